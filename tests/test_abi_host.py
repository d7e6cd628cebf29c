"""Host-only checks of the C-ABI library: it loads without a GPU, exports every symbol the
headers declare, validates arguments, sizes its arenas like the paper's block table, and its
window scheduler orders loads the way Sec. 3.3 describes (checked against the oracle's
time-slot model with the paper's worked example)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2410_00531_b200 as P
import paper_2410_00531_b200.ops as K
import tpi_synth as S
from oracle import window_model as W
from tests.helpers import tpi_config

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for hdr in ("tpi.h", "tpi_ops.h", "tpi_tp.h"):
        src = open(os.path.join(ROOT, "include", hdr)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names += re.findall(r"\b(tpi_[a-z0-9_]+)\s*\(", src)
    return sorted(set(n for n in names if n != "tpi_fill_fn"))


def test_library_exports_every_declared_symbol():
    lib = P.lib()
    decl = declared_functions()
    assert len(decl) >= 30
    for name in decl:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    import paper_2410_00531_b200.tp as TP
    bound = set(P.binding.SYMBOLS) | set(K.OPS_SYMBOLS) | set(TP.TP_SYMBOLS)
    assert set(decl) <= bound, set(decl) - bound


def test_strerror_and_argument_validation():
    lib = P.lib()
    assert lib.tpi_strerror(0) == b"ok" and b"arena" in lib.tpi_strerror(-3)
    cfg = tpi_config(S.CONFIGS["C1"], 64, 16)
    with pytest.raises(P.TpiError) as e:
        P.query_arena(cfg, 2, -1, False)
    assert e.value.code == -1
    bad = tpi_config(S.CONFIGS["C1"].with_(n_heads=6, n_kv_heads=4), 64, 16)
    with pytest.raises(P.TpiError) as e:
        P.query_arena(bad, 2, 0, False)
    assert e.value.code == -2
    with pytest.raises(P.TpiError):
        P.ring_trace(7, 2, 4)                  # odd number of blocks


def test_load_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    cfg = tpi_config(S.CONFIGS["C1"], 64, 16)
    with pytest.raises(RuntimeError):
        P.Session(cfg, S.synth_fill(S.CONFIGS["C1"]), 2)
    # and the raw C call reports a CUDA error instead of computing anything on the host
    buf = (C.c_char * 4096)()
    res = P.binding.TpiResources(C.addressof(buf), 4096, C.addressof(buf), 4096, None, None)
    cb = P.binding.FILL_FN(lambda *a: 0)
    with pytest.raises(P.TpiError) as e:
        P.load_model(cfg, res, cb, 2, 0)
    assert e.value.code in (-1, -3, -6)


def test_block_bytes_match_table5():
    """Table 5 (Llama 2-7B, n = 4, p = 0.25, FP32): attention 64 MB, FFN 129 MB per device."""
    sh = S.CONFIGS["C2"].with_(dtype="f32")
    attn, ffn = P.block_bytes(tpi_config(sh, 256, 128))
    n = 4
    assert round(attn / n / 2**20) == 64 and round(ffn / n / 2**20) == 129
    want_a = W.block_params("attn", sh.hidden, sh.vocab, sh.n_heads, sh.n_kv_heads, sh.ffn, 1.0) * 4
    want_f = W.block_params("ffn", sh.hidden, sh.vocab, sh.n_heads, sh.n_kv_heads, sh.ffn, 1.0) * 4
    assert 0 <= attn - want_a < 1024 and 0 <= ffn - want_f < 1024      # only alignment padding on top


def test_arena_grows_with_window_like_prop5():
    sh = S.CONFIGS["C4"]
    cfg = tpi_config(sh, 1024, 512)
    attn, ffn = P.block_bytes(cfg)
    base = P.query_arena(cfg, 8, 1, True)[0] - ffn
    for w in (1, 2, 3, 4, 8, 16, 32):
        d, h = P.query_arena(cfg, 8, w, True)
        # floor(w/2) attention + floor((w+1)/2) FFN blocks (w = 1: one slot)
        assert d - base == (w // 2) * attn + ((w + 1) // 2) * ffn
        assert h > 2 * sh.n_layers * 0 + sh.n_layers * (attn + ffn)
    resident = P.query_arena(cfg, 8, 0, False)[0]
    assert resident - base == sh.n_layers * (attn + ffn)


# ----------------------------------------------------------------- window scheduler ordering
def replay(ops, t_exec, t_ar, tau, n_blocks):
    """Event simulation of the recorded operations on two in-order queues with the given
    durations; returns per executed block how long compute waited for its weights."""
    copy_t = 0.0
    comp_t = 0.0
    loaded = {}
    released = {}
    stalls = []
    k = 0
    for op, slot, blk in ops:
        if op == 0:
            copy_t = max(copy_t, released[slot])
        elif op == 1:
            copy_t += tau[blk % 2]
        elif op == 2:
            loaded[slot] = copy_t
        elif op == 3:
            stalls.append(max(0.0, loaded[slot] - comp_t))
            comp_t = max(comp_t, loaded[slot])
        elif op == 4:
            comp_t += t_exec[k % 2] + t_ar
            released[slot] = comp_t
            k += 1
        elif op == 5:                                           # a retained block: no window operation
            stalls.append(0.0)
            comp_t += t_exec[k % 2] + t_ar
            k += 1
    return stalls, comp_t


@pytest.mark.parametrize("w", [1, 2, 4, 6])
def test_ring_reproduces_the_oracle_timeline(w):
    ta, tf, tr, la, lf = 11.0, 17.0, 14.0, 18.0, 30.0          # the paper's worked example
    n_blocks, n_exec = 64, 160                                  # crosses the token boundary (cyclic)
    ops = P.ring_trace(n_blocks, w, n_exec)
    stalls, end = replay(ops, (ta, tf), tr, (la, lf), n_blocks)
    want, _, want_end = W.timeline(ta, tf, tr, la, lf, n_exec, w)
    assert len(stalls) == n_exec
    assert np.allclose(stalls, want) and np.isclose(end, want_end)


@pytest.mark.parametrize("w,T", [(1, 2), (2, 1), (2, 3), (4, 2), (6, 4), (8, 5)])
def test_ring_with_block_retention_reproduces_the_oracle_timeline(w, T):
    ta, tf, tr, la, lf = 11.0, 17.0, 14.0, 18.0, 60.0           # a link too slow for Prop. 3
    L, n_exec = 16, 100                                         # crosses the token boundary (cyclic)
    ops = P.ring_trace(2 * L, w, n_exec, ffn_every_T=T)
    keep = {2 * l + 1 for l in W.retained_ffn_layers(L, T)}
    assert {int(b) for op, _, b in ops if op == 5} == keep     # exactly the kept blocks run without a load
    assert not any(int(b) in keep for op, _, b in ops if op == 1)
    stalls, end = replay(ops, (ta, tf), tr, (la, lf), 2 * L)
    want, _, want_end = W.timeline_retained(ta, tf, tr, la, lf, n_exec, w, T, L)
    assert len(stalls) == n_exec
    assert np.allclose(stalls, want) and np.isclose(end, want_end)


@pytest.mark.parametrize("w", [3, 5, 7])
def test_ring_with_an_odd_window_follows_the_per_kind_places_of_prop5(w):
    """Prop. 5 splits an odd window into floor(w/2) attention and ceil(w/2) FFN places; the ring deals its slots the
    same way, so its stalls are those of the oracle's per-kind event model (retention off)."""
    ta, tf, tr, la, lf = 11.0, 17.0, 2.0, 18.0, 30.0            # loads slower than compute: the window size matters
    L, n_exec = 12, 70
    ops = P.ring_trace(2 * L, w, n_exec)
    stalls, end = replay(ops, (ta, tf), tr, (la, lf), 2 * L)
    want, _, want_end = W.timeline_retained(ta, tf, tr, la, lf, n_exec, w, 0, L)
    assert np.allclose(stalls, want) and np.isclose(end, want_end)
    slots = {int(sl) for op, sl, _ in ops if op == 1}
    assert len(slots) == w                                      # every place of the window gets used


def test_ring_invariants():
    for w in (1, 2, 3, 5, 8):
        n_blocks = 8
        ops = P.ring_trace(n_blocks, w, 40)
        holds, resident, next_copy, next_exec = {}, set(), 0, 0
        for op, slot, blk in ops:
            if op == 1:
                assert blk == next_copy % n_blocks              # loads strictly in execution order
                next_copy += 1
                assert slot not in resident                     # never overwrite a block still in use
                holds[slot] = blk
                resident.add(slot)
                assert len(resident) <= max(w, 1)               # at most w blocks held (Prop. 5)
            elif op == 3:
                assert holds[slot] == next_exec % n_blocks      # compute waits for the block it needs
            elif op == 4:
                resident.discard(slot)
                next_exec += 1
        assert next_exec == 40 and next_copy >= 40
        # attention blocks (even) and FFN blocks (odd) never share a slot unless w == 1
        if w > 1:
            kinds = {}
            for op, slot, blk in ops:
                if op == 1:
                    kinds.setdefault(slot, set()).add(blk % 2)
            assert all(len(k) == 1 for k in kinds.values())
            n_attn = sum(1 for k in kinds.values() if k == {0})
            assert n_attn == w // 2 and len(kinds) - n_attn == (w + 1) // 2


@pytest.mark.parametrize("w,T", [(1, 0), (2, 0), (3, 0), (4, 2), (8, 0)])
def test_a_failed_block_copy_propagates_and_leaves_the_ring_consistent(w, T):
    """Failure injection on the host: the back end's k-th block copy fails once (what a cudaMemcpyAsync error looks
    like to the scheduler).  Without a retry the status comes back unchanged from wherever the loader was pumped
    (start-up, a block's wait, a block's release).  With a retry the ring must carry on as if nothing had happened:
    the copies, waits and releases are exactly those of a fault-free run, in the same order."""
    n_blocks, n_exec = 12, 40
    clean = P.ring_trace(n_blocks, w, n_exec, ffn_every_T=T)
    n_copies = int((clean[:, 0] == 1).sum())
    essential = lambda ops: [tuple(o) for o in ops if o[0] in (1, 2, 3, 4, 5)]
    for k in list(range(0, min(n_copies, 30))) + [n_copies - 1]:
        for status in (-6, -7):                                   # TPI_ERR_CUDA, TPI_ERR_TIMEOUT
            with pytest.raises(P.TpiError) as e:
                P.ring_trace_faulty(n_blocks, w, n_exec, k, status, False, ffn_every_T=T)
            assert e.value.code == status
        ops = P.ring_trace_faulty(n_blocks, w, n_exec, k, -6, True, ffn_every_T=T)
        marks = [tuple(o) for o in ops if o[0] == 6]
        assert len(marks) == 1 and marks[0][1] == -6             # seen once, with the injected status
        assert essential(ops) == essential(clean)
        # the retried load waits for its slot's release again, never less often than the fault-free run
        assert int((ops[:, 0] == 0).sum()) >= int((clean[:, 0] == 0).sum())
    # a copy index beyond the run never fires
    assert essential(P.ring_trace_faulty(n_blocks, w, n_exec, 10 ** 6, -6, False, ffn_every_T=T)) == essential(clean)
    with pytest.raises(P.TpiError):
        P.ring_trace_faulty(n_blocks, w, n_exec, 0, 3, True)      # a failure needs a negative status


# ----------------------------------------------------------------- steady-state diagnostics (Prop. 3, 4, 6)
def test_steady_conditions_match_the_oracle_and_the_worked_example():
    # the paper's worked example: tight fails, loose holds, so no retention is needed
    assert P.steady_conditions(11, 17, 14, 18, 30, 32) == (False, True, 0)
    rng = np.random.default_rng(7)
    seen = set()
    for _ in range(400):
        ta, tf, la, lf = rng.integers(1, 40, 4).astype(float)
        tr = float(rng.integers(0, 12))
        L = int(rng.integers(1, 20))
        tight, loose, T = P.steady_conditions(ta, tf, tr, la, lf, L)
        assert tight == W.tight_condition(ta, tf, tr, la, lf)
        assert loose == W.loose_condition(ta, tf, tr, la, lf, L)
        ok = [t for t in range(1, L + 1) if W.retention_condition(ta, tf, tr, la, lf, L, t)]
        want = 0 if loose else (max(ok) if ok else -1)
        assert T == want, (ta, tf, tr, la, lf, L)
        seen.add(min(T, 1))
    assert seen == {-1, 0, 1}                                   # every outcome occurred
    # the allreduce term only ever appears added to a block's compute time
    assert P.steady_conditions(11, 17, 14, 18, 30, 32) == P.steady_conditions(25, 31, 0, 18, 30, 32)
    with pytest.raises(P.TpiError):
        P.steady_conditions(-1, 1, 1, 1, 1, 4)


def test_timeline_variant_compiles_and_the_plain_library_carries_no_stamps(tmp_path):
    """The decode kernels' device-side timeline is an opt-in build (-DTPI_TIMELINE, see build.py): the translation units
    that hold its macro, a stamped kernel, and the hook must compile for sm_100a with the flag, and the plain library's
    hook must answer 0 ("no stamps here") while still reporting the buffer layout."""
    import shutil
    import subprocess
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not (os.path.exists(nvcc) or shutil.which("nvcc")):
        pytest.skip("no nvcc on this machine")
    csrc = os.path.join(os.path.dirname(P.__file__), "csrc")
    procs = [subprocess.Popen([nvcc if os.path.exists(nvcc) else "nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O1",
                               "-std=c++17", "-Xcompiler", "-fPIC", "-DTPI_TIMELINE", "-c", os.path.join(csrc, src), "-o",
                               str(tmp_path / (src + ".o"))]) for src in ("attn_prefill_mma.cu", "ops.cu")]
    assert all(p.wait() == 0 for p in procs)
    fn = P.lib().tpi_internal_timeline
    fn.argtypes, fn.restype = [C.c_void_p, C.POINTER(C.c_int)], C.c_int
    lay = (C.c_int * 4)()
    if os.environ.get("TPI_TIMELINE", "0") in ("", "0"):
        assert fn(None, lay) == 0
    assert lay[0] >= 7 and lay[1] >= 148 and lay[2] >= 4 + 32 and lay[3] == 4
