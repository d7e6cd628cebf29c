"""The one-shard-per-rank form on the host: the slice table of Sec. 3.1 Step 1 (which part of every unsharded tensor a
rank holds) and, with two gloo ranks on CPU, the exchange it implies: every rank computes the partial sums of Eq. 1-2
from ITS slices alone (cut with the library's table), the ranks exchange them, and the rank-ordered sum plus shortcut
must equal the oracle's per-device form.  No GPU involved; the arithmetic here is numpy fp64 inside the test."""
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest

import paper_2410_00531_b200 as P
import paper_2410_00531_b200.tp as TP
import tpi_synth as S
from tests.helpers import tpi_config

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("cfg_name,R", [("C1", 2), ("C1", 4), ("C3", 8), ("C5", 2), ("C2", 1)])
def test_rank_slices_tile_every_tensor_exactly_once(cfg_name, R):
    sh = S.CONFIGS[cfg_name]
    cfg = tpi_config(sh, 64, 16)
    d = sh.head_dim
    for tid in (S.WQ, S.WK, S.WV, S.WO, S.WGATE, S.WUP, S.WDOWN):
        rows, cols = sh.tensor_shape(tid)
        cell = 0
        for r in range(R):
            r0, nr, c0, nc = TP.rank_slice(cfg, R, r, tid)
            assert 0 <= r0 and r0 + nr <= rows and 0 <= c0 and c0 + nc <= cols and nr > 0 and nc > 0
            cell += nr * nc
            # whole heads / whole kv-head groups / contiguous FFN columns, in rank order
            if tid == S.WQ:
                assert (r0, nr, c0, nc) == (r * sh.n_heads // R * d, sh.n_heads // R * d, 0, sh.hidden)
            if tid in (S.WK, S.WV):
                assert (r0, nr) == (r * sh.n_kv_heads // R * d, sh.n_kv_heads // R * d)
            if tid == S.WO:
                assert (r0, nr, c0, nc) == (0, sh.hidden, r * sh.n_heads // R * d, sh.n_heads // R * d)
            if tid in (S.WGATE, S.WUP):
                assert (r0, nr) == (r * sh.ffn // R, sh.ffn // R)
            if tid == S.WDOWN:
                assert (r0, nr, c0, nc) == (0, sh.hidden, r * sh.ffn // R, sh.ffn // R)
        assert cell == rows * cols                                           # every element on exactly one rank
    for r in range(R):                                                       # norm gains everywhere; emb / head on the master
        assert TP.rank_slice(cfg, R, r, S.ATTN_NORM)[1] == 1 and TP.rank_slice(cfg, R, r, S.FFN_NORM)[1] == 1
        for tid in (S.EMB, S.HEAD):
            assert TP.rank_slice(cfg, R, r, tid)[1] == (sh.vocab if r == 0 else 0)
        assert TP.rank_slice(cfg, R, r, S.FINAL_NORM)[1] == (1 if r == 0 else 0)
    with pytest.raises(P.TpiError) as e:
        TP.rank_slice(cfg, 3, 0, S.WQ)
    assert e.value.code == -2
    with pytest.raises(P.TpiError):
        TP.rank_slice(cfg, R, R, S.WQ)
    # arena: a worker needs no embedding and no head
    if R > 1:
        d1, _ = TP.query_arena(cfg, R, 1)
        esz = 2 if sh.dtype == "bf16" else 4
        assert TP.query_arena(cfg, R, 0)[0] - d1 >= 2 * (sh.vocab - 1) * sh.hidden * esz


def test_rank_slices_of_a_heterogeneous_partition():
    """Sec. 3.1's proportions p_i as slices: whole kv-head groups and contiguous FFN columns in rank order, every element
    of every matrix on exactly one rank; malformed partitions are refused."""
    sh = S.CONFIGS["C3"]                                   # 32 heads over 8 kv heads (4 per group), FFN 14336
    cfg = tpi_config(sh, 64, 16)
    part = ([4, 2, 1, 1], [7168, 3584, 2048, 1536])
    d, grp = sh.head_dim, sh.n_heads // sh.n_kv_heads
    kv0 = np.concatenate([[0], np.cumsum(part[0])])
    f0 = np.concatenate([[0], np.cumsum(part[1])])
    for r in range(4):
        assert TP.rank_slice(cfg, 4, r, S.WQ, part) == (kv0[r] * grp * d, part[0][r] * grp * d, 0, sh.hidden)
        assert TP.rank_slice(cfg, 4, r, S.WK, part)[:2] == (kv0[r] * d, part[0][r] * d)
        assert TP.rank_slice(cfg, 4, r, S.WO, part) == (0, sh.hidden, kv0[r] * grp * d, part[0][r] * grp * d)
        assert TP.rank_slice(cfg, 4, r, S.WUP, part)[:2] == (f0[r], part[1][r])
        assert TP.rank_slice(cfg, 4, r, S.WDOWN, part) == (0, sh.hidden, f0[r], part[1][r])
    big, small = TP.query_arena(cfg, 4, 1, 0, part)[0], TP.query_arena(cfg, 4, 3, 0, part)[0]
    assert big > small                                     # a rank with more heads and columns needs more memory
    for bad in (([4, 2, 1, 2], part[1]), (part[0], [7168, 3584, 2048, 1535]), ([4, 2, 2, 0], part[1]), ([8], [14336])):
        with pytest.raises((P.TpiError, ValueError)):
            TP.rank_slice(cfg, 4, 0, S.WQ, bad)


WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np
    import torch, torch.distributed as dist
    import tpi_synth as S
    import paper_2410_00531_b200.tp as TP
    from oracle import llama_oracle as O
    from tests.helpers import TINY, make_oracle, tpi_config

    dist.init_process_group("gloo")
    rank, R = dist.get_rank(), dist.get_world_size()
    sh = TINY.with_(n_layers=2, n_heads=4, n_kv_heads=2, head_dim=8, hidden=32, ffn=48)
    cfg = tpi_config(sh, 32, 8)
    d, h = sh.head_dim, sh.hidden

    def mine(layer, tid):          # this rank's slice of the unsharded tensor, cut with the library's table
        r0, nr, c0, nc = TP.rank_slice(cfg, R, rank, tid)
        return S.as_f64(S.gen_tensor(sh, layer, tid)).reshape(sh.tensor_shape(tid)[0], -1)[r0:r0 + nr, c0:c0 + nc]

    def allreduce_rank_order(p):   # the star sum: gather every rank's partial sums, add them in rank order
        parts = [torch.zeros_like(torch.from_numpy(p)) for _ in range(R)]
        dist.all_gather(parts, torch.from_numpy(np.ascontiguousarray(p)))
        red = parts[0].numpy().copy()
        for q in parts[1:]:
            red = red + q.numpy()
        return red

    toks = S.prompt_tokens(sh, 5)
    # the master embeds and broadcasts H^0 (only rank 0 reads the embedding table)
    x = torch.zeros(len(toks), h, dtype=torch.float64)
    if rank == 0:
        x = torch.from_numpy(S.as_f64(S.gen_tensor(sh, 0, S.EMB))[toks])
    dist.broadcast(x, 0)
    x = x.numpy()
    pos = np.arange(len(toks))
    taps = {}
    for l in range(sh.n_layers):
        xn = O.rmsnorm(x, S.as_f64(S.gen_tensor(sh, l, S.ATTN_NORM)), sh.rms_eps)
        q = O.rope((xn @ mine(l, S.WQ).T).reshape(len(toks), -1, d), pos, sh.rope_base)
        k = O.rope((xn @ mine(l, S.WK).T).reshape(len(toks), -1, d), pos, sh.rope_base)
        v = (xn @ mine(l, S.WV).T).reshape(len(toks), -1, d)
        o = O.attention(q, np.swapaxes(k, 0, 1), np.swapaxes(v, 0, 1), pos).reshape(len(toks), -1)
        x = allreduce_rank_order(o @ mine(l, S.WO).T) + x
        taps[(l, "attn")] = x
        xn = O.rmsnorm(x, S.as_f64(S.gen_tensor(sh, l, S.FFN_NORM)), sh.rms_eps)
        act = O.silu(xn @ mine(l, S.WGATE).T) * (xn @ mine(l, S.WUP).T)
        x = allreduce_rank_order(act @ mine(l, S.WDOWN).T) + x
        taps[(l, "ffn")] = x
    orc = make_oracle(sh)
    orc.forward(toks, n_shards=R)
    err = max(float(np.abs(taps[k] - orc.taps[k]).max()) for k in taps)
    gathered = [None] * R
    dist.all_gather_object(gathered, err)
    if rank == 0:
        print(json.dumps({"world": R, "max_abs_err": max(gathered)}))
    dist.destroy_process_group()
""") % ROOT


def test_two_ranks_each_with_its_own_slices_reproduce_the_oracle(tmp_path):
    script = tmp_path / "tp_worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29541", OMP_NUM_THREADS="1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-3000:]
    import json
    d = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][0])
    assert d["world"] == 2 and d["max_abs_err"] < 1e-12
