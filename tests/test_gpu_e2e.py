"""End-to-end parity of the CUDA library against the CPU oracle through the C ABI
(tiny fp32 workload C1, full depth; small bf16 / grouped-head variants)."""
import numpy as np
import torch
import pytest

import tpi_synth as S
from tests.helpers import check_logits, close_elementwise, gpu_session, make_oracle, rel_l2, tol_for

pytestmark = pytest.mark.gpu


def _run_and_compare(shape, n_shards, window=0, n_decode=8, prompt_len=None, max_prefill=None, opts=(), max_ambiguous=None):
    """Prompt pass + teacher-forced decode against the oracle.  Every hidden state, cache row and logits vector must
    meet the vector bar (rel-L2 <= tol) and the element bar (max |delta| <= 3 tol rms); every step must satisfy the
    token rule.  Returns (tokens, mismatches, ambiguous steps): a mismatch is only ever accepted on a step whose
    oracle top-2 gap is within twice the per-logit allowance, and the number of such steps is bounded by the caller."""
    import paper_2410_00531_b200 as P
    tol = tol_for(shape)
    toks = S.prompt_tokens(shape, prompt_len or shape.prompt_len)
    T = len(toks)
    orc = make_oracle(shape)
    with gpu_session(shape, T + n_decode + 1, max_prefill or T, n_shards, window) as ses:
        for o, v in opts:
            P.set_option(ses.h, o, v)
        tok, lg = P.prefill(ses.h, toks, shape.vocab)
        want = orc.forward(toks)
        ok, amb = check_logits(lg, tok, want, tol)
        mismatches, ambiguous = int(not ok), int(amb)
        for l in range(shape.n_layers):
            assert close_elementwise(P.get_hidden(ses.h, l, 0, shape.hidden), orc.taps[(l, "attn")][-1], tol)
            assert close_elementwise(P.get_hidden(ses.h, l, 1, shape.hidden), orc.taps[(l, "ffn")][-1], tol)
        # cache contents and indexing: slot p holds position p
        for l in range(shape.n_layers):
            for g in range(shape.n_kv_heads):
                k, v = P.get_kv(ses.h, l, g, 0, T, shape.head_dim)
                assert close_elementwise(k, orc.cache.K[l][g], tol) and close_elementwise(v, orc.cache.V[l][g], tol)
        out_tokens = [tok]
        feed = int(np.argmax(want))
        for step in range(n_decode):
            tok, lg = P.decode_step(ses.h, feed, shape.vocab)   # teacher-forced with the oracle's token
            want = orc.forward([feed])
            ok, amb = check_logits(lg, tok, want, tol)
            mismatches += (not ok)
            ambiguous += amb
            for l in range(shape.n_layers):
                assert close_elementwise(P.get_hidden(ses.h, l, 0, shape.hidden), orc.taps[(l, "attn")][-1], tol)
                assert close_elementwise(P.get_hidden(ses.h, l, 1, shape.hidden), orc.taps[(l, "ffn")][-1], tol)
            feed = int(np.argmax(want))
            out_tokens.append(tok)
        assert P.position(ses.h) == T + n_decode
        k, v = P.get_kv(ses.h, shape.n_layers - 1, 0, T, n_decode, shape.head_dim)
        assert close_elementwise(k, orc.cache.K[-1][0][T:], tol)
        print(f"[parity] {shape.name} N={n_shards} T={T}: {mismatches} mismatches, {ambiguous} ambiguous of {n_decode + 1} steps")
        assert mismatches <= ambiguous
        if max_ambiguous is not None:
            assert ambiguous <= max_ambiguous
        return out_tokens, mismatches


@pytest.mark.parametrize("n_shards", [1, 2, 4])
def test_c1_full_depth(n_shards):
    shape = S.CONFIGS["C1"]
    toks, mism = _run_and_compare(shape, n_shards)
    assert mism == 0                           # fp32: gaps are far above the tolerance
    ref, _ = make_oracle(shape).greedy(S.prompt_tokens(shape), 9)
    assert toks == list(ref)                   # "identical to single-server inference"


def test_c1_every_decode_driver():
    """The default is a CUDA graph of per-phase kernels with programmatic dependent launch; the same
    kernels also run without PDL or as plain stream launches."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"]
    _run_and_compare(shape, 2, opts=((P.OPT_GRAPH, 0), (P.OPT_PDL, 0)))
    _run_and_compare(shape, 2, opts=((P.OPT_GRAPH, 0), (P.OPT_PDL, 1)))
    _run_and_compare(shape, 2, opts=((P.OPT_GRAPH, 1), (P.OPT_PDL, 0)))


def test_chunked_prefill_matches():
    shape = S.CONFIGS["C1"]
    _run_and_compare(shape, 2, prompt_len=23, max_prefill=8, n_decode=3)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_degenerate_prompts(dtype):
    """The smallest and the tightest cases of Algorithm 1's loop: a prompt of ONE token (no earlier key to attend to),
    a prompt whose last chunk holds one position (chunks 8, 8, 1), a prompt that fills the cache to its last slot (the
    step after it must be refused, nothing may be written past the cache), and an empty prompt (refused)."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"].with_(dtype=dtype, seed=91)
    _run_and_compare(shape, 2, prompt_len=1, n_decode=3)
    _run_and_compare(shape, 2, prompt_len=17, max_prefill=8, n_decode=2)
    toks = S.prompt_tokens(shape, 24)
    orc = make_oracle(shape)
    want = orc.forward(toks)
    with gpu_session(shape, 24, 24, 2) as ses:               # max_seq == prompt length
        with pytest.raises(P.TpiError) as e:
            P.prefill(ses.h, [], 0)
        assert e.value.code == -1 and P.position(ses.h) == 0
        tok, lg = P.prefill(ses.h, toks, shape.vocab)
        check_logits(lg, tok, want, tol_for(shape))
        k, v = P.get_kv(ses.h, shape.n_layers - 1, shape.n_kv_heads - 1, 23, 1, shape.head_dim)   # the last slot
        assert close_elementwise(k, orc.cache.K[-1][-1][23:24], tol_for(shape))
        assert P.position(ses.h) == 24
        with pytest.raises(P.TpiError) as e:
            P.decode_step(ses.h, tok, 0)
        assert e.value.code == -4 and P.position(ses.h) == 24


def test_small_bf16_gqa():
    shape = S.CONFIGS["C1"].with_(dtype="bf16", n_heads=8, n_kv_heads=2, head_dim=32, seed=77, rope_base=500000.0)
    _run_and_compare(shape, 2)


def test_small_f32_gqa8_d128():
    shape = S.ModelShape("gqa8", 2, 1024, 8, 1, 128, 1408, 3001, 1e-5, 500000.0, "f32", 78, 1, 40, 4)
    _run_and_compare(shape, 1)


@pytest.mark.parametrize("window", [1, 2, 3, 4])
def test_streamed_is_bit_identical_to_resident(window):
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"].with_(n_layers=4)
    toks = S.prompt_tokens(shape)
    res = {}
    for w in (0, window):
        with gpu_session(shape, 64, 16, 2, w) as ses:
            t0, lg0 = P.prefill(ses.h, toks, shape.vocab)
            seq = P.decode_run(ses.h, t0, 6)
            t1, lg1 = P.decode_step(ses.h, int(seq[-1]), shape.vocab)
            res[w] = (t0, lg0, seq, t1, lg1)
            st = P.get_stats(ses.h)
            if w:
                assert st["blocks_loaded"] >= 8 * 8 and st["link_bytes_total"] > 0
    a, b = res[0], res[window]
    assert a[0] == b[0] and a[3] == b[3] and (a[2] == b[2]).all()
    assert np.array_equal(a[1], b[1]) and np.array_equal(a[4], b[4])


@pytest.mark.parametrize("window,T", [(1, 2), (2, 1), (4, 3)])
def test_block_retention_is_bit_identical_and_loads_less(window, T):
    """Prop. 6's retention: the kept FFN blocks never cross the link again, the rest stream as before,
    and the tokens and logits are the same bits as the resident run's."""
    import paper_2410_00531_b200 as P
    from tests.helpers import tpi_config
    shape = S.CONFIGS["C1"].with_(n_layers=6)
    toks = S.prompt_tokens(shape)
    _, ffn_bytes = P.block_bytes(tpi_config(shape, 64, 16))
    n_keep = len(range(0, shape.n_layers, T))
    res, loads = {}, {}
    for mode in ("resident", "streamed", "retained"):
        extra = n_keep * ffn_bytes if mode == "retained" else 0
        with gpu_session(shape, 64, 16, 2, 0 if mode == "resident" else window, extra_dev_bytes=extra) as ses:
            if mode == "retained":
                P.set_retention(ses.h, T)
            t0, lg0 = P.prefill(ses.h, toks, shape.vocab)
            seq = P.decode_run(ses.h, t0, 5)
            t1, lg1 = P.decode_step(ses.h, int(seq[-1]), shape.vocab)
            res[mode] = (t0, lg0, seq, t1, lg1)
            st = P.get_stats(ses.h)
            loads[mode] = st["link_bytes_total"]
            if mode == "retained":
                assert st["retained_blocks"] == n_keep and st["retained_bytes"] == n_keep * ffn_bytes
            elif mode == "streamed":
                assert st["retained_blocks"] == 0
                with pytest.raises(P.TpiError) as e:           # no room was given for kept blocks
                    P.set_retention(ses.h, T)
                assert e.value.code == -3
                t2, _ = P.prefill(ses.h, toks, 0)               # ... and the model still works as before
                assert t2 == t0
    a = res["resident"]
    for mode in ("streamed", "retained"):
        b = res[mode]
        assert a[0] == b[0] and a[3] == b[3] and (a[2] == b[2]).all()
        assert np.array_equal(a[1], b[1]) and np.array_equal(a[4], b[4])
    assert loads["retained"] < loads["streamed"]
    # automatic period: the smallest T whose kept blocks fit the room that the arena has beside the window
    for room, want_T in ((shape.n_layers, 1), (3, 2), (2, 3), (1, 6), (0, 0)):
        with gpu_session(shape, 64, 16, 2, window, extra_dev_bytes=room * ffn_bytes + 64) as ses:
            P.set_retention(ses.h, -1)
            r = P.scheduler_report(ses.h)
            assert r["retain_every_T"] == want_T and P.get_stats(ses.h)["retained_blocks"] == (len(range(0, 6, want_T)) if want_T else 0)


def test_scheduler_report_measures_the_propositions_inputs():
    """Sec. 3.3's diagnostics: block compute and load latencies measured on the run, Prop. 3/4/6 evaluated on them."""
    import paper_2410_00531_b200 as P
    from tests.helpers import tpi_config
    shape = S.CONFIGS["C1"].with_(n_layers=4)
    toks = S.prompt_tokens(shape)
    attn_b, ffn_b = P.block_bytes(tpi_config(shape, 64, 16))
    with gpu_session(shape, 64, 16, 2, 3) as ses:
        P.set_option(ses.h, P.OPT_PROFILE, 1)
        t0, _ = P.prefill(ses.h, toks, 0)
        assert P.scheduler_report(ses.h)["n_t_attn"] == 0          # the prompt pass is not sampled
        P.decode_run(ses.h, t0, 5)
        torch.cuda.synchronize()
        r = P.scheduler_report(ses.h)
        assert r["n_t_attn"] == r["n_t_ffn"] == 5 * shape.n_layers
        assert r["n_tau_attn"] >= 5 * shape.n_layers - 2 and r["n_tau_ffn"] >= 5 * shape.n_layers - 2
        assert min(r["t_attn_ms"], r["t_ffn_ms"], r["tau_attn_ms"], r["tau_ffn_ms"]) > 0 and r["t_all_reduce_ms"] == 0
        want = P.steady_conditions(r["t_attn_ms"], r["t_ffn_ms"], 0.0, r["tau_attn_ms"], r["tau_ffn_ms"], shape.n_layers)
        assert (bool(r["tight_holds"]), bool(r["loose_holds"]), r["retention_T"]) == want
        assert r["window_blocks"] == 3 and r["m_worker_bytes"] == attn_b + 2 * ffn_b == r["window_device_bytes"]
        P.scheduler_reset(ses.h)
        assert P.scheduler_report(ses.h)["n_t_ffn"] == 0
    with gpu_session(shape, 64, 16, 2, 0) as ses:                  # resident: compute samples only, no verdicts
        P.set_option(ses.h, P.OPT_PROFILE, 1)
        t0, _ = P.prefill(ses.h, toks, 0)
        P.decode_run(ses.h, t0, 3)
        r = P.scheduler_report(ses.h)
        assert r["n_t_attn"] == 3 * shape.n_layers and r["n_tau_attn"] == 0
        assert r["tight_holds"] == r["loose_holds"] == r["retention_T"] == -2 and r["m_worker_bytes"] == 0


@pytest.mark.parametrize("case", ["f32_gqa", "bf16_wide"])
def test_heterogeneous_partition_matches_the_oracle(case):
    """Sec. 3.1's proportions p_i: unequal shares of heads and FFN columns, prompt pass and decode, resident and streamed."""
    import paper_2410_00531_b200 as P
    if case == "f32_gqa":
        shape = S.CONFIGS["C1"].with_(n_heads=8, n_kv_heads=4, head_dim=32, hidden=256, ffn=688, n_layers=3)
        parts = [([2, 1, 1], [344, 200, 144]), ([3, 1], [512, 176])]
    else:   # 7B-shaped widths, two layers: the tensor-core prompt pass with per-shard contractions of unequal length
        shape = S.CONFIGS["C2"].with_(n_layers=2)
        parts = [([24, 8], [8256, 2752]), ([16, 8, 4, 4], [5504, 2752, 1408, 1344])]
    toks = S.prompt_tokens(shape)[:24]
    tol = tol_for(shape)
    for kv, ff in parts:
        orc = make_oracle(shape)
        want0 = orc.forward(toks, n_shards=len(kv), partition=(kv, ff))
        for window in (0, 3):
            with gpu_session(shape, 48, 16, 1, window) as ses:
                P.set_partition(ses.h, kv, ff)
                assert P.get_stats(ses.h)["n_shards"] == len(kv)
                t0, lg0 = P.prefill(ses.h, toks, shape.vocab)
                check_logits(lg0, t0, want0, tol)
                for l in range(shape.n_layers):
                    for which, key in ((0, "attn"), (1, "ffn")):
                        assert rel_l2(P.get_hidden(ses.h, l, which, shape.hidden), orc.taps[(l, key)][-1]) <= tol
                if window == 0:
                    o2 = make_oracle(shape)
                    o2.forward(toks, n_shards=len(kv), partition=(kv, ff))
                    tok, want = int(np.argmax(want0)), None
                    for _ in range(3):                                  # teacher-forced decode steps
                        want = o2.forward([tok], n_shards=len(kv), partition=(kv, ff))
                        got_tok, lg = P.decode_step(ses.h, tok, shape.vocab)
                        check_logits(lg, got_tok, want, tol)
                        tok = int(np.argmax(want))
                    P.set_shards(ses.h, 1)                              # back to the uniform split
                    t1, lg1 = P.prefill(ses.h, toks, shape.vocab)
                    check_logits(lg1, t1, want0, tol)
    with gpu_session(shape, 48, 16, 1) as ses:
        for bad in (([1], [shape.ffn]), ([shape.n_kv_heads, 1], [shape.ffn - 8, 8]), ([shape.n_kv_heads - 1, 1], [shape.ffn - 3, 3]),
                    ([shape.n_kv_heads, 0], [shape.ffn - 8, 8])):
            with pytest.raises(P.TpiError):
                P.set_partition(ses.h, *bad)


def test_heterogeneous_partition_long_prompt():
    """Unequal shares with more than 128 prompt positions: one CTA-pair GEMM per shard with contractions of unequal
    length (the star sum then runs as its own kernel), 7B-shaped widths, two layers, against the oracle."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C2"].with_(n_layers=2, vocab=32000)
    kv, ff = [16, 8, 4, 4], [5504, 2752, 1408, 1344]
    toks = S.prompt_tokens(shape, 160)
    tol = tol_for(shape)
    orc = make_oracle(shape)
    want = orc.forward(toks, n_shards=len(kv), partition=(kv, ff))
    with gpu_session(shape, 176, 160, 1, 0) as ses:
        P.set_partition(ses.h, kv, ff)
        t0, lg0 = P.prefill(ses.h, toks, shape.vocab)
        check_logits(lg0, t0, want, tol)
        for l in range(shape.n_layers):
            for which, key in ((0, "attn"), (1, "ffn")):
                assert rel_l2(P.get_hidden(ses.h, l, which, shape.hidden), orc.taps[(l, key)][-1]) <= tol


def test_set_shards_and_set_window_roundtrip():
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"]
    toks = S.prompt_tokens(shape)
    want = make_oracle(shape).forward(toks)
    with gpu_session(shape, 64, 16, 2, 0, other_windows=(2,)) as ses:
        for n, w in ((2, 0), (4, 0), (4, 2), (1, 2), (1, 0)):
            P.set_shards(ses.h, n)
            P.set_window(ses.h, w)
            tok, lg = P.prefill(ses.h, toks, shape.vocab)
            check_logits(lg, tok, want, 1e-5)
            st = P.get_stats(ses.h)
            assert st["n_shards"] == n and st["window_blocks"] == w


def test_error_codes():
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"]
    with pytest.raises(P.TpiError) as e:
        gpu_session(shape, 64, 16, 3)                      # 3 does not divide 4 heads
    assert e.value.code == -2
    with gpu_session(shape, 20, 16, 2) as ses:
        with pytest.raises(P.TpiError) as e:
            P.prefill(ses.h, [1, 2, shape.vocab], 0)
        assert e.value.code == -5
        tok, _ = P.prefill(ses.h, S.prompt_tokens(shape), 0)
        P.decode_run(ses.h, tok, 4)
        with pytest.raises(P.TpiError) as e:
            P.decode_step(ses.h, 1, 0)                     # position 20 == max_seq
        assert e.value.code == -4
        with pytest.raises(P.TpiError) as e:
            P.set_window(ses.h, 2)                         # resident load kept no host images
        assert e.value.code in (-9, -3)


def test_full_size_7b_shape_sampled_outputs_and_size_independent_properties():
    """The benchmarked 7B-shaped workload at FULL depth in bench.py's launch configuration (graph + PDL).  The oracle
    cannot run 32 layers in seconds, so (a) it computes what it can one by one: layer 0's two hidden states of the last
    prompt position (a one-layer oracle sees the same embedding and layer-0 weights); (b) properties that hold at any
    size: the result does not depend on the number of shards (the paper's identity with single-server inference, here
    up to the fp32 order of the partial sums), a streamed model gives the resident model's bits, and one enqueue of
    several tokens gives the per-token calls' tokens."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C2"]
    toks = S.prompt_tokens(shape)
    T, n_dec = len(toks), 6
    one = make_oracle(shape.with_(n_layers=1))
    one.forward(toks)
    res = {}
    with gpu_session(shape, T + 2 * n_dec + 2, T, 4, 0, keep_host_images=True, other_windows=(4,)) as ses:
        for key, n, w in (("n4", 4, 0), ("n1", 1, 0), ("n4w4", 4, 4)):
            P.set_shards(ses.h, n)
            P.set_window(ses.h, w)
            t0, lg = P.prefill(ses.h, toks, shape.vocab)
            h_attn, h_ffn = P.get_hidden(ses.h, 0, 0, shape.hidden), P.get_hidden(ses.h, 0, 1, shape.hidden)
            assert rel_l2(h_attn, one.taps[(0, "attn")][-1]) <= 1e-2 and rel_l2(h_ffn, one.taps[(0, "ffn")][-1]) <= 1e-2
            seq = P.decode_run(ses.h, t0, n_dec)                        # one enqueue (graph replay when resident)
            P.set_position(ses.h, T)                                    # rewind: the same steps, one call each
            step, tok = [], t0
            for _ in range(n_dec):
                tok, _ = P.decode_step(ses.h, tok, 0)
                step.append(tok)
            assert list(seq) == step
            res[key] = (t0, lg, list(seq))
    assert np.isfinite(res["n4"][1]).all()
    assert res["n4w4"][0] == res["n4"][0] and np.array_equal(res["n4w4"][1], res["n4"][1]) and res["n4w4"][2] == res["n4"][2]
    # Same bf16 weights and exact products; only the fp32 order of the partial sums differs.  Where that moves a key or
    # value across a bf16 rounding boundary the cache entry changes by one bf16 ulp, and 32 layers carry it on:
    # 1.7e-3 observed, inside the 1e-2 bar that bf16 weights are given.
    assert rel_l2(res["n1"][1], res["n4"][1]) < 1e-2
    g = np.sort(res["n4"][1])[::-1]
    if g[0] - g[1] > 3e-2 * np.sqrt(np.mean(g * g)):
        assert res["n1"][0] == res["n4"][0]


def _golden(name):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", f"{name.lower()}_full_depth.txt")
    return [ln.split() for ln in open(path) if ln[0] != "#"]


def _check_stored_logits(gold, prefix, lg, tok, tol):
    """Sampled logits, the oracle's 32 largest, the root mean square and the token rule against stored oracle values;
    the vector bar is taken over the 64 evenly spaced stored logits (an estimate of the relative L2 distance over the
    whole vocabulary).  Returns that estimate."""
    rms = float(next(g[1] for g in gold if g[0] == prefix + "logits_rms"))
    top = [(int(g[1]), float(g[2])) for g in gold if g[0] == prefix + "top"]
    sampled = [(int(g[1]), float(g[2])) for g in gold if g[0] == prefix + "logit"]
    e = 3 * tol * rms                                            # the token rule's per-logit allowance
    assert abs(np.sqrt(np.mean(lg.astype(np.float64) ** 2)) - rms) <= tol * rms
    rel = float(np.sqrt(np.mean([(lg[i] - v) ** 2 for i, v in sampled])) / rms)
    assert rel <= tol, (prefix, rel)
    for i, v in sampled + top:
        assert abs(lg[i] - v) <= e, (prefix, i, lg[i], v)
    assert int(np.argmax(lg)) == tok
    if top[0][1] - top[1][1] > 2 * e:
        assert tok == top[0][0]
    else:
        assert tok in (top[0][0], top[1][0])
    assert lg.max() <= top[0][1] + e                             # nothing outside the oracle's 32 largest may win by more
    return rel


# Bars of the full-depth test as multiples of the 1e-2 bar for bf16 weights.  At 32 layers the distance to the oracle is
# 0.35-0.45e-2 and the bar holds with room.  At 80 layers (70B shape) the distance itself is about 1e-2: measured 0.80e-2
# on the last layer's hidden states, 0.84e-2 on the prompt's logits and 1.21e-2 on the logits of the decode step on top
# of it, tokens identical (with every GEMM in fp32 on the CUDA cores instead of the tensor cores the prompt's logits
# are at 0.63e-2: a random-weight model of that depth amplifies last-bit differences, among them the rounding of
# the bf16 KV cache).  The distance moves by +-15 % with any change of summation order, so this one case is held to
# 1.5e-2 and the figures above are reported instead of claiming the 1e-2 bar at 80 layers.
FULL_DEPTH_BAR = {"C2": 1.0, "C3": 1.0, "C5": 1.5}


@pytest.mark.parametrize("name", ["C2", "C3", "C5"])
def test_full_size_against_the_oracle_s_stored_values(name):
    """The benchmarked workloads at FULL depth and full vocabulary, in bench.py's launch configuration (prompt in one
    chunk, graph + PDL decode), against values the CPU oracle computed for them offline (tests/golden/*_full_depth.txt,
    written by tests/golden/make_full_depth_golden.py): 7B shape with its 128-token prompt, 8B shape with its
    4096-token prompt, 70B shape (139 GB resident) with its 512-token prompt.  Hidden states of the first, middle and
    last layer, sampled logits, the 32 largest logits and the greedy token of the last prompt position at the 1e-2 bar
    for bf16 weights (1.5e-2 at 80 layers, see FULL_DEPTH_BAR); for the 8B and 70B shapes also ONE decode step on top
    of the prompt, teacher-forced with the oracle's token."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS[name]
    gold = _golden(name)
    toks = S.prompt_tokens(shape)
    tol = tol_for(shape) * FULL_DEPTH_BAR[name]
    layers = sorted({int(g[1]) for g in gold if g[0] == "hidden_rms"})
    with gpu_session(shape, len(toks) + 8, min(len(toks), 4096)) as ses:
        tok, lg = P.prefill(ses.h, toks, shape.vocab)
        for l in layers:
            for which, key in ((0, "attn"), (1, "ffn")):
                hr = float(next(g[3] for g in gold if g[0] == "hidden_rms" and int(g[1]) == l and g[2] == key))
                got = P.get_hidden(ses.h, l, which, shape.hidden)
                for g in gold:
                    if g[0] == "hidden" and int(g[1]) == l and g[2] == key:
                        assert abs(got[int(g[3])] - float(g[4])) <= 3 * tol * hr, (l, key, g[3])
                assert abs(np.sqrt(np.mean(got.astype(np.float64) ** 2)) - hr) <= tol * hr
        rel = [_check_stored_logits(gold, "", lg, tok, tol)]
        feed = [int(g[1]) for g in gold if g[0] == "dfeed"]
        if feed:
            tok2, lg2 = P.decode_step(ses.h, feed[0], shape.vocab)
            rel.append(_check_stored_logits(gold, "d", lg2, tok2, tol))
        print(f"[parity] {name} full depth: sampled logits off by {', '.join(f'{r:.2e}' for r in rel)} (prompt, decode step)")


def test_second_model_family_non_power_of_two_widths():
    """A shape from the paper's model list outside the Llama 2/3 sizes (Yi-34B: hidden 7168, 56 heads over 8 kv
    heads, FFN 20480): widths that are not powers of two, 7 query heads per kv head group... per shard, bf16,
    N = 8; two layers and a 32000-entry vocabulary so that the oracle finishes in seconds."""
    shape = S.CONFIGS["C3"].with_(n_layers=2, hidden=7168, n_heads=56, n_kv_heads=8, head_dim=128, ffn=20480, vocab=32000,
                                  rope_base=5000000.0)
    toks, mism = _run_and_compare(shape, 8, n_decode=4, prompt_len=96, max_ambiguous=3)
    assert mism <= 2


@pytest.mark.parametrize("cfg,n_shards,T,chunk", [("C2", 4, 128, None), ("C3", 8, 200, None), ("C3", 8, 300, None),
                                                   ("C3", 8, 300, 256)])
def test_full_width_reduced_depth(cfg, n_shards, T, chunk):
    """The benchmarked shapes end to end at full width (bf16, launch configuration of bench.py:
    graph + PDL), depth reduced to 2 layers and the vocabulary to 32000 so that the fp64 oracle
    finishes in seconds; teacher-forced, token rule applied at every step.  300 positions take the
    long-prompt kernels (CTA-pair projections, star sum in the GEMM epilogue, tcgen05 attention); in chunks
    of 256 + 44 the second chunk takes the short-prompt kernels on top of the first chunk's cache."""
    shape = S.CONFIGS[cfg].with_(n_layers=2, vocab=32000)
    toks, mism = _run_and_compare(shape, n_shards, n_decode=6, prompt_len=T, max_prefill=chunk, max_ambiguous=4)
    assert mism <= 3


def test_long_prompt_streamed_is_bit_identical_to_resident():
    """A 300-token prompt of the 8B shape (2 layers) through the long-prompt kernels: the window-streamed model must
    produce the resident model's bits (first token, its logits, and the tokens after it)."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C3"].with_(n_layers=2, vocab=32000)
    toks = S.prompt_tokens(shape, 300)
    res = {}
    for w in (0, 2):
        with gpu_session(shape, 320, 300, 8, w) as ses:
            t0, lg0 = P.prefill(ses.h, toks, shape.vocab)
            seq = P.decode_run(ses.h, t0, 4)
            res[w] = (t0, lg0, seq)
    assert res[0][0] == res[2][0] and (res[0][2] == res[2][2]).all()
    assert np.array_equal(res[0][1], res[2][1])
