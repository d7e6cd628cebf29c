"""Parity at the benchmarked shapes the fp64 oracle cannot run at full depth: the 70B widths end to end at reduced
depth (bf16 and fp32), one full-shape layer decoding over a synthetic cache of the workload's context length (Eq. 1
over the whole KV cache, Algorithm 1's loop body), and one 4096-token prompt through the single-chunk prompt pass."""
import numpy as np
import pytest

import tpi_synth as S
from tests.helpers import check_logits, close_elementwise, gpu_session, make_oracle, rel_l2, tol_for
from tests.test_gpu_e2e import _run_and_compare

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,n_shards,T", [("C5", 8, 96), ("C5", 2, 160), ("C4", 8, 40)])
def test_70b_widths_reduced_depth(cfg, n_shards, T):
    """Hidden 8192, 64 query / 8 kv heads, FFN 28672 end to end: two layers, vocabulary 32000 (so that the oracle
    finishes in a minute), prompt pass + teacher-forced decode.  bf16: 96 positions take the single-CTA GEMM tiles,
    160 the CTA-pair tiles with the star sum in the epilogue; fp32 (the streamed workload's kernels): 1e-5 bar."""
    shape = S.CONFIGS[cfg].with_(n_layers=2, vocab=32000)
    toks, mism = _run_and_compare(shape, n_shards, n_decode=4, prompt_len=T, max_ambiguous=3)
    if shape.dtype == "f32":
        assert mism == 0


@pytest.mark.parametrize("window", [8, 3])
def test_70b_fp32_streamed_is_bit_identical_to_resident(window):
    """The fp32 70B-shaped blocks (0.6 GB attention, 2.8 GB FFN) through the window ring: four layers = eight blocks,
    window 8 (every block has its own slot, loads run a full pass ahead) and window 3 (one attention + two FFN slots,
    every slot reused many times per token) must give the resident model's bits."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C4"].with_(n_layers=4, vocab=32000)
    toks = S.prompt_tokens(shape, 24)
    res = {}
    for w in (0, window):
        with gpu_session(shape, 40, 24, 8, w) as ses:
            t0, lg0 = P.prefill(ses.h, toks, shape.vocab)
            seq = P.decode_run(ses.h, t0, 4)
            t1, lg1 = P.decode_step(ses.h, int(seq[-1]), shape.vocab)
            res[w] = (t0, lg0, seq, t1, lg1)
            if w:
                st = P.get_stats(ses.h)
                assert st["blocks_loaded"] >= 6 * 8 and st["window_blocks"] == w
    a, b = res[0], res[window]
    assert a[0] == b[0] and a[3] == b[3] and (a[2] == b[2]).all()
    assert np.array_equal(a[1], b[1]) and np.array_equal(a[4], b[4])


@pytest.mark.parametrize("cfg,n_shards,ctx", [("C3", 8, 4096), ("C5", 8, 8192), ("C5", 2, 2048), ("C2", 4, 255)])
def test_single_layer_full_shape_decode_over_a_synthetic_cache(cfg, n_shards, ctx):
    """One layer at the workload's full shape (full vocabulary) decoding one token on top of a seeded cache of the
    workload's context length: the cache goes in through tpi_put_kv, the position through tpi_set_position, and
    H_attn (Eq. 1), H_ffn (Eq. 2), the logits, the token and the appended cache row are compared with a one-layer
    oracle holding the same cache."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS[cfg].with_(n_layers=1)
    b, d = shape.n_kv_heads, shape.head_dim
    tol = tol_for(shape)
    k = S.kv_contents(101, (b, ctx, d))
    v = S.kv_contents(102, (b, ctx, d))
    if shape.dtype == "bf16":   # the values as the cache stores them
        k = S.bf16_bits_to_f32(S.f32_to_bf16_bits(k)).reshape(k.shape)
        v = S.bf16_bits_to_f32(S.f32_to_bf16_bits(v)).reshape(v.shape)
    orc = make_oracle(shape)
    orc.cache.K, orc.cache.V = [k.astype(np.float64)], [v.astype(np.float64)]
    tok_in = int(S.prompt_tokens(shape, 1)[0])
    want = orc.forward([tok_in])
    with gpu_session(shape, ctx + 8, 16, n_shards) as ses:
        for g in range(b):
            P.put_kv(ses.h, 0, g, 0, k[g], v[g])
        P.set_position(ses.h, ctx)
        kb, vb = P.get_kv(ses.h, 0, b - 1, ctx - 3, 3, d)            # what went in comes back (exact for stored values)
        assert np.array_equal(kb, k[b - 1, ctx - 3:]) and np.array_equal(vb, v[b - 1, ctx - 3:])
        tok, lg = P.decode_step(ses.h, tok_in, shape.vocab)
        assert P.position(ses.h) == ctx + 1
        check_logits(lg, tok, want, tol)
        assert close_elementwise(P.get_hidden(ses.h, 0, 0, shape.hidden), orc.taps[(0, "attn")][-1], tol)
        assert close_elementwise(P.get_hidden(ses.h, 0, 1, shape.hidden), orc.taps[(0, "ffn")][-1], tol)
        for g in (0, b - 1):
            kn, vn = P.get_kv(ses.h, 0, g, ctx, 1, d)
            assert close_elementwise(kn, orc.cache.K[0][g][ctx:], tol) and close_elementwise(vn, orc.cache.V[0][g][ctx:], tol)
            ko, _ = P.get_kv(ses.h, 0, g, 0, ctx, d)                 # the older rows were not touched
            assert np.array_equal(ko, k[g])
        # a tighter look at Eq. 1 alone: with one layer, H_attn - embedding is W_O applied to the attention output
        emb = orc.w(0, S.EMB)[tok_in]
        got_delta = P.get_hidden(ses.h, 0, 0, shape.hidden).astype(np.float64) - emb
        assert rel_l2(got_delta, orc.taps[(0, "attn")][-1] - emb) < 1e-4


def test_long_prompt_single_chunk_full_width():
    """The 8B shape's 4096-token prompt as bench.py runs it: ONE chunk (CTA-pair projections over 16 position tiles,
    star sum in the GEMM epilogue, tcgen05 attention with 32 query tiles per head), one layer, vocabulary 32000.
    Last position: hidden states, logits, token; earlier positions: sampled cache rows of every kv head."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C3"].with_(n_layers=1, vocab=32000)
    T = 4096
    toks = S.prompt_tokens(shape, T)
    tol = tol_for(shape)
    orc = make_oracle(shape)
    want = orc.forward(toks)
    with gpu_session(shape, T + 8, T, 8) as ses:
        tok, lg = P.prefill(ses.h, toks, shape.vocab)
        check_logits(lg, tok, want, tol)
        assert close_elementwise(P.get_hidden(ses.h, 0, 0, shape.hidden), orc.taps[(0, "attn")][-1], tol)
        assert close_elementwise(P.get_hidden(ses.h, 0, 1, shape.hidden), orc.taps[(0, "ffn")][-1], tol)
        for g in range(shape.n_kv_heads):
            k, v = P.get_kv(ses.h, 0, g, 0, T, shape.head_dim)
            assert close_elementwise(k, orc.cache.K[0][g], tol) and close_elementwise(v, orc.cache.V[0][g], tol)
            for p in (0, 127, 128, 255, 256, 2047, 2048, 4095):      # tile edges of the position dimension
                assert close_elementwise(k[p], orc.cache.K[0][g][p], tol), (g, p)
        # one decode step on top of the 4096 cached positions (teacher-forced)
        feed = int(np.argmax(want))
        tok2, lg2 = P.decode_step(ses.h, feed, shape.vocab)
        check_logits(lg2, tok2, orc.forward([feed]), tol)
        assert close_elementwise(P.get_hidden(ses.h, 0, 1, shape.hidden), orc.taps[(0, "ffn")][-1], tol)


def test_stream_launches_with_dependent_launch_match_the_graph_bit_for_bit():
    """Without the CUDA graph the kernels of consecutive tokens are adjacent programmatic dependent launches; the
    attention kernel reads the position ahead of its dependency wait, which is only sound because the step's first
    kernel holds its dependents back until the previous token's head has advanced the position.  40 chained steps
    (bf16, head dimension 128: the tensor-core attention kernel) must give the graph replay's tokens and logits."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C3"].with_(n_layers=3, vocab=32000)
    toks = S.prompt_tokens(shape, 300)
    res = {}
    with gpu_session(shape, 400, 300, 8) as ses:
        for graph in (1, 0):
            P.set_option(ses.h, P.OPT_GRAPH, graph)
            P.set_option(ses.h, P.OPT_PDL, 1)
            P.reset(ses.h)
            t0, _ = P.prefill(ses.h, toks, 0)
            seq = P.decode_run(ses.h, t0, 40)
            assert bool(P.get_stats(ses.h)["graph_active"]) == bool(graph)
            t1, lg = P.decode_step(ses.h, int(seq[-1]), shape.vocab)
            res[graph] = (t0, seq, t1, lg)
    assert res[0][0] == res[1][0] and (res[0][1] == res[1][1]).all() and res[0][2] == res[1][2]
    assert np.array_equal(res[0][3], res[1][3])
