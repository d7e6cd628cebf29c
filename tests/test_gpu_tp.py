"""The one-shard-per-rank form (tpi_tp.h) on ONE GPU: R ranks as R models with their own arenas and streams in this
process, receive areas cross-wired, every exchange ordered by events between the streams (the flags are already set when
a consumer starts; its bounded wait is a backstop).  Against the oracle's per-device form (Eq. 1-2 as N devices compute
them), bit for bit against the emulated-shard model, and the failure path of a rank that never publishes."""
import numpy as np
import pytest

import tpi_synth as S
from tests.helpers import check_logits, close_elementwise, gpu_session, make_oracle, tol_for, tpi_config

pytestmark = pytest.mark.gpu


def _group(shape, R, max_seq, window=0, max_prefill=None, partition=None):
    import paper_2410_00531_b200.tp as TP
    return TP.Group(tpi_config(shape, max_seq, max_prefill or max_seq), S.synth_fill(shape), R, window, partition=partition)


CASES = {
    "c1_r2": (S.CONFIGS["C1"], 2, 12, 5),
    "c1_r4": (S.CONFIGS["C1"], 4, 12, 5),
    "bf16_gqa_r2": (S.CONFIGS["C1"].with_(dtype="bf16", n_heads=8, n_kv_heads=2, head_dim=32, seed=77, rope_base=500000.0), 2, 10, 4),
    "c3_widths_r8": (S.CONFIGS["C3"].with_(n_layers=2, vocab=32000), 8, 20, 3),
    "c3_widths_r8_long": (S.CONFIGS["C3"].with_(n_layers=2, vocab=32000), 8, 300, 2),
    "c5_widths_r2": (S.CONFIGS["C5"].with_(n_layers=1, vocab=32000), 2, 140, 2),
    "c2_widths_r4": (S.CONFIGS["C2"].with_(n_layers=2), 4, 12, 3),
    "f32_gqa_r1": (S.CONFIGS["C1"].with_(n_heads=8, n_kv_heads=4, head_dim=32), 1, 8, 3),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_ranks_match_the_oracle_s_per_device_form(case):
    """Prompt pass (all positions per pass, every rank on its slices; 300 positions take the CTA-pair GEMMs and the
    tcgen05 attention) + teacher-forced decode against `forward(n_shards=R)`: logits and token rule on the master, H_attn / H_ffn of every layer on EVERY rank (all ranks must hold the same bits after an allreduce), cache
    rows of every kv head on the rank that owns it."""
    shape, R, T, n_dec = CASES[case]
    tol = tol_for(shape)
    toks = S.prompt_tokens(shape, T)
    orc = make_oracle(shape)
    with _group(shape, R, T + n_dec + 2) as g:
        tok, lg = g.prefill(toks, shape.vocab)
        want = orc.forward(toks, n_shards=R)
        check_logits(lg, tok, want, tol)
        assert g.position() == T
        for step in range(n_dec + 1):
            for l in range(shape.n_layers):
                for which, key in ((0, "attn"), (1, "ffn")):
                    h0 = g.get_hidden(0, l, which)
                    assert close_elementwise(h0, orc.taps[(l, key)][-1], tol)
                    for r in range(1, R):
                        assert np.array_equal(g.get_hidden(r, l, which), h0), (r, l, key)
            if step == n_dec:
                break
            feed = int(np.argmax(want))
            tok, lg = g.decode_step(feed, shape.vocab)
            want = orc.forward([feed], n_shards=R)
            check_logits(lg, tok, want, tol)
        n = T + n_dec
        for l in range(shape.n_layers):
            for kvh in range(shape.n_kv_heads):
                k, v = g.get_kv(l, kvh, 0, n)
                assert close_elementwise(k, orc.cache.K[l][kvh], tol) and close_elementwise(v, orc.cache.V[l][kvh], tol)
        st = g.stats()
        assert st["n_ranks"] == R and st["position"] == n
        assert st["exchange_bytes_per_token"] == 2 * shape.n_layers * shape.hidden * 4 * (R - 1)
        # per position: master embed + broadcast, then per rank 1 + 2 * L consumers, 4 * L + ... kernels; the head once
        base = 2 + R * (1 + shape.n_layers * 7) + 1
        assert st["kernel_launches_last"] in (base, base + R)    # + one guard-zone check per rank under TPI_DEBUG=1


@pytest.mark.parametrize("case", ["c1_r2", "bf16_gqa_r2", "c3_widths_r8"])
def test_ranks_give_the_emulated_shard_model_s_bits(case):
    """R real ranks == N = R shards emulated on one model, bit for bit, when that model runs its row-sharded projections in
    the two-kernel form (partial sums through memory, then the rank-ordered sum) and is fed the prompt one position at a
    time through the same decode kernels.  Contexts stay within one attention split (256 positions)."""
    import paper_2410_00531_b200 as P
    import paper_2410_00531_b200.tp as TP
    shape, R, T, n_dec = CASES[case]
    toks = S.prompt_tokens(shape, T)
    with _group(shape, R, T + n_dec + 2) as g:
        g.set_option(TP.OPT_BATCHED_PROMPT, 0)                   # the prompt through the decode kernels, like the model below
        t_tp, lg_tp = g.prefill(toks, shape.vocab)
        seq_tp = g.decode_run(t_tp, n_dec)
        h_tp = [g.get_hidden(R - 1, l, w) for l in range(shape.n_layers) for w in (0, 1)]
    with gpu_session(shape, T + n_dec + 2, 1, R) as ses:
        P.set_option(ses.h, P.OPT_ROWSHARD_FUSED, 0)
        for t in toks[:-1]:
            P.decode_step(ses.h, int(t), 0)
        t_em, lg_em = P.decode_step(ses.h, int(toks[-1]), shape.vocab)
        seq_em = P.decode_run(ses.h, t_em, n_dec)
        h_em = [P.get_hidden(ses.h, l, w, shape.hidden) for l in range(shape.n_layers) for w in (0, 1)]
    assert t_tp == t_em and np.array_equal(lg_tp, lg_em) and (seq_tp == seq_em).all()
    for a, b in zip(h_tp, h_em):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("case,chunk", [("c1_r2", None), ("c1_r4", 5), ("bf16_gqa_r2", None), ("c3_widths_r8", None),
                                        ("c3_widths_r8_long", None), ("c3_widths_r8_long", 128)])
def test_prompt_pass_of_the_ranks_gives_the_emulated_model_s_prompt_pass_bits(case, chunk):
    """The batched prompt pass on R ranks against the emulated model's (N = R): the same GEMM, attention and row kernels
    run on slices instead of on the whole, every output element is accumulated in the same order, and the partial
    sums are added in rank order on both sides, so first token, logits and the last position's hidden states agree
    bit for bit; chunked prompts (a last chunk shorter than the others) included."""
    import paper_2410_00531_b200 as P
    shape, R, T, _ = CASES[case]
    toks = S.prompt_tokens(shape, T)
    with _group(shape, R, T + 4, max_prefill=chunk) as g:
        t_tp, lg_tp = g.prefill(toks, shape.vocab)
        h_tp = [g.get_hidden(0, l, w) for l in range(shape.n_layers) for w in (0, 1)]
        kv_tp = g.get_kv(shape.n_layers - 1, shape.n_kv_heads - 1, 0, T)
    with gpu_session(shape, T + 4, chunk or T, R) as ses:
        t_em, lg_em = P.prefill(ses.h, toks, shape.vocab)
        h_em = [P.get_hidden(ses.h, l, w, shape.hidden) for l in range(shape.n_layers) for w in (0, 1)]
        kv_em = P.get_kv(ses.h, shape.n_layers - 1, shape.n_kv_heads - 1, 0, T, shape.head_dim)
    assert t_tp == t_em and np.array_equal(lg_tp, lg_em)
    for a, b in zip(h_tp, h_em):
        assert np.array_equal(a, b)
    assert np.array_equal(kv_tp[0], kv_em[0]) and np.array_equal(kv_tp[1], kv_em[1])


@pytest.mark.parametrize("case", ["f32_gqa", "bf16_8b_widths"])
def test_ranks_with_unequal_shares_match_the_oracle(case):
    """Sec. 3.1's proportions p_i on real ranks: every rank holds a different number of kv-head groups and FFN columns
    (different kernels' shapes per rank), against the oracle's per-device form with the same partition; prompt pass
    (batched), decode, all ranks' hidden states equal, cache rows on their owners."""
    if case == "f32_gqa":
        shape = S.CONFIGS["C1"].with_(n_heads=8, n_kv_heads=4, head_dim=32, hidden=256, ffn=688, n_layers=3)
        part, T = ([2, 1, 1], [344, 200, 144]), 11
    else:
        shape = S.CONFIGS["C3"].with_(n_layers=2, vocab=32000)
        part, T = ([4, 2, 1, 1], [7168, 3584, 2048, 1536]), 150
    R, tol = len(part[0]), tol_for(shape)
    toks = S.prompt_tokens(shape, T)
    orc = make_oracle(shape)
    with _group(shape, R, T + 6, partition=part) as g:
        tok, lg = g.prefill(toks, shape.vocab)
        want = orc.forward(toks, n_shards=R, partition=part)
        check_logits(lg, tok, want, tol)
        for step in range(3):
            for l in range(shape.n_layers):
                for which, key in ((0, "attn"), (1, "ffn")):
                    h0 = g.get_hidden(0, l, which)
                    assert close_elementwise(h0, orc.taps[(l, key)][-1], tol)
                    for r in range(1, R):
                        assert np.array_equal(g.get_hidden(r, l, which), h0)
            feed = int(np.argmax(want))
            tok, lg = g.decode_step(feed, shape.vocab)
            want = orc.forward([feed], n_shards=R, partition=part)
            check_logits(lg, tok, want, tol)
        for kvh in range(shape.n_kv_heads):
            k, v = g.get_kv(shape.n_layers - 1, kvh, 0, T + 3)
            assert close_elementwise(k, orc.cache.K[-1][kvh], tol) and close_elementwise(v, orc.cache.V[-1][kvh], tol)
    with pytest.raises(Exception):
        _group(shape, R, 16, partition=(part[0][::-1][:R - 1] + [1], part[1]))   # heads do not add up


def test_one_graph_over_all_ranks_matches_stream_launches():
    """By default a decode position of all ranks is one CUDA graph (captured across the ranks' streams); the same kernels
    as plain stream launches, with and without programmatic dependent launch, must give the same tokens and logits."""
    import paper_2410_00531_b200.tp as TP
    shape, R, T, _ = CASES["c3_widths_r8"]
    toks = S.prompt_tokens(shape, T)
    res = {}
    with _group(shape, R, T + 40) as g:
        for key, graph, pdl in (("graph", 1, 1), ("stream", 0, 1), ("stream_no_pdl", 0, 0), ("graph_again", 1, 0)):
            g.set_option(TP.OPT_GRAPH, graph)
            g.set_option(TP.OPT_PDL, pdl)
            g.reset()
            t0, _ = g.prefill(toks, 0)
            seq = g.decode_run(t0, 24)
            t1, lg = g.decode_step(int(seq[-1]), shape.vocab)
            res[key] = (t0, seq, t1, lg)
            assert g.stats()["kernel_launches_last"] in (2 + R * (1 + shape.n_layers * 7) + 1, 2 + R * (2 + shape.n_layers * 7) + 1)
    for key in ("stream", "stream_no_pdl", "graph_again"):
        a, b = res["graph"], res[key]
        assert a[0] == b[0] and (a[1] == b[1]).all() and a[2] == b[2] and np.array_equal(a[3], b[3]), key


def test_streamed_ranks_give_the_resident_ranks_bits():
    """Every rank streams its own blocks through its own window (Sec. 3.3 runs on every device)."""
    shape = S.CONFIGS["C1"].with_(n_layers=4)
    toks = S.prompt_tokens(shape, 9)
    res = {}
    for w in (0, 2, 3):
        with _group(shape, 2, 32, w, max_prefill=4) as g:        # 9 prompt positions in chunks of 4 + 4 + 1
            t0, lg = g.prefill(toks, shape.vocab)
            res[w] = (t0, lg, g.decode_run(t0, 5))
    for w in (2, 3):
        assert res[w][0] == res[0][0] and np.array_equal(res[w][1], res[0][1]) and (res[w][2] == res[0][2]).all()


def test_a_rank_that_never_publishes_ends_in_a_timeout_status_and_reset_recovers():
    """Failure injection on the host: one rank's next push computes its partial sums but never publishes them.  The
    other ranks' consumers find no flag, give up after their poll limit (a few thousand polls here), the kernels
    return, and the call reports TPI_ERR_TIMEOUT naming a rank.  Further calls are refused until tpi_tp_reset, after
    which the same prompt gives the same tokens."""
    import paper_2410_00531_b200 as P
    import paper_2410_00531_b200.tp as TP
    shape = S.CONFIGS["C1"]
    toks = S.prompt_tokens(shape, 8)
    with _group(shape, 2, 32) as g:
        t0, lg0 = g.prefill(toks, shape.vocab)
        seq0 = g.decode_run(t0, 4)
        with pytest.raises(P.TpiError) as e:
            g.set_option(TP.OPT_EVENTS, 0)                       # two ranks on one device must be ordered by events
        assert e.value.code == -9
        for victim in (1, 0):
            g.set_option(TP.OPT_WAIT_POLLS, 4000)
            g.set_option(TP.OPT_DROP_PUSH, victim + 1)
            with pytest.raises(P.TpiError) as e:
                g.decode_step(int(seq0[-1]), 0)
            assert e.value.code == -7 and "rank" in str(e.value)
            with pytest.raises(P.TpiError) as e:
                g.decode_step(int(seq0[-1]), 0)                  # refused until the group is reset
            assert e.value.code == -9
            g.reset()
            # the same failure inside a prompt pass
            g.set_option(TP.OPT_DROP_PUSH, victim + 1)
            with pytest.raises(P.TpiError) as e:
                g.prefill(toks, 0)
            assert e.value.code == -7
            g.reset()
            g.set_option(TP.OPT_WAIT_POLLS, 1 << 21)
            t1, lg1 = g.prefill(toks, shape.vocab)
            seq1 = g.decode_run(t1, 4)
            assert t1 == t0 and np.array_equal(lg1, lg0) and (seq1 == seq0).all()
        with pytest.raises(P.TpiError) as e:
            g.decode_run(t1, 64)                                 # position + steps beyond max_seq
        assert e.value.code == -4
    with pytest.raises(P.TpiError) as e:
        _group(shape, 3, 32)                                     # 3 does not divide 4 heads
    assert e.value.code == -2
