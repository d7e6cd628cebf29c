"""Pins for the window-scheduler model: the paper's printed block sizes, its
worked timing example with the time-slot expressions of Appendix A.3, Prop. 5."""
import os

from oracle import window_model as W

G = os.path.join(os.path.dirname(__file__), "golden")


def _read(name):
    rows = []
    for line in open(os.path.join(G, name)):
        if line.strip() and not line.startswith("#"):
            rows.append(line.split())
    return rows


def test_table5_block_sizes():
    h, v, a, b, s, p = 4096, 32000, 32, 32, 11008, 0.25
    for kind, mb in _read("table5_block_sizes.txt"):
        got = W.block_params(kind, h, v, a, b, s, p) * 4 / 2**20
        assert round(got) == int(mb), (kind, got)


def test_table6_required_memory_70b():
    (_, L, h, a, b, s, v, gb), = _read("table6_required_mem.txt")
    L, h, a, b, s, v = map(int, (L, h, a, b, s, v))
    params = (L * (W.block_params("attn", h, v, a, b, s, 1.0) + W.block_params("ffn", h, v, a, b, s, 1.0))
              + W.block_params("pre", h, v, a, b, s, 1.0) + W.block_params("post", h, v, a, b, s, 1.0))
    assert round(params * 4 / 2**30) == int(gb)


def test_worked_example_conditions_and_timeline():
    ex = {k: float(v) for k, v in _read("worked_timing_example.txt")}
    t = (ex["t_attn"], ex["t_ffn"], ex["t_all_reduce"], ex["tau_attn"], ex["tau_ffn"])
    assert W.tight_condition(*t) == bool(ex["tight"])
    assert W.loose_condition(*t, L=32) == bool(ex["loose"])
    ta, tf, tr, la, lf = t
    # Appendix A.3's slot expressions, evaluated by hand for this example with an unbounded window:
    stall, slack, _ = W.timeline(*t, n_blocks=64, w=10**6)
    assert stall[0] == la                                     # slot 1: the first block must load first
    assert stall[1] == -(ta + tr - lf) == 5                   # slot 3: t' = 11 + 14 - 30 = -5
    assert slack[2] == max(0, ta + tr - lf) + tf + tr - la == 13          # slot 5
    assert slack[3] == 13 + ta + tr - lf == 8                 # slot 7
    assert slack[4] == ta + 2 * tf + 3 * tr - 2 * la - lf == 21           # slot 9 (case 2)
    assert all(s == 0 for s in stall[2:])
    # with the paper's w = 4 the run reaches the steady state too: one 5 ms stall, then none
    stall4, _, end4 = W.timeline(*t, n_blocks=64, w=int(ex["w"]))
    assert stall4[1] == 5 and all(s == 0 for s in stall4[2:])
    assert end4 == la + 5 + 32 * (ta + tf + 2 * tr)


def test_window_one_blocks_on_every_load():
    stall, _, end = W.timeline(11, 17, 14, 18, 30, n_blocks=6, w=1)
    assert stall == [18, 30, 18, 30, 18, 30]
    assert end == 3 * (18 + 30 + 11 + 17 + 28)


def test_timeline_steady_when_tight_condition_holds():
    stall, _, _ = W.timeline(20, 25, 14, 18, 30, n_blocks=40, w=2)
    assert W.tight_condition(20, 25, 14, 18, 30) and all(s == 0 for s in stall[1:])


def test_prop5_worker_peak_counts_blocks():
    h, a, b, s, p = 8192, 64, 8, 28672, 0.125
    attn = 2 * (1 + b / a) * h * h * p + h
    ffn = 3 * h * s * p + h
    assert W.worker_peak(1, h, a, b, s, p) == ffn
    assert W.worker_peak(2, h, a, b, s, p) == attn + ffn
    assert W.worker_peak(5, h, a, b, s, p) == 2 * attn + 3 * ffn
    v = 32000
    assert W.master_peak(1, h, v, a, b, s, p) == h * v + h
    assert W.master_peak(4, h, v, a, b, s, p) == 2 * h * v + h + attn + ffn
    # the attention block of Table 5 and the one of Prop. 5 are the same count
    assert W.block_params("attn", h, v, a, b, s, p) == attn


def test_prop5_peaks_add_up_table5_s_printed_block_sizes():
    """Prop. 5 against numbers the paper prints, not against the formula typed again: Table 5 gives the blocks of
    Llama 2-7B with n = 4, p = 0.25 in FP32 as 500 / 64 / 129 / 500 MB, and Prop. 5 says which of them a window of w
    blocks holds: a worker floor(w/2) attention + ceil(w/2) FFN blocks (w = 1: the larger, FFN); the master its
    pre/postprocess blocks first (w = 1: the postprocess block, w = 2: both) and the layer blocks in what is left."""
    import os
    rows = [ln.split() for ln in open(os.path.join(os.path.dirname(__file__), "golden", "table5_block_sizes.txt")) if ln[0] != "#"]
    mb = {k: float(v) for k, v in rows}
    h, v, a, b, s, p = 4096, 32000, 32, 32, 11008, 0.25
    MiB = 2.0 ** 20 / 4          # parameters per printed MB (FP32)
    for w, want in ((1, mb["ffn"]), (2, mb["attn"] + mb["ffn"]), (3, mb["attn"] + 2 * mb["ffn"]),
                    (4, 2 * mb["attn"] + 2 * mb["ffn"]), (8, 4 * (mb["attn"] + mb["ffn"]))):
        assert abs(W.worker_peak(w, h, a, b, s, p) / MiB - want) < 0.5 * w, w        # the printed sizes are rounded to 1 MB
    for w, want in ((1, mb["post"]), (2, mb["pre"] + mb["post"]), (3, mb["pre"] + mb["post"] + mb["ffn"]),
                    (4, mb["pre"] + mb["post"] + mb["attn"] + mb["ffn"]), (6, mb["pre"] + mb["post"] + 2 * (mb["attn"] + mb["ffn"]))):
        assert abs(W.master_peak(w, h, v, a, b, s, p) / MiB - want) < 0.5 * w, w


def test_retention_slot_expressions_and_prop6():
    """Appendix A.6's time-slot expressions evaluated by hand on the paper's measured latencies
    (t_attn 11, t_ffn 17, tau_attn 18, tau_ffn 30; allreduce 14 as in the worked example) with T = 2."""
    ta, tf, tr, la, lf = 11.0, 17.0, 14.0, 18.0, 30.0
    stall, slack, _ = W.timeline_retained(ta, tf, tr, la, lf, n_blocks=64, w=10**6, T=2, L=32)
    assert stall[0] == la and all(s == 0 for s in stall[1:])
    assert slack[1] == 0                                                   # slot 3: layer 1's FFN block is kept
    assert slack[2] == ta + tf + 2 * tr - la == 38                         # slot 5 with the indicator = 1
    assert slack[3] == 2 * ta + tf + 3 * tr - lf - la == 33                # slot 7: one FFN load so far
    assert slack[4] == 2 * ta + 2 * tf + 4 * tr - lf - 2 * la == 46        # slot 9
    assert W.retained_ffn_layers(7, 3) == {0, 3, 6} and W.retained_ffn_layers(7, 0) == set()
    # no retention: the same model as the plain timeline, at every window size
    for w in (1, 2, 4, 6, 10**6):
        assert W.timeline_retained(ta, tf, tr, la, lf, 64, w, 0, 32) == W.timeline(ta, tf, tr, la, lf, 64, w)


def test_prop6_decides_the_steady_state_of_the_timeline():
    """A link twice as slow for FFN blocks (tau_ffn 60) breaks Prop. 3; Prop. 6 says which T repairs it,
    and the event model with an unbounded window stalls exactly when Prop. 6 fails."""
    ta, tf, tr, la, lf = 11.0, 17.0, 14.0, 18.0, 60.0
    assert not W.loose_condition(ta, tf, tr, la, lf, L=32)
    verdicts = {}
    for T in (1, 2, 3, 4, 8):
        stall, _, end = W.timeline_retained(ta, tf, tr, la, lf, n_blocks=64, w=10**6, T=T, L=32)
        steady = all(s == 0 for s in stall[1:])
        verdicts[T] = steady
        assert steady == W.retention_condition(ta, tf, tr, la, lf, L=32, T=T), T
        if steady:
            assert end == la + 32 * (ta + tf + 2 * tr)
    assert verdicts == {1: True, 2: True, 3: False, 4: False, 8: False}
    # by hand for T = 3 at l = 3: 3*56 = 168 < (3 - 1)*60 + 3*18 = 174
    assert 3 * (ta + tf + 2 * tr) < 2 * lf + 3 * la
