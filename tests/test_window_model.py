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
