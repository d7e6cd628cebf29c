"""Pins for the oracle's building blocks: closed forms, invariants, special
cases that reduce to a library routine (torch CPU fp64), high-precision angles."""
import mpmath
import numpy as np
import torch
import torch.nn.functional as F

from oracle import llama_oracle as O

RNG = np.random.default_rng(11)


# ------------------------------------------------------------------ RMSNorm
def test_rmsnorm_unit_rms_and_scale_invariance():
    x = RNG.standard_normal((3, 64))
    y = O.rmsnorm(x, np.ones(64), 0.0)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0, atol=1e-14)
    assert np.allclose(O.rmsnorm(7.5 * x, np.ones(64), 0.0), y, atol=1e-14)


def test_rmsnorm_matches_torch():
    x, g = RNG.standard_normal((5, 96)), RNG.standard_normal(96)
    want = F.rms_norm(torch.from_numpy(x), (96,), torch.from_numpy(g), eps=1e-5).numpy()
    assert np.abs(O.rmsnorm(x, g, 1e-5) - want).max() < 1e-14


def test_rmsnorm_eps_is_inside_the_root():
    x = np.full(4, 2.0)
    assert np.allclose(O.rmsnorm(x, np.ones(4), 5.0), 2.0 / 3.0)      # 2 / sqrt(4 + 5)


# --------------------------------------------------------------------- RoPE
def test_rope_identity_at_zero_and_norm_preserved():
    u = RNG.standard_normal((4, 3, 16))
    assert np.array_equal(O.rope(u, np.zeros(4), 10000.0), u)
    r = O.rope(u, np.array([1, 17, 300, 8191]), 500000.0)
    pair = lambda t: t[..., :8] ** 2 + t[..., 8:] ** 2
    assert np.abs(pair(r) / pair(u) - 1).max() < 1e-13


def test_rope_inner_product_depends_on_offset_only():
    q, k = RNG.standard_normal((1, 1, 32)), RNG.standard_normal((1, 1, 32))
    dot = lambda m, n: float((O.rope(q, np.array([m]), 1e4) * O.rope(k, np.array([n]), 1e4)).sum())
    assert abs(dot(5, 2) - dot(105, 102)) < 1e-11
    assert abs(dot(5, 2) - dot(7, 2)) > 1e-3


def test_rope_angles_high_precision():
    mpmath.mp.dps = 50
    d, base, p = 128, 500000.0, 8191
    th = O.rope_angles(np.array([p]), d, base)[0]
    for i in (0, 1, 31, 63):
        want = mpmath.mpf(p) * mpmath.power(base, mpmath.mpf(-2 * i) / d)
        assert abs(th[i] - float(want)) <= 4e-16 * float(want) + 1e-18
    u = np.zeros((1, 1, d)); u[0, 0, 1] = 1.0          # unit vector in pair 1
    r = O.rope(u, np.array([p]), base)[0, 0]
    want = mpmath.mpf(p) * mpmath.power(base, mpmath.mpf(-2) / d)
    assert abs(r[1] - float(mpmath.cos(want))) < 1e-11 and abs(r[1 + d // 2] - float(mpmath.sin(want))) < 1e-11


def test_rope_hand_example():
    # d = 2: a single pair rotated by p radians (base^0 = 1): (1, 0) -> (cos p, sin p)
    u = np.array([[[1.0, 0.0]]])
    r = O.rope(u, np.array([2]), 10000.0)[0, 0]
    assert np.allclose(r, [np.cos(2.0), np.sin(2.0)], atol=1e-15)


# ------------------------------------------------------------ softmax / SiLU
def test_softmax_rows_sum_to_one_and_shift_invariance():
    sc = RNG.standard_normal((6, 50)) * 30
    w = O.softmax(sc)
    assert np.abs(w.sum(-1) - 1).max() < 1e-14
    assert np.abs(O.softmax(sc + 1000.0) - w).max() < 1e-13


def test_silu_identities_and_torch():
    t = RNG.standard_normal(1000) * 4
    assert O.silu(np.zeros(1))[0] == 0.0
    assert np.abs(O.silu(t) - O.silu(-t) - t).max() < 1e-14
    assert np.abs(O.silu(t) - F.silu(torch.from_numpy(t)).numpy()).max() < 1e-15


# ---------------------------------------------------------------- attention
def test_attention_special_cases():
    d, b, a, n = 8, 2, 4, 6
    K, V = RNG.standard_normal((b, n, d)), RNG.standard_normal((b, n, d))
    q = RNG.standard_normal((1, a, d))
    # only position 0 visible -> output is V[g, 0]
    o = O.attention(q, K, V, np.array([0]))
    for j in range(a):
        assert np.allclose(o[0, j], V[j // 2, 0], atol=1e-15)
    # q = 0 -> uniform weights -> mean of the visible values
    o = O.attention(np.zeros((1, a, d)), K, V, np.array([3]))
    assert np.allclose(o[0, 3], V[1, :4].mean(0), atol=1e-15)
    # identical value rows -> that row
    Vc = np.broadcast_to(V[:, :1], V.shape)
    o = O.attention(q, K, Vc, np.array([n - 1]))
    assert np.allclose(o[0, 0], V[0, 0], atol=1e-14)


def test_attention_matches_torch_sdpa_gqa_causal():
    d, b, a, T = 16, 2, 6, 9
    q = RNG.standard_normal((T, a, d))
    K, V = RNG.standard_normal((b, T, d)), RNG.standard_normal((b, T, d))
    got = O.attention(q, K, V, np.arange(T))
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]            # [1, a, T, d]
    want = F.scaled_dot_product_attention(tq, torch.from_numpy(K)[None], torch.from_numpy(V)[None],
                                          is_causal=True, enable_gqa=True)[0].permute(1, 0, 2).numpy()
    assert np.abs(got - want).max() < 1e-13


def test_attention_ignores_positions_beyond_the_query():
    d, n = 8, 10
    K, V = RNG.standard_normal((1, n, d)), RNG.standard_normal((1, n, d))
    q = RNG.standard_normal((1, 1, d))
    ref = O.attention(q, K[:, :5], V[:, :5], np.array([4]))
    Kp, Vp = K.copy(), V.copy()
    Kp[:, 5:] = 1e30; Vp[:, 5:] = -1e30                        # garbage tail must not leak
    assert np.array_equal(O.attention(q, Kp, Vp, np.array([4])), ref)


def test_round_bf16():
    x = np.array([1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8, -0.3, 123.456])
    r = O.round_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 + 2.0**-6
    assert np.all(np.abs(r / x - 1) <= 2.0**-8)
    assert np.array_equal(O.round_bf16(r), r)
