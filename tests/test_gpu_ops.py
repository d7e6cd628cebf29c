"""Kernel-level parity at the workloads' real shapes: each step of the decoder path,
called alone through the C ABI (tpi_ops.h) on seeded inputs, against the CPU oracle's
definition of that step (fp64).  Shapes span many tiles and ragged tails."""
import numpy as np
import pytest

import tpi_synth as S
from oracle import llama_oracle as O
from tests.helpers import rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def T():
    import torch
    assert torch.cuda.is_available()
    return torch


_KEEP = []          # device tensors must outlive the asynchronous launches that read them


def dev(T, a):
    """numpy array -> device tensor holding the same bytes (uint16 bf16 bits travel as int16).
    The tensor is kept alive until the end of the test (see the autouse fixture)."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    t = T.from_numpy(a).cuda()
    _KEEP.append(t)
    return t


@pytest.fixture(autouse=True)
def _release_device_tensors():
    yield
    import torch
    torch.cuda.synchronize()
    _KEEP.clear()


def dt_of(shape):
    return 1 if shape.dtype == "bf16" else 0


def matvec64(w_stored, x64, chunk=8192):
    """fp64 W x for a stored (fp32 or bf16-bits) matrix, a band of rows at a time so that the fp64 copy of a
    70B-sized matrix never exists at once."""
    out = np.empty(w_stored.shape[0], np.float64)
    for r0 in range(0, w_stored.shape[0], chunk):
        out[r0:r0 + chunk] = S.as_f64(w_stored[r0:r0 + chunk]) @ x64
    return out


def pack_rows_sharded(w, n):           # row-sharded [h][K] -> [N][h][K/N]
    h, K = w.shape
    return np.ascontiguousarray(w.reshape(h, n, K // n).transpose(1, 0, 2))


def pack_gate_up(wg, wu, n):           # -> per shard rows gate_0, up_0, gate_1, up_1, ...
    s, h = wg.shape
    g = wg.reshape(n, s // n, 1, h)
    u = wu.reshape(n, s // n, 1, h)
    return np.ascontiguousarray(np.concatenate([g, u], axis=2).reshape(2 * s, h))


@pytest.mark.parametrize("cfg,n_shards", [("C2", 4), ("C1", 2), ("C3", 8), ("C5", 8), ("C5", 2), ("C4", 8)])
def test_gateup_swiglu(T, cfg, n_shards):
    import paper_2410_00531_b200.ops as K
    shape = S.CONFIGS[cfg]
    h, s = shape.hidden, shape.ffn
    wg, wu = S.gen_tensor(shape, 1, S.WGATE), S.gen_tensor(shape, 1, S.WUP)
    gain = S.as_f64(S.gen_tensor(shape, 1, S.FFN_NORM)).astype(np.float32)
    xhat = S.hidden_state(5, h, 1.0)
    act = T.empty(s, dtype=T.float32, device="cuda")
    K.gemv_gateup(dt_of(shape), dev(T, pack_gate_up(wg, wu, n_shards)).data_ptr(), dev(T, xhat).data_ptr(),
                  dev(T, gain).data_ptr(), h, s, n_shards, act.data_ptr())
    xn = xhat.astype(np.float64) * gain
    want = O.silu(matvec64(wg, xn)) * matvec64(wu, xn)
    got = act.cpu().numpy()
    assert rel_l2(got, want) < 2e-6
    assert np.abs(got - want).max() < 2e-5 * np.sqrt(np.mean(want * want))


@pytest.mark.parametrize("cfg,n_shards,which", [("C2", 4, S.WDOWN), ("C2", 4, S.WO), ("C3", 8, S.WO),
                                                ("C1", 2, S.WDOWN), ("C2", 1, S.WDOWN), ("C2", 2, S.WDOWN),
                                                ("C4", 8, S.WDOWN), ("C4", 8, S.WO), ("C5", 8, S.WO)])
def test_rowshard_partials_and_star_sum(T, cfg, n_shards, which):
    import paper_2410_00531_b200.ops as K
    shape = S.CONFIGS[cfg]
    w = S.gen_tensor(shape, 0, which)
    h, Kdim = w.shape
    x_in = S.hidden_state(6, Kdim, 0.7)
    resid = S.hidden_state(7, h, 0.5)
    Wd = dev(T, pack_rows_sharded(w, n_shards))
    part = T.empty((n_shards, h), dtype=T.float32, device="cuda")
    K.gemv_partials(dt_of(shape), Wd.data_ptr(), dev(T, x_in).data_ptr(), h, Kdim // n_shards, n_shards, part.data_ptr())
    w64, x64 = S.as_f64(w), x_in.astype(np.float64)
    cols = Kdim // n_shards
    want_p = np.stack([w64[:, i * cols:(i + 1) * cols] @ x64[i * cols:(i + 1) * cols] for i in range(n_shards)])
    assert rel_l2(part.cpu().numpy(), want_p) < 2e-6
    # allreduce + shortcut + norm statistics in one call, partials in caller scratch
    x = dev(T, resid.copy())
    xhat = T.empty(h, dtype=T.float32, device="cuda")
    scratch = T.empty(n_shards * h, dtype=T.float32, device="cuda")
    K.rowshard_project(dt_of(shape), Wd.data_ptr(), dev(T, x_in).data_ptr(), h, cols, n_shards, shape.rms_eps,
                       scratch.data_ptr(), x.data_ptr(), xhat.data_ptr())
    want_x = w64 @ x64 + resid
    assert rel_l2(x.cpu().numpy(), want_x) < 2e-6
    assert rel_l2(xhat.cpu().numpy(), O.rmsnorm(want_x, np.ones(h), shape.rms_eps)) < 2e-6
    # rank order matters for bit-reproducibility: the device sum equals ((P0 + P1) + ...) + x in fp32
    p32 = part.cpu().numpy()
    acc = p32[0].copy()
    for i in range(1, n_shards):
        acc = acc + p32[i]
    assert np.array_equal(x.cpu().numpy(), acc + resid)


@pytest.mark.parametrize("cfg,n_shards,p", [("C3", 8, 4095), ("C2", 4, 0), ("C1", 2, 17), ("C5", 8, 8191), ("C4", 8, 575)])
def test_qkv_rope_kv_append(T, cfg, n_shards, p):
    import paper_2410_00531_b200.ops as K
    shape = S.CONFIGS[cfg]
    h, a, b, d = shape.hidden, shape.n_heads, shape.n_kv_heads, shape.head_dim
    max_seq = p + 3
    wq, wk, wv = (S.gen_tensor(shape, 2, t) for t in (S.WQ, S.WK, S.WV))
    hps, kps = a // n_shards * d, b // n_shards * d
    packed = np.concatenate([np.concatenate([wq[i * hps:(i + 1) * hps], wk[i * kps:(i + 1) * kps],
                                             wv[i * kps:(i + 1) * kps]]) for i in range(n_shards)])
    gain = S.as_f64(S.gen_tensor(shape, 2, S.ATTN_NORM)).astype(np.float32)
    xhat = S.hidden_state(8, h, 1.0)
    esz = T.bfloat16 if shape.dtype == "bf16" else T.float32
    kc = T.zeros((b, max_seq, d), dtype=esz, device="cuda")
    vc = T.zeros((b, max_seq, d), dtype=esz, device="cuda")
    rope = T.empty((max_seq, d // 2, 2), dtype=T.float32, device="cuda")
    invf = T.empty(d // 2, dtype=T.float64, device="cuda")
    K.rope_table(shape.rope_base, d, max_seq, invf.data_ptr(), rope.data_ptr())
    q = T.empty(a * d, dtype=T.float32, device="cuda")
    pos = T.tensor([p], dtype=T.int32, device="cuda")
    K.gemv_qkv(dt_of(shape), dev(T, packed).data_ptr(), dev(T, xhat).data_ptr(), dev(T, gain).data_ptr(), h, a, b, d,
               n_shards, max_seq, pos.data_ptr(), rope.data_ptr(), q.data_ptr(), kc.data_ptr(), vc.data_ptr())
    xn = xhat.astype(np.float64) * gain
    pp = np.array([p])
    q_want = O.rope((S.as_f64(wq) @ xn).reshape(1, a, d), pp, shape.rope_base)[0]
    k_want = O.rope((S.as_f64(wk) @ xn).reshape(1, b, d), pp, shape.rope_base)[0]
    v_want = (S.as_f64(wv) @ xn).reshape(b, d)
    assert rel_l2(q.cpu().numpy(), q_want) < 3e-6
    kg, vg = kc.float().cpu().numpy(), vc.float().cpu().numpy()
    tol = 4e-3 if shape.dtype == "bf16" else 3e-6
    assert rel_l2(kg[:, p], k_want) < tol and rel_l2(vg[:, p], v_want) < tol
    if shape.dtype == "bf16":       # apart from rare last-bit flips the stored values ARE the RNE-rounded ones
        assert (kg[:, p] != O.round_bf16(k_want)).mean() < 0.02
    # nothing but row p was touched
    kg[:, p] = 0
    vg[:, p] = 0
    assert not kg.any() and not vg.any()
    # the table itself against the fp64 definition
    th = O.rope_angles(np.arange(max_seq), d, shape.rope_base)
    r = rope.cpu().numpy()
    assert np.abs(r[..., 0] - np.cos(th)).max() < 1e-7 and np.abs(r[..., 1] - np.sin(th)).max() < 1e-7


@pytest.mark.parametrize("dtype,a,b,d,n,nsplit", [
    ("bf16", 32, 8, 128, 4096, 34),      # C3: grouped heads, long cache
    ("bf16", 64, 8, 128, 8192, 37),      # C5 at context 8192
    ("bf16", 32, 32, 128, 200, 2),       # C2
    ("f32", 4, 4, 64, 24, 1),            # C1
    ("f32", 64, 8, 128, 577, 5),         # C4, ragged split
    ("bf16", 8, 2, 32, 1, 3),            # a single cached position, empty splits
    ("bf16", 8, 2, 128, 1, 3),           # the same on the tensor-core path
    ("bf16", 16, 2, 64, 700, 4),         # 8 heads per kv head, d = 64, three active splits
    ("bf16", 32, 8, 128, 257, 33),       # just past one split
    ("bf16", 56, 8, 128, 300, 3),        # 7 query heads per kv head (Yi-34B shape)
    ("bf16", 12, 4, 64, 95, 2),          # 3 per group, ragged 32-key tiles
    ("f32", 8, 4, 64, 33, 8),
])
def test_decode_attention(T, dtype, a, b, d, n, nsplit):
    import paper_2410_00531_b200.ops as K
    max_seq = n + 5
    k = S.kv_contents(11, (b, max_seq, d))
    v = S.kv_contents(12, (b, max_seq, d))
    if dtype == "bf16":
        k, v = S.bf16_bits_to_f32(S.f32_to_bf16_bits(k)).reshape(k.shape), S.bf16_bits_to_f32(S.f32_to_bf16_bits(v)).reshape(v.shape)
    k[:, n:], v[:, n:] = np.nan, np.nan        # nothing beyond the current position may be read
    q = S.hidden_state(13, a * d, 1.3)
    tt = T.bfloat16 if dtype == "bf16" else T.float32
    kc, vc = T.from_numpy(k).cuda().to(tt), T.from_numpy(v).cuda().to(tt)
    scratch = T.empty(K.attention_scratch_floats(a, b, d, nsplit), dtype=T.float32, device="cuda")
    tickets = T.zeros(b, dtype=T.int32, device="cuda")
    o = T.empty(a * d, dtype=T.float32, device="cuda")
    pos = T.tensor([n - 1], dtype=T.int32, device="cuda")
    for _ in range(2):                         # twice: the tickets must come back to zero
        K.decode_attention(1 if dtype == "bf16" else 0, dev(T, q).data_ptr(), kc.data_ptr(), vc.data_ptr(), pos.data_ptr(),
                           a, b, d, max_seq, nsplit, scratch.data_ptr(), tickets.data_ptr(), o.data_ptr())
    want = O.attention(q.astype(np.float64).reshape(1, a, d), k[:, :n].astype(np.float64), v[:, :n].astype(np.float64),
                       np.array([n - 1]))[0]
    # bf16 caches with d = 64 / 128 run on tensor cores with split-bf16 queries and weights (~2^-17 per operand)
    assert rel_l2(o.cpu().numpy(), want) < (2e-5 if dtype == "bf16" and d >= 64 else 5e-6)
    assert not tickets.cpu().numpy().any()


@pytest.mark.parametrize("cfg,vocab", [("C2", None), ("C1", None), ("C1", 999), ("C3", None), ("C5", None), ("C4", None),
                                       ("C3", 128255)])
def test_head_argmax(T, cfg, vocab):
    """Task head + greedy argmax at every benchmarked (vocabulary, hidden) pair: 32000 x 4096 (7B shape), 128256 x 4096
    (8B), 128256 x 8192 (70B, bf16), 32000 x 8192 in fp32, and odd vocabularies."""
    import paper_2410_00531_b200.ops as K
    shape = S.CONFIGS[cfg]
    if vocab:
        shape = shape.with_(vocab=vocab)
    h, v = shape.hidden, shape.vocab
    w = S.gen_tensor(shape, 0, S.HEAD)
    gain = S.as_f64(S.gen_tensor(shape, 0, S.FINAL_NORM)).astype(np.float32)
    xhat = S.hidden_state(21, h, 1.0)
    nb = K.head_blocks(v)
    logits = T.empty(v, dtype=T.float32, device="cuda")
    av, ai = T.empty(nb, dtype=T.float32, device="cuda"), T.empty(nb, dtype=T.int32, device="cuda")
    ticket = T.zeros(1, dtype=T.int32, device="cuda")
    tok = T.full((2,), -7, dtype=T.int32, device="cuda")
    wd = dev(T, w)
    K.head_argmax(dt_of(shape), wd.data_ptr(), dev(T, xhat).data_ptr(), dev(T, gain).data_ptr(), h, v,
                  logits.data_ptr(), av.data_ptr(), ai.data_ptr(), ticket.data_ptr(), tok.data_ptr())
    want = matvec64(w, xhat.astype(np.float64) * gain)
    lg = logits.cpu().numpy()
    assert rel_l2(lg, want) < 2e-6
    assert np.abs(lg - want).max() < 2e-5 * np.sqrt(np.mean(want * want))
    assert int(tok[1]) == int(np.argmax(lg)) and int(ticket[0]) == 0
    order = np.argsort(-want, kind="stable")
    if want[order[0]] - want[order[1]] > 1e-4:      # far above the fp32 accumulation error: the id is the oracle's
        assert int(tok[1]) == int(order[0])
    # ties go to the lowest index: duplicate the winning row at a lower and a higher index
    win = int(np.argmax(lg))
    lo, hi = (win // 2, min(v - 1, win + 5)) if win > 0 else (0, 5)
    wd[lo], wd[hi] = wd[win].clone(), wd[win].clone()      # in place on the device copy (a 2 GB matrix at the 70B shape)
    K.head_argmax(dt_of(shape), wd.data_ptr(), dev(T, xhat).data_ptr(), dev(T, gain).data_ptr(), h, v,
                  logits.data_ptr(), av.data_ptr(), ai.data_ptr(), ticket.data_ptr(), tok.data_ptr())
    assert int(tok[1]) == min(lo, win)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gemm_batched_ragged(T, dtype):
    import paper_2410_00531_b200.ops as K
    rng = np.random.default_rng(3)
    Tn, Kd, n_out, nb = 100, 344, 203, 2
    X = rng.standard_normal((Tn, nb * Kd)).astype(np.float32)           # batch b reads columns [b*Kd, (b+1)*Kd)
    W = (rng.standard_normal((nb, n_out, Kd)) * 0.02).astype(np.float32)
    Wst = S.f32_to_bf16_bits(W).reshape(W.shape) if dtype == "bf16" else W
    Y = T.zeros((nb, Tn, n_out), dtype=T.float32, device="cuda")
    K.gemm(1 if dtype == "bf16" else 0, dev(T, X).data_ptr(), Kd, nb * Kd, dev(T, Wst).data_ptr(), n_out * Kd,
           Y.data_ptr(), Tn * n_out, n_out, Tn, n_out, Kd, nb)
    W64 = S.as_f64(Wst)
    want = np.stack([X[:, b * Kd:(b + 1) * Kd].astype(np.float64) @ W64[b].T for b in range(nb)])
    assert rel_l2(Y.cpu().numpy(), want) < 2e-6


@pytest.mark.parametrize("dtype,a,b,d,Tq,pos0", [("f32", 4, 4, 64, 16, 0), ("bf16", 8, 2, 128, 37, 20), ("bf16", 8, 1, 32, 5, 0),
                                                    ("bf16", 4, 4, 128, 200, 0), ("bf16", 8, 2, 64, 130, 77), ("bf16", 2, 1, 128, 64, 64),
                                                    ("bf16", 4, 2, 128, 1, 300), ("bf16", 8, 2, 128, 300, 77),
                                                    ("bf16", 2, 1, 128, 513, 0), ("bf16", 2, 2, 128, 257, 1000),
                                                    ("bf16", 16, 2, 128, 300, 5)])
def test_prefill_attention(T, dtype, a, b, d, Tq, pos0):
    import paper_2410_00531_b200.ops as K
    n = pos0 + Tq
    max_seq = n + 2
    k, v = S.kv_contents(31, (b, max_seq, d)), S.kv_contents(32, (b, max_seq, d))
    if dtype == "bf16":
        k, v = S.bf16_bits_to_f32(S.f32_to_bf16_bits(k)).reshape(k.shape), S.bf16_bits_to_f32(S.f32_to_bf16_bits(v)).reshape(v.shape)
    q = S.kv_contents(33, (Tq, a, d))
    tt = T.bfloat16 if dtype == "bf16" else T.float32
    kc, vc = T.from_numpy(k).cuda().to(tt), T.from_numpy(v).cuda().to(tt)
    kc[:, n:], vc[:, n:] = float("nan"), float("nan")                # nothing past the newest position may be read
    o = T.empty((Tq, a, d), dtype=T.float32, device="cuda")
    K.prefill_attention(1 if dtype == "bf16" else 0, dev(T, q).data_ptr(), kc.data_ptr(), vc.data_ptr(), Tq, pos0, a, b, d,
                        max_seq, o.data_ptr())
    want = O.attention(q.astype(np.float64), k[:, :n].astype(np.float64), v[:, :n].astype(np.float64), np.arange(pos0, n))
    # bf16 caches with d = 64 / 128 run on tensor cores with split-bf16 queries and weights (~2^-17 per operand)
    assert rel_l2(o.cpu().numpy(), want) < (2e-5 if dtype == "bf16" else 5e-6)


@pytest.mark.parametrize("cfg,n_shards,which", [("C2", 4, S.WDOWN), ("C2", 4, S.WO), ("C3", 8, S.WO), ("C1", 2, S.WDOWN),
                                                ("C2", 1, S.WDOWN), ("C5", 8, S.WDOWN), ("C5", 2, S.WDOWN),
                                                ("C4", 8, S.WDOWN), ("C4", 8, S.WO)])
def test_rowshard_fused_is_bit_identical_to_partials_then_sum(T, cfg, n_shards, which):
    """The model driver's fused kernel keeps the N partial sums in registers; the result must be the
    same bits as partial sums through memory followed by the rank-ordered sum kernel."""
    import paper_2410_00531_b200.ops as K
    shape = S.CONFIGS[cfg]
    w = S.gen_tensor(shape, 3, which)
    h, Kdim = w.shape
    cols = Kdim // n_shards
    Wd = dev(T, pack_rows_sharded(w, n_shards))
    x_in = dev(T, S.hidden_state(16, Kdim, 0.7))
    resid = S.hidden_state(17, h, 0.5)
    x_a, x_b = dev(T, resid.copy()), dev(T, resid.copy())
    xhat = T.empty(h, dtype=T.float32, device="cuda")
    scratch = T.empty(n_shards * h, dtype=T.float32, device="cuda")
    K.rowshard_project(dt_of(shape), Wd.data_ptr(), x_in.data_ptr(), h, cols, n_shards, shape.rms_eps,
                       scratch.data_ptr(), x_a.data_ptr(), xhat.data_ptr())
    parts = T.empty(K.rowshard_fused_parts(h), dtype=T.float32, device="cuda")
    K.rowshard_fused(dt_of(shape), Wd.data_ptr(), x_in.data_ptr(), h, cols, n_shards, x_b.data_ptr(), parts.data_ptr())
    a, b = x_a.cpu().numpy(), x_b.cpu().numpy()
    assert np.array_equal(a, b)
    want = S.as_f64(w) @ S.hidden_state(16, Kdim, 0.7).astype(np.float64) + resid
    assert rel_l2(b, want) < 2e-6
    assert abs(float(parts.double().sum()) / float((want * want).sum()) - 1) < 1e-5


@pytest.mark.parametrize("Tn,K,n_out,nb", [(128, 4096, 12288, 1), (100, 4096, 1024, 1), (300, 1024, 4096, 4),
                                           (128, 2752, 4096, 4), (37, 64, 200, 2), (512, 3584, 640, 8),
                                           (300, 4160, 1000, 1), (513, 8192, 2048, 1), (1400, 1024, 768, 1)])
@pytest.mark.parametrize("split", [False, True])
def test_gemm_tensor_core_bf16(T, Tn, K, n_out, nb, split):
    """Prompt-pass projection on tcgen05: bf16 inputs, fp32 accumulation, against fp64 on the same
    bf16 values.  Batches model the row-sharded projections (batch b reads A's columns b*K..)."""
    import paper_2410_00531_b200.ops as KK
    rng = np.random.default_rng(Tn + K)
    A32 = rng.standard_normal((Tn, nb * K)).astype(np.float32)
    A = S.f32_to_bf16_bits(A32).reshape(Tn, nb * K)
    Alo = S.f32_to_bf16_bits(A32 - S.bf16_bits_to_f32(A).reshape(A32.shape)).reshape(Tn, nb * K) if split else None
    W = S.f32_to_bf16_bits((rng.standard_normal((nb, n_out, K)) * 0.02).astype(np.float32)).reshape(nb, n_out, K)
    Y = T.full((nb, Tn, n_out), float("nan"), dtype=T.float32, device="cuda")
    err = T.zeros(1, dtype=T.int32, device="cuda")
    KK.gemm_bf16(dev(T, A).data_ptr(), nb * K, K, dev(T, W).data_ptr(), n_out, Y.data_ptr(), Tn * n_out, n_out,
                 Tn, n_out, K, nb, err.data_ptr(), A_lo=dev(T, Alo).data_ptr() if split else None)
    T.cuda.synchronize()
    assert int(err[0]) == 0
    A64, W64 = S.as_f64(A), S.as_f64(W)
    if split:                       # hi + lo carries the fp32 activation to ~2^-17
        assert rel_l2(A64 + S.as_f64(Alo), A32) < 2e-5
        A64 = A64 + S.as_f64(Alo)
    want = np.stack([A64[:, b * K:(b + 1) * K] @ W64[b].T for b in range(nb)])
    got = Y.cpu().numpy()
    assert np.isfinite(got).all()
    # products of bf16 pairs are exact in fp32; what is left is the tensor core's fp32 accumulation
    # over K / 16 (split: K / 8) steps, each of which truncates: 9.3e-6 at K = 4096 in one chain
    assert rel_l2(got, want) < 2e-5
    if split and nb == 1 and Tn > 128 and K > 512:   # accumulated in chunks of 512 inputs (ragged last chunk included)
        assert rel_l2(got, want) < 3e-6


def test_tensor_core_accumulator_drift_and_what_the_chunks_do_about_it(T):
    """Why long contractions are accumulated in pieces: the tensor core truncates its fp32 accumulator at every step, so
    a long chain comes out too SMALL in magnitude (a systematic bias, not noise).  A batch of 2 forces the one-chain
    form at 300 positions: at K = 8192 its result is biased towards zero by about 1.6e-5 of the mean magnitude; the
    single batch at the same size runs in 512-input chunks and is ten times closer to the exact product of the same
    bf16 values; at 128 positions the two half chains sit in between."""
    import paper_2410_00531_b200.ops as KK
    rng = np.random.default_rng(5)
    K, n_out = 8192, 512
    err = T.zeros(1, dtype=T.int32, device="cuda")

    def run(Tn, nb):
        A32 = rng.standard_normal((Tn, nb * K)).astype(np.float32)
        A = S.f32_to_bf16_bits(A32).reshape(Tn, nb * K)
        Alo = S.f32_to_bf16_bits(A32 - S.bf16_bits_to_f32(A).reshape(A32.shape)).reshape(Tn, nb * K)
        W = S.f32_to_bf16_bits((rng.standard_normal((nb, n_out, K)) * 0.02).astype(np.float32)).reshape(nb, n_out, K)
        Y = T.zeros((nb, Tn, n_out), dtype=T.float32, device="cuda")
        KK.gemm_bf16(dev(T, A).data_ptr(), nb * K, K, dev(T, W).data_ptr(), n_out, Y.data_ptr(), Tn * n_out, n_out,
                     Tn, n_out, K, nb, err.data_ptr(), A_lo=dev(T, Alo).data_ptr())
        T.cuda.synchronize()
        assert int(err[0]) == 0
        A64, W64 = S.as_f64(A) + S.as_f64(Alo), S.as_f64(W)
        want = np.stack([A64[:, b * K:(b + 1) * K] @ W64[b].T for b in range(nb)])
        d = Y.cpu().numpy().astype(np.float64) - want
        return rel_l2(Y.cpu().numpy(), want), float((d * np.sign(want)).mean() / np.abs(want).mean())

    one_chain, bias = run(300, 2)
    assert 1e-5 < one_chain < 3e-5 and -3e-5 < bias < -1e-5, (one_chain, bias)
    chunked, bias_c = run(300, 1)
    assert chunked < 2e-6 and abs(bias_c) < 2e-6, (chunked, bias_c)
    halves, bias_h = run(128, 1)
    assert chunked < halves < one_chain and bias_h < 0, (halves, bias_h)


@pytest.mark.parametrize("shape", [0, 1, 2, 3])
@pytest.mark.parametrize("Tn,K,n_out,nb", [(300, 1024, 1000, 2), (513, 192, 2048, 1)])
def test_gemm_tensor_core_pair_shapes(T, monkeypatch, shape, Tn, K, n_out, nb):
    """Every CTA-pair tile shape (M = 256, one or two accumulators) on ragged position and column counts, pinned
    through the environment, against fp64 on the same bf16 values; tiles past the edge must not write."""
    import paper_2410_00531_b200.ops as KK
    monkeypatch.setenv("TPI_GEMM_PAIR_SHAPE", str(shape))
    rng = np.random.default_rng(Tn + K + shape)
    A32 = rng.standard_normal((Tn, nb * K)).astype(np.float32)
    A = S.f32_to_bf16_bits(A32).reshape(Tn, nb * K)
    Alo = S.f32_to_bf16_bits(A32 - S.bf16_bits_to_f32(A).reshape(A32.shape)).reshape(Tn, nb * K)
    W = S.f32_to_bf16_bits((rng.standard_normal((nb, n_out, K)) * 0.02).astype(np.float32)).reshape(nb, n_out, K)
    Y = T.full((nb * Tn * n_out + 4096,), 7.0, dtype=T.float32, device="cuda")
    err = T.zeros(1, dtype=T.int32, device="cuda")
    KK.gemm_bf16(dev(T, A).data_ptr(), nb * K, K, dev(T, W).data_ptr(), n_out, Y.data_ptr(), Tn * n_out, n_out,
                 Tn, n_out, K, nb, err.data_ptr(), A_lo=dev(T, Alo).data_ptr())
    T.cuda.synchronize()
    assert int(err[0]) == 0
    A64 = S.as_f64(A) + S.as_f64(Alo)
    W64 = S.as_f64(W)
    want = np.stack([A64[:, b * K:(b + 1) * K] @ W64[b].T for b in range(nb)])
    got = Y.cpu().numpy()
    assert (got[nb * Tn * n_out:] == 7.0).all()
    assert rel_l2(got[:nb * Tn * n_out].reshape(nb, Tn, n_out), want) < 2e-5


@pytest.mark.parametrize("Tn,K,n_out,nb", [(300, 512, 1000, 4), (513, 192, 4096, 8), (129, 64, 260, 1), (1024, 1792, 512, 3),
                                           (1700, 256, 1024, 2)])   # 7 position tiles: a band of 4 and a lower last band of 3
def test_gemm_rowsum_star_sum_in_epilogue(T, Tn, K, n_out, nb):
    """Row-sharded projection with the star sum and shortcut in the GEMM's epilogue (Eq. 1-2 for T positions): against
    fp64, and bit for bit against the two-kernel path (partial sums in memory, then the rank-ordered sum)."""
    import paper_2410_00531_b200.ops as KK
    rng = np.random.default_rng(Tn + K + nb)
    A32 = rng.standard_normal((Tn, nb * K)).astype(np.float32)
    A = S.f32_to_bf16_bits(A32).reshape(Tn, nb * K)
    Alo = S.f32_to_bf16_bits(A32 - S.bf16_bits_to_f32(A).reshape(A32.shape)).reshape(Tn, nb * K)
    W = S.f32_to_bf16_bits((rng.standard_normal((nb, n_out, K)) * 0.02).astype(np.float32)).reshape(nb, n_out, K)
    X0 = rng.standard_normal((Tn, n_out)).astype(np.float32)
    Ad, Ald, Wd = dev(T, A), dev(T, Alo), dev(T, W)
    err = T.zeros(1, dtype=T.int32, device="cuda")
    Xa = T.cat([dev(T, X0.copy()).flatten(), T.full((1024,), 7.0, dtype=T.float32, device="cuda")])
    KK.gemm_bf16_rowsum(Ad.data_ptr(), Ald.data_ptr(), nb * K, K, Wd.data_ptr(), n_out, Xa.data_ptr(), n_out, Tn, n_out, K, nb,
                        err.data_ptr())
    T.cuda.synchronize()
    assert int(err[0]) == 0
    got = Xa.cpu().numpy()
    assert (got[Tn * n_out:] == 7.0).all()
    got = got[:Tn * n_out].reshape(Tn, n_out)
    A64, W64 = S.as_f64(A) + S.as_f64(Alo), S.as_f64(W)
    want = sum(A64[:, b * K:(b + 1) * K] @ W64[b].T for b in range(nb)) + X0
    assert rel_l2(got, want) < 2e-5
    # the same partial sums through memory, summed by the row kernel in rank order
    P = T.empty((nb, Tn, n_out), dtype=T.float32, device="cuda")
    KK.gemm_bf16(Ad.data_ptr(), nb * K, K, Wd.data_ptr(), n_out, P.data_ptr(), Tn * n_out, n_out, Tn, n_out, K, nb,
                 err.data_ptr(), A_lo=Ald.data_ptr())
    Xb = dev(T, X0.copy())
    g = T.ones(n_out, dtype=T.float32, device="cuda")
    Xn = T.empty((Tn, n_out), dtype=T.float32, device="cuda")
    KK.reduce_residual_norm_rows(P.data_ptr(), nb, Tn, n_out, Xb.data_ptr(), g.data_ptr(), 1e-5, Xn.data_ptr())
    T.cuda.synchronize()
    assert int(err[0]) == 0
    assert np.array_equal(Xb.cpu().numpy(), got)


@pytest.mark.parametrize("Tn,K,s", [(128, 4096, 11008), (70, 1024, 1360), (300, 512, 48), (300, 4160, 496), (513, 8192, 1360)])
@pytest.mark.parametrize("split_out", [False, True])
def test_gemm_tensor_core_swiglu_epilogue(T, Tn, K, s, split_out):
    """Eq. 2's gate/up projection for T positions with SwiGLU applied in the GEMM's epilogue (gate_j, up_j rows
    interleaved): against the oracle's silu on the fp64 product of the same bf16 values."""
    import paper_2410_00531_b200.ops as KK
    rng = np.random.default_rng(Tn + K + s)
    A32 = rng.standard_normal((Tn, K)).astype(np.float32)
    A = S.f32_to_bf16_bits(A32).reshape(Tn, K)
    Alo = S.f32_to_bf16_bits(A32 - S.bf16_bits_to_f32(A).reshape(A32.shape)).reshape(Tn, K)
    W = S.f32_to_bf16_bits((rng.standard_normal((2 * s, K)) * 0.05).astype(np.float32)).reshape(2 * s, K)
    ACT = T.full((2, Tn, s), -1, dtype=T.int16, device="cuda")       # hi plane, lo plane (bf16 bits)
    err = T.zeros(1, dtype=T.int32, device="cuda")
    KK.gemm_bf16_swiglu(dev(T, A).data_ptr(), K, dev(T, W).data_ptr(), ACT.data_ptr(), split_out, Tn, s, K,
                        err.data_ptr(), A_lo=dev(T, Alo).data_ptr())
    T.cuda.synchronize()
    assert int(err[0]) == 0
    y = (S.as_f64(A) + S.as_f64(Alo)) @ S.as_f64(W).T
    want = O.silu(y[:, 0::2]) * y[:, 1::2]
    planes = ACT.cpu().numpy().view(np.uint16)
    hi = S.as_f64(planes[0])
    if split_out:
        got = hi + S.as_f64(planes[1])
        assert rel_l2(got, want) < 2e-5                              # hi + lo keeps ~16 bits of the fp32 value
    else:
        assert (planes[1] == 0xFFFF).all()                           # the second plane is not touched
        got = hi
        assert rel_l2(got, want) < 3e-3                              # one bf16 rounding of each output
    # element by element: the high plane is the fp32 result rounded to bf16 (half an ulp, 2^-9 relative), on top of
    # the fp32 accumulation error of the two dot products, which scales with the size of y, not of the output
    bound = np.abs(want) * 2.0 ** -8 + 2e-5 * np.abs(y).max() * (1 + np.abs(y[:, 1::2]))
    assert (np.abs(hi - want) <= bound).all()


@pytest.mark.parametrize("Tn,h,N", [(128, 4096, 4), (37, 8192, 8), (5, 256, 2), (200, 1000, 3)])
def test_reduce_residual_norm_rows(T, Tn, h, N):
    """Star sum in rank order + shortcut for T positions, then the next block's RMSNorm (Eq. 1-2 and the norm
    of Step 3), against the oracle; the residual stream itself must equal the stand-alone sum kernel's bits."""
    import paper_2410_00531_b200.ops as KK
    rng = np.random.default_rng(Tn * h + N)
    P = rng.standard_normal((N, Tn, h)).astype(np.float32)
    X0 = rng.standard_normal((Tn, h)).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(h)).astype(np.float32)
    eps = 1e-5
    X = dev(T, X0.copy())
    Xn = T.full((Tn, h), float("nan"), dtype=T.float32, device="cuda")
    KK.reduce_residual_norm_rows(dev(T, P).data_ptr(), N, Tn, h, X.data_ptr(), dev(T, g).data_ptr(), eps, Xn.data_ptr())
    T.cuda.synchronize()
    want_x = P.astype(np.float64).sum(0) + X0
    assert rel_l2(X.cpu().numpy(), want_x) < 1e-6
    acc = P[0].copy()
    for i in range(1, N):
        acc = acc + P[i]                                             # fp32, rank order, shortcut last
    assert np.array_equal(X.cpu().numpy(), acc + X0)
    assert rel_l2(Xn.cpu().numpy(), O.rmsnorm(want_x, g.astype(np.float64), eps)) < 2e-6
