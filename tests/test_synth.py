"""The seeded input generator: the numpy and compiled twins agree bit for bit,
values have the stated distribution, bf16 rounding is round-to-nearest-even."""
import ml_dtypes
import numpy as np

import tpi_synth as S
from tpi_synth import gen


def test_twins_agree_bitwise():
    n = 1_000_000
    for uid, start, off, sc in ((20, 5, 0.0, 0.02), (3, 0, 1.0, 0.02), (16 * 79 + 11, 2**33, 0.0, 0.02)):
        a = gen.weight_values_numpy(2024, uid, start, n, off, sc)
        b = np.empty(n, np.float32)
        gen.fill_raw(2024, uid, start, n, off, sc, False, b.ctypes.data)
        assert (a.view(np.uint32) == b.view(np.uint32)).all()
        c = np.empty(n, np.uint16)
        gen.fill_raw(2024, uid, start, n, off, sc, True, c.ctypes.data)
        assert (gen.f32_to_bf16_bits(a) == c).all()


def test_distribution():
    n = 1_000_000
    a = gen.weight_values_numpy(1, 4, 0, n, 0.0, 0.02).astype(np.float64)
    assert abs(a.mean()) < 3 * 0.02 / np.sqrt(n)
    assert abs(a.std() / 0.02 - 1) < 2e-3
    assert np.abs(a).max() < 0.02 * 4.95           # Irwin-Hall(8) support


def test_bf16_is_rne_and_exact_upcast():
    a = gen.weight_values_numpy(9, 9, 0, 200_000, 0.0, 0.02)
    bits = gen.f32_to_bf16_bits(a)
    assert (bits == a.astype(ml_dtypes.bfloat16).view(np.uint16)).all()
    back = gen.bf16_bits_to_f32(bits)
    assert (back == a.astype(ml_dtypes.bfloat16).astype(np.float32)).all()
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    t = np.array([1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8], np.float32)
    assert list(gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(t))) == [1.0, 1.0 + 2.0**-6]


def test_tensors_do_not_depend_on_chunking_or_shards():
    sh = S.CONFIGS["C1"]
    full = S.gen_tensor(sh, 1, gen.WO)
    part = np.empty(1000, np.float32)
    gen.fill_raw(sh.seed, gen.tensor_uid(1, gen.WO), 12345, 1000, 0.0, 0.02, False, part.ctypes.data)
    assert (full.ravel()[12345:13345] == part).all()
    assert (S.gen_tensor(sh, 1, gen.WO, fast=False) == full).all()
    assert S.gen_tensor(sh, 0, gen.ATTN_NORM).mean() > 0.9      # gains are 1 + noise


def test_prompt_is_seeded():
    sh = S.CONFIGS["C1"]
    p = S.prompt_tokens(sh)
    assert p.shape == (16,) and p.dtype == np.int32
    assert (p == S.prompt_tokens(sh)).all() and p.min() >= 0 and p.max() < sh.vocab
