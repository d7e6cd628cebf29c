"""Glue between the seeded input generator and the CPU oracle (tests only)."""
from __future__ import annotations

import functools

import numpy as np

import tpi_synth as S
from oracle.llama_oracle import LlamaOracle, OracleConfig


def oracle_cfg(shape: S.ModelShape, kv_round: str | None = None) -> OracleConfig:
    if kv_round is None:
        kv_round = "bf16" if shape.dtype == "bf16" else "none"
    return OracleConfig(shape.n_layers, shape.hidden, shape.n_heads, shape.n_kv_heads,
                        shape.head_dim, shape.ffn, shape.vocab, shape.rms_eps,
                        shape.rope_base, kv_round)


def weight_fn(shape: S.ModelShape, cache: int = 64):
    """(layer, tensor id) -> float64 array of the stored (possibly bf16-rounded) values."""
    @functools.lru_cache(maxsize=cache)
    def w(layer: int, tid: int) -> np.ndarray:
        return S.as_f64(S.gen_tensor(shape, layer, tid))
    return w


def make_oracle(shape: S.ModelShape, kv_round: str | None = None, cache: int = 64) -> LlamaOracle:
    return LlamaOracle(oracle_cfg(shape, kv_round), weight_fn(shape, cache))


def rel_l2(got, want) -> float:
    got = np.asarray(got, dtype=np.float64).ravel()
    want = np.asarray(want, dtype=np.float64).ravel()
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


TINY = S.ModelShape("tiny-test", 2, 32, 4, 2, 8, 48, 37, 1e-5, 10000.0, "f32", 7, 2, 5, 3)
