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


def close_elementwise(got, want, tol) -> bool:
    """The vector bar plus an element bar: rel-L2 <= tol AND no entry further than 3 * tol * rms(want) from the
    oracle's (a norm alone would let one entry of a long vector drift by a large multiple of the rms).
    Raises with the measured numbers when a bar is missed; returns True otherwise."""
    want = np.asarray(want, dtype=np.float64).ravel()
    got = np.asarray(got, dtype=np.float64).ravel()
    rms = float(np.sqrt(np.mean(want * want)))
    r, worst = rel_l2(got, want), float(np.abs(got - want).max())
    assert r <= tol, f"rel-L2 {r:.3e} > {tol:g}"
    assert worst <= 3 * tol * max(rms, 1e-300), f"max |delta| {worst:.3e} > 3 * {tol:g} * rms {rms:.3e} (rel-L2 {r:.3e})"
    return True


TINY = S.ModelShape("tiny-test", 2, 32, 4, 2, 8, 48, 37, 1e-5, 10000.0, "f32", 7, 2, 5, 3)


# ------------------------------------------------------------------ GPU harness
def tpi_config(shape: S.ModelShape, max_seq: int, max_prefill: int):
    import paper_2410_00531_b200 as P
    return P.make_config(n_layers=shape.n_layers, hidden=shape.hidden, n_heads=shape.n_heads,
                         n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, ffn=shape.ffn,
                         vocab=shape.vocab, max_seq=max_seq, max_prefill=max_prefill,
                         rms_eps=shape.rms_eps, rope_base=shape.rope_base, dtype=shape.dtype)


def gpu_session(shape: S.ModelShape, max_seq: int, max_prefill: int, n_shards: int | None = None,
                window: int = 0, alias_layers: int | None = None, **kw):
    import paper_2410_00531_b200 as P
    cfg = tpi_config(shape, max_seq, max_prefill)
    return P.Session(cfg, S.synth_fill(shape, alias_layers), n_shards or shape.n_shards, window, **kw)


def tol_for(shape: S.ModelShape) -> float:
    """Relative-L2 bar on hidden states and logits: 1e-5 for fp32 weights, 1e-2 for bf16."""
    return 1e-5 if shape.dtype == "f32" else 1e-2


def check_logits(gpu_logits, gpu_token, oracle_logits, tol) -> tuple[bool, bool]:
    """The token rule.  Returns (token_matches, step_was_ambiguous); raises on a violation.

    (1) rel-L2(logits) <= tol; (2) each of the oracle's top-8 logits is reproduced within
    e = 3 * tol * rms(oracle logits); (3) the GPU's greedy token equals the oracle's, or the
    oracle's top-2 gap is <= 2e and the GPU picked the runner-up."""
    o = np.asarray(oracle_logits, np.float64)
    g = np.asarray(gpu_logits, np.float64)
    assert rel_l2(g, o) <= tol, f"logits rel-L2 {rel_l2(g, o):.3e} > {tol}"
    e = 3 * tol * float(np.sqrt(np.mean(o * o)))
    top = np.argsort(-o, kind="stable")[:8]
    assert np.abs(g[top] - o[top]).max() <= e
    ambiguous = (o[top[0]] - o[top[1]]) <= 2 * e
    assert int(np.argmax(g)) == gpu_token, "device argmax disagrees with the logits it returned"
    if gpu_token == int(top[0]):
        return True, ambiguous
    assert ambiguous and gpu_token == int(top[1]), "token differs although the oracle's gap exceeds the tolerance"
    return False, True
