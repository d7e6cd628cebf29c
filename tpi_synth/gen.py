"""Seeded synthetic inputs shared by the CPU oracle's tests and the GPU harness.

Nothing in this module belongs to the inference method: it only produces
reproducible pseudo-random weights, prompts, hidden states and KV contents with
the shapes and value scales of the paper's Llama-family workloads (Table 6 gives
layers / hidden / heads / kv heads; the paper runs pretrained checkpoints, which
do not exist here, so i.i.d. N(0, 0.02^2)-like weights stand in for them).

Weights come from a counter-based generator (see ``weight_values``): element
``idx`` of tensor ``uid`` depends on nothing but ``(seed, uid, idx)``, so a
70B-shaped model never has to be held in memory and the values do not depend on
the number of shards.  A compiled twin (``cgen.c``) produces the same bits
faster; ``tests/test_synth.py`` checks that the two agree exactly.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace

import numpy as np

# tensor ids (also the ids the C-ABI weight callback receives)
EMB, HEAD, FINAL_NORM = 0, 1, 2
ATTN_NORM, WQ, WK, WV, WO, FFN_NORM, WGATE, WUP, WDOWN = 3, 4, 5, 6, 7, 8, 9, 10, 11
TENSOR_NAMES = {
    EMB: "emb", HEAD: "head", FINAL_NORM: "final_norm", ATTN_NORM: "attn_norm",
    WQ: "wq", WK: "wk", WV: "wv", WO: "wo", FFN_NORM: "ffn_norm",
    WGATE: "wgate", WUP: "wup", WDOWN: "wdown",
}
NORM_IDS = (FINAL_NORM, ATTN_NORM, FFN_NORM)

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_IH_MEAN = 262140.0
_IH_STD = 53509.91992145008


@dataclass(frozen=True)
class ModelShape:
    """Shape of a Llama-style decoder (the paper's notation in comments)."""
    name: str
    n_layers: int      # L
    hidden: int        # h
    n_heads: int       # a
    n_kv_heads: int    # b
    head_dim: int      # d
    ffn: int           # s
    vocab: int         # v
    rms_eps: float
    rope_base: float
    dtype: str         # "f32" | "bf16": storage type of weights and KV cache
    seed: int
    n_shards: int      # N (default for this config)
    prompt_len: int
    decode_len: int

    def tensor_shape(self, tid: int) -> tuple[int, ...]:
        h, a, b, d, s, v = (self.hidden, self.n_heads, self.n_kv_heads,
                            self.head_dim, self.ffn, self.vocab)
        return {
            EMB: (v, h), HEAD: (v, h), FINAL_NORM: (h,), ATTN_NORM: (h,),
            WQ: (a * d, h), WK: (b * d, h), WV: (b * d, h), WO: (h, a * d),
            FFN_NORM: (h,), WGATE: (s, h), WUP: (s, h), WDOWN: (h, s),
        }[tid]

    def with_(self, **kw) -> "ModelShape":
        return replace(self, **kw)


def _cfg(i, name, L, h, a, b, d, s, v, base, dtype, N, T, G):
    return ModelShape(name, L, h, a, b, d, s, v, 1e-5, base, dtype, 20241000 + i, N, T, G)


# The five workloads of this build, in order (C1..C5).
CONFIGS = {
    "C1": _cfg(1, "tiny-f32", 2, 256, 4, 4, 64, 688, 1000, 10000.0, "f32", 2, 16, 8),
    "C2": _cfg(2, "llama2-7b-shape-bf16", 32, 4096, 32, 32, 128, 11008, 32000, 10000.0, "bf16", 4, 128, 128),
    "C3": _cfg(3, "llama3.1-8b-shape-bf16", 32, 4096, 32, 8, 128, 14336, 128256, 500000.0, "bf16", 8, 4096, 256),
    "C4": _cfg(4, "llama2-70b-shape-f32", 80, 8192, 64, 8, 128, 28672, 32000, 10000.0, "f32", 8, 512, 64),
    "C5": _cfg(5, "llama3.1-70b-shape-bf16", 80, 8192, 64, 8, 128, 28672, 128256, 500000.0, "bf16", 8, 512, 128),
}


# ---------------------------------------------------------------- generator
def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on uint64 arrays (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        x = x + np.uint64(0x9E3779B97F4A7C15)
        x = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        x = (x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return x ^ (x >> np.uint64(31))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even of finite float32 values to bf16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def weight_values_numpy(seed: int, uid: int, start: int, count: int,
                        offset: float, scale: float) -> np.ndarray:
    """Reference implementation of the counter-based generator (float32 out)."""
    key = _mix64(np.array([(seed ^ uid) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))[0]
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        r1 = _mix64(key + np.uint64(2) * idx)
        r2 = _mix64(key + np.uint64(2) * idx + np.uint64(1))
    s = np.zeros(count, dtype=np.int64)
    for k in range(4):
        sh = np.uint64(16 * k)
        s += ((r1 >> sh) & np.uint64(0xFFFF)).astype(np.int64)
        s += ((r2 >> sh) & np.uint64(0xFFFF)).astype(np.int64)
    z = (s.astype(np.float64) - _IH_MEAN) / _IH_STD
    return (offset + scale * z).astype(np.float32)


_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


def build_cgen(force: bool = False) -> str:
    """Compile cgen.c into tpi_synth/libtpisynth.so (gcc, OpenMP)."""
    src = os.path.join(_HERE, "cgen.c")
    out = os.path.join(_HERE, "libtpisynth.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O3", "-fopenmp", "-shared", "-fPIC", "-o", out, src])
    return out


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(build_cgen())
        lib.tpi_synth_fill.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                                       ctypes.c_uint64, ctypes.c_double, ctypes.c_double,
                                       ctypes.c_int, ctypes.c_void_p]
        lib.tpi_synth_fill.restype = None
        _LIB = lib
    return _LIB


def fill_raw(seed: int, uid: int, start: int, count: int, offset: float, scale: float,
             as_bf16: bool, dst_ptr: int) -> None:
    """Write ``count`` generated elements straight to a raw address (compiled path)."""
    _lib().tpi_synth_fill(seed, uid, start, count, offset, scale, int(as_bf16), dst_ptr)


def tensor_uid(layer: int, tid: int) -> int:
    return (layer if tid >= ATTN_NORM else 0) * 16 + tid


def offset_scale(tid: int) -> tuple[float, float]:
    """Matrices ~ N(0, 0.02^2); norm gains = 1 + N(0, 0.02^2) so the multiply is exercised."""
    return (1.0, 0.02) if tid in NORM_IDS else (0.0, 0.02)


def gen_tensor(shape: ModelShape, layer: int, tid: int, *, fast: bool = True) -> np.ndarray:
    """One UNSHARDED tensor, [out][in] row-major, in storage form:
    float32 array for "f32" models, uint16 bf16 bit patterns for "bf16" models."""
    dims = shape.tensor_shape(tid)
    n = int(np.prod(dims))
    off, sc = offset_scale(tid)
    uid = tensor_uid(layer, tid)
    bf = shape.dtype == "bf16"
    if fast:
        out = np.empty(n, dtype=np.uint16 if bf else np.float32)
        fill_raw(shape.seed, uid, 0, n, off, sc, bf, out.ctypes.data)
    else:
        out = weight_values_numpy(shape.seed, uid, 0, n, off, sc)
        if bf:
            out = f32_to_bf16_bits(out)
    return out.reshape(dims)


def as_f64(stored: np.ndarray) -> np.ndarray:
    """Exact upcast of a stored tensor (float32, or bf16 bits) to float64."""
    if stored.dtype == np.uint16:
        return bf16_bits_to_f32(stored).astype(np.float64)
    return stored.astype(np.float64)


def prompt_tokens(shape: ModelShape, n: int | None = None) -> np.ndarray:
    n = shape.prompt_len if n is None else n
    rng = np.random.Generator(np.random.PCG64(shape.seed + 1))
    return rng.integers(0, shape.vocab, n).astype(np.int32)


def hidden_state(seed: int, n: int, scale: float = 0.5) -> np.ndarray:
    """A float32 stand-in for a residual-stream vector (single-kernel tests)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return (rng.standard_normal(n) * scale).astype(np.float32)


def kv_contents(seed: int, shape_: tuple[int, ...], scale: float = 1.3) -> np.ndarray:
    """Float32 stand-in for cached keys/values: N(0, 1.3^2) matches 0.02*sqrt(h)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return (rng.standard_normal(shape_) * scale).astype(np.float32)


def synth_fill(shape: ModelShape, alias_layers: int | None = None):
    """Weight source for the GPU library's load callback:
    fill(tensor_id, layer, row0, n_rows, dst_address, n_bytes) writes rows of the unsharded tensor.

    alias_layers = K maps layer l to l mod K (declared stand-in when a model's
    distinct layers would not fit in host memory; the oracle side must alias too)."""
    esz = 2 if shape.dtype == "bf16" else 4

    def fill(tid: int, layer: int, row0: int, n_rows: int, dst: int, n_bytes: int) -> None:
        dims = shape.tensor_shape(tid)
        row_len = dims[-1]
        if alias_layers:
            layer = layer % alias_layers
        assert n_bytes == n_rows * row_len * esz
        off, sc = offset_scale(tid)
        fill_raw(shape.seed, tensor_uid(layer, tid), row0 * row_len, n_rows * row_len, off, sc,
                 shape.dtype == "bf16", dst)
    return fill
