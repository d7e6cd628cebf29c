"""CPU fp64 oracle for the TPI-LLM decoder step.  TEST INFRASTRUCTURE ONLY.

This is the plain, slow, obviously-correct statement of what the GPU library
must compute.  Only tests, the smoke check and the benchmark's CPU-baseline leg
may import it; the product never does, and this file imports nothing from the
product (no shared kernels, tables, helpers or post-processing).

What it computes, following the paper:

* Sec. 3.1 Step 2: the master turns a token into an embedding row, H^0.
* Sec. 3.1 Step 3, Eq. 1: every device normalises the hidden state, projects
  it with ITS heads' slices of W_Q, W_K, W_V, attends over its own KV cache,
  and the per-device results are summed by an allreduce and added to the
  shortcut.  (Eq. 1 as printed omits the output projection; Table 5's
  attention-block parameter count 2(a+b)h^2 p/a + h only adds up with a
  row-sliced W_O applied before the allreduce, which is the reading used.)
* Eq. 2: the FFN block with column-sliced gate/up, row-sliced down, allreduce
  and shortcut.
* Step 4 / Algorithm 1: final sum, norm, task head, next token (greedy).

Because Eq. 1-2 only re-associate a sum, the result equals the unsharded
Llama forward; ``layer_unsharded`` is that definition written out and
``layer_sharded`` is the paper's per-device form (the meaning of "N shards"),
kept as a second path and tied to the first by an invariant test.

Readings where the paper is silent: "norm" = RMSNorm (eps inside the root, gain
applied after); positions enter through rotary embeddings with the
rotate-half pairing (i, i + d/2), angle p * base^(-2i/d), keys cached AFTER
rotation; sigma = SiLU; greedy argmax with ties to the lowest index; the KV
cache may be stored in bf16 (``kv_round="bf16"``), rounding to nearest even at
the moment of the store.

All arithmetic is float64.  Parity pinned: see tests/test_oracle_*.py.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable

import numpy as np

# tensor ids of the weight provider (the same numbering the input generator uses)
EMB, HEAD, FINAL_NORM = 0, 1, 2
ATTN_NORM, WQ, WK, WV, WO, FFN_NORM, WGATE, WUP, WDOWN = 3, 4, 5, 6, 7, 8, 9, 10, 11


@dataclass(frozen=True)
class OracleConfig:
    n_layers: int
    hidden: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0
    kv_round: str = "none"      # "none" | "bf16": storage rounding of cached K, V


# --------------------------------------------------------------- primitives
def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * g over the last axis ("norm" in Sec. 3.1 Step 3)."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope_angles(pos: np.ndarray, head_dim: int, base: float) -> np.ndarray:
    """theta[p, i] = p * base^(-2i/d), i in [0, d/2)."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = base ** (-2.0 * i / head_dim)
    return np.asarray(pos, dtype=np.float64)[..., None] * inv_freq


def rope(u: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotate head vectors u[..., T, n_heads, d] at positions pos[T].

    Pair (i, i + d/2) is rotated by theta[p, i]:
      u_i'       = u_i cos - u_{i+d/2} sin
      u_{i+d/2}' = u_{i+d/2} cos + u_i sin
    """
    d = u.shape[-1]
    th = rope_angles(pos, d, base)[:, None, :]       # [T, 1, d/2]
    c, s = np.cos(th), np.sin(th)
    lo, hi = u[..., : d // 2], u[..., d // 2:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def softmax(sc: np.ndarray) -> np.ndarray:
    e = np.exp(sc - np.max(sc, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def silu(t: np.ndarray) -> np.ndarray:
    return t / (1.0 + np.exp(-t))


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64 values to the bf16 grid (returned as float64)."""
    u = x.astype(np.float32).view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(np.float64)


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, q_pos: np.ndarray) -> np.ndarray:
    """Scaled dot-product attention of Eq. 1 with grouped heads and a causal mask.

    q [T, a, d] (rotated queries at absolute positions q_pos[T]);
    K, V [b, n, d] cached keys/values for positions 0..n-1;
    query head j reads kv head j // (a/b) and sees positions t <= q_pos.
    Returns o [T, a, d].
    """
    T, a, d = q.shape
    b, n, _ = K.shape
    grp = a // b
    o = np.empty_like(q)
    t_idx = np.arange(n)
    for j in range(a):
        g = j // grp
        sc = (q[:, j, :] @ K[g].T) / np.sqrt(d)                   # [T, n]
        sc = np.where(t_idx[None, :] <= np.asarray(q_pos)[:, None], sc, -np.inf)
        o[:, j, :] = softmax(sc) @ V[g]
    return o


# -------------------------------------------------------------------- model
WeightFn = Callable[[int, int], np.ndarray]   # (layer, tensor id) -> float64 array [out][in]


@dataclass
class KVCache:
    """D^k of Algorithms 1-2: per layer, keys/values by kv head and position."""
    K: list = field(default_factory=list)    # per layer: [b, n, d]
    V: list = field(default_factory=list)

    @property
    def length(self) -> int:
        return 0 if not self.K else self.K[0].shape[1]


class LlamaOracle:
    def __init__(self, cfg: OracleConfig, weights: WeightFn):
        self.cfg = cfg
        self.w = weights
        self.cache = KVCache()
        self.taps: dict = {}     # (layer, "attn"|"ffn") -> H [T, h] of the last forward

    def reset(self) -> None:
        self.cache = KVCache()

    # -- attention block inputs shared by both forms
    def _qkv(self, l: int, xn: np.ndarray, pos: np.ndarray, heads=None, kv_heads=None):
        c = self.cfg
        d = c.head_dim
        Wq, Wk, Wv = self.w(l, WQ), self.w(l, WK), self.w(l, WV)
        if heads is not None:            # a device's own slices (Sec. 3.1 Step 3)
            Wq = Wq.reshape(c.n_heads, d, c.hidden)[heads].reshape(-1, c.hidden)
            Wk = Wk.reshape(c.n_kv_heads, d, c.hidden)[kv_heads].reshape(-1, c.hidden)
            Wv = Wv.reshape(c.n_kv_heads, d, c.hidden)[kv_heads].reshape(-1, c.hidden)
        T = xn.shape[0]
        q = (xn @ Wq.T).reshape(T, -1, d)
        k = (xn @ Wk.T).reshape(T, -1, d)
        v = (xn @ Wv.T).reshape(T, -1, d)
        q = rope(q, pos, c.rope_base)
        k = rope(k, pos, c.rope_base)
        if c.kv_round == "bf16":
            k, v = round_bf16(k), round_bf16(v)
        return q, k, v

    # -- one decoder layer, unsharded definition
    def layer_unsharded(self, l: int, x: np.ndarray, pos: np.ndarray, Kprev, Vprev):
        c = self.cfg
        xn = rmsnorm(x, self.w(l, ATTN_NORM), c.rms_eps)
        q, k, v = self._qkv(l, xn, pos)
        K = np.swapaxes(k, 0, 1) if Kprev is None else np.concatenate([Kprev, np.swapaxes(k, 0, 1)], axis=1)
        V = np.swapaxes(v, 0, 1) if Vprev is None else np.concatenate([Vprev, np.swapaxes(v, 0, 1)], axis=1)
        o = attention(q, K, V, pos).reshape(x.shape[0], -1)
        h_attn = o @ self.w(l, WO).T + x
        xn2 = rmsnorm(h_attn, self.w(l, FFN_NORM), c.rms_eps)
        act = silu(xn2 @ self.w(l, WGATE).T) * (xn2 @ self.w(l, WUP).T)
        h_ffn = act @ self.w(l, WDOWN).T + h_attn
        return h_attn, h_ffn, K, V

    # -- the same layer as N devices compute it (Eq. 1-2): per-device partials, rank-ordered sum
    def layer_sharded(self, l: int, x: np.ndarray, pos: np.ndarray, Kprev, Vprev, n_shards: int, partition=None):
        """Eq. 1-2 as N devices compute them.  ``partition`` = (kv heads per device, FFN columns per device)
        gives device i the proportion p_i of the heads and of the FFN columns (Sec. 3.1: stronger devices take
        more); None is the uniform p_i = 1/N.  A device's query heads are those of its kv heads' groups."""
        c = self.cfg
        a, b, d, s = c.n_heads, c.n_kv_heads, c.head_dim, c.ffn
        if partition is None:
            if a % n_shards or b % n_shards or s % n_shards:
                raise ValueError("N must divide heads, kv heads and FFN width")
            kv_cnt, ffn_cnt = [b // n_shards] * n_shards, [s // n_shards] * n_shards
        else:
            kv_cnt, ffn_cnt = [int(v) for v in partition[0]], [int(v) for v in partition[1]]
            if len(kv_cnt) != n_shards or len(ffn_cnt) != n_shards or sum(kv_cnt) != b or sum(ffn_cnt) != s \
                    or min(kv_cnt) < 1 or min(ffn_cnt) < 1:
                raise ValueError("a partition gives every device at least one kv head and one FFN column, all of them once")
        kv0 = np.concatenate([[0], np.cumsum(kv_cnt)])
        f0 = np.concatenate([[0], np.cumsum(ffn_cnt)])
        grp = a // b
        T = x.shape[0]
        xn = rmsnorm(x, self.w(l, ATTN_NORM), c.rms_eps)     # replicated norm on every device
        Wo = self.w(l, WO)
        partials, Ks, Vs = [], [], []
        for i in range(n_shards):
            heads = np.arange(kv0[i] * grp, kv0[i + 1] * grp)
            kvh = np.arange(kv0[i], kv0[i + 1])
            q, k, v = self._qkv(l, xn, pos, heads, kvh)
            Ki = np.swapaxes(k, 0, 1) if Kprev is None else np.concatenate([Kprev[kvh], np.swapaxes(k, 0, 1)], axis=1)
            Vi = np.swapaxes(v, 0, 1) if Vprev is None else np.concatenate([Vprev[kvh], np.swapaxes(v, 0, 1)], axis=1)
            o_i = attention(q, Ki, Vi, pos).reshape(T, -1)
            cols = np.arange(heads[0] * d, (heads[-1] + 1) * d)
            partials.append(o_i @ Wo[:, cols].T)
            Ks.append(Ki)
            Vs.append(Vi)
        red = partials[0]
        for p in partials[1:]:
            red = red + p                                     # star allreduce: master sums in rank order
        h_attn = red + x
        xn2 = rmsnorm(h_attn, self.w(l, FFN_NORM), c.rms_eps)
        Wg, Wu, Wd = self.w(l, WGATE), self.w(l, WUP), self.w(l, WDOWN)
        partials = []
        for i in range(n_shards):
            cols = np.arange(f0[i], f0[i + 1])
            act_i = silu(xn2 @ Wg[cols].T) * (xn2 @ Wu[cols].T)
            partials.append(act_i @ Wd[:, cols].T)
        red = partials[0]
        for p in partials[1:]:
            red = red + p
        h_ffn = red + h_attn
        return h_attn, h_ffn, np.concatenate(Ks, axis=0), np.concatenate(Vs, axis=0)

    # -- Algorithm 1's loop body for T new positions
    def forward(self, tokens, n_shards: int | None = None, all_logits: bool = False, partition=None) -> np.ndarray:
        """Feed ``tokens`` at positions cache.length .. cache.length+T-1.

        Returns logits of the last position [v] (or of every position [T, v])."""
        c = self.cfg
        tokens = np.asarray(tokens, dtype=np.int64).reshape(-1)
        T = tokens.shape[0]
        p0 = self.cache.length
        pos = np.arange(p0, p0 + T)
        x = self.w(0, EMB)[tokens]                            # H^0 = x W_emb
        first = not self.cache.K
        for l in range(c.n_layers):
            Kp = None if first else self.cache.K[l]
            Vp = None if first else self.cache.V[l]
            if n_shards is None:
                h_attn, h_ffn, K, V = self.layer_unsharded(l, x, pos, Kp, Vp)
            else:
                h_attn, h_ffn, K, V = self.layer_sharded(l, x, pos, Kp, Vp, n_shards, partition)
            if first:
                self.cache.K.append(K)
                self.cache.V.append(V)
            else:
                self.cache.K[l], self.cache.V[l] = K, V
            self.taps[(l, "attn")], self.taps[(l, "ffn")] = h_attn, h_ffn
            x = h_ffn
        xn = rmsnorm(x if all_logits else x[-1:], self.w(0, FINAL_NORM), c.rms_eps)
        logits = xn @ self.w(0, HEAD).T
        return logits if all_logits else logits[0]

    def greedy(self, prompt, n_new: int, n_shards: int | None = None):
        """Prefill the prompt, then decode greedily.  Returns (tokens [n_new], logits [n_new, v])."""
        self.reset()
        out, lg = [], []
        logits = self.forward(prompt, n_shards)
        for _ in range(n_new):
            tok = int(np.argmax(logits))                      # first maximum = lowest index on ties
            out.append(tok)
            lg.append(logits)
            if len(out) == n_new:
                break
            logits = self.forward([tok], n_shards)
        return np.array(out, dtype=np.int32), np.stack(lg)
