"""Scalar-loop restatement of the decoder forward.  TEST INFRASTRUCTURE ONLY.

Pure Python floats and ``math`` only (no numpy vector ops), written straight
from the definitions in Sec. 3.1 (Eq. 1-2, Step 4) so that an indexing, sign or
transposition mistake in the vectorised oracle shows up as a disagreement on
tiny models.  Exponentially slower than the oracle; use hidden sizes <= 32.
"""
from __future__ import annotations

import math


def _rmsnorm(x, g, eps):
    ms = sum(t * t for t in x) / len(x)
    r = 1.0 / math.sqrt(ms + eps)
    return [x[i] * r * g[i] for i in range(len(x))]


def _matvec(W, x):
    """y[o] = sum_i W[o][i] x[i]  (weights are [out][in])."""
    return [sum(W[o][i] * x[i] for i in range(len(x))) for o in range(len(W))]


def _rope_head(u, p, base):
    d = len(u)
    out = [0.0] * d
    for i in range(d // 2):
        th = p * base ** (-2.0 * i / d)
        c, s = math.cos(th), math.sin(th)
        out[i] = u[i] * c - u[i + d // 2] * s
        out[i + d // 2] = u[i + d // 2] * c + u[i] * s
    return out


def forward_tokens(cfg, W, tokens):
    """Run the whole prompt position by position; returns logits of every position.

    cfg: dict with n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab,
    rms_eps, rope_base.  W(layer, tensor_id) -> nested lists [out][in]
    (tensor ids: 0 emb, 1 head, 2 final norm, 3 attn norm, 4 q, 5 k, 6 v, 7 o,
    8 ffn norm, 9 gate, 10 up, 11 down).
    """
    L, a, b, d = cfg["n_layers"], cfg["n_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    eps, base = cfg["rms_eps"], cfg["rope_base"]
    Kc = [[[] for _ in range(b)] for _ in range(L)]      # Kc[l][g][t] -> list of d
    Vc = [[[] for _ in range(b)] for _ in range(L)]
    all_logits = []
    for p, z in enumerate(tokens):
        x = list(W(0, 0)[z])
        for l in range(L):
            xn = _rmsnorm(x, W(l, 3), eps)
            q, k, v = _matvec(W(l, 4), xn), _matvec(W(l, 5), xn), _matvec(W(l, 6), xn)
            for g in range(b):
                Kc[l][g].append(_rope_head(k[g * d:(g + 1) * d], p, base))
                Vc[l][g].append(v[g * d:(g + 1) * d])
            o = []
            for j in range(a):
                g = j // (a // b)
                qj = _rope_head(q[j * d:(j + 1) * d], p, base)
                sc = [sum(qj[i] * Kc[l][g][t][i] for i in range(d)) / math.sqrt(d) for t in range(p + 1)]
                m = max(sc)
                e = [math.exp(t - m) for t in sc]
                tot = sum(e)
                o += [sum(e[t] / tot * Vc[l][g][t][i] for t in range(p + 1)) for i in range(d)]
            att = _matvec(W(l, 7), o)
            h_attn = [att[i] + x[i] for i in range(len(x))]
            xn = _rmsnorm(h_attn, W(l, 8), eps)
            gate, up = _matvec(W(l, 9), xn), _matvec(W(l, 10), xn)
            act = [gate[i] / (1.0 + math.exp(-gate[i])) * up[i] for i in range(len(gate))]
            dn = _matvec(W(l, 11), act)
            x = [dn[i] + h_attn[i] for i in range(len(x))]
        all_logits.append(_matvec(W(0, 1), _rmsnorm(x, W(0, 2), eps)))
    return all_logits
