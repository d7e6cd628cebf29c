"""ctypes binding of the single-operation entry points (include/tpi_ops.h).

Arguments are raw device addresses (ints, e.g. ``tensor.data_ptr()``) and sizes;
nothing is computed here."""
from __future__ import annotations

import ctypes as C

from .binding import TPI_BF16, TPI_F32, _check, lib  # noqa: F401

_P, _I, _F, _LL = C.c_void_p, C.c_int, C.c_float, C.c_longlong

OPS_SYMBOLS = {
    "tpi_op_gemv_gateup": (_I, [_I, _P, _P, _P, _I, _I, _I, _P, _P]),
    "tpi_op_gemv_qkv": (_I, [_I, _P, _P, _P, _I, _I, _I, _I, _I, _I, _P, _P, _P, _P, _P, _P]),
    "tpi_op_rope_table": (_I, [_F, _I, _I, _P, _P, _P]),
    "tpi_op_gemv_partials": (_I, [_I, _P, _P, _I, _I, _I, _P, _P]),
    "tpi_op_reduce_residual": (_I, [_P, _I, _I, _F, _P, _P, _P]),
    "tpi_op_rowshard_project": (_I, [_I, _P, _P, _I, _I, _I, _F, _P, _P, _P, _P]),
    "tpi_op_rowshard_fused_parts": (_I, [_I]),
    "tpi_op_rowshard_fused": (_I, [_I, _P, _P, _I, _I, _I, _P, _P, _P]),
    "tpi_op_static_scratch_floats": (C.c_size_t, []),
    "tpi_op_rowshard_project_static": (_I, [_I, _P, _P, _I, _I, _I, _F, _P, _P, _P]),
    "tpi_op_attention_scratch_floats": (C.c_size_t, [_I, _I, _I, _I]),
    "tpi_op_decode_attention": (_I, [_I, _P, _P, _P, _P, _I, _I, _I, _I, _I, _P, _P, _P, _P]),
    "tpi_op_head_blocks": (_I, [_I]),
    "tpi_op_head_argmax": (_I, [_I, _P, _P, _P, _I, _I, _P, _P, _P, _P, _P, _P]),
    "tpi_op_gemm": (_I, [_I, _P, _LL, _I, _P, _LL, _P, _LL, _I, _I, _I, _I, _I, _P]),
    "tpi_op_gemm_bf16": (_I, [_P, _P, _I, _I, _P, _I, _P, _LL, _I, _I, _I, _I, _I, _P, _P]),
    "tpi_op_gemm_bf16_starved": (_I, [_P, _I, _P, _P, _I, _I, _I, _I, _I, _P, _P]),
    "tpi_op_prefill_attention": (_I, [_I, _P, _P, _P, _I, _I, _I, _I, _I, _I, _P, _P]),
    "tpi_op_gemm_bf16_swiglu": (_I, [_P, _P, _I, _P, _P, _I, _I, _I, _I, _P, _P]),
    "tpi_op_gemm_bf16_rowsum": (_I, [_P, _P, _I, _I, _P, _I, _P, _I, _I, _I, _I, _I, _P, _P]),
    "tpi_op_reduce_residual_norm_rows": (_I, [_P, _I, _I, _I, _P, _P, _F, _P, _P]),
}
_BOUND = False


def _ops():
    global _BOUND
    L = lib()
    if not _BOUND:
        for name, (res, args) in OPS_SYMBOLS.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _BOUND = True
    return L


def gemv_gateup(dtype, Wgu, xhat, gain, h, s, n_shards, act, stream=None):
    _check(_ops().tpi_op_gemv_gateup(dtype, Wgu, xhat, gain, h, s, n_shards, act, stream))


def gemv_qkv(dtype, Wqkv, xhat, gain, h, a, b, d, n_shards, max_seq, pos, rope, q_out, kcache, vcache, stream=None):
    _check(_ops().tpi_op_gemv_qkv(dtype, Wqkv, xhat, gain, h, a, b, d, n_shards, max_seq, pos, rope, q_out,
                                  kcache, vcache, stream))


def rope_table(rope_base, d, max_seq, inv_freq_scratch, rope, stream=None):
    _check(_ops().tpi_op_rope_table(rope_base, d, max_seq, inv_freq_scratch, rope, stream))


def gemv_partials(dtype, W, x, rows, Ks, n_shards, partials, stream=None):
    _check(_ops().tpi_op_gemv_partials(dtype, W, x, rows, Ks, n_shards, partials, stream))


def reduce_residual(partials, n_shards, h, eps, x, xhat, stream=None):
    _check(_ops().tpi_op_reduce_residual(partials, n_shards, h, eps, x, xhat, stream))


def rowshard_project(dtype, W, x_in, rows, Ks, n_shards, eps, scratch, x, xhat, stream=None):
    _check(_ops().tpi_op_rowshard_project(dtype, W, x_in, rows, Ks, n_shards, eps, scratch, x, xhat, stream))


def rowshard_fused_parts(rows) -> int:
    return _check(_ops().tpi_op_rowshard_fused_parts(rows))


def rowshard_fused(dtype, W, x_in, rows, Ks, n_shards, x, ss_part, stream=None):
    _check(_ops().tpi_op_rowshard_fused(dtype, W, x_in, rows, Ks, n_shards, x, ss_part, stream))


def static_scratch_floats() -> int:
    return int(_ops().tpi_op_static_scratch_floats())


def rowshard_project_static(dtype, W, x_in, rows, Ks, n_shards, eps, x, xhat, stream=None):
    """Like rowshard_project, but the partial sums live in the library's built-in array, so the
    call needs no scratch buffer (for callers that cannot allocate device memory)."""
    _check(_ops().tpi_op_rowshard_project_static(dtype, W, x_in, rows, Ks, n_shards, eps, x, xhat, stream))


def attention_scratch_floats(a, b, d, nsplit) -> int:
    return int(_ops().tpi_op_attention_scratch_floats(a, b, d, nsplit))


def decode_attention(dtype, q, kcache, vcache, pos, a, b, d, max_seq, nsplit, scratch, tickets, o, stream=None):
    _check(_ops().tpi_op_decode_attention(dtype, q, kcache, vcache, pos, a, b, d, max_seq, nsplit, scratch,
                                          tickets, o, stream))


def head_blocks(vocab) -> int:
    return _check(_ops().tpi_op_head_blocks(vocab))


def head_argmax(dtype, Whead, xhat, gain, h, vocab, logits, amax_val, amax_idx, ticket, token_out, stream=None):
    _check(_ops().tpi_op_head_argmax(dtype, Whead, xhat, gain, h, vocab, logits, amax_val, amax_idx, ticket,
                                     token_out, stream))


def gemm(dtype, X, x_bs, ldx, W, w_bs, Y, y_bs, ldy, T, n_out, K, n_batch, stream=None):
    _check(_ops().tpi_op_gemm(dtype, X, x_bs, ldx, W, w_bs, Y, y_bs, ldy, T, n_out, K, n_batch, stream))


def gemm_bf16(A, lda, a_col_batch, W, w_row_batch, Y, y_bs, ldy, T, n_out, K, n_batch, err_word, stream=None, A_lo=None):
    _check(_ops().tpi_op_gemm_bf16(A, A_lo, lda, a_col_batch, W, w_row_batch, Y, y_bs, ldy, T, n_out, K, n_batch, err_word, stream))


def gemm_bf16_starved(A, lda, W, Y, ldy, T, n_out, K, wait_polls, err_word, stream=None):
    _check(_ops().tpi_op_gemm_bf16_starved(A, lda, W, Y, ldy, T, n_out, K, wait_polls, err_word, stream))


def gemm_bf16_swiglu(A, lda, Wgu, ACT, split_out, T, s, K, err_word, stream=None, A_lo=None):
    _check(_ops().tpi_op_gemm_bf16_swiglu(A, A_lo, lda, Wgu, ACT, int(split_out), T, s, K, err_word, stream))


def gemm_bf16_rowsum(A, A_lo, lda, a_col_batch, W, w_row_batch, X, ldx, T, n_out, K, n_shards, err_word, stream=None):
    _check(_ops().tpi_op_gemm_bf16_rowsum(A, A_lo, lda, a_col_batch, W, w_row_batch, X, ldx, T, n_out, K, n_shards, err_word, stream))


def reduce_residual_norm_rows(partials, n_shards, T, h, X, gain, rms_eps, Xn, stream=None):
    _check(_ops().tpi_op_reduce_residual_norm_rows(partials, n_shards, T, h, X, gain, rms_eps, Xn, stream))


def prefill_attention(dtype, Q, kcache, vcache, T, pos0, a, b, d, max_seq, O, stream=None):
    _check(_ops().tpi_op_prefill_attention(dtype, Q, kcache, vcache, T, pos0, a, b, d, max_seq, O, stream))
