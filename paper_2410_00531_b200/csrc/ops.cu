// Single-operation entry points (include/tpi_ops.h): thin wrappers that launch one kernel
// of the decoder path on caller-provided device buffers.
#include <cuda_runtime.h>
#include <math.h>

#include "../../include/tpi.h"
#include "../../include/tpi_ops.h"
#include "kernels.h"

using namespace tpi;

static int cu(cudaError_t e) { return e == cudaSuccess ? TPI_OK : TPI_ERR_CUDA; }
static bool bad_dtype(int dt) { return dt != TPI_F32 && dt != TPI_BF16; }
static int vec_of(int dt) { return dt == TPI_BF16 ? 8 : 4; }
static LaunchCtx ctx(void* stream) { return LaunchCtx{(cudaStream_t)stream, false, nullptr}; }

extern "C" int tpi_op_gemv_gateup(int dtype, const void* Wgu, const float* xhat, const float* gain, int h, int s,
                                  int n_shards, float* act, void* stream) {
  if (bad_dtype(dtype) || !Wgu || !xhat || !act || h < 1 || s < 1 || n_shards < 1) return TPI_ERR_INVALID_ARG;
  if (s % n_shards || h % vec_of(dtype) || h % 4) return TPI_ERR_SHAPE;
  return cu(launch_gemv_gateup(ctx(stream), dtype, Wgu, (size_t)2 * (s / n_shards) * h, NormIn{xhat, gain, nullptr, 0, 0.f}, h, n_shards, s, act));
}

extern "C" int tpi_op_gemv_qkv(int dtype, const void* Wqkv, const float* xhat, const float* gain, int h, int a, int b,
                               int d, int n_shards, int max_seq, const int32_t* pos, const void* rope, float* q_out,
                               void* kcache, void* vcache, void* stream) {
  if (bad_dtype(dtype) || !Wqkv || !xhat || !pos || !rope || !q_out || !kcache || !vcache) return TPI_ERR_INVALID_ARG;
  if (a % n_shards || b % n_shards || d % 2 || h % vec_of(dtype) || h % 4) return TPI_ERR_SHAPE;
  return cu(launch_gemv_qkv(ctx(stream), dtype, Wqkv, (size_t)(a + 2 * b) / n_shards * d * h, NormIn{xhat, gain, nullptr, 0, 0.f}, h, n_shards, a,
                            b, d, max_seq, pos, (const float2*)rope, q_out, kcache, vcache));
}

extern "C" int tpi_op_rope_table(float rope_base, int d, int max_seq, double* inv_freq_scratch, void* rope,
                                 void* stream) {
  if (!inv_freq_scratch || !rope || d < 2 || d % 2 || d > 512 || max_seq < 1) return TPI_ERR_INVALID_ARG;
  double invf[256];
  for (int i = 0; i < d / 2; ++i) invf[i] = pow((double)rope_base, -2.0 * i / d);
  cudaError_t e = cudaMemcpyAsync(inv_freq_scratch, invf, (size_t)(d / 2) * 8, cudaMemcpyHostToDevice, (cudaStream_t)stream);
  if (e != cudaSuccess) return TPI_ERR_CUDA;
  e = cudaStreamSynchronize((cudaStream_t)stream);  // invf lives on this stack frame
  if (e != cudaSuccess) return TPI_ERR_CUDA;
  return cu(launch_rope_table(ctx(stream), inv_freq_scratch, max_seq, d / 2, (float2*)rope));
}

extern "C" int tpi_op_gemv_partials(int dtype, const void* W, const float* x, int rows, int Ks, int n_shards,
                                    float* partials, void* stream) {
  if (bad_dtype(dtype) || !W || !x || !partials || rows < 1 || Ks < 1 || n_shards < 1) return TPI_ERR_INVALID_ARG;
  if (Ks % vec_of(dtype) || Ks % 4) return TPI_ERR_SHAPE;
  return cu(launch_gemv_partials(ctx(stream), dtype, W, (size_t)rows * Ks, x, rows, Ks, n_shards, partials));
}

extern "C" int tpi_op_reduce_residual(const float* partials, int n_shards, int h, float eps, float* x, float* xhat,
                                      void* stream) {
  if (!partials || !x || !xhat || n_shards < 1 || h < 1) return TPI_ERR_INVALID_ARG;
  return cu(launch_reduce_residual(ctx(stream), partials, n_shards, h, eps, x, xhat, nullptr, nullptr, 0));
}

extern "C" int tpi_op_rowshard_project(int dtype, const void* W, const float* x_in, int rows, int Ks, int n_shards,
                                       float eps, float* scratch, float* x, float* xhat, void* stream) {
  if (!scratch) return TPI_ERR_INVALID_ARG;
  const int rc = tpi_op_gemv_partials(dtype, W, x_in, rows, Ks, n_shards, scratch, stream);
  if (rc) return rc;
  return tpi_op_reduce_residual(scratch, n_shards, rows, eps, x, xhat, stream);
}

extern "C" int tpi_op_rowshard_fused_parts(int rows) { return rows < 1 ? TPI_ERR_INVALID_ARG : rowshard_fused_parts(rows); }

extern "C" int tpi_op_rowshard_fused(int dtype, const void* W, const float* x_in, int rows, int Ks, int n_shards,
                                     float* x, float* ss_part, void* stream) {
  if (bad_dtype(dtype) || !W || !x_in || !x || !ss_part || rows < 1 || Ks < 1 || n_shards < 1) return TPI_ERR_INVALID_ARG;
  if (Ks % vec_of(dtype) || Ks % 4 || !rowshard_fused_supported(Ks, n_shards)) return TPI_ERR_SHAPE;
  return cu(launch_gemv_rowshard_fused(ctx(stream), dtype, W, (size_t)rows * Ks, x_in, rows, Ks, n_shards, x, ss_part, nullptr));
}

extern "C" size_t tpi_op_attention_scratch_floats(int a, int b, int d, int nsplit) {
  if (a < 1 || b < 1 || d < 1 || nsplit < 1) return 0;
  return decode_attention_scratch_floats(a, b, d, nsplit);
}

extern "C" int tpi_op_decode_attention(int dtype, const float* q, const void* kcache, const void* vcache,
                                       const int32_t* pos, int a, int b, int d, int max_seq, int nsplit, float* scratch,
                                       uint32_t* tickets, float* o, void* stream) {
  if (bad_dtype(dtype) || !q || !kcache || !vcache || !pos || !scratch || !tickets || !o || nsplit < 1)
    return TPI_ERR_INVALID_ARG;
  if (a % b) return TPI_ERR_SHAPE;
  const cudaError_t e = launch_decode_attention(ctx(stream), dtype, q, kcache, vcache, pos, a, b, d, max_seq, nsplit,
                                                scratch, tickets, o);
  return e == cudaErrorInvalidValue ? TPI_ERR_SHAPE : cu(e);
}

extern "C" int tpi_op_head_blocks(int vocab) { return vocab < 1 ? TPI_ERR_INVALID_ARG : head_argmax_blocks(vocab); }

extern "C" int tpi_op_head_argmax(int dtype, const void* Whead, const float* xhat, const float* gain, int h, int vocab,
                                  float* logits, float* amax_val, int32_t* amax_idx, uint32_t* ticket,
                                  int32_t* token_out, void* stream) {
  if (bad_dtype(dtype) || !Whead || !xhat || !logits || !amax_val || !amax_idx || !ticket || !token_out)
    return TPI_ERR_INVALID_ARG;
  if (h % vec_of(dtype) || h % 4) return TPI_ERR_SHAPE;
  // the kernel writes tok_hist[*pos + 1]; token_out[0] serves as a zero position, token_out[1] gets the id
  if (cudaMemsetAsync(token_out, 0, 4, (cudaStream_t)stream) != cudaSuccess) return TPI_ERR_CUDA;
  return cu(launch_head_argmax(ctx(stream), dtype, Whead, NormIn{xhat, gain, nullptr, 0, 0.f}, h, vocab, logits, amax_val, amax_idx, ticket,
                               token_out, token_out, 0));
}

extern "C" int tpi_op_gemm(int dtype, const float* X, long long x_bs, int ldx, const void* W, long long w_bs, float* Y,
                           long long y_bs, int ldy, int T, int n_out, int K, int n_batch, void* stream) {
  if (bad_dtype(dtype) || !X || !W || !Y || T < 1 || n_out < 1 || K < 1 || n_batch < 1) return TPI_ERR_INVALID_ARG;
  if (K % 4 || ldx % 4 || x_bs % 4 || w_bs % 4) return TPI_ERR_SHAPE;
  return cu(launch_gemm_simt(ctx(stream), dtype, X, x_bs, ldx, W, w_bs, Y, y_bs, ldy, T, n_out, K, n_batch));
}

extern "C" int tpi_op_gemm_bf16(const void* A, const void* A_lo, int lda, int a_col_batch, const void* W, int w_row_batch, float* Y,
                                long long y_bs, int ldy, int T, int n_out, int K, int n_batch, int32_t* err_word,
                                void* stream) {
  if (!A || !W || !Y || !err_word || T < 1 || n_out < 1 || K < 1 || n_batch < 1) return TPI_ERR_INVALID_ARG;
  if (!gemm_tc_supported(K, lda, ldy) || a_col_batch % 8) return TPI_ERR_SHAPE;
  const cudaError_t e = launch_gemm_tc(ctx(stream), A, A_lo, lda, a_col_batch, W, w_row_batch, Y, y_bs, ldy, T, n_out, K,
                                       n_batch, err_word, true);
  return e == cudaErrorInvalidValue ? TPI_ERR_SHAPE : cu(e);
}

extern "C" int tpi_op_gemm_bf16_starved(const void* A, int lda, const void* W, float* Y, int ldy, int T, int n_out, int K,
                                        int wait_polls, int32_t* err_word, void* stream) {
  if (!A || !W || !Y || !err_word || T < 1 || n_out < 1 || K < 1 || wait_polls < 1 || wait_polls > 65536) return TPI_ERR_INVALID_ARG;
  if (!gemm_tc_supported(K, lda, ldy)) return TPI_ERR_SHAPE;
  const cudaError_t e = launch_gemm_tc_starved(ctx(stream), A, lda, W, Y, ldy, T, n_out, K, err_word, wait_polls);
  return e == cudaErrorInvalidValue ? TPI_ERR_SHAPE : cu(e);
}

extern "C" int tpi_op_gemm_bf16_swiglu(const void* A, const void* A_lo, int lda, const void* Wgu, void* ACT, int split_out, int T,
                                       int s, int K, int32_t* err_word, void* stream) {
  if (!A || !Wgu || !ACT || !err_word || T < 1 || s < 1 || K < 1) return TPI_ERR_INVALID_ARG;
  if (!gemm_tc_swiglu_supported(K, lda, s)) return TPI_ERR_SHAPE;
  const cudaError_t e = launch_gemm_tc_swiglu(ctx(stream), A, A_lo, lda, Wgu, ACT, split_out ? 2 : 1, T, s, K, err_word);
  return e == cudaErrorInvalidValue ? TPI_ERR_SHAPE : cu(e);
}

extern "C" int tpi_op_gemm_bf16_rowsum(const void* A, const void* A_lo, int lda, int a_col_batch, const void* W, int w_row_batch,
                                       float* X, int ldx, int T, int n_out, int K, int n_shards, int32_t* err_word, void* stream) {
  if (!A || !A_lo || !W || !X || !err_word || T < 1 || n_out < 1 || K < 1 || n_shards < 1) return TPI_ERR_INVALID_ARG;
  if (!gemm_tc_rowsum_supported(T, K, lda, n_out, ldx)) return TPI_ERR_SHAPE;
  const cudaError_t e = launch_gemm_tc_rowsum(ctx(stream), A, A_lo, lda, a_col_batch, W, w_row_batch, X, ldx, T, n_out, K, n_shards,
                                              err_word);
  return e == cudaErrorInvalidValue ? TPI_ERR_SHAPE : cu(e);
}

extern "C" int tpi_op_reduce_residual_norm_rows(const float* partials, int n_shards, int T, int h, float* X, const float* gain,
                                                float rms_eps, float* Xn, void* stream) {
  if (!partials || !X || !gain || !Xn || n_shards < 1 || T < 1 || h < 1) return TPI_ERR_INVALID_ARG;
  return cu(launch_reduce_residual_norm_rows(ctx(stream), partials, n_shards, T, h, X, nullptr, gain, rms_eps, Xn, 0));
}

extern "C" int tpi_op_prefill_attention(int dtype, const float* Q, const void* kcache, const void* vcache, int T,
                                        int pos0, int a, int b, int d, int max_seq, float* O, void* stream) {
  if (bad_dtype(dtype) || !Q || !kcache || !vcache || !O || T < 1 || pos0 < 0) return TPI_ERR_INVALID_ARG;
  if (a % b) return TPI_ERR_SHAPE;
  const cudaError_t e = prefill_attention_tc_supported(dtype, d, T)
                            ? launch_prefill_attention_tc(ctx(stream), Q, kcache, vcache, T, pos0, a, b, max_seq, O, 0, nullptr)
                        : prefill_attention_mma_supported(dtype, d)
                            ? launch_prefill_attention_mma(ctx(stream), Q, kcache, vcache, T, pos0, a, b, d, max_seq, O, 0)
                            : launch_prefill_attention(ctx(stream), dtype, Q, kcache, vcache, T, pos0, a, b, d, max_seq, O, 0);
  return e == cudaErrorInvalidValue ? TPI_ERR_SHAPE : cu(e);
}

// Internal hook (not part of the public interface): hands the decode kernels a device buffer of
// layout[0] * layout[1] * layout[2] 64-bit words for their timeline stamps (NULL switches it off again).
// Returns 1, or 0 when the library was built without -DTPI_TIMELINE (the kernels then carry no stamps).
extern "C" int tpi_internal_timeline(void* dev_buf, int* layout) {
  if (layout) { layout[0] = TL_KERNELS; layout[1] = TL_CTAS; layout[2] = TL_SLOTS; layout[3] = TL_WARP0; }
#ifdef TPI_TIMELINE
  set_timeline_decode(dev_buf);
  set_timeline_attn(dev_buf);
  return 1;
#else
  (void)dev_buf;
  return 0;
#endif
}

// Internal tuning hook (not part of the public interface): see kernels.h set_tuning.
extern "C" void tpi_internal_tune(int key, int value) { set_tuning(key, value); }
