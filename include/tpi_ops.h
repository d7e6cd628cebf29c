/* tpi_ops.h - single-operation entry points of libtpi.so.
 *
 * Each call launches one step of the decoder path (the same kernels the model
 * driver in tpi.h strings together) on caller-provided DEVICE buffers, so that a
 * step can be checked or timed alone at any shape.  All pointers are DEVICE
 * pointers unless they say HOST; `stream` is a cudaStream_t (NULL = default
 * stream).  Calls are asynchronous: they return after the launch.  dtype is a
 * tpi_dtype (storage type of weights / KV); activations are fp32.
 * Return value: 0 or a negative tpi_status (see tpi.h).
 */
#ifndef TPI_OPS_H
#define TPI_OPS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Column-sharded gate/up projection with SwiGLU (Eq. 2, inner part):
 *   act[i*s/N + j] = SiLU(W_gate^i[j,:] . xn) * (W_up^i[j,:] . xn),  xn = xhat * gain.
 * Wgu: per shard i a [2 s/N][h] matrix whose rows alternate gate_j, up_j; shards
 * are contiguous.  xhat, gain: float[h]; act: float[s]. */
int tpi_op_gemv_gateup(int dtype, const void *Wgu, const float *xhat, const float *gain, int h, int s,
                       int n_shards, float *act, void *stream);

/* Column-sharded QKV projection + rotary embedding + KV append (Eq. 1 inputs,
 * Algorithm 1 "store (K, V) in KVCache").  Wqkv: per shard i rows
 * [W_Q^i ; W_K^i ; W_V^i] x h.  pos: int32* current position p.  rope:
 * float2[max_seq][d/2] = (cos, sin)(p * base^(-2i/d)).  q_out: float[a d]
 * (rotated).  kcache/vcache: [b][max_seq][d] in dtype; row p is written. */
int tpi_op_gemv_qkv(int dtype, const void *Wqkv, const float *xhat, const float *gain, int h, int a, int b,
                    int d, int n_shards, int max_seq, const int32_t *pos, const void *rope, float *q_out,
                    void *kcache, void *vcache, void *stream);

/* cos/sin table for tpi_op_gemv_qkv: rope[p][i] for p < max_seq, i < d/2 (fp64 inside).
 * inv_freq_scratch: double[d/2] device scratch the call fills from rope_base. */
int tpi_op_rope_table(float rope_base, int d, int max_seq, double *inv_freq_scratch, void *rope, void *stream);

/* Row-sharded projection (W_O of Eq. 1 / W_down of Eq. 2): one partial sum per shard,
 *   partials[i][r] = W^i[r,:] . x[i*Ks : (i+1)*Ks],  W: [N][rows][Ks] contiguous. */
int tpi_op_gemv_partials(int dtype, const void *W, const float *x, int rows, int Ks, int n_shards,
                         float *partials, void *stream);

/* The star allreduce of Sec. 3.2 emulated on one GPU, plus the shortcut of Eq. 1-2
 * and the next norm's statistics:  x <- ((P_0 + P_1) + ... + P_{N-1}) + x;
 * xhat <- x * rsqrt(mean(x^2) + eps).  partials: float[N][h]; x, xhat: float[h]. */
int tpi_op_reduce_residual(const float *partials, int n_shards, int h, float eps, float *x, float *xhat,
                           void *stream);

/* Both of the above back to back: x <- sum_i W^i x_i + x, xhat as above.
 * scratch: float[n_shards * rows] DEVICE memory owned by the caller (the N partials). */
int tpi_op_rowshard_project(int dtype, const void *W, const float *x_in, int rows, int Ks, int n_shards,
                            float eps, float *scratch, float *x, float *xhat, void *stream);

/* The same step as the model driver runs it: the N per-shard partial sums are formed in
 * registers (shard by shard, rank order) and folded straight into the shortcut, so they never
 * pass through memory:  x[r] <- ((P_0[r] + P_1[r]) + ... + P_{N-1}[r]) + x[r].  Bit-identical
 * to tpi_op_rowshard_project.  ss_part: float[tpi_op_rowshard_fused_parts(rows)], receives each
 * CTA's sum of squares of its new x entries (the next RMSNorm's statistics; unused entries are
 * zeroed).  The whole x_in must fit in shared memory: n_shards * Ks * 4 <= 200 KiB. */
int tpi_op_rowshard_fused_parts(int rows);
int tpi_op_rowshard_fused(int dtype, const void *W, const float *x_in, int rows, int Ks, int n_shards,
                          float *x, float *ss_part, void *stream);

/* Allocation-free variant of tpi_op_rowshard_project (the paper has no counterpart: it is
 * an addition for callers that cannot allocate device memory when they need this step,
 * such as code inside a memory-capped plug-in or a real-time loop where cudaMalloc is
 * off limits).  Same arguments minus `scratch`: the N partial sums live in an array built
 * into the library (tpi_op_static_scratch_floats() floats = 256 KiB, held on every GPU that
 * loads the library until the process exits).  Returns TPI_ERR_NOMEM, with a message in
 * tpi_last_error(), when n_shards * rows exceeds that size.  The call allocates nothing.
 * All calls on a GPU share the array and it keeps the previous call's contents (each call
 * overwrites all it reads, so nothing needs clearing); calls that overlap on the GPU race,
 * so issue them in one stream order.  The first call on each GPU looks up the array's
 * device address; make that call before any stream capture begins. */
size_t tpi_op_static_scratch_floats(void);
int tpi_op_rowshard_project_static(int dtype, const void *W, const float *x_in, int rows, int Ks,
                                   int n_shards, float eps, float *x, float *xhat, void *stream);

/* Split-K attention of one query position over cache positions 0..*pos (Eq. 1).
 * q: float[a d] rotated queries; kcache/vcache [b][max_seq][d]; o: float[a d].
 * scratch: float[tpi_op_attention_scratch_floats(...)]; tickets: uint32[b], zero on entry
 * (the kernel leaves them zero). */
size_t tpi_op_attention_scratch_floats(int a, int b, int d, int nsplit);
int tpi_op_decode_attention(int dtype, const float *q, const void *kcache, const void *vcache,
                            const int32_t *pos, int a, int b, int d, int max_seq, int nsplit, float *scratch,
                            uint32_t *tickets, float *o, void *stream);

/* Task head + greedy argmax (Step 4): logits = W_head . (xhat * gain); token =
 * lowest index of the maximum.  amax_val/amax_idx: scratch of tpi_op_head_blocks(vocab)
 * entries; ticket: uint32, zero on entry.  token_out: int32[2]; token_out[1] receives the id. */
int tpi_op_head_blocks(int vocab);
int tpi_op_head_argmax(int dtype, const void *Whead, const float *xhat, const float *gain, int h, int vocab,
                       float *logits, float *amax_val, int32_t *amax_idx, uint32_t *ticket,
                       int32_t *token_out, void *stream);

/* Prompt-pass projection: Y[b][t][o] = sum_k X[b][t][k] W[b][o][k] for n_batch independent
 * problems (batch = shard for the row-sharded projections), fp32 accumulate.
 * X: float, row stride ldx, batch stride x_bs; W: dtype, [n_out][K], batch stride w_bs elements;
 * Y: float, row stride ldy, batch stride y_bs. */
int tpi_op_gemm(int dtype, const float *X, long long x_bs, int ldx, const void *W, long long w_bs, float *Y,
                long long y_bs, int ldy, int T, int n_out, int K, int n_batch, void *stream);

/* The prompt-pass projection on the tensor cores (bf16 configurations): same contraction with bf16
 * activations, tcgen05.mma with an fp32 accumulator in tensor memory, operands staged by TMA.
 * A: bf16 [T][lda]; batch b reads K columns starting at column b * a_col_batch (a multiple of 8).
 * A_lo: NULL, or a second bf16 tensor like A holding bf16(x - A) so that A + A_lo carries ~16 mantissa
 * bits of the fp32 activations x (each k-block is then multiplied twice onto one accumulator).
 * W: bf16 [n_batch * w_row_batch][K], batch b uses rows [b * w_row_batch, b * w_row_batch + n_out).
 * Y: float, row stride ldy (multiple of 4), batch stride y_bs floats.  K must be a multiple of 64.
 * A single batch with A_lo, more than 128 positions and K > 512 is accumulated in chunks of 512 inputs (each
 * chunk in tensor memory, the chunks added in fp32 registers): the tensor core truncates its accumulator at every
 * step, and a long chain drifts by ~2^-26 of the sum per step (1.9e-5 of the result at K = 8192, 1.1e-6 in chunks).
 * err_word: int32 DEVICE word, zero on entry; the kernel's bounded waits write 3 there if one runs out. */
int tpi_op_gemm_bf16(const void *A, const void *A_lo, int lda, int a_col_batch, const void *W, int w_row_batch, float *Y,
                     long long y_bs, int ldy, int T, int n_out, int K, int n_batch, int32_t *err_word,
                     void *stream);

/* Failure-path check of the kernels' bounded waits (a test aid; the paper has no counterpart): launches the
 * kernel of tpi_op_gemm_bf16 (single-CTA tiles, one batch, A without a low half) with its loader switched
 * off and every wait limited to `wait_polls` polls (1..65536, about 0.1 us each), so that no operand ever
 * arrives and every wait in the kernel runs out.  The kernel must then return by itself within
 * milliseconds, store nothing to Y, release its tensor memory, and leave 3 (wait timeout) in *err_word;
 * the device context stays usable.  Nothing in it can wait without a limit and nothing faults. */
int tpi_op_gemm_bf16_starved(const void *A, int lda, const void *W, float *Y, int ldy, int T, int n_out, int K,
                             int wait_polls, int32_t *err_word, void *stream);

/* The gate/up projection of Eq. 2 for T positions with SwiGLU applied in the GEMM's epilogue:
 * ACT[t][j] = silu(y[t][2j]) * y[t][2j+1], y = A . Wgu^T, Wgu bf16 [2 s][K] with rows interleaved
 * gate_j, up_j (all shards, shard-major).  A, A_lo as tpi_op_gemm_bf16 (one batch).  ACT: bf16 [T][s];
 * with split_out != 0 a second bf16 tensor bf16(v - hi) follows T*s elements later.  s % 16 == 0. */
int tpi_op_gemm_bf16_swiglu(const void *A, const void *A_lo, int lda, const void *Wgu, void *ACT, int split_out, int T,
                            int s, int K, int32_t *err_word, void *stream);

/* A row-sharded projection of Eq. 1-2 for T > 128 positions with the star sum and the shortcut in the GEMM's epilogue:
 * X[t][o] <- ((P_0[t][o] + P_1[t][o]) + ...) + X[t][o],  P_i = A[:, i*a_col_batch : i*a_col_batch + K] . W_i^T,
 * W_i = rows [i * w_row_batch, i * w_row_batch + n_out) of W (bf16, [.][K]); the partial sums P_i are formed in tensor
 * memory one shard after the other and added in rank order in fp32, the shortcut last; they never reach memory.
 * A, A_lo (required), err_word as tpi_op_gemm_bf16; X float [T][ldx] in/out (ldx, n_out multiples of 4).
 * TPI_ERR_SHAPE when T <= 128 or a size rule fails. */
int tpi_op_gemm_bf16_rowsum(const void *A, const void *A_lo, int lda, int a_col_batch, const void *W, int w_row_batch,
                            float *X, int ldx, int T, int n_out, int K, int n_shards, int32_t *err_word, void *stream);

/* Eq. 1-2's star sum and shortcut for T positions followed by the next block's RMSNorm:
 * X[t] <- ((P_0[t] + P_1[t]) + ...) + X[t];  Xn[t] = X[t] * rsqrt(mean(X[t]^2) + rms_eps) * gain.
 * partials: float[n_shards][T][h]; X in/out float[T][h]; gain float[h]; Xn float[T][h]. */
int tpi_op_reduce_residual_norm_rows(const float *partials, int n_shards, int T, int h, float *X, const float *gain,
                                     float rms_eps, float *Xn, void *stream);

/* Causal attention (Eq. 1) of T query positions [pos0, pos0+T) over cache positions [0, pos0+T); position pos0+t sees
 * cache rows 0 .. pos0+t.  Q, O: float[T][a][d] (Q after the rotation); kcache, vcache: one layer's cache,
 * [b][max_seq][d] in dtype, of which nothing past row pos0+T-1 is read.  bf16 caches run on tensor cores with the
 * queries and the softmax weights split into bf16 hi + lo (d = 128 and T >= 256: tcgen05 with S, P and O in tensor
 * memory; d = 64 / 128 otherwise: mma.sync); fp32 caches and other d on the fp32 SIMT kernel.  a % b == 0. */
int tpi_op_prefill_attention(int dtype, const float *Q, const void *kcache, const void *vcache, int T, int pos0,
                             int a, int b, int d, int max_seq, float *O, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TPI_OPS_H */
