// Host-side launchers of the CUDA kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tpi {

struct LaunchCtx {
  cudaStream_t stream = nullptr;
  bool pdl = false;        // programmatic dependent launch between consecutive kernels
  int* launches = nullptr; // counter of kernels launched (may be null)
};

enum { DT_F32 = 0, DT_BF16 = 1 };
// codes written to the device error word by kernel self-checks (the host reads it after a step)
// DEVERR_CANARY + i: the guard zone after the i-th carved arena buffer no longer holds its pattern (debug arenas)
enum : int { DEVERR_NONE = 0, DEVERR_TOKEN_RANGE = 1, DEVERR_POS_RANGE = 2, DEVERR_WAIT_TIMEOUT = 3, DEVERR_CANARY = 100 };
static inline size_t dt_size(int dt) { return dt == DT_BF16 ? 2 : 4; }

// A function attribute (e.g. the dynamic shared memory limit) belongs to one device: this remembers, per device
// ordinal, whether the current device already has it.
struct PerDeviceOnce {
  bool done[64] = {};
  static int cur() {
    int dev = 0;
    return cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64 ? dev : -1;
  }
  bool get() const { const int d = cur(); return d >= 0 && done[d]; }
  void set() { const int d = cur(); if (d >= 0) done[d] = true; }
};

// Input of a GEMV that starts a block: x is either already normalised (ss_part == nullptr) or the
// raw residual stream together with the producer's partial sums of squares, in which case the kernel
// applies x * rsqrt(sum(ss_part) / h + eps) while staging; gain (may be null) is the block's norm gain.
struct NormIn {
  const float* x;
  const float* gain;
  const float* ss_part;
  int n_parts;
  float eps;
};

// ---------------------------------------------------------------- decode (one position)
// x = W_emb[tok_hist[*pos]] (fp32); xhat = x * rsqrt(mean(x^2) + eps).
cudaError_t launch_embed(const LaunchCtx& c, int dt, const void* emb, const int* tok_hist,
                         const int* pos, int vocab, int max_seq, int h, float eps, float* x,
                         float* xhat, float* ss_part, int n_parts, int* err);

// Column-sharded QKV GEMV with fused rotary embedding and KV-cache append (Eq. 1 inputs).
// Wqkv: shard-major [(a/N + 2b/N) d][h] per shard.  q_out fp32 [a d] (rotated, unscaled).
cudaError_t launch_gemv_qkv(const LaunchCtx& c, int dt, const void* Wqkv, size_t shard_stride_elems,
                            const NormIn& in, int h, int n_shards, int a, int b,
                            int d, int max_seq, const int* pos, const float2* rope, float* q_out,
                            void* kcache_layer, void* vcache_layer);

// Column-sharded gate/up GEMV (rows interleaved gate_j, up_j) with SwiGLU epilogue (Eq. 2).
cudaError_t launch_gemv_gateup(const LaunchCtx& c, int dt, const void* Wgu, size_t shard_stride_elems,
                               const NormIn& in, int h, int n_shards, int s, float* act);

// Row-sharded GEMV: partials[i][r] = W^i[r, :] . x[i*Ks : (i+1)*Ks]   (per-device partial sums).
cudaError_t launch_gemv_partials(const LaunchCtx& c, int dt, const void* W, size_t shard_stride_elems,
                                 const float* x, int rows, int Ks, int n_shards, float* partials);

// The emulated star allreduce + shortcut + the next block's norm statistics:
// x <- ((P_0 + P_1) + ... + P_{N-1}) + x ; xhat = x * rsqrt(mean(x^2) + eps); tap (may be null) <- x.
// ss_part (may be null): also publish the sum of squares as ss_part[0], zeros in [1, n_parts).
cudaError_t launch_reduce_residual(const LaunchCtx& c, const float* partials, int n_shards, int h,
                                   float eps, float* x, float* xhat, float* tap, float* ss_part,
                                   int n_parts);

// Row-sharded projection fused with the star sum and the shortcut: x[r] <- ((P_0[r] + P_1[r]) + ...) + x[r]
// with P_i[r] = W^i[r,:] . x_in[i*Ks:(i+1)*Ks] formed in registers; ss_part[cta] <- sum of squares of the
// CTA's new entries (rowshard_fused_parts(rows) entries, zeros beyond the grid); tap (may be null) <- new x.
// Needs the whole x_in in shared memory (N * Ks * 4 <= 200 KiB).
cudaError_t launch_gemv_rowshard_fused(const LaunchCtx& c, int dt, const void* W, size_t shard_stride_elems,
                                       const float* x_in, int rows, int Ks, int n_shards, float* x,
                                       float* ss_part, float* tap);
// The same for shards of unequal width (heterogeneous p_i): shard i owns columns [k0[i], k0[i+1]) of the K = k0[n_shards]
// inputs, its matrix [rows][k0[i+1]-k0[i]] starts rows * k0[i] elements into W.  n_shards <= ROWSHARD_MAX_UNEQUAL.
constexpr int ROWSHARD_MAX_UNEQUAL = 16;
cudaError_t launch_gemv_rowshard_fused_unequal(const LaunchCtx& c, int dt, const void* W, const float* x_in, int rows,
                                               const int* k0, int n_shards, float* x, float* ss_part, float* tap);
int rowshard_fused_parts(int rows);
bool rowshard_fused_supported(int Ks, int n_shards);

// Split-K attention of one query position over the cache (Eq. 1), grouped heads.
// scratch: float[b * nsplit * (a/b) * (d + 2)], tickets: unsigned[b] (zero between launches).
cudaError_t launch_decode_attention(const LaunchCtx& c, int dt, const float* q, const void* kcache_layer,
                                    const void* vcache_layer, const int* pos, int a, int b, int d,
                                    int max_seq, int nsplit, float* scratch, unsigned* tickets,
                                    float* o);
size_t decode_attention_scratch_floats(int a, int b, int d, int nsplit);
// tensor-core form (bf16 cache, head dim 64 / 128, up to 8 query heads per kv head); launch_decode_attention uses it when it applies
bool decode_attention_mma_supported(int dt, int a, int b, int d, int nsplit);
cudaError_t launch_decode_attention_mma(const LaunchCtx& c, const float* q, const void* kcache_layer,
                                        const void* vcache_layer, const int* pos, int a, int b, int d, int max_seq,
                                        int nsplit, float* scratch, unsigned* tickets, float* o);

// Task head (Step 4): logits = W_head . (xhat * gain), greedy argmax (lowest index on ties);
// writes tok_hist[*pos + 1] and advances *pos.  amax scratch: >= grid blocks entries.
cudaError_t launch_head_argmax(const LaunchCtx& c, int dt, const void* Whead, const NormIn& in, int h,
                               int vocab, float* logits, float* amax_val, int* amax_idx, unsigned* ticket,
                               int* tok_hist, int* pos, int advance);
int head_argmax_blocks(int vocab);

// cos/sin table for positions [0, max_seq): table[p][i] = (cos, sin)(p * inv_freq[i]), fp64 inside.
cudaError_t launch_rope_table(const LaunchCtx& c, const double* inv_freq, int max_seq, int half,
                              float2* table);

// ---------------------------------------------------------------- prefill (T positions)
cudaError_t launch_embed_rows(const LaunchCtx& c, int dt, const void* emb, const int* tok_hist, int pos0,
                              int T, int vocab, int h, float* X, int* err);
// Xn[t] = X[t] * rsqrt(mean + eps) * gain.  out_bf16: 0 = fp32; 1 = bf16; 2 = split bf16 (hi at Xn,
// lo = bf16(v - hi) at Xn + T*h bf16 elements).  The same convention holds for the attention and SwiGLU outputs.
cudaError_t launch_rmsnorm_rows(const LaunchCtx& c, const float* X, const float* gain, int T, int h,
                                float eps, void* Xn, int out_bf16);
// Y[t][o] = sum_k X[t][k] W[o][k] for a batch of `n_batch` independent problems
// (batch = shard for the row-sharded projections).  X fp32, row stride ldx; Y fp32, row stride ldy.
cudaError_t launch_gemm_simt(const LaunchCtx& c, int dt, const float* X, long long x_batch_stride, int ldx,
                             const void* W, long long w_batch_stride_elems, float* Y,
                             long long y_batch_stride, int ldy, int T, int n_out, int K, int n_batch);
// The same contraction on the tensor cores (bf16 x bf16 -> fp32, tcgen05 + TMA): A is bf16 [T][lda], batch b
// reads K columns starting at b * a_col_batch; W is bf16 [n_batch * w_row_batch][K]; Y fp32.
// Needs gemm_tc_supported(K, lda, ldy).  err: device error word (bounded waits report there).
bool gemm_tc_supported(int K, int a_cols_total, int ldy);
// A_lo_bf16 (may be null): second bf16 tensor of the same shape with A = A_bf16 + A_lo_bf16 (split activations).
cudaError_t launch_gemm_tc(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                           const void* W_bf16, int w_row_batch, float* Y, long long y_batch_stride, int ldy, int T,
                           int n_out, int K, int n_batch, int* err, bool chunk_k = false);
// (chunk_k: a single-batch contraction over more than 128 positions is accumulated in chunks, see
// launch_gemm_tc_chunked; the column-sharded projections ask for it, the per-shard partial sums do not)
// Gate/up projection with the SwiGLU of launch_swiglu_rows applied in the epilogue (same arithmetic, same bits):
// Wgu rows interleaved gate_j, up_j; ACT [T][s] bf16 (out_mode 1) or split bf16 (2: lo at + T*s elements).
// CTA-pair tiles (tcgen05.mma.cta_group::2) for the same contract, split activations only.  gemm_tc_pair_choose returns
// the tile shape with the lowest predicted time (us_out), or -1 when none applies (T <= 128); launch_gemm_tc_pair
// runs that shape (act != nullptr: SwiGLU epilogue as above).
int gemm_tc_pair_choose(int T, int n_out, int K, int n_batch, int nsm, double* us_out);
cudaError_t launch_gemm_tc_pair(const LaunchCtx& c, int shape, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                                const void* W_bf16, int w_row_batch, float* Y, long long y_batch_stride, int ldy, int T, int n_out,
                                int K, int n_batch, int* err, void* act, int act_ld, long long act_lo_off, int act_split);
// Row-sharded projection of T > 128 positions with the star sum in its epilogue: X[t][o] = ((P_0 + P_1) + ... ) + X[t][o],
// P_i[t][o] = sum_k (A_hi + A_lo)[t][i*a_col_batch + k] * W[i*w_row_batch + o][k]; the partial sums stay on chip.
bool gemm_tc_rowsum_supported(int T, int K, int a_cols_total, int n_out, int ldx);
// The same pair kernel for the column-sharded projections, the contraction cut into chunks whose partial sums are added
// in registers (the tensor core truncates its fp32 accumulator at every step; short chains keep that drift small).
bool gemm_tc_chunked_supported(int T, int K, int lda, int n_out, int ldy, bool swiglu);
cudaError_t launch_gemm_tc_chunked(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, const void* W_bf16, float* Y,
                                   int ldy, int T, int n_out, int K, int* err, void* act, int act_ld, long long act_lo_off,
                                   int act_split);
cudaError_t launch_gemm_tc_rowsum(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                                  const void* W_bf16, int w_row_batch, float* X, int ldx, int T, int n_out, int K, int n_shards,
                                  int* err);
// Failure-path test aid: the single-CTA-tile kernel with its loader switched off and every wait cut to `wait_polls`
// polls (1..65536).  Every wait runs out: the kernel must return by itself, leave Y alone, free its tensor memory and
// report DEVERR_WAIT_TIMEOUT in *err.
cudaError_t launch_gemm_tc_starved(const LaunchCtx& c, const void* A_bf16, int lda, const void* W_bf16, float* Y, int ldy, int T,
                                   int n_out, int K, int* err, int wait_polls);
bool gemm_tc_swiglu_supported(int K, int lda, int s);
cudaError_t launch_gemm_tc_swiglu(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, const void* Wgu_bf16,
                                  void* ACT, int out_mode, int T, int s, int K, int* err);
// rotate q and k of T positions, append k, v to the cache. QKV rows: [shard][q | k | v] packed as the GEMV.
cudaError_t launch_rope_kv_rows(const LaunchCtx& c, int dt, const float* QKV, int T, int pos0, int n_shards,
                                int a, int b, int d, int max_seq, const float2* rope, float* Q,
                                void* kcache_layer, void* vcache_layer);
// causal attention of T query positions [pos0, pos0+T) over cache positions [0, pos0+T)
cudaError_t launch_prefill_attention(const LaunchCtx& c, int dt, const float* Q, const void* kcache_layer,
                                     const void* vcache_layer, int T, int pos0, int a, int b, int d,
                                     int max_seq, void* O, int out_bf16);
// the same on tensor cores (mma.sync m16n8k16) for a bf16 cache with head dim 64 or 128; out_mode as out_bf16 above
bool prefill_attention_mma_supported(int dt, int d);
cudaError_t launch_prefill_attention_mma(const LaunchCtx& c, const float* Q, const void* kcache_layer,
                                         const void* vcache_layer, int T, int pos0, int a, int b, int d, int max_seq,
                                         void* O, int out_mode);
// The same on tcgen05 (head dimension 128, bf16 cache, at least 256 positions): 128 queries x 128 keys per step, S and
// O in tensor memory.  err: device error word for the bounded waits (may be null).
bool prefill_attention_tc_supported(int dt, int d, int T);
cudaError_t launch_prefill_attention_tc(const LaunchCtx& c, const float* Q, const void* kcache_layer, const void* vcache_layer,
                                        int T, int pos0, int a, int b, int max_seq, void* O, int out_mode, int* err);
// act[t][j] = silu(GU[t][2j]) * GU[t][2j+1] per shard-major interleaved rows
cudaError_t launch_swiglu_rows(const LaunchCtx& c, const float* GU, int T, int s, void* ACT, int out_bf16);
// X[t] <- sum_i P_i[t] + X[t]; optional tap of the last row
cudaError_t launch_reduce_residual_rows(const LaunchCtx& c, const float* partials, int n_shards, int T,
                                        int h, float* X, float* tap_last);
// The same followed by the next block's RMSNorm (gain: that block's norm gain): Xn as launch_rmsnorm_rows writes it.
// Bit-identical to launch_reduce_residual_rows + launch_rmsnorm_rows.
cudaError_t launch_reduce_residual_norm_rows(const LaunchCtx& c, const float* partials, int n_shards, int T, int h,
                                             float* X, float* tap_last, const float* gain, float eps, void* Xn,
                                             int out_bf16);
// xhat of one row of X (to hand the last position to the decode-style head)
// (also sets *pos = pos_value when pos is not null)
cudaError_t launch_rmsnorm_stat_row(const LaunchCtx& c, const float* xrow, int h, float eps, float* x,
                                    float* xhat, float* ss_part, int n_parts, int* pos, int pos_value);

// Timeline buffer layout (see common.cuh): kernel ids 0 QKV, 1 gate/up, 3 task head (the column-sharded GEMVs' epilogue
// ids), 4 O projection, 5 down projection, 6 decode attention; slots TL_ENTRY, TL_WAIT (dependency wait returned),
// TL_STAGED (inputs in shared memory), TL_SMID (1 + the SM the CTA ran on), then one per warp from TL_WARP0 (the
// warp's last row is done).
enum { TL_KERNELS = 7, TL_CTAS = 160, TL_SLOTS = 40, TL_ENTRY = 0, TL_WAIT = 1, TL_STAGED = 2, TL_SMID = 3, TL_WARP0 = 4,
       TL_ID_O = 4, TL_ID_DOWN = 5, TL_ID_ATTN = 6 };
#ifdef TPI_TIMELINE
void set_timeline_decode(void* dev_buf);
void set_timeline_attn(void* dev_buf);
#endif

// tuning knobs (0: CTAs per SM of the column-sharded GEMVs, 1: of the fused row-sharded GEMVs,
// 2: L2 prefetch bytes per row before the dependency wait)
void set_tuning(int key, int value);
int get_tuning(int key);

// ---------------------------------------------------------------- one shard per rank: the exchange kernels
// Every rank has, in its own memory, a receive area of two halves of `half` floats each (fp32) and flags[2][R] (int):
// parity of the rank's exchange counter, then the R sources side by side, n floats each (n = h for a decode step,
// T * h for a prompt pass of T positions; R * n <= half).  Exchange number c (0-based, counted per rank in *epoch)
// uses parity c & 1; source j stores its n values at recv + (c & 1) * half + j * n of every destination and then sets
// flags[c & 1][j] = c + 1.
constexpr int TP_MAX_RANKS = 16;
struct TpPeers {
  int n_ranks, rank;
  long long half;             // floats per parity half of a receive area
  float* recv[TP_MAX_RANKS];  // destination ranks' receive areas (this rank's own included)
  int* flags[TP_MAX_RANKS];
};
// This rank's partial sums of a row-sharded projection, P[r] = W[r, :] . x_in (W [rows][Ks], the rank's own columns),
// stored into every rank's receive area, then published.  Same per-row arithmetic as launch_gemv_partials.
// ticket: unsigned, zero between launches.  drop != 0: compute but never publish (failure injection).
cudaError_t launch_tp_rowpush(const LaunchCtx& c, int dt, const void* W, const float* x_in, int rows, int Ks, const int* epoch,
                              unsigned* ticket, const TpPeers& peers, int drop);
// The master's broadcast of the embedded hidden state: x[h] into every rank's recv[c & 1][0], then the flags.
cudaError_t launch_tp_bcast(const LaunchCtx& c, const float* x, int h, const int* epoch, const TpPeers& peers, int drop);
// The consumer: waits (at most wait_polls polls per flag) until all sources of exchange *epoch have published, then
// mode 0: x <- ((P_0 + P_1) + ... + P_{R-1}) + x (rank order, shortcut last); mode 1: x <- P_0 (broadcast).
// Also tap (may be null) <- x, xhat, ss_part[0] = sum of squares (zeros in [1, n_parts)), ++*epoch, and
// (pos_advance != null) ++*pos_advance.  A wait that runs out sets DEVERR_WAIT_TIMEOUT in *err and changes nothing.
cudaError_t launch_tp_recv(const LaunchCtx& c, const float* recv, long long half, const int* flags, int* epoch, int n_ranks, int h,
                           int mode, float eps, float* x, float* xhat, float* tap, float* ss_part, int n_parts, int* pos_advance,
                           int* err, int wait_polls);
// Prompt pass: n floats of src (T x h partial sums, or the embedded rows with as_rank0 != 0) into every rank's slot of
// this source, then the flags; and the consumer's wait alone (n_src sources, 1 for the broadcast), which also advances
// the counter, so that the ordinary row kernels can read the receive area afterwards.
cudaError_t launch_tp_push_rows(const LaunchCtx& c, const float* src, size_t n, const int* epoch, unsigned* ticket,
                                const TpPeers& peers, int as_rank0, int drop);
cudaError_t launch_tp_wait(const LaunchCtx& c, const int* flags, int* epoch, int n_ranks, int n_src, int* err, int wait_polls);

// Guard zones of a debug arena: up to 64 zones of 256 bytes at base + off[i].  fill writes the pattern, check compares
// it and reports the first damaged zone as DEVERR_CANARY + i in *err (one CTA per zone, no other effect).
struct CanaryList {
  int n;
  unsigned long long off[64];
};
cudaError_t launch_canary_fill(const LaunchCtx& c, char* base, const CanaryList& L);
cudaError_t launch_canary_check(const LaunchCtx& c, const char* base, const CanaryList& L, int* err);

// misc
cudaError_t launch_fill_u32(const LaunchCtx& c, uint32_t* p, size_t n, uint32_t v);
cudaError_t launch_kv_convert(const LaunchCtx& c, int dt, void* cache_rows, float* f32_rows, size_t n,
                              int to_float);

}  // namespace tpi
