// Decode-step kernels (one position, batch 1): weight-streaming GEMVs with
// fused epilogues, the emulated star allreduce, split-K attention, task head.
//
// All of them are HBM-bound on the weight (or KV) bytes: 16-byte streaming
// loads, many in flight per lane, activations staged in shared memory, warp
// shuffle reductions, and an L2 bulk prefetch of each CTA's weight rows issued
// BEFORE the programmatic-dependent-launch wait so that the weight stream of
// kernel k+1 starts while kernel k (often a one-CTA reduction) is still running.
#include "common.cuh"
#include "gemv_bodies.cuh"
#include "kernels.h"
#include "launch.cuh"

namespace tpi {
#ifdef TPI_TIMELINE
void set_timeline_decode(void* dev_buf) { cudaMemcpyToSymbol(g_tl, &dev_buf, sizeof dev_buf); }
#endif

// =====================================================================================
// GEMV family
// =====================================================================================
struct Tuning {
  int cps_cols = 4;          // CTAs per SM, column-sharded GEMVs
  int cps_rows = 4;          // CTAs per SM, fused row-sharded GEMVs
  int prefetch_bytes = 1024; // L2 prefetch per row issued before the dependency wait (more than ~2 KB measured slower)
  int warps = 0;             // 0: one CTA per SM with a balanced warp count; 8, 16, 32: that many warps, cps CTAs per SM
};
static Tuning g_tune;
void set_tuning(int key, int value) {
  if (key == 0) g_tune.cps_cols = value;
  if (key == 1) g_tune.cps_rows = value;
  if (key == 2) g_tune.prefetch_bytes = value;
  if (key == 3) g_tune.warps = value;
}
int get_tuning(int key) {
  return key == 0 ? g_tune.cps_cols : key == 1 ? g_tune.cps_rows : key == 2 ? g_tune.prefetch_bytes : key == 3 ? g_tune.warps : 0;
}
static int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
  }
  return n;
}

// Work split of the persistent GEMVs.  `items` equal work items go to one CTA per SM as contiguous ranges, and
// inside a CTA warp w takes items w, w + W, ...: the kernel ends when the fullest warp ends, so W is chosen so
// that the busiest CTA's items fill its warps' rounds with little left over (a 7B-shaped gate/up projection has
// 74.4 row pairs per SM: 32 warps would need 3 rounds for 2.3 rounds of work, 25 warps fill 3 rounds exactly).
// Fewer warps keep fewer loads in flight, hence the weight below 20 warps.
constexpr int lb_threads(int w) { return w > 0 ? w * 32 : 1024; }
constexpr int lb_blocks(int w) { return w > 0 ? 32 / w : 1; }
static void balance_split(long long items, int* grid, int* warps) {
  const int sms = sm_count();
  const int g = (int)(items < sms ? (items < 1 ? 1 : items) : sms);
  const long long per = (items + g - 1) / g;  // items of the busiest CTA
  double best = -1.0;
  int bw = 8;
  for (int w = 32; w >= 4; --w) {
    const long long rounds = (per + w - 1) / w;
    const double fill = (double)items / g / (double)(rounds * w);
    const double score = fill * (w >= 20 ? 1.0 : w / 20.0);
    if (score > best + 1e-9) { best = score; bw = w; }
  }
  *grid = g;
  *warps = bw;
}

template <typename WT, int R, int EPI, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) wstream_rows_kernel(const GemvArgs A) {
  extern __shared__ __align__(16) float xs[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int bps = (A.items_per_shard + WARPS - 1) / WARPS;
  const int shard = blockIdx.x / bps;
  const int item = (blockIdx.x - shard * bps) * WARPS + warp;
  const bool valid = item < A.items_per_shard;

  int rows[R];
  item_rows<EPI, R>(A, valid ? item : 0, rows);
  const WT* Wsh = reinterpret_cast<const WT*>(A.W) + (size_t)shard * A.shard_stride;
  const uint4* wp[R];
#pragma unroll
  for (int r = 0; r < R; ++r) wp[r] = reinterpret_cast<const uint4*>(Wsh + (size_t)rows[r] * A.K);

  // Weights do not depend on the previous kernel: start pulling them into L2 now.
  if (valid && lane == 0) {
    const uint32_t row_bytes = (uint32_t)(A.K * sizeof(WT));
#pragma unroll
    for (int r = 0; r < R; ++r) l2_prefetch_bulk(wp[r], row_bytes);
  }
  pdl_launch_dependents();
  pdl_wait();  // the activation vector is written by the previous kernel

  float acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = 0.f;

  float rnorm = 1.f;
  if (A.ss_part) {  // every CTA sums the producer's partial sums in the same fixed order
    __shared__ float red[32];
    float ss = 0.f;
    for (int i = threadIdx.x; i < A.n_parts; i += WARPS * 32) ss += A.ss_part[i];
    ss = block_sum(ss, red);
    rnorm = rsqrtf(ss / (float)A.ss_dim + A.eps);
  }
  const float* xg = A.x + (size_t)shard * A.x_shard_stride;
  for (int k0 = 0; k0 < A.K; k0 += A.kc) {
    const int kc = min(A.kc, A.K - k0);
    if (k0) __syncthreads();
    for (int k = threadIdx.x * 4; k < kc; k += WARPS * 32 * 4) {
      float4 v = *reinterpret_cast<const float4*>(xg + k0 + k);
      if (A.ss_part) { v.x *= rnorm; v.y *= rnorm; v.z *= rnorm; v.w *= rnorm; }
      if (A.gain) {
        const float4 g = *reinterpret_cast<const float4*>(A.gain + k0 + k);
        v.x *= g.x; v.y *= g.y; v.z *= g.z; v.w *= g.w;
      }
      *reinterpret_cast<float4*>(xs + k) = v;
    }
    __syncthreads();
    if (valid) warp_dot<WT, R>(wp, k0 / Elem<WT>::VEC, xs, kc / Elem<WT>::VEC, lane, acc);
  }
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = warp_sum(acc[r]);

  // ---------------------------------------------------------------- epilogues
  if constexpr (EPI == EPI_QKV) {
    if (valid && lane == 0) {
      const int half = A.d >> 1;
      const int qp = A.hps * half, kp = A.kps * half;
      const int p = *A.pos;
      if (item < qp + kp) {
        const bool is_q = item < qp;
        const int t = is_q ? item : item - qp;
        const int hl = t / half, ii = t - hl * half;
        const float2 cs = A.rope[(size_t)p * half + ii];
        const float lo = acc[0] * cs.x - acc[1] * cs.y;
        const float hi = acc[1] * cs.x + acc[0] * cs.y;
        if (is_q) {
          float* q = A.out + (size_t)(shard * A.hps + hl) * A.d;
          q[ii] = lo;
          q[ii + half] = hi;
        } else {
          WT* kr = reinterpret_cast<WT*>(A.kcache) + ((size_t)(shard * A.kps + hl) * A.max_seq + p) * A.d;
          Elem<WT>::store(kr + ii, lo);
          Elem<WT>::store(kr + ii + half, hi);
        }
      } else {
        const int t2 = 2 * (item - qp - kp);
        const int hl = t2 / A.d, idx = t2 - hl * A.d;
        WT* vr = reinterpret_cast<WT*>(A.vcache) + ((size_t)(shard * A.kps + hl) * A.max_seq + p) * A.d;
        Elem<WT>::store(vr + idx, acc[0]);
        Elem<WT>::store(vr + idx + 1, acc[1]);
      }
    }
  } else if constexpr (EPI == EPI_SWIGLU) {
    if (valid && lane == 0) {
      const float g = acc[0], u = acc[1];
      A.out[(size_t)shard * A.out_shard_stride + item] = g / (1.f + expf(-g)) * u;
    }
  } else if constexpr (EPI == EPI_PARTIAL) {
    if (valid && lane == 0) {
      float* o = A.out + (size_t)shard * A.out_shard_stride + (size_t)item * R;
#pragma unroll
      for (int r = 0; r < R; ++r) o[r] = acc[r];
    }
  } else {  // EPI_LOGITS: write logits, then a grid-wide argmax with lowest index on ties
    __shared__ float s_val[WARPS];
    __shared__ int s_idx[WARPS];
    __shared__ bool s_last;
    float bv = -INFINITY;
    int bi = 0x7FFFFFFF;
    if (valid && lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        A.out[(size_t)item * R + r] = acc[r];
        if (acc[r] > bv) { bv = acc[r]; bi = item * R + r; }
      }
    }
    if (lane == 0) { s_val[warp] = bv; s_idx[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < WARPS; ++w)
        if (s_val[w] > bv || (s_val[w] == bv && s_idx[w] < bi)) { bv = s_val[w]; bi = s_idx[w]; }
      A.amax_val[blockIdx.x] = bv;
      A.amax_idx[blockIdx.x] = bi;
      __threadfence();
      const unsigned t = atomicAdd(A.ticket, 1u);
      s_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (s_last && warp == 0) {
      __threadfence();
      bv = -INFINITY;
      bi = 0x7FFFFFFF;
      for (int b = lane; b < (int)gridDim.x; b += 32) {
        const float v = __ldcg(A.amax_val + b);
        const int i = __ldcg(A.amax_idx + b);
        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float v = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
        const int i = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
      }
      if (lane == 0) {
        const int p = *A.pos_rw;
        A.tok_hist[p + 1] = bi;  // the token to feed at the next position
        if (A.advance) *A.pos_rw = p + 1;
        *A.ticket = 0u;
      }
    }
  }
}


template <typename WT, int EPI, int WARPS>
__global__ void __launch_bounds__(lb_threads(WARPS), lb_blocks(WARPS)) wstream_cols_kernel(const GemvArgs A) {
  extern __shared__ __align__(16) float xs[];
  cols_body<WT, EPI, WARPS>(A, xs, blockIdx.x, gridDim.x);
}

template <typename WT, int EPI, int WARPS>
static cudaError_t launch_gemv_cols_w(const LaunchCtx& c, GemvArgs& A) {
  A.prefetch_bytes = g_tune.prefetch_bytes;
  const long long total = (long long)A.items_per_shard * A.n_shards;
  long long grid = (long long)sm_count() * g_tune.cps_cols;
  int warps = WARPS;
  if constexpr (WARPS > 0) {
    if (grid > (total + WARPS - 1) / WARPS) grid = (total + WARPS - 1) / WARPS;
    if (grid < 1) grid = 1;
  } else {
    int g;
    balance_split(total, &g, &warps);
    grid = g;
  }
  auto kern = wstream_cols_kernel<WT, EPI, WARPS>;
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  return launch_kernel(c, kern, dim3((unsigned)grid), dim3(warps * 32), (size_t)A.K * sizeof(float), A);
}
template <typename WT, int EPI>
static cudaError_t launch_gemv_cols_t(const LaunchCtx& c, GemvArgs& A) {
  if (g_tune.warps <= 0) return launch_gemv_cols_w<WT, EPI, 0>(c, A);
  if (g_tune.warps >= 32) return launch_gemv_cols_w<WT, EPI, 32>(c, A);
  if (g_tune.warps >= 16) return launch_gemv_cols_w<WT, EPI, 16>(c, A);
  return launch_gemv_cols_w<WT, EPI, 8>(c, A);
}
static bool cols_persistent_ok(const GemvArgs& A) { return A.K <= 16384 && A.K % 4 == 0; }

static int pick_kc(int K) {
  // whole vector in shared memory up to 64 KiB, else chunks of 16384 floats
  return K <= 16384 ? K : 16384;
}

template <typename WT, int R, int EPI>
static cudaError_t launch_gemv_t(const LaunchCtx& c, GemvArgs& A) {
  constexpr int WARPS = 8;
  A.kc = pick_kc(A.K);
  const int bps = (A.items_per_shard + WARPS - 1) / WARPS;
  const size_t smem = (size_t)A.kc * sizeof(float);
  auto kern = wstream_rows_kernel<WT, R, EPI, WARPS>;
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  return launch_kernel(c, kern, dim3((unsigned)(bps * A.n_shards)), dim3(WARPS * 32), smem, A);
}

static void set_norm_in(GemvArgs& A, const NormIn& in, int h) {
  A.x = in.x; A.gain = in.gain; A.ss_part = in.ss_part; A.n_parts = in.n_parts; A.eps = in.eps; A.ss_dim = h;
}

cudaError_t launch_gemv_qkv(const LaunchCtx& c, int dt, const void* Wqkv, size_t shard_stride_elems,
                            const NormIn& in, int h, int n_shards, int a, int b,
                            int d, int max_seq, const int* pos, const float2* rope, float* q_out,
                            void* kcache_layer, void* vcache_layer) {
  GemvArgs A{};
  A.W = Wqkv; A.shard_stride = (long long)shard_stride_elems; set_norm_in(A, in, h); A.x_shard_stride = 0;
  A.K = h; A.n_shards = n_shards;
  A.hps = a / n_shards; A.kps = b / n_shards; A.d = d; A.max_seq = max_seq;
  A.items_per_shard = (A.hps + 2 * A.kps) * (d / 2);
  A.out = q_out; A.kcache = kcache_layer; A.vcache = vcache_layer; A.pos = pos; A.rope = rope;
  if (cols_persistent_ok(A))
    return dt == DT_BF16 ? launch_gemv_cols_t<__nv_bfloat16, EPI_QKV>(c, A) : launch_gemv_cols_t<float, EPI_QKV>(c, A);
  return dt == DT_BF16 ? launch_gemv_t<__nv_bfloat16, 2, EPI_QKV>(c, A) : launch_gemv_t<float, 2, EPI_QKV>(c, A);
}

cudaError_t launch_gemv_gateup(const LaunchCtx& c, int dt, const void* Wgu, size_t shard_stride_elems,
                               const NormIn& in, int h, int n_shards, int s,
                               float* act) {
  GemvArgs A{};
  A.W = Wgu; A.shard_stride = (long long)shard_stride_elems; set_norm_in(A, in, h); A.x_shard_stride = 0;
  A.K = h; A.n_shards = n_shards; A.items_per_shard = s / n_shards;
  A.out = act; A.out_shard_stride = s / n_shards;
  if (cols_persistent_ok(A))
    return dt == DT_BF16 ? launch_gemv_cols_t<__nv_bfloat16, EPI_SWIGLU>(c, A) : launch_gemv_cols_t<float, EPI_SWIGLU>(c, A);
  return dt == DT_BF16 ? launch_gemv_t<__nv_bfloat16, 2, EPI_SWIGLU>(c, A)
                       : launch_gemv_t<float, 2, EPI_SWIGLU>(c, A);
}

cudaError_t launch_gemv_partials(const LaunchCtx& c, int dt, const void* W, size_t shard_stride_elems,
                                 const float* x, int rows, int Ks, int n_shards, float* partials) {
  GemvArgs A{};
  A.W = W; A.shard_stride = (long long)shard_stride_elems; A.x = x; A.x_shard_stride = Ks;
  A.gain = nullptr; A.K = Ks; A.n_shards = n_shards; A.out = partials; A.out_shard_stride = rows;
  // rows per warp: keep >= ~8 KiB of weights per warp so that loads stay in flight
  const size_t row_bytes = (size_t)Ks * dt_size(dt);
  int R = 2;
  if (row_bytes <= 4096 && rows % 4 == 0) R = 4;
  if (rows % 2) R = 1;
  A.items_per_shard = rows / R;
  if (dt == DT_BF16) {
    if (R == 4) return launch_gemv_t<__nv_bfloat16, 4, EPI_PARTIAL>(c, A);
    if (R == 2) return launch_gemv_t<__nv_bfloat16, 2, EPI_PARTIAL>(c, A);
    return launch_gemv_t<__nv_bfloat16, 1, EPI_PARTIAL>(c, A);
  }
  if (R == 4) return launch_gemv_t<float, 4, EPI_PARTIAL>(c, A);
  if (R == 2) return launch_gemv_t<float, 2, EPI_PARTIAL>(c, A);
  return launch_gemv_t<float, 1, EPI_PARTIAL>(c, A);
}

static int head_rows_per_warp(int vocab) { return vocab % 2 == 0 ? 2 : 1; }
int head_argmax_blocks(int vocab) {
  const int R = head_rows_per_warp(vocab);
  const int per_item = (vocab / R + 7) / 8, per_sm = sm_count() * 4;  // an upper bound of every grid the head kernel uses
  return per_item > per_sm ? per_item : per_sm;
}

cudaError_t launch_head_argmax(const LaunchCtx& c, int dt, const void* Whead, const NormIn& in,
                               int h, int vocab, float* logits, float* amax_val,
                               int* amax_idx, unsigned* ticket, int* tok_hist, int* pos, int advance) {
  GemvArgs A{};
  A.W = Whead; A.shard_stride = 0; set_norm_in(A, in, h); A.x_shard_stride = 0; A.K = h;
  A.n_shards = 1; A.out = logits; A.amax_val = amax_val; A.amax_idx = amax_idx; A.ticket = ticket;
  A.tok_hist = tok_hist; A.pos_rw = pos; A.rows_total = vocab; A.advance = advance;
  if (cols_persistent_ok(A)) {  // row pairs; an odd last row is masked by rows_total
    A.items_per_shard = (vocab + 1) / 2;
    return dt == DT_BF16 ? launch_gemv_cols_t<__nv_bfloat16, EPI_LOGITS>(c, A) : launch_gemv_cols_t<float, EPI_LOGITS>(c, A);
  }
  const int R = head_rows_per_warp(vocab);
  A.items_per_shard = vocab / R;
  if (dt == DT_BF16)
    return R == 2 ? launch_gemv_t<__nv_bfloat16, 2, EPI_LOGITS>(c, A) : launch_gemv_t<__nv_bfloat16, 1, EPI_LOGITS>(c, A);
  return R == 2 ? launch_gemv_t<float, 2, EPI_LOGITS>(c, A) : launch_gemv_t<float, 1, EPI_LOGITS>(c, A);
}

template <typename WT, int R, int NS, int WARPS>
__global__ void __launch_bounds__(lb_threads(WARPS), lb_blocks(WARPS))
    wstream_rowshard_fused_kernel(const RowFusedArgs A) {
  extern __shared__ __align__(16) float xs[];
  rowfused_body<WT, R, NS, WARPS>(A, xs, blockIdx.x, gridDim.x);
}

// Entries of the per-CTA partial sums of squares that producers fill (zeros beyond their grid) and consumers add up:
// one per SM with the balanced one-CTA-per-SM launch, four per SM when a fixed warp count is forced.  Never more than
// the 1024 entries the arena plan reserves.
int rowshard_fused_parts(int) {
  const int n = g_tune.warps > 0 ? sm_count() * 4 : sm_count();
  return n > 1024 ? 1024 : n;
}
bool rowshard_fused_supported(int Ks, int n_shards) { return (size_t)Ks * n_shards * sizeof(float) <= 200 * 1024; }

template <typename WT, int R, int NS, int WARPS>
static cudaError_t launch_rowfused_w(const LaunchCtx& c, RowFusedArgs& A) {
  auto kern = wstream_rowshard_fused_kernel<WT, R, NS, WARPS>;
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  const size_t smem = (size_t)A.Ks * A.n_shards * sizeof(float);
  int cps = g_tune.cps_rows < 1 ? 1 : (g_tune.cps_rows > 4 ? 4 : g_tune.cps_rows);
  const int fit = (int)((220 * 1024) / (smem + 1024));
  if (cps > fit) cps = fit < 1 ? 1 : fit;
  const int groups = A.rows / R;
  int grid = sm_count() * cps, warps = WARPS;
  if constexpr (WARPS > 0) {
    if (grid > (groups + WARPS - 1) / WARPS) grid = (groups + WARPS - 1) / WARPS;
    if (grid < 1) grid = 1;
  } else {
    balance_split(groups, &grid, &warps);
  }
  return launch_kernel(c, kern, dim3(grid), dim3(warps * 32), smem, A);
}

template <typename WT, int R, int NS>
static cudaError_t launch_rowfused_t(const LaunchCtx& c, RowFusedArgs& A) {
  // Keep about 32 warps per SM: when the staged x_in is so large that fewer than four CTAs fit in an
  // SM's shared memory, make the CTAs bigger instead (70B-shaped down projection: 112 KiB of x_in).
  if (g_tune.warps <= 0) return launch_rowfused_w<WT, R, NS, 0>(c, A);
  const size_t smem = (size_t)A.Ks * A.n_shards * sizeof(float);
  const int fit = (int)((220 * 1024) / (smem + 1024));
  int warps = g_tune.warps;
  if (fit < 2 && warps < 32) warps = 32;
  else if (fit < 4 && warps < 16) warps = 16;
  if (warps >= 32) return launch_rowfused_w<WT, R, NS, 32>(c, A);
  if (warps >= 16) return launch_rowfused_w<WT, R, NS, 16>(c, A);
  return launch_rowfused_w<WT, R, NS, 8>(c, A);
}

cudaError_t launch_gemv_rowshard_fused(const LaunchCtx& c, int dt, const void* W, size_t shard_stride_elems,
                                       const float* x_in, int rows, int Ks, int n_shards, float* x,
                                       float* ss_part, float* tap) {
  if (!rowshard_fused_supported(Ks, n_shards)) return cudaErrorInvalidValue;
  RowFusedArgs A{};
  A.W = W; A.shard_stride = (long long)shard_stride_elems; A.x_in = x_in; A.Ks = Ks; A.n_shards = n_shards;
  A.rows = rows; A.x = x; A.ss_part = ss_part; A.tap = tap;
  A.n_parts = rowshard_fused_parts(rows);
  A.prefetch_bytes = g_tune.prefetch_bytes;
#define TPI_RF(WT)                                                      \
  do {                                                                  \
    switch (n_shards) {                                                 \
      case 1: return launch_rowfused_t<WT, 1, 1>(c, A);                 \
      case 2: return launch_rowfused_t<WT, 1, 2>(c, A);                 \
      case 4: return launch_rowfused_t<WT, 1, 4>(c, A);                 \
      case 8: return launch_rowfused_t<WT, 1, 8>(c, A);                 \
      default: return launch_rowfused_t<WT, 1, 0>(c, A);                \
    }                                                                   \
  } while (0)
  if (dt == DT_BF16) TPI_RF(__nv_bfloat16);
  TPI_RF(float);
#undef TPI_RF
}

cudaError_t launch_gemv_rowshard_fused_unequal(const LaunchCtx& c, int dt, const void* W, const float* x_in, int rows,
                                               const int* k0, int n_shards, float* x, float* ss_part, float* tap) {
  if (n_shards < 1 || n_shards > ROWSHARD_MAX_UNEQUAL || !k0 || k0[0] != 0) return cudaErrorInvalidValue;
  const int vec = dt == DT_BF16 ? 8 : 4;
  for (int i = 0; i < n_shards; ++i)
    if (k0[i + 1] <= k0[i] || (k0[i + 1] - k0[i]) % vec) return cudaErrorInvalidValue;
  const int K = k0[n_shards];
  if ((size_t)K * sizeof(float) > 200 * 1024) return cudaErrorInvalidValue;
  RowFusedArgs A{};
  A.W = W; A.shard_stride = 0; A.x_in = x_in; A.Ks = K; A.n_shards = n_shards;  // Ks * 1 shard sizes the staged x_in
  A.rows = rows; A.x = x; A.ss_part = ss_part; A.tap = tap;
  A.n_parts = rowshard_fused_parts(rows);
  A.prefetch_bytes = 0;
  A.unequal = 1;
  for (int i = 0; i <= n_shards; ++i) A.k0[i] = k0[i];
  // shared memory is sized from Ks * n_shards by the launcher: present the staged vector as one slice of K floats
  RowFusedArgs L = A;
  auto go = [&](auto wt) -> cudaError_t {
    using WT = decltype(wt);
    auto kern = wstream_rowshard_fused_kernel<WT, 1, 0, 0>;
    static PerDeviceOnce attr_done;
    if (!attr_done.get()) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return e;
      attr_done.set();
    }
    int grid, warps;
    balance_split(rows, &grid, &warps);
    return launch_kernel(c, kern, dim3(grid), dim3(warps * 32), (size_t)K * sizeof(float), L);
  };
  return dt == DT_BF16 ? go(__nv_bfloat16{}) : go(float{});
}

// =====================================================================================
// Embedding row + norm statistics (Algorithm 1 "Preprocess")
// =====================================================================================
template <typename WT>
__global__ void __launch_bounds__(1024) embed_kernel(const WT* emb, const int* tok_hist, const int* pos,
                                                    int vocab, int max_seq, int h, float eps, float* x,
                                                    float* xhat, float* ss_part, int n_parts, int* err) {
  __shared__ float red[32];
  // The step's first kernel waits for the previous token's task head (which advances *pos) BEFORE it lets its
  // dependents start: no kernel of this step can then be resident while the position is still the old one, which
  // is what lets the attention kernel read *pos ahead of its own dependency wait.
  pdl_wait();
  pdl_launch_dependents();
  const int p = *pos;
  int tok = (p >= 0 && p < max_seq) ? tok_hist[p] : -1;
  if (p < 0 || p >= max_seq) {
    if (threadIdx.x == 0) atomicCAS(err, DEVERR_NONE, DEVERR_POS_RANGE);
    tok = 0;
  } else if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0) atomicCAS(err, DEVERR_NONE, DEVERR_TOKEN_RANGE);
    tok = 0;
  }
  const WT* row = emb + (size_t)tok * h;
  float ss = 0.f;
  for (int k = threadIdx.x; k < h; k += blockDim.x) {
    const float v = Elem<WT>::load(row + k);
    x[k] = v;
    ss = fmaf(v, v, ss);
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)h + eps);
  for (int k = threadIdx.x; k < h; k += blockDim.x) xhat[k] = x[k] * r;
  for (int i = threadIdx.x; i < n_parts; i += blockDim.x) ss_part[i] = i ? 0.f : ss;
}

cudaError_t launch_embed(const LaunchCtx& c, int dt, const void* emb, const int* tok_hist,
                         const int* pos, int vocab, int max_seq, int h, float eps, float* x,
                         float* xhat, float* ss_part, int n_parts, int* err) {
  if (dt == DT_BF16)
    return launch_kernel(c, embed_kernel<__nv_bfloat16>, dim3(1), dim3(1024), 0,
                         (const __nv_bfloat16*)emb, tok_hist, pos, vocab, max_seq, h, eps, x, xhat, ss_part,
                         n_parts, err);
  return launch_kernel(c, embed_kernel<float>, dim3(1), dim3(1024), 0, (const float*)emb, tok_hist, pos,
                       vocab, max_seq, h, eps, x, xhat, ss_part, n_parts, err);
}

// =====================================================================================
// Emulated star allreduce + shortcut (+ norm statistics of the next block)
// =====================================================================================
__global__ void __launch_bounds__(1024) reduce_residual_kernel(const float* __restrict__ partials,
                                                              int n_shards, int h, float eps, float* x,
                                                              float* xhat, float* tap, float* ss_part,
                                                              int n_parts) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  float ss = 0.f;
  for (int k = threadIdx.x; k < h; k += blockDim.x) {
    float s = partials[k];  // master's own partial (rank 0) ...
    for (int i = 1; i < n_shards; ++i) s += partials[(size_t)i * h + k];  // ... plus workers, rank order
    s += x[k];              // shortcut is added after the allreduce (Eq. 1-2)
    x[k] = s;
    if (tap) tap[k] = s;
    ss = fmaf(s, s, ss);
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)h + eps);
  for (int k = threadIdx.x; k < h; k += blockDim.x) xhat[k] = x[k] * r;
  if (ss_part)
    for (int i = threadIdx.x; i < n_parts; i += blockDim.x) ss_part[i] = i ? 0.f : ss;
}

cudaError_t launch_reduce_residual(const LaunchCtx& c, const float* partials, int n_shards, int h,
                                   float eps, float* x, float* xhat, float* tap, float* ss_part,
                                   int n_parts) {
  return launch_kernel(c, reduce_residual_kernel, dim3(1), dim3(1024), 0, partials, n_shards, h, eps, x,
                       xhat, tap, ss_part, n_parts);
}

// =====================================================================================
// Split-K decode attention (Eq. 1) over cache positions 0..p, grouped query heads
// =====================================================================================
// One CTA = (kv head, split).  A "row group" of LPR lanes owns one cached position at a
// time (LPR * 16 bytes = one K or V row), keeps online-softmax state (m, l, acc) for the GRP
// query heads of the kv head, and walks the split's positions in batches of P.
// The split's K and V rows (contiguous in the cache) are first copied to shared memory with
// cp.async, all requests in flight at once, so the split costs one DRAM round trip instead of
// one per batch; splits longer than CH positions are walked CH positions at a time.
template <typename KT, int GRP, int LPR>
__global__ void __launch_bounds__(256) decode_attn_kernel(const float* __restrict__ q, const KT* kc,
                                                          const KT* vc, const int* pos, int max_seq,
                                                          int nsplit, float* scratch, unsigned* tickets,
                                                          float* o) {
  constexpr int VEC = Elem<KT>::VEC;
  constexpr int D = LPR * VEC;
  constexpr int WARPS = 8, RG = 32 / LPR, G = WARPS * RG, P = 4;  // 8 warps: enough warps per scheduler to hide ALU latency
  extern __shared__ __align__(16) float sm[];
  constexpr int CH = 256 / (int)sizeof(KT);  // positions staged at a time: 128 (bf16) or 64 (fp32)
  KT* k_s = reinterpret_cast<KT*>(sm);        // [CH][D], then V [CH][D]; reused by the merge buffers below
  KT* v_s = k_s + CH * D;
  float* sm_m = sm;                 // [G][GRP]
  float* sm_l = sm + G * GRP;       // [G][GRP]
  float* sm_acc = sm + 2 * G * GRP; // [G][GRP][D]
  __shared__ bool s_last;

  const int g = blockIdx.x, split = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp_id = warp * RG + lane / LPR, sub = lane % LPR;
  pdl_launch_dependents();
  pdl_wait();
  const int n = *pos + 1;  // visible positions (the current one was appended by the QKV kernel)
  int chunk = (n + nsplit - 1) / nsplit;
  chunk = (chunk + 31) & ~31;
  const int s0 = split * chunk, s1 = min(n, s0 + chunk);

  // scores are kept in the log2 domain: q is scaled by log2(e)/sqrt(d)
  const float qscale = 1.4426950408889634f * rsqrtf((float)D);
  float qr[GRP][VEC], acc[GRP][VEC], m[GRP], l[GRP];
#pragma unroll
  for (int hh = 0; hh < GRP; ++hh) {
    const float* qp = q + (size_t)(g * GRP + hh) * D + sub * VEC;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { qr[hh][v] = qp[v] * qscale; acc[hh][v] = 0.f; }
    m[hh] = -INFINITY;
    l[hh] = 0.f;
  }
  const KT* kg = kc + (size_t)g * max_seq * D;
  const KT* vg = vc + (size_t)g * max_seq * D;
  const KT* kbase = k_s + sub * VEC;  // rows are addressed relative to the staged window
  const KT* vbase = v_s + sub * VEC;

  // The trip count is the same for every lane of the warp (the loop variable is the CTA-wide batch
  // base), because the score reduction below shuffles across the whole warp.
  for (int w0 = s0; w0 < s1; w0 += CH) {
  const int wn = min(CH, s1 - w0);  // positions in this window
  if (w0 != s0) __syncthreads();    // everyone is done reading the previous window
  {
    const int n16 = wn * D * (int)sizeof(KT) / 16;  // 16-byte pieces per tensor
    const char* ksrc = reinterpret_cast<const char*>(kg + (size_t)w0 * D);
    const char* vsrc = reinterpret_cast<const char*>(vg + (size_t)w0 * D);
    for (int i = threadIdx.x; i < n16; i += WARPS * 32) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(reinterpret_cast<char*>(k_s) + i * 16)), "l"(ksrc + (size_t)i * 16) : "memory");
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(reinterpret_cast<char*>(v_s) + i * 16)), "l"(vsrc + (size_t)i * 16) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
  }
  for (int tb = 0; tb < wn; tb += G * P) {
    const int t0 = tb + grp_id;
    // the batch's K and V rows are requested together: one DRAM round trip per batch, not two
    uint4 kv[P], vv[P];
#pragma unroll
    for (int pp = 0; pp < P; ++pp) {
      const int t = t0 + pp * G;
      const bool in = t < wn;
      kv[pp] = in ? *reinterpret_cast<const uint4*>(kbase + (size_t)t * D) : make_uint4(0, 0, 0, 0);
      vv[pp] = in ? *reinterpret_cast<const uint4*>(vbase + (size_t)t * D) : make_uint4(0, 0, 0, 0);
    }
    float sc[P][GRP];
#pragma unroll
    for (int pp = 0; pp < P; ++pp) {
      float kf[VEC];
      Elem<KT>::unpack(kv[pp], kf);
#pragma unroll
      for (int hh = 0; hh < GRP; ++hh) {
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VEC; ++v) s = fmaf(qr[hh][v], kf[v], s);
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        sc[pp][hh] = (t0 + pp * G < wn) ? s : -INFINITY;
      }
    }
#pragma unroll
    for (int hh = 0; hh < GRP; ++hh) {
      float mx = sc[0][hh];
#pragma unroll
      for (int pp = 1; pp < P; ++pp) mx = fmaxf(mx, sc[pp][hh]);
      const float mn = fmaxf(m[hh], mx);
      // a group that has seen no position yet keeps m = -inf; use 0 as the reference then so that
      // exp2(-inf - ref) = 0 instead of exp2(-inf + inf) = NaN
      const float ref = (mn == -INFINITY) ? 0.f : mn;
      const float scale = exp2f(m[hh] - ref);
      m[hh] = mn;
      l[hh] *= scale;
#pragma unroll
      for (int v = 0; v < VEC; ++v) acc[hh][v] *= scale;
#pragma unroll
      for (int pp = 0; pp < P; ++pp) sc[pp][hh] = exp2f(sc[pp][hh] - ref);  // 0 for masked positions
    }
#pragma unroll
    for (int pp = 0; pp < P; ++pp) {
      float vf[VEC];
      Elem<KT>::unpack(vv[pp], vf);
#pragma unroll
      for (int hh = 0; hh < GRP; ++hh) {
        l[hh] += sc[pp][hh];
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[hh][v] = fmaf(sc[pp][hh], vf[v], acc[hh][v]);
      }
    }
  }
  }  // windows
  __syncthreads();  // the merge buffers alias the staged window
  // ---- merge the G row groups of this CTA (fixed order)
#pragma unroll
  for (int hh = 0; hh < GRP; ++hh) {
    if (sub == 0) { sm_m[grp_id * GRP + hh] = m[hh]; sm_l[grp_id * GRP + hh] = l[hh]; }
#pragma unroll
    for (int v = 0; v < VEC; ++v) sm_acc[(grp_id * GRP + hh) * D + sub * VEC + v] = acc[hh][v];
  }
  __syncthreads();
  float* part = scratch + ((size_t)g * nsplit + split) * GRP * (D + 2);
  for (int e = threadIdx.x; e < GRP * D; e += blockDim.x) {
    const int hh = e / D, dd = e - hh * D;
    float M = -INFINITY;
    for (int gi = 0; gi < G; ++gi) M = fmaxf(M, sm_m[gi * GRP + hh]);
    float A = 0.f, L = 0.f;
    if (M > -INFINITY) {
      for (int gi = 0; gi < G; ++gi) {
        const float w = exp2f(sm_m[gi * GRP + hh] - M);
        A = fmaf(w, sm_acc[(gi * GRP + hh) * D + dd], A);
        L = fmaf(w, sm_l[gi * GRP + hh], L);
      }
    }
    part[hh * (D + 2) + 2 + dd] = A;
    if (dd == 0) { part[hh * (D + 2)] = M; part[hh * (D + 2) + 1] = L; }
  }
  // ---- the last CTA of this kv head to arrive merges the splits in split order (one thread fences for the CTA:
  // the barrier orders every thread's stores before its fence, and its second fence precedes the barrier after which
  // the last CTA reads the other splits' results through L2)
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned t = atomicAdd(tickets + g, 1u);
    s_last = (t == (unsigned)nsplit - 1);
    __threadfence();
  }
  __syncthreads();
  if (!s_last) return;
  const int nact = (n + chunk - 1) / chunk;  // splits that saw at least one position
  const float* pg = scratch + (size_t)g * nsplit * GRP * (D + 2);
  // weights of the splits first (one exp2 per head and split, kept in shared memory; the row-group
  // buffers are free by now), then every thread sums its output elements over the splits in split order
  float* w_s = sm;                       // [GRP][nact] normalised weights
  __syncthreads();
  for (int hh = warp; hh < GRP; hh += WARPS) {
    float M = -INFINITY;
    for (int s = lane; s < nact; s += 32) M = fmaxf(M, __ldcg(pg + (size_t)(s * GRP + hh) * (D + 2)));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, off));
    float L = 0.f;  // fixed order: lane-strided partial sums, then the warp tree
    for (int s = lane; s < nact; s += 32) {
      const float* ps = pg + (size_t)(s * GRP + hh) * (D + 2);
      const float w = exp2f(__ldcg(ps) - M);
      w_s[hh * nact + s] = w;
      L = fmaf(w, __ldcg(ps + 1), L);
    }
    L = warp_sum(L);
    const float inv = 1.f / L;
    for (int s = lane; s < nact; s += 32) w_s[hh * nact + s] *= inv;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < GRP * D; e += blockDim.x) {
    const int hh = e / D, dd = e - hh * D;
    float A = 0.f;
#pragma unroll 8
    for (int s = 0; s < nact; ++s)
      A = fmaf(w_s[hh * nact + s], __ldcg(pg + (size_t)(s * GRP + hh) * (D + 2) + 2 + dd), A);
    o[(size_t)(g * GRP + hh) * D + dd] = A;
  }
  if (threadIdx.x == 0) tickets[g] = 0u;
}

size_t decode_attention_scratch_floats(int a, int b, int d, int nsplit) {
  return (size_t)b * nsplit * (a / b) * (d + 2);
}

template <typename KT, int GRP, int LPR>
static cudaError_t launch_attn_t(const LaunchCtx& c, const float* q, const void* kc, const void* vc,
                                 const int* pos, int b, int max_seq, int nsplit, float* scratch,
                                 unsigned* tickets, float* o) {
  constexpr int D = LPR * Elem<KT>::VEC, G = 8 * (32 / LPR);
  size_t smem = (size_t)(2 * G * GRP + G * GRP * D) * sizeof(float);
  if (smem < (size_t)GRP * nsplit * sizeof(float)) smem = (size_t)GRP * nsplit * sizeof(float);
  if (smem < (size_t)2 * 256 * D) smem = (size_t)2 * 256 * D;  // K and V windows: 2 x CH x D x sizeof = 512 D bytes
  auto kern = decode_attn_kernel<KT, GRP, LPR>;
  static PerDeviceOnce attr_done;
  if (smem > 48 * 1024 && !attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  return launch_kernel(c, kern, dim3(b, nsplit), dim3(256), smem, q, (const KT*)kc, (const KT*)vc, pos,
                       max_seq, nsplit, scratch, tickets, o);
}

template <typename KT, int LPR>
static cudaError_t launch_attn_g(const LaunchCtx& c, int grp, const float* q, const void* kc,
                                 const void* vc, const int* pos, int b, int max_seq, int nsplit,
                                 float* scratch, unsigned* tickets, float* o) {
  switch (grp) {
    case 1: return launch_attn_t<KT, 1, LPR>(c, q, kc, vc, pos, b, max_seq, nsplit, scratch, tickets, o);
    case 2: return launch_attn_t<KT, 2, LPR>(c, q, kc, vc, pos, b, max_seq, nsplit, scratch, tickets, o);
    case 4: return launch_attn_t<KT, 4, LPR>(c, q, kc, vc, pos, b, max_seq, nsplit, scratch, tickets, o);
    case 8: return launch_attn_t<KT, 8, LPR>(c, q, kc, vc, pos, b, max_seq, nsplit, scratch, tickets, o);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_decode_attention(const LaunchCtx& c, int dt, const float* q, const void* kcache_layer,
                                    const void* vcache_layer, const int* pos, int a, int b, int d,
                                    int max_seq, int nsplit, float* scratch, unsigned* tickets,
                                    float* o) {
  if (decode_attention_mma_supported(dt, a, b, d, nsplit))
    return launch_decode_attention_mma(c, q, kcache_layer, vcache_layer, pos, a, b, d, max_seq, nsplit, scratch, tickets, o);
  const int grp = a / b;
  const int lpr = (int)(d * dt_size(dt) / 16);
  if (dt == DT_BF16) {
    if (lpr == 16) return launch_attn_g<__nv_bfloat16, 16>(c, grp, q, kcache_layer, vcache_layer, pos, b, max_seq, nsplit, scratch, tickets, o);
    if (lpr == 8) return launch_attn_g<__nv_bfloat16, 8>(c, grp, q, kcache_layer, vcache_layer, pos, b, max_seq, nsplit, scratch, tickets, o);
    if (lpr == 4) return launch_attn_g<__nv_bfloat16, 4>(c, grp, q, kcache_layer, vcache_layer, pos, b, max_seq, nsplit, scratch, tickets, o);
  } else {
    if (lpr == 32) return launch_attn_g<float, 32>(c, grp, q, kcache_layer, vcache_layer, pos, b, max_seq, nsplit, scratch, tickets, o);
    if (lpr == 16) return launch_attn_g<float, 16>(c, grp, q, kcache_layer, vcache_layer, pos, b, max_seq, nsplit, scratch, tickets, o);
    if (lpr == 8) return launch_attn_g<float, 8>(c, grp, q, kcache_layer, vcache_layer, pos, b, max_seq, nsplit, scratch, tickets, o);
  }
  return cudaErrorInvalidValue;
}

// =====================================================================================
// Rotary table (built once per model)
// =====================================================================================
__global__ void rope_table_kernel(const double* inv_freq, int max_seq, int half, float2* table) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)max_seq * half) return;
  const int p = (int)(i / half), k = (int)(i - (size_t)p * half);
  double s, cth;
  sincos((double)p * inv_freq[k], &s, &cth);
  table[i] = make_float2((float)cth, (float)s);
}

cudaError_t launch_rope_table(const LaunchCtx& c, const double* inv_freq, int max_seq, int half,
                              float2* table) {
  const size_t n = (size_t)max_seq * half;
  return launch_kernel(c, rope_table_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, inv_freq,
                       max_seq, half, table);
}

}  // namespace tpi
