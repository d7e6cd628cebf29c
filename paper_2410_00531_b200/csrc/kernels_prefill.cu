// Prefill kernels: the same decoder block over T prompt positions at once
// (Algorithm 1, first pass of the loop: causal mask, cache positions pos0..pos0+T-1).
// This file holds the fp32-accurate SIMT path used for fp32 models and as the
// general fallback; the bf16 tensor-core GEMM lives in gemm_tcgen05.cu.
#include "common.cuh"
#include "kernels.h"
#include "launch.cuh"

namespace tpi {

// Activation store for the GEMM that follows: MODE 0 fp32, 1 bf16, 2 split bf16 (hi, and lo = v - hi at +lo_off).
template <int MODE>
__device__ __forceinline__ void store_act(void* base, size_t i, size_t lo_off, float v) {
  if (MODE == 0) reinterpret_cast<float*>(base)[i] = v;
  else {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    reinterpret_cast<__nv_bfloat16*>(base)[i] = hi;
    if (MODE == 2) reinterpret_cast<__nv_bfloat16*>(base)[lo_off + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
  }
}

// ------------------------------------------------------------------ embedding rows
template <typename WT>
__global__ void embed_rows_kernel(const WT* emb, const int* tok_hist, int pos0, int vocab, int h, float* X,
                                  int* err) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  const int t = blockIdx.x;
  int tok = tok_hist[pos0 + t];
  if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0) atomicCAS(err, DEVERR_NONE, DEVERR_TOKEN_RANGE);
    tok = 0;
  }
  const WT* row = emb + (size_t)tok * h;
  for (int k = threadIdx.x; k < h; k += blockDim.x) X[(size_t)t * h + k] = Elem<WT>::load(row + k);
}

cudaError_t launch_embed_rows(const LaunchCtx& c, int dt, const void* emb, const int* tok_hist, int pos0,
                              int T, int vocab, int h, float* X, int* err) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  if (dt == DT_BF16)
    return launch_kernel(nc, embed_rows_kernel<__nv_bfloat16>, dim3(T), dim3(256), 0,
                         (const __nv_bfloat16*)emb, tok_hist, pos0, vocab, h, X, err);
  return launch_kernel(nc, embed_rows_kernel<float>, dim3(T), dim3(256), 0, (const float*)emb, tok_hist,
                       pos0, vocab, h, X, err);
}

// ------------------------------------------------------------------ RMSNorm rows
// Row kernels below share one mapping so that their sums agree to the bit: thread tid owns the float4 groups
// tid, tid + B, ... of the row (B threads), adds the squares of its elements in index order, then block_sum.
constexpr int ROW_KEEP = 8;  // most float4 groups a thread keeps in registers (rows up to 32 * B elements)
__device__ __forceinline__ float sq4(float4 v, float ss) {
  ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
  return ss;
}
template <int MODE>
__device__ __forceinline__ void store_act4(void* base, size_t i, size_t lo_off, float4 v) {
  if (MODE == 0) *reinterpret_cast<float4*>(reinterpret_cast<float*>(base) + i) = v;
  else {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y), h2 = __float2bfloat16_rn(v.z),
                        h3 = __float2bfloat16_rn(v.w);
    __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(base) + i;
    *reinterpret_cast<uint2*>(o) = make_uint2((uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16),
                                              (uint32_t)__bfloat16_as_ushort(h2) | ((uint32_t)__bfloat16_as_ushort(h3) << 16));
    if (MODE == 2) {
      const __nv_bfloat16 l0 = __float2bfloat16_rn(v.x - __bfloat162float(h0)), l1 = __float2bfloat16_rn(v.y - __bfloat162float(h1)),
                          l2 = __float2bfloat16_rn(v.z - __bfloat162float(h2)), l3 = __float2bfloat16_rn(v.w - __bfloat162float(h3));
      *reinterpret_cast<uint2*>(o + lo_off) =
          make_uint2((uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16),
                     (uint32_t)__bfloat16_as_ushort(l2) | ((uint32_t)__bfloat16_as_ushort(l3) << 16));
    }
  }
}
// threads per row: enough float4 groups per thread to keep many loads in flight, few enough to stay in registers
static inline int row_threads(int h) { return h / 4 <= 8 * 256 ? 256 : 1024; }

// PARTS: 0 = plain RMSNorm of X; 1 = first X <- ((P_0 + P_1) + ...) + X (star sum in rank order + shortcut), then the norm.
template <int MODE, int PARTS, int THREADS, int KEEP>
__global__ void __launch_bounds__(THREADS) norm_rows_kernel(const float* __restrict__ partials, int n_shards, int T, int h,
                                                        float* X, float* tap_last, const float* __restrict__ gain,
                                                        float eps, void* Xn, size_t lo_off) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  __shared__ float red[32];
  const int B = blockDim.x, ng = h >> 2;
  const size_t n = (size_t)T * h, row = (size_t)blockIdx.x * h;
  float4 v[KEEP];
#pragma unroll
  for (int j = 0; j < KEEP; ++j) {
    const int g = threadIdx.x + j * B;
    if (g < ng) v[j] = *reinterpret_cast<const float4*>(X + row + 4 * g);
  }
  if (PARTS) {
    float4 acc[KEEP];
    for (int sh = 0; sh < n_shards; ++sh) {
#pragma unroll
      for (int j = 0; j < KEEP; ++j) {
        const int g = threadIdx.x + j * B;
        if (g < ng) {
          const float4 p = *reinterpret_cast<const float4*>(partials + (size_t)sh * n + row + 4 * g);
          if (sh == 0) acc[j] = p;
          else { acc[j].x += p.x; acc[j].y += p.y; acc[j].z += p.z; acc[j].w += p.w; }
        }
      }
    }
#pragma unroll
    for (int j = 0; j < KEEP; ++j) {
      const int g = threadIdx.x + j * B;
      if (g < ng) {
        v[j].x = acc[j].x + v[j].x; v[j].y = acc[j].y + v[j].y; v[j].z = acc[j].z + v[j].z; v[j].w = acc[j].w + v[j].w;
        *reinterpret_cast<float4*>(X + row + 4 * g) = v[j];
        if (tap_last && blockIdx.x == T - 1) *reinterpret_cast<float4*>(tap_last + 4 * g) = v[j];
      }
    }
  }
  if (!gain) return;  // sum and shortcut only
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < KEEP; ++j) {
    const int g = threadIdx.x + j * B;
    if (g < ng) ss = sq4(v[j], ss);
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)h + eps);
#pragma unroll
  for (int j = 0; j < KEEP; ++j) {
    const int g = threadIdx.x + j * B;
    if (g < ng) {
      const float4 gn = *reinterpret_cast<const float4*>(gain + 4 * g);
      store_act4<MODE>(Xn, row + 4 * g, lo_off,
                       make_float4(v[j].x * r * gn.x, v[j].y * r * gn.y, v[j].z * r * gn.z, v[j].w * r * gn.w));
    }
  }
}
static inline bool norm_rows_vec_ok(int h) { return h % 4 == 0 && h / 4 <= ROW_KEEP * 1024; }

// scalar form for widths the vector form does not take
template <int OUT_BF16>
__global__ void __launch_bounds__(1024) rmsnorm_rows_kernel(const float* X, const float* gain, int h, float eps,
                                                          void* Xn, size_t lo_off) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  __shared__ float red[32];
  const float* x = X + (size_t)blockIdx.x * h;
  float ss = 0.f;
  for (int k = threadIdx.x; k < h; k += blockDim.x) ss = fmaf(x[k], x[k], ss);
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)h + eps);
  for (int k = threadIdx.x; k < h; k += blockDim.x) {
    store_act<OUT_BF16>(Xn, (size_t)blockIdx.x * h + k, lo_off, x[k] * r * gain[k]);
  }
}

template <int PARTS>
static cudaError_t launch_norm_rows_vec(const LaunchCtx& c, const float* partials, int n_shards, int T, int h, float* X,
                                        float* tap_last, const float* gain, float eps, void* Xn, int mode) {
  const size_t lo = (size_t)T * h;
#define TPI_NR(MODE, THREADS, KEEP) \
  launch_kernel(c, norm_rows_kernel<MODE, PARTS, THREADS, KEEP>, dim3(T), dim3(THREADS), 0, partials, n_shards, T, h, X, tap_last, gain, eps, Xn, lo)
  if (row_threads(h) == 256) {
    if (h / 4 <= 4 * 256)  // rows up to 4096: half the registers, more rows in flight per SM
      return mode == 2 ? TPI_NR(2, 256, 4) : mode == 1 ? TPI_NR(1, 256, 4) : TPI_NR(0, 256, 4);
    return mode == 2 ? TPI_NR(2, 256, 8) : mode == 1 ? TPI_NR(1, 256, 8) : TPI_NR(0, 256, 8);
  }
  return mode == 2 ? TPI_NR(2, 1024, 8) : mode == 1 ? TPI_NR(1, 1024, 8) : TPI_NR(0, 1024, 8);
#undef TPI_NR
}

cudaError_t launch_rmsnorm_rows(const LaunchCtx& c, const float* X, const float* gain, int T, int h,
                                float eps, void* Xn, int out_bf16) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  if (norm_rows_vec_ok(h))
    return launch_norm_rows_vec<0>(nc, nullptr, 0, T, h, const_cast<float*>(X), nullptr, gain, eps, Xn, out_bf16);
  const size_t lo = (size_t)T * h;
  if (out_bf16 == 2) return launch_kernel(nc, rmsnorm_rows_kernel<2>, dim3(T), dim3(h >= 4096 ? 1024 : 256), 0, X, gain, h, eps, Xn, lo);
  if (out_bf16) return launch_kernel(nc, rmsnorm_rows_kernel<1>, dim3(T), dim3(h >= 4096 ? 1024 : 256), 0, X, gain, h, eps, Xn, lo);
  return launch_kernel(nc, rmsnorm_rows_kernel<0>, dim3(T), dim3(h >= 4096 ? 1024 : 256), 0, X, gain, h, eps, Xn, lo);
}

__global__ void __launch_bounds__(1024) rmsnorm_stat_row_kernel(const float* xrow, int h, float eps, float* x,
                                                               float* xhat, float* ss_part, int n_parts,
                                                               int* pos, int pos_value) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  __shared__ float red[32];
  float ss = 0.f;
  for (int k = threadIdx.x; k < h; k += blockDim.x) {
    const float v = xrow[k];
    x[k] = v;
    ss = fmaf(v, v, ss);
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)h + eps);
  for (int k = threadIdx.x; k < h; k += blockDim.x) xhat[k] = xrow[k] * r;
  for (int i = threadIdx.x; i < n_parts; i += blockDim.x) ss_part[i] = i ? 0.f : ss;
  if (threadIdx.x == 0 && pos) *pos = pos_value;
}

cudaError_t launch_rmsnorm_stat_row(const LaunchCtx& c, const float* xrow, int h, float eps, float* x,
                                    float* xhat, float* ss_part, int n_parts, int* pos, int pos_value) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  return launch_kernel(nc, rmsnorm_stat_row_kernel, dim3(1), dim3(1024), 0, xrow, h, eps, x, xhat, ss_part,
                       n_parts, pos, pos_value);
}

// ------------------------------------------------------------------ SIMT GEMM (fp32 accumulate)
// Y[b][t][o] = sum_k X[b][t][k] * W[b][o][k];   64x64 tile, 16-deep slices, 4x4 per thread.
template <typename WT>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const float* __restrict__ X, long long xbs, int ldx,
                                                        const WT* __restrict__ W, long long wbs,
                                                        float* __restrict__ Y, long long ybs, int ldy, int T,
                                                        int n_out, int K) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ __align__(16) float Xs[BK][BM + 4];
  __shared__ __align__(16) float Ws[BK][BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  X += (size_t)blockIdx.z * xbs;
  W += (size_t)blockIdx.z * wbs;
  Y += (size_t)blockIdx.z * ybs;
  const int lrow = tid >> 2, lk = (tid & 3) * 4;
  // Two-level accumulation: products are added into `acc` (fp32) for 64 consecutive k, then `acc` is folded into
  // `tot` (fp64).  A single fp32 running sum over K = 8192 terms loses ~2e-6 of relative accuracy per projection, too
  // close to the 1e-5 bar that fp32 models are held to over a whole network (an fp32 fold every 512: 1e-6, which over
  // 16 layers of the 70B widths still added up to the whole bar); with 64-term chains and an fp64 total it is ~3e-7,
  // for one conversion and one fp64 add per 64 products.
  constexpr int FOLD = 64;
  float acc[4][4];
  double tot[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; tot[i][j] = 0.0; }

  for (int k0 = 0; k0 < K; k0 += BK) {
    if (k0 && k0 % FOLD == 0) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { tot[i][j] += (double)acc[i][j]; acc[i][j] = 0.f; }
    }
    float xv[4] = {0.f, 0.f, 0.f, 0.f}, wv[4] = {0.f, 0.f, 0.f, 0.f};
    if (m0 + lrow < T && k0 + lk < K) {
      const float4 v = *reinterpret_cast<const float4*>(X + (size_t)(m0 + lrow) * ldx + k0 + lk);
      xv[0] = v.x; xv[1] = v.y; xv[2] = v.z; xv[3] = v.w;
    }
    if (n0 + lrow < n_out && k0 + lk < K) {
      const WT* wp = W + (size_t)(n0 + lrow) * K + k0 + lk;
      if constexpr (sizeof(WT) == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(wp);
        wv[0] = bf16lo(v.x); wv[1] = bf16hi(v.x); wv[2] = bf16lo(v.y); wv[3] = bf16hi(v.y);
      } else {
        const float4 v = *reinterpret_cast<const float4*>(wp);
        wv[0] = v.x; wv[1] = v.y; wv[2] = v.z; wv[3] = v.w;
      }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) { Xs[lk + i][lrow] = xv[i]; Ws[lk + i][lrow] = wv[i]; }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&Xs[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Ws[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= T) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < n_out) Y[(size_t)m * ldy + n] = (float)(tot[i][j] + (double)acc[i][j]);
    }
  }
}

// The same contraction on 128 x 64 tiles for more than 64 positions: 8 x 4 outputs per thread, the next 16-deep slice
// in flight (registers) while the current one is multiplied.  Every output is still ONE thread's running sum over k in
// ascending order with the fold (into an fp64 total) every 64, so the bits equal the 64 x 64 kernel's.
template <typename WT>
__global__ void __launch_bounds__(256, 2) gemm_simt_wide_kernel(const float* __restrict__ X, long long xbs, int ldx,
                                                             const WT* __restrict__ W, long long wbs,
                                                             float* __restrict__ Y, long long ybs, int ldy, int T,
                                                             int n_out, int K) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  constexpr int BM = 128, BN = 64, BK = 16, FOLD = 64;
  __shared__ __align__(16) float Xs[2][BK][BM + 4];
  __shared__ __align__(16) float Ws[2][BK][BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;  // thread: rows ty*4 + {0..3} and 64 + ty*4 + {0..3}, cols tx*4 + {0..3}
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  X += (size_t)blockIdx.z * xbs;
  W += (size_t)blockIdx.z * wbs;
  Y += (size_t)blockIdx.z * ybs;
  const int lrow = tid >> 2, lk = (tid & 3) * 4;  // loader: rows lrow and lrow + 64 of X, row lrow of W, 4 consecutive k
  // The fp64 totals live in shared memory (slot [output][thread]: no two threads share one, no barrier needed, no bank
  // conflict); in registers they would take the kernel from two CTAs per SM to one.
  extern __shared__ double tot_s[];  // [32][256]
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; tot_s[(i * 4 + j) * 256 + tid] = 0.0; }
  float4 xa, xb, wv;
  auto fetch = [&](int k0) {
    xa = xb = wv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (k0 + lk < K) {
      if (m0 + lrow < T) xa = *reinterpret_cast<const float4*>(X + (size_t)(m0 + lrow) * ldx + k0 + lk);
      if (m0 + 64 + lrow < T) xb = *reinterpret_cast<const float4*>(X + (size_t)(m0 + 64 + lrow) * ldx + k0 + lk);
      if (n0 + lrow < n_out) {
        const WT* wp = W + (size_t)(n0 + lrow) * K + k0 + lk;
        if constexpr (sizeof(WT) == 2) {
          const uint2 v = *reinterpret_cast<const uint2*>(wp);
          wv = make_float4(bf16lo(v.x), bf16hi(v.x), bf16lo(v.y), bf16hi(v.y));
        } else {
          wv = *reinterpret_cast<const float4*>(wp);
        }
      }
    }
  };
  auto stash = [&](int buf) {
    Xs[buf][lk + 0][lrow] = xa.x; Xs[buf][lk + 1][lrow] = xa.y; Xs[buf][lk + 2][lrow] = xa.z; Xs[buf][lk + 3][lrow] = xa.w;
    Xs[buf][lk + 0][64 + lrow] = xb.x; Xs[buf][lk + 1][64 + lrow] = xb.y; Xs[buf][lk + 2][64 + lrow] = xb.z; Xs[buf][lk + 3][64 + lrow] = xb.w;
    Ws[buf][lk + 0][lrow] = wv.x; Ws[buf][lk + 1][lrow] = wv.y; Ws[buf][lk + 2][lrow] = wv.z; Ws[buf][lk + 3][lrow] = wv.w;
  };
  fetch(0);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < K; k0 += BK) {
    if (k0 && k0 % FOLD == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { tot_s[(i * 4 + j) * 256 + tid] += (double)acc[i][j]; acc[i][j] = 0.f; }
    }
    const bool more = k0 + BK < K;
    if (more) fetch(k0 + BK);  // in flight while this slice is multiplied
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4*>(&Xs[buf][kk][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&Xs[buf][kk][64 + ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Ws[buf][kk][tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    if (more) {
      stash(buf ^ 1);  // the other buffer was last read one iteration ago, behind the barrier below
      __syncthreads();
      buf ^= 1;
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    if (m >= T) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < n_out) Y[(size_t)m * ldy + n] = (float)(tot_s[(i * 4 + j) * 256 + tid] + (double)acc[i][j]);
    }
  }
}

cudaError_t launch_gemm_simt(const LaunchCtx& c, int dt, const float* X, long long x_batch_stride, int ldx,
                             const void* W, long long w_batch_stride_elems, float* Y,
                             long long y_batch_stride, int ldy, int T, int n_out, int K, int n_batch) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  if (T > 64) {
    dim3 gridw((n_out + 63) / 64, (T + 127) / 128, n_batch);
    constexpr size_t tot_bytes = 32 * 256 * sizeof(double);  // the fp64 totals, one slot per output and thread
    static PerDeviceOnce attr_done;
    if (!attr_done.get()) {
      cudaError_t e = cudaFuncSetAttribute(gemm_simt_wide_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tot_bytes);
      if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_simt_wide_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tot_bytes);
      if (e != cudaSuccess) return e;
      attr_done.set();
    }
    if (dt == DT_BF16)
      return launch_kernel(nc, gemm_simt_wide_kernel<__nv_bfloat16>, gridw, dim3(256), tot_bytes, X, x_batch_stride, ldx,
                           (const __nv_bfloat16*)W, w_batch_stride_elems, Y, y_batch_stride, ldy, T, n_out, K);
    return launch_kernel(nc, gemm_simt_wide_kernel<float>, gridw, dim3(256), tot_bytes, X, x_batch_stride, ldx, (const float*)W,
                         w_batch_stride_elems, Y, y_batch_stride, ldy, T, n_out, K);
  }
  dim3 grid((n_out + 63) / 64, (T + 63) / 64, n_batch);
  if (dt == DT_BF16)
    return launch_kernel(nc, gemm_simt_kernel<__nv_bfloat16>, grid, dim3(256), 0, X, x_batch_stride, ldx,
                         (const __nv_bfloat16*)W, w_batch_stride_elems, Y, y_batch_stride, ldy, T, n_out, K);
  return launch_kernel(nc, gemm_simt_kernel<float>, grid, dim3(256), 0, X, x_batch_stride, ldx,
                       (const float*)W, w_batch_stride_elems, Y, y_batch_stride, ldy, T, n_out, K);
}

// ------------------------------------------------------------------ rotary + KV append for T rows
// QKV[t] holds, per shard i, [q heads | k heads | v heads] of that shard (the GEMM's column order).
template <typename WT>
__global__ void rope_kv_rows_kernel(const float* QKV, int pos0, int n_shards, int a, int b, int d, int max_seq,
                                    const float2* rope, float* Q, WT* kc, WT* vc) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  const int t = blockIdx.x, half = d >> 1;
  const int hps = a / n_shards, kps = b / n_shards;
  const int per_shard = (hps + 2 * kps) * d;
  const float* row = QKV + (size_t)t * per_shard * n_shards;
  const int p = pos0 + t;
  const int pairs = (a + b) * half;  // rotary pairs of q and k
  for (int e = blockIdx.y * blockDim.x + threadIdx.x; e < pairs + b * d; e += gridDim.y * blockDim.x) {
    if (e < pairs) {
      const int head = e / half, ii = e - head * half;  // heads 0..a-1 are q, a..a+b-1 are k
      const bool is_q = head < a;
      const int gh = is_q ? head : head - a;
      const int shard = is_q ? gh / hps : gh / kps;
      const int hl = is_q ? gh - shard * hps : gh - shard * kps;
      const float* src = row + (size_t)shard * per_shard + (is_q ? 0 : hps * d) + hl * d;
      const float2 cs = rope[(size_t)p * half + ii];
      const float lo = src[ii] * cs.x - src[ii + half] * cs.y;
      const float hi = src[ii + half] * cs.x + src[ii] * cs.y;
      if (is_q) {
        float* q = Q + ((size_t)t * a + gh) * d;
        q[ii] = lo;
        q[ii + half] = hi;
      } else {
        WT* kr = kc + ((size_t)gh * max_seq + p) * d;
        Elem<WT>::store(kr + ii, lo);
        Elem<WT>::store(kr + ii + half, hi);
      }
    } else {
      const int e2 = e - pairs, gh = e2 / d, idx = e2 - gh * d;
      const int shard = gh / kps, hl = gh - shard * kps;
      const float* src = row + (size_t)shard * per_shard + (hps + kps) * d + hl * d;
      Elem<WT>::store(vc + ((size_t)gh * max_seq + p) * d + idx, src[idx]);
    }
  }
}

// The same, four consecutive elements per thread (16-byte loads of the projections and the rotation table, 16- or
// 8-byte stores); needs d % 8 == 0.  Same expressions per element as the scalar kernel.
__device__ __forceinline__ void store4(float* p, const float (&v)[4]) { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }
__device__ __forceinline__ void store4(__nv_bfloat16* p, const float (&v)[4]) {
  const __nv_bfloat162 a = __halves2bfloat162(__float2bfloat16_rn(v[0]), __float2bfloat16_rn(v[1]));
  const __nv_bfloat162 b = __halves2bfloat162(__float2bfloat16_rn(v[2]), __float2bfloat16_rn(v[3]));
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
}
template <typename WT>
__global__ void __launch_bounds__(256) rope_kv_rows_vec_kernel(const float* QKV, int pos0, int n_shards, int a, int b, int d,
                                                               int max_seq, const float2* rope, float* Q, WT* kc, WT* vc) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  const int t = blockIdx.x, half = d >> 1, hq = half >> 2, dq = d >> 2;
  const int hps = a / n_shards, kps = b / n_shards;
  const int per_shard = (hps + 2 * kps) * d;
  const float* row = QKV + (size_t)t * per_shard * n_shards;
  const int p = pos0 + t;
  const int groups = (a + b) * hq;  // groups of 4 rotary pairs of q and k
  for (int e = blockIdx.y * blockDim.x + threadIdx.x; e < groups + b * dq; e += gridDim.y * blockDim.x) {
    if (e < groups) {
      const int head = e / hq, ii = (e - head * hq) * 4;  // heads 0..a-1 are q, a..a+b-1 are k
      const bool is_q = head < a;
      const int gh = is_q ? head : head - a;
      const int shard = is_q ? gh / hps : gh / kps;
      const int hl = is_q ? gh - shard * hps : gh - shard * kps;
      const float* src = row + (size_t)shard * per_shard + (is_q ? 0 : hps * d) + hl * d;
      const float4 x0 = *reinterpret_cast<const float4*>(src + ii), x1 = *reinterpret_cast<const float4*>(src + ii + half);
      const float4 r0 = *reinterpret_cast<const float4*>(rope + (size_t)p * half + ii);
      const float4 r1 = *reinterpret_cast<const float4*>(rope + (size_t)p * half + ii + 2);
      const float xl[4] = {x0.x, x0.y, x0.z, x0.w}, xh[4] = {x1.x, x1.y, x1.z, x1.w};
      const float cs[4] = {r0.x, r0.z, r1.x, r1.z}, sn[4] = {r0.y, r0.w, r1.y, r1.w};
      float lo[4], hi[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        lo[j] = xl[j] * cs[j] - xh[j] * sn[j];
        hi[j] = xh[j] * cs[j] + xl[j] * sn[j];
      }
      if (is_q) {
        float* q = Q + ((size_t)t * a + gh) * d;
        store4(q + ii, lo);
        store4(q + ii + half, hi);
      } else {
        WT* kr = kc + ((size_t)gh * max_seq + p) * d;
        store4(kr + ii, lo);
        store4(kr + ii + half, hi);
      }
    } else {
      const int e2 = e - groups, gh = e2 / dq, idx = (e2 - gh * dq) * 4;
      const int shard = gh / kps, hl = gh - shard * kps;
      const float* src = row + (size_t)shard * per_shard + (hps + kps) * d + hl * d;
      const float4 x = *reinterpret_cast<const float4*>(src + idx);
      const float v[4] = {x.x, x.y, x.z, x.w};
      store4(vc + ((size_t)gh * max_seq + p) * d + idx, v);
    }
  }
}

cudaError_t launch_rope_kv_rows(const LaunchCtx& c, int dt, const float* QKV, int T, int pos0, int n_shards,
                                int a, int b, int d, int max_seq, const float2* rope, float* Q,
                                void* kcache_layer, void* vcache_layer) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  if (d % 8 == 0) {
    const int work4 = (a + b) * (d / 8) + b * (d / 4);  // groups of four per position
    const dim3 grid4(T, (work4 + 255) / 256);
    if (dt == DT_BF16)
      return launch_kernel(nc, rope_kv_rows_vec_kernel<__nv_bfloat16>, grid4, dim3(256), 0, QKV, pos0, n_shards, a, b, d, max_seq,
                           rope, Q, (__nv_bfloat16*)kcache_layer, (__nv_bfloat16*)vcache_layer);
    return launch_kernel(nc, rope_kv_rows_vec_kernel<float>, grid4, dim3(256), 0, QKV, pos0, n_shards, a, b, d, max_seq, rope, Q,
                         (float*)kcache_layer, (float*)vcache_layer);
  }
  const int work = (a + b) * (d / 2) + b * d;  // elements per position; two per thread and slice
  const dim3 grid(T, (work + 511) / 512);
  if (dt == DT_BF16)
    return launch_kernel(nc, rope_kv_rows_kernel<__nv_bfloat16>, grid, dim3(256), 0, QKV, pos0, n_shards, a,
                         b, d, max_seq, rope, Q, (__nv_bfloat16*)kcache_layer, (__nv_bfloat16*)vcache_layer);
  return launch_kernel(nc, rope_kv_rows_kernel<float>, grid, dim3(256), 0, QKV, pos0, n_shards, a, b, d,
                       max_seq, rope, Q, (float*)kcache_layer, (float*)vcache_layer);
}

// ------------------------------------------------------------------ causal attention, T queries
// One warp = one (query position, head).  Per tile of 32 cached positions: each lane scores one
// position (full dot product, q broadcast from shared memory), the tile's softmax statistics go
// through shuffles, then each lane accumulates its d/32 output dims over the tile's values.
template <typename KT, int D, int OUT_BF16>
__global__ void __launch_bounds__(128) prefill_attn_kernel(const float* __restrict__ Q, const KT* kc,
                                                           const KT* vc, int T, int pos0, int a, int b,
                                                           int max_seq, void* O, size_t lo_off) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  constexpr int VEC = Elem<KT>::VEC, DPL = D / 32;
  __shared__ __align__(16) float qs[4][D];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * 4 + warp, j = blockIdx.y, g = j / (a / b);
  const bool active = t < T;
  const float qscale = 1.4426950408889634f * rsqrtf((float)D);
  if (active)
    for (int i = lane; i < D; i += 32) qs[warp][i] = Q[((size_t)t * a + j) * D + i] * qscale;
  __syncwarp();
  if (!active) return;
  const int n = pos0 + t + 1;
  const KT* kb = kc + (size_t)g * max_seq * D;
  const KT* vb = vc + (size_t)g * max_seq * D;
  float m = -INFINITY, l = 0.f, acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  for (int p0 = 0; p0 < n; p0 += 32) {
    const int p = p0 + lane;
    float s = -INFINITY;
    if (p < n) {
      s = 0.f;
      const uint4* kr = reinterpret_cast<const uint4*>(kb + (size_t)p * D);
#pragma unroll 4
      for (int v = 0; v < D / VEC; ++v) s = Elem<KT>::dot(kr[v], &qs[warp][v * VEC], s);
    }
    float mx = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    const float mn = fmaxf(m, mx);
    const float scale = exp2f(m - mn);
    const float w = exp2f(s - mn);
    l = l * scale + warp_sum(w);
    m = mn;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] *= scale;
    const int cnt = min(32, n - p0);
    for (int u = 0; u < cnt; ++u) {
      const float wu = __shfl_sync(0xFFFFFFFFu, w, u);
      const KT* vr = vb + (size_t)(p0 + u) * D + lane * DPL;
#pragma unroll
      for (int i = 0; i < DPL; ++i) acc[i] = fmaf(wu, Elem<KT>::load(vr + i), acc[i]);
    }
  }
  const size_t off = ((size_t)t * a + j) * D + lane * DPL;
#pragma unroll
  for (int i = 0; i < DPL; ++i) store_act<OUT_BF16>(O, off + i, lo_off, acc[i] / l);
}

cudaError_t launch_prefill_attention(const LaunchCtx& c, int dt, const float* Q, const void* kcache_layer,
                                     const void* vcache_layer, int T, int pos0, int a, int b, int d,
                                     int max_seq, void* O, int out_bf16) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  dim3 grid((T + 3) / 4, a);
  const size_t lo = (size_t)T * a * d;
#define TPI_PA_M(KT, DD, MM)                                                                           \
  launch_kernel(nc, prefill_attn_kernel<KT, DD, MM>, grid, dim3(128), 0, Q, (const KT*)kcache_layer,   \
                (const KT*)vcache_layer, T, pos0, a, b, max_seq, O, lo)
#define TPI_PA(KT, DD) \
  return out_bf16 == 2 ? TPI_PA_M(KT, DD, 2) : (out_bf16 ? TPI_PA_M(KT, DD, 1) : TPI_PA_M(KT, DD, 0))
  if (dt == DT_BF16) {
    if (d == 128) TPI_PA(__nv_bfloat16, 128);
    if (d == 64) TPI_PA(__nv_bfloat16, 64);
    if (d == 32) TPI_PA(__nv_bfloat16, 32);
  } else {
    if (d == 128) TPI_PA(float, 128);
    if (d == 64) TPI_PA(float, 64);
    if (d == 32) TPI_PA(float, 32);
  }
#undef TPI_PA
#undef TPI_PA_M
  return cudaErrorInvalidValue;
}

// ------------------------------------------------------------------ SwiGLU rows
template <int OUT_BF16>
__global__ void swiglu_rows_kernel(const float* GU, size_t n_pairs, void* ACT) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pairs) return;
  const float2 gu = reinterpret_cast<const float2*>(GU)[i];
  store_act<OUT_BF16>(ACT, i, n_pairs, gu.x / (1.f + expf(-gu.x)) * gu.y);
}

cudaError_t launch_swiglu_rows(const LaunchCtx& c, const float* GU, int T, int s, void* ACT, int out_bf16) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  const size_t n = (size_t)T * s;
  const dim3 grid((unsigned)((n + 255) / 256));
  if (out_bf16 == 2) return launch_kernel(nc, swiglu_rows_kernel<2>, grid, dim3(256), 0, GU, n, ACT);
  if (out_bf16) return launch_kernel(nc, swiglu_rows_kernel<1>, grid, dim3(256), 0, GU, n, ACT);
  return launch_kernel(nc, swiglu_rows_kernel<0>, grid, dim3(256), 0, GU, n, ACT);
}

// ------------------------------------------------------------------ allreduce + shortcut, T rows
__global__ void reduce_residual_rows_kernel(const float* __restrict__ partials, int n_shards, int T, int h,
                                            float* X, float* tap_last) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  const size_t n = (size_t)T * h;
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = partials[i];
  for (int k = 1; k < n_shards; ++k) s += partials[(size_t)k * n + i];
  s += X[i];
  X[i] = s;
  if (tap_last && i >= n - h) tap_last[i - (n - h)] = s;
}

cudaError_t launch_reduce_residual_rows(const LaunchCtx& c, const float* partials, int n_shards, int T,
                                        int h, float* X, float* tap_last) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  if (norm_rows_vec_ok(h)) return launch_norm_rows_vec<1>(nc, partials, n_shards, T, h, X, tap_last, nullptr, 0.f, nullptr, 0);
  const size_t n = (size_t)T * h;
  return launch_kernel(nc, reduce_residual_rows_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0,
                       partials, n_shards, T, h, X, tap_last);
}

// The same followed by the next block's RMSNorm in one pass over the row (one CTA per position): the element to
// thread mapping and the order of every sum are those of the two separate kernels, so the results are the same bits.
template <int MODE>
__global__ void __launch_bounds__(1024) reduce_residual_norm_rows_kernel(const float* __restrict__ partials, int n_shards,
                                                                        int T, int h, float* X, float* tap_last,
                                                                        const float* __restrict__ gain, float eps,
                                                                        void* Xn, size_t lo_off) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  __shared__ float red[32];
  constexpr int KEEP = 8;
  const size_t n = (size_t)T * h, row = (size_t)blockIdx.x * h;
  float v[KEEP];
  float ss = 0.f;
  int j = 0;
  for (int k = threadIdx.x; k < h; k += blockDim.x, ++j) {
    const size_t i = row + k;
    float s = partials[i];
    for (int sh = 1; sh < n_shards; ++sh) s += partials[(size_t)sh * n + i];
    s += X[i];
    X[i] = s;
    if (tap_last && blockIdx.x == T - 1) tap_last[k] = s;
    if (j < KEEP) v[j] = s;
    ss = fmaf(s, s, ss);
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)h + eps);
  j = 0;
  for (int k = threadIdx.x; k < h; k += blockDim.x, ++j) {
    const float x = j < KEEP ? v[j] : X[row + k];  // a thread re-reads only what it wrote itself
    store_act<MODE>(Xn, row + k, lo_off, x * r * gain[k]);
  }
}

cudaError_t launch_reduce_residual_norm_rows(const LaunchCtx& c, const float* partials, int n_shards, int T, int h,
                                             float* X, float* tap_last, const float* gain, float eps, void* Xn,
                                             int out_bf16) {
  LaunchCtx nc = c;
  if (norm_rows_vec_ok(h)) return launch_norm_rows_vec<1>(nc, partials, n_shards, T, h, X, tap_last, gain, eps, Xn, out_bf16);
  const size_t lo = (size_t)T * h;
  const dim3 block(h >= 4096 ? 1024 : 256);  // as launch_rmsnorm_rows: the same per-thread sums
  if (out_bf16 == 2)
    return launch_kernel(nc, reduce_residual_norm_rows_kernel<2>, dim3(T), block, 0, partials, n_shards, T, h, X, tap_last, gain, eps, Xn, lo);
  if (out_bf16)
    return launch_kernel(nc, reduce_residual_norm_rows_kernel<1>, dim3(T), block, 0, partials, n_shards, T, h, X, tap_last, gain, eps, Xn, lo);
  return launch_kernel(nc, reduce_residual_norm_rows_kernel<0>, dim3(T), block, 0, partials, n_shards, T, h, X, tap_last, gain, eps, Xn, lo);
}

// ------------------------------------------------------------------ misc
__global__ void fill_u32_kernel(uint32_t* p, size_t n, uint32_t v) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    p[i] = v;
}
cudaError_t launch_fill_u32(const LaunchCtx& c, uint32_t* p, size_t n, uint32_t v) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  const unsigned blocks = (unsigned)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
  return launch_kernel(nc, fill_u32_kernel, dim3(blocks ? blocks : 1), dim3(256), 0, p, n, v);
}

// ------------------------------------------------------------------ guard zones of a debug arena
__device__ __forceinline__ uint32_t canary_word(int zone, int i) { return 0xC0DE0000u ^ ((uint32_t)zone << 8) ^ (uint32_t)i; }
__global__ void canary_kernel(char* base, const CanaryList L, int* err, int fill) {
  pdl_launch_dependents();
  pdl_wait();  // everything the step wrote is in memory
  const int z = blockIdx.x, i = threadIdx.x;  // 64 words per zone
  uint32_t* w = reinterpret_cast<uint32_t*>(base + L.off[z]);
  if (fill) w[i] = canary_word(z, i);
  else if (__ldcg(w + i) != canary_word(z, i)) atomicCAS(err, DEVERR_NONE, DEVERR_CANARY + z);
}
cudaError_t launch_canary_fill(const LaunchCtx& c, char* base, const CanaryList& L) {
  if (L.n < 1) return cudaSuccess;
  return launch_kernel(c, canary_kernel, dim3(L.n), dim3(64), 0, base, L, (int*)nullptr, 1);
}
cudaError_t launch_canary_check(const LaunchCtx& c, const char* base, const CanaryList& L, int* err) {
  if (L.n < 1) return cudaSuccess;
  return launch_kernel(c, canary_kernel, dim3(L.n), dim3(64), 0, const_cast<char*>(base), L, err, 0);
}

template <typename WT, int TO_FLOAT>
__global__ void kv_convert_kernel(WT* cache, float* f, size_t n) {
  pdl_launch_dependents();
  pdl_wait();  // inputs come from the previous kernel in the stream
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  if (TO_FLOAT) f[i] = Elem<WT>::load(cache + i);
  else Elem<WT>::store(cache + i, f[i]);
}
cudaError_t launch_kv_convert(const LaunchCtx& c, int dt, void* cache_rows, float* f32_rows, size_t n,
                              int to_float) {
  LaunchCtx nc = c;  // PDL allowed: every kernel below waits on its predecessor before touching memory
  dim3 grid((unsigned)((n + 255) / 256));
  if (dt == DT_BF16) {
    if (to_float) return launch_kernel(nc, kv_convert_kernel<__nv_bfloat16, 1>, grid, dim3(256), 0, (__nv_bfloat16*)cache_rows, f32_rows, n);
    return launch_kernel(nc, kv_convert_kernel<__nv_bfloat16, 0>, grid, dim3(256), 0, (__nv_bfloat16*)cache_rows, f32_rows, n);
  }
  if (to_float) return launch_kernel(nc, kv_convert_kernel<float, 1>, grid, dim3(256), 0, (float*)cache_rows, f32_rows, n);
  return launch_kernel(nc, kv_convert_kernel<float, 0>, grid, dim3(256), 0, (float*)cache_rows, f32_rows, n);
}

}  // namespace tpi
