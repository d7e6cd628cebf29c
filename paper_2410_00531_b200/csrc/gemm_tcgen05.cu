// Prompt-pass projections on the 5th-generation tensor cores (sm_100a):
//   Y[b][t][o] = sum_k A[t][b*Ka + k] * W[b*rows_b + o][k]     (bf16 x bf16 -> fp32)
// One CTA computes a 128 x BN tile.  Warp 0 streams 128B-swizzled K-major tiles of A and W into a
// shared-memory ring with TMA (cp.async.bulk.tensor, every CTA loading its own tiles), one thread of warp 1 issues
// tcgen05.mma (kind::f16, fp32 accumulator in tensor memory), warps 2-5 read the accumulator back
// with tcgen05.ld and store fp32 rows.  Every wait on an mbarrier is bounded: when a limit runs
// out the kernel writes DEVERR_WAIT_TIMEOUT to the error word, skips its remaining work, frees its
// tensor memory and returns.
#include <stdlib.h>

#include "gemm_tc_common.cuh"

namespace tpi {

namespace {

using namespace tc;

constexpr int kBM = 128;
// tensor-memory columns are allocated in powers of two
__host__ __device__ constexpr uint32_t tmem_cols(int bn) { return bn <= 32 ? 32u : bn <= 64 ? 64u : bn <= 128 ? 128u : 256u; }
// pipeline depth that fits one SM's shared memory
constexpr int stages_for(int bn, int split) {
  const int stage = (1 + split) * kBM * kBK * 2 + bn * kBK * 2;
  const int n = (226 * 1024 - 1024) / stage;
  return n > 8 ? 8 : n;
}

// SPLIT = 1: the activations come as two bf16 tensors, A = A_hi + A_lo (A_lo = bf16(A - A_hi)), and every
// k-block issues the MMAs twice onto the same accumulator.  That keeps ~16 mantissa bits of the fp32
// activations while the weights stay exact bf16; the weight tile in shared memory is shared by both.
//
// n_acc = 2: the first and the second half of the k-blocks accumulate in two accumulators side by side in tensor
// memory, added in fp32 in the epilogue.  The tensor core truncates its fp32 accumulator at every step (16 products),
// so a chain drifts towards zero by about 2^-26 of the sum per step (9.3e-6 of the result at K = 4096 with the two
// products per k-block); two half chains added with round to nearest halve that.  (Four accumulators halve it again
// but take all of tensor memory for tiles of 160 outputs and measured 6 % slower at 128 positions.)
template <int BN, int STAGES, int SPLIT>
__global__ void __launch_bounds__(192) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                      const __grid_constant__ CUtensorMap tmAlo,
                                                      const __grid_constant__ CUtensorMap tmW, const GemmTcArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], acc_ready;
  __shared__ uint32_t tmem_base_s;
  static_assert(BN % 32 == 0 && BN <= 256, "the epilogue reads 32 accumulator columns at a time");
  constexpr uint32_t ACOLS = tmem_cols(BN);  // columns of one accumulator
  const int n_acc = (a.n_acc >= 2 && a.K / kBK >= 2) ? 2 : 1;
  const uint32_t TCOLS = ACOLS * (uint32_t)n_acc;
  constexpr uint32_t A_BYTES = kBM * kBK * 2, B_BYTES = BN * kBK * 2, STAGE_BYTES = (1 + SPLIT) * A_BYTES + B_BYTES;
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * kBM, batch = blockIdx.z;
  const int kblocks = a.K / kBK;
  const int polls = a.wait_polls > 0 ? a.wait_polls : kWaitPolls;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(&acc_ready, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // one warp allocates BN columns of tensor memory for the fp32 accumulator
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(TCOLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_s;
  // set-up above overlaps the previous kernel's tail; the activations it wrote are needed from here on
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0) {
    if (lane == 0 && !a.starve) {  // ---- TMA producer
      for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, a.err, polls)) break;
        uint8_t* sa = smem + (size_t)s * STAGE_BYTES;
        mbar_expect_tx(&full[s], STAGE_BYTES);
        tma_load_2d(sa, &tmA, &full[s], batch * a.a_col_batch + kb * kBK, m0);
        if (SPLIT) tma_load_2d(sa + A_BYTES, &tmAlo, &full[s], batch * a.a_col_batch + kb * kBK, m0);
        tma_load_2d(sa + (1 + SPLIT) * A_BYTES, &tmW, &full[s], kb * kBK, batch * a.w_row_batch + n0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {  // ---- MMA issuer
      // instruction descriptor: D fp32, A and B bf16, both K-major, N = BN, M = 128
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
      bool ok = true;
      const int kb_half = n_acc == 2 ? kblocks / 2 : kblocks;  // the second accumulator takes the k-blocks from here on
      for (int kb = 0; kb < kblocks && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(&full[s], ph, a.err, polls);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d = tmem_acc + (kb >= kb_half ? ACOLS : 0u);
        const bool first = kb == 0 || kb == kb_half;
        const uint32_t sa = smem_u32(smem + (size_t)s * STAGE_BYTES);
        const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + (1 + SPLIT) * A_BYTES);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k)  // 16 bf16 = 32 bytes per step inside the swizzle atom
          umma_bf16(d, da + 2 * k, db + 2 * k, idesc, (!first || k) ? 1u : 0u);
        if (SPLIT) {
          const uint64_t dl = umma_desc_sw128(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) umma_bf16(d, dl + 2 * k, db + 2 * k, idesc, 1u);
        }
        umma_commit(&empty[s]);  // the stage is free once these MMAs have read it
      }
      // after a wait that ran out the accumulator is incomplete: leave acc_ready alone, so that the epilogue's own
      // (bounded) wait runs out too and nothing is read back or stored
      if (ok) umma_commit(&acc_ready);
    }
  } else {  // ---- epilogue: warps 2..5 cover the four 32-lane quarters of tensor memory
    const int q = warp & 3;
    const bool ok = mbar_wait(&acc_ready, 0, a.err, polls);
    tc_fence_after();
    const int row = m0 + q * 32 + lane;
    float* yrow = a.Y + (size_t)batch * a.y_bs + (size_t)row * a.ldy + n0;
    if (ok && kblocks > 0) {
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t r[32];
        if (n_acc == 2) {  // both halves of the contraction: two loads in flight, one wait, first half + second half
          uint32_t r2[32];
          tmem_ld32_nowait(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
          tmem_ld32_nowait(tmem_acc + ((uint32_t)(q * 32) << 16) + ACOLS + (uint32_t)c0, r2);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
        } else {
          tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
        }
        if (row < a.T && a.act) {
          __nv_bfloat16* arow = a.act + (size_t)row * a.act_ld + ((n0 + c0) >> 1);
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int j = 0; j < 32; j += 4) {  // two (gate, up) pairs -> two activations packed in one word
            float v[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const float g = __uint_as_float(r[j + 2 * e]), u = __uint_as_float(r[j + 2 * e + 1]);
              v[e] = g / (1.f + expf(-g)) * u;
            }
            const __nv_bfloat16 h0 = __float2bfloat16_rn(v[0]), h1 = __float2bfloat16_rn(v[1]);
            hi[j >> 2] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
            const __nv_bfloat16 l0 = __float2bfloat16_rn(v[0] - __bfloat162float(h0)),
                                l1 = __float2bfloat16_rn(v[1] - __bfloat162float(h1));
            lo[j >> 2] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
          }
          if (n0 + c0 + 32 <= a.n_out) {
            *reinterpret_cast<uint4*>(arow) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(arow + 8) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
            if (a.act_split) {
              *reinterpret_cast<uint4*>(arow + a.act_lo_off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
              *reinterpret_cast<uint4*>(arow + a.act_lo_off + 8) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
            }
          } else {
            for (int j = 0; j < 16; ++j)
              if (n0 + c0 + 2 * j + 1 < a.n_out) {
                arow[j] = __ushort_as_bfloat16((unsigned short)(hi[j >> 1] >> ((j & 1) * 16)));
                if (a.act_split) arow[a.act_lo_off + j] = __ushort_as_bfloat16((unsigned short)(lo[j >> 1] >> ((j & 1) * 16)));
              }
          }
        } else if (row < a.T) {
          if (n0 + c0 + 32 <= a.n_out) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(yrow + c0 + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                                       __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
          } else {
            for (int j = 0; j < 32; ++j)
              if (n0 + c0 + j < a.n_out) yrow[c0 + j] = __uint_as_float(r[j]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(TCOLS) : "memory");
  }
}

}  // namespace

bool gemm_tc_supported(int K, int a_cols_total, int ldy) {
  return K > 0 && K % kBK == 0 && a_cols_total % 8 == 0 && ldy % 4 == 0;
}

template <int BN, int STAGES, int SPLIT>
static cudaError_t launch_tc_t(const LaunchCtx& c, const CUtensorMap& tmA, const CUtensorMap& tmAlo, const CUtensorMap& tmW,
                               const GemmTcArgs& a, int n_batch) {
  auto kern = gemm_tc_kernel<BN, STAGES, SPLIT>;
  const size_t smem = (size_t)STAGES * ((1 + SPLIT) * kBM * kBK * 2 + BN * kBK * 2) + 1024;
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  if (c.launches) ++*c.launches;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((a.n_out + BN - 1) / BN, (a.T + kBM - 1) / kBM, n_batch);
  cfg.blockDim = dim3(192);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c.stream;
  cudaLaunchAttribute attr[1];
  if (c.pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmAlo, tmW, a);
}

// TPI_GEMM_PAIR=0 in the environment keeps every projection on single-CTA tiles (for comparisons)
static bool gemm_pair_enabled() {
  static int on = -1;
  if (on < 0) {
    const char* e = getenv("TPI_GEMM_PAIR");
    on = !(e && e[0] == '0');
  }
  return on != 0;
}

static cudaError_t launch_gemm_tc_any(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                                      const void* W_bf16, int w_row_batch, float* Y, long long y_batch_stride, int ldy, int T,
                                      int n_out, int K, int n_batch, int* err, void* act, int act_ld, long long act_lo_off,
                                      int act_split, int wait_polls = 0, int starve = 0, bool chunk_k = false) {
  // Tile width: one CTA computes 128 positions x BN outputs and, per 64-wide k-block, pulls the activation tile(s)
  // plus BN weight rows through shared memory; a CTA's ingest rate is what bounds it, so the cost of a choice is
  // (waves of CTAs over the SMs) x (bytes per k-block), and widths that leave SMs idle or spill into another wave lose.
  int nsm = 148, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev);
  static const int cand[4] = {256, 160, 128, 96};  // 112 (148 CTAs for a 4096-wide output x 4 shards) measured slower than 128
  static const double tile_us[4] = {0.97, 0.66, 0.55, 0.47};  // measured per tile and k-block at more than 128 positions
  const long long mt = (T + kBM - 1) / kBM;
  int BN = 128;
  double best = 1e30, best_us = 1e30;
  for (int i = 0; i < 4; ++i) {
    const int bn = cand[i];
    if (act && bn % 32) continue;                 // the SwiGLU epilogue works on 32-column groups
    if (bn > 128 && n_out < bn) continue;
    const long long tiles = (long long)((n_out + bn - 1) / bn) * mt * n_batch;
    const long long waves = (tiles + nsm - 1) / nsm;
    // up to 128 positions a CTA's ingest bounds it: bytes per k-block; beyond, the measured tile times
    const double cost = T <= kBM ? (double)waves * ((A_lo_bf16 ? 2 : 1) * kBM * kBK * 2 + bn * kBK * 2)
                                 : (double)waves * ((K / kBK) * tile_us[i] + 4.0 + bn / 64.0);
    if (cost < best - 1e-9) { best = cost; BN = bn; best_us = cost; }
  }
  // long contractions of the column-sharded projections: chunks of the contraction, added in registers
  if (chunk_k && A_lo_bf16 && n_batch == 1 && gemm_pair_enabled() && !starve &&
      gemm_tc_chunked_supported(T, K, lda, n_out, ldy, act != nullptr))
    return launch_gemm_tc_chunked(c, A_bf16, A_lo_bf16, lda, W_bf16, Y, ldy, T, n_out, K, err, act, act_ld, act_lo_off, act_split);
  if (A_lo_bf16 && T > kBM && gemm_pair_enabled() && !starve) {  // a CTA pair (M = 256) pulls half the weight bytes per MMA
    double pair_us = 0;
    const int shape = gemm_tc_pair_choose(T, n_out, K, n_batch, nsm, &pair_us);
    if (shape >= 0 && pair_us < best_us)
      return launch_gemm_tc_pair(c, shape, A_bf16, A_lo_bf16, lda, a_col_batch, W_bf16, w_row_batch, Y, y_batch_stride, ldy, T,
                                 n_out, K, n_batch, err, act, act_ld, act_lo_off, act_split);
  }
  CUtensorMap tmA, tmAlo, tmW;
  // A: [T][lda] (each batch reads K columns starting at batch * a_col_batch); W: [n_batch * w_row_batch][K]
  if (!make_map(&tmA, A_bf16, (uint64_t)lda, (uint64_t)T, (uint64_t)lda, kBM)) return cudaErrorInvalidValue;
  if (!make_map(&tmAlo, A_lo_bf16 ? A_lo_bf16 : A_bf16, (uint64_t)lda, (uint64_t)T, (uint64_t)lda, kBM)) return cudaErrorInvalidValue;
  const uint64_t w_rows = (uint64_t)(n_batch - 1) * w_row_batch + n_out;
  if (!make_map(&tmW, W_bf16, (uint64_t)K, w_rows, (uint64_t)K, (uint32_t)BN)) return cudaErrorInvalidValue;
  // up to 128 positions no other kernel computes the same outputs, and the contraction is spread over two accumulators
  // whatever the tile width (so the bits do not depend on it); beyond, the single chain that the CTA-pair kernels
  // and the star sum in their epilogue reproduce
  GemmTcArgs a{Y, y_batch_stride, ldy, T, n_out, K, a_col_batch, w_row_batch, err, (__nv_bfloat16*)act, act_lo_off, act_ld, act_split,
               wait_polls, starve, T <= kBM ? 2 : 1};
#define TPI_TC(BNV) \
  return A_lo_bf16 ? launch_tc_t<BNV, stages_for(BNV, 1), 1>(c, tmA, tmAlo, tmW, a, n_batch) \
                   : launch_tc_t<BNV, stages_for(BNV, 0), 0>(c, tmA, tmAlo, tmW, a, n_batch)
  switch (BN) {
    case 256: TPI_TC(256);
    case 160: TPI_TC(160);
    case 96: TPI_TC(96);
    default: TPI_TC(128);
  }
#undef TPI_TC
}

cudaError_t launch_gemm_tc(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                           const void* W_bf16, int w_row_batch, float* Y, long long y_batch_stride, int ldy, int T,
                           int n_out, int K, int n_batch, int* err, bool chunk_k) {
  return launch_gemm_tc_any(c, A_bf16, A_lo_bf16, lda, a_col_batch, W_bf16, w_row_batch, Y, y_batch_stride, ldy, T, n_out, K,
                            n_batch, err, nullptr, 0, 0, 0, 0, 0, chunk_k);
}

cudaError_t launch_gemm_tc_starved(const LaunchCtx& c, const void* A_bf16, int lda, const void* W_bf16, float* Y, int ldy, int T,
                                   int n_out, int K, int* err, int wait_polls) {
  if (wait_polls < 1 || wait_polls > (1 << 16)) return cudaErrorInvalidValue;
  return launch_gemm_tc_any(c, A_bf16, nullptr, lda, 0, W_bf16, n_out, Y, 0, ldy, T, n_out, K, 1, err, nullptr, 0, 0, 0, wait_polls, 1);
}

bool gemm_tc_swiglu_supported(int K, int lda, int s) { return gemm_tc_supported(K, lda, 2 * s) && s % 16 == 0; }

cudaError_t launch_gemm_tc_swiglu(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, const void* Wgu_bf16,
                                  void* ACT, int out_mode, int T, int s, int K, int* err) {
  if (out_mode != 1 && out_mode != 2) return cudaErrorInvalidValue;
  return launch_gemm_tc_any(c, A_bf16, A_lo_bf16, lda, 0, Wgu_bf16, 2 * s, nullptr, 0, 2 * s, T, 2 * s, K, 1, err, ACT, s,
                            (long long)T * s, out_mode == 2, 0, 0, true);
}

}  // namespace tpi
