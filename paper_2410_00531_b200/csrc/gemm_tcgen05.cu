// Prompt-pass projections on the 5th-generation tensor cores (sm_100a):
//   Y[b][t][o] = sum_k A[t][b*Ka + k] * W[b*rows_b + o][k]     (bf16 x bf16 -> fp32)
// One CTA computes a 128 x BN tile.  Warp 0 streams 128B-swizzled K-major tiles of A and W into a
// shared-memory ring with TMA (cp.async.bulk.tensor, no multicast), one thread of warp 1 issues
// tcgen05.mma (kind::f16, fp32 accumulator in tensor memory), warps 2-5 read the accumulator back
// with tcgen05.ld and store fp32 rows.  Every wait on an mbarrier is bounded: when a limit runs
// out the kernel writes DEVERR_WAIT_TIMEOUT to the error word, skips its remaining work, frees its
// tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.h"

namespace tpi {

namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: about a quarter of a second at most, then the error word is set.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* err) {
  for (int i = 0; i < (1 << 21); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 128) __nanosleep(100);
  }
  atomicCAS(err, DEVERR_NONE, DEVERR_WAIT_TIMEOUT);
  return false;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}

// K-major operand tile written by TMA with the 128-byte swizzle: rows of 64 bf16 (128 B), groups of
// 8 rows 1024 B apart.  Descriptor: start address >> 4, leading offset (unused for this layout) 1,
// stride offset 1024 >> 4, version 1 (sm_100), layout type 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct GemmTcArgs {
  float* Y;
  long long y_bs;   // floats between batches of Y
  int ldy, T, n_out, K;
  int a_col_batch;  // A's column offset per batch (elements)
  int w_row_batch;  // W's row offset per batch
  int* err;
  // SwiGLU epilogue (gate/up projection whose output columns are interleaved gate_j, up_j): when act != nullptr
  // nothing is written to Y; act[t][c / 2] = silu(y[t][c]) * y[t][c + 1] goes out as bf16 (hi, and in split mode
  // lo = bf16(v - hi) act_lo_off elements further), row stride act_ld.
  __nv_bfloat16* act;
  long long act_lo_off;
  int act_ld, act_split;
};

constexpr int kBM = 128, kBK = 64;
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
template <int BN, int STAGES, int SPLIT>
__global__ void __launch_bounds__(192) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                      const __grid_constant__ CUtensorMap tmAlo,
                                                      const __grid_constant__ CUtensorMap tmW, const GemmTcArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], acc_ready;
  __shared__ uint32_t tmem_base_s;
  static_assert(BN % 32 == 0 && BN <= 256, "the epilogue reads 32 accumulator columns at a time");
  constexpr uint32_t TCOLS = tmem_cols(BN);
  constexpr uint32_t A_BYTES = kBM * kBK * 2, B_BYTES = BN * kBK * 2, STAGE_BYTES = (1 + SPLIT) * A_BYTES + B_BYTES;
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * kBM, batch = blockIdx.z;
  const int kblocks = a.K / kBK;

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
    if (lane == 0) {  // ---- TMA producer
      for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, a.err)) break;
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
      for (int kb = 0; kb < kblocks && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(&full[s], ph, a.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + (size_t)s * STAGE_BYTES);
        const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + (1 + SPLIT) * A_BYTES);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k)  // 16 bf16 = 32 bytes per step inside the swizzle atom
          umma_bf16(tmem_acc, da + 2 * k, db + 2 * k, idesc, (kb | k) ? 1u : 0u);
        if (SPLIT) {
          const uint64_t dl = umma_desc_sw128(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) umma_bf16(tmem_acc, dl + 2 * k, db + 2 * k, idesc, 1u);
        }
        umma_commit(&empty[s]);  // the stage is free once these MMAs have read it
      }
      umma_commit(&acc_ready);
    }
  } else {  // ---- epilogue: warps 2..5 cover the four 32-lane quarters of tensor memory
    const int q = warp & 3;
    const bool ok = mbar_wait(&acc_ready, 0, a.err);
    tc_fence_after();
    const int row = m0 + q * 32 + lane;
    float* yrow = a.Y + (size_t)batch * a.y_bs + (size_t)row * a.ldy + n0;
    if (ok && kblocks > 0) {
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// 2-D bf16 tensor [rows][cols] with row stride ld elements; box = 64 columns x box_rows rows, 128B swizzle.
bool make_map(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t ld, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {kBK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
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
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done = true;
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

static cudaError_t launch_gemm_tc_any(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                                      const void* W_bf16, int w_row_batch, float* Y, long long y_batch_stride, int ldy, int T,
                                      int n_out, int K, int n_batch, int* err, void* act, int act_ld, long long act_lo_off,
                                      int act_split) {
  // Tile width: one CTA computes 128 positions x BN outputs and, per 64-wide k-block, pulls the activation tile(s)
  // plus BN weight rows through shared memory; a CTA's ingest rate is what bounds it, so the cost of a choice is
  // (waves of CTAs over the SMs) x (bytes per k-block), and widths that leave SMs idle or spill into another wave lose.
  int nsm = 148, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev);
  static const int cand[4] = {256, 160, 128, 96};  // 112 (148 CTAs for a 4096-wide output x 4 shards) measured slower than 128
  const long long mt = (T + kBM - 1) / kBM;
  int BN = 128;
  double best = 1e30;
  for (int i = 0; i < 4; ++i) {
    const int bn = cand[i];
    if (act && bn % 32) continue;                 // the SwiGLU epilogue works on 32-column groups
    if (bn > 128 && n_out < bn) continue;
    const long long tiles = (long long)((n_out + bn - 1) / bn) * mt * n_batch;
    const long long waves = (tiles + nsm - 1) / nsm;
    const double cost = (double)waves * ((A_lo_bf16 ? 2 : 1) * kBM * kBK * 2 + bn * kBK * 2);
    if (cost < best - 1e-9) { best = cost; BN = bn; }
  }
  CUtensorMap tmA, tmAlo, tmW;
  // A: [T][lda] (each batch reads K columns starting at batch * a_col_batch); W: [n_batch * w_row_batch][K]
  if (!make_map(&tmA, A_bf16, (uint64_t)lda, (uint64_t)T, (uint64_t)lda, kBM)) return cudaErrorInvalidValue;
  if (!make_map(&tmAlo, A_lo_bf16 ? A_lo_bf16 : A_bf16, (uint64_t)lda, (uint64_t)T, (uint64_t)lda, kBM)) return cudaErrorInvalidValue;
  const uint64_t w_rows = (uint64_t)(n_batch - 1) * w_row_batch + n_out;
  if (!make_map(&tmW, W_bf16, (uint64_t)K, w_rows, (uint64_t)K, (uint32_t)BN)) return cudaErrorInvalidValue;
  GemmTcArgs a{Y, y_batch_stride, ldy, T, n_out, K, a_col_batch, w_row_batch, err, (__nv_bfloat16*)act, act_lo_off, act_ld, act_split};
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
                           int n_out, int K, int n_batch, int* err) {
  return launch_gemm_tc_any(c, A_bf16, A_lo_bf16, lda, a_col_batch, W_bf16, w_row_batch, Y, y_batch_stride, ldy, T, n_out, K,
                            n_batch, err, nullptr, 0, 0, 0);
}

bool gemm_tc_swiglu_supported(int K, int lda, int s) { return gemm_tc_supported(K, lda, 2 * s) && s % 16 == 0; }

cudaError_t launch_gemm_tc_swiglu(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, const void* Wgu_bf16,
                                  void* ACT, int out_mode, int T, int s, int K, int* err) {
  if (out_mode != 1 && out_mode != 2) return cudaErrorInvalidValue;
  return launch_gemm_tc_any(c, A_bf16, A_lo_bf16, lda, 0, Wgu_bf16, 2 * s, nullptr, 0, 2 * s, T, 2 * s, K, 1, err, ACT, s,
                            (long long)T * s, out_mode == 2);
}

}  // namespace tpi
