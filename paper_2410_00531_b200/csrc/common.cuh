// Device-side helpers shared by the kernels of this library (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.h"

namespace tpi {

// Device-side timeline of the decode kernels (builds with -DTPI_TIMELINE only; compiled out otherwise): a CTA stamps
// the global nanosecond timer when it starts, when its dependency wait returns, when its inputs are staged and when
// each of its warps ends, into a caller-provided buffer [TL_KERNELS][TL_CTAS][TL_SLOTS] of 64-bit words.  Each launch
// of a kernel overwrites the stamps of the launch before, so after a run the buffer holds the LAST layer's kernels:
// one layer's schedule under graph replay with programmatic dependent launch, gaps between kernels included.
#ifdef TPI_TIMELINE
static __device__ unsigned long long* g_tl;  // one copy per translation unit, all set by set_timeline_*()
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define TL(id, cta, slot)                                                                              \
  do {                                                                                                 \
    if (g_tl && (cta) < TL_CTAS) {                                                                     \
      g_tl[((id) * TL_CTAS + (cta)) * TL_SLOTS + (slot)] = global_ns();                                \
      if ((slot) == TL_ENTRY) {  /* which SM runs this CTA (slow SMs show up as late CTAs) */          \
        unsigned sm_;                                                                                  \
        asm volatile("mov.u32 %0, %%smid;" : "=r"(sm_));                                               \
        g_tl[((id) * TL_CTAS + (cta)) * TL_SLOTS + TL_SMID] = sm_ + 1;                                 \
      }                                                                                                \
    }                                                                                                  \
  } while (0)
#else
#define TL(id, cta, slot) do {} while (0)
#endif
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// 16-byte streaming load of read-only weights: no L1 allocation, each byte is used once.
__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];"
      : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
      : "l"(p));
  return v;
}
// 16-byte load through L2 only (data written by another CTA of the same grid)
__device__ __forceinline__ float ld_cg(const float* p) { return __ldcg(p); }

// Ask L2 to fetch [p, p+bytes) ahead of use (bytes: multiple of 16, p 16-byte aligned).
__device__ __forceinline__ void l2_prefetch_bulk(const void* p, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Storage element traits: how many elements a 16-byte vector holds and how to
// accumulate vector * x[0..VEC) into acc.
template <typename T>
struct Elem;
template <>
struct Elem<float> {
  static constexpr int VEC = 4;
  // fp32 weights are held to 1e-5 against an fp64 oracle over a whole network: a lane's running sum over hundreds of
  // products would alone lose ~1e-6 per projection.  The four products of one vector are summed in fp32 and the
  // vectors in fp64 (free in a kernel that waits for HBM); the result is rounded to fp32 once, after the warp's sum.
  using Acc = double;
  static __device__ __forceinline__ double dot(uint4 w, const float* x, double acc) {
    const float4 a = *reinterpret_cast<const float4*>(x);
    float p = __uint_as_float(w.x) * a.x;
    p = fmaf(__uint_as_float(w.y), a.y, p);
    p = fmaf(__uint_as_float(w.z), a.z, p);
    p = fmaf(__uint_as_float(w.w), a.w, p);
    return acc + (double)p;
  }
  static __device__ __forceinline__ void unpack(uint4 w, float* f) {
    f[0] = __uint_as_float(w.x); f[1] = __uint_as_float(w.y);
    f[2] = __uint_as_float(w.z); f[3] = __uint_as_float(w.w);
  }
  static __device__ __forceinline__ float load(const float* p) { return *p; }
  static __device__ __forceinline__ void store(float* p, float v) { *p = v; }
};
template <>
struct Elem<__nv_bfloat16> {
  static constexpr int VEC = 8;
  using Acc = float;
  static __device__ __forceinline__ float dot(uint4 w, const float* x, float acc) {
    const float4 a = *reinterpret_cast<const float4*>(x);
    const float4 b = *reinterpret_cast<const float4*>(x + 4);
    acc = fmaf(bf16lo(w.x), a.x, acc);
    acc = fmaf(bf16hi(w.x), a.y, acc);
    acc = fmaf(bf16lo(w.y), a.z, acc);
    acc = fmaf(bf16hi(w.y), a.w, acc);
    acc = fmaf(bf16lo(w.z), b.x, acc);
    acc = fmaf(bf16hi(w.z), b.y, acc);
    acc = fmaf(bf16lo(w.w), b.z, acc);
    acc = fmaf(bf16hi(w.w), b.w, acc);
    return acc;
  }
  static __device__ __forceinline__ void unpack(uint4 w, float* f) {
    f[0] = bf16lo(w.x); f[1] = bf16hi(w.x); f[2] = bf16lo(w.y); f[3] = bf16hi(w.y);
    f[4] = bf16lo(w.z); f[5] = bf16hi(w.z); f[6] = bf16lo(w.w); f[7] = bf16hi(w.w);
  }
  static __device__ __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, float v) {
    *p = __float2bfloat16_rn(v);  // round to nearest even: the KV cache's storage rounding
  }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
// the same tree in fp64, rounded to fp32 at the end (the fp32-weight GEMVs)
__device__ __forceinline__ float warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return (float)v;
}

// Sum over a block in a fixed order (warp trees, then warp 0 over the per-warp sums).
// scratch: >= 32 floats of shared memory.  Every thread gets the result.
__device__ __forceinline__ float block_sum(float v, float* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float t = (lane < nwarp) ? scratch[lane] : 0.f;
  t = warp_sum(t);
  return t;
}

}  // namespace tpi
