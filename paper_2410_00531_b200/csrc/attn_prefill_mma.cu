// Causal attention of the prompt pass on tensor cores (bf16 KV cache): Eq. 1's softmax(QK^T/sqrt d)V for
// T query positions at once.  One CTA = 64 queries of one head (4 warps x 16 rows); keys are walked in
// tiles of 64 staged in shared memory (cp.async, two stages, XOR-swizzled 16-byte chunks); S = QK^T and
// O += PV run on mma.sync m16n8k16 (bf16 inputs, fp32 accumulate) with an online softmax in between.
// K and V are exact bf16 (the cache's storage type); the fp32 queries and the softmax weights are each
// split into bf16 hi + lo and multiplied twice, so the result keeps fp32-level accuracy.
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "kernels.h"
#include "launch.cuh"

namespace tpi {
#ifdef TPI_TIMELINE
void set_timeline_attn(void* dev_buf) { cudaMemcpyToSymbol(g_tl, &dev_buf, sizeof dev_buf); }
#endif

namespace {

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// (x, y) -> packed bf16 pair of the rounded values, and the pair of the remainders
__device__ __forceinline__ void split_pack(float x, float y, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 hx = __float2bfloat16_rn(x), hy = __float2bfloat16_rn(y);
  const __nv_bfloat162 h = __halves2bfloat162(hx, hy);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - __bfloat162float(hx), y - __bfloat162float(hy));
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

template <int MODE>
__device__ __forceinline__ void store_out(void* base, size_t i, size_t lo_off, float v) {
  if (MODE == 0) reinterpret_cast<float*>(base)[i] = v;
  else {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    reinterpret_cast<__nv_bfloat16*>(base)[i] = hi;
    if (MODE == 2) reinterpret_cast<__nv_bfloat16*>(base)[lo_off + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
  }
}

constexpr int KB = 64;  // keys per tile of the prompt kernel
// decode kernel: DW warps per CTA, each takes DKB-key tiles (shorter tiles, more warps: a shorter dependent MMA chain per warp)
constexpr int DW = 8, DKB = 32;

// byte offset of 16-byte chunk c of row r in a tile whose rows hold D bf16 (chunks XOR-swizzled in groups of 8)
template <int D>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return (uint32_t)(r * (D * 2) + (((c & ~7) | ((c ^ r) & 7)) << 4));
}

// QBT queries per CTA (16 per warp): 64, or 32 when 64-query tiles would leave most of the machine idle
template <int D, int MODE, int QBT>
__global__ void __launch_bounds__(QBT * 2) prefill_attn_mma_kernel(const float* __restrict__ Q, const __nv_bfloat16* kc,
                                                               const __nv_bfloat16* vc, int T, int pos0, int a, int b,
                                                               int max_seq, void* O, size_t lo_off) {
  constexpr int KS = D / 16;       // k-steps of the QK^T contraction
  constexpr int ND = D / 8;        // 8-wide output blocks of O
  constexpr int CPR = D / 8;       // 16-byte chunks per row
  constexpr int TILE = KB * D * 2; // bytes of one K (or V) tile
  extern __shared__ __align__(128) uint8_t smem[];  // [2 stages][K tile | V tile]
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int j = blockIdx.y, kvh = j / (a / b);
  const int q0 = blockIdx.x * QBT;                      // first query row of the CTA
  const int row_lo = q0 + warp * 16 + g, row_hi = row_lo + 8;
  const int n_keys = min(pos0 + min(q0 + QBT, T), pos0 + T);  // keys any row of this CTA may see
  const __nv_bfloat16* kg = kc + (size_t)kvh * max_seq * D;
  const __nv_bfloat16* vg = vc + (size_t)kvh * max_seq * D;
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);

  auto stage_tile = [&](int stage, int k0) {
    // 64 rows x CPR chunks for K and for V; rows beyond the cache's valid range are zero-filled
    for (int i = threadIdx.x; i < KB * CPR; i += QBT * 2) {
      const int r = i / CPR, c = i - r * CPR;
      const uint32_t dk = smem_base + stage * 2 * TILE + tile_off<D>(r, c);
      const uint32_t dv = dk + TILE;
      if (k0 + r < n_keys) {
        const size_t src = (size_t)(k0 + r) * D + c * 8;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dk), "l"(kg + src) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dv), "l"(vg + src) : "memory");
      } else {
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(dk), "r"(0u) : "memory");
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(dv), "r"(0u) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  // ---- Q fragments (scaled into the log2 domain, split hi/lo)
  const float qscale = 1.4426950408889634f * rsqrtf((float)D);
  uint32_t qh[KS][4], ql[KS][4];
  {
    const float* q_lo = Q + ((size_t)min(row_lo, T - 1) * a + j) * D;
    const float* q_hi = Q + ((size_t)min(row_hi, T - 1) * a + j) * D;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const float2 v0 = *reinterpret_cast<const float2*>(q_lo + ks * 16 + 2 * t);
      const float2 v1 = *reinterpret_cast<const float2*>(q_hi + ks * 16 + 2 * t);
      const float2 v2 = *reinterpret_cast<const float2*>(q_lo + ks * 16 + 8 + 2 * t);
      const float2 v3 = *reinterpret_cast<const float2*>(q_hi + ks * 16 + 8 + 2 * t);
      split_pack(v0.x * qscale, v0.y * qscale, qh[ks][0], ql[ks][0]);
      split_pack(v1.x * qscale, v1.y * qscale, qh[ks][1], ql[ks][1]);
      split_pack(v2.x * qscale, v2.y * qscale, qh[ks][2], ql[ks][2]);
      split_pack(v3.x * qscale, v3.y * qscale, qh[ks][3], ql[ks][3]);
    }
  }
  float o[ND][4];
#pragma unroll
  for (int nd = 0; nd < ND; ++nd) { o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  const int qpos_lo = pos0 + row_lo, qpos_hi = pos0 + row_hi;

  const int n_tiles = (n_keys + KB - 1) / KB;
  stage_tile(0, 0);
  for (int kt = 0; kt < n_tiles; ++kt) {
    const int k0 = kt * KB, stage = kt & 1;
    if (kt + 1 < n_tiles) {
      stage_tile(stage ^ 1, k0 + KB);  // next tile streams in while this one is used
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const uint32_t ks_base = smem_base + stage * 2 * TILE, vs_base = ks_base + TILE;

    // ---- S = Q K^T for this warp's 16 rows x 64 keys
    float s[KB / 8][4];
#pragma unroll
    for (int nb = 0; nb < KB / 8; ++nb) {
      s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
        uint32_t kb[4];
        ldsm_x4(kb, ks_base + tile_off<D>(nb * 8 + (lane & 7), ks * 2 + (lane >> 3)));
        mma_bf16(s[nb], qh[ks], kb[0], kb[1]);
        mma_bf16(s[nb], ql[ks], kb[0], kb[1]);
        mma_bf16(s[nb], qh[ks + 1], kb[2], kb[3]);
        mma_bf16(s[nb], ql[ks + 1], kb[2], kb[3]);
      }
    }
    // ---- causal mask + online softmax (rows g and g + 8 of the warp's block)
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < KB / 8; ++nb) {
      const int key = k0 + nb * 8 + 2 * t;
      if (key > qpos_lo) s[nb][0] = -INFINITY;
      if (key + 1 > qpos_lo) s[nb][1] = -INFINITY;
      if (key > qpos_hi) s[nb][2] = -INFINITY;
      if (key + 1 > qpos_hi) s[nb][3] = -INFINITY;
      mx_lo = fmaxf(mx_lo, fmaxf(s[nb][0], s[nb][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[nb][2], s[nb][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xFFFFFFFFu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xFFFFFFFFu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xFFFFFFFFu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xFFFFFFFFu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float ref_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, ref_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
    const float sc_lo = exp2f(m_lo - ref_lo), sc_hi = exp2f(m_hi - ref_hi);
    m_lo = mn_lo;
    m_hi = mn_hi;
    l_lo *= sc_lo;
    l_hi *= sc_hi;
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) { o[nd][0] *= sc_lo; o[nd][1] *= sc_lo; o[nd][2] *= sc_hi; o[nd][3] *= sc_hi; }
    uint32_t ph[KB / 16][4], pl[KB / 16][4];  // P as A-operand fragments: k-step kk covers key blocks 2kk, 2kk+1
#pragma unroll
    for (int nb = 0; nb < KB / 8; ++nb) {
      const float p0 = exp2f(s[nb][0] - ref_lo), p1 = exp2f(s[nb][1] - ref_lo);
      const float p2 = exp2f(s[nb][2] - ref_hi), p3 = exp2f(s[nb][3] - ref_hi);
      l_lo += p0 + p1;
      l_hi += p2 + p3;
      const int kk = nb >> 1, half = nb & 1;
      split_pack(p0, p1, ph[kk][half * 2 + 0], pl[kk][half * 2 + 0]);
      split_pack(p2, p3, ph[kk][half * 2 + 1], pl[kk][half * 2 + 1]);
    }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < KB / 16; ++kk) {
#pragma unroll
      for (int nd = 0; nd < ND; nd += 2) {
        uint32_t vb[4];
        ldsm_x4_trans(vb, vs_base + tile_off<D>(kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), nd + (lane >> 4)));
        mma_bf16(o[nd], ph[kk], vb[0], vb[1]);
        mma_bf16(o[nd], pl[kk], vb[0], vb[1]);
        mma_bf16(o[nd + 1], ph[kk], vb[2], vb[3]);
        mma_bf16(o[nd + 1], pl[kk], vb[2], vb[3]);
      }
    }
    __syncthreads();  // the stage is overwritten two iterations from now
  }
  // ---- normalise and store
  l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 2);
  const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
#pragma unroll
  for (int nd = 0; nd < ND; ++nd) {
    const int col = nd * 8 + 2 * t;
    if (row_lo < T) {
      const size_t i = ((size_t)row_lo * a + j) * D + col;
      store_out<MODE>(O, i, lo_off, o[nd][0] * inv_lo);
      store_out<MODE>(O, i + 1, lo_off, o[nd][1] * inv_lo);
    }
    if (row_hi < T) {
      const size_t i = ((size_t)row_hi * a + j) * D + col;
      store_out<MODE>(O, i, lo_off, o[nd][2] * inv_hi);
      store_out<MODE>(O, i + 1, lo_off, o[nd][3] * inv_hi);
    }
  }
}

template <int D, int MODE, int QBT>
cudaError_t launch_tq(const LaunchCtx& c, const float* Q, const void* kc, const void* vc, int T, int pos0, int a, int b,
                      int max_seq, void* O) {
  auto kern = prefill_attn_mma_kernel<D, MODE, QBT>;
  const size_t smem = (size_t)2 * 2 * KB * D * 2;
  static PerDeviceOnce attr_done;
  if (!attr_done.get() && smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  return launch_kernel(c, kern, dim3((T + QBT - 1) / QBT, a), dim3(QBT * 2), smem, Q, (const __nv_bfloat16*)kc,
                       (const __nv_bfloat16*)vc, T, pos0, a, b, max_seq, O, (size_t)T * a * D);
}

template <int D, int MODE>
cudaError_t launch_t(const LaunchCtx& c, const float* Q, const void* kc, const void* vc, int T, int pos0, int a, int b,
                     int max_seq, void* O) {
  // 64-query tiles unless they would fill less than one CTA per SM: then 32-query tiles (twice the CTAs, half the
  // serial work of each; a row's arithmetic does not depend on the tile it sits in, so the bits are the same)
  int sms = 148, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if ((long long)((T + 63) / 64) * a < sms) return launch_tq<D, MODE, 32>(c, Q, kc, vc, T, pos0, a, b, max_seq, O);
  return launch_tq<D, MODE, 64>(c, Q, kc, vc, T, pos0, a, b, max_seq, O);
}

}  // namespace

// =====================================================================================================
// Decode attention on tensor cores: one query position, the GRP query heads of a kv head are the rows
// (padded to 16) of the same m16n8k16 tiles.  Grid (kv head, split); the 8 warps of a CTA take 32 keys each per
// round of the split, staged in shared memory as two 16-key half tiles with a buffer each.  A split of one round
// (256 positions) requests both halves up front and multiplies them in one step; longer splits (chosen so that the
// grid stays within one wave of CTAs: at most SMs / kv heads splits per head) pipeline the halves, the one after
// next loading while one is multiplied.  Then the CTA folds the warps' partial results, and the last split of a kv
// head to finish merges the splits in split order.
// =====================================================================================================
namespace {

template <int D>
__global__ void __launch_bounds__(DW * 32) decode_attn_mma_kernel(const float* __restrict__ q, const __nv_bfloat16* kc,
                                                              const __nv_bfloat16* vc, const int* pos, int grp,
                                                              int max_seq, int nsplit, int max_sph, float* scratch,
                                                              unsigned* tickets, float* o_out) {
  constexpr int KB = DKB;  // keys per warp and round: two halves of HK keys, each in its own buffer
  constexpr int HK = KB / 2;
  constexpr int KS = D / 16, ND = D / 8, CPR = D / 8, TILE = KB * D * 2, HALF = HK * D * 2;
  extern __shared__ __align__(128) uint8_t smem[];  // [DW warps][K tile | V tile], reused by the merge buffers
  __shared__ bool s_last;
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int kvh = blockIdx.x, split = blockIdx.y;
  if (threadIdx.x == 0) TL(TL_ID_ATTN, blockIdx.x + gridDim.x * blockIdx.y, TL_ENTRY);
  // The position counter was advanced by the previous token's task head, and the embedding kernel that opens a step
  // lets no later kernel of the step start before that head has completed; only the cache row of the newest position
  // (and the queries) come from the kernel just before this one.  Read through L2: the line may sit stale in this
  // SM's L1 from the step before.
  const int n = __ldcg(pos) + 1;
  // splits of at least 256 positions, and no more of them per kv head than keeps the grid within one wave of CTAs
  // (max_sph): a warp then walks several rounds of its split, the next half tile loading while one is multiplied
  const int lim = max(1, min(nsplit, max_sph));
  int chunk = (n + lim - 1) / lim;
  chunk = max(256, (chunk + 63) & ~63);
  const int nact = (n + chunk - 1) / chunk;
  if (split >= nact) return;  // this split sees no position (its ticket is not counted)
  const int s0 = split * chunk, s1 = min(n, s0 + chunk);
  const __nv_bfloat16* kg = kc + (size_t)kvh * max_seq * D;
  const __nv_bfloat16* vg = vc + (size_t)kvh * max_seq * D;
  // per warp: two buffers, each a K half tile and a V half tile of HK rows (64-byte-swizzled 16-byte chunks)
  const uint32_t my_base = (uint32_t)__cvta_generic_to_shared(smem) + warp * 2 * TILE;
  // half h of this warp: round h / 2 of the split (DW * KB keys per round), first or second HK keys of the warp's KB
  auto half_k0 = [&](int hI) { return s0 + (hI >> 1) * (DW * KB) + warp * KB + (hI & 1) * HK; };
  auto issue_half = [&](int hI) {  // always commits a group, so that "all but the newest group" means "half h landed"
    const int k0 = half_k0(hI);
    const uint32_t bk = my_base + (uint32_t)(hI & 1) * 2 * HALF, bv = bk + HALF;
    if (k0 < s1 || hI < 2) {  // the first two halves are always defined (zeros past the split's end)
      for (int i = lane; i < HK * CPR; i += 32) {
        const int r = i / CPR, c = i - r * CPR;
        const uint32_t off = tile_off<D>(r, c);
        if (k0 + r < s1) {
          const size_t src = (size_t)(k0 + r) * D + c * 8;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(bk + off), "l"(kg + src) : "memory");
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(bv + off), "l"(vg + src) : "memory");
        } else {
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(bk + off), "r"(0u) : "memory");
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(bv + off), "r"(0u) : "memory");
        }
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // halves of older positions only are requested ahead of the dependency wait (the newest row comes from the kernel before)
  const bool early0 = half_k0(0) + HK <= n - 1, early1 = half_k0(1) + HK <= n - 1;
  if (early0) issue_half(0);
  if (early0 && early1) issue_half(1);
  pdl_wait();
  if (threadIdx.x == 0) TL(TL_ID_ATTN, blockIdx.x + gridDim.x * blockIdx.y, TL_WAIT);
  if (!early0) issue_half(0);
  if (!(early0 && early1)) issue_half(1);

  // Q fragments: row g = head g of the group (rows >= grp and rows 8..15 are zero)
  const float qscale = 1.4426950408889634f * rsqrtf((float)D);
  uint32_t qh[KS][4], ql[KS][4];
  {
    const float* qrow = q + (size_t)(kvh * grp + min(g, grp - 1)) * D;
    const float on = g < grp ? qscale : 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const float2 v0 = *reinterpret_cast<const float2*>(qrow + ks * 16 + 2 * t);
      const float2 v2 = *reinterpret_cast<const float2*>(qrow + ks * 16 + 8 + 2 * t);
      split_pack(v0.x * on, v0.y * on, qh[ks][0], ql[ks][0]);
      split_pack(v2.x * on, v2.y * on, qh[ks][2], ql[ks][2]);
      qh[ks][1] = ql[ks][1] = qh[ks][3] = ql[ks][3] = 0u;
    }
  }
  float o[ND][4];
#pragma unroll
  for (int nd = 0; nd < ND; ++nd) { o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f; }
  float m_r = -INFINITY, l_r = 0.f;

  // NH half tiles (buffers hI & 1, (hI + 1) & 1) as one step of the online softmax: scores, weights, O += P V
  auto step = [&](auto nh_c, int hI) {
    constexpr int NH = decltype(nh_c)::value, NK = NH * HK;
    const int k0 = half_k0(hI);
    float s[NK / 8][4];
#pragma unroll
    for (int nb = 0; nb < NK / 8; ++nb) {
      const uint32_t my_k = my_base + (uint32_t)((hI + nb / (HK / 8)) & 1) * 2 * HALF;
      s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
        uint32_t kb[4];
        ldsm_x4(kb, my_k + tile_off<D>((nb % (HK / 8)) * 8 + (lane & 7), ks * 2 + (lane >> 3)));
        mma_bf16(s[nb], qh[ks], kb[0], kb[1]);
        mma_bf16(s[nb], ql[ks], kb[0], kb[1]);
        mma_bf16(s[nb], qh[ks + 1], kb[2], kb[3]);
        mma_bf16(s[nb], ql[ks + 1], kb[2], kb[3]);
      }
    }
    float mx = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < NK / 8; ++nb) {
      const int key = k0 + nb * 8 + 2 * t;  // the NH halves cover NK consecutive keys
      if (key >= s1) s[nb][0] = -INFINITY;
      if (key + 1 >= s1) s[nb][1] = -INFINITY;
      mx = fmaxf(mx, fmaxf(s[nb][0], s[nb][1]));
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
    const float mn = fmaxf(m_r, mx);  // finite: the step's first key is valid
    const float sc = exp2f(m_r - mn);
    m_r = mn;
    l_r *= sc;
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) { o[nd][0] *= sc; o[nd][1] *= sc; }
    uint32_t ph[NK / 16][4], pl[NK / 16][4];
#pragma unroll
    for (int nb = 0; nb < NK / 8; ++nb) {
      const float p0 = exp2f(s[nb][0] - mn), p1 = exp2f(s[nb][1] - mn);
      l_r += p0 + p1;
      const int kk = nb >> 1, half = nb & 1;
      split_pack(p0, p1, ph[kk][half * 2], pl[kk][half * 2]);
      ph[kk][half * 2 + 1] = pl[kk][half * 2 + 1] = 0u;
    }
#pragma unroll
    for (int kk = 0; kk < NK / 16; ++kk) {
      const uint32_t my_v = my_base + (uint32_t)((hI + kk / (HK / 16)) & 1) * 2 * HALF + HALF;
#pragma unroll
      for (int nd = 0; nd < ND; nd += 2) {
        uint32_t vb[4];
        ldsm_x4_trans(vb, my_v + tile_off<D>((kk % (HK / 16)) * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), nd + (lane >> 4)));
        mma_bf16(o[nd], ph[kk], vb[0], vb[1]);
        mma_bf16(o[nd], pl[kk], vb[0], vb[1]);
        mma_bf16(o[nd + 1], ph[kk], vb[2], vb[3]);
        mma_bf16(o[nd + 1], pl[kk], vb[2], vb[3]);
      }
    }
  };
  if (chunk <= DW * KB) {  // one round per warp: both halves were requested up front and make one step
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncwarp();
    if (half_k0(0) < s1) step(std::integral_constant<int, 2>{}, 0);
  } else {
    for (int hI = 0; half_k0(hI) < s1; ++hI) {  // several rounds: halves hI and hI + 1 are in flight
      asm volatile("cp.async.wait_group 1;" ::: "memory");
      __syncwarp();
      step(std::integral_constant<int, 1>{}, hI);
      __syncwarp();        // every lane is done reading this buffer
      issue_half(hI + 2);  // the half after next goes into it
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  l_r += __shfl_xor_sync(0xFFFFFFFFu, l_r, 1);
  l_r += __shfl_xor_sync(0xFFFFFFFFu, l_r, 2);

  // ---- fold the 4 warps (fixed order).  Buffers alias the tiles, so everyone must be done reading them.
  __syncthreads();
  float* w_m = reinterpret_cast<float*>(smem);  // [DW][8]
  float* w_l = w_m + DW * 8;                    // [DW][8]
  float* w_o = w_l + DW * 8;                    // [DW][8][D]
  float* mw = w_o + DW * 8 * D;                 // [grp][nsplit] weights of the final merge
  if (t == 0) { w_m[warp * 8 + g] = m_r; w_l[warp * 8 + g] = l_r; }
#pragma unroll
  for (int nd = 0; nd < ND; ++nd) {
    w_o[(warp * 8 + g) * D + nd * 8 + 2 * t] = o[nd][0];
    w_o[(warp * 8 + g) * D + nd * 8 + 2 * t + 1] = o[nd][1];
  }
  __syncthreads();
  float* part = scratch + ((size_t)kvh * nsplit + split) * grp * (D + 2);
  for (int e = threadIdx.x; e < grp * D; e += DW * 32) {
    const int hh = e / D, dd = e - hh * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < DW; ++w) M = fmaxf(M, w_m[w * 8 + hh]);
    float A = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < DW; ++w) {
      const float sc = exp2f(w_m[w * 8 + hh] - M);  // a warp that saw no tile has m = -inf, weight 0
      A = fmaf(sc, w_o[(w * 8 + hh) * D + dd], A);
      L = fmaf(sc, w_l[w * 8 + hh], L);
    }
    if (nact == 1) {
      o_out[(size_t)(kvh * grp + hh) * D + dd] = A / L;  // a single split is the answer
    } else {
      part[hh * (D + 2) + 2 + dd] = A;
      if (dd == 0) { part[hh * (D + 2)] = M; part[hh * (D + 2) + 1] = L; }
    }
  }
  if (threadIdx.x == 0) TL(TL_ID_ATTN, blockIdx.x + gridDim.x * blockIdx.y, TL_WARP0);
  if (nact == 1) return;
  // One thread publishes the CTA's partial results (the barrier orders every thread's stores before its fence, the
  // fence before the ticket) and, in the CTA that arrives last, fences again before the barrier that lets the other
  // threads read the other splits' results through L2: one fence per CTA on either side instead of one per thread.
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned tk = atomicAdd(tickets + kvh, 1u);
    s_last = (tk == (unsigned)nact - 1);
    __threadfence();
  }
  __syncthreads();
  if (!s_last) return;
  const float* pg = scratch + (size_t)kvh * nsplit * grp * (D + 2);
  constexpr int MAXN = 24, EPT = 2;  // register path: up to MAXN splits, up to EPT outputs per thread
  if (nact <= MAXN && grp * D <= EPT * DW * 32) {
    // Few splits: every thread requests the partial values of its own outputs straight away (independent loads, one
    // trip to L2) while the first warps turn the splits' maxima and sums into merge weights; then the weighted sums.
    float v[EPT][MAXN];
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
      const int e = threadIdx.x + j * DW * 32;
      const int hh = e / D, dd = e - hh * D;
#pragma unroll
      for (int sI = 0; sI < MAXN; ++sI)
        if (e < grp * D && sI < nact) v[j][sI] = __ldcg(pg + (size_t)(sI * grp + hh) * (D + 2) + 2 + dd);
    }
    for (int hh = warp; hh < grp; hh += DW) {
      const float m_s = lane < nact ? __ldcg(pg + (size_t)(lane * grp + hh) * (D + 2)) : -INFINITY;  // nact <= 24 < 32 lanes
      const float l_s = lane < nact ? __ldcg(pg + (size_t)(lane * grp + hh) * (D + 2) + 1) : 0.f;
      float M = m_s;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, off));
      const float w = lane < nact ? exp2f(m_s - M) : 0.f;
      const float L = warp_sum(w * l_s);
      if (lane < nact) mw[hh * nact + lane] = w / L;
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
      const int e = threadIdx.x + j * DW * 32;
      if (e < grp * D) {
        const int hh = e / D, dd = e - hh * D;
        float A = 0.f;
#pragma unroll
        for (int sI = 0; sI < MAXN; ++sI)
          if (sI < nact) A = fmaf(mw[hh * nact + sI], v[j][sI], A);
        o_out[(size_t)(kvh * grp + hh) * D + dd] = A;
      }
    }
    if (threadIdx.x == 0) tickets[kvh] = 0u;
    if (threadIdx.x == 0) TL(TL_ID_ATTN, blockIdx.x + gridDim.x * blockIdx.y, TL_WARP0 + 1);  // merge done
    return;
  }
  // All partial results of this kv head come into shared memory in one batch of independent loads (one trip to L2
  // instead of a dependent chain per pass) when they fit: nact * grp * (D + 2) floats next to the merge weights.
  constexpr int SMEM_FLOATS = DW * 2 * DKB * D * 2 / 4;
  const int tot = nact * grp * (D + 2);
  const bool staged = tot + grp * nact <= SMEM_FLOATS;
  float* sp = reinterpret_cast<float*>(smem);
  if (staged) {
    for (int i = threadIdx.x; i < tot / 2; i += DW * 32)
      reinterpret_cast<float2*>(sp)[i] = __ldcg(reinterpret_cast<const float2*>(pg) + i);
    mw = sp + tot;
    __syncthreads();
  }
  auto part_at = [&](int idx) { return staged ? sp[idx] : __ldcg(pg + idx); };
  for (int hh = warp; hh < grp; hh += DW) {
    float M = -INFINITY;
    for (int sI = lane; sI < nact; sI += 32) M = fmaxf(M, part_at((sI * grp + hh) * (D + 2)));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, off));
    float L = 0.f;
    for (int sI = lane; sI < nact; sI += 32) {
      const int ps = (sI * grp + hh) * (D + 2);
      const float w = exp2f(part_at(ps) - M);
      mw[hh * nact + sI] = w;
      L = fmaf(w, part_at(ps + 1), L);
    }
    L = warp_sum(L);
    const float inv = 1.f / L;
    for (int sI = lane; sI < nact; sI += 32) mw[hh * nact + sI] *= inv;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < grp * D; e += DW * 32) {
    const int hh = e / D, dd = e - hh * D;
    float A = 0.f;
#pragma unroll 8
    for (int sI = 0; sI < nact; ++sI) A = fmaf(mw[hh * nact + sI], part_at((sI * grp + hh) * (D + 2) + 2 + dd), A);
    o_out[(size_t)(kvh * grp + hh) * D + dd] = A;
  }
  if (threadIdx.x == 0) tickets[kvh] = 0u;
  if (threadIdx.x == 0) TL(TL_ID_ATTN, blockIdx.x + gridDim.x * blockIdx.y, TL_WARP0 + 1);  // merge done
}

template <int D>
cudaError_t launch_dec_t(const LaunchCtx& c, const float* q, const void* kc, const void* vc, const int* pos, int a,
                         int b, int max_seq, int nsplit, float* scratch, unsigned* tickets, float* o) {
  auto kern = decode_attn_mma_kernel<D>;
  const size_t smem = (size_t)DW * 2 * DKB * D * 2;  // >= merge buffers (16 DW + 8 DW D + grp * nsplit floats)
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  int sms = 148, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return launch_kernel(c, kern, dim3(b, nsplit), dim3(DW * 32), smem, q, (const __nv_bfloat16*)kc,
                       (const __nv_bfloat16*)vc, pos, a / b, max_seq, nsplit, sms / b, scratch, tickets, o);
}

}  // namespace

bool decode_attention_mma_supported(int dt, int a, int b, int d, int nsplit) {
  const int grp = a / b;
  return dt == DT_BF16 && (d == 128 || d == 64) && grp <= 8 && (size_t)(16 * DW + 8 * DW * d + grp * nsplit) * 4 <= (size_t)DW * 2 * DKB * d * 2;
}

cudaError_t launch_decode_attention_mma(const LaunchCtx& c, const float* q, const void* kcache_layer,
                                        const void* vcache_layer, const int* pos, int a, int b, int d, int max_seq,
                                        int nsplit, float* scratch, unsigned* tickets, float* o) {
  if (d == 128) return launch_dec_t<128>(c, q, kcache_layer, vcache_layer, pos, a, b, max_seq, nsplit, scratch, tickets, o);
  if (d == 64) return launch_dec_t<64>(c, q, kcache_layer, vcache_layer, pos, a, b, max_seq, nsplit, scratch, tickets, o);
  return cudaErrorInvalidValue;
}

bool prefill_attention_mma_supported(int dt, int d) { return dt == DT_BF16 && (d == 128 || d == 64); }

cudaError_t launch_prefill_attention_mma(const LaunchCtx& c, const float* Q, const void* kcache_layer,
                                         const void* vcache_layer, int T, int pos0, int a, int b, int d, int max_seq,
                                         void* O, int out_mode) {
#define TPI_AM(DD)                                                                                         \
  return out_mode == 2 ? launch_t<DD, 2>(c, Q, kcache_layer, vcache_layer, T, pos0, a, b, max_seq, O)       \
         : out_mode == 1 ? launch_t<DD, 1>(c, Q, kcache_layer, vcache_layer, T, pos0, a, b, max_seq, O)     \
                         : launch_t<DD, 0>(c, Q, kcache_layer, vcache_layer, T, pos0, a, b, max_seq, O)
  if (d == 128) TPI_AM(128);
  if (d == 64) TPI_AM(64);
#undef TPI_AM
  return cudaErrorInvalidValue;
}

}  // namespace tpi
