// Prompt-pass projections on CTA pairs (tcgen05.mma.cta_group::2), for the same contract as gemm_tcgen05.cu:
//   Y[b][t][o] = sum_k (A_hi + A_lo)[t][b*Ka + k] * W[b*rows_b + o][k]     (bf16 x bf16 -> fp32)
// The two CTAs of a cluster sit on the two SMs of one TPC and compute ONE tile of 256 positions x BNT outputs:
// each CTA stages its own 128 positions of the activations and only its own BNT/2 weight rows, and the pair's
// MMA (M = 256) reads both halves: per MMA every SM pulls half the weight bytes of a single-CTA tile of the same
// width.  Used for prompts of more than 128 positions, where it measured 5-20 % faster on the wide projections;
// a pair with M = 128 (64 positions per CTA, half the activation bytes per SM) was also built and measured
// slower at 128 positions than single-CTA tiles, since 64 rows per SM run the tensor pipe at half rate.
//
// Roles per CTA: warp 0 lane 0 issues the TMA loads of its halves (completion bytes are counted on the LEADER's
// barrier, the CTA with cluster rank 0); warp 1 lane 0 of the leader issues every MMA and releases a stage in both
// CTAs with tcgen05.commit; warps 2-5 of each CTA read their own accumulator rows back (a CTA's tensor memory
// holds its 128 positions x N columns).
// Every mbarrier wait is bounded; every CTA loads its own tiles.
#include <stdlib.h>

#include "gemm_tc_common.cuh"

namespace tpi {

namespace {

using namespace tc;

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA tile load into this CTA's shared memory whose completion bytes go to a barrier of either CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// arrive on a barrier (shared::cluster address, either CTA) once the pair's MMAs issued so far have completed
__device__ __forceinline__ void umma2_commit(uint32_t bar_cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__host__ __device__ constexpr uint32_t pow2_cols(int c) { return c <= 32 ? 32u : c <= 64 ? 64u : c <= 128 ? 128u : c <= 256 ? 256u : 512u; }
constexpr int kMH = 128;  // positions per CTA; the pair's MMA has M = 256
__host__ __device__ constexpr int pair_stage_bytes(int BNT) { return 2 * kMH * kBK * 2 + (BNT / 2) * kBK * 2; }
constexpr int pair_stages(int BNT) {
  const int n = (226 * 1024 - 1024) / pair_stage_bytes(BNT);
  return n > 8 ? 8 : n;
}

// 32 accumulator values of one position, output columns col .. col + 31 (col a multiple of 32): plain fp32 stores,
// or SwiGLU on the (gate, up) pairs -> 16 activations as bf16 hi (+ lo)
__device__ __forceinline__ void store32(const GemmTcArgs& a, int batch, int row, int col, const uint32_t (&r)[32]) {
  if (row >= a.T || col >= a.n_out) return;
  if (a.act) {
    __nv_bfloat16* arow = a.act + (size_t)row * a.act_ld + (col >> 1);
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
      const __nv_bfloat16 l0 = __float2bfloat16_rn(v[0] - __bfloat162float(h0)), l1 = __float2bfloat16_rn(v[1] - __bfloat162float(h1));
      lo[j >> 2] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
    }
    if (col + 32 <= a.n_out) {
      *reinterpret_cast<uint4*>(arow) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *reinterpret_cast<uint4*>(arow + 8) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
      if (a.act_split) {
        *reinterpret_cast<uint4*>(arow + a.act_lo_off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        *reinterpret_cast<uint4*>(arow + a.act_lo_off + 8) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
      }
    } else {
      for (int j = 0; j < 16; ++j)
        if (col + 2 * j + 1 < a.n_out) {
          arow[j] = __ushort_as_bfloat16((unsigned short)(hi[j >> 1] >> ((j & 1) * 16)));
          if (a.act_split) arow[a.act_lo_off + j] = __ushort_as_bfloat16((unsigned short)(lo[j >> 1] >> ((j & 1) * 16)));
        }
    }
    return;
  }
  float* y = a.Y + (size_t)batch * a.y_bs + (size_t)row * a.ldy + col;
  if (col + 32 <= a.n_out) {
#pragma unroll
    for (int j = 0; j < 32; j += 4)
      *reinterpret_cast<float4*>(y + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
  } else {
    for (int j = 0; j < 32; ++j)
      if (col + j < a.n_out) y[j] = __uint_as_float(r[j]);
  }
}

// BNA = N of one MMA of the pair (multiple of 64); NACC accumulators share one activation tile; the pair's tile is
// 256 positions x BNT = NACC*BNA outputs.  CTA r of the pair loads weight rows n0 + r*BNT/2 + [0, BNT/2);
// accumulator j multiplies rows [j*BNA/2, (j+1)*BNA/2) of both CTAs' slices, so its output column n is weight row
// n0 + j*BNA/2 + n of the leader's slice for n < BNA/2 and row n0 + BNT/2 + j*BNA/2 + (n - BNA/2) otherwise.
template <int BNA, int NACC, int STAGES>
__global__ void __launch_bounds__(192) gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA,
                                                           const __grid_constant__ CUtensorMap tmAlo,
                                                           const __grid_constant__ CUtensorMap tmW, const GemmTcArgs a) {
  static_assert(BNA % 64 == 0 && BNA <= 256, "each CTA's half of an MMA's width is read back 32 columns at a time");
  constexpr int BNT = NACC * BNA, HALF = BNA / 2;  // HALF: this CTA's weight rows per accumulator
  constexpr uint32_t A_BYTES = kMH * kBK * 2, B_BYTES = (BNT / 2) * kBK * 2, STAGE_BYTES = 2 * A_BYTES + B_BYTES;
  constexpr uint32_t TCOLS = pow2_cols(BNT);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], acc_ready;
  __shared__ uint32_t tmem_base_s;
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();  // 0 = leader
  // position tiles run fastest over the grid: the pairs in flight share a few weight tiles (read from DRAM once) and
  // sweep the activations, which fit in L2
  const int n0 = blockIdx.y * BNT, m0 = (blockIdx.x >> 1) * 2 * kMH + (int)rank * kMH, batch = blockIdx.z;
  const int kblocks = a.K / kBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(&acc_ready, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // the same warp of both CTAs allocates the pair's tensor memory
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(TCOLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers exist before either signals the other's
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_s;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {  // ---- TMA producer of this CTA's halves
      const uint32_t bar0 = map_to_cta(smem_u32(&full[0]), 0);
      for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, a.err)) break;
        uint8_t* sa = smem + (size_t)s * STAGE_BYTES;
        if (rank == 0) mbar_expect_tx(&full[s], 2 * STAGE_BYTES);  // both CTAs' bytes land on the leader's barrier
        const uint32_t bar = bar0 + (uint32_t)s * 8;
        const int kx = batch * a.a_col_batch + kb * kBK;
        tma_load_2d_pair(sa, &tmA, bar, kx, m0);
        tma_load_2d_pair(sa + A_BYTES, &tmAlo, bar, kx, m0);
        tma_load_2d_pair(sa + 2 * A_BYTES, &tmW, bar, kb * kBK, batch * a.w_row_batch + n0 + (int)rank * (BNT / 2));
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {  // ---- the leader issues the pair's MMAs
      // instruction descriptor: D fp32, A and B bf16, both K-major, N = BNA, M = 256
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BNA >> 3) << 17) | ((uint32_t)((2 * kMH) >> 4) << 24);
      const uint32_t empty0_peer = map_to_cta(smem_u32(&empty[0]), 1);
      bool ok = true;
      for (int kb = 0; kb < kblocks && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(&full[s], ph, a.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + (size_t)s * STAGE_BYTES);
        const uint64_t dh = umma_desc_sw128(sa), dl = umma_desc_sw128(sa + A_BYTES);
#pragma unroll
        for (int j = 0; j < NACC; ++j) {
          const uint64_t db = umma_desc_sw128(sa + 2 * A_BYTES + (uint32_t)j * HALF * kBK * 2);
          const uint32_t d = tmem_acc + (uint32_t)(j * BNA);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) umma2_bf16(d, dh + 2 * k, db + 2 * k, idesc, (kb | k) ? 1u : 0u);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) umma2_bf16(d, dl + 2 * k, db + 2 * k, idesc, 1u);
        }
        umma2_commit(smem_u32(&empty[s]));           // the stage is free in this CTA ...
        umma2_commit(empty0_peer + (uint32_t)s * 8);  // ... and in the other one
      }
      umma2_commit(smem_u32(&acc_ready));
      umma2_commit(map_to_cta(smem_u32(&acc_ready), 1));
    }
  } else {  // ---- epilogue: warps 2..5 cover the four 32-lane quarters of this CTA's tensor memory
    const int q = warp & 3;
    const bool ok = mbar_wait(&acc_ready, 0, a.err);
    tc_fence_after();
    if (ok && kblocks > 0) {
      const int row = m0 + q * 32 + lane;
#pragma unroll 1
      for (int j = 0; j < NACC; ++j)
#pragma unroll 1
        for (int hh = 0; hh < 2; ++hh)
#pragma unroll 1
          for (int c = 0; c < HALF; c += 32) {
            uint32_t r[32];
            tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(j * BNA + hh * HALF + c), r);
            store32(a, batch, row, n0 + hh * (BNT / 2) + j * HALF + c, r);
          }
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA frees tensor memory or leaves while the other may still use the pair's state
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(TCOLS) : "memory");
  }
}

// Row-sharded projection with the star sum in the epilogue (Eq. 1-2 for T positions): for each of n_shards shards
// in rank order the pair's MMA forms the shard's partial sum P_i of a 256-position x 256-column tile in tensor
// memory (two accumulator buffers, so shard i+1 multiplies while shard i is read back); 8 epilogue warps per CTA
// keep the running sum ((P_0 + P_1) + ...) in registers (one row and 128 columns per thread), add the shortcut X
// last and write the new residual stream over X.  The partial sums never reach memory.
//
//
// The same kernel runs the COLUMN-sharded projections (QKV, gate/up; modes 1: plain store, 2: SwiGLU) with their
// contraction over the whole hidden state cut into CHUNKS of 512 inputs that take the place of the shards: each chunk
// is formed in tensor memory by itself and added to the running sum in registers.  The reason is the tensor core's
// accumulator: every tcgen05.mma step adds 16 products to the fp32 value in tensor memory and TRUNCATES the result,
// so a chain of K / 16 steps (twice that with the hi + lo activations) drifts towards zero by about 2^-26 of the sum
// per step: measured 9e-6 of the output's norm at K = 4096 and 1.9e-5 at K = 8192, against 2.4e-6 for the hi + lo
// split itself.  In chunks of 512 inputs, added in registers with round to nearest, the chain is 64 steps long
// whatever K is (1.1e-6).  On the 70B shape at full depth this halves the distance to the fp64 oracle (logits 2.0e-2
// -> 0.9e-2; with fp32 SIMT GEMMs throughout it is 0.6e-2).  A shard's contraction (512 to 3584 inputs) stays one
// chain: cutting it as well changed nothing measurable at full depth, and the partial sum P_i of a shard keeps the
// bits a real rank computes for it.
constexpr int RS_BN = 256, RS_THREADS = 320;
constexpr uint32_t RS_A_BYTES = kMH * kBK * 2, RS_B_BYTES = (RS_BN / 2) * kBK * 2, RS_STAGE = 2 * RS_A_BYTES + RS_B_BYTES;
constexpr int RS_STAGES = (226 * 1024 - 1024) / RS_STAGE;

struct RowSumArgs {
  float* X;  // [T][ldx] fp32: mode 0 residual in, new residual out; mode 1 output
  int ldx, T, n_out, K, n_shards;  // K: contraction length of one shard
  int a_col_batch;  // A's column offset per shard (elements)
  int w_row_batch;  // W's row offset per shard
  int* err;
  int chunks;       // chunks per shard; chunk c of a shard covers its k-blocks [c * kb_chunk, min((c + 1) * kb_chunk, K / 64))
  int kb_chunk;     // 64-wide k-blocks per chunk
  int mode;         // 0: X <- sum + X (star sum + shortcut); 1: X <- sum; 2: act <- SwiGLU(sum) as bf16 hi (+ lo)
  __nv_bfloat16* act;
  long long act_lo_off;
  int act_ld, act_split;
  int band;         // position-pair tiles per band (0: one band): the pairs sweep the column tiles band by band
};

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}

__global__ void __launch_bounds__(RS_THREADS) gemm_tc_pair_rowsum_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                         const __grid_constant__ CUtensorMap tmAlo,
                                                                         const __grid_constant__ CUtensorMap tmW,
                                                                         const RowSumArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full[RS_STAGES], empty[RS_STAGES], acc_ready[2], acc_free[2];
  __shared__ uint32_t tmem_base_s;
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();  // 0 = leader
  // Order of the pairs' tiles: position tiles run fastest inside a band of `band` position tiles, then the column
  // tiles of that band, then the next band: the pairs in flight share a few weight tiles, and a band's activations
  // (not the whole chunk's) are what has to stay in L2 while the column tiles sweep over them.
  int pt = (int)(blockIdx.x >> 1), ct = (int)blockIdx.y;
  if (a.band > 0) {
    const int PT = (int)(gridDim.x >> 1), NCT = (int)gridDim.y;
    const long long L = (long long)ct * PT + pt;
    const int full = PT / a.band;                       // bands of the full height; the rest forms a last, lower band
    const long long per_band = (long long)a.band * NCT;
    int b = (int)(L / per_band);
    if (b >= full) b = full;
    const long long rem = L - (long long)b * per_band;
    const int hb = b < full ? a.band : PT - full * a.band;  // height of this band
    ct = (int)(rem / hb);
    pt = b * a.band + (int)(rem % hb);
  }
  const int n0 = ct * RS_BN, m0 = pt * 2 * kMH + (int)rank * kMH;
  const int kblocks = a.K / kBK;  // per shard

  if (threadIdx.x == 0) {
    for (int s = 0; s < RS_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_ready[i], 1); mbar_init(&acc_free[i], 16); }  // 8 warps of each CTA
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_s;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {  // ---- TMA producer: shard after shard, the stage ring runs on across shards
      const uint32_t bar0 = map_to_cta(smem_u32(&full[0]), 0);
      int it = 0;
      bool ok = true;
      for (int sh = 0; sh < a.n_shards && ok; ++sh)
        for (int kb = 0; kb < kblocks; ++kb, ++it) {  // the loader does not care where a chunk ends
          const int s = it % RS_STAGES;
          const uint32_t ph = (it / RS_STAGES) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1, a.err)) { ok = false; break; }
          uint8_t* sa = smem + (size_t)s * RS_STAGE;
          if (rank == 0) mbar_expect_tx(&full[s], 2 * RS_STAGE);
          const uint32_t bar = bar0 + (uint32_t)s * 8;
          const int kx = sh * a.a_col_batch + kb * kBK;
          tma_load_2d_pair(sa, &tmA, bar, kx, m0);
          tma_load_2d_pair(sa + RS_A_BYTES, &tmAlo, bar, kx, m0);
          tma_load_2d_pair(sa + 2 * RS_A_BYTES, &tmW, bar, kb * kBK, sh * a.w_row_batch + n0 + (int)rank * (RS_BN / 2));
        }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {  // ---- the leader issues the pair's MMAs; chunk g (counted over all shards) accumulates in buffer g & 1
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(RS_BN >> 3) << 17) | ((uint32_t)((2 * kMH) >> 4) << 24);
      const uint32_t empty0_peer = map_to_cta(smem_u32(&empty[0]), 1);
      int it = 0;
      bool ok = true;
      const int n_seg = a.n_shards * a.chunks;
      for (int g = 0; g < n_seg && ok; ++g) {
        const int bi = g & 1;
        ok = mbar_wait(&acc_free[bi], ((g >> 1) & 1) ^ 1, a.err);  // both CTAs have read this buffer's previous chunk back
        if (!ok) break;
        tc_fence_after();
        const uint32_t d = tmem_acc + (uint32_t)bi * RS_BN;
        const int kb0 = (g % a.chunks) * a.kb_chunk, kb1 = min(kb0 + a.kb_chunk, kblocks);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % RS_STAGES;
          const uint32_t ph = (it / RS_STAGES) & 1;
          ok = mbar_wait(&full[s], ph, a.err);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)s * RS_STAGE);
          const uint64_t dh = umma_desc_sw128(sa), dl = umma_desc_sw128(sa + RS_A_BYTES), db = umma_desc_sw128(sa + 2 * RS_A_BYTES);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) umma2_bf16(d, dh + 2 * k, db + 2 * k, idesc, (kb > kb0 || k) ? 1u : 0u);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) umma2_bf16(d, dl + 2 * k, db + 2 * k, idesc, 1u);
          umma2_commit(smem_u32(&empty[s]));
          umma2_commit(empty0_peer + (uint32_t)s * 8);
        }
        umma2_commit(smem_u32(&acc_ready[bi]));
        umma2_commit(map_to_cta(smem_u32(&acc_ready[bi]), 1));
      }
    }
  } else {  // ---- epilogue: warps 2..9; warp (q, hs) owns rows 32q.. and columns 128 hs .. 128 hs + 127 of the CTA's tile
    const int q = warp & 3, hs = (warp - 2) >> 2;
    const uint32_t tbase = tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)hs * 128;
    const uint32_t free0 = map_to_cta(smem_u32(&acc_free[0]), 0);
    float sum[128];
    bool ok = true;
    const int n_seg = a.n_shards * a.chunks;
    for (int sh = 0; sh < n_seg && ok; ++sh) {  // sh counts chunks over all shards
      const int bi = sh & 1;
      ok = mbar_wait(&acc_ready[bi], (sh >> 1) & 1, a.err);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 128; c += 16) {  // 16 columns at a time: the running sum takes 128 of the thread's registers
        uint32_t r[16];
        tmem_ld16(tbase + (uint32_t)bi * RS_BN + (uint32_t)c, r);
#pragma unroll
        for (int e = 0; e < 16; ++e) sum[c + e] = sh ? sum[c + e] + __uint_as_float(r[e]) : __uint_as_float(r[e]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(free0 + (uint32_t)bi * 8);  // on the leader's barrier: its MMA thread reuses the buffer
    }
    const int row = m0 + q * 32 + lane;
    if (ok && row < a.T && a.n_shards > 0 && kblocks > 0 && a.mode == 2) {
      // SwiGLU on the (gate, up) column pairs: 16 columns -> 8 activations -> one 16-byte store of the high halves
      // (and one of the low halves); n_out is a multiple of 32 here, so a group of 16 columns is whole or absent
      __nv_bfloat16* arow = a.act + (size_t)row * a.act_ld + ((n0 + hs * 128) >> 1);
#pragma unroll
      for (int c = 0; c < 128; c += 16) {
        if (n0 + hs * 128 + c + 16 > a.n_out) break;
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float v[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float g = sum[c + 4 * j + 2 * e], u = sum[c + 4 * j + 2 * e + 1];
            v[e] = g / (1.f + expf(-g)) * u;
          }
          const __nv_bfloat16 h0 = __float2bfloat16_rn(v[0]), h1 = __float2bfloat16_rn(v[1]);
          hi[j] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
          const __nv_bfloat16 l0 = __float2bfloat16_rn(v[0] - __bfloat162float(h0)), l1 = __float2bfloat16_rn(v[1] - __bfloat162float(h1));
          lo[j] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
        }
        *reinterpret_cast<uint4*>(arow + (c >> 1)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        if (a.act_split) *reinterpret_cast<uint4*>(arow + a.act_lo_off + (c >> 1)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
    } else if (ok && row < a.T && a.n_shards > 0 && kblocks > 0) {
      // column hs*128 + c of the CTA's tile is weight row n0 + hs * 128 + c (the leader's half first)
      float* x = a.X + (size_t)row * a.ldx + n0 + hs * 128;
      const bool add = a.mode == 0;  // the shortcut comes after the star sum; the column-sharded projections have none
#pragma unroll
      for (int c = 0; c < 128; c += 4) {
        const int col = n0 + hs * 128 + c;
        if (col + 4 <= a.n_out) {
          const float4 v = add ? *reinterpret_cast<const float4*>(x + c) : make_float4(0.f, 0.f, 0.f, 0.f);
          *reinterpret_cast<float4*>(x + c) = make_float4(sum[c] + v.x, sum[c + 1] + v.y, sum[c + 2] + v.z, sum[c + 3] + v.w);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (col + e < a.n_out) x[c + e] = add ? sum[c + e] + x[c + e] : sum[c + e];
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(512u) : "memory");
  }
}

template <int BNA, int NACC>
cudaError_t launch_pair_t(const LaunchCtx& c, const void* A, const void* Alo, int lda, const void* W, uint64_t w_rows,
                          const GemmTcArgs& a, int n_batch) {
  constexpr int BNT = NACC * BNA, STAGES = pair_stages(BNT);
  CUtensorMap tmA, tmAlo, tmW;
  if (!make_map(&tmA, A, (uint64_t)lda, (uint64_t)a.T, (uint64_t)lda, kMH)) return cudaErrorInvalidValue;
  if (!make_map(&tmAlo, Alo, (uint64_t)lda, (uint64_t)a.T, (uint64_t)lda, kMH)) return cudaErrorInvalidValue;
  if (!make_map(&tmW, W, (uint64_t)a.K, w_rows, (uint64_t)a.K, BNT / 2)) return cudaErrorInvalidValue;
  auto kern = gemm_tc_pair_kernel<BNA, NACC, STAGES>;
  const size_t smem = (size_t)STAGES * pair_stage_bytes(BNT) + 1024;
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  if (c.launches) ++*c.launches;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * ((a.T + 2 * kMH - 1) / (2 * kMH)), (a.n_out + BNT - 1) / BNT, n_batch);
  cfg.blockDim = dim3(192);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c.stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.numAttrs = 1;
  if (c.pdl) {
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmAlo, tmW, a);
}

struct PairShape { int bna, nacc; };
constexpr PairShape kShapes[] = {{128, 1}, {192, 1}, {256, 1}, {256, 2}};
constexpr int kNumShapes = (int)(sizeof(kShapes) / sizeof(kShapes[0]));

}  // namespace

// Predicted time of the best pair shape for this problem, from the measured time one tile takes per 64-wide k-block
// (0.53 / 0.66 / 0.82 / 1.57 us for the four shapes) plus a fixed cost per tile, times the waves of pairs over the
// TPCs.  Returns the index into kShapes, or -1 when no pair shape applies (T <= 128).
int gemm_tc_pair_choose(int T, int n_out, int K, int n_batch, int nsm, double* us_out) {
  if (T <= kMH) return -1;
  static const double tile_us[kNumShapes] = {0.53, 0.66, 0.82, 1.57};
  int best_i = -1;
  double best = 1e30;
  const char* force = getenv("TPI_GEMM_PAIR_SHAPE");  // development aid: pin one shape
  for (int i = 0; i < kNumShapes; ++i) {
    const int bnt = kShapes[i].bna * kShapes[i].nacc;
    if (force && atoi(force) != i) continue;
    if (bnt > 128 && n_out < bnt) continue;
    const long long pairs = (long long)((n_out + bnt - 1) / bnt) * ((T + 2 * kMH - 1) / (2 * kMH)) * n_batch;
    const long long waves = (pairs + nsm / 2 - 1) / (nsm / 2);
    const double us = (double)waves * ((K / kBK) * tile_us[i] + 6.0 + bnt / 64.0);
    if (us < best - 1e-9) { best = us; best_i = i; }
  }
  if (us_out) *us_out = force && best_i >= 0 ? 0 : best;
  return best_i;
}

cudaError_t launch_gemm_tc_pair(const LaunchCtx& c, int shape, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                                const void* W_bf16, int w_row_batch, float* Y, long long y_batch_stride, int ldy, int T, int n_out,
                                int K, int n_batch, int* err, void* act, int act_ld, long long act_lo_off, int act_split) {
  if (shape < 0 || shape >= kNumShapes || !A_lo_bf16) return cudaErrorInvalidValue;
  const uint64_t w_rows = (uint64_t)(n_batch - 1) * w_row_batch + n_out;
  GemmTcArgs a{Y, y_batch_stride, ldy, T, n_out, K, a_col_batch, w_row_batch, err, (__nv_bfloat16*)act, act_lo_off, act_ld, act_split, 0, 0, 1};
  switch (shape) {
    case 0: return launch_pair_t<128, 1>(c, A_bf16, A_lo_bf16, lda, W_bf16, w_rows, a, n_batch);
    case 1: return launch_pair_t<192, 1>(c, A_bf16, A_lo_bf16, lda, W_bf16, w_rows, a, n_batch);
    case 2: return launch_pair_t<256, 1>(c, A_bf16, A_lo_bf16, lda, W_bf16, w_rows, a, n_batch);
    case 3: return launch_pair_t<256, 2>(c, A_bf16, A_lo_bf16, lda, W_bf16, w_rows, a, n_batch);
  }
  return cudaErrorInvalidValue;
}

bool gemm_tc_rowsum_supported(int T, int K, int a_cols_total, int n_out, int ldx) {
  const char* e = getenv("TPI_GEMM_ROWSUM");  // TPI_GEMM_ROWSUM=0 keeps the partial sums in memory (for comparisons)
  return !(e && e[0] == '0') && T > kMH && K > 0 && K % kBK == 0 && a_cols_total % 8 == 0 && ldx % 4 == 0 && n_out % 4 == 0;
}

static cudaError_t launch_rowsum_args(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, const void* W_bf16,
                                      uint64_t w_cols, uint64_t w_rows, const RowSumArgs& a);

// Band height of the tile order, in position tiles of 256 (see the kernel).  With P position tiles and C column tiles
// in flight at once the pairs pull P activation tiles and C weight tiles per k-block, P * C = the 74 pairs of the
// machine: position tiles fastest over ALL positions (P = 16 at 4096 positions, 32 at 8192) is far from the balance
// P ~ C; 4 measured best (8B shape, 4096-token prompt: TTFT 109.6 -> 107.9 ms; 70B shape, 8192 tokens: 2.03 -> 1.91 s;
// 8 within noise of it, 2 in between).
static int band_tiles() {
  static int band = -1;
  if (band < 0) {
    const char* e = getenv("TPI_GEMM_BAND");  // development aid: 0 = one band (position tiles fastest over the whole chunk)
    band = e ? atoi(e) : 4;
    if (band < 0) band = 4;
  }
  return band;
}

int gemm_tc_chunk_len() {
  static int len = -1;
  if (len < 0) {
    const char* e = getenv("TPI_GEMM_CHUNK");  // development aid: 0 = one accumulation chain per contraction, else the longest chunk
    len = e ? atoi(e) : 512;
    if (len < 0 || len % kBK) len = 512;
  }
  return len;
}
// chunks of a contraction of K inputs: as few as keep every chunk within the limit, of equal length up to one k-block
static void chunking(int K, int* chunks, int* kb_chunk) {
  const int len = gemm_tc_chunk_len(), kblocks = K / kBK;
  const int n = len > 0 ? (K + len - 1) / len : 1;
  *chunks = n < 1 ? 1 : n;
  *kb_chunk = (kblocks + *chunks - 1) / *chunks;
  if (*kb_chunk < 1) *kb_chunk = 1;
  *chunks = (kblocks + *kb_chunk - 1) / *kb_chunk;
  if (*chunks < 1) *chunks = 1;
}

cudaError_t launch_gemm_tc_rowsum(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, int a_col_batch,
                                  const void* W_bf16, int w_row_batch, float* X, int ldx, int T, int n_out, int K, int n_shards,
                                  int* err) {
  if (!A_lo_bf16 || n_shards < 1) return cudaErrorInvalidValue;
  RowSumArgs a{X, ldx, T, n_out, K, n_shards, a_col_batch, w_row_batch, err, 1, K / kBK, 0, nullptr, 0, 0, 0, band_tiles()};  // one chain per shard
  return launch_rowsum_args(c, A_bf16, A_lo_bf16, lda, W_bf16, (uint64_t)K, (uint64_t)(n_shards - 1) * w_row_batch + n_out, a);
}

// Column-sharded projection (one matrix, no shortcut): Y[t][o] = sum over the chunks of the contraction.
// act != nullptr: SwiGLU epilogue as in launch_gemm_tc_swiglu (act_ld, act_lo_off, act_split), nothing is written to Y.
bool gemm_tc_chunked_supported(int T, int K, int lda, int n_out, int ldy, bool swiglu) {
  const int len = gemm_tc_chunk_len();
  return len > 0 && T > kMH && K > len && K % kBK == 0 && lda % 8 == 0 && n_out % 4 == 0 && (swiglu ? n_out % 32 == 0 : ldy % 4 == 0);
}
cudaError_t launch_gemm_tc_chunked(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, const void* W_bf16, float* Y,
                                   int ldy, int T, int n_out, int K, int* err, void* act, int act_ld, long long act_lo_off,
                                   int act_split) {
  if (!A_lo_bf16) return cudaErrorInvalidValue;
  int chunks, kb_chunk;
  chunking(K, &chunks, &kb_chunk);
  RowSumArgs a{Y, ldy, T, n_out, K, 1, 0, 0, err, chunks, kb_chunk, act ? 2 : 1, (__nv_bfloat16*)act, act_lo_off, act_ld, act_split, band_tiles()};
  return launch_rowsum_args(c, A_bf16, A_lo_bf16, lda, W_bf16, (uint64_t)K, (uint64_t)n_out, a);
}

static cudaError_t launch_rowsum_args(const LaunchCtx& c, const void* A_bf16, const void* A_lo_bf16, int lda, const void* W_bf16,
                                      uint64_t w_cols, uint64_t w_rows, const RowSumArgs& a) {
  const int T = a.T, n_out = a.n_out;
  CUtensorMap tmA, tmAlo, tmW;
  if (!make_map(&tmA, A_bf16, (uint64_t)lda, (uint64_t)T, (uint64_t)lda, kMH)) return cudaErrorInvalidValue;
  if (!make_map(&tmAlo, A_lo_bf16, (uint64_t)lda, (uint64_t)T, (uint64_t)lda, kMH)) return cudaErrorInvalidValue;
  if (!make_map(&tmW, W_bf16, w_cols, w_rows, w_cols, RS_BN / 2)) return cudaErrorInvalidValue;
  auto kern = gemm_tc_pair_rowsum_kernel;
  const size_t smem = (size_t)RS_STAGES * RS_STAGE + 1024;
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  if (c.launches) ++*c.launches;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * ((T + 2 * kMH - 1) / (2 * kMH)), (n_out + RS_BN - 1) / RS_BN, 1);
  cfg.blockDim = dim3(RS_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c.stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.numAttrs = 1;
  if (c.pdl) {
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmAlo, tmW, a);
}

}  // namespace tpi
