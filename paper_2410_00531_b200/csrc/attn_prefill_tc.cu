// Causal attention of the prompt pass on the 5th-generation tensor cores (bf16 KV cache, head dimension 128):
// Eq. 1's softmax(QK^T/sqrt d)V for T query positions at once.  One CTA = 128 queries of one head; keys are walked
// in tiles of 128.  Per tile: S = Q K^T (tcgen05.mma, fp32 in tensor memory), an online softmax by 4 warps in
// which every thread owns one query row (no shuffles), the weights P written back over S in tensor memory as packed
// bf16 (the MMA's A operand is read from there), and O += P V (tcgen05.mma, V read in place as an MN-major operand)
// accumulated in tensor memory.
//   * K and V tiles come straight from the cache by TMA (128B swizzle; rows past the last valid position are
//     zero-filled by the tensor map's bounds, so nothing beyond position pos0 + T - 1 is read).
//   * The fp32 queries and the softmax weights are split into bf16 hi + lo and multiplied twice (K and V are exact
//     bf16, the cache's storage type), as in the mma.sync kernel this replaces for long prompts.
//   * Two softmax streams: warps 2-5 take the even key tiles (S / P buffer 0, accumulator O_0), warps 6-9 the odd
//     ones (buffer 1, O_1), each with its own running reference and sum; one warp per SM sub-partition cannot issue
//     the softmax of a tile as fast as the tensor core multiplies it, two can.  The epilogue merges the two
//     streams (weights 2^(m - M)), so tensor memory holds S_0, S_1, O_0, O_1 = 512 columns.
//   * O is rescaled only when a row's maximum has grown by more than 2^8 since the reference in use (the final
//     1/l normalisation makes a stale reference exact), and only then does a stream wait for its previous P V.
// Roles: warp 0 lane 0 TMA producer, warp 1 lane 0 MMA issuer, warps 2-9 softmax and epilogue.  Every mbarrier
// wait is bounded; a role that gives up leaves its loop, the others follow at their next wait, and the error word
// is set.
#include <stdlib.h>

#include "gemm_tc_common.cuh"

namespace tpi {

namespace {

using namespace tc;

constexpr int AD = 128;          // head dimension
constexpr int AQ = 128, AK = 128;  // queries per CTA, keys per tile
constexpr uint32_t BLK = AQ * 64 * 2;    // one [128 rows][64 elements] bf16 block, 128B-swizzled: 16 KB
constexpr uint32_t OFF_QH = 0, OFF_QL = 2 * BLK, OFF_K = 4 * BLK, OFF_V = 8 * BLK, ATT_SMEM = 12 * BLK;  // 192 KB: Q, 2 x K, 2 x V
constexpr uint32_t TM_S0 = 0, TM_S1 = 128, TM_O = 256, TM_COLS = 512;  // O_0 at TM_O, O_1 at TM_O + 128
constexpr int ATT_THREADS = 320;

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void umma_bf16_ta(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(  // A operand from tensor memory (row = lane, two bf16 per column), B from shared memory
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// V tile as the B operand of O += P V: the contraction runs over keys, and a key's row holds the 64 output columns
// of a block contiguously (MN-major, 128-byte swizzle): 8 keys per 1024-byte group (stride offset), the second
// block of 64 columns one block further (leading offset).
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(BLK >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// byte offset of 16-byte chunk c8 (8 elements) of row r in a [128][128]-element operand made of two 64-wide blocks
__device__ __forceinline__ uint32_t op_off(int r, int c8) {
  return (uint32_t)((c8 >> 3) * BLK + r * 128 + (((c8 & 7) ^ (r & 7)) << 4));
}
// two fp32 values -> packed bf16 pair of the rounded values (x in the low half) and the pair of the remainders
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(y), "f"(x));
  const float rx = x - __uint_as_float(hi << 16), ry = y - __uint_as_float(hi & 0xFFFF0000u);
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(ry), "f"(rx));
}
__device__ __forceinline__ void split8(const float (&v)[8], uint4& hi, uint4& lo) {
  split2(v[0], v[1], hi.x, lo.x);
  split2(v[2], v[3], hi.y, lo.y);
  split2(v[4], v[5], hi.z, lo.z);
  split2(v[6], v[7], hi.w, lo.w);
}
// 2^x for x <= 8 or so (softmax weights against a running reference); -inf -> 0
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int MODE>
__device__ __forceinline__ void store_row32(void* base, size_t i, size_t lo_off, const float (&v)[32]) {
  if (MODE == 0) {
    float* p = reinterpret_cast<float*>(base) + i;
#pragma unroll
    for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(p + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
  } else {
    __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(base) + i;
#pragma unroll
    for (int j = 0; j < 32; j += 8) {
      float w[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) w[e] = v[j + e];
      uint4 hi, lo;
      split8(w, hi, lo);
      *reinterpret_cast<uint4*>(p + j) = hi;
      if (MODE == 2) *reinterpret_cast<uint4*>(p + lo_off + j) = lo;
    }
  }
}

template <int MODE>
__global__ void __launch_bounds__(ATT_THREADS) prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                              const __grid_constant__ CUtensorMap tmV,
                                                              const float* __restrict__ Q, int T, int pos0, int a, int b,
                                                              void* O, size_t lo_off, int* err) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2], s_ready[2], p_ready[2], pv_done[2];
  __shared__ float st_m[2][AQ], st_l[2][AQ];  // the two streams' final reference and sum per row
  __shared__ uint32_t tmem_base_s;
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = gridDim.x - 1 - blockIdx.x;  // the longest rows (last query tiles) start first
  const int j = blockIdx.y, kvh = j / (a / b);
  const int q0 = qt * AQ;
  const int n_keys = pos0 + min(q0 + AQ, T);  // keys any row of this CTA may see
  const int n_tiles = (n_keys + AK - 1) / AK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1); mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1); mbar_init(&s_ready[i], 1);
      mbar_init(&p_ready[i], 4); mbar_init(&pv_done[i], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(TM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (warp >= 2) {  // stage the CTA's queries: scaled into the log2 domain, split hi / lo, in MMA operand layout
    const float qscale = 1.4426950408889634f * rsqrtf((float)AD);
    for (int i = threadIdx.x - 64; i < AQ * 16; i += ATT_THREADS - 64) {
      const int r = i >> 4, c8 = i & 15;
      float v[8];
      if (q0 + r < T) {
        const float* src = Q + ((size_t)(q0 + r) * a + j) * AD + c8 * 8;
        const float4 x = *reinterpret_cast<const float4*>(src), y = *reinterpret_cast<const float4*>(src + 4);
        v[0] = x.x * qscale; v[1] = x.y * qscale; v[2] = x.z * qscale; v[3] = x.w * qscale;
        v[4] = y.x * qscale; v[5] = y.y * qscale; v[6] = y.z * qscale; v[7] = y.w * qscale;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = 0.f;
      }
      uint4 hi, lo;
      split8(v, hi, lo);
      *reinterpret_cast<uint4*>(smem + OFF_QH + op_off(r, c8)) = hi;
      *reinterpret_cast<uint4*>(smem + OFF_QL + op_off(r, c8)) = lo;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const bool live = err == nullptr || *reinterpret_cast<volatile int*>(err) == DEVERR_NONE;  // an earlier CTA gave up: skip

  if (warp == 0) {
    if (lane == 0 && live) {  // ---- TMA producer: K and V tiles kt into their buffers kt & 1
      for (int kt = 0; kt < n_tiles; ++kt) {
        const int bi = kt & 1;
        const uint32_t ph = (kt >> 1) & 1;
        if (!mbar_wait(&k_empty[bi], ph ^ 1, err)) break;
        uint8_t* kd = smem + OFF_K + bi * 2 * BLK;
        mbar_expect_tx(&k_full[bi], 2 * BLK);
        tma_load_3d(kd, &tmK, &k_full[bi], 0, kt * AK, kvh);
        tma_load_3d(kd + BLK, &tmK, &k_full[bi], 64, kt * AK, kvh);
        if (!mbar_wait(&v_empty[bi], ph ^ 1, err)) break;
        uint8_t* vd = smem + OFF_V + bi * 2 * BLK;
        mbar_expect_tx(&v_full[bi], 2 * BLK);
        tma_load_3d(vd, &tmV, &v_full[bi], 0, kt * AK, kvh);
        tma_load_3d(vd + BLK, &tmV, &v_full[bi], 64, kt * AK, kvh);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && live) {  // ---- MMA issuer
      // D fp32, A and B bf16, N = 128, M = 128; S: both operands K-major; O: B (the V tile) MN-major
      constexpr uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(AK >> 3) << 17) | ((uint32_t)(AQ >> 4) << 24);
      constexpr uint32_t idesc_o = idesc_s | (1u << 16);
      const uint32_t sb = smem_u32(smem);
      auto issue_s = [&](int kt) -> bool {  // S(kt) = Q K(kt)^T into S buffer kt & 1 (free: P V of tile kt - 2 is complete)
        const int bi = kt & 1;
        if (!mbar_wait(&k_full[bi], (kt >> 1) & 1, err)) return false;
        tc_fence_after();
        const uint32_t kb = sb + OFF_K + (uint32_t)bi * 2 * BLK, d = tmem + (bi ? TM_S1 : TM_S0);
#pragma unroll
        for (int ks = 0; ks < AD / 16; ++ks) {
          const uint32_t o = (uint32_t)(ks >> 2) * BLK;
          const uint64_t dk = umma_desc_sw128(kb + o) + 2 * (ks & 3);
          umma_bf16(d, umma_desc_sw128(sb + OFF_QH + o) + 2 * (ks & 3), dk, idesc_s, ks ? 1u : 0u);
          umma_bf16(d, umma_desc_sw128(sb + OFF_QL + o) + 2 * (ks & 3), dk, idesc_s, 1u);
        }
        umma_commit(&s_ready[bi]);
        umma_commit(&k_empty[bi]);
        return true;
      };
      bool ok = n_tiles > 0 && issue_s(0);
      if (ok && n_tiles > 1) ok = issue_s(1);
      for (int kt = 0; kt < n_tiles && ok; ++kt) {
        const int bi = kt & 1;
        ok = mbar_wait(&p_ready[bi], (kt >> 1) & 1, err) && mbar_wait(&v_full[bi], (kt >> 1) & 1, err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t pa = tmem + (bi ? TM_S1 : TM_S0), vb = sb + OFF_V + (uint32_t)bi * 2 * BLK;
#pragma unroll
        for (int ks = 0; ks < AK / 16; ++ks) {  // 16 keys per step: 8 columns of P (hi, then lo 16 columns on), two 8-key groups of V
          const uint64_t dv = umma_desc_sw128_mn(vb + (uint32_t)ks * 2048);
          const uint32_t pc = pa + (uint32_t)((ks >> 1) * 32 + (ks & 1) * 8);
          umma_bf16_ta(tmem + TM_O + (uint32_t)bi * 128, pc, dv, idesc_o, ((kt >> 1) | ks) ? 1u : 0u);
          umma_bf16_ta(tmem + TM_O + (uint32_t)bi * 128, pc + 16, dv, idesc_o, 1u);
        }
        umma_commit(&pv_done[bi]);
        umma_commit(&v_empty[bi]);
        if (kt + 2 < n_tiles) {  // the S / P buffer of tile kt is rewritten only after its P V has completed
          ok = mbar_wait(&pv_done[bi], (kt >> 1) & 1, err) && issue_s(kt + 2);
        }
      }
    }
  } else {  // ---- softmax and epilogue: thread = query row, warp q covers tensor-memory lanes 32q..32q+31
    const int strm = warp >= 6 ? 1 : 0;  // stream 0: even key tiles, stream 1: odd key tiles
    const int q = warp & 3, r = q * 32 + lane;
    const uint32_t lane_sel = (uint32_t)(q * 32) << 16;
    const int qpos = pos0 + q0 + r;
    const uint32_t ts = tmem + lane_sel + (strm ? TM_S1 : TM_S0), to = tmem + lane_sel + TM_O + (uint32_t)strm * 128;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = live;
    for (int kt = strm; kt < n_tiles && ok; kt += 2) {
      const int k0 = kt * AK;
      const uint32_t ph = (kt >> 1) & 1;
      ok = mbar_wait(&s_ready[strm], ph, err);
      if (!ok) break;
      tc_fence_after();
      // tiles left of the diagonal are visible to every row of the warp: no masking there
      const bool full = k0 + AK - 1 <= pos0 + q0 + q * 32;
      float mx = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < AK; c += 32) {
        uint32_t s[32];
        tmem_ld32(ts + (uint32_t)c, s);
        if (full) {
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            m0 = fmaxf(m0, __uint_as_float(s[e])); m1 = fmaxf(m1, __uint_as_float(s[e + 1]));
            m2 = fmaxf(m2, __uint_as_float(s[e + 2])); m3 = fmaxf(m3, __uint_as_float(s[e + 3]));
          }
          mx = fmaxf(mx, fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)));
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (k0 + c + e <= qpos) mx = fmaxf(mx, __uint_as_float(s[e]));
        }
      }
      // the reference moves only when the row's maximum outgrew it by more than 2^8 (always on a stream's first tile
      // that shows the row a key; a row that sees none keeps -inf and weights 0)
      const bool need = mx > m_ref + 8.f;
      if (kt >= 2 && __any_sync(0xFFFFFFFFu, need)) {
        ok = mbar_wait(&pv_done[strm], ph ^ 1, err);  // O holds the stream's earlier tiles and nothing is adding to it
        if (!ok) break;
        tc_fence_after();
        const float alpha = need ? ex2(m_ref - mx) : 1.f;  // m_ref = -inf: the row has added nothing yet, alpha = 0
#pragma unroll 1
        for (int c = 0; c < AD; c += 32) {
          uint32_t o[32];
          tmem_ld32(to + (uint32_t)c, o);
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st32(to + (uint32_t)c, o);
        }
        l *= alpha;
      }
      if (need) m_ref = mx;
#pragma unroll 1
      for (int c = 0; c < AK; c += 32) {  // 32 scores -> 16 columns of packed P_hi and 16 of P_lo, in place
        uint32_t s[32], pk[32];
        tmem_ld32(ts + (uint32_t)c, s);
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float p0 = ex2(__uint_as_float(s[e]) - m_ref), p1 = ex2(__uint_as_float(s[e + 1]) - m_ref);
          if (!full) {
            if (k0 + c + e > qpos) p0 = 0.f;
            if (k0 + c + e + 1 > qpos) p1 = 0.f;
          }
          l += p0 + p1;
          split2(p0, p1, pk[e >> 1], pk[16 + (e >> 1)]);
        }
        tmem_st32(ts + (uint32_t)c, pk);
      }
      tc_fence_before();  // this thread's reads of S and writes of P and O are done
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_ready[strm]);
    }
    // ---- merge the two streams and store: each stream's warp takes half of the output columns of its rows
    const int my_tiles = (n_tiles - strm + 1) / 2;  // key tiles this stream has seen
    if (ok && my_tiles > 0) ok = mbar_wait(&pv_done[strm], (my_tiles - 1) & 1, err);
    st_m[strm][r] = m_ref;
    st_l[strm][r] = l;
    tc_fence_before();
    asm volatile("bar.sync 1, 256;" ::: "memory");  // the 8 softmax warps (every one of them reaches this point)
    tc_fence_after();
    if (ok && n_tiles > 0 && (err == nullptr || *reinterpret_cast<volatile int*>(err) == DEVERR_NONE)) {
      const bool two = n_tiles > 1;
      const float m0 = st_m[0][r], m1 = two ? st_m[1][r] : -INFINITY;
      const float M = fmaxf(m0, m1);
      const float w0 = ex2(m0 - M), w1 = two ? ex2(m1 - M) : 0.f;  // a stream whose rows saw no key has m = -inf, weight 0
      const float inv = 1.f / (st_l[0][r] * w0 + (two ? st_l[1][r] * w1 : 0.f));
      const float f0 = w0 * inv, f1 = w1 * inv;
      const int row = q0 + r;
#pragma unroll 1
      for (int c = strm * 64; c < strm * 64 + 64; c += 32) {
        uint32_t o0[32];
        float v[32];
        tmem_ld32(tmem + lane_sel + TM_O + (uint32_t)c, o0);
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(o0[e]) * f0;
        if (two) {
          uint32_t o1[32];
          tmem_ld32(tmem + lane_sel + TM_O + 128 + (uint32_t)c, o1);
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = fmaf(__uint_as_float(o1[e]), f1, v[e]);
        }
        if (row < T) store_row32<MODE>(O, ((size_t)row * a + j) * AD + c, lo_off, v);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
  }
}

// cache of one layer: [kv heads][max_seq][128] bf16; only rows below n_rows are readable through the map
bool make_cache_map(CUtensorMap* m, const void* base, int n_rows, int max_seq, int b) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)AD, (cuuint64_t)n_rows, (cuuint64_t)b};
  const cuuint64_t strides[2] = {(cuuint64_t)AD * 2, (cuuint64_t)max_seq * AD * 2};
  const cuuint32_t box[3] = {64, AK, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int MODE>
cudaError_t launch_att_t(const LaunchCtx& c, const CUtensorMap& tmK, const CUtensorMap& tmV, const float* Q, int T, int pos0,
                         int a, int b, void* O, int* err) {
  auto kern = prefill_attn_tc_kernel<MODE>;
  const size_t smem = ATT_SMEM + 1024;
  static PerDeviceOnce attr_done;
  if (!attr_done.get()) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  if (c.launches) ++*c.launches;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((T + AQ - 1) / AQ, a);
  cfg.blockDim = dim3(ATT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c.stream;
  cudaLaunchAttribute attr[1];
  if (c.pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kern, tmK, tmV, Q, T, pos0, a, b, O, (size_t)T * a * AD, err);
}

}  // namespace

// TPI_ATTN_TC=0 in the environment keeps the prompt pass on the mma.sync kernel (for comparisons)
bool prefill_attention_tc_supported(int dt, int d, int T) {
  static int on = -1;
  if (on < 0) {
    const char* e = getenv("TPI_ATTN_TC");
    on = !(e && e[0] == '0');
  }
  return on && dt == DT_BF16 && d == AD && T >= 256;  // below that the 64-query tiles of the mma.sync kernel fill more SMs
}

cudaError_t launch_prefill_attention_tc(const LaunchCtx& c, const float* Q, const void* kcache_layer, const void* vcache_layer,
                                        int T, int pos0, int a, int b, int max_seq, void* O, int out_mode, int* err) {
  CUtensorMap tmK, tmV;
  if (!make_cache_map(&tmK, kcache_layer, pos0 + T, max_seq, b) || !make_cache_map(&tmV, vcache_layer, pos0 + T, max_seq, b))
    return cudaErrorInvalidValue;
  return out_mode == 2   ? launch_att_t<2>(c, tmK, tmV, Q, T, pos0, a, b, O, err)
         : out_mode == 1 ? launch_att_t<1>(c, tmK, tmV, Q, T, pos0, a, b, O, err)
                         : launch_att_t<0>(c, tmK, tmV, Q, T, pos0, a, b, O, err);
}

}  // namespace tpi
