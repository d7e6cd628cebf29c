// Persistent weight-streaming GEMV bodies of the decode kernels (kernels_decode.cu).  A body is written for CTA
// `cta` of `ncta` CTAs that are all resident; `xs` is the CTA's dynamic shared memory (the staged activation vector).
#pragma once
#include "common.cuh"

namespace tpi {

enum { EPI_QKV = 0, EPI_SWIGLU = 1, EPI_PARTIAL = 2, EPI_LOGITS = 3 };

struct GemvArgs {
  const void* W;              // shard 0's matrix, [rows][K] row-major
  long long shard_stride;     // elements between consecutive shards' matrices
  const float* x;             // input vector (fp32)
  int x_shard_stride;         // 0: every shard reads the same x; Ks: shard i reads x + i*Ks
  const float* gain;          // optional per-element gain applied while staging x (norm gain)
  const float* ss_part;       // optional: partial sums of x^2 written by the producer; x is scaled by
  int n_parts;                //   rsqrt(sum(ss_part[0..n_parts)) / ss_dim + eps) while staging (RMSNorm)
  float eps;
  int ss_dim;
  int K;                      // dot length
  int kc;                     // shared-memory chunk of K in floats (multiple of 8)
  int items_per_shard;        // warp work items per shard
  int n_shards;
  float* out;
  long long out_shard_stride;
  // EPI_QKV
  void* kcache;
  void* vcache;
  const int* pos;
  const float2* rope;
  int hps, kps, d, max_seq;   // q heads per shard, kv heads per shard, head dim
  // EPI_LOGITS
  float* amax_val;
  int* amax_idx;
  unsigned* ticket;
  int* tok_hist;
  int* pos_rw;
  int rows_total;
  int advance;
  int prefetch_bytes;
};

template <int EPI, int R>
__device__ __forceinline__ void item_rows(const GemvArgs& A, int item, int (&rows)[R]) {
  if constexpr (EPI == EPI_QKV) {
    static_assert(R == 2, "qkv items are row pairs");
    const int half = A.d >> 1;
    const int qp = A.hps * half, kp = A.kps * half;
    if (item < qp + kp) {  // rotary pair (i, i + d/2) of one q or k head
      const int hl = item / half, ii = item - hl * half;
      rows[0] = hl * A.d + ii;
      rows[1] = rows[0] + half;
    } else {  // two adjacent v rows
      const int t = item - qp - kp;
      rows[0] = (A.hps + A.kps) * A.d + 2 * t;
      rows[1] = rows[0] + 1;
    }
  } else {
#pragma unroll
    for (int r = 0; r < R; ++r) rows[r] = item * R + r;
  }
}

// One warp accumulates R dot products of length nvec 16-byte vectors: row r's vectors start at
// wp[r] + v0, the matching activations at xs.  Lane l takes vectors l, l+32, ...; U batches of
// loads are issued before the first FMA so that R*U 16-byte loads per lane are in flight.
template <typename WT, int R>
__device__ __forceinline__ void warp_dot(const uint4* const (&wp)[R], int v0, const float* xs, int nvec,
                                         int lane, float (&acc)[R]) {
  constexpr int VEC = Elem<WT>::VEC;
  constexpr int U = 4;
  typename Elem<WT>::Acc a[R];  // fp32 weights: the vectors' partial sums are added in fp64 (see Elem<float>)
#pragma unroll
  for (int r = 0; r < R; ++r) a[r] = acc[r];
  int v = lane;
  for (; v + 32 * (U - 1) < nvec; v += 32 * U) {
    uint4 w[U][R];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int r = 0; r < R; ++r) w[u][r] = ldg_stream16(wp[r] + v0 + v + 32 * u);
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int r = 0; r < R; ++r) a[r] = Elem<WT>::dot(w[u][r], xs + (v + 32 * u) * VEC, a[r]);
  }
  if (v < nvec) {  // ragged tail: one more batch with the out-of-range loads masked, still issued together
    uint4 w[U][R];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int r = 0; r < R; ++r)
        w[u][r] = (v + 32 * u < nvec) ? ldg_stream16(wp[r] + v0 + v + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (v + 32 * u < nvec) {
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] = Elem<WT>::dot(w[u][r], xs + (v + 32 * u) * VEC, a[r]);
      }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = (float)a[r];
}

// -------------------------------------------------------------------------------------
// Persistent form for the column-sharded projections (QKV, gate/up, head): x is the same for
// every shard, so the grid is sized to the machine (a few CTAs per SM), each CTA stages x ONCE
// and walks a contiguous range of row pairs.  No wave quantisation, one prologue per CTA, all
// CTAs finish together.
// -------------------------------------------------------------------------------------
template <typename WT, int EPI, int WARPS>
__device__ __forceinline__ void cols_body(const GemvArgs& A, float* xs, const int cta, const int ncta) {
  constexpr int R = 2, XR = 4;
  __shared__ float red[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nw = WARPS > 0 ? WARPS : (int)(blockDim.x >> 5);  // WARPS == 0: the launch decides (up to 32 warps)
  const long long total = (long long)A.items_per_shard * A.n_shards;
  const int lo = (int)(total * cta / ncta), hi = (int)(total * (cta + 1) / ncta);
  const uint32_t row_bytes = (uint32_t)(A.K * sizeof(WT));
  if (threadIdx.x == 0) TL(EPI, cta, TL_ENTRY);

  auto row_ptrs = [&](int it, int& shard, int& item, const uint4* (&wp)[R]) {
    shard = it / A.items_per_shard;
    item = it - shard * A.items_per_shard;
    int rows[R];
    item_rows<EPI, R>(A, item, rows);
    if constexpr (EPI == EPI_LOGITS) {  // an odd vocabulary's last pair re-reads the last row (result unused)
#pragma unroll
      for (int r = 0; r < R; ++r) rows[r] = min(rows[r], A.rows_total - 1);
    }
    const WT* Wsh = reinterpret_cast<const WT*>(A.W) + (size_t)shard * A.shard_stride;
#pragma unroll
    for (int r = 0; r < R; ++r) wp[r] = reinterpret_cast<const uint4*>(Wsh + (size_t)rows[r] * A.K);
  };

  // weights do not depend on the previous kernel: start pulling this warp's first rows into L2
  if (lo + warp < hi && lane == 0) {
    int sh, itm;
    const uint4* wp[R];
    row_ptrs(lo + warp, sh, itm, wp);
    const uint32_t pf = min(row_bytes, (uint32_t)A.prefetch_bytes) & ~15u;
#pragma unroll
    for (int r = 0; r < R; ++r)
      if (pf) l2_prefetch_bulk(wp[r], pf);
  }
  pdl_launch_dependents();
  // the norm gain is a weight of this block: it is read ahead of the wait, so that afterwards every CTA asks L2 only
  // for x and the statistics (the same few lines for all CTAs)
  float4 xr[XR], gr[XR];
#pragma unroll
  for (int j = 0; j < XR; ++j) {
    const int k = (threadIdx.x + j * nw * 32) * 4;
    if (k < A.K) gr[j] = A.gain ? *reinterpret_cast<const float4*>(A.gain + k) : make_float4(1.f, 1.f, 1.f, 1.f);
  }
  pdl_wait();  // x (and its norm statistics) come from the previous kernel
  if (threadIdx.x == 0) TL(EPI, cta, TL_WAIT);

  // ---- prologue: one round trip to L2 for the statistics and x
  float ss = 0.f;
  if (A.ss_part)
    for (int i = threadIdx.x; i < A.n_parts; i += nw * 32) ss += A.ss_part[i];
#pragma unroll
  for (int j = 0; j < XR; ++j) {
    const int k = (threadIdx.x + j * nw * 32) * 4;
    if (k < A.K) xr[j] = *reinterpret_cast<const float4*>(A.x + k);
  }
  float rnorm = 1.f;
  if (A.ss_part) {
    ss = block_sum(ss, red);
    rnorm = rsqrtf(ss / (float)A.ss_dim + A.eps);
  }
#pragma unroll
  for (int j = 0; j < XR; ++j) {
    const int k = (threadIdx.x + j * nw * 32) * 4;
    if (k < A.K) {
      float4 v = xr[j];
      if (A.ss_part) { v.x *= rnorm; v.y *= rnorm; v.z *= rnorm; v.w *= rnorm; }
      v.x *= gr[j].x; v.y *= gr[j].y; v.z *= gr[j].z; v.w *= gr[j].w;
      *reinterpret_cast<float4*>(xs + k) = v;
    }
  }
  for (int k = (threadIdx.x + XR * nw * 32) * 4; k < A.K; k += nw * 32 * 4) {
    float4 v = *reinterpret_cast<const float4*>(A.x + k);
    if (A.ss_part) { v.x *= rnorm; v.y *= rnorm; v.z *= rnorm; v.w *= rnorm; }
    if (A.gain) {
      const float4 g = *reinterpret_cast<const float4*>(A.gain + k);
      v.x *= g.x; v.y *= g.y; v.z *= g.z; v.w *= g.w;
    }
    *reinterpret_cast<float4*>(xs + k) = v;
  }
  __syncthreads();
  if (threadIdx.x == 0) TL(EPI, cta, TL_STAGED);

  // ---- main loop over this CTA's row pairs
  const int nvec = A.K / Elem<WT>::VEC;
  float bv = -INFINITY;  // EPI_LOGITS: this warp's running best
  int bi = 0x7FFFFFFF;
  for (int it = lo + warp; it < hi; it += nw) {
    int shard, item;
    const uint4* wp[R];
    row_ptrs(it, shard, item, wp);
    // QKV: the position and this pair's rotation are requested before the weight stream, not after it
    int p_cur = 0;
    float2 cs_cur = make_float2(1.f, 0.f);
    if constexpr (EPI == EPI_QKV) {
      const int half = A.d >> 1;
      p_cur = *A.pos;
      if (item < (A.hps + A.kps) * half) cs_cur = A.rope[(size_t)p_cur * half + (item % half)];
    }
    float acc[R] = {0.f, 0.f};
    warp_dot<WT, R>(wp, 0, xs, nvec, lane, acc);
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = warp_sum(acc[r]);
    if (lane == 0) {
      if constexpr (EPI == EPI_QKV) {
        const int half = A.d >> 1;
        const int qp = A.hps * half, kp = A.kps * half;
        const int p = p_cur;
        if (item < qp + kp) {
          const bool is_q = item < qp;
          const int t = is_q ? item : item - qp;
          const int hl = t / half, ii = t - hl * half;
          const float2 cs = cs_cur;
          const float lo_v = acc[0] * cs.x - acc[1] * cs.y;
          const float hi_v = acc[1] * cs.x + acc[0] * cs.y;
          if (is_q) {
            float* q = A.out + (size_t)(shard * A.hps + hl) * A.d;
            q[ii] = lo_v;
            q[ii + half] = hi_v;
          } else {
            WT* kr = reinterpret_cast<WT*>(A.kcache) + ((size_t)(shard * A.kps + hl) * A.max_seq + p) * A.d;
            Elem<WT>::store(kr + ii, lo_v);
            Elem<WT>::store(kr + ii + half, hi_v);
          }
        } else {
          const int t2 = 2 * (item - qp - kp);
          const int hl = t2 / A.d, idx = t2 - hl * A.d;
          WT* vr = reinterpret_cast<WT*>(A.vcache) + ((size_t)(shard * A.kps + hl) * A.max_seq + p) * A.d;
          Elem<WT>::store(vr + idx, acc[0]);
          Elem<WT>::store(vr + idx + 1, acc[1]);
        }
      } else if constexpr (EPI == EPI_SWIGLU) {
        const float g = acc[0], u = acc[1];
        A.out[(size_t)shard * A.out_shard_stride + item] = g / (1.f + expf(-g)) * u;
      } else {  // EPI_LOGITS (rows ascend within a warp, so '>' keeps the lowest index on ties)
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const int row = item * R + r;
          if (row < A.rows_total) {
            A.out[row] = acc[r];
            if (acc[r] > bv) { bv = acc[r]; bi = row; }
          }
        }
      }
    }
  }
  if (lane == 0) TL(EPI, cta, TL_WARP0 + warp);
  if constexpr (EPI == EPI_LOGITS) {
    __shared__ float s_val[WARPS > 0 ? WARPS : 32];
    __shared__ int s_idx[WARPS > 0 ? WARPS : 32];
    __shared__ bool s_last;
    if (lane == 0) { s_val[warp] = bv; s_idx[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < nw; ++w)
        if (s_val[w] > bv || (s_val[w] == bv && s_idx[w] < bi)) { bv = s_val[w]; bi = s_idx[w]; }
      A.amax_val[cta] = bv;
      A.amax_idx[cta] = bi;
      __threadfence();
      const unsigned t = atomicAdd(A.ticket, 1u);
      s_last = (t == ncta - 1);
    }
    __syncthreads();
    if (s_last && warp == 0) {
      __threadfence();
      bv = -INFINITY;
      bi = 0x7FFFFFFF;
      for (int b = lane; b < ncta; b += 32) {
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

// =====================================================================================
// Row-sharded projection fused with the emulated star allreduce and the shortcut
// =====================================================================================
// One warp owns R output rows and visits the N shards in rank order: it forms shard i's partial sum
// P_i[r] = W^i[r,:] . x_i exactly as the stand-alone partials kernel does, then folds it into
// ((P_0 + P_1) + ... + P_{N-1}) + residual in registers, so the N partial sums never travel through
// memory.  Each CTA also emits the sum of squares of its new residual entries for the next RMSNorm.
struct RowFusedArgs {
  const void* W;           // [N][rows][Ks]
  long long shard_stride;  // elements
  const float* x_in;       // [N * Ks]
  int Ks, n_shards, rows, n_parts, prefetch_bytes;
  int unequal;             // 1: shard i owns inputs [k0[i], k0[i+1]) and its matrix starts rows * k0[i] elements into W
  int k0[ROWSHARD_MAX_UNEQUAL + 1];
  float* x;                // residual stream, in/out [rows]
  float* ss_part;          // [n_parts]: per-CTA sum of squares of its new entries (zeros beyond the grid)
  float* tap;              // optional copy of the new residual
};

// Persistent: a few CTAs per SM, the whole x_in staged once per CTA, each CTA owns a contiguous
// range of row groups.
// NS > 0: the shard count is a compile-time constant (1, 2, 4, 8); NS == 0: any N, shard by shard.
template <typename WT, int R, int NS, int WARPS>
__device__ __forceinline__ void rowfused_body(const RowFusedArgs& A, float* xs, const int cta, const int ncta) {
  __shared__ float s_sq[WARPS > 0 ? WARPS : 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nw = WARPS > 0 ? WARPS : (int)(blockDim.x >> 5);
  const int groups = A.rows / R;
  const int lo = (int)((long long)groups * cta / ncta);
  const int hi = (int)((long long)groups * (cta + 1) / ncta);
  const WT* Wall = reinterpret_cast<const WT*>(A.W);
  [[maybe_unused]] const int tlid = (A.Ks * A.n_shards == A.rows) ? TL_ID_O : TL_ID_DOWN;  // timeline id (square: O)
  if (threadIdx.x == 0) TL(tlid, cta, TL_ENTRY);
  if (lo + warp < hi && !A.unequal) {
    const uint32_t pf = min((uint32_t)(R * A.Ks * sizeof(WT)), (uint32_t)A.prefetch_bytes) & ~15u;
    for (int sh = lane; sh < A.n_shards; sh += 32)
      if (pf) l2_prefetch_bulk(Wall + (size_t)sh * A.shard_stride + (size_t)(lo + warp) * R * A.Ks, pf);
  }
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) TL(tlid, cta, TL_WAIT);

  const int ktot = A.unequal ? A.k0[A.n_shards] : A.n_shards * A.Ks;
  for (int k = threadIdx.x * 4; k < ktot; k += nw * 32 * 4)
    *reinterpret_cast<float4*>(xs + k) = *reinterpret_cast<const float4*>(A.x_in + k);
  __syncthreads();
  if (threadIdx.x == 0) TL(tlid, cta, TL_STAGED);

  constexpr int VEC = Elem<WT>::VEC;
  const int nvec = A.Ks / VEC;
  float sq = 0.f;
  for (int g = lo + warp; g < hi; g += nw) {
    const int row0 = g * R;
    float sum[R], res[R];
#pragma unroll
    for (int r = 0; r < R; ++r) res[r] = A.x[row0 + r];  // shortcut operand, requested ahead of the weight stream
    if constexpr (NS > 0) {
      // Every shard's slice of these rows is requested in the same batch (NS * R * U 16-byte loads
      // per lane in flight); each shard keeps its own accumulator, so the partial sums stay per device.
      constexpr int U = (8 / (NS * R)) > 0 ? (8 / (NS * R)) : 1;
      typename Elem<WT>::Acc acc[NS][R];
#pragma unroll
      for (int sh = 0; sh < NS; ++sh)
#pragma unroll
        for (int r = 0; r < R; ++r) acc[sh][r] = 0;
      const uint4* base = reinterpret_cast<const uint4*>(Wall + (size_t)row0 * A.Ks);
      const size_t sstride = (size_t)A.shard_stride / VEC, rstride = (size_t)nvec;
      for (int v = lane; v < nvec; v += 32 * U) {
        uint4 w[NS][R][U];
#pragma unroll
        for (int sh = 0; sh < NS; ++sh)
#pragma unroll
          for (int r = 0; r < R; ++r)
#pragma unroll
            for (int u = 0; u < U; ++u)
              w[sh][r][u] = (v + 32 * u < nvec) ? ldg_stream16(base + sh * sstride + r * rstride + v + 32 * u)
                                                : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < U; ++u)
          if (v + 32 * u < nvec) {
#pragma unroll
            for (int sh = 0; sh < NS; ++sh)
#pragma unroll
              for (int r = 0; r < R; ++r)
                acc[sh][r] = Elem<WT>::dot(w[sh][r][u], xs + (size_t)sh * A.Ks + (v + 32 * u) * VEC, acc[sh][r]);
          }
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        sum[r] = warp_sum((float)acc[0][r]);                               // the master's own partial sum
#pragma unroll
        for (int sh = 1; sh < NS; ++sh) sum[r] += warp_sum((float)acc[sh][r]);  // + workers', in rank order
      }
    } else {
#pragma unroll
      for (int r = 0; r < R; ++r) sum[r] = 0.f;
      for (int sh = 0; sh < A.n_shards; ++sh) {
        const uint4* wp[R];
        float acc[R];
        const int kb = A.unequal ? A.k0[sh] : sh * A.Ks;                 // first input of this shard
        const int kw = A.unequal ? A.k0[sh + 1] - kb : A.Ks;             // its width
        const size_t wbase = A.unequal ? (size_t)A.rows * kb : (size_t)sh * A.shard_stride;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          wp[r] = reinterpret_cast<const uint4*>(Wall + wbase + (size_t)(row0 + r) * kw);
          acc[r] = 0.f;
        }
        warp_dot<WT, R>(wp, 0, xs + kb, kw / VEC, lane, acc);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const float p = warp_sum(acc[r]);         // device sh's partial sum
          sum[r] = (sh == 0) ? p : sum[r] + p;      // the master adds them in rank order
        }
      }
    }
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float v = sum[r] + res[r];          // shortcut after the allreduce
        A.x[row0 + r] = v;
        if (A.tap) A.tap[row0 + r] = v;
        sq = fmaf(v, v, sq);
      }
    }
  }
  if (lane == 0) TL(tlid, cta, TL_WARP0 + warp);
  if (lane == 0) s_sq[warp] = sq;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = s_sq[0];
    for (int w = 1; w < nw; ++w) t += s_sq[w];
    A.ss_part[cta] = t;
    for (int i = cta + ncta; i < A.n_parts; i += ncta) A.ss_part[i] = 0.f;
  }
}

}  // namespace tpi
