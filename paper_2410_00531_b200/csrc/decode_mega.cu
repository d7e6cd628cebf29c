// Whole-token decode kernel: one cooperative launch runs every step of Algorithm 1's loop body for
// one position (embedding, L x [QKV + RoPE + KV append, attention, O -> star sum + shortcut, gate/up +
// SwiGLU, down -> star sum + shortcut], head + argmax) with one persistent CTA per SM.
//
// Why: with batch 1 each phase streams 30-200 MB of weights in 5-30 us, so per-launch costs (launch
// gap, prologue, DRAM ramp, tail) are 30 % of a step when the phases are separate kernels.  Here the
// phases are separated by a grid barrier (one atomic per CTA + a bounded spin), and before a CTA
// arrives at the barrier it asks L2 to fetch the first weight rows it will need in the NEXT phase, so
// HBM keeps streaming across the barrier.
//
// Every spin is bounded: when a limit runs out the kernel writes DEVERR_WAIT_TIMEOUT to the error word,
// later barriers return at once, and the kernel runs to its end (with meaningless results that the
// host discards).  Co-residency of all CTAs is guaranteed by the cooperative launch.
#include "common.cuh"
#include "gemv_bodies.cuh"
#include "kernels.h"

namespace tpi {

namespace {

constexpr int MW = 32;  // warps per CTA (one CTA of 1024 threads per SM)

struct MegaLayer {
  GemvArgs qkv;
  RowFusedArgs oproj;
  GemvArgs gateup;
  RowFusedArgs down;
  const void* kc;
  const void* vc;
};

static_assert(sizeof(MegaLayer) <= 1024, "the memory plan reserves 1024 bytes per layer");

struct MegaArgs {
  const MegaLayer* layers;  // device array [n_layers]
  int n_layers;
  const void* emb;
  int vocab, max_seq, h;
  float* x;
  float* ss_part;
  int n_parts;
  int* tok_hist;
  int* pos;
  int* err;
  float* q;
  float* o;
  float* attn_scratch;
  unsigned* tickets;
  int a, b, nsplit;
  GemvArgs head;
  unsigned* bar;  // grid-barrier counter, zero when the kernel starts
  int prefetch;
  unsigned long long* ts;  // optional: CTA 0 stamps the global timer after every barrier (phase timing aid)
};

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// k-th barrier of the launch: every CTA adds one, then waits for (k + 1) * ncta.  Bounded.
__device__ __forceinline__ void grid_barrier(unsigned* bar, unsigned k, int ncta, int* err,
                                             unsigned long long* ts = nullptr) {
  if (ts && blockIdx.x == 0 && threadIdx.x == 0) {  // arrival time of CTA 0 (even slots), release time (odd slots)
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    ts[2 * k] = t;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(bar, 1u);
    const unsigned target = (k + 1u) * (unsigned)ncta;
    if (*reinterpret_cast<volatile int*>(err) == DEVERR_NONE) {
      int spins = 0;
      while (ld_acquire_u32(bar) < target) {
        if (++spins > (1 << 21)) {  // tens of milliseconds: far beyond any phase of a decode step
          atomicCAS(err, DEVERR_NONE, DEVERR_WAIT_TIMEOUT);
          break;
        }
        if (spins > 4096) __nanosleep(64);
      }
    }
    __threadfence();
    if (ts && blockIdx.x == 0) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
      ts[2 * k + 1] = t;
    }
  }
  __syncthreads();
}

// ---- L2 prefetch of the rows a CTA will read first in a coming phase (hints only)
template <typename WT, int EPI>
__device__ __forceinline__ void cols_prefetch(const GemvArgs& A, int cta, int ncta, int bytes_per_row) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long total = (long long)A.items_per_shard * A.n_shards;
  const int lo = (int)(total * cta / ncta), hi = (int)(total * (cta + 1) / ncta);
  const int it = lo + warp;
  if (it >= hi || lane != 0) return;
  const int shard = it / A.items_per_shard, item = it - shard * A.items_per_shard;
  int rows[2];
  item_rows<EPI, 2>(A, item, rows);
  const WT* Wsh = reinterpret_cast<const WT*>(A.W) + (size_t)shard * A.shard_stride;
  const uint32_t pf = min((uint32_t)(A.K * sizeof(WT)), (uint32_t)bytes_per_row) & ~15u;
  if (!pf) return;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    int row = rows[r];
    if (EPI == EPI_LOGITS) row = min(row, A.rows_total - 1);
    l2_prefetch_bulk(Wsh + (size_t)row * A.K, pf);
  }
}

template <typename WT>
__device__ __forceinline__ void rowfused_prefetch(const RowFusedArgs& A, int cta, int ncta, int bytes_per_row) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int lo = (int)((long long)A.rows * cta / ncta), hi = (int)((long long)A.rows * (cta + 1) / ncta);
  if (lo + warp >= hi) return;
  const uint32_t pf = min((uint32_t)(A.Ks * sizeof(WT)), (uint32_t)bytes_per_row) & ~15u;
  const WT* Wall = reinterpret_cast<const WT*>(A.W);
  for (int sh = lane; sh < A.n_shards; sh += 32)
    if (pf) l2_prefetch_bulk(Wall + (size_t)sh * A.shard_stride + (size_t)(lo + warp) * A.Ks, pf);
}

template <typename WT>
__device__ __forceinline__ void rowfused_phase(const RowFusedArgs& A, float* xs, int cta, int ncta) {
  switch (A.n_shards) {  // compile-time shard counts keep every shard's slice of a row in flight together
    case 1: rowfused_body<WT, 1, 1, MW>(A, xs, cta, ncta); break;
    case 2: rowfused_body<WT, 1, 2, MW>(A, xs, cta, ncta); break;
    case 4: rowfused_body<WT, 1, 4, MW>(A, xs, cta, ncta); break;
    default: rowfused_body<WT, 1, 0, MW>(A, xs, cta, ncta); break;
  }
}

// ---- embedding row and its norm statistics (one CTA)
template <typename WT>
__device__ __forceinline__ void embed_phase(const MegaArgs& A, float* red) {
  const int p = *A.pos;
  int tok = (p >= 0 && p < A.max_seq) ? A.tok_hist[p] : -1;
  if (p < 0 || p >= A.max_seq) {
    if (threadIdx.x == 0) atomicCAS(A.err, DEVERR_NONE, DEVERR_POS_RANGE);
    tok = 0;
  } else if (tok < 0 || tok >= A.vocab) {
    if (threadIdx.x == 0) atomicCAS(A.err, DEVERR_NONE, DEVERR_TOKEN_RANGE);
    tok = 0;
  }
  const WT* row = reinterpret_cast<const WT*>(A.emb) + (size_t)tok * A.h;
  float ss = 0.f;
  for (int k = threadIdx.x; k < A.h; k += blockDim.x) {
    const float v = Elem<WT>::load(row + k);
    A.x[k] = v;
    ss = fmaf(v, v, ss);
  }
  ss = block_sum(ss, red);
  for (int i = threadIdx.x; i < A.n_parts; i += blockDim.x) A.ss_part[i] = i ? 0.f : ss;
}

// ---- split-K attention over the cache; work items (kv head, active split) are dealt round-robin to CTAs.
// One query head at a time (the K/V window sits in shared memory, so re-reading it per head is cheap and
// keeps the register footprint small); row groups of LPR lanes own positions; the last split of a kv head
// to finish (atomic ticket) merges that head group's splits in split order.
template <typename KT, int LPR>
__device__ __forceinline__ void attn_phase(const MegaArgs& A, const KT* kc, const KT* vc, float* sm, int cta, int ncta) {
  constexpr int VEC = Elem<KT>::VEC, D = LPR * VEC, RG = 32 / LPR, G = MW * RG;
  constexpr int CH = 256 / (int)sizeof(KT);
  KT* k_s = reinterpret_cast<KT*>(sm);
  KT* v_s = k_s + CH * D;
  float* g_m = reinterpret_cast<float*>(v_s + CH * D);  // [G]
  float* g_l = g_m + G;                                 // [G]
  float* g_acc = g_l + G;                               // [G][D]
  float* w_s = g_acc + G * D;                           // [grp][nsplit]
  __shared__ bool s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp_id = warp * RG + lane / LPR, sub = lane % LPR;
  const int grp = A.a / A.b, nsplit = A.nsplit;
  const int n = *A.pos + 1;
  int chunk = (n + nsplit - 1) / nsplit;
  chunk = (chunk + 31) & ~31;
  const int nact = (n + chunk - 1) / chunk;
  const float qscale = 1.4426950408889634f * rsqrtf((float)D);

  for (int item = cta; item < A.b * nact; item += ncta) {
    const int g = item / nact, split = item - g * nact;
    const int s0 = split * chunk, s1 = min(n, s0 + chunk);
    const KT* kg = kc + (size_t)g * A.max_seq * D;
    const KT* vg = vc + (size_t)g * A.max_seq * D;
    float* part = A.attn_scratch + ((size_t)g * nsplit + split) * grp * (D + 2);
    // online-softmax state of every head for this row group lives in registers only one head at a time,
    // so splits longer than one window keep per-head running state in shared memory (g_m / g_l / g_acc
    // are per window; the per-head running merge below folds windows together in `part`)
    for (int hh = 0; hh < grp; ++hh) {
      float run_m = -INFINITY, run_l = 0.f, run_a = 0.f;  // thread e < D owns output dim e across windows
      for (int w0 = s0; w0 < s1; w0 += CH) {
        const int wn = min(CH, s1 - w0);
        if (hh == 0 || s1 - s0 > CH) {  // (re)stage the window: once per item unless the split spans windows
          __syncthreads();
          const int n16 = wn * D * (int)sizeof(KT) / 16;
          const char* ksrc = reinterpret_cast<const char*>(kg + (size_t)w0 * D);
          const char* vsrc = reinterpret_cast<const char*>(vg + (size_t)w0 * D);
          for (int i = threadIdx.x; i < n16; i += MW * 32) {
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(reinterpret_cast<char*>(k_s) + i * 16)), "l"(ksrc + (size_t)i * 16) : "memory");
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(reinterpret_cast<char*>(v_s) + i * 16)), "l"(vsrc + (size_t)i * 16) : "memory");
          }
          asm volatile("cp.async.commit_group;" ::: "memory");
          asm volatile("cp.async.wait_group 0;" ::: "memory");
          __syncthreads();
        }
        // this row group's positions of the window: t = grp_id, grp_id + G, ...
        float qr[VEC], acc[VEC], m = -INFINITY, l = 0.f;
        {
          const float* qp = A.q + (size_t)(g * grp + hh) * D + sub * VEC;
#pragma unroll
          for (int v = 0; v < VEC; ++v) { qr[v] = qp[v] * qscale; acc[v] = 0.f; }
        }
        for (int tb = 0; tb < wn; tb += G) {  // same trip count for every lane (shuffles below)
          const int t = tb + grp_id;
          const bool in = t < wn;
          float kf[VEC], vf[VEC];
          Elem<KT>::unpack(in ? *reinterpret_cast<const uint4*>(k_s + (size_t)t * D + sub * VEC) : make_uint4(0, 0, 0, 0), kf);
          Elem<KT>::unpack(in ? *reinterpret_cast<const uint4*>(v_s + (size_t)t * D + sub * VEC) : make_uint4(0, 0, 0, 0), vf);
          float s = 0.f;
#pragma unroll
          for (int v = 0; v < VEC; ++v) s = fmaf(qr[v], kf[v], s);
#pragma unroll
          for (int off = LPR / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
          if (!in) s = -INFINITY;
          const float mn = fmaxf(m, s);
          const float ref = (mn == -INFINITY) ? 0.f : mn;
          const float scale = exp2f(m - ref), w = exp2f(s - ref);
          m = mn;
          l = l * scale + w;
#pragma unroll
          for (int v = 0; v < VEC; ++v) acc[v] = fmaf(w, vf[v], acc[v] * scale);
        }
        if (sub == 0) { g_m[grp_id] = m; g_l[grp_id] = l; }
#pragma unroll
        for (int v = 0; v < VEC; ++v) g_acc[grp_id * D + sub * VEC + v] = acc[v];
        __syncthreads();
        if (threadIdx.x < D) {  // fold the G row groups (fixed order), then fold the window into the running state
          const int dd = threadIdx.x;
          float M = -INFINITY;
          for (int gi = 0; gi < G; ++gi) M = fmaxf(M, g_m[gi]);
          float Aw = 0.f, Lw = 0.f;
          if (M > -INFINITY)
            for (int gi = 0; gi < G; ++gi) {
              const float w = exp2f(g_m[gi] - M);
              Aw = fmaf(w, g_acc[gi * D + dd], Aw);
              Lw = fmaf(w, g_l[gi], Lw);
            }
          const float mn = fmaxf(run_m, M);
          const float ref = (mn == -INFINITY) ? 0.f : mn;
          const float sa = exp2f(run_m - ref), sb = exp2f(M - ref);
          run_a = run_a * sa + Aw * sb;
          run_l = run_l * sa + Lw * sb;
          run_m = mn;
        }
        __syncthreads();
      }
      if (threadIdx.x < D) {
        part[hh * (D + 2) + 2 + threadIdx.x] = run_a;
        if (threadIdx.x == 0) { part[hh * (D + 2)] = run_m; part[hh * (D + 2) + 1] = run_l; }
      }
    }
    // ---- ticket: the last split of kv head g merges all its splits
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const unsigned t = atomicAdd(A.tickets + g, 1u);
      s_last = (t == (unsigned)nact - 1);
    }
    __syncthreads();
    if (s_last) {
      __threadfence();
      const float* pg = A.attn_scratch + (size_t)g * nsplit * grp * (D + 2);
      for (int hh = warp; hh < grp; hh += MW) {
        float M = -INFINITY;
        for (int s = lane; s < nact; s += 32) M = fmaxf(M, __ldcg(pg + (size_t)(s * grp + hh) * (D + 2)));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, off));
        float L = 0.f;
        for (int s = lane; s < nact; s += 32) {
          const float* ps = pg + (size_t)(s * grp + hh) * (D + 2);
          const float w = exp2f(__ldcg(ps) - M);
          w_s[hh * nact + s] = w;
          L = fmaf(w, __ldcg(ps + 1), L);
        }
        L = warp_sum(L);
        const float inv = 1.f / L;
        for (int s = lane; s < nact; s += 32) w_s[hh * nact + s] *= inv;
      }
      __syncthreads();
      for (int e = threadIdx.x; e < grp * D; e += blockDim.x) {
        const int hh = e / D, dd = e - hh * D;
        float acc = 0.f;
#pragma unroll 8
        for (int s = 0; s < nact; ++s)
          acc = fmaf(w_s[hh * nact + s], __ldcg(pg + (size_t)(s * grp + hh) * (D + 2) + 2 + dd), acc);
        A.o[(size_t)(g * grp + hh) * D + dd] = acc;
      }
      if (threadIdx.x == 0) A.tickets[g] = 0u;
    }
    __syncthreads();
  }
}

template <typename WT, int LPR>
__global__ void __launch_bounds__(MW * 32, 1) decode_token_kernel(const MegaArgs A) {
  extern __shared__ __align__(16) float smem[];
  __shared__ float red[32];
  const int cta = blockIdx.x, ncta = gridDim.x;
  const int PF = A.prefetch;  // bytes per row requested from L2 ahead of a barrier
  unsigned k = 0;

  if (cta == 0) embed_phase<WT>(A, red);
  cols_prefetch<WT, EPI_QKV>(A.layers[0].qkv, cta, ncta, PF);
  grid_barrier(A.bar, k++, ncta, A.err, A.ts);

  for (int l = 0; l < A.n_layers; ++l) {
    const MegaLayer& Ly = A.layers[l];
    cols_body<WT, EPI_QKV, MW>(Ly.qkv, smem, cta, ncta);
    rowfused_prefetch<WT>(Ly.oproj, cta, ncta, PF);
    grid_barrier(A.bar, k++, ncta, A.err, A.ts);

    attn_phase<WT, LPR>(A, reinterpret_cast<const WT*>(Ly.kc), reinterpret_cast<const WT*>(Ly.vc), smem, cta, ncta);
    cols_prefetch<WT, EPI_SWIGLU>(Ly.gateup, cta, ncta, PF);
    grid_barrier(A.bar, k++, ncta, A.err, A.ts);

    rowfused_phase<WT>(Ly.oproj, smem, cta, ncta);
    grid_barrier(A.bar, k++, ncta, A.err, A.ts);

    cols_body<WT, EPI_SWIGLU, MW>(Ly.gateup, smem, cta, ncta);
    rowfused_prefetch<WT>(Ly.down, cta, ncta, PF);
    grid_barrier(A.bar, k++, ncta, A.err, A.ts);

    rowfused_phase<WT>(Ly.down, smem, cta, ncta);
    if (l + 1 < A.n_layers) cols_prefetch<WT, EPI_QKV>(A.layers[l + 1].qkv, cta, ncta, PF);
    else cols_prefetch<WT, EPI_LOGITS>(A.head, cta, ncta, PF);
    grid_barrier(A.bar, k++, ncta, A.err, A.ts);
  }
  cols_body<WT, EPI_LOGITS, MW>(A.head, smem, cta, ncta);
}

}  // namespace

// ---------------------------------------------------------------------------------------------- host side
size_t mega_layer_table_bytes(int n_layers) { return (size_t)n_layers * sizeof(MegaLayer); }

static void fill_cols(GemvArgs& G, const void* W, size_t shard_stride, const NormIn& in, int h, int n_shards,
                      int items_per_shard) {
  G = GemvArgs{};
  G.W = W; G.shard_stride = (long long)shard_stride; G.x = in.x; G.gain = in.gain; G.ss_part = in.ss_part;
  G.n_parts = in.n_parts; G.eps = in.eps; G.ss_dim = h; G.x_shard_stride = 0; G.K = h; G.kc = h;
  G.n_shards = n_shards; G.items_per_shard = items_per_shard; G.prefetch_bytes = 0;
}

void mega_fill_layer(void* table_host, int l, const MegaLayerDesc& d) {
  MegaLayer& L = reinterpret_cast<MegaLayer*>(table_host)[l];
  const NormIn in_attn{d.x, d.gain_attn, d.ss_part, d.n_parts, d.eps};
  const NormIn in_ffn{d.x, d.gain_ffn, d.ss_part, d.n_parts, d.eps};
  const int hps = d.a / d.n_shards, kps = d.b / d.n_shards;
  fill_cols(L.qkv, d.wqkv, (size_t)(d.a + 2 * d.b) / d.n_shards * d.d * d.h, in_attn, d.h, d.n_shards, (hps + 2 * kps) * (d.d / 2));
  L.qkv.hps = hps; L.qkv.kps = kps; L.qkv.d = d.d; L.qkv.max_seq = d.max_seq; L.qkv.out = d.q;
  L.qkv.kcache = d.kc; L.qkv.vcache = d.vc; L.qkv.pos = d.pos; L.qkv.rope = d.rope;
  fill_cols(L.gateup, d.wgu, (size_t)2 * (d.s / d.n_shards) * d.h, in_ffn, d.h, d.n_shards, d.s / d.n_shards);
  L.gateup.out = d.act; L.gateup.out_shard_stride = d.s / d.n_shards;
  auto rf = [&](RowFusedArgs& R, const void* W, const float* xin, int Ks, float* tap) {
    R = RowFusedArgs{};
    R.W = W; R.shard_stride = (long long)d.h * Ks; R.x_in = xin; R.Ks = Ks; R.n_shards = d.n_shards; R.rows = d.h;
    R.n_parts = d.n_parts; R.prefetch_bytes = 0; R.x = d.x; R.ss_part = d.ss_part; R.tap = tap;
  };
  rf(L.oproj, d.wo, d.o, d.a * d.d / d.n_shards, d.tap_attn);
  rf(L.down, d.wdown, d.act, d.s / d.n_shards, d.tap_ffn);
  L.kc = d.kc;
  L.vc = d.vc;
}

bool mega_supported(int dt, int h, int a, int b, int d, int s) {
  const size_t esz = dt == DT_BF16 ? 2 : 4;
  const int lpr = (int)(d * esz / 16);
  if (lpr != 4 && lpr != 8 && lpr != 16 && lpr != 32) return false;
  if (h > 16384 || h % 4) return false;
  const int grp = a / b;
  if (grp != 1 && grp != 2 && grp != 4 && grp != 8) return false;
  return mega_smem_bytes(dt, h, a, b, d, s, 128) <= 200 * 1024;
}

size_t mega_smem_bytes(int dt, int h, int a, int b, int d, int s, int nsplit) {
  const size_t esz = dt == DT_BF16 ? 2 : 4;
  const int lpr = (int)(d * esz / 16), G = MW * (32 / (lpr ? lpr : 1));
  size_t attn = (size_t)2 * 256 * d + (size_t)(2 * G + (size_t)G * d) * 4 + (size_t)(a / b) * nsplit * 4;
  size_t x = (size_t)(s > a * d ? s : a * d) * 4;
  if ((size_t)h * 4 > x) x = (size_t)h * 4;
  return (attn > x ? attn : x) + 256;
}

template <typename WT, int LPR>
static cudaError_t launch_mega_t(cudaStream_t stream, MegaArgs& A, size_t smem, int grid) {
  auto kern = decode_token_kernel<WT, LPR>;
  static size_t attr_smem = 0;
  if (smem > attr_smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_smem = smem;
  }
  void* args[] = {&A};
  return cudaLaunchCooperativeKernel((void*)kern, dim3(grid), dim3(MW * 32), args, smem, stream);
}

cudaError_t launch_decode_token(const LaunchCtx& c, const MegaTokenDesc& t) {
  MegaArgs A{};
  A.layers = reinterpret_cast<const MegaLayer*>(t.layer_table_dev);
  A.n_layers = t.n_layers; A.emb = t.emb; A.vocab = t.vocab; A.max_seq = t.max_seq; A.h = t.h;
  A.x = t.x; A.ss_part = t.ss_part; A.n_parts = t.n_parts; A.tok_hist = t.tok_hist; A.pos = t.pos; A.err = t.err;
  A.q = t.q; A.o = t.o; A.attn_scratch = t.attn_scratch; A.tickets = t.tickets; A.a = t.a; A.b = t.b; A.nsplit = t.nsplit;
  A.bar = t.bar;
  A.ts = t.ts;
  A.prefetch = get_tuning(4);
  fill_cols(A.head, t.head, 0, NormIn{t.x, t.gain_final, t.ss_part, t.n_parts, t.eps}, t.h, 1, (t.vocab + 1) / 2);
  A.head.out = t.logits; A.head.amax_val = t.amax_val; A.head.amax_idx = t.amax_idx; A.head.ticket = t.tickets + t.b;
  A.head.tok_hist = t.tok_hist; A.head.pos_rw = t.pos; A.head.rows_total = t.vocab; A.head.advance = 1;
  int dev = 0, nsm = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, dev);
  const size_t smem = mega_smem_bytes(t.dt, t.h, t.a, t.b, t.d, t.s, t.nsplit);
  cudaError_t e = cudaMemsetAsync(t.bar, 0, 4, c.stream);
  if (e != cudaSuccess) return e;
  if (c.launches) ++*c.launches;
  const int lpr = (int)(t.d * dt_size(t.dt) / 16);
  if (t.dt == DT_BF16) {
    if (lpr == 16) return launch_mega_t<__nv_bfloat16, 16>(c.stream, A, smem, nsm);
    if (lpr == 8) return launch_mega_t<__nv_bfloat16, 8>(c.stream, A, smem, nsm);
    if (lpr == 4) return launch_mega_t<__nv_bfloat16, 4>(c.stream, A, smem, nsm);
  } else {
    if (lpr == 32) return launch_mega_t<float, 32>(c.stream, A, smem, nsm);
    if (lpr == 16) return launch_mega_t<float, 16>(c.stream, A, smem, nsm);
    if (lpr == 8) return launch_mega_t<float, 8>(c.stream, A, smem, nsm);
  }
  return cudaErrorInvalidValue;
}

}  // namespace tpi
