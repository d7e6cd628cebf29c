// Exchange kernels of the one-shard-per-rank form (Sec. 3.2's star allreduce in its one-hop shape): a rank stores its
// partial sums into every rank's receive area with plain stores and then sets one flag per destination; the consumer
// waits for the flags with a limit, adds the partial sums in rank order and the shortcut last.  Remote memory is only
// ever WRITTEN, never read, and every store names one destination.
#include "common.cuh"
#include "gemv_bodies.cuh"
#include "kernels.h"
#include "launch.cuh"

namespace tpi {

namespace {

// The flags of one exchange are published by ONE system-scope fence followed by relaxed stores, one per destination (a
// release store each would repeat the fence R times: measured 15 us of a 21 us kernel).
__device__ __forceinline__ void st_flag_sys(int* p, int v) {
  asm volatile("st.relaxed.sys.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_sys(const int* p) {
  int v;
  asm volatile("ld.acquire.sys.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

int sm_count_tp() {
  int dev = 0, n = 0;
  cudaGetDevice(&dev);
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
  return n;
}

struct RowPushArgs {
  const void* W;  // [rows][Ks]
  const float* x_in;
  int rows, Ks, seg_cap, drop;
  const int* epoch;
  unsigned* ticket;
  TpPeers peers;
};

// Persistent: one CTA per SM, x_in staged once, CTA `cta` owns rows [rows * cta / ncta, rows * (cta + 1) / ncta); its
// partial sums are collected in shared memory and leave as contiguous runs, one run per destination rank.
template <typename WT>
__global__ void __launch_bounds__(1024) tp_rowpush_kernel(const RowPushArgs A) {
  extern __shared__ __align__(16) float xs[];  // [Ks] staged inputs | [seg_cap] this CTA's partial sums
  float* seg = xs + A.Ks;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int cta = blockIdx.x, ncta = gridDim.x;
  const int lo = (int)((long long)A.rows * cta / ncta), hi = (int)((long long)A.rows * (cta + 1) / ncta);
  const WT* Wall = reinterpret_cast<const WT*>(A.W);
  pdl_wait();  // x_in and the exchange counter come from the kernels before
  pdl_launch_dependents();
  for (int k = threadIdx.x * 4; k < A.Ks; k += blockDim.x * 4)
    *reinterpret_cast<float4*>(xs + k) = *reinterpret_cast<const float4*>(A.x_in + k);
  __syncthreads();
  const int nvec = A.Ks / Elem<WT>::VEC;
  for (int g = lo + warp; g < hi; g += nw) {
    const uint4* wp[1] = {reinterpret_cast<const uint4*>(Wall + (size_t)g * A.Ks)};
    float acc[1] = {0.f};
    warp_dot<WT, 1>(wp, 0, xs, nvec, lane, acc);
    const float p = warp_sum(acc[0]);
    if (lane == 0) seg[g - lo] = p;
  }
  __syncthreads();
  const int c = __ldcg(A.epoch), parity = c & 1, R = A.peers.n_ranks;
  if (!A.drop) {
    for (int j = 0; j < R; ++j) {
      float* dst = A.peers.recv[j] + ((size_t)parity * A.peers.half + (size_t)A.peers.rank * A.rows + lo);
      for (int i = threadIdx.x; i < hi - lo; i += blockDim.x) dst[i] = seg[i];
    }
  }
  // One fence per CTA, not per thread (a system-scope fence in every thread cost five times the weight stream): the
  // barrier orders the CTA's stores before thread 0, whose fence then orders them, cumulatively, before its ticket.
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence_system();
    const unsigned t = atomicAdd(A.ticket, 1u);
    if (t == (unsigned)ncta - 1) {  // every CTA's stores are out: publish
      __threadfence_system();
      if (!A.drop)
        for (int j = 0; j < R; ++j) st_flag_sys(A.peers.flags[j] + parity * R + A.peers.rank, c + 1);
      *A.ticket = 0u;
    }
  }
}

__global__ void __launch_bounds__(1024) tp_bcast_kernel(const float* x, int h, const int* epoch, const TpPeers P, int drop) {
  pdl_wait();
  pdl_launch_dependents();
  const int c = __ldcg(epoch), parity = c & 1, R = P.n_ranks;
  if (drop) return;
  for (int j = 0; j < R; ++j) {
    float* dst = P.recv[j] + (size_t)parity * P.half;  // source 0
    for (int k = threadIdx.x; k < h; k += blockDim.x) dst[k] = x[k];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence_system();
    for (int j = 0; j < R; ++j) st_flag_sys(P.flags[j] + parity * R + 0, c + 1);
  }
}

struct RecvArgs {
  const float* recv;
  long long half;
  const int* flags;
  int* epoch;
  int n_ranks, h, mode, n_parts, wait_polls;
  float eps;
  float *x, *xhat, *tap, *ss_part;
  int* pos_advance;
  int* err;
};

__global__ void __launch_bounds__(1024) tp_recv_kernel(const RecvArgs A) {
  __shared__ float red[32];
  __shared__ int s_ok;
  pdl_wait();  // the counter was advanced by this rank's previous consumer
  pdl_launch_dependents();
  const int c = __ldcg(A.epoch), parity = c & 1, R = A.n_ranks;
  const int n_src = A.mode == 1 ? 1 : R;
  if (threadIdx.x == 0) s_ok = 1;
  __syncthreads();
  if ((int)threadIdx.x < n_src) {  // one thread per source; every wait has a limit
    const int* f = A.flags + parity * R + threadIdx.x;
    bool got = false;
    for (int i = 0; i < A.wait_polls; ++i) {
      if (ld_acquire_sys(f) == c + 1) { got = true; break; }
      if (i > 64) __nanosleep(100);
    }
    if (!got) {
      atomicCAS(A.err, DEVERR_NONE, DEVERR_WAIT_TIMEOUT);
      s_ok = 0;
    }
  }
  __syncthreads();
  if (!s_ok) return;  // nothing is changed: the host sees the error word and resets the group
  const float* P = A.recv + (size_t)parity * A.half;
  float ss = 0.f;
  for (int k = threadIdx.x; k < A.h; k += blockDim.x) {
    float s = __ldcg(P + k);  // the master's own partial (rank 0) ...
    if (A.mode == 0) {
      for (int i = 1; i < R; ++i) s += __ldcg(P + (size_t)i * A.h + k);  // ... plus the workers', rank order
      s += A.x[k];            // shortcut is added after the allreduce (Eq. 1-2)
    }
    A.x[k] = s;
    if (A.tap) A.tap[k] = s;
    ss = fmaf(s, s, ss);
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)A.h + A.eps);
  for (int k = threadIdx.x; k < A.h; k += blockDim.x) A.xhat[k] = A.x[k] * r;
  for (int i = threadIdx.x; i < A.n_parts; i += blockDim.x) A.ss_part[i] = i ? 0.f : ss;
  if (threadIdx.x == 0) {
    *A.epoch = c + 1;
    if (A.pos_advance) *A.pos_advance += 1;
  }
}


// Prompt pass: a block of n floats (T x h) goes to every rank's slot of this source.  Many CTAs copy, the last to
// finish publishes the flags.
__global__ void __launch_bounds__(256) tp_push_rows_kernel(const float* src, size_t n, const int* epoch, unsigned* ticket,
                                                           const TpPeers P, int src_rank, int drop) {
  pdl_wait();
  pdl_launch_dependents();
  const int c = __ldcg(epoch), parity = c & 1, R = P.n_ranks;
  if (!drop) {
    const size_t n4 = n >> 2;
    for (int j = 0; j < R; ++j) {
      float4* dst = reinterpret_cast<float4*>(P.recv[j] + (size_t)parity * P.half + (size_t)src_rank * n);
      const float4* s4 = reinterpret_cast<const float4*>(src);
      for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) dst[i] = s4[i];
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence_system();
    const unsigned t = atomicAdd(ticket, 1u);
    if (t == gridDim.x - 1) {
      __threadfence_system();
      if (!drop)
        for (int j = 0; j < R; ++j) st_flag_sys(P.flags[j] + parity * R + src_rank, c + 1);
      *ticket = 0u;
    }
  }
}

// The consumer's wait alone: one thread per source, bounded; then the counter moves on.
__global__ void tp_wait_kernel(const int* flags, int* epoch, int n_ranks, int n_src, int* err, int wait_polls) {
  __shared__ int s_ok;
  pdl_wait();
  pdl_launch_dependents();
  const int c = __ldcg(epoch), parity = c & 1;
  if (threadIdx.x == 0) s_ok = 1;
  __syncthreads();
  if ((int)threadIdx.x < n_src) {
    const int* f = flags + parity * n_ranks + threadIdx.x;
    bool got = false;
    for (int i = 0; i < wait_polls; ++i) {
      if (ld_acquire_sys(f) == c + 1) { got = true; break; }
      if (i > 64) __nanosleep(100);
    }
    if (!got) {
      atomicCAS(err, DEVERR_NONE, DEVERR_WAIT_TIMEOUT);
      s_ok = 0;
    }
  }
  __syncthreads();
  if (s_ok && threadIdx.x == 0) *epoch = c + 1;
}

}  // namespace

cudaError_t launch_tp_rowpush(const LaunchCtx& c, int dt, const void* W, const float* x_in, int rows, int Ks, const int* epoch,
                              unsigned* ticket, const TpPeers& peers, int drop) {
  const int vec = dt == DT_BF16 ? 8 : 4;
  if (rows < 1 || Ks < vec || Ks % vec || peers.n_ranks < 1 || peers.n_ranks > TP_MAX_RANKS) return cudaErrorInvalidValue;
  int grid = sm_count_tp();
  if (grid > rows) grid = rows;
  const int per = (rows + grid - 1) / grid;
  int warps = per < 32 ? per : 32;
  if (warps < 4) warps = 4;
  RowPushArgs A{W, x_in, rows, Ks, per + 1, drop, epoch, ticket, peers};
  const size_t smem = ((size_t)Ks + per + 1) * sizeof(float);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  auto go = [&](auto wt) -> cudaError_t {
    using WT = decltype(wt);
    auto kern = tp_rowpush_kernel<WT>;
    static PerDeviceOnce attr_done;
    if (!attr_done.get()) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return e;
      attr_done.set();
    }
    return launch_kernel(c, kern, dim3(grid), dim3(warps * 32), smem, A);
  };
  return dt == DT_BF16 ? go(__nv_bfloat16{}) : go(float{});
}

cudaError_t launch_tp_push_rows(const LaunchCtx& c, const float* src, size_t n, const int* epoch, unsigned* ticket,
                                const TpPeers& peers, int as_rank0, int drop) {
  if (n < 4 || n % 4 || (long long)(n * peers.n_ranks) > peers.half) return cudaErrorInvalidValue;
  size_t blocks = (n / 4 + 255) / 256;
  const size_t cap = (size_t)sm_count_tp() * 4;
  if (blocks > cap) blocks = cap;
  return launch_kernel(c, tp_push_rows_kernel, dim3((unsigned)blocks), dim3(256), 0, src, n, epoch, ticket, peers,
                       as_rank0 ? 0 : peers.rank, drop);
}

cudaError_t launch_tp_wait(const LaunchCtx& c, const int* flags, int* epoch, int n_ranks, int n_src, int* err, int wait_polls) {
  if (n_ranks < 1 || n_ranks > TP_MAX_RANKS || n_src < 1 || n_src > n_ranks || wait_polls < 1 || !err) return cudaErrorInvalidValue;
  return launch_kernel(c, tp_wait_kernel, dim3(1), dim3(32), 0, flags, epoch, n_ranks, n_src, err, wait_polls);
}

cudaError_t launch_tp_bcast(const LaunchCtx& c, const float* x, int h, const int* epoch, const TpPeers& peers, int drop) {
  return launch_kernel(c, tp_bcast_kernel, dim3(1), dim3(1024), 0, x, h, epoch, peers, drop);
}

cudaError_t launch_tp_recv(const LaunchCtx& c, const float* recv, long long half, const int* flags, int* epoch, int n_ranks, int h,
                           int mode, float eps, float* x, float* xhat, float* tap, float* ss_part, int n_parts, int* pos_advance,
                           int* err, int wait_polls) {
  if (n_ranks < 1 || n_ranks > TP_MAX_RANKS || wait_polls < 1 || !err || half < (long long)n_ranks * h) return cudaErrorInvalidValue;
  RecvArgs A{recv, half, flags, epoch, n_ranks, h, mode, n_parts, wait_polls, eps, x, xhat, tap, ss_part, pos_advance, err};
  return launch_kernel(c, tp_recv_kernel, dim3(1), dim3(1024), 0, A);
}

}  // namespace tpi
