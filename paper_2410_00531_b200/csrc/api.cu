// C ABI of the library: model set-up (weight partition + packing), the per-token
// step driver, the prompt pass, and the sliding-window block ring on CUDA streams.
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <chrono>
#include <new>
#include <thread>
#include <vector>

#include <cuda_bf16.h>

#include "../../include/tpi.h"
#include "kernels.h"
#include "plan.h"
#include "ring.h"

using namespace tpi;

// ------------------------------------------------------------------------------ errors
static thread_local char g_err[512] = "";
static int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof g_err, fmt, ap);
  va_end(ap);
  return code;
}
#define CK(call)                                                                                          \
  do {                                                                                                    \
    cudaError_t e_ = (call);                                                                              \
    if (e_ != cudaSuccess)                                                                                \
      return fail(TPI_ERR_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
  } while (0)
#define TRY(call)                  \
  do {                             \
    int rc_ = (call);              \
    if (rc_ != TPI_OK) return rc_; \
  } while (0)

extern "C" const char* tpi_last_error(void) { return g_err; }
// lets the library's other translation units leave a message for tpi_last_error()
extern "C" void tpi_internal_set_error(const char* msg) { snprintf(g_err, sizeof g_err, "%s", msg ? msg : ""); }
extern "C" const char* tpi_strerror(int code) {
  switch (code) {
    case TPI_OK: return "ok";
    case TPI_ERR_INVALID_ARG: return "invalid argument";
    case TPI_ERR_SHAPE: return "unsupported shape or shard count";
    case TPI_ERR_NOMEM: return "arena too small";
    case TPI_ERR_SEQ_OVERFLOW: return "sequence capacity exceeded";
    case TPI_ERR_TOKEN_RANGE: return "token id out of range";
    case TPI_ERR_CUDA: return "CUDA runtime error";
    case TPI_ERR_TIMEOUT: return "bounded wait ran out";
    case TPI_ERR_DEVICE_CHECK: return "device-side self check failed";
    case TPI_ERR_STATE: return "call not valid in this state";
    case TPI_ERR_CALLBACK: return "weight callback failed";
    default: return "unknown error";
  }
}

// ------------------------------------------------------------------------------ model
struct tpi_model {
  tpi_config cfg{};
  tpi_resources res{};
  tpi_fill_fn fill = nullptr;
  void* user = nullptr;
  int N = 1, window = 0;
  bool host_images = false;
  Plan plan{};
  char* dev = nullptr;
  char* host = nullptr;
  cudaStream_t cs = nullptr, ps = nullptr;
  bool own_cs = false, own_ps = false;
  int opt_graph = 1, opt_pdl = 1, opt_profile = 0, opt_tensor = 1, opt_mega = 0;
  bool mega_ready = false;  // the whole-token kernel's layer table is in device memory
  int position = 0;
  // window ring
  Ring ring;
  // partition of the kv heads (with their query-head groups) and of the FFN columns over the shards: prefix sums,
  // N + 1 entries each.  unequal = false: the uniform p_i = 1/N.  With unequal proportions the QKV rows are packed
  // in the unsharded order (their results do not depend on who computes them) and the row-sharded O / down
  // matrices follow the partition, which is where it decides the grouping of the partial sums.
  std::vector<int> kv0, f0;
  bool unequal = false;
  int retain_T = 0;                  // keep the FFN block of every T-th layer resident beside the window (0: none)
  std::vector<char> retained;        // per block
  std::vector<size_t> retained_off;  // byte offset of a retained block after the window slots
  size_t retained_bytes = 0;
  std::vector<cudaEvent_t> ev_loaded, ev_released;
  uint64_t link_bytes = 0;
  // graph of one resident decode step
  cudaGraphExec_t graph_exec = nullptr;
  int graph_launches = 0;
  // timing
  cudaEvent_t ev_t0 = nullptr, ev_t1 = nullptr, ev_done = nullptr;
  std::vector<cudaEvent_t> prof_ev;  // pairs around gate/up GEMVs (profile mode)
  size_t prof_used = 0;
  double prof_ms_sum = 0;
  uint32_t prof_samples = 0;
  // scheduler diagnostics (profile mode, decode only): event pairs around each block's kernels on the
  // compute stream (kinds 0 attention, 1 FFN) and around each block copy on the copy stream (kinds 2, 3)
  struct TimedPair { cudaEvent_t a, b; int kind; };
  std::vector<TimedPair> sched_pending;
  std::vector<cudaEvent_t> sched_free;
  cudaEvent_t sched_open = nullptr;
  bool sched_rec = false;
  double sched_sum[4] = {0, 0, 0, 0};
  uint32_t sched_n[4] = {0, 0, 0, 0};
  std::vector<cudaEvent_t> stall_ev;  // pairs around window waits (profile mode)
  size_t stall_used = 0;
  double stall_ms = 0;
  tpi_stats st{};
  double wait_deadline_s = 900.0;
};

template <typename T>
static T* dptr(tpi_model* m, size_t off) { return reinterpret_cast<T*>(m->dev + off); }

static void uniform_partition(tpi_model* m) {
  const int N = m->N;
  m->kv0.assign(N + 1, 0);
  m->f0.assign(N + 1, 0);
  for (int i = 0; i <= N; ++i) { m->kv0[i] = m->cfg.n_kv_heads / N * i; m->f0[i] = m->cfg.ffn / N * i; }
  m->unequal = false;
}

static int validate(const tpi_config* c, int N) {
  if (!c) return fail(TPI_ERR_INVALID_ARG, "null config");
  if (c->n_layers < 1 || c->hidden < 1 || c->n_heads < 1 || c->n_kv_heads < 1 || c->head_dim < 1 ||
      c->ffn < 1 || c->vocab < 1 || c->max_seq < 1 || c->max_prefill < 1)
    return fail(TPI_ERR_INVALID_ARG, "config sizes must be positive");
  if (c->dtype != TPI_F32 && c->dtype != TPI_BF16) return fail(TPI_ERR_INVALID_ARG, "unknown dtype %d", c->dtype);
  if (N < 1) return fail(TPI_ERR_INVALID_ARG, "n_shards must be >= 1");
  const int vec = c->dtype == TPI_BF16 ? 8 : 4;
  if (c->n_heads % c->n_kv_heads) return fail(TPI_ERR_SHAPE, "kv heads must divide heads");
  const int grp = c->n_heads / c->n_kv_heads;
  // the tensor-core attention kernels (bf16 cache, head_dim 64 or 128) take any group of up to 8 query heads
  const bool any_grp = c->dtype == TPI_BF16 && (c->head_dim == 64 || c->head_dim == 128) && grp <= 8;
  if (!any_grp && grp != 1 && grp != 2 && grp != 4 && grp != 8)
    return fail(TPI_ERR_SHAPE, "heads per kv head must be 1, 2, 4 or 8 (any count up to 8 for bf16 with head_dim 64 or 128)");
  if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return fail(TPI_ERR_SHAPE, "head_dim must be 32, 64 or 128");
  if (c->n_heads % N || c->n_kv_heads % N || c->ffn % N)
    return fail(TPI_ERR_SHAPE, "n_shards=%d must divide heads (%d), kv heads (%d) and ffn (%d)", N, c->n_heads,
                c->n_kv_heads, c->ffn);
  if (c->hidden % vec || (c->ffn / N) % vec || (c->n_heads / N * c->head_dim) % vec)
    return fail(TPI_ERR_SHAPE, "hidden, ffn/N and heads*d/N must be multiples of %d elements (16 bytes)", vec);
  if (c->hidden % 4) return fail(TPI_ERR_SHAPE, "hidden must be a multiple of 4");
  return TPI_OK;
}

extern "C" int tpi_query_arena(const tpi_config* cfg, int n_shards_max, int window_blocks, int keep_host_images,
                               size_t* dev_bytes, size_t* host_bytes) {
  TRY(validate(cfg, 1));
  if (n_shards_max < 1 || window_blocks < 0) return fail(TPI_ERR_INVALID_ARG, "bad shard/window count");
  if (n_shards_max < 8) n_shards_max = 8;  // tpi_load_model always plans for at least 8 shards
  Plan p;
  make_plan(*cfg, n_shards_max, window_blocks, keep_host_images, head_argmax_blocks(cfg->vocab), &p, dev_bytes,
            host_bytes);
  return TPI_OK;
}

extern "C" int tpi_block_bytes(const tpi_config* cfg, size_t* attn_block_bytes, size_t* ffn_block_bytes) {
  TRY(validate(cfg, 1));
  const BlockLayout b = block_layout(*cfg);
  if (attn_block_bytes) *attn_block_bytes = b.attn_bytes;
  if (ffn_block_bytes) *ffn_block_bytes = b.ffn_bytes;
  return TPI_OK;
}

// ------------------------------------------------------------------------------ host-side wait
static int wait_event(tpi_model* m, cudaEvent_t ev) {
  const auto t0 = std::chrono::steady_clock::now();
  for (long spins = 0;; ++spins) {
    cudaError_t e = cudaEventQuery(ev);
    if (e == cudaSuccess) return TPI_OK;
    if (e != cudaErrorNotReady) return fail(TPI_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
    if (spins > 2000) std::this_thread::yield();
    if ((spins & 1023) == 0) {
      const double s = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
      if (s > m->wait_deadline_s) return fail(TPI_ERR_TIMEOUT, "device did not finish within %.0f s", s);
    }
  }
}

// ------------------------------------------------------------------------------ weight packing
namespace {
struct RowCopy {  // destination of one source row (or row segment) inside a block image
  size_t dst_off;
};
}  // namespace

static void f32_from_storage(const void* src, int dtype, float* dst, size_t n) {
  if (dtype == TPI_F32) memcpy(dst, src, n * 4);
  else {
    const uint16_t* s = (const uint16_t*)src;
    for (size_t i = 0; i < n; ++i) {
      uint32_t u = (uint32_t)s[i] << 16;
      memcpy(dst + i, &u, 4);
    }
  }
}

// Copies rows [row0, row0+n) of tensor `tid` from `src` into the layer's attention or FFN image.
static void place_rows(const tpi_config& c, const BlockLayout& bl, int N, const int* kv0, const int* f0, bool unequal,
                       int tid, int64_t row0, int64_t n, const char* src, char* attn_img, char* ffn_img) {
  const size_t B = elem_size(c.dtype), h = c.hidden, d = c.head_dim;
  const int Nq = unequal ? 1 : N;  // column-sharded rows of an unequal partition are packed as one shard
  const int64_t hps_rows = (int64_t)c.n_heads / Nq * d, kps_rows = (int64_t)c.n_kv_heads / Nq * d;
  const int64_t qkv_rows = hps_rows + 2 * kps_rows, spn = c.ffn / Nq;
  const int grp = c.n_heads / c.n_kv_heads;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    const int64_t r = row0 + i;
    switch (tid) {
      case TPI_T_WQ: {
        const int64_t sh = r / hps_rows, rl = r % hps_rows;
        memcpy(attn_img + bl.off_qkv + (size_t)(sh * qkv_rows + rl) * h * B, src + (size_t)i * h * B, h * B);
      } break;
      case TPI_T_WK: {
        const int64_t sh = r / kps_rows, rl = r % kps_rows;
        memcpy(attn_img + bl.off_qkv + (size_t)(sh * qkv_rows + hps_rows + rl) * h * B, src + (size_t)i * h * B, h * B);
      } break;
      case TPI_T_WV: {
        const int64_t sh = r / kps_rows, rl = r % kps_rows;
        memcpy(attn_img + bl.off_qkv + (size_t)(sh * qkv_rows + hps_rows + kps_rows + rl) * h * B,
               src + (size_t)i * h * B, h * B);
      } break;
      case TPI_T_WGATE:
      case TPI_T_WUP: {
        const int64_t sh = r / spn, j = r % spn;
        memcpy(ffn_img + bl.off_gu + (size_t)(sh * 2 * spn + 2 * j + (tid == TPI_T_WUP)) * h * B,
               src + (size_t)i * h * B, h * B);
      } break;
      case TPI_T_WO: {  // shard sh: [h][its heads' columns], shards one after another
        const size_t K = (size_t)c.n_heads * d;
        for (int sh = 0; sh < N; ++sh) {
          const size_t k_lo = (size_t)kv0[sh] * grp * d, Ks = (size_t)(kv0[sh + 1] - kv0[sh]) * grp * d;
          memcpy(attn_img + bl.off_wo + (h * k_lo + (size_t)r * Ks) * B, src + ((size_t)i * K + k_lo) * B, Ks * B);
        }
      } break;
      case TPI_T_WDOWN: {
        const size_t K = c.ffn;
        for (int sh = 0; sh < N; ++sh) {
          const size_t k_lo = (size_t)f0[sh], Ks = (size_t)(f0[sh + 1] - f0[sh]);
          memcpy(ffn_img + bl.off_down + (h * k_lo + (size_t)r * Ks) * B, src + ((size_t)i * K + k_lo) * B, Ks * B);
        }
      } break;
      default: break;
    }
  }
}

static int64_t tensor_rows(const tpi_config& c, int tid, size_t* row_len) {
  const int64_t h = c.hidden, d = c.head_dim;
  switch (tid) {
    case TPI_T_EMB: case TPI_T_HEAD: *row_len = h; return c.vocab;
    case TPI_T_FINAL_NORM: case TPI_T_ATTN_NORM: case TPI_T_FFN_NORM: *row_len = h; return 1;
    case TPI_T_WQ: *row_len = h; return c.n_heads * d;
    case TPI_T_WK: case TPI_T_WV: *row_len = h; return c.n_kv_heads * d;
    case TPI_T_WO: *row_len = c.n_heads * d; return h;
    case TPI_T_WGATE: case TPI_T_WUP: *row_len = h; return c.ffn;
    case TPI_T_WDOWN: *row_len = c.ffn; return h;
    default: *row_len = 0; return 0;
  }
}

static char* host_image(tpi_model* m, int block) {  // block = 2*layer + (0 attn | 1 ffn)
  const BlockLayout& bl = m->plan.bl;
  const size_t per_layer = bl.attn_bytes + bl.ffn_bytes;
  return m->host + m->plan.h_images + (size_t)(block / 2) * per_layer + (block % 2 ? bl.attn_bytes : 0);
}
static size_t block_size(const tpi_model* m, int block) {
  return block % 2 ? m->plan.bl.ffn_bytes : m->plan.bl.attn_bytes;
}
static char* resident_block(tpi_model* m, int block) {
  const BlockLayout& bl = m->plan.bl;
  const size_t per_layer = bl.attn_bytes + bl.ffn_bytes;
  return m->dev + m->plan.blocks + (size_t)(block / 2) * per_layer + (block % 2 ? bl.attn_bytes : 0);
}
static char* slot_ptr(tpi_model* m, int slot) {
  const BlockLayout& bl = m->plan.bl;
  const int nA = m->ring.n_attn_slots();
  if (slot < nA) return m->dev + m->plan.blocks + (size_t)slot * bl.attn_bytes;
  return m->dev + m->plan.blocks + (size_t)nA * bl.attn_bytes + (size_t)(slot - nA) * bl.ffn_bytes;
}

// Streams one global tensor (EMB / HEAD) to the device through the staging buffer.
static int load_global(tpi_model* m, int tid, size_t dev_off) {
  const tpi_config& c = m->cfg;
  size_t row_len;
  const int64_t rows = tensor_rows(c, tid, &row_len);
  const size_t rb = row_len * elem_size(c.dtype);
  const int64_t chunk = (int64_t)(m->plan.h_stage_bytes / rb);
  char* stage = m->host + m->plan.h_stage;
  for (int64_t r0 = 0; r0 < rows; r0 += chunk) {
    const int64_t n = rows - r0 < chunk ? rows - r0 : chunk;
    if (m->fill(m->user, tid, 0, r0, n, stage)) return fail(TPI_ERR_CALLBACK, "fill(tensor %d) failed", tid);
    CK(cudaMemcpyAsync(m->dev + dev_off + (size_t)r0 * rb, stage, (size_t)n * rb, cudaMemcpyHostToDevice, m->cs));
    CK(cudaStreamSynchronize(m->cs));
  }
  return TPI_OK;
}

// Builds the two block images of one layer in host memory (Step 1: partition for N devices).
static int build_layer_images(tpi_model* m, int layer, char* attn_img, char* ffn_img) {
  const tpi_config& c = m->cfg;
  char* stage = m->host + m->plan.h_stage;
  static const int tids[] = {TPI_T_ATTN_NORM, TPI_T_WQ, TPI_T_WK, TPI_T_WV, TPI_T_WO,
                             TPI_T_FFN_NORM, TPI_T_WGATE, TPI_T_WUP, TPI_T_WDOWN};
  for (int tid : tids) {
    size_t row_len;
    const int64_t rows = tensor_rows(c, tid, &row_len);
    const size_t rb = row_len * elem_size(c.dtype);
    const int64_t chunk = (int64_t)(m->plan.h_stage_bytes / rb);
    for (int64_t r0 = 0; r0 < rows; r0 += chunk) {
      const int64_t n = rows - r0 < chunk ? rows - r0 : chunk;
      if (m->fill(m->user, tid, layer, r0, n, stage))
        return fail(TPI_ERR_CALLBACK, "fill(tensor %d, layer %d) failed", tid, layer);
      if (tid == TPI_T_ATTN_NORM) f32_from_storage(stage, c.dtype, (float*)attn_img, c.hidden);
      else if (tid == TPI_T_FFN_NORM) f32_from_storage(stage, c.dtype, (float*)ffn_img, c.hidden);
      else place_rows(c, m->plan.bl, m->N, m->kv0.data(), m->f0.data(), m->unequal, tid, r0, n, stage, attn_img, ffn_img);
    }
  }
  return TPI_OK;
}

static int load_layers(tpi_model* m) {
  const tpi_config& c = m->cfg;
  const BlockLayout& bl = m->plan.bl;
  for (int l = 0; l < c.n_layers; ++l) {
    char *ai, *fi;
    if (m->host_images) { ai = host_image(m, 2 * l); fi = host_image(m, 2 * l + 1); }
    else { ai = m->host + m->plan.h_bounce; fi = ai; }
    if (m->host_images) {
      TRY(build_layer_images(m, l, ai, fi));
      if (m->window == 0) {
        CK(cudaMemcpyAsync(resident_block(m, 2 * l), ai, bl.attn_bytes, cudaMemcpyHostToDevice, m->cs));
        CK(cudaMemcpyAsync(resident_block(m, 2 * l + 1), fi, bl.ffn_bytes, cudaMemcpyHostToDevice, m->cs));
      }
    } else {
      // one bounce buffer: build and ship the attention image, then the FFN image
      const tpi_config& cc = m->cfg;
      char* stage = m->host + m->plan.h_stage;
      for (int pass = 0; pass < 2; ++pass) {
        static const int at[] = {TPI_T_ATTN_NORM, TPI_T_WQ, TPI_T_WK, TPI_T_WV, TPI_T_WO};
        static const int ft[] = {TPI_T_FFN_NORM, TPI_T_WGATE, TPI_T_WUP, TPI_T_WDOWN};
        const int* tids = pass ? ft : at;
        const int nt = pass ? 4 : 5;
        for (int k = 0; k < nt; ++k) {
          const int tid = tids[k];
          size_t row_len;
          const int64_t rows = tensor_rows(cc, tid, &row_len);
          const size_t rb = row_len * elem_size(cc.dtype);
          const int64_t chunk = (int64_t)(m->plan.h_stage_bytes / rb);
          for (int64_t r0 = 0; r0 < rows; r0 += chunk) {
            const int64_t n = rows - r0 < chunk ? rows - r0 : chunk;
            if (m->fill(m->user, tid, l, r0, n, stage))
              return fail(TPI_ERR_CALLBACK, "fill(tensor %d, layer %d) failed", tid, l);
            if (tid == TPI_T_ATTN_NORM || tid == TPI_T_FFN_NORM) f32_from_storage(stage, cc.dtype, (float*)ai, cc.hidden);
            else place_rows(cc, bl, m->N, m->kv0.data(), m->f0.data(), m->unequal, tid, r0, n, stage, ai, ai);
          }
        }
        CK(cudaMemcpyAsync(resident_block(m, 2 * l + pass), ai, pass ? bl.ffn_bytes : bl.attn_bytes,
                           cudaMemcpyHostToDevice, m->cs));
        CK(cudaStreamSynchronize(m->cs));
      }
    }
  }
  CK(cudaStreamSynchronize(m->cs));
  return TPI_OK;
}

// ------------------------------------------------------------------------------ scheduler diagnostics
static cudaEvent_t sched_event(tpi_model* m) {
  if (!m->sched_free.empty()) { cudaEvent_t e = m->sched_free.back(); m->sched_free.pop_back(); return e; }
  if (m->sched_pending.size() >= 8192) return nullptr;  // bounded: further samples are dropped until a harvest
  cudaEvent_t e = nullptr;
  return cudaEventCreate(&e) == cudaSuccess ? e : nullptr;
}
// completed pairs go into the running means; pairs still in flight (the loader runs ahead) stay for the next call
static void sched_harvest(tpi_model* m) {
  size_t keep = 0;
  for (size_t i = 0; i < m->sched_pending.size(); ++i) {
    tpi_model::TimedPair tp = m->sched_pending[i];
    float ms = 0;
    if (cudaEventQuery(tp.b) == cudaSuccess && cudaEventElapsedTime(&ms, tp.a, tp.b) == cudaSuccess) {
      m->sched_sum[tp.kind] += ms;
      ++m->sched_n[tp.kind];
      m->sched_free.push_back(tp.a);
      m->sched_free.push_back(tp.b);
    } else {
      cudaGetLastError();  // cudaErrorNotReady is expected here
      m->sched_pending[keep++] = tp;
    }
  }
  m->sched_pending.resize(keep);
}

// ------------------------------------------------------------------------------ ring back end (CUDA)
static int be_copy_wait_released(void* ctx, int slot) {
  tpi_model* m = (tpi_model*)ctx;
  CK(cudaStreamWaitEvent(m->ps, m->ev_released[slot], 0));
  return 0;
}
static int be_copy_block(void* ctx, int slot, int block) {
  tpi_model* m = (tpi_model*)ctx;
  const size_t n = block_size(m, block);
  cudaEvent_t a = nullptr, b = nullptr;
  if (m->sched_rec && (a = sched_event(m)) && (b = sched_event(m))) CK(cudaEventRecord(a, m->ps));
  CK(cudaMemcpyAsync(slot_ptr(m, slot), host_image(m, block), n, cudaMemcpyHostToDevice, m->ps));
  if (a && b) {
    CK(cudaEventRecord(b, m->ps));
    m->sched_pending.push_back({a, b, 2 + (block & 1)});
  } else if (a) m->sched_free.push_back(a);
  m->link_bytes += n;
  return 0;
}
static int be_copy_record_loaded(void* ctx, int slot) {
  tpi_model* m = (tpi_model*)ctx;
  CK(cudaEventRecord(m->ev_loaded[slot], m->ps));
  return 0;
}
static int be_compute_wait_loaded(void* ctx, int slot) {
  tpi_model* m = (tpi_model*)ctx;
  cudaEvent_t a = nullptr, b = nullptr;
  if (m->opt_profile && m->stall_used + 2 <= m->stall_ev.size()) {
    a = m->stall_ev[m->stall_used++];
    b = m->stall_ev[m->stall_used++];
    CK(cudaEventRecord(a, m->cs));
  }
  CK(cudaStreamWaitEvent(m->cs, m->ev_loaded[slot], 0));
  if (b) CK(cudaEventRecord(b, m->cs));
  return 0;
}
static int be_compute_record_released(void* ctx, int slot) {
  tpi_model* m = (tpi_model*)ctx;
  CK(cudaEventRecord(m->ev_released[slot], m->cs));
  return 0;
}

static void drop_graph(tpi_model* m);
// Whole-token kernel: per-layer argument table (pointers into the resident block images and the arena).
static int ensure_mega(tpi_model* m) {
  if (m->mega_ready) return TPI_OK;
  const tpi_config& c = m->cfg;
  const Plan& p = m->plan;
  const BlockLayout& bl = p.bl;
  char* tab = m->host + p.h_stage;  // staging area is free outside of loading
  const int n_parts = rowshard_fused_parts(c.hidden);
  for (int l = 0; l < c.n_layers; ++l) {
    char* ab = m->dev + p.blocks + (size_t)l * (bl.attn_bytes + bl.ffn_bytes);
    char* fb = ab + bl.attn_bytes;
    MegaLayerDesc d{};
    d.wqkv = ab + bl.off_qkv; d.wo = ab + bl.off_wo; d.wgu = fb + bl.off_gu; d.wdown = fb + bl.off_down;
    d.gain_attn = (const float*)ab; d.gain_ffn = (const float*)fb;
    d.kc = m->dev + p.kcache + (size_t)l * p.kv_layer_bytes;
    d.vc = m->dev + p.vcache + (size_t)l * p.kv_layer_bytes;
    d.tap_attn = (float*)(m->dev + p.taps) + (size_t)(2 * l) * c.hidden;
    d.tap_ffn = d.tap_attn + c.hidden;
    d.x = (float*)(m->dev + p.x); d.ss_part = (float*)(m->dev + p.ss_part); d.q = (float*)(m->dev + p.q);
    d.o = (float*)(m->dev + p.o); d.act = (float*)(m->dev + p.act);
    d.pos = (const int*)(m->dev + p.pos); d.rope = (const float2*)(m->dev + p.rope);
    d.n_parts = n_parts; d.h = c.hidden; d.a = c.n_heads; d.b = c.n_kv_heads; d.d = c.head_dim; d.s = c.ffn;
    d.n_shards = m->N; d.max_seq = c.max_seq; d.eps = c.rms_eps;
    mega_fill_layer(tab, l, d);
  }
  CK(cudaMemcpyAsync(m->dev + p.mega_table, tab, mega_layer_table_bytes(c.n_layers), cudaMemcpyHostToDevice, m->cs));
  CK(cudaStreamSynchronize(m->cs));
  m->mega_ready = true;
  return TPI_OK;
}

static bool mega_usable(const tpi_model* m) {
  const tpi_config& c = m->cfg;
  return m->opt_mega && m->window <= 0 && !m->opt_profile && !m->unequal &&
         mega_supported(c.dtype, c.hidden, c.n_heads, c.n_kv_heads, c.head_dim, c.ffn) &&
         mega_layer_table_bytes(c.n_layers) <= m->plan.h_stage_bytes &&
         mega_smem_bytes(c.dtype, c.hidden, c.n_heads, c.n_kv_heads, c.head_dim, c.ffn, m->plan.nsplit) <= 200 * 1024;
}

static int enqueue_decode_mega(tpi_model* m, LaunchCtx& lc) {
  const tpi_config& c = m->cfg;
  const Plan& p = m->plan;
  MegaTokenDesc t{};
  t.layer_table_dev = m->dev + p.mega_table;
  t.n_layers = c.n_layers; t.dt = c.dtype; t.vocab = c.vocab; t.max_seq = c.max_seq; t.h = c.hidden; t.a = c.n_heads;
  t.b = c.n_kv_heads; t.d = c.head_dim; t.s = c.ffn; t.nsplit = p.nsplit; t.n_parts = rowshard_fused_parts(c.hidden);
  t.eps = c.rms_eps; t.emb = m->dev + p.emb; t.head = m->dev + p.head; t.gain_final = (const float*)(m->dev + p.final_gain);
  t.x = (float*)(m->dev + p.x); t.ss_part = (float*)(m->dev + p.ss_part); t.q = (float*)(m->dev + p.q);
  t.o = (float*)(m->dev + p.o); t.attn_scratch = (float*)(m->dev + p.attn_scratch); t.logits = (float*)(m->dev + p.logits);
  t.amax_val = (float*)(m->dev + p.amax_val); t.amax_idx = (int*)(m->dev + p.amax_idx);
  t.tickets = (unsigned*)(m->dev + p.tickets); t.bar = (unsigned*)(m->dev + p.mega_bar);
  t.tok_hist = (int*)(m->dev + p.tok_hist); t.pos = (int*)(m->dev + p.pos); t.err = (int*)(m->dev + p.err);
  static const bool want_ts = getenv("TPI_MEGA_TS") != nullptr;  // phase-timing aid: stamps go to the prefill scratch
  t.ts = want_ts ? (unsigned long long*)(m->dev + p.pX) : nullptr;
  CK(launch_decode_token(lc, t));
  if (want_ts) {
    const int nb = 1 + 5 * c.n_layers;
    std::vector<unsigned long long> h(2 * nb);
    CK(cudaMemcpyAsync(h.data(), t.ts, h.size() * 8, cudaMemcpyDeviceToHost, m->cs));
    CK(cudaStreamSynchronize(m->cs));
    // per phase kind: time from the previous barrier's release to CTA 0's arrival (work) and arrival -> release (wait)
    double work[5] = {0, 0, 0, 0, 0}, wait[5] = {0, 0, 0, 0, 0};
    for (int l = 0; l < c.n_layers; ++l)
      for (int ph = 0; ph < 5; ++ph) {
        const int k = 1 + 5 * l + ph;
        work[ph] += (double)(h[2 * k] - h[2 * k - 1]);
        wait[ph] += (double)(h[2 * k + 1] - h[2 * k]);
      }
    static const char* nm[5] = {"qkv", "attn", "oproj", "gateup", "down"};
    for (int ph = 0; ph < 5; ++ph)
      fprintf(stderr, "[mega] %-6s work %.2f us  barrier wait %.2f us (per layer)\n", nm[ph], work[ph] / c.n_layers * 1e-3,
              wait[ph] / c.n_layers * 1e-3);
    fprintf(stderr, "[mega] token %.1f us\n", (double)(h[2 * nb - 1] - h[0]) * 1e-3);
  }
  return TPI_OK;
}

static void drop_graph(tpi_model* m) {
  m->mega_ready = false;
  if (m->graph_exec) cudaGraphExecDestroy(m->graph_exec);
  m->graph_exec = nullptr;
}

static int start_window(tpi_model* m) {
  for (auto e : m->ev_loaded) cudaEventDestroy(e);
  for (auto e : m->ev_released) cudaEventDestroy(e);
  m->ev_loaded.clear();
  m->ev_released.clear();
  if (m->window <= 0) return TPI_OK;
  RingBackend be;
  be.ctx = m;
  be.copy_wait_released = be_copy_wait_released;
  be.copy_block = be_copy_block;
  be.copy_record_loaded = be_copy_record_loaded;
  be.compute_wait_loaded = be_compute_wait_loaded;
  be.compute_record_released = be_compute_record_released;
  // Block retention (Prop. 6): the FFN block of every T-th layer stays resident after the window slots.
  const int nb = 2 * m->cfg.n_layers;
  m->retained.assign(nb, 0);
  m->retained_off.assign(nb, 0);
  m->retained_bytes = 0;
  {
    int nA, nF;
    window_slots(m->window, &nA, &nF);
    const size_t slots = (size_t)nA * m->plan.bl.attn_bytes + (size_t)nF * m->plan.bl.ffn_bytes;
    size_t off = slots;
    if (m->retain_T > 0)
      for (int l = 0; l < m->cfg.n_layers; l += m->retain_T) {
        m->retained[2 * l + 1] = 1;
        m->retained_off[2 * l + 1] = off;
        off += m->plan.bl.ffn_bytes;
      }
    m->retained_bytes = off - slots;
    if (m->plan.blocks + off > m->res.dev_bytes)
      return fail(TPI_ERR_NOMEM, "device arena too small for the window plus retained blocks: need %zu bytes, have %zu",
                  m->plan.blocks + off, m->res.dev_bytes);
    for (int b = 0; b < nb; ++b)
      if (m->retained[b])
        CK(cudaMemcpyAsync(m->dev + m->plan.blocks + m->retained_off[b], host_image(m, b), block_size(m, b),
                           cudaMemcpyHostToDevice, m->cs));
    CK(cudaStreamSynchronize(m->cs));
  }
  m->ring.configure(nb, m->window, be, m->retained.data());
  for (int i = 0; i < m->ring.n_slots(); ++i) {
    cudaEvent_t a, b;
    CK(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
    m->ev_loaded.push_back(a);
    m->ev_released.push_back(b);
  }
  const int rc = m->ring.pump();  // preload the first w blocks
  if (rc) return rc < 0 ? rc : fail(TPI_ERR_CUDA, "window start failed");
  return TPI_OK;
}

// ------------------------------------------------------------------------------ set-up
static int init_device_state(tpi_model* m) {
  const tpi_config& c = m->cfg;
  const Plan& p = m->plan;
  LaunchCtx lc{m->cs, false, nullptr};
  // rotary frequencies base^(-2i/d) in fp64 on the host, cos/sin table on the device
  const int half = c.head_dim / 2;
  double* invf = (double*)(m->host + p.h_stage);
  for (int i = 0; i < half; ++i) invf[i] = pow((double)c.rope_base, -2.0 * i / c.head_dim);
  CK(cudaMemcpyAsync(m->dev + p.inv_freq, invf, half * 8, cudaMemcpyHostToDevice, m->cs));
  CK(cudaStreamSynchronize(m->cs));
  CK(launch_rope_table(lc, dptr<double>(m, p.inv_freq), c.max_seq, half, dptr<float2>(m, p.rope)));
  CK(cudaMemsetAsync(m->dev + p.tickets, 0, (c.n_kv_heads + 1) * 4, m->cs));
  CK(cudaMemsetAsync(m->dev + p.tok_hist, 0, (c.max_seq + 2) * 4, m->cs));
  CK(cudaMemsetAsync(m->dev + p.pos, 0, 4, m->cs));
  CK(cudaMemsetAsync(m->dev + p.err, 0, 4, m->cs));
  CK(cudaMemsetAsync(m->dev + p.taps, 0, (size_t)c.n_layers * 2 * c.hidden * 4, m->cs));
  CK(cudaStreamSynchronize(m->cs));
  return TPI_OK;
}

static int load_all(tpi_model* m) {
  const tpi_config& c = m->cfg;
  TRY(load_global(m, TPI_T_EMB, m->plan.emb));
  TRY(load_global(m, TPI_T_HEAD, m->plan.head));
  {
    char* stage = m->host + m->plan.h_stage;
    if (m->fill(m->user, TPI_T_FINAL_NORM, 0, 0, 1, stage)) return fail(TPI_ERR_CALLBACK, "fill(final norm) failed");
    float* g = (float*)(stage + align_up((size_t)c.hidden * 4, 256));
    f32_from_storage(stage, c.dtype, g, c.hidden);
    CK(cudaMemcpyAsync(m->dev + m->plan.final_gain, g, c.hidden * 4, cudaMemcpyHostToDevice, m->cs));
    CK(cudaStreamSynchronize(m->cs));
  }
  return load_layers(m);
}

static int check_arenas(tpi_model* m, int window, bool host_images, Plan* out) {
  size_t need_d, need_h;
  make_plan(m->cfg, m->plan.n_shards_max, window, host_images, head_argmax_blocks(m->cfg.vocab), out, &need_d,
            &need_h);
  if (need_d > m->res.dev_bytes)
    return fail(TPI_ERR_NOMEM, "device arena too small: need %zu bytes, have %zu", need_d, m->res.dev_bytes);
  if (need_h > m->res.host_bytes)
    return fail(TPI_ERR_NOMEM, "host arena too small: need %zu bytes, have %zu", need_h, m->res.host_bytes);
  return TPI_OK;
}

extern "C" int tpi_load_model(const tpi_config* cfg, const tpi_resources* res, tpi_fill_fn fill, void* user,
                              int n_shards, int window_blocks, tpi_model** out) {
  if (!cfg || !res || !fill || !out) return fail(TPI_ERR_INVALID_ARG, "null argument");
  if (window_blocks < 0) return fail(TPI_ERR_INVALID_ARG, "window_blocks must be >= 0");
  TRY(validate(cfg, n_shards));
  if (!res->dev_arena || !res->host_arena) return fail(TPI_ERR_INVALID_ARG, "both arenas are required");
  if (((uintptr_t)res->dev_arena | (uintptr_t)res->host_arena) & 255)
    return fail(TPI_ERR_INVALID_ARG, "arenas must be 256-byte aligned");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1)
    return fail(TPI_ERR_CUDA, "no CUDA device: this library has no CPU path");
  tpi_model* m = new (std::nothrow) tpi_model();
  if (!m) return fail(TPI_ERR_NOMEM, "out of host memory");
  m->cfg = *cfg;
  m->res = *res;
  m->fill = fill;
  m->user = user;
  m->N = n_shards;
  uniform_partition(m);
  m->window = window_blocks;
  m->dev = (char*)res->dev_arena;
  m->host = (char*)res->host_arena;
  m->plan.n_shards_max = n_shards > 8 ? n_shards : 8;
  if (const char* tn = getenv("TPI_TUNE")) {  // "key=value,key=value": kernel tuning knobs (see kernels.h)
    int k = 0, v = 0, n = 0;
    while (sscanf(tn, "%d=%d%n", &k, &v, &n) == 2) {
      set_tuning(k, v);
      tn += n;
      if (*tn == ',') ++tn;
    }
  }
  if (const char* dl = getenv("TPI_WAIT_DEADLINE_S")) {  // bound on every host-side wait for the device
    const double v = atof(dl);
    if (v > 0) m->wait_deadline_s = v;
  }
  // keep host images when streaming, or when the host arena has room for them anyway
  Plan with_images;
  size_t nd, nh;
  make_plan(*cfg, m->plan.n_shards_max, window_blocks, 1, head_argmax_blocks(cfg->vocab), &with_images, &nd, &nh);
  m->host_images = window_blocks > 0 || nh <= res->host_bytes;
  int rc = check_arenas(m, window_blocks, m->host_images, &m->plan);
  if (rc) { delete m; return rc; }
  auto bail = [&](int code) { tpi_free(m); return code; };
  if (res->compute_stream) m->cs = (cudaStream_t)res->compute_stream;
  else { if (cudaStreamCreateWithFlags(&m->cs, cudaStreamNonBlocking) != cudaSuccess) return bail(fail(TPI_ERR_CUDA, "stream")); m->own_cs = true; }
  if (res->copy_stream) m->ps = (cudaStream_t)res->copy_stream;
  else { if (cudaStreamCreateWithFlags(&m->ps, cudaStreamNonBlocking) != cudaSuccess) return bail(fail(TPI_ERR_CUDA, "stream")); m->own_ps = true; }
  if (cudaEventCreate(&m->ev_t0) != cudaSuccess || cudaEventCreate(&m->ev_t1) != cudaSuccess ||
      cudaEventCreateWithFlags(&m->ev_done, cudaEventDisableTiming) != cudaSuccess)
    return bail(fail(TPI_ERR_CUDA, "event creation failed"));
  if ((rc = init_device_state(m))) return bail(rc);
  if ((rc = load_all(m))) return bail(rc);
  if ((rc = start_window(m))) return bail(rc);
  *out = m;
  return TPI_OK;
}

extern "C" void tpi_free(tpi_model* m) {
  if (!m) return;
  if (m->cs) cudaStreamSynchronize(m->cs);
  if (m->ps) cudaStreamSynchronize(m->ps);
  drop_graph(m);
  for (auto e : m->ev_loaded) cudaEventDestroy(e);
  for (auto e : m->ev_released) cudaEventDestroy(e);
  for (auto e : m->prof_ev) cudaEventDestroy(e);
  for (auto e : m->stall_ev) cudaEventDestroy(e);
  for (auto& tp : m->sched_pending) { cudaEventDestroy(tp.a); cudaEventDestroy(tp.b); }
  for (auto e : m->sched_free) cudaEventDestroy(e);
  if (m->sched_open) cudaEventDestroy(m->sched_open);
  if (m->ev_t0) cudaEventDestroy(m->ev_t0);
  if (m->ev_t1) cudaEventDestroy(m->ev_t1);
  if (m->ev_done) cudaEventDestroy(m->ev_done);
  if (m->own_cs) cudaStreamDestroy(m->cs);
  if (m->own_ps) cudaStreamDestroy(m->ps);
  delete m;
}

static int quiesce(tpi_model* m) {
  CK(cudaStreamSynchronize(m->cs));
  CK(cudaStreamSynchronize(m->ps));
  return TPI_OK;
}

static int write_position(tpi_model* m, int p) {
  int* io = (int*)(m->host + m->plan.h_io);
  io[0] = p;
  CK(cudaMemcpyAsync(m->dev + m->plan.pos, io, 4, cudaMemcpyHostToDevice, m->cs));
  CK(cudaStreamSynchronize(m->cs));
  m->position = p;
  return TPI_OK;
}

extern "C" int tpi_set_shards(tpi_model* m, int n_shards) {
  if (!m) return fail(TPI_ERR_INVALID_ARG, "null model");
  TRY(validate(&m->cfg, n_shards));
  if (n_shards > m->plan.n_shards_max) return fail(TPI_ERR_INVALID_ARG, "n_shards exceeds the planned maximum %d", m->plan.n_shards_max);
  TRY(quiesce(m));
  drop_graph(m);
  m->N = n_shards;
  uniform_partition(m);
  TRY(load_layers(m));
  TRY(start_window(m));
  return write_position(m, 0);
}

extern "C" int tpi_set_partition(tpi_model* m, int n_shards, const int32_t* kv_heads_per_shard,
                                 const int32_t* ffn_cols_per_shard) {
  if (!m || !kv_heads_per_shard || !ffn_cols_per_shard) return fail(TPI_ERR_INVALID_ARG, "null argument");
  const tpi_config& c = m->cfg;
  if (n_shards < 1 || n_shards > ROWSHARD_MAX_UNEQUAL || n_shards > m->plan.n_shards_max)
    return fail(TPI_ERR_INVALID_ARG, "n_shards must be in [1, %d]", ROWSHARD_MAX_UNEQUAL < m->plan.n_shards_max ? ROWSHARD_MAX_UNEQUAL : m->plan.n_shards_max);
  const int vec = c.dtype == TPI_BF16 ? 8 : 4, grp = c.n_heads / c.n_kv_heads;
  long long kv = 0, ff = 0;
  for (int i = 0; i < n_shards; ++i) {
    if (kv_heads_per_shard[i] < 1 || ffn_cols_per_shard[i] < 1) return fail(TPI_ERR_SHAPE, "every shard needs at least one kv head and one FFN column");
    if (ffn_cols_per_shard[i] % vec || (kv_heads_per_shard[i] * grp * c.head_dim) % vec)
      return fail(TPI_ERR_SHAPE, "a shard's FFN columns and heads*d must be multiples of %d elements (16 bytes)", vec);
    kv += kv_heads_per_shard[i];
    ff += ffn_cols_per_shard[i];
  }
  if (kv != c.n_kv_heads || ff != c.ffn) return fail(TPI_ERR_SHAPE, "the shards' kv heads (%lld of %d) and FFN columns (%lld of %d) must add up", kv, c.n_kv_heads, ff, c.ffn);
  if (!rowshard_fused_supported(c.ffn, 1)) return fail(TPI_ERR_SHAPE, "ffn too wide for an unequal partition");
  TRY(quiesce(m));
  drop_graph(m);
  m->N = n_shards;
  m->kv0.assign(n_shards + 1, 0);
  m->f0.assign(n_shards + 1, 0);
  for (int i = 0; i < n_shards; ++i) { m->kv0[i + 1] = m->kv0[i] + kv_heads_per_shard[i]; m->f0[i + 1] = m->f0[i] + ffn_cols_per_shard[i]; }
  m->unequal = true;
  TRY(load_layers(m));
  TRY(start_window(m));
  return write_position(m, 0);
}

extern "C" int tpi_set_window(tpi_model* m, int window_blocks) {
  if (!m || window_blocks < 0) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  if (window_blocks == m->window) return TPI_OK;
  if (!m->host_images) return fail(TPI_ERR_STATE, "no host images were kept: load with a larger host arena or a window");
  Plan np;
  TRY(quiesce(m));
  TRY(check_arenas(m, window_blocks, true, &np));
  drop_graph(m);
  m->plan = np;
  m->window = window_blocks;
  m->retain_T = 0;  // retention is chosen per window size: set it again after this call
  if (window_blocks == 0) {
    for (int b = 0; b < 2 * m->cfg.n_layers; ++b)
      CK(cudaMemcpyAsync(resident_block(m, b), host_image(m, b), block_size(m, b), cudaMemcpyHostToDevice, m->cs));
    CK(cudaStreamSynchronize(m->cs));
  }
  return start_window(m);
}

extern "C" int tpi_set_retention(tpi_model* m, int ffn_every_T) {
  if (!m || ffn_every_T < -1) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  if (m->window <= 0) return fail(TPI_ERR_STATE, "block retention applies to a streamed model (window >= 1)");
  if (ffn_every_T == -1) {  // as many FFN blocks as the device arena has room for beside the window: the smallest T that fits
    int nA, nF;
    window_slots(m->window, &nA, &nF);
    const size_t used = m->plan.blocks + (size_t)nA * m->plan.bl.attn_bytes + (size_t)nF * m->plan.bl.ffn_bytes;
    const size_t spare = m->res.dev_bytes > used ? m->res.dev_bytes - used : 0;
    const long long fit = (long long)(spare / m->plan.bl.ffn_bytes);
    ffn_every_T = 0;
    for (int T = 1; T <= m->cfg.n_layers && fit > 0; ++T)
      if ((m->cfg.n_layers + T - 1) / T <= fit) { ffn_every_T = T; break; }
  }
  TRY(quiesce(m));
  drop_graph(m);
  const int old = m->retain_T;
  m->retain_T = ffn_every_T;
  const int rc = start_window(m);
  if (rc) {  // put the previous setting back so that the model stays usable
    m->retain_T = old;
    start_window(m);
  }
  return rc;
}

extern "C" int tpi_reset(tpi_model* m) {
  if (!m) return fail(TPI_ERR_INVALID_ARG, "null model");
  return write_position(m, 0);
}
extern "C" int tpi_position(const tpi_model* m) { return m ? m->position : TPI_ERR_INVALID_ARG; }
extern "C" int tpi_set_position(tpi_model* m, int position) {
  if (!m || position < 0 || position > m->cfg.max_seq) return fail(TPI_ERR_INVALID_ARG, "bad position");
  return write_position(m, position);
}

extern "C" int tpi_set_option(tpi_model* m, int option, int value) {
  if (!m) return fail(TPI_ERR_INVALID_ARG, "null model");
  TRY(quiesce(m));
  switch (option) {
    case TPI_OPT_GRAPH: m->opt_graph = value != 0; break;
    case TPI_OPT_PDL: m->opt_pdl = value != 0; break;
    case TPI_OPT_MEGA: m->opt_mega = value != 0; break;
    case TPI_OPT_TENSOR: m->opt_tensor = value < 0 ? 0 : (value > 2 ? 2 : value); break;
    case TPI_OPT_PROFILE:
      m->opt_profile = value != 0;
      if (value && m->prof_ev.empty()) {
        const size_t want = 2 * (size_t)m->cfg.n_layers * 8;
        for (size_t i = 0; i < want; ++i) {
          cudaEvent_t e;
          CK(cudaEventCreate(&e));
          m->prof_ev.push_back(e);
        }
        for (size_t i = 0; i < 4 * (size_t)m->cfg.n_layers * 8; ++i) {
          cudaEvent_t e;
          CK(cudaEventCreate(&e));
          m->stall_ev.push_back(e);
        }
      }
      break;
    default: return fail(TPI_ERR_INVALID_ARG, "unknown option %d", option);
  }
  drop_graph(m);
  return TPI_OK;
}

// ------------------------------------------------------------------------------ block access during a step
struct BlockRef {
  char* base;
  int slot;
};
static int acquire_block(tpi_model* m, int block, BlockRef* r) {
  if (m->window <= 0) { r->base = resident_block(m, block); r->slot = -1; }
  else if (m->retained[block]) { r->base = m->dev + m->plan.blocks + m->retained_off[block]; r->slot = -1; }
  else {
    const int s = m->ring.acquire(block);
    if (s < 0) return s == -1000 || s == -1001 ? fail(TPI_ERR_STATE, "window ring out of order (%d)", s) : s;
    r->base = slot_ptr(m, s);
    r->slot = s;
  }
  if (m->sched_rec && (m->sched_open = sched_event(m))) CK(cudaEventRecord(m->sched_open, m->cs));  // after the wait
  return TPI_OK;
}
static int release_block(tpi_model* m, int block) {
  if (m->sched_open) {
    cudaEvent_t b = sched_event(m);
    if (b) {
      CK(cudaEventRecord(b, m->cs));
      m->sched_pending.push_back({m->sched_open, b, block & 1});
    } else m->sched_free.push_back(m->sched_open);
    m->sched_open = nullptr;
  }
  if (m->window <= 0 || m->retained[block]) return TPI_OK;
  const int rc = m->ring.release(block);
  if (rc == -1000) return fail(TPI_ERR_STATE, "window ring out of order");
  return rc;
}

// ------------------------------------------------------------------------------ one decode step (enqueue only)
static int enqueue_decode(tpi_model* m, LaunchCtx& lc) {
  const tpi_config& c = m->cfg;
  const Plan& p = m->plan;
  const BlockLayout& bl = p.bl;
  const int dt = c.dtype, h = c.hidden, a = c.n_heads, b = c.n_kv_heads, d = c.head_dim, s = c.ffn, N = m->N;
  float* x = dptr<float>(m, p.x);
  float* xhat = dptr<float>(m, p.xhat);
  float* q = dptr<float>(m, p.q);
  float* o = dptr<float>(m, p.o);
  float* act = dptr<float>(m, p.act);
  float* partials = dptr<float>(m, p.partials);
  int* pos = dptr<int>(m, p.pos);
  int* tok_hist = dptr<int>(m, p.tok_hist);
  const float2* rope = dptr<float2>(m, p.rope);
  unsigned* tickets = dptr<unsigned>(m, p.tickets);
  const int Nc = m->unequal ? 1 : N;  // the column-sharded projections of an unequal partition run as one shard
  const size_t qkv_shard = (size_t)(a + 2 * b) / Nc * d * h;
  // unequal partition: input ranges of the row-sharded projections (O: a shard's heads x d; down: its FFN columns)
  std::vector<int> ko(N + 1), kd(N + 1);
  for (int i = 0; i <= N; ++i) { ko[i] = m->kv0[i] * (a / b) * d; kd[i] = m->f0[i]; }

  // The kernel that ends a block leaves the raw residual x plus partial sums of x^2; the GEMV that
  // starts the next block normalises and applies its own block's gain while staging x.
  float* ss_part = dptr<float>(m, p.ss_part);
  const int n_parts = rowshard_fused_parts(h);
  auto norm_in = [&](const float* gain) { return NormIn{x, gain, ss_part, n_parts, c.rms_eps}; };
  auto rowshard = [&](const void* W, const float* xin, int Ks, const int* k0, float* tap) -> int {
    if (m->unequal) {
      CK(launch_gemv_rowshard_fused_unequal(lc, dt, W, xin, h, k0, N, x, ss_part, tap));
    } else if (rowshard_fused_supported(Ks, N)) {
      CK(launch_gemv_rowshard_fused(lc, dt, W, (size_t)h * Ks, xin, h, Ks, N, x, ss_part, tap));
    } else {  // very long shard slices: partial sums through memory, then the sum kernel
      CK(launch_gemv_partials(lc, dt, W, (size_t)h * Ks, xin, h, Ks, N, partials));
      CK(launch_reduce_residual(lc, partials, N, h, c.rms_eps, x, xhat, tap, ss_part, n_parts));
    }
    return TPI_OK;
  };
  CK(launch_embed(lc, dt, m->dev + p.emb, tok_hist, pos, c.vocab, c.max_seq, h, c.rms_eps, x, xhat, ss_part, n_parts,
                  dptr<int>(m, p.err)));
  for (int l = 0; l < c.n_layers; ++l) {
    BlockRef br;
    // ---- attention block: norm gain | QKV (column-sharded) | O (row-sharded)
    TRY(acquire_block(m, 2 * l, &br));
    void* kc = m->dev + p.kcache + (size_t)l * p.kv_layer_bytes;
    void* vc = m->dev + p.vcache + (size_t)l * p.kv_layer_bytes;
    CK(launch_gemv_qkv(lc, dt, br.base + bl.off_qkv, qkv_shard, norm_in((const float*)br.base), h, Nc, a, b, d,
                       c.max_seq, pos, rope, q, kc, vc));
    CK(launch_decode_attention(lc, dt, q, kc, vc, pos, a, b, d, c.max_seq, p.nsplit,
                               dptr<float>(m, p.attn_scratch), tickets, o));
    TRY(rowshard(br.base + bl.off_wo, o, a * d / N, ko.data(), dptr<float>(m, p.taps) + (size_t)(2 * l) * h));
    TRY(release_block(m, 2 * l));
    // ---- FFN block: norm gain | gate/up (column-sharded) | down (row-sharded)
    TRY(acquire_block(m, 2 * l + 1, &br));
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (m->opt_profile && m->prof_used + 2 <= m->prof_ev.size()) {
      e0 = m->prof_ev[m->prof_used++];
      e1 = m->prof_ev[m->prof_used++];
      CK(cudaEventRecord(e0, lc.stream));
    }
    CK(launch_gemv_gateup(lc, dt, br.base + bl.off_gu, (size_t)2 * (s / Nc) * h, norm_in((const float*)br.base), h, Nc, s, act));
    if (e1) CK(cudaEventRecord(e1, lc.stream));
    TRY(rowshard(br.base + bl.off_down, act, s / N, kd.data(), dptr<float>(m, p.taps) + (size_t)(2 * l + 1) * h));
    TRY(release_block(m, 2 * l + 1));
  }
  CK(launch_head_argmax(lc, dt, m->dev + p.head, norm_in(dptr<float>(m, p.final_gain)), h, c.vocab,
                        dptr<float>(m, p.logits), dptr<float>(m, p.amax_val), dptr<int>(m, p.amax_idx),
                        tickets + b, tok_hist, pos, 1));
  return TPI_OK;
}

static int ensure_graph(tpi_model* m) {
  if (m->graph_exec) return TPI_OK;
  int launches = 0;
  LaunchCtx lc{m->cs, m->opt_pdl != 0, &launches};
  cudaGraph_t g = nullptr;
  CK(cudaStreamBeginCapture(m->cs, cudaStreamCaptureModeThreadLocal));
  const int rc = enqueue_decode(m, lc);
  cudaError_t e = cudaStreamEndCapture(m->cs, &g);
  if (rc) { if (g) cudaGraphDestroy(g); return rc; }
  if (e != cudaSuccess) return fail(TPI_ERR_CUDA, "graph capture failed: %s", cudaGetErrorString(e));
  e = cudaGraphInstantiate(&m->graph_exec, g, 0);
  cudaGraphDestroy(g);
  if (e != cudaSuccess) { m->graph_exec = nullptr; return fail(TPI_ERR_CUDA, "graph instantiate failed: %s", cudaGetErrorString(e)); }
  m->graph_launches = launches;
  return TPI_OK;
}

static void harvest_profile(tpi_model* m) {
  for (size_t i = 0; i + 1 < m->prof_used; i += 2) {
    float ms = 0;
    if (cudaEventElapsedTime(&ms, m->prof_ev[i], m->prof_ev[i + 1]) == cudaSuccess) { m->prof_ms_sum += ms; ++m->prof_samples; }
  }
  m->prof_used = 0;
  for (size_t i = 0; i + 1 < m->stall_used; i += 2) {
    float ms = 0;
    if (cudaEventElapsedTime(&ms, m->stall_ev[i], m->stall_ev[i + 1]) == cudaSuccess) m->stall_ms += ms;
  }
  m->stall_used = 0;
  sched_harvest(m);
}

static int check_device_error(tpi_model* m, const int* io_err) {
  if (*io_err == DEVERR_NONE) return TPI_OK;
  const int code = *io_err;
  cudaMemsetAsync(m->dev + m->plan.err, 0, 4, m->cs);
  cudaStreamSynchronize(m->cs);
  if (code == DEVERR_TOKEN_RANGE) return fail(TPI_ERR_TOKEN_RANGE, "a token id was outside [0, vocab)");
  return fail(TPI_ERR_DEVICE_CHECK, "device error word = %d", code);
}

// io layout (pinned): [0] scratch int, [1] device error word, [2..] token ids
static int run_decode(tpi_model* m, int32_t token_in, int n_steps, int32_t* tokens_out, float* logits) {
  if (!m || n_steps < 1 || !tokens_out) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  const tpi_config& c = m->cfg;
  if (token_in < 0 || token_in >= c.vocab) return fail(TPI_ERR_TOKEN_RANGE, "token %d outside [0, %d)", token_in, c.vocab);
  if (m->position + n_steps > c.max_seq) return fail(TPI_ERR_SEQ_OVERFLOW, "position %d + %d steps exceeds max_seq %d", m->position, n_steps, c.max_seq);
  const Plan& p = m->plan;
  int* io = (int*)(m->host + p.h_io);
  const auto w0 = std::chrono::steady_clock::now();
  io[2] = token_in;
  CK(cudaMemcpyAsync(dptr<int>(m, p.tok_hist) + m->position, io + 2, 4, cudaMemcpyHostToDevice, m->cs));
  const bool use_mega = mega_usable(m);
  const bool use_graph = !use_mega && m->opt_graph && m->window <= 0 && !m->opt_profile;
  if (use_mega) TRY(ensure_mega(m));
  if (use_graph) TRY(ensure_graph(m));
  int launches = 0;
  CK(cudaEventRecord(m->ev_t0, m->cs));
  for (int i = 0; i < n_steps; ++i) {
    if (use_mega) {
      LaunchCtx lc{m->cs, false, &launches};
      TRY(enqueue_decode_mega(m, lc));
    } else if (use_graph) { CK(cudaGraphLaunch(m->graph_exec, m->cs)); launches += m->graph_launches; }
    else {
      LaunchCtx lc{m->cs, m->opt_pdl != 0 && !m->opt_profile, &launches};
      m->sched_rec = m->opt_profile != 0;
      const int rc = enqueue_decode(m, lc);
      m->sched_rec = false;
      TRY(rc);
    }
  }
  CK(cudaEventRecord(m->ev_t1, m->cs));
  CK(cudaMemcpyAsync(io + 3, dptr<int>(m, p.tok_hist) + m->position + 1, (size_t)n_steps * 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaMemcpyAsync(io + 1, m->dev + p.err, 4, cudaMemcpyDeviceToHost, m->cs));
  if (logits) CK(cudaMemcpyAsync(m->host + p.h_logits, m->dev + p.logits, (size_t)c.vocab * 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaEventRecord(m->ev_done, m->cs));
  TRY(wait_event(m, m->ev_done));
  m->position += n_steps;
  memcpy(tokens_out, io + 3, (size_t)n_steps * 4);
  if (logits) memcpy(logits, m->host + p.h_logits, (size_t)c.vocab * 4);
  float ms = 0;
  cudaEventElapsedTime(&ms, m->ev_t0, m->ev_t1);
  m->st.last_decode_dev_ms = ms;
  m->st.last_decode_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - w0).count();
  m->st.kernel_launches_last = launches;
  if (m->opt_profile) harvest_profile(m);
  return check_device_error(m, io + 1);
}

extern "C" int tpi_decode_step(tpi_model* m, int32_t token_in, int32_t* token_out, float* logits_or_null) {
  return run_decode(m, token_in, 1, token_out, logits_or_null);
}
extern "C" int tpi_decode_run(tpi_model* m, int32_t token_in, int n_steps, int32_t* tokens_out) {
  if (m && n_steps + 3 > m->cfg.max_seq + 2 + m->cfg.max_prefill) return fail(TPI_ERR_INVALID_ARG, "n_steps too large");
  return run_decode(m, token_in, n_steps, tokens_out, nullptr);
}

// ------------------------------------------------------------------------------ prompt pass
static int enqueue_prefill_chunk(tpi_model* m, LaunchCtx& lc, int pos0, int T, bool last) {
  const tpi_config& c = m->cfg;
  const Plan& p = m->plan;
  const BlockLayout& bl = p.bl;
  const int dt = c.dtype, h = c.hidden, a = c.n_heads, b = c.n_kv_heads, d = c.head_dim, s = c.ffn, N = m->N;
  float* X = dptr<float>(m, p.pX);
  float* Xn = dptr<float>(m, p.pXn);
  float* QKV = dptr<float>(m, p.pQKV);
  float* Q = dptr<float>(m, p.pQ);
  float* O = dptr<float>(m, p.pO);
  float* GU = dptr<float>(m, p.pGU);
  float* ACT = dptr<float>(m, p.pACT);
  float* PART = dptr<float>(m, p.pPART);
  const float2* rope = dptr<float2>(m, p.rope);
  const int qkv_cols = (a + 2 * b) * d;
  const int Ko = a * d / N, Kd = s / N;
  const int Nc = m->unequal ? 1 : N;  // column-sharded rows of an unequal partition are packed as one shard
  std::vector<int> ko(N + 1), kd(N + 1);  // input ranges of the row-sharded projections per shard
  for (int i = 0; i <= N; ++i) { ko[i] = m->kv0[i] * (a / b) * d; kd[i] = m->f0[i]; }
  bool k64 = true;  // the tensor-core GEMM takes contractions that are multiples of 64
  for (int i = 0; i < N; ++i) k64 = k64 && (ko[i + 1] - ko[i]) % 64 == 0 && (kd[i + 1] - kd[i]) % 64 == 0;
  // bf16 models run the projections on the tensor cores (activations rounded to bf16, fp32 accumulate);
  // fp32 models, and shapes the tensor-core kernel does not take, use the fp32 SIMT GEMM.
  const bool tc = m->opt_tensor && dt == TPI_BF16 && gemm_tc_supported(h, h, qkv_cols) && gemm_tc_supported(h, h, 2 * s) &&
                  (m->unequal ? k64 && gemm_tc_supported(64, a * d, h) && gemm_tc_supported(64, s, h)
                              : gemm_tc_supported(Ko, a * d, h) && gemm_tc_supported(Kd, s, h));
  const int act_mode = tc ? (m->opt_tensor == 2 ? 1 : 2) : 0;  // 0 fp32, 1 bf16, 2 split bf16 (default)
  int* err = dptr<int>(m, p.err);
  // Y[b] = A[:, b*a_col : b*a_col+K] . W[b]^T for n_batch shards (1 for the column-sharded projections)
  auto proj = [&](const float* A, int lda, int a_col, const void* W, int w_rows_b, float* Y, long long y_bs, int ldy,
                  int n_out, int K, int n_batch) -> int {
    if (tc) {  // split mode: the low halves sit T * lda bf16 elements after the high halves
      const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(A);
      CK(launch_gemm_tc(lc, hi, act_mode == 2 ? hi + (size_t)T * lda : nullptr, lda, a_col, W, w_rows_b, Y, y_bs, ldy, T,
                        n_out, K, n_batch, err));
    }
    else CK(launch_gemm_simt(lc, dt, A, a_col, lda, W, (long long)w_rows_b * K, Y, y_bs, ldy, T, n_out, K, n_batch));
    return TPI_OK;
  };
  // row-sharded projection: shard i multiplies its slice of the inputs by its own matrix -> partial sums P_i
  auto proj_rows = [&](const float* A, int lda, const void* W, const int* k0, int Ks) -> int {
    if (!m->unequal) return proj(A, lda, Ks, W, h, PART, (long long)T * h, h, h, Ks, N);
    const size_t B = elem_size(dt);
    for (int i = 0; i < N; ++i) {
      const int kw = k0[i + 1] - k0[i];
      const char* Wi = (const char*)W + (size_t)h * k0[i] * B;
      // split-bf16 activations: the column offset applies to both halves, which are T * lda elements apart
      const float* Ai = tc ? reinterpret_cast<const float*>(reinterpret_cast<const __nv_bfloat16*>(A) + k0[i]) : A + k0[i];
      if (tc) {
        const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(Ai);
        CK(launch_gemm_tc(lc, hi, act_mode == 2 ? hi + (size_t)T * lda : nullptr, lda, 0, Wi, h, PART + (size_t)i * T * h, 0, h, T,
                          h, kw, 1, err));
      } else {
        CK(launch_gemm_simt(lc, dt, Ai, 0, lda, Wi, 0, PART + (size_t)i * T * h, 0, h, T, h, kw, 1));
      }
    }
    return TPI_OK;
  };
  CK(launch_embed_rows(lc, dt, m->dev + p.emb, dptr<int>(m, p.tok_hist), pos0, T, c.vocab, h, X, err));
  // With every block resident, the kernel that ends a block (star sum + shortcut) also applies the next block's
  // RMSNorm, whose gain lives in that next block's image; a streamed model may not hold the next block yet.
  const bool fuse_norm = m->window <= 0;
  bool normed = false;  // Xn already holds the input of the block about to start
  for (int l = 0; l < c.n_layers; ++l) {
    BlockRef br;
    TRY(acquire_block(m, 2 * l, &br));
    void* kc = m->dev + p.kcache + (size_t)l * p.kv_layer_bytes;
    void* vc = m->dev + p.vcache + (size_t)l * p.kv_layer_bytes;
    if (!normed) CK(launch_rmsnorm_rows(lc, X, (const float*)br.base, T, h, c.rms_eps, Xn, act_mode));
    TRY(proj(Xn, h, 0, br.base + bl.off_qkv, qkv_cols, QKV, 0, qkv_cols, qkv_cols, h, 1));
    CK(launch_rope_kv_rows(lc, dt, QKV, T, pos0, Nc, a, b, d, c.max_seq, rope, Q, kc, vc));
    if (m->opt_tensor && prefill_attention_mma_supported(dt, d))
      CK(launch_prefill_attention_mma(lc, Q, kc, vc, T, pos0, a, b, d, c.max_seq, O, act_mode));
    else
      CK(launch_prefill_attention(lc, dt, Q, kc, vc, T, pos0, a, b, d, c.max_seq, O, act_mode));
    TRY(proj_rows(O, a * d, br.base + bl.off_wo, ko.data(), Ko));
    float* tap_a = last ? dptr<float>(m, p.taps) + (size_t)(2 * l) * h : nullptr;
    if (fuse_norm)
      CK(launch_reduce_residual_norm_rows(lc, PART, N, T, h, X, tap_a, (const float*)resident_block(m, 2 * l + 1), c.rms_eps, Xn, act_mode));
    else
      CK(launch_reduce_residual_rows(lc, PART, N, T, h, X, tap_a));
    TRY(release_block(m, 2 * l));
    TRY(acquire_block(m, 2 * l + 1, &br));
    if (!fuse_norm) CK(launch_rmsnorm_rows(lc, X, (const float*)br.base, T, h, c.rms_eps, Xn, act_mode));
    if (tc && gemm_tc_swiglu_supported(h, h, s)) {  // SwiGLU in the GEMM's epilogue: the fp32 gate/up rows never reach memory
      const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(Xn);
      CK(launch_gemm_tc_swiglu(lc, hi, act_mode == 2 ? hi + (size_t)T * h : nullptr, h, br.base + bl.off_gu, ACT, act_mode, T, s, h, err));
    } else {
      TRY(proj(Xn, h, 0, br.base + bl.off_gu, 2 * s, GU, 0, 2 * s, 2 * s, h, 1));
      CK(launch_swiglu_rows(lc, GU, T, s, ACT, act_mode));
    }
    TRY(proj_rows(ACT, s, br.base + bl.off_down, kd.data(), Kd));
    float* tap_f = last ? dptr<float>(m, p.taps) + (size_t)(2 * l + 1) * h : nullptr;
    normed = fuse_norm && l + 1 < c.n_layers;
    if (normed)
      CK(launch_reduce_residual_norm_rows(lc, PART, N, T, h, X, tap_f, (const float*)resident_block(m, 2 * l + 2), c.rms_eps, Xn, act_mode));
    else
      CK(launch_reduce_residual_rows(lc, PART, N, T, h, X, tap_f));
    TRY(release_block(m, 2 * l + 1));
  }
  if (last) {
    const int n_parts = rowshard_fused_parts(h);
    CK(launch_rmsnorm_stat_row(lc, X + (size_t)(T - 1) * h, h, c.rms_eps, dptr<float>(m, p.x), dptr<float>(m, p.xhat),
                               dptr<float>(m, p.ss_part), n_parts,
                               dptr<int>(m, p.pos), pos0 + T - 1));
    CK(launch_head_argmax(lc, dt, m->dev + p.head,
                          NormIn{dptr<float>(m, p.x), dptr<float>(m, p.final_gain), dptr<float>(m, p.ss_part), n_parts, c.rms_eps},
                          h, c.vocab,
                          dptr<float>(m, p.logits), dptr<float>(m, p.amax_val), dptr<int>(m, p.amax_idx),
                          dptr<unsigned>(m, p.tickets) + b, dptr<int>(m, p.tok_hist), dptr<int>(m, p.pos), 1));
  }
  return TPI_OK;
}

extern "C" int tpi_prefill(tpi_model* m, const int32_t* tokens, int n_tokens, int32_t* first_token,
                           float* logits_or_null) {
  if (!m || !tokens || n_tokens < 1 || !first_token) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  const tpi_config& c = m->cfg;
  const Plan& p = m->plan;
  if (m->position + n_tokens > c.max_seq) return fail(TPI_ERR_SEQ_OVERFLOW, "position %d + %d tokens exceeds max_seq %d", m->position, n_tokens, c.max_seq);
  for (int i = 0; i < n_tokens; ++i)
    if (tokens[i] < 0 || tokens[i] >= c.vocab) return fail(TPI_ERR_TOKEN_RANGE, "token %d outside [0, %d)", tokens[i], c.vocab);
  int* io = (int*)(m->host + p.h_io);
  const auto w0 = std::chrono::steady_clock::now();
  int launches = 0;
  LaunchCtx lc{m->cs, m->opt_pdl != 0 && !m->opt_profile, &launches};
  const int p_begin = m->position;
  CK(cudaEventRecord(m->ev_t0, m->cs));
  for (int t0 = 0; t0 < n_tokens; t0 += c.max_prefill) {
    const int T = n_tokens - t0 < c.max_prefill ? n_tokens - t0 : c.max_prefill;
    // token ids go through the pinned io area, one chunk at a time
    if (t0) TRY(wait_event(m, m->ev_done));
    memcpy(io + 3, tokens + t0, (size_t)T * 4);
    CK(cudaMemcpyAsync(dptr<int>(m, p.tok_hist) + p_begin + t0, io + 3, (size_t)T * 4, cudaMemcpyHostToDevice, m->cs));
    CK(cudaEventRecord(m->ev_done, m->cs));
    TRY(enqueue_prefill_chunk(m, lc, p_begin + t0, T, t0 + T == n_tokens));
  }
  CK(cudaEventRecord(m->ev_t1, m->cs));
  m->st.last_prefill_enqueue_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - w0).count();
  CK(cudaMemcpyAsync(io + 2, dptr<int>(m, p.tok_hist) + p_begin + n_tokens, 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaMemcpyAsync(io + 1, m->dev + p.err, 4, cudaMemcpyDeviceToHost, m->cs));
  if (logits_or_null) CK(cudaMemcpyAsync(m->host + p.h_logits, m->dev + p.logits, (size_t)c.vocab * 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaEventRecord(m->ev_done, m->cs));
  TRY(wait_event(m, m->ev_done));
  m->position = p_begin + n_tokens;
  *first_token = io[2];
  if (logits_or_null) memcpy(logits_or_null, m->host + p.h_logits, (size_t)c.vocab * 4);
  m->st.last_prefill_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - w0).count();
  {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, m->ev_t0, m->ev_t1) == cudaSuccess) m->st.last_prefill_dev_ms = ms;
  }
  m->st.kernel_launches_last = launches;
  if (m->opt_profile) harvest_profile(m);
  return check_device_error(m, io + 1);
}

// ------------------------------------------------------------------------------ taps, cache access, stats
extern "C" int tpi_get_hidden(tpi_model* m, int layer, int which, float* dst_host) {
  if (!m || !dst_host || layer < 0 || layer >= m->cfg.n_layers || (which != 0 && which != 1))
    return fail(TPI_ERR_INVALID_ARG, "bad argument");
  CK(cudaMemcpyAsync(dst_host, dptr<float>(m, m->plan.taps) + (size_t)(2 * layer + which) * m->cfg.hidden,
                     (size_t)m->cfg.hidden * 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaStreamSynchronize(m->cs));
  return TPI_OK;
}

static int kv_io(tpi_model* m, int layer, int kv_head, int pos0, int n, float* k, float* v, bool put) {
  const tpi_config& c = m->cfg;
  if (!m || layer < 0 || layer >= c.n_layers || kv_head < 0 || kv_head >= c.n_kv_heads || pos0 < 0 || n < 1 ||
      pos0 + n > c.max_seq || !k || !v)
    return fail(TPI_ERR_INVALID_ARG, "bad argument");
  const Plan& p = m->plan;
  const size_t B = elem_size(c.dtype), d = c.head_dim;
  float* tmp = dptr<float>(m, p.pX);  // prefill activations double as conversion scratch
  const size_t cap = (size_t)c.max_prefill * c.hidden / d;  // rows that fit
  LaunchCtx lc{m->cs, false, nullptr};
  for (int which = 0; which < 2; ++which) {
    char* base = m->dev + (which ? p.vcache : p.kcache) + (size_t)layer * p.kv_layer_bytes +
                 ((size_t)kv_head * c.max_seq + pos0) * d * B;
    float* hostp = which ? v : k;
    for (size_t r0 = 0; r0 < (size_t)n; r0 += cap) {
      const size_t rows = (size_t)n - r0 < cap ? (size_t)n - r0 : cap;
      if (put) {
        CK(cudaMemcpyAsync(tmp, hostp + r0 * d, rows * d * 4, cudaMemcpyHostToDevice, m->cs));
        CK(launch_kv_convert(lc, c.dtype, base + r0 * d * B, tmp, rows * d, 0));
      } else {
        CK(launch_kv_convert(lc, c.dtype, base + r0 * d * B, tmp, rows * d, 1));
        CK(cudaMemcpyAsync(hostp + r0 * d, tmp, rows * d * 4, cudaMemcpyDeviceToHost, m->cs));
      }
      CK(cudaStreamSynchronize(m->cs));
    }
  }
  return TPI_OK;
}
extern "C" int tpi_get_kv(tpi_model* m, int layer, int kv_head, int pos0, int n, float* k_dst, float* v_dst) {
  if (!m) return fail(TPI_ERR_INVALID_ARG, "null model");
  return kv_io(m, layer, kv_head, pos0, n, k_dst, v_dst, false);
}
extern "C" int tpi_put_kv(tpi_model* m, int layer, int kv_head, int pos0, int n, const float* k_src,
                          const float* v_src) {
  if (!m) return fail(TPI_ERR_INVALID_ARG, "null model");
  return kv_io(m, layer, kv_head, pos0, n, (float*)k_src, (float*)v_src, true);
}

extern "C" int tpi_get_stats(tpi_model* m, tpi_stats* out) {
  if (!m || !out) return fail(TPI_ERR_INVALID_ARG, "null argument");
  const tpi_config& c = m->cfg;
  const size_t B = elem_size(c.dtype);
  tpi_stats s = m->st;
  const uint64_t layer_bytes = ((uint64_t)(c.n_heads + 2 * c.n_kv_heads) * c.head_dim * c.hidden +
                                (uint64_t)c.hidden * c.n_heads * c.head_dim + 3ull * c.hidden * c.ffn) * B +
                               2ull * c.hidden * 4;
  s.weight_bytes_per_token = layer_bytes * c.n_layers + (uint64_t)c.vocab * c.hidden * B + (uint64_t)c.hidden * 4;
  s.link_bytes_total = m->link_bytes;
  s.blocks_loaded = m->window > 0 ? (uint64_t)m->ring.loads_issued() : 0;
  s.stall_ms_total = m->stall_ms;
  s.dominant_kernel_ms = m->prof_samples ? m->prof_ms_sum / m->prof_samples : 0.0;
  s.dominant_kernel_bytes = 2ull * c.ffn * c.hidden * B + (uint64_t)c.hidden * 8 + (uint64_t)c.ffn * 4;
  s.dominant_kernel_samples = m->prof_samples;
  s.window_blocks = m->window;
  s.n_shards = m->N;
  s.position = m->position;
  s.graph_active = m->graph_exec != nullptr;
  if (m->window > 0) {
    s.window_peak_bytes = (uint64_t)m->ring.n_attn_slots() * m->plan.bl.attn_bytes +
                          (uint64_t)m->ring.n_ffn_slots() * m->plan.bl.ffn_bytes;
  } else s.window_peak_bytes = 0;
  s.retained_bytes = m->window > 0 ? m->retained_bytes : 0;
  s.retained_blocks = 0;
  if (m->window > 0)
    for (char r : m->retained) s.retained_blocks += r != 0;
  *out = s;
  return TPI_OK;
}

// ------------------------------------------------------------------------------ ring trace (host-only test hook)
namespace {
struct TraceCtx {
  int* ops;
  int max_ops, n;
};
int tr_push(void* ctx, int op, int slot, int block) {
  TraceCtx* t = (TraceCtx*)ctx;
  if (t->n < t->max_ops) { t->ops[3 * t->n] = op; t->ops[3 * t->n + 1] = slot; t->ops[3 * t->n + 2] = block; }
  ++t->n;
  return 0;
}
int tr_cwr(void* c, int s) { return tr_push(c, 0, s, -1); }
int tr_cb(void* c, int s, int b) { return tr_push(c, 1, s, b); }
int tr_crl(void* c, int s) { return tr_push(c, 2, s, -1); }
int tr_xwl(void* c, int s) { return tr_push(c, 3, s, -1); }
int tr_xrr(void* c, int s) { return tr_push(c, 4, s, -1); }
}  // namespace

// Runs the window ring's ordering logic against a recording back end (no GPU needed): executes
// `n_exec` blocks in cyclic order over `n_blocks` with window `w`.  ops receives up to max_ops
// triples (op, slot, block): op 0 copy-queue waits for release of slot, 1 copy block into slot,
// 2 copy-queue marks slot loaded, 3 compute-queue waits for slot, 4 compute-queue releases slot.
// Returns the number of operations (may exceed max_ops) or a negative status.
// ------------------------------------------------------------------------------ steady-state diagnostics
// Prop. 3, Prop. 4 and Prop. 6 evaluated on given latencies (host arithmetic only).
extern "C" int tpi_steady_conditions(double t_attn, double t_ffn, double t_all_reduce, double tau_attn, double tau_ffn,
                                     int n_layers, int* tight, int* loose, int* retention_T) {
  if (n_layers < 1 || !(t_attn >= 0) || !(t_ffn >= 0) || !(t_all_reduce >= 0) || !(tau_attn >= 0) || !(tau_ffn >= 0))
    return fail(TPI_ERR_INVALID_ARG, "bad argument");
  const double ca = t_attn + t_all_reduce, cf = t_ffn + t_all_reduce;  // a block's compute with its allreduce
  if (tight) *tight = ca >= tau_ffn && cf >= tau_attn;
  // Prop. 3: one layer's compute covers one layer's loads, and one of the two prefix families holds for every l
  bool fam_a = true, fam_b = true;
  for (int l = 1; l <= n_layers; ++l) {
    if (l * ca + (l - 1) * cf < l * tau_ffn + (l - 1) * tau_attn) fam_a = false;
    if ((l - 1) * ca + l * cf < (l - 1) * tau_ffn + l * tau_attn) fam_b = false;
  }
  const bool loose_ok = ca + cf >= tau_ffn + tau_attn && (fam_a || fam_b);
  if (loose) *loose = loose_ok;
  if (retention_T) {
    // Prop. 6: with one FFN block in every T kept, ceil(l/T) of the first l FFN loads disappear; both prefix
    // families must hold.  Fewer kept blocks (larger T) only add loads, so scan from the cheapest setting down.
    int best = -1;
    for (int T = n_layers; T >= 1 && best < 0; --T) {
      bool ok = true;
      for (int l = 1; l <= n_layers && ok; ++l) {
        const double ffn_loads = (double)(l - (l + T - 1) / T) * tau_ffn;
        if (l * ca + l * cf < ffn_loads + l * tau_attn) ok = false;
        if (l * ca + (l - 1) * cf < ffn_loads + (l - 1) * tau_attn) ok = false;
      }
      if (ok) best = T;
    }
    *retention_T = loose_ok ? 0 : best;
  }
  return TPI_OK;
}

extern "C" int tpi_scheduler_report(tpi_model* m, tpi_sched_report* out) {
  if (!m || !out) return fail(TPI_ERR_INVALID_ARG, "null argument");
  sched_harvest(m);
  tpi_sched_report r;
  memset(&r, 0, sizeof r);
  double mean[4];
  for (int k = 0; k < 4; ++k) mean[k] = m->sched_n[k] ? m->sched_sum[k] / m->sched_n[k] : 0.0;
  r.t_attn_ms = mean[0]; r.t_ffn_ms = mean[1]; r.tau_attn_ms = mean[2]; r.tau_ffn_ms = mean[3];
  r.n_t_attn = m->sched_n[0]; r.n_t_ffn = m->sched_n[1]; r.n_tau_attn = m->sched_n[2]; r.n_tau_ffn = m->sched_n[3];
  r.t_all_reduce_ms = 0.0;  // the rank-ordered sum runs inside the block's last kernel: it is part of t_attn / t_ffn
  r.stall_ms_total = m->stall_ms;
  r.tight_holds = r.loose_holds = r.retention_T = -2;
  const bool have_t = r.n_t_attn && r.n_t_ffn;
  // a retained or resident block has no load: its tau counts as 0 only when nothing of that kind is streamed
  const bool streams_ffn = m->window > 0 && m->retain_T != 1;
  const bool have_tau = m->window > 0 && r.n_tau_attn && (r.n_tau_ffn || !streams_ffn);
  if (have_t && have_tau)
    TRY(tpi_steady_conditions(r.t_attn_ms, r.t_ffn_ms, 0.0, r.tau_attn_ms, r.tau_ffn_ms, m->cfg.n_layers, &r.tight_holds,
                              &r.loose_holds, &r.retention_T));
  r.window_blocks = m->window;
  r.retain_every_T = m->window > 0 ? m->retain_T : 0;
  if (m->window > 0) {
    int nA, nF;
    window_slots(m->window, &nA, &nF);
    // Prop. 5 without the empirical factor: floor(w/2) attention blocks + ceil(w/2) FFN blocks
    r.m_worker_bytes = (uint64_t)(m->window / 2) * m->plan.bl.attn_bytes + (uint64_t)((m->window + 1) / 2) * m->plan.bl.ffn_bytes;
    r.window_device_bytes = (uint64_t)nA * m->plan.bl.attn_bytes + (uint64_t)nF * m->plan.bl.ffn_bytes + m->retained_bytes;
  }
  *out = r;
  return TPI_OK;
}

extern "C" int tpi_scheduler_reset(tpi_model* m) {
  if (!m) return fail(TPI_ERR_INVALID_ARG, "null model");
  TRY(quiesce(m));
  sched_harvest(m);
  for (int k = 0; k < 4; ++k) { m->sched_sum[k] = 0; m->sched_n[k] = 0; }
  m->stall_ms = 0;
  return TPI_OK;
}

extern "C" int tpi_ring_trace(int n_blocks, int w, int n_exec, int* ops, int max_ops) {
  return tpi_ring_trace_retained(n_blocks, w, n_exec, 0, ops, max_ops);
}

extern "C" int tpi_ring_trace_retained(int n_blocks, int w, int n_exec, int ffn_every_T, int* ops, int max_ops) {
  if (n_blocks < 2 || n_blocks % 2 || w < 1 || n_exec < 0 || ffn_every_T < 0 || (!ops && max_ops > 0))
    return fail(TPI_ERR_INVALID_ARG, "bad argument");
  std::vector<char> keep(n_blocks, 0);
  if (ffn_every_T > 0)
    for (int l = 0; l < n_blocks / 2; l += ffn_every_T) keep[2 * l + 1] = 1;
  TraceCtx t{ops, max_ops, 0};
  RingBackend be;
  be.ctx = &t;
  be.copy_wait_released = tr_cwr;
  be.copy_block = tr_cb;
  be.copy_record_loaded = tr_crl;
  be.compute_wait_loaded = tr_xwl;
  be.compute_record_released = tr_xrr;
  Ring r;
  r.configure(n_blocks, w, be, keep.data());
  if (r.pump()) return TPI_ERR_STATE;
  for (int i = 0; i < n_exec; ++i) {
    const int blk = i % n_blocks;
    if (keep[blk]) { tr_push(&t, 5, -1, blk); continue; }  // a retained block runs without any window operation
    if (r.acquire(blk) < 0) return TPI_ERR_STATE;
    if (r.release(blk)) return TPI_ERR_STATE;
  }
  return t.n;
}
