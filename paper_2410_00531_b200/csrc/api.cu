// C ABI of the library, part 1: errors, arena planning, weight partition + packing, loading and the calls that
// re-shape a loaded model (shards, partition, window, retention, options).
#include "model.h"

// ------------------------------------------------------------------------------ errors
static thread_local char g_err[512] = "";
int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof g_err, fmt, ap);
  va_end(ap);
  return code;
}

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

void uniform_partition(tpi_model* m) {
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

// TPI_DEBUG=1 in the environment builds the device arena with guard zones (read at tpi_query_arena and tpi_load_model,
// which must see the same setting).
static bool debug_env() {
  const char* e = getenv("TPI_DEBUG");
  return e && e[0] && e[0] != '0';
}

static CanaryList canary_list(const tpi_model* m) {
  CanaryList L{};
  L.n = m->plan.n_canaries;
  for (int i = 0; i < L.n; ++i) L.off[i] = m->plan.canary_off[i];
  return L;
}
int fill_canaries(tpi_model* m) {
  LaunchCtx lc{m->cs, false, nullptr};
  CK(launch_canary_fill(lc, m->dev, canary_list(m)));
  return TPI_OK;
}
int enqueue_canary_check(tpi_model* m, LaunchCtx& lc) {
  if (m->plan.n_canaries < 1) return TPI_OK;
  CK(launch_canary_check(lc, m->dev, canary_list(m), dptr<int>(m, m->plan.err)));
  return TPI_OK;
}

extern "C" int tpi_query_arena(const tpi_config* cfg, int n_shards_max, int window_blocks, int keep_host_images,
                               size_t* dev_bytes, size_t* host_bytes) {
  TRY(validate(cfg, 1));
  if (n_shards_max < 1 || window_blocks < 0) return fail(TPI_ERR_INVALID_ARG, "bad shard/window count");
  if (n_shards_max < 8) n_shards_max = 8;  // tpi_load_model always plans for at least 8 shards
  Plan p;
  make_plan(*cfg, n_shards_max, window_blocks, keep_host_images, head_argmax_blocks(cfg->vocab), &p, dev_bytes,
            host_bytes, debug_env());
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
int wait_event(tpi_model* m, cudaEvent_t ev) {
  const auto t0 = std::chrono::steady_clock::now();
  for (long spins = 0;; ++spins) {
    cudaError_t e = cudaEventQuery(ev);
    if (e == cudaSuccess) return TPI_OK;
    if (e != cudaErrorNotReady) return fail(TPI_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
    if (spins > 2000) std::this_thread::yield();
    if ((spins & 1023) == 0) {
      const double s = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
      if (s > m->wait_deadline_s) {
        m->desync = true;  // the enqueued work is still running: host and device positions no longer agree
        return fail(TPI_ERR_TIMEOUT, "device did not finish within %.3f s", s);
      }
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

char* host_image(tpi_model* m, int block) {  // block = 2*layer + (0 attn | 1 ffn)
  const BlockLayout& bl = m->plan.bl;
  const size_t per_layer = bl.attn_bytes + bl.ffn_bytes;
  return m->host + m->plan.h_images + (size_t)(block / 2) * per_layer + (block % 2 ? bl.attn_bytes : 0);
}
size_t block_size(const tpi_model* m, int block) {
  return block % 2 ? m->plan.bl.ffn_bytes : m->plan.bl.attn_bytes;
}
char* resident_block(tpi_model* m, int block) {
  const BlockLayout& bl = m->plan.bl;
  const size_t per_layer = bl.attn_bytes + bl.ffn_bytes;
  return m->dev + m->plan.blocks + (size_t)(block / 2) * per_layer + (block % 2 ? bl.attn_bytes : 0);
}
char* slot_ptr(tpi_model* m, int slot) {
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
  TRY(fill_canaries(m));
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
            &need_h, m->debug);
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
  m->debug = debug_env();
  make_plan(*cfg, m->plan.n_shards_max, window_blocks, 1, head_argmax_blocks(cfg->vocab), &with_images, &nd, &nh, m->debug);
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

int quiesce(tpi_model* m) {
  CK(cudaStreamSynchronize(m->cs));
  CK(cudaStreamSynchronize(m->ps));
  return TPI_OK;
}

int write_position(tpi_model* m, int p) {
  int* io = (int*)(m->host + m->plan.h_io);
  io[0] = p;
  CK(cudaMemcpyAsync(m->dev + m->plan.pos, io, 4, cudaMemcpyHostToDevice, m->cs));
  CK(cudaStreamSynchronize(m->cs));
  m->position = p;
  m->desync = false;
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
    case TPI_OPT_TENSOR: m->opt_tensor = value < 0 ? 0 : (value > 2 ? 2 : value); break;
    case TPI_OPT_ROWSHARD_FUSED: m->opt_rowshard_fused = value != 0; break;
    case TPI_OPT_WAIT_DEADLINE_MS:
      if (value < 1) return fail(TPI_ERR_INVALID_ARG, "the wait deadline must be at least 1 ms");
      m->wait_deadline_s = value * 1e-3;
      return TPI_OK;  // nothing about the launch sequence changes: the captured graph stays
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

