// Debug taps, KV-cache access and statistics.
#include "model.h"

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

