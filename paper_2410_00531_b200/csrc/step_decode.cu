// The per-token step driver: the five kernels per layer (graph + programmatic dependent launch when all blocks are
// resident, plain launches between the window's events otherwise), the optional whole-token kernel, tpi_decode_*.
#include "model.h"

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

void drop_graph(tpi_model* m) {
  m->mega_ready = false;
  if (m->graph_exec) cudaGraphExecDestroy(m->graph_exec);
  m->graph_exec = nullptr;
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

void harvest_profile(tpi_model* m) {
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

int check_device_error(tpi_model* m, const int* io_err) {
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

