// The per-token step driver: the five kernels per layer (graph + programmatic dependent launch when all blocks are
// resident, plain launches between the window's events otherwise), tpi_decode_*.
#include "model.h"

void drop_graph(tpi_model* m) {
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
    } else if (m->opt_rowshard_fused && rowshard_fused_supported(Ks, N)) {
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
  return enqueue_canary_check(m, lc);
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
  if (code == DEVERR_WAIT_TIMEOUT) return fail(TPI_ERR_TIMEOUT, "a bounded wait inside a kernel ran out (the kernel returned early)");
  if (code >= DEVERR_CANARY)
    return fail(TPI_ERR_DEVICE_CHECK, "guard zone %d of the device arena was overwritten (the buffer carved before it, at arena offset < %zu, was overrun)",
                code - DEVERR_CANARY, code - DEVERR_CANARY < m->plan.n_canaries ? m->plan.canary_off[code - DEVERR_CANARY] : (size_t)0);
  return fail(TPI_ERR_DEVICE_CHECK, "device error word = %d", code);
}

// An enqueue that fails part-way leaves kernels of an unfinished step in the stream and, in window mode, the ring
// between an acquire and its release: drain both streams, restart the ring at block 0 and put the device's position
// counter back to the host's, so that the next call starts from a consistent state.
void recover_after_failed_step(tpi_model* m) {
  char saved[512];
  snprintf(saved, sizeof saved, "%s", tpi_last_error());  // keep the original failure's message
  cudaStreamSynchronize(m->cs);
  cudaStreamSynchronize(m->ps);
  cudaGetLastError();
  if (m->sched_open) { m->sched_free.push_back(m->sched_open); m->sched_open = nullptr; }
  if (m->window > 0) start_window(m);
  write_position(m, m->position);
  fail(0, "%s", saved);
}

// io layout (pinned): [0] scratch int, [1] device error word, [2..] token ids
static int run_decode(tpi_model* m, int32_t token_in, int n_steps, int32_t* tokens_out, float* logits) {
  if (!m || n_steps < 1 || !tokens_out) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  if (m->desync) return fail(TPI_ERR_STATE, "an earlier call timed out with work in flight: call tpi_reset or tpi_set_position first");
  const tpi_config& c = m->cfg;
  if (token_in < 0 || token_in >= c.vocab) return fail(TPI_ERR_TOKEN_RANGE, "token %d outside [0, %d)", token_in, c.vocab);
  if (m->position + n_steps > c.max_seq) return fail(TPI_ERR_SEQ_OVERFLOW, "position %d + %d steps exceeds max_seq %d", m->position, n_steps, c.max_seq);
  const Plan& p = m->plan;
  int* io = (int*)(m->host + p.h_io);
  const auto w0 = std::chrono::steady_clock::now();
  io[2] = token_in;
  CK(cudaMemcpyAsync(dptr<int>(m, p.tok_hist) + m->position, io + 2, 4, cudaMemcpyHostToDevice, m->cs));
  const bool use_graph = m->opt_graph && m->window <= 0 && !m->opt_profile;
  if (use_graph) TRY(ensure_graph(m));
  int launches = 0;
  CK(cudaEventRecord(m->ev_t0, m->cs));
  for (int i = 0; i < n_steps; ++i) {
    if (use_graph) { CK(cudaGraphLaunch(m->graph_exec, m->cs)); launches += m->graph_launches; }
    else {
      LaunchCtx lc{m->cs, m->opt_pdl != 0 && !m->opt_profile, &launches};
      m->sched_rec = m->opt_profile != 0;
      const int rc = enqueue_decode(m, lc);
      m->sched_rec = false;
      if (rc) { recover_after_failed_step(m); return rc; }
    }
  }
  CK(cudaEventRecord(m->ev_t1, m->cs));
  CK(cudaMemcpyAsync(io + 3, dptr<int>(m, p.tok_hist) + m->position + 1, (size_t)n_steps * 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaMemcpyAsync(io + 1, m->dev + p.err, 4, cudaMemcpyDeviceToHost, m->cs));
  if (logits) CK(cudaMemcpyAsync(m->host + p.h_logits, m->dev + p.logits, (size_t)c.vocab * 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaEventRecord(m->ev_done, m->cs));
  TRY(wait_event(m, m->ev_done));
  if (io[1] != DEVERR_NONE) {  // the step's results are void: the host position stays, the device counter goes back to it
    const int rc = check_device_error(m, io + 1);
    write_position(m, m->position);
    return rc;
  }
  m->position += n_steps;
  memcpy(tokens_out, io + 3, (size_t)n_steps * 4);
  if (logits) memcpy(logits, m->host + p.h_logits, (size_t)c.vocab * 4);
  float ms = 0;
  cudaEventElapsedTime(&ms, m->ev_t0, m->ev_t1);
  m->st.last_decode_dev_ms = ms;
  m->st.last_decode_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - w0).count();
  m->st.kernel_launches_last = launches;
  if (m->opt_profile) harvest_profile(m);
  return TPI_OK;
}

extern "C" int tpi_decode_step(tpi_model* m, int32_t token_in, int32_t* token_out, float* logits_or_null) {
  return run_decode(m, token_in, 1, token_out, logits_or_null);
}
extern "C" int tpi_decode_run(tpi_model* m, int32_t token_in, int n_steps, int32_t* tokens_out) {
  if (m && n_steps + 3 > m->cfg.max_seq + 2 + m->cfg.max_prefill) return fail(TPI_ERR_INVALID_ARG, "n_steps too large");
  return run_decode(m, token_in, n_steps, tokens_out, nullptr);
}

