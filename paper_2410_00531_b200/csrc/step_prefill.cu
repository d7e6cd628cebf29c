// The prompt pass: Algorithm 1's loop body over T positions at a time (tensor-core projections for bf16 models).
#include "model.h"

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
                  int n_out, int K, int n_batch, bool chunk_k = false) -> int {
    if (tc) {  // split mode: the low halves sit T * lda bf16 elements after the high halves
      const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(A);
      CK(launch_gemm_tc(lc, hi, act_mode == 2 ? hi + (size_t)T * lda : nullptr, lda, a_col, W, w_rows_b, Y, y_bs, ldy, T,
                        n_out, K, n_batch, err, chunk_k));
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
  // What ends a block: the row-sharded projection -> per-shard partial sums, their star sum in rank order + the shortcut
  // (Eq. 1-2), the hidden-state tap of the last position, and (next_gain != nullptr) the next block's RMSNorm.  More
  // than 128 positions of an equal partition: the partial sums are formed and summed inside the GEMM (tensor memory
  // and registers); otherwise they go through PART.
  auto block_end = [&](const float* A, int lda, const void* W, const int* k0, int Ks, float* tap, const float* next_gain) -> int {
    if (tc && act_mode == 2 && !m->unequal && gemm_tc_rowsum_supported(T, Ks, lda, h, h)) {
      const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(A);
      CK(launch_gemm_tc_rowsum(lc, hi, hi + (size_t)T * lda, lda, Ks, W, h, X, h, T, h, Ks, N, err));
      if (tap) CK(cudaMemcpyAsync(tap, X + (size_t)(T - 1) * h, (size_t)h * 4, cudaMemcpyDeviceToDevice, lc.stream));
      if (next_gain) CK(launch_rmsnorm_rows(lc, X, next_gain, T, h, c.rms_eps, Xn, act_mode));
      return TPI_OK;
    }
    TRY(proj_rows(A, lda, W, k0, Ks));
    if (next_gain) CK(launch_reduce_residual_norm_rows(lc, PART, N, T, h, X, tap, next_gain, c.rms_eps, Xn, act_mode));
    else CK(launch_reduce_residual_rows(lc, PART, N, T, h, X, tap));
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
    TRY(proj(Xn, h, 0, br.base + bl.off_qkv, qkv_cols, QKV, 0, qkv_cols, qkv_cols, h, 1, true));
    CK(launch_rope_kv_rows(lc, dt, QKV, T, pos0, Nc, a, b, d, c.max_seq, rope, Q, kc, vc));
    if (m->opt_tensor && prefill_attention_tc_supported(dt, d, T))
      CK(launch_prefill_attention_tc(lc, Q, kc, vc, T, pos0, a, b, c.max_seq, O, act_mode, err));
    else if (m->opt_tensor && prefill_attention_mma_supported(dt, d))
      CK(launch_prefill_attention_mma(lc, Q, kc, vc, T, pos0, a, b, d, c.max_seq, O, act_mode));
    else
      CK(launch_prefill_attention(lc, dt, Q, kc, vc, T, pos0, a, b, d, c.max_seq, O, act_mode));
    float* tap_a = last ? dptr<float>(m, p.taps) + (size_t)(2 * l) * h : nullptr;
    TRY(block_end(O, a * d, br.base + bl.off_wo, ko.data(), Ko, tap_a, fuse_norm ? (const float*)resident_block(m, 2 * l + 1) : nullptr));
    TRY(release_block(m, 2 * l));
    TRY(acquire_block(m, 2 * l + 1, &br));
    if (!fuse_norm) CK(launch_rmsnorm_rows(lc, X, (const float*)br.base, T, h, c.rms_eps, Xn, act_mode));
    if (tc && gemm_tc_swiglu_supported(h, h, s)) {  // SwiGLU in the GEMM's epilogue: the fp32 gate/up rows never reach memory
      const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(Xn);
      CK(launch_gemm_tc_swiglu(lc, hi, act_mode == 2 ? hi + (size_t)T * h : nullptr, h, br.base + bl.off_gu, ACT, act_mode, T, s, h, err));
    } else {
      TRY(proj(Xn, h, 0, br.base + bl.off_gu, 2 * s, GU, 0, 2 * s, 2 * s, h, 1, true));
      CK(launch_swiglu_rows(lc, GU, T, s, ACT, act_mode));
    }
    float* tap_f = last ? dptr<float>(m, p.taps) + (size_t)(2 * l + 1) * h : nullptr;
    normed = fuse_norm && l + 1 < c.n_layers;
    TRY(block_end(ACT, s, br.base + bl.off_down, kd.data(), Kd, tap_f, normed ? (const float*)resident_block(m, 2 * l + 2) : nullptr));
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
  return enqueue_canary_check(m, lc);
}

extern "C" int tpi_prefill(tpi_model* m, const int32_t* tokens, int n_tokens, int32_t* first_token,
                           float* logits_or_null) {
  if (!m || !tokens || n_tokens < 1 || !first_token) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  if (m->desync) return fail(TPI_ERR_STATE, "an earlier call timed out with work in flight: call tpi_reset or tpi_set_position first");
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
    const int rc = enqueue_prefill_chunk(m, lc, p_begin + t0, T, t0 + T == n_tokens);
    if (rc) { recover_after_failed_step(m); return rc; }
  }
  CK(cudaEventRecord(m->ev_t1, m->cs));
  m->st.last_prefill_enqueue_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - w0).count();
  CK(cudaMemcpyAsync(io + 2, dptr<int>(m, p.tok_hist) + p_begin + n_tokens, 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaMemcpyAsync(io + 1, m->dev + p.err, 4, cudaMemcpyDeviceToHost, m->cs));
  if (logits_or_null) CK(cudaMemcpyAsync(m->host + p.h_logits, m->dev + p.logits, (size_t)c.vocab * 4, cudaMemcpyDeviceToHost, m->cs));
  CK(cudaEventRecord(m->ev_done, m->cs));
  TRY(wait_event(m, m->ev_done));
  if (io[1] != DEVERR_NONE) {  // results are void: keep the host position and put the device counter back to it
    const int rc = check_device_error(m, io + 1);
    write_position(m, m->position);
    return rc;
  }
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
  return TPI_OK;
}

