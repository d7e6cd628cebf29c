// One shard per rank (include/tpi_tp.h): every rank is a model of its own over its slices of the weights (a decoder
// with a / R heads, b / R kv heads and s / R FFN columns, one "shard"), with its own arenas, streams and KV cache; this
// file slices the weight source per rank, wires the ranks' receive areas together and drives them in lock step.
#include "../../include/tpi_tp.h"
#include "model.h"

namespace {

// Sec. 3.1 Step 1: rank i takes the proportion p_i of the attention heads (whole kv-head groups) and of the FFN columns.
// Prefix sums over the ranks, R + 1 entries each.
struct Partition {
  std::vector<int> kv0, f0;
};

struct RankFill {  // the weight source as rank `rank` sees it: local tensors cut out of the unsharded ones
  tpi_fill_fn fill = nullptr;
  void* user = nullptr;
  tpi_config cfg{};  // the unsharded model
  int R = 1, rank = 0;
  Partition part;
  std::vector<char> tmp;
};

struct TpRank {
  tpi_model* m = nullptr;
  int device = 0;
  tpi_config lcfg{};
  RankFill rf;
  float* recv = nullptr;  // [2][R][h]
  int* flags = nullptr;   // [2][R]
  int* epoch = nullptr;
  unsigned* ticket = nullptr;
  char* tail = nullptr;
  size_t tail_bytes = 0;
  cudaEvent_t ev_push = nullptr, ev_done = nullptr;
};

// floats of one parity half of a rank's receive area: R sources x (one position's hidden state for a decode step, up
// to max_prefill positions for a prompt pass)
size_t tp_half_floats(const tpi_config& c, int R) { return (size_t)R * c.max_prefill * c.hidden; }
size_t tp_tail_bytes(const tpi_config& c, int R) { return align_up((size_t)2 * tp_half_floats(c, R) * 4, 256) + 3 * 256; }

// The uniform partition p_i = 1/R (lists null), or the given one; validated.
int make_partition(const tpi_config& c, int R, const int32_t* kv_heads, const int32_t* ffn_cols, Partition* out) {
  if (R < 1 || R > TPI_TP_MAX_RANKS) return fail(TPI_ERR_INVALID_ARG, "n_ranks must be in [1, %d]", TPI_TP_MAX_RANKS);
  if ((kv_heads == nullptr) != (ffn_cols == nullptr)) return fail(TPI_ERR_INVALID_ARG, "give both lists or neither");
  if (c.n_heads % c.n_kv_heads) return fail(TPI_ERR_SHAPE, "kv heads must divide heads");
  out->kv0.assign(R + 1, 0);
  out->f0.assign(R + 1, 0);
  if (!kv_heads) {
    if (c.n_heads % R || c.n_kv_heads % R || c.ffn % R)
      return fail(TPI_ERR_SHAPE, "n_ranks=%d must divide heads (%d), kv heads (%d) and ffn (%d)", R, c.n_heads, c.n_kv_heads, c.ffn);
    for (int i = 0; i <= R; ++i) { out->kv0[i] = c.n_kv_heads / R * i; out->f0[i] = c.ffn / R * i; }
    return TPI_OK;
  }
  const int vec = c.dtype == TPI_BF16 ? 8 : 4, grp = c.n_heads / c.n_kv_heads;
  for (int i = 0; i < R; ++i) {
    if (kv_heads[i] < 1 || ffn_cols[i] < 1) return fail(TPI_ERR_SHAPE, "every rank needs at least one kv head and one FFN column");
    if (ffn_cols[i] % vec || (kv_heads[i] * grp * c.head_dim) % vec)
      return fail(TPI_ERR_SHAPE, "a rank's FFN columns and heads*d must be multiples of %d elements (16 bytes)", vec);
    out->kv0[i + 1] = out->kv0[i] + kv_heads[i];
    out->f0[i + 1] = out->f0[i] + ffn_cols[i];
  }
  if (out->kv0[R] != c.n_kv_heads || out->f0[R] != c.ffn)
    return fail(TPI_ERR_SHAPE, "the ranks' kv heads (%d of %d) and FFN columns (%d of %d) must add up", out->kv0[R], c.n_kv_heads, out->f0[R], c.ffn);
  return TPI_OK;
}

int slice_of(const tpi_config& c, const Partition& part, int rank, int tid, int64_t* row0, int64_t* n_rows, int64_t* col0, int64_t* n_cols) {
  const int R = (int)part.kv0.size() - 1;
  if (rank < 0 || rank >= R) return fail(TPI_ERR_INVALID_ARG, "rank %d of %d", rank, R);
  const int64_t h = c.hidden, d = c.head_dim, grp = c.n_heads / c.n_kv_heads;
  const int64_t q0 = (int64_t)part.kv0[rank] * grp * d, qn = (int64_t)(part.kv0[rank + 1] - part.kv0[rank]) * grp * d;  // query rows
  const int64_t k0 = (int64_t)part.kv0[rank] * d, kn = (int64_t)(part.kv0[rank + 1] - part.kv0[rank]) * d;              // key / value rows
  const int64_t s0 = part.f0[rank], sn = part.f0[rank + 1] - part.f0[rank];                                                // FFN columns
  int64_t r0 = 0, nr = 0, c0 = 0, nc = h;
  switch (tid) {
    case TPI_T_EMB: case TPI_T_HEAD: nr = rank == 0 ? c.vocab : 0; break;
    case TPI_T_FINAL_NORM: nr = rank == 0 ? 1 : 0; break;
    case TPI_T_ATTN_NORM: case TPI_T_FFN_NORM: nr = 1; break;
    case TPI_T_WQ: r0 = q0; nr = qn; break;
    case TPI_T_WK: case TPI_T_WV: r0 = k0; nr = kn; break;
    case TPI_T_WO: nr = h; c0 = q0; nc = qn; break;
    case TPI_T_WGATE: case TPI_T_WUP: r0 = s0; nr = sn; break;
    case TPI_T_WDOWN: nr = h; c0 = s0; nc = sn; break;
    default: return fail(TPI_ERR_INVALID_ARG, "unknown tensor id %d", tid);
  }
  if (row0) *row0 = r0;
  if (n_rows) *n_rows = nr;
  if (col0) *col0 = c0;
  if (n_cols) *n_cols = nc;
  return TPI_OK;
}

// tpi_fill_fn of a rank's local model: rows [row0, row0 + n) of the LOCAL tensor.
int rank_fill(void* user, int tid, int layer, int64_t row0, int64_t n, void* dst) {
  RankFill* f = (RankFill*)user;
  const tpi_config& c = f->cfg;
  const size_t B = elem_size(c.dtype);
  int64_t r0, nr, c0, nc;
  if (slice_of(c, f->part, f->rank, tid, &r0, &nr, &c0, &nc)) return 1;
  if (nr == 0) {  // a tensor this rank does not hold (workers: embedding, head, final norm): a one-row placeholder
    memset(dst, 0, (size_t)n * nc * B);
    return 0;
  }
  const bool col_slice = tid == TPI_T_WO || tid == TPI_T_WDOWN;
  if (!col_slice) return f->fill(f->user, tid, layer, r0 + row0, n, dst);
  const int64_t full = tid == TPI_T_WO ? (int64_t)c.n_heads * c.head_dim : c.ffn;  // unsharded row length
  int64_t per = (int64_t)((size_t)(32u << 20) / ((size_t)full * B));
  if (per < 1) per = 1;
  if (f->tmp.size() < (size_t)per * full * B) f->tmp.resize((size_t)per * full * B);
  for (int64_t i = 0; i < n; i += per) {
    const int64_t m = n - i < per ? n - i : per;
    if (f->fill(f->user, tid, layer, row0 + i, m, f->tmp.data())) return 1;
    for (int64_t r = 0; r < m; ++r)
      memcpy((char*)dst + (size_t)(i + r) * nc * B, f->tmp.data() + ((size_t)r * full + c0) * B, (size_t)nc * B);
  }
  return 0;
}

tpi_config local_cfg(const tpi_config& c, const Partition& part, int rank) {
  tpi_config l = c;
  l.n_kv_heads = part.kv0[rank + 1] - part.kv0[rank];
  l.n_heads = l.n_kv_heads * (c.n_heads / c.n_kv_heads);
  l.ffn = part.f0[rank + 1] - part.f0[rank];
  if (rank != 0) l.vocab = 1;  // workers hold no embedding and no head (Sec. 3.1: they reside on the master)
  return l;
}

}  // namespace

struct tpi_tp_group {
  tpi_config cfg{};
  int R = 0, window = 0;
  Partition part;
  std::vector<TpRank> ranks;
  int events = 1, wait_polls = 1 << 21, drop_rank = -1, pdl = 1, batched_prompt = 1, use_graph = 1;
  cudaGraphExec_t graph_exec = nullptr;  // one decode position of ALL ranks (resident groups only)
  int graph_launches = 0;
  cudaEvent_t ev_graph = nullptr;
  int position = 0, launches_last = 0;
  bool broken = false;  // a call failed or timed out: tpi_tp_reset first
  uint64_t exchanges = 0;
  double last_decode_ms = 0;
};

namespace {

struct DeviceGuard {  // calls switch between the ranks' devices and put the caller's back at the end
  int saved = 0;
  DeviceGuard() { cudaGetDevice(&saved); }
  ~DeviceGuard() { cudaSetDevice(saved); }
};

TpPeers peers_of(const tpi_tp_group* g, int rank) {
  TpPeers P{};
  P.n_ranks = g->R;
  P.rank = rank;
  P.half = (long long)tp_half_floats(g->cfg, g->R);
  for (int j = 0; j < g->R; ++j) { P.recv[j] = g->ranks[j].recv; P.flags[j] = g->ranks[j].flags; }
  return P;
}

bool share_a_device(const tpi_tp_group* g) {
  for (int i = 0; i < g->R; ++i)
    for (int j = i + 1; j < g->R; ++j)
      if (g->ranks[i].device == g->ranks[j].device) return true;
  return false;
}

// One position through all ranks (enqueue only).  with_head: the master runs the task head and the greedy argmax
// (which advance its position); otherwise (a prompt position that is not the last) its last consumer advances it.
int enqueue_step(tpi_tp_group* g, bool with_head, int* launches, bool force_edges = false) {
  const tpi_config& c = g->cfg;
  const bool edges = g->events || force_edges;  // inside a graph capture the cross-stream waits ARE the graph's edges
  const int R = g->R, h = c.hidden, d = c.head_dim, dt = c.dtype, L = c.n_layers;
  auto ctx = [&](TpRank& r) { return LaunchCtx{r.m->cs, g->pdl != 0, launches}; };
  auto drop_now = [&](int rank) {  // one-shot failure injection: this rank computes but never publishes
    if (g->drop_rank != rank) return 0;
    g->drop_rank = -1;
    return 1;
  };
  auto consume = [&](int mode, int layer_tap, bool advance_workers) -> int {  // every rank waits for the sources, then sums
    for (int i = 0; i < R; ++i) {
      TpRank& r = g->ranks[i];
      tpi_model* m = r.m;
      const Plan& p = m->plan;
      CK(cudaSetDevice(r.device));
      if (edges) {
        if (mode == 1) { if (i != 0) CK(cudaStreamWaitEvent(m->cs, g->ranks[0].ev_push, 0)); }
        else
          for (int j = 0; j < R; ++j)
            if (j != i) CK(cudaStreamWaitEvent(m->cs, g->ranks[j].ev_push, 0));
      }
      LaunchCtx lc = ctx(r);
      float* tap = layer_tap >= 0 ? dptr<float>(m, p.taps) + (size_t)layer_tap * h : nullptr;
      const bool adv = advance_workers && !(i == 0 && with_head);
      CK(launch_tp_recv(lc, r.recv, (long long)tp_half_floats(c, R), r.flags, r.epoch, R, h, mode, c.rms_eps, dptr<float>(m, p.x), dptr<float>(m, p.xhat), tap,
                        dptr<float>(m, p.ss_part), rowshard_fused_parts(h), adv ? dptr<int>(m, p.pos) : nullptr,
                        dptr<int>(m, p.err), g->wait_polls));
    }
    ++g->exchanges;
    return TPI_OK;
  };
  // ---- the master embeds the token and sends the hidden state to every rank (Algorithm 1: preprocess, broadcast)
  {
    TpRank& r = g->ranks[0];
    tpi_model* m = r.m;
    const Plan& p = m->plan;
    CK(cudaSetDevice(r.device));
    LaunchCtx lc = ctx(r);
    CK(launch_embed(lc, dt, m->dev + p.emb, dptr<int>(m, p.tok_hist), dptr<int>(m, p.pos), c.vocab, c.max_seq, h, c.rms_eps,
                    dptr<float>(m, p.x), dptr<float>(m, p.xhat), dptr<float>(m, p.ss_part), rowshard_fused_parts(h),
                    dptr<int>(m, p.err)));
    CK(launch_tp_bcast(lc, dptr<float>(m, p.x), h, r.epoch, peers_of(g, 0), drop_now(0)));
    if (edges) CK(cudaEventRecord(r.ev_push, m->cs));
  }
  TRY(consume(1, -1, false));
  for (int l = 0; l < L; ++l) {
    for (int blk = 0; blk < 2; ++blk) {
      for (int i = 0; i < R; ++i) {  // every rank: its block's column-sharded part, then its partial sums go out
        TpRank& r = g->ranks[i];
        tpi_model* m = r.m;
        const Plan& p = m->plan;
        const BlockLayout& bl = p.bl;
        CK(cudaSetDevice(r.device));
        LaunchCtx lc = ctx(r);
        const int al = r.lcfg.n_heads, bl_ = r.lcfg.n_kv_heads, sl = r.lcfg.ffn;  // this rank's share
        BlockRef br;
        TRY(acquire_block(m, 2 * l + blk, &br));
        const NormIn in{dptr<float>(m, p.x), (const float*)br.base, dptr<float>(m, p.ss_part), rowshard_fused_parts(h), c.rms_eps};
        if (blk == 0) {
          void* kc = m->dev + p.kcache + (size_t)l * p.kv_layer_bytes;
          void* vc = m->dev + p.vcache + (size_t)l * p.kv_layer_bytes;
          CK(launch_gemv_qkv(lc, dt, br.base + bl.off_qkv, (size_t)(al + 2 * bl_) * d * h, in, h, 1, al, bl_, d, c.max_seq,
                             dptr<int>(m, p.pos), dptr<float2>(m, p.rope), dptr<float>(m, p.q), kc, vc));
          CK(launch_decode_attention(lc, dt, dptr<float>(m, p.q), kc, vc, dptr<int>(m, p.pos), al, bl_, d, c.max_seq, p.nsplit,
                                     dptr<float>(m, p.attn_scratch), dptr<unsigned>(m, p.tickets), dptr<float>(m, p.o)));
          CK(launch_tp_rowpush(lc, dt, br.base + bl.off_wo, dptr<float>(m, p.o), h, al * d, r.epoch, r.ticket, peers_of(g, i),
                               drop_now(i)));
        } else {
          CK(launch_gemv_gateup(lc, dt, br.base + bl.off_gu, (size_t)2 * sl * h, in, h, 1, sl, dptr<float>(m, p.act)));
          CK(launch_tp_rowpush(lc, dt, br.base + bl.off_down, dptr<float>(m, p.act), h, sl, r.epoch, r.ticket, peers_of(g, i),
                               drop_now(i)));
        }
        TRY(release_block(m, 2 * l + blk));
        if (edges) CK(cudaEventRecord(r.ev_push, m->cs));
      }
      TRY(consume(0, 2 * l + blk, l == L - 1 && blk == 1));
    }
  }
  if (with_head) {  // Algorithm 1: the master alone runs the task head (postprocess) and picks the token
    TpRank& r = g->ranks[0];
    tpi_model* m = r.m;
    const Plan& p = m->plan;
    CK(cudaSetDevice(r.device));
    LaunchCtx lc = ctx(r);
    CK(launch_head_argmax(lc, dt, m->dev + p.head,
                          NormIn{dptr<float>(m, p.x), dptr<float>(m, p.final_gain), dptr<float>(m, p.ss_part), rowshard_fused_parts(h), c.rms_eps},
                          h, c.vocab, dptr<float>(m, p.logits), dptr<float>(m, p.amax_val), dptr<int>(m, p.amax_idx),
                          dptr<unsigned>(m, p.tickets) + r.lcfg.n_kv_heads, dptr<int>(m, p.tok_hist), dptr<int>(m, p.pos), 1));
  }
  for (int i = 0; i < R; ++i) {  // debug arenas (TPI_DEBUG=1): every rank's guard zones are compared after the step
    TpRank& r = g->ranks[i];
    if (r.m->plan.n_canaries < 1) break;
    CK(cudaSetDevice(r.device));
    LaunchCtx lc = ctx(r);
    TRY(enqueue_canary_check(r.m, lc));
  }
  return TPI_OK;
}

// T prompt positions [pos0, pos0 + T) through all ranks at once (enqueue only): Algorithm 1's loop body with T
// positions per rank, every rank on its own heads and FFN columns.  The row-sharded projections leave T x h partial
// sums per rank, which go to every rank's receive area (tp_push_rows_kernel); the consumer is the wait kernel followed
// by the ordinary row kernel that adds R partial sums in rank order and the shortcut (and applies the next RMSNorm).
// The host addresses the receive area by the parity of its own exchange count, which equals the device counter as long
// as no wait ran out (after one, the call fails and tpi_tp_reset puts both back to zero).
int enqueue_prompt_chunk(tpi_tp_group* g, int pos0, int T, bool last, int* launches) {
  const tpi_config& c = g->cfg;
  const int R = g->R, h = c.hidden, d = c.head_dim, dt = c.dtype, L = c.n_layers;
  const size_t half = tp_half_floats(c, R);
  auto ctx = [&](TpRank& r) { return LaunchCtx{r.m->cs, g->pdl != 0, launches}; };
  auto drop_now = [&](int rank) {
    if (g->drop_rank != rank) return 0;
    g->drop_rank = -1;
    return 1;
  };
  // split bf16 activations on the tensor cores where every contraction of EVERY rank qualifies (all ranks use the same
  // arithmetic, so that the partition does not change which kernels run), fp32 SIMT otherwise
  bool tc = dt == TPI_BF16 && g->ranks[0].m->opt_tensor;
  for (int i = 0; i < R && tc; ++i) {
    const tpi_config& lc_ = g->ranks[i].lcfg;
    tc = gemm_tc_supported(h, h, (lc_.n_heads + 2 * lc_.n_kv_heads) * d) && gemm_tc_supported(h, h, 2 * lc_.ffn) &&
         gemm_tc_supported(lc_.n_heads * d, lc_.n_heads * d, h) && gemm_tc_supported(lc_.ffn, lc_.ffn, h);
  }
  const int act_mode = tc ? 2 : 0;
  const bool fuse_norm = g->window <= 0;  // a streamed rank may not hold the next block's gain yet
  auto gemm = [&](TpRank& r, LaunchCtx& lc, const float* A, int lda, const void* W, float* Y, int ldy, int n_out, int K,
                  bool chunk_k = false) -> int {
    if (tc) {
      const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(A);
      CK(launch_gemm_tc(lc, hi, hi + (size_t)T * lda, lda, 0, W, n_out, Y, 0, ldy, T, n_out, K, 1, dptr<int>(r.m, r.m->plan.err), chunk_k));
    } else {
      CK(launch_gemm_simt(lc, dt, A, 0, lda, W, 0, Y, 0, ldy, T, n_out, K, 1));
    }
    return TPI_OK;
  };
  // every rank waits for `n_src` sources of the current exchange; returns the receive parity in *parity
  auto wait_all = [&](int n_src) -> int {
    for (int i = 0; i < R; ++i) {
      TpRank& r = g->ranks[i];
      CK(cudaSetDevice(r.device));
      if (g->events)
        for (int j = 0; j < (n_src == 1 ? 1 : R); ++j)
          if (j != i) CK(cudaStreamWaitEvent(r.m->cs, g->ranks[j].ev_push, 0));
      LaunchCtx lc = ctx(r);
      CK(launch_tp_wait(lc, r.flags, r.epoch, R, n_src, dptr<int>(r.m, r.m->plan.err), g->wait_polls));
    }
    return TPI_OK;
  };
  // ---- the master embeds the T tokens and sends the rows to every rank
  {
    TpRank& r = g->ranks[0];
    tpi_model* m = r.m;
    const Plan& p = m->plan;
    CK(cudaSetDevice(r.device));
    LaunchCtx lc = ctx(r);
    CK(launch_embed_rows(lc, dt, m->dev + p.emb, dptr<int>(m, p.tok_hist), pos0, T, c.vocab, h, dptr<float>(m, p.pX), dptr<int>(m, p.err)));
    CK(launch_tp_push_rows(lc, dptr<float>(m, p.pX), (size_t)T * h, r.epoch, r.ticket, peers_of(g, 0), 1, drop_now(0)));
    if (g->events) CK(cudaEventRecord(r.ev_push, m->cs));
  }
  {
    const int parity = (int)(g->exchanges & 1);
    TRY(wait_all(1));
    for (int i = 1; i < R; ++i) {  // the workers take the rows out of the master's slot
      TpRank& r = g->ranks[i];
      CK(cudaSetDevice(r.device));
      CK(cudaMemcpyAsync(dptr<float>(r.m, r.m->plan.pX), r.recv + (size_t)parity * half, (size_t)T * h * 4,
                         cudaMemcpyDeviceToDevice, r.m->cs));
    }
    ++g->exchanges;
  }
  std::vector<char> normed(R, 0);  // Xn already holds the input of the block about to start
  for (int l = 0; l < L; ++l) {
    for (int blk = 0; blk < 2; ++blk) {
      for (int i = 0; i < R; ++i) {
        TpRank& r = g->ranks[i];
        tpi_model* m = r.m;
        const Plan& p = m->plan;
        const BlockLayout& bl = p.bl;
        CK(cudaSetDevice(r.device));
        LaunchCtx lc = ctx(r);
        const int al = r.lcfg.n_heads, bl_ = r.lcfg.n_kv_heads, sl = r.lcfg.ffn, qkv_cols = (al + 2 * bl_) * d;
        float *X = dptr<float>(m, p.pX), *Xn = dptr<float>(m, p.pXn), *PART = dptr<float>(m, p.pPART);
        BlockRef br;
        TRY(acquire_block(m, 2 * l + blk, &br));
        if (!normed[i]) CK(launch_rmsnorm_rows(lc, X, (const float*)br.base, T, h, c.rms_eps, Xn, act_mode));
        if (blk == 0) {
          float *QKV = dptr<float>(m, p.pQKV), *Q = dptr<float>(m, p.pQ), *O = dptr<float>(m, p.pO);
          void* kc = m->dev + p.kcache + (size_t)l * p.kv_layer_bytes;
          void* vc = m->dev + p.vcache + (size_t)l * p.kv_layer_bytes;
          TRY(gemm(r, lc, Xn, h, br.base + bl.off_qkv, QKV, qkv_cols, qkv_cols, h, true));
          CK(launch_rope_kv_rows(lc, dt, QKV, T, pos0, 1, al, bl_, d, c.max_seq, dptr<float2>(m, p.rope), Q, kc, vc));
          if (m->opt_tensor && prefill_attention_tc_supported(dt, d, T))
            CK(launch_prefill_attention_tc(lc, Q, kc, vc, T, pos0, al, bl_, c.max_seq, O, act_mode, dptr<int>(m, p.err)));
          else if (m->opt_tensor && prefill_attention_mma_supported(dt, d))
            CK(launch_prefill_attention_mma(lc, Q, kc, vc, T, pos0, al, bl_, d, c.max_seq, O, act_mode));
          else
            CK(launch_prefill_attention(lc, dt, Q, kc, vc, T, pos0, al, bl_, d, c.max_seq, O, act_mode));
          TRY(gemm(r, lc, O, al * d, br.base + bl.off_wo, PART, h, h, al * d));
        } else {
          float *GU = dptr<float>(m, p.pGU), *ACT = dptr<float>(m, p.pACT);
          if (tc && gemm_tc_swiglu_supported(h, h, sl)) {
            const __nv_bfloat16* hi = reinterpret_cast<const __nv_bfloat16*>(Xn);
            CK(launch_gemm_tc_swiglu(lc, hi, hi + (size_t)T * h, h, br.base + bl.off_gu, ACT, act_mode, T, sl, h, dptr<int>(m, p.err)));
          } else {
            TRY(gemm(r, lc, Xn, h, br.base + bl.off_gu, GU, 2 * sl, 2 * sl, h, true));
            CK(launch_swiglu_rows(lc, GU, T, sl, ACT, act_mode));
          }
          TRY(gemm(r, lc, ACT, sl, br.base + bl.off_down, PART, h, h, sl));
        }
        CK(launch_tp_push_rows(lc, PART, (size_t)T * h, r.epoch, r.ticket, peers_of(g, i), 0, drop_now(i)));
        TRY(release_block(m, 2 * l + blk));
        if (g->events) CK(cudaEventRecord(r.ev_push, m->cs));
      }
      const int parity = (int)(g->exchanges & 1);
      TRY(wait_all(R));
      const bool more = !(l == L - 1 && blk == 1);
      for (int i = 0; i < R; ++i) {  // ((P_0 + P_1) + ...) + X for T rows, and the next block's norm where its gain is at hand
        TpRank& r = g->ranks[i];
        tpi_model* m = r.m;
        const Plan& p = m->plan;
        CK(cudaSetDevice(r.device));
        LaunchCtx lc = ctx(r);
        const float* parts = r.recv + (size_t)parity * half;  // [R][T][h]: source j's rows at j * T * h
        float* tap = last ? dptr<float>(m, p.taps) + (size_t)(2 * l + blk) * h : nullptr;
        normed[i] = fuse_norm && more;
        if (normed[i])
          CK(launch_reduce_residual_norm_rows(lc, parts, R, T, h, dptr<float>(m, p.pX), tap, (const float*)resident_block(m, 2 * l + blk + 1),
                                              c.rms_eps, dptr<float>(m, p.pXn), act_mode));
        else
          CK(launch_reduce_residual_rows(lc, parts, R, T, h, dptr<float>(m, p.pX), tap));
      }
      ++g->exchanges;
    }
  }
  if (last) {
    TpRank& r = g->ranks[0];
    tpi_model* m = r.m;
    const Plan& p = m->plan;
    CK(cudaSetDevice(r.device));
    LaunchCtx lc = ctx(r);
    const int n_parts = rowshard_fused_parts(h);
    CK(launch_rmsnorm_stat_row(lc, dptr<float>(m, p.pX) + (size_t)(T - 1) * h, h, c.rms_eps, dptr<float>(m, p.x), dptr<float>(m, p.xhat),
                               dptr<float>(m, p.ss_part), n_parts, dptr<int>(m, p.pos), pos0 + T - 1));
    CK(launch_head_argmax(lc, dt, m->dev + p.head,
                          NormIn{dptr<float>(m, p.x), dptr<float>(m, p.final_gain), dptr<float>(m, p.ss_part), n_parts, c.rms_eps}, h,
                          c.vocab, dptr<float>(m, p.logits), dptr<float>(m, p.amax_val), dptr<int>(m, p.amax_idx),
                          dptr<unsigned>(m, p.tickets) + r.lcfg.n_kv_heads, dptr<int>(m, p.tok_hist), dptr<int>(m, p.pos), 1));
  }
  for (int i = 0; i < R; ++i) {  // debug arenas (TPI_DEBUG=1): every rank's guard zones are compared after the step
    TpRank& r = g->ranks[i];
    if (r.m->plan.n_canaries < 1) break;
    CK(cudaSetDevice(r.device));
    LaunchCtx lc = ctx(r);
    TRY(enqueue_canary_check(r.m, lc));
  }
  return TPI_OK;
}

// The prompt in chunks of max_prefill positions through enqueue_prompt_chunk.
int run_prompt(tpi_tp_group* g, const int32_t* tokens, int n, int32_t* first, float* logits) {
  if (g->broken) return fail(TPI_ERR_STATE, "an earlier call failed or timed out: call tpi_tp_reset first");
  const tpi_config& c = g->cfg;
  if (g->position + n > c.max_seq) return fail(TPI_ERR_SEQ_OVERFLOW, "position %d + %d exceeds max_seq %d", g->position, n, c.max_seq);
  for (int i = 0; i < n; ++i)
    if (tokens[i] < 0 || tokens[i] >= c.vocab) return fail(TPI_ERR_TOKEN_RANGE, "token %d outside [0, %d)", tokens[i], c.vocab);
  DeviceGuard guard;
  const auto w0 = std::chrono::steady_clock::now();
  tpi_model* m0 = g->ranks[0].m;
  int* io0 = (int*)(m0->host + m0->plan.h_io);
  int launches = 0;
  g->broken = true;
  const int p_begin = g->position;
  for (int t0 = 0; t0 < n; t0 += c.max_prefill) {
    const int T = n - t0 < c.max_prefill ? n - t0 : c.max_prefill;
    CK(cudaSetDevice(g->ranks[0].device));
    if (t0) TRY(wait_event(m0, g->ranks[0].ev_done));  // the pinned token area is free again
    memcpy(io0 + 3, tokens + t0, (size_t)T * 4);
    CK(cudaMemcpyAsync(dptr<int>(m0, m0->plan.tok_hist) + p_begin + t0, io0 + 3, (size_t)T * 4, cudaMemcpyHostToDevice, m0->cs));
    CK(cudaEventRecord(g->ranks[0].ev_done, m0->cs));
    TRY(enqueue_prompt_chunk(g, p_begin + t0, T, t0 + T == n, &launches));
  }
  for (int i = 1; i < g->R; ++i) {  // the workers' position counters (the master's was set by its head)
    TpRank& r = g->ranks[i];
    int* io = (int*)(r.m->host + r.m->plan.h_io);
    io[0] = p_begin + n;
    CK(cudaSetDevice(r.device));
    CK(cudaMemcpyAsync(r.m->dev + r.m->plan.pos, io, 4, cudaMemcpyHostToDevice, r.m->cs));
  }
  CK(cudaSetDevice(g->ranks[0].device));
  CK(cudaMemcpyAsync(io0 + 2, dptr<int>(m0, m0->plan.tok_hist) + p_begin + n, 4, cudaMemcpyDeviceToHost, m0->cs));
  if (logits) CK(cudaMemcpyAsync(m0->host + m0->plan.h_logits, m0->dev + m0->plan.logits, (size_t)c.vocab * 4, cudaMemcpyDeviceToHost, m0->cs));
  for (int i = 0; i < g->R; ++i) {
    TpRank& r = g->ranks[i];
    int* io = (int*)(r.m->host + r.m->plan.h_io);
    CK(cudaSetDevice(r.device));
    CK(cudaMemcpyAsync(io + 1, r.m->dev + r.m->plan.err, 4, cudaMemcpyDeviceToHost, r.m->cs));
    CK(cudaEventRecord(r.ev_done, r.m->cs));
  }
  for (int i = 0; i < g->R; ++i) {
    CK(cudaSetDevice(g->ranks[i].device));
    TRY(wait_event(g->ranks[i].m, g->ranks[i].ev_done));
  }
  for (int i = 0; i < g->R; ++i) {
    const int code = ((int*)(g->ranks[i].m->host + g->ranks[i].m->plan.h_io))[1];
    if (code == DEVERR_NONE) continue;
    if (code == DEVERR_WAIT_TIMEOUT)
      return fail(TPI_ERR_TIMEOUT, "rank %d gave up waiting for another rank's partial sums (bounded wait ran out); call tpi_tp_reset", i);
    if (code == DEVERR_TOKEN_RANGE) return fail(TPI_ERR_TOKEN_RANGE, "a token id was outside [0, vocab)");
    return fail(TPI_ERR_DEVICE_CHECK, "rank %d: device error word = %d", i, code);
  }
  g->broken = false;
  g->position = p_begin + n;
  for (auto& r : g->ranks) r.m->position = g->position;
  *first = io0[2];
  if (logits) memcpy(logits, m0->host + m0->plan.h_logits, (size_t)c.vocab * 4);
  g->launches_last = launches;
  g->last_decode_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - w0).count();
  return TPI_OK;
}

void drop_group_graph(tpi_tp_group* g) {
  if (g->graph_exec) cudaGraphExecDestroy(g->graph_exec);
  g->graph_exec = nullptr;
}

// One decode position of all ranks as ONE CUDA graph: captured from the master's compute stream, the other ranks'
// streams join the capture through the exchange's event waits (which become the graph's edges) and are joined back at
// the end.  A token then costs the host one launch instead of 2 + R (1 + 7 L).
int ensure_group_graph(tpi_tp_group* g) {
  if (g->graph_exec) return TPI_OK;
  TpRank& r0 = g->ranks[0];
  cudaStream_t origin = r0.m->cs;
  CK(cudaSetDevice(r0.device));
  const uint64_t saved = g->exchanges;
  int launches = 0;
  cudaGraph_t graph = nullptr;
  CK(cudaStreamBeginCapture(origin, cudaStreamCaptureModeThreadLocal));
  int rc = enqueue_step(g, true, &launches, true);
  cudaError_t e = cudaSuccess;
  for (int i = 1; i < g->R && rc == TPI_OK && e == cudaSuccess; ++i) {  // join every rank's stream back
    TpRank& r = g->ranks[i];
    cudaSetDevice(r.device);
    e = cudaEventRecord(r.ev_push, r.m->cs);
    cudaSetDevice(r0.device);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(origin, r.ev_push, 0);
  }
  cudaSetDevice(r0.device);
  const cudaError_t e2 = cudaStreamEndCapture(origin, &graph);
  g->exchanges = saved;
  if (rc) { if (graph) cudaGraphDestroy(graph); return rc; }
  if (e != cudaSuccess || e2 != cudaSuccess) {
    if (graph) cudaGraphDestroy(graph);
    cudaGetLastError();
    return fail(TPI_ERR_CUDA, "capturing the ranks' decode step failed: %s", cudaGetErrorString(e != cudaSuccess ? e : e2));
  }
  e = cudaGraphInstantiate(&g->graph_exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e != cudaSuccess) { g->graph_exec = nullptr; return fail(TPI_ERR_CUDA, "graph instantiate failed: %s", cudaGetErrorString(e)); }
  g->graph_launches = launches;
  return TPI_OK;
}

// Feeds n positions: tokens[] (n_given of them, the rest are the ranks' own outputs chained on the master) and returns
// the master's tokens after each of the last n_out positions.
int run_positions(tpi_tp_group* g, const int32_t* tokens, int n_given, int n_pos, bool head_every, int32_t* out, int n_out,
                  float* logits) {
  if (g->broken) return fail(TPI_ERR_STATE, "an earlier call failed or timed out: call tpi_tp_reset first");
  const tpi_config& c = g->cfg;
  if (g->position + n_pos > c.max_seq) return fail(TPI_ERR_SEQ_OVERFLOW, "position %d + %d exceeds max_seq %d", g->position, n_pos, c.max_seq);
  for (int i = 0; i < n_given; ++i)
    if (tokens[i] < 0 || tokens[i] >= c.vocab) return fail(TPI_ERR_TOKEN_RANGE, "token %d outside [0, %d)", tokens[i], c.vocab);
  DeviceGuard guard;
  const auto w0 = std::chrono::steady_clock::now();
  tpi_model* m0 = g->ranks[0].m;
  int* io0 = (int*)(m0->host + m0->plan.h_io);
  CK(cudaSetDevice(g->ranks[0].device));
  memcpy(io0 + 3, tokens, (size_t)n_given * 4);
  CK(cudaMemcpyAsync(dptr<int>(m0, m0->plan.tok_hist) + g->position, io0 + 3, (size_t)n_given * 4, cudaMemcpyHostToDevice, m0->cs));
  int launches = 0;
  g->broken = true;  // until the call has gone through
  const bool graph = g->use_graph && g->window <= 0 && head_every && g->drop_rank < 0;
  if (graph) TRY(ensure_group_graph(g));
  for (int i = 0; i < n_pos; ++i) {
    if (graph) {
      CK(cudaSetDevice(g->ranks[0].device));
      CK(cudaGraphLaunch(g->graph_exec, m0->cs));
      launches += g->graph_launches;
      g->exchanges += 2ull * c.n_layers + 1;
    } else {
      TRY(enqueue_step(g, head_every || i == n_pos - 1, &launches));
    }
  }
  if (graph) {  // the other ranks' streams took no part in the launch: what they do next comes after the graph
    CK(cudaSetDevice(g->ranks[0].device));
    CK(cudaEventRecord(g->ev_graph, m0->cs));
    for (int i = 1; i < g->R; ++i) {
      CK(cudaSetDevice(g->ranks[i].device));
      CK(cudaStreamWaitEvent(g->ranks[i].m->cs, g->ev_graph, 0));
    }
  }
  // results and error words
  CK(cudaSetDevice(g->ranks[0].device));
  CK(cudaMemcpyAsync(io0 + 3, dptr<int>(m0, m0->plan.tok_hist) + g->position + n_pos - n_out + 1, (size_t)n_out * 4,
                     cudaMemcpyDeviceToHost, m0->cs));
  if (logits) CK(cudaMemcpyAsync(m0->host + m0->plan.h_logits, m0->dev + m0->plan.logits, (size_t)c.vocab * 4, cudaMemcpyDeviceToHost, m0->cs));
  for (int i = 0; i < g->R; ++i) {
    TpRank& r = g->ranks[i];
    int* io = (int*)(r.m->host + r.m->plan.h_io);
    CK(cudaSetDevice(r.device));
    CK(cudaMemcpyAsync(io + 1, r.m->dev + r.m->plan.err, 4, cudaMemcpyDeviceToHost, r.m->cs));
    CK(cudaEventRecord(r.ev_done, r.m->cs));
  }
  for (int i = 0; i < g->R; ++i) {
    CK(cudaSetDevice(g->ranks[i].device));
    TRY(wait_event(g->ranks[i].m, g->ranks[i].ev_done));
  }
  for (int i = 0; i < g->R; ++i) {
    const int code = ((int*)(g->ranks[i].m->host + g->ranks[i].m->plan.h_io))[1];
    if (code == DEVERR_NONE) continue;
    if (code == DEVERR_WAIT_TIMEOUT)
      return fail(TPI_ERR_TIMEOUT, "rank %d gave up waiting for another rank's partial sums (bounded wait ran out); call tpi_tp_reset", i);
    if (code == DEVERR_TOKEN_RANGE) return fail(TPI_ERR_TOKEN_RANGE, "a token id was outside [0, vocab)");
    return fail(TPI_ERR_DEVICE_CHECK, "rank %d: device error word = %d", i, code);
  }
  g->broken = false;
  g->position += n_pos;
  for (auto& r : g->ranks) r.m->position = g->position;
  memcpy(out, io0 + 3, (size_t)n_out * 4);
  if (logits) memcpy(logits, m0->host + m0->plan.h_logits, (size_t)c.vocab * 4);
  g->launches_last = launches;
  g->last_decode_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - w0).count();
  return TPI_OK;
}

}  // namespace

extern "C" int tpi_tp_rank_slice_p(const tpi_config* cfg, int n_ranks, int rank, const int32_t* kv_heads_per_rank,
                                   const int32_t* ffn_cols_per_rank, int tensor_id, int64_t* row0, int64_t* n_rows, int64_t* col0,
                                   int64_t* n_cols) {
  if (!cfg) return fail(TPI_ERR_INVALID_ARG, "null config");
  Partition part;
  TRY(make_partition(*cfg, n_ranks, kv_heads_per_rank, ffn_cols_per_rank, &part));
  return slice_of(*cfg, part, rank, tensor_id, row0, n_rows, col0, n_cols);
}
extern "C" int tpi_tp_rank_slice(const tpi_config* cfg, int n_ranks, int rank, int tensor_id, int64_t* row0, int64_t* n_rows,
                                 int64_t* col0, int64_t* n_cols) {
  return tpi_tp_rank_slice_p(cfg, n_ranks, rank, nullptr, nullptr, tensor_id, row0, n_rows, col0, n_cols);
}

extern "C" int tpi_tp_query_arena(const tpi_config* cfg, int n_ranks, int rank, int window_blocks, size_t* dev_bytes,
                                  size_t* host_bytes) {
  return tpi_tp_query_arena_p(cfg, n_ranks, rank, nullptr, nullptr, window_blocks, dev_bytes, host_bytes);
}
extern "C" int tpi_tp_query_arena_p(const tpi_config* cfg, int n_ranks, int rank, const int32_t* kv_heads_per_rank,
                                    const int32_t* ffn_cols_per_rank, int window_blocks, size_t* dev_bytes, size_t* host_bytes) {
  if (!cfg) return fail(TPI_ERR_INVALID_ARG, "null config");
  Partition part;
  TRY(make_partition(*cfg, n_ranks, kv_heads_per_rank, ffn_cols_per_rank, &part));
  TRY(slice_of(*cfg, part, rank, TPI_T_WQ, nullptr, nullptr, nullptr, nullptr));
  const tpi_config l = local_cfg(*cfg, part, rank);
  size_t d = 0, hb = 0;
  TRY(tpi_query_arena(&l, 1, window_blocks, window_blocks > 0, &d, &hb));
  if (dev_bytes) *dev_bytes = align_up(d, 256) + tp_tail_bytes(*cfg, n_ranks);
  if (host_bytes) *host_bytes = hb;
  return TPI_OK;
}

extern "C" void tpi_tp_free(tpi_tp_group* g) {
  if (!g) return;
  DeviceGuard guard;
  drop_group_graph(g);
  if (g->ev_graph) cudaEventDestroy(g->ev_graph);
  for (auto& r : g->ranks) {
    cudaSetDevice(r.device);
    if (r.m) tpi_free(r.m);
    if (r.ev_push) cudaEventDestroy(r.ev_push);
    if (r.ev_done) cudaEventDestroy(r.ev_done);
  }
  delete g;
}

extern "C" int tpi_tp_create(const tpi_config* cfg, int n_ranks, const tpi_resources* res, const int* devices, tpi_fill_fn fill,
                             void* user, int window_blocks, tpi_tp_group** out) {
  return tpi_tp_create_p(cfg, n_ranks, nullptr, nullptr, res, devices, fill, user, window_blocks, out);
}
extern "C" int tpi_tp_create_p(const tpi_config* cfg, int n_ranks, const int32_t* kv_heads_per_rank, const int32_t* ffn_cols_per_rank,
                               const tpi_resources* res, const int* devices, tpi_fill_fn fill, void* user, int window_blocks,
                               tpi_tp_group** out) {
  if (!cfg || !res || !fill || !out || window_blocks < 0) return fail(TPI_ERR_INVALID_ARG, "null or negative argument");
  Partition part;
  TRY(make_partition(*cfg, n_ranks, kv_heads_per_rank, ffn_cols_per_rank, &part));
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return fail(TPI_ERR_CUDA, "no CUDA device: this library has no CPU path");
  DeviceGuard guard;
  tpi_tp_group* g = new (std::nothrow) tpi_tp_group();
  if (!g) return fail(TPI_ERR_NOMEM, "out of host memory");
  g->cfg = *cfg;
  g->R = n_ranks;
  g->part = part;
  g->window = window_blocks;
  g->ranks.resize(n_ranks);  // never resized again: the ranks' weight sources are referenced by address
  auto bail = [&](int code) { tpi_tp_free(g); return code; };
  for (int i = 0; i < n_ranks; ++i) {
    TpRank& r = g->ranks[i];
    r.device = devices ? devices[i] : guard.saved;
    if (r.device < 0 || r.device >= ndev) return bail(fail(TPI_ERR_INVALID_ARG, "rank %d: device %d does not exist", i, r.device));
    if (!res[i].compute_stream || !res[i].copy_stream) return bail(fail(TPI_ERR_INVALID_ARG, "rank %d: both streams are required", i));
  }
  for (int i = 0; i < n_ranks; ++i)  // a rank stores into every other rank's receive area
    for (int j = 0; j < n_ranks; ++j)
      if (g->ranks[i].device != g->ranks[j].device) {
        if (cudaSetDevice(g->ranks[i].device) != cudaSuccess) return bail(fail(TPI_ERR_CUDA, "cudaSetDevice(%d) failed", g->ranks[i].device));
        const cudaError_t e = cudaDeviceEnablePeerAccess(g->ranks[j].device, 0);
        if (e != cudaSuccess && e != cudaErrorPeerAccessAlreadyEnabled)
          return bail(fail(TPI_ERR_CUDA, "no peer access from device %d to device %d: %s", g->ranks[i].device, g->ranks[j].device, cudaGetErrorString(e)));
        cudaGetLastError();
      }
  for (int i = 0; i < n_ranks; ++i) {
    TpRank& r = g->ranks[i];
    if (cudaSetDevice(r.device) != cudaSuccess) return bail(fail(TPI_ERR_CUDA, "cudaSetDevice(%d) failed", r.device));
    r.lcfg = local_cfg(*cfg, part, i);
    r.rf.fill = fill; r.rf.user = user; r.rf.cfg = *cfg; r.rf.R = n_ranks; r.rf.rank = i; r.rf.part = part;
    size_t need_d = 0, need_h = 0;
    int rc = tpi_tp_query_arena_p(cfg, n_ranks, i, kv_heads_per_rank, ffn_cols_per_rank, window_blocks, &need_d, &need_h);
    if (rc) return bail(rc);
    if (res[i].dev_bytes < need_d) return bail(fail(TPI_ERR_NOMEM, "rank %d: device arena too small: need %zu bytes, have %zu", i, need_d, res[i].dev_bytes));
    r.tail_bytes = tp_tail_bytes(*cfg, n_ranks);
    tpi_resources lres = res[i];
    lres.dev_bytes = (res[i].dev_bytes - r.tail_bytes) & ~(size_t)255;  // the rank's model takes the front, the exchange the tail
    r.tail = (char*)res[i].dev_arena + lres.dev_bytes;
    rc = tpi_load_model(&r.lcfg, &lres, rank_fill, &r.rf, 1, window_blocks, &r.m);
    if (rc) return bail(rc);
    r.rf.tmp.clear();
    r.rf.tmp.shrink_to_fit();
    r.recv = (float*)r.tail;
    char* t = r.tail + align_up((size_t)2 * tp_half_floats(*cfg, n_ranks) * 4, 256);
    r.flags = (int*)t;
    r.epoch = (int*)(t + 256);
    r.ticket = (unsigned*)(t + 512);
    if (cudaMemsetAsync(r.tail, 0, r.tail_bytes, r.m->cs) != cudaSuccess || cudaStreamSynchronize(r.m->cs) != cudaSuccess)
      return bail(fail(TPI_ERR_CUDA, "rank %d: clearing the exchange area failed", i));
    if (cudaEventCreateWithFlags(&r.ev_push, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&r.ev_done, cudaEventDisableTiming) != cudaSuccess)
      return bail(fail(TPI_ERR_CUDA, "event creation failed"));
  }
  cudaSetDevice(g->ranks[0].device);
  if (cudaEventCreateWithFlags(&g->ev_graph, cudaEventDisableTiming) != cudaSuccess) return bail(fail(TPI_ERR_CUDA, "event creation failed"));
  *out = g;
  return TPI_OK;
}

extern "C" int tpi_tp_prefill(tpi_tp_group* g, const int32_t* tokens, int n_tokens, int32_t* first_token, float* logits_or_null) {
  if (!g || !tokens || n_tokens < 1 || !first_token) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  if (g->batched_prompt) return run_prompt(g, tokens, n_tokens, first_token, logits_or_null);
  return run_positions(g, tokens, n_tokens, n_tokens, false, first_token, 1, logits_or_null);
}
extern "C" int tpi_tp_decode_step(tpi_tp_group* g, int32_t token_in, int32_t* token_out, float* logits_or_null) {
  if (!g || !token_out) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  return run_positions(g, &token_in, 1, 1, true, token_out, 1, logits_or_null);
}
extern "C" int tpi_tp_decode_run(tpi_tp_group* g, int32_t token_in, int n_steps, int32_t* tokens_out) {
  if (!g || !tokens_out || n_steps < 1) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  return run_positions(g, &token_in, 1, n_steps, true, tokens_out, n_steps, nullptr);
}

extern "C" int tpi_tp_reset(tpi_tp_group* g) {
  if (!g) return fail(TPI_ERR_INVALID_ARG, "null group");
  DeviceGuard guard;
  for (auto& r : g->ranks) {  // first everything drains, then every rank's exchange state goes back to zero
    CK(cudaSetDevice(r.device));
    TRY(quiesce(r.m));
  }
  for (auto& r : g->ranks) {
    CK(cudaSetDevice(r.device));
    CK(cudaMemsetAsync(r.tail, 0, r.tail_bytes, r.m->cs));
    CK(cudaMemsetAsync(r.m->dev + r.m->plan.err, 0, 4, r.m->cs));
    CK(cudaMemsetAsync(r.m->dev + r.m->plan.tickets, 0, (size_t)(r.lcfg.n_kv_heads + 1) * 4, r.m->cs));
    if (r.m->sched_open) { r.m->sched_free.push_back(r.m->sched_open); r.m->sched_open = nullptr; }
    if (g->window > 0) TRY(start_window(r.m));
    TRY(write_position(r.m, 0));
  }
  g->position = 0;
  g->exchanges = 0;
  g->broken = false;
  g->drop_rank = -1;
  return TPI_OK;
}

extern "C" int tpi_tp_position(const tpi_tp_group* g) { return g ? g->position : TPI_ERR_INVALID_ARG; }
extern "C" int tpi_tp_n_ranks(const tpi_tp_group* g) { return g ? g->R : TPI_ERR_INVALID_ARG; }

extern "C" int tpi_tp_get_hidden(tpi_tp_group* g, int rank, int layer, int which, float* dst_host) {
  if (!g || rank < 0 || rank >= g->R) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  DeviceGuard guard;
  CK(cudaSetDevice(g->ranks[rank].device));
  return tpi_get_hidden(g->ranks[rank].m, layer, which, dst_host);
}

extern "C" int tpi_tp_get_kv(tpi_tp_group* g, int layer, int kv_head, int pos0, int n, float* k_dst, float* v_dst) {
  if (!g || kv_head < 0 || kv_head >= g->cfg.n_kv_heads) return fail(TPI_ERR_INVALID_ARG, "bad argument");
  int owner = 0;
  while (kv_head >= g->part.kv0[owner + 1]) ++owner;
  DeviceGuard guard;
  CK(cudaSetDevice(g->ranks[owner].device));
  return tpi_get_kv(g->ranks[owner].m, layer, kv_head - g->part.kv0[owner], pos0, n, k_dst, v_dst);
}

extern "C" int tpi_tp_set_option(tpi_tp_group* g, int option, int value) {
  if (!g) return fail(TPI_ERR_INVALID_ARG, "null group");
  switch (option) {
    case TPI_TP_OPT_EVENTS:
      if (!value && share_a_device(g))
        return fail(TPI_ERR_STATE, "ranks that share a device must be ordered by events: a kernel may not wait for a kernel that is not running");
      g->events = value != 0;
      // Without events a consumer really waits for its peers (they run on other GPUs at their own pace: first-launch
      // set-up, a window stall), so the default limit grows from a quarter of a second to about ten seconds.
      if (!g->events && g->wait_polls == (1 << 21)) g->wait_polls = 1 << 26;
      if (g->events && g->wait_polls == (1 << 26)) g->wait_polls = 1 << 21;
      drop_group_graph(g);
      return TPI_OK;
    case TPI_TP_OPT_GRAPH:
      g->use_graph = value != 0;
      drop_group_graph(g);
      return TPI_OK;
    case TPI_TP_OPT_WAIT_POLLS:
      if (value < 1) return fail(TPI_ERR_INVALID_ARG, "the poll limit must be positive");
      g->wait_polls = value;
      drop_group_graph(g);  // the limit is a kernel argument
      return TPI_OK;
    case TPI_TP_OPT_DROP_PUSH:
      if (value < 0 || value > g->R) return fail(TPI_ERR_INVALID_ARG, "rank + 1 expected");
      g->drop_rank = value - 1;
      return TPI_OK;
    case TPI_TP_OPT_PDL: g->pdl = value != 0; drop_group_graph(g); return TPI_OK;
    case TPI_TP_OPT_BATCHED_PROMPT: g->batched_prompt = value != 0; return TPI_OK;
    default: return fail(TPI_ERR_INVALID_ARG, "unknown option %d", option);
  }
}

extern "C" int tpi_tp_get_stats(tpi_tp_group* g, tpi_tp_stats* out) {
  if (!g || !out) return fail(TPI_ERR_INVALID_ARG, "null argument");
  tpi_tp_stats s{};
  const tpi_config& c = g->cfg;
  s.n_ranks = g->R;
  s.position = g->position;
  s.events = g->events;
  s.kernel_launches_last = g->launches_last;
  s.exchanges_total = g->exchanges;
  s.exchange_bytes_per_token = (uint64_t)2 * c.n_layers * c.hidden * 4 * (g->R - 1);  // a worker; the master adds one broadcast
  const uint64_t B = elem_size(c.dtype);
  auto layers_of = [&](const tpi_config& l) {  // the bytes of its slices that a rank streams per decoded token
    return (((uint64_t)(l.n_heads + 2 * l.n_kv_heads) * l.head_dim * l.hidden + (uint64_t)l.hidden * l.n_heads * l.head_dim +
             3ull * l.hidden * l.ffn) * B + 2ull * l.hidden * 4) * l.n_layers;
  };
  s.weight_bytes_worker = layers_of(g->ranks[g->R > 1 ? 1 : 0].lcfg);  // rank 1's share (every worker's, when p_i is uniform)
  s.weight_bytes_rank0 = layers_of(g->ranks[0].lcfg) + (uint64_t)c.vocab * c.hidden * B + (uint64_t)c.hidden * 4;
  s.last_decode_ms = g->last_decode_ms;
  *out = s;
  return TPI_OK;
}
