// The sliding-window block ring on CUDA streams (copy stream + loaded / released events), block retention, the
// scheduler's diagnostics (per-block latencies, Prop. 3-6) and the host-only ordering trace.
#include "model.h"

// ------------------------------------------------------------------------------ scheduler diagnostics
cudaEvent_t sched_event(tpi_model* m) {
  if (!m->sched_free.empty()) { cudaEvent_t e = m->sched_free.back(); m->sched_free.pop_back(); return e; }
  if (m->sched_pending.size() >= 8192) return nullptr;  // bounded: further samples are dropped until a harvest
  cudaEvent_t e = nullptr;
  return cudaEventCreate(&e) == cudaSuccess ? e : nullptr;
}
// completed pairs go into the running means; pairs still in flight (the loader runs ahead) stay for the next call
void sched_harvest(tpi_model* m) {
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

int start_window(tpi_model* m) {
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

// ------------------------------------------------------------------------------ block access during a step
int acquire_block(tpi_model* m, int block, BlockRef* r) {
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
int release_block(tpi_model* m, int block) {
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
int tr_crl(void* c, int s) { return tr_push(c, 2, s, -1); }
int tr_xwl(void* c, int s) { return tr_push(c, 3, s, -1); }
int tr_xrr(void* c, int s) { return tr_push(c, 4, s, -1); }
}  // namespace

// Runs the window ring's ordering logic against a recording back end (no GPU needed): executes
// `n_exec` blocks in cyclic order over `n_blocks` with window `w`.  ops receives up to max_ops
// triples (op, slot, block): op 0 copy-queue waits for release of slot, 1 copy block into slot,
// 2 copy-queue marks slot loaded, 3 compute-queue waits for slot, 4 compute-queue releases slot.
// Returns the number of operations (may exceed max_ops) or a negative status.
extern "C" int tpi_ring_trace(int n_blocks, int w, int n_exec, int* ops, int max_ops) {
  return tpi_ring_trace_retained(n_blocks, w, n_exec, 0, ops, max_ops);
}

extern "C" int tpi_ring_trace_retained(int n_blocks, int w, int n_exec, int ffn_every_T, int* ops, int max_ops) {
  return tpi_ring_trace_faulty(n_blocks, w, n_exec, ffn_every_T, -1, 0, 0, ops, max_ops);
}

namespace {
struct FaultyCtx {
  TraceCtx t;
  int copies, fail_copy, fail_status;
};
int ft_cb(void* c, int s, int b) {
  FaultyCtx* f = (FaultyCtx*)c;
  if (f->copies++ == f->fail_copy) return f->fail_status;  // the copy was not issued: nothing is recorded
  return tr_push(&f->t, 1, s, b);
}
}  // namespace

extern "C" int tpi_ring_trace_faulty(int n_blocks, int w, int n_exec, int ffn_every_T, int fail_copy, int fail_status,
                                     int retry, int* ops, int max_ops) {
  if (fail_copy >= 0 && fail_status >= 0) return fail(TPI_ERR_INVALID_ARG, "fail_status must be a negative status");
  if (n_blocks < 2 || n_blocks % 2 || w < 1 || n_exec < 0 || ffn_every_T < 0 || (!ops && max_ops > 0))
    return fail(TPI_ERR_INVALID_ARG, "bad argument");
  std::vector<char> keep(n_blocks, 0);
  if (ffn_every_T > 0)
    for (int l = 0; l < n_blocks / 2; l += ffn_every_T) keep[2 * l + 1] = 1;
  FaultyCtx f{{ops, max_ops, 0}, 0, fail_copy, fail_status};
  TraceCtx& t = f.t;
  RingBackend be;
  be.ctx = &f;  // TraceCtx is FaultyCtx's first member: the recording callbacks take the same pointer
  be.copy_wait_released = tr_cwr;
  be.copy_block = ft_cb;
  be.copy_record_loaded = tr_crl;
  be.compute_wait_loaded = tr_xwl;
  be.compute_record_released = tr_xrr;
  Ring r;
  r.configure(n_blocks, w, be, keep.data());
  // a failure surfaces from the call that pumped the loader; with `retry` that call's pending part is issued again
  auto failed = [&](int rc, int blk) -> bool {  // true: give up with rc
    if (rc != fail_status || !retry) return true;
    tr_push(&t, 6, fail_status, blk);
    return false;
  };
  int rc = r.pump();
  if (rc) {
    if (failed(rc, -1)) return rc < 0 ? rc : TPI_ERR_STATE;
    if ((rc = r.pump())) return rc < 0 ? rc : TPI_ERR_STATE;
  }
  for (int i = 0; i < n_exec; ++i) {
    const int blk = i % n_blocks;
    if (keep[blk]) { tr_push(&t, 5, -1, blk); continue; }  // a retained block runs without any window operation
    int s = r.acquire(blk);
    if (s < 0) {
      if (failed(s, blk)) return s == -1000 || s == -1001 ? TPI_ERR_STATE : s;
      if ((s = r.acquire(blk)) < 0) return s == -1000 || s == -1001 ? TPI_ERR_STATE : s;
    }
    rc = r.release(blk);
    if (rc) {  // the block itself was released before the loader was pumped: only the pump is repeated
      if (failed(rc, blk)) return rc == -1000 ? TPI_ERR_STATE : rc;
      if ((rc = r.pump())) return rc < 0 ? rc : TPI_ERR_STATE;
    }
  }
  return t.n;
}

