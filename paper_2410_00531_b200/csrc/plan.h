// Memory plan: where every buffer of a model lives inside the caller's arenas,
// and how a layer's two weight blocks are packed.  Pure host arithmetic.
#pragma once
#include <stddef.h>
#include <stdint.h>

#include "../../include/tpi.h"

namespace tpi {

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline size_t elem_size(int dtype) { return dtype == TPI_BF16 ? 2 : 4; }

// Layout of the two block images of one layer (byte offsets inside the image).
// Attention block (Table 5: 2(a+b)h^2 p/a + h parameters per device, all N devices side by side):
//   gain fp32[h] | shard 0..N-1: [W_Q^i ; W_K^i ; W_V^i] rows x h | shard 0..N-1: W_O^i [h][a d / N]
// FFN block (3 h s p + h per device):
//   gain fp32[h] | shard 0..N-1: gate/up rows interleaved [2 s / N][h] | shard 0..N-1: W_down^i [h][s / N]
struct BlockLayout {
  size_t attn_bytes, ffn_bytes;
  size_t off_qkv, off_wo, off_gu, off_down;
};

static inline BlockLayout block_layout(const tpi_config& c) {
  BlockLayout b{};
  const size_t B = elem_size(c.dtype), h = c.hidden, d = c.head_dim;
  const size_t gain = align_up(h * 4, 256);
  b.off_qkv = gain;
  b.off_wo = align_up(b.off_qkv + (size_t)(c.n_heads + 2 * c.n_kv_heads) * d * h * B, 256);
  b.attn_bytes = align_up(b.off_wo + h * (size_t)c.n_heads * d * B, 256);
  b.off_gu = gain;
  b.off_down = align_up(b.off_gu + 2 * (size_t)c.ffn * h * B, 256);
  b.ffn_bytes = align_up(b.off_down + h * (size_t)c.ffn * B, 256);
  return b;
}

constexpr int kMaxCanaries = 64;
constexpr size_t kCanaryBytes = 256;

struct Plan {
  BlockLayout bl;
  int nsplit, head_blocks, n_shards_max;
  // device arena offsets
  size_t emb, head, final_gain, rope, inv_freq, kcache, vcache, kv_layer_bytes;
  size_t x, xhat, ss_part, q, o, act, partials, logits, attn_scratch, amax_val, amax_idx, tickets, tok_hist, pos, err,
      taps;
  size_t pX, pXn, pQKV, pQ, pO, pGU, pACT, pPART;
  size_t blocks;      // start of the weight-block region (resident images or window slots)
  size_t dev_fixed;   // bytes before the block region
  // host arena offsets
  size_t h_io, h_logits, h_stage, h_stage_bytes, h_bounce, h_images, host_fixed;
  // debug build of the arena (TPI_DEBUG=1): a guard zone of kCanaryBytes follows every carved device buffer; the
  // zones hold a known pattern that a check kernel compares after every step (an overrun of buffer i lands in zone i)
  int n_canaries;
  size_t canary_off[kMaxCanaries];
};

static inline int attn_nsplit(const tpi_config& c) {
  // one split per 128 cached positions (what a CTA stages in shared memory in one go), at most 128 splits
  int n = (c.max_seq + 127) / 128;
  if (n > 128) n = 128;
  return n < 1 ? 1 : n;
}

static inline int window_slots(int w, int* nA, int* nF) {
  if (w <= 1) { *nA = 0; *nF = 1; }
  else { *nA = w / 2; *nF = (w + 1) / 2; }
  return *nA + *nF;
}

// Upper bound of the entries the kernels use for the per-CTA partial sums of squares (4 per SM, up to 256 SMs).
constexpr size_t kMaxNormParts = 1024;

// Fills `p`; returns the bytes needed in each arena for the given residency mode.
static inline void make_plan(const tpi_config& c, int n_shards_max, int window_blocks, int keep_host,
                             int head_blocks, Plan* p, size_t* dev_bytes, size_t* host_bytes, bool canaries = false) {
  const size_t B = elem_size(c.dtype), h = c.hidden, d = c.head_dim, a = c.n_heads, b = c.n_kv_heads,
               s = c.ffn, v = c.vocab, L = c.n_layers, S = c.max_seq, T = c.max_prefill;
  p->bl = block_layout(c);
  p->nsplit = attn_nsplit(c);
  p->head_blocks = head_blocks;
  p->n_shards_max = n_shards_max;
  size_t o = 0;
  p->n_canaries = 0;
  auto take = [&](size_t bytes) {
    size_t r = o;
    o = align_up(o + bytes, 256);
    if (canaries && p->n_canaries < kMaxCanaries) { p->canary_off[p->n_canaries++] = o; o += kCanaryBytes; }
    return r;
  };
  p->emb = take(v * h * B);
  p->head = take(v * h * B);
  p->final_gain = take(h * 4);
  p->rope = take(S * (d / 2) * 8);
  p->inv_freq = take((d / 2) * 8);
  p->kv_layer_bytes = align_up(b * S * d * B, 256);
  p->kcache = take(L * p->kv_layer_bytes);
  p->vcache = take(L * p->kv_layer_bytes);
  p->x = take(h * 4);
  p->xhat = take(h * 4);
  p->ss_part = take((h > kMaxNormParts ? h : kMaxNormParts) * 4);  // per-CTA partial sums of x^2: up to kMaxNormParts entries
  p->q = take(a * d * 4);
  p->o = take(a * d * 4);
  p->act = take(s * 4);
  p->partials = take((size_t)n_shards_max * h * 4);
  p->logits = take(v * 4);
  p->attn_scratch = take(b * p->nsplit * (a / b) * (d + 2) * 4);
  p->amax_val = take((size_t)head_blocks * 4);
  p->amax_idx = take((size_t)head_blocks * 4);
  p->tickets = take((b + 1) * 4);
  p->tok_hist = take((S + 2) * 4);
  p->pos = take(4);
  p->err = take(4);
  p->taps = take(L * 2 * h * 4);
  p->pX = take(T * h * 4);
  p->pXn = take(T * h * 4);
  p->pQKV = take(T * (a + 2 * b) * d * 4);
  p->pQ = take(T * a * d * 4);
  p->pO = take(T * a * d * 4);
  p->pGU = take(T * 2 * s * 4);
  p->pACT = take(T * s * 4);
  p->pPART = take((size_t)n_shards_max * T * h * 4);
  p->dev_fixed = o;
  p->blocks = o;
  size_t blocks_bytes;
  if (window_blocks <= 0) blocks_bytes = L * (p->bl.attn_bytes + p->bl.ffn_bytes);
  else {
    int nA, nF;
    window_slots(window_blocks, &nA, &nF);
    blocks_bytes = nA * p->bl.attn_bytes + nF * p->bl.ffn_bytes;
  }
  if (dev_bytes) *dev_bytes = o + blocks_bytes;

  size_t ho = 0;
  auto htake = [&](size_t bytes) { size_t r = ho; ho = align_up(ho + bytes, 256); return r; };
  p->h_io = htake((S + 2 + T) * 4 + 256);
  p->h_logits = htake(v * 4);
  p->h_stage_bytes = (size_t)64 << 20;
  {  // at least one row of the widest tensor
    size_t widest = (s > a * d ? s : a * d);
    if (h > widest) widest = h;
    if (widest * B > p->h_stage_bytes) p->h_stage_bytes = align_up(widest * B, 256);
  }
  p->h_stage = htake(p->h_stage_bytes);
  p->host_fixed = ho;
  if (keep_host || window_blocks > 0) {
    p->h_bounce = 0;
    p->h_images = htake(L * (p->bl.attn_bytes + p->bl.ffn_bytes));
  } else {
    p->h_images = 0;
    p->h_bounce = htake(p->bl.ffn_bytes > p->bl.attn_bytes ? p->bl.ffn_bytes : p->bl.attn_bytes);
  }
  if (host_bytes) *host_bytes = ho;
}

}  // namespace tpi
