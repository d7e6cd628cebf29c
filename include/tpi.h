/* tpi.h - C ABI of the B200 implementation of the TPI-LLM decoder hot path.
 *
 * The library runs the batch-1 Llama-style decoder step under the paper's
 * tensor-parallel partition (Sec. 3.1, Steps 1-4, Eq. 1-2, Algorithms 1-2) on
 * ONE GPU: all N shards ("devices" in the paper) are emulated side by side,
 * each row-sharded projection produces one partial sum per shard, and the star
 * allreduce (Sec. 3.2, Prop. 2) becomes an on-device sum of the N partials in
 * ascending rank order followed by the shortcut add.  Layer weights that do
 * not fit in device memory are fed by the sliding-window memory scheduler of
 * Sec. 3.3 / Appendix A.2, rebuilt as a pinned-host -> device copy ring.
 *
 * General rules
 *  - Plain C types only.  Every pointer says whether it is HOST or DEVICE memory.
 *  - The library allocates no device memory and no pinned memory: the caller
 *    hands in two arenas (tpi_resources) that must outlive the model.
 *  - Every call returns 0 (TPI_OK) or a negative tpi_status.  Nothing aborts.
 *  - A model is used by one host thread at a time.
 *  - Weights are [out][in] row-major, no biases (Table 5's counts have none).
 *  - Debug aid: with TPI_DEBUG=1 in the environment when tpi_query_arena and
 *    tpi_load_model are called, every buffer carved from the device arena is
 *    followed by a 256-byte guard zone holding a known pattern, and a small
 *    kernel compares all zones at the end of every tpi_prefill / tpi_decode_*
 *    call: a kernel that wrote past its buffer makes the call return
 *    TPI_ERR_DEVICE_CHECK, and tpi_last_error() names the zone.
 */
#ifndef TPI_H
#define TPI_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tpi_model tpi_model; /* opaque */

typedef enum {
  TPI_OK = 0,
  TPI_ERR_INVALID_ARG = -1,  /* null pointer, negative size, unknown enum            */
  TPI_ERR_SHAPE = -2,        /* N must divide heads, kv heads and FFN width; d even.. */
  TPI_ERR_NOMEM = -3,        /* an arena is too small (tpi_last_error() says by how much) */
  TPI_ERR_SEQ_OVERFLOW = -4, /* position would reach max_seq                          */
  TPI_ERR_TOKEN_RANGE = -5,  /* token id outside [0, vocab)                           */
  TPI_ERR_CUDA = -6,         /* a CUDA runtime call failed (message in tpi_last_error)*/
  TPI_ERR_TIMEOUT = -7,      /* a bounded wait ran out                                */
  TPI_ERR_DEVICE_CHECK = -8, /* a kernel's self-check wrote the device error word     */
  TPI_ERR_STATE = -9,        /* call not valid in this state (e.g. no host images)    */
  TPI_ERR_CALLBACK = -10     /* the weight callback returned non-zero                 */
} tpi_status;

typedef enum { TPI_F32 = 0, TPI_BF16 = 1 } tpi_dtype;

/* Model shape, in the paper's notation (Appendix A.5): L layers, hidden h,
 * a heads, b kv heads, head dim d, intermediate size s, vocabulary v. */
typedef struct {
  int32_t n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab;
  int32_t max_seq;       /* KV-cache capacity in positions                         */
  int32_t max_prefill;   /* largest number of prompt positions processed at once
                            (longer prompts are fed in chunks of this size)        */
  float rms_eps, rope_base;
  int32_t dtype;         /* tpi_dtype: storage type of weights AND of the KV cache */
} tpi_config;

/* Caller-owned memory and streams.  dev_arena: DEVICE memory, 256-byte aligned.
 * host_arena: PINNED HOST memory, 256-byte aligned.  Streams are cudaStream_t
 * handles; compute_stream may be NULL (legacy default stream is NOT used: the
 * library then creates its own non-blocking streams). */
typedef struct {
  void *dev_arena;
  size_t dev_bytes;
  void *host_arena;
  size_t host_bytes;
  void *compute_stream;
  void *copy_stream;
} tpi_resources;

/* Tensor ids handed to the weight callback. */
enum {
  TPI_T_EMB = 0, TPI_T_HEAD = 1, TPI_T_FINAL_NORM = 2,
  TPI_T_ATTN_NORM = 3, TPI_T_WQ = 4, TPI_T_WK = 5, TPI_T_WV = 6, TPI_T_WO = 7,
  TPI_T_FFN_NORM = 8, TPI_T_WGATE = 9, TPI_T_WUP = 10, TPI_T_WDOWN = 11
};

/* Weight source (Sec. 3.1 Step 1: the master partitions the pretrained weights
 * and hands each device its slices).  The library asks for rows
 * [row0, row0 + n_rows) of the UNSHARDED tensor `tensor_id` of `layer`
 * (layer is 0 for EMB / HEAD / FINAL_NORM; a norm gain is one row of h
 * elements) and the callback writes them, row-major, in cfg.dtype, to the HOST
 * buffer dst (n_rows * row_len * element size bytes).  Return 0 on success. */
typedef int (*tpi_fill_fn)(void *user, int tensor_id, int layer, int64_t row0, int64_t n_rows,
                           void *dst);

/* Arena sizes needed for a configuration.  window_blocks = 0: every layer block
 * resident in device memory; >= 1: streamed through a window of that many
 * blocks.  keep_host_images != 0 additionally keeps every packed block image
 * in the host arena (required for window_blocks >= 1, and for switching a
 * resident model to streaming later).  n_shards_max bounds later tpi_set_shards.
 * Pure host arithmetic; needs no GPU. */
int tpi_query_arena(const tpi_config *cfg, int n_shards_max, int window_blocks,
                    int keep_host_images, size_t *dev_bytes, size_t *host_bytes);

/* Sizes of the paper's blocks (Table 5) as this library packs them for one
 * shard fraction 1/n_shards ... and for the whole layer: bytes of one attention
 * block image and one FFN block image (all N shards together, gains included). */
int tpi_block_bytes(const tpi_config *cfg, size_t *attn_block_bytes, size_t *ffn_block_bytes);

/* Step 1 (Algorithm 1, line 1 / Algorithm 2, line 1): build the shard-major
 * block images from the callback, place them (device, or host + window), and
 * set up the step driver.  `fill` and `user` are kept and called again by
 * tpi_set_shards, so they must stay valid for the model's lifetime.
 * On success *out owns nothing but bookkeeping; free it with tpi_free. */
int tpi_load_model(const tpi_config *cfg, const tpi_resources *res, tpi_fill_fn fill, void *user,
                   int n_shards, int window_blocks, tpi_model **out);

/* Re-partition for N devices (Sec. 3.1 Step 1).  Repacks the images through
 * the callback, clears the KV cache and the position. */
int tpi_set_shards(tpi_model *m, int n_shards);

/* Window size w of the memory scheduler IN BLOCKS (one attention block or one
 * FFN block, Sec. 3.3; the executing block counts, Prop. 5).  0 = all resident.
 * w = 1 loads then computes with no overlap.  Keeps the KV cache and position.
 * Needs host images unless going 0 -> 0. */
int tpi_set_window(tpi_model *m, int window_blocks);

/* Heterogeneous partition (Sec. 3.1: device i takes the proportion p_i of the attention heads and of the
 * FFN columns, stronger devices more): shard i owns kv_heads_per_shard[i] kv heads together with their
 * query-head groups and ffn_cols_per_shard[i] FFN columns, in rank order.  Both lists have n_shards
 * entries (1 <= n_shards <= 16), every entry >= 1, sums equal to n_kv_heads and ffn, and a shard's
 * heads*head_dim and FFN columns must be multiples of 16 bytes of weights (TPI_ERR_SHAPE otherwise).
 * Re-packs the layer blocks like tpi_set_shards (which returns to the uniform p_i = 1/N) and resets the
 * position.  The partition decides which inputs each per-shard partial sum of the O and down
 * projections covers; the column-sharded projections give the same values whoever computes them. */
int tpi_set_partition(tpi_model *m, int n_shards, const int32_t *kv_heads_per_shard,
                      const int32_t *ffn_cols_per_shard);

/* Block retention (Sec. 3.3, Prop. 6 / Appendix A.6): when the link is the bottleneck, keep ONE FFN
 * block in every `ffn_every_T` FFN blocks resident (layers 0, T, 2T, ...) beside the window and stream
 * only the rest; 0 turns retention off, 1 keeps every FFN block, -1 picks the smallest T whose kept
 * blocks fit in the device arena beside the window (0 if none fits).  Only for a streamed model
 * (window >= 1).  The retained blocks live in the device arena after the window slots: the arena must
 * have room for them (TPI_ERR_NOMEM otherwise, and the previous setting stays in force).  Keeps the KV
 * cache and the position; results are bit-identical with and without retention.  tpi_set_window turns
 * retention off again (it is chosen per window size). */
int tpi_set_retention(tpi_model *m, int ffn_every_T);

/* One pass of Algorithm 1's loop body over n_tokens prompt positions starting
 * at the current position (usually 0): fills the KV cache and returns the
 * greedy next token.  tokens: HOST int32[n_tokens].  first_token: HOST int32*.
 * logits_or_null: HOST float[vocab] (last position's logits) or NULL.
 * Synchronous: returns when the token has arrived on the host. */
int tpi_prefill(tpi_model *m, const int32_t *tokens, int n_tokens, int32_t *first_token,
                float *logits_or_null);

/* One pass of the loop body for ONE position: feed token_in at the current
 * position, append its K/V, return the greedy next token (ties -> lowest id).
 * token_out: HOST int32*; logits_or_null: HOST float[vocab] or NULL. */
int tpi_decode_step(tpi_model *m, int32_t token_in, int32_t *token_out, float *logits_or_null);

/* Enqueue `n_steps` decode steps back to back, each feeding the previous
 * step's output token (the first feeds token_in), with ONE host wait at the
 * end.  tokens_out: HOST int32[n_steps].  Same arithmetic as tpi_decode_step. */
int tpi_decode_run(tpi_model *m, int32_t token_in, int n_steps, int32_t *tokens_out);

int tpi_reset(tpi_model *m);           /* position = 0 (cache contents become dead) */
int tpi_position(const tpi_model *m);  /* number of cached positions                */

/* Debug taps of the LAST processed position: which = 0 -> H_attn (Eq. 1),
 * 1 -> H_ffn (Eq. 2) of `layer`.  dst_host: HOST float[hidden]. */
int tpi_get_hidden(tpi_model *m, int layer, int which, float *dst_host);

/* Read cached keys/values of one kv head: positions [pos0, pos0+n) as float
 * (exact upcast of the stored type).  k_dst, v_dst: HOST float[n * head_dim]. */
int tpi_get_kv(tpi_model *m, int layer, int kv_head, int pos0, int n, float *k_dst, float *v_dst);

/* Overwrite cached keys/values (tests: synthetic caches of a given length).
 * k_src, v_src: HOST float[n * head_dim], rounded to the storage type.
 * tpi_set_position then declares how many positions are valid. */
int tpi_put_kv(tpi_model *m, int layer, int kv_head, int pos0, int n, const float *k_src,
               const float *v_src);
int tpi_set_position(tpi_model *m, int position);

typedef struct {
  double last_prefill_ms;      /* host wall time of the last tpi_prefill (TTFT)          */
  double last_decode_ms;       /* host wall time of the last tpi_decode_step / _run      */
  double last_decode_dev_ms;   /* the same region timed with CUDA events                 */
  uint64_t weight_bytes_per_token; /* layer blocks + head, algorithmic                   */
  uint64_t link_bytes_total;   /* bytes copied host -> device by the window so far       */
  uint64_t blocks_loaded;      /* window loads issued so far                             */
  double stall_ms_total;       /* compute-stream time spent waiting for loads (profile)  */
  double dominant_kernel_ms;   /* mean duration of the gate/up GEMV launch (profile)     */
  uint64_t dominant_kernel_bytes; /* algorithmic bytes of one such launch                */
  uint32_t dominant_kernel_samples;
  int32_t kernel_launches_last; /* kernels launched by the last prefill/decode call      */
  int32_t window_blocks, n_shards, position, graph_active;
  uint64_t window_peak_bytes;  /* device bytes held by window slots                      */
  uint64_t retained_bytes;     /* device bytes held by retained blocks (block retention) */
  int32_t retained_blocks, reserved_;
  double last_prefill_dev_ms;     /* the last tpi_prefill's kernels timed with CUDA events             */
  double last_prefill_enqueue_ms; /* host time that call spent enqueueing them (before it waited)      */
} tpi_stats;
int tpi_get_stats(tpi_model *m, tpi_stats *out);

/* The paper's scheduler diagnostics (Sec. 3.3): the latencies that Prop. 3-6 are stated in, measured
 * on this run, and the propositions evaluated on them.  Samples are taken by decode calls while
 * TPI_OPT_PROFILE is 1 (CUDA events around every block's kernels on the compute stream and around
 * every block copy on the copy stream; means over all samples since load or tpi_scheduler_reset).
 * The emulated allreduce (the rank-ordered sum) runs inside each block's last kernel, so it is part
 * of t_attn / t_ffn and t_all_reduce is reported as 0; every proposition only uses the sums
 * t + t_all_reduce, so the verdicts are unaffected.  tight_holds / loose_holds: Prop. 4 / Prop. 3
 * (1 or 0); retention_T: 0 if Prop. 3 holds without retention, else the largest T for which Prop. 6
 * holds, -1 if none does; all three are -2 while a needed sample is missing (e.g. a resident model
 * has no loads).  m_worker_bytes: Prop. 5's M_worker for the current window without the empirical
 * factor; window_device_bytes: what the window slots plus retained blocks occupy. */
typedef struct {
  double t_attn_ms, t_ffn_ms, t_all_reduce_ms, tau_attn_ms, tau_ffn_ms, stall_ms_total;
  uint32_t n_t_attn, n_t_ffn, n_tau_attn, n_tau_ffn;
  int32_t tight_holds, loose_holds, retention_T, window_blocks, retain_every_T, reserved_;
  uint64_t m_worker_bytes, window_device_bytes;
} tpi_sched_report;
int tpi_scheduler_report(tpi_model *m, tpi_sched_report *out);
int tpi_scheduler_reset(tpi_model *m);

/* Prop. 3 (loose), Prop. 4 (tight) and Prop. 6 (retention) on given latencies; host arithmetic only,
 * any consistent time unit.  Outputs may be null.  *retention_T as in tpi_sched_report. */
int tpi_steady_conditions(double t_attn, double t_ffn, double t_all_reduce, double tau_attn, double tau_ffn,
                          int n_layers, int *tight, int *loose, int *retention_T);

/* Options: TPI_OPT_GRAPH (1 = replay the decode step as a CUDA graph when all
 * blocks are resident; default 1), TPI_OPT_PDL (1 = programmatic dependent
 * launch between kernels; default 1), TPI_OPT_PROFILE (1 = CUDA events around
 * each gate/up GEMV launch and each window wait; default 0), TPI_OPT_TENSOR (1 =
 * bf16 models run the prompt pass's projections on the tensor cores with each
 * fp32 activation split into two bf16 values, hi + lo, so ~16 mantissa bits
 * survive; 2 = a single bf16 per activation: twice the tensor throughput, but
 * the rounding alone costs ~1e-2 relative error on the logits after two
 * layers of the synthetic workloads; 0 = fp32 SIMT GEMM everywhere; default 1),
 * TPI_OPT_WAIT_DEADLINE_MS (value > 0: how long tpi_prefill / tpi_decode_* wait for the device
 * before they give up with TPI_ERR_TIMEOUT; default 900000, or TPI_WAIT_DEADLINE_S seconds from the
 * environment.  After a timeout the enqueued work still runs to its end on the device; the host
 * position is unchanged, and tpi_reset / tpi_set_position drain the stream and re-synchronise),
 * TPI_OPT_ROWSHARD_FUSED (default 1: a decode step's row-sharded projections keep the N partial sums
 * in registers and add them in rank order in the same kernel; 0: the partial sums go through memory
 * and a second kernel adds them - the same residual bits, the form whose norm statistics a group of
 * real ranks (tpi_tp.h) reproduces bit for bit). */
enum { TPI_OPT_GRAPH = 0, TPI_OPT_PDL = 1, TPI_OPT_PROFILE = 2, TPI_OPT_TENSOR = 3, TPI_OPT_WAIT_DEADLINE_MS = 4,
       TPI_OPT_ROWSHARD_FUSED = 5 };
int tpi_set_option(tpi_model *m, int option, int value);

/* Host-only test hook (needs no GPU): drives the window scheduler's ordering
 * logic (Sec. 3.3: loads in execution order, at most w blocks held, a slot is
 * reloaded only after its block was released) against a recording back end.
 * Executes n_exec blocks in cyclic order over n_blocks (even) with window w and
 * writes up to max_ops triples (op, slot, block) to ops (HOST int[3*max_ops]):
 * op 0 = copy queue waits for the release of `slot`, 1 = copy `block` into
 * `slot`, 2 = copy queue marks `slot` loaded, 3 = compute queue waits for
 * `slot`, 4 = compute queue releases `slot`.  Returns the number of operations
 * (which may exceed max_ops) or a negative tpi_status. */
int tpi_ring_trace(int n_blocks, int w, int n_exec, int *ops, int max_ops);
/* The same with block retention: the FFN block of layers 0, T, 2T, ... is retained; executing a
 * retained block is recorded as op 5 (slot -1) and touches neither queue. */
int tpi_ring_trace_retained(int n_blocks, int w, int n_exec, int ffn_every_T, int *ops, int max_ops);

/* Host-only test hook for the failure path of the window scheduler (needs no GPU): as
 * tpi_ring_trace_retained, but the back end's block copy number `fail_copy` (0-based, counted over the
 * whole run, the start-up loads included) fails once with `fail_status` (a negative tpi_status), the
 * way a cudaMemcpyAsync that returns an error would.  retry == 0: the run stops where a decoder step
 * would stop and the call returns fail_status (the failure propagates unchanged).  retry != 0: the
 * failure is recorded as op 6 (slot = fail_status, block = the block being executed, -1 during
 * start-up) and the interrupted operation is issued again; the ring must carry on as if nothing had
 * happened: no block skipped or loaded twice into a live slot, loads still in execution order. */
int tpi_ring_trace_faulty(int n_blocks, int w, int n_exec, int ffn_every_T, int fail_copy, int fail_status,
                          int retry, int *ops, int max_ops);

void tpi_free(tpi_model *m);
const char *tpi_strerror(int code);
const char *tpi_last_error(void); /* thread-local detail of the last failure */

#ifdef __cplusplus
}
#endif
#endif /* TPI_H */
