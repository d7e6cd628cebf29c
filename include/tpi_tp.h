/* tpi_tp.h - the decoder step on R real devices ("ranks"), one shard each.
 *
 * tpi.h emulates the paper's N devices side by side on one GPU.  This header is
 * the form in which every device of Sec. 3.1 is a rank of its own (Algorithm 1:
 * rank 0, the master; Algorithm 2: the workers):
 *
 *  - rank i holds ONLY its slices of the weights (Sec. 3.1 Step 1: its share of
 *    the attention heads with their W_Q, W_K, W_V rows and W_O columns, its
 *    share of the FFN columns of W_gate / W_up and rows-of-columns of W_down)
 *    and the KV cache of its own heads (Eq. 1: "cached locally");
 *  - W_emb, W_head and the final norm live on the master only, and only the
 *    master ever sees token ids (the placement of Sec. 3.1; workers receive
 *    the embedded hidden state, Algorithm 2 line "receive H^0");
 *  - every row-sharded projection (O, down) ends in the star allreduce of
 *    Sec. 3.2 in its one-hop form: each rank STORES its h fp32 partial sums
 *    into every rank's receive buffer (plain stores into the consumer's own
 *    memory, then one flag per source), and every rank adds the R partial sums
 *    in ascending rank order and the shortcut last (Eq. 1-2), so all ranks hold
 *    the same bits.  No rank ever loads from another rank's memory, every store
 *    names a single destination, and every wait for a flag is bounded: when it runs
 *    out the kernel returns, the device error word reads "wait timeout", and
 *    the call returns TPI_ERR_TIMEOUT.
 *
 * A group lives in ONE host process and drives all ranks; each rank has its own
 * device arena, pinned host arena and streams (tpi_resources), on the device
 * given for it.  Ranks may share a device (this is how the path is tested on a
 * single GPU): the exchange is then ordered by CUDA events between the ranks'
 * streams, so that a flag is always set before the kernel that waits for it
 * starts, and the bounded device-side wait is only a backstop.  With one device
 * per rank the events can be switched off (TPI_TP_OPT_EVENTS = 0) and the flags
 * alone order the exchange.
 *
 * The arithmetic is that of tpi.h's two-kernel form of the row-sharded
 * projections (partial sums through memory, then the rank-ordered sum), so a
 * group of R ranks gives the same bits as an emulated model with N = R shards
 * run with TPI_OPT_ROWSHARD_FUSED = 0.
 *
 * A prompt is processed in chunks of up to cfg.max_prefill positions per pass
 * over the weights, with the kernels of tpi.h's prompt pass on every rank's
 * slices; the partial sums of a chunk (positions x hidden, fp32) travel the same
 * way.  TPI_TP_OPT_BATCHED_PROMPT = 0 feeds the prompt one position at a time
 * through the decode kernels instead.
 */
#ifndef TPI_TP_H
#define TPI_TP_H

#include "tpi.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tpi_tp_group tpi_tp_group; /* opaque */

#define TPI_TP_MAX_RANKS 16

/* Sec. 3.1 Step 1 as a table: which part of the UNSHARDED tensor `tensor_id`
 * (ids of tpi.h) rank `rank` of `n_ranks` holds under the uniform partition
 * p_i = 1/R: rows [row0, row0 + n_rows) x columns [col0, col0 + n_cols).
 * Norm gains are held whole by every rank; EMB / HEAD / FINAL_NORM by rank 0
 * only (n_rows = 0 elsewhere).  Pure host arithmetic; needs no GPU.
 * TPI_ERR_SHAPE when n_ranks does not divide heads, kv heads and FFN width. */
int tpi_tp_rank_slice(const tpi_config *cfg, int n_ranks, int rank, int tensor_id, int64_t *row0, int64_t *n_rows,
                      int64_t *col0, int64_t *n_cols);

/* The same for a heterogeneous partition (Sec. 3.1: device i takes the
 * proportion p_i of the heads and FFN columns, stronger devices more): rank i
 * owns kv_heads_per_rank[i] kv heads with their query-head groups and
 * ffn_cols_per_rank[i] FFN columns, in rank order; both lists have n_ranks
 * entries >= 1 that add up to n_kv_heads and ffn, and a rank's heads * head_dim
 * and FFN columns are multiples of 16 bytes of weights (TPI_ERR_SHAPE
 * otherwise).  NULL lists = the uniform partition. */
int tpi_tp_rank_slice_p(const tpi_config *cfg, int n_ranks, int rank, const int32_t *kv_heads_per_rank,
                        const int32_t *ffn_cols_per_rank, int tensor_id, int64_t *row0, int64_t *n_rows, int64_t *col0,
                        int64_t *n_cols);

/* Arena sizes rank `rank` needs (its slice of the model, its KV heads, its
 * receive buffers).  Pure host arithmetic. */
int tpi_tp_query_arena(const tpi_config *cfg, int n_ranks, int rank, int window_blocks, size_t *dev_bytes,
                       size_t *host_bytes);

int tpi_tp_query_arena_p(const tpi_config *cfg, int n_ranks, int rank, const int32_t *kv_heads_per_rank,
                         const int32_t *ffn_cols_per_rank, int window_blocks, size_t *dev_bytes, size_t *host_bytes);

/* Builds the R ranks.  res: HOST array of n_ranks resource sets (arenas on the
 * rank's device, streams of that device; both streams required).  devices: HOST
 * array of n_ranks CUDA device ordinals, or NULL = every rank on the current
 * device.  fill / user: the weight source of tpi.h (unsharded tensors); the
 * group asks it for each rank's slices only.  When two ranks sit on different
 * devices, peer access between them must be possible (it is enabled here). */
int tpi_tp_create(const tpi_config *cfg, int n_ranks, const tpi_resources *res, const int *devices, tpi_fill_fn fill,
                  void *user, int window_blocks, tpi_tp_group **out);
/* The same with a heterogeneous partition (lists as in tpi_tp_rank_slice_p). */
int tpi_tp_create_p(const tpi_config *cfg, int n_ranks, const int32_t *kv_heads_per_rank, const int32_t *ffn_cols_per_rank,
                    const tpi_resources *res, const int *devices, tpi_fill_fn fill, void *user, int window_blocks,
                    tpi_tp_group **out);
void tpi_tp_free(tpi_tp_group *g);

/* Algorithm 1 / 2 for a prompt and for one position; arguments as tpi_prefill /
 * tpi_decode_step / tpi_decode_run (tokens and logits are the master's). */
int tpi_tp_prefill(tpi_tp_group *g, const int32_t *tokens, int n_tokens, int32_t *first_token, float *logits_or_null);
int tpi_tp_decode_step(tpi_tp_group *g, int32_t token_in, int32_t *token_out, float *logits_or_null);
int tpi_tp_decode_run(tpi_tp_group *g, int32_t token_in, int n_steps, int32_t *tokens_out);

/* Position 0 on every rank, exchange counters and flags cleared (also the way
 * back to a consistent state after a failed or timed-out call). */
int tpi_tp_reset(tpi_tp_group *g);
int tpi_tp_position(const tpi_tp_group *g);
int tpi_tp_n_ranks(const tpi_tp_group *g);

/* Debug taps: H_attn (which = 0) / H_ffn (1) of `layer` as rank `rank` holds it
 * after the allreduce (every rank holds the same bits).  dst_host: float[hidden]. */
int tpi_tp_get_hidden(tpi_tp_group *g, int rank, int layer, int which, float *dst_host);
/* Cached keys / values of GLOBAL kv head `kv_head` (read from the rank that owns it). */
int tpi_tp_get_kv(tpi_tp_group *g, int layer, int kv_head, int pos0, int n, float *k_dst, float *v_dst);

/* Options.  TPI_TP_OPT_EVENTS (default 1): order every exchange by CUDA events
 * between the ranks' streams; 0 is refused while two ranks share a device.
 * TPI_TP_OPT_WAIT_POLLS: poll limit of the device-side flag waits (default
 * 2097152, about a quarter of a second, while events order the exchange and the
 * wait is a backstop; 67108864, about ten seconds, once events are off and a
 * consumer really waits for ranks that run at their own pace).  TPI_TP_OPT_DROP_PUSH = r + 1: failure
 * injection on the host - rank r's next push computes its partial sums but
 * never publishes them (a rank that "never joins"); the other ranks' waits then
 * run out and the call returns TPI_ERR_TIMEOUT; one-shot, 0 clears it.
 * TPI_TP_OPT_PDL: programmatic dependent launch between a rank's kernels
 * (default 1).  TPI_TP_OPT_BATCHED_PROMPT (default 1): see above.
 * TPI_TP_OPT_GRAPH (default 1): with every block resident, a decode position of
 * ALL ranks is one CUDA graph (captured from the master's stream; the other
 * ranks' streams join through the exchange's event waits, which become graph
 * edges), so a token costs the host one launch; 0 = stream launches. */
enum { TPI_TP_OPT_EVENTS = 0, TPI_TP_OPT_WAIT_POLLS = 1, TPI_TP_OPT_DROP_PUSH = 2, TPI_TP_OPT_PDL = 3,
       TPI_TP_OPT_BATCHED_PROMPT = 4, TPI_TP_OPT_GRAPH = 5 };
int tpi_tp_set_option(tpi_tp_group *g, int option, int value);

typedef struct {
  int32_t n_ranks, position, events, kernel_launches_last; /* launches summed over the ranks */
  uint64_t exchanges_total;          /* allreduces + broadcasts completed so far (per rank)       */
  uint64_t exchange_bytes_per_token; /* bytes one rank stores into OTHER ranks' buffers per token */
  uint64_t weight_bytes_rank0, weight_bytes_worker; /* bytes a decode step streams on that rank    */
  double last_decode_ms;             /* host wall time of the last decode call                    */
} tpi_tp_stats;
int tpi_tp_get_stats(tpi_tp_group *g, tpi_tp_stats *out);

#ifdef __cplusplus
}
#endif
#endif /* TPI_TP_H */
