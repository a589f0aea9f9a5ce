/*
 * headcast.h - C ABI of the HeadCast attention path for NVIDIA B200 (sm_100a).
 *
 * HeadCast (Sec. 4 of the paper) serves the attention layers of an autoregressive video
 * diffusion transformer that generates a video block by block over a KV cache (Sec. 3.1):
 *   warm-up with full attention -> one-time head classification (Sec. 4.2, Eq. 2-5) ->
 *   split of the monolithic cache into per-archetype buffers (Sec. 4.3) ->
 *   head-specific attention (Sec. 4.4) with a per-block append and roll of those buffers.
 * One headcast_ctx is one attention layer.  Batch size is 1.
 *
 * Conventions for every call:
 *   - returns HC_OK (0) or a negative HC_ERR_* code; never throws, aborts or prints.
 *     headcast_last_error() gives a context-owned, human-readable reason for the last failure.
 *   - tensor arguments named *_dev are DEVICE pointers owned by the caller, 16-byte aligned,
 *     contiguous, bf16, layout [L][H][d]: L = frames_per_block*grid_h*grid_w tokens of one
 *     block in (frame, grid row, grid column) order, H = n_heads, d = head_dim.
 *     arguments named *_host are HOST pointers.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is enqueued
 *     on it and the call returns without waiting, except where a call says it synchronises.
 *   - the context owns every cache, table and scratch buffer (device memory it allocates at
 *     headcast_create / headcast_split_cache and frees at headcast_destroy).  The caller must
 *     keep the context's device current and must not use one context from two threads at once.
 *   - a kernel that gave up on a bounded wait sets a device status word; the next synchronising
 *     call, or headcast_check(), reports it as HC_ERR_TIMEOUT.  Until it has been reported, later
 *     attention launches of the context return at once without computing anything (their
 *     outputs are undefined); reading the status clears it and puts the context back to work.
 *
 * States: FILLING (monolithic cache only) --headcast_split_cache--> SPLIT.  A call made in
 * the wrong state returns HC_ERR_STATE and changes nothing.
 */
#ifndef HEADCAST_H_
#define HEADCAST_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  HC_OK = 0,
  HC_ERR_INVALID_ARG = -1,
  HC_ERR_STATE = -2,
  HC_ERR_CUDA = -3,
  HC_ERR_NOMEM = -4,
  HC_ERR_UNSUPPORTED = -5,
  HC_ERR_TIMEOUT = -6
};

/* Head archetypes (Sec. 3.2, Eq. 5). */
enum { HC_SINK = 0, HC_DUMMY = 1, HC_SPATIAL = 2, HC_GLOBAL = 3 };

/* Per-head score vector written by headcast_classify. */
enum {
  HC_SCORE_COS_SINK = 0,    /* Eq. 3, m = sink   */
  HC_SCORE_COS_DUMMY = 1,   /* Eq. 3, m = dummy  */
  HC_SCORE_COS_SPATIAL = 2, /* Eq. 3, m = spatial */
  HC_SCORE_P5_SPATIAL = 3,  /* 5th percentile of the token-wise spatial cosines (Eq. 4) */
  HC_SCORE_MSE_SPATIAL = 4, /* MSE(O_spatial, O_ref) over all L*d elements (Eq. 4) */
  HC_SCORE_SCORE = 5,       /* P5 - gamma * MSE (Eq. 4) */
  HC_SCORE_MASS_FIRST = 6,  /* mean attention mass on the first cached block */
  HC_SCORE_MASS_LAST = 7,   /* ... on the newest block */
  HC_SCORE_MASS_SPATIAL = 8,/* ... inside the (2r+1)x(2r+1) neighbourhood, any frame */
  HC_SCORE_MASS_REST = 9,   /* ... on everything else */
  HC_N_SCORES = 10
};

/* Decision rule of headcast_classify. */
enum {
  HC_RULE_COSINE = 0, /* Eq. 5 of the paper: mean cosines and the Spatial score against their thresholds */
  HC_RULE_MASS = 1    /* not in the paper: the same cascade on the mean attention masses (first block, newest block,
                         (2r+1)^2 neighbourhood) against one threshold mass_tau */
};

typedef struct headcast_config {
  int32_t n_heads;          /* H, 1..64 */
  int32_t head_dim;         /* d, 64 or 128 */
  int32_t grid_h, grid_w;   /* latent token grid of one frame */
  int32_t frames_per_block; /* 3 in the paper (Sec. 5.1) */
  int32_t n_blocks;         /* cache capacity in blocks (2..32), counting the sink block and the newest block */
  int32_t cell_h, cell_w;   /* deployed Spatial cell, 10 x 10 in the paper (Sec. 5.1) */
  /* optional explicit cell edges (HOST arrays, copied at create; 0 = first edge, grid = last).
   * NULL/0 selects the default rule: n = max(1, floor(grid/cell + 1/2)) cells per axis, edge i = floor(i*grid/n). */
  const int32_t* row_edges_host;
  int32_t n_row_edges;
  const int32_t* col_edges_host;
  int32_t n_col_edges;
  int32_t proxy_radius;     /* r of the Spatial proxy, 2 in the paper */
  float theta_sink, theta_dummy, theta_spatial; /* 0.95 each (Sec. 5.1) */
  float theta_score;        /* 0.755 */
  float gamma;              /* 5 */
  float softmax_scale;      /* 0 selects 1/sqrt(d) */
  int32_t keep_monolithic;  /* nonzero: keep appending to the monolithic cache after the split, so that
                               headcast_full_attend (the dense baseline) stays usable on the same history */
  int32_t sd_mode;          /* 0: Sink and Dummy heads keep exactly one block (Sec. 4.3, 4.4).  1: the accounting of
                               Appendix B / C: Sink keeps its anchor block plus the current block, Dummy the previous
                               plus the current block (2L tokens each) */
  int32_t rule;             /* HC_RULE_COSINE (default, Eq. 5) or HC_RULE_MASS */
  float mass_tau;           /* HC_RULE_MASS only: Sink if mass_first >= tau, else Dummy if mass_last >= tau, else Spatial
                               if mass_spatial >= tau, else Global.  0 < tau <= 1; default 0.9 (the paper gives none) */
} headcast_config;

typedef struct headcast_ctx headcast_ctx;

/* Fills *cfg with the paper's constants (Sec. 5.1); sizes are left zero for the caller. */
void headcast_default_config(headcast_config* cfg);

/* Validates cfg, allocates on the current device the (zeroed) monolithic cache and an equally large zeroed arena
 * from which headcast_split_cache later carves the per-archetype buffers, and returns a context in *out.
 * Synchronises the device. */
int headcast_create(const headcast_config* cfg, headcast_ctx** out);

/* Frees everything the context owns.  Synchronises the device.  NULL is accepted. */
int headcast_destroy(headcast_ctx* ctx);

/* Sec. 3.1 / 4.3: adds one generated block's K and V ([L][H][d] each, device) to the cache.
 * While the cache is not full the block is placed after the newest one; once full, the oldest block other
 * than the first (sink) block is evicted.  Before the split this updates the monolithic cache; after it,
 * the per-archetype buffers: Sink heads keep their frozen first block, Dummy heads overwrite their single
 * block, Global and Spatial heads slide their window.  Pure byte movement: stored values are bit-identical. */
int headcast_append(headcast_ctx* ctx, const void* k_new_dev, const void* v_new_dev, void* stream);

/* Per-denoise-step refresh: replaces the K and V of the NEWEST cached block wherever it is kept as the newest block
 * (monolithic cache, Global / Spatial windows, a Dummy head's current block, a Sink head's current block with
 * sd_mode 1); no block is evicted and a Sink head's anchor block stays frozen.  Needs at least one cached block. */
int headcast_overwrite_last(headcast_ctx* ctx, const void* k_new_dev, const void* v_new_dev, void* stream);

/* Dense baseline and warm-up path (Sec. 3.1; "Global Path", Sec. 4.4): every head attends to every cached
 * token of the monolithic cache.  q_dev and out_dev are [L][H][d] bf16.  Needs at least one cached block;
 * after the split it needs keep_monolithic. */
int headcast_full_attend(headcast_ctx* ctx, const void* q_dev, void* out_dev, void* stream);

/* Sec. 4.2: one-time classification with the block's queries q_dev at the maximum-noise step.  Computes the
 * full-context reference output (Eq. 2) and the Sink, Dummy and Spatial proxy outputs, the mean cosines
 * (Eq. 3), the Spatial score (Eq. 4) and the label of every head (Eq. 5).  Needs >= 2 cached blocks and
 * state FILLING.  Synchronises `stream`; writes labels_host[H] and, if not NULL, scores_host[H][HC_N_SCORES];
 * the labels are also stored in the context. */
int headcast_classify(headcast_ctx* ctx, const void* q_dev, int32_t* labels_host, float* scores_host, void* stream);

/* Overrides / reads the stored labels (seeded head mixes, ablations).  Host arrays of H int32. State FILLING. */
int headcast_set_labels(headcast_ctx* ctx, const int32_t* labels_host);
int headcast_get_labels(const headcast_ctx* ctx, int32_t* labels_host);

/* Sec. 4.3: slices the monolithic cache along the head dimension into the Sink-Dummy buffer (one block per
 * head), the Global buffer and the Spatial buffer (full window each).  Needs labels and >= 1 cached block.
 * Allocates nothing (the buffers come from the arena reserved at create); unless keep_monolithic, the monolithic
 * cache is released in stream order after the gather (cudaFreeAsync: no host or device stall).  State becomes SPLIT. */
int headcast_split_cache(headcast_ctx* ctx, void* stream);

/* Sec. 4.4: head-specific attention of one block's queries, one launch for all pathways.  Sink heads read
 * their first block, Dummy heads the newest block, Global heads the whole window, Spatial heads the keys of
 * the query's own grid cell in every cached frame.  out_dev[L][H][d]: every head's rows land at its original
 * head index (the paper's concatenation along heads).  State SPLIT. */
int headcast_attend(headcast_ctx* ctx, const void* q_dev, void* out_dev, void* stream);

/* Copies what the cache currently keeps for one head into k_out_dev / v_out_dev ([n_tokens][d] bf16, room for
 * n_blocks*L rows) in LOGICAL order - oldest kept block first, tokens in (frame, row, column) order - whatever
 * the private physical layout is.  *n_tokens_host receives the row count.  Either output may be NULL. */
int headcast_export_cache(headcast_ctx* ctx, int32_t head, void* k_out_dev, void* v_out_dev,
                          int32_t* n_tokens_host, void* stream);

/* Number of cached blocks (before the split: of the monolithic cache; after: of the sliding window). */
int headcast_n_filled(const headcast_ctx* ctx);

/* Number of kernels this context has launched so far (bookkeeping for benchmarks). */
int64_t headcast_launch_count(const headcast_ctx* ctx);

/* The same two steps for callers whose tensors live in HOST memory (the paper's pipeline keeps them on the GPU; this
 * is for measuring, or serving, the path end to end across PCIe).  k_host/v_host/q_host/out_host: host pointers to
 * [L][H][d] bf16; pinned memory lets the copies overlap the kernels, pageable memory works but serialises.
 * headcast_append_host copies the block into device staging owned by the context and appends it.
 * headcast_attend_host splits the call into four stages (first half of the Global heads' query rows; Sink + Dummy
 * heads; Spatial heads; second half of the Global heads' rows): each stage's part of Q is copied in, attended
 * (Sec. 4.4, as headcast_attend) and its part of the output copied out, on two copy streams of the context, so that
 * transfers in both directions overlap the attention of the other stages.  Both
 * return once everything is enqueued; out_host is complete when work enqueued on `stream` after the call runs (e.g.
 * after synchronising `stream`).  q_host must stay unchanged and out_host untouched until then.  Staging buffers,
 * streams and events are created on the first call.  Errors as headcast_attend / headcast_append. */
int headcast_append_host(headcast_ctx* ctx, const void* k_host, const void* v_host, void* stream);
int headcast_attend_host(headcast_ctx* ctx, const void* q_host, void* out_host, void* stream);

/* Algorithmic FLOPs (4 * L_q * L_k * d per head, Appendix B) of the next headcast_attend (dense = 0) or
 * headcast_full_attend (dense = 1) with the current cache fill and labels. */
double headcast_attend_flops(const headcast_ctx* ctx, int32_t dense);

/* Benchmark aid.  With enable != 0 every later attention call records CUDA events on its stream directly
 * before and after its tensor-core attention kernel (not around the small merge kernel that may follow).
 * headcast_last_attention_kernel_ms waits for the most recent pair and writes the elapsed milliseconds. */
int headcast_set_kernel_timing(headcast_ctx* ctx, int32_t enable);
int headcast_last_attention_kernel_ms(headcast_ctx* ctx, float* ms_host);

/* Scheduling aid.  With enable != 0 every later attention launch records, per work item, the GPU global timer
 * (ns) at which the item's first query tile started and finished.  headcast_read_trace synchronises the device
 * and writes, for each work item of the most recent attention launch, 8 int64 values to rows_host
 * ([capacity][8]): CTA index (the CTA count for items of the shared queue), head, Spatial cell (-1 if none), query
 * rows, key tiles, output mode
 * (0 final, 1 partial, 2 fp32), start ns, end ns.  *n_items_host receives the item count. */
int headcast_set_tracing(headcast_ctx* ctx, int32_t enable);
int headcast_read_trace(headcast_ctx* ctx, int64_t* rows_host, int32_t capacity, int32_t* n_items_host);

/* Host-only (no GPU needed): the work list headcast_attend (dense = 0, labels_host[H] given) or headcast_full_attend
 * (dense = 1) would run with n_filled cached blocks on n_ctas persistent CTAs.  Every item is 16 int32:
 * head, Spatial cell or -1, first query (token, or packed index inside the cell) of query tile 0 and 1, valid rows of
 * tile 0 and 1, buffer (0 monolithic, 1 Sink-Dummy, 2 Global, 3 Spatial), element column, first key row, row stride
 * between key segments, keys per segment, 128-key tiles per segment, first and one-past-last tile of this item,
 * output mode (0 final, 1 partial to be merged), partial slot.  items_host has room for `capacity` items,
 * cta_first_host for n_ctas + 1 entries (items of CTA b are [cta_first[b], cta_first[b+1])); either may be NULL.
 * Items from cta_first[n_ctas] up to *n_items_host belong to no CTA: they form the shared queue (the last ~2 % of
 * the work, cut into small pieces) that CTAs draw from, in order, once their own lists are done. */
int headcast_plan_schedule(const headcast_config* cfg, const int32_t* labels_host, int32_t n_filled, int32_t n_ctas,
                           int32_t dense, int32_t* items_host, int32_t capacity, int32_t* n_items_host,
                           int32_t* cta_first_host);

/* Self-test of the failure path.  Launches one small kernel that waits on a barrier nobody will ever signal; the wait
 * is bounded like every wait in this library, so after limit_ms (1..1000) the kernel records its give-up in the status
 * word and returns normally.  The call synchronises `stream` and returns HC_ERR_TIMEOUT - that is the expected
 * result; the context stays fully usable afterwards.  Nothing faults, traps or hangs. */
int headcast_selftest_bounded_wait(headcast_ctx* ctx, int32_t limit_ms, void* stream);

/* Synchronises `stream` and reports a device-side status raised by any earlier kernel of this context
 * (HC_ERR_TIMEOUT if a bounded wait expired). */
int headcast_check(headcast_ctx* ctx, void* stream);

const char* headcast_last_error(const headcast_ctx* ctx);

/* ---- Dense attention without any allocation -------------------------------------------------------------
 * (This entry point has no counterpart in the paper; it exists for integration.)
 *
 * Some hosts of this library cannot let it allocate device memory: an inference server that has handed the whole
 * GPU to its own pool (a cudaMalloc from a plug-in then fails, or fragments what the pool believes it owns), or a
 * frame loop that cannot afford the device-wide synchronisation an allocation or free implies.  For them,
 * headcast_dense_attend_noalloc computes out[t][h][:] = softmax(scale * q[t][h] . k[:][h]^T) v[:][h] for every head
 * - the same result as headcast_full_attend on a cache holding k and v - and calls no cudaMalloc, cudaFree or
 * other allocating routine.  q_dev and out_dev are [n_queries][n_heads][head_dim] bf16, k_dev and v_dev
 * [n_keys][n_heads][head_dim] bf16, all caller-owned, 16-byte aligned and contiguous.
 *
 * The scratch the kernel needs in global memory (work list, per-CTA ranges, status word; about 140 KB) is a fixed device array inside
 * the library: every GPU that loads the library holds it until the process exits.  Consequences:
 *   - size limit: n_heads * ceil(n_queries / 256) <= HEADCAST_NOALLOC_MAX_ITEMS, head_dim 64 or 128,
 *     n_heads <= 64; anything larger returns HC_ERR_UNSUPPORTED and does nothing;
 *   - all calls on one GPU share that array, which keeps the previous call's contents (each call rewrites what
 *     it uses and clears the status word): two calls whose GPU work overlaps - different streams, or different
 *     host threads - race on it.  Keep calls on one GPU in one stream, or order them with events;
 *   - the first call on each device looks up the array's device address and sets the kernel's shared-memory
 *     attribute (with that device current).  Make that first call before starting any stream capture;
 *   - a call on a stream that is being captured returns HC_ERR_UNSUPPORTED (the work list is copied from a host
 *     image that the next call rewrites).
 * softmax_scale = 0 selects 1/sqrt(head_dim).  Asynchronous on `stream`.  headcast_noalloc_status synchronises
 * the stream and reports HC_ERR_TIMEOUT if the kernel gave up on a bounded wait; headcast_noalloc_last_error
 * returns the reason of the last failing call (process-wide buffer). */
#define HEADCAST_NOALLOC_MAX_ITEMS 2048
int headcast_dense_attend_noalloc(const void* q_dev, const void* k_dev, const void* v_dev, void* out_dev,
                                  int32_t n_queries, int32_t n_keys, int32_t n_heads, int32_t head_dim,
                                  float softmax_scale, void* stream);
int headcast_noalloc_status(void* stream);
const char* headcast_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HEADCAST_H_ */
