/*
 * pasta.h — C ABI of the decode-attention path for interpreter-driven asynchronous decoding
 * ("Learning to Keep a Promise", PASTA; Section 3 "Efficiency", Fig. 2b/2c, Appendix B).
 *
 * Several threads of one response decode one token each in the same model step.  All of them
 * keep their KV in ONE pool; a thread attends to the main-thread tokens that existed when it was
 * spawned plus its own chunk; after <sync/> the main thread attends to everything, each chunk
 * placed logically right after its <promise/>, and nothing is copied.  This library owns the
 * bookkeeping of that pool (pages, per-thread segment lists) and runs the per-step attention on
 * one NVIDIA B200 (sm_100a).  There is no CPU fallback: every compute entry point needs the GPU.
 *
 * General conventions
 *  - Every function returns a pasta_status_t and never throws, aborts or exits.
 *  - Out-parameters are written only on success.  A failed call leaves the pool unchanged.
 *  - "host" pointers are read or written during the call only.  "device" pointers must stay
 *    valid until the stream has executed the work enqueued by the call.
 *  - One pool belongs to one GPU and is not thread-safe: calls on one pool must not overlap.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All device
 *    work of a pool must be issued on streams that are ordered with respect to each other by the
 *    caller; the simplest use is one stream per pool.
 *  - Tensors are dense, row-major, bf16 unless stated; the last index is contiguous.
 */
#ifndef PASTA_H_
#define PASTA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pasta_pool pasta_pool_t;   /* opaque; created by pasta_pool_create, freed by pasta_pool_destroy */
typedef int32_t pasta_status_t;

enum {
  PASTA_OK = 0,
  PASTA_ERR_INVALID_ARG = 1,   /* unknown id, thread listed twice, finished thread in a step, bad pointer or size */
  PASTA_ERR_OUT_OF_PAGES = 2,  /* the pool has too few free pages for the request */
  PASTA_ERR_BAD_STATE = 3,     /* e.g. merging a fork that is still decoding, compute call on a host-only pool */
  PASTA_ERR_CAPACITY = 4,      /* more requests / threads / segments / step entries than the pool was created for */
  PASTA_ERR_CUDA = 5,          /* a CUDA runtime call failed; pasta_last_cuda_error() gives its code */
  PASTA_ERR_DEVICE_CHECK = 6,  /* a kernel found an out-of-range page id or offset and skipped the access */
  PASTA_ERR_TIMEOUT = 7        /* a bounded wait inside a kernel expired; the kernel returned early */
};

enum {
  PASTA_FLAG_HOST_ONLY = 1,      /* bookkeeping only: no CUDA call is ever made, compute entry points return BAD_STATE */
  PASTA_FLAG_NO_TENSOR_PATH = 2, /* route every stream through the warp-shuffle kernel (debugging / comparison) */
  PASTA_FLAG_OUT_BF16 = 4        /* `out` of pasta_decode_attn, pasta_step_device and pasta_step_host is bf16 instead of
                                    fp32 (same shape; the sums stay fp32, one rounding at the end; lse stays fp32).
                                    pasta_decode_attn_noalloc writes fp32 only and returns BAD_STATE on such a pool. */
};

/* thread states reported by pasta_pool_dump */
enum { PASTA_THREAD_ACTIVE = 0, PASTA_THREAD_FINISHED = 1, PASTA_THREAD_MERGED = 2 };

typedef struct {
  int32_t n_layers;                 /* independent layers stored in the pool (page ids are shared by all layers) */
  int32_t n_q_heads, n_kv_heads;    /* n_q_heads must be a multiple of n_kv_heads; group = n_q_heads / n_kv_heads in {1,2,4,8} */
  int32_t head_dim;                 /* 64 or 128 */
  int32_t page_size;                /* tokens per page; must be 16 */
  int32_t n_pages;                  /* pages per layer */
  int32_t max_requests;             /* requests alive at the same time */
  int32_t max_threads_per_request;  /* main thread + every fork ever spawned by one request (ids are not reused) */
  int32_t max_segments_per_thread;  /* longest segment list of one thread */
  int32_t max_step_queries;         /* most queries in one step (one per entry, or per new token); 0 = max_requests * 17 */
  int32_t max_partial_rows;         /* split/segment partial results per layer; 0 = derived from max_step_queries */
  int32_t max_layers_per_launch;    /* layers whose partials fit the workspace at once; 0 = min(n_layers, 8) */
  int32_t flags;                    /* PASTA_FLAG_* */
  int32_t device;                   /* CUDA device ordinal the pool lives on */
  void *kv_base;                    /* device; pasta_kv_bytes() bytes, 1024-byte aligned, allocated and freed by the caller */
  size_t kv_bytes;
  void *workspace;                  /* device; pasta_workspace_bytes() bytes, 256-byte aligned, caller-owned */
  size_t workspace_bytes;
  const int32_t *free_order;        /* host; n_pages entries, a permutation: order in which free pages are handed out
                                       (NULL = 0, 1, 2, …) */
} pasta_pool_config_t;

/* Sizes of the two device buffers the caller has to provide for this configuration. */
pasta_status_t pasta_kv_bytes(const pasta_pool_config_t *cfg, size_t *out);
pasta_status_t pasta_workspace_bytes(const pasta_pool_config_t *cfg, size_t *out);

/*
 * The single pre-allocated KV pool of Section 3 "Efficiency" (here paged: 16 tokens per page, one
 * page list per stream, where a stream is the main thread's tokens or one fork's chunk).  The
 * layout inside a page is private to the library; results do not depend on which pages a stream
 * receives.  Create zero-fills the KV memory once (bytes of a page beyond a stream's end are read
 * and multiplied by zero weights, so they have to be finite); destroy does not touch it.
 */
pasta_status_t pasta_pool_create(const pasta_pool_config_t *cfg, pasta_pool_t **out);
pasta_status_t pasta_pool_destroy(pasta_pool_t *pool);

/* ---- thread lifecycle: host only, integers only (Section 3 "Interpreter") -------------------- */

/* A new response; its main thread has id 0.  The request gets the lowest id not in use. */
pasta_status_t pasta_request_begin(pasta_pool_t *pool, int32_t *out_req);
/* Returns every page of the request: stream by stream (ascending id), page by page, each to the
 * FRONT of the free sequence. */
pasta_status_t pasta_request_end(pasta_pool_t *pool, int32_t req);
/* <promise/>: a fork whose view is the main thread's view at this moment (call it after the promise
 * token was appended), followed by its own chunk.  Forks are numbered 1, 2, 3, … per request. */
pasta_status_t pasta_thread_spawn(pasta_pool_t *pool, int32_t req, int32_t *out_thread);
/*
 * <promise/> with a length prediction (Section 4 "Training a PASTA-SFT model" and Section 6 "Positional
 * Embedding": the main thread cannot know how long the asynchronous block will be, so it assigns position
 * ids past the promise as if the block had the predicted length).  Like pasta_thread_spawn, and also:
 * the fork's first token takes the position id right after the promise token, the main thread's next token
 * takes that id plus predicted_tokens (>= 0; e.g. 10 x the promise's `tokens` attribute for the paper's
 * Pred-10X scheme, 40 for Fixed-40).  Ids are never revised: a chunk longer than predicted runs into ids
 * the main thread has used (not monotone after sync), a shorter one leaves a gap.
 *
 * pending (0 or 1): 1 = the promise has been decoded but is not in the pool yet; it is the main thread's next
 * token (Section 3 "Efficiency", the walk through Fig. 2b: the <async> tag joins the pool at the timestamp of its
 * promise, so the promise and the fork's first token are fed to the model in one step).  The fork's view then
 * counts that token in, the promise keeps the main thread's next position id and the jump by predicted_tokens
 * follows it.  The outcome equals appending the promise first and spawning with pending = 0.  Until the promise
 * is in the pool (by the appends of the same step at the latest) the fork can neither take part in a step, nor
 * append a run, nor be merged: PASTA_ERR_BAD_STATE.  PASTA_ERR_CAPACITY if the main thread's segment list is full.
 * pasta_thread_spawn is the same with predicted_tokens = 0 and pending = 0.
 */
pasta_status_t pasta_thread_spawn_predicted(pasta_pool_t *pool, int32_t req, int32_t predicted_tokens, int32_t pending,
                                            int32_t *out_thread);
/* </async>: the fork decodes no more; its chunk stays invisible to the main thread until merged. */
pasta_status_t pasta_thread_finish(pasta_pool_t *pool, int32_t req, int32_t thread);

/*
 * <sync/> (Section 3: the main thread waits for the forks, then conditions on their chunks; the
 * paper's pool moves no KV at this point and neither does this call).  The named finished forks
 * are merged into the main thread's segment list: each chunk goes right after the main-stream
 * piece that ends at the fork's cut-off (ties: ascending thread id).  n_threads < 0 merges every
 * finished, unmerged fork.  Naming a fork that is still decoding returns BAD_STATE: waiting is
 * the caller's job.  Host only; the <sync/> token itself is appended by the next step.
 */
pasta_status_t pasta_sync_merge(pasta_pool_t *pool, int32_t req, int32_t n_threads, const int32_t *thread_ids);

/* ---- one decode step (Section 3: every active thread decodes one token in the same step) ----- */

/*
 * Reserves the pool slot of every token appended in this step and plans the attention of the
 * step.  Entry i is thread thread_ids[i] of request req_ids[i] (host arrays, n entries, each
 * thread at most once, ACTIVE threads only) and appends n_new[i] >= 0 tokens (NULL = all 1).
 * Pages are taken in list order, one whenever a stream's token index is a multiple of 16.
 * An entry that would see nothing (no visible token and n_new == 0) is INVALID_ARG.
 * QUERIES.  An entry with n_new <= 1 issues one attention query (for its new token, or over what the thread
 * sees already).  An entry with n_new = m > 1 (several tokens of one thread fed in one step: a prompt chunk, a
 * promise together with what follows it) issues m queries, one per new token in order, each seeing the
 * thread's view up to and including its own token and none of the later ones — causal attention among the new
 * tokens, the same results as m steps of one token.  The step's queries are numbered in entry order; every
 * per-query array of the calls below (q, out, lse, slots, positions) has one row per query, and k_new / v_new
 * one row per appended token in the same order.  The number of queries is bounded by max_step_queries
 * (CAPACITY, nothing reserved).
 * If the bookkeeping succeeds but the step cannot be planned within the pool's capacities (partial rows, plan
 * words), the call returns CAPACITY and takes the reservation back: the pool is as it was, only the previous
 * step's plan is no longer valid.
 * The plan is uploaded on `stream`; it is used by the pasta_kv_append and pasta_decode_attn calls
 * that follow, for every layer, until the next pasta_step_begin.
 */
pasta_status_t pasta_step_begin(pasta_pool_t *pool, int32_t n, const int32_t *req_ids,
                                const int32_t *thread_ids, const int32_t *n_new, void *stream);

/* (page, offset) reserved by the last pasta_step_begin for the token of each of its queries, two int32 per
 * query, (-1, -1) for the query of an entry with n_new == 0.  Host array; capacity in queries (CAPACITY if
 * smaller than the step's number of queries). */
pasta_status_t pasta_step_slots(pasta_pool_t *pool, int32_t *out_slots, int32_t capacity_queries);

/* Position id of each query's token for the last pasta_step_begin.  Host array; capacity in queries. */
pasta_status_t pasta_step_positions(pasta_pool_t *pool, int32_t *out_pos, int32_t capacity_queries);

/*
 * pasta_kv_append with rotary position embedding fused in: every new K vector is rotated by its token's
 * position id before it is stored (rotate-half form: element i pairs with element i + head_dim/2,
 * angle = position * theta^(-2i/head_dim), angles evaluated in double precision, result rounded to bf16);
 * V is copied unchanged.  theta > 1 (10000 for the usual base).
 */
pasta_status_t pasta_kv_append_rope(pasta_pool_t *pool, int32_t layer_begin, int32_t layer_count,
                                    const void *k_new, const void *v_new, float theta, void *stream);
/* Rotates the step's queries in place by the same rule: q device bf16 [layer_count, n, n_q_heads, head_dim]. */
pasta_status_t pasta_rope_queries(pasta_pool_t *pool, int32_t layer_count, void *q, float theta, void *stream);

/*
 * Copies the new tokens' K and V into their reserved slots for layers
 * [layer_begin, layer_begin + layer_count).  k_new, v_new: device bf16
 * [layer_count, n_app, n_kv_heads, head_dim], where n_app is the number of step entries with
 * n_new == 1, in entry order.  A pure bit copy.
 */
pasta_status_t pasta_kv_append(pasta_pool_t *pool, int32_t layer_begin, int32_t layer_count,
                               const void *k_new, const void *v_new, void *stream);

/*
 * Decode attention of the planned step.  For entry i and query head h (kv head h / group):
 *     out[l, i, h, :] = softmax(q[l, i, h, :] . K_vis^T * scale) V_vis
 * over the tokens visible to that thread (its segment list; the token appended in this step
 * included).  q: device bf16 [layer_count, n, n_q_heads, head_dim]; out: device fp32 of the same
 * shape; lse: optional device fp32 [layer_count, n, n_q_heads] (natural-log sum of exponentials of
 * the scaled scores), may be NULL; scale 0 means 1/sqrt(head_dim).
 * With head_dim 128, the streams a request's threads read are staged into shared memory once per kv
 * head and scored against all those threads' queries on tensor cores (rows that may not see a page are
 * masked), as long as threads x (n_q_heads / n_kv_heads) <= 128 and the request has at most 4095 streams;
 * other requests and head sizes take a warp-shuffle kernel; a merge kernel combines the partial results
 * (fp32 throughout).  Where one piece of work covers everything a (query, kv head) pair reads, the tensor-core pass
 * writes that pair's rows of out and lse itself; a step made of such pieces only launches no merge kernel.
 */
pasta_status_t pasta_decode_attn(pasta_pool_t *pool, int32_t layer_begin, int32_t layer_count,
                                 const void *q, void *out, float *lse, float scale, void *stream);

/*
 * Appends m tokens to one thread outside a decode step (prompt prefill, benchmark set-up):
 * reserves slots like m steps of that thread alone would, then copies k, v
 * (device bf16 [layer_count, m, n_kv_heads, head_dim]).  With layer_count == 0 only the
 * bookkeeping is done.  Invalidates the current step plan.
 */
pasta_status_t pasta_kv_append_run(pasta_pool_t *pool, int32_t req, int32_t thread, int32_t m,
                                   int32_t layer_begin, int32_t layer_count,
                                   const void *k, const void *v, void *stream);

/* pasta_kv_append_run with the rotary embedding of pasta_kv_append_rope (consecutive position ids from the
 * thread's next one). */
pasta_status_t pasta_kv_append_run_rope(pasta_pool_t *pool, int32_t req, int32_t thread, int32_t m,
                                        int32_t layer_begin, int32_t layer_count, const void *k, const void *v,
                                        float theta, void *stream);

/*
 * One whole step with DEVICE tensors in one call: pasta_step_begin, pasta_kv_append and pasta_decode_attn for all
 * layers (Section 3: a decoding step of every active thread).  Arguments as in those three calls: k_new, v_new
 * device bf16 [n_layers, appended tokens, n_kv_heads, head_dim]; q device bf16 [n_layers, queries, n_q_heads,
 * head_dim]; out device fp32 like q; lse optional.  Saves the caller two library calls per step, which is what
 * bounds small steps.  Errors as in the three calls; after a failure of the first nothing is enqueued.
 */
pasta_status_t pasta_step_device(pasta_pool_t *pool, int32_t n, const int32_t *req_ids, const int32_t *thread_ids,
                                 const int32_t *n_new, const void *k_new, const void *v_new, const void *q, void *out,
                                 float *lse, float scale, void *stream);

/*
 * One whole step with HOST tensors: the copies of k_new / v_new / q to the device are enqueued, the step is
 * planned while they are in flight (step_begin), then kv_append and decode_attn for all layers, `out` is copied
 * back and the stream synchronised.  k_new, v_new:
 * host bf16 [n_layers, n_app, n_kv_heads, head_dim]; q: host bf16 [n_layers, n, n_q_heads, head_dim];
 * out: host fp32 like q.  staging: device scratch of at least pasta_step_host_bytes(pool, n)
 * bytes, caller-owned.  Pinned host memory makes the copies asynchronous; pageable works too.
 * Entries append at most one token each here (n_new[i] > 1: INVALID_ARG, nothing reserved).
 */
pasta_status_t pasta_step_host_bytes(pasta_pool_t *pool, int32_t n, size_t *out);
/*
 * The same step in two halves, so that a caller can keep two or three steps in flight (Section 3: the decode loop is
 * one step after the other; what overlaps here are the copies and the host's planning of one step with the kernels of
 * its neighbours).
 * pasta_step_host_begin enqueues everything pasta_step_host does (the input copies and the copy of `out` back to
 * the host run on streams of the pool's own, ordered with `stream` by events) and returns without waiting;
 * pasta_step_host_wait blocks until the OLDEST step begun and not yet waited for has delivered its `out`.
 * k_new, v_new, q and out must stay untouched between the two calls.  At most two steps may be begun and not
 * waited for, three when `staging_bytes` is at least three times pasta_step_host_bytes (one begin more: BAD_STATE, as
 * is a wait with nothing begun).  With `staging_bytes` of at least twice pasta_step_host_bytes the inputs of a step
 * are copied while the step before still computes; with less, the copies wait for that step to leave the area.  With
 * three steps in flight the host never waits for a step's outputs to cross the bus before it plans the next but one.
 * Pinned host memory is required for any overlap; use the same staging area and size for all steps in flight.
 */
pasta_status_t pasta_step_host_begin(pasta_pool_t *pool, int32_t n, const int32_t *req_ids,
                                     const int32_t *thread_ids, const int32_t *n_new,
                                     const void *k_new, const void *v_new, const void *q, void *out,
                                     void *staging, size_t staging_bytes, float scale, void *stream);
pasta_status_t pasta_step_host_wait(pasta_pool_t *pool);
pasta_status_t pasta_step_host(pasta_pool_t *pool, int32_t n, const int32_t *req_ids,
                               const int32_t *thread_ids, const int32_t *n_new,
                               const void *k_new, const void *v_new, const void *q, void *out,
                               void *staging, size_t staging_bytes, float scale, void *stream);

/*
 * (No counterpart in the paper: an addition for callers that are not allowed to allocate.)
 *
 * pasta_decode_attn for ONE layer of the planned step, with the intermediate partial results (one
 * (max, sum, unnormalised output) row per query head and per piece of the visible set) kept in a fixed
 * array inside the library's own device image instead of in workspace memory.  The call itself calls no
 * allocation routine of any kind, which is what code running under a memory budget that is frozen after
 * start-up needs: inference-engine plug-ins, real-time loops, or a process whose GPU memory is entirely
 * owned by a framework's arena.
 *   - The array holds PASTA_NOALLOC_MAX_ROWS partial rows (about 8 MiB; every GPU that loads the library
 *     carries it until the process exits).  A step whose plan needs more rows is refused with
 *     PASTA_ERR_CAPACITY; use pasta_decode_attn for those.
 *   - The first call on a device looks up the array's device address (a runtime query, no allocation).
 *     Make that first call outside any stream capture.  The pool's device must be the current device.
 *     The address is kept for the life of the device's primary context: after cudaDeviceReset the library
 *     has to be reloaded before this entry point is used again.
 *   - All calls, from all pools, share the one array per GPU and each overwrites what the previous one
 *     left: two calls whose kernels may run at the same time on one GPU (different streams, different
 *     pools or processes' threads) race on it and corrupt each other's results.  Serialise them.
 * q, out, lse, scale, stream: as for pasta_decode_attn with layer_count == 1
 * (q: device bf16 [n, n_q_heads, head_dim]; out: device fp32 of the same shape).
 */
#define PASTA_NOALLOC_MAX_ROWS 16384
pasta_status_t pasta_decode_attn_noalloc(pasta_pool_t *pool, int32_t layer, const void *q, void *out,
                                         float *lse, float scale, void *stream);

/* ---- comparison layout: the paper's dense pool with a boolean mask ------------------------------ */

/*
 * The layout the paper itself describes (Section 3 "Efficiency", Fig. 2b/2c): ONE dense, token-granular pool per
 * response, filled in decode order so that the tokens of the threads interleave, and a boolean attention mask per
 * thread over the pool's slots.  Kept here as a measured comparison for the paged pool above (next to the duplicated
 * rows of Appendix B); these calls own no state: the caller holds the tensors (paper_2502_11517_b200/dense_mask.py).
 *   k_pool, v_pool  device bf16 [max_slots, n_kv_heads, head_dim], slot = position in decode order
 *   mask, own       device bytes [n_threads, mask_stride]: mask[t, s] != 0 iff thread t may attend to slot s;
 *                   own[t, s] != 0 iff thread t decoded slot s (what <sync/> adds to the main thread's row)
 * pasta_dense_append copies n_new (<= 64) tokens k_new / v_new [n_new, n_kv_heads, head_dim] to slots slot0 ...
 * and sets mask and own of token i in row rows[i] (host array).  pasta_dense_mask_attn computes, for query i
 * (q device bf16 [n_queries, n_q_heads, head_dim]; mask_row device int32 [n_queries]: its thread's mask row),
 * softmax(q K^T scale + (mask ? 0 : -inf)) V over slots [0, n_slots) into out (device fp32 like q) and the
 * log-sum-exp into lse (optional): every query reads every slot, whatever the mask says, as masked attention over
 * a dense cache does.  scratch: device, 256-byte aligned, pasta_dense_mask_scratch_bytes() bytes.  head_dim 64 or
 * 128, n_q_heads / n_kv_heads in {1, 2, 4}.  Errors: INVALID_ARG, CUDA.
 */
pasta_status_t pasta_dense_mask_scratch_bytes(int32_t n_queries, int32_t n_slots, int32_t n_q_heads, int32_t n_kv_heads,
                                              int32_t head_dim, size_t *out);
pasta_status_t pasta_dense_append(void *k_pool, void *v_pool, uint8_t *mask, uint8_t *own, int64_t mask_stride,
                                  int32_t slot0, int32_t n_new, const int32_t *rows, const void *k_new,
                                  const void *v_new, int32_t n_kv_heads, int32_t head_dim, void *stream);
pasta_status_t pasta_dense_mask_attn(const void *k_pool, const void *v_pool, const uint8_t *mask, int64_t mask_stride,
                                     const int32_t *mask_row, const void *q, void *out, float *lse, void *scratch,
                                     size_t scratch_bytes, int32_t n_queries, int32_t n_slots, int32_t n_q_heads,
                                     int32_t n_kv_heads, int32_t head_dim, float scale, void *stream);

/* ---- introspection ---------------------------------------------------------------------------- */

/*
 * Reads tokens [start, start + m) of one stream (stream id = thread id; 0 = main) of one layer back
 * into dense device bf16 arrays k_out, v_out [m, n_kv_heads, head_dim].
 */
pasta_status_t pasta_kv_read(pasta_pool_t *pool, int32_t layer, int32_t req, int32_t stream_id,
                             int32_t start, int32_t m, void *k_out, void *v_out, void *stream);

/*
 * Serialises the bookkeeping state into host int32 words:
 *   n_requests, then per live request (ascending id):
 *     req, n_streams, per stream (ascending id): stream, len, n_pages, page ids…
 *     n_threads, per thread (ascending id): thread, state, cutoff, next position id, n_segments, (stream, start, len)…
 *   n_free, free page ids in hand-out order.
 * *needed receives the number of words; nothing is written when capacity_words is too small
 * (the call then still returns PASTA_OK so that the size can be queried with host_buf == NULL).
 */
pasta_status_t pasta_pool_dump(pasta_pool_t *pool, int32_t *host_buf, size_t capacity_words, size_t *needed);

/*
 * The current step plan as uploaded to the device (int32 words, layout documented in
 * pasta_plan.h inside the package).  Same size protocol as pasta_pool_dump.  For tests.
 */
pasta_status_t pasta_plan_dump(pasta_pool_t *pool, int32_t *host_buf, size_t capacity_words, size_t *needed);

/* Synchronises `stream`, returns and clears the status word the kernels write
 * (PASTA_OK, PASTA_ERR_DEVICE_CHECK or PASTA_ERR_TIMEOUT). */
pasta_status_t pasta_pool_status(pasta_pool_t *pool, void *stream);

/*
 * Test hooks for the bounded waits inside the kernels (no counterpart in the paper, whose only wait is the
 * interpreter's, on the host, at <sync/>).  Every wait of one kernel role for another gives up after a number of SM
 * clock cycles, the kernel then returns early and pasta_pool_status reports PASTA_ERR_TIMEOUT.
 * pasta_debug_set_wait_limit sets that number for the kernels this pool launches from now on (cycles <= 0 restores
 * the default of 3e9, about 1.5 s).  pasta_debug_wait_expiry enqueues a one-warp kernel that waits, with the pool's
 * limit, for a barrier nobody completes: with a short limit it returns after that many cycles and leaves
 * PASTA_ERR_TIMEOUT in the status word, which is how the tests see the limit, the report and the recovery work.
 * With the default limit it occupies one warp for 1.5 s.  Neither touches the pool's bookkeeping or KV memory.
 */
pasta_status_t pasta_debug_set_wait_limit(pasta_pool_t *pool, int64_t cycles);
/*
 * Makes the wait of a role of the tensor-core attention kernel run out for real: the roles whose bit is set in
 * role_mask (1 page producer, 2 MMA issue, 4 query-operand builder, 8 / 16 the two softmax groups) do not start in
 * the launches that follow, the roles that wait for them give up after the pool's wait limit, every CTA drains what
 * it has in flight, frees its tensor memory and returns, and the status word holds PASTA_ERR_TIMEOUT.  The outputs
 * of such a launch are undefined.  Set a short limit first (pasta_debug_set_wait_limit); 0 switches the hook off.
 */
pasta_status_t pasta_debug_hold_roles(pasta_pool_t *pool, int32_t role_mask);
/*
 * Tuning hook (no counterpart in the paper).  The tensor-core kernel assigns the tiles of a step to its CTAs in
 * advance, except that of the short (request, kv head) runs, those of at most 4 x `tiles` tiles, every so often a whole
 * one is kept back, `percent` of their tiles in all (0 to 50; 10 by default), in units of at most `tiles` tiles (2 to
 * 1024; 16 by default).  The CTAs take these from a shared counter once their own work is done: SMs that stream faster
 * than others then do more of it.  0 percent assigns everything in advance.  Takes effect from the next
 * pasta_step_begin, and only for steps large enough for it to matter (16 tiles per CTA).
 */
pasta_status_t pasta_debug_set_tail(pasta_pool_t *pool, int32_t percent, int32_t tiles);
/*
 * Tuning hook (no counterpart in the paper), process-wide.  The kernels of a step (append, the two attention passes, the
 * merge) are launched so that each may set itself up while the one ahead of it in the stream drains (programmatic
 * dependent launch); every kernel waits for the one ahead to have completed before it touches anything that one reads
 * or writes, so results do not depend on the setting.  on = 0 launches them one strictly after the other; on = 1
 * (default) overlaps them.  Takes effect from the next launch.
 */
void pasta_debug_set_launch_overlap(int32_t on);
/*
 * Measurement aid (no counterpart in the paper): enqueues a kernel that reads `bytes` of device memory at `src`
 * (16-byte aligned; NULL = the pool's own KV memory, all of it) and does nothing with them, so that a benchmark can
 * time what a read-only kernel is given on this GPU next to the attention kernel.  mode 0: plain 16-byte loads;
 * mode 1: bulk copies into shared memory, one CTA per SM with 3 x 64 KB in flight, the mechanism of the tensor-core
 * attention kernel (whole 64 KB chunks only); mode 2: the same, every 8 KB piece taken from a pseudo-random place of
 * the buffer, the way a stream's pages lie in a pool that hands pages out in random order.  Writes nothing but 8
 * scratch bytes of the workspace.
 */
pasta_status_t pasta_debug_stream_read(pasta_pool_t *pool, const void *src, size_t bytes, int32_t mode, void *stream);
pasta_status_t pasta_debug_wait_expiry(pasta_pool_t *pool, void *stream);

/* Number of kernels this pool has launched so far (for launch accounting). */
pasta_status_t pasta_launch_count(pasta_pool_t *pool, int64_t *out);

/*
 * Kernel timing for benchmarks.  on = 0 switches it off; on = k >= 1 makes every k-th pasta_decode_attn launch group
 * (the first one included) bracket each of its kernels with CUDA events on the launching stream (at most 512 timed
 * groups are kept between two reads; on < 0 is INVALID_ARG).  A timing event between two kernels keeps the second from
 * starting until its time stamp is written, which costs a few microseconds per event: time every launch (k = 1) only
 * where that does not matter, and sample (k = 8, say) inside a region whose total time is being measured.
 * pasta_profile_read waits for the recorded events and returns, accumulated since the previous read:
 * out_ms[0..2] = device milliseconds of the tensor-core pass, the warp-shuffle pass and the merge,
 * out_launches[0..2] = how many launches of each were timed.  Both arrays are host memory.
 */
pasta_status_t pasta_profile_enable(pasta_pool_t *pool, int32_t on);
pasta_status_t pasta_profile_read(pasta_pool_t *pool, double *out_ms, int64_t *out_launches);

/* cudaError_t of the last failed CUDA call made by the library in this process (0 if none). */
int32_t pasta_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PASTA_H_ */
