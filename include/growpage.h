/*
 * growpage.h: C ABI of the GrowPage paged-decode library for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-step decode path of GrowPage (on-demand KV budgeting): every
 * request owns a page table over a shared pool of fixed-size KV pages; a decode step appends the
 * new token, runs GQA paged attention fused with the update of the two exponentially smoothed
 * query summaries (Sec. 3.2, Eq. 6), and, for requests whose allocation is now full, estimates
 * the short- and long-horizon attention working sets (Eq. 7, Eq. 8) and either acquires one
 * more page or evicts one page worth of tokens and compacts in place (Sec. 3.3, Eq. 9, Eq. 10).
 *
 * Conventions
 *   - All functions return an int status (GP_OK or a negative GP_ERR_*), never throw or abort.
 *   - "device pointer" = memory of the pool's CUDA device; "host pointer" = ordinary host memory.
 *   - The caller owns every buffer it passes.  The pool owns only the partition of the single
 *     device blob handed to gp_pool_create; the library never allocates device memory.
 *   - `stream` arguments are CUDA stream handles (cudaStream_t) passed as void*; NULL is the
 *     default stream.  Work is enqueued in stream order.
 *   - bf16 tensors are raw 16-bit patterns, row-major with the last index fastest.
 */
#ifndef GROWPAGE_H_
#define GROWPAGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define GP_OK             0
#define GP_ERR_INVALID   (-1)  /* bad argument, unknown or dead request id                        */
#define GP_ERR_NO_SLOT   (-2)  /* all max_requests summary slots are bound                        */
#define GP_ERR_NO_PAGES  (-3)  /* the free list or the per-request cap cannot supply the pages    */
#define GP_ERR_CUDA      (-4)  /* a CUDA call failed or a kernel reported an internal error       */
#define GP_ERR_STATE     (-5)  /* call not possible in the pool's current state                   */
#define GP_ERR_TOO_LARGE (-6)  /* problem exceeds the fixed scratch of gp_attention_noalloc        */

/* per-request action written by gp_decode_step (Sec. 3.3, Sec. 4.2) */
#define GP_ACT_NONE               0   /* no capacity boundary this step                           */
#define GP_ACT_GROW               1   /* Delta_t > tau: one page appended to the block table      */
#define GP_ACT_COMPRESS           2   /* Compress & Hold: one page worth of slots freed in place  */
#define GP_ACT_COMPRESS_FALLBACK  3   /* wanted to grow, cap or free list said no, compressed     */
#define GP_ACT_SHRINK             4   /* GP_POLICY_SHRINK: two pages worth of slots freed in place,
                                         the last page returned to the pool (Eq. 13)              */
#define GP_ACT_PENDING            5   /* asynchronous boundary work only: the request reached its capacity boundary
                                         with this step; its demand estimate, decision and compaction run beside the
                                         next step (gp_boundary_outcome tells the decision afterwards)             */
#define GP_ACT_HELD               6   /* asynchronous boundary work only: the request reached its boundary at the step
                                         before and sits this step out (not stepped, nothing of it read or written by
                                         the step; `out` row not written); it decodes again from the next step on   */
#define GP_ACT_STALLED          (-1)  /* full and neither a page nor copy-on-write targets could
                                         be had: page state untouched, the caller should release
                                         (preempt) the request; it is skipped while it stays full */
#define GP_ACT_SCRATCH          (-2)  /* the batch exceeds max_batch_tokens and this request's work did
                                         not fit the step's scratch: it was not stepped, its state is
                                         unchanged, and it can be stepped again in a later batch     */
#define GP_ACT_INVALID          (-3)  /* id out of range, not live, or repeated in the batch      */

typedef struct gp_pool gp_pool; /* opaque */

/* Capacity-control policies: the default and the controls of the paper's ablation ("Alternative
 * Capacity-Control Policies", with Eq. 13).  The fixed-budget control needs no policy of its own: a
 * threshold tau that Delta_t never exceeds (Delta_t <= 1) with initial_pages = the budget.
 *   DEMAND   grow iff Delta_t > tau (Sec. 3.2, Eq. 8)
 *   INVERSE  the reversed reading of the signal: grow iff Delta_t <= tau
 *   RANDOM   ignores Delta_t: Compress & Hold with probability p_compress, else grow.  The draw of request
 *            r whose step processes the token at absolute position pos is
 *            u = (mix(policy_seed + 0x9E3779B97F4A7C15 * (r + 1) + 0xBF58476D1CE4E5B9 * pos) >> 11) * 2^-53,
 *            arithmetic modulo 2^64, mix = the SplitMix64 finaliser; compress iff u < p_compress.
 *            Working sets and Delta_t are still computed and reported.
 *   SHRINK   Eq. 13, three actions: grow iff Delta_t > tau; Shrink iff Delta_t < shrink_below (and not
 *            growing); Compress & Hold in between.  A Shrink evicts two pages worth of the candidate set C
 *            per (layer, KV head) by the rule of Eq. 10 with the target |C| - 2b, compacts in place, and
 *            returns the request's last page to the pool: P pages become P - 1 with one page of free slots.
 *            It needs P >= 3 and (P - 1) * page_size >= min_capacity (the capacity left); otherwise the
 *            boundary is a Compress & Hold.  Shared pages are copied first as for a compression. */
#define GP_POLICY_DEMAND   0
#define GP_POLICY_INVERSE  1
#define GP_POLICY_RANDOM   2
#define GP_POLICY_SHRINK   3

#define GP_METRIC_TOP_P    0
#define GP_METRIC_ENTROPY  1

typedef struct gp_config {
  int32_t n_layers;          /* L                                                                  */
  int32_t n_q_heads;         /* H_q, a multiple of n_kv_heads; group size G = H_q/H_kv <= 8        */
  int32_t n_kv_heads;        /* H_kv                                                               */
  int32_t head_dim;          /* d_h: 64 or 128                                                     */
  int32_t page_size;         /* b: tokens per page, a power of two from 16 to 256 (the paper's default: 256).
                                The page is the unit in which capacity grows, local-quota blocks are formed
                                and slots are freed; n_pages, max_pages_per_req, initial_pages and every
                                page count the calls report are in these pages.  Inside, a page is a group
                                of page_size / 16 tiles of 16 tokens that are taken, shared and returned
                                together                                                            */
  int32_t max_requests;      /* M: summary slots = highest request id + 1 (App. D.1, default 512)  */
  int32_t max_pages_per_req; /* per-request page cap and page-table stride, >= 1; at most about 61 000
                                * 16 / page_size (the selection kernel keeps one bit per candidate token on
                                chip)                                                             */
  int32_t recent_window;     /* |R_t| protected newest tokens: 16 (the paper's default; equals the page at
                                page_size 16).  With a larger page the working sets of Eq. 7 are taken over
                                the history minus the newest page, the candidates of Eq. 10 are the history
                                minus these 16 tokens, each with its own softmax (App. D.1, Sec. 3.3)   */
  int32_t k_loc;             /* block-local retention quota of Eq. 10, at most page_size (default 4 = a
                                quarter of the default page of 16; the paper's 64 at its page of 256)  */
  int32_t host_staging;      /* 1: reserve staging so that gp_decode_step_host can be used         */
  int32_t policy;            /* GP_POLICY_*: how Delta_t becomes an action (default: demand)       */
  int32_t policy_seed;       /* GP_POLICY_RANDOM: seed of its counter-based draws                  */
  int32_t async_boundary;    /* 1: asynchronous boundary work (App. "Asynchronous Decoding and Compression"),
                                see gp_decode_step; default 0                                       */
  int32_t demand_metric;     /* GP_METRIC_TOP_P (default): working-set size of Eq. 7; GP_METRIC_ENTROPY: the
                                ablation's other metric, the view's attention entropy H over ln |C| in the
                                place of K / |C| (Delta_t is then a floating-point mean)               */
  int32_t overlap_slots;     /* synchronous mode, how the boundary work of a step (selection jobs, decisions,
                                compaction) is launched.  -2: one kernel behind the attention kernel, whose
                                thread blocks take their places as that kernel's leave and whose jobs start as
                                soon as the boundary requests' summary logits are reported complete (three
                                launches per step).  -1: a selection and a compaction kernel, one after the
                                other (four launches per step; what gp_step_end runs).  0 (default): -2 when
                                max_requests * n_layers * n_kv_heads <= 1024 (a step's boundary work is then a
                                few hundred jobs at most and the saved kernel boundary counts), else -1 (the
                                compaction of thousands of units wants its own, larger grid).  N > 0: as -2,
                                beside the attention kernel on N thread-block slots that kernel's grid gives
                                up.  Same results in every case                                        */
  int32_t async_slots;       /* asynchronous boundary work: thread blocks of the attention kernel's grid
                                given up so that the boundary kernel finds room on the SMs beside it;
                                0 = a default (64)                                                    */
  int32_t kv_shard_count;    /* pools that together hold the model's KV heads (Eq. 11's heads per GPU): this pool
                                has n_kv_heads of n_kv_heads * kv_shard_count, and Delta_t is a mean over all of
                                them (gp_decode_step_local / gp_decode_step_finish); default 1               */
  int32_t reserved;          /* keep 0                                                              */
  int64_t n_pages;           /* physical pages; one page id covers all layers and KV heads         */
  int64_t min_capacity;      /* GP_POLICY_SHRINK: tokens of capacity a Shrink must leave, default 1024 */
  int64_t max_batch_tokens;  /* bound on the summed sequence lengths of one decode batch, used to
                                size scratch; 0 = n_pages * page_size, which bounds it only while
                                no prompt pages are shared (a shared page counts once in the pool
                                and once per request in a batch).  A batch above the bound is not
                                an error: requests that do not fit report GP_ACT_SCRATCH          */
  int64_t max_boundary_tokens; /* bound on the summed candidate tokens of the requests that reach their
                                boundary in one step; sizes the boundary scratch (summary logits,
                                per-page softmax partials, large-set scores), 50 to 60 bytes per token,
                                layer and KV head.  0 = max_batch_tokens: every request of a batch may be
                                at its boundary (equal prompts reach it together).  On average one
                                request in sixteen is, so a large pool can set an eighth of that, at
                                least one request at the page cap.  More boundary tokens in a step are
                                not an error: the requests that do not fit report GP_ACT_SCRATCH, are
                                not stepped, and reach their boundary in a later step               */
  double  beta_s, beta_l;    /* Eq. 6, defaults 0.9 and 0.999                                      */
  double  top_p;             /* Eq. 7, default 0.99                                                */
  double  tau;               /* decision threshold, default 0                                      */
  double  rope_theta;        /* RoPE base (rotate-half pairing); 0 = no rotation                   */
  double  p_compress;        /* GP_POLICY_RANDOM: probability of Compress & Hold, default 0.7      */
  double  shrink_below;      /* GP_POLICY_SHRINK: Shrink iff Delta_t is under it, default -0.005    */
} gp_config;

/* Fills *cfg with the paper's defaults (Sec. 3.2, Sec. 5.1, App. B.2, App. D.1); the geometry
 * fields (layers, heads, pages) are set to zero and must be filled by the caller. */
int gp_config_default(gp_config* cfg);

/* Bytes of device memory a pool of this configuration needs; 0 if the configuration is invalid. */
size_t gp_pool_bytes(const gp_config* cfg);

/* Creates a pool inside `dev_blob` (device pointer, 256-byte aligned, at least gp_pool_bytes(cfg)
 * bytes, on CUDA device `device`).  The blob is cleared; every page starts on the free list (the
 * pool-wide stock of free pages that growth draws on, Sec. 4.2).  Synchronous.  The blob must outlive
 * the pool.  The only memory the library obtains itself is 64 bytes of page-locked host memory per pool
 * for the kernels' error word (see gp_pool_status). */
int gp_pool_create(const gp_config* cfg, void* dev_blob, size_t bytes, int device, gp_pool** out);

/* Frees the host-side handle.  Synchronises the device first.  The blob is left to its owner. */
int gp_pool_destroy(gp_pool* pool);

/* Admits a request: binds a summary slot to it at admission (App. D.1) and gives it its pages, the
 * leading ones possibly shared (App. D.2 prefix sharing).  Its first `n_shared_pages` pages are shared by reference
 * count with live request `share_from` (-1 for none), which must still hold them as untouched
 * full prompt pages.  The rest of the prompt, `n_tail` tokens, is copied from k_tail / v_tail:
 * device pointers, bf16 [L][n_tail][H_kv][d], keys already in cache form (post-RoPE).
 * The request starts with max(initial_pages, floor(n_prompt / b) + 1) pages.
 * On success *out_req receives the request id (the lowest free slot).  The summaries of the slot
 * are not cleared: the first decode step overwrites them.  Synchronises `stream`.
 * Errors, checked in this order: GP_ERR_INVALID (arguments; donor dead or with fewer shareable pages),
 * GP_ERR_STATE (between gp_step_begin and gp_step_end: the open step holds a snapshot of the free list),
 * GP_ERR_NO_SLOT, GP_ERR_NO_PAGES (nothing is changed in these cases). */
int gp_request_add(gp_pool* pool, int32_t share_from, int32_t n_shared_pages,
                   const void* k_tail, const void* v_tail, int32_t n_tail,
                   int32_t initial_pages, void* stream, int32_t* out_req);

/* One decode step for `n_req` requests (Sec. 3.2 - 3.3, App. D.1, App. D.2).
 *   dev_req_ids  device int32 [n_req]: request ids, each at most once
 *   q            device bf16 [L][n_req][H_q][d]: normalised queries before RoPE
 *   k, v         device bf16 [L][n_req][H_kv][d]: the new token's key (cache form) and value
 *   out          device fp32 [L][n_req][H_q][d]: attention output over all retained tokens,
 *                the new one included; rows of requests whose action is GP_ACT_INVALID, or that
 *                were already full on entry, are not written
 *   dev_actions  device int32 [n_req]: GP_ACT_* per request
 * q, k, v and out must be 16-byte aligned (the kernels move rows in 16-byte pieces), dev_req_ids and
 * dev_actions 4-byte aligned: GP_ERR_INVALID otherwise, nothing is launched.
 * Asynchronous on `stream`; nothing is read back to the host and the step's number lives on the device,
 * so (with profiling off, synchronous mode) a step over fixed buffers, or a sequence of steps, can be captured
 * into a CUDA graph and replayed any number of times.  The step's kernels are chained with
 * programmatic dependent launch.  Steps of one pool must be issued on one stream (or otherwise
 * serialised): they share scratch inside the blob.  See gp_set_early_plan for an option that lets
 * the step's first kernel start its work beside the last kernel of the step before.
 *
 * Asynchronous boundary work (gp_config.async_boundary = 1; App. "Asynchronous Decoding and Compression":
 * requests that compress leave the decode batch, the others keep decoding, the compressed ones rejoin a later
 * batch).  Here the whole boundary chain of a step (demand estimate, decision, page grant or eviction and
 * compaction) leaves the step's critical path: one kernel runs it beside the attention kernel of the next
 * step, on the same stream, on SM room that kernel leaves free (async_slots), and ends with it.  A request that
 * reaches its boundary at step t reports GP_ACT_PENDING at step t, is skipped at step t + 1 (GP_ACT_HELD if the
 * batch names it: the caller keeps that token's inputs for step t + 2), and decodes again from step t + 2 on, by
 * which time its pages are in their new state; a request whose boundary ended without pages reports
 * GP_ACT_STALLED then.  "Step" counts the pool's decode steps, whatever their batches.  Every token still sees
 * exactly the state the synchronous mode gives it; only the step at which it is decoded moves.  `dev_actions`
 * carries what is known when the step's own work ends (NONE, PENDING, HELD, STALLED, SCRATCH, INVALID); the
 * decisions are read with gp_boundary_outcome.  The boundary chain of the LAST step issued has not been launched
 * yet: gp_request_add, gp_release and the introspection calls launch it themselves (on the stream of that step);
 * a caller that looks at the pool's pages in any other way calls gp_async_join first.  Early planning does not
 * apply, the layer-by-layer calls are not available in this mode (GP_ERR_STATE from gp_step_begin), and its steps
 * are numbered on the host: do not replay them from a CUDA graph. */
int gp_decode_step(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req,
                   const void* q, const void* k, const void* v,
                   void* out, int32_t* dev_actions, void* stream);

/* Asynchronous boundary work: launches the boundary chain of the last decode step on `stream` if it is still
 * outstanding (it otherwise rides behind the next step's attention kernel); a no-op in the synchronous mode. */
int gp_async_join(gp_pool* pool, void* stream);

/* The decision taken at the request's most recent capacity boundary (GP_ACT_GROW, GP_ACT_COMPRESS,
 * GP_ACT_COMPRESS_FALLBACK, GP_ACT_SHRINK, GP_ACT_STALLED; GP_ACT_NONE if it has not reached one) and the
 * number of that decode step, counted from 0 over the pool's decode steps (host outputs, either may be NULL).
 * Synchronises the device.  In the synchronous mode it repeats what dev_actions said. */
int gp_boundary_outcome(gp_pool* pool, int32_t req, int32_t* action, int64_t* step);

/* The same step, layer by layer, for a model's forward pass, where layer l + 1's query exists only after
 * layer l's attention output (the paper's setting: attention and the summary update run inside every
 * layer, the capacity decision once per step, Sec. 3.2, Sec. 4.1):
 *   gp_step_begin   validates the batch and plans the step (what gp_decode_step does first);
 *   gp_attn_layer   for one layer: append, attention, summary update and, for requests at their
 *                   boundary, the summary logits; q [n_req][H_q][d], k, v [n_req][H_kv][d] bf16 and
 *                   out [n_req][H_q][d] fp32 are this layer's tensors (device pointers); when the call's
 *                   work has run, `out` is complete.  Every layer exactly once, in any order;
 *   gp_step_end     working sets, decisions, allocation, compaction; writes `dev_actions`.
 * Same ids, n_req, alignment and stream discipline as gp_decode_step; between gp_step_begin and gp_step_end
 * no other step of the pool may be issued, and no request admitted or released (GP_ERR_STATE: the open step
 * holds a snapshot of the free list).  A layer given twice is refused (GP_ERR_STATE), and so is gp_step_end
 * while layers are missing; gp_step_abort leaves an open step without committing it: no request has advanced,
 * rows the finished layers appended lie beyond the occupied slots and are overwritten by the next step.  Actions, page state, retained sets and summaries
 * equal gp_decode_step's bit for bit; the attention outputs agree to fp32 rounding (long requests
 * are cut into work items of different sizes, so partial results are merged in another order). */
int gp_step_begin(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, int32_t* dev_actions,
                  void* stream);
int gp_attn_layer(gp_pool* pool, int32_t layer, const int32_t* dev_req_ids, int32_t n_req,
                  const void* q, const void* k, const void* v, void* out, void* stream);
int gp_step_end(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, int32_t* dev_actions,
                void* stream);
int gp_step_abort(gp_pool* pool);

/* gp_attn_layer with the model's query / key normalisation fused in (Sec. 3.2: the summaries follow the query
 * after its normalisation and before its rotation).  q_raw [n_req][H_q][d] and k_raw [n_req][H_kv][d] are the
 * projections' bf16 outputs; per head, x <- x / sqrt(mean(x^2) + eps) * weight (q_weight, k_weight: device fp32
 * [d], one learned weight per element of the head dimension).  The normalised query, rounded to bf16, is the
 * query of the layer (attention rotates it when RoPE is on, the summaries take it as it is); the normalised key
 * is rotated to its position when RoPE is on and rounded to bf16 in that cache form.  Arithmetic in fp64, rounded
 * double -> float -> bf16.  Otherwise as gp_attn_layer (v in cache form, same alignment rules; the weights 4-byte
 * aligned). */
int gp_attn_layer_qknorm(gp_pool* pool, int32_t layer, const int32_t* dev_req_ids, int32_t n_req,
                         const void* q_raw, const void* k_raw, const void* v, const float* q_weight,
                         const float* k_weight, double eps, void* out, void* stream);

/* The step of a pool that holds a part of the model's KV heads (Eq. 11: "query heads per GPU"; every GPU of a
 * tensor-parallel group has its own pool over the same requests, page ids and batches, with n_kv_heads of the
 * model's n_kv_heads * kv_shard_count heads).  Scoring, working sets, selection and compaction are per (layer, KV
 * head); the one coupling is the mean of Eq. 8, i.e. two integers per boundary request:
 *   gp_decode_step_local   plan, attention, selection jobs (arguments as gp_decode_step, this pool's heads only);
 *                          leaves, per boundary request in batch order, the sums of K^S and of K^L over this
 *                          pool's units in the device array gp_shard_sums returns (int32 [max_requests][2],
 *                          zero past the step's boundary requests);
 *   (the caller adds the arrays of all pools up, element by element, in place: one all-reduce of
 *    2 * max_requests int32 on `stream`, e.g. ncclAllReduce with ncclSum; nothing to do for a single pool)
 *   gp_decode_step_finish  decisions from the completed sums (every pool takes the same ones, on its replica of the
 *                          page tables and the free list), allocation, compaction; writes `dev_actions`.
 * Between the two calls the pool accepts nothing else (GP_ERR_STATE).  Synchronous mode and the Top-p metric only
 * (the entropy variant would sum doubles, in an order that differs from a single pool's).  With one pool the pair
 * gives exactly what gp_decode_step gives. */
int gp_decode_step_local(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req,
                         const void* q, const void* k, const void* v,
                         void* out, int32_t* dev_actions, void* stream);
int gp_shard_sums(gp_pool* pool, int32_t** dev_sums, int64_t* n_ints);
int gp_decode_step_finish(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, int32_t* dev_actions,
                          void* stream);

/* As gp_decode_step with HOST pointers: brings the inputs to staging inside the blob, runs the
 * step, delivers `out` and `actions` and synchronises `stream`.  When the four input buffers are
 * page-locked, mapped host memory (cudaHostAlloc / cudaHostRegister: "pinned") and q, k, v are
 * 16-byte aligned, one kernel fetches them over the bus; otherwise four copies do.  When
 * `out` and `actions` are pinned, the kernels write them directly while they run; otherwise the
 * results are staged on the device and copied back.
 * Needs host_staging = 1 at creation, else GP_ERR_STATE.  After its synchronisation the call looks at the
 * kernels' error word and returns GP_ERR_CUDA when a kernel reported an internal error (gp_pool_status). */
int gp_decode_step_host(gp_pool* pool, const int32_t* host_req_ids, int32_t n_req,
                        const void* q, const void* k, const void* v,
                        void* out, int32_t* actions, void* stream);

/* The same step without the synchronisation at the end: everything is enqueued and the call returns.  With
 * page-locked buffers the copy engine moves the inputs in on a stream of the pool's own, beside the step before on
 * `stream` (two staging sets), and the kernels write the results into the caller's buffers as they run: a serving
 * loop issues step t + 1 while step t runs and reads the results of step t from a second pair of result buffers
 * meanwhile; the GPU never waits for the host's wake-up and launches between steps.  The caller's input buffers
 * must stay as they are, and `out` and `actions` are not to be read, until gp_decode_step_host_wait has returned for
 * the call (calls are waited for in the order they were made; at most two can be outstanding: a third call first
 * waits for the oldest itself) or `stream` has been synchronised. */
int gp_decode_step_host_async(gp_pool* pool, const int32_t* host_req_ids, int32_t n_req,
                              const void* q, const void* k, const void* v,
                              void* out, int32_t* actions, void* stream);

/* Waits until the results of the oldest gp_decode_step_host_async call not yet waited for are in the caller's
 * buffers (a device-wide synchronisation when there is none), then looks at the kernels' error word: GP_OK, or
 * GP_ERR_CUDA when a kernel reported an internal error (gp_pool_status). */
int gp_decode_step_host_wait(gp_pool* pool);

/* Ends a request: every page of its table loses one reference and returns to the free list at
 * zero; the summary slot is recycled without clearing (App. D.1).  Asynchronous on `stream`.
 * GP_ERR_STATE between gp_step_begin and gp_step_end. */
int gp_release(gp_pool* pool, int32_t req, void* stream);

/* Internal errors reported by the kernels (a bounded wait that ran out, a failed bounds check, free-list
 * accounting gone wrong): GP_OK, or GP_ERR_CUDA with the bits in *error_bits (may be NULL).  The kernels set
 * the bits in a word of page-locked host memory, so this call neither synchronises nor copies; it reflects
 * the work that has completed.  gp_decode_step is asynchronous and cannot report them itself:
 * call this after synchronising its stream.  The bits are sticky for the life of the pool:
 *   1 a bounded wait inside the attention kernel gave up   2 free-list accounting out of range
 *   4 an index failed a bounds check (the access was skipped)   8 a bounded wait inside the compaction kernel gave up
 * (bits 7 and up say which wait of the attention kernel it was). */
int gp_pool_status(gp_pool* pool, int32_t* error_bits);

/* Text for a status code. */
const char* gp_strerror(int status);

/* ---- introspection (host outputs; each call synchronises the device) ------------------------ */

/* Pages P, occupied slots n, absolute position pos and the page table (host int32, room for
 * max_pages_per_req entries; may be NULL) of a live request. */
int gp_debug_request(gp_pool* pool, int32_t req, int32_t* P, int32_t* n, int64_t* pos, int32_t* page_table);

/* Pages and occupied slots of every request slot at once: host int32 [max_requests] each (either may be
 * NULL); slots that are not live read 0. */
int gp_debug_state(gp_pool* pool, int32_t* P, int32_t* n);

/* Original token index of every occupied slot of one (layer, KV head) stream, in slot order:
 * host int32 [n].  This is the retained-index set of Sec. 3.3. */
int gp_debug_retained(gp_pool* pool, int32_t req, int32_t layer, int32_t kv_head, int32_t* token_ids);

/* K and V rows of the occupied slots of one (layer, KV head) stream in slot order:
 * host bf16 [n][d] each (either may be NULL). */
int gp_debug_kv(gp_pool* pool, int32_t req, int32_t layer, int32_t kv_head, void* k_rows, void* v_rows);

/* The two summaries of a request: host double [L][2][H_q][d], short then long (Eq. 6, Eq. 11). */
int gp_debug_summaries(gp_pool* pool, int32_t req, double* out);

/* Working-set sizes of the request's most recent boundary: host int32 [L][H_kv] each, and
 * Delta_t (Eq. 7, Eq. 8). */
int gp_debug_boundary(gp_pool* pool, int32_t req, int32_t* K_S, int32_t* K_L, double* delta);

/* Entropy metric only: the entropies of the two views at the request's most recent boundary, host double
 * [L][H_kv] each (either may be NULL). */
int gp_debug_entropy(gp_pool* pool, int32_t req, double* H_S, double* H_L);

/* Free pages, per-page reference counts (host int32 [n_pages], may be NULL) and event counters:
 * [0] grow [1] compress [2] fallback-compress [3] stalled [4] copy-on-write pages
 * [5] decode steps [6] tokens decoded [7] internal error bits (0 when healthy)
 * [8] (layer, head, token) rows rewritten by compaction [9] candidate tokens scored at boundaries
 * [10] Shrink events (not counted under [1]) [11] reserved. */
int gp_debug_pool(gp_pool* pool, int64_t* n_free, int32_t* refcounts, int64_t counters[12]);

/* ---- measurement ----------------------------------------------------------------------------- */

#define GP_N_KERNELS 4   /* plan, attention (+ boundary logits), selection + decision, compaction; with the boundary
                            work in one kernel (overlap_slots >= 0, the default) the third entry is that kernel and
                            the fourth stays zero */

/* With profiling on, every kernel of gp_decode_step is bracketed by CUDA events on the step's
 * stream (this serialises nothing but adds event records).  Off by default. */
int gp_set_profiling(gp_pool* pool, int32_t enable);

/* Early planning (off by default).  The first kernel of gp_decode_step is launched as a programmatic
 * dependent of whatever kernel precedes it on the stream.  With the option off it waits for that
 * kernel to end before it reads anything: always safe.  With it on, it reads dev_req_ids and q, plans
 * the step and updates the query summaries before that wait, beside the compaction kernel of the
 * step before, and waits only before it looks at the free list.  That is correct only if
 * dev_req_ids and q are complete in memory by the time the preceding kernel on the stream lets
 * its dependents be scheduled: true when they were produced by copies or by kernels that do not
 * signal programmatic launch completion (or when nothing was enqueued since the step before);
 * not true when the query projection enqueued just before the step signals completion ahead of its
 * stores.  gp_decode_step_host always plans early (its inputs arrive by copies).  The
 * layer-by-layer calls are not affected. */
int gp_set_early_plan(gp_pool* pool, int32_t enable);

/* Synchronises, then returns the accumulated device time in milliseconds and the launch count of
 * each kernel since profiling was switched on (host arrays of GP_N_KERNELS), and resets them. */
int gp_get_kernel_times(gp_pool* pool, float* ms, int64_t* launches);

/* Kernels launched by this pool since creation (all calls). */
int64_t gp_launch_count(gp_pool* pool);

/* ---- test support --------------------------------------------------------------------------------------------- */

/* Every wait of one thread block for another inside the kernels is bounded: after a number of iterations it gives
 * up, sets an error bit (gp_pool_status) and the kernel runs to its end, with wrong results for the work concerned
 * but without hanging and with the pool's page accounting intact.  This call lets a test see that happen without
 * any fault: `what` names hand-overs that are then simply not made (1 the attention kernel's first thread block
 * never completes its second work item for its consumer warps; 2 the first chunk of every compaction unit never
 * says that its sources are read; 4 the deciding thread block of the boundary kernel never tells the others; 8 the
 * attention kernel never reports a boundary unit's summary logits complete; 0 none; and, not a withheld hand-over
 * but a switch for tests: 16 the compaction claims a whole unit per ticket however few units there are),
 * `spin_limit` the iterations after which waits give up (0 = the default, 2^21).  Applies to the steps issued
 * after it.  The error bits stay set; results of such a pool are not meaningful afterwards. */
int gp_test_withhold(gp_pool* pool, int32_t what, int32_t spin_limit);

/* ---- attention without any allocation ------------------------------------------------------------ */

#define GP_NOALLOC_SPLITS   8      /* parts a request's tokens are split into                           */
#define GP_NOALLOC_MAX_ROWS 2048   /* limit on n_req * n_q_heads                                        */

/* (The paper has no counterpart of this call; it exists for deployments, not for the method.)
 *
 * GQA decode attention over plain, un-paged K/V, for callers that cannot give the library any memory to
 * work in and must not have it allocate: for instance a server that handed every byte of the GPU to its KV
 * pool at start-up, or a host that loads this library as a plug-in and forbids allocator calls from it.
 * The split-KV partial results go to an 8.5 MB array that is part of the library image; each GPU that loads
 * the library holds that array until the process exits.
 *
 *   q     device bf16 [n_req][n_q_heads][d]
 *   k, v  device bf16 [n_req][n_kv_heads][max_len][d], rows in plain order (no page layout, no swizzle)
 *   lens  device int32 [n_req]: tokens of each request, 1..max_len (values above max_len are clipped;
 *         a request with lens <= 0 attends to nothing and gets an output row of zeros)
 *   out   device fp32 [n_req][n_q_heads][d]: softmax(q.K/sqrt(d)).V per query head, KV head g / G
 *
 * Limits: d is 64 or 128, G = n_q_heads / n_kv_heads <= 8, n_req * n_q_heads <= GP_NOALLOC_MAX_ROWS;
 * beyond that the call returns GP_ERR_TOO_LARGE and does nothing.  It calls no cudaMalloc, cudaFree or
 * other allocating routine.  The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress) with that device current; make that first call outside any stream capture.
 * All calls share the one array and nothing in it has to be cleared (every slot a call reads it has
 * written first), but two calls that overlap on the GPU, e.g. on different streams, race on it:
 * serialise them.  Asynchronous on `stream`. */
int gp_attention_noalloc(const void* q, const void* k, const void* v, const int32_t* lens, int32_t n_req,
                         int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t max_len,
                         void* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GROWPAGE_H_ */
