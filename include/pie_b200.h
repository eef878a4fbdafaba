/*
 * pie_b200.h - C ABI of the B200-native batched `forward` attention handler.
 *
 * The calls follow the inference-layer handler API of the Pie paper (Table 1: alloc_kvpage,
 * dealloc_kvpage, copy_kvpage, forward; Section 4.1 "Resources" for KvPages; Section 4.2
 * "Forward API" for masks and positions; Section 5.2 for the batch the control layer hands
 * to a handler).  One `forward` batch = many inferlets' calls coalesced: per request the new
 * K/V rows are appended to its output KvPages and every query token attends over the
 * request's page list under its mask.
 *
 * Conventions
 *   - Every function returns PIE_OK (0) or a negative pie_status.  Nothing throws, aborts or
 *     traps on the device.  pie_strerror() names a status.
 *   - "host" / "device" below says where a pointer must live.  Index arrays given to the
 *     planner are host memory, read during the call and not retained.
 *   - Device work is enqueued on the caller's stream (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream) and is asynchronous unless stated otherwise.  Ordering
 *     between calls is stream order (the paper's command-queue order).
 *   - The KvPage pool is owned by the library; its layout is private.  Q / K_new / V_new /
 *     output / LSE buffers are owned by the caller.
 *   - Element type: bf16 or fp32 for Q, K, V and the output; LSE is always fp32.
 *   - Threads: a context (and its plans and scheduler objects) must not be used from two host
 *     threads at the same time.  A plan owns the scratch of its split partials, so two
 *     pie_forward calls on the SAME plan must not overlap on the GPU (same stream order is fine);
 *     different plans may run concurrently on different streams.
 */
#ifndef PIE_B200_H_
#define PIE_B200_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum pie_status {
  PIE_OK = 0,
  PIE_ERR_INVALID = -1,         /* bad argument (null pointer, size out of range, bad config)   */
  PIE_ERR_NO_PAGES = -2,        /* pool exhausted; nothing was allocated                        */
  PIE_ERR_BAD_PAGE = -3,        /* page id out of range, not allocated, or freed twice          */
  PIE_ERR_CONFLICT = -4,        /* two batched calls touch the same KvPage slot, one writing    */
  PIE_ERR_BATCH_TOO_LARGE = -5, /* more requests / query tokens than the configured maximum     */
  PIE_ERR_MASK = -6,            /* mask range size != q_len * kv_len, or a byte not 0/1         */
  PIE_ERR_CUDA = -7,            /* a CUDA runtime call failed (see pie_last_cuda_error)         */
  PIE_ERR_NO_DEVICE = -8,       /* the context was created host-only (device = -1)              */
  PIE_ERR_UNSUPPORTED = -9,     /* shape / type combination the kernels do not cover            */
  PIE_ERR_DEVICE_TIMEOUT = -10  /* a bounded device-side wait gave up (results invalid)         */
} pie_status;

enum { PIE_DTYPE_BF16 = 0, PIE_DTYPE_F32 = 1 };

/* Start-up configuration (Section 5.2 "Resource management": the pool is sized once at
 * start-up; Section 5.2 "Batch scheduler": the backend has a maximum batch size). */
typedef struct pie_config {
  int32_t num_pages;        /* KvPages in the pool                                    */
  int32_t page_size;        /* tokens per KvPage: 8, 16 or 32 (Section 4.1)            */
  int32_t num_q_heads;      /* H_q                                                    */
  int32_t num_kv_heads;     /* H_kv, divides H_q; kv head of q head h is h / (H_q/H_kv) */
  int32_t head_dim;         /* D: 64 or 128                                           */
  int32_t dtype;            /* PIE_DTYPE_BF16 or PIE_DTYPE_F32                         */
  int32_t max_requests;     /* largest batch (requests) pie_plan_forward accepts       */
  int32_t max_query_tokens; /* largest total of query tokens in one batch              */
  int32_t device;           /* CUDA device ordinal; -1 = host-only context (planner,
                               allocator and validation work; device calls return
                               PIE_ERR_NO_DEVICE)                                      */
  float rope_theta;         /* 0: Q / K arrive position-encoded (default).  > 0: rotary
                               position embedding inside the path with this base (Llama-3:
                               500000): forward rotates Q for the attention and rotates each
                               new K row before storing it, at the token's position
                               (rotate-half form: pairs (i, i + D/2), angle pos * theta^(-2i/D)).
                               `forward` "operates based on explicit sequence positions"
                               (Section 4.2); the paper gives no formula.               */
} pie_config;

typedef struct pie_ctx pie_ctx;
typedef struct pie_plan pie_plan;

const char* pie_strerror(int status);
/* Text of the last CUDA error seen by this context ("" if none).  Host. */
const char* pie_last_cuda_error(const pie_ctx* ctx);

/* Create a context and its KvPage pool (Section 5.3: the inference layer holds the physical
 * memory).  Allocates num_pages * page_size * 2 * H_kv * D elements on the device and
 * zero-fills them once.  *out is set only on success.  Synchronous. */
int pie_create(const pie_config* cfg, pie_ctx** out);
/* Free the pool and everything the context owns.  Plans must be destroyed first. */
int pie_destroy(pie_ctx* ctx);

/* alloc_kvpage / dealloc_kvpage (Table 1).  Host free list; no device work.
 * pie_alloc_kvpages writes n page ids to out_ids (host) or fails with PIE_ERR_NO_PAGES and
 * allocates nothing (the caller applies the first-come-first-served policy of Section 5.2).
 * Page contents are NOT cleared.  pie_dealloc_kvpages rejects ids that are out of range or
 * not allocated (PIE_ERR_BAD_PAGE) without freeing any. */
int pie_alloc_kvpages(pie_ctx* ctx, int32_t n, int32_t* out_ids);
int pie_dealloc_kvpages(pie_ctx* ctx, int32_t n, const int32_t* ids);
/* Free pages, counting the pages that forwards of requests without output KvPages (no_store) have
 * borrowed: both pie_num_free_kvpages and, when the free list is short, pie_alloc_kvpages wait for such
 * forwards to finish before they answer. */
int pie_num_free_kvpages(const pie_ctx* ctx, int32_t* out);

/* Write / read whole pages in the canonical layout  K[n][page_size][H_kv][D], V[same]
 * (the save / restore side of export_kvpage / import_kvpage, Table 1; also how tests install
 * context).  ids: host.  K, V: host memory if on_device == 0 (the call then synchronises the
 * stream before returning), device memory if on_device == 1 (asynchronous). */
int pie_kvpage_write(pie_ctx* ctx, int32_t n, const int32_t* ids, const void* K, const void* V,
                     int on_device, void* stream);
int pie_kvpage_read(pie_ctx* ctx, int32_t n, const int32_t* ids, void* K, void* V,
                    int on_device, void* stream);

/* copy_kvpage (Table 1: "copy KV cache contents at token-level").  For op k, rows
 * [src_off[k], src_off[k]+ntok[k]) of page src[k] are copied (K and V, all heads, bit for bit)
 * to rows starting at dst_off[k] of page dst[k].  All arrays: host, n entries.
 * Errors: ranges outside a page or unallocated pages (PIE_ERR_BAD_PAGE / PIE_ERR_INVALID);
 * two ops writing the same slot, or an op reading a slot another op of the same call writes
 * (PIE_ERR_CONFLICT).  Asynchronous on `stream`. */
int pie_copy_kvpage(pie_ctx* ctx, int32_t n, const int32_t* src, const int32_t* dst,
                    const int32_t* src_off, const int32_t* dst_off, const int32_t* ntok,
                    void* stream);

/* mask_kvpage (Table 1: "masks the KV cache in a token-level manner"; used by the attention-sink,
 * windowed- and hierarchical-attention inferlets of Section 7).  Sets the persistent visibility
 * mask of n pages: bit s of masks[k] set = slot s of page ids[k] may be attended to.  The mask
 * stays with the page until it is set again; allocating a page resets it to all-visible.
 * In forward a position is attended iff the batch mask (explicit or inferred) allows it AND its
 * page-mask bit is set; a page none of whose slots is visible to a request is never fetched
 * (the same as leaving the page out of the list, Section 4.2).  Host bookkeeping only; it
 * affects plans made afterwards.  ids, masks: host, n entries.  PIE_ERR_BAD_PAGE if a page is
 * out of range or not allocated (nothing is changed then). */
int pie_mask_kvpage(pie_ctx* ctx, int32_t n, const int32_t* ids, const uint32_t* masks);

/* One coalesced `forward` batch as the control layer hands it over (Section 5.2).
 * Request r has q_len = qo_indptr[r+1]-qo_indptr[r] >= 1 new tokens and the page list
 * page_indices[page_indptr[r] .. page_indptr[r+1]) (input KvPages followed by output KvPages;
 * ids may repeat across requests: shared pages).  last_page_len[r] in [1, page_size] counts the
 * filled slots of the last page AFTER the append, so the context length is
 * kv_len = (num_pages_r - 1) * page_size + last_page_len[r] and the new tokens occupy
 * positions kv_len - q_len .. kv_len - 1.
 * Mask (Section 4.2): mask_indptr == NULL, or an empty range for request r, means "infer from
 * positions": token i attends to positions <= kv_len - q_len + i.  Otherwise
 * mask[mask_indptr[r] .. mask_indptr[r+1]) holds q_len * kv_len bytes, row major, 1 = attend,
 * 0 = masked; it is the complete specification (not combined with causality) and is shared by
 * all heads.  A row with no allowed position yields output 0 and LSE = -inf. */
typedef struct pie_batch_desc {
  int32_t num_requests;
  const int32_t* qo_indptr;     /* [R+1], qo_indptr[0] == 0                       */
  const int32_t* page_indptr;   /* [R+1], page_indptr[0] == 0                     */
  const int32_t* page_indices;  /* [page_indptr[R]]                               */
  const int32_t* last_page_len; /* [R]                                            */
  const int64_t* mask_indptr;   /* [R+1] or NULL: request r's explicit mask is mask[mask_indptr[r] ..
                                   mask_indptr[r+1]); an empty range = causal mask inferred from positions */
  const uint8_t* mask;          /* q_len x kv_len bool bytes (1 = attend) per request with a mask, or NULL;
                                   packed bits instead with PIE_PLAN_MASK_BITS                             */
  uint32_t flags;               /* PIE_PLAN_* below, 0 for the default path       */
  const int32_t* positions;     /* [T] explicit position of every new token, or NULL for the
                                   default kv_len - q_len + i.  Used only when the context
                                   was created with rope_theta > 0.                 */
  const int32_t* out_len;       /* [R] or NULL.  Section 4.2: a forward call fills output Embeds
                                   and / or output KvPages.  Request r produces outputs (out, lse)
                                   for its LAST out_len[r] query tokens only, 0 <= out_len[r] <=
                                   q_len; 0 = its rows are stored and nothing is attended.  All
                                   q_len rows are appended and keep their positions and mask rows;
                                   out / lse rows of tokens without output are left untouched.
                                   NULL = every token produces an output.             */
  const uint8_t* no_store;      /* [R] or NULL.  Section 4.2: a forward call may have NO output KvPages
                                   (`forward(kv, iemb[-1:], oemb)`, `forward([], iemb, [], oemb)` in the
                                   paper's listing).  no_store[r] != 0: request r's new rows take part in
                                   the attention as the last q_len positions of its context but are not
                                   written to its pages.  For such a request the page list and
                                   last_page_len describe the EXISTING context only (an empty page range =
                                   none; last_page_len is then ignored) and an explicit mask is
                                   [q_len x (existing + q_len)].  The plan borrows pages from the context's
                                   free list for its lifetime (PIE_ERR_NO_PAGES if too few are free; the
                                   caller's pages are never written).  When the plan is destroyed the
                                   pages return to the free list behind its latest forward: they are held
                                   until the work enqueued on that forward's stream has finished.          */
} pie_batch_desc;

enum {
  PIE_PLAN_FORCE_SIMPLE = 1u,   /* run every request through the plain CUDA-core kernel   */
  PIE_PLAN_NO_TENSOR_TILES = 2u, /* keep prefill / tree requests off the tcgen05 tile path (ignored with 8-token pages) */
  PIE_PLAN_NO_CASCADE = 4u,     /* never attend a shared prefix once for a group of requests */
  PIE_PLAN_CASCADE_ALWAYS = 8u, /* cascade every shared prefix, however small the saving (tests, tuning) */
  PIE_PLAN_MASK_BITS = 16u      /* `mask` holds bits, not bool bytes: for a request with a mask, q_len rows of
                                   ceil(kv_len / 32) uint32 words (bit j of the row = position j, LSB first; bits
                                   past kv_len are ignored), `mask` 4-byte aligned, mask_indptr counting WORDS */
};

typedef struct pie_plan_info {
  int32_t num_requests;
  int32_t num_query_tokens;
  int32_t num_split_items;      /* work items of the split-KV (decode) kernel      */
  int32_t num_tile_items;       /* work items of the prefill / tree tile kernel    */
  int32_t num_simple_rows;      /* (token, head) rows given to the plain kernel    */
  int32_t num_merge_groups;     /* groups whose split partials the merge combines  */
  int32_t launches;             /* kernels one pie_forward enqueues                */
  int32_t side_by_side_sms;     /* SMs given to the row-tile kernel when it runs next to the decode kernel (0: one after the other) */
  int32_t split_unit_kv_heads;  /* adjacent kv heads that one split-KV work item covers: 1, or 2 (one copy of twice the size per page) */
  int32_t reserved0;
  int64_t kept_pages;           /* pages left in the lists after dropping fully masked ones */
  int64_t mask_words;           /* 32-bit words of packed mask                     */
  int64_t workspace_bytes;      /* device scratch for split partials               */
} pie_plan_info;

/* Batch planner (host side of `forward`): validates the batch, infers or bit-packs the masks
 * (LSB first, 32-bit words, rows padded to 128 bits), drops pages no query row attends to,
 * splits the work across SMs, and uploads the result.  Errors: PIE_ERR_BAD_PAGE (id out of
 * range / not allocated), PIE_ERR_INVALID (last_page_len outside [1,page_size], q_len < 1,
 * kv_len < q_len, non-monotone indptr), PIE_ERR_CONFLICT (two requests append to the same
 * slot, or a request reads a slot that a LATER request of the batch appends: the
 * vertical-batching rule of Section 5.2; reading rows an EARLIER request appends is legal,
 * because the whole batch is appended before any request attends),
 * PIE_ERR_BATCH_TOO_LARGE, PIE_ERR_MASK.  *out is set only on success.  The upload uses
 * `stream`; the call returns after it completed. */
int pie_plan_forward(pie_ctx* ctx, const pie_batch_desc* batch, void* stream, pie_plan** out);
/* Ends the plan's life.  The context keeps a few destroyed plans - host arrays, pinned upload
 * image and device arrays - and pie_plan_forward reuses them, so a loop that plans every step
 * stops allocating after its first steps (no cudaMalloc, no cudaFree and its device-wide
 * synchronisation per batch).  The call does not wait: it marks the point behind the plan's
 * latest pie_forward on that forward's stream, and the reuse waits for that point.  Destroy a
 * plan only when no captured graph that holds its forward will be launched again, and before
 * the stream of its latest forward is destroyed.  pie_destroy releases the kept plans. */
int pie_plan_destroy(pie_plan* plan);
int pie_plan_get_info(const pie_plan* plan, pie_plan_info* out);

/* Planner introspection for tests: copy one of the plan's host-side arrays into buf (host).
 * which: 0 = packed mask words (uint32), 1 = kept page list (int32 pairs: physical id,
 * logical page | 0x80000000 if the page needs mask evaluation), 2 = append destinations
 * (int32 per query token: page * page_size + slot), 3 = the plan's whole upload image (request
 * records, kept pages, masks, append destinations, work items, share boundaries, merge groups
 * and counters in device layout, gaps zeroed; size a multiple of 4), 4 / 5 = the work items of
 * the split-KV / row-tile launch (16 int32 each: request, kv head, first row, rows, first and
 * end kept page, partial slot or -1, six fields of the request record, flags - for row-tile
 * items flags >> 8 = leading pages every row of the tile sees in full -, mask word offset as two
 * words).  *out_bytes receives the
 * array size; data is copied only if cap_bytes is large enough. */
int pie_plan_debug_read(const pie_plan* plan, int which, void* buf, int64_t cap_bytes,
                        int64_t* out_bytes);

/* forward (Table 1; Section 4.2).  Device pointers: q [T][H_q][D], k_new / v_new
 * [T][H_kv][D], out [T][H_q][D] in the configured element type, lse [T][H_q] fp32 (natural log
 * of the sum of exp of the scaled scores).  Enqueues on `stream`: append of the new rows into
 * the pool, then attention (scale 1/sqrt(D)) reading the pool, then the merge of split
 * partials.  The plan may be reused for repeated calls with the same batch structure.
 * All five pointers must be 16-byte aligned (rows are moved in 16-byte pieces); an `out` that
 * is 32-byte aligned is written with wider stores, with identical results. */
int pie_forward(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new,
                const void* v_new, void* out, float* lse, void* stream);

/* The same call for callers whose tensors live in HOST memory: plans the batch, copies
 * q / k_new / v_new to the device, runs pie_forward, copies out / lse back and synchronises.
 * All pointers host (pinned memory makes the copies asynchronous with respect to the host,
 * but the call still returns only after the results arrived). */
int pie_forward_host(pie_ctx* ctx, const pie_batch_desc* batch, const void* q, const void* k_new,
                     const void* v_new, void* out, float* lse, void* stream);

/* get_next_dist from the logits on (Table 1 `get_next_dist`; Section 4.2 "Sample API": the next-token
 * probability distribution, truncated to the top-K tokens, K configurable, 256 by default).  The LM head
 * that turns output Embeds into logits is a plain GEMM and not part of this library.
 *   logits    device, [n_rows] rows of `vocab` entries, `row_stride` entries apart (>= vocab), of type
 *             `dtype` (PIE_DTYPE_BF16 or PIE_DTYPE_F32; independent of the context's KV type).  16-byte
 *             aligned rows are read with vector loads, others entry by entry.  Every row needs at
 *             least one finite entry; -inf entries get probability 0.
 *   top_k     1 .. 1024 and <= vocab.
 *   out_ids   device, [n_rows][top_k] int32: the top_k most probable tokens of every row in order of
 *             descending probability; equal logits in order of ascending token id (so the result is unique).
 *   out_probs device, [n_rows][top_k] float: their probabilities in the softmax over the WHOLE vocabulary
 *             (not renormalised over the kept tokens).
 * Asynchronous on `stream`; buffers are the caller's.  Errors: PIE_ERR_INVALID (sizes, type, null
 * pointers), PIE_ERR_NO_DEVICE, PIE_ERR_CUDA. */
int pie_get_next_dist(pie_ctx* ctx, const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                      int64_t row_stride, int32_t top_k, int32_t* out_ids, float* out_probs, void* stream);

/* Device-side status word: 0, or PIE_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel
 * gave up since the last call.  Synchronises `stream`, reads and clears the word. */
int pie_get_last_device_status(pie_ctx* ctx, void* stream, int* out);

/* Test hook for the failure path.  Every wait inside the kernels is bounded: after about a second it
 * gives up, sets the status word and the kernel drains.  This call enqueues a one-warp kernel whose only
 * wait can never complete, so that a test can watch exactly that: pie_get_last_device_status then returns
 * PIE_ERR_DEVICE_TIMEOUT once, and the context keeps working. */
int pie_debug_bounded_wait(pie_ctx* ctx, void* stream);

/* forward for callers that must not allocate device memory.  (The paper has no counterpart:
 * this entry point exists for the embedding application, not for the method.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they run a batch: code
 * running under a memory manager that owns the whole device heap, code that must not trigger the
 * implicit synchronisation of cudaMalloc / cudaFree inside a latency-critical serving loop, or
 * code running after its allocator has been frozen.  pie_plan_forward allocates the device copy
 * of the plan and the fp32 scratch of the split-KV kernels; this call does the same work as
 * pie_plan_forward + pie_forward but keeps both in one fixed array that is part of the library
 * image (a file-scope `static __device__` array of PIE_STATIC_SCRATCH_BYTES bytes; every GPU that
 * loads the library holds it until the process exits).  It calls no cudaMalloc, no cudaFree and
 * no allocating library routine; host-side planning uses ordinary host memory.
 *
 *   - Arguments, results and errors are those of pie_forward, with `batch` (host) as in
 *     pie_plan_forward; q / k_new / v_new / out / lse are device pointers owned by the caller.
 *   - The host blocks while the plan image (ordinary pageable host memory) is handed to the copy
 *     engine; the kernels run asynchronously on `stream` as in pie_forward.
 *   - Requests without output KvPages (no_store) work as in pie_forward: the pool pages they borrow
 *     are handed back when the call returns and rejoin the free list once the work enqueued on
 *     `stream` has finished (one CUDA event per such call, recycled - a host-side object, no device
 *     memory).
 *   - A batch whose plan arrays plus split partials need more than PIE_STATIC_SCRATCH_BYTES is
 *     refused with PIE_ERR_BATCH_TOO_LARGE and nothing is enqueued.
 *   - The first call on a device looks up the array's device address (one cudaGetSymbolAddress,
 *     with that device current); make that first call before any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents.  Nothing in it has
 *     to start at zero (each call overwrites the plan arrays it reads and writes every partial
 *     before reading it), but two calls whose device work overlaps - different streams, or
 *     different contexts on the same GPU - race on it: keep them in one stream order. */
enum { PIE_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024 };
int pie_forward_static_scratch(pie_ctx* ctx, const pie_batch_desc* batch, const void* q,
                               const void* k_new, const void* v_new, void* out, float* lse,
                               void* stream);

/* ---- Batch scheduler of the control layer (Section 5.2 "Batch scheduler", Section 6.1) ------------
 * Host-only bookkeeping that decides WHICH pending calls form the next batch; it does not touch
 * the device.  Calls are submitted to command queues (Section 4.1 "Command queue": order inside a
 * queue is dependency order; queues carry a priority).  pie_sched_next_batch - to be called the
 * moment the GPU reports idle (work-conserving dispatch) - forms one batch:
 *   1. API type: the one whose oldest eligible call has waited longest (eligible = the run of
 *      consecutive same-type calls at the head of a queue);
 *   2. vertical batching: a queue contributes its head run, in order, up to (not including) the
 *      first call that writes a KvPage already written by a call of this batch;
 *   3. horizontal batching: all queues whose head call has that type take part, higher priority
 *      first (ties: lower queue id), so that
 *   4. the batch is cut from the tail at min(max_batch_calls, cap).
 * Chosen calls leave their queues; tags (caller's handles) come back in batch order, with their
 * queue ids if out_queues != NULL.  *out_n = 0 and *out_type = -1 when nothing is pending.
 * Types are small integers chosen by the caller (< PIE_SCHED_MAX_TYPES); write_pages lists the
 * KvPages a call writes (forward: its output pages; copy_kvpage: its destinations).  A request
 * reading rows that an EARLIER call of the same batch appends is not a conflict: pie_forward
 * appends the whole batch before attending (the two-call split of Section 4.2 runs as one batch). */
enum { PIE_SCHED_MAX_TYPES = 16 };
typedef struct pie_sched pie_sched;
int pie_sched_create(int32_t max_batch_calls, pie_sched** out);
int pie_sched_destroy(pie_sched* s);
int pie_sched_create_queue(pie_sched* s, int32_t priority, int32_t* out_queue);
int pie_sched_set_queue_priority(pie_sched* s, int32_t queue, int32_t priority);
int pie_sched_submit(pie_sched* s, int32_t queue, int32_t type, int32_t n_write, const int32_t* write_pages,
                     int64_t arrival_ns, int64_t tag);
int pie_sched_pending(const pie_sched* s, int32_t* out);
int pie_sched_next_batch(pie_sched* s, int32_t* out_type, int32_t cap, int64_t* out_tags, int32_t* out_queues,
                         int32_t* out_n);

/* Tuning knobs (all optional; 0 restores the default).  They affect plans made afterwards.
 *   PIE_OPT_SPLIT_SMS  SMs the split-KV decode kernel may use (default: all).
 *   PIE_OPT_TILE_SMS   SMs the prefill / tree kernel may use (default: all).
 *   PIE_OPT_OVERLAP    mixed batches (decode requests and prefill / tree requests in one call):
 *                      0 = automatic (default): the HBM-bound decode kernel and the tensor-bound
 *                      prefill / tree kernel run side by side on disjoint SM sets - the second on an
 *                      internal stream that forks from and joins the caller's stream - when a model
 *                      of the two kernels (the decode kernel keeps the memory system saturated
 *                      with about 60 % of the SMs) predicts at least 10 % over running them one
 *                      after the other; 1 = side by side whenever both kinds are present;
 *                      2 = never.  With 1 and PIE_OPT_SPLIT_SMS and PIE_OPT_TILE_SMS both set,
 *                      those are the two SM sets.
 *   PIE_OPT_NO_FUSION  bit mask of fusions of the decode path to switch off (default 0: all on;
 *                      results are identical up to fp32 summation order, pool contents bit-identical).
 *                      Bit 0: always launch the append kernel.  By default a decode batch (every
 *                      request one new token, all on the split-KV kernel, no request listing a
 *                      page another one appends to) lets the attention kernel write the new K/V
 *                      rows itself.  Bit 1: always merge split partials with the merge kernel.  By
 *                      default short decode launches keep all pieces of a (request, kv head)
 *                      inside one thread block, which merges them itself, and those where whole
 *                      units cannot fill the blocks evenly (a few long requests) cut units across
 *                      thread blocks and still merge inside the kernel: every block combines what it
 *                      holds of a unit, the block that writes its partial last combines the
 *                      blocks' partials (fixed order: results do not depend on timing).  Bit 3:
 *                      partials of merges inside a thread block always go through global memory.
 *                      By default a group whose pieces are the last work of their warps leaves
 *                      them in the warps' idle staging buffers in shared memory.  Bit 2: one kv head per
 *                      decode unit.  By default, with 64-wide heads and pages of 8 or 16 tokens, a
 *                      unit is a pair of adjacent kv heads (one copy of twice the size per page). */
enum { PIE_OPT_SPLIT_SMS = 0, PIE_OPT_TILE_SMS = 1, PIE_OPT_OVERLAP = 2, PIE_OPT_NO_FUSION = 3, PIE_NUM_OPTIONS = 4 };
int pie_set_option(pie_ctx* ctx, int option, int value);

/* Per-kernel device timing for benchmarks.  While enabled, pie_forward and pie_copy_kvpage
 * bracket each kernel they enqueue with CUDA events on the caller's stream.
 * pie_get_kernel_times waits for the recorded events, adds the elapsed milliseconds and the
 * launch counts per kernel kind into ms[PIE_NUM_KERNEL_KINDS] / launches[PIE_NUM_KERNEL_KINDS]
 * (host arrays, overwritten), and forgets the records.  Off by default (no events, no cost). */
enum {
  PIE_KERNEL_APPEND = 0,
  PIE_KERNEL_SIMPLE = 1,
  PIE_KERNEL_SPLIT = 2,   /* split-KV decode attention   */
  PIE_KERNEL_TILES = 3,   /* prefill / tree row tiles    */
  PIE_KERNEL_MERGE = 4,
  PIE_KERNEL_COPY = 5,
  PIE_NUM_KERNEL_KINDS = 6
};
int pie_set_kernel_timing(pie_ctx* ctx, int enable);
int pie_get_kernel_times(pie_ctx* ctx, float* ms, int32_t* launches);

#ifdef __cplusplus
}
#endif
#endif /* PIE_B200_H_ */
