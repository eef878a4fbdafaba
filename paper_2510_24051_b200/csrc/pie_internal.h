// Internal structures shared by the host code and the kernels of libpie_b200.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "pie_b200.h"

// ---------------------------------------------------------------------------------------------
// KvPage pool layout (private to the library).
//
//   pool[page][kv_head][K|V][slab][slot][128 bytes]
//
// A "block" is the K (or V) data of one (page, kv head): page_size rows of D elements.  Each
// row is cut into 128-byte slabs; inside a slab the eight 16-byte chunks of row `slot` are
// stored at chunk position (chunk ^ (slot & 7)).  This is exactly the 128-byte shared-memory
// swizzle that ldmatrix and the tcgen05 matrix descriptors want, so a plain linear bulk copy of
// a block lands in shared memory bank-conflict free and MMA ready, with no tensor map.
// K and V of the same (page, head) are adjacent: one copy of 2 blocks feeds one attention step.
// ---------------------------------------------------------------------------------------------
struct PoolGeom {
  int32_t page_size, n_kv_heads, head_dim, esize;
  int32_t row_bytes;    // D * esize
  int32_t n_slabs;      // row_bytes / 128
  int32_t slab_bytes;   // page_size * 128
  int32_t block_bytes;  // page_size * row_bytes
  int64_t page_bytes;   // n_kv_heads * 2 * block_bytes
};

// Byte offset inside a block of the 16-byte chunk `chunk` (0 .. row_bytes/16) of row `slot`.
__host__ __device__ inline int32_t pie_chunk_offset(int32_t slab_bytes, int32_t slot, int32_t chunk) {
  return (chunk >> 3) * slab_bytes + slot * 128 + (((chunk & 7) ^ (slot & 7)) << 4);
}

// Per-request record read by the attention kernels.
struct PieReq {
  int32_t q_start;         // first query token (qo_indptr[r])
  int32_t q_len;
  int32_t kv_len;
  int32_t kept_start;      // first entry in the kept-page list
  int32_t kept_count;
  int32_t mask_row_words;  // 0: causal mask inferred from positions
  int64_t mask_word_off;   // first packed mask word of this request
  int32_t last_logical;    // logical index of the last page
  int32_t last_page_len;
};

// One unit of work of a tile kernel: rows [row0, row0+nrows) of the request's (token, head-in-
// group) row space for one kv head, attended over kept pages [page_begin, page_end).
struct PieItem {
  int32_t req, kv_head, row0, nrows;
  int32_t page_begin, page_end;  // absolute indices into the kept-page list
  int32_t partial_slot;          // -1: write the final output; else slot of the fp32 partial
  // copy of the request record, so that a kernel can start an item from this one 64-byte line
  int32_t q_start, q_len, kv_len, mask_row_words, last_logical, last_page_len;
  uint32_t flags;                // PIE_ITEM_*
  int64_t mask_word_off;
};
static_assert(sizeof(PieItem) == 64, "PieItem is one 64-byte line");
// The split-KV warp that owns this item also writes the request's one new K/V row (decode batches
// whose append is fused into the attention kernel): into the pool and into its staged copy of the page.
#define PIE_ITEM_APPEND 1u
// Split-KV, fixed shares: the pieces of a cut unit that lie in ONE thread block are merged inside the
// kernel.  Every piece but the block's first writes its fp32 partial and counts itself in on a
// shared-memory counter (block-scope fence, no device-wide one); the warp with the first piece - its
// last item, so it finishes last - waits for the count and combines the partials with its own
// registers.  PIE_ITEM_LOCAL_GID = the group's counter in the block, PIE_ITEM_LOCAL_NP = its pieces.
#define PIE_ITEM_LOCAL_PIECE 2u
#define PIE_ITEM_LOCAL_MERGER 4u
#define PIE_MAX_LOCAL_GROUPS 8
// A unit cut across thread blocks: what a block holds of it (one piece, or the combination of its
// pieces made as above) is written as ONE fp32 partial, into the slot of the block's first piece,
// made visible device-wide and counted on the unit's counter in global memory (behind the launch's
// two work counters, indexed by the unit's first slot); the warp that finds all other blocks counted
// combines the block partials in slot order.  No warp waits for another block.  PIE_ITEM_GRID_NB =
// blocks the unit spans, PIE_ITEM_GRID_KB = index of this block among them, PIE_ITEM_GRID_N0 =
// pieces in the first of these blocks (every block between the first and the last holds one piece
// per warp, so block partial k > 0 sits n0 + warps_per_block (k - 1) slots behind the first).
#define PIE_ITEM_GRID_PIECE 8u
// A block-local group all of whose pieces are the LAST items of their warps: the partials are left in the
// warps' own (idle) rings in shared memory instead of global memory.
#define PIE_ITEM_LOCAL_SMEM 0x80000000u
#define PIE_ITEM_LOCAL_GID(f) (((f) >> 4) & 7u)
#define PIE_ITEM_LOCAL_NP(f) (((f) >> 7) & 15u)
#define PIE_ITEM_GRID_NB(f) (((f) >> 11) & 255u)
#define PIE_ITEM_GRID_KB(f) (((f) >> 19) & 255u)
#define PIE_ITEM_GRID_N0(f) (((f) >> 27) & 15u)
#define PIE_ITEM_LOCAL_BITS(gid, np) (((uint32_t)(gid) << 4) | ((uint32_t)(np) << 7))
#define PIE_ITEM_GRID_BITS(nb, kb, n0) (((uint32_t)(nb) << 11) | ((uint32_t)(kb) << 19) | ((uint32_t)(n0) << 27))
// Row-tile items: flags >> PIE_ITEM_CLEAN_SHIFT = number of leading pages of the item that every
// row of the tile sees in full (no page record and no mask word needs to be looked at for them).
#define PIE_ITEM_CLEAN_SHIFT 8

// A group of partial slots that the merge kernel combines into final rows.
struct PieMerge {
  int32_t req, kv_head, row0, nrows;
  int32_t slot0, nslots;
  // Shared-prefix cascade: further partials of the same rows, written by the row-tile launch for a
  // group of requests at once.  They sit in that launch's workspace, slots [x_slot0, x_slot0 +
  // x_nslots), where this group's rows start at row x_row0 of the slot (x_nslots = 0: none).
  int32_t x_slot0, x_nslots, x_row0;
};

#define PIE_KEPT_NEEDS_MASK 0x80000000u

struct PieLaunchList {           // one tile-kernel launch (split-KV decode, or row tiles)
  std::vector<PieItem> items;
  std::vector<int32_t> cta_ptr;  // [grid+1] items of each CTA
  std::vector<PieMerge> merges;
  int32_t grid = 0;
  int32_t n_slots = 0;
  int32_t slot_rows = 0;
  int32_t n_static = 0;          // split-KV: items [n_static, size) are taken from the work counter
  bool grid_merge = false;       // split-KV: cut units are merged inside the kernel by their last piece (one counter per slot behind d_work_ctr)
  int32_t heads_per_unit = 1;    // split-KV: 2 = every item covers kv heads 2 kv_head and 2 kv_head + 1 (rows of the first, then of the second)
  // device copies
  PieItem* d_items = nullptr;
  int32_t* d_cta_ptr = nullptr;
  PieMerge* d_merges = nullptr;
  int32_t* d_work_ctr = nullptr; // [2] dynamic-scheduling counters (split-KV kernel), re-armed by the kernel; then [n_slots] group counters if grid_merge
  float* d_ws_o = nullptr;       // [n_slots][slot_rows][D]
  float* d_ws_lse = nullptr;     // [n_slots][slot_rows]
};

struct pie_plan {
  pie_ctx* ctx = nullptr;
  uint32_t flags = 0;
  int32_t R = 0, T = 0;
  std::vector<PieReq> reqs;
  std::vector<int32_t> kept;        // pairs (phys, logical|flag)
  std::vector<int32_t> kept_scratch; // planner scratch (per-request slices before packing)
  std::vector<int32_t> clean_kept;   // [R] kept pages of the request before the first one some row sees only in part
  std::vector<int32_t> req_note;     // planner scratch: per request, the outcome of a pass over its page list
  std::vector<int32_t> slot_group;   // planner scratch: partial slot -> its merge group
  std::vector<int32_t> local_key;    // planner scratch: the batch's decode units as a key of the context's list cache
  // requests without output KvPages: pages of the library's own behind their page lists
  std::vector<int32_t> scratch_pages;                                   // held until the plan is destroyed or rebuilt
  std::vector<int32_t> pre_copies;                                      // (src, dst, src_off, dst_off, ntok) per copy, run before the append
  std::vector<int32_t> int_page_indptr, int_page_indices, int_last_page_len;   // the rewritten batch
  int32_t* d_pre_copies = nullptr;
  std::vector<uint32_t> mask_words;
  std::vector<int32_t> append_dst;  // [T] page*P + slot
  std::vector<int32_t> tok_req;     // [T]
  std::vector<int32_t> positions;   // [T] position of every new token (RoPE contexts only)
  std::vector<int32_t> simple_rows; // (token*H_q + head) rows for the plain kernel
  PieLaunchList split, tile;
  bool tile_tc = false;             // row tiles run on the tcgen05 kernel (256-row items)
  bool overlap = false;             // decode and tile kernels run side by side on disjoint SM sets
  bool append_fused = false;        // the split-KV kernel writes the new K/V rows itself (no append launch)
  pie_plan_info info{};
  // device
  void* d_blob = nullptr;           // one allocation holding every array below
  size_t d_blob_bytes = 0;
  void* h_image = nullptr;          // pinned host copy of the uploaded part (pie_plan_forward)
  size_t h_image_bytes = 0;
  // recycling (pie_plan_destroy parks the object, pie_plan_forward takes it back): the device
  // arrays may be overwritten only after the last forward that read them has finished
  mutable cudaStream_t last_stream = nullptr;   // stream of the latest pie_forward with this plan
  mutable bool used = false;                    // some pie_forward has read the device arrays
  mutable bool many_streams = false;            // ... and not all of them on last_stream
  cudaEvent_t idle = nullptr;                   // recorded behind that forward when the plan is parked
  bool idle_pending = false;
  PieReq* d_reqs = nullptr;
  int2* d_kept = nullptr;
  uint32_t* d_mask = nullptr;
  int32_t* d_append_dst = nullptr;
  int32_t* d_tok_req = nullptr;
  int32_t* d_positions = nullptr;
  int32_t* d_simple_rows = nullptr;
};

struct pie_plan;
// Host worker threads of a context (planner.cpp): started on the first batch that is worth them, parked on a
// condition variable between batches, joined by pie_destroy.
struct PieWorkers;
void pie_workers_destroy(PieWorkers* w);

struct pie_ctx {
  pie_config cfg{};
  PieWorkers* workers = nullptr;
  PoolGeom geom{};
  int32_t G = 1;
  int32_t n_sms = 148;
  bool host_only = false;
  // allocator
  std::vector<int32_t> free_list;
  std::vector<uint8_t> allocated;
  std::vector<uint32_t> page_mask;   // mask_kvpage: bit s = slot s visible (all ones by default)
  int64_t n_masked_pages = 0;        // pages whose mask hides at least one slot
  // device
  uint8_t* pool = nullptr;
  int* d_status = nullptr;
  void* d_stage = nullptr;  // staging for host <-> device calls
  size_t stage_bytes = 0;
  void* d_io = nullptr;     // device arena of pie_forward_host: q/k/v/out/lse
  size_t io_bytes = 0;
  void* d_planbuf = nullptr;  // device arena of pie_forward_host: plan image + partial workspaces
  size_t planbuf_bytes = 0;
  void* d_qrot = nullptr;        // rotated copy of Q (RoPE contexts): [max_query_tokens][H_q][D]
  double* d_inv_freq = nullptr;  // [D/2] theta^(-2i/D)
  void* h_stage = nullptr;  // pinned host staging of the plan image (pie_forward_host)
  size_t h_stage_bytes = 0;
  pie_plan* host_plan = nullptr;  // reused plan object of pie_forward_host
  std::vector<pie_plan*> parked_plans;  // destroyed plans kept for reuse: host arrays, pinned image, device arrays
  // Pages a plan borrowed for requests without output KvPages go back to the free list only when the
  // forward that used them is over: they wait here behind an event recorded on that forward's stream.
  struct HeldPages { cudaEvent_t done; std::vector<int32_t> pages; };
  std::vector<HeldPages> held_pages;
  std::vector<cudaEvent_t> held_events;   // recycled events of held_pages
  bool tc_configured = false, split_configured = false, split_pair_configured = false, tile_configured = false, nd_configured = false;   // kernel attributes set for this context's device
  // The block-local work list of the latest decode batch.  Consecutive steps of a serving loop bring the same
  // requests with the same page counts (a request grows by a page every page_size steps), and then the list is
  // the same up to the fields copied from the request records: the planner reuses it instead of dealing the
  // units to thread blocks again.
  struct LocalListCache {
    bool valid = false, balanced = false;
    int32_t sms = 0, warps = 0, slot_rows = 0;
    std::vector<int32_t> key;        // (request, kv head, first row, rows, first page, end page) of every unit
    std::vector<PieItem> items;
    std::vector<int32_t> cta_ptr;
    int32_t grid = 0, n_slots = 0;
  } local_cache;
  std::string cuda_error;
  int options[PIE_NUM_OPTIONS] = {0, 0, 0, 0};
  cudaStream_t side_stream = nullptr;  // second stream of overlapped mixed batches
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  // optional per-kernel timing (pie_set_kernel_timing)
  bool timing = false;
  struct TimedLaunch { int kind; cudaEvent_t start, stop; };
  std::vector<TimedLaunch> timed;
  std::vector<cudaEvent_t> free_events;
  // scratch for validation (sized num_pages)
  std::vector<uint32_t> wmask;
  std::vector<int32_t> writer;
};

// ---- kernels (defined in the .cu files) --------------------------------------------------------
struct AttnParams {
  const uint8_t* pool;
  const void* q;
  void* out;
  float* lse;
  const PieReq* reqs;
  const int2* kept;
  const uint32_t* mask;
  const PieItem* items;
  const int32_t* cta_ptr;
  int32_t* work_ctr;
  int32_t n_shares;   // split-KV kernel with fixed shares: entries of cta_ptr minus one
  int32_t n_static;   // first item that is taken dynamically (items before it belong to fixed shares)
  int32_t slot_rows;
  float* ws_o;
  float* ws_lse;
  const void* k_new;         // fused append: new rows [T][H_kv][D]
  const void* v_new;
  int* status;
  int64_t page_bytes;
  int32_t n_q_heads, n_kv_heads;
  int32_t G;         // rows per query token of an item: query heads per kv head, times the kv heads of a unit
  int32_t G_head;    // query heads per kv head
  float scale_log2;  // log2(e) / sqrt(D)
  // 1: signal dependent launches only when a block is done.  Side by side with another kernel an
  // early signal would let the NEXT kernel of the stream (a merge) occupy the SMs meant for the
  // neighbour with blocks that only wait; alone, the early signal hides the next launch.
  int32_t late_trigger;
};

int pie_launch_append(pie_ctx* ctx, const pie_plan* plan, const void* k_new, const void* v_new, cudaStream_t s);
// RoPE contexts: append with rotated K and a rotated copy of Q (rope.cu); *q_eff is what attention reads
int pie_launch_rope(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new, const void* v_new, cudaStream_t s);
// append (plain or RoPE) and the Q the attention kernels must read
int pie_append_and_q(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new, const void* v_new, cudaStream_t s,
                     const void** q_eff);
int pie_launch_copy(pie_ctx* ctx, int n, const int32_t* d_ops, cudaStream_t s);
int pie_launch_page_io(pie_ctx* ctx, int n, const int32_t* d_ids, void* K, void* V, bool write, cudaStream_t s);
int pie_launch_simple(pie_ctx* ctx, const pie_plan* plan, const void* q, void* out, float* lse, cudaStream_t s);
int pie_launch_split(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new, const void* v_new, void* out,
                     float* lse, cudaStream_t s);
int pie_launch_tiles(pie_ctx* ctx, const pie_plan* plan, const void* q, void* out, float* lse, cudaStream_t s);
int pie_launch_merge(pie_ctx* ctx, const pie_plan* plan, const PieLaunchList& ll, void* out, float* lse, cudaStream_t s);
bool pie_split_supported(const pie_ctx* ctx);
bool pie_split_pair_supported(const pie_ctx* ctx);   // ... with units of two adjacent kv heads
int pie_split_warps_per_block(const pie_ctx* ctx);
bool pie_tc_supported(const pie_ctx* ctx);
// n_tokens: rows of the Q tensor (the batch's query tokens), for the bounds of the Q tensor map
int pie_launch_tc_tiles(pie_ctx* ctx, const AttnParams& p, int grid, int64_t n_tokens, cudaStream_t s);

// Device image of a plan (every array the kernels read, 256-byte aligned, then the fp32 partial
// workspaces of the two tile launches): offsets, host-side fill of the uploaded part, binding of the
// plan's device pointers to an image at `base`.
struct PlanLayout {
  size_t reqs, kept, mask, app, tok, pos, simple, copies, items[2], cta[2], merges[2], ctr[2], ws_o[2], ws_lse[2];
  size_t upload, total;
};

PlanLayout pie_plan_layout(const pie_ctx* ctx, const pie_plan* plan);
void pie_plan_fill(const pie_plan* plan, const PlanLayout& L, uint8_t* dst);
void pie_plan_bind(pie_plan* plan, const PlanLayout& L, uint8_t* base);

int pie_build_plan(pie_ctx* ctx, const pie_batch_desc* b, pie_plan* plan);
// Borrowed pages of a plan (requests without output KvPages), host bookkeeping in planner.cpp:
// back to the free list at once (no forward has used them, or it is known to be over) ...
void pie_plan_release_scratch(pie_plan* plan);
// ... or held until everything enqueued on `s` so far has finished (api.cu).
void pie_plan_hold_scratch(pie_plan* plan, cudaStream_t s);
// Returns held pages whose forward is over to the free list; wait = block until all of them are.
void pie_reclaim_pages(pie_ctx* ctx, bool wait);
void pie_free_pages(pie_ctx* ctx, const std::vector<int32_t>& ids);

#define PIE_CUDA(ctx, expr)                                   \
  do {                                                        \
    cudaError_t e__ = (expr);                                 \
    if (e__ != cudaSuccess) {                                 \
      (ctx)->cuda_error = std::string(#expr) + ": " + cudaGetErrorString(e__); \
      return PIE_ERR_CUDA;                                    \
    }                                                         \
  } while (0)

// Programmatic dependent launch: every kernel of the path is launched with the stream-serialisation
// attribute, lets its successor start launching at once (pie_pdl_launch_dependents) and waits for its
// predecessor's results only where it first needs them (pie_pdl_wait), so launch latencies and
// prologues overlap the previous kernel's tail.  pie_pdl_wait returns once every earlier grid of the
// stream has completed and its writes are visible.
#ifdef __CUDACC__
__device__ __forceinline__ void pie_pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pie_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t pie_launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif
