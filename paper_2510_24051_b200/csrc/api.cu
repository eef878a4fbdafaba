// C ABI entry points, the KvPage allocator, and the bit-exact data-movement kernels
// (append of new K/V rows, token-level page copy, canonical page import / export).
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "pie_internal.h"

// ------------------------------------------------------------------------------------ kernels
namespace {

// K1: append (Table 1 `forward`, output KvPages).  One thread moves one 16-byte chunk of one new K
// or V row into the swizzled pool block of its destination (page, slot).  A thread keeps its place
// inside a token (K or V, head, chunk: found once, with shifts - chunks per row and page size are
// powers of two) and walks over tokens, four at a time so that four loads are in flight before
// the first store.  tok_shift > 0: a token has fewer chunks than the block has threads and every
// block covers 2^tok_shift tokens per step.
constexpr int kAppendUnroll = 4;
__global__ void append_kernel(uint8_t* __restrict__ pool, const uint8_t* __restrict__ k_new,
                              const uint8_t* __restrict__ v_new, const int32_t* __restrict__ append_dst,
                              int T, PoolGeom g, int chunk_shift, int page_shift, int tok_shift) {
  pie_pdl_launch_dependents();
  pie_pdl_wait();
  const int per_tok = (2 * g.n_kv_heads) << chunk_shift;     // chunks per token
  const int lanes = blockDim.x >> tok_shift;                 // threads that work on one token
  const int tl = threadIdx.x / lanes;                        // token of this thread inside the block's group
  const int j0 = threadIdx.x - tl * lanes;
  const int n_groups = (T + (1 << tok_shift) - 1) >> tok_shift;
  for (int j = j0; j < per_tok; j += lanes) {                // (one pass unless a token has more chunks than the block has threads)
    const int c = j & ((1 << chunk_shift) - 1), hk = j >> chunk_shift;
    const int kv = hk >= g.n_kv_heads ? 1 : 0, head = hk - kv * g.n_kv_heads;
    const uint8_t* src0 = (kv ? v_new : k_new) + (int64_t)head * g.row_bytes + c * 16;
    const int64_t tok_stride = (int64_t)g.n_kv_heads * g.row_bytes;
    uint8_t* dst0 = pool + (int64_t)(head * 2 + kv) * g.block_bytes;
    for (int grp = blockIdx.x; grp < n_groups; grp += kAppendUnroll * gridDim.x) {
      uint4 v[kAppendUnroll];
      int dst[kAppendUnroll];
#pragma unroll
      for (int u = 0; u < kAppendUnroll; ++u) {
        const int t = ((grp + u * (int)gridDim.x) << tok_shift) + tl;
        dst[u] = -1;
        if (grp + u * (int)gridDim.x < n_groups && t < T) {
          dst[u] = append_dst[t];
          v[u] = *reinterpret_cast<const uint4*>(src0 + t * tok_stride);
        }
      }
#pragma unroll
      for (int u = 0; u < kAppendUnroll; ++u) {
        if (dst[u] < 0) continue;
        const int page = dst[u] >> page_shift, slot = dst[u] & ((1 << page_shift) - 1);
        *reinterpret_cast<uint4*>(dst0 + (int64_t)page * g.page_bytes + pie_chunk_offset(g.slab_bytes, slot, c)) = v[u];
      }
    }
  }
}

// K2: copy_kvpage (Table 1).  ops[k] = {src, dst, src_off, dst_off, ntok}; kCopySplit blocks per
// op, 16 bytes per thread and step, four loads in flight before the first store (the copy is pure
// latency: a page is a few tens of KB).
constexpr int kCopySplit = 4;
__global__ void copy_kernel(uint8_t* __restrict__ pool, const int32_t* __restrict__ ops, PoolGeom g) {
  pie_pdl_launch_dependents();
  pie_pdl_wait();
  const int32_t* op = ops + blockIdx.x * 5;
  const int src = op[0], dst = op[1], so = op[2], dof = op[3], n = op[4];
  const int chunks = g.row_bytes >> 4;
  const int per_tok = 2 * g.n_kv_heads * chunks;
  const int total = n * per_tok, stride = blockDim.x * kCopySplit;
  auto addr = [&](int i, int page, int off) -> int64_t {
    const int t = i / per_tok, rem = i - t * per_tok;
    const int blk = rem / chunks, c = rem - blk * chunks;  // blk = head*2 + kv
    return (int64_t)page * g.page_bytes + (int64_t)blk * g.block_bytes + pie_chunk_offset(g.slab_bytes, off + t, c);
  };
  for (int i0 = blockIdx.y * blockDim.x + threadIdx.x; i0 < total; i0 += 4 * stride) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (i0 + k * stride < total) v[k] = *reinterpret_cast<const uint4*>(pool + addr(i0 + k * stride, src, so));
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (i0 + k * stride < total) *reinterpret_cast<uint4*>(pool + addr(i0 + k * stride, dst, dof)) = v[k];
  }
}

// Canonical [n][slot][head][D] <-> pool layout, 16 bytes per thread.
__global__ void page_io_kernel(uint8_t* __restrict__ pool, const int32_t* __restrict__ ids, uint8_t* K,
                               uint8_t* V, int n, int write, PoolGeom g) {
  const int chunks = g.row_bytes >> 4;
  const int64_t per_page = (int64_t)g.page_size * g.n_kv_heads * chunks;
  const int64_t total = (int64_t)n * per_page * 2;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int kv = (int)(i / ((int64_t)n * per_page));
    int64_t j = i - (int64_t)kv * n * per_page;  // chunk index inside canonical K or V
    int pg = (int)(j / per_page);
    int rem = (int)(j - (int64_t)pg * per_page);
    int slot = rem / (g.n_kv_heads * chunks);
    rem -= slot * g.n_kv_heads * chunks;
    int head = rem / chunks, c = rem - head * chunks;
    uint8_t* canon = (kv ? V : K) + j * 16;
    uint8_t* p = pool + (int64_t)ids[pg] * g.page_bytes + (int64_t)(head * 2 + kv) * g.block_bytes +
                 pie_chunk_offset(g.slab_bytes, slot, c);
    if (write) *reinterpret_cast<uint4*>(p) = *reinterpret_cast<const uint4*>(canon);
    else *reinterpret_cast<uint4*>(canon) = *reinterpret_cast<const uint4*>(p);
  }
}

int grid_for(int64_t work_items, int threads, int n_sms) {
  int64_t blocks = (work_items + threads - 1) / threads;
  return (int)std::max<int64_t>(1, std::min<int64_t>(blocks, (int64_t)n_sms * 8));
}

int ensure_buffer(pie_ctx* ctx, void** buf, size_t* cap, size_t need) {
  if (*cap >= need) return PIE_OK;
  if (*buf) PIE_CUDA(ctx, cudaFree(*buf));
  *buf = nullptr;
  *cap = 0;
  // half as much again: a serving loop's batches grow step by step, and every regrowth is a cudaFree +
  // cudaMalloc (a device-wide synchronisation of several hundred microseconds)
  size_t want = std::max(need + need / 2, (size_t)1 << 20);
  PIE_CUDA(ctx, cudaMalloc(buf, want));
  *cap = want;
  return PIE_OK;
}

// Runs `launch` bracketed by events when timing is on.
template <typename F>
int timed_launch(pie_ctx* ctx, int kind, cudaStream_t s, F&& launch) {
  if (!ctx->timing) return launch();
  cudaEvent_t ev[2];
  for (int k = 0; k < 2; ++k) {
    if (!ctx->free_events.empty()) {
      ev[k] = ctx->free_events.back();
      ctx->free_events.pop_back();
    } else {
      PIE_CUDA(ctx, cudaEventCreate(&ev[k]));
    }
  }
  PIE_CUDA(ctx, cudaEventRecord(ev[0], s));
  int rc = launch();
  PIE_CUDA(ctx, cudaEventRecord(ev[1], s));
  ctx->timed.push_back({kind, ev[0], ev[1]});
  return rc;
}

bool page_ok(const pie_ctx* ctx, int32_t id) {
  return id >= 0 && id < ctx->cfg.num_pages && ctx->allocated[id];
}

}  // namespace

// Device image of a plan: every array the kernels read, 256-byte aligned, followed by the fp32
// partial workspaces of the two tile launches.

PlanLayout pie_plan_layout(const pie_ctx* ctx, const pie_plan* plan) {
  PlanLayout L{};
  size_t off = 0;
  auto place = [&](size_t bytes) {
    size_t o = off;
    off = (off + bytes + 255) & ~(size_t)255;
    return o;
  };
  L.reqs = place(plan->reqs.size() * sizeof(PieReq));
  L.kept = place(plan->kept.size() * 4);
  L.mask = place(plan->mask_words.size() * 4);
  L.app = place(plan->append_dst.size() * 4);
  L.tok = place(plan->tok_req.size() * 4);
  L.pos = place(plan->positions.size() * 4);
  L.simple = place(plan->simple_rows.size() * 4);
  L.copies = place(plan->pre_copies.size() * 4);
  const PieLaunchList* lls[2] = {&plan->split, &plan->tile};
  for (int k = 0; k < 2; ++k) {
    L.items[k] = place(lls[k]->items.size() * sizeof(PieItem));
    L.cta[k] = place(lls[k]->cta_ptr.size() * 4);
    L.merges[k] = place(lls[k]->merges.size() * sizeof(PieMerge));
    L.ctr[k] = place(8 + (lls[k]->grid_merge ? (size_t)lls[k]->n_slots * 4 : 0));
  }
  L.upload = off;
  const size_t D = ctx->cfg.head_dim;
  for (int k = 0; k < 2; ++k) {
    L.ws_o[k] = place((size_t)lls[k]->n_slots * lls[k]->slot_rows * D * 4);
    L.ws_lse[k] = place((size_t)lls[k]->n_slots * lls[k]->slot_rows * 4);
  }
  L.total = off;
  return L;
}

void pie_plan_fill(const pie_plan* plan, const PlanLayout& L, uint8_t* dst) {
  auto cp = [&](size_t off, const void* p, size_t bytes) {
    if (bytes) std::memcpy(dst + off, p, bytes);
  };
  cp(L.reqs, plan->reqs.data(), plan->reqs.size() * sizeof(PieReq));
  cp(L.kept, plan->kept.data(), plan->kept.size() * 4);
  cp(L.mask, plan->mask_words.data(), plan->mask_words.size() * 4);
  cp(L.app, plan->append_dst.data(), plan->append_dst.size() * 4);
  cp(L.tok, plan->tok_req.data(), plan->tok_req.size() * 4);
  cp(L.pos, plan->positions.data(), plan->positions.size() * 4);
  cp(L.simple, plan->simple_rows.data(), plan->simple_rows.size() * 4);
  cp(L.copies, plan->pre_copies.data(), plan->pre_copies.size() * 4);
  const PieLaunchList* lls[2] = {&plan->split, &plan->tile};
  for (int k = 0; k < 2; ++k) {
    cp(L.items[k], lls[k]->items.data(), lls[k]->items.size() * sizeof(PieItem));
    cp(L.cta[k], lls[k]->cta_ptr.data(), lls[k]->cta_ptr.size() * 4);
    cp(L.merges[k], lls[k]->merges.data(), lls[k]->merges.size() * sizeof(PieMerge));
    {
      const int32_t ctr0[2] = {lls[k]->n_static, 0};  // next dynamic item, finished warps; the kernel re-arms them
      std::memcpy(dst + L.ctr[k], ctr0, 8);
      if (lls[k]->grid_merge) std::memset(dst + L.ctr[k] + 8, 0, (size_t)lls[k]->n_slots * 4);   // pieces written so far, per group
    }
  }
}

void pie_plan_bind(pie_plan* plan, const PlanLayout& L, uint8_t* base) {
  plan->d_reqs = (PieReq*)(base + L.reqs);
  plan->d_kept = (int2*)(base + L.kept);
  plan->d_mask = (uint32_t*)(base + L.mask);
  plan->d_append_dst = (int32_t*)(base + L.app);
  plan->d_tok_req = (int32_t*)(base + L.tok);
  plan->d_positions = (int32_t*)(base + L.pos);
  plan->d_simple_rows = (int32_t*)(base + L.simple);
  plan->d_pre_copies = (int32_t*)(base + L.copies);
  PieLaunchList* lls[2] = {&plan->split, &plan->tile};
  for (int k = 0; k < 2; ++k) {
    lls[k]->d_items = (PieItem*)(base + L.items[k]);
    lls[k]->d_cta_ptr = (int32_t*)(base + L.cta[k]);
    lls[k]->d_merges = (PieMerge*)(base + L.merges[k]);
    lls[k]->d_work_ctr = (int32_t*)(base + L.ctr[k]);
    lls[k]->d_ws_o = (float*)(base + L.ws_o[k]);
    lls[k]->d_ws_lse = (float*)(base + L.ws_lse[k]);
  }
}


int pie_launch_append(pie_ctx* ctx, const pie_plan* plan, const void* k_new, const void* v_new, cudaStream_t s) {
  if (plan->T == 0) return PIE_OK;
  const PoolGeom& g = ctx->geom;
  auto log2i = [](int x) {
    int l = 0;
    while ((1 << l) < x) ++l;
    return l;
  };
  const int chunk_shift = log2i(g.row_bytes >> 4), page_shift = log2i(g.page_size);   // (both powers of two: D 64 / 128, page size 8 / 16 / 32)
  const int per_tok = (2 * g.n_kv_heads) << chunk_shift;
  int tok_shift = 0;   // tokens per block and step: as many as fit into 256 threads, a power of two
  while ((per_tok << (tok_shift + 1)) <= 256) ++tok_shift;
  const int n_groups = (plan->T + (1 << tok_shift) - 1) >> tok_shift;
  const int grid = std::max(1, std::min((n_groups + kAppendUnroll - 1) / kAppendUnroll, ctx->n_sms * 8));
  PIE_CUDA(ctx, pie_launch_pdl(append_kernel, dim3(grid), dim3(256), 0, s, ctx->pool, (const uint8_t*)k_new, (const uint8_t*)v_new,
                               (const int32_t*)plan->d_append_dst, plan->T, g, chunk_shift, page_shift, tok_shift));
  return PIE_OK;
}

int pie_append_and_q(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new, const void* v_new, cudaStream_t s,
                     const void** q_eff) {
  *q_eff = q;
  if (plan->append_fused) return PIE_OK;  // the split-KV kernel writes the new rows itself
  if (ctx->cfg.rope_theta > 0.f) {  // positions inside the path: rotated K goes to the pages, attention reads rotated Q
    *q_eff = ctx->d_qrot;
    return pie_launch_rope(ctx, plan, q, k_new, v_new, s);
  }
  return pie_launch_append(ctx, plan, k_new, v_new, s);
}

int pie_launch_copy(pie_ctx* ctx, int n, const int32_t* d_ops, cudaStream_t s) {
  PIE_CUDA(ctx, pie_launch_pdl(copy_kernel, dim3(n, kCopySplit), dim3(256), 0, s, ctx->pool, d_ops, ctx->geom));
  return PIE_OK;
}

int pie_launch_page_io(pie_ctx* ctx, int n, const int32_t* d_ids, void* K, void* V, bool write, cudaStream_t s) {
  const PoolGeom& g = ctx->geom;
  int64_t work = (int64_t)n * g.page_size * g.n_kv_heads * (g.row_bytes >> 4) * 2;
  page_io_kernel<<<grid_for(work, 256, ctx->n_sms), 256, 0, s>>>(ctx->pool, d_ids, (uint8_t*)K, (uint8_t*)V, n,
                                                                  write ? 1 : 0, g);
  PIE_CUDA(ctx, cudaGetLastError());
  return PIE_OK;
}

// ------------------------------------------------------------------------------------ borrowed pages
void pie_reclaim_pages(pie_ctx* ctx, bool wait) {
  if (ctx->held_pages.empty()) return;
  cudaSetDevice(ctx->cfg.device);
  size_t kept = 0;
  for (size_t k = 0; k < ctx->held_pages.size(); ++k) {
    pie_ctx::HeldPages& h = ctx->held_pages[k];
    cudaError_t e = wait ? cudaEventSynchronize(h.done) : cudaEventQuery(h.done);
    if (e == cudaErrorNotReady) {
      cudaGetLastError();
      if (kept != k) ctx->held_pages[kept] = std::move(h);
      ++kept;
      continue;
    }
    if (e != cudaSuccess) cudaGetLastError();   // (a failed device: nothing is running on the pages any more)
    pie_free_pages(ctx, h.pages);
    ctx->held_events.push_back(h.done);
  }
  ctx->held_pages.resize(kept);
}

void pie_plan_hold_scratch(pie_plan* plan, cudaStream_t s) {
  pie_ctx* ctx = plan->ctx;
  if (plan->scratch_pages.empty() || ctx->host_only) {
    pie_plan_release_scratch(plan);
    return;
  }
  cudaSetDevice(ctx->cfg.device);
  cudaEvent_t ev = nullptr;
  cudaError_t e = cudaSuccess;
  if (!ctx->held_events.empty()) {
    ev = ctx->held_events.back();
    ctx->held_events.pop_back();
  } else {
    e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaEventRecord(ev, s);
  if (e != cudaSuccess) {   // no event to wait behind: wait for the device instead, then the pages are free
    cudaGetLastError();
    cudaDeviceSynchronize();
    if (ev) ctx->held_events.push_back(ev);
    pie_plan_release_scratch(plan);
    return;
  }
  ctx->held_pages.push_back(pie_ctx::HeldPages{ev, std::move(plan->scratch_pages)});
  plan->scratch_pages.clear();
  plan->pre_copies.clear();
}

// ------------------------------------------------------------------------------------ C ABI
extern "C" {

const char* pie_strerror(int status) {
  switch (status) {
    case PIE_OK: return "ok";
    case PIE_ERR_INVALID: return "invalid argument";
    case PIE_ERR_NO_PAGES: return "out of KvPages";
    case PIE_ERR_BAD_PAGE: return "bad KvPage id";
    case PIE_ERR_CONFLICT: return "conflicting KvPage access inside one batch";
    case PIE_ERR_BATCH_TOO_LARGE: return "batch exceeds the configured maximum";
    case PIE_ERR_MASK: return "malformed mask";
    case PIE_ERR_CUDA: return "CUDA error";
    case PIE_ERR_NO_DEVICE: return "host-only context";
    case PIE_ERR_UNSUPPORTED: return "unsupported shape or type";
    case PIE_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

const char* pie_last_cuda_error(const pie_ctx* ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }

int pie_create(const pie_config* cfg, pie_ctx** out) {
  if (!cfg || !out) return PIE_ERR_INVALID;
  const int P = cfg->page_size, D = cfg->head_dim;
  if (P != 8 && P != 16 && P != 32) return PIE_ERR_INVALID;
  if (D != 64 && D != 128) return PIE_ERR_INVALID;
  if (cfg->dtype != PIE_DTYPE_BF16 && cfg->dtype != PIE_DTYPE_F32) return PIE_ERR_INVALID;
  if (cfg->num_pages < 1 || cfg->num_q_heads < 1 || cfg->num_kv_heads < 1) return PIE_ERR_INVALID;
  if (cfg->num_q_heads % cfg->num_kv_heads) return PIE_ERR_INVALID;
  if (cfg->max_requests < 1 || cfg->max_query_tokens < 1) return PIE_ERR_INVALID;
  if (!(cfg->rope_theta >= 0.f)) return PIE_ERR_INVALID;
  if ((int64_t)cfg->num_pages * P > 0x7FFFFFFF) return PIE_ERR_INVALID;
  if ((int64_t)cfg->num_pages * cfg->num_kv_heads > 0x7FFFFFFF) return PIE_ERR_INVALID;
  pie_ctx* ctx = new (std::nothrow) pie_ctx();
  if (!ctx) return PIE_ERR_INVALID;
  ctx->cfg = *cfg;
  ctx->G = cfg->num_q_heads / cfg->num_kv_heads;
  PoolGeom& g = ctx->geom;
  g.page_size = P;
  g.n_kv_heads = cfg->num_kv_heads;
  g.head_dim = D;
  g.esize = cfg->dtype == PIE_DTYPE_BF16 ? 2 : 4;
  g.row_bytes = D * g.esize;
  g.n_slabs = g.row_bytes / 128;
  g.slab_bytes = P * 128;
  g.block_bytes = P * g.row_bytes;
  g.page_bytes = (int64_t)cfg->num_kv_heads * 2 * g.block_bytes;
  ctx->allocated.assign(cfg->num_pages, 0);
  ctx->page_mask.assign(cfg->num_pages, 0xFFFFFFFFu);
  ctx->free_list.resize(cfg->num_pages);
  for (int i = 0; i < cfg->num_pages; ++i) ctx->free_list[i] = cfg->num_pages - 1 - i;  // pop from the back: 0,1,2,..
  ctx->wmask.assign(cfg->num_pages, 0u);
  ctx->writer.assign(cfg->num_pages, -1);
  ctx->host_only = cfg->device < 0;
  if (!ctx->host_only) {
    auto fail = [&](cudaError_t e, const char* what) {
      (void)e;
      (void)what;
      if (ctx->pool) cudaFree(ctx->pool);
      if (ctx->d_status) cudaFree(ctx->d_status);
      if (ctx->d_qrot) cudaFree(ctx->d_qrot);
      if (ctx->d_inv_freq) cudaFree(ctx->d_inv_freq);
      delete ctx;
      return PIE_ERR_CUDA;
    };
    cudaError_t e;
    if ((e = cudaSetDevice(cfg->device)) != cudaSuccess) return fail(e, "cudaSetDevice");
    int sms = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device)) != cudaSuccess)
      return fail(e, "attr");
    ctx->n_sms = sms;
    size_t bytes = (size_t)cfg->num_pages * (size_t)g.page_bytes;
    if ((e = cudaMalloc((void**)&ctx->pool, bytes)) != cudaSuccess) return fail(e, "cudaMalloc pool");
    if ((e = cudaMemset(ctx->pool, 0, bytes)) != cudaSuccess) return fail(e, "memset");
    if ((e = cudaMalloc((void**)&ctx->d_status, 256)) != cudaSuccess) return fail(e, "cudaMalloc status");
    if ((e = cudaMemset(ctx->d_status, 0, 256)) != cudaSuccess) return fail(e, "memset");
    if (cfg->rope_theta > 0.f) {
      const size_t qb = (size_t)cfg->max_query_tokens * cfg->num_q_heads * g.row_bytes;
      std::vector<double> inv((size_t)D / 2);
      for (int i = 0; i < D / 2; ++i) inv[i] = std::pow((double)cfg->rope_theta, -2.0 * i / D);
      if ((e = cudaMalloc(&ctx->d_qrot, qb)) != cudaSuccess) return fail(e, "cudaMalloc qrot");
      if ((e = cudaMalloc((void**)&ctx->d_inv_freq, inv.size() * 8)) != cudaSuccess) return fail(e, "cudaMalloc inv_freq");
      if ((e = cudaMemcpy(ctx->d_inv_freq, inv.data(), inv.size() * 8, cudaMemcpyHostToDevice)) != cudaSuccess)
        return fail(e, "upload inv_freq");
    }
    if ((e = cudaDeviceSynchronize()) != cudaSuccess) return fail(e, "sync");
  }
  *out = ctx;
  return PIE_OK;
}

int pie_destroy(pie_ctx* ctx) {
  if (!ctx) return PIE_ERR_INVALID;
  if (!ctx->host_only) {
    cudaSetDevice(ctx->cfg.device);
    cudaDeviceSynchronize();
    if (ctx->pool) cudaFree(ctx->pool);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->d_stage) cudaFree(ctx->d_stage);
    if (ctx->d_io) cudaFree(ctx->d_io);
    if (ctx->d_planbuf) cudaFree(ctx->d_planbuf);
    if (ctx->h_stage) cudaFreeHost(ctx->h_stage);
    if (ctx->d_qrot) cudaFree(ctx->d_qrot);
    if (ctx->d_inv_freq) cudaFree(ctx->d_inv_freq);
    if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    for (auto& t : ctx->timed) {
      cudaEventDestroy(t.start);
      cudaEventDestroy(t.stop);
    }
    for (auto e : ctx->free_events) cudaEventDestroy(e);
    for (auto& h : ctx->held_pages) cudaEventDestroy(h.done);
    for (auto e : ctx->held_events) cudaEventDestroy(e);
  }
  pie_workers_destroy(ctx->workers);
  ctx->workers = nullptr;
  delete ctx->host_plan;
  for (pie_plan* plan : ctx->parked_plans) {
    if (!ctx->host_only) {
      if (plan->d_blob) cudaFree(plan->d_blob);
      if (plan->h_image) cudaFreeHost(plan->h_image);
      if (plan->idle) cudaEventDestroy(plan->idle);
    }
    delete plan;
  }
  delete ctx;
  return PIE_OK;
}

int pie_alloc_kvpages(pie_ctx* ctx, int32_t n, int32_t* out_ids) {
  if (!ctx || n < 0 || (n > 0 && !out_ids)) return PIE_ERR_INVALID;
  pie_reclaim_pages(ctx, false);
  if ((size_t)n > ctx->free_list.size()) pie_reclaim_pages(ctx, true);   // pages still borrowed by a running forward
  if ((size_t)n > ctx->free_list.size()) return PIE_ERR_NO_PAGES;
  for (int i = 0; i < n; ++i) {
    int32_t id = ctx->free_list.back();
    ctx->free_list.pop_back();
    ctx->allocated[id] = 1;
    if (ctx->page_mask[id] != 0xFFFFFFFFu) {  // a fresh page is fully visible
      ctx->page_mask[id] = 0xFFFFFFFFu;
      --ctx->n_masked_pages;
    }
    out_ids[i] = id;
  }
  return PIE_OK;
}

int pie_dealloc_kvpages(pie_ctx* ctx, int32_t n, const int32_t* ids) {
  if (!ctx || n < 0 || (n > 0 && !ids)) return PIE_ERR_INVALID;
  for (int i = 0; i < n; ++i) {
    if (!page_ok(ctx, ids[i])) return PIE_ERR_BAD_PAGE;
    for (int j = 0; j < i; ++j)  // a repeated id inside one call is a double free
      if (ids[j] == ids[i]) return PIE_ERR_BAD_PAGE;
  }
  for (int i = 0; i < n; ++i) {
    ctx->allocated[ids[i]] = 0;
    ctx->free_list.push_back(ids[i]);
  }
  return PIE_OK;
}

int pie_mask_kvpage(pie_ctx* ctx, int32_t n, const int32_t* ids, const uint32_t* masks) {
  if (!ctx || n < 0 || (n > 0 && (!ids || !masks))) return PIE_ERR_INVALID;
  for (int i = 0; i < n; ++i)
    if (!page_ok(ctx, ids[i])) return PIE_ERR_BAD_PAGE;
  const int P = ctx->cfg.page_size;
  const uint32_t full = P >= 32 ? 0xFFFFFFFFu : ((1u << P) - 1u);
  for (int i = 0; i < n; ++i) {
    const uint32_t m = ((masks[i] & full) == full) ? 0xFFFFFFFFu : (masks[i] & full);
    uint32_t& cur = ctx->page_mask[ids[i]];
    ctx->n_masked_pages += (m != 0xFFFFFFFFu) - (cur != 0xFFFFFFFFu);
    cur = m;
  }
  return PIE_OK;
}

int pie_num_free_kvpages(const pie_ctx* ctx, int32_t* out) {
  if (!ctx || !out) return PIE_ERR_INVALID;
  pie_reclaim_pages(const_cast<pie_ctx*>(ctx), true);
  *out = (int32_t)ctx->free_list.size();
  return PIE_OK;
}

static int page_io(pie_ctx* ctx, int32_t n, const int32_t* ids, void* K, void* V, int on_device, void* stream,
                   bool write) {
  if (!ctx || n < 0 || (n > 0 && (!ids || !K || !V))) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  for (int i = 0; i < n; ++i)
    if (!page_ok(ctx, ids[i])) return PIE_ERR_BAD_PAGE;
  if (n == 0) return PIE_OK;
  cudaStream_t s = (cudaStream_t)stream;
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  const size_t canon = (size_t)ctx->geom.page_size * ctx->geom.n_kv_heads * ctx->geom.row_bytes;  // K (or V) bytes per page
  if (on_device) {
    int rc = ensure_buffer(ctx, &ctx->d_stage, &ctx->stage_bytes, (size_t)n * 4);
    if (rc) return rc;
    PIE_CUDA(ctx, cudaMemcpyAsync(ctx->d_stage, ids, (size_t)n * 4, cudaMemcpyHostToDevice, s));
    return pie_launch_page_io(ctx, n, (const int32_t*)ctx->d_stage, K, V, write, s);
  }
  const int chunk = (int)std::max<size_t>(1, std::min<size_t>((size_t)n, ((size_t)64 << 20) / canon));
  size_t ids_bytes = ((size_t)chunk * 4 + 255) & ~(size_t)255;
  int rc = ensure_buffer(ctx, &ctx->d_stage, &ctx->stage_bytes, ids_bytes + 2 * chunk * canon);
  if (rc) return rc;
  uint8_t* dK = (uint8_t*)ctx->d_stage + ids_bytes;
  uint8_t* dV = dK + (size_t)chunk * canon;
  for (int i0 = 0; i0 < n; i0 += chunk) {
    int m = std::min(chunk, n - i0);
    PIE_CUDA(ctx, cudaMemcpyAsync(ctx->d_stage, ids + i0, (size_t)m * 4, cudaMemcpyHostToDevice, s));
    if (write) {
      PIE_CUDA(ctx, cudaMemcpyAsync(dK, (const uint8_t*)K + (size_t)i0 * canon, (size_t)m * canon, cudaMemcpyHostToDevice, s));
      PIE_CUDA(ctx, cudaMemcpyAsync(dV, (const uint8_t*)V + (size_t)i0 * canon, (size_t)m * canon, cudaMemcpyHostToDevice, s));
    }
    rc = pie_launch_page_io(ctx, m, (const int32_t*)ctx->d_stage, dK, dV, write, s);
    if (rc) return rc;
    if (!write) {
      PIE_CUDA(ctx, cudaMemcpyAsync((uint8_t*)K + (size_t)i0 * canon, dK, (size_t)m * canon, cudaMemcpyDeviceToHost, s));
      PIE_CUDA(ctx, cudaMemcpyAsync((uint8_t*)V + (size_t)i0 * canon, dV, (size_t)m * canon, cudaMemcpyDeviceToHost, s));
    }
    PIE_CUDA(ctx, cudaStreamSynchronize(s));
  }
  return PIE_OK;
}

int pie_kvpage_write(pie_ctx* ctx, int32_t n, const int32_t* ids, const void* K, const void* V, int on_device,
                     void* stream) {
  return page_io(ctx, n, ids, const_cast<void*>(K), const_cast<void*>(V), on_device, stream, true);
}

int pie_kvpage_read(pie_ctx* ctx, int32_t n, const int32_t* ids, void* K, void* V, int on_device, void* stream) {
  return page_io(ctx, n, ids, K, V, on_device, stream, false);
}

int pie_copy_kvpage(pie_ctx* ctx, int32_t n, const int32_t* src, const int32_t* dst, const int32_t* src_off,
                    const int32_t* dst_off, const int32_t* ntok, void* stream) {
  if (!ctx || n < 0 || (n > 0 && (!src || !dst || !src_off || !dst_off || !ntok))) return PIE_ERR_INVALID;
  const int P = ctx->cfg.page_size;
  for (int k = 0; k < n; ++k) {
    if (!page_ok(ctx, src[k]) || !page_ok(ctx, dst[k])) return PIE_ERR_BAD_PAGE;
    if (ntok[k] < 0 || src_off[k] < 0 || dst_off[k] < 0 || src_off[k] + ntok[k] > P || dst_off[k] + ntok[k] > P)
      return PIE_ERR_INVALID;
  }
  auto bits = [](int lo, int n_) -> uint32_t {
    if (n_ <= 0) return 0u;
    uint32_t m = (n_ >= 32) ? 0xFFFFFFFFu : ((1u << n_) - 1u);
    return m << lo;
  };
  int status = PIE_OK;
  for (int k = 0; k < n && status == PIE_OK; ++k) {
    uint32_t m = bits(dst_off[k], ntok[k]);
    if (ctx->wmask[dst[k]] & m) status = PIE_ERR_CONFLICT;
    ctx->wmask[dst[k]] |= m;
  }
  for (int k = 0; k < n && status == PIE_OK; ++k)
    if (ctx->wmask[src[k]] & bits(src_off[k], ntok[k])) status = PIE_ERR_CONFLICT;
  for (int k = 0; k < n; ++k) ctx->wmask[dst[k]] = 0;
  if (status != PIE_OK) return status;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  if (n == 0) return PIE_OK;
  cudaStream_t s = (cudaStream_t)stream;
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  std::vector<int32_t> ops((size_t)n * 5);
  for (int k = 0; k < n; ++k) {
    ops[k * 5 + 0] = src[k];
    ops[k * 5 + 1] = dst[k];
    ops[k * 5 + 2] = src_off[k];
    ops[k * 5 + 3] = dst_off[k];
    ops[k * 5 + 4] = ntok[k];
  }
  int rc = ensure_buffer(ctx, &ctx->d_stage, &ctx->stage_bytes, ops.size() * 4);
  if (rc) return rc;
  PIE_CUDA(ctx, cudaMemcpyAsync(ctx->d_stage, ops.data(), ops.size() * 4, cudaMemcpyHostToDevice, s));
  return timed_launch(ctx, PIE_KERNEL_COPY, s, [&] { return pie_launch_copy(ctx, n, (const int32_t*)ctx->d_stage, s); });
}

// Plans are recycled: pie_plan_destroy parks up to kParkedPlans objects in the context, with their
// host vectors, pinned image and device arrays, and pie_plan_forward takes one back.  A serving
// loop that plans every step therefore stops allocating after its first steps: no cudaMalloc and
// no cudaFree (with its device-wide synchronisation) per batch.
static const size_t kParkedPlans = 4;

static void release_plan(pie_plan* plan) {
  if (plan->ctx) {
    if (plan->used && !plan->ctx->host_only && !plan->scratch_pages.empty()) {
      cudaSetDevice(plan->ctx->cfg.device);
      cudaDeviceSynchronize();   // its forwards may still be running on the borrowed pages
    }
    pie_plan_release_scratch(plan);
  }
  if (plan->d_blob || plan->h_image || plan->idle) {
    cudaSetDevice(plan->ctx->cfg.device);
    if (plan->d_blob) cudaFree(plan->d_blob);   // (synchronises: nothing can still be reading the arrays afterwards)
    if (plan->h_image) cudaFreeHost(plan->h_image);
    if (plan->idle) cudaEventDestroy(plan->idle);
  }
  delete plan;
}

int pie_plan_forward(pie_ctx* ctx, const pie_batch_desc* batch, void* stream, pie_plan** out) {
  if (!ctx || !batch || !out) return PIE_ERR_INVALID;
  pie_plan* plan = nullptr;
  if (!ctx->parked_plans.empty()) {
    plan = ctx->parked_plans.back();
    ctx->parked_plans.pop_back();
  } else {
    plan = new (std::nothrow) pie_plan();
  }
  if (!plan) return PIE_ERR_INVALID;
  plan->ctx = ctx;
  auto give_back = [&]() {   // the object goes back as it came: its device arrays were not touched
    if (ctx->parked_plans.size() < kParkedPlans) ctx->parked_plans.push_back(plan);
    else release_plan(plan);
  };
  int rc = pie_build_plan(ctx, batch, plan);
  if (rc != PIE_OK) {
    give_back();
    return rc;
  }
  if (!ctx->host_only && plan->R > 0) {
    cudaStream_t s = (cudaStream_t)stream;
    const PlanLayout L = pie_plan_layout(ctx, plan);
    cudaError_t e = cudaSetDevice(ctx->cfg.device);
    if (e == cudaSuccess && plan->idle_pending) {   // the forward that last read the device arrays must be over
      e = cudaEventSynchronize(plan->idle);
      plan->idle_pending = false;
    }
    if (e == cudaSuccess && plan->h_image_bytes < L.upload) {
      if (plan->h_image) cudaFreeHost(plan->h_image);
      plan->h_image = nullptr;
      plan->h_image_bytes = 0;
      const size_t want = std::max(L.upload + L.upload / 4, (size_t)1 << 16);
      e = cudaMallocHost(&plan->h_image, want);
      if (e == cudaSuccess) plan->h_image_bytes = want;
    }
    if (e == cudaSuccess && plan->d_blob_bytes < L.total) {
      if (plan->d_blob) cudaFree(plan->d_blob);
      plan->d_blob = nullptr;
      plan->d_blob_bytes = 0;
      const size_t want = std::max(L.total + L.total / 4, (size_t)1 << 16);
      e = cudaMalloc(&plan->d_blob, want);
      if (e == cudaSuccess) plan->d_blob_bytes = want;
    }
    if (e == cudaSuccess) {
      pie_plan_fill(plan, L, (uint8_t*)plan->h_image);
      if (L.upload) e = cudaMemcpyAsync(plan->d_blob, plan->h_image, L.upload, cudaMemcpyHostToDevice, s);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
      ctx->cuda_error = std::string("plan upload: ") + cudaGetErrorString(e);
      release_plan(plan);
      return PIE_ERR_CUDA;
    }
    pie_plan_bind(plan, L, (uint8_t*)plan->d_blob);
  }
  plan->used = false;
  plan->many_streams = false;
  *out = plan;
  return PIE_OK;
}

int pie_plan_destroy(pie_plan* plan) {
  if (!plan) return PIE_ERR_INVALID;
  pie_ctx* ctx = plan->ctx;
  if (!ctx || ctx->parked_plans.size() >= kParkedPlans) {
    release_plan(plan);
    return PIE_OK;
  }
  // pages borrowed for requests without output KvPages go back once the plan's forwards are over
  if (plan->used && !plan->scratch_pages.empty() && !ctx->host_only) {
    if (plan->many_streams) {
      cudaSetDevice(ctx->cfg.device);
      cudaDeviceSynchronize();
      pie_plan_release_scratch(plan);
    } else {
      pie_plan_hold_scratch(plan, plan->last_stream);
    }
  } else {
    pie_plan_release_scratch(plan);
  }
  if (plan->used && plan->d_blob) {
    // a forward may still be reading the device arrays: mark the point behind it on its stream
    cudaSetDevice(ctx->cfg.device);
    cudaError_t e = cudaSuccess;
    if (plan->many_streams) e = cudaErrorInvalidValue;   // forwards on several streams: one event cannot follow them all
    if (e == cudaSuccess && !plan->idle) e = cudaEventCreateWithFlags(&plan->idle, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventRecord(plan->idle, plan->last_stream);
    if (e == cudaSuccess) {
      plan->idle_pending = true;
    } else {   // (e.g. the stream no longer exists) fall back to waiting for the whole device
      cudaGetLastError();
      cudaDeviceSynchronize();
      plan->idle_pending = false;
    }
  }
  plan->used = false;
  plan->many_streams = false;
  ctx->parked_plans.push_back(plan);
  return PIE_OK;
}

int pie_plan_get_info(const pie_plan* plan, pie_plan_info* out) {
  if (!plan || !out) return PIE_ERR_INVALID;
  *out = plan->info;
  return PIE_OK;
}

int pie_plan_debug_read(const pie_plan* plan, int which, void* buf, int64_t cap_bytes, int64_t* out_bytes) {
  if (!plan || !out_bytes) return PIE_ERR_INVALID;
  const void* p = nullptr;
  int64_t n = 0;
  if (which == 3) {   // the whole image as it is uploaded: every array the kernels read, in device layout
    const PlanLayout L = pie_plan_layout(plan->ctx, plan);
    *out_bytes = (int64_t)L.upload;
    if (buf && cap_bytes >= (int64_t)L.upload && L.upload > 0) {
      std::memset(buf, 0, L.upload);   // (alignment gaps between the arrays)
      pie_plan_fill(plan, L, (uint8_t*)buf);
    }
    return PIE_OK;
  }
  switch (which) {
    case 0: p = plan->mask_words.data(); n = (int64_t)plan->mask_words.size() * 4; break;
    case 1: p = plan->kept.data(); n = (int64_t)plan->kept.size() * 4; break;
    case 2: p = plan->append_dst.data(); n = (int64_t)plan->append_dst.size() * 4; break;
    case 4: p = plan->split.items.data(); n = (int64_t)plan->split.items.size() * (int64_t)sizeof(PieItem); break;
    case 5: p = plan->tile.items.data(); n = (int64_t)plan->tile.items.size() * (int64_t)sizeof(PieItem); break;
    default: return PIE_ERR_INVALID;
  }
  *out_bytes = n;
  if (buf && cap_bytes >= n && n > 0) std::memcpy(buf, p, (size_t)n);
  return PIE_OK;
}

int pie_forward(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new, const void* v_new, void* out,
                float* lse, void* stream) {
  if (!ctx || !plan || plan->ctx != ctx) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  if (plan->T == 0) return PIE_OK;
  if (!q || !k_new || !v_new || !out || !lse) return PIE_ERR_INVALID;
  cudaStream_t s = (cudaStream_t)stream;
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  // (a recycled plan's device arrays are rewritten only behind the forwards that read them)
  if (plan->used && plan->last_stream != s) plan->many_streams = true;
  plan->last_stream = s;
  plan->used = true;
  if (!plan->pre_copies.empty()) {   // rows of partly filled input pages of requests without output KvPages, into the plan's own pages
    const int n_ops = (int)plan->pre_copies.size() / 5;
    const int rc0 = timed_launch(ctx, PIE_KERNEL_COPY, s, [&] { return pie_launch_copy(ctx, n_ops, (const int32_t*)plan->d_pre_copies, s); });
    if (rc0) return rc0;
  }
  const void* q_in = q;
  int rc = plan->append_fused ? PIE_OK  // (q stays q_in: the split-KV kernel writes the new rows itself)
                              : timed_launch(ctx, PIE_KERNEL_APPEND, s, [&] { return pie_append_and_q(ctx, plan, q_in, k_new, v_new, s, &q); });
  if (rc) return rc;
  if (!plan->simple_rows.empty() &&
      (rc = timed_launch(ctx, PIE_KERNEL_SIMPLE, s, [&] { return pie_launch_simple(ctx, plan, q, out, lse, s); })))
    return rc;
  const bool side = plan->overlap && !plan->split.items.empty() && !plan->tile.items.empty();
  cudaStream_t s2 = s;
  if (side) {
    // fork: the tile kernel (and its merge) runs on the context's side stream, next to the
    // decode kernel on the caller's stream; both joined again before the call returns
    if (!ctx->side_stream) {
      PIE_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking));
      PIE_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming));
      PIE_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming));
    }
    s2 = ctx->side_stream;
    PIE_CUDA(ctx, cudaEventRecord(ctx->ev_fork, s));
    PIE_CUDA(ctx, cudaStreamWaitEvent(s2, ctx->ev_fork, 0));
  }
  auto launch_tiles = [&]() -> int {
    int r = PIE_OK;
    if (!plan->tile.items.empty() &&
        (r = timed_launch(ctx, PIE_KERNEL_TILES, s2, [&] { return pie_launch_tiles(ctx, plan, q, out, lse, s2); })))
      return r;
    if (!plan->tile.merges.empty() &&
        (r = timed_launch(ctx, PIE_KERNEL_MERGE, s2, [&] { return pie_launch_merge(ctx, plan, plan->tile, out, lse, s2); })))
      return r;
    return PIE_OK;
  };
  // Side by side, the decode kernel is enqueued first: measured on B200, a running row-tile kernel
  // keeps the decode kernel's blocks from being dispatched until it ends, while the other order
  // lets both run.  One after the other, the row tiles go first (cascade partials feed the split merge).
  if (!side && (rc = launch_tiles())) return rc;
  if (!plan->split.items.empty() &&
      (rc = timed_launch(ctx, PIE_KERNEL_SPLIT, s, [&] { return pie_launch_split(ctx, plan, q, k_new, v_new, out, lse, s); })))
    return rc;
  if (side) {   // row tiles on the side stream, then join: the split merge may read their partials (cascade)
    if ((rc = launch_tiles())) return rc;
    PIE_CUDA(ctx, cudaEventRecord(ctx->ev_join, s2));
    PIE_CUDA(ctx, cudaStreamWaitEvent(s, ctx->ev_join, 0));
  }
  if (!plan->split.merges.empty() &&
      (rc = timed_launch(ctx, PIE_KERNEL_MERGE, s, [&] { return pie_launch_merge(ctx, plan, plan->split, out, lse, s); })))
    return rc;
  return PIE_OK;
}

int pie_forward_host(pie_ctx* ctx, const pie_batch_desc* batch, const void* q, const void* k_new, const void* v_new,
                     void* out, float* lse, void* stream) {
  if (!ctx || !batch) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  // The context keeps one plan object, one pinned staging buffer and two device arenas (tensors,
  // plan image) for this entry point and reuses them call after call: no allocation in the
  // steady state.  The Q / K / V uploads are started first, so the DMA runs while the host plans.
  if (!ctx->host_plan) ctx->host_plan = new (std::nothrow) pie_plan();
  pie_plan* plan = ctx->host_plan;
  if (!plan) return PIE_ERR_INVALID;
  plan->ctx = ctx;
  cudaStream_t s = (cudaStream_t)stream;
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  const int R = batch->num_requests;
  const bool early = R > 0 && R <= ctx->cfg.max_requests && batch->qo_indptr && batch->qo_indptr[R] > 0 &&
                     batch->qo_indptr[R] <= ctx->cfg.max_query_tokens && q && k_new && v_new && out && lse;
  const size_t es = ctx->geom.esize, D = ctx->cfg.head_dim;
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  size_t T = 0, q_bytes = 0, kv_bytes = 0, lse_bytes = 0, o_k = 0, o_v = 0, o_out = 0, o_lse = 0;
  auto io_layout = [&](size_t tokens) {
    T = tokens;
    q_bytes = T * ctx->cfg.num_q_heads * D * es;
    kv_bytes = T * ctx->cfg.num_kv_heads * D * es;
    lse_bytes = T * ctx->cfg.num_q_heads * 4;
    o_k = al(q_bytes);
    o_v = o_k + al(kv_bytes);
    o_out = o_v + al(kv_bytes);
    o_lse = o_out + al(q_bytes);
    return o_lse + al(lse_bytes);
  };
  auto upload_inputs = [&]() -> int {
    uint8_t* io = (uint8_t*)ctx->d_io;
    PIE_CUDA(ctx, cudaMemcpyAsync(io, q, q_bytes, cudaMemcpyHostToDevice, s));
    PIE_CUDA(ctx, cudaMemcpyAsync(io + o_k, k_new, kv_bytes, cudaMemcpyHostToDevice, s));
    PIE_CUDA(ctx, cudaMemcpyAsync(io + o_v, v_new, kv_bytes, cudaMemcpyHostToDevice, s));
    return PIE_OK;
  };
  int rc;
  if (early) {
    if ((rc = ensure_buffer(ctx, &ctx->d_io, &ctx->io_bytes, io_layout((size_t)batch->qo_indptr[R])))) return rc;
    if ((rc = upload_inputs())) return rc;
  }
  rc = pie_build_plan(ctx, batch, plan);
  if (rc) {
    if (early) cudaStreamSynchronize(s);  // the caller's buffers must outlive the copies already queued
    return rc;
  }
  if (plan->T == 0) return PIE_OK;
  if (!q || !k_new || !v_new || !out || !lse) return PIE_ERR_INVALID;
  if (!early) {
    if ((rc = ensure_buffer(ctx, &ctx->d_io, &ctx->io_bytes, io_layout((size_t)plan->T)))) return rc;
    if ((rc = upload_inputs())) return rc;
  }
  const PlanLayout L = pie_plan_layout(ctx, plan);
  if ((rc = ensure_buffer(ctx, &ctx->d_planbuf, &ctx->planbuf_bytes, L.total))) return rc;
  if (ctx->h_stage_bytes < L.upload) {
    if (ctx->h_stage) PIE_CUDA(ctx, cudaFreeHost(ctx->h_stage));
    ctx->h_stage = nullptr;
    ctx->h_stage_bytes = 0;
    const size_t want = std::max(L.upload * 2, (size_t)1 << 20);
    PIE_CUDA(ctx, cudaMallocHost(&ctx->h_stage, want));
    ctx->h_stage_bytes = want;
  }
  uint8_t* io = (uint8_t*)ctx->d_io;
  pie_plan_fill(plan, L, (uint8_t*)ctx->h_stage);
  pie_plan_bind(plan, L, (uint8_t*)ctx->d_planbuf);
  PIE_CUDA(ctx, cudaMemcpyAsync(ctx->d_planbuf, ctx->h_stage, L.upload, cudaMemcpyHostToDevice, s));
  if ((rc = pie_forward(ctx, plan, io, io + o_k, io + o_v, io + o_out, (float*)(io + o_lse), stream))) return rc;
  PIE_CUDA(ctx, cudaMemcpyAsync(out, io + o_out, q_bytes, cudaMemcpyDeviceToHost, s));
  PIE_CUDA(ctx, cudaMemcpyAsync(lse, io + o_lse, lse_bytes, cudaMemcpyDeviceToHost, s));
  PIE_CUDA(ctx, cudaStreamSynchronize(s));
  pie_plan_release_scratch(plan);   // (pages borrowed for requests without output KvPages: the forward is over)
  return PIE_OK;
}

int pie_get_last_device_status(pie_ctx* ctx, void* stream, int* out) {
  if (!ctx || !out) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  cudaStream_t s = (cudaStream_t)stream;
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  int v = 0;
  PIE_CUDA(ctx, cudaMemcpyAsync(&v, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, s));
  PIE_CUDA(ctx, cudaStreamSynchronize(s));
  if (v != 0) {
    PIE_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(int), s));
    PIE_CUDA(ctx, cudaStreamSynchronize(s));
  }
  *out = v;
  return PIE_OK;
}

int pie_set_option(pie_ctx* ctx, int option, int value) {
  if (!ctx || option < 0 || option >= PIE_NUM_OPTIONS || value < 0) return PIE_ERR_INVALID;
  ctx->options[option] = value;
  return PIE_OK;
}

int pie_set_kernel_timing(pie_ctx* ctx, int enable) {
  if (!ctx) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  for (auto& t : ctx->timed) {
    ctx->free_events.push_back(t.start);
    ctx->free_events.push_back(t.stop);
  }
  ctx->timed.clear();
  ctx->timing = enable != 0;
  return PIE_OK;
}

int pie_get_kernel_times(pie_ctx* ctx, float* ms, int32_t* launches) {
  if (!ctx || !ms || !launches) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  for (int k = 0; k < PIE_NUM_KERNEL_KINDS; ++k) {
    ms[k] = 0.f;
    launches[k] = 0;
  }
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  for (auto& t : ctx->timed) {
    PIE_CUDA(ctx, cudaEventSynchronize(t.stop));
    float e = 0.f;
    PIE_CUDA(ctx, cudaEventElapsedTime(&e, t.start, t.stop));
    ms[t.kind] += e;
    launches[t.kind] += 1;
    ctx->free_events.push_back(t.start);
    ctx->free_events.push_back(t.stop);
  }
  ctx->timed.clear();
  return PIE_OK;
}

}  // extern "C"
