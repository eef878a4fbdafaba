// Prefill / token-tree attention on the 5th-generation tensor cores (Section 4.2 "Forward API":
// chunked prefill, speculative-tree verification under explicit masks).
//
// One CTA per SM walks its share of work items.  An item is up to 256 rows (row = query token *
// G + head-in-group, one kv head) = two 128-row Q tiles, attended over the item's kept pages in
// KV tiles of 128 tokens that are handled as two halves of 64 columns.  Roles (352 threads):
//   warps 0-3 / 4-7  softmax warpgroup of Q tile 0 / 1: one row per thread.  Reads a half of S
//                    from TMEM, masks, exponentiates, writes bf16 P back over that half of S,
//                    keeps the running (max, sum), rescales O in TMEM only when the row max grew
//                    by more than 2^8, and runs the epilogue.
//   warp 8           producer: linear bulk copies of page blocks into the K / V stage rings.  The
//                    pool's storage order is the 128-byte-swizzled canonical operand layout, so a
//                    page block drops into its 16-row band of the tile with no tensor map.
//   warp 9, one lane MMA issuer: S_t^h = Q_t K_h^T (N = 64), O_t += P_t^h V_h with tcgen05.mma,
//                    accumulators and P in TMEM; completion is tracked with tcgen05.commit.
//   warp 10          Q loader (TMA): runs one item ahead, so that the first S of the next item is
//                    computed while the warpgroups are still in the epilogue of this one.
// The tensor pipe takes instructions synchronously from the issuing thread (measured: a group of
// eight MMAs returns after ~8 x 64 cycles and any other work of that thread is idle pipe time), so
// the issuer is a single thread that does nothing but wait, issue and commit.  The two halves
// break the chain S -> softmax -> PV -> next S of a Q tile: while a warpgroup works on one half,
// the PV of the other half and the next S into the columns it frees are already running.
// TMEM (512 columns): S0a S0b | S1a S1b | O0 | O1; P_t^h overlays the first 32 columns of S_t^h.
#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "pie_internal.h"
#include "ptx_helpers.cuh"

namespace {

using namespace pie_ptx;

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, M x N, A K-major, B K- or MN-major.
__device__ __forceinline__ uint32_t instr_desc(int M, int N, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
               "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
               : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
               "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
               : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// A load that stays where it is written (the compiler neither sinks it to its first use nor
// merges it with a later one).
__device__ __forceinline__ uint32_t ldg_early(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
// Tiled TMA load of a 3-D box (no multicast); x is the innermost coordinate in elements.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
               "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
               : "memory");
}
// Tiled TMA store of a 3-D box from shared memory (bulk async-group completion).
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(map), "r"(src), "r"(x), "r"(y),
               "r"(z)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// every bulk store of this thread has finished READING shared memory / has completed altogether
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// barrier among the 128 threads of one softmax warpgroup (ids 1 and 2; 0 is __syncthreads)
template <int ID>
__device__ __forceinline__ void wg_sync() { asm volatile("bar.sync %0, 128;" ::"n"(ID) : "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// 32-byte global store (the address must be 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t* w) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]),
               "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}
// One lane of the (converged) warp, the same one every time.
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred P;\nelect.sync _|P, 0xffffffff;\nselp.u32 %0, 1, 0, P;\n}\n" : "=r"(pred));
  return pred;
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%"
      "31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
               "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
               "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
               : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
}
// packed fp32x2 arithmetic (two independent fp32 lanes in one 64-bit register) and 3-input max
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0,%1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

constexpr float kNegInf = -__builtin_huge_valf();
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTileM = 128;    // rows per Q tile
constexpr int kTileN = 128;    // tokens per KV tile (one stage of the K / V rings)
constexpr int kHalf = 64;      // columns per half tile: the unit handed between softmax and MMA
constexpr int kThreads = 352;

template <int D, int P>
struct TcCfg {
  static constexpr int NSLAB = D / 64;                 // 128-byte slabs per row
  static constexpr int PPT = kTileN / P;               // pages per KV tile
  static constexpr int PPH = kHalf / P;                // pages per half
  static constexpr int SLAB_TILE = kTileN * 128;       // bytes of one slab of a 128-row tile (16 KB)
  static constexpr int SLAB_PAGE = P * 128;            // bytes of one slab of a page block
  static constexpr int BLK = P * D * 2;                // K (or V) block of one page and head
  static constexpr int QTILE = kTileM * D * 2;
  static constexpr int KVTILE = kTileN * D * 2;
  static constexpr int STAGES = D == 128 ? 2 : 4;
  static constexpr int NBAR = 4 * STAGES + 19;
  static constexpr int OSLAB = kTileM * 128;           // output staging: one 64-column slab of a 128-row tile per warpgroup
  static constexpr int SMEM = 2 * QTILE + 2 * STAGES * KVTILE + 2 * OSLAB + NBAR * 8 + 64;
};

template <int D, int P>
__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(const AttnParams p, const __grid_constant__ CUtensorMap qmap,
                                                              const __grid_constant__ CUtensorMap omap, const int kflags) {
  using C = TcCfg<D, P>;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sQ = smem;
  uint8_t* sK = smem + 2 * C::QTILE;
  uint8_t* sV = sK + C::STAGES * C::KVTILE;
  uint8_t* sO = sV + C::STAGES * C::KVTILE;   // [2][128 rows][128 B], 128-byte swizzle like the Q tiles
  uint64_t* bars = reinterpret_cast<uint64_t*>(sO + 2 * C::OSLAB);
  uint64_t* k_full = bars;
  uint64_t* k_empty = k_full + C::STAGES;
  uint64_t* v_full = k_empty + C::STAGES;
  uint64_t* v_empty = v_full + C::STAGES;
  uint64_t* q_full = v_empty + C::STAGES;  // [2]      Q tile t is in shared memory
  uint64_t* q_free = q_full + 2;           // [2]      every S MMA of the item that reads Q tile t is complete
  uint64_t* s_full = q_free + 2;           // [2][2]   S_t^h is complete in TMEM
  uint64_t* p_full = s_full + 4;           // [2][2]   P_t^h is written (128 arrivals)
  uint64_t* pv_done = p_full + 4;          // [2]      one phase per PV group of Q tile t
  uint64_t* o_done = pv_done + 2;          // [2]      last PV of the item is complete
  uint64_t* o_free = o_done + 2;           // [2]      the epilogue has read O_t (128 arrivals)
  uint64_t* v_land = o_free + 2;           // [1]      producer-private: V tile that needs its tail cleared
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(v_land + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool use_qmap = kflags & 1;      // Q tiles come through the tensor map
  const bool out_wide = kflags & 2;      // the output pointer allows 32-byte stores
  const bool use_omap = kflags & 4;      // full output tiles leave through shared memory and a TMA store
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(smem_u32(k_full + s), 1);
      mbar_init(smem_u32(k_empty + s), 1);
      mbar_init(smem_u32(v_full + s), 1);
      mbar_init(smem_u32(v_empty + s), 1);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(q_full + t), 1);
      mbar_init(smem_u32(q_free + t), 1);
      for (int h = 0; h < 2; ++h) {
        mbar_init(smem_u32(s_full + 2 * t + h), 1);
        mbar_init(smem_u32(p_full + 2 * t + h), kTileM);
      }
      mbar_init(smem_u32(pv_done + t), 1);
      mbar_init(smem_u32(o_done + t), 1);
      mbar_init(smem_u32(o_free + t), kTileM);
    }
    mbar_init(smem_u32(v_land), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (!p.late_trigger) pie_pdl_launch_dependents();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pie_pdl_wait();  // the append (and whatever produced Q) is complete from here on

  const int it0 = p.cta_ptr[blockIdx.x], it1 = p.cta_ptr[blockIdx.x + 1];

  if (warp == 8) {
    // ================================================================ producer
    uint32_t tile_cnt = 0, land_cnt = 0;
    for (int it = it0; it < it1; ++it) {
      const PieItem item = p.items[it];
      const uint8_t* base = p.pool + (int64_t)item.kv_head * (2 * C::BLK);
      const int npages = item.page_end - item.page_begin;
      const int ntiles = (npages + C::PPT - 1) / C::PPT;
      const bool ragged = item.last_page_len < P;   // slots past the end of the context may hold anything
      for (int j = 0; j < ntiles; ++j, ++tile_cnt) {
        const uint32_t s = tile_cnt % C::STAGES, ph = (tile_cnt / C::STAGES) & 1;
        const int nvalid = min(C::PPT, npages - j * C::PPT);
        const int ncopies = nvalid * C::NSLAB;
        int2 rec = make_int2(0, -1);
        if (lane < nvalid) rec = __ldg(&p.kept[item.page_begin + j * C::PPT + lane]);
        const int pg = lane / C::NSLAB, sl = lane % C::NSLAB;   // copy `lane`: page pg of the tile, slab sl
        const int ph_pg = __shfl_sync(0xFFFFFFFFu, rec.x, pg);   // (at most PPT * NSLAB <= 32 copies per tile)
        // ---- K
        mbar_wait(smem_u32(k_empty + s), ph ^ 1, p.status);
        if (lane == 0) mbar_expect_tx(smem_u32(k_full + s), nvalid * C::BLK);
        __syncwarp();
        if (lane < ncopies)
          bulk_g2s(smem_u32(sK + s * C::KVTILE + sl * C::SLAB_TILE + pg * C::SLAB_PAGE),
                   base + (int64_t)ph_pg * p.page_bytes + sl * C::SLAB_PAGE, C::SLAB_PAGE, smem_u32(k_full + s));
        __syncwarp();
        // ---- V.  A tile that holds the request's partly filled last page lands on a private
        // barrier first: the rows past the end of the context are cleared (they may hold NaN
        // patterns, and 0 x NaN would poison O) before the tile is handed to the MMA thread.
        mbar_wait(smem_u32(v_empty + s), ph ^ 1, p.status);
        unsigned hit = 0;
        if (ragged) hit = __ballot_sync(0xFFFFFFFFu, lane < nvalid && (int)((uint32_t)rec.y & ~PIE_KEPT_NEEDS_MASK) == item.last_logical);
        const bool odd_end = P == 8 && (nvalid & 1);   // half of the tile's last 16-token step has no page
        const uint32_t vbar = (hit || odd_end) ? smem_u32(v_land) : smem_u32(v_full + s);
        if (lane == 0) mbar_expect_tx(vbar, nvalid * C::BLK);
        __syncwarp();
        if (lane < ncopies)
          bulk_g2s(smem_u32(sV + s * C::KVTILE + sl * C::SLAB_TILE + pg * C::SLAB_PAGE),
                   base + (int64_t)ph_pg * p.page_bytes + C::BLK + sl * C::SLAB_PAGE, C::SLAB_PAGE, vbar);
        __syncwarp();
        if (hit || odd_end) {
          mbar_wait(smem_u32(v_land), land_cnt & 1, p.status);
          ++land_cnt;
          constexpr int CH = D * 2 / 16;
          auto clear_rows = [&](int first, int n) {   // V rows [first, first + n) of the tile
            for (int c = lane; c < n * CH; c += 32) {
              const int tkn = first + c / CH, ch = c % CH;
              *reinterpret_cast<uint4*>(sV + s * C::KVTILE + (ch >> 3) * C::SLAB_TILE + tkn * 128 + (((ch & 7) ^ (tkn & 7)) << 4)) =
                  make_uint4(0, 0, 0, 0);
            }
          };
          if (hit) clear_rows((__ffs(hit) - 1) * P + item.last_page_len, P - item.last_page_len);
          if (odd_end) clear_rows(nvalid * P, P);
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(v_full + s));
        }
      }
    }
  } else if (warp == 9) {
    // ================================================================ MMA issuer
    // One elected lane runs the whole role.  (Electing the lane, rather than testing the lane id,
    // lets the compiler keep descriptors and loop state in uniform registers; measured, it halves
    // the cost of issuing an MMA.)  Everything between two batches of MMAs is time the tensor pipe
    // may run dry, so interior KV tiles take a fully unrolled path with constant offsets.
    if (elect_one()) {
      uint32_t tile_cnt = 0;
      uint32_t item_ph = 0;   // bit t: phase of q_full / o_free of Q tile t
      uint32_t half_ph = 0;   // bit 2t+h: phase of p_full[t][h]
      const uint32_t idesc_pv = instr_desc(kTileM, D, 1);
      const uint32_t idesc_s = instr_desc(kTileM, kHalf, 0);
      const uint64_t k_desc0 = smem_desc(smem_u32(sK), 16, 1024);            // K-major
      const uint64_t v_desc0 = smem_desc(smem_u32(sV), C::SLAB_TILE, 1024);  // MN-major: LBO = slab stride
      const uint64_t q_desc0 = smem_desc(smem_u32(sQ), 16, 1024);
      const uint32_t bar_p = smem_u32(p_full), bar_s = smem_u32(s_full), bar_pv = smem_u32(pv_done);
      // the next item's page count and row count are fetched one item ahead (their latency would
      // otherwise sit between the last MMA of an item and the first of the next)
      // (raw loaded values are kept and only combined when the item starts: nothing waits for the loads here)
      uint32_t nx_end = 0, nx_begin = 0, nx_nrows = 0;
      if (it0 < it1) {
        nx_end = ldg_early(reinterpret_cast<const uint32_t*>(&p.items[it0].page_end));
        nx_begin = ldg_early(reinterpret_cast<const uint32_t*>(&p.items[it0].page_begin));
        nx_nrows = ldg_early(reinterpret_cast<const uint32_t*>(&p.items[it0].nrows));
      }
      for (int it = it0; it < it1; ++it) {
        const int npages = (int)(nx_end - nx_begin), nrows = (int)nx_nrows;
        if (it + 1 < it1) {
          nx_end = ldg_early(reinterpret_cast<const uint32_t*>(&p.items[it + 1].page_end));
          nx_begin = ldg_early(reinterpret_cast<const uint32_t*>(&p.items[it + 1].page_begin));
          nx_nrows = ldg_early(reinterpret_cast<const uint32_t*>(&p.items[it + 1].nrows));
        }
        if (npages == 0) continue;  // the softmax warpgroups write zeros / -inf on their own
        const int ntiles = (npages + C::PPT - 1) / C::PPT;
        const int nhalf = (npages + C::PPH - 1) / C::PPH;           // halves of the item
        // columns of the last half, as a whole number of 16-token MMA steps (with 8-token pages the last step may
        // be half empty: its scores are masked off like any column past the end, its V rows are cleared)
        const int last_cols = ((npages - (nhalf - 1) * C::PPH) * P + 15) & ~15;
        const int nt = nrows > kTileM ? 2 : 1;
        // Phase of q_full / o_free of Q tile t: bit t of item_ph counts the items the tile took part in.
        const uint32_t ph_item = item_ph;
        for (int t = 0; t < nt; ++t) {
          mbar_wait(smem_u32(q_full + t), (ph_item >> t) & 1, p.status);
          item_ph ^= 1u << t;
        }
        tc_fence_after();

        // Descriptors are built once (per kernel for the K / V stages, per item for Q); a k-step only
        // adds its byte offset >> 4 to the start-address field.
        auto issue_s = [&](int t, int i, uint32_t stage) {   // S_t^h = Q_t K_h^T for half i of the item (h = i & 1)
          const int h = i & 1;
          const uint32_t idesc = instr_desc(kTileM, i + 1 < nhalf ? kHalf : last_cols, 0);
          const uint64_t qd = q_desc0 + (uint64_t)(t * (C::QTILE >> 4));
          const uint64_t kd = k_desc0 + (uint64_t)(stage * (C::KVTILE >> 4) + h * ((kHalf * 128) >> 4));
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint64_t off = (uint64_t)(((ks >> 2) * C::SLAB_TILE + (ks & 3) * 32) >> 4);
            umma_ss(tmem + t * 128 + h * kHalf, qd + off, kd + off, idesc, ks > 0);
          }
          umma_commit(bar_s + 8 * (2 * t + h));
        };

        // prologue: both halves of S_t for the first KV tile
        {
          const uint32_t s = tile_cnt % C::STAGES, ph = (tile_cnt / C::STAGES) & 1;
          mbar_wait(smem_u32(k_full + s), ph, p.status);
          tc_fence_after();
          for (int h = 0; h < min(2, nhalf); ++h)
            for (int t = 0; t < nt; ++t) issue_s(t, h, s);
          umma_commit(smem_u32(k_empty + s));
          if (ntiles == 1)
            for (int t = 0; t < nt; ++t) umma_commit(smem_u32(q_free + t));
        }
        for (int j = 0; j < ntiles; ++j) {
          const uint32_t cnt = tile_cnt + j;
          const uint32_t s = cnt % C::STAGES, ph = (cnt / C::STAGES) & 1;
          const uint32_t sn = (cnt + 1) % C::STAGES, phn = ((cnt + 1) / C::STAGES) & 1;
          mbar_wait(smem_u32(v_full + s), ph, p.status);
          if (nt == 2 && j > 0 && 2 * j + 5 <= nhalf) {
            // ---- interior tile: this tile and the next both have two full halves
            mbar_wait(smem_u32(k_full + sn), phn, p.status);
            const uint64_t vd0 = v_desc0 + (uint64_t)(s * (C::KVTILE >> 4));
            const uint64_t kd0 = k_desc0 + (uint64_t)(sn * (C::KVTILE >> 4));
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
              for (int t = 0; t < 2; ++t) {
                mbar_wait(bar_p + 8 * (2 * t + h), (half_ph >> (2 * t + h)) & 1, p.status);
                tc_fence_after();
                const uint32_t dO = tmem + 256 + t * D, dS = tmem + t * 128 + h * kHalf;
#pragma unroll
                for (int ks = 0; ks < kHalf / 16; ++ks)   // 16 token rows = 2048 bytes per k-step
                  umma_ts(dO, dS + ks * 8, vd0 + (uint64_t)((h * (kHalf / 16) + ks) * 128), idesc_pv, 1u);
                umma_commit(bar_pv + 8 * t);
                if (h == 1 && t == 1) umma_commit(smem_u32(v_empty + s));
                const uint64_t qd = q_desc0 + (uint64_t)(t * (C::QTILE >> 4));
                const uint64_t kd = kd0 + (uint64_t)(h * ((kHalf * 128) >> 4));
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                  const uint64_t off = (uint64_t)(((ks >> 2) * C::SLAB_TILE + (ks & 3) * 32) >> 4);
                  umma_ss(dS, qd + off, kd + off, idesc_s, ks > 0);
                }
                umma_commit(bar_s + 8 * (2 * t + h));
                if (h == 1 && t == 1) umma_commit(smem_u32(k_empty + sn));
              }
            }
            half_ph ^= 0xFu;
            continue;
          }
          // ---- first / last tiles of an item, ragged halves, single Q tile
          const int nh = min(2, nhalf - 2 * j);                            // halves of this tile
          const int nhn = j + 1 < ntiles ? min(2, nhalf - 2 * j - 2) : 0;   // halves of the next one
          bool k_ready = false;
          for (int h = 0; h < nh; ++h) {
            const int i = 2 * j + h;
            const int ksteps = (i + 1 < nhalf ? kHalf : last_cols) / 16;
            for (int t = 0; t < nt; ++t) {
              mbar_wait(bar_p + 8 * (2 * t + h), (half_ph >> (2 * t + h)) & 1, p.status);
              half_ph ^= 1u << (2 * t + h);
              if (h < nhn && !k_ready) {
                mbar_wait(smem_u32(k_full + sn), phn, p.status);
                k_ready = true;
              }
              if (i == 0) mbar_wait(smem_u32(o_free + t), ((ph_item >> t) & 1) ^ 1, p.status);  // the previous epilogue has drained O_t
              tc_fence_after();
              const uint64_t vd = v_desc0 + (uint64_t)(s * (C::KVTILE >> 4) + h * (kHalf / 16) * 128);
              const uint32_t dO = tmem + 256 + t * D, aP = tmem + t * 128 + h * kHalf;
              for (int ks = 0; ks < ksteps; ++ks)
                umma_ts(dO, aP + ks * 8, vd + (uint64_t)(ks * 128), idesc_pv, (i > 0 || ks > 0) ? 1u : 0u);
              umma_commit(bar_pv + 8 * t);
              if (h == nh - 1 && t == nt - 1) umma_commit(smem_u32(v_empty + s));
              if (i + 1 == nhalf) umma_commit(smem_u32(o_done + t));
              if (h < nhn) {   // S_t^h of the next tile goes into the columns this PV frees
                issue_s(t, i + 2, sn);
                if (h == nhn - 1 && t == nt - 1) umma_commit(smem_u32(k_empty + sn));
              }
            }
          }
          if (j + 2 == ntiles)   // the S MMAs of the last tile are all issued: Q may be replaced once they are done
            for (int t = 0; t < nt; ++t) umma_commit(smem_u32(q_free + t));
        }
        tile_cnt += ntiles;
      }
    }
  } else if (warp >= 10) {
    // ================================================================ Q loader (warp 10)
    // Runs one item ahead: the next item's Q rows go into shared memory (K-major, 128-byte
    // swizzle) as soon as the S MMAs of the current item no longer read the tile.  A Q tile is
    // the box (64 dims, G heads of the group, 128 / G tokens) of the Q tensor: two TMA loads per
    // tile (one per 64-dim slab) when 128 is a multiple of G; plain 16-byte asynchronous copies
    // otherwise.
    uint32_t n_t[2] = {0, 0};   // items Q tile t took part in
    const int G = p.G;
    if (use_qmap && lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&qmap) : "memory");
    for (int it = it0; it < it1; ++it) {
      const PieItem item = p.items[it];
      if (item.page_end == item.page_begin) continue;
      const int nt = item.nrows > kTileM ? 2 : 1;
      for (int t = 0; t < nt; ++t) {
        mbar_wait(smem_u32(q_free + t), (n_t[t & 1] & 1) ^ 1, p.status);
        ++n_t[t & 1];
        if (use_qmap) {
          if (elect_one()) {
            mbar_expect_tx(smem_u32(q_full + t), C::QTILE);
            const int tok0 = item.q_start + (item.row0 + t * kTileM) / G;   // row0 is a multiple of the tile height
#pragma unroll
            for (int sl = 0; sl < C::NSLAB; ++sl)
              tma_load_3d(smem_u32(sQ + t * C::QTILE + sl * C::SLAB_TILE), &qmap, sl * 64, item.kv_head * G, tok0, smem_u32(q_full + t));
          }
          __syncwarp();
        } else {
          constexpr int CPR = D * 2 / 16;        // 16-byte chunks per row
          constexpr int RPI = 32 / CPR;          // rows per warp instruction
          const int ch = lane % CPR;
          const char* qbase = reinterpret_cast<const char*>(p.q) + ((int64_t)item.q_start * p.n_q_heads + item.kv_head * G) * (D * 2) + ch * 16;
          const uint32_t dst0 = smem_u32(sQ + t * C::QTILE + (ch >> 3) * C::SLAB_TILE);
#pragma unroll 4
          for (int r = 0; r < kTileM; r += RPI) {
            const int row = r + lane / CPR, gr = t * kTileM + row;   // row inside the tile / the item
            const bool ok = gr < item.nrows;
            const int tok = (item.row0 + gr) / G, hg = (item.row0 + gr) % G;
            const char* src = ok ? qbase + ((int64_t)tok * p.n_q_heads + hg) * (D * 2) : qbase;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst0 + row * 128 + (((ch & 7) ^ (row & 7)) << 4)),
                         "l"(__cvta_generic_to_global(src)), "r"(ok ? 16 : 0)
                         : "memory");
          }
          asm volatile("cp.async.wait_all;" ::: "memory");
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(q_full + t));
        }
      }
    }
  } else {
    // ================================================================ softmax warpgroups
    const int t = warp >> 2;                       // Q tile of this warpgroup
    const int rho = (warp & 3) * 32 + lane;        // row inside the tile = TMEM lane
    const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + t * 128 + lane_sel, tO = tmem + 256 + t * D + lane_sel;
    uint32_t my_items = 0;   // phase of o_done
    uint32_t s_ph = 0;       // bit h: phase of s_full[t][h]
    uint32_t n_arr = 0;      // p_full arrivals so far = PV groups of this Q tile issued or about to be
    // The record of the next item is fetched before the wait for the last PV of the current one, so that its
    // latency is not added to the gap between two items (where the tensor pipe is idle).
    PieItem item_nxt = PieItem{};
    if (it0 < it1) item_nxt = p.items[it0];
    for (int it = it0; it < it1; ++it) {
      const PieItem item = item_nxt;
      const int npages = item.page_end - item.page_begin;
      const int nhalf = (npages + C::PPH - 1) / C::PPH;
      const int nt = item.nrows > kTileM ? 2 : 1;
      if (t >= nt) {
        if (it + 1 < it1) item_nxt = p.items[it + 1];
        continue;
      }
      const int gr = item.row0 + t * kTileM + rho;
      const bool valid = gr < item.row0 + item.nrows;
      const int tok = valid ? gr / p.G : 0;
      const int head = item.kv_head * p.G + (valid ? gr % p.G : 0);
      const int64_t oi = (int64_t)(item.q_start + tok) * p.n_q_heads + head;
      const int lim = valid ? item.kv_len - item.q_len + tok : -1;
      const uint32_t* mrow = p.mask + item.mask_word_off + (int64_t)tok * item.mask_row_words;
      const bool explicit_mask = item.mask_row_words != 0;
      float m_ref = kNegInf, l_sum = 0.f;

      if (nhalf > 0) {
        // Page records (logical page | needs-mask flag; same addresses for all threads) and the
        // allowed-position bits of this row run two halves ahead of the softmax.  The loads are
        // volatile so that they are issued here and not next to their first use, where their
        // latency would be exposed on every half.
        const int2* krec = p.kept + item.page_begin;
        auto load_recs = [&](int i, uint32_t* rec) {
#pragma unroll
          for (int g = 0; g < C::PPH; ++g) {
            const int pg = i * C::PPH + g;
            rec[g] = 0xFFFFFFFFu;   // all ones: no such page
            if (pg < npages) rec[g] = ldg_early(reinterpret_cast<const uint32_t*>(&krec[pg].y));
          }
        };
        auto make_bits = [&](const uint32_t* rec, uint32_t* bits) -> bool {
          uint32_t any = valid ? 0u : PIE_KEPT_NEEDS_MASK;
#pragma unroll
          for (int g = 0; g < C::PPH; ++g) any |= rec[g];
          if (!(any & PIE_KEPT_NEEDS_MASK)) return false;   // common case: every page fully visible (warp-uniform unless rows are padding)
#pragma unroll
          for (int g = 0; g < C::PPH; ++g) {
            const uint32_t lpf = rec[g];
            bits[g] = 0xFFFFFFFFu;
            if (lpf == 0xFFFFFFFFu || !valid) {
              bits[g] = 0u;
            } else if (lpf & PIE_KEPT_NEEDS_MASK) {
              const int j0 = (int)(lpf & ~PIE_KEPT_NEEDS_MASK) * P;
              if (explicit_mask) bits[g] = ldg_early(mrow + (j0 >> 5)) >> (j0 & 31);
              else bits[g] = lim >= j0 + P - 1 ? 0xFFFFFFFFu : (lim < j0 ? 0u : ((1u << (lim - j0 + 1)) - 1u));
            }
          }
          return true;
        };
        // Halves that lie inside the item's clean prefix (pages every row of the tile sees in full,
        // counted by the planner) need neither records nor bits; the look-ahead starts two halves
        // before the first half that does.
        const int clean_halves = (int)(item.flags >> PIE_ITEM_CLEAN_SHIFT) / C::PPH;
        uint32_t rec_nxt[C::PPH], bits_nxt[C::PPH], bits[C::PPH];
#pragma unroll
        for (int g = 0; g < C::PPH; ++g) bits_nxt[g] = 0xFFFFFFFFu;
        bool mask_nxt = false;
        if (clean_halves <= 0) {
          load_recs(0, rec_nxt);
          mask_nxt = make_bits(rec_nxt, bits_nxt);
        }
        if (clean_halves <= 1) load_recs(1, rec_nxt);

        // P = exp2(x * scale - m) for one chunk of 32 columns: bf16 pairs into pk, the sums onto sa / sb.
        auto exp_chunk = [&](const float* x, const uint64_t scale2, const uint64_t negm2, uint64_t& sa, uint64_t& sb, uint32_t* pk) {
#pragma unroll
          for (int c = 0; c < 32; c += 4) {
            float e0, e1, e2, e3;
            unpack_f32x2(fma_f32x2(pack_f32x2(x[c], x[c + 1]), scale2, negm2), e0, e1);
            unpack_f32x2(fma_f32x2(pack_f32x2(x[c + 2], x[c + 3]), scale2, negm2), e2, e3);
            const float p0 = fast_exp2(e0), p1 = fast_exp2(e1), p2 = fast_exp2(e2), p3 = fast_exp2(e3);
            sa = add_f32x2(sa, pack_f32x2(p0, p1));
            sb = add_f32x2(sb, pack_f32x2(p2, p3));
            pk[c >> 1] = pack_bf16(p0, p1);
            pk[(c >> 1) + 1] = pack_bf16(p2, p3);
          }
        };
        // One half of the item.  The body exists twice: a lean copy for the halves of the clean
        // prefix (no records, no bits, no masking code in the loop) and the general one.
        auto do_half = [&](const int i, auto masked_tag) {
          constexpr bool kMasked = decltype(masked_tag)::value;
          const int h = i & 1;
          const uint32_t tSh = tS + h * kHalf;
          bool half_mask = false;
          if constexpr (kMasked) {
            half_mask = mask_nxt;
#pragma unroll
            for (int g = 0; g < C::PPH; ++g) bits[g] = bits_nxt[g];
            mask_nxt = false;
            if (i + 1 >= clean_halves) mask_nxt = make_bits(rec_nxt, bits_nxt);   // half i + 1 (all "no such page" past the end)
            if (i + 2 >= clean_halves) load_recs(i + 2, rec_nxt);
          }

          mbar_wait(smem_u32(s_full + 2 * t + h), (s_ph >> h) & 1, p.status);
          s_ph ^= 1u << h;
          tc_fence_after();
          // ---- one pass over the half in 32-column chunks (online softmax with a lagging reference):
          // P = exp2(S * scale - m_ref) goes back as bf16 over the first 32 columns of S_t^h.  m_ref may
          // lag the true running maximum by up to 2^8; when a chunk exceeds that (rare after the first
          // chunk of an item), O_t, the sums and the P chunk already written for this half are brought
          // to the new reference.  Scale-and-shift and the row sum use packed fp32x2 arithmetic.
          uint64_t psum_a = pack_f32x2(0.f, 0.f), psum_b = pack_f32x2(0.f, 0.f);
          const uint64_t scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
          float xbuf[2][32];   // double buffer: chunk 1 is in flight while chunk 0 is processed
          tmem_ld32(tSh, reinterpret_cast<uint32_t*>(xbuf[0]));
          tmem_wait_ld();
#pragma unroll
          for (int k = 0; k < kHalf / 32; ++k) {
            float* x = xbuf[k & 1];
            if (k + 1 < kHalf / 32) tmem_ld32(tSh + (k + 1) * 32, reinterpret_cast<uint32_t*>(xbuf[(k + 1) & 1]));
            if (kMasked && half_mask) {
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (!((bits[(k * 32 + c) / P] >> ((k * 32 + c) % P)) & 1u)) x[c] = kNegInf;
            }
            // Lean form (the whole of the lean copy; in the general copy the first attempt on every chunk, masked
            // scores being -inf by now - the halves around an item's first masked page and the diagonal of a
            // causal chunk are a quarter of a short item): no maximum is taken while the sums stay small.  The exponentials are computed
            // against the current reference straight away; the chunk's sum bounds its largest term, so a
            // sum below 2^16 proves that no score runs ahead of the reference by more than 16 binades
            // (fp32 sums and bf16 P keep their relative precision at any such lag).  Otherwise - or when a
            // row of the warp has no reference yet - the chunk is redone the careful way below.
            if constexpr (!kMasked || P != 8) {   // (with 8-token pages the general loop has no registers left for it)
              if (__all_sync(0xFFFFFFFFu, m_ref != kNegInf)) {
                const uint64_t negm2 = pack_f32x2(-m_ref, -m_ref);
                uint64_t ca = pack_f32x2(0.f, 0.f), cb = pack_f32x2(0.f, 0.f);
                uint32_t pk[16];
                exp_chunk(x, scale2, negm2, ca, cb, pk);
                float s0, s1;
                unpack_f32x2(add_f32x2(ca, cb), s0, s1);
                if (!__any_sync(0xFFFFFFFFu, !(s0 + s1 <= 65536.f))) {   // (also catches inf and NaN)
                  psum_a = add_f32x2(psum_a, ca);
                  psum_b = add_f32x2(psum_b, cb);
                  tmem_st16(tSh + k * 16, pk);
                  if (k + 1 < kHalf / 32) tmem_wait_ld();
                  continue;
                }
              }
            }
            float cm0 = max3(x[0], x[1], x[2]), cm1 = max3(x[3], x[4], x[5]);   // two chains
#pragma unroll
            for (int c = 6; c < 30; c += 4) {
              cm0 = max3(cm0, x[c], x[c + 1]);
              cm1 = max3(cm1, x[c + 2], x[c + 3]);
            }
            const float cmax = fmaxf(max3(cm0, x[30], x[31]), cm1);
            const float m_new = fmaxf(m_ref, cmax * p.scale_log2);   // -inf stays -inf
            if (__any_sync(0xFFFFFFFFu, m_new > m_ref + 8.f)) {       // also when m_ref is -inf and m_new finite
              const float f = (m_ref == kNegInf) ? 1.f : fast_exp2(m_ref - m_new);
              if (m_new != kNegInf) m_ref = m_new;
              l_sum *= f;
              psum_a = fma_f32x2(psum_a, pack_f32x2(f, f), pack_f32x2(0.f, 0.f));
              psum_b = fma_f32x2(psum_b, pack_f32x2(f, f), pack_f32x2(0.f, 0.f));
              if (i > 0) {
                // O_t holds the PV groups of halves 0..i-1; the latest may still be running.  All but
                // the latest are known complete (S_t^h of this half was issued after them), so the
                // barrier is at most one phase behind and the parity wait is unambiguous.
                mbar_wait(smem_u32(pv_done + t), (n_arr - 1) & 1, p.status);
                tc_fence_after();
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 16) {
                  uint32_t o[16];
                  tmem_ld16(tO + c0, o);
                  tmem_wait_ld();
#pragma unroll
                  for (int c = 0; c < 16; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
                  tmem_st16(tO + c0, o);
                }
              }
#pragma unroll 1
              for (int kk = 0; kk < k; ++kk) {   // P chunks of this half written under the old reference
                uint32_t pp[16];
                tmem_wait_st();
                tmem_ld16(tSh + kk * 16, pp);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                  const float lo = __uint_as_float(pp[c] << 16) * f, hi = __uint_as_float(pp[c] & 0xFFFF0000u) * f;
                  pp[c] = pack_bf16(lo, hi);
                }
                tmem_st16(tSh + kk * 16, pp);
              }
              tmem_wait_st();
            }
            const float neg_m = (m_ref == kNegInf) ? 0.f : -m_ref;
            const uint64_t negm2 = pack_f32x2(neg_m, neg_m);
            uint32_t pk[16];
            exp_chunk(x, scale2, negm2, psum_a, psum_b, pk);
            tmem_st16(tSh + k * 16, pk);   // columns [16k, 16k+16): below every S column still to be read
            if (k + 1 < kHalf / 32) tmem_wait_ld();
          }
          {
            float s0, s1;
            unpack_f32x2(add_f32x2(psum_a, psum_b), s0, s1);
            l_sum += s0 + s1;
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(smem_u32(p_full + 2 * t + h));
          ++n_arr;
        };
        const int n_lean = min(nhalf, max(0, clean_halves - 2));   // (the look-ahead of the general loop starts two halves early)
        for (int i = 0; i < n_lean; ++i) do_half(i, std::false_type{});
        for (int i = n_lean; i < nhalf; ++i) do_half(i, std::true_type{});
        if (it + 1 < it1) item_nxt = p.items[it + 1];
        mbar_wait(smem_u32(o_done + t), my_items & 1, p.status);
        ++my_items;
        tc_fence_after();
      }

      if (nhalf == 0 && it + 1 < it1) item_nxt = p.items[it + 1];
      // ---- epilogue: normalise, store
      const bool live = m_ref != kNegInf && l_sum > 0.f;   // a row with no allowed position: O = 0, LSE = -inf
      const float inv = live ? 1.f / l_sum : 0.f;
      const float lse = live ? (m_ref + log2f(l_sum)) * kLn2 : kNegInf;
      // A full tile of final rows leaves through shared memory: every thread converts its row, 64 columns at a
      // time, into the warpgroup's staging slab (the swizzled image of the box 64 dims x G heads x 128 / G tokens
      // of the output tensor) and one thread hands the slab to a TMA store.  The accumulator is free for the next
      // item as soon as it has been read into registers, and the stores to global memory run while the warpgroup
      // is already in the next item's softmax - the epilogue sits between the last MMA of an item and the first
      // of the next, so every cycle of it is idle tensor-pipe time.  (All conditions are uniform over the
      // warpgroup: the barriers below always see their 128 threads.)
      const bool via_tma = use_omap && nhalf > 0 && item.partial_slot < 0 && item.nrows >= (t + 1) * kTileM;
      if (via_tma) {
        const uint32_t stg = smem_u32(sO + t * C::OSLAB) + rho * 128;
        const bool lead = (warp & 3) == 0;
        const int tok0 = item.q_start + (item.row0 + t * kTileM) / p.G;
        auto sync_wg = [&]() {
          if (t == 0) wg_sync<1>();
          else wg_sync<2>();
        };
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t o[32];
          tmem_ld32(tO + c0, o);
          tmem_wait_ld();
          if (c0 + 32 == D) {   // O_t is in registers: the next item's PV may overwrite it
            tc_fence_before();
            mbar_arrive(smem_u32(o_free + t));
          }
          uint32_t w[16];
#pragma unroll
          for (int c = 0; c < 32; c += 2) w[c >> 1] = pack_bf16(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
          if ((c0 & 63) == 0) {   // the slab's previous store must have read it before it is overwritten
            if (lead) {
              if (elect_one()) bulk_wait_read();
              __syncwarp();
            }
            sync_wg();
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int ch = ((c0 & 63) >> 3) + k;   // 16-byte chunk of the row inside the slab
            st_shared_v4(stg + ((ch ^ (rho & 7)) << 4), w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]);
          }
          if ((c0 & 63) == 32) {
            fence_async_smem();
            sync_wg();
            if (lead) {
              if (elect_one()) {
                tma_store_3d(&omap, smem_u32(sO + t * C::OSLAB), c0 & ~63, item.kv_head * p.G, tok0);
                bulk_commit();
              }
              __syncwarp();
            }
          }
        }
        p.lse[oi] = lse;
      } else {
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t o[32];
          if (nhalf > 0) {
            tmem_ld32(tO + c0, o);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] = 0u;
          }
          if (valid) {
            if (item.partial_slot < 0) {
              // 32-byte stores: every thread writes its own row, so the store path is bound by the number
              // of (thread, instruction) pairs, not by bytes
              __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + oi * D + c0;
              uint32_t w[16];
#pragma unroll
              for (int c = 0; c < 32; c += 2) w[c >> 1] = pack_bf16(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
              if (out_wide) {
                st_global_v8(dst, w);
                st_global_v8(dst + 16, w + 8);
              } else {
#pragma unroll
                for (int c = 0; c < 16; c += 4) reinterpret_cast<uint4*>(dst)[c >> 2] = make_uint4(w[c], w[c + 1], w[c + 2], w[c + 3]);
              }
            } else {
              float* dst = p.ws_o + ((int64_t)item.partial_slot * 256 + (gr - item.row0)) * D + c0;
#pragma unroll
              for (int c = 0; c < 32; c += 8) {
                uint32_t w[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) w[k] = __float_as_uint(__uint_as_float(o[c + k]) * inv);
                st_global_v8(dst + c, w);
              }
            }
          }
        }
        if (valid) {
          if (item.partial_slot < 0) p.lse[oi] = lse;
          else p.ws_lse[(int64_t)item.partial_slot * 256 + (gr - item.row0)] = lse;
        }
        if (nhalf > 0) {
          tc_fence_before();
          mbar_arrive(smem_u32(o_free + t));
        }
      }
    }
    // the last output tiles must have left shared memory (and reached global memory) before the block ends
    if ((warp & 3) == 0) {
      if (elect_one()) bulk_wait_all();
      __syncwarp();
    }
  }

  // ---- teardown: everyone is done with TMEM before it is released
  if (p.late_trigger) pie_pdl_launch_dependents();
  tc_fence_before();
  __syncthreads();
  if (warp == 8) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

}  // namespace
bool pie_tc_supported(const pie_ctx* ctx) {
  const pie_config& c = ctx->cfg;
  return c.dtype == PIE_DTYPE_BF16 && (c.page_size == 8 || c.page_size == 16 || c.page_size == 32) &&
         (c.head_dim == 64 || c.head_dim == 128);
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// Tensor map of Q [tokens][q heads][D] (bf16) whose box is one Q tile: 64 dims x G heads x 128/G
// tokens, 128-byte swizzle.  Returns false when the shape does not fit (128 not a multiple of G,
// unaligned pointer): the kernel then loads Q with plain asynchronous copies.
static bool make_q_map(const pie_ctx* ctx, const void* q, int64_t n_tokens, int G, CUtensorMap* map) {   // (also the map of the output tensor: same shape)
  const int D = ctx->cfg.head_dim, Hq = ctx->cfg.num_q_heads;
  if (G <= 0 || kTileM % G != 0 || n_tokens <= 0 || (reinterpret_cast<uintptr_t>(q) & 15) != 0) return false;
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t gdim[3] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)n_tokens};
  const cuuint64_t gstride[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hq * D * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(kTileM / G)};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int P>
static int launch_tc(pie_ctx* ctx, const AttnParams& p, int grid, int64_t n_tokens, cudaStream_t s) {
  using C = TcCfg<D, P>;
  auto kern = attn_tc_kernel<D, P>;
  if (!ctx->tc_configured) {   // (a context has one shape, hence one instantiation, and one device)
    PIE_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
    ctx->tc_configured = true;
  }
  CUtensorMap qmap, omap;
  memset(&qmap, 0, sizeof(qmap));
  memset(&omap, 0, sizeof(omap));
  const int kflags = (make_q_map(ctx, p.q, n_tokens, p.G, &qmap) ? 1 : 0) | ((reinterpret_cast<uintptr_t>(p.out) & 31) == 0 ? 2 : 0) |
                     (make_q_map(ctx, p.out, n_tokens, p.G, &omap) ? 4 : 0);
  PIE_CUDA(ctx, pie_launch_pdl(kern, dim3(grid), dim3(kThreads), C::SMEM, s, p, qmap, omap, kflags));
  return PIE_OK;
}

int pie_launch_tc_tiles(pie_ctx* ctx, const AttnParams& p, int grid, int64_t n_tokens, cudaStream_t s) {
  const int D = ctx->cfg.head_dim, P = ctx->cfg.page_size;
  if (D == 128 && P == 8) return launch_tc<128, 8>(ctx, p, grid, n_tokens, s);
  if (D == 64 && P == 8) return launch_tc<64, 8>(ctx, p, grid, n_tokens, s);
  if (D == 128 && P == 16) return launch_tc<128, 16>(ctx, p, grid, n_tokens, s);
  if (D == 64 && P == 16) return launch_tc<64, 16>(ctx, p, grid, n_tokens, s);
  if (D == 128 && P == 32) return launch_tc<128, 32>(ctx, p, grid, n_tokens, s);
  if (D == 64 && P == 32) return launch_tc<64, 32>(ctx, p, grid, n_tokens, s);
  return PIE_ERR_UNSUPPORTED;
}
