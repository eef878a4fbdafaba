// Attention kernels of the `forward` handler (Section 4.2 "Forward API": attention over the
// request's KvPages under an explicit or inferred mask):
//   * attn_split_kernel - decode: split-KV over scattered pages, HBM bound.  Every warp is an
//     independent pipeline: it streams its share of (page, kv head) blocks into a private
//     shared-memory ring with bulk async copies, runs QK^T / PV on tensor cores with the
//     grouped query heads stacked in the M dimension, and writes a final row or an fp32 partial.
//   * attn_tile_kernel  - row tiles (prefill chunks, token trees): each consumer warp owns 16
//     query rows and every warp walks the same page stream filled by a producer warp.
//   * merge_kernel                 - LSE-weighted merge of split partials.
//   * simple_kernel                - plain CUDA-core kernel (fp32 pools and shapes the tile
//     kernels do not cover); one warp per (token, head) row, sequential online softmax.
#include <cuda_bf16.h>

#include <cstring>
#include <type_traits>

#include "pie_internal.h"
#include "ptx_helpers.cuh"

namespace {

// ------------------------------------------------------------------------------ PTX helpers
using namespace pie_ptx;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
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

// ------------------------------------------------------------------------------ warp-level core
// One warp attends 16 query rows (row = query token * G + head-in-group, for one kv head) over a
// stream of KvPage blocks.  Per thread: rows r_lo = lane/4 and r_lo + 8, columns cpair, cpair+1
// of every 8-wide block (the m16n8k16 accumulator layout).
template <int D>
struct RowState {
  uint32_t qf[D / 16][4];  // Q fragments (A operand)
  float o[D / 8][4];       // un-normalised output accumulators
  float m_run[2], l_run[2];
  int lim[2];              // last visible position under the inferred causal mask (-1: no row)
  const uint32_t* mrow[2]; // packed explicit mask row
  bool valid[2];
  int hsel[2];             // head of the row inside its unit (units of two adjacent kv heads; else 0)
  bool explicit_mask;
  bool any_rows;
};

template <int D>
__device__ __forceinline__ void rows_init(RowState<D>& st, const AttnParams& p, const PieItem& item, const PieReq& rq,
                                          int rbase, int lane) {
  const int r_lo = lane >> 2, cpair = (lane & 3) * 2;
  const int row_end = item.row0 + item.nrows;
  st.explicit_mask = rq.mask_row_words != 0;
  st.any_rows = rbase < row_end;
  const __nv_bfloat16* qptr[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int gr = rbase + r_lo + r * 8;
    st.valid[r] = gr < row_end;
    const int tok = st.valid[r] ? gr / p.G : 0;
    const int head = item.kv_head * p.G + (st.valid[r] ? gr % p.G : 0);
    st.lim[r] = st.valid[r] ? rq.kv_len - rq.q_len + tok : -1;
    st.hsel[r] = st.valid[r] ? (gr % p.G) / p.G_head : -1;
    st.mrow[r] = p.mask + rq.mask_word_off + (int64_t)tok * rq.mask_row_words;
    qptr[r] = reinterpret_cast<const __nv_bfloat16*>(p.q) + ((int64_t)(rq.q_start + tok) * p.n_q_heads + head) * D;
    st.m_run[r] = kNegInf;
    st.l_run[r] = 0.f;
  }
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      uint32_t lo = 0, hi = 0;
      if (st.valid[r]) {
        lo = __ldg(reinterpret_cast<const uint32_t*>(qptr[r] + ks * 16 + cpair));
        hi = __ldg(reinterpret_cast<const uint32_t*>(qptr[r] + ks * 16 + 8 + cpair));
      }
      st.qf[ks][r] = lo;
      st.qf[ks][2 + r] = hi;
    }
  }
#pragma unroll
  for (int nb = 0; nb < D / 8; ++nb) st.o[nb][0] = st.o[nb][1] = st.o[nb][2] = st.o[nb][3] = 0.f;
}

// Attend the warp's rows to one visit resident in shared memory: PPV pages, each a K block then a V
// block ([slab][slot][128 B] with the 16-byte chunks XOR-swizzled by slot & 7), handled in steps of 16
// tokens (one m16n8k16 k-step of P V).  Pages of 16 or 32 tokens are one visit each; pages of 8 tokens
// come in pairs, so that a step is filled by two pages (lpf[i] = logical page | needs-mask flag of page i,
// 0xFFFFFFFF when the visit has no page i: the odd page at the end of a piece).
// HP = 2: the unit is a PAIR of adjacent kv heads (their blocks of a page are contiguous in the pool, so one
// copy of twice the size brings both).  Rows of the first head take their scores from the first head's K
// and their probabilities meet only its V; likewise for the second: two sets of MMAs, one softmax.
#define PIE_NO_PAGE 0xFFFFFFFFu
template <int D, int P, int PPV, int HP>
__device__ __forceinline__ void visit_compute(RowState<D>& st, uint8_t* stage, const PieReq& rq, const uint32_t* lpf,
                                              float scale_log2, int lane) {
  constexpr int KSTEPS = D / 16, VT = P * PPV, SUBS = VT / 16, BLK = P * D * 2, SLAB = P * 128, PAGE = 2 * BLK;
  constexpr int VP = HP * PAGE;   // bytes of one page in the stage: the blocks of its HP heads
  constexpr int PIECES = P >= 16 ? 1 : 16 / P, PW = 16 / PIECES;   // a 16-token step is made of PIECES runs of PW tokens, each inside one page
  static_assert(VT % 16 == 0, "a visit is a whole number of 16-token steps");
  const int cpair = (lane & 3) * 2;
  const uint32_t sbase = smem_u32(stage);

#pragma unroll
  for (int i = 0; i < PPV; ++i) {
    // slots past the end of the context (and a page the visit does not have) may hold anything: clear their V
    // rows so that a zero probability times a NaN bit pattern cannot leak into the output
    int first_bad = P;
    if (lpf[i] == PIE_NO_PAGE) first_bad = 0;
    else if ((int)(lpf[i] & ~PIE_KEPT_NEEDS_MASK) == rq.last_logical && rq.last_page_len < P) first_bad = rq.last_page_len;
    if (first_bad < P) {
      constexpr int CH = D * 2 / 16;
      const int nz = (P - first_bad) * CH;
#pragma unroll
      for (int hh = 0; hh < HP; ++hh)
        for (int c = lane; c < nz; c += 32) {
          const int t = first_bad + c / CH, ch = c % CH;
          *reinterpret_cast<uint4*>(stage + i * VP + hh * PAGE + BLK + pie_chunk_offset(SLAB, t, ch)) = make_uint4(0, 0, 0, 0);
        }
      // these generic-proxy writes must be ordered before the bulk copy that later refills the stage
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
    }
  }
  if (!st.any_rows) return;

#pragma unroll
  for (int sub = 0; sub < SUBS; ++sub) {
    uint32_t bits[2] = {0u, 0u};
    bool needs_mask = false;
#pragma unroll
    for (int pc = 0; pc < PIECES; ++pc) {
      const int pg = (sub * 16 + pc * PW) / P, off = (sub * 16 + pc * PW) % P;
      const uint32_t l = lpf[pg], full = (1u << PW) - 1u;
      uint32_t piece[2] = {full, full};
      if (l == PIE_NO_PAGE) {
        needs_mask = true;
        piece[0] = piece[1] = 0u;
      } else if (l & PIE_KEPT_NEEDS_MASK) {
        needs_mask = true;
        const int j0 = (int)(l & ~PIE_KEPT_NEEDS_MASK) * P + off;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          if (!st.valid[r]) piece[r] = 0u;
          else if (st.explicit_mask) piece[r] = (__ldg(st.mrow[r] + (j0 >> 5)) >> (j0 & 31)) & full;
          else piece[r] = st.lim[r] >= j0 + PW - 1 ? full : (st.lim[r] < j0 ? 0u : ((1u << (st.lim[r] - j0 + 1)) - 1u));
        }
      }
      bits[0] |= piece[0] << (pc * PW);
      bits[1] |= piece[1] << (pc * PW);
    }
    if (needs_mask && __all_sync(0xFFFFFFFFu, (bits[0] | bits[1]) == 0)) continue;  // nothing visible to this warp
    // ---- S = Q K^T for 16 tokens
    float sacc[2][4];
    {
      float sh[HP][2][4];
      const int t = sub * 16 + ((lane >> 4) << 3) + (lane & 7);   // token of the visit whose K row this lane addresses
      const uint32_t rowaddr = sbase + (t / P) * VP + (t % P) * 128;
      const int csel = (lane >> 3) & 1;
#pragma unroll
      for (int hh = 0; hh < HP; ++hh) {
#pragma unroll
        for (int e = 0; e < 4; ++e) sh[hh][0][e] = sh[hh][1][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
          const int c = (ks & 3) * 2 + csel;
          uint32_t b0, b1, b2, b3;
          ldsm_x4(rowaddr + hh * PAGE + (ks >> 2) * SLAB + ((c ^ (t & 7)) << 4), b0, b1, b2, b3);
          mma_bf16(sh[hh][0], st.qf[ks], b0, b1);
          mma_bf16(sh[hh][1], st.qf[ks], b2, b3);
        }
      }
#pragma unroll
      for (int nb = 0; nb < 2; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) sacc[nb][e] = (HP > 1 && st.hsel[e >> 1] == 1) ? sh[HP - 1][nb][e] : sh[0][nb][e];
    }
    // ---- mask, online softmax (base-2 domain)
    float mx[2] = {kNegInf, kNegInf};
#pragma unroll
    for (int nb = 0; nb < 2; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = e >> 1, col = nb * 8 + cpair + (e & 1);
        float v = sacc[nb][e] * scale_log2;
        if (needs_mask && !((bits[r] >> col) & 1u)) v = kNegInf;
        sacc[nb][e] = v;
        mx[r] = fmaxf(mx[r], v);
      }
    float alpha[2], m_use[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 2));
      const float m_new = fmaxf(st.m_run[r], mx[r]);
      m_use[r] = (m_new == kNegInf) ? 0.f : m_new;
      alpha[r] = fast_exp2(st.m_run[r] - m_use[r]);
      st.m_run[r] = m_new;
    }
    float psum[2] = {0.f, 0.f};
#pragma unroll
    for (int nb = 0; nb < 2; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float pv = fast_exp2(sacc[nb][e] - m_use[e >> 1]);
        sacc[nb][e] = pv;
        psum[e >> 1] += pv;
      }
    st.l_run[0] = st.l_run[0] * alpha[0] + psum[0];
    st.l_run[1] = st.l_run[1] * alpha[1] + psum[1];
#pragma unroll
    for (int nb = 0; nb < D / 8; ++nb) {
      st.o[nb][0] *= alpha[0];
      st.o[nb][1] *= alpha[0];
      st.o[nb][2] *= alpha[1];
      st.o[nb][3] *= alpha[1];
    }
    uint32_t pa[4];
    pa[0] = pack_bf16(sacc[0][0], sacc[0][1]);
    pa[1] = pack_bf16(sacc[0][2], sacc[0][3]);
    pa[2] = pack_bf16(sacc[1][0], sacc[1][1]);
    pa[3] = pack_bf16(sacc[1][2], sacc[1][3]);
    // ---- O += P V
    {
      const int t = sub * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
      const uint32_t rowaddr = sbase + (t / P) * VP + BLK + (t % P) * 128;
      const int csel = lane >> 4;
#pragma unroll
      for (int hh = 0; hh < HP; ++hh) {
        uint32_t ph[4] = {pa[0], pa[1], pa[2], pa[3]};
        if (HP > 1) {   // the probabilities of the other head's rows do not meet this head's V
          if (st.hsel[0] != hh) ph[0] = ph[2] = 0u;
          if (st.hsel[1] != hh) ph[1] = ph[3] = 0u;
        }
#pragma unroll
        for (int db = 0; db < KSTEPS; ++db) {
          const int c = (db & 3) * 2 + csel;
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(rowaddr + hh * PAGE + (db >> 2) * SLAB + ((c ^ (t & 7)) << 4), b0, b1, b2, b3);
          mma_bf16(st.o[2 * db], ph, b0, b1);
          mma_bf16(st.o[2 * db + 1], ph, b2, b3);
        }
      }
    }
  }
}

// One page per visit (pages of 16 or 32 tokens).
template <int D, int P>
__device__ __forceinline__ void page_compute(RowState<D>& st, uint8_t* stage, const PieReq& rq, uint32_t lpf,
                                             float scale_log2, int lane) {
  visit_compute<D, P, 1, 1>(st, stage, rq, &lpf, scale_log2, lane);
}

// Normalise and store the warp's rows: final bf16 output + LSE, or an fp32 partial for the merge.
template <int D>
__device__ __forceinline__ void rows_store(RowState<D>& st, const AttnParams& p, const PieItem& item, const PieReq& rq,
                                           int rbase, int slot_rows, int lane) {
  const int r_lo = lane >> 2, cpair = (lane & 3) * 2;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    st.l_run[r] += __shfl_xor_sync(0xFFFFFFFFu, st.l_run[r], 1);
    st.l_run[r] += __shfl_xor_sync(0xFFFFFFFFu, st.l_run[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (!st.valid[r]) continue;
    const int gr = rbase + r_lo + r * 8;
    const int tok = gr / p.G, head = item.kv_head * p.G + gr % p.G;
    const float L = st.l_run[r];
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const float lse = L > 0.f ? (st.m_run[r] + log2f(L)) * kLn2 : kNegInf;
    if (item.partial_slot < 0) {
      const int64_t oi = ((int64_t)(rq.q_start + tok) * p.n_q_heads + head);
      __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + oi * D;
#pragma unroll
      for (int nb = 0; nb < D / 8; ++nb)
        *reinterpret_cast<uint32_t*>(dst + nb * 8 + cpair) = pack_bf16(st.o[nb][2 * r] * inv, st.o[nb][2 * r + 1] * inv);
      if ((lane & 3) == 0) p.lse[oi] = lse;
    } else {
      const int64_t si = (int64_t)item.partial_slot * slot_rows + (gr - item.row0);
      float* dst = p.ws_o + si * D;
#pragma unroll
      for (int nb = 0; nb < D / 8; ++nb)
        *reinterpret_cast<float2*>(dst + nb * 8 + cpair) = make_float2(st.o[nb][2 * r] * inv, st.o[nb][2 * r + 1] * inv);
      if ((lane & 3) == 0) p.ws_lse[si] = lse;
    }
  }
}

// The same partial, written into shared memory (the warp's own, now idle, ring of stages) for a merge by
// another warp of the block: [16 rows][D] fp32, then 16 LSEs.
template <int D>
__device__ __forceinline__ void rows_store_smem(RowState<D>& st, float* base, int lane) {
  const int r_lo = lane >> 2, cpair = (lane & 3) * 2;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    st.l_run[r] += __shfl_xor_sync(0xFFFFFFFFu, st.l_run[r], 1);
    st.l_run[r] += __shfl_xor_sync(0xFFFFFFFFu, st.l_run[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (!st.valid[r]) continue;
    const int row = r_lo + r * 8;
    const float L = st.l_run[r];
    const float inv = L > 0.f ? 1.f / L : 0.f;
    float* dst = base + row * D;
#pragma unroll
    for (int nb = 0; nb < D / 8; ++nb)
      *reinterpret_cast<float2*>(dst + nb * 8 + cpair) = make_float2(st.o[nb][2 * r] * inv, st.o[nb][2 * r + 1] * inv);
    if ((lane & 3) == 0) base[16 * D + row] = L > 0.f ? (st.m_run[r] + log2f(L)) * kLn2 : kNegInf;
  }
}

// In-kernel merge of fp32 partial rows by one warp (the split-KV kernel's block-local and cross-block
// merges).  Sources: slot0, then slot0 + first, slot0 + first + stride, ... (n in all), combined in that
// order: lse = ln sum_c exp(lse_c), o = sum_c exp(lse_c - lse) o_c - whichever warp ends up doing it reads
// the same values in the same order, so results do not depend on timing.  dst_slot < 0: final rows (bf16
// output and LSE); else the combination is itself a partial and goes to that slot (which may be slot0:
// a lane reads exactly the addresses it later writes).  A merge is a handful of round trips to L2 and
// nothing else, so the rows of kBatch sources are fetched at once, all loads issued before the first is
// used.
struct MergeArgs {
  const float* ws_o;
  const float* ws_lse;
  float* ws_o_w;
  float* ws_lse_w;
  __nv_bfloat16* out;
  float* lse;
  int slot0, n, first, stride, dst_slot;
  int nrows, slot_rows, row0, kv_head, G, n_q_heads, q_start;
  const float* sm_base;   // SMEM variant: source c is the partial that warp (own + c) left in its ring
  int sm_stride;          // floats between the rings of consecutive warps
};
template <int D, bool SMEM>
__device__ __forceinline__ void merge_slots(const MergeArgs& a, int lane) {
  constexpr int kBatch = D == 64 ? 4 : 2;
  const int r_lo = lane >> 2, cpair = (lane & 3) * 2;
  auto slot_of = [&](int c) { return c == 0 ? a.slot0 : a.slot0 + a.first + a.stride * (c - 1); };
#pragma unroll 1
  for (int r = 0; r < 2; ++r) {
    const int row = r_lo + r * 8;   // row inside the unit
    if (row >= a.nrows) continue;
    float2 v[kBatch][D / 8];
    float l[kBatch];
    auto load = [&](int c0) {
#pragma unroll
      for (int u = 0; u < kBatch; ++u)
        if (c0 + u < a.n) {
          if constexpr (SMEM) {
            const float* src = a.sm_base + (size_t)(c0 + u) * a.sm_stride;
            l[u] = src[16 * D + row];
#pragma unroll
            for (int nb = 0; nb < D / 8; ++nb) v[u][nb] = *reinterpret_cast<const float2*>(src + row * D + nb * 8 + cpair);
          } else {
            const int64_t si = (int64_t)slot_of(c0 + u) * a.slot_rows + row;
            l[u] = __ldcg(a.ws_lse + si);
            const float* src = a.ws_o + si * D;
#pragma unroll
            for (int nb = 0; nb < D / 8; ++nb) v[u][nb] = __ldcg(reinterpret_cast<const float2*>(src + nb * 8 + cpair));
          }
        }
    };
    load(0);
    float M = kNegInf;
#pragma unroll 4
    for (int c = 0; c < a.n; ++c)
      M = fmaxf(M, SMEM ? a.sm_base[(size_t)c * a.sm_stride + 16 * D + row] : __ldcg(a.ws_lse + (int64_t)slot_of(c) * a.slot_rows + row));
    float Z = 0.f, acc[D / 8][2];
#pragma unroll
    for (int nb = 0; nb < D / 8; ++nb) acc[nb][0] = acc[nb][1] = 0.f;
    for (int c0 = 0; c0 < a.n; c0 += kBatch) {
      if (c0 > 0) load(c0);
#pragma unroll
      for (int u = 0; u < kBatch; ++u)
        if (c0 + u < a.n) {
          float wc = 0.f;
          if (M != kNegInf) wc = __expf(l[u] - M);
          Z += wc;
#pragma unroll
          for (int nb = 0; nb < D / 8; ++nb) {
            acc[nb][0] += wc * v[u][nb].x;
            acc[nb][1] += wc * v[u][nb].y;
          }
        }
    }
    const float invZ = Z > 0.f ? 1.f / Z : 0.f;
    const float lse = Z > 0.f ? M + logf(Z) : kNegInf;
    if (a.dst_slot < 0) {
      const int gr = a.row0 + row;
      const int tok = gr / a.G, head = a.kv_head * a.G + gr % a.G;
      const int64_t oi = ((int64_t)(a.q_start + tok) * a.n_q_heads + head);
      __nv_bfloat16* dst = a.out + oi * D;
#pragma unroll
      for (int nb = 0; nb < D / 8; ++nb)
        *reinterpret_cast<uint32_t*>(dst + nb * 8 + cpair) = pack_bf16(acc[nb][0] * invZ, acc[nb][1] * invZ);
      if ((lane & 3) == 0) a.lse[oi] = lse;
    } else {
      const int64_t si = (int64_t)a.dst_slot * a.slot_rows + row;
      float* dst = a.ws_o_w + si * D;
#pragma unroll
      for (int nb = 0; nb < D / 8; ++nb) *reinterpret_cast<float2*>(dst + nb * 8 + cpair) = make_float2(acc[nb][0] * invZ, acc[nb][1] * invZ);
      if ((lane & 3) == 0) a.ws_lse_w[si] = lse;
    }
  }
}

// What a split-KV warp still owes for a piece of a unit that is merged inside the kernel (PIE_ITEM_LOCAL_MERGER /
// PIE_ITEM_GRID_PIECE), once the piece's rows have been written as an fp32 partial.  It runs after the warp's
// last item: nothing of the attention loop is live any more, so this code does not weigh on the loop's registers
// (inlined at the end of every item it cost the loop spills and up to half its speed; as a call of its own, too).
template <int D, int NW>
__device__ __forceinline__ void split_piece_finish(const AttnParams& p, int item_idx, const float* ring, int ring_floats, int* local_cnt,
                                                   int lane) {
  const PieItem item = p.items[item_idx];
  const uint32_t fl = item.flags;
  MergeArgs margs;
  margs.sm_base = ring, margs.sm_stride = ring_floats;
  margs.ws_o = p.ws_o, margs.ws_lse = p.ws_lse, margs.ws_o_w = p.ws_o, margs.ws_lse_w = p.ws_lse;
  margs.out = reinterpret_cast<__nv_bfloat16*>(p.out), margs.lse = p.lse;
  margs.nrows = item.nrows, margs.slot_rows = p.slot_rows, margs.row0 = item.row0, margs.kv_head = item.kv_head;
  margs.G = p.G, margs.n_q_heads = p.n_q_heads, margs.q_start = item.q_start;
  if (fl & PIE_ITEM_LOCAL_MERGER) {
    const int gid = PIE_ITEM_LOCAL_GID(fl), np = PIE_ITEM_LOCAL_NP(fl);
    // wait (bounded) until the other pieces of the group have been written
    if (lane == 0) {
      volatile int* cnt = local_cnt + gid;
      uint64_t t0 = 0;
      for (uint32_t spin = 1; *cnt < np - 1; ++spin) {
        if ((spin & 255u) == 0) {
          if (*reinterpret_cast<volatile int*>(p.status) != 0) break;
          const uint64_t now = global_ns();
          if (t0 == 0) t0 = now;
          if (now - t0 > 1000000000ull) {
            atomicExch(p.status, (int)PIE_ERR_DEVICE_TIMEOUT);
            break;
          }
        }
      }
    }
    __syncwarp();
    __threadfence_block();
    margs.slot0 = item.partial_slot, margs.n = np, margs.first = 1, margs.stride = 1;
    margs.dst_slot = (fl & PIE_ITEM_GRID_PIECE) ? item.partial_slot : -1;
    if (fl & PIE_ITEM_LOCAL_SMEM) merge_slots<D, true>(margs, lane);
    else merge_slots<D, false>(margs, lane);
  }
  if (fl & PIE_ITEM_GRID_PIECE) {
    // make the block partial visible device-wide and count it; the warp that finds all other blocks of the
    // unit counted combines them (no warp waits for another block)
    const int nb = PIE_ITEM_GRID_NB(fl), kb = PIE_ITEM_GRID_KB(fl), n0 = PIE_ITEM_GRID_N0(fl);
    const int slot0 = item.partial_slot - (kb == 0 ? 0 : n0 + NW * (kb - 1));
    __threadfence();
    __syncwarp();
    int32_t* cnt = p.work_ctr + 2 + slot0;
    int seen = 0;
    if (lane == 0) seen = atomicAdd(cnt, 1);
    seen = __shfl_sync(0xFFFFFFFFu, seen, 0);
    if (seen == nb - 1) {
      __threadfence();
      if (lane == 0) *cnt = 0;   // re-armed for the next launch
      margs.slot0 = slot0, margs.n = nb, margs.first = n0, margs.stride = NW, margs.dst_slot = -1;
      merge_slots<D, false>(margs, lane);
    }
  }
}

// ------------------------------------------------------------------------------ split-KV decode
// Every warp is an independent pipeline.  The planner cuts every (request, kv head) into chunks
// of pages - large ones first, small ones for the tail - and the warps of the grid take chunks
// from a global counter as they go, so SMs that get less memory bandwidth simply take fewer
// chunks and all of them finish together.  A warp keeps DEPTH bulk copies in flight into a
// private ring and refills a stage as soon as it has consumed it: no producer warp, no empty
// barrier, no block-level sync.  The chunk after the current one is taken a few pages early so
// that neither the atomic nor the chunk record is ever waited for.
template <int D, int P, int NW, int DEPTH, int HP>
struct SplitCfg {
  static constexpr int PPV = P == 8 ? 2 : 1;   // pages per visit: 8-token pages are handled in pairs (16 tokens fill an MMA step)
  static constexpr int PAGE = 2 * P * D * 2;   // K block + V block of one (page, kv head)
  static constexpr int VP = HP * PAGE;         // one copy: the blocks of the unit's HP adjacent kv heads of one page
  static constexpr int STAGE = PPV * VP;
  static constexpr int QUEUE = 8;  // chunk ids a warp has started fetching but not finished (<= DEPTH + 2)
  static constexpr int SMEM = NW * DEPTH * STAGE + NW * DEPTH * (8 + 8 * PPV) + NW * QUEUE * 4 + PIE_MAX_LOCAL_GROUPS * 4 + 64;
};

template <int D, int P, int NW, int DEPTH, int HP>
__global__ void __launch_bounds__(NW * 32, 1) attn_split_kernel(const AttnParams p, int n_items, int n_warps) {
  using C = SplitCfg<D, P, NW, DEPTH, HP>;
  static_assert(DEPTH + 2 <= C::QUEUE, "queue too small");
  extern __shared__ __align__(1024) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* stages = smem + warp * DEPTH * C::STAGE;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + NW * DEPTH * C::STAGE) + warp * DEPTH;
  constexpr int PPV = C::PPV;
  volatile uint32_t* meta = reinterpret_cast<uint32_t*>(smem + NW * DEPTH * C::STAGE + NW * DEPTH * 8) + warp * DEPTH * PPV;
  volatile int* meta_phys = reinterpret_cast<int*>(smem + NW * DEPTH * C::STAGE + NW * DEPTH * (8 + 4 * PPV)) + warp * DEPTH * PPV;
  volatile int* queue = reinterpret_cast<int*>(smem + NW * DEPTH * C::STAGE + NW * DEPTH * (8 + 8 * PPV)) + warp * C::QUEUE;
  int* local_cnt = reinterpret_cast<int*>(smem + NW * DEPTH * C::STAGE + NW * DEPTH * (8 + 8 * PPV) + NW * C::QUEUE * 4);  // block-local merge groups
  if (threadIdx.x < PIE_MAX_LOCAL_GROUPS) local_cnt[threadIdx.x] = 0;
  __syncthreads();   // the only block-wide sync of the kernel (counters are zero before any warp counts itself in)
  if (!p.late_trigger) pie_pdl_launch_dependents();
  if (lane == 0) {
    for (int s = 0; s < DEPTH; ++s) mbar_init(smem_u32(full_bar + s), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();

  // ---- prefetch side: a cursor DEPTH page visits ahead of the consumer
  int q_head = 0, q_tail = 0;                       // queue of chunk ids, pushed here, popped by the consumer
  int pf_k = 0, pf_end = 0, pf_head = 0;            // cursor inside its current chunk
  int nx_begin = 0, nx_end = 0, nx_head = 0, nx_idx = -1;  // record of the chunk after it (when nx_idx >= 0)
  int grabbed = 0;                                  // lane 0: result of an atomic whose value is not needed yet
  bool grab_pending = false, exhausted = false, pf_live = true;

  // Short launches give every warp a fixed share first (cta_ptr != nullptr: warp w owns items
  // [cta_ptr[w], cta_ptr[w+1])) and leave only the last part of the work, cut into small chunks
  // [n_static, n_items), to the counter: few pieces and partials, yet no SM is left waiting at the end.
  const int wg = blockIdx.x * NW + warp;
  int own_next = 0, own_end = 0;
  if (p.cta_ptr != nullptr && wg < p.n_shares) {
    own_next = p.cta_ptr[wg];
    own_end = p.cta_ptr[wg + 1];
  }
  auto take = [&]() {  // synchronous: next chunk id for this warp
    if (own_next < own_end) return own_next++;
    int v = 0;
    if (lane == 0) v = atomicAdd(p.work_ctr, 1);
    return __shfl_sync(0xFFFFFFFFu, v, 0);
  };
  auto load_next_record = [&](int idx) {
    if (idx >= n_items) {
      exhausted = true;
      return;
    }
    const int4 r0 = __ldg(reinterpret_cast<const int4*>(p.items + idx));      // req, kv_head, row0, nrows
    const int2 r1 = __ldg(reinterpret_cast<const int2*>(p.items + idx) + 2);  // page_begin, page_end
    nx_head = r0.y;
    nx_begin = r1.x;
    nx_end = r1.y;
    nx_idx = idx;
  };
  auto pf_settle = [&]() {  // enter the next chunk while the current one is used up
    while (pf_live && pf_k >= pf_end) {
      if (nx_idx < 0 && !exhausted) {  // start-up, or chunks shorter than the look-ahead
        const int idx = grab_pending ? __shfl_sync(0xFFFFFFFFu, grabbed, 0) : take();
        grab_pending = false;
        load_next_record(idx);
      }
      if (nx_idx < 0) {
        pf_live = false;
        break;
      }
      pf_k = nx_begin;
      pf_end = nx_end;
      pf_head = nx_head;
      if (lane == 0) queue[q_tail % C::QUEUE] = nx_idx;
      ++q_tail;
      nx_idx = -1;
      __syncwarp();
    }
  };
  auto pf_lookahead = [&]() {  // two steps, a few pages apart, so that nothing is waited for
    if (!pf_live || nx_idx >= 0 || exhausted) return;
    const int left = pf_end - pf_k;
    if (!grab_pending) {
      if (left <= 4 * PPV) {
        if (own_next < own_end) grabbed = own_next++;
        else if (lane == 0) grabbed = atomicAdd(p.work_ctr, 1);
        grab_pending = true;
      }
    } else if (left <= 2 * PPV) {
      const int idx = __shfl_sync(0xFFFFFFFFu, grabbed, 0);
      grab_pending = false;
      load_next_record(idx);
    }
  };
  // (The stage was last read with ldmatrix by this same warp, and those reads have returned
  // their registers before the warp gets here, so the overwrite needs no proxy fence; the one
  // generic-proxy write to a stage, clearing rows of a last page, fences for itself.)
  auto issue = [&](int n, const int2* rec, int cnt, int head) {   // one visit: cnt <= PPV pages
    const uint32_t s = n % DEPTH;
#pragma unroll
    for (int i = 0; i < PPV; ++i) {
      meta[s * PPV + i] = i < cnt ? (uint32_t)rec[i].y : PIE_NO_PAGE;  // logical page | needs-mask flag, read back by the warp after the wait
      meta_phys[s * PPV + i] = rec[i].x;                                // physical page (the fused append writes its row back to it)
    }
    mbar_expect_tx(smem_u32(full_bar + s), cnt * C::VP);
#pragma unroll
    for (int i = 0; i < PPV; ++i)
      if (i < cnt)
        bulk_g2s(smem_u32(stages + s * C::STAGE + i * C::VP), p.pool + ((int64_t)rec[i].x * p.n_kv_heads + head * HP) * C::PAGE, C::VP,
                 smem_u32(full_bar + s));
  };
  auto load_visit = [&](int2* rec) {   // records of the visit at the prefetch cursor; returns its page count
    const int cnt = min(PPV, pf_end - pf_k);
#pragma unroll
    for (int i = 0; i < PPV; ++i) {
      rec[i] = make_int2(0, 0);
      if (i < cnt) rec[i] = __ldg(&p.kept[pf_k + i]);
    }
    return cnt;
  };

  // Prologue.  The plan arrays are not written by the kernels that precede this one in the stream, so
  // a warp with a fixed share walks its first DEPTH page records BEFORE waiting for those kernels:
  // under programmatic dependent launch this runs while the previous kernel drains.  The work
  // counter, the pool, Q and every output are touched only after the wait.
  int2 pre_rec[DEPTH][PPV];
  int n_pre = 0;
  if (own_next < own_end) {
    pf_settle();  // enters the first item of the fixed share (no counter access)
    n_pre = min(DEPTH, (pf_end - pf_k + PPV - 1) / PPV);
#pragma unroll
    for (int i = 0; i < DEPTH; ++i)
#pragma unroll
      for (int j = 0; j < PPV; ++j) {
        pre_rec[i][j] = make_int2(0, 0);
        if (i < n_pre && pf_k + i * PPV + j < pf_end) pre_rec[i][j] = __ldg(&p.kept[pf_k + i * PPV + j]);
      }
  }
  pie_pdl_wait();  // the append (and whatever produced Q) is complete from here on
#pragma unroll
  for (int i = 0; i < DEPTH; ++i)
    if (i < n_pre && lane == 0) issue(i, pre_rec[i], min(PPV, pf_end - pf_k - i * PPV), pf_head);
  pf_k = min(pf_k + n_pre * PPV, pf_end);
  pf_settle();  // (may take from the counter now)
  for (int n = n_pre; n < DEPTH && pf_live; ++n) {  // rest of the ring
    int2 rec[PPV];
    const int cnt = load_visit(rec);
    if (lane == 0) issue(n, rec, cnt, pf_head);
    pf_k += cnt;
    pf_lookahead();
    pf_settle();
  }

  // ---- consumer side
  int n = 0;  // visits consumed so far (ring position)
  int owed0 = 0, owed1 = 0, n_owed = 0;   // items whose merge duties are carried out after the last item
  while (q_head < q_tail) {
    const int idx = queue[q_head % C::QUEUE];
    ++q_head;
    const PieItem item = p.items[idx];
    PieReq rq;  // the chunk carries its request's record
    rq.q_start = item.q_start;
    rq.q_len = item.q_len;
    rq.kv_len = item.kv_len;
    rq.kept_start = 0;
    rq.kept_count = 0;
    rq.mask_row_words = item.mask_row_words;
    rq.mask_word_off = item.mask_word_off;
    rq.last_logical = item.last_logical;
    rq.last_page_len = item.last_page_len;
    // Fused append (decode batches): this piece ends with the request's last page, so this warp
    // also owns the request's one new K/V row of its kv head(s).  The row's 16-byte chunks are
    // fetched now (per head CH lanes for K, then CH for V) and written, once the page has landed, into
    // the staged copy and into the pool at the same offset (the stage is an image of the blocks).
    constexpr int CH = D * 2 / 16;
    static_assert(2 * CH * HP <= 32, "one lane per 16-byte chunk of the new row");
    const bool do_append = (item.flags & PIE_ITEM_APPEND) != 0;
    const int a_head = lane / (2 * CH), a_v = (lane / CH) & 1;   // which head of the unit, K or V
    uint4 new_chunk = make_uint4(0, 0, 0, 0);
    if (do_append && lane < 2 * CH * HP)
      new_chunk = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(a_v ? p.v_new : p.k_new) +
                                                       ((int64_t)item.q_start * p.n_kv_heads + item.kv_head * HP + a_head) * (D * 2)) + (lane % CH));
    RowState<D> st;
    rows_init<D>(st, p, item, rq, item.row0, lane);
    for (int k = item.page_begin; k < item.page_end; k += PPV, ++n) {
      const uint32_t s = n % DEPTH, ph = (n / DEPTH) & 1;
      int2 rec_next[PPV];
      int cnt_next = 0;
      if (pf_live) cnt_next = load_visit(rec_next);  // latency hides behind the wait
      mbar_wait(smem_u32(full_bar + s), ph, p.status);
      uint32_t lpf[PPV];
#pragma unroll
      for (int i = 0; i < PPV; ++i) lpf[i] = meta[s * PPV + i];
#pragma unroll
      for (int i = 0; i < PPV; ++i) {
        if (do_append && lpf[i] != PIE_NO_PAGE && (int)(lpf[i] & ~PIE_KEPT_NEEDS_MASK) == item.last_logical) {
          if (lane < 2 * CH * HP) {
            const int off = a_head * C::PAGE + (a_v ? C::PAGE / 2 : 0) + pie_chunk_offset(P * 128, item.last_page_len - 1, lane % CH);
            *reinterpret_cast<uint4*>(stages + s * C::STAGE + i * C::VP + off) = new_chunk;
            const int phys = meta_phys[s * PPV + i];
            *reinterpret_cast<uint4*>(const_cast<uint8_t*>(p.pool) + ((int64_t)phys * p.n_kv_heads + item.kv_head * HP) * C::PAGE + off) = new_chunk;
          }
          // the generic-proxy write must be ordered before the bulk copy that later refills the stage
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
        }
      }
      visit_compute<D, P, PPV, HP>(st, stages + s * C::STAGE, rq, lpf, p.scale_log2, lane);
      __syncwarp();
      if (pf_live) {
        if (lane == 0) issue(n + DEPTH, rec_next, cnt_next, pf_head);
        pf_k += cnt_next;
        pf_lookahead();
        pf_settle();
      }
    }
    // Rows out: final, or an fp32 partial - in global memory, or, for a block-local group all of whose pieces are
    // the last items of their warps (so that their rings are idle), in the warp's ring, where the merging warp
    // finds it without a round trip to L2.
    const uint32_t fl = item.flags;
    if (fl & PIE_ITEM_LOCAL_SMEM) rows_store_smem<D>(st, reinterpret_cast<float*>(stages), lane);
    else rows_store<D>(st, p, item, rq, item.row0, p.slot_rows, lane);
    if ((fl & PIE_ITEM_LOCAL_PIECE) && !(fl & PIE_ITEM_LOCAL_MERGER)) {
      __threadfence_block();   // the merging warp runs on this SM: block scope is enough
      __syncwarp();
      if (lane == 0) atomicAdd(local_cnt + PIE_ITEM_LOCAL_GID(fl), 1);
    } else if (fl & (PIE_ITEM_LOCAL_MERGER | PIE_ITEM_GRID_PIECE)) {
      // merging and cross-block counting wait until the warp has no item left (at most two pieces per warp owe
      // any: the one that ends a unit begun in an earlier block, and the warp's last item)
      if (n_owed == 0) owed0 = idx;
      else owed1 = idx;
      ++n_owed;
    }
  }
  if (n_owed > 0) split_piece_finish<D, NW>(p, owed0, reinterpret_cast<const float*>(stages), DEPTH * C::STAGE / 4, local_cnt, lane);
  if (n_owed > 1) split_piece_finish<D, NW>(p, owed1, reinterpret_cast<const float*>(stages), DEPTH * C::STAGE / 4, local_cnt, lane);

  if (p.late_trigger) pie_pdl_launch_dependents();
  // ---- the last warp of the grid to finish re-arms the counters for the next launch
  if (lane == 0) {
    __threadfence();
    if (atomicAdd(p.work_ctr + 1, 1) == n_warps - 1) {
      p.work_ctr[0] = p.n_static;
      p.work_ctr[1] = 0;
    }
  }
}

// ------------------------------------------------------------------------------ row-tile kernel
// Prefill chunks and token trees: NW consumer warps own 16 query rows each and all walk the same
// page stream, which a producer warp keeps filled through a ring of full / empty barriers.
template <int D, int P, int NW, int NSTAGES>
struct TileCfg {
  static constexpr int BLK = P * D * 2;       // one K (or V) block, bytes
  static constexpr int STAGE = 2 * BLK;       // K block then V block
  static constexpr int SMEM = NSTAGES * STAGE + 2 * NSTAGES * 8 + ((NSTAGES + 3) & ~3) * 4 + 64;
};

template <int D, int P, int NW, int NSTAGES>
__global__ void __launch_bounds__((NW + 1) * 32, 1) attn_tile_kernel(const AttnParams p) {
  using C = TileCfg<D, P, NW, NSTAGES>;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* stages = smem;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + NSTAGES * C::STAGE);
  uint64_t* empty_bar = full_bar + NSTAGES;
  uint32_t* meta = reinterpret_cast<uint32_t*>(empty_bar + NSTAGES);  // per stage: logical page | flag

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGES; ++s) {
      mbar_init(smem_u32(full_bar + s), 1);
      mbar_init(smem_u32(empty_bar + s), NW);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  pie_pdl_launch_dependents();
  __syncthreads();
  pie_pdl_wait();

  const int it0 = p.cta_ptr[blockIdx.x], it1 = p.cta_ptr[blockIdx.x + 1];

  if (warp == NW) {
    // ---- producer warp: LANES copies per step; stages of one step are distinct, and the warp
    // re-converges after every step so that no lane runs ahead into a later ring phase
    constexpr int LANES = NSTAGES / 2 < 32 ? NSTAGES / 2 : 32;
    uint32_t cnt_base = 0;
    for (int it = it0; it < it1; ++it) {
      const PieItem item = p.items[it];
      const uint8_t* base = p.pool + (int64_t)item.kv_head * C::STAGE;
      const int npages = item.page_end - item.page_begin;
      for (int k0 = 0; k0 < npages; k0 += LANES) {
        const int kk = k0 + lane;
        if (lane < LANES && kk < npages) {
          const uint32_t cnt = cnt_base + kk;
          const uint32_t s = cnt % NSTAGES, ph = (cnt / NSTAGES) & 1;
          const int2 kp = __ldg(p.kept + item.page_begin + kk);
          mbar_wait(smem_u32(empty_bar + s), ph ^ 1, p.status);
          meta[s] = (uint32_t)kp.y;
          mbar_expect_tx(smem_u32(full_bar + s), C::STAGE);
          bulk_g2s(smem_u32(stages + s * C::STAGE), base + (int64_t)kp.x * p.page_bytes, C::STAGE,
                   smem_u32(full_bar + s));
        }
        __syncwarp();
      }
      cnt_base += npages;
    }
    return;
  }

  // ---- consumers
  uint32_t cnt = 0;
  for (int it = it0; it < it1; ++it) {
    const PieItem item = p.items[it];
    const PieReq rq = p.reqs[item.req];
    const int rbase = item.row0 + warp * 16;
    RowState<D> st;
    rows_init<D>(st, p, item, rq, rbase, lane);
    const int npages = item.page_end - item.page_begin;
    for (int kk = 0; kk < npages; ++kk, ++cnt) {
      const uint32_t s = cnt % NSTAGES, ph = (cnt / NSTAGES) & 1;
      mbar_wait(smem_u32(full_bar + s), ph, p.status);
      const uint32_t lpf = meta[s];
      page_compute<D, P>(st, stages + s * C::STAGE, rq, lpf, p.scale_log2, lane);
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(empty_bar + s));
    }
    rows_store<D>(st, p, item, rq, rbase, NW * 16, lane);
  }
}

// ------------------------------------------------------------------------------ merge kernel
// lse = ln sum_c exp(lse_c), o = sum_c exp(lse_c - lse) o_c over the partial slots of a group.
template <typename T, int D>
__global__ void merge_kernel(const PieMerge* __restrict__ merges, const PieReq* __restrict__ reqs,
                             const float* __restrict__ ws_o, const float* __restrict__ ws_lse, T* __restrict__ out,
                             float* __restrict__ lse_out, int slot_rows, int n_q_heads, int G,
                             const float* __restrict__ x_ws_o, const float* __restrict__ x_ws_lse, int x_slot_rows) {
  // One warp per (merge group, row).  Lanes share the slots for the max and the weights, then each
  // lane owns D/32 consecutive columns and the slot loop issues independent, coalesced row loads.
  // (Every partial row is written by its kernel, with zeros when its part of the context was empty.)
  // A group may name further partials of its rows in the row-tile launch's workspace (x_*: the
  // shared-prefix cascade); they are combined after the group's own slots.
  constexpr int EPL = D / 32;
  pie_pdl_launch_dependents();
  pie_pdl_wait();
  const PieMerge mg = merges[blockIdx.x];
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.y * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= mg.nrows) return;
  const PieReq rq = reqs[mg.req];
  const int ntot = mg.nslots + mg.x_nslots;
  // source c: own slot c, or cascade slot c - nslots
  auto lse_of = [&](int c) -> float {
    return c < mg.nslots ? ws_lse[(int64_t)(mg.slot0 + c) * slot_rows + row]
                         : x_ws_lse[(int64_t)(mg.x_slot0 + c - mg.nslots) * x_slot_rows + mg.x_row0 + row];
  };
  auto row_of = [&](int c) -> const float* {
    return c < mg.nslots ? ws_o + ((int64_t)(mg.slot0 + c) * slot_rows + row) * D + lane * EPL
                         : x_ws_o + ((int64_t)(mg.x_slot0 + c - mg.nslots) * x_slot_rows + mg.x_row0 + row) * D + lane * EPL;
  };
  // The first sources' rows are fetched together with the LSEs (their addresses need neither the
  // maximum nor the weights), the others in batches of the same size: one round trip to memory per
  // batch instead of one after the LSEs and then one per four sources.
  constexpr int BATCH = EPL == 4 ? 4 : 8;   // (16 registers of loads in flight: more would cost large merge grids their occupancy)
  typedef typename std::conditional<EPL == 4, float4, float2>::type Vec;
  Vec pre[BATCH];
#pragma unroll
  for (int u = 0; u < BATCH; ++u)
    if (u < ntot) pre[u] = *reinterpret_cast<const Vec*>(row_of(u));
  float M = kNegInf;
  for (int c = lane; c < ntot; c += 32) M = fmaxf(M, lse_of(c));
  for (int sft = 16; sft > 0; sft >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, sft));
  float Z = 0.f, acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  auto add = [&](float wu, const Vec& v) {
    if constexpr (EPL == 4) acc[0] += wu * v.x, acc[1] += wu * v.y, acc[2] += wu * v.z, acc[3] += wu * v.w;
    else acc[0] += wu * v.x, acc[1] += wu * v.y;
  };
  for (int base = 0; base < ntot; base += 32) {
    const int c = base + lane;
    float w = 0.f;
    if (c < ntot && M != kNegInf) w = __expf(lse_of(c) - M);  // exp(-inf) = 0
    Z += w;
    const int cnt = min(32, ntot - base);
    int u0 = 0;
    if (base == 0) {
#pragma unroll
      for (int u = 0; u < BATCH; ++u)
        if (u < cnt) add(__shfl_sync(0xFFFFFFFFu, w, u), pre[u]);
      u0 = BATCH;
    }
    for (int ub = u0; ub < cnt; ub += BATCH) {
      Vec v[BATCH];
#pragma unroll
      for (int u = 0; u < BATCH; ++u)
        if (ub + u < cnt) v[u] = *reinterpret_cast<const Vec*>(row_of(base + ub + u));
#pragma unroll
      for (int u = 0; u < BATCH; ++u)
        if (ub + u < cnt) add(__shfl_sync(0xFFFFFFFFu, w, ub + u), v[u]);
    }
  }
  for (int sft = 16; sft > 0; sft >>= 1) Z += __shfl_xor_sync(0xFFFFFFFFu, Z, sft);
  const int gr = mg.row0 + row;
  const int tok = gr / G, head = mg.kv_head * G + gr % G;
  const int64_t oi = (int64_t)(rq.q_start + tok) * n_q_heads + head;
  const float inv = Z > 0.f ? 1.f / Z : 0.f;
#pragma unroll
  for (int e = 0; e < EPL; ++e) out[oi * D + lane * EPL + e] = (T)(acc[e] * inv);
  if (lane == 0) lse_out[oi] = Z > 0.f ? M + logf(Z) : kNegInf;
}

// The same for groups of row-tile partials (up to 256 rows per group, few sources each: the pieces of a cut unit,
// or a request's private part plus the shared-prefix cascade).  One thread block per group, its record read
// once; every warp takes eight rows at a time (four when there are three or four sources): one lane per (row,
// source) pair fetches the pair's LSE while every lane already fetches its columns of all sources of those rows -
// one round trip to memory per eight rows instead of a chain of four per row.  Sources are combined in slot order
// (own slots, then the cascade's), as above.
template <typename T, int D>
__global__ void __launch_bounds__(256) merge_tiles_kernel(const PieMerge* __restrict__ merges, const PieReq* __restrict__ reqs,
                                                          const float* __restrict__ ws_o, const float* __restrict__ ws_lse,
                                                          T* __restrict__ out, float* __restrict__ lse_out, int slot_rows,
                                                          int n_q_heads, int G, const float* __restrict__ x_ws_o,
                                                          const float* __restrict__ x_ws_lse, int x_slot_rows) {
  constexpr int EPL = D / 32;
  pie_pdl_launch_dependents();
  pie_pdl_wait();
  const PieMerge mg = merges[blockIdx.x];
  const PieReq rq = reqs[mg.req];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ntot = mg.nslots + mg.x_nslots;
  auto lse_at = [&](int c, int row) -> const float* {
    return c < mg.nslots ? ws_lse + (int64_t)(mg.slot0 + c) * slot_rows + row
                         : x_ws_lse + (int64_t)(mg.x_slot0 + c - mg.nslots) * x_slot_rows + mg.x_row0 + row;
  };
  auto row_at = [&](int c, int row) -> const float* {
    return c < mg.nslots ? ws_o + ((int64_t)(mg.slot0 + c) * slot_rows + row) * D + lane * EPL
                         : x_ws_o + ((int64_t)(mg.x_slot0 + c - mg.nslots) * x_slot_rows + mg.x_row0 + row) * D + lane * EPL;
  };
  auto store_row = [&](int row, const float* acc, float M, float Z) {
    const int gr = mg.row0 + row;
    const int tok = gr / G, head = mg.kv_head * G + gr % G;
    const int64_t oi = (int64_t)(rq.q_start + tok) * n_q_heads + head;
    const float inv = Z > 0.f ? 1.f / Z : 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) out[oi * D + lane * EPL + e] = (T)(acc[e] * inv);
    if (lane == 0) lse_out[oi] = Z > 0.f ? M + logf(Z) : kNegInf;
  };
  // Few sources: RPW rows per warp and step, 32 / RPW lanes per row fetch the row's LSEs (one per source).
  auto run_few = [&](auto rpw_c, auto ns_c) {
    constexpr int RPW = decltype(rpw_c)::value, NS = decltype(ns_c)::value, LPR = 32 / RPW;
    static_assert(NS <= LPR, "one lane per (row, source) pair");
    for (int row0 = warp * RPW; row0 < mg.nrows; row0 += (blockDim.x >> 5) * RPW) {
      const int nr = min(RPW, mg.nrows - row0);   // (warp uniform)
      float v[RPW][NS][EPL];
#pragma unroll
      for (int k = 0; k < RPW; ++k)
#pragma unroll
        for (int c = 0; c < NS; ++c) {
          if (k < nr && c < ntot) {
            const float* src = row_at(c, row0 + k);
            if constexpr (EPL == 4) {
              const float4 x = __ldcg(reinterpret_cast<const float4*>(src));
              v[k][c][0] = x.x, v[k][c][1] = x.y, v[k][c][2] = x.z, v[k][c][3] = x.w;
            } else {
              const float2 x = __ldcg(reinterpret_cast<const float2*>(src));
              v[k][c][0] = x.x, v[k][c][1] = x.y;
            }
          } else {
#pragma unroll
            for (int e = 0; e < EPL; ++e) v[k][c][e] = 0.f;
          }
        }
      const int lk = lane / LPR, lc = lane % LPR;   // this lane's (row, source) pair
      float l = kNegInf;
      if (lk < nr && lc < ntot) l = *lse_at(lc, row0 + lk);
      float M = l;
#pragma unroll
      for (int sft = LPR / 2; sft > 0; sft >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, sft));   // over the lanes of the row
      const float w = M != kNegInf ? __expf(l - M) : 0.f;   // exp(-inf) = 0
#pragma unroll
      for (int k = 0; k < RPW; ++k) {
        float acc[EPL], Z = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
#pragma unroll
        for (int c = 0; c < NS; ++c) {
          const float wu = __shfl_sync(0xFFFFFFFFu, w, k * LPR + c);
          Z += wu;
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[e] += wu * v[k][c][e];
        }
        const float Mk = __shfl_sync(0xFFFFFFFFu, M, k * LPR);
        if (k < nr) store_row(row0 + k, acc, Mk, Z);
      }
    }
  };
  if (ntot <= 2) {   // (a request's private part plus the cascade's shared part, a unit cut once: the common cases)
    run_few(std::integral_constant<int, 8>{}, std::integral_constant<int, 2>{});
    return;
  }
  if (ntot <= 4) {
    run_few(std::integral_constant<int, 4>{}, std::integral_constant<int, 4>{});
    return;
  }
  for (int row = warp; row < mg.nrows; row += blockDim.x >> 5) {   // many sources: row by row
    float M = kNegInf;
    for (int c = lane; c < ntot; c += 32) M = fmaxf(M, *lse_at(c, row));
    for (int sft = 16; sft > 0; sft >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, sft));
    float Z = 0.f, acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int base = 0; base < ntot; base += 32) {
      const int c = base + lane;
      float w = 0.f;
      if (c < ntot && M != kNegInf) w = __expf(*lse_at(c, row) - M);
      Z += w;
      const int cnt = min(32, ntot - base);
      for (int u = 0; u < cnt; ++u) {
        const float wu = __shfl_sync(0xFFFFFFFFu, w, u);
        const float* src = row_at(base + u, row);
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] += wu * src[e];
      }
    }
    for (int sft = 16; sft > 0; sft >>= 1) Z += __shfl_xor_sync(0xFFFFFFFFu, Z, sft);
    store_row(row, acc, M, Z);
  }
}

// ------------------------------------------------------------------------------ simple kernel
template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T, int D>
__global__ void simple_kernel(const uint8_t* __restrict__ pool, const T* __restrict__ q, T* __restrict__ out,
                              float* __restrict__ lse_out, const PieReq* __restrict__ reqs,
                              const int2* __restrict__ kept, const uint32_t* __restrict__ mask,
                              const int32_t* __restrict__ tok_req, const int32_t* __restrict__ rows, int n_rows,
                              PoolGeom g, int n_q_heads, int G, float scale) {
  constexpr int EPL = D / 32;  // elements per lane
  pie_pdl_launch_dependents();
  pie_pdl_wait();
  const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (wid >= n_rows) return;
  const int row = rows[wid];
  const int t = row / n_q_heads, h = row - t * n_q_heads;
  const PieReq rq = reqs[tok_req[t]];
  const int i = t - rq.q_start, kvh = h / G;
  const int lim = rq.kv_len - rq.q_len + i;
  const uint32_t* mrow = mask + rq.mask_word_off + (int64_t)i * rq.mask_row_words;
  float qv[EPL], acc[EPL];
  for (int e = 0; e < EPL; ++e) {
    qv[e] = to_f32<T>(q[(int64_t)row * D + lane * EPL + e]);
    acc[e] = 0.f;
  }
  const int byte_off = lane * EPL * (int)sizeof(T);
  const int chunk = byte_off >> 4, within = byte_off & 15;
  float m = kNegInf, l = 0.f;
  for (int k = 0; k < rq.kept_count; ++k) {
    const int2 kp = kept[rq.kept_start + k];
    const int lp = (int)((uint32_t)kp.y & ~PIE_KEPT_NEEDS_MASK);
    const uint8_t* blockK = pool + (int64_t)kp.x * g.page_bytes + (int64_t)(kvh * 2) * g.block_bytes;
    const uint8_t* blockV = blockK + g.block_bytes;
    for (int slot = 0; slot < g.page_size; ++slot) {
      const int j = lp * g.page_size + slot;
      if (j >= rq.kv_len) break;
      const bool allowed = rq.mask_row_words ? ((mrow[j >> 5] >> (j & 31)) & 1u) : (j <= lim);
      if (!allowed) continue;
      const int off = pie_chunk_offset(g.slab_bytes, slot, chunk) + within;
      const T* kp_ = reinterpret_cast<const T*>(blockK + off);
      const T* vp_ = reinterpret_cast<const T*>(blockV + off);
      float dot = 0.f;
      for (int e = 0; e < EPL; ++e) dot += qv[e] * to_f32<T>(kp_[e]);
      for (int sft = 16; sft > 0; sft >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, sft);
      const float s = dot * scale;
      const float m_new = fmaxf(m, s);
      const float a = expf(m - m_new), pw = expf(s - m_new);
      l = l * a + pw;
      for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * a + pw * to_f32<T>(vp_[e]);
      m = m_new;
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  for (int e = 0; e < EPL; ++e) out[(int64_t)row * D + lane * EPL + e] = (T)(acc[e] * inv);
  if (lane == 0) lse_out[row] = l > 0.f ? m + logf(l) : kNegInf;
}

// ------------------------------------------------------------------------------ launchers
AttnParams make_params(pie_ctx* ctx, const pie_plan* plan, const PieLaunchList& ll, const void* q, void* out,
                       float* lse) {
  AttnParams p{};
  p.pool = ctx->pool;
  p.q = q;
  p.out = out;
  p.lse = lse;
  p.reqs = plan->d_reqs;
  p.kept = plan->d_kept;
  p.mask = plan->d_mask;
  p.items = ll.d_items;
  p.cta_ptr = ll.cta_ptr.empty() ? nullptr : ll.d_cta_ptr;
  p.n_shares = ll.cta_ptr.empty() ? 0 : (int)ll.cta_ptr.size() - 1;
  p.n_static = ll.n_static;
  p.work_ctr = ll.d_work_ctr;
  p.slot_rows = ll.slot_rows;
  p.ws_o = ll.d_ws_o;
  p.ws_lse = ll.d_ws_lse;
  p.status = ctx->d_status;
  p.page_bytes = ctx->geom.page_bytes;
  p.n_q_heads = ctx->cfg.num_q_heads;
  p.n_kv_heads = ctx->cfg.num_kv_heads;
  p.G_head = ctx->G;
  p.G = ctx->G * ll.heads_per_unit;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)ctx->cfg.head_dim);
  p.late_trigger = plan->overlap ? 1 : 0;
  return p;
}

template <int D, int P, int NW, int DEPTH, int HP = 1>
int launch_split(pie_ctx* ctx, const AttnParams& p, int n_items, int n_warps, cudaStream_t s) {
  using C = SplitCfg<D, P, NW, DEPTH, HP>;
  auto kern = attn_split_kernel<D, P, NW, DEPTH, HP>;
  bool& configured = HP == 1 ? ctx->split_configured : ctx->split_pair_configured;
  if (!configured) {   // (a context has one shape and one device, hence one instantiation per unit width)
    PIE_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
    configured = true;
  }
  const int blocks = (n_warps + NW - 1) / NW;
  PIE_CUDA(ctx, pie_launch_pdl(kern, dim3(blocks), dim3(NW * 32), C::SMEM, s, p, n_items, blocks * NW));
  return PIE_OK;
}

template <int D, int P, int NW>
int launch_tiles(pie_ctx* ctx, const AttnParams& p, int grid, cudaStream_t s) {
  constexpr int NSTAGES = (128 * 1024) / (2 * P * D * 2);
  using C = TileCfg<D, P, NW, NSTAGES>;
  auto kern = attn_tile_kernel<D, P, NW, NSTAGES>;
  if (!ctx->tile_configured) {
    PIE_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
    ctx->tile_configured = true;
  }
  PIE_CUDA(ctx, pie_launch_pdl(kern, dim3(grid), dim3((NW + 1) * 32), C::SMEM, s, p));
  return PIE_OK;
}

}  // namespace

bool pie_split_supported(const pie_ctx* ctx) {
  const pie_config& c = ctx->cfg;
  return c.dtype == PIE_DTYPE_BF16 && (c.page_size == 8 || c.page_size == 16 || c.page_size == 32) &&
         (c.head_dim == 64 || c.head_dim == 128) && ctx->G <= 16;
}

// Units of two adjacent kv heads (copies of twice the size): the shapes whose blocks are 2 or 4 KB.
bool pie_split_pair_supported(const pie_ctx* ctx) {
  const pie_config& c = ctx->cfg;
  return pie_split_supported(ctx) && c.head_dim == 64 && (c.page_size == 8 || c.page_size == 16) && c.num_kv_heads % 2 == 0 &&
         2 * ctx->G <= 16;
}

// Warps per block of the split-KV kernel (the planner sizes its shares with this).
int pie_split_warps_per_block(const pie_ctx* ctx) {
  return (ctx->cfg.page_size == 32 && ctx->cfg.head_dim == 128) ? 4 : 8;
}

int pie_launch_split(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new, const void* v_new, void* out,
                     float* lse, cudaStream_t s) {
  AttnParams p = make_params(ctx, plan, plan->split, q, out, lse);
  p.k_new = k_new;
  p.v_new = v_new;
  const int D = ctx->cfg.head_dim, P = ctx->cfg.page_size, n = plan->split.grid, ni = (int)plan->split.items.size();
  // ring depth: 128 - 192 KB of copies in flight per SM (measured on the 64-request decode batch with 4 KB stages:
  // depths 3 and 4 run 1.5 % faster than 5 and 6 - a deeper ring only lengthens the queue in front of every copy)
  if (plan->split.heads_per_unit == 2) {   // units of two adjacent kv heads: copies of 8 KB instead of 4 KB (of 4 KB instead of 2 KB)
    if (D == 64 && P == 16) return launch_split<64, 16, 8, 3, 2>(ctx, p, ni, n, s);
    if (D == 64 && P == 8) return launch_split<64, 8, 8, 3, 2>(ctx, p, ni, n, s);
    return PIE_ERR_UNSUPPORTED;
  }
  if (D == 64 && P == 8) return launch_split<64, 8, 8, 4>(ctx, p, ni, n, s);     // (a visit is two pages: the same 4 / 8 KB as with 16-token pages)
  if (D == 128 && P == 8) return launch_split<128, 8, 8, 3>(ctx, p, ni, n, s);
  if (D == 64 && P == 16) return launch_split<64, 16, 8, 4>(ctx, p, ni, n, s);
  if (D == 128 && P == 16) return launch_split<128, 16, 8, 3>(ctx, p, ni, n, s);
  if (D == 64 && P == 32) return launch_split<64, 32, 8, 3>(ctx, p, ni, n, s);
  if (D == 128 && P == 32) return launch_split<128, 32, 4, 3>(ctx, p, ni, n, s);
  return PIE_ERR_UNSUPPORTED;
}

int pie_launch_tiles(pie_ctx* ctx, const pie_plan* plan, const void* q, void* out, float* lse, cudaStream_t s) {
  AttnParams p = make_params(ctx, plan, plan->tile, q, out, lse);
  const int D = ctx->cfg.head_dim, P = ctx->cfg.page_size, grid = plan->tile.grid;
  if (plan->tile_tc) return pie_launch_tc_tiles(ctx, p, grid, plan->info.num_query_tokens, s);
  if (D == 64 && P == 16) return launch_tiles<64, 16, 4>(ctx, p, grid, s);
  if (D == 128 && P == 16) return launch_tiles<128, 16, 4>(ctx, p, grid, s);
  if (D == 64 && P == 32) return launch_tiles<64, 32, 4>(ctx, p, grid, s);
  if (D == 128 && P == 32) return launch_tiles<128, 32, 4>(ctx, p, grid, s);
  return PIE_ERR_UNSUPPORTED;
}

int pie_launch_merge(pie_ctx* ctx, const pie_plan* plan, const PieLaunchList& ll, void* out, float* lse, cudaStream_t s) {
  const int D = ctx->cfg.head_dim;
  const bool tiles = ll.slot_rows >= 32;      // groups of row-tile partials: one block per group
  const int wpb = ll.slot_rows >= 8 ? 8 : 4;  // warps (= rows) per block
  const dim3 n((unsigned)ll.merges.size(), tiles ? 1u : (unsigned)((ll.slot_rows + wpb - 1) / wpb));
#define PIE_MERGE(T, DD)                                                                                                   \
  PIE_CUDA(ctx, pie_launch_pdl(tiles ? merge_tiles_kernel<T, DD> : merge_kernel<T, DD>, n, dim3(tiles ? 256 : wpb * 32), 0, s, \
                               (const PieMerge*)ll.d_merges, (const PieReq*)plan->d_reqs, (const float*)ll.d_ws_o,         \
                               (const float*)ll.d_ws_lse, (T*)out, lse, ll.slot_rows, ctx->cfg.num_q_heads, ctx->G * ll.heads_per_unit, \
                               (const float*)plan->tile.d_ws_o, (const float*)plan->tile.d_ws_lse, plan->tile.slot_rows))
  if (ctx->cfg.dtype == PIE_DTYPE_BF16) {
    if (D == 64) PIE_MERGE(__nv_bfloat16, 64);
    else PIE_MERGE(__nv_bfloat16, 128);
  } else {
    if (D == 64) PIE_MERGE(float, 64);
    else PIE_MERGE(float, 128);
  }
#undef PIE_MERGE
  PIE_CUDA(ctx, cudaGetLastError());
  return PIE_OK;
}

int pie_launch_simple(pie_ctx* ctx, const pie_plan* plan, const void* q, void* out, float* lse, cudaStream_t s) {
  const int n = (int)plan->simple_rows.size();
  const int D = ctx->cfg.head_dim;
  const float scale = 1.f / sqrtf((float)D);
  const int threads = 128, grid = (n * 32 + threads - 1) / threads;
#define PIE_SIMPLE(T, DD)                                                                                              \
  PIE_CUDA(ctx, pie_launch_pdl(simple_kernel<T, DD>, dim3(grid), dim3(threads), 0, s, (const uint8_t*)ctx->pool,     \
                               (const T*)q, (T*)out, lse, (const PieReq*)plan->d_reqs, (const int2*)plan->d_kept,     \
                               (const uint32_t*)plan->d_mask, (const int32_t*)plan->d_tok_req,                         \
                               (const int32_t*)plan->d_simple_rows, n, ctx->geom, ctx->cfg.num_q_heads, ctx->G, scale))
  if (ctx->cfg.dtype == PIE_DTYPE_BF16) {
    if (D == 64) PIE_SIMPLE(__nv_bfloat16, 64);
    else PIE_SIMPLE(__nv_bfloat16, 128);
  } else {
    if (D == 64) PIE_SIMPLE(float, 64);
    else PIE_SIMPLE(float, 128);
  }
#undef PIE_SIMPLE
  PIE_CUDA(ctx, cudaGetLastError());
  return PIE_OK;
}


// ------------------------------------------------------------------------------ forward without allocation
// Scratch for pie_forward_static_scratch: the uploaded plan arrays and the fp32 split partials
// live in this file-scope array instead of a cudaMalloc'd buffer.  Every GPU that loads the
// library holds it until the process exits.  In host code the name below is only a stand-in
// for the symbol; its device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char pie_static_scratch[PIE_STATIC_SCRATCH_BYTES];
static void* g_static_scratch_addr[64] = {};  // per device ordinal, filled on first use

extern "C" int pie_forward_static_scratch(pie_ctx* ctx, const pie_batch_desc* batch, const void* q, const void* k_new,
                                          const void* v_new, void* out, float* lse, void* stream) {
  if (!ctx || !batch) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  const int dev = ctx->cfg.device;
  if (dev < 0 || dev >= 64) return PIE_ERR_INVALID;
  cudaStream_t s = (cudaStream_t)stream;
  PIE_CUDA(ctx, cudaSetDevice(dev));
  if (!g_static_scratch_addr[dev]) {  // set-up, once per device, with that device current
    void* ptr = nullptr;
    PIE_CUDA(ctx, cudaGetSymbolAddress(&ptr, pie_static_scratch));
    g_static_scratch_addr[dev] = ptr;
  }
  uint8_t* base = static_cast<uint8_t*>(g_static_scratch_addr[dev]);

  pie_plan plan;  // host-side only; its device pointers will point into the static scratch
  plan.ctx = ctx;
  const int saved_overlap = ctx->options[PIE_OPT_OVERLAP];
  ctx->options[PIE_OPT_OVERLAP] = 2;  // this entry point enqueues its kernels one after the other
  int rc = pie_build_plan(ctx, batch, &plan);
  ctx->options[PIE_OPT_OVERLAP] = saved_overlap;
  if (rc != PIE_OK) return rc;   // (a failed build has given its borrowed pages back)
  // Pages borrowed for requests without output KvPages: on every way out from here they are handed to
  // the context, which returns them to the free list once the work enqueued on `s` so far is over.
  struct Holder {
    pie_plan* plan;
    cudaStream_t s;
    ~Holder() { pie_plan_hold_scratch(plan, s); }
  } holder{&plan, s};
  if (plan.T == 0) return PIE_OK;
  if (!q || !k_new || !v_new || !out || !lse) return PIE_ERR_INVALID;

  const PlanLayout L = pie_plan_layout(ctx, &plan);
  if (L.total > (size_t)PIE_STATIC_SCRATCH_BYTES) return PIE_ERR_BATCH_TOO_LARGE;  // plan + partials exceed the static scratch
  // Nothing in the scratch has to start at zero: every plan array is overwritten by this copy
  // and every partial row is written by the attention kernel before a merge reads it.
  // (The image is ordinary pageable host memory: the copy call returns once the runtime has staged it,
  //  so the vector may go when this function returns.)
  std::vector<uint8_t> host(L.upload);
  pie_plan_fill(&plan, L, host.data());
  PIE_CUDA(ctx, cudaMemcpyAsync(base, host.data(), host.size(), cudaMemcpyHostToDevice, s));
  pie_plan_bind(&plan, L, base);
  // rows of partly filled last input pages of requests without output KvPages, into the borrowed pages
  if (!plan.pre_copies.empty() && (rc = pie_launch_copy(ctx, (int)plan.pre_copies.size() / 5, plan.d_pre_copies, s))) return rc;
  if ((rc = pie_append_and_q(ctx, &plan, q, k_new, v_new, s, &q))) return rc;
  if (!plan.simple_rows.empty() && (rc = pie_launch_simple(ctx, &plan, q, out, lse, s))) return rc;
  if (!plan.tile.items.empty() && (rc = pie_launch_tiles(ctx, &plan, q, out, lse, s))) return rc;
  if (!plan.tile.merges.empty() && (rc = pie_launch_merge(ctx, &plan, plan.tile, out, lse, s))) return rc;
  if (!plan.split.items.empty() && (rc = pie_launch_split(ctx, &plan, q, k_new, v_new, out, lse, s))) return rc;
  if (!plan.split.merges.empty() && (rc = pie_launch_merge(ctx, &plan, plan.split, out, lse, s))) return rc;
  return PIE_OK;
}


// ------------------------------------------------------------------------------ failure path probe
// A warp waits on a barrier nobody arrives at.  The bounded wait gives up after about a second,
// writes PIE_ERR_DEVICE_TIMEOUT to the status word and the kernel returns: the context stays usable.
namespace {
__global__ void wait_probe_kernel(int* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    pie_ptx::mbar_init(pie_ptx::smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  pie_ptx::mbar_wait(pie_ptx::smem_u32(&bar), 0, status);
}
}  // namespace

int pie_debug_bounded_wait(pie_ctx* ctx, void* stream) {
  if (!ctx) return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  wait_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(ctx->d_status);
  PIE_CUDA(ctx, cudaGetLastError());
  return PIE_OK;
}
