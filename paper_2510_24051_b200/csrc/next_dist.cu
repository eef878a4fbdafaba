// get_next_dist from the logits on (Table 1 `get_next_dist`; Section 4.2 "Sample API": the
// next-token probability distribution, truncated to the top-K tokens, K = 256 by default).
//
// Two kernels.  Aligned bf16 rows of at least 8,192 logits run with a CLUSTER of thread blocks per row
// (next_dist_cluster_kernel, described where it is defined).  Everything else - fp32 logits, unaligned or short
// rows - runs with one thread block per row (next_dist_kernel), two passes over the row (the second finds it in
// L2: a row is 256 - 512 KB):
//  1. Every thread takes the maximum of its own entries; every warp sorts its 32 maxima and offers
//     its ceil(K / 32)-th largest.  The smallest offer, tau, has at least K entries of the row at
//     or above it (that many thread maxima alone), so the K-th largest entry of the row is >= tau
//     and nothing below tau can be part of the answer.  The largest maximum is the row maximum.
//  2. The sum of exp(x - max) over the whole vocabulary, and the entries >= tau - a few hundred
//     for continuous data - collected in shared memory.  They are sorted there by (logit
//     descending, token id ascending), which is exactly the order of the result; the first K are
//     written with their probabilities exp(x - max) / sum, not renormalised.
// Rows with so many equal entries around the K-th place that more than 4,096 entries pass the
// filter (quantised logits, constant rows) take the general way instead (radix_path): radix selection of the
// K-th largest key, eight bits per pass, then the entries above it and, in ascending token order,
// as many entries equal to it as are still missing.
#include <cuda_bf16.h>

#include <cooperative_groups.h>

#include "pie_internal.h"
#include "ptx_helpers.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxK = 1024;
#ifndef ND_IN_FLIGHT
#define ND_IN_FLIGHT 4
#endif
constexpr int kInFlight = ND_IN_FLIGHT;
constexpr int kMaxCand = 4096;   // entries the filter may pass before the radix path takes over
static_assert(kMaxCand * 8 >= kWarps * 256 * 4, "the histograms fit into the candidate buffer");

// Order-preserving key: larger logit <=> larger unsigned key.  bf16 keys sit in the upper half.
// (-0 and +0 are the same logit: both get the key of +0, so that only the token id orders them.)
__device__ __forceinline__ uint32_t key_of_bits(uint32_t u) {
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float value_of_key(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

template <typename T>
struct Elem;
template <>
struct Elem<float> {
  static constexpr int VEC = 4;
  static constexpr int DIGITS = 4;
  static __device__ __forceinline__ uint32_t key(float v) { return key_of_bits(__float_as_uint(v)); }
};
template <>
struct Elem<__nv_bfloat16> {
  static constexpr int VEC = 8;
  static constexpr int DIGITS = 2;
  static __device__ __forceinline__ uint32_t key(__nv_bfloat16 v) {
    return key_of_bits((uint32_t)__bfloat16_as_ushort(v) << 16);
  }
};

__device__ __forceinline__ float exp2f_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __uint_as_float((uint32_t)__bfloat16_as_ushort(v) << 16); }

// Calls f(value, token id) for every entry of the row, each thread of the block taking groups of VEC
// consecutive entries.  The 16-byte loads of kInFlight groups are issued back to back, with no branch
// between them (a group past the end re-reads the thread's first group and is then skipped), so that
// they are all in flight before the first value is used.
template <typename T, bool kAligned, typename F>
__device__ __forceinline__ void walk_row(const T* __restrict__ row, int vocab, F&& f) {
  constexpr int VEC = Elem<T>::VEC;
  const int n_groups = vocab / VEC;   // whole groups; the remaining entries follow below
  for (int g0 = threadIdx.x; g0 < n_groups; g0 += kInFlight * kThreads) {
    uint4 raw[kInFlight];
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) {
      const int g = g0 + u * kThreads;
      const T* src = row + (int64_t)(g < n_groups ? g : g0) * VEC;
      if (kAligned) {
        raw[u] = *reinterpret_cast<const uint4*>(src);
      } else {
        T* dst = reinterpret_cast<T*>(&raw[u]);
#pragma unroll
        for (int e = 0; e < VEC; ++e) dst[e] = src[e];
      }
    }
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) {
      const int g = g0 + u * kThreads;
      if (g < n_groups) {
        const T* v = reinterpret_cast<const T*>(&raw[u]);
#pragma unroll
        for (int e = 0; e < VEC; ++e) f(to_float(v[e]), g * VEC + e);
      }
    }
  }
  const int t = n_groups * VEC + (int)threadIdx.x;
  if (t < vocab) f(to_float(row[t]), t);
}

// VEC consecutive entries of the row starting at `base` as keys; returns how many of them lie
// inside the row (the others get key 0 and are ignored by their index).
template <typename T, bool kAligned>
__device__ __forceinline__ int load_keys(const T* __restrict__ row, int base, int vocab, uint32_t* keys) {
  constexpr int VEC = Elem<T>::VEC;
  const int n_valid = min(VEC, vocab - base);
  if (kAligned && n_valid == VEC) {
    const uint4 raw = *reinterpret_cast<const uint4*>(row + base);
    const T* v = reinterpret_cast<const T*>(&raw);
#pragma unroll
    for (int e = 0; e < VEC; ++e) keys[e] = Elem<T>::key(v[e]);
  } else {
#pragma unroll
    for (int e = 0; e < VEC; ++e) keys[e] = e < n_valid ? Elem<T>::key(row[base + e]) : 0u;
  }
  return n_valid;
}

// Bitonic sort of a[0, n) in shared memory, descending; n is a power of two, the whole block takes part.
__device__ __forceinline__ void sort_descending(unsigned long long* a, int n) {
  for (int size = 2; size <= n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int p = threadIdx.x; p < (n >> 1); p += kThreads) {
        const int i = 2 * p - (p & (stride - 1)), j = i + stride;   // the p-th pair of this step
        const unsigned long long x = a[i], y = a[j];
        if ((x < y) == ((i & size) == 0)) {
          a[i] = y;
          a[j] = x;
        }
      }
      __syncthreads();
    }
  }
}

// The same for n <= kThreads with one element per thread: steps whose partner sits in the same warp
// exchange registers by shuffle, only the others go through shared memory and a block barrier.
__device__ __forceinline__ void sort_descending_small(unsigned long long* a, int n) {
  const int tid = threadIdx.x;
  unsigned long long v = tid < n ? a[tid] : 0ull;
  for (int size = 2; size <= n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      const bool keep_larger = ((tid & stride) == 0) == ((tid & size) == 0);   // lower index of a descending pair, or upper of an ascending one
      unsigned long long other;
      if (stride < 32) {
        other = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
      } else {
        __syncthreads();
        if (tid < n) a[tid] = v;
        __syncthreads();
        other = tid < n ? a[tid ^ stride] : 0ull;
      }
      v = keep_larger ? (v > other ? v : other) : (v < other ? v : other);
    }
  }
  __syncthreads();
  if (tid < n) a[tid] = v;
  __syncthreads();
}

// Scratch of one thread block in shared memory (both kernels).
struct NdScratch {
  unsigned long long pool[kMaxCand];   // filtered entries (key << 32 | ~token id); the radix path keeps its histograms here
  unsigned long long cand[kMaxK];      // the K survivors of the radix path
  float red[kWarps];
  uint32_t scan[kWarps];
  uint32_t sh_prefix, sh_krem, sh_cnt;
  float sh_max, sh_sum;
};

// The general way for rows with many equal entries around the K-th place: radix selection of the K-th largest
// key, eight bits per pass (the first pass also finds the row maximum, the second the sum of exp(x - max) over
// the whole row), then the entries above it and, in ascending token order, as many entries equal to it as are
// still missing.  The whole block takes part; reads the row from global memory.
template <typename T, bool kAligned>
__device__ __noinline__ void radix_path(const T* __restrict__ row, int vocab, int K, int64_t row_idx, int32_t* __restrict__ out_ids,
                                        float* __restrict__ out_probs, NdScratch& sc) {
  constexpr int VEC = Elem<T>::VEC;
  unsigned long long* const pool = sc.pool;
  unsigned long long* const cand = sc.cand;
  uint32_t (*hist)[256] = reinterpret_cast<uint32_t (*)[256]>(pool);   // [kWarps][256], one histogram per warp
  float* const red = sc.red;
  uint32_t* const scan = sc.scan;
  uint32_t& sh_prefix = sc.sh_prefix;
  uint32_t& sh_krem = sc.sh_krem;
  uint32_t& sh_cnt = sc.sh_cnt;
  float& sh_max = sc.sh_max;
  float& sh_sum = sc.sh_sum;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __syncthreads();
  if (tid == 0) {
    sh_cnt = 0u;
    sh_prefix = 0u;
    sh_krem = (uint32_t)K;
  }

  float m_loc = -__builtin_huge_valf(), s_loc = 0.f;
  for (int d = 0; d < Elem<T>::DIGITS; ++d) {
    const int shift = 24 - 8 * d;
    for (int b = tid; b < kWarps * 256; b += kThreads) (&hist[0][0])[b] = 0u;
    __syncthreads();
    const uint32_t prefix = sh_prefix;
    const uint32_t himask = d == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
    const float row_max = sh_max;   // (valid from the second pass on)
    for (int base0 = 0; base0 < vocab; base0 += kThreads * VEC) {   // (every thread walks every group: the warp votes below need whole warps)
      const int base = base0 + tid * VEC;
      uint32_t keys[VEC] = {};
      int nv = 0;
      if (base < vocab) nv = load_keys<T, kAligned>(row, base, vocab, keys);
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        const bool in_row = e < nv;
        if (d == 0 && in_row) m_loc = fmaxf(m_loc, value_of_key(keys[e]));
        if (d == 1 && in_row) s_loc += expf(value_of_key(keys[e]) - row_max);
        // entries whose higher digits match take part; equal digits in a warp are counted once
        const bool take = in_row && ((keys[e] & himask) == prefix);
        if (!__any_sync(0xFFFFFFFFu, take)) continue;
        const uint32_t digit = (keys[e] >> shift) & 0xFFu;
        const uint32_t peers = __match_any_sync(0xFFFFFFFFu, take ? digit : 0x100u + (uint32_t)lane);
        if (take && lane == __ffs(peers) - 1) atomicAdd(&hist[warp][digit], (uint32_t)__popc(peers));
      }
    }
    if (d == 0) {   // row maximum
      for (int o = 16; o > 0; o >>= 1) m_loc = fmaxf(m_loc, __shfl_xor_sync(0xFFFFFFFFu, m_loc, o));
      if (lane == 0) red[warp] = m_loc;
    }
    if (d == 1) {   // sum of exp(x - max) over the whole row
      for (int o = 16; o > 0; o >>= 1) s_loc += __shfl_xor_sync(0xFFFFFFFFu, s_loc, o);
      if (lane == 0) red[warp] = s_loc;
    }
    __syncthreads();
    if (tid < 256) {   // combine the warps' histograms
      uint32_t c = 0;
#pragma unroll 8
      for (int w = 0; w < kWarps; ++w) c += hist[w][tid];
      hist[0][tid] = c;
    }
    if (warp == 8 && d <= 1) {
      float v = red[lane];
      for (int o = 16; o > 0; o >>= 1) v = d == 0 ? fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o)) : v + __shfl_xor_sync(0xFFFFFFFFu, v, o);
      if (lane == 0) (d == 0 ? sh_max : sh_sum) = v;
    }
    __syncthreads();
    if (warp == 0) {
      // the digit that holds the k_rem-th largest of the entries that took part: walk the bins from the
      // top, eight per lane, with a warp scan over the lanes' totals
      const uint32_t k_rem = sh_krem;
      uint32_t mine[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        mine[j] = hist[0][255 - (lane * 8 + j)];   // lane 0 holds the top eight bins
        tot += mine[j];
      }
      uint32_t incl = tot;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
      }
      uint32_t above = incl - tot;   // entries in bins above this lane's bins
      if (above < k_rem && k_rem <= incl) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (above < k_rem && k_rem <= above + mine[j]) {
            sh_prefix = prefix | ((uint32_t)(255 - (lane * 8 + j)) << shift);
            sh_krem = k_rem - above;   // still to take among the entries with this digit
          }
          above += mine[j];
        }
      }
    }
    __syncthreads();
  }
  static_assert(Elem<T>::DIGITS >= 2, "the second pass is where the sum over the row is taken");

  // ---- collect: keys above the threshold, and the first k_rem keys equal to it in token order
  const uint32_t thr = sh_prefix, need_eq = sh_krem, n_gt = (uint32_t)K - need_eq;
  uint32_t eq_before = 0;   // equal keys in the groups already walked (same value in every thread)
  for (int base0 = 0; base0 < vocab; base0 += kThreads * VEC) {
    const int base = base0 + tid * VEC;
    uint32_t keys[VEC] = {};
    int nv = 0;
    if (base < vocab) nv = load_keys<T, kAligned>(row, base, vocab, keys);
    uint32_t n_eq = 0;
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      if (e < nv && keys[e] > thr) cand[atomicAdd(&sh_cnt, 1u)] = ((unsigned long long)keys[e] << 32) | (0xFFFFFFFFu - (uint32_t)(base + e));
      n_eq += (e < nv && keys[e] == thr) ? 1u : 0u;
    }
    if (eq_before < need_eq) {   // (uniform) rank the equal keys of this group in token order: block-wide exclusive scan
      uint32_t incl = n_eq;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
      }
      if (lane == 31) scan[warp] = incl;
      __syncthreads();
      uint32_t warp_base = 0, total = 0;
      for (int w = 0; w < kWarps; ++w) {
        const uint32_t c = scan[w];
        if (w < warp) warp_base += c;
        total += c;
      }
      uint32_t rank = eq_before + warp_base + incl - n_eq;
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        if (e < nv && keys[e] == thr) {
          if (rank < need_eq) cand[n_gt + rank] = ((unsigned long long)thr << 32) | (0xFFFFFFFFu - (uint32_t)(base + e));
          ++rank;
        }
      }
      eq_before += total;
      __syncthreads();   // `scan` is reused by the next group
    }
  }
  __syncthreads();

  // ---- sort the K survivors and write them out
  int n_sort = 1;
  while (n_sort < K) n_sort <<= 1;
  for (int i = K + tid; i < n_sort; i += kThreads) cand[i] = 0ull;   // padding sorts to the end
  __syncthreads();
  sort_descending(cand, n_sort);
  if (tid < K) {
    const unsigned long long c = cand[tid];
    const float x = value_of_key((uint32_t)(c >> 32));
    out_ids[row_idx * K + tid] = (int32_t)(0xFFFFFFFFu - (uint32_t)c);
    out_probs[row_idx * K + tid] = expf(x - sh_max) / sh_sum;
  }
}

template <typename T, bool kAligned>
__global__ void __launch_bounds__(kThreads, 1)
next_dist_kernel(const T* __restrict__ logits, int64_t row_stride, int vocab, int K, int32_t* __restrict__ out_ids,
                 float* __restrict__ out_probs) {
  constexpr int VEC = Elem<T>::VEC;
  __shared__ NdScratch sc;
  unsigned long long* const pool = sc.pool;
  float* const red = sc.red;
  uint32_t* const scan = sc.scan;
  uint32_t& sh_prefix = sc.sh_prefix;
  uint32_t& sh_krem = sc.sh_krem;
  uint32_t& sh_cnt = sc.sh_cnt;
  float& sh_max = sc.sh_max;
  float& sh_sum = sc.sh_sum;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* row = logits + (int64_t)blockIdx.x * row_stride;
  if (tid == 0) {
    sh_prefix = 0u;
    sh_krem = (uint32_t)K;
    sh_cnt = 0u;
  }

  // ---- pass 1: thread maxima (as keys), sorted; tau = the K-th largest of them
  {
    float fmax_t = -__builtin_huge_valf();
    walk_row<T, kAligned>(row, vocab, [&](float x, int) { fmax_t = fmaxf(fmax_t, x); });
    const uint32_t kmax = key_of_bits(__float_as_uint(fmax_t));   // (threads without entries offer -inf)
    // every warp sorts its 32 maxima (shuffles only) and offers its ceil(K / 32)-th largest; the smallest
    // offer is a threshold with at least K entries of the row at or above it
    uint32_t v = kmax;
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1)
#pragma unroll
      for (int stride = size >> 1; stride > 0; stride >>= 1) {
        const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
        const bool keep_larger = ((lane & stride) == 0) == ((lane & size) == 0);
        v = keep_larger ? max(v, other) : min(v, other);
      }
    const int j = (K + 31) / 32;   // 1 .. 32
    const uint32_t offer = __shfl_sync(0xFFFFFFFFu, v, j - 1), top = __shfl_sync(0xFFFFFFFFu, v, 0);
    if (lane == 0) {
      scan[warp] = offer;
      red[warp] = __uint_as_float(top);
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t lo = scan[lane], hi = __float_as_uint(red[lane]);
      for (int o = 16; o > 0; o >>= 1) {
        lo = min(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
        hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
      }
      if (lane == 0) {
        sh_prefix = lo;                 // (the radix path, if it runs, resets this)
        sh_max = value_of_key(hi);
      }
    }
    __syncthreads();
  }
  const uint32_t tau = sh_prefix;
  const float row_max_f = sh_max;
  __syncthreads();
  // ---- pass 2: the sum over the row, and the entries at or above tau
  {
    // (plain fp32 arithmetic per entry: exp2 of a fused multiply-add, one comparison with tau as a float; the
    //  integer key is only made for the few entries that pass)
    float s_acc = 0.f;
    const float tau_f = value_of_key(tau), kLog2e = 1.4426950408889634f;
    walk_row<T, kAligned>(row, vocab, [&](float x, int token) {
      s_acc += exp2f_fast((x - row_max_f) * kLog2e);   // (the difference first: exact enough for logits of any magnitude)
      if (x >= tau_f) {
        const uint32_t at = atomicAdd(&sh_cnt, 1u);
        if (at < (uint32_t)kMaxCand) pool[at] = ((unsigned long long)key_of_bits(__float_as_uint(x)) << 32) | (0xFFFFFFFFu - (uint32_t)token);
      }
    });
    for (int o = 16; o > 0; o >>= 1) s_acc += __shfl_xor_sync(0xFFFFFFFFu, s_acc, o);
    if (lane == 0) red[warp] = s_acc;
    __syncthreads();
    if (warp == 0) {
      float v = red[lane];
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
      if (lane == 0) sh_sum = v;
    }
    __syncthreads();
  }
  const uint32_t n_pass = sh_cnt;
  if (n_pass <= (uint32_t)kMaxCand) {   // (n_pass >= K: the K thread maxima at or above tau are entries of the row)
    int n_sort = 1;
    while (n_sort < (int)n_pass) n_sort <<= 1;
    for (int i = (int)n_pass + tid; i < n_sort; i += kThreads) pool[i] = 0ull;   // padding sorts to the end
    __syncthreads();
    if (n_sort <= kThreads) sort_descending_small(pool, n_sort);
    else sort_descending(pool, n_sort);
    if (tid < K) {
      const unsigned long long c = pool[tid];
      out_ids[(int64_t)blockIdx.x * K + tid] = (int32_t)(0xFFFFFFFFu - (uint32_t)c);
      out_probs[(int64_t)blockIdx.x * K + tid] = expf(value_of_key((uint32_t)(c >> 32)) - sh_max) / sh_sum;
    }
    return;
  }
  // ---- too many entries at or above tau (ties): the general way
  radix_path<T, kAligned>(row, vocab, K, (int64_t)blockIdx.x, out_ids, out_probs, sc);
}

// ---------------------------------------------------------------------------------------------
// Decode-sized batches of bf16 logits: a CLUSTER of thread blocks per row.  With one block per row a batch of
// 64 rows fills 64 of 148 SMs and every block is bound by the arithmetic of its two passes.  Here the row is
// cut into S parts; every block of the cluster
//   * brings its part into shared memory with bulk copies (one read of the row from HBM, all of it in flight
//     at once, no registers spent on it);
//   * takes thread maxima and, relative to them, the sum of exponentials in ONE pass while the copies land
//     (the sum is rescaled when a thread's maximum grows; blocks and threads are combined with the factors
//     exp(m_part - m_row) afterwards); finds its ceil(K / S)-th largest thread maximum exactly; the smallest of
//     the blocks' values is tau (at least K entries of the row lie at or above it, and few more), the largest
//     maximum the row maximum - exchanged through distributed shared memory;
//   * collects its entries at or above tau from shared memory with packed comparisons.
// The candidates go straight into block 0's pool through distributed shared memory (their order there is
// arbitrary: they are sorted afterwards); block 0 adds the partial sums in rank order (the result does not
// depend on timing), sorts and writes the row.  A row with more than kMaxCand candidates (many equal logits)
// is redone by block 0 alone the general way.  Every block passes the same two cluster barriers.
constexpr int kNdMaxPart = 160 * 1024;   // bytes of a row that one block keeps in shared memory
constexpr int kNdChunk = kThreads * 16;  // bytes per bulk copy: one 16-byte group per thread
constexpr int kNdMaxChunks = kNdMaxPart / kNdChunk;
constexpr int kNdMaxCluster = 8;
constexpr int kNdBins = 2048;            // distinct bf16 values between tau and the row maximum that the counting sort covers

struct NdClusterShared {
  NdScratch sc;
  uint32_t x_lo[kNdMaxCluster], x_hi[kNdMaxCluster];   // every block's threshold / largest maximum (written by the peers)
  float x_sum[kNdMaxCluster];                           // block 0: partial sums, each relative to its block's maximum
  uint32_t l_cnt, l_base;                               // candidates staged in this block, their place in block 0's pool
  uint32_t bin_start[kNdBins], bin_cur[kNdBins];        // block 0: counting sort of the candidates by logit
  unsigned long long bar[kNdMaxChunks];
};

__global__ void __launch_bounds__(kThreads, 1)
next_dist_cluster_kernel(const __nv_bfloat16* __restrict__ logits, int64_t row_stride, int vocab, int K, int groups_per_part,
                         int32_t* __restrict__ out_ids, float* __restrict__ out_probs, int* status) {
  namespace cg = cooperative_groups;
  using namespace pie_ptx;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  extern __shared__ __align__(128) uint8_t nd_smem[];
  const uint4* part = reinterpret_cast<const uint4*>(nd_smem);   // this block's groups of 8 entries
  NdClusterShared& sh = *reinterpret_cast<NdClusterShared*>(nd_smem + kNdMaxPart);
  NdScratch& sc = sh.sc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t row_idx = blockIdx.x / S;
  const __nv_bfloat16* row = logits + row_idx * row_stride;
  const int n_groups = vocab / 8;
  const int g0 = rank * groups_per_part, n_mine = max(0, min(groups_per_part, n_groups - g0));
  const int n_chunks = (n_mine + kThreads - 1) / kThreads;
  constexpr float kLog2e = 1.4426950408889634f, kNegInf = -__builtin_huge_valf();

  // one thread per chunk sets up the chunk's barrier and starts its copy (the barrier is only waited on by
  // threads that pass the block barrier below, i.e. after its initialisation)
  if (tid < n_chunks) {
    const int c = tid;
    mbar_init(smem_u32(&sh.bar[c]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const uint32_t bytes = (uint32_t)min(kThreads, n_mine - c * kThreads) * 16u;
    mbar_expect_tx(smem_u32(&sh.bar[c]), bytes);
    bulk_g2s(smem_u32(nd_smem + (size_t)c * kNdChunk), row + ((int64_t)g0 + (int64_t)c * kThreads) * 8, bytes, smem_u32(&sh.bar[c]));
  }
  if (tid == 0) {
    sc.sh_cnt = 0u;
    sh.l_cnt = 0u;
  }
  __syncthreads();

  // ---- the one pass over the part, chunk by chunk as the copies land: the thread's maximum and, relative to
  // it, the thread's share of the sum of exponentials (rescaled when the maximum grows: the arithmetic of this
  // pass hides behind the arrival of the data).  Packed bf16 maxima, packed fp32 multiply-adds and sums.
  float m_t = kNegInf;
  uint64_t acc_a = 0ull, acc_b = 0ull;   // two fp32 pairs (0, 0)
  uint64_t scale2;
  asm("mov.b64 %0, {%1,%1};" : "=l"(scale2) : "f"(kLog2e));
  auto add_entry = [&](float x, float& acc) {   // (the few entries behind the last whole group)
    if (x > m_t) {
      const float f = exp2f_fast((m_t - x) * kLog2e);
      uint64_t f2;
      asm("mov.b64 %0, {%1,%1};" : "=l"(f2) : "f"(f));
      asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(acc_a) : "l"(f2));
      asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(acc_b) : "l"(f2));
      acc *= f;
      m_t = x;
    }
    if (m_t != kNegInf) acc += exp2f_fast((x - m_t) * kLog2e);
  };
  for (int c = 0; c < n_chunks; ++c) {
    mbar_wait(smem_u32(&sh.bar[c]), 0, status);
    if (c * kThreads + tid < n_mine) {
      const uint4 v = part[c * kThreads + tid];
      uint32_t g2 = v.x;
      asm("max.bf16x2 %0, %0, %1;" : "+r"(g2) : "r"(v.y));
      asm("max.bf16x2 %0, %0, %1;" : "+r"(g2) : "r"(v.z));
      asm("max.bf16x2 %0, %0, %1;" : "+r"(g2) : "r"(v.w));
      const float gmax = fmaxf(__uint_as_float(g2 << 16), __uint_as_float(g2 & 0xFFFF0000u));
      if (gmax > m_t) {
        const float f = exp2f_fast((m_t - gmax) * kLog2e);   // (0 when there was no maximum yet: the sums are 0 then)
        uint64_t f2;
        asm("mov.b64 %0, {%1,%1};" : "=l"(f2) : "f"(f));
        asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(acc_a) : "l"(f2));
        asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(acc_b) : "l"(f2));
        m_t = gmax;
      }
      if (m_t != kNegInf) {
        uint64_t negm2;   // (x - m first, then the scale: the rounded product m * log2(e) would cost accuracy at large |m|)
        asm("mov.b64 %0, {%1,%1};" : "=l"(negm2) : "f"(-m_t));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          uint64_t x2, y2, p2;
          float e0, e1;
          asm("mov.b64 %0, {%1,%2};" : "=l"(x2) : "r"(w[e] << 16), "r"(w[e] & 0xFFFF0000u));
          asm("add.rn.f32x2 %0, %1, %2;" : "=l"(y2) : "l"(x2), "l"(negm2));
          asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(y2) : "l"(scale2));
          asm("mov.b64 {%0,%1}, %2;" : "=f"(e0), "=f"(e1) : "l"(y2));
          asm("mov.b64 %0, {%1,%2};" : "=l"(p2) : "f"(exp2f_fast(e0)), "f"(exp2f_fast(e1)));
          if (e & 1) asm("add.rn.f32x2 %0, %0, %1;" : "+l"(acc_b) : "l"(p2));
          else asm("add.rn.f32x2 %0, %0, %1;" : "+l"(acc_a) : "l"(p2));
        }
      }
    }
  }
  float s_tail = 0.f;
  if (rank == S - 1 && n_groups * 8 + tid < vocab) add_entry(to_float(row[n_groups * 8 + tid]), s_tail);
  const uint32_t tmax_key = key_of_bits(__float_as_uint(m_t));

  // The block's maximum and sum; its ceil(K / S)-th largest thread maximum, exactly: the largest key v with at
  // least that many thread maxima >= v, found bit by bit (bf16 keys: the upper 16 bits).  The smallest of the S
  // blocks' values is tau: at least K entries of the row lie at or above it, and few more than K do.
  {
    uint32_t hi = tmax_key;
    for (int o = 16; o > 0; o >>= 1) hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
    if (lane == 0) sc.scan[warp] = hi;
    const int kb = (K + S - 1) / S;   // <= kThreads
    uint32_t prefix = 0u;
#pragma unroll 1
    for (int bit = 31; bit >= 16; --bit) {
      const uint32_t v = prefix | (1u << bit);
      if (__syncthreads_count(tmax_key >= v) >= kb) prefix = v;
    }
    hi = sc.scan[lane];   // (written before the barriers of the loop above)
    for (int o = 16; o > 0; o >>= 1) hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
    const float m_block = value_of_key(hi);
    float s_acc = 0.f;
    if (m_t != kNegInf) {
      float a0, a1, b0, b1;
      asm("mov.b64 {%0,%1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc_a));
      asm("mov.b64 {%0,%1}, %2;" : "=f"(b0), "=f"(b1) : "l"(acc_b));
      s_acc = (((a0 + a1) + (b0 + b1)) + s_tail) * exp2f_fast((m_t - m_block) * kLog2e);
    }
    for (int o = 16; o > 0; o >>= 1) s_acc += __shfl_xor_sync(0xFFFFFFFFu, s_acc, o);
    if (lane == 0) sc.red[warp] = s_acc;
    __syncthreads();
    if (warp == 0) {
      float v = sc.red[lane];
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
      if (lane < S) {   // lane r tells block r
        *cluster.map_shared_rank(&sh.x_lo[rank], lane) = prefix;
        *cluster.map_shared_rank(&sh.x_hi[rank], lane) = hi;
      }
      if (lane == 0) *cluster.map_shared_rank(&sh.x_sum[rank], 0) = v;
    }
  }
  cluster.sync();   // (1) every block has every block's threshold and maximum, block 0 the partial sums
  uint32_t tau = 0xFFFFFFFFu, top = 0u;
  for (int r = 0; r < S; ++r) {
    tau = min(tau, sh.x_lo[r]);
    top = max(top, sh.x_hi[r]);
  }
  const float row_max_f = value_of_key(top);

  // ---- the entries at or above tau (packed bf16 comparisons on the part in shared memory): staged in this
  // block, then copied into block 0's pool through distributed shared memory
  {
    const float tau_f = value_of_key(tau);
    unsigned long long* pool0 = cluster.map_shared_rank(&sc.pool[0], 0);
    uint32_t* cnt0 = cluster.map_shared_rank(&sc.sh_cnt, 0);
    auto offer = [&](uint32_t bits16, int token) {
      const unsigned long long c = ((unsigned long long)key_of_bits(bits16 << 16) << 32) | (0xFFFFFFFFu - (uint32_t)token);
      const uint32_t at = atomicAdd(&sh.l_cnt, 1u);
      if (at < (uint32_t)kMaxK) {
        sc.cand[at] = c;
      } else {   // (more than the staging area holds: many equal logits; straight to block 0)
        const uint32_t at0 = atomicAdd(cnt0, 1u);
        if (at0 < (uint32_t)kMaxCand) pool0[at0] = c;
      }
    };
    const uint32_t tau16 = __float_as_uint(tau_f) >> 16;
    const uint32_t tau2 = tau16 | (tau16 << 16);
    for (int c = 0; c < n_chunks; ++c) {
      const int g = c * kThreads + tid;
      if (g < n_mine) {
        const uint4 v = part[g];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t m[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(m[e]) : "r"(w[e]), "r"(tau2));
        if ((m[0] | m[1] | m[2] | m[3]) != 0u) {
          const int token = (g0 + g) * 8;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (m[e] & 0x0000FFFFu) offer(w[e] & 0xFFFFu, token + 2 * e);
            if (m[e] & 0xFFFF0000u) offer(w[e] >> 16, token + 2 * e + 1);
          }
        }
      }
    }
    if (rank == S - 1) {   // entries behind the last whole group of the row
      const int t = n_groups * 8 + tid;
      if (t < vocab && to_float(row[t]) >= tau_f) offer((uint32_t)__bfloat16_as_ushort(row[t]), t);
    }
    __syncthreads();
    const uint32_t n_loc = min(sh.l_cnt, (uint32_t)kMaxK);
    if (tid == 0) sh.l_base = atomicAdd(cnt0, n_loc);
    __syncthreads();
    const uint32_t base = sh.l_base;
    for (uint32_t i = tid; i < n_loc; i += kThreads)
      if (base + i < (uint32_t)kMaxCand) pool0[base + i] = sc.cand[i];
  }
  cluster.sync();   // (2) block 0 holds every block's candidates; the peers are done
  if (rank != 0) return;
  const uint32_t n_pass = sc.sh_cnt;
  if (n_pass > (uint32_t)kMaxCand) {   // many equal logits around the K-th place: the general way
    radix_path<__nv_bfloat16, true>(row, vocab, K, row_idx, out_ids, out_probs, sc);
    return;
  }
  float sum = 0.f;   // in rank order: the result does not depend on timing
  for (int r = 0; r < S; ++r) sum += sh.x_sum[r] * exp2f_fast((value_of_key(sh.x_hi[r]) - row_max_f) * kLog2e);

  const uint32_t hi16 = top >> 16, span = hi16 - (tau >> 16) + 1u;
  if (span <= (uint32_t)kNdBins && n_pass <= (uint32_t)kMaxK) {
    // ---- counting sort: the candidates' logits are bf16 values between tau and the maximum, a few hundred
    // distinct keys at most.  Bin b holds the key hi16 - b (descending logit); inside a bin the order is
    // ascending token id.
    for (uint32_t b = tid; b < span; b += kThreads) sh.bin_cur[b] = 0u;
    __syncthreads();
    unsigned long long mine = 0ull;
    uint32_t my_bin = 0u;
    if (tid < (int)n_pass) {
      mine = sc.pool[tid];
      my_bin = hi16 - (uint32_t)(mine >> 48);
      atomicAdd(&sh.bin_cur[my_bin], 1u);
    }
    __syncthreads();
    {   // exclusive scan over the bins: two bins per thread, warp scans, then the warps' totals
      const uint32_t b0 = 2u * tid, c0 = b0 < span ? sh.bin_cur[b0] : 0u, c1 = b0 + 1 < span ? sh.bin_cur[b0 + 1] : 0u;
      uint32_t incl = c0 + c1;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
      }
      if (lane == 31) sc.scan[warp] = incl;
      __syncthreads();
      uint32_t warp_base = 0;
      for (int w = 0; w < warp; ++w) warp_base += sc.scan[w];
      const uint32_t excl = warp_base + incl - (c0 + c1);
      if (b0 < span) sh.bin_start[b0] = sh.bin_cur[b0] = excl;
      if (b0 + 1 < span) sh.bin_start[b0 + 1] = sh.bin_cur[b0 + 1] = excl + c0;
    }
    __syncthreads();
    if (tid < (int)n_pass) sc.cand[atomicAdd(&sh.bin_cur[my_bin], 1u)] = mine;   // grouped by bin, any order inside
    __syncthreads();
    if (tid < (int)n_pass) {
      const uint32_t first = sh.bin_start[my_bin], end = sh.bin_cur[my_bin];
      uint32_t pos = first;
      for (uint32_t j = first; j < end; ++j) pos += sc.cand[j] > mine ? 1u : 0u;   // equal keys: larger value = smaller token id
      if (pos < (uint32_t)K) {
        out_ids[row_idx * K + pos] = (int32_t)(0xFFFFFFFFu - (uint32_t)mine);
        out_probs[row_idx * K + pos] = expf(value_of_key((uint32_t)(mine >> 32)) - row_max_f) / sum;
      }
    }
    return;
  }
  int n_sort = 1;
  while (n_sort < (int)n_pass) n_sort <<= 1;
  for (int i = (int)n_pass + tid; i < n_sort; i += kThreads) sc.pool[i] = 0ull;   // padding sorts to the end
  __syncthreads();
  if (n_sort <= kThreads) sort_descending_small(sc.pool, n_sort);
  else sort_descending(sc.pool, n_sort);
  if (tid < K) {
    const unsigned long long c = sc.pool[tid];
    out_ids[row_idx * K + tid] = (int32_t)(0xFFFFFFFFu - (uint32_t)c);
    out_probs[row_idx * K + tid] = expf(value_of_key((uint32_t)(c >> 32)) - row_max_f) / sum;
  }
}

}  // namespace

int pie_get_next_dist(pie_ctx* ctx, const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab, int64_t row_stride,
                      int32_t top_k, int32_t* out_ids, float* out_probs, void* stream) {
  if (!ctx || n_rows < 0 || vocab < 1 || top_k < 1 || top_k > kMaxK || top_k > vocab || row_stride < vocab ||
      (dtype != PIE_DTYPE_BF16 && dtype != PIE_DTYPE_F32))
    return PIE_ERR_INVALID;
  if (ctx->host_only) return PIE_ERR_NO_DEVICE;
  if (n_rows == 0) return PIE_OK;
  if (!logits || !out_ids || !out_probs) return PIE_ERR_INVALID;
  cudaStream_t s = (cudaStream_t)stream;
  PIE_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  const size_t esize = dtype == PIE_DTYPE_BF16 ? 2 : 4;
  const bool aligned = ((uintptr_t)logits % 16 == 0) && ((size_t)row_stride * esize % 16 == 0);
  if (dtype == PIE_DTYPE_BF16 && aligned && vocab >= 8 * kThreads) {
    // a cluster per row: the smallest power of two of blocks whose part of the row fits into shared memory,
    // doubled while the batch still leaves SMs without a block
    const int n_groups = vocab / 8;
    int S = 1;
    while (S < kNdMaxCluster && (int64_t)((n_groups + S - 1) / S) * 16 > kNdMaxPart) S *= 2;
    while (S < kNdMaxCluster && (int64_t)n_rows * S * 2 <= ctx->n_sms && n_groups / (2 * S) >= 2 * kThreads) S *= 2;   // (parts stay >= 2 groups per thread)
    const int gpp = (n_groups + S - 1) / S;
    if ((int64_t)gpp * 16 <= kNdMaxPart) {
      const size_t smem = kNdMaxPart + sizeof(NdClusterShared);
      if (!ctx->nd_configured) {
        PIE_CUDA(ctx, cudaFuncSetAttribute(next_dist_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        ctx->nd_configured = true;
      }
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)(n_rows * S));
      cfg.blockDim = dim3(kThreads);
      cfg.dynamicSmemBytes = smem;
      cfg.stream = s;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = (unsigned)S;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      // (a device that cannot place such clusters - fewer SMs per GPC, a partitioned GPU - refuses the launch:
      //  the one-block kernel below then does the work)
      if (cudaLaunchKernelEx(&cfg, next_dist_cluster_kernel, (const __nv_bfloat16*)logits, row_stride, (int)vocab, (int)top_k, gpp, out_ids,
                             out_probs, ctx->d_status) == cudaSuccess)
        return PIE_OK;
      cudaGetLastError();
    }
  }
  if (dtype == PIE_DTYPE_BF16) {
    auto* p = (const __nv_bfloat16*)logits;
    if (aligned) next_dist_kernel<__nv_bfloat16, true><<<n_rows, kThreads, 0, s>>>(p, row_stride, vocab, top_k, out_ids, out_probs);
    else next_dist_kernel<__nv_bfloat16, false><<<n_rows, kThreads, 0, s>>>(p, row_stride, vocab, top_k, out_ids, out_probs);
  } else {
    auto* p = (const float*)logits;
    if (aligned) next_dist_kernel<float, true><<<n_rows, kThreads, 0, s>>>(p, row_stride, vocab, top_k, out_ids, out_probs);
    else next_dist_kernel<float, false><<<n_rows, kThreads, 0, s>>>(p, row_stride, vocab, top_k, out_ids, out_probs);
  }
  PIE_CUDA(ctx, cudaGetLastError());
  return PIE_OK;
}
