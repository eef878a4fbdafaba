// get_next_dist from the logits on (Table 1 `get_next_dist`; Section 4.2 "Sample API": the
// next-token probability distribution, truncated to the top-K tokens, K = 256 by default).
//
// One thread block per row of logits, two passes over the row (the second finds it in L2: a row
// is 256 - 512 KB).
//  1. Every thread takes the maximum of its own entries; every warp sorts its 32 maxima and offers
//     its ceil(K / 32)-th largest.  The smallest offer, tau, has at least K entries of the row at
//     or above it (that many thread maxima alone), so the K-th largest entry of the row is >= tau
//     and nothing below tau can be part of the answer.  The largest maximum is the row maximum.
//  2. The sum of exp(x - max) over the whole vocabulary, and the entries >= tau - a few hundred
//     for continuous data - collected in shared memory.  They are sorted there by (logit
//     descending, token id ascending), which is exactly the order of the result; the first K are
//     written with their probabilities exp(x - max) / sum, not renormalised.
// Rows with so many equal entries around the K-th place that more than 4,096 entries pass the
// filter (quantised logits, constant rows) take the general way instead: radix selection of the
// K-th largest key, eight bits per pass, then the entries above it and, in ascending token order,
// as many entries equal to it as are still missing.
#include <cuda_bf16.h>

#include "pie_internal.h"

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

template <typename T, bool kAligned>
__global__ void __launch_bounds__(kThreads, 1)
next_dist_kernel(const T* __restrict__ logits, int64_t row_stride, int vocab, int K, int32_t* __restrict__ out_ids,
                 float* __restrict__ out_probs) {
  constexpr int VEC = Elem<T>::VEC;
  __shared__ unsigned long long pool[kMaxCand];   // filtered entries (key << 32 | ~token id); the radix path keeps its histograms here
  __shared__ unsigned long long cand[kMaxK];      // thread maxima, then the K survivors of the radix path
  uint32_t (*hist)[256] = reinterpret_cast<uint32_t (*)[256]>(pool);   // [kWarps][256], one histogram per warp
  __shared__ float red[kWarps];
  __shared__ uint32_t scan[kWarps];
  __shared__ uint32_t sh_prefix, sh_krem, sh_cnt;
  __shared__ float sh_max, sh_sum;

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
    const float tau_f = value_of_key(tau), kLog2e = 1.4426950408889634f, neg_max_l2 = -row_max_f * kLog2e;
    walk_row<T, kAligned>(row, vocab, [&](float x, int token) {
      s_acc += exp2f_fast(fmaf(x, kLog2e, neg_max_l2));   // (about 2^-21 relative: the kept tokens below use expf)
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
  // ---- too many entries at or above tau (ties): radix selection of the K-th largest key
  __syncthreads();
  if (tid == 0) {
    sh_cnt = 0u;
    sh_prefix = 0u;
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
    out_ids[(int64_t)blockIdx.x * K + tid] = (int32_t)(0xFFFFFFFFu - (uint32_t)c);
    out_probs[(int64_t)blockIdx.x * K + tid] = expf(x - sh_max) / sh_sum;
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
