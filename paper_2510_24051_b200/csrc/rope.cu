// Positions inside the path (Section 4.2: `forward` "operates based on explicit sequence
// positions"): for contexts created with rope_theta > 0 the new K rows are rotated before they are
// stored in their KvPages and Q is rotated into a scratch copy that the attention kernels read.
// Rotate-half rotary embedding: pairs (i, i + D/2), angle pos * theta^(-2i/D).  The angle is formed
// and reduced in fp64 (positions reach 10^5, fp32 would lose the fraction), sine / cosine and the
// rotation itself are fp32, results are rounded to the element type.
#include <cuda_bf16.h>

#include <algorithm>

#include "pie_internal.h"

namespace {

template <typename T>
struct Vec16;  // 16 bytes of elements
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const void* p, float* f) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      f[2 * k] = __uint_as_float(w[k] << 16);
      f[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
    }
  }
  __device__ static void store(void* p, const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
      w[k] = *reinterpret_cast<uint32_t*>(&b);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void load(const void* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x, f[1] = v.y, f[2] = v.z, f[3] = v.w;
  }
  __device__ static void store(void* p, const float* f) { *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]); }
};

__device__ __forceinline__ void rotate(float* lo, float* hi, int n, int i0, int pos, const double* __restrict__ inv_freq) {
  constexpr double kTwoPi = 6.283185307179586476925286766559;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    if (e >= n) break;
    double a = (double)pos * inv_freq[i0 + e];
    a -= kTwoPi * floor(a * (1.0 / kTwoPi));  // into [0, 2 pi)
    float sn, cs;
    sincosf((float)a, &sn, &cs);
    const float x = lo[e], y = hi[e];
    lo[e] = x * cs - y * sn;
    hi[e] = y * cs + x * sn;
  }
}

// One thread: one 16-byte chunk of the first half of a row and its partner in the second half.
// Rows: T * H_q query rows (rotated into qrot) followed by T * H_kv new K rows (rotated into the
// pool) and T * H_kv new V rows (copied into the pool).
template <typename T>
__global__ void rope_kernel(uint8_t* __restrict__ pool, const uint8_t* __restrict__ q, uint8_t* __restrict__ qrot,
                            const uint8_t* __restrict__ k_new, const uint8_t* __restrict__ v_new,
                            const int32_t* __restrict__ append_dst, const int32_t* __restrict__ positions,
                            const double* __restrict__ inv_freq, int Tn, int n_q_heads, PoolGeom g) {
  pie_pdl_launch_dependents();
  pie_pdl_wait();
  constexpr int N = Vec16<T>::N;
  const int half_chunks = g.row_bytes >> 5;                 // 16-byte chunks in half a row
  const int64_t q_items = (int64_t)Tn * n_q_heads * half_chunks;
  const int64_t k_items = (int64_t)Tn * g.n_kv_heads * half_chunks;
  const int64_t total = q_items + 2 * k_items;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    if (i < q_items) {
      const int c = (int)(i % half_chunks);
      const int64_t row = i / half_chunks;                   // t * H_q + h
      const int t = (int)(row / n_q_heads);
      const uint8_t* src = q + row * g.row_bytes;
      float lo[8], hi[8];
      Vec16<T>::load(src + c * 16, lo);
      Vec16<T>::load(src + (half_chunks + c) * 16, hi);
      rotate(lo, hi, N, c * N, positions[t], inv_freq);
      Vec16<T>::store(qrot + row * g.row_bytes + c * 16, lo);
      Vec16<T>::store(qrot + row * g.row_bytes + (half_chunks + c) * 16, hi);
    } else {
      int64_t j = i - q_items;
      const int kv = j >= k_items;
      if (kv) j -= k_items;
      const int c = (int)(j % half_chunks);
      const int64_t row = j / half_chunks;                   // t * H_kv + head
      const int t = (int)(row / g.n_kv_heads), head = (int)(row % g.n_kv_heads);
      const uint8_t* src = (kv ? v_new : k_new) + row * g.row_bytes;
      const int dst = append_dst[t];
      const int page = dst / g.page_size, slot = dst - page * g.page_size;
      uint8_t* blk = pool + (int64_t)page * g.page_bytes + (int64_t)(head * 2 + kv) * g.block_bytes;
      if (kv) {
        *reinterpret_cast<uint4*>(blk + pie_chunk_offset(g.slab_bytes, slot, c)) = *reinterpret_cast<const uint4*>(src + c * 16);
        *reinterpret_cast<uint4*>(blk + pie_chunk_offset(g.slab_bytes, slot, half_chunks + c)) =
            *reinterpret_cast<const uint4*>(src + (half_chunks + c) * 16);
      } else {
        float lo[8], hi[8];
        Vec16<T>::load(src + c * 16, lo);
        Vec16<T>::load(src + (half_chunks + c) * 16, hi);
        rotate(lo, hi, N, c * N, positions[t], inv_freq);
        Vec16<T>::store(blk + pie_chunk_offset(g.slab_bytes, slot, c), lo);
        Vec16<T>::store(blk + pie_chunk_offset(g.slab_bytes, slot, half_chunks + c), hi);
      }
    }
  }
}

}  // namespace

int pie_launch_rope(pie_ctx* ctx, const pie_plan* plan, const void* q, const void* k_new, const void* v_new, cudaStream_t s) {
  const PoolGeom& g = ctx->geom;
  const int64_t work = (int64_t)plan->T * (ctx->cfg.num_q_heads + 2 * g.n_kv_heads) * (g.row_bytes >> 5);
  const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((work + 255) / 256, (int64_t)ctx->n_sms * 8));
  if (ctx->cfg.dtype == PIE_DTYPE_BF16)
    PIE_CUDA(ctx, pie_launch_pdl(rope_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, s, ctx->pool, (const uint8_t*)q,
                                 (uint8_t*)ctx->d_qrot, (const uint8_t*)k_new, (const uint8_t*)v_new,
                                 (const int32_t*)plan->d_append_dst, (const int32_t*)plan->d_positions,
                                 (const double*)ctx->d_inv_freq, plan->T, ctx->cfg.num_q_heads, g));
  else
    PIE_CUDA(ctx, pie_launch_pdl(rope_kernel<float>, dim3(grid), dim3(256), 0, s, ctx->pool, (const uint8_t*)q,
                                 (uint8_t*)ctx->d_qrot, (const uint8_t*)k_new, (const uint8_t*)v_new,
                                 (const int32_t*)plan->d_append_dst, (const int32_t*)plan->d_positions,
                                 (const double*)ctx->d_inv_freq, plan->T, ctx->cfg.num_q_heads, g));
  return PIE_OK;
}
