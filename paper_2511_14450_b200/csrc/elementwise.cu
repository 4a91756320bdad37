// Small HBM-trivial kernels of the decoder block: embedding gather, RMSNorm, RoPE + paged KV write.
#include "common.cuh"
#include "hyperion.h"

namespace hyp {

// x[t, :] = E[ids[t], :]  (bf16 -> fp32, exact).  Ids outside [0, V) are clamped (the host
// cannot validate device-resident ids without a sync).
__global__ void embed_kernel(const int32_t* __restrict__ ids, const __nv_bfloat16* __restrict__ E,
                             float* __restrict__ x, int H, int V) {
  pdl_trigger();
  pdl_wait();
  const int t = blockIdx.x;
  int id = ids[t];
  id = id < 0 ? 0 : (id >= V ? V - 1 : id);
  const uint4* src = reinterpret_cast<const uint4*>(E + (size_t)id * H);
  float4* dst = reinterpret_cast<float4*>(x + (size_t)t * H);
  for (int i = threadIdx.x; i < H / 8; i += blockDim.x) {
    const uint4 v = src[i];
    dst[2 * i] = make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    dst[2 * i + 1] = make_float4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w));
  }
}

int launch_embed(const int32_t* ids, const __nv_bfloat16* E, float* x, int M, int H, int V, cudaStream_t st) {
  HYP_CUDA_TRY(launch_pdl(embed_kernel, dim3(M), dim3(128), 0, st, ids, E, x, H, V));
  return 1;
}

__global__ void copy_f32_kernel(const float4* __restrict__ src, float4* __restrict__ dst, size_t n4) {
  pdl_trigger();
  pdl_wait();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

int launch_copy_f32(const float* src, float* dst, size_t n, cudaStream_t st) {
  const size_t n4 = n / 4;  // H is a multiple of 8, so n is a multiple of 4
  int blocks = (int)((n4 + 255) / 256);
  if (blocks > sm_count() * 8) blocks = sm_count() * 8;
  if (blocks < 1) blocks = 1;
  HYP_CUDA_TRY(launch_pdl(copy_f32_kernel, dim3(blocks), dim3(256), 0, st, reinterpret_cast<const float4*>(src),
                          reinterpret_cast<float4*>(dst), n4));
  return 1;
}

// h[r, :] = x[row, :] * rsqrt(mean(x[row, :]^2) + eps) * g, one CTA per output row.
// row = row_index ? row_index[r] : r.  fp32 statistics; output bf16, or fp16 for the q/k/v projection
// (whose inputs need fp16's 11 mantissa bits to keep the softmax weights inside the logit tolerance).
// DEFER (the model's first block, whose input rows are embedding rows, i.e. bf16 values): the row is written
// as x * g * 2^e with 2^e the power of two just below the normalisation factor, and the remaining factor
// rstd / 2^e in [1, 2) goes to row_scale[r] for the consumer of the projection to apply.  x * 2^e is exact, so
// with unit gains the projection's fp16 input carries no rounding error at all (and never more than before).
template <int THREADS, bool F16, bool DEFER = false>
__global__ void __launch_bounds__(THREADS, 1280 / THREADS)  // <= 51 registers: five 256-thread CTAs per SM
rmsnorm_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ g, void* __restrict__ h,
                               int H, float eps, const int32_t* __restrict__ row_index, float* __restrict__ row_scale) {
  constexpr int CACHE = 5;  // float4 per thread kept in registers: rows up to THREADS * 20 wide are read once
  __shared__ float red[THREADS / 32];
  const int r = blockIdx.x;
  const int n4 = H / 4;
  // the gains are weights: fetch them (a DRAM miss, they are read once per step) while the predecessor still runs
  const uint2* gr = reinterpret_cast<const uint2*>(g);
  uint2 gk[CACHE];
#pragma unroll
  for (int c = 0; c < CACHE; ++c) {
    const int i = threadIdx.x + c * THREADS;
    gk[c] = i < n4 ? gr[i] : make_uint2(0u, 0u);
  }
  pdl_trigger();
  pdl_wait();
  const int row = row_index ? row_index[r] : r;
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)row * H);
  float4 keep[CACHE];
  float ss = 0.f;
#pragma unroll
  for (int c = 0; c < CACHE; ++c) {
    const int i = threadIdx.x + c * THREADS;
    keep[c] = i < n4 ? xr[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    ss += keep[c].x * keep[c].x + keep[c].y * keep[c].y + keep[c].z * keep[c].z + keep[c].w * keep[c].w;
  }
  for (int i = threadIdx.x + CACHE * THREADS; i < n4; i += THREADS) {
    const float4 v = xr[i];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < THREADS / 32; ++w) tot += red[w];
  float rstd = rsqrtf(tot / (float)H + eps);
  if (DEFER) {
    const float pow2 = __uint_as_float(__float_as_uint(rstd) & 0x7f800000u);  // 2^floor(log2(rstd))
    if (threadIdx.x == 0) row_scale[r] = rstd / pow2;
    rstd = pow2;
  }
  uint2* hr = reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(h) + (size_t)r * H);
  auto emit = [&](int i, const float4& v, const uint2 gg) {
    const float y0 = v.x * rstd * bf16_lo(gg.x), y1 = v.y * rstd * bf16_hi(gg.x);
    const float y2 = v.z * rstd * bf16_lo(gg.y), y3 = v.w * rstd * bf16_hi(gg.y);
    uint2 o;
    o.x = F16 ? pack_f16_sat(y0, y1) : pack_bf16(y0, y1);
    o.y = F16 ? pack_f16_sat(y2, y3) : pack_bf16(y2, y3);
    hr[i] = o;
  };
#pragma unroll
  for (int c = 0; c < CACHE; ++c) {
    const int i = threadIdx.x + c * THREADS;
    if (i < n4) emit(i, keep[c], gk[c]);
  }
  for (int i = threadIdx.x + CACHE * THREADS; i < n4; i += THREADS) emit(i, xr[i], gr[i]);
}

int launch_rmsnorm(const float* x, const __nv_bfloat16* g, void* h, bool out_f16, int M, int H, float eps,
                   const int32_t* row_index, cudaStream_t st, bool gains_are_constant, float* defer_scale) {
  // the kernel reads g before it waits for its predecessor: only launched early when g cannot be that
  // predecessor's output
  if (defer_scale) {
    if (!out_f16 || !gains_are_constant) return HYP_EINVAL;
    HYP_CUDA_TRY(launch_pdl<2>(rmsnorm_kernel<256, true, true>, dim3(M), dim3(256), 0, st, x, g, h, H, eps, row_index,
                               defer_scale));
    return 1;
  }
  float* none = nullptr;
  if (gains_are_constant) {
    if (out_f16)
      HYP_CUDA_TRY(launch_pdl<2>(rmsnorm_kernel<256, true>, dim3(M), dim3(256), 0, st, x, g, h, H, eps, row_index, none));
    else
      HYP_CUDA_TRY(launch_pdl<2>(rmsnorm_kernel<256, false>, dim3(M), dim3(256), 0, st, x, g, h, H, eps, row_index, none));
  } else {
    if (out_f16)
      HYP_CUDA_TRY(launch_pdl<4>(rmsnorm_kernel<256, true>, dim3(M), dim3(256), 0, st, x, g, h, H, eps, row_index, none));
    else
      HYP_CUDA_TRY(launch_pdl<4>(rmsnorm_kernel<256, false>, dim3(M), dim3(256), 0, st, x, g, h, H, eps, row_index, none));
  }
  return 1;
}

// Rotate q and k of every new row by its position and append k, v to the sequence's pages.
// Input row layout (fp32, straight from the projection's accumulators): [Q heads | K heads | V heads],
// each head D wide.  Outputs are fp16 (rounded once): q to its own [M, Hq*D] buffer, k and v to the pages.
// One thread handles 8 rotation pairs (i .. i+7, i+D/2 .. i+D/2+7) of one head of one row.
// SPLIT (the model's first block): every element of the row is first multiplied by row_scale[t] (the RMSNorm
// factor that this block applies after the projection instead of before it), and the rotated queries and keys are
// stored as two fp16 terms, value = hi + lo with lo the rounding residue of hi: the high terms where the plain
// kernel stores them, the low terms in q_lo (layout of q16) and in klo_layer ([page][Hkv][16][D], the cache's row
// order).
__device__ __forceinline__ uint32_t pack_f16_residue(float a, float b, uint32_t hi) {
  const __half2 h = *reinterpret_cast<const __half2*>(&hi);
  return pack_f16(a - __low2float(h), b - __high2float(h));
}
template <bool SPLIT>
__global__ void __launch_bounds__(256, 4)
rope_kv_write_kernel(const float* __restrict__ qkv, __half* __restrict__ q16, __half* __restrict__ kv_layer,
                     const float2* __restrict__ rope_table, const float* __restrict__ row_scale,
                     __half* __restrict__ q_lo, __half* __restrict__ klo_layer, BatchMeta bm, ModelDims d) {
  pdl_trigger();
  pdl_wait();
  constexpr int ITEMS = 2;  // work items of a thread whose loads are issued together
  const int t = blockIdx.x;
  const int vec_per_head = d.D / 16;
  const int n_heads = d.Hq + 2 * d.Hkv;
  const int n_work = n_heads * vec_per_head;
  const float* row = qkv + (size_t)t * d.qkv_rows;
  for (int w0 = threadIdx.x; w0 < n_work; w0 += ITEMS * blockDim.x) {
    // the projection's rows first: they depend on nothing, the token's position and page are a chain of two loads
    float4 a[ITEMS][2], b[ITEMS][2];
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const int w = w0 + it * blockDim.x;
      if (w < n_work) {
        const float* hp = row + (size_t)(w / vec_per_head) * d.D + (w % vec_per_head) * 8;
        a[it][0] = *reinterpret_cast<const float4*>(hp);
        a[it][1] = *reinterpret_cast<const float4*>(hp + 4);
        b[it][0] = *reinterpret_cast<const float4*>(hp + d.D / 2);
        b[it][1] = *reinterpret_cast<const float4*>(hp + d.D / 2 + 4);
      }
    }
    const int pos = bm.tok_pos[t];
    const int sq = bm.tok_seq[t];
    const int page = bm.block_table[(size_t)sq * bm.max_pages_per_seq + pos / d.page_tokens];
    const int slot = pos % d.page_tokens;
    const size_t page_base = (size_t)page * kv_page_elems(d.Hkv, d.page_tokens, d.D);
    const float scale = SPLIT ? row_scale[t] : 1.f;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const int w = w0 + it * blockDim.x;
      if (w >= n_work) break;
      const int head = w / vec_per_head;
      const int i0 = (w % vec_per_head) * 8;
      float x1[8] = {a[it][0].x, a[it][0].y, a[it][0].z, a[it][0].w, a[it][1].x, a[it][1].y, a[it][1].z, a[it][1].w};
      float x2[8] = {b[it][0].x, b[it][0].y, b[it][0].z, b[it][0].w, b[it][1].x, b[it][1].y, b[it][1].z, b[it][1].w};
      if (SPLIT) {
#pragma unroll
        for (int j = 0; j < 8; ++j) { x1[j] *= scale; x2[j] *= scale; }
      }
      __half* dst;
      __half* dst_lo = nullptr;
      if (head < d.Hq + d.Hkv) {
        const float4* cs = reinterpret_cast<const float4*>(rope_table + (size_t)pos * (d.D / 2) + i0);  // (cos, sin) pairs
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float4 c = cs[j];
          const float u0 = x1[2 * j], v0 = x2[2 * j], u1 = x1[2 * j + 1], v1 = x2[2 * j + 1];
          x1[2 * j] = u0 * c.x - v0 * c.y;
          x2[2 * j] = v0 * c.x + u0 * c.y;
          x1[2 * j + 1] = u1 * c.z - v1 * c.w;
          x2[2 * j + 1] = v1 * c.z + u1 * c.w;
        }
        dst = head < d.Hq ? q16 + (size_t)t * d.Hq * d.D + (size_t)head * d.D
                          : kv_layer + page_base + ((size_t)(head - d.Hq) * d.page_tokens + slot) * d.D;
        if (SPLIT)
          dst_lo = head < d.Hq ? q_lo + (size_t)t * d.Hq * d.D + (size_t)head * d.D
                               : klo_layer + (((size_t)page * d.Hkv + (head - d.Hq)) * d.page_tokens + slot) * d.D;
      } else {
        dst = kv_layer + page_base + (size_t)d.Hkv * d.page_tokens * d.D +
              ((size_t)(head - d.Hq - d.Hkv) * d.page_tokens + slot) * d.D;
      }
      // cache rows keep their 16-byte chunks XOR-permuted by the token's slot (see kv_chunk_pos); q rows are plain
      const int sw = head < d.Hq ? 0 : (slot & 7);
      const uint4 h1 = make_uint4(pack_f16_sat(x1[0], x1[1]), pack_f16_sat(x1[2], x1[3]), pack_f16_sat(x1[4], x1[5]),
                                  pack_f16_sat(x1[6], x1[7]));
      const uint4 h2 = make_uint4(pack_f16_sat(x2[0], x2[1]), pack_f16_sat(x2[2], x2[3]), pack_f16_sat(x2[4], x2[5]),
                                  pack_f16_sat(x2[6], x2[7]));
      *reinterpret_cast<uint4*>(dst + (((i0 >> 3) ^ sw) << 3)) = h1;
      *reinterpret_cast<uint4*>(dst + ((((d.D / 2 + i0) >> 3) ^ sw) << 3)) = h2;
      if (SPLIT && dst_lo) {
        *reinterpret_cast<uint4*>(dst_lo + (((i0 >> 3) ^ sw) << 3)) =
            make_uint4(pack_f16_residue(x1[0], x1[1], h1.x), pack_f16_residue(x1[2], x1[3], h1.y),
                       pack_f16_residue(x1[4], x1[5], h1.z), pack_f16_residue(x1[6], x1[7], h1.w));
        *reinterpret_cast<uint4*>(dst_lo + ((((d.D / 2 + i0) >> 3) ^ sw) << 3)) =
            make_uint4(pack_f16_residue(x2[0], x2[1], h2.x), pack_f16_residue(x2[2], x2[3], h2.y),
                       pack_f16_residue(x2[4], x2[5], h2.z), pack_f16_residue(x2[6], x2[7], h2.w));
      }
    }
  }
}

int launch_rope_kv_write(const float* qkv, __half* q16, __half* kv_layer, const float2* rope_table,
                         const BatchMeta& bm, const ModelDims& d, cudaStream_t st, const float* row_scale,
                         __half* q_lo, __half* klo_layer) {
  const int work = (d.Hq + 2 * d.Hkv) * (d.D / 16);
  int threads = ((work / 2 + 31) / 32) * 32;  // two work items per thread
  if (threads > 256) threads = 256;
  if (threads < 32) threads = 32;
  if (row_scale) {
    if (!q_lo || !klo_layer) return HYP_EINVAL;
    HYP_CUDA_TRY(launch_pdl<2>(rope_kv_write_kernel<true>, dim3(bm.n_tokens), dim3(threads), 0, st, qkv, q16, kv_layer,
                               rope_table, row_scale, q_lo, klo_layer, bm, d));
  } else {
    HYP_CUDA_TRY(launch_pdl<2>(rope_kv_write_kernel<false>, dim3(bm.n_tokens), dim3(threads), 0, st, qkv, q16, kv_layer,
                               rope_table, row_scale, q_lo, klo_layer, bm, d));
  }
  return 1;
}

}  // namespace hyp
