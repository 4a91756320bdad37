// Prefill attention over the paged KV cache: causal, grouped-query, fp32 softmax.
// Query row t of sequence s sits at absolute position tok_pos[t] and sees cached positions
// 0 .. tok_pos[t] (its own k, v were appended by the RoPE/KV-write kernel beforehand).
#include "common.cuh"
#include "hyperion.h"

namespace hyp {

// Simple kernel: one warp per (row, query head); lanes split the head dimension.
template <int D>
__global__ void attn_prefill_rowwarp_kernel(const __nv_bfloat16* __restrict__ qkv,
                                            const __nv_bfloat16* __restrict__ kv_layer,
                                            __nv_bfloat16* __restrict__ out, BatchMeta bm, ModelDims d) {
  constexpr int EPL = D / 32;  // elements per lane
  constexpr int PT = 16;
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp_global >= bm.n_tokens * d.Hq) return;
  const int t = warp_global / d.Hq, hq = warp_global % d.Hq;
  const int kvh = hq / (d.Hq / d.Hkv);
  const int pos = bm.tok_pos[t];
  const int32_t* bt = bm.block_table + (size_t)bm.tok_seq[t] * bm.max_pages_per_seq;
  const size_t page_elems = kv_page_elems(d.Hkv, PT, D);
  const size_t v_off = (size_t)d.Hkv * PT * D;
  const float scale = rsqrtf((float)D);

  float q[EPL], acc[EPL];
  const __nv_bfloat16* qp = qkv + (size_t)t * d.qkv_rows + (size_t)hq * D + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; ++e) {
    q[e] = __bfloat162float(qp[e]) * scale;
    acc[e] = 0.f;
  }
  float m = -1e30f, l = 0.f;
  for (int j = 0; j <= pos; ++j) {
    const __nv_bfloat16* kp =
        kv_layer + (size_t)bt[j / PT] * page_elems + ((size_t)kvh * PT + (j % PT)) * D + lane * EPL;
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) s += q[e] * __bfloat162float(kp[e]);
    s = warp_sum(s);
    const float m_new = fmaxf(m, s);
    const float corr = __expf(m - m_new), p = __expf(s - m_new);
    l = l * corr + p;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * corr + p * __bfloat162float(kp[v_off + e]);
    m = m_new;
  }
  __nv_bfloat16* op = out + (size_t)t * d.Hq * D + (size_t)hq * D + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; ++e) op[e] = __float2bfloat16_rn(acc[e] / l);
}

int launch_attn_prefill(const __nv_bfloat16* qkv, const __nv_bfloat16* kv_layer, __nv_bfloat16* attn_out,
                        const BatchMeta& bm, const ModelDims& d, cudaStream_t st) {
  const long warps = (long)bm.n_tokens * d.Hq;
  const int block = 128;
  const int grid = (int)((warps * 32 + block - 1) / block);
  if (d.D == 128)
    attn_prefill_rowwarp_kernel<128><<<grid, block, 0, st>>>(qkv, kv_layer, attn_out, bm, d);
  else if (d.D == 64)
    attn_prefill_rowwarp_kernel<64><<<grid, block, 0, st>>>(qkv, kv_layer, attn_out, bm, d);
  else
    return HYP_EINVAL;
  return 1;
}

}  // namespace hyp
