// Decode attention: one query row per sequence against its paged KV cache, split along the
// context so that a small batch still fills the GPU, followed by a log-sum-exp merge.
//
//   partial kernel: grid (n_splits, Hkv, n_seqs), 4 warps.  A CTA streams its context slice of one KV
//   head through shared memory in 64-token tiles (double-buffered cp.async, 128-bit, each byte read
//   once) and serves the G = Hq/Hkv query heads that share the head as the rows of one
//   mma.sync.m16n8k16 operand (rows >= G are padding; q, k, v and the softmax weights are fp16).  Warp w owns keys 16w..16w+15 of every tile:
//   it forms their scores, keeps its own online-softmax state and its own O += P V partial, so there is
//   no cross-warp traffic inside the loop; the four warps are combined once at the end.  Tensor cores
//   are used because the scalar version needs ~130 instructions per KB of cache and is issue-bound at
//   HBM speed; the roofline of this kernel is HBM.
//   merge kernel: grid (n_seqs * Hq).  Combines the split partials and writes fp16.
//
// Scratch layout (fp32): acc [n_seqs][Hq][n_splits][D], then ml [n_seqs][Hq][n_splits][2].
#include "attn_common.cuh"
#include "hyperion.h"

namespace hyp {

constexpr int AD_WARPS = 4;
constexpr int AD_TILE = 64;
constexpr float AD_NEG = -1e30f;

size_t attn_decode_scratch_bytes(int max_seqs, int Hq, int D, int max_splits) {
  return (size_t)max_seqs * Hq * max_splits * (D + 2) * sizeof(float);
}

int attn_decode_splits(int n_seqs, int Hkv, int max_ctx) {
  int want = (3 * sm_count() + n_seqs * Hkv - 1) / (n_seqs * Hkv);
  int cap = (max_ctx + 2 * AD_TILE - 1) / (2 * AD_TILE);  // at least two tiles per split
  if (want > cap) want = cap;
  if (want > 32) want = 32;
  if (want < 1) want = 1;
  return want;
}

template <int D, int G>
__global__ void __launch_bounds__(AD_WARPS * 32)
attn_decode_partial_kernel(const __half* __restrict__ qkv, const __half* __restrict__ kv_layer,
                           float* __restrict__ part_acc, float* __restrict__ part_ml, int n_splits,
                           BatchMeta bm, ModelDims d) {
  constexpr int KS = D / 16, DN = D / 8, CPR = D / 8, PT = 16;
  constexpr int TILE_BYTES = AD_TILE * D * 2;
  extern __shared__ __align__(128) uint8_t ad_smem[];
  const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(ad_smem);
  auto k_tile = [&](int buf) { return smem0 + buf * TILE_BYTES; };
  auto v_tile = [&](int buf) { return smem0 + (2 + buf) * TILE_BYTES; };

  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  pdl_trigger();
  pdl_wait();  // the cache pages, the query row and the metadata all come from earlier kernels / copies

  const int ctx_total = bm.ctx_lens[b] + 1;  // the new token's k, v are already in the cache
  int tps = (ctx_total + n_splits - 1) / n_splits;
  tps = ((tps + AD_TILE - 1) / AD_TILE) * AD_TILE;
  const int t_begin = split * tps;
  const int t_end = min(ctx_total, t_begin + tps);
  const int n_tiles = t_begin < t_end ? (t_end - t_begin + AD_TILE - 1) / AD_TILE : 0;

  const int32_t* bt = bm.block_table + (size_t)b * bm.max_pages_per_seq;
  const size_t page_elems = kv_page_elems(d.Hkv, PT, D);
  const size_t v_off = (size_t)d.Hkv * PT * D;

  auto load_tile = [&](int j, int buf) {
    for (int idx = threadIdx.x; idx < AD_TILE * CPR; idx += AD_WARPS * 32) {
      const int r = idx / CPR, c = idx % CPR;
      const int key = t_begin + j * AD_TILE + r;
      const bool ok = key < t_end;
      const int kk = ok ? key : t_begin;
      const __half* src =
          kv_layer + (size_t)bt[kk / PT] * page_elems + ((size_t)kvh * PT + (kk % PT)) * D + c * 8;
      // the cache row is stored with the tile's own chunk permutation (tiles start on page boundaries, so
      // r & 7 is the token's slot & 7): chunk positions copy one to one
      cp_async16(k_tile(buf) + r * (D * 2) + c * 16, src, ok);
      cp_async16(v_tile(buf) + r * (D * 2) + c * 16, src + v_off, ok);
    }
  };
  if (n_tiles > 0) load_tile(0, 0);
  cp_async_commit();

  // query heads kvh*G .. kvh*G+G-1 of row b as operand rows 0..G-1 (rows G..15 are zero)
  uint32_t qf[KS][2];  // [k step][k half]; only the "row g" halves of the fragment are non-zero
  {
    const __half* qrow = qkv + (size_t)b * d.qkv_rows + (size_t)(kvh * G + (g < G ? g : 0)) * D;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qf[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * tq) : 0u;
      qf[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * tq) : 0u;
    }
  }
  const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;

  float o[DN][2];  // row g of each 8-wide output column tile (rows 8..15 are padding and dropped)
#pragma unroll
  for (int i = 0; i < DN; ++i) o[i][0] = o[i][1] = 0.f;
  float m_run = AD_NEG, l_run = 0.f;

  for (int j = 0; j < n_tiles; ++j) {
    const int buf = j & 1;
    if (j + 1 < n_tiles) load_tile(j + 1, buf ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();

    // scores of this warp's 16 keys: two 8-key column tiles
    float s[2][4];
    s[0][0] = s[0][1] = s[0][2] = s[0][3] = 0.f;
    s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int r = 16 * warp + (lane & 7) + ((lane >> 4) << 3);
      const int c = 2 * ks + ((lane >> 3) & 1);
      uint32_t b0, b1, b2, b3;
      ldsm_x4(k_tile(buf) + tile_off<D>(r, c), b0, b1, b2, b3);
      mma_f16_16816(s[0], qf[ks][0], 0u, qf[ks][1], 0u, b0, b1);
      mma_f16_16816(s[1], qf[ks][0], 0u, qf[ks][1], 0u, b2, b3);
    }
    const int key0 = t_begin + j * AD_TILE + 16 * warp + 2 * tq;
    float mx = m_run;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float v = (key0 + 8 * nt + e < t_end) ? s[nt][e] * sl2 : AD_NEG;
        s[nt][e] = v;
        mx = fmaxf(mx, v);
      }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float corr = exp2f(m_run - mx);
    m_run = mx;
    float p[2][2];
    float sum = 0.f;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        p[nt][e] = (key0 + 8 * nt + e < t_end) ? exp2f(s[nt][e] - mx) : 0.f;
        sum += p[nt][e];
      }
    l_run = l_run * corr + sum;
    const uint32_t pa0 = pack_f16(p[0][0], p[0][1]), pa2 = pack_f16(p[1][0], p[1][1]);
#pragma unroll
    for (int dp = 0; dp < DN / 2; ++dp) {
      const int r = 16 * warp + (lane & 7) + (((lane >> 3) & 1) << 3);
      const int c = 2 * dp + (lane >> 4);
      uint32_t b0, b1, b2, b3;
      ldsm_x4_t(v_tile(buf) + tile_off<D>(r, c), b0, b1, b2, b3);
      float c0[4] = {o[2 * dp][0] * corr, o[2 * dp][1] * corr, 0.f, 0.f};
      float c1[4] = {o[2 * dp + 1][0] * corr, o[2 * dp + 1][1] * corr, 0.f, 0.f};
      mma_f16_16816(c0, pa0, 0u, pa2, 0u, b0, b1);
      mma_f16_16816(c1, pa0, 0u, pa2, 0u, b2, b3);
      o[2 * dp][0] = c0[0]; o[2 * dp][1] = c0[1];
      o[2 * dp + 1][0] = c1[0]; o[2 * dp + 1][1] = c1[1];
    }
    __syncthreads();
  }
  cp_async_wait<0>();
  __syncthreads();  // the staging buffers are reused below

  // combine the four warps: (m, l) per head, then rescaled O
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  float* sm_m = reinterpret_cast<float*>(ad_smem);                 // [AD_WARPS][8]
  float* sm_l = sm_m + AD_WARPS * 8;                               // [AD_WARPS][8]
  float* sm_o = sm_l + AD_WARPS * 8;                               // [AD_WARPS][G][D]
  if (g < G) {
    if (tq == 0) {
      sm_m[warp * 8 + g] = m_run;
      sm_l[warp * 8 + g] = l_run;
    }
#pragma unroll
    for (int dn = 0; dn < DN; ++dn) {
      sm_o[(warp * G + g) * D + 8 * dn + 2 * tq] = o[dn][0];
      sm_o[(warp * G + g) * D + 8 * dn + 2 * tq + 1] = o[dn][1];
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < G * D; e += AD_WARPS * 32) {
    const int gq = e / D, dd = e % D;
    float mx = AD_NEG;
#pragma unroll
    for (int w = 0; w < AD_WARPS; ++w) mx = fmaxf(mx, sm_m[w * 8 + gq]);
    float l = 0.f, a = 0.f;
#pragma unroll
    for (int w = 0; w < AD_WARPS; ++w) {
      const float wgt = exp2f(sm_m[w * 8 + gq] - mx);
      l += wgt * sm_l[w * 8 + gq];
      a += wgt * sm_o[(w * G + gq) * D + dd];
    }
    const size_t slot = ((size_t)b * d.Hq + kvh * G + gq) * n_splits + split;
    part_acc[slot * D + dd] = a;
    if (dd == 0) {
      part_ml[slot * 2] = mx;  // log2 units
      part_ml[slot * 2 + 1] = l;
    }
  }
}

template <int D>
__global__ void attn_decode_merge_kernel(const float* __restrict__ part_acc, const float* __restrict__ part_ml,
                                         __half* __restrict__ out, int n_splits, int Hq) {
  const int bh = blockIdx.x;  // b * Hq + hq
  const int dd = threadIdx.x;
  pdl_trigger();
  pdl_wait();
  float mx = AD_NEG;
  for (int s = 0; s < n_splits; ++s) mx = fmaxf(mx, part_ml[((size_t)bh * n_splits + s) * 2]);
  float l = 0.f, a = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const size_t slot = (size_t)bh * n_splits + s;
    const float wgt = exp2f(part_ml[slot * 2] - mx);
    l += wgt * part_ml[slot * 2 + 1];
    a += wgt * part_acc[slot * D + dd];
  }
  out[(size_t)bh * D + dd] = __float2half_rn(fminf(fmaxf(a / l, -65504.f), 65504.f));
}

template <int D, int G>
static int launch_dg(const __half* qkv, const __half* kv_layer, __half* attn_out,
                     float* scratch, int n_splits, const BatchMeta& bm, const ModelDims& d, cudaStream_t st) {
  static bool configured = false;
  constexpr int smem = 4 * AD_TILE * D * 2;  // K[2] + V[2]; also covers the end-of-kernel combine buffers
  static_assert(smem >= (int)((2 * AD_WARPS * 8 + AD_WARPS * G * D) * sizeof(float)), "combine buffers must fit");
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(attn_decode_partial_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured = true;
  }
  float* part_acc = scratch;
  float* part_ml = scratch + (size_t)bm.n_seqs * d.Hq * n_splits * D;
  HYP_CUDA_TRY(launch_pdl(attn_decode_partial_kernel<D, G>, dim3(n_splits, d.Hkv, bm.n_seqs), dim3(AD_WARPS * 32), smem,
                          st, qkv, kv_layer, part_acc, part_ml, n_splits, bm, d));
  HYP_CUDA_TRY(launch_pdl(attn_decode_merge_kernel<D>, dim3(bm.n_seqs * d.Hq), dim3(D), 0, st, part_acc, part_ml,
                          attn_out, n_splits, d.Hq));
  return 2;
}

int launch_attn_decode(const __half* qkv, int q_stride, const __half* kv_layer, __half* attn_out,
                       float* scratch, int n_splits, const BatchMeta& bm, const ModelDims& d_in, cudaStream_t st) {
  ModelDims d = d_in;
  d.qkv_rows = q_stride;
  const int G = d.Hq / d.Hkv;
#define HYP_AD_CASE(DD, GG) \
  if (d.D == DD && G == GG) return launch_dg<DD, GG>(qkv, kv_layer, attn_out, scratch, n_splits, bm, d, st);
  HYP_AD_CASE(128, 1) HYP_AD_CASE(128, 2) HYP_AD_CASE(128, 4) HYP_AD_CASE(128, 8)
  HYP_AD_CASE(64, 1) HYP_AD_CASE(64, 2) HYP_AD_CASE(64, 4) HYP_AD_CASE(64, 8)
#undef HYP_AD_CASE
  return HYP_EINVAL;
}

}  // namespace hyp
