// Decode attention: one query row per sequence against its paged KV cache, split along the
// context so that a small batch still fills the GPU, followed by a log-sum-exp merge.
//
//   partial kernel: grid (n_splits, Hkv, n_seqs).  A CTA streams its context slice of one KV head
//   once with 128-bit loads and serves all G = Hq/Hkv query heads that share it.  Each group of
//   D/8 lanes owns one token per iteration; the dot product is finished with warp shuffles and a
//   running (max, sum, weighted V) state is kept in fp32 per lane group, then combined in shared
//   memory.
//   merge kernel: grid (n_seqs * Hq).  Combines the split partials and writes bf16.
//
// Scratch layout (fp32): acc [n_seqs][Hq][n_splits][D], then ml [n_seqs][Hq][n_splits][2].
#include "common.cuh"
#include "hyperion.h"

namespace hyp {

constexpr int AD_WARPS = 4;
constexpr int AD_UNROLL = 4;
constexpr float AD_NEG = -1e30f;

size_t attn_decode_scratch_bytes(int max_seqs, int Hq, int D, int max_splits) {
  return (size_t)max_seqs * Hq * max_splits * (D + 2) * sizeof(float);
}

int attn_decode_splits(int n_seqs, int Hkv, int max_ctx) {
  int want = (4 * 148 + n_seqs * Hkv - 1) / (n_seqs * Hkv);
  int cap = (max_ctx + 63) / 64;
  if (want > cap) want = cap;
  if (want > 32) want = 32;
  if (want < 1) want = 1;
  return want;
}

template <int D, int G>
__global__ void __launch_bounds__(AD_WARPS * 32)
attn_decode_partial_kernel(const __nv_bfloat16* __restrict__ qkv, const __nv_bfloat16* __restrict__ kv_layer,
                           float* __restrict__ part_acc, float* __restrict__ part_ml, int n_splits,
                           BatchMeta bm, ModelDims d) {
  constexpr int LPT = D / 8;          // lanes per token
  constexpr int TPW = 32 / LPT;       // tokens per warp iteration
  constexpr int GROUPS = AD_WARPS * TPW;
  constexpr int PT = 16;              // tokens per page
  __shared__ float sm_m[GROUPS][G], sm_l[GROUPS][G];
  __shared__ float sm_acc[GROUPS][G][D];

  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPT, dl = (lane % LPT) * 8;
  const int grp = warp * TPW + sub;

  const int ctx_total = bm.ctx_lens[b] + 1;  // the new token's k, v are already in the cache
  int tps = (ctx_total + n_splits - 1) / n_splits;
  tps = ((tps + PT - 1) / PT) * PT;
  const int t_begin = split * tps;
  const int t_end = min(ctx_total, t_begin + tps);

  // query heads kvh*G .. kvh*G+G-1 of row b, pre-scaled by 1/sqrt(D)
  const float scale = rsqrtf((float)D);
  float q[G][8];
  const __nv_bfloat16* qrow = qkv + (size_t)b * d.qkv_rows + (size_t)kvh * G * D;  // decode: row b is sequence b
#pragma unroll
  for (int gq = 0; gq < G; ++gq) {
    const uint4 v = *reinterpret_cast<const uint4*>(qrow + gq * D + dl);
    q[gq][0] = bf16_lo(v.x) * scale; q[gq][1] = bf16_hi(v.x) * scale;
    q[gq][2] = bf16_lo(v.y) * scale; q[gq][3] = bf16_hi(v.y) * scale;
    q[gq][4] = bf16_lo(v.z) * scale; q[gq][5] = bf16_hi(v.z) * scale;
    q[gq][6] = bf16_lo(v.w) * scale; q[gq][7] = bf16_hi(v.w) * scale;
  }

  float m_run[G], l_run[G], acc[G][8];
#pragma unroll
  for (int gq = 0; gq < G; ++gq) {
    m_run[gq] = AD_NEG;
    l_run[gq] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[gq][e] = 0.f;
  }

  const int32_t* bt = bm.block_table + (size_t)b * bm.max_pages_per_seq;
  const size_t page_elems = kv_page_elems(d.Hkv, PT, D);
  const size_t v_off = (size_t)d.Hkv * PT * D;

  for (int base = t_begin; base < t_end; base += GROUPS * AD_UNROLL) {
    uint4 kreg[AD_UNROLL], vreg[AD_UNROLL];
    bool ok[AD_UNROLL];
#pragma unroll
    for (int u = 0; u < AD_UNROLL; ++u) {
      const int tok = base + u * GROUPS + grp;
      ok[u] = tok < t_end;
      const int tk = ok[u] ? tok : t_begin;
      const int page = bt[tk / PT];
      const __nv_bfloat16* kp = kv_layer + (size_t)page * page_elems + ((size_t)kvh * PT + (tk % PT)) * D + dl;
      kreg[u] = ldg_stream(kp);
      vreg[u] = ldg_stream(kp + v_off);
    }
    float s[AD_UNROLL][G];
#pragma unroll
    for (int u = 0; u < AD_UNROLL; ++u) {
      const float k0 = bf16_lo(kreg[u].x), k1 = bf16_hi(kreg[u].x), k2 = bf16_lo(kreg[u].y), k3 = bf16_hi(kreg[u].y);
      const float k4 = bf16_lo(kreg[u].z), k5 = bf16_hi(kreg[u].z), k6 = bf16_lo(kreg[u].w), k7 = bf16_hi(kreg[u].w);
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
        float p = q[gq][0] * k0 + q[gq][1] * k1 + q[gq][2] * k2 + q[gq][3] * k3 + q[gq][4] * k4 + q[gq][5] * k5 +
                  q[gq][6] * k6 + q[gq][7] * k7;
#pragma unroll
        for (int o = LPT / 2; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
        s[u][gq] = ok[u] ? p : AD_NEG;
      }
    }
#pragma unroll
    for (int gq = 0; gq < G; ++gq) {
      float m_new = m_run[gq];
#pragma unroll
      for (int u = 0; u < AD_UNROLL; ++u) m_new = fmaxf(m_new, s[u][gq]);
      const float corr = __expf(m_run[gq] - m_new);
      m_run[gq] = m_new;
      l_run[gq] *= corr;
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[gq][e] *= corr;
#pragma unroll
      for (int u = 0; u < AD_UNROLL; ++u) {
        const float p = ok[u] ? __expf(s[u][gq] - m_new) : 0.f;
        l_run[gq] += p;
        acc[gq][0] += p * bf16_lo(vreg[u].x); acc[gq][1] += p * bf16_hi(vreg[u].x);
        acc[gq][2] += p * bf16_lo(vreg[u].y); acc[gq][3] += p * bf16_hi(vreg[u].y);
        acc[gq][4] += p * bf16_lo(vreg[u].z); acc[gq][5] += p * bf16_hi(vreg[u].z);
        acc[gq][6] += p * bf16_lo(vreg[u].w); acc[gq][7] += p * bf16_hi(vreg[u].w);
      }
    }
  }

  // combine the lane groups of the CTA
#pragma unroll
  for (int gq = 0; gq < G; ++gq) {
    if ((lane % LPT) == 0) {
      sm_m[grp][gq] = m_run[gq];
      sm_l[grp][gq] = l_run[gq];
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) sm_acc[grp][gq][dl + e] = acc[gq][e];
  }
  __syncthreads();
  for (int o = threadIdx.x; o < G * D; o += AD_WARPS * 32) {
    const int gq = o / D, dd = o % D;
    float mx = AD_NEG;
#pragma unroll
    for (int r = 0; r < GROUPS; ++r) mx = fmaxf(mx, sm_m[r][gq]);
    float l = 0.f, a = 0.f;
#pragma unroll
    for (int r = 0; r < GROUPS; ++r) {
      const float wgt = __expf(sm_m[r][gq] - mx);
      l += wgt * sm_l[r][gq];
      a += wgt * sm_acc[r][gq][dd];
    }
    const int hq = kvh * G + gq;
    const size_t slot = ((size_t)b * d.Hq + hq) * n_splits + split;
    part_acc[slot * D + dd] = a;
    if (dd == 0) {
      part_ml[slot * 2] = mx;
      part_ml[slot * 2 + 1] = l;
    }
  }
}

template <int D>
__global__ void attn_decode_merge_kernel(const float* __restrict__ part_acc, const float* __restrict__ part_ml,
                                         __nv_bfloat16* __restrict__ out, int n_splits, int Hq) {
  const int bh = blockIdx.x;  // b * Hq + hq
  const int dd = threadIdx.x;
  float mx = AD_NEG;
  for (int s = 0; s < n_splits; ++s) mx = fmaxf(mx, part_ml[((size_t)bh * n_splits + s) * 2]);
  float l = 0.f, a = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const size_t slot = (size_t)bh * n_splits + s;
    const float wgt = __expf(part_ml[slot * 2] - mx);
    l += wgt * part_ml[slot * 2 + 1];
    a += wgt * part_acc[slot * D + dd];
  }
  out[(size_t)bh * D + dd] = __float2bfloat16_rn(a / l);
}

template <int D, int G>
static int launch_dg(const __nv_bfloat16* qkv, const __nv_bfloat16* kv_layer, __nv_bfloat16* attn_out,
                     float* scratch, int n_splits, const BatchMeta& bm, const ModelDims& d, cudaStream_t st) {
  float* part_acc = scratch;
  float* part_ml = scratch + (size_t)bm.n_seqs * d.Hq * n_splits * D;
  attn_decode_partial_kernel<D, G><<<dim3(n_splits, d.Hkv, bm.n_seqs), AD_WARPS * 32, 0, st>>>(
      qkv, kv_layer, part_acc, part_ml, n_splits, bm, d);
  attn_decode_merge_kernel<D><<<bm.n_seqs * d.Hq, D, 0, st>>>(part_acc, part_ml, attn_out, n_splits, d.Hq);
  return 2;
}

int launch_attn_decode(const __nv_bfloat16* qkv, const __nv_bfloat16* kv_layer, __nv_bfloat16* attn_out,
                       float* scratch, int n_splits, const BatchMeta& bm, const ModelDims& d, cudaStream_t st) {
  const int G = d.Hq / d.Hkv;
#define HYP_AD_CASE(DD, GG) \
  if (d.D == DD && G == GG) return launch_dg<DD, GG>(qkv, kv_layer, attn_out, scratch, n_splits, bm, d, st);
  HYP_AD_CASE(128, 1) HYP_AD_CASE(128, 2) HYP_AD_CASE(128, 4) HYP_AD_CASE(128, 8)
  HYP_AD_CASE(64, 1) HYP_AD_CASE(64, 2) HYP_AD_CASE(64, 4) HYP_AD_CASE(64, 8)
#undef HYP_AD_CASE
  return HYP_EINVAL;
}

}  // namespace hyp
