// Prefill attention over the paged KV cache: causal, grouped-query, fp32 online softmax.
//
// Flash-attention tiling on tensor cores: one CTA = 64 query rows of one sequence and one query head
// (4 warps x 16 rows); keys/values stream through shared memory in 64-token tiles (4 pages), double-buffered,
// one bulk copy per page and operand (the cache keeps a page's rows in the tile's chunk-permuted order); S = Q K^T and O += P V run on mma.sync.m16n8k16 (fp16 in, fp32 accumulate: q, k,
// v and the softmax weights carry 11 mantissa bits - bf16's 8 bits alone cost ~0.5 % error in the softmax
// weights), the probabilities never leave registers.  New rows of a sequence sit at positions
// ctx_len .. ctx_len + q_len - 1 and see every cached position up to their own (their k, v were
// appended by the RoPE / KV-write kernel beforehand), so chunked prefill needs no special case.
#include "attn_common.cuh"
#include "hyperion.h"
#include "gemm_tc.cuh"
#include "sm100_common.cuh"

namespace hyp {

namespace {

constexpr int FA_BQ = 64, FA_BKV = 64, FA_THREADS = 128, PT = 16;

// SPLIT: the scores are formed from two-term operands, q = q_hi + q_lo and k = k_hi + k_lo (each term fp16, the low
// term the rounding residue of the high one), as q_hi k_hi + q_lo k_hi + q_hi k_lo: ~21 significant bits instead of
// 11.  `q_lo` has the layout of `qkv`; `klo_layer` is a pool [page][Hkv][16][D] with the cache's row order.  Used for
// the model's first block, whose attention errors the rest of the network amplifies most (see stage.cu).
template <int D, bool SPLIT>
__global__ void __launch_bounds__(FA_THREADS, SPLIT ? 2 : 3)
attn_prefill_fa_kernel(const __half* __restrict__ qkv, const __half* __restrict__ kv_layer,
                       const __half* __restrict__ q_lo_buf, const __half* __restrict__ klo_layer,
                       __half* __restrict__ out, BatchMeta bm, ModelDims d, int* __restrict__ err) {
  constexpr int KS = D / 16;       // k-steps of the QK^T contraction
  constexpr int DN = D / 8;        // 8-wide output column tiles of O
  constexpr int CPR = D / 8;       // 16-byte chunks per K/V row
  constexpr int TILE_BYTES = FA_BKV * D * 2;
  extern __shared__ __align__(128) uint8_t fa_smem[];
  const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(fa_smem);
  // layout: K[2] then V[2] (then the low terms of K[2])
  auto k_tile = [&](int buf) { return smem0 + buf * TILE_BYTES; };
  auto v_tile = [&](int buf) { return smem0 + (2 + buf) * TILE_BYTES; };
  auto klo_tile = [&](int buf) { return smem0 + (4 + buf) * TILE_BYTES; };

  __shared__ uint64_t kv_bars[2];
  constexpr int PAGE_BYTES = PT * D * 2;  // the 16 keys (or values) of one page and KV head: contiguous in the cache
  pdl_trigger();
  pdl_wait();
  // which (sequence, query tile) is this CTA?  The last tiles of a sequence see the most keys: they go first.
  int t = (int)gridDim.y - 1 - (int)blockIdx.y, seq = -1, q0 = 0, q_len = 0;
  for (int i = 0; i < bm.n_seqs; ++i) {
    const int ql = bm.cu_q[i + 1] - bm.cu_q[i];
    const int nt = (ql + FA_BQ - 1) / FA_BQ;
    if (t < nt) { seq = i; q0 = t * FA_BQ; q_len = ql; break; }
    t -= nt;
  }
  if (seq < 0) return;
  const int hq = blockIdx.x;  // heads vary fastest: every head's heaviest tile is scheduled before any lighter one
  const int kvh = hq / (d.Hq / d.Hkv);
  const int ctx = bm.ctx_lens[seq];
  const int row_base = bm.cu_q[seq] + q0;               // first packed row of this tile
  const int rows_here = min(FA_BQ, q_len - q0);
  const int kv_total = ctx + q0 + rows_here;             // keys this tile may need: positions < kv_total
  const int n_kv_tiles = (kv_total + FA_BKV - 1) / FA_BKV;
  const int32_t* bt = bm.block_table + (size_t)seq * bm.max_pages_per_seq;
  const size_t page_elems = kv_page_elems(d.Hkv, PT, D);
  const size_t v_off = (size_t)d.Hkv * PT * D;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;

  // One tile = 4 pages.  The cache stores a page's rows with the tile's own chunk permutation, so thread 0 brings a
  // tile in with one bulk copy per page for the keys and one for the values; pages past the sequence's last one
  // are not copied but cleared (their probabilities are zero, and 0 x stale bits must not become NaN).
  const int n_pages_seq = (kv_total + PT - 1) / PT;
  const uint32_t bar0 = smem_u32(kv_bars);
  if (threadIdx.x == 0) {
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  auto load_kv_tile = [&](int j, int buf) {
    const int p0 = j * (FA_BKV / PT);
    const int n_valid = min(FA_BKV / PT, n_pages_seq - p0);
    if (threadIdx.x == 0) {
      mbar_expect_tx(bar0 + 8u * buf, (uint32_t)((SPLIT ? 3 : 2) * n_valid * PAGE_BYTES));
      for (int pi = 0; pi < n_valid; ++pi) {
        const __half* src = kv_layer + (size_t)bt[p0 + pi] * page_elems + (size_t)kvh * PT * D;
        bulk_load(k_tile(buf) + pi * PAGE_BYTES, src, PAGE_BYTES, bar0 + 8u * buf);
        bulk_load(v_tile(buf) + pi * PAGE_BYTES, src + v_off, PAGE_BYTES, bar0 + 8u * buf);
        if (SPLIT)
          bulk_load(klo_tile(buf) + pi * PAGE_BYTES, klo_layer + ((size_t)bt[p0 + pi] * d.Hkv + kvh) * PT * D, PAGE_BYTES,
                    bar0 + 8u * buf);
      }
    }
    if (n_valid < FA_BKV / PT) {
      const int bytes = (FA_BKV / PT - n_valid) * PAGE_BYTES;
      for (int o = threadIdx.x * 16; o < bytes; o += FA_THREADS * 16) {
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(k_tile(buf) + n_valid * PAGE_BYTES + o), "r"(0u) : "memory");
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(v_tile(buf) + n_valid * PAGE_BYTES + o), "r"(0u) : "memory");
        if (SPLIT)
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(klo_tile(buf) + n_valid * PAGE_BYTES + o), "r"(0u) : "memory");
      }
    }
  };

  load_kv_tile(0, 0);

  // Q fragments of this warp's 16 rows, straight from global memory
  uint32_t qf[KS][4];
  {
    const int r_lo = 16 * warp + g, r_hi = r_lo + 8;
    const __half* q_lo = qkv + (size_t)(row_base + r_lo) * d.qkv_rows + (size_t)hq * D;
    const __half* q_hi = qkv + (size_t)(row_base + r_hi) * d.qkv_rows + (size_t)hq * D;
    const bool ok_lo = r_lo < rows_here, ok_hi = r_hi < rows_here;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qf[ks][0] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + 16 * ks + 2 * tq) : 0u;
      qf[ks][1] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + 16 * ks + 2 * tq) : 0u;
      qf[ks][2] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + 16 * ks + 8 + 2 * tq) : 0u;
      qf[ks][3] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + 16 * ks + 8 + 2 * tq) : 0u;
    }
  }
  uint32_t qfl[SPLIT ? KS : 1][4];  // low terms of the same fragments
  if (SPLIT) {
    const int r_lo = 16 * warp + g, r_hi = r_lo + 8;
    const __half* q_lo = q_lo_buf + (size_t)(row_base + r_lo) * d.qkv_rows + (size_t)hq * D;
    const __half* q_hi = q_lo_buf + (size_t)(row_base + r_hi) * d.qkv_rows + (size_t)hq * D;
    const bool ok_lo = r_lo < rows_here, ok_hi = r_hi < rows_here;
#pragma unroll
    for (int ks = 0; ks < (SPLIT ? KS : 1); ++ks) {
      qfl[ks][0] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + 16 * ks + 2 * tq) : 0u;
      qfl[ks][1] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + 16 * ks + 2 * tq) : 0u;
      qfl[ks][2] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + 16 * ks + 8 + 2 * tq) : 0u;
      qfl[ks][3] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + 16 * ks + 8 + 2 * tq) : 0u;
    }
  }

  const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;  // scores are kept in log2 units
  // absolute positions of this thread's two rows (rows past the end are clamped: computed, never stored)
  const int pos_lo = ctx + q0 + min(16 * warp + g, rows_here - 1);
  const int pos_hi = ctx + q0 + min(16 * warp + g + 8, rows_here - 1);

  float o[DN][4];
#pragma unroll
  for (int i = 0; i < DN; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -1e30f, m_hi = -1e30f, l_lo = 0.f, l_hi = 0.f;

  bool ok = true;
  for (int j = 0; j < n_kv_tiles; ++j) {
    const int buf = j & 1;
    if (j + 1 < n_kv_tiles) load_kv_tile(j + 1, buf ^ 1);
    const bool landed = mbar_wait(bar0 + 8u * buf, (uint32_t)((j >> 1) & 1), nullptr);
    // one decision for the whole CTA (a bounded wait could expire for some threads only); as a barrier it also
    // makes the cleared pages of a last tile visible
    if (!__syncthreads_and(landed)) { ok = false; break; }

    // ---- S = Q K^T (16 rows x 64 keys per warp) ----
    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {  // pairs of 8-key tiles
        const int r = 16 * np + (lane & 7) + ((lane >> 4) << 3);
        const int c = 2 * ks + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4(k_tile(buf) + tile_off<D>(r, c), b0, b1, b2, b3);
        mma_f16_16816(s[2 * np], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b0, b1);
        mma_f16_16816(s[2 * np + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b2, b3);
        if (SPLIT) {
          const int kq = SPLIT ? ks : 0;
          mma_f16_16816(s[2 * np], qfl[kq][0], qfl[kq][1], qfl[kq][2], qfl[kq][3], b0, b1);
          mma_f16_16816(s[2 * np + 1], qfl[kq][0], qfl[kq][1], qfl[kq][2], qfl[kq][3], b2, b3);
          ldsm_x4(klo_tile(buf) + tile_off<D>(r, c), b0, b1, b2, b3);
          mma_f16_16816(s[2 * np], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b0, b1);
          mma_f16_16816(s[2 * np + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b2, b3);
        }
      }
    }

    // ---- scale, causal mask, online softmax ----
    const int key0 = j * FA_BKV;
    const bool need_mask = key0 + FA_BKV - 1 > ctx + q0;  // some key of the tile may lie past a row's position
    float mx_lo = m_lo, mx_hi = m_hi;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[nt][e] * sl2;
        if (need_mask) {
          const int key = key0 + 8 * nt + 2 * tq + (e & 1);
          if (key > ((e < 2) ? pos_lo : pos_hi)) v = -1e30f;
        }
        s[nt][e] = v;
      }
      mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float corr_lo = exp2f(m_lo - mx_lo), corr_hi = exp2f(m_hi - mx_hi);
    m_lo = mx_lo;
    m_hi = mx_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
    uint32_t pf[8][2];  // probabilities as fp16 pairs: [key tile][row lo / hi]
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p0 = exp2f(s[nt][0] - mx_lo), p1 = exp2f(s[nt][1] - mx_lo);
      const float p2 = exp2f(s[nt][2] - mx_hi), p3 = exp2f(s[nt][3] - mx_hi);
      sum_lo += p0 + p1;
      sum_hi += p2 + p3;
      pf[nt][0] = pack_f16(p0, p1);
      pf[nt][1] = pack_f16(p2, p3);
    }
    l_lo = l_lo * corr_lo + sum_lo;
    l_hi = l_hi * corr_hi + sum_hi;
#pragma unroll
    for (int dn = 0; dn < DN; ++dn) {
      o[dn][0] *= corr_lo; o[dn][1] *= corr_lo;
      o[dn][2] *= corr_hi; o[dn][3] *= corr_hi;
    }

    // ---- O += P V ----
#pragma unroll
    for (int kk = 0; kk < FA_BKV / 16; ++kk) {
#pragma unroll
      for (int dp = 0; dp < DN / 2; ++dp) {  // pairs of 8-wide output column tiles
        const int r = 16 * kk + (lane & 7) + (((lane >> 3) & 1) << 3);
        const int c = 2 * dp + (lane >> 4);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(v_tile(buf) + tile_off<D>(r, c), b0, b1, b2, b3);
        mma_f16_16816(o[2 * dp], pf[2 * kk][0], pf[2 * kk][1], pf[2 * kk + 1][0], pf[2 * kk + 1][1], b0, b1);
        mma_f16_16816(o[2 * dp + 1], pf[2 * kk][0], pf[2 * kk][1], pf[2 * kk + 1][0], pf[2 * kk + 1][1], b2, b3);
      }
    }
    __syncthreads();  // everyone is done with `buf` before the next iteration's loads overwrite it
  }
  if (!ok) {
    // a copy never landed (bounded wait expired): record it; the rows of this tile are not written
    if (threadIdx.x == 0) atomicCAS(err, 0, 12);
    return;
  }

  // row sums live spread over the 4 lanes of a quad
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
  const int r_lo = 16 * warp + g, r_hi = r_lo + 8;
  __half* o_lo = out + (size_t)(row_base + r_lo) * d.Hq * D + (size_t)hq * D;
  __half* o_hi = out + (size_t)(row_base + r_hi) * d.Hq * D + (size_t)hq * D;
#pragma unroll
  for (int dn = 0; dn < DN; ++dn) {
    if (r_lo < rows_here)
      *reinterpret_cast<uint32_t*>(o_lo + 8 * dn + 2 * tq) = pack_f16_sat(o[dn][0] * inv_lo, o[dn][1] * inv_lo);
    if (r_hi < rows_here)
      *reinterpret_cast<uint32_t*>(o_hi + 8 * dn + 2 * tq) = pack_f16_sat(o[dn][2] * inv_hi, o[dn][3] * inv_hi);
  }
}

template <int D, bool SPLIT>
int launch_fa(const __half* qkv, const __half* kv_layer, const __half* q_lo, const __half* klo_layer, __half* attn_out,
              const BatchMeta& bm, const ModelDims& d, cudaStream_t st) {
  static bool configured = false;
  constexpr int smem = (SPLIT ? 6 : 4) * FA_BKV * D * 2;
  int rc = tc_prepare();  // the device word that bounded waits report to
  if (rc) return rc;
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(attn_prefill_fa_kernel<D, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured = true;
  }
  // every sequence adds at most one ragged tile on top of floor(rows / 64)
  const int max_tiles = bm.n_tokens / FA_BQ + bm.n_seqs;
  HYP_CUDA_TRY(launch_pdl<2>(attn_prefill_fa_kernel<D, SPLIT>, dim3(d.Hq, max_tiles), dim3(FA_THREADS), smem, st, qkv,
                             kv_layer, q_lo, klo_layer, attn_out, bm, d, tc_err_flag_ptr()));
  return 1;
}

}  // namespace

// Needs bm.cu_q, bm.ctx_lens, bm.block_table, bm.n_seqs, bm.n_tokens.  Head h of row t: q + t*q_stride + h*D.
int launch_attn_prefill(const __half* q, int q_stride, const __half* kv_layer, __half* attn_out,
                        const BatchMeta& bm, const ModelDims& d_in, cudaStream_t st) {
  ModelDims d = d_in;
  d.qkv_rows = q_stride;
  if (d.D == 128) return launch_fa<128, false>(q, kv_layer, nullptr, nullptr, attn_out, bm, d, st);
  if (d.D == 64) return launch_fa<64, false>(q, kv_layer, nullptr, nullptr, attn_out, bm, d, st);
  return HYP_EINVAL;
}

// The same attention with two-term queries and keys (q_lo: layout of q; klo_layer: [page][Hkv][16][D]).
int launch_attn_prefill_split(const __half* q, const __half* q_lo, int q_stride, const __half* kv_layer,
                              const __half* klo_layer, __half* attn_out, const BatchMeta& bm, const ModelDims& d_in,
                              cudaStream_t st) {
  ModelDims d = d_in;
  d.qkv_rows = q_stride;
  if (!q_lo || !klo_layer) return HYP_EINVAL;
  if (d.D == 128) return launch_fa<128, true>(q, kv_layer, q_lo, klo_layer, attn_out, bm, d, st);
  if (d.D == 64) return launch_fa<64, true>(q, kv_layer, q_lo, klo_layer, attn_out, bm, d, st);
  return HYP_EINVAL;
}

}  // namespace hyp
