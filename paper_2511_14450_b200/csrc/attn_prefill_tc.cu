// Prefill attention on the tcgen05 tensor cores (head_dim 128): causal, grouped-query, paged cache, fp32 softmax.
//
// One CTA = 128 query rows of one sequence and one query head; keys / values go by in tiles of 64 tokens (4 pages),
// two tiles in flight.
//   warp 0   lanes 0-15 issue TMA: the query tile once (two 64-wide k-blocks, 128-byte swizzle), then per tile one
//            2-D box per page and 64-wide half of head_dim for keys and for values (two stages each).  The cache
//            keeps a token's row chunk-permuted inside each 128-byte half, so a box of 16 rows x 128 bytes lands
//            as a ready 128-byte-swizzled operand tile (no swizzle in the copy).
//   warp 1   one lane issues tcgen05.mma: S_b = Q K^T (128 x 64 per tile, K-major operands) into one of two score
//            buffers in tensor memory, and, once the softmax warps have written the probabilities, O += P V (P
//            from tensor memory as the A operand, the value pages as MN-major B operands, two 64-column halves of
//            O).  The scores of tile j + 2 are issued right after the value product of tile j, so the tensor core
//            works on tile j + 1 while the softmax of tile j runs.
//   warps 2-5  softmax, one thread per query row (tensor-memory lane): read the 64 scores of the row (four loads,
//            one wait), scale, mask, exponentiate against a reference maximum, write P as packed fp16 over the
//            upper half of the score buffer's own columns, keep the running denominator.  The reference maximum is
//            only moved (and O rescaled in tensor memory, after the previous value product has drained) when the
//            row's maximum has grown by more than 2^8, so most tiles need no rescaling pass; fp16 holds P < 2^8
//            easily.  At the end they read O, divide by the denominator and store fp16.
// 96 KB of shared memory and 256 tensor-memory columns per CTA let two CTAs share an SM.
// Every barrier exists once per buffer (phase = tile / 2), so a waiter can never be lapped; every wait is bounded
// and failure unwinds through a shared flag.
#include <cuda.h>

#include "attn_common.cuh"
#include "gemm_tc.cuh"
#include "hyperion.h"
#include "tcgen05.cuh"

namespace hyp {

namespace {

constexpr int PT_Q = 128, PT_KV = 64, PT_D = 128, PT_PAGE = 16, PT_THREADS = 192;
constexpr int PT_TILE = 128 * 64 * 2;              // one [128][64] fp16 operand tile
constexpr int PT_STAGE = PT_KV * PT_D * 2;         // one tile of keys (or values): 4 pages x 2 halves x 2 KB
constexpr int PT_SMEM = 2 * PT_TILE + 4 * PT_STAGE + 1024;  // Q[2 k-blocks], K[2 stages], V[2 stages]
constexpr float PT_NEG = -1e30f;

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// MMA whose A operand is read from tensor memory (lane = row, two fp16 k-values per 32-bit column).
__device__ __forceinline__ void tc_mma_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// MN-major operand of 128 (MN) x 16 (K) fp16, 128-byte swizzle: the two 64-wide pieces of a page are 4 x 2 KB apart,
// 8-row groups along K are 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((4 * 2048) >> 4) << 16;  // leading byte offset: next 64 elements along MN
  d |= (uint64_t)(1024 >> 4) << 32;  // stride byte offset
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// fp16 x fp16 -> fp32, M = 128: N = 64 keys, K-major B (scores) / N = 128 dims, MN-major B (values)
constexpr uint32_t IDESC_S = (1u << 4) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 16) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);


__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Softmax of one 64-key tile for one query row (= tensor-memory lane): reads the row of the score buffer, moves
// the reference maximum when needed (rescaling O once the previous value product has drained: o_prev / o_parity
// name its barrier and phase), writes P as packed fp16 over columns 32-63 of the buffer and adds to the
// denominator.  The buffer holds raw scores; sl2 = log2(e) / sqrt(head_dim) is folded into the exponent.
template <bool MASKED>
__device__ __forceinline__ bool softmax_tile(uint32_t tmem_sb, uint32_t tmem_o, uint32_t lane_off, int key0, int pos, float sl2,
                                             int j, uint32_t o_prev, uint32_t o_parity, volatile int* abort_flag, float& m_ref,
                                             float& l) {
  uint32_t sv[PT_KV];
  float mx = PT_NEG;
#pragma unroll
  for (int c = 0; c < PT_KV; c += 16) tmem_ld16(tmem_sb + lane_off + c, reinterpret_cast<uint32_t(&)[16]>(sv[c]));
  tmem_ld_wait();
  {  // four independent chains: one or two warps per scheduler leave little else to hide the latency behind
    float m4[4] = {PT_NEG, PT_NEG, PT_NEG, PT_NEG};
#pragma unroll
    for (int i = 0; i < PT_KV; ++i) m4[i & 3] = fmaxf(m4[i & 3], !MASKED || key0 + i <= pos ? __uint_as_float(sv[i]) : PT_NEG);
    mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * sl2;  // sl2 > 0: the maximum of the scaled scores
  }
  // Move the reference maximum only when some row of the warp has outgrown it by 2^8 (the tensor-memory loads
  // and stores of the rescaling pass are warp-wide, so the decision is too); a row that has not grown keeps
  // its reference (corr = 1).
  if (__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
    const float new_ref = fmaxf(m_ref, mx);
    if (j > 0) {
      if (!mbar_wait(o_prev, o_parity, abort_flag)) return false;  // O must hold every earlier tile before it is scaled
      tc_fence_after();
      const float corr = ex2_approx(m_ref - new_ref);
      l *= corr;
#pragma unroll
      for (int c = 0; c < PT_D; c += 32) {
        uint32_t v[16], w[16];
        tmem_ld16(tmem_o + lane_off + c, v);
        tmem_ld16(tmem_o + lane_off + c + 16, w);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          v[i] = __float_as_uint(__uint_as_float(v[i]) * corr);
          w[i] = __float_as_uint(__uint_as_float(w[i]) * corr);
        }
        tmem_st16(tmem_o + lane_off + c, v);
        tmem_st16(tmem_o + lane_off + c + 16, w);
      }
    }
    m_ref = new_ref;
  }
  const float neg_ref = -m_ref;
  float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int c = 0; c < PT_KV; c += 32) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
      float p0 = ex2_approx(fmaf(__uint_as_float(sv[c + i]), sl2, neg_ref));
      float p1 = ex2_approx(fmaf(__uint_as_float(sv[c + i + 1]), sl2, neg_ref));
      if (MASKED) {
        p0 = key0 + c + i <= pos ? p0 : 0.f;
        p1 = key0 + c + i + 1 <= pos ? p1 : 0.f;
      }
      l4[(i >> 1) & 3] += p0 + p1;
      pk[i >> 1] = pack_f16(p0, p1);
    }
    tmem_st16(tmem_sb + lane_off + 32 + (c >> 1), pk);  // key k of the tile: 16-bit half k & 1 of column 32 + k / 2
  }
  l += (l4[0] + l4[1]) + (l4[2] + l4[3]);
  tmem_st_wait();
  return true;
}

}  // namespace

namespace {

__global__ void __launch_bounds__(PT_THREADS, 2)
attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kv,
                       __half* __restrict__ out, BatchMeta bm, ModelDims d, int* __restrict__ err) {
  extern __shared__ uint8_t pt_smem[];
  __shared__ uint64_t bars[16];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_word;
  const uint32_t base = (smem_u32(pt_smem) + 1023u) & ~1023u;
  const uint32_t sQ = base, sK = base + 2 * PT_TILE, sV = sK + 2 * PT_STAGE;
  // barriers: one per buffer b = tile & 1 (add 8 * b); phase of tile j = j / 2
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t q_full = bar0, k_full = bar0 + 16, v_full = bar0 + 32, s_full = bar0 + 80, p_full = bar0 + 96,
                 o_done = bar0 + 112;
  volatile int* abort_flag = &abort_word;
  pdl_trigger();
  pdl_wait();  // the queries and the cache rows come from the kernel launched just before

  // which (sequence, query tile) is this CTA?  The last tiles of a sequence see the most keys: they go first.
  int t = (int)gridDim.y - 1 - (int)blockIdx.y, seq = -1, q0 = 0, q_len = 0;
  for (int i = 0; i < bm.n_seqs; ++i) {
    const int ql = bm.cu_q[i + 1] - bm.cu_q[i];
    const int nt = (ql + PT_Q - 1) / PT_Q;
    if (t < nt) { seq = i; q0 = t * PT_Q; q_len = ql; break; }
    t -= nt;
  }
  if (seq < 0) return;
  const int hq = blockIdx.x;  // heads vary fastest: every head's heaviest tile is scheduled before any lighter one
  const int kvh = hq / (d.Hq / d.Hkv);
  const int ctx = bm.ctx_lens[seq];
  const int row_base = bm.cu_q[seq] + q0;
  const int rows_here = min(PT_Q, q_len - q0);
  const int kv_total = ctx + q0 + rows_here;  // keys this tile may need: positions < kv_total
  const int n_tiles = (kv_total + PT_KV - 1) / PT_KV;
  const int n_pages_seq = (kv_total + PT_PAGE - 1) / PT_PAGE;
  const int32_t* bt = bm.block_table + (size_t)seq * bm.max_pages_per_seq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 16; ++i) mbar_init(bar0 + 8u * i, (i == 12 || i == 13) ? 128u : 1u);  // p_full: every softmax thread
    abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(256));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // columns 0-63 / 64-127: the two score buffers (P over the upper half of each); 128-255: O
  const uint32_t tmem_s = tmem_slot, tmem_o = tmem_slot + 128u;

  if (warp == 0) {
    // ---------------- TMA producer: one box per lane and tile, the sixteen boxes of a tile side by side ----------
    // lanes 0-7 bring the keys, 8-15 the values; within each, lane = page (0-3) x half of head_dim
    if (lane == 0) {
      mbar_expect_tx(q_full, 2 * PT_TILE);
      tma_load_2d(sQ, &tm_q, hq * PT_D, row_base, q_full);
      tma_load_2d(sQ + PT_TILE, &tm_q, hq * PT_D + 64, row_base, q_full);
    }
    if (lane < 16) {
      const int is_v = lane >> 3, p = (lane >> 1) & 3, h = lane & 1;
      const uint32_t full = is_v ? v_full : k_full;
      const uint32_t empty = is_v ? o_done : s_full;  // a stage is free once the product that read it has drained
      // keys: k-block h = [64 tokens][64 dims], pages stacked; values: one 2 KB piece per (half, page)
      const uint32_t dst = is_v ? sV + (h * 4 + p) * 2048 : sK + h * (PT_STAGE / 2) + p * 2048;
      // Key lanes and value lanes advance independently (their stages drain at different times), so no lane may
      // block in a wait the others have to reconverge with: every lane polls its own barrier once per turn.
      bool ok = true;
      int j = 0;
      uint32_t idle = 0;
      uint64_t t_idle = 0;
      while (j < n_tiles) {
        const uint32_t b = (uint32_t)(j & 1);
        if (j < 2 || mbar_try(empty + 8 * b, (uint32_t)(((j >> 1) - 1) & 1))) {
          // rows of the pool seen as [page][K, V][kv head][16 tokens] x head_dim
          const int pi = min(4 * j + p, n_pages_seq - 1);  // past the last page: any valid page (its keys are masked)
          const int row0 = ((bt[pi] * 2 + is_v) * d.Hkv + kvh) * PT_PAGE;
          if ((lane & 7) == 0) mbar_expect_tx(full + 8 * b, PT_STAGE);  // a copy may land first: the count goes negative meanwhile
          tma_load_2d(dst + b * PT_STAGE, &tm_kv, h * 64, row0, full + 8 * b);
          ++j;
          idle = 0;
        } else if ((++idle & 1023u) == 0) {
          const uint64_t now = globaltimer();
          if (idle == 1024u) t_idle = now;
          if (*abort_flag || now - t_idle > WAIT_LIMIT_NS) { ok = false; break; }
        }
      }
      if (!ok && (lane & 7) == 0) {
        *abort_flag = 1;
        atomicCAS(err, 0, 13);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      bool ok = mbar_wait(q_full, 0, abort_flag);
      // operand descriptors differ from tile to tile by a constant in the address field only
      const uint64_t dq = smem_desc(sQ), dk = smem_desc(sK), dv = smem_desc_mn(sV);
      // S_b = Q K^T of tile j: two 64-wide k-blocks of head_dim, four 16-wide steps each
      auto scores = [&](int j) -> bool {
        const uint32_t b = (uint32_t)(j & 1);
        if (!mbar_wait(k_full + 8 * b, (uint32_t)((j >> 1) & 1), abort_flag)) return false;
        tc_fence_after();
        const uint64_t dkb = dk + (uint64_t)(b * (PT_STAGE >> 4));
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma(tmem_s + 64u * b, dq + (uint64_t)(kb * (PT_TILE >> 4) + ks * 2),
                   dkb + (uint64_t)(kb * (PT_STAGE >> 5) + ks * 2), IDESC_S, (kb | ks) ? 1u : 0u);
        tc_commit(s_full + 8 * b);  // also frees the key stage
        return true;
      };
      ok = ok && scores(0);
      if (ok && n_tiles > 1) ok = scores(1);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const uint32_t b = (uint32_t)(j & 1), ph = (uint32_t)((j >> 1) & 1);
        if (!mbar_wait(p_full + 8 * b, ph, abort_flag) || !mbar_wait(v_full + 8 * b, ph, abort_flag)) { ok = false; break; }
        tc_fence_after();
        // O += P V: 4 pages of 16 keys; P sits in tensor memory (8 columns per page); a value page is an MN-major
        // operand of two 64-wide pieces
        const uint64_t dvb = dv + (uint64_t)(b * (PT_STAGE >> 4));
#pragma unroll
        for (int p = 0; p < 4; ++p)
          tc_mma_ta(tmem_o, tmem_s + 64u * b + 32u + (uint32_t)(8 * p), dvb + (uint64_t)(p * (2048 >> 4)), IDESC_PV,
                    (j > 0 || p > 0) ? 1u : 0u);
        tc_commit(o_done + 8 * b);  // also frees the value stage
        // the scores of tile j + 2 reuse this tile's buffer: issued behind its value product
        if (j + 2 < n_tiles) ok = scores(j + 2);
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(err, 0, 14);
      }
    }
  } else {
    // ---------------- softmax / epilogue: thread = query row = tensor-memory lane ----------------
    const int q = warp & 3;
    const int r = 32 * q + lane;
    const uint32_t lane_off = (uint32_t)(32 * q) << 16;
    const int pos = ctx + q0 + min(r, rows_here - 1);  // rows past the end are clamped: computed, never stored
    const float sl2 = rsqrtf((float)PT_D) * 1.4426950408889634f;
    float m_ref = PT_NEG, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const uint32_t b = (uint32_t)(j & 1);
      if (!mbar_wait(s_full + 8 * b, (uint32_t)((j >> 1) & 1), abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int key0 = j * PT_KV;
      // the value product of tile j - 1: buffer (j - 1) & 1, phase (j - 1) / 2
      const uint32_t o_prev = o_done + 8 * (b ^ 1), o_parity = (uint32_t)(((j - 1) >> 1) & 1);
      // only the tiles that reach past some row's own position need the causal mask
      if (__any_sync(0xffffffffu, key0 + PT_KV - 1 > pos))
        ok = softmax_tile<true>(tmem_s + 64u * b, tmem_o, lane_off, key0, pos, sl2, j, o_prev, o_parity, abort_flag, m_ref, l);
      else
        ok = softmax_tile<false>(tmem_s + 64u * b, tmem_o, lane_off, key0, pos, sl2, j, o_prev, o_parity, abort_flag, m_ref, l);
      if (!ok) break;
      tc_fence_before();
      mbar_arrive(p_full + 8 * b);
    }
    // the last value product (a commit follows every earlier one too)
    if (ok && !mbar_wait(o_done + 8 * ((n_tiles - 1) & 1), (uint32_t)(((n_tiles - 1) >> 1) & 1), abort_flag)) ok = false;
    tc_fence_after();
    if (ok) {
      const float inv = 1.f / l;
      __half* orow = out + (size_t)(row_base + min(r, rows_here - 1)) * d.Hq * PT_D + (size_t)hq * PT_D;
#pragma unroll
      for (int c = 0; c < PT_D; c += 32) {  // warp-wide loads; only rows of this tile store
        uint32_t v[16], w[16];
        tmem_ld16(tmem_o + lane_off + c, v);
        tmem_ld16(tmem_o + lane_off + c + 16, w);
        tmem_ld_wait();
        if (r < rows_here) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            pk[i] = pack_f16_sat(__uint_as_float(v[2 * i]) * inv, __uint_as_float(v[2 * i + 1]) * inv);
            pk[8 + i] = pack_f16_sat(__uint_as_float(w[2 * i]) * inv, __uint_as_float(w[2 * i + 1]) * inv);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
            reinterpret_cast<uint4*>(orow + c)[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
        }
      }
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(err, 0, 15);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"(256));
  }
}

}  // namespace


int& attn_prefill_tc_enabled() {
  static int v = 1;
  return v;
}

// q_map: the rotated queries [rows, Hq * 128] fp16 with 128-row x 64-column boxes (128-byte swizzle);
// kv_map: the block's page pool seen as rows of head_dim fp16 (tc_make_kv_map).
int launch_attn_prefill_tc(const CUtensorMap& q_map, const CUtensorMap& kv_map, __half* attn_out, const BatchMeta& bm,
                           const ModelDims& d, cudaStream_t st) {
  static bool configured = false;
  if (d.D != PT_D || d.Hkv < 1 || d.Hq % d.Hkv) return HYP_EINVAL;
  int rc = tc_prepare();
  if (rc) return rc;
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(attn_prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PT_SMEM));
    configured = true;
  }
  const int max_tiles = bm.n_tokens / PT_Q + bm.n_seqs;  // every sequence adds at most one ragged tile
  HYP_CUDA_TRY(launch_pdl<2>(attn_prefill_tc_kernel, dim3(d.Hq, max_tiles), dim3(PT_THREADS), (size_t)PT_SMEM, st, q_map, kv_map,
                          attn_out, bm, d, tc_err_flag_ptr()));
  return 1;
}

}  // namespace hyp
