// Decode attention of the stage path, fused with what precedes and follows it (one launch per block):
// rotary encoding of the new token's query and key, append of its key / value to the paged cache,
// split-context attention, and the merge of the splits.
//
//   grid (n_splits, Hkv, n_seqs), 4 warps.  Page p of a sequence belongs to split p % n_splits; warp w takes every
//   fourth page of its split and streams them through its own ring: one bulk copy brings the 16 keys of a page for this KV head (contiguous in the
//   cache, already chunk-permuted for ldmatrix), another the 16 values; the warp waits on the slot's mbarrier,
//   forms the scores of its 16 keys for the G = Hq/Hkv query heads (rows of one mma.sync.m16n8k16 operand, rows
//   >= G are padding), keeps its own online-softmax state and O += P V partial, and lane 0 refills the slot.
//   No CTA-wide synchronisation inside the loop; a slot has one waiter.
//   Prologue: the page copies are issued first (older cache entries do not depend on the predecessor); then the
//   CTA rotates its G query heads from the projection's fp32 output into shared memory, and the CTA whose run
//   ends with the new token rotates that token's key, rounds key and value to fp16, writes them to the page
//   (for the following steps) and, once that page has landed in its ring, over the stale row in shared memory.
//   Epilogue: the four warps are combined in shared memory; then the splits are merged, in one of two ways.
//   Cluster variant (the op-level entry point: no scratch memory, no atomics): the n_splits CTAs form a thread-block
//   cluster; after a cluster barrier every CTA merges a slice of the G x D outputs over all splits, reading the
//   other CTAs' partials through distributed shared memory.  Global variant (the stage path): every CTA writes its
//   partial to a scratch row and takes a ticket; the CTA with the last ticket merges.  A cluster's CTAs must be
//   co-scheduled, which made an early (programmatic) launch of the cluster variant slower than a plain one; the
//   global variant is launched early, so its CTAs move in as the q/k/v projection's CTAs leave and have their first
//   pages on the way before the projection has finished (14-block decode step, batch 8: 1784 -> 1768 us).
//   Every mbarrier wait is bounded; the cluster barriers are reached by every CTA; nothing waits for another CTA.
#include "attn_common.cuh"
#include "hyperion.h"
#include "sm100_common.cuh"

namespace hyp {

namespace {

constexpr int AF_WARPS = 4;
constexpr int AF_THREADS = 32 * AF_WARPS;
constexpr int AF_MAX_SLOTS = 4;
constexpr int AF_PT = 16;  // tokens per page
constexpr float AF_NEG = -1e30f;

struct AttnFusedArgs {
  const float* qkv32;        // [n_seqs, stride] fp32: Q heads | K heads | V heads of the new token, not rotated
  int stride;
  __half* kv_layer;          // the block's page pool, written (new token) and read
  const float2* rope_table;  // [max_ctx, D/2] (cos, sin)
  __half* out;               // [n_seqs, Hq * D]
  int slots;                 // ring slots per warp
  int* err;
  // SPLIT instantiation only (the model's first block): the rows of qkv32 still lack the RMSNorm factor
  // row_scale[b], and queries / keys are two-term fp16 values, the keys' low terms cached in klo_layer
  // ([page][Hkv][16][D], the cache's row order), so that the scores carry ~21 significant bits
  const float* row_scale;
  __half* klo_layer;
  // GLOBAL instantiation only: the splits meet in global memory instead of a cluster's shared memory
  float* scratch;            // [n_seqs * Hkv][n_splits][G * D + 16] partial outputs, then maxima and denominators
  int* tickets;              // [n_seqs * Hkv], zero between launches
};

__device__ __forceinline__ __half f16_sat(float x) { return __float2half_rn(fminf(fmaxf(x, -65504.f), 65504.f)); }
// GLOBAL: no cluster.  Every CTA writes its partial (G x D sums, G maxima, G denominators) to a scratch row, fences,
// and takes a ticket on the (sequence, KV head)'s counter; the CTA that takes the last ticket reads the n_splits
// rows back (L2) and merges them.  Nothing waits for another CTA, and without the co-scheduling that a cluster
// needs the grid can be launched early (programmatic dependent launch): its CTAs take the SMs' slots as the
// projection's CTAs leave them and have their first pages on the way before the projection has finished.
template <int D, int G, bool SPLIT, bool GLOBAL>
__global__ void __launch_bounds__(AF_THREADS)
attn_decode_fused_kernel(AttnFusedArgs a, BatchMeta bm, ModelDims d) {
  constexpr int KS = D / 16, DN = D / 8, CPR = D / 8;
  constexpr int PAGE_BYTES = AF_PT * D * 2;   // 16 keys (or values) of one KV head
  constexpr int SLOT_BYTES = (SPLIT ? 3 : 2) * PAGE_BYTES;  // keys, then values (then the keys' low terms)
  extern __shared__ __align__(128) uint8_t af_smem[];
  __shared__ uint64_t bars[AF_WARPS * AF_MAX_SLOTS];
  __shared__ float ex_m[8], ex_l[8];              // this CTA's partial: running maximum (log2 units), denominator
  __shared__ __align__(16) float ex_o[G * D];     // and weighted value sum, read by the whole cluster
  __shared__ __align__(16) __half sq[G * D];      // rotated queries
  __shared__ __align__(16) __half snew[3 * D];    // the new token's rotated key, then its value (then the key's low term)
  __shared__ __align__(16) __half sq_lo[SPLIT ? G * D : 8];  // low terms of the rotated queries
  const int S = a.slots;
  const uint32_t ring0 = (smem_u32(af_smem) + 127u) & ~127u;
  uint8_t* ring_ptr = af_smem + (ring0 - smem_u32(af_smem));

  const int n_splits = gridDim.x;
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;

  // Which pages are mine does not depend on the sequence's length: page p belongs to split p % n_splits, and inside
  // the CTA the pages of a split go round-robin over the warps, so this warp's i-th page is
  // split + n_splits * (warp + AF_WARPS * i).  The block-table entries (one per lane, two rounds) are therefore
  // fetched together with the length instead of behind it; only "how many of them exist" waits for the length.
  // Metadata and cache pages written by earlier steps do not depend on the predecessor kernel.
  const int32_t* bt = bm.block_table + (size_t)b * bm.max_pages_per_seq;
  auto page_index = [&](int i) { return split + n_splits * (warp + AF_WARPS * i); };
  const int pi_lo = page_index(lane), pi_hi = page_index(lane + 32);
  const int32_t bt_lo = pi_lo < bm.max_pages_per_seq ? bt[pi_lo] : 0;
  const int32_t bt_hi = pi_hi < bm.max_pages_per_seq ? bt[pi_hi] : 0;
  const int pos = bm.ctx_lens[b];  // the new token's position
  const int ctx_total = pos + 1;
  const int n_pages = (ctx_total + AF_PT - 1) / AF_PT;
  const size_t page_elems = kv_page_elems(d.Hkv, AF_PT, D);
  const size_t v_off = (size_t)d.Hkv * AF_PT * D;
  const uint32_t my_bars = smem_u32(bars) + 8u * (warp * AF_MAX_SLOTS);
  const uint32_t my_ring = ring0 + (uint32_t)(warp * S) * SLOT_BYTES;
  const int first = page_index(0), stride_p = n_splits * AF_WARPS;
  const int my_n = first < n_pages ? (n_pages - first + stride_p - 1) / stride_p : 0;
  auto page_of = [&](int i) {  // all lanes call; page id of this warp's i-th page
    const int32_t lo = __shfl_sync(0xffffffffu, bt_lo, i & 31), hi = __shfl_sync(0xffffffffu, bt_hi, i & 31);
    return i < 32 ? lo : i < 64 ? hi : bt[page_index(i)];
  };
  auto issue = [&](int page, int slot) {  // lane 0: copy one page's keys and values of this head into a slot
    const __half* src = a.kv_layer + (size_t)page * page_elems + (size_t)kvh * AF_PT * D;
    const uint32_t dst = my_ring + slot * SLOT_BYTES, bar = my_bars + 8u * slot;
    mbar_expect_tx(bar, SLOT_BYTES);
    bulk_load(dst, src, PAGE_BYTES, bar);
    bulk_load(dst + PAGE_BYTES, src + v_off, PAGE_BYTES, bar);
    if (SPLIT) bulk_load(dst + 2 * PAGE_BYTES, a.klo_layer + ((size_t)page * d.Hkv + kvh) * AF_PT * D, PAGE_BYTES, bar);
  };
  pdl_trigger();
  if (lane == 0) {
    for (int sl = 0; sl < S; ++sl) mbar_init(my_bars + 8u * sl, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int sl = 0; sl < S && sl < my_n; ++sl) {
    const int page = page_of(sl);
    if (lane == 0) issue(page, sl);
  }
  pdl_wait();  // the projection's output

  // rotate: this CTA's G query heads; and, in the CTA whose run holds the new token's page, its key (+ value)
  const int page_new = pos / AF_PT, slot_new = pos % AF_PT;
  const bool owner_cta = page_new % n_splits == split;
  {
    const float* row = a.qkv32 + (size_t)b * a.stride;
    const float2* cs = a.rope_table + (size_t)pos * (D / 2);
    const float rs = SPLIT ? a.row_scale[b] : 1.f;
    for (int e = threadIdx.x; e < G * (D / 2); e += AF_THREADS) {
      const int gq = e / (D / 2), i = e % (D / 2);
      const float* hp = row + (size_t)(kvh * G + gq) * D;
      const float x1 = hp[i] * rs, x2 = hp[i + D / 2] * rs;
      const float2 c = cs[i];
      const float r1 = x1 * c.x - x2 * c.y, r2 = x2 * c.x + x1 * c.y;
      const __half h1 = f16_sat(r1), h2 = f16_sat(r2);
      sq[gq * D + i] = h1;
      sq[gq * D + i + D / 2] = h2;
      if (SPLIT) {
        sq_lo[gq * D + i] = __float2half_rn(r1 - __half2float(h1));
        sq_lo[gq * D + i + D / 2] = __float2half_rn(r2 - __half2float(h2));
      }
    }
    if (owner_cta) {
      const float* kp = row + (size_t)(d.Hq + kvh) * D;
      const float* vp = row + (size_t)(d.Hq + d.Hkv + kvh) * D;
      __half* dk = a.kv_layer + (size_t)bt[page_new] * page_elems + ((size_t)kvh * AF_PT + slot_new) * D;
      __half* dkl = SPLIT ? a.klo_layer + (((size_t)bt[page_new] * d.Hkv + kvh) * AF_PT + slot_new) * D : nullptr;
      for (int i = threadIdx.x; i < D / 2; i += AF_THREADS) {
        const float x1 = kp[i] * rs, x2 = kp[i + D / 2] * rs;
        const float2 c = cs[i];
        const float r1 = x1 * c.x - x2 * c.y, r2 = x2 * c.x + x1 * c.y;
        const __half k1 = f16_sat(r1), k2 = f16_sat(r2);
        const __half v1 = f16_sat(vp[i] * rs), v2 = f16_sat(vp[i + D / 2] * rs);
        snew[i] = k1; snew[i + D / 2] = k2;
        snew[D + i] = v1; snew[D + i + D / 2] = v2;
        // the cache keeps them for the following steps, in its chunk-permuted row layout
        const int j1 = (kv_chunk_pos(i >> 3, slot_new) << 3) + (i & 7);
        const int j2 = (kv_chunk_pos((i + D / 2) >> 3, slot_new) << 3) + (i & 7);
        dk[j1] = k1; dk[j2] = k2;
        dk[v_off + j1] = v1; dk[v_off + j2] = v2;
        if (SPLIT) {
          const __half l1 = __float2half_rn(r1 - __half2float(k1)), l2 = __float2half_rn(r2 - __half2float(k2));
          snew[2 * D + i] = l1; snew[2 * D + i + D / 2] = l2;
          dkl[j1] = l1; dkl[j2] = l2;
        }
      }
    }
  }
  __syncthreads();

  // query heads kvh*G .. kvh*G+G-1 as operand rows 0..G-1 (rows G..15 are zero)
  uint32_t qf[KS][2];  // [k step][k half]; only the "row g" halves of the fragment are non-zero
  {
    const __half* qrow = sq + (g < G ? g : 0) * D;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qf[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * tq) : 0u;
      qf[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * tq) : 0u;
    }
  }
  uint32_t qfl[SPLIT ? KS : 1][2];
  if (SPLIT) {
    const __half* qrow = sq_lo + (g < G ? g : 0) * D;
#pragma unroll
    for (int ks = 0; ks < (SPLIT ? KS : 1); ++ks) {
      qfl[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * tq) : 0u;
      qfl[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * tq) : 0u;
    }
  }
  const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;

  float o[DN][2];  // row g of each 8-wide output column tile (rows 8..15 are padding and dropped)
#pragma unroll
  for (int i = 0; i < DN; ++i) o[i][0] = o[i][1] = 0.f;
  float m_run = AF_NEG, l_run = 0.f;

  bool ok = true;
  int slot = 0;
  uint32_t phase = 0;
  for (int i = 0; i < my_n; ++i) {
    const int pi = page_index(i);
    if (!mbar_wait(my_bars + 8u * slot, phase, nullptr)) { ok = false; break; }
    const uint32_t kt = my_ring + slot * SLOT_BYTES, vt = kt + PAGE_BYTES;
    const bool patched = pi == page_new;
    if (patched) {
      // this page was copied while its last row was being written: put the new key / value over it
      for (int e = lane; e < (SPLIT ? 3 : 2) * CPR; e += 32) {
        const int which = e / CPR, c = e % CPR;   // 0 key, 1 value, 2 key's low term
        const uint4 v = *reinterpret_cast<const uint4*>(snew + which * D + c * 8);
        const uint32_t dst = kt + which * PAGE_BYTES + tile_off<D>(slot_new, c);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
      }
      __syncwarp();
    }

    // scores of the page's 16 keys: two 8-key column tiles
    float s[2][4];
    s[0][0] = s[0][1] = s[0][2] = s[0][3] = 0.f;
    s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int r = (lane & 7) + ((lane >> 4) << 3);
      const int c = 2 * ks + ((lane >> 3) & 1);
      uint32_t b0, b1, b2, b3;
      ldsm_x4(kt + tile_off<D>(r, c), b0, b1, b2, b3);
      mma_f16_16816(s[0], qf[ks][0], 0u, qf[ks][1], 0u, b0, b1);
      mma_f16_16816(s[1], qf[ks][0], 0u, qf[ks][1], 0u, b2, b3);
      if (SPLIT) {
        const int kq = SPLIT ? ks : 0;
        mma_f16_16816(s[0], qfl[kq][0], 0u, qfl[kq][1], 0u, b0, b1);
        mma_f16_16816(s[1], qfl[kq][0], 0u, qfl[kq][1], 0u, b2, b3);
        ldsm_x4(kt + 2 * PAGE_BYTES + tile_off<D>(r, c), b0, b1, b2, b3);
        mma_f16_16816(s[0], qf[ks][0], 0u, qf[ks][1], 0u, b0, b1);
        mma_f16_16816(s[1], qf[ks][0], 0u, qf[ks][1], 0u, b2, b3);
      }
    }
    const int key0 = pi * AF_PT + 2 * tq;
    float mx = m_run;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float v = (key0 + 8 * nt + e < ctx_total) ? s[nt][e] * sl2 : AF_NEG;
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
        p[nt][e] = (key0 + 8 * nt + e < ctx_total) ? exp2f(s[nt][e] - mx) : 0.f;
        sum += p[nt][e];
      }
    l_run = l_run * corr + sum;
    const uint32_t pa0 = pack_f16(p[0][0], p[0][1]), pa2 = pack_f16(p[1][0], p[1][1]);
#pragma unroll
    for (int dp = 0; dp < DN / 2; ++dp) {
      const int r = (lane & 7) + (((lane >> 3) & 1) << 3);
      const int c = 2 * dp + (lane >> 4);
      uint32_t b0, b1, b2, b3;
      ldsm_x4_t(vt + tile_off<D>(r, c), b0, b1, b2, b3);
      float c0[4] = {o[2 * dp][0] * corr, o[2 * dp][1] * corr, 0.f, 0.f};
      float c1[4] = {o[2 * dp + 1][0] * corr, o[2 * dp + 1][1] * corr, 0.f, 0.f};
      mma_f16_16816(c0, pa0, 0u, pa2, 0u, b0, b1);
      mma_f16_16816(c1, pa0, 0u, pa2, 0u, b2, b3);
      o[2 * dp][0] = c0[0]; o[2 * dp][1] = c0[1];
      o[2 * dp + 1][0] = c1[0]; o[2 * dp + 1][1] = c1[1];
    }
    // all reads of the slot are consumed by issued MMAs; hand it back to the copy engine
    __syncwarp();
    if (i + S < my_n) {
      const int page = page_of(i + S);
      if (lane == 0) {
        if (patched) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(page, slot);
      }
    }
    if (++slot == S) { slot = 0; phase ^= 1u; }
  }
  if (!ok) {
    if (lane == 0) atomicCAS(a.err, 0, 5);
    for (int sl = 0; sl < S; ++sl) mbar_wait(my_bars + 8u * sl, 0, nullptr), mbar_wait(my_bars + 8u * sl, 1, nullptr);
  }
  __syncthreads();  // every warp is done with its ring: the space is reused below

  // combine the four warps: (m, l) per head, then rescaled O
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  float* sm_m = reinterpret_cast<float*>(ring_ptr);  // [AF_WARPS][8]
  float* sm_l = sm_m + AF_WARPS * 8;                 // [AF_WARPS][8]
  float* sm_o = sm_l + AF_WARPS * 8;                 // [AF_WARPS][G][D]
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
  for (int e = threadIdx.x; e < G * D; e += AF_THREADS) {
    const int gq = e / D, dd = e % D;
    float mx = AF_NEG;
#pragma unroll
    for (int w = 0; w < AF_WARPS; ++w) mx = fmaxf(mx, sm_m[w * 8 + gq]);
    float l = 0.f, acc = 0.f;
#pragma unroll
    for (int w = 0; w < AF_WARPS; ++w) {
      const float wgt = exp2f(sm_m[w * 8 + gq] - mx);
      l += wgt * sm_l[w * 8 + gq];
      acc += wgt * sm_o[(w * G + gq) * D + dd];
    }
    ex_o[e] = acc;
    if (dd == 0) {
      ex_m[gq] = mx;
      ex_l[gq] = l;
    }
  }

  if (GLOBAL) {
    __shared__ int last_flag;
    __shared__ float all_m[8 * 8], all_l[8 * 8];  // [head][split]
    constexpr int ROW = G * D + 16;
    const int group = b * d.Hkv + kvh;
    float* grp = a.scratch + (size_t)group * n_splits * ROW;
    __syncthreads();  // ex_o, ex_m, ex_l are complete
    float* mine = grp + (size_t)split * ROW;
    for (int e = threadIdx.x * 4; e < G * D; e += AF_THREADS * 4)
      __stcg(reinterpret_cast<float4*>(mine + e), *reinterpret_cast<const float4*>(ex_o + e));
    if ((int)threadIdx.x < G) {
      __stcg(mine + G * D + threadIdx.x, ex_m[threadIdx.x]);
      __stcg(mine + G * D + 8 + threadIdx.x, ex_l[threadIdx.x]);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const int t = atomicAdd(a.tickets + group, 1);
      last_flag = t == n_splits - 1;
      if (last_flag) a.tickets[group] = 0;  // for the next launch (it starts after this grid has completed)
    }
    __syncthreads();
    if (!last_flag) return;
    __threadfence();
    if ((int)threadIdx.x < G * n_splits) {
      const int gq = threadIdx.x / n_splits, sp = threadIdx.x % n_splits;
      all_m[gq * 8 + sp] = sp == split ? ex_m[gq] : __ldcg(grp + (size_t)sp * ROW + G * D + gq);
      all_l[gq * 8 + sp] = sp == split ? ex_l[gq] : __ldcg(grp + (size_t)sp * ROW + G * D + 8 + gq);
    }
    __syncthreads();
    // every thread fetches the n_splits partial sums of its four outputs in one batch, then combines them
    for (int e = threadIdx.x * 4; e < G * D; e += AF_THREADS * 4) {
      const int gq = e / D, dd = e % D;
      float4 ov[8];
#pragma unroll
      for (int sp = 0; sp < 8; ++sp)
        ov[sp] = sp < n_splits ? __ldcg(reinterpret_cast<const float4*>(grp + (size_t)sp * ROW + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
      float mx = AF_NEG;
#pragma unroll
      for (int sp = 0; sp < 8; ++sp)
        if (sp < n_splits) mx = fmaxf(mx, all_m[gq * 8 + sp]);
      float l = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int sp = 0; sp < 8; ++sp) {
        if (sp < n_splits) {
          const float wgt = exp2f(all_m[gq * 8 + sp] - mx);
          l += wgt * all_l[gq * 8 + sp];
          acc.x += wgt * ov[sp].x; acc.y += wgt * ov[sp].y; acc.z += wgt * ov[sp].z; acc.w += wgt * ov[sp].w;
        }
      }
      __half* op = a.out + ((size_t)b * d.Hq + kvh * G + gq) * D + dd;
      uint2 pk;  // the same quotient as the cluster variant forms: both variants give the same bits
      pk.x = pack_f16_sat(acc.x / l, acc.y / l);
      pk.y = pack_f16_sat(acc.z / l, acc.w / l);
      *reinterpret_cast<uint2*>(op) = pk;
    }
    return;
  }

  // merge over the splits: every CTA of the cluster takes a slice of the G x D outputs.  Loads from a peer's shared
  // memory have a long latency, so none of them may wait for another: first one thread per (head, split) fetches
  // that split's maximum and denominator into this CTA's own shared memory, then every thread fetches the n_splits
  // partial outputs of its element in one batch and only then combines them.
  __syncthreads();
  cluster_barrier();
  {
    __shared__ float all_m[8 * 8], all_l[8 * 8];  // [head][split]
    const uint32_t rank = cluster_rank_x();  // == split
    const uint32_t a_m = smem_u32(ex_m), a_l = smem_u32(ex_l), a_o = smem_u32(ex_o);
    if ((int)threadIdx.x < G * n_splits) {
      const int gq = threadIdx.x / n_splits, sp = threadIdx.x % n_splits;
      const float mv = ld_cluster_f32(a_m + 4u * gq, sp), lv = ld_cluster_f32(a_l + 4u * gq, sp);
      all_m[gq * 8 + sp] = mv;
      all_l[gq * 8 + sp] = lv;
    }
    __syncthreads();
    const int per = (G * D + n_splits - 1) / n_splits;
    const int e0 = (int)rank * per, e1 = min(G * D, e0 + per);
    for (int e = e0 + threadIdx.x; e < e1; e += AF_THREADS) {
      const int gq = e / D, dd = e % D;
      float ov[8];
#pragma unroll
      for (int sp = 0; sp < 8; ++sp) ov[sp] = sp < n_splits ? ld_cluster_f32(a_o + 4u * e, sp) : 0.f;
      float mx = AF_NEG;
#pragma unroll
      for (int sp = 0; sp < 8; ++sp)
        if (sp < n_splits) mx = fmaxf(mx, all_m[gq * 8 + sp]);
      float l = 0.f, acc = 0.f;
#pragma unroll
      for (int sp = 0; sp < 8; ++sp) {
        if (sp < n_splits) {
          const float wgt = exp2f(all_m[gq * 8 + sp] - mx);
          l += wgt * all_l[gq * 8 + sp];
          acc += wgt * ov[sp];
        }
      }
      a.out[((size_t)b * d.Hq + kvh * G + gq) * D + dd] = f16_sat(acc / l);
    }
  }
  __syncthreads();
  cluster_barrier();  // nobody leaves while a peer may still read its partial
}

template <int D, int G, bool SPLIT, bool GLOBAL>
int launch_dg(const AttnFusedArgs& a_in, int n_splits, const BatchMeta& bm, const ModelDims& d, cudaStream_t st) {
  static bool configured = false;
  constexpr int SLOT_BYTES = (SPLIT ? 3 : 2) * AF_PT * D * 2;
  constexpr int COMBINE_BYTES = (2 * AF_WARPS * 8 + AF_WARPS * G * D) * 4;
  constexpr int MAX_DYN = AF_WARPS * AF_MAX_SLOTS * SLOT_BYTES + 128;
  static_assert(AF_WARPS * 2 * SLOT_BYTES >= COMBINE_BYTES, "the combine buffers reuse the ring");
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(attn_decode_fused_kernel<D, G, SPLIT, GLOBAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_DYN));
    configured = true;
  }
  AttnFusedArgs a = a_in;
  if (attn_fused_slots_override() > 0) a.slots = attn_fused_slots_override();
  if (a.slots < 2) a.slots = 2;
  if (a.slots > AF_MAX_SLOTS) a.slots = AF_MAX_SLOTS;
  const size_t smem = (size_t)AF_WARPS * a.slots * SLOT_BYTES + 128;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_splits, d.Hkv, bm.n_seqs);
  cfg.blockDim = dim3(AF_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  if (GLOBAL) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_level() >= 2 ? 1 : 0;
  } else {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = n_splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_level() >= 3 ? 2 : 1;  // measured: launching the cluster variant early costs 2 %
  }
  HYP_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_decode_fused_kernel<D, G, SPLIT, GLOBAL>, a, bm, d));
  return 1;
}

}  // namespace

int& attn_fused_splits_override() {
  static int v = 0;
  return v;
}
int& first_block_split() {
  static int v = 1;
  return v;
}
int& attn_global_merge() {
  static int v = 1;
  return v;
}
int& attn_fused_slots_override() {
  static int v = 0;
  return v;
}

int attn_decode_fused_splits(int n_seqs, int Hkv, int max_ctx) {
  if (attn_fused_splits_override() > 0) return attn_fused_splits_override();
  // one resident wave: about three CTAs per SM; at least 8 pages (two per warp) per split; clusters of up to 8
  int want = (3 * sm_count()) / (n_seqs * Hkv);
  const int pages = (max_ctx + AF_PT - 1) / AF_PT;
  const int cap = (pages + 7) / 8;
  if (want > cap) want = cap;
  if (want > 8) want = 8;
  if (want < 1) want = 1;
  return want;
}

int launch_attn_decode_fused(const float* qkv32, int stride, __half* kv_layer, const float2* rope_table, __half* attn_out,
                             int n_splits, int slots, int* err, const BatchMeta& bm, const ModelDims& d, cudaStream_t st,
                             const float* row_scale, __half* klo_layer, float* scratch, int* tickets) {
  if (n_splits < 1 || n_splits > 8 || !err || (row_scale != nullptr) != (klo_layer != nullptr)) return HYP_EINVAL;
  if ((scratch != nullptr) != (tickets != nullptr)) return HYP_EINVAL;
  AttnFusedArgs a;
  a.qkv32 = qkv32; a.stride = stride; a.kv_layer = kv_layer; a.rope_table = rope_table; a.out = attn_out;
  a.slots = slots; a.err = err; a.row_scale = row_scale; a.klo_layer = klo_layer;
  a.scratch = scratch; a.tickets = tickets;
  const int G = d.Hq / d.Hkv;
#define HYP_AF_CASE(DD, GG)                                                \
  if (d.D == DD && G == GG)                                                \
    return scratch ? (row_scale ? launch_dg<DD, GG, true, true>(a, n_splits, bm, d, st)                            \
                                : launch_dg<DD, GG, false, true>(a, n_splits, bm, d, st))                          \
                   : (row_scale ? launch_dg<DD, GG, true, false>(a, n_splits, bm, d, st)                           \
                                : launch_dg<DD, GG, false, false>(a, n_splits, bm, d, st));
  HYP_AF_CASE(128, 1) HYP_AF_CASE(128, 2) HYP_AF_CASE(128, 4) HYP_AF_CASE(128, 8)
  HYP_AF_CASE(64, 1) HYP_AF_CASE(64, 2) HYP_AF_CASE(64, 4) HYP_AF_CASE(64, 8)
#undef HYP_AF_CASE
  return HYP_EINVAL;
}

}  // namespace hyp
