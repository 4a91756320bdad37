// Tensor-core projection for prefill: out[m, n] (+)= sum_k act[m, k] * w[n, k], bf16 in, fp32 accumulate.
//
// Persistent, warp-specialised sm_100a kernel:
//   warp 0   one lane issues TMA tile loads (128B-swizzled, K-major) into a 4-stage shared-memory ring;
//   warp 1   one lane issues tcgen05.mma (128 x 256 x 16 per instruction) into tensor memory; the
//            accumulator is double-buffered (2 x 256 columns) so the epilogue of tile i overlaps the
//            main loop of tile i+1;
//   warps 2-5  read the accumulator with tcgen05.ld and apply the epilogue (bf16 store, residual add,
//            SiLU(gate) * up, fp32 store) straight to global memory.
// For the SwiGLU epilogue the 256 accumulator columns are 128 gate columns and the 128 matching up
// columns (two weight boxes per stage), so gate and up never leave the chip.
// Work split: for the bf16 / fp32-store epilogues each CTA takes whole output tiles.  For the residual
// epilogue (out += acc) the k-blocks of all tiles form one list that is cut into equal contiguous
// ranges, one per CTA ("stream-K"); a CTA that holds only part of a tile's k range adds its partial
// sum with fp32 reductions, so 80 tiles still keep 148 SMs busy (used up to 2048 rows).  The order of
// those additions is not fixed, so the last bits of a split tile can differ between runs.
// Every mbarrier wait is bounded: on expiry the kernel records an error code and unwinds.
#include <cuda.h>

#include <algorithm>

#include "gemm_tc.cuh"
#include "sm100_common.cuh"
#include "tcgen05.cuh"
#include "hyperion.h"

namespace hyp {

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment*/ + 1024 /*barriers*/ + 4 * 2 * 32 * 128 /*epilogue boxes*/;
constexpr int TC_THREADS = 192;

// Instruction descriptor: (bf16 x bf16 | fp16 x fp16) -> fp32, both operands K-major, M = 128, N = 256.
constexpr uint32_t IDESC_BF16 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
constexpr uint32_t IDESC_F16 = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

// Walks the work of one CTA as a sequence of (tile, k-block range) segments.  All three roles of a CTA
// run the same walk, so they agree on the order without communicating.
//
// Stream-K mode: CTAs form teams of `team` members; member j of a team owns M-tile (group * team + j).
// The list of (M-tile group, N-tile, k-block) columns is cut into equal contiguous ranges, one per team,
// so the members of a team walk the same weight k-blocks at the same time (one HBM fetch, the rest L2
// hits) and every CTA gets the same number of k-blocks.
struct Segments {
  long u, u_end;  // stream-K: position in the column list
  int tile, n_tiles, stride, KB, tiles_m, tiles_n, team, member;
  bool streamk;
  // `unit` of `n_units`: the CTA's index in the grid, or the CTA pair's index for the two-CTA kernel (whose
  // M-tiles are 256 rows high)
  __device__ Segments(bool sk, int tiles_m_, int tiles_n_, int KB_, int team_, int unit, int n_units)
      : n_tiles(tiles_m_ * tiles_n_), KB(KB_), tiles_m(tiles_m_), tiles_n(tiles_n_), team(team_), streamk(sk) {
    if (sk) {
      const int n_teams = n_units / team_;
      const int my_team = unit / team_;
      member = unit % team_;
      const long total = (long)(tiles_m_ / team_) * tiles_n_ * KB_;
      u = total * my_team / n_teams;
      u_end = total * (my_team + 1) / n_teams;
    } else {
      tile = unit;
      stride = n_units;
    }
  }
  __device__ bool next(int& t, int& kb0, int& kb1) {
    if (streamk) {
      if (u >= u_end) return false;
      const long per_group = (long)tiles_n * KB;
      const int mg = (int)(u / per_group);
      const long rem = u % per_group;
      const int nt = (int)(rem / KB);
      kb0 = (int)(rem % KB);
      const long room = u_end - u;
      kb1 = (KB - kb0 < room) ? KB : kb0 + (int)room;
      u += kb1 - kb0;
      t = nt * tiles_m + mg * team + member;
      return true;
    }
    if (tile >= n_tiles) return false;
    t = tile;
    kb0 = 0;
    kb1 = KB;
    tile += stride;
    return true;
  }
};

// ---------------------------------------------------------------------------------------------------------
// Epilogue through shared memory and TMA.  An accumulator row lives in one thread (tcgen05.ld, lane = row), so
// direct global stores touch 32 rows per warp instruction, 16 bytes each.  Instead every epilogue warp turns its
// 32 rows x 128 bytes of results through a 4 KB staging box (128-byte swizzle: chunk c of row r at c ^ (r & 7),
// conflict-free for 16-byte stores by rows) and one lane hands the box to the copy engine: a tensor store, or - for
// the residual epilogue, whole tiles and split-K partial tiles alike - a tensor reduction that adds the box to
// the residual stream in L2.  The tensor map clips rows >= M and columns >= N, so ragged tiles need no predicates.
// Two boxes per warp: the next one is filled while the copy engine reads the previous one.
// ---------------------------------------------------------------------------------------------------------
constexpr int EPI_BOX_BYTES = 32 * 128;                 // 32 rows x 128 bytes
constexpr int EPI_STAGING_BYTES = 4 * 2 * EPI_BOX_BYTES;  // 4 epilogue warps x 2 boxes

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// One warp's share (32 rows) of one accumulator tile.  t0: tensor-memory address of the warp's lane quarter at
// the accumulator's first column; up_cols: column distance from a gate column to its up column (SwiGLU);
// boxes: shared address of the warp's two staging boxes; n_box: running count of boxes this warp has issued.
template <int EPI, int BN_ACC>
__device__ __forceinline__ void epilogue_warp(uint32_t t0, const CUtensorMap* tm_out, uint32_t boxes, int lane, int row0,
                                              int n0, int N, bool f16, uint32_t& n_box) {
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  constexpr bool OUT16 = EPI == EPI_STORE_BF16 || EPI == EPI_SWIGLU_BF16;
  constexpr int BN_OUT = SWIGLU ? BN_ACC / 2 : BN_ACC;
  constexpr int BOX_COLS = OUT16 ? 64 : 32;  // 128 bytes of output per row
  const uint32_t sw = (uint32_t)(lane & 7);
#pragma unroll 1
  for (int c = 0; c < BN_OUT; c += BOX_COLS) {
    if (n0 + c >= N) break;  // uniform across the warp
    const uint32_t box = boxes + (n_box & 1u) * EPI_BOX_BYTES;
    const uint32_t rowp = box + (uint32_t)lane * 128u;
    // the copy that last read this box (two boxes ago) must have finished reading it
    if (n_box >= 2) {
      if (lane == 0) bulk_wait_read<1>();
      __syncwarp();
    }
#pragma unroll
    for (int hh = 0; hh < (OUT16 ? 2 : 1); ++hh) {  // 32 accumulator columns at a time
      uint32_t v[32], u[SWIGLU ? 32 : 1];
      tmem_ld16(t0 + c + 32 * hh, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
      tmem_ld16(t0 + c + 32 * hh + 16, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
      if (SWIGLU) {
        tmem_ld16(t0 + BN_ACC / 2 + c + 32 * hh, *reinterpret_cast<uint32_t(*)[16]>(&u[0]));
        tmem_ld16(t0 + BN_ACC / 2 + c + 32 * hh + 16, *reinterpret_cast<uint32_t(*)[16]>(&u[SWIGLU ? 16 : 0]));
      }
      tmem_ld_wait();
      if (OUT16) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float y0 = __uint_as_float(v[2 * i]), y1 = __uint_as_float(v[2 * i + 1]);
          if (SWIGLU) {
            y0 = y0 / (1.f + __expf(-y0)) * __uint_as_float(u[SWIGLU ? 2 * i : 0]);
            y1 = y1 / (1.f + __expf(-y1)) * __uint_as_float(u[SWIGLU ? 2 * i + 1 : 0]);
          }
          pk[i] = f16 ? pack_f16_sat(y0, y1) : pack_bf16(y0, y1);  // 16-bit results take the operands' type
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
          st_shared_v4(rowp + ((((uint32_t)(4 * hh + j)) ^ sw) << 4), pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          st_shared_v4(rowp + (((uint32_t)j ^ sw) << 4), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the copy engine must see these stores
    __syncwarp();
    if (lane == 0) {
      if (EPI == EPI_RESID_F32)
        tma_reduce_add_2d(tm_out, box, n0 + c, row0);
      else
        tma_store_2d(tm_out, box, n0 + c, row0);
      bulk_commit();
    }
    ++n_box;
  }
}

template <int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
               const __grid_constant__ CUtensorMap tm_out, int M, int N, int K, int up_tile0, int team, uint32_t idesc,
               int* __restrict__ err) {
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  const bool STREAMK = EPI == EPI_RESID_F32 && team > 0;
  constexpr int BN_OUT = SWIGLU ? BN / 2 : BN;  // output columns per tile
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* aligned = smem_raw + (base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(aligned + STAGES * STAGE_BYTES);
  // bars: full[STAGES] | empty[STAGES] | tmem_full[2] | tmem_empty[2] | tmem base (u32) | abort (int)
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t staging = base + STAGES * STAGE_BYTES + 1024;  // 1024-aligned: the boxes are 128-byte swizzled

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN_OUT - 1) / BN_OUT;
  const int KB = (K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tm_a);
    prefetch_tensormap(&tm_b);
    prefetch_tensormap(&tm_out);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 128);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_trigger();

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer ----------------
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      int tile, kb0, kb1;
      // The weight boxes of the first ring-full of k-blocks go out before the wait for the predecessor (weights are
      // never written by a kernel); the activation boxes of the same stages follow it.  When this kernel was
      // launched early, its weights are then on their way while the predecessor drains.
      {
        Segments pre(STREAMK, tiles_m, tiles_n, KB, team, (int)blockIdx.x, (int)gridDim.x);
        int n = 0;
        while (n < STAGES && pre.next(tile, kb0, kb1)) {
          const int n0 = (tile / tiles_m) * BN_OUT;
          const int tb0 = n0 >> 4, tb1 = SWIGLU ? up_tile0 + (n0 >> 4) : (n0 >> 4) + 8;
          for (int kb = kb0; kb < kb1 && n < STAGES; ++kb, ++n) {
            const uint32_t sb = base + n * STAGE_BYTES + A_BYTES;
            mbar_expect_tx(full_bar(n), STAGE_BYTES);
            tma_load_4d(sb, &tm_b, 0, 0, kb, tb0, full_bar(n));
            tma_load_4d(sb + B_BYTES / 2, &tm_b, 0, 0, kb, tb1, full_bar(n));
          }
        }
      }
      pdl_wait();  // the activation operand is the predecessor's output
      Segments seg(STREAMK, tiles_m, tiles_n, KB, team, (int)blockIdx.x, (int)gridDim.x);
      while (ok && seg.next(tile, kb0, kb1)) {
        const int m0 = (tile % tiles_m) * BM;
        const int n0 = (tile / tiles_m) * BN_OUT;
        // weight tiles (16 rows each) of the two 128-row boxes: SwiGLU pairs gate rows with the matching up rows
        const int tb0 = n0 >> 4, tb1 = SWIGLU ? up_tile0 + (n0 >> 4) : (n0 >> 4) + 8;
        for (int kb = kb0; kb < kb1; ++kb, ++issued) {
          const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
          if (issued >= STAGES) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1, abort_flag)) { ok = false; break; }
            mbar_expect_tx(full_bar(stage), STAGE_BYTES);
            tma_load_4d(sb, &tm_b, 0, 0, kb, tb0, full_bar(stage));
            tma_load_4d(sb + B_BYTES / 2, &tm_b, 0, 0, kb, tb1, full_bar(stage));
          }
          tma_load_2d(sa, &tm_a, kb * BK, m0, full_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(err, 0, 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      Segments seg(STREAMK, tiles_m, tiles_n, KB, team, (int)blockIdx.x, (int)gridDim.x);
      int tile, kb0, kb1;
      while (ok && seg.next(tile, kb0, kb1)) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
          const uint64_t da = smem_desc(sa), db = smem_desc(sb);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            tc_mma(d_tmem, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                   (kb > kb0 || k > 0) ? 1u : 0u);
          tc_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc_commit(tfull_bar(acc));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1;
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(err, 0, 2);
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    const int q = warp & 3;  // tensor-memory lane quarter this warp may read
    pdl_wait();              // the output buffer may still be in use by the predecessor
    int acc = 0;
    uint32_t acc_phase = 0, n_box = 0;
    bool ok = true;
    const uint32_t boxes = staging + (uint32_t)q * (2 * EPI_BOX_BYTES);
    Segments seg(STREAMK, tiles_m, tiles_n, KB, team, (int)blockIdx.x, (int)gridDim.x);
    int tile, kb0, kb1;
    while (ok && seg.next(tile, kb0, kb1)) {
      const int m0 = (tile % tiles_m) * BM;
      const int n0 = (tile / tiles_m) * BN_OUT;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t0 = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(acc * BN);
      epilogue_warp<EPI, BN>(t0, &tm_out, boxes, lane, m0 + 32 * q, n0, N, idesc == IDESC_F16, n_box);
      tc_fence_before();
      mbar_arrive(tempty_bar(acc));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
    if (lane == 0) bulk_wait_all();  // the boxes must outlive the copies that read them; results complete before exit
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(err, 0, 3);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

// ---------------------------------------------------------------------------------------------------------
// Two-CTA variant (thread-block cluster of 2, tcgen05 cta_group::2): a CTA pair computes a 256 x 256 tile.
// Each CTA loads its own 128 activation rows and HALF of the weight tile (128 of the 256 rows; for SwiGLU the
// leader holds the gate rows, its peer the matching up rows), so a k-block costs 32 KB of shared-memory
// fill per SM instead of 48 KB and the ring is 6 stages deep.  The leader's lane issues one MMA for both
// CTAs; each CTA keeps its 128 x 256 half of the accumulator in its own tensor memory and runs its own
// epilogue.  All copies of a stage (from both CTAs) complete on the leader's "full" barrier; the MMA commit
// is multicast to both CTAs' "empty" / "accumulator ready" barriers; the peer's epilogue threads arrive
// remotely on the leader's "accumulator free" barrier.  No multicast loads.  Used for the non-residual
// epilogues (whole tiles per pair).
// ---------------------------------------------------------------------------------------------------------
constexpr int STAGES2 = 6;
constexpr int STAGE2_BYTES = A_BYTES + B_BYTES / 2;  // per CTA: 16 KB of A + 16 KB of its half of B
constexpr int SMEM2_BYTES = STAGES2 * STAGE2_BYTES + 1024 /*alignment*/ + 1024 /*barriers*/ + EPI_STAGING_BYTES;
constexpr uint32_t idesc2(bool f16, int bn) {  // M = 256 (the pair), N = bn, fp32 accumulate, both operands K-major
  return (1u << 4) | (f16 ? 0u : ((1u << 7) | (1u << 10))) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {  // same offset in CTA `rank`
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load of a CTA pair: data lands in the executing CTA, completion bytes go to `bar` (a
// shared::cluster address, here always the leader's barrier).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                 uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {  // arrive on `bar` (same offset) in both CTAs
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}

// BNT: accumulator columns of the pair's tile, 256 or 224 (each CTA supplies BNT / 2 weight rows = 8 or 7 packed
// tiles per k-block; the launcher picks the width that leaves the fewest idle pairs in the last wave).
template <int EPI, int BNT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const __grid_constant__ CUtensorMap tm_out, int M, int N, int K, int up_tile0, int team, uint32_t idesc,
                int* __restrict__ err) {
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  const bool STREAMK = EPI == EPI_RESID_F32 && team > 0;
  constexpr int BN_OUT = SWIGLU ? BNT / 2 : BNT;
  constexpr int B_HALF_BYTES = (BNT / 2) * BK * 2;  // this CTA's half of the weight tile
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* aligned = smem_raw + (base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(aligned + STAGES2 * STAGE2_BYTES);
  // bars: full[STAGES2] | empty[STAGES2] | tmem_full[2] | tmem_empty[2] | tmem base (u32) | abort (int)
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES2 + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES2 + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES2 + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES2 + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t staging = base + STAGES2 * STAGE2_BYTES + 1024;  // 1024-aligned: the boxes are 128-byte swizzled

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();      // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int pairs_m = (M + 2 * BM - 1) / (2 * BM), tiles_n = (N + BN_OUT - 1) / BN_OUT;
  const int n_tiles = pairs_m * tiles_n;
  const int KB = (K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tm_a);
    prefetch_tensormap(&tm_b);
    prefetch_tensormap(&tm_out);
    for (int s = 0; s < STAGES2; ++s) {
      mbar_init(full_bar(s), 1);    // the leader's arrive.expect_tx; bytes come from both CTAs' copies
      mbar_init(empty_bar(s), 1);   // the leader's MMA commit (multicast)
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);      // MMA commit (multicast)
      mbar_init(tempty_bar(a), 256);   // 128 epilogue threads of each CTA (used in the leader only)
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers exist before anybody signals across
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_trigger();

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer (both CTAs) ----------------
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      int tile, kb0, kb1;
      // weight boxes of the first ring-full of k-blocks before the wait for the predecessor, see gemm_tc_kernel
      {
        Segments pre(STREAMK, pairs_m, tiles_n, KB, team, pair, n_pairs);
        int n = 0;
        while (n < STAGES2 && pre.next(tile, kb0, kb1)) {
          const int n0 = (tile / pairs_m) * BN_OUT;
          const int tb = SWIGLU ? (int)rank * up_tile0 + (n0 >> 4) : (n0 >> 4) + (int)rank * (BNT / 32);
          for (int kb = kb0; kb < kb1 && n < STAGES2; ++kb, ++n) {
            if (rank == 0) mbar_expect_tx(full_bar(n), 2 * (A_BYTES + B_HALF_BYTES));
            tma_load_4d_pair(base + n * STAGE2_BYTES + A_BYTES, &tm_b, 0, 0, kb, tb, mapa_rank(full_bar(n), 0));
          }
        }
      }
      pdl_wait();
      Segments seg(STREAMK, pairs_m, tiles_n, KB, team, pair, n_pairs);
      while (ok && seg.next(tile, kb0, kb1)) {
        const int m0 = (tile % pairs_m) * (2 * BM) + (int)rank * BM;
        const int n0 = (tile / pairs_m) * BN_OUT;
        // this CTA's half of the weight tile, as an index of 16-row packed tiles
        const int tb = SWIGLU ? (int)rank * up_tile0 + (n0 >> 4) : (n0 >> 4) + (int)rank * (BNT / 32);
        for (int kb = kb0; kb < kb1; ++kb, ++issued) {
          const uint32_t sa = base + stage * STAGE2_BYTES, sb = sa + A_BYTES;
          const uint32_t lead_full = mapa_rank(full_bar(stage), 0);
          if (issued >= STAGES2) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1, abort_flag)) { ok = false; break; }
            if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * (A_BYTES + B_HALF_BYTES));
            tma_load_4d_pair(sb, &tm_b, 0, 0, kb, tb, lead_full);
          }
          tma_load_2d_pair(sa, &tm_a, kb * BK, m0, lead_full);
          if (++stage == STAGES2) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(err, 0, 6);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ---------------- MMA issuer (leader only) ----------------
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      Segments seg(STREAMK, pairs_m, tiles_n, KB, team, pair, n_pairs);
      int tile, kb0, kb1;
      while (ok && seg.next(tile, kb0, kb1)) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + stage * STAGE2_BYTES, sb = sa + A_BYTES;
          const uint64_t da = smem_desc(sa), db = smem_desc(sb);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            tc_mma_pair(d_tmem, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                        (kb > kb0 || k > 0) ? 1u : 0u);
          tc_commit_pair(empty_bar(stage));
          if (++stage == STAGES2) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc_commit_pair(tfull_bar(acc));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1;
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(err, 0, 7);
      }
    }
  } else {
    // ---------------- epilogue warps (both CTAs, each its own 128 rows) ----------------
    const int q = warp & 3;
    pdl_wait();
    int acc = 0;
    uint32_t acc_phase = 0, n_box = 0;
    bool ok = true;
    const uint32_t boxes = staging + (uint32_t)q * (2 * EPI_BOX_BYTES);
    Segments seg(STREAMK, pairs_m, tiles_n, KB, team, pair, n_pairs);
    int tile, kb0, kb1;
    while (ok && seg.next(tile, kb0, kb1)) {
      const int m0 = (tile % pairs_m) * (2 * BM) + (int)rank * BM;
      const int n0 = (tile / pairs_m) * BN_OUT;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t0 = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(acc * BN);
      epilogue_warp<EPI, BNT>(t0, &tm_out, boxes, lane, m0 + 32 * q, n0, N, (idesc & (1u << 7)) == 0, n_box);
      tc_fence_before();
      mbar_arrive_cluster(mapa_rank(tempty_bar(acc), 0));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
    if (lane == 0) bulk_wait_all();  // the boxes must outlive the copies that read them; results complete before exit
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(err, 0, 8);
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // nobody leaves (or frees tensor memory) while its peer may still signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

int encode_map(CUtensorMap* map, const void* ptr, int rows, int K, int box_rows, bool f16) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return HYP_ECUDA;
  if ((K % 8) != 0 || ((uintptr_t)ptr & 15) != 0) return HYP_EINVAL;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  CUresult r = enc(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)ptr, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return HYP_ECUDA;
  }
  return HYP_OK;
}

// Output matrix [M, N] (row stride ldo elements) as the epilogue's boxes see it: 32 rows x 128 bytes, 128-byte
// swizzle, extents M and N so that the copy engine clips ragged tiles.
int encode_out_map(CUtensorMap* map, void* out, int ldo, int M, int N, int epi, bool f16) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return HYP_ECUDA;
  const bool out16 = epi == EPI_STORE_BF16 || epi == EPI_SWIGLU_BF16;
  const size_t es = out16 ? 2 : 4;
  const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)ldo * es};
  const cuuint32_t box[2] = {(cuuint32_t)(128 / es), 32u};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUtensorMapDataType dt = !out16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                 : f16  ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  CUresult r = enc(map, dt, 2, out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return HYP_ECUDA;
  }
  return HYP_OK;
}

int* g_err_flag = nullptr;  // one device word per process: first non-zero code wins

template <int EPI, int BNT>
int launch_pair_bn(const TcAct& act, const TcWeight& w, int M, int N, int K, void* out, int ldo, cudaStream_t st,
                   long pairs, int team, bool early) {
  static bool configured = false;
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(gemm_tc2_kernel<EPI, BNT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    configured = true;
  }
  CUtensorMap tm_out;
  const int mrc = encode_out_map(&tm_out, out, ldo, M, N, EPI, act.f16);
  if (mrc) return mrc;
  const CUtensorMap& tm_b = BNT == 256 ? w.map : w.map7;
  if (early)
    HYP_CUDA_TRY(launch_pdl<1>(gemm_tc2_kernel<EPI, BNT>, dim3((unsigned)(2 * pairs)), dim3(TC_THREADS), (size_t)SMEM2_BYTES, st,
                               act.map, tm_b, tm_out, M, N, K, w.N16p, team, idesc2(act.f16, BNT), g_err_flag));
  else
    HYP_CUDA_TRY(launch_pdl(gemm_tc2_kernel<EPI, BNT>, dim3((unsigned)(2 * pairs)), dim3(TC_THREADS), (size_t)SMEM2_BYTES, st,
                            act.map, tm_b, tm_out, M, N, K, w.N16p, team, idesc2(act.f16, BNT), g_err_flag));
  return 1;
}

template <int EPI>
int launch_pair(const TcAct& act, const TcWeight& w, int M, int N, int K, void* out, int ldo, cudaStream_t st,
                int num_sms, bool early) {
  constexpr int OUT_PER_ACC = EPI == EPI_SWIGLU_BF16 ? 2 : 1;  // SwiGLU: a gate and an up column per output column
  const int pairs_m = (M + 2 * BM - 1) / (2 * BM);
  long pairs = num_sms / 2;
  int team = 0;  // 0 = whole tiles per CTA pair
  if (EPI == EPI_RESID_F32) {
    // stream-K over CTA pairs: teams of `team` pairs (a divisor of the 256-row M-tiles) share the weight k-blocks
    // they walk; every team gets the same number of k-blocks
    const int tiles_n = (N + BN - 1) / BN;
    double best = -1.0;
    team = 1;
    for (int ts = 1; ts <= pairs_m && ts <= pairs; ++ts) {
      if (pairs_m % ts) continue;
      const long teams = pairs / ts;
      const double score = (double)(teams * ts) / (double)pairs + 0.003 * ts;
      if (score > best) { best = score; team = ts; }
    }
    long teams = pairs / team;
    const long cols = (long)(pairs_m / team) * tiles_n * ((K + BK - 1) / BK);
    if (teams > cols) teams = cols;
    pairs = teams * team;
    return launch_pair_bn<EPI, 256>(act, w, M, N, K, out, ldo, st, pairs, team, early);
  }
  // whole tiles per pair: a 224-column tile is taken when it needs less tensor time over all waves than a 256-column
  // one (7680 columns at 512 rows: 70 tiles of 224 fill 74 pairs once, 60 tiles of 256 leave 14 idle for longer)
  auto waves_cost = [&](int bn, long* tiles_out) {
    const long tiles = (long)pairs_m * ((N + bn / OUT_PER_ACC - 1) / (bn / OUT_PER_ACC));
    *tiles_out = tiles;
    return ((tiles + pairs - 1) / pairs) * bn;
  };
  long tiles256, tiles224;
  const long c256 = waves_cost(256, &tiles256), c224 = waves_cost(224, &tiles224);
  // (fp32 stores only: their 32-column output boxes divide 224, the 64-column boxes of the 16-bit epilogues do not)
  if (EPI == EPI_STORE_F32 && c224 < c256 && tile_width_224_enabled())
    return launch_pair_bn<EPI, 224>(act, w, M, N, K, out, ldo, st, tiles224 < pairs ? tiles224 : pairs, 0, early);
  return launch_pair_bn<EPI, 256>(act, w, M, N, K, out, ldo, st, tiles256 < pairs ? tiles256 : pairs, 0, early);
}

template <int EPI>
int launch_epi(const TcAct& act, const TcWeight& w, int M, int N, int K, void* out, int ldo, cudaStream_t st, bool early) {
  static bool configured = false;
  static int num_sms = 0;
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    int dev = 0;
    HYP_CUDA_TRY(cudaGetDevice(&dev));
    HYP_CUDA_TRY(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    configured = true;
  }
  constexpr int BN_OUT = EPI == EPI_SWIGLU_BF16 ? BN / 2 : BN;
  const int tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN_OUT - 1) / BN_OUT;
  // two-CTA tiles (a third less shared-memory fill per flop) from 129 rows on; the residual epilogue only up to 1024
  // rows: measured on B200 (N 5120, K 17920) the pair kernel's stream-K takes 75 / 154 us at 512 / 1024 rows against
  // 79 / 161 for one-CTA stream-K, but 359 / 679 against 299 / 590 at 2048 / 4096 rows
  if (tiles_m >= 2 && (EPI != EPI_RESID_F32 || tiles_m <= 8)) return launch_pair<EPI>(act, w, M, N, K, out, ldo, st, num_sms, early);
  int grid, team = 0;  // team 0 = whole tiles per CTA
  if (EPI == EPI_RESID_F32 && tiles_m <= 16) {
    // stream-K (up to 2048 rows; beyond that whole tiles already balance and reuse A better): pick the team size (a divisor of tiles_m) that keeps most SMs busy, larger teams preferred
    double best = -1.0;
    team = 1;
    for (int ts = 1; ts <= tiles_m && ts <= num_sms; ++ts) {
      if (tiles_m % ts) continue;
      const int teams = num_sms / ts;
      const double score = (double)(teams * ts) / num_sms + 0.003 * ts;
      if (score > best) { best = score; team = ts; }
    }
    long teams = num_sms / team;
    const long cols = (long)(tiles_m / team) * tiles_n * ((K + BK - 1) / BK);
    if (teams > cols) teams = cols;
    grid = (int)teams * team;
  } else {
    const long tiles = (long)tiles_m * tiles_n;
    grid = (int)(tiles < num_sms ? tiles : num_sms);
  }
  // launched early (set-up under the predecessor's tail; every load waits for it) where the caller allows
  CUtensorMap tm_out;
  const int mrc = encode_out_map(&tm_out, out, ldo, M, N, EPI, act.f16);
  if (mrc) return mrc;
  if (early)
    HYP_CUDA_TRY(launch_pdl<1>(gemm_tc_kernel<EPI>, dim3(grid), dim3(TC_THREADS), (size_t)SMEM_BYTES, st, act.map, w.map,
                               tm_out, M, N, K, w.N16p, team, act.f16 ? IDESC_F16 : IDESC_BF16, g_err_flag));
  else
    HYP_CUDA_TRY(launch_pdl(gemm_tc_kernel<EPI>, dim3(grid), dim3(TC_THREADS), (size_t)SMEM_BYTES, st, act.map, w.map,
                            tm_out, M, N, K, w.N16p, team, act.f16 ? IDESC_F16 : IDESC_BF16, g_err_flag));
  return 1;
}

}  // namespace

// Packed weights: one 4-D descriptor whose box is eight 16-row tiles of one k-block (a 128-row operand tile).  The
// tiles already carry the 128-byte swizzle, so the copy itself applies none.
int tc_make_weight(TcWeight* w, const void* packed, int rows, int halves, int K, bool f16) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return HYP_ECUDA;
  if (rows < 1 || (halves != 1 && halves != 2) || K < 8 || (K % 8) != 0 || ((uintptr_t)packed & 127) != 0) return HYP_EINVAL;
  w->packed = packed; w->rows = rows; w->halves = halves; w->K = K; w->f16 = f16;
  w->KBp = pk_kbp(K);
  w->N16p = pk_n16p(rows);
  const cuuint64_t dims[4] = {64, 16, (cuuint64_t)w->KBp, (cuuint64_t)halves * w->N16p};
  const cuuint64_t strides[3] = {128, (cuuint64_t)PK_TILE_BYTES, (cuuint64_t)w->KBp * PK_TILE_BYTES};
  const cuuint32_t box[4] = {64, 16, 1, 8};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  CUresult r = enc(&w->map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, (void*)packed, dims,
                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  const cuuint32_t box7[4] = {64, 16, 1, 7};  // 112 rows: a CTA's half of a 224-column pair tile
  if (r == CUDA_SUCCESS)
    r = enc(&w->map7, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, (void*)packed, dims, strides,
            box7, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return HYP_ECUDA;
  }
  return HYP_OK;
}

int& tile_width_224_enabled() {
  static int v = 1;
  return v;
}

namespace {
// One thread per 16-byte chunk of the packed buffer: finds the source row and k of its chunk, converts, stores.
__global__ void pack_weight_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int rows, int halves, int K,
                                   int N16p, int KBp, bool to_f16) {
  const size_t total = (size_t)halves * N16p * KBp * (PK_TILE_BYTES / 16);
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int c_sw = (int)(idx & 7), r = (int)((idx >> 3) & 15);
    const size_t tile = idx >> 7;
    const int kb = (int)(tile % KBp);
    const int t = (int)(tile / KBp);
    const int half = t / N16p, n = (t % N16p) * 16 + r;
    const int k = kb * 64 + ((c_sw ^ (r & 7)) << 3);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (n < rows && k < K) {
      v = src[((size_t)(half * rows + n) * K + k) >> 3];
      if (to_f16) {
        uint32_t* p = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = pack_f16_sat(bf16_lo(p[i]), bf16_hi(p[i]));
      }
    }
    dst[idx] = v;
  }
}
}  // namespace

int tc_pack_weight(const void* src, void* dst, int rows, int halves, int K, bool to_f16, cudaStream_t st) {
  if (!src || !dst || rows < 1 || (halves != 1 && halves != 2) || K < 8 || (K % 8) != 0) return HYP_EINVAL;
  if (((uintptr_t)src & 15) != 0 || ((uintptr_t)dst & 15) != 0) return HYP_EINVAL;
  const size_t chunks = tc_packed_bytes(rows, halves, K) / 16;
  const int blocks = (int)std::min<size_t>((chunks + 255) / 256, (size_t)sm_count() * 16);
  pack_weight_kernel<<<blocks, 256, 0, st>>>((const uint4*)src, (uint4*)dst, rows, halves, K, pk_n16p(rows), pk_kbp(K), to_f16);
  return 1;
}

// One block's KV page pool [pages][K, V][Hkv][16 tokens][D] fp16 seen as a matrix of D-wide rows; box = 16 rows (one
// page of one head) x 64 columns.  The rows are stored chunk-permuted inside each 128-byte half, so such a box lands
// in shared memory as a 128-byte-swizzled operand tile without any swizzle in the copy.
int tc_make_kv_map(CUtensorMap* map, const void* kv_layer, size_t n_pages, int Hkv, int D) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return HYP_ECUDA;
  if (D != 128 || ((uintptr_t)kv_layer & 15) != 0 || n_pages < 1) return HYP_EINVAL;
  const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)(n_pages * 2 * (size_t)Hkv * 16)};
  const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
  const cuuint32_t box[2] = {64u, 16u};
  const cuuint32_t estr[2] = {1u, 1u};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (void*)kv_layer, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return HYP_ECUDA;
  }
  return HYP_OK;
}

// Activations: 128-row boxes for the tile kernels, 16/32/64-row boxes for the swapped-operand kernel.
int tc_make_act(TcAct* a, const void* ptr, int rows, int K, bool f16) {
  a->ptr = ptr; a->rows = rows; a->K = K; a->f16 = f16;
  int rc = encode_map(&a->map, ptr, rows, K, 128, f16);
  for (int i = 0; i < 3 && !rc; ++i) rc = encode_map(&a->map_small[i], ptr, rows, K, 16 << i, f16);
  a->has_a8 = false;
  if (!rc && K % 64 == 0) {
    EncodeTiledFn enc = encode_fn();
    const cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(K / 64)};
    const cuuint64_t strides[2] = {(cuuint64_t)K * 2, 128};
    const cuuint32_t box[3] = {64, 8, 2};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult r = enc(&a->map_a8, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void*)ptr, dims,
                     strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    a->has_a8 = r == CUDA_SUCCESS;  // without it the streaming kernel reads its fragments from global memory
  }
  return rc;
}

int* tc_err_flag_ptr() { return g_err_flag; }

int tc_prepare() {
  if (!g_err_flag) {
    HYP_CUDA_TRY(cudaMalloc((void**)&g_err_flag, sizeof(int)));
    HYP_CUDA_TRY(cudaMemset(g_err_flag, 0, sizeof(int)));
  }
  return HYP_OK;
}

int tc_error_flag(int* value_out) {
  *value_out = 0;
  if (!g_err_flag) return HYP_OK;
  HYP_CUDA_TRY(cudaMemcpy(value_out, g_err_flag, sizeof(int), cudaMemcpyDeviceToHost));
  return HYP_OK;
}

int tc_error_flag_take(int* value_out, bool clear) {
  const int rc = tc_error_flag(value_out);
  if (rc == HYP_OK && clear && g_err_flag && *value_out) HYP_CUDA_TRY(cudaMemset(g_err_flag, 0, sizeof(int)));
  return rc;
}

int launch_gemm_tc(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                   cudaStream_t st, bool early) {
  if (M < 1 || N < 1 || K < 8 || act.K != K || w.K != K || M > act.rows || !g_err_flag) return HYP_EINVAL;
  if (w.rows != N || w.halves != (epi == EPI_SWIGLU_BF16 ? 2 : 1)) return HYP_EINVAL;
  if (act.f16 != w.f16) return HYP_EINVAL;  // one instruction takes both operands in the same 16-bit type
  // the epilogues write 16 bytes per lane at out + row * ldo + col (col a multiple of 16)
  const int row_align = (epi == EPI_RESID_F32 || epi == EPI_STORE_F32) ? 4 : 8;
  if (!out || ((uintptr_t)out & 15) != 0 || ldo < N || ldo % row_align) return HYP_EINVAL;
  switch (epi) {
    case EPI_STORE_BF16: return launch_epi<EPI_STORE_BF16>(act, w, M, N, K, out, ldo, st, early);
    case EPI_RESID_F32: return launch_epi<EPI_RESID_F32>(act, w, M, N, K, out, ldo, st, early);
    case EPI_SWIGLU_BF16: return launch_epi<EPI_SWIGLU_BF16>(act, w, M, N, K, out, ldo, st, early);
    case EPI_STORE_F32: return launch_epi<EPI_STORE_F32>(act, w, M, N, K, out, ldo, st, early);
    default: return HYP_EINVAL;
  }
}

}  // namespace hyp
