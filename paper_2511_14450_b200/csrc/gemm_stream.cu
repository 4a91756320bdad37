// Weight-streaming projection for M <= 32 rows (decode): out[m, n] (+)= sum_k a[m, k] * w[n, k].
//
// HBM-bound: every weight byte is read exactly once.  A CTA owns 16 (or 2 x 16) weight rows; its four
// warps take the 64-wide k-blocks round-robin.  Each warp runs its own TMA ring: lane 0 keeps a run of
// k-blocks (weight tile + the matching slice of the <= 32 activation rows, 128-byte swizzle) in flight
// into the warp's shared-memory slots, the warp reads a landed slot back with ldmatrix, runs
// mma.sync.m16n8k16 (weights are the 16-row operand, tokens the 8-wide operand) and lane 0 refills the
// slot at once.  The bytes in flight are set by the ring depth, not by registers or occupancy, a slot
// only ever has one waiter, and four lanes per CTA issue copies in parallel.  Batch 8-32 costs no more
// issue slots than batch 1.  Each warp keeps a partial sum over its k-blocks; the warps meet in shared
// memory and the epilogue (bf16 store, residual add, SiLU(gate) * up, fp32 store) is applied once.
// Every mbarrier wait is bounded.
#include "gemm_tc.cuh"
#include "hyperion.h"
#include "sm100_common.cuh"

namespace hyp {

namespace {

constexpr int GS_BK = 64;
constexpr int GS_WARPS = 4;
constexpr int GS_THREADS = 32 * GS_WARPS;
constexpr int GS_MAX_SLOTS = 16;  // ring slots per warp
constexpr int W_TILE_BYTES = 16 * GS_BK * 2;  // 16 rows x 64 k
constexpr int A_TILE_BYTES = 8 * GS_BK * 2;   // 8 tokens x 64 k

__device__ __forceinline__ uint32_t sw_off(int r, int c) {  // 128-byte rows, 16-byte chunks XOR-swizzled by the row
  return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
}
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

// TILES = 1: 16 output columns per CTA.  TILES = 2: 32 adjacent columns, or (SwiGLU) 16 gate rows and
// the 16 matching up rows.  S = ring slots per warp.
template <int NB, int EPI, int TILES, bool F16>
__global__ void __launch_bounds__(GS_THREADS)
gemm_stream_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_a, int N, int K,
                   int M, void* __restrict__ out, int ldo, int S, int* __restrict__ err) {
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  static_assert(!SWIGLU || TILES == 2, "SwiGLU pairs a gate tile with an up tile");
  constexpr int OUT_COLS = (TILES == 2 && !SWIGLU) ? 32 : 16;
  constexpr int STAGE_BYTES = TILES * W_TILE_BYTES + NB * A_TILE_BYTES;
  extern __shared__ uint8_t gs_smem_raw[];
  __shared__ float red[GS_WARPS][16 * TILES][NB * 8 + 1];
  __shared__ uint64_t bars[GS_WARPS * GS_MAX_SLOTS];
  const uint32_t base = (smem_u32(gs_smem_raw) + 1023u) & ~1023u;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * OUT_COLS;
  const int KB = (K + GS_BK - 1) / GS_BK;
  const uint32_t my_bars = smem_u32(bars) + 8u * (warp * GS_MAX_SLOTS);
  const uint32_t my_ring = base + (uint32_t)(warp * S) * STAGE_BYTES;
  const int row1 = N + n0;  // SwiGLU: the up rows that pair with this CTA's gate rows

  // one k-block into one of this warp's slots (lane 0 only).  CTAs walk K from staggered starting points
  // (a fixed rotation per CTA, so the summation order stays reproducible): otherwise every resident CTA
  // would ask for the same activation slice and the same column offsets of its rows at the same moment.
  const int rot = (int)((blockIdx.x * 13u) % (unsigned)KB);
  // weights: never written by any kernel, may be fetched before the predecessor has finished
  auto issue_w = [&](int kb_logical, int slot) {
    int kb = kb_logical + rot;
    if (kb >= KB) kb -= KB;
    const uint32_t dst = my_ring + slot * STAGE_BYTES, bar = my_bars + 8u * slot;
    mbar_expect_tx(bar, STAGE_BYTES);
    tma_load_2d(dst, &tm_w, kb * GS_BK, n0, bar);  // 16 rows, or one 32-row box
    if (SWIGLU) tma_load_2d(dst + W_TILE_BYTES, &tm_w, kb * GS_BK, row1, bar);
  };
  // activations: produced by the predecessor
  auto issue_a = [&](int kb_logical, int slot) {
    int kb = kb_logical + rot;
    if (kb >= KB) kb -= KB;
    tma_load_2d(my_ring + slot * STAGE_BYTES + TILES * W_TILE_BYTES, &tm_a, kb * GS_BK, 0, my_bars + 8u * slot);
  };

  if (lane == 0) {
    for (int sl = 0; sl < S; ++sl) mbar_init(my_bars + 8u * sl, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int sl = 0; sl < S; ++sl)
      if (warp + GS_WARPS * sl < KB) issue_w(warp + GS_WARPS * sl, sl);
  }
  pdl_wait();
  if (lane == 0) {
    for (int sl = 0; sl < S; ++sl)
      if (warp + GS_WARPS * sl < KB) issue_a(warp + GS_WARPS * sl, sl);
  }
  __syncwarp();

  float acc[TILES][NB][4];
#pragma unroll
  for (int i = 0; i < TILES; ++i)
#pragma unroll
    for (int j = 0; j < NB; ++j) acc[i][j][0] = acc[i][j][1] = acc[i][j][2] = acc[i][j][3] = 0.f;

  bool ok = true;
  int slot = 0;
  uint32_t phase = 0;
  for (int kb = warp; kb < KB; kb += GS_WARPS) {
    if (!mbar_wait(my_bars + 8u * slot, phase, nullptr)) { ok = false; break; }
    const uint32_t sw = my_ring + slot * STAGE_BYTES, sa = sw + TILES * W_TILE_BYTES;
#pragma unroll
    for (int kp = 0; kp < 2; ++kp) {  // pairs of 16-wide k steps
      uint32_t bf[NB][4];              // [n tile]: b0, b1 of step 2kp, then of step 2kp + 1
#pragma unroll
      for (int j = 0; j < NB; ++j)
        ldsm4(sa + sw_off(8 * j + (lane & 7), 4 * kp + (lane >> 3)), bf[j][0], bf[j][1], bf[j][2], bf[j][3]);
#pragma unroll
      for (int i = 0; i < TILES; ++i) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int ks = 2 * kp + h;
          uint32_t a0, a1, a2, a3;
          ldsm4(sw + i * W_TILE_BYTES + sw_off((lane & 7) + (((lane >> 3) & 1) << 3), 2 * ks + (lane >> 4)), a0, a1, a2, a3);
#pragma unroll
          for (int j = 0; j < NB; ++j) {
            if (F16)
              mma_f16_16816(acc[i][j], a0, a1, a2, a3, bf[j][2 * h], bf[j][2 * h + 1]);
            else
              mma_bf16_16816(acc[i][j], a0, a1, a2, a3, bf[j][2 * h], bf[j][2 * h + 1]);
          }
        }
      }
    }
    // Every ldmatrix result above has been consumed by an MMA that is already issued, so after this
    // warp barrier no lane still reads the slot and lane 0 may hand it back to the copy engine.
    __syncwarp();
    if (lane == 0) {
      const int next = kb + GS_WARPS * S;
      if (next < KB) {
        issue_w(next, slot);
        issue_a(next, slot);
      }
    }
    if (++slot == S) { slot = 0; phase ^= 1u; }
  }
  pdl_trigger();  // this warp has no more copies to issue: the successor may begin its own prefetch
  if (!ok) {
    // a copy never landed: record it and let whatever is still in flight arrive (bounded) before leaving
    if (lane == 0) atomicCAS(err, 0, 4);
    for (int sl = 0; sl < S; ++sl) mbar_wait(my_bars + 8u * sl, 0, nullptr), mbar_wait(my_bars + 8u * sl, 1, nullptr);
  }
  {
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int i = 0; i < TILES; ++i)
#pragma unroll
      for (int j = 0; j < NB; ++j) {
        red[warp][16 * i + g][8 * j + 2 * t] = acc[i][j][0];
        red[warp][16 * i + g][8 * j + 2 * t + 1] = acc[i][j][1];
        red[warp][16 * i + g + 8][8 * j + 2 * t] = acc[i][j][2];
        red[warp][16 * i + g + 8][8 * j + 2 * t + 1] = acc[i][j][3];
      }
  }
  __syncthreads();

  for (int e = threadIdx.x; e < OUT_COLS * NB * 8; e += GS_THREADS) {
    const int r = e % OUT_COLS, m = e / OUT_COLS;  // r fastest: consecutive threads -> consecutive n
    const int n = n0 + r;
    if (m >= M || n >= N) continue;
    float v = 0.f, v2 = 0.f;
#pragma unroll
    for (int ww = 0; ww < GS_WARPS; ++ww) {
      v += red[ww][r][m];
      if (SWIGLU) v2 += red[ww][16 + r][m];
    }
    const size_t o = (size_t)m * ldo + n;
    if (EPI == EPI_STORE_BF16 || EPI == EPI_SWIGLU_BF16) {
      // 16-bit results take the operands' type
      const float y = EPI == EPI_SWIGLU_BF16 ? v / (1.f + __expf(-v)) * v2 : v;
      if (F16)
        reinterpret_cast<__half*>(out)[o] = __float2half_rn(fminf(fmaxf(y, -65504.f), 65504.f));
      else
        reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(y);
    } else if (EPI == EPI_RESID_F32) {
      reinterpret_cast<float*>(out)[o] += v;
    } else {
      reinterpret_cast<float*>(out)[o] = v;
    }
  }
}

template <int NB, int EPI, int TILES, bool F16>
int launch_cfg(const TcAct& act, const TcWeight& w, int M, int N, int K, void* out, int ldo, cudaStream_t st) {
  static bool configured = false;
  static int num_sms = 0;
  constexpr int STAGE_BYTES = TILES * W_TILE_BYTES + NB * A_TILE_BYTES;
  constexpr int MAX_DYN = GS_WARPS * GS_MAX_SLOTS * STAGE_BYTES + 1024 > 200 * 1024 ? 200 * 1024
                                                                                       : GS_WARPS * GS_MAX_SLOTS * STAGE_BYTES + 1024;
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(gemm_stream_kernel<NB, EPI, TILES, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_DYN));
    // several CTAs per SM share the ring space: ask for the largest shared-memory carve-out
    HYP_CUDA_TRY(cudaFuncSetAttribute(gemm_stream_kernel<NB, EPI, TILES, F16>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                      cudaSharedmemCarveoutMaxShared));
    int dev = 0;
    HYP_CUDA_TRY(cudaGetDevice(&dev));
    HYP_CUDA_TRY(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    configured = true;
  }
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  constexpr int OUT_COLS = (TILES == 2 && !SWIGLU) ? 32 : 16;
  const int n_ctas = (N + OUT_COLS - 1) / OUT_COLS;
  // Ring depth (slots per warp).  Measured on B200: throughput peaks when roughly 28 k-block copies (and
  // no more than ~110 KB) are in flight per SM and falls off sharply beyond that (3 slots at 3.2 CTAs/SM run at half the speed of 2),
  // so the depth follows from how many CTAs share an SM; two slots are the floor (one slot exposes the
  // full memory latency), four the ceiling.
  double ctas_per_sm = (double)n_ctas / num_sms;
  if (ctas_per_sm > 5.0) ctas_per_sm = 5.0;
  int slots = (int)(28.0 / (GS_WARPS * ctas_per_sm));
  const int by_bytes = (int)(110.0 * 1024 / (GS_WARPS * ctas_per_sm * STAGE_BYTES));  // and ~110 KB in flight per SM
  if (by_bytes < slots) slots = by_bytes;
  if (slots > 4) slots = 4;
  if (slots < 2) slots = 2;
  while (slots > 1 && GS_WARPS * slots * STAGE_BYTES + 1024 > MAX_DYN) --slots;
  const int smem = GS_WARPS * slots * STAGE_BYTES + 1024;
  HYP_CUDA_TRY(launch_pdl(gemm_stream_kernel<NB, EPI, TILES, F16>, dim3(n_ctas), dim3(GS_THREADS), (size_t)smem, st,
                          (TILES == 2 && !SWIGLU) ? w.map_small[1] : w.map_small[0], act.map_small[NB - 1], N, K, M, out,
                          ldo, slots, tc_err_flag_ptr()));
  return 1;
}

template <int NB, bool F16>
int launch_nb(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo, cudaStream_t st) {
  const bool wide = N > 8192;  // many rows: 32 columns per CTA keep the CTA count within one resident wave
  switch (epi) {
    case EPI_STORE_BF16:
      return wide ? launch_cfg<NB, EPI_STORE_BF16, 2, F16>(act, w, M, N, K, out, ldo, st)
                  : launch_cfg<NB, EPI_STORE_BF16, 1, F16>(act, w, M, N, K, out, ldo, st);
    case EPI_RESID_F32:
      return wide ? launch_cfg<NB, EPI_RESID_F32, 2, F16>(act, w, M, N, K, out, ldo, st)
                  : launch_cfg<NB, EPI_RESID_F32, 1, F16>(act, w, M, N, K, out, ldo, st);
    case EPI_STORE_F32:
      return wide ? launch_cfg<NB, EPI_STORE_F32, 2, F16>(act, w, M, N, K, out, ldo, st)
                  : launch_cfg<NB, EPI_STORE_F32, 1, F16>(act, w, M, N, K, out, ldo, st);
    case EPI_SWIGLU_BF16: return launch_cfg<NB, EPI_SWIGLU_BF16, 2, F16>(act, w, M, N, K, out, ldo, st);
    default: return HYP_EINVAL;
  }
}

template <bool F16>
int launch_type(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo, cudaStream_t st) {
  switch ((M + 7) / 8) {
    case 1: return launch_nb<1, F16>(act, w, M, N, K, epi, out, ldo, st);
    case 2: return launch_nb<2, F16>(act, w, M, N, K, epi, out, ldo, st);
    case 3: return launch_nb<3, F16>(act, w, M, N, K, epi, out, ldo, st);
    default: return launch_nb<4, F16>(act, w, M, N, K, epi, out, ldo, st);
  }
}

}  // namespace

int launch_gemm_stream(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                       cudaStream_t st) {
  if (M < 1 || M > 32 || N < 1 || K < 8 || act.K != K || w.K != K || !tc_err_flag_ptr()) return HYP_EINVAL;
  if (act.f16 != w.f16) return HYP_EINVAL;  // one instruction takes both operands in the same 16-bit type
  return act.f16 ? launch_type<true>(act, w, M, N, K, epi, out, ldo, st)
                 : launch_type<false>(act, w, M, N, K, epi, out, ldo, st);
}

}  // namespace hyp
