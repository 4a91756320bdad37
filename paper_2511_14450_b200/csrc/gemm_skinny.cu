// Weight-streaming projection for M <= 32 rows (decode): out[m, n] = sum_k a[m, k] * w[n, k].
//
// The weight matrix is read exactly once with 128-bit loads straight into mma.sync fragments
// (weights are the 16-row operand, the <= 32 activation rows the 8-wide operand), so the kernel
// stays HBM-bound up to batch 32 instead of running out of fp32 FMA issue slots.  The contraction
// index inside one instruction is permuted (each thread owns 16 consecutive k of its row); the
// same permutation is applied to the activation fragment, which leaves the sum unchanged.
//
// One CTA feeds two 16-row operand tiles (32 adjacent rows; or 16 gate rows and the matching 16 up
// rows for the SwiGLU epilogue; or, for matrices with few rows, the same 16 rows at two k slices so
// that twice as many CTAs are in flight) and splits K across its 8 warps in interleaved steps;
// partial sums meet in shared memory and the epilogue is applied once.
#include "common.cuh"
#include "hyperion.h"

namespace hyp {

constexpr int SK_WARPS = 8;
constexpr int SK_STEP = 64;  // k per tile and warp step

// How a CTA's two 16-row operand tiles are used.
enum SkMode : int {
  SK_ROWS32 = 0,  // two adjacent row tiles: 32 output columns per CTA
  SK_SWIGLU = 1,  // 16 gate rows and the 16 matching up rows: 16 output columns per CTA
  SK_KPAIR = 2    // the same 16 rows at two consecutive 64-wide k slices: 16 output columns per CTA,
                  // twice as many CTAs - for matrices with few rows (N <= 8192)
};

template <int NB, bool KPAIR>
struct Frags {
  uint4 a[2][2][2];               // [tile][row g / g+8][k half]
  uint4 b[KPAIR ? 2 : 1][NB][2];  // [tile (only if the tiles sit at different k)][n tile][k half]
};

// k: step start (row pointers already include the thread's 16 t offset and the tile's k offset);
// k_room[i]: how far tile i of this thread may reach (only read when !FULL).
template <int NB, bool KPAIR, bool FULL>
__device__ __forceinline__ void load_frags(Frags<NB, KPAIR>& f, const __nv_bfloat16* const (&wrow)[2][2],
                                           const __nv_bfloat16* const (&arow)[2][NB], const bool (&a_ok)[NB], int k,
                                           const int (&k_room)[2]) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int kk = k + 8 * h;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const bool ok = FULL || (kk + 8 <= k_room[i]);
#pragma unroll
      for (int r = 0; r < 2; ++r) f.a[i][r][h] = ok ? ldg_stream(wrow[i][r] + kk) : make_uint4(0, 0, 0, 0);
      if (i == 0 || KPAIR) {
#pragma unroll
        for (int j = 0; j < NB; ++j)
          f.b[i][j][h] = (ok && a_ok[j]) ? *reinterpret_cast<const uint4*>(arow[i][j] + kk) : make_uint4(0, 0, 0, 0);
      }
    }
  }
}

template <int NB, bool KPAIR>
__device__ __forceinline__ void mma_frags(float (&acc)[2][NB][4], const Frags<NB, KPAIR>& f) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint4 x = f.a[i][0][h], y = f.a[i][1][h];
#pragma unroll
      for (int j = 0; j < NB; ++j) {
        const uint4 b = f.b[KPAIR ? i : 0][j][h];
        mma_bf16_16816(acc[i][j], x.x, y.x, x.y, y.y, b.x, b.y);
        mma_bf16_16816(acc[i][j], x.z, y.z, x.w, y.w, b.z, b.w);
      }
    }
  }
}

template <int NB, int EPI, int MODE>
__global__ void __launch_bounds__(SK_WARPS * 32)
gemm_skinny_kernel(const __nv_bfloat16* __restrict__ a, int lda, const __nv_bfloat16* __restrict__ w, int N,
                   int K, int M, void* __restrict__ out, int ldo) {
  constexpr bool SWIGLU = MODE == SK_SWIGLU, KPAIR = MODE == SK_KPAIR;
  static_assert((EPI == EPI_SWIGLU_BF16) == SWIGLU, "the SwiGLU epilogue needs the gate/up tile pairing");
  constexpr int OUT_ROWS = MODE == SK_ROWS32 ? 32 : 16;
  constexpr int WSTEP = KPAIR ? 2 * SK_STEP : SK_STEP;  // k covered by one warp step
  __shared__ float red[SK_WARPS][32][NB * 8 + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int r0 = blockIdx.x * OUT_ROWS;
  const int n_w_rows = SWIGLU ? 2 * N : N;

  // row pointers (rows past the end are clamped for loading and never stored)
  const __nv_bfloat16* wrow[2][2];
  int k_room[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int koff = KPAIR ? i * SK_STEP : 0;
    k_room[i] = K - 16 * t - koff;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      int row = SWIGLU ? (i * N + r0 + 8 * r + g) : KPAIR ? (r0 + 8 * r + g) : (r0 + 16 * i + 8 * r + g);
      if (SWIGLU && r0 + 8 * r + g >= N) row = i * N + N - 1;
      if (row >= n_w_rows) row = n_w_rows - 1;
      wrow[i][r] = w + (size_t)row * K + 16 * t + koff;
    }
  }
  const __nv_bfloat16* arow[2][NB];
  bool a_ok[NB];
#pragma unroll
  for (int j = 0; j < NB; ++j) {
    const int m = 8 * j + g;
    a_ok[j] = m < M;
#pragma unroll
    for (int i = 0; i < 2; ++i) arow[i][j] = a + (size_t)(a_ok[j] ? m : 0) * lda + 16 * t + (KPAIR ? i * SK_STEP : 0);
  }

  float acc[2][NB][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < NB; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[i][j][c] = 0.f;

  const int full_steps = K / WSTEP;
  Frags<NB, KPAIR> cur, nxt;
  int s = warp;
  if (s < full_steps) load_frags<NB, KPAIR, true>(cur, wrow, arow, a_ok, s * WSTEP, k_room);
  while (s < full_steps) {
    const int sn = s + SK_WARPS;
    if (sn < full_steps) load_frags<NB, KPAIR, true>(nxt, wrow, arow, a_ok, sn * WSTEP, k_room);
    mma_frags<NB, KPAIR>(acc, cur);
    cur = nxt;
    s = sn;
  }
  // ragged K tail (K is a multiple of 8): one predicated step, taken by the warp whose turn it is
  if ((K % WSTEP) != 0 && (full_steps % SK_WARPS) == warp) {
    Frags<NB, KPAIR> tl;
    load_frags<NB, KPAIR, false>(tl, wrow, arow, a_ok, full_steps * WSTEP, k_room);
    mma_frags<NB, KPAIR>(acc, tl);
  }

  // cross-warp reduction through shared memory
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < NB; ++j) {
      red[warp][16 * i + g][8 * j + 2 * t] = acc[i][j][0];
      red[warp][16 * i + g][8 * j + 2 * t + 1] = acc[i][j][1];
      red[warp][16 * i + g + 8][8 * j + 2 * t] = acc[i][j][2];
      red[warp][16 * i + g + 8][8 * j + 2 * t + 1] = acc[i][j][3];
    }
  __syncthreads();

  for (int e = threadIdx.x; e < OUT_ROWS * NB * 8; e += SK_WARPS * 32) {
    const int r = e % OUT_ROWS, m = e / OUT_ROWS;  // r fastest: consecutive threads -> consecutive n
    const int n = r0 + r;
    if (m >= M || n >= N) continue;
    float v = 0.f, v2 = 0.f;
#pragma unroll
    for (int ww = 0; ww < SK_WARPS; ++ww) {
      v += red[ww][r][m];
      if (MODE != SK_ROWS32) v2 += red[ww][16 + r][m];
    }
    if (KPAIR) v += v2;  // the second tile held the other k slices of the same rows
    const size_t o = (size_t)m * ldo + n;
    if (EPI == EPI_STORE_BF16) {
      reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(v);
    } else if (EPI == EPI_RESID_F32) {
      reinterpret_cast<float*>(out)[o] += v;
    } else if (EPI == EPI_SWIGLU_BF16) {
      reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(v / (1.f + __expf(-v)) * v2);
    } else {
      reinterpret_cast<float*>(out)[o] = v;
    }
  }
}

template <int NB, int EPI>
static void launch_mode(bool kpair, const __nv_bfloat16* a, int lda, const __nv_bfloat16* w, int N, int K, int M,
                        void* out, int ldo, cudaStream_t st) {
  const dim3 block(SK_WARPS * 32);
  if (kpair)
    gemm_skinny_kernel<NB, EPI, SK_KPAIR><<<(N + 15) / 16, block, 0, st>>>(a, lda, w, N, K, M, out, ldo);
  else
    gemm_skinny_kernel<NB, EPI, SK_ROWS32><<<(N + 31) / 32, block, 0, st>>>(a, lda, w, N, K, M, out, ldo);
}

template <int NB>
static int launch_nb(const __nv_bfloat16* a, int lda, const __nv_bfloat16* w, int N, int K, int M, int epi,
                     void* out, int ldo, cudaStream_t st) {
  const bool kpair = N <= 8192 && K >= 2 * SK_STEP * SK_WARPS;  // few rows: trade rows per CTA for more CTAs
  switch (epi) {
    case EPI_STORE_BF16: launch_mode<NB, EPI_STORE_BF16>(kpair, a, lda, w, N, K, M, out, ldo, st); break;
    case EPI_RESID_F32: launch_mode<NB, EPI_RESID_F32>(kpair, a, lda, w, N, K, M, out, ldo, st); break;
    case EPI_STORE_F32: launch_mode<NB, EPI_STORE_F32>(kpair, a, lda, w, N, K, M, out, ldo, st); break;
    case EPI_SWIGLU_BF16:
      gemm_skinny_kernel<NB, EPI_SWIGLU_BF16, SK_SWIGLU><<<(N + 15) / 16, dim3(SK_WARPS * 32), 0, st>>>(a, lda, w, N, K,
                                                                                                      M, out, ldo);
      break;
    default:
      return HYP_EINVAL;
  }
  return 1;
}

// N = output columns (for SwiGLU: F, with w holding 2F rows).  K multiple of 8, 1 <= M <= 32.
int launch_gemm_skinny(const __nv_bfloat16* a, int lda, const __nv_bfloat16* w, int N, int K, int M, int epi,
                       void* out, int ldo, cudaStream_t st) {
  if (M < 1 || M > 32 || (K % 8) != 0 || (lda % 8) != 0) return HYP_EINVAL;
  switch ((M + 7) / 8) {
    case 1: return launch_nb<1>(a, lda, w, N, K, M, epi, out, ldo, st);
    case 2: return launch_nb<2>(a, lda, w, N, K, M, epi, out, ldo, st);
    case 3: return launch_nb<3>(a, lda, w, N, K, M, epi, out, ldo, st);
    default: return launch_nb<4>(a, lda, w, N, K, M, epi, out, ldo, st);
  }
}

}  // namespace hyp
