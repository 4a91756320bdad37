// Projection for a few dozen rows (decode batches of 9-128 tokens): out[m, n] (+)= sum_k a[m, k] * w[n, k] with
// the operands swapped on the tensor cores.
//
// The weight-streaming kernel re-reads the activations from L2 once per 16- or 32-row weight strip; from 16
// tokens on those reads outweigh the weights and L2 -> SM traffic becomes the bound.  Here a CTA owns 128 weight
// rows as the M operand of tcgen05.mma (a 16 KB tile per k-block, eight packed 2 KB strips) and the tokens are
// the N operand (16-128 rows, 2-16 KB per k-block): activation bytes per weight byte drop to NT / 128.  The
// accumulator is 128 lanes (weight rows) x NT columns (tokens) of tensor memory; SwiGLU keeps a second one for
// the matching up rows, so gate and up meet lane by lane in the epilogue.
// There are only N / 128 such tiles, so K is split over the CTAs of a thread-block cluster (<= 8): each takes a
// contiguous share of the k-blocks; the non-leaders copy their accumulators to shared memory and the leader adds
// them in rank order through distributed shared memory before the epilogue: deterministic, no atomics.
//   warp 0   one lane issues TMA loads into a ring (weights before the dependency wait, activations after);
//   warp 1   one lane issues tcgen05.mma (128 x NT x 16, kind::f16) and commits stages / the accumulator;
//   warps 2-5  read the accumulator (lane = weight row) and write out[token][row]: for a fixed token the 32 lanes
//            of a warp store 32 consecutive columns.
// Every mbarrier wait is bounded; the cluster barriers are reached by every thread of every CTA.
#include <cuda.h>

#include "gemm_tc.cuh"
#include "hyperion.h"
#include "tcgen05.cuh"

namespace hyp {

int& gemm_swap_min_rows() {
  static int v = 9;
  return v;
}
int& gemm_swap_max_rows() {
  static int v = 128;
  return v;
}


int& gemm_swap_epilogues() {
  static int v = (1 << EPI_STORE_BF16) | (1 << EPI_STORE_F32);
  return v;
}

namespace {

constexpr int SW_ROWS = 128, SW_BK = 64, SW_THREADS = 192, SW_MAX_STAGES = 8;
constexpr int SW_A_BYTES = SW_ROWS * SW_BK * 2;

struct SwapArgs {
  int M, N, K, up_tile0, ldo;
  int NT;       // token tile: 16, 32, 64 or 128 (>= M)
  int stages;   // ring depth
  int ksplit;   // cluster size = K shares
  int tmem_cols;
  uint32_t idesc;
  void* out;
  int* err;
};

template <int EPI>
__global__ void __launch_bounds__(SW_THREADS)
gemm_swap_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_a, SwapArgs p) {
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  constexpr int A_TILES = SWIGLU ? 2 : 1;
  extern __shared__ uint8_t sw_smem[];
  __shared__ uint64_t bars[2 * SW_MAX_STAGES + 1];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_word;
  const uint32_t base = (smem_u32(sw_smem) + 1023u) & ~1023u;
  float* dump = reinterpret_cast<float*>(sw_smem + (base - smem_u32(sw_smem)));  // accumulator copy, [col][128 rows]
  const int NT = p.NT, S = p.stages;
  const int B_BYTES = NT * SW_BK * 2;
  const int STAGE_BYTES = A_TILES * SW_A_BYTES + B_BYTES;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (SW_MAX_STAGES + s); };
  const uint32_t tfull_bar = bar0 + 8u * (2 * SW_MAX_STAGES);
  volatile int* abort_flag = &abort_word;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = p.ksplit > 1 ? (int)(blockIdx.x % (unsigned)p.ksplit) : 0;
  const int tile = p.ksplit > 1 ? (int)(blockIdx.x / (unsigned)p.ksplit) : (int)blockIdx.x;
  const int n0 = tile * SW_ROWS;
  const int KB = (p.K + SW_BK - 1) / SW_BK;
  const int kb0 = (int)((long)KB * rank / p.ksplit), kb1 = (int)((long)KB * (rank + 1) / p.ksplit);

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(tfull_bar, 1);
    abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(p.tmem_cols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  pdl_trigger();

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer ----------------
      auto load_w = [&](int kb, int stage) {
        const uint32_t sa = base + stage * STAGE_BYTES;
        mbar_expect_tx(full_bar(stage), STAGE_BYTES);
        tma_load_4d(sa, &tm_w, 0, 0, kb, tile * 8, full_bar(stage));
        if (SWIGLU) tma_load_4d(sa + SW_A_BYTES, &tm_w, 0, 0, kb, p.up_tile0 + tile * 8, full_bar(stage));
      };
      auto load_a = [&](int kb, int stage) {
        tma_load_2d(base + stage * STAGE_BYTES + A_TILES * SW_A_BYTES, &tm_a, kb * SW_BK, 0, full_bar(stage));
      };
      // the ring starts empty: weights of the first stages go out before the wait, their activations after it
      const int n_first = min(S, kb1 - kb0);
      for (int i = 0; i < n_first; ++i) load_w(kb0 + i, i);
      pdl_wait();
      for (int i = 0; i < n_first; ++i) load_a(kb0 + i, i);
      int stage = n_first == S ? 0 : n_first;
      uint32_t phase = n_first == S ? 1 : 0;  // parity of the "empty" phase waited on next
      bool ok = true;
      for (int kb = kb0 + n_first; kb < kb1; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1, abort_flag)) { ok = false; break; }
        load_w(kb, stage);
        load_a(kb, stage);
        if (++stage == S) { stage = 0; phase ^= 1; }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(p.err, 0, 9);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_TILES * SW_A_BYTES;
        const uint64_t da = smem_desc(sa), db = smem_desc(sb);
#pragma unroll
        for (int k = 0; k < SW_BK / 16; ++k) {
          const uint32_t accum = (kb > kb0 || k > 0) ? 1u : 0u;
          tc_mma(tmem_base, da + (uint64_t)(k * 32 / 16), db + (uint64_t)(k * 32 / 16), p.idesc, accum);
          if (SWIGLU)
            tc_mma(tmem_base + (uint32_t)NT, smem_desc(sa + SW_A_BYTES) + (uint64_t)(k * 32 / 16), db + (uint64_t)(k * 32 / 16),
                   p.idesc, accum);
        }
        tc_commit(empty_bar(stage));
        if (++stage == S) { stage = 0; phase ^= 1; }
      }
      if (ok) {
        tc_commit(tfull_bar);
      } else {
        *abort_flag = 1;
        atomicCAS(p.err, 0, 10);
      }
    }
  }

  // ---------------- epilogue warps ----------------
  const int q = warp & 3;  // tensor-memory lane quarter this warp may read
  const int row = 32 * q + lane;
  const uint32_t t0 = tmem_base + ((uint32_t)(32 * q) << 16);
  bool acc_ok = true;
  if (warp >= 2) {
    pdl_wait();  // the output buffer may still be in use by the predecessor
    acc_ok = mbar_wait(tfull_bar, 0, abort_flag);
    tc_fence_after();
    if (!acc_ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(p.err, 0, 11);
    }
    if (acc_ok && rank != 0) {
      // a K share that is not the leader's: leave the accumulator where the leader can read it
      for (int c = 0; c < NT && c < p.M; c += 16) {
        uint32_t v[16], v2[16];
        tmem_ld16(t0 + c, v);
        if (SWIGLU) tmem_ld16(t0 + NT + c, v2);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          dump[(c + i) * SW_ROWS + row] = __uint_as_float(v[i]);
          if (SWIGLU) dump[(NT + c + i) * SW_ROWS + row] = __uint_as_float(v2[i]);
        }
      }
    }
  }
  if (p.ksplit > 1) {
    __syncthreads();
    cluster_barrier();
  }
  if (warp >= 2 && rank == 0 && acc_ok) {
    const int n = n0 + row;
    const uint32_t dump_addr = smem_u32(dump);
    const bool f16 = (p.idesc & (1u << 7)) == 0;  // operand type bits of the instruction descriptor
    for (int c = 0; c < NT && c < p.M; c += 16) {
      uint32_t v[16], v2[16];
      tmem_ld16(t0 + c, v);
      if (SWIGLU) tmem_ld16(t0 + NT + c, v2);
      tmem_ld_wait();
      float a[16], b[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        a[i] = __uint_as_float(v[i]);
        b[i] = SWIGLU ? __uint_as_float(v2[i]) : 0.f;
      }
      for (int rr = 1; rr < p.ksplit; ++rr) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          a[i] += ld_cluster_f32(dump_addr + 4u * ((c + i) * SW_ROWS + row), rr);
          if (SWIGLU) b[i] += ld_cluster_f32(dump_addr + 4u * ((NT + c + i) * SW_ROWS + row), rr);
        }
      }
      if (n < p.N) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int m = c + i;
          if (m >= p.M) break;
          const size_t o = (size_t)m * p.ldo + n;
          if (EPI == EPI_STORE_BF16 || EPI == EPI_SWIGLU_BF16) {
            const float y = SWIGLU ? a[i] / (1.f + __expf(-a[i])) * b[i] : a[i];
            if (f16)
              reinterpret_cast<__half*>(p.out)[o] = __float2half_rn(fminf(fmaxf(y, -65504.f), 65504.f));
            else
              reinterpret_cast<__nv_bfloat16*>(p.out)[o] = __float2bfloat16_rn(y);
          } else if (EPI == EPI_RESID_F32) {
            reinterpret_cast<float*>(p.out)[o] += a[i];
          } else {
            reinterpret_cast<float*>(p.out)[o] = a[i];
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (p.ksplit > 1) cluster_barrier();  // nobody leaves while the leader may still read its accumulator copy
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols));
  }
}

template <int EPI>
int launch_epi(const TcAct& act, const TcWeight& w, int M, int N, int K, void* out, int ldo, cudaStream_t st, bool early) {
  static bool configured = false;
  static int num_sms = 0, smem_per_sm = 0;
  constexpr int A_TILES = EPI == EPI_SWIGLU_BF16 ? 2 : 1;
  constexpr int MAX_DYN = 200 * 1024;
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(gemm_swap_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_DYN));
    int dev = 0;
    HYP_CUDA_TRY(cudaGetDevice(&dev));
    HYP_CUDA_TRY(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    HYP_CUDA_TRY(cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev));
    configured = true;
  }
  SwapArgs p;
  p.M = M; p.N = N; p.K = K; p.up_tile0 = w.N16p; p.ldo = ldo; p.out = out; p.err = tc_err_flag_ptr();
  p.NT = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128;
  const CUtensorMap& amap = p.NT == 128 ? act.map : act.map_small[p.NT == 16 ? 0 : p.NT == 32 ? 1 : 2];
  const int tiles = (N + SW_ROWS - 1) / SW_ROWS;
  const int KB = (K + SW_BK - 1) / SW_BK;
  // K shares: about 1.5 CTAs per SM in all, two resident per SM, at least four k-blocks per share
  int ks = (3 * num_sms / 2 + tiles / 2) / tiles;
  if (ks > KB / 4) ks = KB / 4;
  if (ks > 8) ks = 8;
  if (ks < 1) ks = 1;
  p.ksplit = ks;
  const int stage_bytes = A_TILES * SW_A_BYTES + p.NT * SW_BK * 2;
  const int dump_bytes = ks > 1 ? A_TILES * p.NT * SW_ROWS * 4 : 0;
  const int budget = tiles * ks > num_sms ? (smem_per_sm / 2 - 3072) : MAX_DYN - 1024;  // two CTAs per SM when there are that many
  int stages = (budget - 1024) / stage_bytes;
  if (stages > SW_MAX_STAGES) stages = SW_MAX_STAGES;
  while (stages * stage_bytes < dump_bytes) ++stages;  // the accumulator copy reuses the ring
  if (stages < 2) stages = 2;
  if (stages > SW_MAX_STAGES || stages * stage_bytes + 1024 > MAX_DYN) return HYP_EINVAL;
  p.stages = stages;
  int cols = 32;
  while (cols < A_TILES * p.NT) cols <<= 1;
  p.tmem_cols = cols;
  p.idesc = (act.f16 ? (1u << 4) : ((1u << 4) | (1u << 7) | (1u << 10))) | ((uint32_t)(p.NT >> 3) << 17) |
            ((uint32_t)(SW_ROWS >> 4) << 24);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles * ks);
  cfg.blockDim = dim3(SW_THREADS);
  cfg.dynamicSmemBytes = (size_t)stages * stage_bytes + 1024;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (early && pdl_level() >= 1) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (ks > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = ks;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  HYP_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_swap_kernel<EPI>, w.map, amap, p));
  return 1;
}

}  // namespace

int launch_gemm_swap(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                     cudaStream_t st, bool early) {
  if (M < 1 || M > 128 || N < 1 || K < 8 || act.K != K || w.K != K || M > act.rows || !tc_err_flag_ptr()) return HYP_EINVAL;
  if (w.rows != N || w.halves != (epi == EPI_SWIGLU_BF16 ? 2 : 1)) return HYP_EINVAL;
  if (act.f16 != w.f16) return HYP_EINVAL;  // one instruction takes both operands in the same 16-bit type
  switch (epi) {
    case EPI_STORE_BF16: return launch_epi<EPI_STORE_BF16>(act, w, M, N, K, out, ldo, st, early);
    case EPI_RESID_F32: return launch_epi<EPI_RESID_F32>(act, w, M, N, K, out, ldo, st, early);
    case EPI_SWIGLU_BF16: return launch_epi<EPI_SWIGLU_BF16>(act, w, M, N, K, out, ldo, st, early);
    case EPI_STORE_F32: return launch_epi<EPI_STORE_F32>(act, w, M, N, K, out, ldo, st, early);
    default: return HYP_EINVAL;
  }
}

// Which kernel runs a projection of M rows (measured on B200, Phi-3-medium shapes, us for the four projections of a
// block: streaming kernel 127 at 8 rows, 146 at 16, 204 at 32; tile kernel + swapped kernel 137-147 from 9 to 64 rows):
//   up to 8 rows     the weight-streaming kernel (HBM-bound; its activation re-reads from L2 grow with the rows);
//   9 to 128 rows    the tcgen05 tile kernel - stream-K keeps every SM busy for the residual epilogues, gate/up has
//                    140 tiles - except the plain-store epilogues with too few 256-column tiles to fill the GPU
//                    (q/k/v: 30), which take the swapped-operand kernel (K split over clusters instead);
//   above            the tile kernels.
int launch_projection(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo, cudaStream_t st,
                      bool early) {
  if (M <= 8 && M < gemm_swap_min_rows()) return launch_gemm_stream(act, w, M, N, K, epi, out, ldo, st, early);
  const bool store = epi >= 0 && epi < 4 && ((gemm_swap_epilogues() >> epi) & 1);
  if (store && M >= gemm_swap_min_rows() && M <= gemm_swap_max_rows() && (N + 255) / 256 < 100)
    return launch_gemm_swap(act, w, M, N, K, epi, out, ldo, st, early);
  return launch_gemm_tc(act, w, M, N, K, epi, out, ldo, st, early);
}

}  // namespace hyp
