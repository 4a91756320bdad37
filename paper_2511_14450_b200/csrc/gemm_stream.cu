// Weight-streaming projection for M <= 8 rows (decode): out[m, n] (+)= sum_k a[m, k] * w[n, k].
//
// HBM-bound: every weight byte is read exactly once.  Weights are held packed (see gemm_tc.cuh): all k-blocks of
// a 16-row strip are contiguous, so a CTA, which owns one strip (or two), reads it as a sequential run of 4 KB
// bulk copies.  Its four warps take the copies round-robin.  Each warp runs its own ring: lane 0 keeps a run of
// copies in flight into the warp's shared-memory slots, the warp reads a landed slot back, runs
// mma.sync.m16n8k16 (weights are the 16-row operand, tokens the 8-wide operand) and lane 0 refills the slot at
// once.  The ring holds weights only and is sized to fill the SM's shared memory when every CTA of the grid is
// resident, so a CTA launched early (programmatic dependent launch) pulls a large part of its strip on chip while
// its predecessor drains.  A slot only ever has one waiter, and four lanes per CTA issue copies in parallel.
// Activations never touch shared memory: each lane reads the 16 bytes (8 consecutive k of one token) it needs
// for a pair of MMAs straight from global memory (L2-resident, written by the predecessor), one copy ahead.  The
// MMA's sixteen k slots are assigned to those k so that a lane's 16 bytes are exactly its fragment entries:
// slots {2t, 2t+1, 2t+8, 2t+9} of the first MMA of a pair hold k = 8t .. 8t+3, the same slots of the second hold
// 8t+4 .. 8t+7 (t = lane % 4); the weight fragments are read from shared memory with the same assignment (two
// 128-bit loads per pair), which a dot product does not notice.
// Each warp keeps a partial sum over its k-blocks; the warps meet in shared memory and the epilogue (16-bit store,
// residual add, SiLU(gate) * up, fp32 store) is applied once.  Every mbarrier wait is bounded.
#include "gemm_tc.cuh"
#include "hyperion.h"
#include "sm100_common.cuh"

namespace hyp {

int& gemm_stream_slots_override() {
  static int v = 0;
  return v;
}
int& gemm_stream_rotation() {
  static int v = 13;
  return v;
}
int& gemm_stream_act_depth() {  // copies ahead that a warp's activation fragments are fetched; 0 = built-in choice
  static int v = 0;
  return v;
}
int& gemm_stream_act_tma() {  // 1 (default): activations ride into the ring by TMA where the operand allows it
  static int v = 1;
  return v;
}
int& gemm_stream_wait_limit_us() {
  static int v = 0;
  return v;
}
int& gemm_stream_withhold_next() {
  static int v = 0;
  return v;
}

namespace {

constexpr int GS_CH = 2;  // k-blocks per weight copy: 4 KB contiguous per 16-row strip
constexpr int GS_WARPS = 4;
constexpr int GS_THREADS = 32 * GS_WARPS;
constexpr int GS_MAX_SLOTS = 8;  // ring slots per warp
constexpr int W_TILE_BYTES = PK_TILE_BYTES;          // 16 rows x 64 k
constexpr int W_CHUNK_BYTES = GS_CH * W_TILE_BYTES;  // one copy
constexpr int GS_CHUNK_K = GS_CH * 64;               // k per copy
constexpr int GS_GROUPS = GS_CHUNK_K / 32;           // 32-k groups (one MMA pair each) per copy

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
// activations are written by the predecessor grid and only read here: the non-coherent path may cache them in L1
__device__ __forceinline__ uint4 ldg_act(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}

// TILES = 1: 16 output columns per CTA (one strip).  TILES = 2: 32 adjacent columns (strips 2b, 2b + 1), or (SwiGLU)
// gate strip b and the matching up strip tile1_off + b.  S = ring slots per warp; a slot holds TILES copies.
// AD = how many of a warp's copies ahead its activation fragments are fetched.  A warp handles one copy per
// iteration; with the fragments of only the next copy in flight an iteration cannot be shorter than one L2 round
// trip.  Measured on the 14-block decode stage (batch 8, us per step): AD 1: 1837, AD 2: 1818, AD 3: 1830 (the
// registers of the third copy cost more than its latency cover gives).
// ATMA: the activations of a copy's k range (8 token rows x 128 k, 2 KB) ride into the same ring slot by one TMA box
// load (tensor map {64 k, rows, K / 64}, box {64, 8, 2}, 128-byte swizzle) instead of per-lane global loads.  Measured
// with the loads taken out, the one-strip projections spend 19-29 % of their loop time on those loads (they
// queue in the load/store unit, 12 warps x 4 x 512 bytes per copy round; a deeper register prefetch does not help),
// and only without them does a warp wait for HBM rather than for its own instructions.  Needs K % 64 == 0.
template <int NB, int EPI, int TILES, bool F16, int AD, bool ATMA>
__global__ void __launch_bounds__(GS_THREADS, 3)
gemm_stream_kernel(const uint8_t* __restrict__ wp, const uint16_t* __restrict__ act, int lda, int K, int N, int KBp,
                   int tile1_off, int M, void* __restrict__ out, int ldo, int S, int rot_mul, int* __restrict__ err,
                   uint64_t wait_ns, int withhold, const __grid_constant__ CUtensorMap tm_act) {
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  static_assert(!SWIGLU || TILES == 2, "SwiGLU pairs a gate strip with an up strip");
  constexpr int OUT_COLS = (TILES == 2 && !SWIGLU) ? 32 : 16;
  constexpr int ACT_BYTES = ATMA ? GS_CHUNK_K * 8 * 2 : 0;  // 8 token rows of the copy's k range
  constexpr int STAGE_BYTES = TILES * W_CHUNK_BYTES + ACT_BYTES;
  constexpr int RED_LD = NB * 8 + 1;
  static_assert(16 * TILES * RED_LD * 4 <= 2 * STAGE_BYTES, "a warp's partial sums reuse its own ring space");
  static_assert(!ATMA || NB == 1, "the activation box holds one group of 8 tokens");
  extern __shared__ uint8_t gs_smem_raw[];
  __shared__ uint64_t bars[GS_WARPS * GS_MAX_SLOTS];
  const uint32_t base = (smem_u32(gs_smem_raw) + 1023u) & ~1023u;  // the activation boxes are 128-byte swizzled
  uint8_t* base_ptr = gs_smem_raw + (base - smem_u32(gs_smem_raw));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n0 = blockIdx.x * OUT_COLS;
  const int NCH = KBp / GS_CH;  // copies per strip
  const uint32_t my_bars = smem_u32(bars) + 8u * (warp * GS_MAX_SLOTS);
  const uint32_t my_ring = base + (uint32_t)(warp * S) * STAGE_BYTES;
  const int strip0 = SWIGLU ? (int)blockIdx.x : (int)blockIdx.x * TILES;
  const int strip1 = SWIGLU ? tile1_off + (int)blockIdx.x : strip0 + 1;
  const uint8_t* w0 = wp + (size_t)strip0 * KBp * W_TILE_BYTES;
  const uint8_t* w1 = wp + (size_t)strip1 * KBp * W_TILE_BYTES;

  // CTAs walk K from staggered starting points (a fixed rotation per CTA, so the summation order stays
  // reproducible): otherwise every resident CTA would ask for the same activation lines at the same moment.
  const int rot = (int)((blockIdx.x * (unsigned)rot_mul) % (unsigned)NCH);
  auto actual = [&](int ch_logical) {
    const int ch = ch_logical + rot;
    return ch >= NCH ? ch - NCH : ch;
  };
  uint32_t inflight = 0;  // lane 0: slots whose copy has been asked for and not yet been waited for
  // weights: never written by any kernel, may be fetched before the predecessor has finished
  auto issue_w = [&](int ch_logical, int slot) {
    const int ch = actual(ch_logical);
    const uint32_t dst = my_ring + slot * STAGE_BYTES, bar = my_bars + 8u * slot;
    inflight |= 1u << slot;
    mbar_expect_tx(bar, STAGE_BYTES);
    bulk_load(dst, w0 + (size_t)ch * W_CHUNK_BYTES, W_CHUNK_BYTES, bar);
    if (TILES == 2) bulk_load(dst + W_CHUNK_BYTES, w1 + (size_t)ch * W_CHUNK_BYTES, W_CHUNK_BYTES, bar);
  };

  // activations of the same copy (the predecessor's output: only after the wait for it)
  auto issue_a = [&](int ch_logical, int slot) {
    if (ATMA) {
      const uint32_t dst = my_ring + slot * STAGE_BYTES + TILES * W_CHUNK_BYTES, bar = my_bars + 8u * slot;
      asm volatile(
          "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
          ::"r"(dst), "l"(&tm_act), "r"(bar), "r"(0), "r"(0), "r"(actual(ch_logical) * GS_CH)
          : "memory");
    }
  };

  // Every CTA of this grid is resident by the time the last one gets here, so the successor may be scheduled
  // into whatever room is left: it only sets up and prefetches until this grid has completed.
  pdl_trigger();
  if (lane == 0) {
    if (ATMA) asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_act) : "memory");
    for (int sl = 0; sl < S; ++sl) mbar_init(my_bars + 8u * sl, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // `withhold` (a test hook, see launch_cfg): warp 0 of CTA 0 never asks for its first copy, so its first
    // wait below runs into the limit and the kernel leaves through the path that a lost copy would take
    for (int sl = 0; sl < S; ++sl)
      if (warp + GS_WARPS * sl < NCH && !(withhold && blockIdx.x == 0 && warp == 0 && sl == 0)) issue_w(warp + GS_WARPS * sl, sl);
  }
  __syncwarp();

  // this lane's activation rows: token 8j + g of group j; rows >= M and k >= K read as zero
  const uint16_t* arow[NB];
  bool avalid[NB];
#pragma unroll
  for (int j = 0; j < NB; ++j) {
    avalid[j] = 8 * j + g < M;
    arow[j] = act + (size_t)(avalid[j] ? 8 * j + g : 0) * lda + 8 * t;
  }
  uint4 bq[AD][GS_GROUPS][NB];  // fragment entries of this warp's next AD copies, refilled group by group as they are used
  auto load_act = [&](int ch_logical, int q, uint4 (&dst)[NB]) {
    const int k = actual(ch_logical) * GS_CHUNK_K + q * 32;
#pragma unroll
    for (int j = 0; j < NB; ++j)
      dst[j] = (avalid[j] && k + 8 * t < K) ? ldg_act(arow[j] + k) : make_uint4(0u, 0u, 0u, 0u);
  };
  pdl_wait();  // activations (and, for the residual epilogue, the output) belong to the predecessor until here
  if (ATMA) {
    if (lane == 0)
      for (int sl = 0; sl < S; ++sl)
        if (warp + GS_WARPS * sl < NCH && !(withhold && blockIdx.x == 0 && warp == 0 && sl == 0)) issue_a(warp + GS_WARPS * sl, sl);
  } else {
#pragma unroll
    for (int a = 0; a < AD; ++a) {
      if (warp + GS_WARPS * a < NCH) {
#pragma unroll
        for (int q = 0; q < GS_GROUPS; ++q) load_act(warp + GS_WARPS * a, q, bq[a][q]);
      }
    }
  }

  // CH independent accumulator chains per output fragment: the MMAs of one copy would otherwise form one chain of
  // eight dependent instructions, and the one-strip kernels then spend their time in that chain's latency instead
  // of waiting for HBM (measured: 8 % of a warp's loop time waiting for copies against 42 % in the two-strip grid)
  constexpr int CH = TILES == 1 ? GS_GROUPS : 2;
  float acc[CH][TILES][NB][4];
#pragma unroll
  for (int c = 0; c < CH; ++c)
#pragma unroll
    for (int i = 0; i < TILES; ++i)
#pragma unroll
      for (int j = 0; j < NB; ++j) acc[c][i][j][0] = acc[c][i][j][1] = acc[c][i][j][2] = acc[c][i][j][3] = 0.f;

  bool ok = true;
  int slot = 0;
  uint32_t phase = 0;
  // shared-memory offset of this lane's 16 bytes in tile row g, first 32-k group (the tile is stored swizzled:
  // 16-byte chunk c of row r sits at chunk position c ^ (r & 7); rows g and g + 8 share g & 7)
  for (int ch0 = warp; ch0 < NCH && ok; ch0 += GS_WARPS * AD) {
#pragma unroll
    for (int a = 0; a < AD; ++a) {
      const int ch = ch0 + GS_WARPS * a;
      if (ch >= NCH) break;
      // one decision for the whole warp (a bounded wait could run out for some lanes only)
      if (!__all_sync(0xffffffffu, mbar_wait(my_bars + 8u * slot, phase, nullptr, wait_ns))) { ok = false; break; }
      inflight &= ~(1u << slot);
      const uint32_t sbase = my_ring + slot * STAGE_BYTES;
      const bool more = ch + GS_WARPS * AD < NCH;
#pragma unroll
      for (int q = 0; q < GS_GROUPS; ++q) {
        const uint32_t off = (uint32_t)((q >> 1) * W_TILE_BYTES + g * 128 + (((4 * (q & 1) + t) ^ g) << 4));
        if (ATMA)  // token g, k 8t .. 8t+7 of the group: the box keeps the weight tiles' chunk permutation
          bq[a][q][0] = lds128(sbase + TILES * W_CHUNK_BYTES + (uint32_t)((q >> 1) * 1024 + g * 128 + (((4 * (q & 1) + t) ^ g) << 4)));
#pragma unroll
        for (int i = 0; i < TILES; ++i) {
          const uint4 lo = lds128(sbase + i * W_CHUNK_BYTES + off);          // row g:     k 8t .. 8t+7 of the group
          const uint4 hi = lds128(sbase + i * W_CHUNK_BYTES + off + 1024u);  // row g + 8
#pragma unroll
          for (int j = 0; j < NB; ++j) {
            if (F16) {
              mma_f16_16816(acc[q % CH][i][j], lo.x, hi.x, lo.y, hi.y, bq[a][q][j].x, bq[a][q][j].y);
              mma_f16_16816(acc[q % CH][i][j], lo.z, hi.z, lo.w, hi.w, bq[a][q][j].z, bq[a][q][j].w);
            } else {
              mma_bf16_16816(acc[q % CH][i][j], lo.x, hi.x, lo.y, hi.y, bq[a][q][j].x, bq[a][q][j].y);
              mma_bf16_16816(acc[q % CH][i][j], lo.z, hi.z, lo.w, hi.w, bq[a][q][j].z, bq[a][q][j].w);
            }
          }
        }
        if (!ATMA && more) load_act(ch + GS_WARPS * AD, q, bq[a][q]);  // the same group, AD copies further on
      }
      // Every shared-memory read above has been consumed by an MMA that is already issued, so after this
      // warp barrier no lane still reads the slot and lane 0 may hand it back to the copy engine.
      __syncwarp();
      if (lane == 0) {
        const int next = ch + GS_WARPS * S;
        if (next < NCH) {
          issue_w(next, slot);
          issue_a(next, slot);
        }
      }
      if (++slot == S) { slot = 0; phase ^= 1u; }
    }
  }
  if (!ok) {
    // a copy never landed: record it and let whatever is still in flight arrive (bounded) before leaving, so that
    // no copy writes into shared memory that already belongs to another CTA.  Slots from the failing one on still
    // owe the current phase, the slots before it were refilled for the next one.
    if (lane == 0) {
      atomicCAS(err, 0, 4);
      for (int sl = 0; sl < S; ++sl)
        if ((inflight >> sl) & 1u) mbar_wait(my_bars + 8u * sl, sl >= slot ? phase : phase ^ 1u, nullptr, wait_ns);
    }
    __syncwarp();
  }
  // partial sums of this warp go to the start of its own ring space (nothing is in flight into it any more)
  float* red = reinterpret_cast<float*>(base_ptr);
  const int red_warp = S * STAGE_BYTES / 4;  // floats between two warps' areas
  {
    float* mine = red + warp * red_warp;
#pragma unroll
    for (int i = 0; i < TILES; ++i)
#pragma unroll
      for (int j = 0; j < NB; ++j) {
        float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < CH; ++c) {  // the chains in a fixed order
          v[0] += acc[c][i][j][0]; v[1] += acc[c][i][j][1]; v[2] += acc[c][i][j][2]; v[3] += acc[c][i][j][3];
        }
        mine[(16 * i + g) * RED_LD + 8 * j + 2 * t] = v[0];
        mine[(16 * i + g) * RED_LD + 8 * j + 2 * t + 1] = v[1];
        mine[(16 * i + g + 8) * RED_LD + 8 * j + 2 * t] = v[2];
        mine[(16 * i + g + 8) * RED_LD + 8 * j + 2 * t + 1] = v[3];
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
      v += red[ww * red_warp + r * RED_LD + m];
      if (SWIGLU) v2 += red[ww * red_warp + (16 + r) * RED_LD + m];
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

template <int NB, int EPI, int TILES, bool F16, int AD, bool ATMA>
int launch_cfg_ad(const TcAct& act, const TcWeight& w, int M, int N, void* out, int ldo, cudaStream_t st, bool early) {
  static bool configured = false;
  static int num_sms = 0, smem_per_sm = 0;
  constexpr int STAGE_BYTES = TILES * W_CHUNK_BYTES + (ATMA ? GS_CHUNK_K * 8 * 2 : 0);
  constexpr int MAX_DYN = GS_WARPS * GS_MAX_SLOTS * STAGE_BYTES + 1024 > 200 * 1024 ? 200 * 1024
                                                                                      : GS_WARPS * GS_MAX_SLOTS * STAGE_BYTES + 1024;
  if (!configured) {
    HYP_CUDA_TRY(cudaFuncSetAttribute(gemm_stream_kernel<NB, EPI, TILES, F16, AD, ATMA>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_DYN));
    // several CTAs per SM share the ring space: ask for the largest shared-memory carve-out
    HYP_CUDA_TRY(cudaFuncSetAttribute(gemm_stream_kernel<NB, EPI, TILES, F16, AD, ATMA>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                      cudaSharedmemCarveoutMaxShared));
    int dev = 0;
    HYP_CUDA_TRY(cudaGetDevice(&dev));
    HYP_CUDA_TRY(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    HYP_CUDA_TRY(cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev));
    configured = true;
  }
  constexpr bool SWIGLU = EPI == EPI_SWIGLU_BF16;
  constexpr int OUT_COLS = (TILES == 2 && !SWIGLU) ? 32 : 16;
  const int n_ctas = (N + OUT_COLS - 1) / OUT_COLS;
  // Ring depth (slots per warp).  A grid whose CTAs are not all resident at once ends with a partial wave that
  // cannot keep HBM busy (measured on B200: 320 CTAs at 2 per SM take 1.4x the time of the same CTAs at 3 per
  // SM), and one that could fit more CTAs per SM than it needs may be placed unevenly when it starts while its
  // predecessor still holds part of the SMs.  So when the grid fits in one wave the ring takes whatever shared
  // memory that residency leaves: this caps the CTAs per SM at ceil(CTAs / SMs), and the more of a strip a CTA
  // holds, the more it fetches while its predecessor drains.  Grids of several waves take two slots (more
  // CTAs per SM hide each other's start and end).  1 KB per CTA is reserved by the driver; 512 B cover barriers
  // and alignment.
  const int per_sm = (n_ctas + num_sms - 1) / num_sms;
  int slots = (smem_per_sm / per_sm - 1024 - 1024 - 384) / (GS_WARPS * STAGE_BYTES);
  if (slots > GS_MAX_SLOTS) slots = GS_MAX_SLOTS;
  if (slots < 2) slots = 2;
  if (gemm_stream_slots_override() > 0) slots = gemm_stream_slots_override();
  if (slots > GS_MAX_SLOTS) slots = GS_MAX_SLOTS;
  while (slots > 2 && GS_WARPS * slots * STAGE_BYTES + 1024 > MAX_DYN) --slots;
  const int smem = GS_WARPS * slots * STAGE_BYTES + 1024;
  // bounded waits: 4 s unless a shorter limit was set (hyp_tune); `withhold` is a one-shot test hook that makes
  // one wait of the next launch run into that limit (nothing faults: the kernel records the code and returns)
  const uint64_t wait_ns = gemm_stream_wait_limit_us() > 0 ? (uint64_t)gemm_stream_wait_limit_us() * 1000ull : WAIT_LIMIT_NS;
  const int withhold = gemm_stream_withhold_next();
  gemm_stream_withhold_next() = 0;
  // the kernel fetches weights before it waits for its predecessor: launched early only when the weights cannot
  // be that predecessor's output
  if (early)
    HYP_CUDA_TRY(launch_pdl<1>(gemm_stream_kernel<NB, EPI, TILES, F16, AD, ATMA>, dim3(n_ctas), dim3(GS_THREADS), (size_t)smem, st,
                               (const uint8_t*)w.packed, (const uint16_t*)act.ptr, act.K, act.K, N, w.KBp, w.N16p, M, out,
                               ldo, slots, gemm_stream_rotation(), tc_err_flag_ptr(), wait_ns, withhold, act.map_a8));
  else
    HYP_CUDA_TRY(launch_pdl<4>(gemm_stream_kernel<NB, EPI, TILES, F16, AD, ATMA>, dim3(n_ctas), dim3(GS_THREADS), (size_t)smem, st,
                               (const uint8_t*)w.packed, (const uint16_t*)act.ptr, act.K, act.K, N, w.KBp, w.N16p, M, out,
                               ldo, slots, gemm_stream_rotation(), tc_err_flag_ptr(), wait_ns, withhold, act.map_a8));
  return 1;
}

template <int NB, int EPI, int TILES, bool F16>
int launch_cfg(const TcAct& act, const TcWeight& w, int M, int N, void* out, int ldo, cudaStream_t st, bool early) {
  // activations by TMA into the ring whenever the operand has the tensor map for it (K a multiple of 64)
  if (act.has_a8 && gemm_stream_act_tma()) return launch_cfg_ad<NB, EPI, TILES, F16, 1, true>(act, w, M, N, out, ldo, st, early);
  int ad = 2;  // measured best, see the kernel
  if (gemm_stream_act_depth() > 0) ad = gemm_stream_act_depth();
  if (ad >= 3) return launch_cfg_ad<NB, EPI, TILES, F16, 3, false>(act, w, M, N, out, ldo, st, early);
  if (ad == 2) return launch_cfg_ad<NB, EPI, TILES, F16, 2, false>(act, w, M, N, out, ldo, st, early);
  return launch_cfg_ad<NB, EPI, TILES, F16, 1, false>(act, w, M, N, out, ldo, st, early);
}

template <int NB, bool F16>
int launch_nb(const TcAct& act, const TcWeight& w, int M, int N, int epi, void* out, int ldo, cudaStream_t st, bool early) {
  const bool wide = N > 8192;  // many rows: 32 columns per CTA keep the CTA count down
  switch (epi) {
    case EPI_STORE_BF16:
      return wide ? launch_cfg<NB, EPI_STORE_BF16, 2, F16>(act, w, M, N, out, ldo, st, early)
                  : launch_cfg<NB, EPI_STORE_BF16, 1, F16>(act, w, M, N, out, ldo, st, early);
    case EPI_RESID_F32:
      return wide ? launch_cfg<NB, EPI_RESID_F32, 2, F16>(act, w, M, N, out, ldo, st, early)
                  : launch_cfg<NB, EPI_RESID_F32, 1, F16>(act, w, M, N, out, ldo, st, early);
    case EPI_STORE_F32:
      return wide ? launch_cfg<NB, EPI_STORE_F32, 2, F16>(act, w, M, N, out, ldo, st, early)
                  : launch_cfg<NB, EPI_STORE_F32, 1, F16>(act, w, M, N, out, ldo, st, early);
    case EPI_SWIGLU_BF16: return launch_cfg<NB, EPI_SWIGLU_BF16, 2, F16>(act, w, M, N, out, ldo, st, early);
    default: return HYP_EINVAL;
  }
}

template <bool F16>
int launch_type(const TcAct& act, const TcWeight& w, int M, int N, int epi, void* out, int ldo, cudaStream_t st, bool early) {
  // One group of 8 tokens.  The kernel is written for NB groups (up to 32 rows), but from 9 rows on the tensor-memory
  // kernels are faster (every CTA here re-reads the activations of its K range from L2, and at 16+ tokens those
  // reads outweigh the weights), so only NB = 1 is built.
  return launch_nb<1, F16>(act, w, M, N, epi, out, ldo, st, early);
}

}  // namespace

int launch_gemm_stream(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                       cudaStream_t st, bool early) {
  if (M < 1 || M > 8 || N < 1 || K < 8 || act.K != K || w.K != K || !tc_err_flag_ptr()) return HYP_EINVAL;
  if (w.rows != N || w.halves != (epi == EPI_SWIGLU_BF16 ? 2 : 1)) return HYP_EINVAL;
  if (act.f16 != w.f16) return HYP_EINVAL;  // one instruction takes both operands in the same 16-bit type
  if (((uintptr_t)act.ptr & 15) != 0 || (K % 8) != 0) return HYP_EINVAL;  // 128-bit activation loads
  return act.f16 ? launch_type<true>(act, w, M, N, epi, out, ldo, st, early) : launch_type<false>(act, w, M, N, epi, out, ldo, st, early);
}

}  // namespace hyp
