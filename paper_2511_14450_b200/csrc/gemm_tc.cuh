// Projection operands (packed weights, activation descriptors) and the launchers of the two projection kernels.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace hyp {

// Packed weight layout.  A projection matrix w[n, k] (n < rows, k < K; SwiGLU: two such halves, gate then up) is
// held as tiles of 16 rows x 64 k (2 KB), tile (t, kb) at byte offset (t * KBp + kb) * 2048 with t = half * N16p +
// n / 16: all k-blocks of one 16-row strip are contiguous, so the weight-streaming kernel reads every strip as one
// sequential run of bulk copies and the tile kernel fetches a 128-row operand tile as eight 2 KB pieces.  Inside a
// tile, row r (128 bytes) keeps its 16-byte chunk c at chunk position c ^ (r & 7): the 128-byte swizzle that
// ldmatrix (conflict-free) and the tcgen05 shared-memory descriptors expect, applied once at load time.  Rows
// beyond `rows` and k beyond K are zero.  N16p = tiles per half (even), KBp = k-blocks per strip (even).
constexpr int PK_TILE_BYTES = 2048;
struct TcWeight {
  const void* packed = nullptr;
  int rows = 0;    // logical rows per half
  int halves = 1;  // 2: SwiGLU gate | up
  int K = 0, KBp = 0, N16p = 0;
  bool f16 = false;
  CUtensorMap map;  // 4-D view {64 k, 16 rows, KBp, halves * N16p}, box = 8 tiles x 1 k-block (128 rows), no swizzle
  CUtensorMap map7;  // the same view with boxes of 7 tiles (112 rows)
};
inline int pk_kbp(int K) { return ((K + 63) / 64 + 1) & ~1; }
inline int pk_n16p(int rows) { return ((rows + 15) / 16 + 1) & ~1; }
inline size_t tc_packed_bytes(int rows, int halves, int K) {
  return (size_t)halves * pk_n16p(rows) * pk_kbp(K) * PK_TILE_BYTES;
}
// src: bf16 [halves * rows, K] row-major (DEVICE, 16-byte aligned, K multiple of 8); dst: tc_packed_bytes(...) bytes.
// to_f16 converts the values to fp16 (exact for |w| >= 2^-17, saturating at +-65504); otherwise they stay bf16.
int tc_pack_weight(const void* src, void* dst, int rows, int halves, int K, bool to_f16, cudaStream_t st);
int tc_make_weight(TcWeight* w, const void* packed, int rows, int halves, int K, bool f16);

// A 16-bit activation matrix [rows, K] row-major (bf16, or fp16 when f16) with the TMA descriptors that tile it.
// Both operands of a projection must have the same type.
struct TcAct {
  CUtensorMap map;  // 128-row boxes (tile kernel)
  const void* ptr = nullptr;
  int rows = 0, K = 0;
  bool f16 = false;
  CUtensorMap map_small[3];  // boxes of 16, 32, 64 rows (swapped-operand kernel: the tokens are the N operand)
  // {64 k, rows, K / 64} view with boxes of 64 k x 8 rows x 2 k-blocks (weight-streaming kernel: the activations of
  // one 128-k copy, 2 KB); only when K is a multiple of 64
  CUtensorMap map_a8;
  bool has_a8 = false;
};
int tc_make_act(TcAct* a, const void* ptr, int rows, int K, bool f16 = false);

// Tensor map over one block's KV page pool for the tcgen05 prefill attention (head_dim 128).
int tc_make_kv_map(CUtensorMap* map, const void* kv_layer, size_t n_pages, int Hkv, int D);
// Prefill attention on tcgen05 (head_dim 128); q_map = TcAct::map of the rotated-query buffer.
int& attn_prefill_tc_enabled();
int launch_attn_prefill_tc(const CUtensorMap& q_map, const CUtensorMap& kv_map, __half* attn_out, const BatchMeta& bm,
                           const ModelDims& d, cudaStream_t st);

// 1 (default): the two-CTA tile kernel may take 224-column tiles where they fill the last wave better.
int& tile_width_224_enabled();

// One-time set-up of the device-side error word (allocates; call from stage creation, not from the hot path).
int tc_prepare();
// Reads the error word (synchronises the device): 0 = no kernel gave up on a wait.
int tc_error_flag(int* value_out);

// Device word that kernels set when a bounded wait expires (null before tc_prepare).
int* tc_err_flag_ptr();

// Ring depth override of the weight-streaming kernel (0 = the built-in choice).
int& gemm_stream_slots_override();
// Per-CTA stagger of the K walk of the weight-streaming kernel: CTA b starts at copy (b * rotation) mod copies.
int& gemm_stream_rotation();

// Limit of the weight-streaming kernel's bounded waits in microseconds (0 = the built-in 4 s), and a one-shot hook
// that makes the next launch of that kernel withhold one copy so that a wait runs into the limit (for the test of
// the HYP_ETIMEOUT path: no fault, the kernel records the code and returns).
int& gemm_stream_act_depth();
int& gemm_stream_act_tma();
int& gemm_stream_wait_limit_us();
int& gemm_stream_withhold_next();
// Reads the device word like tc_error_flag and, if `clear`, zeroes it afterwards.
int tc_error_flag_take(int* value_out, bool clear);

// Weight-streaming projection for M <= 8 rows (decode); same contract as launch_gemm_tc.  `early`: the packed
// weights are long-lived (not written by the kernel launched just before), so the launch may overlap that kernel.
int launch_gemm_stream(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                       cudaStream_t st, bool early = false);

// The same projection for 1..128 rows with the operands swapped on the tensor cores (128 weight rows = the M
// operand, the tokens = the N operand, K split over a cluster): activation traffic per weight byte is rows / 128.
// launch_projection routes the plain-store epilogues of row counts in [gemm_swap_min_rows(), gemm_swap_max_rows()]
// (default 9..128) to it when the matrix has too few 256-column tiles for the tile kernel.
int& gemm_swap_min_rows();
int& gemm_swap_max_rows();
int& gemm_swap_epilogues();  // bit e set: epilogue e may take the swapped kernel (default: the two plain stores)
int launch_gemm_swap(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                     cudaStream_t st, bool early = false);

// out[m, n] (+)= sum_k act[m, k] * w[n, k] for m < M, n < N (SwiGLU: w holds two halves of N rows).
int launch_gemm_tc(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                   cudaStream_t st, bool early = false);

// Picks the kernel by row count and epilogue (see its definition) and launches it.
int launch_projection(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo, cudaStream_t st,
                      bool early = false);

}  // namespace hyp
