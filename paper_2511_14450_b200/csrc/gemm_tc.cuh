// Tensor-core projection for any row count (prefill): operand descriptors and launcher.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace hyp {

// A 16-bit matrix [rows, K] row-major (bf16, or fp16 when f16) together with the TMA descriptors that tile
// it.  Both operands of a projection must have the same type.
struct TcOperand {
  CUtensorMap map;
  const __nv_bfloat16* ptr = nullptr;
  int rows = 0, K = 0;
  bool f16 = false;
  CUtensorMap map_small[4];  // weight-streaming kernel: weights [0], [1] = 16-, 32-row boxes; activations [nb-1] = 8*nb rows
};
typedef TcOperand TcWeight;
typedef TcOperand TcAct;

int tc_make_weight(TcWeight* w, const void* ptr, int rows, int K, bool f16 = false);
int tc_make_act(TcAct* a, const void* ptr, int rows, int K, bool f16 = false);

// One-time set-up of the device-side error word (allocates; call from stage creation, not from the hot path).
int tc_prepare();
// Reads the error word (synchronises the device): 0 = no kernel gave up on a wait.
int tc_error_flag(int* value_out);

// Device word that kernels set when a bounded wait expires (null before tc_prepare).
int* tc_err_flag_ptr();

// Weight-streaming projection for M <= 32 rows (decode), fed by TMA; same contract as launch_gemm_tc.
int launch_gemm_stream(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                       cudaStream_t st);

// out[m, n] (+)= sum_k act[m, k] * w[n, k] for m < M, n < N (SwiGLU: w holds 2N rows).
int launch_gemm_tc(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                   cudaStream_t st);

}  // namespace hyp
