// Bring-up body: row chunks through the weight-streaming kernel (replaced by tcgen05 tiles).
#include "gemm_tc.cuh"
#include "hyperion.h"

namespace hyp {

int tc_make_weight(TcWeight* w, const __nv_bfloat16* ptr, int rows, int K) {
  w->ptr = ptr; w->rows = rows; w->K = K;
  return HYP_OK;
}
int tc_make_act(TcAct* a, const __nv_bfloat16* ptr, int rows, int K) {
  a->ptr = ptr; a->rows = rows; a->K = K;
  return HYP_OK;
}

int launch_gemm_tc(const TcAct& act, const TcWeight& w, int M, int N, int K, int epi, void* out, int ldo,
                   cudaStream_t st) {
  int n = 0;
  const size_t esz = (epi == EPI_STORE_BF16 || epi == EPI_SWIGLU_BF16) ? 2 : 4;
  for (int m0 = 0; m0 < M; m0 += 32) {
    const int rows = M - m0 < 32 ? M - m0 : 32;
    int rc = launch_gemm_skinny(act.ptr + (size_t)m0 * K, K, w.ptr, N, K, rows, epi,
                                (char*)out + (size_t)m0 * ldo * esz, ldo, st);
    if (rc < 0) return rc;
    n += rc;
  }
  return n;
}

}  // namespace hyp
