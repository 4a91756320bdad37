// Decode attention with library-resident scratch: the same kernels as hyp_op_attn_decode, but the
// per-split partial results live in a fixed array inside the library image instead of a buffer the
// caller had to allocate.
#include <mutex>

#include "common.cuh"
#include "hyperion_ops.h"

using namespace hyp;

namespace {

// Scratch shared by every call on a device.  It is part of the loaded module, so each GPU that loads
// the library carries these 4 MiB until the process exits.
static __device__ __align__(256) float g_static_scratch[HYP_STATIC_SCRATCH_BYTES / sizeof(float)];

constexpr int MAX_DEVICES = 64;
float* g_scratch_addr[MAX_DEVICES] = {};  // device address of g_static_scratch, per device ordinal
std::mutex g_scratch_mutex;

// `g_static_scratch` named in host code is only a handle for the runtime, not something a kernel can
// dereference; the real device address has to be asked for, once per device, with that device current.
int scratch_for_current_device(float** out) {
  int dev = 0;
  HYP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return HYP_EINVAL;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    float* p = nullptr;
    HYP_CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_static_scratch));
    if (!p) return HYP_ECUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return HYP_OK;
}

}  // namespace

extern "C" int hyp_op_attn_decode_static(const hyp_attn_shape* shape, int32_t n_seqs, const void* q, int32_t q_stride,
                                         const void* kv_pages, const int32_t* block_table,
                                         int32_t max_pages_per_seq, const int32_t* ctx_lens, int32_t n_splits,
                                         void* out, void* stream) {
  if (!shape || !q || !kv_pages || !block_table || !ctx_lens || !out) return HYP_EINVAL;
  if (shape->n_kv_heads < 1 || shape->n_q_heads < shape->n_kv_heads || shape->n_q_heads % shape->n_kv_heads)
    return HYP_EINVAL;
  const int G = shape->n_q_heads / shape->n_kv_heads;
  if (!(G == 1 || G == 2 || G == 4 || G == 8) || !(shape->head_dim == 64 || shape->head_dim == 128)) return HYP_EINVAL;
  if (n_seqs < 1 || n_seqs > 65535 || max_pages_per_seq < 1 || n_splits < 1 || n_splits > 32) return HYP_EINVAL;
  if (q_stride < shape->n_q_heads * shape->head_dim || q_stride % 8) return HYP_EINVAL;
  // the partials of this batch must fit the fixed array
  if (attn_decode_scratch_bytes(n_seqs, shape->n_q_heads, shape->head_dim, n_splits) > (size_t)HYP_STATIC_SCRATCH_BYTES)
    return HYP_ECAPACITY;
  float* scratch = nullptr;
  int rc = scratch_for_current_device(&scratch);
  if (rc) return rc;

  BatchMeta bm{};
  bm.n_seqs = n_seqs;
  bm.n_tokens = n_seqs;
  bm.max_pages_per_seq = max_pages_per_seq;
  bm.ctx_lens = ctx_lens;
  bm.block_table = block_table;
  ModelDims d{};
  d.Hq = shape->n_q_heads; d.Hkv = shape->n_kv_heads; d.D = shape->head_dim;
  d.qkv_rows = q_stride;
  d.page_tokens = 16;
  // Nothing in the array has to be cleared first: the partial kernel writes every (sequence, head,
  // split) slot - weighted sum, running maximum and denominator - before the merge kernel reads it.
  rc = launch_attn_decode((const __half*)q, q_stride, (const __half*)kv_pages, (__half*)out, scratch, n_splits,
                          bm, d, (cudaStream_t)stream);
  if (rc < 0) return rc;
  cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) {
    set_last_cuda_error((int)e);
    return HYP_ECUDA;
  }
  return HYP_OK;
}
