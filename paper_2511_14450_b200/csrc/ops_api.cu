// Single-kernel C entry points: argument checks, then the same launchers the stage runtime uses.
#include "common.cuh"
#include "gemm_tc.cuh"
#include "hyperion_ops.h"

using namespace hyp;

namespace {

bool attn_shape_ok(const hyp_attn_shape* s) {
  if (!s || s->n_kv_heads < 1 || s->n_q_heads < s->n_kv_heads || s->n_q_heads % s->n_kv_heads) return false;
  const int G = s->n_q_heads / s->n_kv_heads;
  return (G == 1 || G == 2 || G == 4 || G == 8) && (s->head_dim == 64 || s->head_dim == 128);
}

ModelDims attn_dims(const hyp_attn_shape* s, int q_stride) {
  ModelDims d{};
  d.Hq = s->n_q_heads; d.Hkv = s->n_kv_heads; d.D = s->head_dim;
  d.qkv_rows = q_stride;
  d.page_tokens = 16;
  return d;
}

int finish(int rc) {
  if (rc < 0) return rc;
  cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) {
    set_last_cuda_error((int)e);
    return HYP_ECUDA;
  }
  return HYP_OK;
}

}  // namespace

extern "C" int hyp_op_rmsnorm(const float* x, const void* g, void* out, int32_t M, int32_t H, float eps, void* stream) {
  if (!x || !g || !out || M < 1 || H < 8 || H % 8 || !(eps > 0.f)) return HYP_EINVAL;
  return finish(launch_rmsnorm(x, (const __nv_bfloat16*)g, out, false, M, H, eps, nullptr,
                               (cudaStream_t)stream));
}

extern "C" size_t hyp_op_weight_packed_bytes(int32_t N, int32_t K, int32_t swiglu) {
  if (N < 1 || K < 8 || K % 8) return 0;
  return tc_packed_bytes(N, swiglu ? 2 : 1, K);
}

namespace {
int pack_weight(const void* w, int32_t N, int32_t K, int32_t swiglu, void* packed, size_t packed_bytes, void* stream,
                bool to_f16) {
  if (!w || !packed || N < 1 || K < 8 || K % 8) return HYP_EINVAL;
  if (((uintptr_t)w & 15) != 0 || ((uintptr_t)packed & 127) != 0) return HYP_EINVAL;
  if (packed_bytes < tc_packed_bytes(N, swiglu ? 2 : 1, K)) return HYP_ECAPACITY;
  return finish(tc_pack_weight(w, packed, N, swiglu ? 2 : 1, K, to_f16, (cudaStream_t)stream));
}
}  // namespace

extern "C" int hyp_op_pack_weight(const void* w, int32_t N, int32_t K, int32_t swiglu, void* packed, size_t packed_bytes,
                                  void* stream) {
  return pack_weight(w, N, K, swiglu, packed, packed_bytes, stream, false);
}
extern "C" int hyp_op_pack_weight_f16(const void* w, int32_t N, int32_t K, int32_t swiglu, void* packed,
                                      size_t packed_bytes, void* stream) {
  return pack_weight(w, N, K, swiglu, packed, packed_bytes, stream, true);
}

extern "C" int hyp_device_wait_status(int32_t* code_out, int32_t clear) {
  if (!code_out) return HYP_EINVAL;
  int v = 0;
  const int rc = tc_error_flag_take(&v, clear != 0);
  *code_out = v;
  return rc;
}

extern "C" int hyp_tune(int32_t key, int32_t value) {
  switch (key) {
    case HYP_TUNE_PDL:
      if (value < 0 || value > 3) return HYP_EINVAL;
      pdl_level() = value;
      return HYP_OK;
    case HYP_TUNE_STREAM_SLOTS:
      if (value < 0 || value > 8) return HYP_EINVAL;
      gemm_stream_slots_override() = value;
      return HYP_OK;
    case HYP_TUNE_STREAM_ROTATION:
      if (value < 0 || value > 1024) return HYP_EINVAL;
      gemm_stream_rotation() = value;
      return HYP_OK;
    case HYP_TUNE_SWAP_MIN_ROWS:
      if (value < 1 || value > 129) return HYP_EINVAL;
      gemm_swap_min_rows() = value;
      return HYP_OK;
    case HYP_TUNE_SWAP_MAX_ROWS:
      if (value < 0 || value > 128) return HYP_EINVAL;
      gemm_swap_max_rows() = value;
      return HYP_OK;
    case HYP_TUNE_SWAP_EPILOGUES:
      if (value < 0 || value > 15) return HYP_EINVAL;
      gemm_swap_epilogues() = value;
      return HYP_OK;
    case HYP_TUNE_PREFILL_ATTN_TC:
      attn_prefill_tc_enabled() = value != 0;
      return HYP_OK;
    case HYP_TUNE_ATTN_SPLITS:
      if (value < 0 || value > 8) return HYP_EINVAL;
      attn_fused_splits_override() = value;
      return HYP_OK;
    case HYP_TUNE_STREAM_ACT_TMA:
      gemm_stream_act_tma() = value != 0;
      return HYP_OK;
    case HYP_TUNE_ATTN_GLOBAL_MERGE:
      attn_global_merge() = value != 0;
      return HYP_OK;
    case HYP_TUNE_STREAM_ACT_DEPTH:
      if (value < 0 || value > 3) return HYP_EINVAL;
      gemm_stream_act_depth() = value;
      return HYP_OK;
    case HYP_TUNE_WAIT_LIMIT_US:
      if (value < 0) return HYP_EINVAL;
      gemm_stream_wait_limit_us() = value;
      return HYP_OK;
    case HYP_TUNE_STREAM_WITHHOLD_COPY:
      gemm_stream_withhold_next() = value != 0;
      return HYP_OK;
    case HYP_TUNE_TILE_224:
      tile_width_224_enabled() = value != 0;
      return HYP_OK;
    case HYP_TUNE_FIRST_BLOCK_SPLIT:
      first_block_split() = value != 0;
      return HYP_OK;
    case HYP_TUNE_ATTN_SLOTS:
      if (value < 0 || value > 4) return HYP_EINVAL;
      attn_fused_slots_override() = value;
      return HYP_OK;
    default: return HYP_EINVAL;
  }
}

namespace {
int op_gemm(const void* a, const void* w, int32_t M, int32_t N, int32_t K, int32_t epilogue, void* out, int32_t ldo,
            void* stream, bool f16) {
  if (!a || !w || !out || M < 1 || N < 1 || K < 8 || K % 8 || ldo < N || ((uintptr_t)w & 127) != 0) return HYP_EINVAL;
  if (epilogue < HYP_EPI_STORE_BF16 || epilogue > HYP_EPI_STORE_F32) return HYP_EINVAL;
  cudaStream_t st = (cudaStream_t)stream;
  if (M > 8 && (N % 16 || ldo % 8)) return HYP_EINVAL;
  int rc = tc_prepare();
  if (rc) return rc;
  TcAct ta;
  TcWeight tw;
  rc = tc_make_act(&ta, a, M, K, f16);
  if (rc) return rc;
  rc = tc_make_weight(&tw, w, N, epilogue == HYP_EPI_SWIGLU_BF16 ? 2 : 1, K, f16);
  if (rc) return rc;
  return finish(launch_projection(ta, tw, M, N, K, epilogue, out, ldo, st));
}
}  // namespace

extern "C" int hyp_op_gemm(const void* a, const void* w, int32_t M, int32_t N, int32_t K, int32_t epilogue, void* out,
                           int32_t ldo, void* stream) {
  return op_gemm(a, w, M, N, K, epilogue, out, ldo, stream, false);
}
extern "C" int hyp_op_gemm_f16(const void* a, const void* w, int32_t M, int32_t N, int32_t K, int32_t epilogue, void* out,
                               int32_t ldo, void* stream) {
  return op_gemm(a, w, M, N, K, epilogue, out, ldo, stream, true);
}

extern "C" int hyp_op_attn_decode_splits(int32_t n_seqs, int32_t n_kv_heads, int32_t max_ctx) {
  if (n_seqs < 1 || n_kv_heads < 1 || max_ctx < 1) return HYP_EINVAL;
  return attn_decode_splits(n_seqs, n_kv_heads, max_ctx);
}

extern "C" size_t hyp_op_attn_decode_scratch_bytes(int32_t n_seqs, int32_t n_q_heads, int32_t head_dim,
                                                   int32_t n_splits) {
  if (n_seqs < 1 || n_q_heads < 1 || head_dim < 1 || n_splits < 1) return 0;
  return attn_decode_scratch_bytes(n_seqs, n_q_heads, head_dim, n_splits);
}

extern "C" int hyp_op_attn_decode(const hyp_attn_shape* shape, int32_t n_seqs, const void* q, int32_t q_stride,
                                  const void* kv_pages, const int32_t* block_table, int32_t max_pages_per_seq,
                                  const int32_t* ctx_lens, int32_t n_splits, float* scratch, size_t scratch_bytes,
                                  void* out, void* stream) {
  if (!attn_shape_ok(shape) || !q || !kv_pages || !block_table || !ctx_lens || !scratch || !out) return HYP_EINVAL;
  if (n_seqs < 1 || n_seqs > 65535 || max_pages_per_seq < 1 || n_splits < 1 || n_splits > 32) return HYP_EINVAL;
  if (q_stride < shape->n_q_heads * shape->head_dim || q_stride % 8) return HYP_EINVAL;
  if (scratch_bytes < attn_decode_scratch_bytes(n_seqs, shape->n_q_heads, shape->head_dim, n_splits)) return HYP_ECAPACITY;
  BatchMeta bm{};
  bm.n_seqs = n_seqs;
  bm.n_tokens = n_seqs;
  bm.max_pages_per_seq = max_pages_per_seq;
  bm.ctx_lens = ctx_lens;
  bm.block_table = block_table;
  const ModelDims d = attn_dims(shape, q_stride);
  return finish(launch_attn_decode((const __half*)q, q_stride, (const __half*)kv_pages, (__half*)out, scratch,
                                   n_splits, bm, d, (cudaStream_t)stream));
}

extern "C" int hyp_op_attn_decode_step(const hyp_attn_shape* shape, int32_t n_seqs, const float* qkv, int32_t stride,
                                       void* kv_pages, const int32_t* block_table, int32_t max_pages_per_seq,
                                       const int32_t* ctx_lens, const float* rope_table, int32_t n_splits, void* out,
                                       void* stream) {
  if (!attn_shape_ok(shape) || !qkv || !kv_pages || !block_table || !ctx_lens || !rope_table || !out) return HYP_EINVAL;
  if (n_seqs < 1 || n_seqs > 65535 || max_pages_per_seq < 1 || n_splits < 0 || n_splits > 8) return HYP_EINVAL;
  if (stride < (shape->n_q_heads + 2 * shape->n_kv_heads) * shape->head_dim) return HYP_EINVAL;
  if (((uintptr_t)kv_pages & 15) != 0 || ((uintptr_t)rope_table & 7) != 0) return HYP_EINVAL;
  int rc = tc_prepare();
  if (rc) return rc;
  BatchMeta bm{};
  bm.n_seqs = n_seqs;
  bm.n_tokens = n_seqs;
  bm.max_pages_per_seq = max_pages_per_seq;
  bm.ctx_lens = ctx_lens;
  bm.block_table = block_table;
  const ModelDims d = attn_dims(shape, stride);
  if (n_splits == 0) n_splits = attn_decode_fused_splits(n_seqs, shape->n_kv_heads, 16 * max_pages_per_seq);
  return finish(launch_attn_decode_fused(qkv, stride, (__half*)kv_pages, (const float2*)rope_table, (__half*)out, n_splits,
                                         2, tc_err_flag_ptr(), bm, d, (cudaStream_t)stream));
}

extern "C" int hyp_op_attn_prefill(const hyp_attn_shape* shape, int32_t n_seqs, int32_t M, const void* q,
                                   int32_t q_stride, const void* kv_pages, const int32_t* block_table,
                                   int32_t max_pages_per_seq, const int32_t* cu_q, const int32_t* ctx_lens, void* out,
                                   void* stream) {
  if (!attn_shape_ok(shape) || !q || !kv_pages || !block_table || !cu_q || !ctx_lens || !out) return HYP_EINVAL;
  if (n_seqs < 1 || M < n_seqs || max_pages_per_seq < 1) return HYP_EINVAL;
  if (q_stride < shape->n_q_heads * shape->head_dim || q_stride % 8) return HYP_EINVAL;
  BatchMeta bm{};
  bm.n_seqs = n_seqs;
  bm.n_tokens = M;
  bm.max_pages_per_seq = max_pages_per_seq;
  bm.cu_q = cu_q;
  bm.ctx_lens = ctx_lens;
  bm.block_table = block_table;
  const ModelDims d = attn_dims(shape, q_stride);
  if (attn_prefill_tc_enabled() && d.D == 128 && ((uintptr_t)q & 15) == 0) {
    // descriptors over the caller's buffers; the pool's size is not known here and only bounds the descriptor
    TcAct qa;
    CUtensorMap kvm;
    int rc = tc_make_act(&qa, q, M, q_stride, true);
    if (!rc) rc = tc_make_kv_map(&kvm, kv_pages, (size_t)1 << 20, d.Hkv, d.D);
    if (rc) return rc;
    ModelDims dd = d;
    return finish(launch_attn_prefill_tc(qa.map, kvm, (__half*)out, bm, dd, (cudaStream_t)stream));
  }
  return finish(launch_attn_prefill((const __half*)q, q_stride, (const __half*)kv_pages, (__half*)out, bm, d,
                                    (cudaStream_t)stream));
}
