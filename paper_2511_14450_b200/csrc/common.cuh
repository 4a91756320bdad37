// Shared device helpers and the internal kernel-launch interface of libhyperion.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hyp {

// ---------------------------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------------------------
void set_last_cuda_error(int e);
#define HYP_CUDA_TRY(expr)                         \
  do {                                             \
    cudaError_t _e = (expr);                       \
    if (_e != cudaSuccess) {                       \
      ::hyp::set_last_cuda_error((int)_e);         \
      return HYP_ECUDA;                            \
    }                                              \
  } while (0)

// Multiprocessors of the current device (asked once; grids are sized from it).
inline int sm_count() {
  static int n = 0;
  if (n <= 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        n <= 0)
      n = 148;
  }
  return n;
}

// ---------------------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float a, float b) {
  __half2 p = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
// fp32 -> fp16 with saturation at the largest finite value (the attention operands are fp16)
__device__ __forceinline__ uint32_t pack_f16_sat(float a, float b) {
  return pack_f16(fminf(fmaxf(a, -65504.f), 65504.f), fminf(fmaxf(b, -65504.f), 65504.f));
}

// ---------------------------------------------------------------------------------------------
// programmatic dependent launch.  A kernel launched with the attribute may start while its predecessor still
// runs; it calls pdl_wait() before the first access to memory the predecessor writes or reads, and everything
// before that - barrier set-up, weight prefetch - overlaps the predecessor.  A kernel calls pdl_trigger() when its
// successor may be scheduled.  Without the attribute both are no-ops.  Only the weight-streaming projections are
// launched with it (launch_pdl<true>): their prefetch is worth overlapping, and a chain of early launches stays
// one kernel deep.  Measured on B200 (14-block decode stage, batch 8): with the attribute on every kernel of the
// block the step got slower (waiting CTAs of several future kernels pile up on the SMs).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Process-wide level: a launch site of level L gets the attribute when L <= pdl_level().
// 0 = nobody, 1 = the weight-streaming projections, 2 = also the norms between them and the kernels only a prefill
// runs (rotation + cache write, prefill attention: a 512-token block went from 330 to 316 us) - the default, measured
// best on the 14-block decode stage, 3 = every kernel.
inline int& pdl_level() {
  static int level = 2;
  return level;
}

template <int OVERLAP = 3, typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (OVERLAP <= pdl_level()) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------------------------------------
// per-call batch metadata as the kernels see it (all DEVICE pointers, int32)
// ---------------------------------------------------------------------------------------------
struct BatchMeta {
  int n_seqs;
  int n_tokens;             // M = sum of q_lens
  int max_pages_per_seq;    // row stride of block_table
  const int32_t* q_lens;    // [n_seqs]
  const int32_t* ctx_lens;  // [n_seqs] cached tokens before this call
  const int32_t* cu_q;      // [n_seqs+1] first row of each sequence
  const int32_t* tok_seq;   // [M] batch-local sequence index of each row
  const int32_t* tok_pos;   // [M] absolute position of each row
  const int32_t* last_row;  // [n_seqs] row index of each sequence's last new token
  const int32_t* block_table;  // [n_seqs, max_pages_per_seq] page ids (batch-local rows)
};

struct ModelDims {
  int H, Hq, Hkv, D, F, V;
  int qkv_rows;       // (Hq + 2 Hkv) D
  int page_tokens;    // 16
  float eps, theta;
};

// KV pool of ONE layer: [n_pages][2 (K,V)][Hkv][page_tokens][D] fp16.  Within a token's row the 16-byte chunk c
// (elements 8c .. 8c+7) is stored at chunk position c ^ (slot & 7), slot = the token's index in its page: a page's
// 16 rows of one head (contiguous) then land in shared memory, by one bulk copy, already in the layout ldmatrix
// reads without bank conflicts.
__host__ __device__ __forceinline__ int kv_chunk_pos(int c, int slot) { return c ^ (slot & 7); }
__host__ __device__ __forceinline__ size_t kv_page_elems(int Hkv, int page_tokens, int D) {
  return (size_t)2 * Hkv * page_tokens * D;
}

// epilogues of the projection kernels
enum Epilogue : int {
  EPI_STORE_BF16 = 0,  // out_16[m, n] = acc            (16-bit results take the operands' type: bf16 or fp16)
  EPI_RESID_F32 = 1,   // out_f32[m, n] += acc         (residual stream)
  EPI_SWIGLU_BF16 = 2, // out_16[m, n] = silu(acc_gate) * acc_up, gate row n, up row n + N
  EPI_STORE_F32 = 3    // out_f32[m, n] = acc          (logits, q/k/v)
};

// ---------------------------------------------------------------------------------------------
// launchers (each enqueues on `st`, returns the number of kernels launched or a negative status)
// ---------------------------------------------------------------------------------------------
int launch_embed(const int32_t* ids, const __nv_bfloat16* E, float* x, int M, int H, int V, cudaStream_t st);
int launch_copy_f32(const float* src, float* dst, size_t n, cudaStream_t st);
// h = norm(x) as bf16, or as fp16 when out_f16 (h then points to __half storage)
int launch_rmsnorm(const float* x, const __nv_bfloat16* g, void* h, bool out_f16, int M, int H, float eps,
                   const int32_t* row_index /* optional gather of rows, may be null */, cudaStream_t st,
                   bool gains_are_constant = false /* true: g is a loaded weight, never a predecessor's output */,
                   float* defer_scale = nullptr /* non-null: h = x * g * 2^e, defer_scale[r] = rstd / 2^e (fp16 only) */);
// rotate q, k of every row (fp32 in), write q as fp16 [M, Hq*D] and append k, v as fp16 to the pages
// row_scale non-null: rows are multiplied by row_scale[t] first, and q, k are stored as two fp16 terms (the low
// terms to q_lo [M, Hq*D] and klo_layer [page][Hkv][16][D])
int launch_rope_kv_write(const float* qkv, __half* q16, __half* kv_layer, const float2* rope_table,
                         const BatchMeta& bm, const ModelDims& d, cudaStream_t st, const float* row_scale = nullptr,
                         __half* q_lo = nullptr, __half* klo_layer = nullptr);
// q: fp16 [M, q_stride]
int launch_attn_prefill(const __half* q, int q_stride, const __half* kv_layer, __half* attn_out,
                        const BatchMeta& bm, const ModelDims& d, cudaStream_t st);
// the same with two-term queries and keys (see launch_rope_kv_write)
int launch_attn_prefill_split(const __half* q, const __half* q_lo, int q_stride, const __half* kv_layer,
                              const __half* klo_layer, __half* attn_out, const BatchMeta& bm, const ModelDims& d,
                              cudaStream_t st);
// decode attention: one query row per sequence; `scratch` holds split partials
size_t attn_decode_scratch_bytes(int max_seqs, int Hq, int D, int max_splits);
int attn_decode_splits(int n_seqs, int Hkv, int max_ctx);
int launch_attn_decode(const __half* q, int q_stride, const __half* kv_layer, __half* attn_out,
                       float* scratch, int n_splits, const BatchMeta& bm, const ModelDims& d, cudaStream_t st);

// decode attention of the stage path, fused with what surrounds it: rotates the new token's q and k (fp32
// projection output, one row per sequence), appends k, v to the pages, attends over n_splits context slices
// (a thread-block cluster, n_splits <= 8) and merges them.  `err`: device word set if a bounded wait expires.
int attn_decode_fused_splits(int n_seqs, int Hkv, int max_ctx);
int& attn_global_merge();           // 1 (default): the stage's decode attention merges its splits through global memory
int& first_block_split();           // 1 (default): the model's first block keeps two-term queries / keys
int& attn_fused_splits_override();  // 0 = built-in choice
int& attn_fused_slots_override();   // 0 = built-in choice
// row_scale / klo_layer (both or neither): the first block's variant - rows of qkv32 are multiplied by row_scale[b]
// first, and queries / keys are two-term fp16 values (the keys' low terms cached in klo_layer [page][Hkv][16][D]).
int launch_attn_decode_fused(const float* qkv32, int stride, __half* kv_layer, const float2* rope_table, __half* attn_out,
                             int n_splits, int slots, int* err, const BatchMeta& bm, const ModelDims& d, cudaStream_t st,
                             const float* row_scale = nullptr, __half* klo_layer = nullptr,
                             float* scratch = nullptr, int* tickets = nullptr);
// scratch / tickets (both or neither): the splits meet in global memory instead of a cluster (see the kernel);
// scratch holds n_seqs * Hkv * n_splits rows of attn_fused_scratch_row(G, D) floats, tickets n_seqs * Hkv zeroed ints
inline size_t attn_fused_scratch_row(int G, int D) { return (size_t)G * D + 16; }

}  // namespace hyp
