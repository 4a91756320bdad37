/*
 * hyperion_ops.h - single-kernel entry points of libhyperion.
 *
 * These run one step of the decoder block (Section III-A of the paper names the steps: RMSNorm,
 * grouped-query attention with rotary encoding, SwiGLU feed-forward) on caller-owned DEVICE buffers.
 * They exist for unit tests, per-kernel measurement and for callers that assemble their own block
 * sequence; hyp_stage_* (hyperion.h) is the full path.  All pointers are DEVICE unless marked HOST;
 * `stream` is a cudaStream_t as void*; calls enqueue and return; status codes as in hyperion.h.
 *
 * KV page pool layout of ONE block (fp16): [n_pages][2 (K then V)][n_kv_heads][16 tokens][head_dim].
 * Inside a token's head_dim-wide row the 16-byte chunk c (elements 8c .. 8c+7) is stored at chunk position
 * c ^ (slot & 7), slot = the token's index in its page: the 16 rows of a page and head are contiguous, and one
 * bulk copy lands them in shared memory in the bank-conflict-free order the tensor-core loads read.
 * Attention operands (queries, cached keys and values) are IEEE fp16: the softmax weights need more
 * mantissa than bf16 offers to stay inside the library's logit tolerance; values are saturated at
 * +-65504 when the library writes them.
 * A block table row lists, in order, the page ids that hold a sequence's tokens 0-15, 16-31, ...
 */
#ifndef HYPERION_OPS_H
#define HYPERION_OPS_H

#include "hyperion.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Epilogues of hyp_op_gemm. */
enum {
  HYP_EPI_STORE_BF16 = 0, /* out bf16 [M, ldo]: out[m, n] = acc                                     */
  HYP_EPI_RESID_F32 = 1,  /* out fp32 [M, ldo]: out[m, n] += acc  (residual stream)                 */
  HYP_EPI_SWIGLU_BF16 = 2,/* out bf16 [M, ldo]: SiLU(acc over weight row n) * (acc over row n + N); */
                          /* w holds 2N rows: gate rows then up rows                                */
  HYP_EPI_STORE_F32 = 3   /* out fp32 [M, ldo]: out[m, n] = acc                                     */
};

typedef struct {
  int32_t n_q_heads, n_kv_heads, head_dim; /* head_dim 64 or 128; n_q_heads / n_kv_heads in 1,2,4,8 */
} hyp_attn_shape;

/* RMSNorm (Section III-A): out[m, :] = x[m, :] / sqrt(mean(x[m, :]^2) + eps) * g.
 * x fp32 [M, H], g bf16 [H], out bf16 [M, H]; H multiple of 8. */
HYP_API int hyp_op_rmsnorm(const float* x, const void* g, void* out, int32_t M, int32_t H, float eps, void* stream);

/* Packed weight layout.  The projection kernels read a weight matrix w[n, k] (row n = output feature, [out, in]
 * as in y = x W^T) from a tiled copy that the library makes once: tiles of 16 rows x 64 k (2 KB each), all
 * k-blocks of a 16-row strip contiguous, each 128-byte tile row stored with its 16-byte chunks XOR-permuted by
 * (row & 7) (the shared-memory swizzle of the tensor-core operands, applied at load time), zero padding to whole
 * tiles.  Decode then streams every strip as one sequential run; prefill fetches 128-row operand tiles as eight
 * 2 KB pieces.  hyp_op_weight_packed_bytes gives the size of that copy (0 on bad arguments); hyp_op_pack_weight
 * writes it.
 *   w       bf16 [N, K] row-major (swiglu != 0: [2N, K], N gate rows then N up rows), 16-byte aligned
 *   packed  at least hyp_op_weight_packed_bytes(N, K, swiglu) bytes, 128-byte aligned; values stay bf16
 * K multiple of 8.  Errors: HYP_EINVAL, HYP_ECAPACITY (packed_bytes too small). */
HYP_API size_t hyp_op_weight_packed_bytes(int32_t N, int32_t K, int32_t swiglu);
HYP_API int hyp_op_pack_weight(const void* w, int32_t N, int32_t K, int32_t swiglu, void* packed, size_t packed_bytes,
                               void* stream);

/* Projection (the QKV, O, gate/up, down and LM-head contractions of the block):
 * acc[m, n] = sum_k a[m, k] * w[n, k], bf16 inputs, fp32 accumulation, then `epilogue`.  (The same kernels
 * run inside hyp_stage_* with fp16 operands; this entry point exposes the bf16 instantiation.)
 * a bf16 [M, K] row-major; w_packed = the output of hyp_op_pack_weight for the same N, K and
 * swiglu = (epilogue == HYP_EPI_SWIGLU_BF16); K multiple of 8, N and ldo multiples of 16 and 8 unless M <= 8.
 * M <= 8 runs the weight-streaming kernel, larger M the tcgen05 kernels (for 9-128 rows the plain-store
 * epilogues of narrow matrices take the variant with the operands swapped and K split over a cluster).
 * The first call on a process allocates one device word for error reporting. */
HYP_API int hyp_op_gemm(const void* a, const void* w_packed, int32_t M, int32_t N, int32_t K, int32_t epilogue,
                        void* out, int32_t ldo, void* stream);

/* The same two calls for the fp16 instantiation, the one hyp_stage_* runs (reading 11 of the block's arithmetic:
 * fp16 operands, fp32 accumulation): hyp_op_pack_weight_f16 converts the bf16 matrix to fp16 while tiling it
 * (exact for |w| >= 2^-17, saturating at +-65504); hyp_op_gemm_f16 takes `a` as fp16 [M, K] and such a packed
 * copy, and its 16-bit epilogues write fp16.  Everything else as above. */
HYP_API int hyp_op_pack_weight_f16(const void* w, int32_t N, int32_t K, int32_t swiglu, void* packed, size_t packed_bytes,
                                   void* stream);
HYP_API int hyp_op_gemm_f16(const void* a, const void* w_packed, int32_t M, int32_t N, int32_t K, int32_t epilogue,
                            void* out, int32_t ldo, void* stream);

/* Device-side wait status.  Every wait inside the library's kernels (on a copy's completion, on tensor memory, on a
 * peer CTA) is bounded; a kernel whose wait runs out records a small non-zero code in one device word, unwinds and
 * returns by itself (its results are invalid).  The calls that synchronise report that word as HYP_ETIMEOUT; this
 * call reads it for the others: it synchronises the device, writes the code to *code_out (HOST; 0 = no wait ever
 * expired) and, if clear != 0, resets the word.  Errors: HYP_EINVAL, HYP_ECUDA. */
HYP_API int hyp_device_wait_status(int32_t* code_out, int32_t clear);

/* Process-wide tuning switches (measurement aids; the defaults are the measured best).
 *   HYP_TUNE_PDL           which kernels are launched with programmatic dependent launch, so that their
 *                          prologue and weight prefetch may overlap the predecessor's tail: 0 none, 1 the
 *                          weight-streaming projections, 2 also the norms between them, 3 every kernel
 *   HYP_TUNE_STREAM_SLOTS  ring slots per warp of the weight-streaming kernel, 1..8 (0 = built-in choice)
 *   HYP_TUNE_ATTN_SPLITS   context splits (cluster size) of the stage's decode attention, 1..8 (0 = built-in)
 *   HYP_TUNE_ATTN_SLOTS    ring slots per warp of that kernel, 2..4 (0 = built-in)
 *   HYP_TUNE_STREAM_ROTATION  CTA b of the weight-streaming kernel starts its K walk at copy (b * value) mod copies
 *                          (0 = all CTAs walk K in the same order)
 *   HYP_TUNE_SWAP_MIN_ROWS / HYP_TUNE_SWAP_MAX_ROWS  row counts (1..128; min 129 or max 0 = never) for which a
 *                          projection may run on the swapped-operand tensor-core kernel (a minimum below 9
 *                          also takes those row counts away from the weight-streaming kernel)
 *   HYP_TUNE_SWAP_EPILOGUES  bit mask over the HYP_EPI_* values: which epilogues may take that kernel
 *                          (default: the two plain stores; it is only chosen for matrices of < 100 tiles of 256 rows)
 *   HYP_TUNE_PREFILL_ATTN_TC  value != 0 (the default): prefill attention at head_dim 128 runs on the tcgen05 kernel
 *                          (scores, probabilities and output in tensor memory, 128 query rows per CTA); 0: on the
 *                          mma.sync kernel that serves the other head sizes
 *   HYP_TUNE_FIRST_BLOCK_SPLIT  value != 0 (the default): in stages that hold block 0 the attention scores of that
 *                          block are formed from two-term fp16 queries and keys (~21 significant bits) and the
 *                          RMSNorm factor is applied after the q/k/v projection, whose input is then the embedding
 *                          row itself; 0: block 0 runs like every other block (11-bit operands)
 *   HYP_TUNE_TILE_224      value != 0 (the default): projections of more than 128 rows with whole-tile epilogues may
 *                          use 256 x 224 tiles per CTA pair where that fills the last wave of the GPU better than
 *                          256 x 256 (e.g. 7680 columns at 512 rows: 70 tiles on 74 pairs); 0: always 256 x 256
 *   HYP_TUNE_STREAM_ACT_TMA  value != 0 (the default): the weight-streaming kernel brings the activations of every weight
 *                          copy's k range into its ring by a TMA box load (when K is a multiple of 64); 0: each
 *                          lane reads its fragment entries from global memory
 *   HYP_TUNE_ATTN_GLOBAL_MERGE  value != 0 (the default): the stage's decode attention merges its context splits through
 *                          a scratch row per split in global memory (the CTA that finishes last merges) and is
 *                          launched early; 0: the splits form a thread-block cluster and merge through distributed
 *                          shared memory (what hyp_op_attn_decode_fused always does)
 *   HYP_TUNE_STREAM_ACT_DEPTH  how many of its weight copies ahead a warp of the weight-streaming kernel fetches its
 *                          activation fragments, 1..3 (0 = built-in: 2)
 *   HYP_TUNE_WAIT_LIMIT_US  limit of the weight-streaming kernel's bounded waits in microseconds (0 = the built-in
 *                          4 s; the other kernels always use 4 s)
 *   HYP_TUNE_STREAM_WITHHOLD_COPY  value != 0: the NEXT launch of the weight-streaming kernel leaves one weight copy
 *                          unissued, so that one warp's wait runs into the limit and the kernel takes its
 *                          give-up path (records code 4, lets its other copies land, returns).  One-shot; exists
 *                          so that the HYP_ETIMEOUT path can be exercised without faulting or hanging anything.
 * Affects launches made after the call; decode graphs already captured keep their setting. */
enum { HYP_TUNE_PDL = 0, HYP_TUNE_STREAM_SLOTS = 1, HYP_TUNE_ATTN_SPLITS = 2, HYP_TUNE_ATTN_SLOTS = 3,
       HYP_TUNE_STREAM_ROTATION = 4, HYP_TUNE_SWAP_MIN_ROWS = 5, HYP_TUNE_SWAP_MAX_ROWS = 6, HYP_TUNE_SWAP_EPILOGUES = 7,
       HYP_TUNE_PREFILL_ATTN_TC = 8, HYP_TUNE_FIRST_BLOCK_SPLIT = 9, HYP_TUNE_TILE_224 = 10,
       HYP_TUNE_WAIT_LIMIT_US = 11, HYP_TUNE_STREAM_WITHHOLD_COPY = 12, HYP_TUNE_STREAM_ACT_DEPTH = 13, HYP_TUNE_STREAM_ACT_TMA = 14,
       HYP_TUNE_ATTN_GLOBAL_MERGE = 15 };
HYP_API int hyp_tune(int32_t key, int32_t value);

/* Number of context splits hyp_op_attn_decode would pick for this batch, and the scratch bytes
 * that n_splits needs.  Pure host helpers. */
HYP_API int hyp_op_attn_decode_splits(int32_t n_seqs, int32_t n_kv_heads, int32_t max_ctx);
HYP_API size_t hyp_op_attn_decode_scratch_bytes(int32_t n_seqs, int32_t n_q_heads, int32_t head_dim, int32_t n_splits);

/* Decode attention (grouped-query attention of Section III-A for one new token per sequence):
 * out[b, h, :] = softmax_j(q[b, h, :] . k[b, j, h/G, :] / sqrt(D)) v[b, j, h/G, :] over cached
 * positions j = 0 .. ctx_lens[b] (the new token's k, v must already be in the cache).
 *   q          fp16 [n_seqs, q_stride], head h of row b at q + b*q_stride + h*D (already rotated)
 *   kv_pages   one block's page pool (layout above)
 *   block_table int32 [n_seqs, max_pages_per_seq];  ctx_lens int32 [n_seqs]
 *   scratch    fp32, at least hyp_op_attn_decode_scratch_bytes(...) bytes: per-split partial results
 *   out        fp16 [n_seqs, n_q_heads * D]
 * n_splits in [1, 32]. */
HYP_API int hyp_op_attn_decode(const hyp_attn_shape* shape, int32_t n_seqs, const void* q, int32_t q_stride,
                               const void* kv_pages, const int32_t* block_table, int32_t max_pages_per_seq,
                               const int32_t* ctx_lens, int32_t n_splits, float* scratch, size_t scratch_bytes,
                               void* out, void* stream);

/* One decode step of the attention sub-layer as hyp_stage_decode runs it, in a single launch: rotary encoding
 * (Section III-A: the block's grouped-query attention carries a rotary position encoding) of the new token's query and key,
 * append of its key and value to the paged cache, attention of the new token over positions
 * 0 .. ctx_lens[b] (itself included) and the merge of the context splits (a thread-block cluster per sequence
 * and KV head, merged through distributed shared memory; no scratch buffer).
 *   qkv        fp32 [n_seqs, stride]: the q/k/v projection of the new token, [Q heads | K heads | V heads], each
 *              head head_dim wide, not rotated; stride >= (n_q_heads + 2 n_kv_heads) * head_dim
 *   kv_pages   one block's page pool (layout above), READ AND WRITTEN: the new token's rotated key and its value
 *              are stored (fp16) at position ctx_lens[b]; the page holding that position must already be
 *              listed in the sequence's block-table row
 *   rope_table fp32 [positions, head_dim / 2, 2]: (cos, sin) of pos * theta^(-2i / head_dim); must cover every
 *              ctx_lens[b] (not checked: the lengths live on the device)
 *   n_splits   1 .. 8 context splits, 0 = the library's choice
 *   out        fp16 [n_seqs, n_q_heads * head_dim]
 * The first call on a process allocates one device word for error reporting (bounded waits). */
HYP_API int hyp_op_attn_decode_step(const hyp_attn_shape* shape, int32_t n_seqs, const float* qkv, int32_t stride,
                                    void* kv_pages, const int32_t* block_table, int32_t max_pages_per_seq,
                                    const int32_t* ctx_lens, const float* rope_table, int32_t n_splits, void* out,
                                    void* stream);

/* Decode attention for callers that must not allocate device memory.  (The paper has no counterpart
 * to this call; it is a packaging variant of hyp_op_attn_decode.)
 *
 * Some users of this library cannot call cudaMalloc at the point where they need attention: an
 * inference server that handed all free HBM to its own KV-cache pool at start-up, a plug-in running
 * inside a host application whose memory budget is fixed after initialisation, or a latency-critical
 * loop where an allocation's implicit device-wide synchronisation is not acceptable.  For them the
 * per-split partial results go to a fixed HYP_STATIC_SCRATCH_BYTES (4 MiB) array that is part of the
 * library image: every GPU that loads the library holds it until the process exits.  The caller
 * passes inputs and outputs exactly as for hyp_op_attn_decode; there is no scratch argument.
 *
 *  - Limit: hyp_op_attn_decode_scratch_bytes(n_seqs, n_q_heads, head_dim, n_splits) must not exceed
 *    HYP_STATIC_SCRATCH_BYTES; otherwise the call returns HYP_ECAPACITY and launches nothing
 *    (4 MiB covers e.g. 8 sequences x 40 heads x 24 splits at head_dim 128).  Use fewer splits, a
 *    smaller batch, or hyp_op_attn_decode with your own buffer.
 *  - The call performs no cudaMalloc/cudaFree and calls no allocating library routine.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current) and caches it; make that first call before starting any stream capture.
 *  - All calls on a device share the one array and it keeps whatever the previous call left there.
 *    Nothing needs clearing (each call overwrites every slot it later reads), but two calls whose
 *    kernels can overlap on the GPU - different streams without an ordering between them - race on
 *    it.  Keep calls on one stream, or order them with events.
 * Other arguments, layouts and errors: as hyp_op_attn_decode. */
#define HYP_STATIC_SCRATCH_BYTES (4u << 20)
HYP_API int hyp_op_attn_decode_static(const hyp_attn_shape* shape, int32_t n_seqs, const void* q, int32_t q_stride,
                                      const void* kv_pages, const int32_t* block_table, int32_t max_pages_per_seq,
                                      const int32_t* ctx_lens, int32_t n_splits, void* out, void* stream);

/* Prefill attention: the same definition for M query rows packed sequence by sequence.  Sequence i
 * owns rows cu_q[i] .. cu_q[i+1]-1; its row r sits at absolute position ctx_lens[i] + (r - cu_q[i]) and
 * sees cached positions 0 .. its own (all of the sequence's k, v, new rows included, must already be in
 * the cache).
 *   q fp16 [M, q_stride]; cu_q int32 [n_seqs + 1] (cu_q[n_seqs] = M); ctx_lens int32 [n_seqs];
 *   block_table int32 [n_seqs, max_pages_per_seq]; out fp16 [M, n_q_heads * D]. */
HYP_API int hyp_op_attn_prefill(const hyp_attn_shape* shape, int32_t n_seqs, int32_t M, const void* q,
                                int32_t q_stride, const void* kv_pages, const int32_t* block_table,
                                int32_t max_pages_per_seq, const int32_t* cu_q, const int32_t* ctx_lens, void* out,
                                void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HYPERION_OPS_H */
