/*
 * hyperion.h - C ABI of libhyperion: run one pipeline stage of a decoder-only LLM on one GPU
 * (batched prefill and paged-KV decode), profile its blocks, and partition / schedule with the
 * paper's two host algorithms.
 *
 * Paper: "Hyperion: Hierarchical Scheduling for Parallel LLM Acceleration in Multi-tier Networks".
 * The paper models the LLM as N sequential decoder blocks B_1 -> B_2 -> ... -> B_N (Section III-A),
 * assigns tier j the contiguous index set I_j(p) = { i : p_{j-1} < i <= p_j } (Section III-C), and
 * feeds tier 1 the tokenised prompt and every later tier the previous tier's activations
 * (Section III-D, sub-problem 2).  A `hyp_stage` is exactly one such I_j(p) resident on one GPU.
 *
 * General rules
 *  - Every function returns 0 (HYP_OK) or a negative hyp_status.  All argument checks run on the
 *    host before anything is launched; on error no output buffer is touched.  Nothing aborts and no
 *    C++ exception crosses this boundary.
 *  - "DEVICE" pointers are CUDA global-memory addresses on the stage's device; "HOST" pointers are
 *    ordinary CPU addresses.  Each argument says which it is.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  prefill/decode
 *    only enqueue work on it and return; outputs are valid once the caller has synchronised the
 *    stream.  The *_host variants synchronise the stream themselves before returning.
 *  - The library owns weights, KV pages, block tables and workspace; they are allocated once in
 *    hyp_stage_create, so prefill/decode never allocate.  The caller owns `in` / `out`.
 *  - A stage is not thread-safe: one thread at a time per stage.  hyp_split_dp, hyp_sched_rt and
 *    hyp_strerror are pure host functions, thread-safe, and never touch a GPU.
 *  - Activations crossing a stage boundary are fp32, row-major [M, hidden], rows packed in batch
 *    order (all rows of sequence 0, then sequence 1, ...).
 *  - Precision.  The residual stream, all accumulation, softmax and norms are fp32.  Every projection
 *    (q/k/v, O, gate/up, down, LM head) multiplies fp16 activations with weights held as fp16 (the bf16
 *    values converted once at load: exact for |w| >= 2^-17, else off by < 3e-8) into fp32.  The q/k/v
 *    projection writes fp32; q, k are rotated in fp32 and q, k, v rounded once to fp16; the KV cache and
 *    the softmax weights are fp16 (values saturate at +-65504).  With bf16 activations instead, their
 *    8 mantissa bits alone put the per-step logits of the 5120-wide 40-block model outside the 5e-2
 *    tolerance.
 *  - Prefill rows: the residual projections split K across CTAs for row counts up to 2048 and add
 *    partial sums with floating-point atomics, so the last bits of a prefill result may differ from
 *    run to run; decode is bit-reproducible.
 */
#ifndef HYPERION_H
#define HYPERION_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HYP_API __attribute__((visibility("default")))
#else
#define HYP_API
#endif

typedef enum {
  HYP_OK = 0,
  HYP_EINVAL = -1,      /* bad argument (null pointer, shape, range, length mismatch)             */
  HYP_ENOMEM = -2,      /* device or host allocation failed                                       */
  HYP_ECAPACITY = -3,   /* KV pages, context length, batch or token workspace exhausted           */
  HYP_EINFEASIBLE = -4, /* hyp_split_dp: no memory-feasible partition (or N < T);                 */
                        /* hyp_sched_rt: no available node with enough memory                     */
  HYP_ECUDA = -5,       /* a CUDA call failed; hyp_last_cuda_error() gives the cudaError_t        */
  HYP_ESTATE = -6,      /* stage not ready (a weight tensor was never loaded)                     */
  HYP_ETIMEOUT = -7     /* a bounded device-side wait expired inside a kernel; reported by the     */
                        /* calls that synchronise (*_host, hyp_stage_profile); results are invalid */
} hyp_status;

typedef struct hyp_stage hyp_stage; /* opaque, library-owned */

/* Decoder shape and capacity limits.  Plain data, caller-owned, copied by hyp_stage_create.
 * The block it describes is the one named in Section III-A: RMSNorm -> grouped-query attention
 * with rotary position encoding -> RMSNorm -> SwiGLU feed-forward, a residual around each
 * sub-layer, the norm applied before the sub-layer.  No biases anywhere. */
typedef struct {
  int32_t n_layers_total; /* N: blocks in the whole model                                          */
  int32_t hidden;         /* H, multiple of 8                                                      */
  int32_t n_q_heads;      /* Hq, multiple of n_kv_heads                                            */
  int32_t n_kv_heads;     /* Hkv; query head h reads KV head floor(h / (Hq/Hkv))                   */
  int32_t head_dim;       /* D: 64 or 128                                                          */
  int32_t ffn;            /* F: SwiGLU inner width, multiple of 8                                  */
  int32_t vocab;          /* V, multiple of 8 (rows of the logits matrix start on 16-byte boundaries) */
  float rms_eps;          /* y = x / sqrt(mean(x^2) + eps) * g                                     */
  float rope_theta;       /* pair (i, i + D/2) rotated by pos * theta^(-2i/D), positions from 0    */
  int32_t kv_block_size;  /* tokens per KV page; must be 16                                        */
  int32_t max_seqs;       /* sequence slots (seq_id in [0, max_seqs))                              */
  int32_t max_ctx;        /* longest context (cached + new tokens) any sequence may reach          */
  int32_t max_tokens;     /* most rows (sum of q_lens) a single prefill call may carry             */
  int32_t kv_pages;       /* pages in the pool; 0 = max_seqs * ceil(max_ctx / 16)                  */
} hyp_cfg;

/* Weight tensor ids for hyp_stage_load.  Every matrix is given as bf16, row-major [out, in] (y = x W^T).
 * The library keeps its own copy of the projection matrices: fp16 values in a tiled order (16-row x 64-k
 * tiles, all k-blocks of a 16-row strip contiguous; see hyperion_ops.h), which decode streams strip by
 * strip and prefill reads tile by tile. */
enum {
  HYP_W_QKV = 0,     /* [(Hq + 2 Hkv) D, H]: rows = Q heads, then K heads, then V heads               */
  HYP_W_O = 1,       /* [H, Hq D]                                                                   */
  HYP_W_GATE_UP = 2, /* [2 F, H]: rows = gate (F) then up (F)                                       */
  HYP_W_DOWN = 3,    /* [H, F]                                                                      */
  HYP_W_NORM1 = 4,   /* [H] gain of the pre-attention RMSNorm                                       */
  HYP_W_NORM2 = 5,   /* [H] gain of the pre-FFN RMSNorm                                             */
  HYP_W_EMBED = 6,   /* [V, H]  (layer = -1; only if the stage holds block 0)                       */
  HYP_W_FINAL_NORM = 7, /* [H]  (layer = n_layers_total; only if the stage holds the last block)    */
  HYP_W_LM_HEAD = 8  /* [V, H]  (layer = n_layers_total; untied from the embedding)                 */
};

#define HYP_BATCH_ALL_LOGITS 1 /* last stage, prefill: return logits of every row, not only last   */
#define HYP_MAX_DECODE_BATCH 128

/* One call's batch.  All arrays are HOST memory, caller-owned, and fully read before the call
 * returns.  Rows of the batch are packed in sequence order: M = sum(q_lens). */
typedef struct {
  int32_t n_seqs;
  const int32_t* seq_ids;  /* [n_seqs] distinct slots in [0, max_seqs)                              */
  const int32_t* q_lens;   /* [n_seqs] new tokens in this call (>= 1; decode: exactly 1)            */
  const int32_t* ctx_lens; /* [n_seqs] tokens already cached for the slot; must equal the           */
                           /*          library's own count (0 for a new sequence)                   */
  int32_t flags;           /* 0 or HYP_BATCH_ALL_LOGITS                                             */
} hyp_batch;

/* Create the stage holding blocks layer_lo .. layer_hi-1 (0-based, hi exclusive; the paper's
 * I_j(p) with p_{j-1} = layer_lo, p_j = layer_hi, Section III-C) on the current CUDA device.
 * Allocates weights, KV pool, block tables and workspace.  *out is written only on success.
 * Errors: HYP_EINVAL (shape / range), HYP_ENOMEM, HYP_ECUDA. */
HYP_API int hyp_stage_create(int32_t layer_lo, int32_t layer_hi, const hyp_cfg* cfg, hyp_stage** out);

/* Copy one weight tensor into the stage (device-to-device, asynchronous on `stream`; projection
 * matrices are converted to fp16 and re-tiled on the way).
 * layer: block index in [layer_lo, layer_hi), or -1 / n_layers_total for embed / head tensors.
 * src: DEVICE, bf16, `bytes` must equal the tensor's exact size.  The caller may free src after
 * synchronising the stream.  Errors: HYP_EINVAL, HYP_ECUDA. */
HYP_API int hyp_stage_load(hyp_stage* s, int32_t layer, int32_t tensor_id, const void* src, size_t bytes,
                   void* stream);

/* Prefill: push q_lens[i] new rows of every listed sequence through the stage's blocks in order
 * (B_i -> B_{i+1}, Section III-A), appending their rotated keys and values to the paged cache.
 * ctx_lens[i] > 0 continues a sequence (chunked prefill): new rows attend to the cached tokens
 * and causally to each other.
 *   in : DEVICE. int32 token ids [M] if layer_lo == 0 (the tokenised prompt of tier 1), else fp32
 *        activations [M, H] from the previous stage.
 *   out: DEVICE. fp32 activations [M, H]; or, if layer_hi == n_layers_total, fp32 logits
 *        [n_seqs, V] of each sequence's last row ([M, V] with HYP_BATCH_ALL_LOGITS).
 *        Both 16-byte aligned (ids: 4-byte).
 * Errors: HYP_EINVAL, HYP_ECAPACITY (M > max_tokens, context > max_ctx, pool empty), HYP_ESTATE,
 * HYP_ECUDA.  Whatever the code, a call that does not return HYP_OK leaves the slot lengths
 * (hyp_stage_seq_len) and the page pool as they were before it: arguments are checked before anything
 * is reserved, and pages reserved for a call whose enqueue then fails (HYP_ECUDA) are handed back. */
HYP_API int hyp_stage_prefill(hyp_stage* s, const hyp_batch* batch, const void* in, void* out, void* stream);

/* Decode: one new row per sequence (q_lens all 1, n_seqs <= HYP_MAX_DECODE_BATCH), attending to
 * the sequence's whole cache.  Same data flow as prefill with M = n_seqs; uses the
 * weight-streaming kernels.  in: ids [B] or activations [B, H]; out: [B, H] or logits [B, V].
 * The kernel sequence of a step is captured into a CUDA graph the second time a (batch size,
 * attention split count) pair is seen and replayed afterwards; `in` is copied into and `out` out of
 * fixed library buffers around the replay, so the caller's pointers may change from call to call.
 * While hyp_stage_kernel_timing is active the step is launched kernel by kernel instead. */
HYP_API int hyp_stage_decode(hyp_stage* s, const hyp_batch* batch, const void* in, void* out, void* stream);

/* Same two calls with HOST `in` / `out` buffers (pinned memory recommended): the library copies
 * the input to the device, runs the stage, copies the result back and synchronises `stream`
 * before returning. */
HYP_API int hyp_stage_prefill_host(hyp_stage* s, const hyp_batch* batch, const void* in, void* out, void* stream);
HYP_API int hyp_stage_decode_host(hyp_stage* s, const hyp_batch* batch, const void* in, void* out, void* stream);

/* Measure the per-block cost vectors the partitioner consumes: f_i as time, m_i as memory
 * (Section III-A defines f_i and m_i per block).  Runs the stage's blocks on scratch sequences
 * (`batch` sequences; mode 0 = a prefill of `ctx` rows each, mode 1 = one decode step at context
 * `ctx`) `iters` times after one warm-up and reports, per block of the stage,
 *   layer_ms[i]   : HOST float [layer_hi - layer_lo], median milliseconds (CUDA events);
 *   layer_bytes[i]: HOST size_t, weight bytes + KV bytes at (max_seqs, max_ctx) + workspace share.
 * Needs batch * ceil((ctx+1)/16) free pages; live sequences are not disturbed.  Synchronises. */
HYP_API int hyp_stage_profile(hyp_stage* s, int32_t mode, int32_t batch, int32_t ctx, int32_t iters,
                      float* layer_ms, size_t* layer_bytes, void* stream);

/* Kernel classes of the block sequence, for per-launch timing. */
enum {
  HYP_K_GEMM_QKV = 0, HYP_K_GEMM_O = 1, HYP_K_GEMM_GATE_UP = 2, HYP_K_GEMM_DOWN = 3,
  HYP_K_ATTN = 4, HYP_K_NORM = 5, HYP_K_ROPE = 6, HYP_K_LM_HEAD = 7
};
/* Bracket every launch of one kernel class with a CUDA event pair on the call's stream (at most
 * max_samples launches are recorded; kernel_class = -1 switches timing off).  Creating the events
 * happens here, not in prefill/decode.  Measurement aid for roofline reporting. */
HYP_API int hyp_stage_kernel_timing(hyp_stage* s, int32_t kernel_class, int32_t max_samples);
/* Wait for the recorded pairs, return their count and summed duration (HOST outputs), and reset
 * the sample counter. */
HYP_API int hyp_stage_kernel_timing_read(hyp_stage* s, int32_t* n_samples, double* total_ms);

/* Return a sequence's KV pages to the pool and zero its cached length. */
HYP_API int hyp_stage_free_seq(hyp_stage* s, int32_t seq_id);
/* Tokens currently cached for a slot, or a negative status. */
HYP_API int hyp_stage_seq_len(const hyp_stage* s, int32_t seq_id);
/* Free pages left in the pool, or a negative status. */
HYP_API int hyp_stage_free_pages(const hyp_stage* s);
/* Kernels launched by this stage since creation (for launch accounting). */
HYP_API int64_t hyp_stage_launch_count(const hyp_stage* s);
/* Release everything.  NULL is allowed. */
HYP_API void hyp_stage_destroy(hyp_stage* s);

/* HypSplit-DP (Algorithm 1; problem P1 of Section III-D): choose p = (p_1 .. p_{T-1}),
 * 1 <= p_1 < ... < p_{T-1} < N, minimising max_j L_j(p), L_j = (S_f[p_j] - S_f[p_{j-1}]) / C_j,
 * subject to S_m[p_j] - S_m[p_{j-1}] <= Mcap_j for every tier.  S_f, S_m are left-to-right prefix
 * sums in double.  The constant communication term of the objective is dropped as in Section IV-A.
 *   f, m : HOST double [N]   block compute cost (any unit, >= 0) and memory (>= 0)
 *   C    : HOST double [T]   tier capacity (> 0), same unit as f per unit time
 *   Mcap : HOST double [T]   tier memory limit (>= 0), same unit as m
 *   eps  : 0  -> exact: the monotone feasibility test of Algorithm 1 is bisected over the finite,
 *                sorted set of values a tier load can take, so the minimum is found exactly;
 *          >0 -> the same search may stop once the bracket around the optimum is narrower than
 *                eps (the paper's tolerance parameter): the result is a memory-feasible partition
 *                whose bottleneck is within eps of the optimum.
 *   p_out  : HOST int32 [T-1], 1-based index of the last block of tiers 1..T-1 (may be NULL if T==1)
 *   tau_out: HOST double, max_j L_j(p_out)
 * Ties between equally good partitions are resolved as Algorithm 1's predecessor choice implies
 * (each tier, from the last one back, takes the smallest feasible predecessor): the result is the
 * smallest vector when read as (p_{T-1}, ..., p_1).
 * Errors: HYP_EINVAL (null, N < 1, T < 1, negative cost, C <= 0, NaN), HYP_EINFEASIBLE. */
HYP_API int hyp_split_dp(int32_t N, int32_t T, const double* f, const double* m, const double* C,
                 const double* Mcap, double eps, int32_t* p_out, double* tau_out);

/* The partitioning steps of the two systems the paper compares against (Section V, the HEFT and GPipe baselines), on the
 * same inputs as hyp_split_dp, so that their bottleneck max_j L_j(p) can be set beside HypSplit-DP's on measured
 * per-block costs.  The paper names the strategies and gives no algorithm; the readings taken here:
 *   hyp_split_even   (GPipe's static split of the block chain into contiguous, equally long segments):
 *                    segments of equal block count, the N mod T leading tiers one block longer; costs,
 *                    capacities and memory limits play no part.  p_out and tau_out are always written for valid
 *                    arguments with N >= T; the return value is HYP_EINFEASIBLE if a segment exceeds its tier's
 *                    memory limit (the partition is reported, not repaired).
 *   hyp_split_greedy (the greedy, memory-checking partitioning step that precedes HEFT's scheduling): tiers are filled in order;
 *                    tier j keeps taking the next block while its memory limit holds and its load stays within
 *                    its capacity-proportional share S_f[N] * C_j / sum(C), takes at least one block, and leaves
 *                    one block for every later tier; the last tier takes the rest.  HYP_EINFEASIBLE (outputs
 *                    untouched) if a tier cannot hold its first block or the last tier cannot hold the rest.
 * Arguments, units and the other errors: as hyp_split_dp (no eps).  Pure host functions, thread-safe. */
HYP_API int hyp_split_even(int32_t N, int32_t T, const double* f, const double* m, const double* C,
                           const double* Mcap, int32_t* p_out, double* tau_out);
HYP_API int hyp_split_greedy(int32_t N, int32_t T, const double* f, const double* m, const double* C,
                             const double* Mcap, int32_t* p_out, double* tau_out);

/* Real-time state of one node of a tier, as Algorithm 2 (HypSched-RT) reads it. */
typedef struct {
  double C;        /* computing capacity C_{j,k} (> 0)                                             */
  double M_avail;  /* memory currently available                                                   */
  double F_rem;    /* remaining workload of the running task (0 if idle)                           */
  double F_wait;   /* total workload of the tasks waiting in the node's FIFO queue                 */
  int32_t available;
} hyp_node_state;

/* HypSched-RT (Algorithm 2, Section IV-B): among nodes that are available and have
 * M_avail >= m_act, pick k* minimising (F_rem + F_wait + F_new) / C; a strictly smaller cost is
 * required to displace an earlier node, so the lowest index wins ties.
 * nodes: HOST [K].  k_out: HOST int32, 0-based node index.  Errors: HYP_EINVAL, HYP_EINFEASIBLE. */
HYP_API int hyp_sched_rt(double F_new, double m_act, const hyp_node_state* nodes, int32_t K, int32_t* k_out);

HYP_API const char* hyp_strerror(int code);
/* cudaError_t of the most recent failing CUDA call on this thread (0 if none). */
HYP_API int hyp_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HYPERION_H */
