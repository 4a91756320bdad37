// Stage runtime: owns weights, the paged KV pool, block tables (host side) and workspace, and
// drives the per-block kernel sequence for prefill and decode.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "hyperion.h"

namespace hyp {
static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }
}  // namespace hyp

using namespace hyp;
typedef __nv_bfloat16 bf16;

namespace {

constexpr int META_RING = 4;

struct LayerW {
  // projection matrices in the packed fp16 layout of gemm_tc.cuh; gains as loaded (bf16)
  void *wqkv = nullptr, *wo = nullptr, *wgu = nullptr, *wd = nullptr;
  bf16 *g1 = nullptr, *g2 = nullptr;
  uint32_t loaded = 0;
  TcWeight tc_qkv, tc_o, tc_gu, tc_d;
};

}  // namespace

struct hyp_stage {
  hyp_cfg cfg;
  int lo = 0, hi = 0, L = 0, device = 0;
  bool first = false, last = false;
  ModelDims dims;
  std::vector<LayerW> layers;
  bf16 *embed = nullptr, *gf = nullptr;
  void* wlm = nullptr;  // packed fp16
  TcWeight tc_lm;
  uint32_t loaded_extra = 0;
  // KV cache (fp16)
  __half* kv_pool = nullptr;
  size_t kv_layer_elems = 0;
  int n_pages = 0, max_pages_per_seq = 0;
  std::vector<int32_t> free_pages;
  std::vector<std::vector<int32_t>> seq_pages;
  std::vector<int32_t> seq_len;
  // workspace
  int max_rows = 0;
  float* x = nullptr;
  float* qkv32 = nullptr;             // q | k | v straight from the projection's accumulators
  __half* q16 = nullptr;              // rotated queries
  // The model's first block (stages with layer_lo == 0) runs its attention scores at higher precision: the
  // projection's input is the embedding row times the gain times a power of two (exact in fp16 for unit gains),
  // the rest of the RMSNorm factor (row_scale) is applied to q, k, v afterwards, and q, k are kept as two fp16
  // terms (q16_lo; klo_pool [page][Hkv][16][D]).  Reason: the residual stream entering block 0 is tiny, so the
  // block's FFN sees its attention output almost alone and amplifies that branch's rounding errors ~10x more than
  // any later block does; measured on the 40-block Phi-3-medium shape, block 0's fp16 score errors alone made up
  // two thirds of the final logit error.
  float* row_scale = nullptr;
  __half* q16_lo = nullptr;
  __half* klo_pool = nullptr;
  float* attn_scratch = nullptr;  // decode attention: the context splits' partial outputs (merged by the last CTA)
  int* attn_tickets = nullptr;    // one counter per (sequence, KV head), zero between launches
  __half *h = nullptr, *attn = nullptr, *u = nullptr;  // projection inputs (fp16)
  TcAct tc_h, tc_attn, tc_u, tc_q16;
  int* err_host = nullptr;  // pinned: the device error word, copied behind a host-buffer call's last kernel
  std::vector<CUtensorMap> kv_maps;  // per block: the page pool as rows (tcgen05 prefill attention, head_dim 128)
  int max_splits = 8;
  float2* rope_table = nullptr;
  size_t workspace_bytes = 0;
  // metadata staging
  size_t meta_ints = 0;
  int32_t* meta_dev = nullptr;
  int32_t* meta_host[META_RING] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t meta_ev[META_RING] = {nullptr, nullptr, nullptr, nullptr};
  bool meta_used[META_RING] = {false, false, false, false};
  int ring_pos = 0;
  // staging for the *_host entry points
  void *io_in = nullptr, *io_out = nullptr;
  size_t io_in_bytes = 0, io_out_bytes = 0;
  int64_t launches = 0;
  // decode steps replay a captured CUDA graph (one per batch size and attention split count); the graph
  // reads its input from g_in and leaves its result in g_out
  struct DecodeGraph {
    int n = 0, n_splits = 0, n_launches = 0;
    cudaGraphExec_t exec = nullptr;  // null until the second use of the key (the first runs eagerly)
  };
  std::vector<DecodeGraph> graphs;
  bool graphs_ok = true;
  cudaStream_t cap_stream = nullptr;
  void *g_in = nullptr, *g_out = nullptr;
  // optional per-launch timing of one kernel class
  int time_cls = -1;
  std::vector<cudaEvent_t> time_ev;
  int time_n = 0;
};

namespace {

template <typename T>
int dev_alloc(T** p, size_t count) {
  if (count == 0) count = 1;
  cudaError_t e = cudaMalloc((void**)p, count * sizeof(T));
  if (e != cudaSuccess) {
    set_last_cuda_error((int)e);
    *p = nullptr;
    return e == cudaErrorMemoryAllocation ? HYP_ENOMEM : HYP_ECUDA;
  }
  return HYP_OK;
}

size_t tensor_elems(const hyp_stage* s, int tensor_id) {
  const ModelDims& d = s->dims;
  switch (tensor_id) {
    case HYP_W_QKV: return (size_t)d.qkv_rows * d.H;
    case HYP_W_O: return (size_t)d.H * d.Hq * d.D;
    case HYP_W_GATE_UP: return (size_t)2 * d.F * d.H;
    case HYP_W_DOWN: return (size_t)d.H * d.F;
    case HYP_W_NORM1:
    case HYP_W_NORM2:
    case HYP_W_FINAL_NORM: return (size_t)d.H;
    case HYP_W_EMBED:
    case HYP_W_LM_HEAD: return (size_t)d.V * d.H;
    default: return 0;
  }
}

// Rows per half, halves and K of a projection matrix (its packed form is sized from these).
bool proj_geometry(const hyp_stage* s, int tensor_id, int* rows, int* halves, int* K) {
  const ModelDims& d = s->dims;
  *halves = 1;
  switch (tensor_id) {
    case HYP_W_QKV: *rows = d.qkv_rows; *K = d.H; return true;
    case HYP_W_O: *rows = d.H; *K = d.Hq * d.D; return true;
    case HYP_W_GATE_UP: *rows = d.F; *halves = 2; *K = d.H; return true;
    case HYP_W_DOWN: *rows = d.H; *K = d.F; return true;
    case HYP_W_LM_HEAD: *rows = d.V; *K = d.H; return true;
    default: return false;
  }
}
size_t proj_packed_bytes(const hyp_stage* s, int tensor_id) {
  int rows, halves, K;
  if (!proj_geometry(s, tensor_id, &rows, &halves, &K)) return 0;
  return tc_packed_bytes(rows, halves, K);
}
int dev_alloc_bytes(void** p, size_t bytes) {
  uint8_t* q = nullptr;
  const int rc = dev_alloc(&q, bytes);
  *p = q;
  return rc;
}

struct HostBatch {
  int n = 0, M = 0;
  std::vector<int32_t> packed;  // q_lens | ctx_lens | cu_q | last_row | tok_seq | tok_pos | block_table
  size_t off_q, off_ctx, off_cu, off_last, off_tseq, off_tpos, off_bt;
  // what admission changed, so that a call that fails after it can put the tables back
  struct Undo { int32_t id, old_len; size_t old_pages; };
  std::vector<Undo> undo;
};

void layout_meta(HostBatch& hb, int n, int M, int mpps) {
  hb.n = n;
  hb.M = M;
  hb.off_q = 0;
  hb.off_ctx = hb.off_q + n;
  hb.off_cu = hb.off_ctx + n;
  hb.off_last = hb.off_cu + n + 1;
  hb.off_tseq = hb.off_last + n;
  hb.off_tpos = hb.off_tseq + M;
  hb.off_bt = hb.off_tpos + M;
  hb.packed.assign(hb.off_bt + (size_t)n * mpps, 0);
}

BatchMeta device_meta(const hyp_stage* s, const HostBatch& hb) {
  BatchMeta bm;
  bm.n_seqs = hb.n;
  bm.n_tokens = hb.M;
  bm.max_pages_per_seq = s->max_pages_per_seq;
  bm.q_lens = s->meta_dev + hb.off_q;
  bm.ctx_lens = s->meta_dev + hb.off_ctx;
  bm.cu_q = s->meta_dev + hb.off_cu;
  bm.last_row = s->meta_dev + hb.off_last;
  bm.tok_seq = s->meta_dev + hb.off_tseq;
  bm.tok_pos = s->meta_dev + hb.off_tpos;
  bm.block_table = s->meta_dev + hb.off_bt;
  return bm;
}

int upload_meta(hyp_stage* s, const HostBatch& hb, cudaStream_t st) {
  const int slot = s->ring_pos;
  s->ring_pos = (s->ring_pos + 1) % META_RING;
  if (s->meta_used[slot]) HYP_CUDA_TRY(cudaEventSynchronize(s->meta_ev[slot]));
  std::memcpy(s->meta_host[slot], hb.packed.data(), hb.packed.size() * sizeof(int32_t));
  HYP_CUDA_TRY(cudaMemcpyAsync(s->meta_dev, s->meta_host[slot], hb.packed.size() * sizeof(int32_t),
                               cudaMemcpyHostToDevice, st));
  HYP_CUDA_TRY(cudaEventRecord(s->meta_ev[slot], st));
  s->meta_used[slot] = true;
  return HYP_OK;
}

// Validate a batch against the stage's tables and reserve the pages it needs.  Nothing is
// changed unless everything fits.
int admit_batch(hyp_stage* s, const hyp_batch* b, bool decode, HostBatch& hb) {
  if (!b || b->n_seqs < 1 || !b->seq_ids || !b->q_lens || !b->ctx_lens) return HYP_EINVAL;
  if (b->flags & ~HYP_BATCH_ALL_LOGITS) return HYP_EINVAL;
  const int n = b->n_seqs;
  if (n > s->cfg.max_seqs) return HYP_ECAPACITY;
  if (decode && n > HYP_MAX_DECODE_BATCH) return HYP_EINVAL;
  const int PT = s->cfg.kv_block_size;
  long M = 0;
  size_t need_pages = 0;
  std::vector<uint8_t> seen(s->cfg.max_seqs, 0);
  for (int i = 0; i < n; ++i) {
    const int id = b->seq_ids[i];
    if (id < 0 || id >= s->cfg.max_seqs || seen[id]) return HYP_EINVAL;
    seen[id] = 1;
    if (b->q_lens[i] < 1 || (decode && b->q_lens[i] != 1)) return HYP_EINVAL;
    if (b->ctx_lens[i] != s->seq_len[id]) return HYP_EINVAL;
    const long total = (long)b->ctx_lens[i] + b->q_lens[i];
    if (total > s->cfg.max_ctx) return HYP_ECAPACITY;
    M += b->q_lens[i];
    need_pages += (size_t)((total + PT - 1) / PT) - s->seq_pages[id].size();
  }
  if (M > s->max_rows || (!decode && M > s->cfg.max_tokens)) return HYP_ECAPACITY;
  if (need_pages > s->free_pages.size()) return HYP_ECAPACITY;

  layout_meta(hb, n, (int)M, s->max_pages_per_seq);
  int32_t* p = hb.packed.data();
  int row = 0;
  for (int i = 0; i < n; ++i) {
    const int id = b->seq_ids[i];
    const int total = b->ctx_lens[i] + b->q_lens[i];
    auto& pages = s->seq_pages[id];
    hb.undo.push_back({id, s->seq_len[id], pages.size()});
    while ((int)pages.size() < (total + PT - 1) / PT) {
      pages.push_back(s->free_pages.back());
      s->free_pages.pop_back();
    }
    s->seq_len[id] = total;
    p[hb.off_q + i] = b->q_lens[i];
    p[hb.off_ctx + i] = b->ctx_lens[i];
    p[hb.off_cu + i] = row;
    for (int t = 0; t < b->q_lens[i]; ++t) {
      p[hb.off_tseq + row] = i;
      p[hb.off_tpos + row] = b->ctx_lens[i] + t;
      ++row;
    }
    p[hb.off_last + i] = row - 1;
    std::copy(pages.begin(), pages.end(), p + hb.off_bt + (size_t)i * s->max_pages_per_seq);
  }
  p[hb.off_cu + n] = row;
  return HYP_OK;
}

// Undo admit_batch: lengths back, the pages taken for this call back on the free list in their old order.
void rollback_batch(hyp_stage* s, const HostBatch& hb) {
  for (auto it = hb.undo.rbegin(); it != hb.undo.rend(); ++it) {
    auto& pages = s->seq_pages[it->id];
    while (pages.size() > it->old_pages) {
      s->free_pages.push_back(pages.back());
      pages.pop_back();
    }
    s->seq_len[it->id] = it->old_len;
  }
}

int check_ready(const hyp_stage* s) {
  for (const LayerW& lw : s->layers)
    if (lw.loaded != 0x3f) return HYP_ESTATE;
  uint32_t want = 0;
  if (s->first) want |= 1u << HYP_W_EMBED;
  if (s->last) want |= (1u << HYP_W_FINAL_NORM) | (1u << HYP_W_LM_HEAD);
  if ((s->loaded_extra & want) != want) return HYP_ESTATE;
  return HYP_OK;
}

#define HYP_LAUNCH(call)                                   \
  do {                                                     \
    int _n = (call);                                       \
    if (_n < 0) return _n;                                 \
    s->launches += _n;                                     \
  } while (0)

// Same as HYP_LAUNCH, bracketed by an event pair when kernel class `cls` is being timed.
#define HYP_LAUNCH_T(cls, call)                                                             \
  do {                                                                                      \
    const bool _t = s->time_cls == (cls) && (size_t)(2 * s->time_n + 1) < s->time_ev.size(); \
    if (_t) HYP_CUDA_TRY(cudaEventRecord(s->time_ev[2 * s->time_n], st));                   \
    HYP_LAUNCH(call);                                                                       \
    if (_t) {                                                                               \
      HYP_CUDA_TRY(cudaEventRecord(s->time_ev[2 * s->time_n + 1], st));                     \
      s->time_n += 1;                                                                       \
    }                                                                                       \
  } while (0)

// out[m, n] (+)= a[m, :] . w[n, :] with the kernel family chosen by the row count.
int project(hyp_stage* s, const TcAct& act, const bf16* a, int lda, const TcWeight& tw, const bf16* w, int N, int K,
            int M, int epi, void* out, int ldo, cudaStream_t st) {
  (void)a; (void)lda; (void)w;
  return launch_projection(act, tw, M, N, K, epi, out, ldo, st, /*early=*/true);
}

// The block sequence B_lo -> ... -> B_{hi-1} on rows already resident in s->x.
// If `marks` is non-null an event is recorded before the first block and after every block.
int run_blocks(hyp_stage* s, const BatchMeta& bm, bool decode, int n_splits, cudaStream_t st, cudaEvent_t* marks) {
  const ModelDims& d = s->dims;
  const int M = bm.n_tokens;
  if (marks) HYP_CUDA_TRY(cudaEventRecord(marks[0], st));
  for (int li = 0; li < s->L; ++li) {
    LayerW& lw = s->layers[li];
    __half* kv_layer = s->kv_pool + (size_t)li * s->kv_layer_elems;
    // every projection runs fp16 x fp16 -> fp32: with bf16 inputs the rounding of the activations alone
    // (8 mantissa bits, amplified from block to block) puts the 40-block logits outside the tolerance
    const bool split = li == 0 && s->klo_pool != nullptr && first_block_split();
    HYP_LAUNCH_T(HYP_K_NORM, launch_rmsnorm(s->x, lw.g1, s->h, true, M, d.H, d.eps, nullptr, st, true,
                                            split ? s->row_scale : nullptr));
    HYP_LAUNCH_T(HYP_K_GEMM_QKV, project(s, s->tc_h, nullptr, d.H, lw.tc_qkv, nullptr, d.qkv_rows, d.H, M,
                                         EPI_STORE_F32, s->qkv32, d.qkv_rows, st));
    if (decode) {
      // rotation, cache append, attention and the merge of its splits in one launch; the two-term variant holds
      // half as much again in shared memory (two CTAs per SM, not three), so it takes fewer context splits to
      // stay within one resident wave
      const int ns = split ? std::max(1, std::min(n_splits, 2 * sm_count() / std::max(1, M * d.Hkv))) : n_splits;
      HYP_LAUNCH_T(HYP_K_ATTN, launch_attn_decode_fused(s->qkv32, d.qkv_rows, kv_layer, s->rope_table, s->attn, ns,
                                                        2, tc_err_flag_ptr(), bm, d, st, split ? s->row_scale : nullptr,
                                                        split ? s->klo_pool : nullptr,
                                                        attn_global_merge() ? s->attn_scratch : nullptr,
                                                        attn_global_merge() ? s->attn_tickets : nullptr));
    } else if (split) {
      HYP_LAUNCH_T(HYP_K_ROPE, launch_rope_kv_write(s->qkv32, s->q16, kv_layer, s->rope_table, bm, d, st, s->row_scale,
                                                    s->q16_lo, s->klo_pool));
      HYP_LAUNCH_T(HYP_K_ATTN, launch_attn_prefill_split(s->q16, s->q16_lo, d.Hq * d.D, kv_layer, s->klo_pool, s->attn, bm,
                                                         d, st));
    } else {
      HYP_LAUNCH_T(HYP_K_ROPE, launch_rope_kv_write(s->qkv32, s->q16, kv_layer, s->rope_table, bm, d, st));
      if (attn_prefill_tc_enabled() && !s->kv_maps.empty())
        HYP_LAUNCH_T(HYP_K_ATTN, launch_attn_prefill_tc(s->tc_q16.map, s->kv_maps[li], s->attn, bm, d, st));
      else
        HYP_LAUNCH_T(HYP_K_ATTN, launch_attn_prefill(s->q16, d.Hq * d.D, kv_layer, s->attn, bm, d, st));
    }
    HYP_LAUNCH_T(HYP_K_GEMM_O, project(s, s->tc_attn, nullptr, d.Hq * d.D, lw.tc_o, nullptr, d.H, d.Hq * d.D, M,
                                       EPI_RESID_F32, s->x, d.H, st));
    HYP_LAUNCH_T(HYP_K_NORM, launch_rmsnorm(s->x, lw.g2, s->h, true, M, d.H, d.eps, nullptr, st, true));
    HYP_LAUNCH_T(HYP_K_GEMM_GATE_UP, project(s, s->tc_h, nullptr, d.H, lw.tc_gu, nullptr, d.F, d.H, M, EPI_SWIGLU_BF16,
                                             s->u, d.F, st));
    HYP_LAUNCH_T(HYP_K_GEMM_DOWN, project(s, s->tc_u, nullptr, d.F, lw.tc_d, nullptr, d.H, d.F, M, EPI_RESID_F32, s->x,
                                          d.H, st));
    if (marks) HYP_CUDA_TRY(cudaEventRecord(marks[li + 1], st));
  }
  return HYP_OK;
}

// Enqueue [embedding gather | input copy] -> blocks -> [final norm + LM head | output copy] on `st`.
int enqueue_stage(hyp_stage* s, const BatchMeta& bm, int n_seqs, bool decode, bool all_rows, int n_splits,
                  const void* in, void* out, cudaStream_t st) {
  const ModelDims& d = s->dims;
  const int M = bm.n_tokens;
  if (s->first)
    HYP_LAUNCH(launch_embed((const int32_t*)in, s->embed, s->x, M, d.H, d.V, st));
  else
    HYP_LAUNCH(launch_copy_f32((const float*)in, s->x, (size_t)M * d.H, st));
  int rc = run_blocks(s, bm, decode, n_splits, st, nullptr);
  if (rc) return rc;
  if (s->last) {
    const int rows = all_rows ? M : n_seqs;
    HYP_LAUNCH(launch_rmsnorm(s->x, s->gf, s->h, true, rows, d.H, d.eps, all_rows ? nullptr : bm.last_row, st, true));
    HYP_LAUNCH_T(HYP_K_LM_HEAD,
                 project(s, s->tc_h, nullptr, d.H, s->tc_lm, nullptr, d.V, d.H, rows, EPI_STORE_F32, out, d.V, st));
  } else {
    HYP_LAUNCH(launch_copy_f32(s->x, (float*)out, (size_t)M * d.H, st));
  }
  return HYP_OK;
}

// Decode through a captured graph.  `in` / `out` may be device or host memory (the copies around the
// graph take either).  Returns HYP_OK, an error, or 1 if the caller should run the step eagerly.
int decode_with_graph(hyp_stage* s, const BatchMeta& bm, int n, int n_splits, const void* in, void* out,
                      cudaStream_t st) {
  const ModelDims& d = s->dims;
  hyp_stage::DecodeGraph* g = nullptr;
  for (auto& e : s->graphs)
    if (e.n == n && e.n_splits == n_splits) g = &e;
  if (!g) {  // first use of this key: run eagerly (also completes one-time kernel configuration)
    hyp_stage::DecodeGraph e;
    e.n = n;
    e.n_splits = n_splits;
    s->graphs.push_back(e);
    return 1;
  }
  if (!g->exec) {
    const int64_t before = s->launches;
    if (cudaStreamBeginCapture(s->cap_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      cudaGetLastError();
      s->graphs_ok = false;
      return 1;
    }
    const int rc = enqueue_stage(s, bm, n, true, true, n_splits, s->g_in, s->g_out, s->cap_stream);
    cudaGraph_t graph = nullptr;
    const cudaError_t e1 = cudaStreamEndCapture(s->cap_stream, &graph);
    g->n_launches = (int)(s->launches - before);
    s->launches = before;
    cudaError_t e2 = cudaErrorUnknown;
    if (rc == HYP_OK && e1 == cudaSuccess && graph) e2 = cudaGraphInstantiate(&g->exec, graph, 0);
    if (graph) cudaGraphDestroy(graph);
    if (e2 != cudaSuccess) {
      cudaGetLastError();
      g->exec = nullptr;
      if (pdl_level() > 0)
        pdl_level() = 0;  // retry on the next step without programmatic launches
      else
        s->graphs_ok = false;   // this driver cannot capture the sequence: stay on the eager path
      return 1;
    }
  }
  const size_t in_bytes = s->first ? (size_t)n * sizeof(int32_t) : (size_t)n * d.H * sizeof(float);
  const size_t out_bytes = (size_t)n * (s->last ? d.V : d.H) * sizeof(float);
  HYP_CUDA_TRY(cudaMemcpyAsync(s->g_in, in, in_bytes, cudaMemcpyDefault, st));
  HYP_CUDA_TRY(cudaGraphLaunch(g->exec, st));
  s->launches += g->n_launches;
  HYP_CUDA_TRY(cudaMemcpyAsync(out, s->g_out, out_bytes, cudaMemcpyDefault, st));
  return HYP_OK;
}

int run_stage(hyp_stage* s, const hyp_batch* b, const void* in, void* out, cudaStream_t st, bool decode,
              bool io_on_host = false) {
  if (!s || !in || !out) return HYP_EINVAL;
  // device buffers are written 16 bytes at a time by the epilogues (host buffers only see copies)
  if (!io_on_host && ((((uintptr_t)in) & 3) != 0 || (((uintptr_t)out) & 15) != 0)) return HYP_EINVAL;
  int rc = check_ready(s);
  if (rc) return rc;
  HostBatch hb;
  rc = admit_batch(s, b, decode, hb);
  if (rc) return rc;
  // from here on the tables say the rows are cached: any failure before the last enqueue puts them back
  rc = upload_meta(s, hb, st);
  if (rc) {
    rollback_batch(s, hb);
    return rc;
  }
  const BatchMeta bm = device_meta(s, hb);
  const ModelDims& d = s->dims;

  int n_splits = 1;
  if (decode) {
    int max_ctx = 1;
    for (int i = 0; i < hb.n; ++i) max_ctx = std::max(max_ctx, b->ctx_lens[i] + 1);
    n_splits = std::min(s->max_splits, attn_decode_fused_splits(hb.n, d.Hkv, max_ctx));
  }
  const bool all = (b->flags & HYP_BATCH_ALL_LOGITS) != 0 || decode;
  auto enqueue = [&]() -> int {
    int r = 1;
    if (decode && s->graphs_ok && s->time_cls < 0) r = decode_with_graph(s, bm, hb.n, n_splits, in, out, st);
    if (r != 1) return r;
    if (io_on_host) {  // eager kernels need device buffers: stage through the I/O buffers
      const size_t in_bytes = s->first ? (size_t)hb.M * sizeof(int32_t) : (size_t)hb.M * d.H * sizeof(float);
      const size_t out_bytes = (size_t)(all ? hb.M : hb.n) * (s->last ? d.V : d.H) * sizeof(float);
      HYP_CUDA_TRY(cudaMemcpyAsync(s->io_in, in, in_bytes, cudaMemcpyHostToDevice, st));
      r = enqueue_stage(s, bm, hb.n, decode, all, n_splits, s->io_in, s->io_out, st);
      if (r == HYP_OK) HYP_CUDA_TRY(cudaMemcpyAsync(out, s->io_out, out_bytes, cudaMemcpyDeviceToHost, st));
      return r;
    }
    return enqueue_stage(s, bm, hb.n, decode, all, n_splits, in, out, st);
  };
  rc = enqueue();
  if (rc == HYP_OK) {
    cudaError_t e = cudaPeekAtLastError();
    if (e != cudaSuccess) {
      set_last_cuda_error((int)e);
      rc = HYP_ECUDA;
    }
  }
  if (rc) rollback_batch(s, hb);
  return rc;
}

int run_stage_host(hyp_stage* s, const hyp_batch* b, const void* in, void* out, cudaStream_t st, bool decode) {
  if (!s || !b || !in || !out || b->n_seqs < 1 || !b->q_lens) return HYP_EINVAL;
  long M = 0;
  for (int i = 0; i < b->n_seqs; ++i) {
    if (b->q_lens[i] < 1) return HYP_EINVAL;
    M += b->q_lens[i];
  }
  const ModelDims& d = s->dims;
  const size_t in_bytes = s->first ? (size_t)M * sizeof(int32_t) : (size_t)M * d.H * sizeof(float);
  const bool all = (b->flags & HYP_BATCH_ALL_LOGITS) != 0 || decode;
  const size_t out_bytes =
      s->last ? (size_t)(all ? M : b->n_seqs) * d.V * sizeof(float) : (size_t)M * d.H * sizeof(float);
  if (in_bytes > s->io_in_bytes || out_bytes > s->io_out_bytes) return HYP_ECAPACITY;
  // validate before the first copy so that a rejected call moves no data: a trial admission, taken back at once
  {
    HostBatch probe;
    int rc = check_ready(s);
    if (!rc) rc = admit_batch(s, b, decode, probe);
    if (rc) return rc;
    rollback_batch(s, probe);
  }
  int rc = run_stage(s, b, in, out, st, decode, /*io_on_host=*/true);
  if (rc) return rc;
  // the error word rides behind the last kernel, so one synchronisation covers the outputs and the status
  *s->err_host = 0;
  if (tc_err_flag_ptr())
    HYP_CUDA_TRY(cudaMemcpyAsync(s->err_host, tc_err_flag_ptr(), sizeof(int), cudaMemcpyDeviceToHost, st));
  HYP_CUDA_TRY(cudaStreamSynchronize(st));
  return *s->err_host ? HYP_ETIMEOUT : HYP_OK;
}

__global__ void fill_pattern_kernel(float* x, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const uint32_t hsh = (uint32_t)i * 2654435761u;
    x[i] = ((float)((hsh >> 8) & 0xffff) / 65536.0f - 0.5f) * 0.1f;
  }
}

}  // namespace

// -------------------------------------------------------------------------------------------------
// C ABI
// -------------------------------------------------------------------------------------------------
extern "C" int hyp_last_cuda_error(void) { return hyp::g_last_cuda_error; }

extern "C" const char* hyp_strerror(int code) {
  switch (code) {
    case HYP_OK: return "ok";
    case HYP_EINVAL: return "invalid argument";
    case HYP_ENOMEM: return "out of memory";
    case HYP_ECAPACITY: return "capacity exceeded (KV pages, context, batch or token workspace)";
    case HYP_EINFEASIBLE: return "no feasible solution";
    case HYP_ECUDA: return "CUDA error (see hyp_last_cuda_error)";
    case HYP_ESTATE: return "stage not ready: a weight tensor has not been loaded";
    case HYP_ETIMEOUT: return "a device-side wait expired inside a kernel (results invalid)";
    default: return "unknown status";
  }
}

extern "C" void hyp_stage_destroy(hyp_stage* s) {
  if (!s) return;
  for (LayerW& lw : s->layers) {
    cudaFree(lw.wqkv); cudaFree(lw.wo); cudaFree(lw.wgu); cudaFree(lw.wd); cudaFree(lw.g1); cudaFree(lw.g2);
  }
  cudaFree(s->embed); cudaFree(s->gf); cudaFree(s->wlm); cudaFree(s->kv_pool);
  cudaFree(s->x); cudaFree(s->h); cudaFree(s->qkv32); cudaFree(s->q16);
  cudaFree(s->row_scale); cudaFree(s->q16_lo); cudaFree(s->klo_pool); cudaFree(s->attn_scratch); cudaFree(s->attn_tickets);
  cudaFree(s->attn); cudaFree(s->u);
  cudaFree(s->rope_table); cudaFree(s->meta_dev);
  cudaFree(s->io_in); cudaFree(s->io_out);
  for (int i = 0; i < META_RING; ++i) {
    if (s->meta_host[i]) cudaFreeHost(s->meta_host[i]);
    if (s->meta_ev[i]) cudaEventDestroy(s->meta_ev[i]);
  }
  if (s->err_host) cudaFreeHost(s->err_host);
  for (cudaEvent_t e : s->time_ev) cudaEventDestroy(e);
  for (auto& g : s->graphs)
    if (g.exec) cudaGraphExecDestroy(g.exec);
  if (s->cap_stream) cudaStreamDestroy(s->cap_stream);
  cudaFree(s->g_in); cudaFree(s->g_out);
  delete s;
}

extern "C" int hyp_stage_create(int32_t layer_lo, int32_t layer_hi, const hyp_cfg* cfg, hyp_stage** out) {
  if (!cfg || !out) return HYP_EINVAL;
  const hyp_cfg& c = *cfg;
  if (c.n_layers_total < 1 || layer_lo < 0 || layer_hi <= layer_lo || layer_hi > c.n_layers_total) return HYP_EINVAL;
  // every row of an activation, logits or weight matrix must start on a 16-byte boundary (vector stores, TMA)
  if (c.hidden < 8 || c.hidden % 8 || c.ffn < 8 || c.ffn % 8 || c.vocab < 8 || c.vocab % 8) return HYP_EINVAL;
  if (c.n_kv_heads < 1 || c.n_q_heads < c.n_kv_heads || c.n_q_heads % c.n_kv_heads) return HYP_EINVAL;
  const int G = c.n_q_heads / c.n_kv_heads;
  if (!(G == 1 || G == 2 || G == 4 || G == 8)) return HYP_EINVAL;
  if (!(c.head_dim == 64 || c.head_dim == 128)) return HYP_EINVAL;
  if (c.kv_block_size != 16) return HYP_EINVAL;
  if (c.max_seqs < 1 || c.max_ctx < 1 || c.max_tokens < 1 || c.kv_pages < 0) return HYP_EINVAL;
  if (!(c.rms_eps > 0.f) || !(c.rope_theta > 1.f)) return HYP_EINVAL;

  hyp_stage* s = new (std::nothrow) hyp_stage();
  if (!s) return HYP_ENOMEM;
  s->cfg = c;
  s->lo = layer_lo; s->hi = layer_hi; s->L = layer_hi - layer_lo;
  s->first = layer_lo == 0;
  s->last = layer_hi == c.n_layers_total;
  ModelDims& d = s->dims;
  d.H = c.hidden; d.Hq = c.n_q_heads; d.Hkv = c.n_kv_heads; d.D = c.head_dim; d.F = c.ffn; d.V = c.vocab;
  d.qkv_rows = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  d.page_tokens = c.kv_block_size; d.eps = c.rms_eps; d.theta = c.rope_theta;

  int rc = HYP_OK;
#define TRY(expr) do { rc = (expr); if (rc) { hyp_stage_destroy(s); return rc; } } while (0)
#define TRY_CUDA(expr) do { cudaError_t _e = (expr); if (_e != cudaSuccess) { set_last_cuda_error((int)_e); \
    hyp_stage_destroy(s); return _e == cudaErrorMemoryAllocation ? HYP_ENOMEM : HYP_ECUDA; } } while (0)
  TRY_CUDA(cudaGetDevice(&s->device));
  s->layers.resize(s->L);
  for (LayerW& lw : s->layers) {
    TRY(dev_alloc_bytes(&lw.wqkv, proj_packed_bytes(s, HYP_W_QKV)));
    TRY(dev_alloc_bytes(&lw.wo, proj_packed_bytes(s, HYP_W_O)));
    TRY(dev_alloc_bytes(&lw.wgu, proj_packed_bytes(s, HYP_W_GATE_UP)));
    TRY(dev_alloc_bytes(&lw.wd, proj_packed_bytes(s, HYP_W_DOWN)));
    TRY(dev_alloc(&lw.g1, (size_t)d.H));
    TRY(dev_alloc(&lw.g2, (size_t)d.H));
  }
  if (s->first) TRY(dev_alloc(&s->embed, tensor_elems(s, HYP_W_EMBED)));
  if (s->last) {
    TRY(dev_alloc(&s->gf, (size_t)d.H));
    TRY(dev_alloc_bytes(&s->wlm, proj_packed_bytes(s, HYP_W_LM_HEAD)));
  }
  // KV pool: [layer][page][K,V][Hkv][16][D]
  s->max_pages_per_seq = (c.max_ctx + c.kv_block_size - 1) / c.kv_block_size;
  s->n_pages = c.kv_pages > 0 ? c.kv_pages : c.max_seqs * s->max_pages_per_seq;
  s->kv_layer_elems = (size_t)s->n_pages * kv_page_elems(d.Hkv, d.page_tokens, d.D);
  TRY(dev_alloc(&s->kv_pool, s->kv_layer_elems * s->L));
  TRY_CUDA(cudaMemset(s->kv_pool, 0, s->kv_layer_elems * s->L * sizeof(__half)));
  s->free_pages.resize(s->n_pages);
  for (int i = 0; i < s->n_pages; ++i) s->free_pages[i] = s->n_pages - 1 - i;
  s->seq_pages.assign(c.max_seqs, {});
  s->seq_len.assign(c.max_seqs, 0);
  // workspace (row capacity covers a full prefill call or a full decode batch; rows are padded to
  // the GEMM tile height so that tile loads never leave the allocation)
  s->max_rows = std::max(c.max_tokens, std::min(c.max_seqs, HYP_MAX_DECODE_BATCH));
  const size_t rows_pad = ((size_t)s->max_rows + 127) / 128 * 128;
  TRY(dev_alloc(&s->x, rows_pad * d.H));
  TRY(dev_alloc(&s->h, rows_pad * d.H));
  TRY(dev_alloc(&s->qkv32, rows_pad * d.qkv_rows));
  TRY(dev_alloc(&s->q16, rows_pad * d.Hq * d.D));
  if (s->first) {
    const size_t klo_elems = (size_t)s->n_pages * d.Hkv * d.page_tokens * d.D;
    TRY(dev_alloc(&s->row_scale, rows_pad));
    TRY(dev_alloc(&s->q16_lo, rows_pad * d.Hq * d.D));
    TRY(dev_alloc(&s->klo_pool, klo_elems));
    TRY_CUDA(cudaMemset(s->klo_pool, 0, klo_elems * sizeof(__half)));
  }
  {
    const size_t groups = (size_t)std::min(c.max_seqs, HYP_MAX_DECODE_BATCH) * d.Hkv;
    TRY(dev_alloc(&s->attn_scratch, groups * 8 * attn_fused_scratch_row(d.Hq / d.Hkv, d.D)));
    TRY(dev_alloc(&s->attn_tickets, groups));
    TRY_CUDA(cudaMemset(s->attn_tickets, 0, groups * sizeof(int)));
  }
  TRY(dev_alloc(&s->attn, rows_pad * d.Hq * d.D));
  TRY(dev_alloc(&s->u, rows_pad * d.F));
  TRY_CUDA(cudaMemset(s->h, 0, rows_pad * d.H * sizeof(__half)));
  TRY_CUDA(cudaMemset(s->attn, 0, rows_pad * d.Hq * d.D * sizeof(__half)));
  TRY_CUDA(cudaMemset(s->u, 0, rows_pad * d.F * sizeof(__half)));
  s->workspace_bytes = rows_pad * ((size_t)d.H * 8 + (size_t)d.qkv_rows * 4 + ((size_t)2 * d.Hq * d.D + d.F) * 2);
  // rotary table: cos/sin of pos * theta^(-2i/D), angles evaluated in double on the host
  {
    const int half = d.D / 2;
    std::vector<float2> tab((size_t)c.max_ctx * half);
    for (int p = 0; p < c.max_ctx; ++p)
      for (int i = 0; i < half; ++i) {
        const double ang = (double)p * std::pow((double)c.rope_theta, -2.0 * i / d.D);
        tab[(size_t)p * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
      }
    TRY(dev_alloc(&s->rope_table, tab.size()));
    TRY_CUDA(cudaMemcpy(s->rope_table, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice));
  }
  // metadata staging
  s->meta_ints = (size_t)4 * c.max_seqs + 1 + (size_t)2 * s->max_rows + (size_t)c.max_seqs * s->max_pages_per_seq;
  TRY(dev_alloc(&s->meta_dev, s->meta_ints));
  for (int i = 0; i < META_RING; ++i) {
    TRY_CUDA(cudaMallocHost((void**)&s->meta_host[i], s->meta_ints * sizeof(int32_t)));
    TRY_CUDA(cudaEventCreateWithFlags(&s->meta_ev[i], cudaEventDisableTiming));
  }
  TRY_CUDA(cudaMallocHost((void**)&s->err_host, sizeof(int)));
  // staging for host-buffer calls
  s->io_in_bytes = (size_t)s->max_rows * (s->first ? sizeof(int32_t) : d.H * sizeof(float));
  s->io_out_bytes = s->last ? (size_t)std::max(c.max_seqs, std::min(s->max_rows, 64)) * d.V * sizeof(float)
                            : (size_t)s->max_rows * d.H * sizeof(float);
  TRY_CUDA(cudaMalloc(&s->io_in, s->io_in_bytes));
  TRY_CUDA(cudaMalloc(&s->io_out, s->io_out_bytes));
  TRY_CUDA(cudaMalloc(&s->g_in, (size_t)HYP_MAX_DECODE_BATCH * std::max((size_t)d.H * sizeof(float), sizeof(int32_t))));
  TRY_CUDA(cudaMalloc(&s->g_out, (size_t)HYP_MAX_DECODE_BATCH * std::max(d.H, d.V) * sizeof(float)));
  TRY_CUDA(cudaStreamCreateWithFlags(&s->cap_stream, cudaStreamNonBlocking));
  // tensor-core operand descriptors over the fixed workspace buffers
  TRY(tc_prepare());
  TRY(tc_make_act(&s->tc_h, s->h, (int)rows_pad, d.H, true));
  TRY(tc_make_act(&s->tc_attn, s->attn, (int)rows_pad, d.Hq * d.D, true));
  TRY(tc_make_act(&s->tc_u, s->u, (int)rows_pad, d.F, true));
  TRY(tc_make_act(&s->tc_q16, s->q16, (int)rows_pad, d.Hq * d.D, true));
  if (d.D == 128) {
    s->kv_maps.resize(s->L);
    for (int li = 0; li < s->L; ++li)
      TRY(tc_make_kv_map(&s->kv_maps[li], s->kv_pool + (size_t)li * s->kv_layer_elems, (size_t)s->n_pages, d.Hkv, d.D));
  }
  for (LayerW& lw : s->layers) {
    // all projection matrices are held packed as fp16, see hyp_stage_load
    TRY(tc_make_weight(&lw.tc_qkv, lw.wqkv, d.qkv_rows, 1, d.H, true));
    TRY(tc_make_weight(&lw.tc_o, lw.wo, d.H, 1, d.Hq * d.D, true));
    TRY(tc_make_weight(&lw.tc_gu, lw.wgu, d.F, 2, d.H, true));
    TRY(tc_make_weight(&lw.tc_d, lw.wd, d.H, 1, d.F, true));
  }
  if (s->last) TRY(tc_make_weight(&s->tc_lm, s->wlm, d.V, 1, d.H, true));
#undef TRY
#undef TRY_CUDA
  *out = s;
  return HYP_OK;
}

extern "C" int hyp_stage_load(hyp_stage* s, int32_t layer, int32_t tensor_id, const void* src, size_t bytes,
                              void* stream) {
  if (!s || !src) return HYP_EINVAL;
  void* dst = nullptr;
  uint32_t* mask = nullptr;
  if (tensor_id >= HYP_W_QKV && tensor_id <= HYP_W_NORM2) {
    if (layer < s->lo || layer >= s->hi) return HYP_EINVAL;
    LayerW& lw = s->layers[layer - s->lo];
    void* ptrs[6] = {lw.wqkv, lw.wo, lw.wgu, lw.wd, lw.g1, lw.g2};
    dst = ptrs[tensor_id];
    mask = &lw.loaded;
  } else if (tensor_id == HYP_W_EMBED) {
    if (!s->first || layer != -1) return HYP_EINVAL;
    dst = s->embed;
    mask = &s->loaded_extra;
  } else if (tensor_id == HYP_W_FINAL_NORM || tensor_id == HYP_W_LM_HEAD) {
    if (!s->last || layer != s->cfg.n_layers_total) return HYP_EINVAL;
    dst = tensor_id == HYP_W_FINAL_NORM ? (void*)s->gf : (void*)s->wlm;
    mask = &s->loaded_extra;
  } else {
    return HYP_EINVAL;
  }
  if (bytes != tensor_elems(s, tensor_id) * sizeof(bf16)) return HYP_EINVAL;
  if (tensor_id <= HYP_W_DOWN || tensor_id == HYP_W_LM_HEAD) {
    // projection matrices are kept as fp16 so that the projections can take fp16 activations
    // (bf16 -> fp16 is exact for |w| >= 2^-17 and off by < 3e-8 below that), in the packed tile order
    if (((uintptr_t)src & 15) != 0) return HYP_EINVAL;
    int rows, halves, K;
    proj_geometry(s, tensor_id, &rows, &halves, &K);
    const int prc = tc_pack_weight(src, dst, rows, halves, K, true, (cudaStream_t)stream);
    if (prc < 0) return prc;
    cudaError_t e = cudaPeekAtLastError();
    if (e != cudaSuccess) {
      set_last_cuda_error((int)e);
      return HYP_ECUDA;
    }
  } else {
    HYP_CUDA_TRY(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  }
  *mask |= 1u << tensor_id;
  return HYP_OK;
}

extern "C" int hyp_stage_prefill(hyp_stage* s, const hyp_batch* b, const void* in, void* out, void* stream) {
  return run_stage(s, b, in, out, (cudaStream_t)stream, false);
}
extern "C" int hyp_stage_decode(hyp_stage* s, const hyp_batch* b, const void* in, void* out, void* stream) {
  return run_stage(s, b, in, out, (cudaStream_t)stream, true);
}
extern "C" int hyp_stage_prefill_host(hyp_stage* s, const hyp_batch* b, const void* in, void* out, void* stream) {
  return run_stage_host(s, b, in, out, (cudaStream_t)stream, false);
}
extern "C" int hyp_stage_decode_host(hyp_stage* s, const hyp_batch* b, const void* in, void* out, void* stream) {
  return run_stage_host(s, b, in, out, (cudaStream_t)stream, true);
}

extern "C" int hyp_stage_free_seq(hyp_stage* s, int32_t seq_id) {
  if (!s || seq_id < 0 || seq_id >= s->cfg.max_seqs) return HYP_EINVAL;
  auto& pages = s->seq_pages[seq_id];
  for (auto it = pages.rbegin(); it != pages.rend(); ++it) s->free_pages.push_back(*it);
  pages.clear();
  s->seq_len[seq_id] = 0;
  return HYP_OK;
}

extern "C" int hyp_stage_seq_len(const hyp_stage* s, int32_t seq_id) {
  if (!s || seq_id < 0 || seq_id >= s->cfg.max_seqs) return HYP_EINVAL;
  return s->seq_len[seq_id];
}

extern "C" int hyp_stage_free_pages(const hyp_stage* s) {
  if (!s) return HYP_EINVAL;
  return (int)s->free_pages.size();
}

extern "C" int64_t hyp_stage_launch_count(const hyp_stage* s) { return s ? s->launches : 0; }

extern "C" int hyp_stage_kernel_timing(hyp_stage* s, int32_t kernel_class, int32_t max_samples) {
  if (!s || kernel_class < -1 || kernel_class > HYP_K_LM_HEAD || max_samples < 0) return HYP_EINVAL;
  s->time_cls = kernel_class;
  s->time_n = 0;
  while (s->time_ev.size() < (size_t)2 * max_samples) {
    cudaEvent_t e;
    HYP_CUDA_TRY(cudaEventCreate(&e));
    s->time_ev.push_back(e);
  }
  return HYP_OK;
}

extern "C" int hyp_stage_kernel_timing_read(hyp_stage* s, int32_t* n_samples, double* total_ms) {
  if (!s || !n_samples || !total_ms) return HYP_EINVAL;
  double tot = 0.0;
  for (int i = 0; i < s->time_n; ++i) {
    HYP_CUDA_TRY(cudaEventSynchronize(s->time_ev[2 * i + 1]));
    float ms = 0.f;
    HYP_CUDA_TRY(cudaEventElapsedTime(&ms, s->time_ev[2 * i], s->time_ev[2 * i + 1]));
    tot += ms;
  }
  *n_samples = s->time_n;
  *total_ms = tot;
  s->time_n = 0;
  return HYP_OK;
}

extern "C" int hyp_stage_profile(hyp_stage* s, int32_t mode, int32_t batch, int32_t ctx, int32_t iters,
                                 float* layer_ms, size_t* layer_bytes, void* stream) {
  if (!s || !layer_ms || !layer_bytes || (mode != 0 && mode != 1) || batch < 1 || ctx < 1 || iters < 1)
    return HYP_EINVAL;
  int rc = check_ready(s);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const bool decode = mode == 1;
  const int PT = s->cfg.kv_block_size;
  const int total = decode ? ctx + 1 : ctx;
  const long M = decode ? batch : (long)batch * ctx;
  if (batch > s->cfg.max_seqs || total > s->cfg.max_ctx || M > s->max_rows) return HYP_ECAPACITY;
  if (decode && batch > HYP_MAX_DECODE_BATCH) return HYP_EINVAL;
  const int pages_per = (total + PT - 1) / PT;
  if ((size_t)batch * pages_per > s->free_pages.size()) return HYP_ECAPACITY;

  // scratch sequences on pages borrowed from the free list (not removed: nothing persists)
  HostBatch hb;
  layout_meta(hb, batch, (int)M, s->max_pages_per_seq);
  int32_t* p = hb.packed.data();
  int row = 0;
  for (int i = 0; i < batch; ++i) {
    const int ql = decode ? 1 : ctx, cl = decode ? ctx : 0;
    p[hb.off_q + i] = ql;
    p[hb.off_ctx + i] = cl;
    p[hb.off_cu + i] = row;
    for (int t = 0; t < ql; ++t) {
      p[hb.off_tseq + row] = i;
      p[hb.off_tpos + row] = cl + t;
      ++row;
    }
    p[hb.off_last + i] = row - 1;
    for (int k = 0; k < pages_per; ++k)
      p[hb.off_bt + (size_t)i * s->max_pages_per_seq + k] = s->free_pages[s->free_pages.size() - 1 - (i * pages_per + k)];
  }
  p[hb.off_cu + batch] = row;
  rc = upload_meta(s, hb, st);
  if (rc) return rc;
  const BatchMeta bm = device_meta(s, hb);
  const int n_splits = decode ? std::min(s->max_splits, attn_decode_fused_splits(batch, s->dims.Hkv, total)) : 1;

  std::vector<cudaEvent_t> ev((size_t)(s->L + 1) * iters, nullptr);
  for (auto& e : ev) HYP_CUDA_TRY(cudaEventCreate(&e));
  rc = HYP_OK;
  for (int it = -1; it < iters && rc == HYP_OK; ++it) {
    fill_pattern_kernel<<<sm_count() * 4, 256, 0, st>>>(s->x, (size_t)M * s->dims.H);
    s->launches += 1;
    rc = run_blocks(s, bm, decode, n_splits, st, it < 0 ? nullptr : &ev[(size_t)it * (s->L + 1)]);
  }
  if (rc == HYP_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = HYP_ECUDA;
  if (rc == HYP_OK) {
    int dev_err = 0;
    rc = tc_error_flag(&dev_err);
    if (rc == HYP_OK && dev_err) rc = HYP_ETIMEOUT;
  }
  if (rc == HYP_OK) {
    std::vector<float> samples(iters);
    for (int li = 0; li < s->L; ++li) {
      for (int it = 0; it < iters; ++it)
        cudaEventElapsedTime(&samples[it], ev[(size_t)it * (s->L + 1) + li], ev[(size_t)it * (s->L + 1) + li + 1]);
      std::sort(samples.begin(), samples.end());
      layer_ms[li] = samples[iters / 2];
      const ModelDims& d = s->dims;
      const size_t wbytes = ((size_t)d.qkv_rows * d.H + (size_t)d.H * d.Hq * d.D + (size_t)3 * d.F * d.H + 2 * d.H) * 2;
      layer_bytes[li] = wbytes + s->kv_layer_elems * sizeof(__half) + s->workspace_bytes / s->L;
      if (li == 0 && s->klo_pool) layer_bytes[li] += s->kv_layer_elems / 2 * sizeof(__half);  // the keys' low terms
    }
  }
  for (auto& e : ev) cudaEventDestroy(e);
  // the scratch rows wrote K/V into free pages only; live sequences were not touched
  return rc;
}
