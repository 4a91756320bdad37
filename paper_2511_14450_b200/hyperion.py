"""ctypes binding of libhyperion: the same names as the C ABI, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  If the shared library has not been
built this module raises on first use; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libhyperion.so")

HYP_OK, HYP_EINVAL, HYP_ENOMEM, HYP_ECAPACITY, HYP_EINFEASIBLE, HYP_ECUDA, HYP_ESTATE = 0, -1, -2, -3, -4, -5, -6
HYP_ETIMEOUT = -7
(HYP_W_QKV, HYP_W_O, HYP_W_GATE_UP, HYP_W_DOWN, HYP_W_NORM1, HYP_W_NORM2, HYP_W_EMBED, HYP_W_FINAL_NORM,
 HYP_W_LM_HEAD) = range(9)
HYP_BATCH_ALL_LOGITS = 1
HYP_MAX_DECODE_BATCH = 128


class hyp_cfg(C.Structure):
    _fields_ = [("n_layers_total", C.c_int32), ("hidden", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("kv_block_size", C.c_int32),
                ("max_seqs", C.c_int32), ("max_ctx", C.c_int32), ("max_tokens", C.c_int32),
                ("kv_pages", C.c_int32)]


class hyp_batch(C.Structure):
    _fields_ = [("n_seqs", C.c_int32), ("seq_ids", C.POINTER(C.c_int32)), ("q_lens", C.POINTER(C.c_int32)),
                ("ctx_lens", C.POINTER(C.c_int32)), ("flags", C.c_int32)]


class hyp_node_state(C.Structure):
    _fields_ = [("C", C.c_double), ("M_avail", C.c_double), ("F_rem", C.c_double), ("F_wait", C.c_double),
                ("available", C.c_int32)]


class hyp_attn_shape(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32)]


class HyperionError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().hyp_strerror(code).decode()
        if code == HYP_ECUDA:
            msg += f" [cudaError {lib().hyp_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")


_LIB: Optional[C.CDLL] = None

# every exported symbol with (restype, argtypes); the export test walks this table
SIGNATURES = {
    "hyp_stage_create": (C.c_int, [C.c_int32, C.c_int32, C.POINTER(hyp_cfg), C.POINTER(C.c_void_p)]),
    "hyp_stage_load": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]),
    "hyp_stage_prefill": (C.c_int, [C.c_void_p, C.POINTER(hyp_batch), C.c_void_p, C.c_void_p, C.c_void_p]),
    "hyp_stage_decode": (C.c_int, [C.c_void_p, C.POINTER(hyp_batch), C.c_void_p, C.c_void_p, C.c_void_p]),
    "hyp_stage_prefill_host": (C.c_int, [C.c_void_p, C.POINTER(hyp_batch), C.c_void_p, C.c_void_p, C.c_void_p]),
    "hyp_stage_decode_host": (C.c_int, [C.c_void_p, C.POINTER(hyp_batch), C.c_void_p, C.c_void_p, C.c_void_p]),
    "hyp_stage_profile": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_float),
                                    C.POINTER(C.c_size_t), C.c_void_p]),
    "hyp_stage_kernel_timing": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32]),
    "hyp_stage_kernel_timing_read": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_double)]),
    "hyp_stage_free_seq": (C.c_int, [C.c_void_p, C.c_int32]),
    "hyp_stage_seq_len": (C.c_int, [C.c_void_p, C.c_int32]),
    "hyp_stage_free_pages": (C.c_int, [C.c_void_p]),
    "hyp_stage_launch_count": (C.c_int64, [C.c_void_p]),
    "hyp_stage_destroy": (None, [C.c_void_p]),
    "hyp_split_dp": (C.c_int, [C.c_int32, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_double),
                               C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_double, C.POINTER(C.c_int32),
                               C.POINTER(C.c_double)]),
    "hyp_split_even": (C.c_int, [C.c_int32, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                 C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int32),
                                 C.POINTER(C.c_double)]),
    "hyp_split_greedy": (C.c_int, [C.c_int32, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                   C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int32),
                                   C.POINTER(C.c_double)]),
    "hyp_sched_rt": (C.c_int, [C.c_double, C.c_double, C.POINTER(hyp_node_state), C.c_int32, C.POINTER(C.c_int32)]),
    "hyp_op_rmsnorm": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_void_p]),
    "hyp_op_weight_packed_bytes": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int32]),
    "hyp_op_pack_weight": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]),
    "hyp_tune": (C.c_int, [C.c_int32, C.c_int32]),
    "hyp_op_gemm": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                              C.c_int32, C.c_void_p]),
    "hyp_op_pack_weight_f16": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]),
    "hyp_op_gemm_f16": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                  C.c_int32, C.c_void_p]),
    "hyp_device_wait_status": (C.c_int, [C.POINTER(C.c_int32), C.c_int32]),
    "hyp_op_attn_decode_splits": (C.c_int, [C.c_int32, C.c_int32, C.c_int32]),
    "hyp_op_attn_decode_scratch_bytes": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int32, C.c_int32]),
    "hyp_op_attn_decode": (C.c_int, [C.POINTER(hyp_attn_shape), C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                     C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t,
                                     C.c_void_p, C.c_void_p]),
    "hyp_op_attn_decode_static": (C.c_int, [C.POINTER(hyp_attn_shape), C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                            C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "hyp_op_attn_decode_step": (C.c_int, [C.POINTER(hyp_attn_shape), C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                          C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                          C.c_void_p]),
    "hyp_op_attn_prefill": (C.c_int, [C.POINTER(hyp_attn_shape), C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
                                      C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p]),
    "hyp_strerror": (C.c_char_p, [C.c_int]),
    "hyp_last_cuda_error": (C.c_int, []),
}


def lib() -> C.CDLL:
    """Load libhyperion.so (built in-tree by `paper_2511_14450_b200.build`)."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_14450_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _LIB = L
    return _LIB


def _check(code: int, where: str):
    if code != HYP_OK:
        raise HyperionError(code, where)


def _i32(seq: Sequence[int]):
    return (C.c_int32 * len(seq))(*[int(v) for v in seq])


def _f64(seq):
    return (C.c_double * len(seq))(*[float(v) for v in seq])


def _ptr(t) -> int:
    """Address of a torch tensor / numpy array / raw int."""
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream_handle(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def make_cfg(shape, max_seqs: int, max_ctx: int, max_tokens: int, kv_pages: int = 0) -> hyp_cfg:
    return hyp_cfg(shape.n_layers_total, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                   shape.ffn, shape.vocab, shape.rms_eps, shape.rope_theta, shape.kv_block_size,
                   max_seqs, max_ctx, max_tokens, kv_pages)


def make_batch(seq_ids, q_lens, ctx_lens, flags: int = 0):
    """Returns (hyp_batch, keepalive) - keep `keepalive` referenced until the call returns."""
    a, b, c = _i32(seq_ids), _i32(q_lens), _i32(ctx_lens)
    hb = hyp_batch(len(seq_ids), a, b, c, flags)
    return hb, (a, b, c)


# --------------------------------------------------------------------------------------------
# same names as the C ABI
# --------------------------------------------------------------------------------------------
def hyp_stage_create(layer_lo: int, layer_hi: int, cfg: hyp_cfg) -> int:
    h = C.c_void_p()
    _check(lib().hyp_stage_create(layer_lo, layer_hi, C.byref(cfg), C.byref(h)), "hyp_stage_create")
    return h.value


def hyp_stage_load(stage: int, layer: int, tensor_id: int, src, stream=None):
    nbytes = src.numel() * src.element_size()
    _check(lib().hyp_stage_load(stage, layer, tensor_id, _ptr(src), nbytes, _stream_handle(stream)),
           "hyp_stage_load")


def _run(fn_name, stage, seq_ids, q_lens, ctx_lens, inp, out, stream, flags):
    hb, keep = make_batch(seq_ids, q_lens, ctx_lens, flags)
    _check(getattr(lib(), fn_name)(stage, C.byref(hb), _ptr(inp), _ptr(out), _stream_handle(stream)), fn_name)
    del keep


def hyp_stage_prefill(stage, seq_ids, q_lens, ctx_lens, inp, out, stream=None, flags=0):
    _run("hyp_stage_prefill", stage, seq_ids, q_lens, ctx_lens, inp, out, stream, flags)


def hyp_stage_decode(stage, seq_ids, ctx_lens, inp, out, stream=None):
    _run("hyp_stage_decode", stage, seq_ids, [1] * len(seq_ids), ctx_lens, inp, out, stream, 0)


def hyp_stage_prefill_host(stage, seq_ids, q_lens, ctx_lens, inp, out, stream=None, flags=0):
    _run("hyp_stage_prefill_host", stage, seq_ids, q_lens, ctx_lens, inp, out, stream, flags)


def hyp_stage_decode_host(stage, seq_ids, ctx_lens, inp, out, stream=None):
    _run("hyp_stage_decode_host", stage, seq_ids, [1] * len(seq_ids), ctx_lens, inp, out, stream, 0)


def hyp_stage_profile(stage, n_layers: int, mode: int, batch: int, ctx: int, iters: int = 5, stream=None):
    ms = (C.c_float * n_layers)()
    by = (C.c_size_t * n_layers)()
    _check(lib().hyp_stage_profile(stage, mode, batch, ctx, iters, ms, by, _stream_handle(stream)),
           "hyp_stage_profile")
    return list(ms), list(by)


(HYP_K_GEMM_QKV, HYP_K_GEMM_O, HYP_K_GEMM_GATE_UP, HYP_K_GEMM_DOWN, HYP_K_ATTN, HYP_K_NORM, HYP_K_ROPE,
 HYP_K_LM_HEAD) = range(8)


def hyp_stage_kernel_timing(stage, kernel_class: int, max_samples: int):
    _check(lib().hyp_stage_kernel_timing(stage, kernel_class, max_samples), "hyp_stage_kernel_timing")


def hyp_stage_kernel_timing_read(stage):
    """Returns (launches recorded, their summed milliseconds)."""
    n, ms = C.c_int32(), C.c_double()
    _check(lib().hyp_stage_kernel_timing_read(stage, C.byref(n), C.byref(ms)), "hyp_stage_kernel_timing_read")
    return n.value, ms.value


def hyp_stage_free_seq(stage, seq_id: int):
    _check(lib().hyp_stage_free_seq(stage, seq_id), "hyp_stage_free_seq")


def hyp_stage_seq_len(stage, seq_id: int) -> int:
    r = lib().hyp_stage_seq_len(stage, seq_id)
    if r < 0:
        raise HyperionError(r, "hyp_stage_seq_len")
    return r


def hyp_stage_free_pages(stage) -> int:
    r = lib().hyp_stage_free_pages(stage)
    if r < 0:
        raise HyperionError(r, "hyp_stage_free_pages")
    return r


def hyp_stage_launch_count(stage) -> int:
    return lib().hyp_stage_launch_count(stage)


def hyp_stage_destroy(stage):
    lib().hyp_stage_destroy(stage)


def hyp_split_dp(f, m, Cap, Mcap, eps: float = 0.0):
    """Returns (p, tau): p = tuple of 1-based last-block indices of tiers 1..T-1."""
    N, T = len(f), len(Cap)
    p = (C.c_int32 * max(T - 1, 1))()
    tau = C.c_double()
    _check(lib().hyp_split_dp(N, T, _f64(f), _f64(m), _f64(Cap), _f64(Mcap), eps, p, C.byref(tau)), "hyp_split_dp")
    return tuple(p[j] for j in range(T - 1)), tau.value


def _split_baseline(name, f, m, Cap, Mcap, tolerate_infeasible):
    N, T = len(f), len(Cap)
    p = (C.c_int32 * max(T - 1, 1))()
    tau = C.c_double()
    code = getattr(lib(), name)(N, T, _f64(f), _f64(m), _f64(Cap), _f64(Mcap), p, C.byref(tau))
    if not (tolerate_infeasible and code == HYP_EINFEASIBLE and N >= T):
        _check(code, name)
    return tuple(p[j] for j in range(T - 1)), tau.value, code == HYP_OK


def hyp_split_even(f, m, Cap, Mcap):
    """Equal-count contiguous partition.  Returns (p, tau, fits): fits is False if a memory limit is exceeded."""
    return _split_baseline("hyp_split_even", f, m, Cap, Mcap, True)


def hyp_split_greedy(f, m, Cap, Mcap):
    """Memory-aware greedy contiguous partition.  Returns (p, tau); raises HYP_EINFEASIBLE if it finds none."""
    p, tau, _ = _split_baseline("hyp_split_greedy", f, m, Cap, Mcap, False)
    return p, tau


def hyp_sched_rt(F_new: float, m_act: float, nodes) -> int:
    """nodes: sequence of (C, M_avail, F_rem, F_wait_total, available).  Returns the 0-based node."""
    arr = (hyp_node_state * len(nodes))(*[hyp_node_state(*n) for n in nodes])
    k = C.c_int32(-1)
    _check(lib().hyp_sched_rt(F_new, m_act, arr, len(nodes), C.byref(k)), "hyp_sched_rt")
    return k.value


# --------------------------------------------------------------------------------------------
# single-kernel entry points (hyperion_ops.h)
# --------------------------------------------------------------------------------------------
HYP_EPI_STORE_BF16, HYP_EPI_RESID_F32, HYP_EPI_SWIGLU_BF16, HYP_EPI_STORE_F32 = range(4)


def hyp_op_rmsnorm(x, g, out, eps: float, stream=None):
    M, H = x.shape
    _check(lib().hyp_op_rmsnorm(_ptr(x), _ptr(g), _ptr(out), M, H, eps, _stream_handle(stream)), "hyp_op_rmsnorm")


(HYP_TUNE_PDL, HYP_TUNE_STREAM_SLOTS, HYP_TUNE_ATTN_SPLITS, HYP_TUNE_ATTN_SLOTS, HYP_TUNE_STREAM_ROTATION,
 HYP_TUNE_SWAP_MIN_ROWS, HYP_TUNE_SWAP_MAX_ROWS, HYP_TUNE_SWAP_EPILOGUES, HYP_TUNE_PREFILL_ATTN_TC,
 HYP_TUNE_FIRST_BLOCK_SPLIT, HYP_TUNE_TILE_224, HYP_TUNE_WAIT_LIMIT_US, HYP_TUNE_STREAM_WITHHOLD_COPY,
 HYP_TUNE_STREAM_ACT_DEPTH, HYP_TUNE_STREAM_ACT_TMA, HYP_TUNE_ATTN_GLOBAL_MERGE) = range(16)


def hyp_tune(key: int, value: int):
    _check(lib().hyp_tune(key, value), "hyp_tune")


def hyp_op_pack_weight(w, N: int, swiglu: bool, stream=None, f16: bool = False):
    """Packed copy of a bf16 [N (2N for SwiGLU), K] weight matrix, as hyp_op_gemm reads it (a uint8 tensor);
    f16: the values converted to fp16 on the way (hyp_op_pack_weight_f16, for hyp_op_gemm_f16)."""
    import torch
    K = w.shape[1]
    nbytes = lib().hyp_op_weight_packed_bytes(N, K, int(swiglu))
    if nbytes == 0:
        raise HyperionError(HYP_EINVAL, "hyp_op_weight_packed_bytes")
    packed = torch.empty(nbytes, dtype=torch.uint8, device=w.device)
    name = "hyp_op_pack_weight_f16" if f16 else "hyp_op_pack_weight"
    _check(getattr(lib(), name)(_ptr(w), N, K, int(swiglu), _ptr(packed), nbytes, _stream_handle(stream)), name)
    return packed


def hyp_op_gemm(a, w_packed, N: int, epilogue: int, out, stream=None):
    M, K = a.shape
    _check(lib().hyp_op_gemm(_ptr(a), _ptr(w_packed), M, N, K, epilogue, _ptr(out), out.stride(0),
                             _stream_handle(stream)), "hyp_op_gemm")


def hyp_op_gemm_f16(a, w_packed, N: int, epilogue: int, out, stream=None):
    M, K = a.shape
    _check(lib().hyp_op_gemm_f16(_ptr(a), _ptr(w_packed), M, N, K, epilogue, _ptr(out), out.stride(0),
                                 _stream_handle(stream)), "hyp_op_gemm_f16")


def hyp_device_wait_status(clear: bool = False) -> int:
    """Code recorded by a kernel whose bounded wait ran out (0 = none); synchronises the device."""
    code = C.c_int32(0)
    _check(lib().hyp_device_wait_status(C.byref(code), int(clear)), "hyp_device_wait_status")
    return code.value


def hyp_op_attn_decode_splits(n_seqs: int, n_kv_heads: int, max_ctx: int) -> int:
    return lib().hyp_op_attn_decode_splits(n_seqs, n_kv_heads, max_ctx)


def hyp_op_attn_decode_scratch_bytes(n_seqs: int, n_q_heads: int, head_dim: int, n_splits: int) -> int:
    return lib().hyp_op_attn_decode_scratch_bytes(n_seqs, n_q_heads, head_dim, n_splits)


def hyp_op_attn_decode(shape3, q, kv_pages, block_table, ctx_lens, n_splits, scratch, out, stream=None):
    """shape3 = (n_q_heads, n_kv_heads, head_dim); tensors are CUDA tensors laid out as the header says."""
    sh = hyp_attn_shape(*shape3)
    _check(lib().hyp_op_attn_decode(C.byref(sh), q.shape[0], _ptr(q), q.stride(0), _ptr(kv_pages), _ptr(block_table),
                                    block_table.stride(0), _ptr(ctx_lens), n_splits, _ptr(scratch),
                                    scratch.numel() * scratch.element_size(), _ptr(out), _stream_handle(stream)),
           "hyp_op_attn_decode")


HYP_STATIC_SCRATCH_BYTES = 4 << 20


def hyp_op_attn_decode_static(shape3, q, kv_pages, block_table, ctx_lens, n_splits, out, stream=None):
    """Decode attention that allocates nothing: split partials go to the library's built-in 4 MiB
    device array (shared by all calls on the device; calls that may overlap on the GPU race on it).
    Raises HYP_ECAPACITY if this batch's partials would not fit."""
    sh = hyp_attn_shape(*shape3)
    _check(lib().hyp_op_attn_decode_static(C.byref(sh), q.shape[0], _ptr(q), q.stride(0), _ptr(kv_pages),
                                           _ptr(block_table), block_table.stride(0), _ptr(ctx_lens), n_splits,
                                           _ptr(out), _stream_handle(stream)), "hyp_op_attn_decode_static")


def hyp_op_attn_decode_step(shape3, qkv, kv_pages, block_table, ctx_lens, rope_table, n_splits, out, stream=None):
    sh = hyp_attn_shape(*shape3)
    _check(lib().hyp_op_attn_decode_step(C.byref(sh), qkv.shape[0], _ptr(qkv), qkv.stride(0), _ptr(kv_pages),
                                         _ptr(block_table), block_table.stride(0), _ptr(ctx_lens), _ptr(rope_table),
                                         n_splits, _ptr(out), _stream_handle(stream)), "hyp_op_attn_decode_step")


def hyp_op_attn_prefill(shape3, q, kv_pages, block_table, cu_q, ctx_lens, out, stream=None):
    sh = hyp_attn_shape(*shape3)
    _check(lib().hyp_op_attn_prefill(C.byref(sh), ctx_lens.shape[0], q.shape[0], _ptr(q), q.stride(0), _ptr(kv_pages),
                                     _ptr(block_table), block_table.stride(0), _ptr(cu_q), _ptr(ctx_lens), _ptr(out),
                                     _stream_handle(stream)), "hyp_op_attn_prefill")


# --------------------------------------------------------------------------------------------
# convenience: a stage with its weights loaded from the seeded generator
# --------------------------------------------------------------------------------------------
class Stage:
    """Owns one hyp_stage handle.  Thin: holds the handle and the shape, forwards calls."""

    def __init__(self, shape, layer_lo: int, layer_hi: int, max_seqs: int, max_ctx: int, max_tokens: int,
                 kv_pages: int = 0):
        self.shape, self.lo, self.hi = shape, layer_lo, layer_hi
        self.cfg = make_cfg(shape, max_seqs, max_ctx, max_tokens, kv_pages)
        self.handle = hyp_stage_create(layer_lo, layer_hi, self.cfg)
        self.first, self.last = layer_lo == 0, layer_hi == shape.n_layers_total

    def load_layer(self, layer: int, w: dict, stream=None):
        for key, tid in (("wqkv", HYP_W_QKV), ("wo", HYP_W_O), ("wgu", HYP_W_GATE_UP), ("wd", HYP_W_DOWN),
                         ("g1", HYP_W_NORM1), ("g2", HYP_W_NORM2)):
            hyp_stage_load(self.handle, layer, tid, w[key].contiguous(), stream)

    def load_embed(self, E, stream=None):
        hyp_stage_load(self.handle, -1, HYP_W_EMBED, E.contiguous(), stream)

    def load_head(self, gf, wlm, stream=None):
        n = self.shape.n_layers_total
        hyp_stage_load(self.handle, n, HYP_W_FINAL_NORM, gf.contiguous(), stream)
        hyp_stage_load(self.handle, n, HYP_W_LM_HEAD, wlm.contiguous(), stream)

    def prefill(self, seq_ids, q_lens, ctx_lens, inp, out, stream=None, flags=0):
        hyp_stage_prefill(self.handle, seq_ids, q_lens, ctx_lens, inp, out, stream, flags)

    def decode(self, seq_ids, ctx_lens, inp, out, stream=None):
        hyp_stage_decode(self.handle, seq_ids, ctx_lens, inp, out, stream)

    def profile(self, mode, batch, ctx, iters=5, stream=None):
        return hyp_stage_profile(self.handle, self.hi - self.lo, mode, batch, ctx, iters, stream)

    def free_seq(self, seq_id):
        hyp_stage_free_seq(self.handle, seq_id)

    def close(self):
        if self.handle:
            hyp_stage_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
