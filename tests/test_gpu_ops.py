"""Single-kernel parity: each kernel through its C entry point against the oracle's matching function,
on small and ragged shapes (tile tails, page boundaries, shuffled block tables) and one full-size case."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs
from tests.helpers import build_cache, f64, kv_rows  # noqa: F401

pytestmark = pytest.mark.gpu


def bf16_normal(stream, shape, std=1.0):
    return inputs.normal_bf16(11, stream, shape, std=std, device="cuda")


@pytest.mark.parametrize("M,H", [(1, 256), (7, 5120), (33, 1000)])
def test_rmsnorm(M, H):
    x = bf16_normal(1, (M, H)).float() * 3.0
    g = inputs.uniform_bf16(11, 2, (H,), 0.5, 1.5, device="cuda")
    out = torch.empty(M, H, dtype=torch.bfloat16, device="cuda")
    hyp.hyp_op_rmsnorm(x, g, out, 1e-5)
    torch.cuda.synchronize()
    want = od.rmsnorm(f64(x), f64(g), 1e-5)
    assert np.max(np.abs(f64(out) - want) / (np.abs(want) + 1e-2)) < 6e-3      # bf16 rounding of the output


GEMM_SHAPES = [  # (M, N, K)
    (1, 256, 256), (8, 512, 256), (32, 256, 688), (5, 1024, 64),          # weight-streaming kernel, K tail
    (8, 528, 1096), (3, 272, 2056), (20, 5120, 17920),                     # its 16-row mode (few rows, long K)
    (24, 7680, 328), (9, 7120, 264),                                       # its 32-column mode for > 8 tokens
    (33, 512, 256), (128, 256, 256), (200, 1024, 688), (129, 272, 328),   # tile kernel: M, N and K tails
    (512, 7680, 5120),                                                     # QKV projection at full size
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("epi", [hyp.HYP_EPI_STORE_BF16, hyp.HYP_EPI_RESID_F32, hyp.HYP_EPI_SWIGLU_BF16,
                                 hyp.HYP_EPI_STORE_F32])
@pytest.mark.parametrize("f16", [False, True])
def test_gemm_all_epilogues(M, N, K, epi, f16):
    """Both instantiations of the projection kernels: bf16 operands (hyp_op_gemm) and fp16 operands
    (hyp_op_gemm_f16, the one the stage path runs)."""
    if M == 512 and epi not in (hyp.HYP_EPI_STORE_BF16, hyp.HYP_EPI_SWIGLU_BF16):
        pytest.skip("full-size case runs the two 16-bit epilogues only")
    swiglu = epi == hyp.HYP_EPI_SWIGLU_BF16
    a = bf16_normal(3, (M, K))
    w = bf16_normal(4, ((2 * N if swiglu else N), K), std=1.0 / np.sqrt(K))
    if f16:
        a = a.half()                       # bf16 values of this size are exact in fp16
    acc = f64(a) @ f64(w.half() if f16 else w).T
    if epi in (hyp.HYP_EPI_STORE_BF16, hyp.HYP_EPI_SWIGLU_BF16):
        out = torch.full((M, N), 7.0, dtype=torch.float16 if f16 else torch.bfloat16, device="cuda")
        want = od.silu(acc[:, :N]) * acc[:, N:] if swiglu else acc
        tol = 6e-3
    else:
        res = bf16_normal(5, (M, N)).float()
        out = res.clone()
        want = acc + (f64(res) if epi == hyp.HYP_EPI_RESID_F32 else 0.0)
        tol = 2e-5 * np.sqrt(K)
    packed = hyp.hyp_op_pack_weight(w, N, swiglu, f16=f16)
    (hyp.hyp_op_gemm_f16 if f16 else hyp.hyp_op_gemm)(a, packed, N, epi, out)
    torch.cuda.synchronize()
    err = np.abs(f64(out) - want) / (np.abs(want) + 1.0)
    assert np.max(err) < tol, (np.max(err), np.unravel_index(np.argmax(err), err.shape))


@pytest.mark.parametrize("M,N,K", [(1, 256, 256), (8, 528, 1096), (20, 5120, 17920), (33, 512, 256), (128, 272, 328),
                                   (100, 1024, 688), (16, 17920, 512)])
@pytest.mark.parametrize("epi", [hyp.HYP_EPI_STORE_BF16, hyp.HYP_EPI_RESID_F32, hyp.HYP_EPI_SWIGLU_BF16,
                                 hyp.HYP_EPI_STORE_F32])
@pytest.mark.parametrize("f16", [False, True])
def test_gemm_swapped_operand_kernel_all_epilogues(M, N, K, epi, f16):
    """Every epilogue and 1-128 rows forced through the swapped-operand kernel (by default it only takes the plain
    stores of 9-128 rows): ragged N (not a multiple of 128), K tails, clusters of 1-8 K shares, all four token tiles."""
    hyp.hyp_tune(hyp.HYP_TUNE_SWAP_MIN_ROWS, 1)
    hyp.hyp_tune(hyp.HYP_TUNE_SWAP_EPILOGUES, 15)
    try:
        test_gemm_all_epilogues(M, N, K, epi, f16)
    finally:
        hyp.hyp_tune(hyp.HYP_TUNE_SWAP_MIN_ROWS, 9)
        hyp.hyp_tune(hyp.HYP_TUNE_SWAP_EPILOGUES, (1 << hyp.HYP_EPI_STORE_BF16) | (1 << hyp.HYP_EPI_STORE_F32))


@pytest.mark.parametrize("N,K,swiglu", [(48, 128, False), (272, 328, True), (1000, 72, False)])
def test_pack_weight_layout(N, K, swiglu):
    """The packed copy against the layout the header states, built with numpy: tile (t, kb) at (t * KBp + kb) * 2 KB,
    t = half * strips + n // 16; inside a tile row r, 16-byte chunk c at chunk position c ^ (r & 7); zero padding."""
    rows = 2 * N if swiglu else N
    w = bf16_normal(8, (rows, K))
    packed = hyp.hyp_op_pack_weight(w, N, swiglu).cpu().numpy().view(np.uint16)
    bits = w.cpu().view(torch.int16).numpy().view(np.uint16)
    strips = -(-N // 16)
    strips += strips & 1
    kbp = -(-K // 64)
    kbp += kbp & 1
    want = np.zeros(((2 if swiglu else 1) * strips, kbp, 16, 8, 8), np.uint16)
    for half in range(2 if swiglu else 1):
        for n in range(N):
            t, r = half * strips + n // 16, n % 16
            for kb in range(-(-K // 64)):
                blk = np.zeros(64, np.uint16)
                seg = bits[half * N + n, kb * 64:min(K, kb * 64 + 64)]
                blk[:len(seg)] = seg
                chunks = blk.reshape(8, 8)
                want[t, kb, r, np.arange(8) ^ (r & 7)] = chunks
    assert packed.size == want.size
    assert np.array_equal(packed, want.reshape(-1))


@pytest.mark.parametrize("Hq,Hkv,D", [(4, 2, 64), (40, 10, 128), (8, 8, 128), (8, 1, 64)])
@pytest.mark.parametrize("n_splits", [1, 3, 8])
def test_attn_decode(Hq, Hkv, D, n_splits):
    lens = [1, 15, 16, 17, 100, 333]                      # tokens visible, new one included
    pool, table, ks, vs = build_cache(lens, Hkv, D, seed=Hq)
    n = len(lens)
    q_stride = (Hq + 2 * Hkv) * D                         # query rows as they sit inside a fused qkv buffer
    q = bf16_normal(50, (n, q_stride)).half()
    ctx = torch.tensor([l - 1 for l in lens], dtype=torch.int32, device="cuda")
    nbytes = hyp.hyp_op_attn_decode_scratch_bytes(n, Hq, D, n_splits)
    scratch = torch.full((nbytes // 4,), float("nan"), dtype=torch.float32, device="cuda")
    out = torch.empty(n, Hq * D, dtype=torch.float16, device="cuda")
    hyp.hyp_op_attn_decode((Hq, Hkv, D), q, pool, table, ctx, n_splits, scratch, out)
    torch.cuda.synchronize()
    for i, L in enumerate(lens):
        qi = f64(q[i, :Hq * D]).reshape(1, Hq, D)
        want = od.attention(qi, f64(ks[i]), f64(vs[i]), q_pos0=L - 1).reshape(-1)
        assert np.max(np.abs(f64(out[i]) - want)) < 1.5e-2, (i, L)


def rope_table(n_pos, D, theta=10000.0):
    """(cos, sin) of pos * theta^(-2i/D), angles in double, stored fp32 [n_pos, D/2, 2]."""
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * theta ** (-2.0 * np.arange(D // 2, dtype=np.float64) / D)
    return torch.from_numpy(np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)).cuda()


@pytest.mark.parametrize("Hq,Hkv,D", [(4, 2, 64), (40, 10, 128), (8, 8, 128), (8, 1, 64)])
@pytest.mark.parametrize("n_splits", [0, 1, 3, 8])
def test_attn_decode_step_rotates_appends_attends_and_merges(Hq, Hkv, D, n_splits):
    """The one-launch decode step against the oracle's rope + attention, on context lengths that sit on, before
    and after page boundaries (0 = the very first token, 16 = the new token opens a page), with more splits than
    pages for the short ones, and a second step on top of the first (the appended key / value must be in the
    cache, in its chunk-permuted place)."""
    cached = [0, 1, 15, 16, 17, 100, 333]                  # tokens already in the cache
    pool, table, ks, vs = build_cache([c + 2 for c in cached], Hkv, D, seed=Hq + 1)   # pages for two more tokens
    n = len(cached)
    tab = rope_table(400, D)
    out = torch.empty(n, Hq * D, dtype=torch.float16, device="cuda")
    stride = (Hq + 2 * Hkv) * D + 8
    ks = [f64(k) for k in ks]
    vs = [f64(v) for v in vs]
    for step in range(2):
        qkv = bf16_normal(70 + step, (n, stride)).float() * 1.5
        ctx = torch.tensor([c + step for c in cached], dtype=torch.int32, device="cuda")
        hyp.hyp_op_attn_decode_step((Hq, Hkv, D), qkv, pool, table, ctx, tab, n_splits, out)
        torch.cuda.synchronize()
        for i, c in enumerate(cached):
            pos = c + step
            row = f64(qkv[i])
            q = od.rope(row[:Hq * D].reshape(1, Hq, D), np.array([pos]), 10000.0)
            k_new = od.rope(row[Hq * D:(Hq + Hkv) * D].reshape(1, Hkv, D), np.array([pos]), 10000.0)
            v_new = row[(Hq + Hkv) * D:(Hq + 2 * Hkv) * D].reshape(1, Hkv, D)
            # what the cache holds after the step: the old rows (fp16 values) and the new one rounded to fp16
            ks[i] = np.concatenate([ks[i][:pos], k_new.astype(np.float16).astype(np.float64)])
            vs[i] = np.concatenate([vs[i][:pos], v_new.astype(np.float16).astype(np.float64)])
            want = od.attention(q, ks[i], vs[i], q_pos0=pos).reshape(-1)
            assert np.max(np.abs(f64(out[i]) - want)) < 1.5e-2, (step, i, pos)
            # the appended row, read back from its page and un-permuted
            page, slot = int(table[i, pos // 16]), pos % 16
            got_k = f64(pool[page, 0, :, slot]).reshape(Hkv, D // 8, 8)
            src = np.arange(D // 8) ^ (slot & 7)
            # fp32 rotation on the device against the float64 one: at most one fp16 step apart after rounding
            assert np.max(np.abs(got_k[:, src].reshape(Hkv, D) - ks[i][pos])) <= 8e-3, (step, i, "key row")
            ks[i][pos] = got_k[:, src].reshape(Hkv, D)      # the next step attends to what the cache really holds
            got_v = f64(pool[page, 1, :, slot]).reshape(Hkv, D // 8, 8)
            assert np.max(np.abs(got_v[:, src].reshape(Hkv, D) - vs[i][pos])) == 0.0, (step, i, "value row")


def test_attn_decode_rejects_small_scratch():
    pool, table, _, _ = build_cache([20], 2, 64, seed=1)
    q = bf16_normal(51, (1, 256)).half()
    ctx = torch.tensor([19], dtype=torch.int32, device="cuda")
    out = torch.empty(1, 256, dtype=torch.float16, device="cuda")
    with pytest.raises(hyp.HyperionError) as ei:
        hyp.hyp_op_attn_decode((4, 2, 64), q, pool, table, ctx, 4, torch.empty(8, device="cuda"), out)
    assert ei.value.code == hyp.HYP_ECAPACITY


@pytest.mark.parametrize("Hq,Hkv", [(40, 10), (8, 8), (8, 1)])
@pytest.mark.parametrize("lens,new", [([37, 5, 64], [37, 2, 20]), ([300, 129, 1, 64], [300, 65, 1, 64]),
                                      ([700, 128, 257], [700, 128, 130]), ([1500, 90, 64], [300, 90, 1])])
def test_attn_prefill_tensor_memory_kernel(Hq, Hkv, lens, new):
    """The tcgen05 prefill attention (head_dim 128, the default there) on the cases of test_attn_prefill plus prompts
    of several key tiles: ragged query tiles, chunked prefill, pages past a sequence's end inside a tile."""
    test_attn_prefill(Hq, Hkv, 128, lens, new)


@pytest.mark.parametrize("lens,new", [([37, 5, 64], [37, 2, 20]), ([300, 129, 1, 64], [300, 65, 1, 64]),
                                      ([700, 128, 257], [700, 128, 130])])
def test_attn_prefill_mma_sync_kernel_head_dim_128(lens, new):
    """head_dim 128 on the mma.sync kernel (otherwise only reached by the other head sizes)."""
    hyp.hyp_tune(hyp.HYP_TUNE_PREFILL_ATTN_TC, 0)
    try:
        test_attn_prefill(40, 10, 128, lens, new)
    finally:
        hyp.hyp_tune(hyp.HYP_TUNE_PREFILL_ATTN_TC, 1)


@pytest.mark.parametrize("Hq,Hkv,D", [(4, 2, 64), (40, 10, 128), (8, 8, 64)])
@pytest.mark.parametrize("lens,new", [([37, 5, 64], [37, 2, 20]), ([300, 129, 1, 64], [300, 65, 1, 64])])
def test_attn_prefill(Hq, Hkv, D, lens, new):
    # lens: cached tokens per sequence (own k, v included); new: query rows = the last `new` positions
    pool, table, ks, vs = build_cache(lens, Hkv, D, seed=3)
    M = sum(new)
    q = bf16_normal(60, (M, Hq * D)).half()
    cu = np.concatenate([[0], np.cumsum(new)]).astype(np.int32)
    cu_q = torch.from_numpy(cu).cuda()
    ctx = torch.tensor([l - c for l, c in zip(lens, new)], dtype=torch.int32, device="cuda")
    out = torch.full((M, Hq * D), 5.0, dtype=torch.float16, device="cuda")
    hyp.hyp_op_attn_prefill((Hq, Hkv, D), q, pool, table, cu_q, ctx, out)
    torch.cuda.synchronize()
    row = 0
    for i, c in enumerate(new):
        qi = f64(q[row:row + c]).reshape(c, Hq, D)
        want = od.attention(qi, f64(ks[i]), f64(vs[i]), q_pos0=lens[i] - c).reshape(c, -1)
        assert np.max(np.abs(f64(out[row:row + c]) - want)) < 2e-2, i
        row += c


def test_expired_wait_is_reported_and_the_next_call_is_clean():
    """The give-up path of a bounded wait, driven once without faulting anything: with the wait limit at 1 ms, one
    launch of the weight-streaming kernel is told to leave one weight copy unissued; the warp that waits for it runs
    into the limit, the kernel records its code, lets its other copies land and returns by itself.  The status
    call reports the code; after clearing it, the same projection is correct again and the status stays clean."""
    M, N, K = 4, 512, 1024
    a = bf16_normal(3, (M, K)).half()
    w = bf16_normal(4, (N, K), std=1.0 / np.sqrt(K))
    packed = hyp.hyp_op_pack_weight(w, N, False, f16=True)
    want = f64(a) @ f64(w.half()).T
    out = torch.zeros(M, N, dtype=torch.float32, device="cuda")
    assert hyp.hyp_device_wait_status() == 0
    hyp.hyp_tune(hyp.HYP_TUNE_WAIT_LIMIT_US, 1000)
    try:
        hyp.hyp_tune(hyp.HYP_TUNE_STREAM_WITHHOLD_COPY, 1)
        hyp.hyp_op_gemm_f16(a, packed, N, hyp.HYP_EPI_STORE_F32, out)      # returns: the kernel gives up by itself
        assert hyp.hyp_device_wait_status(clear=True) == 4                  # the streaming kernel's code
        assert hyp.hyp_device_wait_status() == 0
        out.zero_()
        hyp.hyp_op_gemm_f16(a, packed, N, hyp.HYP_EPI_STORE_F32, out)      # the hook was one-shot
        torch.cuda.synchronize()
        assert np.max(np.abs(f64(out) - want)) < 2e-5 * np.sqrt(K) * (np.max(np.abs(want)) + 1.0)
        assert hyp.hyp_device_wait_status() == 0
    finally:
        hyp.hyp_tune(hyp.HYP_TUNE_WAIT_LIMIT_US, 0)
        hyp.hyp_tune(hyp.HYP_TUNE_STREAM_WITHHOLD_COPY, 0)
