"""Single-kernel parity: each kernel through its C entry point against the oracle's matching function,
on small and ragged shapes (tile tails, page boundaries, shuffled block tables) and one full-size case."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs

pytestmark = pytest.mark.gpu


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


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
    (33, 512, 256), (128, 256, 256), (200, 1024, 688), (129, 272, 328),   # tile kernel: M, N and K tails
    (512, 7680, 5120),                                                     # QKV projection at full size
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("epi", [hyp.HYP_EPI_STORE_BF16, hyp.HYP_EPI_RESID_F32, hyp.HYP_EPI_SWIGLU_BF16,
                                 hyp.HYP_EPI_STORE_F32])
def test_gemm_all_epilogues(M, N, K, epi):
    if M == 512 and epi not in (hyp.HYP_EPI_STORE_BF16, hyp.HYP_EPI_SWIGLU_BF16):
        pytest.skip("full-size case runs the two bf16 epilogues only")
    swiglu = epi == hyp.HYP_EPI_SWIGLU_BF16
    a = bf16_normal(3, (M, K))
    w = bf16_normal(4, ((2 * N if swiglu else N), K), std=1.0 / np.sqrt(K))
    acc = f64(a) @ f64(w).T
    if epi in (hyp.HYP_EPI_STORE_BF16, hyp.HYP_EPI_SWIGLU_BF16):
        out = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
        want = od.silu(acc[:, :N]) * acc[:, N:] if swiglu else acc
        tol = 6e-3
    else:
        res = bf16_normal(5, (M, N)).float()
        out = res.clone()
        want = acc + (f64(res) if epi == hyp.HYP_EPI_RESID_F32 else 0.0)
        tol = 2e-5 * np.sqrt(K)
    hyp.hyp_op_gemm(a, hyp.hyp_op_pack_weight(w, N, swiglu), N, epi, out)
    torch.cuda.synchronize()
    err = np.abs(f64(out) - want) / (np.abs(want) + 1.0)
    assert np.max(err) < tol, (np.max(err), np.unravel_index(np.argmax(err), err.shape))


def kv_rows(x):
    """Token rows [slots, Hkv, D] -> the cache's row layout [Hkv, slots, D]: 16-byte chunk c of the token in
    page slot s sits at chunk position c ^ (s & 7)."""
    slots, Hkv, D = x.shape
    c = torch.arange(D // 8, device=x.device)
    src = (c[None, :] ^ (torch.arange(slots, device=x.device)[:, None] & 7))          # [slots, chunks]
    xc = x.reshape(slots, Hkv, D // 8, 8)
    out = torch.gather(xc, 2, src[:, None, :, None].expand(slots, Hkv, D // 8, 8))
    return out.reshape(slots, Hkv, D).permute(1, 0, 2)


def build_cache(seq_lens, Hkv, D, seed):
    """Random rotated keys / values (fp16) for each sequence, scattered into a shuffled page pool."""
    n = len(seq_lens)
    mpps = max((l + 15) // 16 for l in seq_lens) + 1
    n_pages = n * mpps + 3
    perm = torch.from_numpy(np.random.default_rng(seed).permutation(n_pages)).to(torch.int32)
    pool = torch.zeros(n_pages, 2, Hkv, 16, D, dtype=torch.float16, device="cuda")
    table = torch.zeros(n, mpps, dtype=torch.int32)
    ks, vs = [], []
    for i, L in enumerate(seq_lens):
        k = bf16_normal(100 + 2 * i + seed, (L, Hkv, D)).half()
        v = bf16_normal(101 + 2 * i + seed, (L, Hkv, D)).half()
        ks.append(k); vs.append(v)
        for p in range((L + 15) // 16):
            page = int(perm[i * mpps + p])
            table[i, p] = page
            t0, t1 = 16 * p, min(L, 16 * p + 16)
            pool[page, 0, :, :t1 - t0] = kv_rows(k[t0:t1])
            pool[page, 1, :, :t1 - t0] = kv_rows(v[t0:t1])
    return pool, table.cuda(), ks, vs


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


def test_attn_decode_rejects_small_scratch():
    pool, table, _, _ = build_cache([20], 2, 64, seed=1)
    q = bf16_normal(51, (1, 256)).half()
    ctx = torch.tensor([19], dtype=torch.int32, device="cuda")
    out = torch.empty(1, 256, dtype=torch.float16, device="cuda")
    with pytest.raises(hyp.HyperionError) as ei:
        hyp.hyp_op_attn_decode((4, 2, 64), q, pool, table, ctx, 4, torch.empty(8, device="cuda"), out)
    assert ei.value.code == hyp.HYP_ECAPACITY


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
