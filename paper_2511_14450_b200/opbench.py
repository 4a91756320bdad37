"""Single-kernel microbenchmarks through the C ABI (hyperion_ops.h).

    python -m paper_2511_14450_b200.opbench gemm --M 8 --N 17920 --K 5120 --epi swiglu
    python -m paper_2511_14450_b200.opbench attn_decode --batch 8 --ctx 1024
    python -m paper_2511_14450_b200.opbench attn_prefill --batch 1 --ctx 512
    python -m paper_2511_14450_b200.opbench layer_gemms --M 512
    python -m paper_2511_14450_b200.opbench decode_stage --layers 2 --batch 8 --ctx 1024
    python -m paper_2511_14450_b200.opbench decode_stage --shape llama3 --layers 11 --batch 8 --ctx 1024

Times with CUDA events after warm-up; weights / KV pools are rotated so that no launch finds its
operands in L2.  Prints one JSON line per case.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2511_14450_b200 import hyperion as hyp  # noqa: E402

EPI = {"bf16": hyp.HYP_EPI_STORE_BF16, "resid": hyp.HYP_EPI_RESID_F32, "swiglu": hyp.HYP_EPI_SWIGLU_BF16,
       "f32": hyp.HYP_EPI_STORE_F32}


def _time(fn, iters, warmup=3):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def gemm(M, N, K, epi, iters=20):
    rows = 2 * N if epi == "swiglu" else N
    n_w = max(2, min(8, int(600e6 // (rows * K * 2)) + 1))     # rotate > L2 worth of weights
    a = torch.randn(M, K, device="cuda").bfloat16()
    ws = [hyp.hyp_op_pack_weight((torch.randn(rows, K, device="cuda") * 0.02).bfloat16(), N, epi == "swiglu")
          for _ in range(n_w)]
    out = torch.zeros(M, N, device="cuda", dtype=torch.bfloat16 if epi in ("bf16", "swiglu") else torch.float32)
    ms = _time(lambda i: hyp.hyp_op_gemm(a, ws[i % n_w], N, EPI[epi], out), iters)
    return {"op": "gemm", "M": M, "N": N, "K": K, "epi": epi, "us": ms * 1e3,
            "tflops": 2.0 * M * rows * K / ms / 1e9, "weight_gbs": rows * K * 2 / ms / 1e6}


def attn_decode(batch, ctx, Hq=40, Hkv=10, D=128, iters=20, splits=0):
    mpps = (ctx + 16) // 16
    n_pages = batch * mpps
    pools = [torch.randn(n_pages, 2, Hkv, 16, D, device="cuda").half() for _ in range(4)]
    table = torch.randperm(n_pages, device="cuda").to(torch.int32).view(batch, mpps)
    q = torch.randn(batch, (Hq + 2 * Hkv) * D, device="cuda").half()
    cl = torch.full((batch,), ctx, dtype=torch.int32, device="cuda")
    ns = splits if splits > 0 else hyp.hyp_op_attn_decode_splits(batch, Hkv, ctx + 1)
    scratch = torch.empty(hyp.hyp_op_attn_decode_scratch_bytes(batch, Hq, D, ns) // 4, device="cuda")
    out = torch.empty(batch, Hq * D, device="cuda", dtype=torch.float16)
    ms = _time(lambda i: hyp.hyp_op_attn_decode((Hq, Hkv, D), q, pools[i % 4], table, cl, ns, scratch, out), iters)
    return {"op": "attn_decode", "batch": batch, "ctx": ctx, "splits": ns, "us": ms * 1e3,
            "kv_gbs": batch * (ctx + 1) * 2 * Hkv * D * 2 / ms / 1e6}


def attn_prefill(batch, ctx, Hq=40, Hkv=10, D=128, iters=10):
    mpps = (ctx + 15) // 16
    n_pages = batch * mpps
    pool = torch.randn(n_pages, 2, Hkv, 16, D, device="cuda").half()
    table = torch.arange(n_pages, dtype=torch.int32, device="cuda").view(batch, mpps)
    M = batch * ctx
    q = torch.randn(M, (Hq + 2 * Hkv) * D, device="cuda").half()
    cu = torch.arange(0, M + 1, ctx, dtype=torch.int32, device="cuda")
    c0 = torch.zeros(batch, dtype=torch.int32, device="cuda")
    out = torch.empty(M, Hq * D, device="cuda", dtype=torch.float16)
    ms = _time(lambda i: hyp.hyp_op_attn_prefill((Hq, Hkv, D), q, pool, table, cu, c0, out), iters, warmup=2)
    return {"op": "attn_prefill", "batch": batch, "ctx": ctx, "us": ms * 1e3,
            "tflops_causal": 4.0 * batch * (ctx * (ctx + 1) / 2) * Hq * D / ms / 1e9}


def _shape(name):
    from paper_2511_14450_b200 import inputs
    return inputs.llama3_8b_shape() if name == "llama3" else inputs.phi3_medium_shape()


def layer_gemms(M, shape="phi3"):
    """The four projections of one block of the given model shape at M rows."""
    sh = _shape(shape)
    H, F, HD = sh.hidden, sh.ffn, sh.n_q_heads * sh.head_dim
    cases = [(sh.qkv_rows, H, "bf16"), (H, HD, "resid"), (F, H, "swiglu"), (H, F, "resid")]
    res = [gemm(M, n, k, e) for n, k, e in cases]
    us = sum(r["us"] for r in res)
    flops = 2.0 * M * sh.layer_linear_params
    return res + [{"op": "layer_gemms", "M": M, "us": us, "tflops": flops / us / 1e6}]


def decode_stage(layers, batch, ctx, iters=20, shape="phi3"):
    """Decode steps of a short stage of Phi-3-medium-shaped blocks (the library's own kernel sequence, graph
    replay): a small stand-in for the benchmark's 14-block stage, e.g. for profiling one of its kernels."""
    from paper_2511_14450_b200 import inputs
    sh = _shape(shape)
    if shape == "llama3":
        sh.vocab = 32768      # only the embedding gather sees it; keeps the table small
    chunk = min(ctx, 2048)
    st = hyp.Stage(sh, 0, layers, max_seqs=batch, max_ctx=ctx + iters + 16, max_tokens=chunk)
    for layer in range(layers):
        st.load_layer(layer, inputs.layer_weights(sh, layer, device="cuda"))
        torch.cuda.synchronize()
    st.load_embed(inputs.embed_weights(sh, device="cuda"))
    hidden = torch.empty(chunk, sh.hidden, dtype=torch.float32, device="cuda")
    for b in range(batch):
        done = 0
        while done < ctx:
            n = min(chunk, ctx - done)
            st.prefill([b], [n], [done], inputs.token_ids(inputs.SEED_PROMPTS, b, n, sh.vocab, device="cuda"), hidden)
            done += n
    out = torch.empty(batch, sh.hidden, dtype=torch.float32, device="cuda")
    ids = inputs.token_ids(inputs.SEED_FORCED, 0, batch, sh.vocab, device="cuda")
    slots = list(range(batch))
    pos = [ctx]

    def step(_):
        st.decode(slots, [pos[0]] * batch, ids, out)
        pos[0] += 1

    ms = _time(step, iters, warmup=4)
    st.close()
    kv = layers * batch * (ctx + iters // 2) * 2 * sh.n_kv_heads * sh.head_dim * 2
    return {"op": "decode_stage", "shape": shape, "layers": layers, "batch": batch, "ctx": ctx, "us_per_step": ms * 1e3,
            "us_per_layer": ms * 1e3 / layers,
            "gbs": (layers * sh.layer_linear_params * 2 + kv) / ms / 1e6}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["gemm", "attn_decode", "attn_prefill", "layer_gemms", "decode_stage"])
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--shape", default="phi3", choices=["phi3", "llama3"], help="model shape of layer_gemms / decode_stage")
    ap.add_argument("--M", type=int, default=8)
    ap.add_argument("--N", type=int, default=17920)
    ap.add_argument("--K", type=int, default=5120)
    ap.add_argument("--epi", default="swiglu", choices=list(EPI))
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--ctx", type=int, default=1024)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--splits", type=int, default=0, help="attn_decode: context splits (0 = the library's choice)")
    a = ap.parse_args()
    if a.op == "gemm":
        out = [gemm(a.M, a.N, a.K, a.epi, a.iters)]
    elif a.op == "attn_decode":
        out = [attn_decode(a.batch, a.ctx, iters=a.iters, splits=a.splits)]
    elif a.op == "attn_prefill":
        out = [attn_prefill(a.batch, a.ctx, iters=a.iters)]
    elif a.op == "decode_stage":
        out = [decode_stage(a.layers, a.batch, a.ctx, iters=a.iters, shape=a.shape)]
    else:
        out = layer_gemms(a.M, a.shape)
    for r in out:
        print(json.dumps(r))


if __name__ == "__main__":
    main()
