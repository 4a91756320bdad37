"""Long-sequence generation on the whole model as ONE stage (40 blocks + LM head): batch 4, 2048-token prompts
prefilled in one 8192-row call, then teacher-forced decode steps with the context growing towards 4096.

    python -m paper_2511_14450_b200.longgen [--steps 2048] [--prompt 2048] [--batch 4]

Prints one JSON line: prefill time and TFLOP/s (linear + causal attention flops), decode tokens/s and the
fraction of the HBM roofline (every weight byte once per step plus the KV cache read).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2511_14450_b200 import hyperion as hyp  # noqa: E402
from paper_2511_14450_b200 import inputs  # noqa: E402


def run(steps: int = 2048, prompt: int = 2048, batch: int = 4, layers: int = 40) -> dict:
    """Prefill of batch x prompt rows in one call, then `steps` teacher-forced decode steps; returns the figures
    main() prints (times from CUDA events on the current stream)."""
    sh = inputs.phi3_medium_shape(layers)
    B, P, S, L = batch, prompt, steps, layers
    st = hyp.Stage(sh, 0, L, max_seqs=B, max_ctx=P + S + 16, max_tokens=B * P)
    for layer in range(L):
        st.load_layer(layer, inputs.layer_weights(sh, layer, device="cuda"))
    st.load_embed(inputs.embed_weights(sh, device="cuda"))
    st.load_head(*inputs.head_weights(sh, device="cuda"))
    torch.cuda.synchronize()
    ids = torch.cat([inputs.token_ids(inputs.SEED_PROMPTS, 500 + b, P, sh.vocab) for b in range(B)]).cuda()
    forced = torch.stack([inputs.token_ids(inputs.SEED_FORCED, 500 + b, S, sh.vocab) for b in range(B)], 1).cuda()
    logits = torch.empty(B, sh.vocab, dtype=torch.float32, device="cuda")
    slots = list(range(B))
    # warm-up prefill on other slots is not possible (pool sized for B): warm the kernels with a short call
    st.prefill(slots, [64] * B, [0] * B, ids[:64 * B], logits)
    for b in slots:
        st.free_seq(b)
    torch.cuda.synchronize()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    e[0].record()
    st.prefill(slots, [P] * B, [0] * B, ids, logits)
    e[1].record()
    torch.cuda.synchronize()
    prefill_ms = e[0].elapsed_time(e[1])
    warm = min(8, S // 4)
    ctx = P
    for i in range(warm):
        st.decode(slots, [ctx] * B, forced[i], logits)
        ctx += 1
    torch.cuda.synchronize()
    e[2].record()
    ctx_sum = 0
    for i in range(warm, S):
        st.decode(slots, [ctx] * B, forced[i], logits)
        ctx_sum += ctx + 1
        ctx += 1
    e[3].record()
    torch.cuda.synchronize()
    n = S - warm
    decode_ms = e[2].elapsed_time(e[3]) / n
    st.close()
    lin_flops = 2.0 * B * P * (L * sh.layer_linear_params + sh.vocab * sh.hidden * 0)   # head: last rows only
    attn_flops = 4.0 * B * (P * (P + 1) / 2) * sh.n_q_heads * sh.head_dim * L
    w_bytes = L * (sh.layer_linear_params * 2 + 4 * sh.hidden) + sh.vocab * sh.hidden * 2 + 2 * sh.hidden
    kv_bytes = L * B * 2 * sh.n_kv_heads * sh.head_dim * 2 * (ctx_sum / n)
    peaks = {}
    pth = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(pth):
        peaks = json.load(open(pth))
    hbm = float(peaks.get("hbm_gbs", 6650.0))
    tf = float(peaks.get("bf16_tflops_sustained", 1400.0))
    gbs = (w_bytes + kv_bytes) / 1e9 / (decode_ms / 1e3)
    return {
        "workload": f"configs[4]: {L} Phi-3-medium-shaped blocks + LM head, batch {B}, prompt {P}, {S} decode steps",
        "prefill_ms": prefill_ms, "prefill_tokens_per_s": B * P / (prefill_ms / 1e3),
        "prefill_tflops": (lin_flops + attn_flops) / prefill_ms / 1e9,
        "prefill_frac_of_measured_sustained": (lin_flops + attn_flops) / prefill_ms / 1e9 / tf,
        "decode_steps_timed": n, "decode_ms_per_step": decode_ms, "decode_tokens_per_s": B / (decode_ms / 1e3),
        "decode_bytes_per_step": w_bytes + kv_bytes, "decode_gbs": gbs, "decode_frac_of_measured_hbm": gbs / hbm,
        "decode_frac_of_nominal_8TBs": gbs / 8000.0, "mean_ctx": ctx_sum / n}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=2048)
    ap.add_argument("--prompt", type=int, default=2048)
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--layers", type=int, default=40)
    a = ap.parse_args()
    print(json.dumps(run(a.steps, a.prompt, a.batch, a.layers)))


if __name__ == "__main__":
    main()
