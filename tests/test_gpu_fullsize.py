"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times
(tcgen05 tiles for prefill, weight-streaming kernels + graph replay for decode).  The oracle computes
sampled outputs: one sequence of the batch, all of its rows, from a full-sequence causal pass."""
import os

import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_config1_single_phi3_layer_prefill_512():
    """One Phi-3-medium-shaped block, batch 1, 512 tokens: stage output and probe logits."""
    sh = inputs.phi3_medium_shape()
    ids = inputs.token_ids(inputs.SEED_PROMPTS, 0, 512, sh.vocab)
    st = H.gpu_stage(sh, 0, 1, max_seqs=1, max_ctx=512, max_tokens=512)
    out = torch.empty(512, sh.hidden, dtype=torch.float32, device="cuda")
    st.prefill([0], [512], [0], ids.cuda(), out)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    want = H.oracle_stage(sh, 0, 1, ids.numpy())
    H.assert_hidden_close(got, want, "config 1 hidden")
    # probe: the oracle's final norm + a seeded head applied to both outputs (a stage without head has
    # no logits of its own); 64 sampled rows
    rows = np.arange(7, 512, 8)
    H.assert_probe_logits_close(sh, got[rows], want[rows], "config 1 probe logits")
    st.close()


def test_config2_stage14_batch8_ctx1024_decode_sampled_sequence():
    """14 blocks, batch 8, 1024-token contexts, paged KV with shuffled tables, 4 forced decode steps (the
    third and fourth replay the captured graph).  Oracle: sequences 3 and 6 of the batch, every row; the
    hidden-state criterion and the logits criterion through the probe head, both on prefill rows and on
    every decode step."""
    sh = inputs.phi3_medium_shape()
    L, B, C, steps, probes = 14, 8, 1024, 4, (3, 6)
    st = H.gpu_stage(sh, 0, L, max_seqs=B + 2, max_ctx=C + steps + 16, max_tokens=C)
    hid = torch.empty(C, sh.hidden, dtype=torch.float32, device="cuda")
    # shuffle the page pool first
    st.prefill([B], [700], [0], inputs.token_ids(9, 1, 700, sh.vocab, device="cuda"), hid)
    st.prefill([B + 1], [300], [0], inputs.token_ids(9, 2, 300, sh.vocab, device="cuda"), hid)
    st.free_seq(B)
    prompts = [inputs.token_ids(inputs.SEED_PROMPTS, 200 + b, C, sh.vocab) for b in range(B)]
    forced = [inputs.token_ids(inputs.SEED_FORCED, 200 + b, steps, sh.vocab) for b in range(B)]
    got_prefill = {}
    for b in range(B):
        st.prefill([b], [C], [0], prompts[b].cuda(), hid)
        if b in probes:
            torch.cuda.synchronize()
            got_prefill[b] = hid.cpu().numpy().astype(np.float64)
    st.free_seq(B + 1)
    out = torch.empty(B, sh.hidden, dtype=torch.float32, device="cuda")
    got_steps = []
    for s in range(steps):
        tok = torch.stack([forced[b][s] for b in range(B)]).cuda()
        st.decode(list(range(B)), [C + s] * B, tok, out)
        torch.cuda.synchronize()
        got_steps.append(out.cpu().numpy().astype(np.float64))
    # batch invariance at full size: the same sequence decoded alone gives the same row
    probe = probes[0]
    alone = H.gpu_stage(sh, 0, 2, max_seqs=1, max_ctx=C + 8, max_tokens=C)
    both = H.gpu_stage(sh, 0, 2, max_seqs=2, max_ctx=C + 8, max_tokens=C)
    h2 = torch.empty(C, sh.hidden, dtype=torch.float32, device="cuda")
    alone.prefill([0], [C], [0], prompts[probe].cuda(), h2)
    both.prefill([0], [C], [0], prompts[0].cuda(), h2)
    both.prefill([1], [C], [0], prompts[probe].cuda(), h2)
    o1 = torch.empty(1, sh.hidden, dtype=torch.float32, device="cuda")
    o2 = torch.empty(2, sh.hidden, dtype=torch.float32, device="cuda")
    alone.decode([0], [C], forced[probe][:1].cuda(), o1)
    both.decode([0, 1], [C, C], torch.stack([forced[0][0], forced[probe][0]]).cuda(), o2)
    torch.cuda.synchronize()
    assert torch.allclose(o1[0], o2[1], rtol=0, atol=2e-3)
    alone.close(); both.close()
    st.close()
    torch.cuda.empty_cache()

    wants = H.oracle_stage_many(sh, 0, L, [torch.cat([prompts[b], forced[b]]).numpy() for b in probes])   # [C + steps, H] each
    for b, want in zip(probes, wants):
        rows = np.concatenate([np.arange(0, C, 37), [C - 1]])
        H.assert_hidden_close(got_prefill[b][rows], want[rows], f"config 2 seq {b} prefill rows")
        H.assert_probe_logits_close(sh, got_prefill[b][rows], want[rows], f"config 2 seq {b} prefill probe logits")
        dec = np.stack([got_steps[s][b] for s in range(steps)])
        H.assert_hidden_close(dec, want[C:C + steps], f"config 2 seq {b} decode steps")
        H.assert_probe_logits_close(sh, dec, want[C:C + steps], f"config 2 seq {b} decode probe logits")


def _full_model_case(prompt_len, steps, B=4, probe=1):
    """40 blocks + LM head as ONE stage, batch B, equal prompts of `prompt_len`, `steps` forced decode steps;
    per-step logits of sequence `probe` against the oracle's full-sequence pass."""
    sh = inputs.phi3_medium_shape()
    L = sh.n_layers_total
    st = H.gpu_stage(sh, 0, L, max_seqs=B, max_ctx=prompt_len + steps + 16, max_tokens=B * prompt_len)
    prompts = [inputs.token_ids(inputs.SEED_PROMPTS, 400 + b, prompt_len, sh.vocab) for b in range(B)]
    forced = [inputs.token_ids(inputs.SEED_FORCED, 400 + b, steps, sh.vocab) for b in range(B)]
    logits = torch.empty(B, sh.vocab, dtype=torch.float32, device="cuda")
    st.prefill(list(range(B)), [prompt_len] * B, [0] * B, torch.cat(prompts).cuda(), logits)   # one call, B * prompt rows
    torch.cuda.synchronize()
    got = [logits[probe].cpu().numpy().astype(np.float64)]
    for s in range(steps):
        tok = torch.stack([forced[b][s] for b in range(B)]).cuda()
        st.decode(list(range(B)), [prompt_len + s] * B, tok, logits)
        torch.cuda.synchronize()
        got.append(logits[probe].cpu().numpy().astype(np.float64))
    st.close()
    torch.cuda.empty_cache()
    want = H.oracle_stage(sh, 0, L, torch.cat([prompts[probe], forced[probe]]).numpy())      # logits of every row
    errs = []
    for i, g in enumerate(got):
        errs.append(H.assert_logits_close(g[None], want[prompt_len - 1 + i][None], f"full model, step {i - 1}"))
    return max(errs)


def test_config4_shape_40_blocks_with_head_prompt_512():
    """The long-generation configuration's model (40 blocks + 32064-way head, batch 4) at a prompt the oracle
    finishes in about two minutes; checks real per-step logits (no probe head involved)."""
    _full_model_case(prompt_len=512, steps=4)


@pytest.mark.skipif(os.environ.get("HYP_SKIP_SLOW") == "1", reason="oracle needs ~3 min; HYP_SKIP_SLOW=1 skips it")
def test_config4_full_size_prompt_2048():
    """configs[4] at full size: batch 4, 2048-token prompts (8192 rows in one prefill call), first decode steps."""
    _full_model_case(prompt_len=2048, steps=2)


def test_llama3_8b_shaped_blocks_prefill_and_batched_decode():
    """The paper's other model shape (32 blocks, hidden 4096, 32 / 8 heads, FFN 14336, rotary base 500000): two
    blocks, two ragged prompts in one prefill call, then three batched decode steps; stage output against the
    oracle, and the logits criterion through a seeded 4096-way probe head."""
    sh = inputs.llama3_8b_shape()
    sh.vocab = 16384          # only the embedding gather sees it: a 128256-row table would cost the oracle 4 GB
    lens, steps = [300, 77], 3
    st = H.gpu_stage(sh, 0, 2, max_seqs=2, max_ctx=320, max_tokens=sum(lens))
    seqs = [inputs.token_ids(inputs.SEED_PROMPTS, 600 + i, lens[i] + steps, sh.vocab) for i in range(2)]
    want = [H.oracle_stage(sh, 0, 2, s.numpy()) for s in seqs]
    out = torch.empty(sum(lens), sh.hidden, dtype=torch.float32, device="cuda")
    st.prefill([0, 1], lens, [0, 0], torch.cat([s[:l] for s, l in zip(seqs, lens)]).cuda(), out,
               flags=hyp.HYP_BATCH_ALL_LOGITS)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    probe = inputs.ModelShape(32, sh.hidden, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.ffn, 4096)
    gf, wlm = (inputs.bf16_bits_to_f64(t) for t in inputs.head_weights(probe))
    row = 0
    for i, l in enumerate(lens):
        H.assert_hidden_close(got[row:row + l], want[i][:l], f"llama3 prefill seq {i}")
        pick = np.arange(row, row + l, 9)
        H.assert_logits_close(od.lm_head(got[pick], gf, wlm, sh.rms_eps),
                              od.lm_head(want[i][pick - row], gf, wlm, sh.rms_eps), f"llama3 prefill probe seq {i}")
        row += l
    dec = torch.empty(2, sh.hidden, dtype=torch.float32, device="cuda")
    for s_ in range(steps):
        tok = torch.stack([seqs[i][lens[i] + s_] for i in range(2)]).cuda()
        st.decode([0, 1], [l + s_ for l in lens], tok, dec)
        torch.cuda.synchronize()
        g = dec.cpu().numpy().astype(np.float64)
        for i in range(2):
            w = want[i][lens[i] + s_][None]
            H.assert_hidden_close(g[i:i + 1], w, f"llama3 decode step {s_} seq {i}")
            H.assert_logits_close(od.lm_head(g[i:i + 1], gf, wlm, sh.rms_eps), od.lm_head(w, gf, wlm, sh.rms_eps),
                                  f"llama3 decode probe step {s_} seq {i}")
    st.close()


@pytest.mark.parametrize("B", [12, 24, 40])
def test_phi3_shaped_blocks_decode_batches_beyond_8(B):
    """Decode batches that leave the weight-streaming kernel (9-128 rows: tile kernel with stream-K, swapped-operand
    kernel for q/k/v) at the Phi-3-medium shape, through the stage path and its graph replay: two blocks, ragged
    prompt lengths, four steps; three sampled sequences against the oracle."""
    sh = inputs.phi3_medium_shape()
    steps = 4
    lens = [17 + (11 * b) % 90 for b in range(B)]
    st = H.gpu_stage(sh, 0, 2, max_seqs=B, max_ctx=128, max_tokens=sum(lens))
    seqs = [inputs.token_ids(inputs.SEED_PROMPTS, 700 + b, lens[b] + steps, sh.vocab) for b in range(B)]
    hid = torch.empty(sum(lens), sh.hidden, dtype=torch.float32, device="cuda")
    st.prefill(list(range(B)), lens, [0] * B, torch.cat([s[:l] for s, l in zip(seqs, lens)]).cuda(), hid)
    out = torch.empty(B, sh.hidden, dtype=torch.float32, device="cuda")
    got = []
    for s_ in range(steps):
        tok = torch.stack([seqs[b][lens[b] + s_] for b in range(B)]).cuda()
        st.decode(list(range(B)), [l + s_ for l in lens], tok, out)
        torch.cuda.synchronize()
        got.append(out.cpu().numpy().astype(np.float64))
    st.close()
    picks = (0, B // 2, B - 1)
    wants = H.oracle_stage_many(sh, 0, 2, [seqs[b].numpy() for b in picks])
    for b, want in zip(picks, wants):
        dec = np.stack([got[s_][b] for s_ in range(steps)])
        H.assert_hidden_close(dec, want[lens[b]:lens[b] + steps], f"batch {B} seq {b}")
        H.assert_probe_logits_close(sh, dec, want[lens[b]:lens[b] + steps], f"batch {B} seq {b} probe logits")
