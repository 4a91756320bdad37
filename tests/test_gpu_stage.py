"""GPU parity: the library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def dev(t):
    return t.to("cuda")


def test_generator_is_identical_on_cpu_and_cuda():
    a = inputs.normal_bf16(0, 77, (513, 129), device="cpu")
    b = inputs.normal_bf16(0, 77, (513, 129), device="cuda").cpu()
    assert torch.equal(a, b)
    assert torch.equal(inputs.token_ids(1, 3, 1000, 32064), inputs.token_ids(1, 3, 1000, 32064, device="cuda").cpu())


def test_config0_tiny_prefill_then_16_forced_decode_steps():
    sh = inputs.tiny_shape()
    prompt = inputs.token_ids(inputs.SEED_PROMPTS, 0, 32, sh.vocab)
    forced = inputs.token_ids(inputs.SEED_FORCED, 0, 16, sh.vocab)
    seq = torch.cat([prompt, forced])
    want = H.oracle_stage(sh, 0, 2, seq.numpy())                     # [48, V]; row t = logits after token t

    st = H.gpu_stage(sh, 0, 2, max_seqs=2, max_ctx=64, max_tokens=64)
    out = torch.empty(1, sh.vocab, dtype=torch.float32, device="cuda")
    st.prefill([0], [32], [0], dev(prompt), out)
    torch.cuda.synchronize()
    H.assert_logits_close(out.cpu().numpy(), want[31:32], "prefill")
    for s in range(16):
        st.decode([0], [32 + s], dev(forced[s:s + 1]), out)
        torch.cuda.synchronize()
        H.assert_logits_close(out.cpu().numpy(), want[32 + s:33 + s], f"decode step {s}")
    assert hyp.hyp_stage_seq_len(st.handle, 0) == 48
    assert hyp.hyp_stage_launch_count(st.handle) > 0
    st.close()


def test_all_rows_logits_and_random_gains():
    sh = inputs.tiny_shape()
    ids = inputs.token_ids(inputs.SEED_PROMPTS, 5, 33, sh.vocab)     # 33 rows: ragged against 16-token pages
    want = H.oracle_stage(sh, 0, 2, ids.numpy(), random_gains=True)
    st = H.gpu_stage(sh, 0, 2, 1, 64, 64, random_gains=True)
    out = torch.empty(33, sh.vocab, dtype=torch.float32, device="cuda")
    st.prefill([0], [33], [0], dev(ids), out, flags=hyp.HYP_BATCH_ALL_LOGITS)
    torch.cuda.synchronize()
    H.assert_logits_close(out.cpu().numpy(), want, "all rows")
    st.close()


@pytest.mark.parametrize("lens", [[15, 16, 17], [1, 40, 7, 2]])
def test_ragged_batch_page_boundaries_and_batched_decode(lens):
    sh = inputs.tiny_shape()
    n = len(lens)
    st = H.gpu_stage(sh, 0, 2, max_seqs=8, max_ctx=64, max_tokens=80)
    # shuffle the page pool: allocate and free a few sequences so block tables are not monotone
    scratch = torch.empty(3, sh.vocab, dtype=torch.float32, device="cuda")
    st.prefill([5, 6, 7], [20, 3, 33], [0, 0, 0], dev(inputs.token_ids(9, 9, 56, sh.vocab)), scratch)
    st.free_seq(6); st.free_seq(5); st.free_seq(7)
    seqs = [inputs.token_ids(inputs.SEED_PROMPTS, 10 + i, lens[i] + 3, sh.vocab) for i in range(n)]
    want = [H.oracle_stage(sh, 0, 2, s.numpy()) for s in seqs]
    slots = list(range(n))
    out = torch.empty(n, sh.vocab, dtype=torch.float32, device="cuda")
    st.prefill(slots, lens, [0] * n, dev(torch.cat([s[:l] for s, l in zip(seqs, lens)])), out)
    torch.cuda.synchronize()
    for i in range(n):
        H.assert_logits_close(out[i:i + 1].cpu().numpy(), want[i][lens[i] - 1:lens[i]], f"prefill seq {i}")
    for step in range(3):
        tok = torch.stack([seqs[i][lens[i] + step] for i in range(n)])
        st.decode(slots, [l + step for l in lens], dev(tok), out)
        torch.cuda.synchronize()
        for i in range(n):
            H.assert_logits_close(out[i:i + 1].cpu().numpy(), want[i][lens[i] + step:lens[i] + step + 1],
                                  f"decode {step} seq {i}")
    st.close()


def test_decode_attention_merge_variants_agree_bit_for_bit():
    """The stage's decode attention merges its context splits through global scratch rows (the last CTA of a
    (sequence, head) merges; launched early); the cluster variant merges through distributed shared memory.  Both add
    the splits in index order, so a decode run gives the same bits either way - over contexts that span several
    splits, a ragged last page and repeated steps (the ticket counters must be back at zero after every launch).
    """
    sh = inputs.tiny_shape()
    lens = [70, 33, 128, 5]
    n = len(lens)
    seqs = [inputs.token_ids(inputs.SEED_PROMPTS, 40 + i, lens[i] + 4, sh.vocab) for i in range(n)]
    outs = {}
    for variant in (1, 0):
        hyp.hyp_tune(hyp.HYP_TUNE_ATTN_GLOBAL_MERGE, variant)
        hyp.hyp_tune(hyp.HYP_TUNE_ATTN_SPLITS, 3)
        try:
            st = H.gpu_stage(sh, 0, 2, max_seqs=8, max_ctx=160, max_tokens=256)
            out = torch.empty(n, sh.vocab, dtype=torch.float32, device="cuda")
            # prompts go in 8 rows at a time: calls of up to 8 rows run the weight-streaming projections, whose sums
            # have a fixed order (a larger prefill adds its split-K partial tiles in arrival order, so two runs of it
            # need not leave the same bits in the cache)
            for i in range(n):
                for lo in range(0, lens[i], 8):
                    hi = min(lens[i], lo + 8)
                    st.prefill([i], [hi - lo], [lo], dev(seqs[i][lo:hi]), out[:1])
            got = []
            for step in range(4):
                tok = torch.stack([seqs[i][lens[i] + step] for i in range(n)])
                st.decode(list(range(n)), [l + step for l in lens], dev(tok), out)
                torch.cuda.synchronize()
                got.append(out.clone())
            outs[variant] = got
            st.close()
        finally:
            hyp.hyp_tune(hyp.HYP_TUNE_ATTN_GLOBAL_MERGE, 1)
            hyp.hyp_tune(hyp.HYP_TUNE_ATTN_SPLITS, 0)
    want = [H.oracle_stage(sh, 0, 2, s.numpy()) for s in seqs]
    for step in range(4):
        assert torch.equal(outs[1][step], outs[0][step]), f"step {step}"
        for i in range(n):
            H.assert_logits_close(outs[1][step][i:i + 1].cpu().numpy(), want[i][lens[i] + step:lens[i] + step + 1],
                                  f"decode {step} seq {i}")
    assert hyp.hyp_device_wait_status() == 0


def test_chunked_prefill_equals_single_prefill_reference():
    sh = inputs.tiny_shape()
    ids = inputs.token_ids(inputs.SEED_PROMPTS, 20, 45, sh.vocab)
    want = H.oracle_stage(sh, 0, 2, ids.numpy())
    st = H.gpu_stage(sh, 0, 2, 1, 64, 64)
    out = torch.empty(1, sh.vocab, dtype=torch.float32, device="cuda")
    st.prefill([0], [18], [0], dev(ids[:18]), out)
    st.prefill([0], [27], [18], dev(ids[18:]), out)
    torch.cuda.synchronize()
    H.assert_logits_close(out.cpu().numpy(), want[44:45], "chunked")
    st.close()


def test_two_stages_chained_equal_oracle_and_hidden_boundary():
    # blocks [0,1) then [1,2): activations cross the boundary as fp32 [M, H]
    sh = inputs.tiny_shape()
    ids = inputs.token_ids(inputs.SEED_PROMPTS, 30, 24, sh.vocab)
    s0 = H.gpu_stage(sh, 0, 1, 1, 32, 32)
    s1 = H.gpu_stage(sh, 1, 2, 1, 32, 32)
    mid = torch.empty(24, sh.hidden, dtype=torch.float32, device="cuda")
    out = torch.empty(24, sh.vocab, dtype=torch.float32, device="cuda")
    s0.prefill([0], [24], [0], dev(ids), mid)
    s1.prefill([0], [24], [0], mid, out, flags=hyp.HYP_BATCH_ALL_LOGITS)
    torch.cuda.synchronize()
    H.assert_hidden_close(mid.cpu().numpy(), H.oracle_stage(sh, 0, 1, ids.numpy()), "stage 0 output")
    H.assert_logits_close(out.cpu().numpy(), H.oracle_stage(sh, 0, 2, ids.numpy()), "chained")
    s0.close(); s1.close()


def test_host_buffer_entry_points_match_device_ones():
    """Same kernels behind both kinds of entry point.  Calls of up to 8 rows take the weight-streaming projections,
    which are bit-reproducible, so there the two paths must agree exactly; a larger prefill adds its split-K
    partial sums with floating-point atomics, whose order (and with it the last bits, amplified by the fp16
    roundings that follow) may change from run to run, on either path."""
    sh = inputs.tiny_shape()
    ids = inputs.token_ids(inputs.SEED_PROMPTS, 40, 29, sh.vocab)
    st = H.gpu_stage(sh, 0, 2, 2, 48, 32)
    out_d = torch.empty(1, sh.vocab, dtype=torch.float32, device="cuda")
    out_h = torch.empty(1, sh.vocab, dtype=torch.float32).pin_memory()
    st.prefill([0], [8], [0], dev(ids[:8]), out_d)
    hyp.hyp_stage_prefill_host(st.handle, [1], [8], [0], ids[:8].pin_memory(), out_h)
    torch.cuda.synchronize()
    assert torch.equal(out_d.cpu(), out_h)
    st.decode([0], [8], dev(ids[8:9]), out_d)
    hyp.hyp_stage_decode_host(st.handle, [1], [8], ids[8:9].pin_memory(), out_h)
    torch.cuda.synchronize()
    assert torch.equal(out_d.cpu(), out_h)
    # a 19-row chunk behind the 9 cached tokens, then one more decode step
    st.prefill([0], [19], [9], dev(ids[9:28]), out_d)
    hyp.hyp_stage_prefill_host(st.handle, [1], [19], [9], ids[9:28].pin_memory(), out_h)
    torch.cuda.synchronize()
    assert torch.allclose(out_d.cpu(), out_h, rtol=0, atol=5e-3)
    st.decode([0], [28], dev(ids[28:29]), out_d)
    hyp.hyp_stage_decode_host(st.handle, [1], [28], ids[28:29].pin_memory(), out_h)
    torch.cuda.synchronize()
    assert torch.allclose(out_d.cpu(), out_h, rtol=0, atol=5e-3)
    st.close()


def test_error_paths_leave_state_untouched():
    sh = inputs.tiny_shape()
    st = hyp.Stage(sh, 0, 2, 2, 32, 16, kv_pages=3)
    out = torch.empty(1, sh.vocab, dtype=torch.float32, device="cuda")
    ids = dev(inputs.token_ids(1, 50, 40, sh.vocab))

    def code(fn):
        with pytest.raises(hyp.HyperionError) as ei:
            fn()
        return ei.value.code
    assert code(lambda: st.prefill([0], [8], [0], ids, out)) == hyp.HYP_ESTATE          # no weights yet
    for layer in range(2):
        st.load_layer(layer, inputs.layer_weights(sh, layer, device="cuda"))
    st.load_embed(inputs.embed_weights(sh, device="cuda"))
    st.load_head(*inputs.head_weights(sh, device="cuda"))
    assert code(lambda: st.prefill([0], [17], [0], ids, out)) == hyp.HYP_ECAPACITY      # > max_tokens
    assert code(lambda: st.prefill([0], [8], [3], ids, out)) == hyp.HYP_EINVAL          # wrong cached length
    assert code(lambda: st.prefill([2], [8], [0], ids, out)) == hyp.HYP_EINVAL          # slot out of range
    assert code(lambda: st.prefill([0, 0], [4, 4], [0, 0], ids, out)) == hyp.HYP_EINVAL  # duplicate slot
    assert code(lambda: st.prefill([0], [8], [0], ids, out.data_ptr() + 4)) == hyp.HYP_EINVAL   # output not 16-byte aligned
    assert hyp.hyp_stage_seq_len(st.handle, 0) == 0 and hyp.hyp_stage_free_pages(st.handle) == 3
    st.prefill([0], [16], [0], ids, out)                                                 # 1 page
    st.prefill([0], [16], [16], ids, out)                                                # 2 pages
    assert code(lambda: st.prefill([0], [1], [32], ids, out)) == hyp.HYP_ECAPACITY      # > max_ctx
    st.prefill([1], [16], [0], ids, out)                                                 # last page
    assert hyp.hyp_stage_free_pages(st.handle) == 0
    assert code(lambda: st.decode([1], [16], ids, out)) == hyp.HYP_ECAPACITY             # pool exhausted
    assert hyp.hyp_stage_seq_len(st.handle, 1) == 16 and hyp.hyp_stage_seq_len(st.handle, 0) == 32
    st.free_seq(0)
    assert hyp.hyp_stage_free_pages(st.handle) == 2
    st.decode([1], [16], ids, out)
    torch.cuda.synchronize()
    st.close()


def test_profile_returns_positive_times_and_bytes():
    sh = inputs.tiny_shape()
    st = H.gpu_stage(sh, 0, 2, 4, 64, 64)
    for mode, batch, ctx in [(0, 2, 32), (1, 4, 40)]:
        ms, by = st.profile(mode, batch, ctx, iters=3)
        assert len(ms) == 2 and all(m > 0 for m in ms) and all(b > 725_504 * 2 for b in by)
    assert hyp.hyp_stage_free_pages(st.handle) == 4 * 4
    st.close()
