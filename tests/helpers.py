"""Glue shared by the GPU parity tests: feed the same seeded inputs to the library and the oracle."""
import numpy as np
import torch

from oracle import decoder as od
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs

LOGIT_MAX_ABS = 5e-2     # per-step logits, max abs error
LOGIT_COSINE = 0.999     # per-step logits, cosine similarity


def oracle_shape(sh):
    return od.Shape(sh.hidden, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.ffn, sh.vocab, sh.rms_eps, sh.rope_theta)


def _gen_device():
    """Where the seeded generator runs.  Its integer hash + table lookup is bit-identical on CPU and CUDA
    (pinned by test_generator_is_identical_on_cpu_and_cuda), so large tensors are generated on the GPU
    when there is one and copied to the host for the oracle."""
    return "cuda" if torch.cuda.is_available() else "cpu"


def oracle_layer(sh, layer, random_gains=False):
    w = inputs.layer_weights(sh, layer, device=_gen_device(), random_gains=random_gains)
    return {k: inputs.bf16_bits_to_f64(v) for k, v in w.items()}


class OracleLayers:
    """Iterable that materialises one layer's float64 weights at a time (bounded memory)."""

    def __init__(self, sh, lo, hi, random_gains=False):
        self.sh, self.lo, self.hi, self.rg = sh, lo, hi, random_gains

    def __iter__(self):
        for layer in range(self.lo, self.hi):
            yield oracle_layer(self.sh, layer, self.rg)


def oracle_stage(sh, lo, hi, x_or_ids, random_gains=False, logits=True):
    """Full-sequence pass of blocks [lo, hi) on one sequence.  ids (int) if lo == 0 else activations."""
    osh = oracle_shape(sh)
    if lo == 0:
        E = inputs.bf16_bits_to_f64(inputs.embed_weights(sh, device=_gen_device()))
        x = od.embed(np.asarray(x_or_ids), E)
    else:
        x = np.asarray(x_or_ids, np.float64)
    x = od.stage_forward(x, OracleLayers(sh, lo, hi, random_gains), osh)
    if hi == sh.n_layers_total and logits:
        gf, wlm = inputs.head_weights(sh, device=_gen_device(), random_gains=random_gains)
        return od.lm_head(x, inputs.bf16_bits_to_f64(gf), inputs.bf16_bits_to_f64(wlm), sh.rms_eps)
    return x


def gpu_stage(sh, lo, hi, max_seqs, max_ctx, max_tokens, random_gains=False, kv_pages=0):
    st = hyp.Stage(sh, lo, hi, max_seqs, max_ctx, max_tokens, kv_pages)
    for layer in range(lo, hi):
        st.load_layer(layer, inputs.layer_weights(sh, layer, device="cuda", random_gains=random_gains))
    if st.first:
        st.load_embed(inputs.embed_weights(sh, device="cuda"))
    if st.last:
        gf, wlm = inputs.head_weights(sh, device="cuda", random_gains=random_gains)
        st.load_head(gf, wlm)
    torch.cuda.synchronize()
    return st


def assert_logits_close(got, want, what=""):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = float(np.max(np.abs(got - want)))
    for r in range(got.shape[0]):
        cs = od.cosine(got[r], want[r])
        assert cs >= LOGIT_COSINE, f"{what}: row {r} cosine {cs}"
    assert err <= LOGIT_MAX_ABS, f"{what}: max abs err {err}"
    return err


HIDDEN_MAX_ABS_OVER_RMS = 1e-1   # stage output without LM head: max abs error / max(1, rms of the oracle output)


def assert_hidden_close(got, want, what=""):
    """Stage output without an LM head (the logits criterion does not apply directly): cosine per row
    >= 0.999 and max-abs <= 0.1 * max(1, rms(oracle output)).  bf16 rounding of q, k, v and of the softmax
    weights gives the attention sub-layer ~0.5 % relative error, which the FFN amplifies to ~1 % of the
    output's rms (0.037 rms / 0.2 max measured on one Phi-3-medium-shaped block); the logits criterion is
    applied separately through a probe head."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape and np.all(np.isfinite(got)), what
    rms = max(1.0, float(np.sqrt(np.mean(want * want))))
    err = float(np.max(np.abs(got - want)))
    for r in range(got.shape[0]):
        assert od.cosine(got[r], want[r]) >= LOGIT_COSINE, f"{what}: row {r}"
    assert err <= HIDDEN_MAX_ABS_OVER_RMS * rms, f"{what}: max abs err {err} (rms {rms})"
    return err
