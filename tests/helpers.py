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


HIDDEN_MAX_ABS_OVER_RMS = 5e-2   # stage output without LM head: max abs error / max(1, rms of the oracle output)


def assert_hidden_close(got, want, what=""):
    """Stage output without an LM head (the logits criterion does not apply to it directly): cosine per row
    >= 0.999 and max-abs <= 5e-2 * max(1, rms(oracle output)) - the logits tolerance carried over to a tensor
    whose scale is not fixed by a final norm.  The logits criterion itself is applied through `assert_probe_logits_close`."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape and np.all(np.isfinite(got)), what
    rms = max(1.0, float(np.sqrt(np.mean(want * want))))
    err = float(np.max(np.abs(got - want)))
    for r in range(got.shape[0]):
        assert od.cosine(got[r], want[r]) >= LOGIT_COSINE, f"{what}: row {r}"
    assert err <= HIDDEN_MAX_ABS_OVER_RMS * rms, f"{what}: max abs err {err} (rms {rms})"
    return err


_PROBE_CACHE = {}


def probe_head(sh, vocab=4096):
    """Seeded probe head for stages that end before the model's last block: (final-norm gain, [vocab, H] matrix)
    as float64.  It is applied ON THE CPU, by the oracle's lm_head, to the library's and to the oracle's stage
    output alike, so the logits criterion can be checked where the stage itself has no head."""
    key = (sh.hidden, vocab)
    if key not in _PROBE_CACHE:
        p = inputs.ModelShape(sh.n_layers_total, sh.hidden, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.ffn, vocab)
        gf, wlm = inputs.head_weights(p, device=_gen_device())
        _PROBE_CACHE[key] = (inputs.bf16_bits_to_f64(gf), inputs.bf16_bits_to_f64(wlm))
    return _PROBE_CACHE[key]


def assert_probe_logits_close(sh, got, want, what=""):
    """The logits criterion (max abs 5e-2, cosine 0.999) on probe-head logits of hidden-state rows."""
    gf, wlm = probe_head(sh)
    return assert_logits_close(od.lm_head(np.asarray(got, np.float64), gf, wlm, sh.rms_eps),
                               od.lm_head(np.asarray(want, np.float64), gf, wlm, sh.rms_eps), what)


def oracle_stage_many(sh, lo, hi, seqs, random_gains=False, logits=True):
    """`oracle_stage` for several independent sequences: every block's float64 weights are materialised once and
    applied to each sequence in turn (the oracle itself still sees one sequence at a time)."""
    osh = oracle_shape(sh)
    if lo == 0:
        E = inputs.bf16_bits_to_f64(inputs.embed_weights(sh, device=_gen_device()))
        xs = [od.embed(np.asarray(s), E) for s in seqs]
        del E
    else:
        xs = [np.asarray(s, np.float64) for s in seqs]
    for w in OracleLayers(sh, lo, hi, random_gains):
        xs = [od.stage_forward(x, [w], osh) for x in xs]
    if hi == sh.n_layers_total and logits:
        gf, wlm = inputs.head_weights(sh, device=_gen_device(), random_gains=random_gains)
        gf, wlm = inputs.bf16_bits_to_f64(gf), inputs.bf16_bits_to_f64(wlm)
        xs = [od.lm_head(x, gf, wlm, sh.rms_eps) for x in xs]
    return xs


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


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
    """Random rotated keys / values (fp16) for each sequence, scattered into a shuffled page pool.
    Returns (pool, block table, keys per sequence, values per sequence)."""
    n = len(seq_lens)
    mpps = max((l + 15) // 16 for l in seq_lens) + 1
    n_pages = n * mpps + 3
    perm = torch.from_numpy(np.random.default_rng(seed).permutation(n_pages)).to(torch.int32)
    pool = torch.zeros(n_pages, 2, Hkv, 16, D, dtype=torch.float16, device="cuda")
    table = torch.zeros(n, mpps, dtype=torch.int32)
    ks, vs = [], []
    for i, L in enumerate(seq_lens):
        k = inputs.normal_bf16(11, 100 + 2 * i + seed, (L, Hkv, D), std=1.0, device="cuda").half()
        v = inputs.normal_bf16(11, 101 + 2 * i + seed, (L, Hkv, D), std=1.0, device="cuda").half()
        ks.append(k); vs.append(v)
        for p in range((L + 15) // 16):
            page = int(perm[i * mpps + p])
            table[i, p] = page
            t0, t1 = 16 * p, min(L, 16 * p + 16)
            pool[page, 0, :, :t1 - t0] = kv_rows(k[t0:t1])
            pool[page, 1, :, :t1 - t0] = kv_rows(v[t0:t1])
    return pool, table.cuda(), ks, vs
