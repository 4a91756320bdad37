"""hyp_op_attn_decode_static: decode attention for callers that cannot allocate device memory
(e.g. a server that gave all free HBM to its KV pool, or a plug-in with a frozen memory budget).
Its split partials live in a 4 MiB array inside the library.  The file sorts last on purpose, so a
run that stops at the first failure has already exercised every other test.

The output must agree with hyp_op_attn_decode (caller-supplied scratch) on two calls in a row: the
second call uses another batch and split count, so stale partials from the first would show.  Both
calls are also held against the oracle's attention directly."""
import numpy as np
import pytest
import torch

from oracle import decoder as od
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

TOL = 1.5e-2      # the absolute tolerance the attention op tests use


def _case(lens, Hq, Hkv, D, seed):
    """Seeded queries and a shuffled paged KV cache for sequences of the given lengths (new token included)."""
    pool, table, ks, vs = H.build_cache(lens, Hkv, D, seed)
    q = inputs.normal_bf16(22, seed, (len(lens), Hq * D), std=1.0, device="cuda").half()
    ctx = torch.tensor([l - 1 for l in lens], dtype=torch.int32, device="cuda")
    return q, pool, table, ctx, ks, vs


def _both(lens, Hq, Hkv, D, n_splits, seed):
    """(static-scratch output, caller-scratch output, oracle attention) for one batch."""
    q, pool, table, ctx, ks, vs = _case(lens, Hq, Hkv, D, seed)
    n = len(lens)
    nbytes = hyp.hyp_op_attn_decode_scratch_bytes(n, Hq, D, n_splits)
    assert nbytes <= hyp.HYP_STATIC_SCRATCH_BYTES
    scratch = torch.zeros(nbytes // 4, dtype=torch.float32, device="cuda")
    want = torch.empty(n, Hq * D, dtype=torch.float16, device="cuda")
    got = torch.full_like(want, 9.0)
    hyp.hyp_op_attn_decode((Hq, Hkv, D), q, pool, table, ctx, n_splits, scratch, want)
    hyp.hyp_op_attn_decode_static((Hq, Hkv, D), q, pool, table, ctx, n_splits, got)
    torch.cuda.synchronize()
    ref = np.stack([od.attention(H.f64(q[i]).reshape(1, Hq, D), H.f64(ks[i]), H.f64(vs[i]), q_pos0=L - 1).reshape(-1)
                    for i, L in enumerate(lens)])
    return got.float().cpu().numpy(), want.float().cpu().numpy(), ref


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row():
    for args in (([1, 17, 200, 1000, 64, 333, 16, 5], 40, 10, 128, 8, 1),
                 ([700, 3, 48], 4, 2, 64, 3, 2)):                        # other shape, fewer splits
        got, want, ref = _both(*args)
        assert np.all(np.isfinite(got)) and np.max(np.abs(got - want)) <= TOL
        assert np.max(np.abs(got - ref)) <= TOL                          # and the oracle's attention itself


def test_static_scratch_rejects_batches_beyond_its_limit():
    q, pool, table, ctx, _, _ = _case([20] * 32, 40, 10, 128, seed=3)
    assert hyp.hyp_op_attn_decode_scratch_bytes(32, 40, 128, 32) > hyp.HYP_STATIC_SCRATCH_BYTES
    out = torch.zeros(32, 40 * 128, dtype=torch.float16, device="cuda")
    with pytest.raises(hyp.HyperionError) as ei:
        hyp.hyp_op_attn_decode_static((40, 10, 128), q, pool, table, ctx, 32, out)
    assert ei.value.code == hyp.HYP_ECAPACITY
    torch.cuda.synchronize()
    assert float(out.float().abs().max()) == 0.0                         # nothing was launched
