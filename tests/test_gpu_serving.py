"""The multi-stage engine: a model split into stages by HypSplit-DP, continuous batching, every generated
token crossing every stage; per-step logits of every request against the oracle."""
import numpy as np
import pytest
import torch

from oracle import split as osp
from paper_2511_14450_b200 import hyperion as hyp
from paper_2511_14450_b200 import inputs, serving
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_three_stage_engine_matches_oracle_under_continuous_batching():
    sh = inputs.tiny_shape(6)
    lens, n_out = [5, 33, 16, 70, 9], 6
    reqs = [serving.Request(i, 0.002 * i, inputs.token_ids(inputs.SEED_PROMPTS, 700 + i, lens[i], sh.vocab),
                            inputs.token_ids(inputs.SEED_FORCED, 700 + i, n_out, sh.vocab), keep_logits=True)
            for i in range(len(lens))]
    eng = serving.PipelineEngine(sh, [0, 1, 4, 6], max_seqs=3, max_ctx=96, max_tokens=48)   # 3 slots < 5 requests
    stats = eng.run(reqs, realtime=True)
    eng.close()
    assert stats["requests"] == 5 and stats["output_tokens"] == 5 * n_out and stats["decode_steps"] >= n_out - 1
    for r in reqs:
        assert len(r.logits) == n_out and r.t_done >= r.t_first >= 0
        seq = torch.cat([r.prompt, r.forced[:n_out - 1]]).numpy()
        want = H.oracle_stage(sh, 0, 6, seq)
        got = np.stack([l.numpy() for l in r.logits]).astype(np.float64)
        H.assert_logits_close(got, want[len(r.prompt) - 1:], f"request {r.rid}")


def test_plan_stages_profiles_and_splits_like_the_enumerator():
    sh = inputs.tiny_shape(8)
    bounds, tau, ms, nbytes = serving.plan_stages(sh, 3, batch=2, ctx=40)
    assert bounds[0] == 0 and bounds[-1] == 8 and all(b > a for a, b in zip(bounds, bounds[1:]))
    assert len(ms) == 8 and all(m > 0 for m in ms)
    total = torch.cuda.get_device_properties(0).total_memory
    p_e, tau_e = osp.enumerate_split(ms, [float(b) for b in nbytes], [1.0] * 3, [total / 3] * 3)
    assert tuple(bounds[1:-1]) == p_e and tau == tau_e
