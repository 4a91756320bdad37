"""The seeded input generators: the torch spelling equals the numpy spelling and a pure-Python
evaluation of the stated definition; distributions have the stated moments.  CPU only."""
import numpy as np
import torch

from paper_2511_14450_b200 import inputs


def test_hash_torch_equals_numpy_equals_python_ints():
    for seed, stream, start in [(0, 74, 0), (3, 1, 12345), (2**31, 999, 2**33)]:
        t = inputs.hash_u64(seed, stream, start, 257).numpy().view(np.uint64)
        n = inputs.hash_u64_numpy(seed, stream, start, 257)
        assert np.array_equal(t, n)
        key = inputs._mix64_int(seed * inputs._GOLDEN + stream)
        for j in (0, 1, 256):
            assert int(n[j]) == inputs._mix64_int(key + (start + j + 1) * inputs._GOLDEN)


def test_normal_weights_moments_and_determinism():
    w = inputs.normal_bf16(0, 5, (512, 1024))
    assert w.dtype == torch.bfloat16 and torch.equal(w, inputs.normal_bf16(0, 5, (512, 1024)))
    x = w.double()
    assert abs(x.mean().item()) < 2e-4 and abs(x.std().item() - 0.02) < 2e-4
    assert abs((x.abs() > 0.04).double().mean().item() - 0.0455) < 2e-3      # two-sigma tail
    assert not torch.equal(w, inputs.normal_bf16(0, 6, (512, 1024)))
    # chunked generation is position-addressed: a different chunk size gives the same tensor
    assert torch.equal(w, inputs.normal_bf16(0, 5, (512, 1024), chunk=1000))


def test_normal_table_is_monotone_and_symmetric():
    tb = torch.from_numpy(inputs.normal_table_bits(0.02).astype(np.int16)).view(torch.bfloat16).double()
    assert torch.all(tb[1:] >= tb[:-1]) and torch.equal(tb, -tb.flip(0))


def test_token_ids_and_lengths_in_range():
    ids = inputs.token_ids(1, 0, 10000, 32064)
    assert ids.dtype == torch.int32 and ids.min() >= 0 and ids.max() < 32064 and ids.unique().numel() > 8000
    ln = inputs.uniform_lengths(1000, 128, 1024)
    assert ln.min() >= 128 and ln.max() <= 1024
    a = inputs.poisson_arrivals(2000, 4.0)
    assert np.all(np.diff(a) > 0) and abs(np.diff(a).mean() - 0.25) < 0.02


def test_layer_weight_shapes():
    sh = inputs.tiny_shape()
    w = inputs.layer_weights(sh, 0)
    assert w["wqkv"].shape == (512, 256) and w["wo"].shape == (256, 256)
    assert w["wgu"].shape == (1376, 256) and w["wd"].shape == (256, 688)
    assert torch.all(w["g1"] == 1)
    assert inputs.phi3_medium_shape().layer_linear_params == 340_787_200
