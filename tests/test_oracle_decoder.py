"""Pins for the decoder-stage oracle: closed forms, brute force on tiny inputs, library routines
on the special cases that reduce to them, and structural identities.  CPU only."""
import cmath
import math
import os

import numpy as np
import pytest
import torch

from oracle import decoder as od


def rng(seed):
    return np.random.default_rng(seed)


def make_layer(r, H, Hq, Hkv, D, F, gains=True):
    return {
        "wqkv": r.normal(0, 0.2, ((Hq + 2 * Hkv) * D, H)),
        "wo": r.normal(0, 0.2, (H, Hq * D)),
        "wgu": r.normal(0, 0.2, (2 * F, H)),
        "wd": r.normal(0, 0.2, (H, F)),
        "g1": r.uniform(0.5, 1.5, H) if gains else np.ones(H),
        "g2": r.uniform(0.5, 1.5, H) if gains else np.ones(H),
    }


SH = od.Shape(hidden=12, n_q_heads=4, n_kv_heads=2, head_dim=4, ffn=10, vocab=17,
              rms_eps=1e-5, rope_theta=10000.0)


# ---------------------------------------------------------------- RMSNorm
def test_rmsnorm_constant_vector_closed_form():
    # c * ones with unit gain -> c / sqrt(c^2 + eps) in every slot
    for c in (0.0, 1.0, -3.0, 1e-3):
        y = od.rmsnorm(np.full((2, 7), c), np.ones(7), 1e-5)
        assert np.allclose(y, c / math.sqrt(c * c + 1e-5), rtol=0, atol=1e-15)


def test_rmsnorm_matches_torch_rms_norm():
    r = rng(0)
    x, g = r.normal(size=(5, 33)), r.uniform(0.5, 1.5, 33)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (33,), torch.from_numpy(g), eps=1e-5)
    assert np.allclose(od.rmsnorm(x, g, 1e-5), ref.numpy(), rtol=1e-12, atol=1e-12)


def test_rmsnorm_eps_is_inside_the_root():
    x = np.array([[3.0, 4.0]])            # mean square 12.5
    y = od.rmsnorm(x, np.ones(2), 0.5)
    assert np.allclose(y, x / math.sqrt(13.0))


# ---------------------------------------------------------------- RoPE
def test_rope_position_zero_is_identity():
    x = rng(1).normal(size=(1, 3, 8))
    assert np.array_equal(od.rope(x, np.array([0]), 10000.0), x)


def test_rope_preserves_norm_and_relative_property():
    r = rng(2)
    q, k = r.normal(size=(1, 1, 16)), r.normal(size=(1, 1, 16))
    for m, n in [(5, 2), (105, 102), (1000, 997)]:
        qm, kn = od.rope(q, np.array([m]), 10000.0), od.rope(k, np.array([n]), 10000.0)
        assert math.isclose(np.linalg.norm(qm), np.linalg.norm(q), rel_tol=1e-12)
        if m == 5:
            base = float(np.sum(qm * kn))
        assert math.isclose(float(np.sum(qm * kn)), base, rel_tol=1e-9, abs_tol=1e-9)


def test_rope_d2_is_plane_rotation_by_pos_radians():
    x = np.array([[[1.0, 0.0]], [[0.3, -0.7]]])
    y = od.rope(x, np.array([2, 3]), 10000.0)
    for t, pos in enumerate((2, 3)):
        z = complex(x[t, 0, 0], x[t, 0, 1]) * cmath.exp(1j * pos)
        assert np.allclose(y[t, 0], [z.real, z.imag], atol=1e-14)


def test_rope_half_split_pairing_and_frequencies():
    # D = 8: element i pairs with i + 4, angle pos * theta^(-2i/8); complex-number restatement
    D, theta, pos = 8, 10000.0, 7
    x = rng(3).normal(size=(1, 1, D))
    y = od.rope(x, np.array([pos]), theta)[0, 0]
    for i in range(D // 2):
        z = complex(x[0, 0, i], x[0, 0, i + D // 2]) * cmath.exp(1j * pos * theta ** (-2.0 * i / D))
        assert math.isclose(y[i], z.real, abs_tol=1e-13)
        assert math.isclose(y[i + D // 2], z.imag, abs_tol=1e-13)


# ---------------------------------------------------------------- attention
def brute_attention(q, k, v, q_pos0):
    """Scalar loops, math.exp, no vector ops: the definition written out."""
    Tq, Hq, D = q.shape
    Tk, Hkv, _ = k.shape
    G = Hq // Hkv
    out = np.zeros((Tq, Hq, D))
    for t in range(Tq):
        for h in range(Hq):
            kvh = h // G
            sc = []
            for j in range(Tk):
                if j <= q_pos0 + t:
                    sc.append(sum(q[t, h, d] * k[j, kvh, d] for d in range(D)) / math.sqrt(D))
            mx = max(sc)
            e = [math.exp(s - mx) for s in sc]
            z = sum(e)
            for d in range(D):
                out[t, h, d] = sum(e[j] / z * v[j, kvh, d] for j in range(len(sc)))
    return out


@pytest.mark.parametrize("Tq,Tk,Hq,Hkv,D", [(5, 5, 4, 2, 4), (1, 6, 4, 1, 2), (3, 7, 6, 3, 8)])
def test_attention_matches_brute_force(Tq, Tk, Hq, Hkv, D):
    r = rng(10 + Tq)
    q, k, v = r.normal(size=(Tq, Hq, D)), r.normal(size=(Tk, Hkv, D)), r.normal(size=(Tk, Hkv, D))
    got = od.attention(q, k, v, q_pos0=Tk - Tq)
    assert np.allclose(got, brute_attention(q, k, v, Tk - Tq), rtol=1e-12, atol=1e-12)


def test_softmax_rows_sum_to_one_and_causal_mass_is_zero():
    r = rng(20)
    q, k = r.normal(size=(9, 4, 8)) * 4, r.normal(size=(9, 2, 8)) * 4
    P = od.attention_probs(q, k, 0)
    assert np.allclose(P.sum(-1), 1.0, atol=1e-12)
    iu = np.triu_indices(9, 1)
    assert np.all(P[:, iu[0], iu[1]] == 0.0)
    assert np.all(P >= 0)


def test_single_token_attention_returns_v():
    r = rng(21)
    q, k, v = r.normal(size=(1, 4, 8)), r.normal(size=(1, 2, 8)), r.normal(size=(1, 2, 8))
    out = od.attention(q, k, v)
    for h in range(4):
        assert np.array_equal(out[0, h], v[0, h // 2])


def test_mha_special_case_matches_torch_sdpa():
    # Hkv == Hq reduces GQA to plain multi-head attention: a library routine exists for it
    r = rng(22)
    T, Hh, D = 11, 3, 8
    q, k, v = (r.normal(size=(T, Hh, D)) for _ in range(3))
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0]
    assert np.allclose(od.attention(q, k, v), ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-10)


def test_gqa_equals_mha_with_repeated_kv_heads():
    r = rng(23)
    T, Hq, Hkv, D = 6, 6, 2, 4
    q, k, v = r.normal(size=(T, Hq, D)), r.normal(size=(T, Hkv, D)), r.normal(size=(T, Hkv, D))
    krep, vrep = np.repeat(k, Hq // Hkv, axis=1), np.repeat(v, Hq // Hkv, axis=1)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (q, krep, vrep))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0]
    assert np.allclose(od.attention(q, k, v), ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-10)


# ---------------------------------------------------------------- FFN
def test_silu_matches_library_and_closed_values():
    z = np.linspace(-6, 6, 25)
    assert np.allclose(od.silu(z), torch.nn.functional.silu(torch.from_numpy(z)).numpy(), atol=1e-14)
    assert od.silu(np.array([0.0]))[0] == 0.0
    assert math.isclose(od.silu(np.array([1.0]))[0], 1 / (1 + math.exp(-1)))


def test_swiglu_scalar_loops():
    r = rng(30)
    H, F, T = 5, 3, 2
    h, wgu, wd = r.normal(size=(T, H)), r.normal(size=(2 * F, H)), r.normal(size=(H, F))
    exp = np.zeros((T, H))
    for t in range(T):
        u = []
        for j in range(F):
            g = sum(h[t, i] * wgu[j, i] for i in range(H))            # gate rows first
            up = sum(h[t, i] * wgu[F + j, i] for i in range(H))       # then up rows
            u.append(g / (1 + math.exp(-g)) * up)
        for o in range(H):
            exp[t, o] = sum(u[j] * wd[o, j] for j in range(F))
    assert np.allclose(od.swiglu_ffn(h, wgu, wd), exp, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- block / stage
def brute_block(x, w, sh):
    """One block with explicit loops for the projections (index conventions written out)."""
    T, H = x.shape
    Hq, Hkv, D = sh.n_q_heads, sh.n_kv_heads, sh.head_dim

    def norm(row, g):
        ms = sum(a * a for a in row) / len(row)
        return [a / math.sqrt(ms + sh.rms_eps) * gg for a, gg in zip(row, g)]

    def rot(vec, pos):
        half = D // 2
        out = list(vec)
        for i in range(half):
            ang = pos * sh.rope_theta ** (-2.0 * i / D)
            a, b = vec[i], vec[i + half]
            out[i] = a * math.cos(ang) - b * math.sin(ang)
            out[i + half] = b * math.cos(ang) + a * math.sin(ang)
        return out

    q = np.zeros((T, Hq, D)); k = np.zeros((T, Hkv, D)); v = np.zeros((T, Hkv, D))
    for t in range(T):
        hrow = norm(x[t], w["g1"])
        qkv = [sum(hrow[i] * w["wqkv"][o, i] for i in range(H)) for o in range((Hq + 2 * Hkv) * D)]
        for h in range(Hq):
            q[t, h] = rot(qkv[h * D:(h + 1) * D], t)
        for h in range(Hkv):
            k[t, h] = rot(qkv[(Hq + h) * D:(Hq + h + 1) * D], t)
            v[t, h] = qkv[(Hq + Hkv + h) * D:(Hq + Hkv + h + 1) * D]
    a = brute_attention(q, k, v, 0).reshape(T, Hq * D)
    y = np.array(x, dtype=float)
    for t in range(T):
        for o in range(H):
            y[t, o] += sum(a[t, i] * w["wo"][o, i] for i in range(Hq * D))
    z = y.copy()
    for t in range(T):
        hrow = np.array(norm(y[t], w["g2"]))[None]
        z[t] += od.swiglu_ffn(hrow, w["wgu"], w["wd"])[0]      # pinned separately above
    return z


def test_block_matches_scalar_loop_restatement():
    r = rng(40)
    w = make_layer(r, SH.hidden, SH.n_q_heads, SH.n_kv_heads, SH.head_dim, SH.ffn)
    x = r.normal(size=(5, SH.hidden))
    got, _, _ = od.block_forward(x, w, SH)
    assert np.allclose(got, brute_block(x, w, SH), rtol=1e-11, atol=1e-11)


def test_zero_output_projections_make_the_stage_the_identity():
    r = rng(41)
    layers = [make_layer(r, SH.hidden, SH.n_q_heads, SH.n_kv_heads, SH.head_dim, SH.ffn) for _ in range(3)]
    for w in layers:
        w["wo"][:] = 0
        w["wd"][:] = 0
    x = r.normal(size=(4, SH.hidden))
    assert np.array_equal(od.stage_forward(x, layers, SH), x)


def test_cached_decode_equals_full_sequence_recompute():
    r = rng(42)
    layers = [make_layer(r, SH.hidden, SH.n_q_heads, SH.n_kv_heads, SH.head_dim, SH.ffn) for _ in range(3)]
    x = r.normal(size=(12, SH.hidden))
    full = od.stage_forward(x, layers, SH)
    cs = od.CachedStage(layers, SH)
    got = [cs.step(x[:5])]                      # prefill of 5 rows
    got.append(cs.step(x[5:8]))                 # a chunked continuation
    for t in range(8, 12):                      # then token-by-token decode
        got.append(cs.step(x[t:t + 1]))
    assert np.allclose(np.concatenate(got), full, rtol=1e-10, atol=1e-10)


def test_stage_composition_equals_single_stage():
    # running blocks [0,mid) then [mid,L) equals running [0,L): the paper's chaining B_i -> B_{i+1}
    r = rng(43)
    layers = [make_layer(r, SH.hidden, SH.n_q_heads, SH.n_kv_heads, SH.head_dim, SH.ffn) for _ in range(4)]
    x = r.normal(size=(6, SH.hidden))
    whole = od.stage_forward(x, layers, SH)
    for mid in (1, 2, 3):
        assert np.array_equal(od.stage_forward(od.stage_forward(x, layers[:mid], SH), layers[mid:], SH), whole)


def test_causality_future_rows_do_not_change_past_outputs():
    r = rng(44)
    layers = [make_layer(r, SH.hidden, SH.n_q_heads, SH.n_kv_heads, SH.head_dim, SH.ffn) for _ in range(2)]
    x = r.normal(size=(7, SH.hidden))
    a = od.stage_forward(x, layers, SH)
    x2 = x.copy(); x2[5:] += 1.0
    b = od.stage_forward(x2, layers, SH)
    assert np.allclose(a[:5], b[:5], rtol=0, atol=1e-12) and not np.allclose(a[5:], b[5:])


def test_embed_and_lm_head():
    r = rng(45)
    E, W, gf = r.normal(size=(17, 12)), r.normal(size=(17, 12)), r.uniform(0.5, 1.5, 12)
    ids = np.array([3, 0, 16, 3])
    x = od.embed(ids, E)
    assert np.array_equal(x[2], E[16]) and np.array_equal(x[0], x[3])
    logits = od.lm_head(x, gf, W, 1e-5)
    for t in range(4):
        ms = sum(a * a for a in x[t]) / 12
        hn = [a / math.sqrt(ms + 1e-5) * g for a, g in zip(x[t], gf)]
        for vv in (0, 9, 16):
            assert math.isclose(logits[t, vv], sum(hn[i] * W[vv, i] for i in range(12)), rel_tol=1e-11, abs_tol=1e-12)


def test_parameter_count_matches_table_1():
    path = os.path.join(os.path.dirname(__file__), "golden", "table1_models.txt")
    rows = {ln.split()[0]: ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")}
    assert rows["Phi-3-medium"][1] == "14B" and rows["Phi-3-medium"][2] == "40" and rows["Phi-3-medium"][3] == "5120"
    H, Hq, Hkv, D, F, V, L = 5120, 40, 10, 128, 17920, 32064, 40
    per_layer = (Hq + 2 * Hkv) * D * H + H * Hq * D + 2 * F * H + H * F + 2 * H
    assert per_layer == 340_797_440
    total = L * per_layer + 2 * V * H + H
    assert abs(total / 1e9 - 14.0) < 0.1
