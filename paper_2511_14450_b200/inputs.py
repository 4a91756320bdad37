"""Seeded synthetic inputs: weights, token ids, split costs, arrival processes.

This module holds no arithmetic of the method itself.  It only turns
(seed, stream id, element index) into reproducible numbers, so that a CPU
checker and the GPU library can be fed bit-identical inputs.

Generator definition (counter based; every element is computable on its own):

    mix64(z): z ^= z >> 30; z *= 0xBF58476D1CE4E5B9
              z ^= z >> 27; z *= 0x94D049BB133111EB
              z ^= z >> 31                      (the splitmix64 finaliser)
    key  = mix64(seed * 0x9E3779B97F4A7C15 + stream)
    h(i) = mix64(key + (i + 1) * 0x9E3779B97F4A7C15)        (all mod 2**64)

* bf16 normal weights: ``table[h(i) >> 48]`` where ``table[j]`` is
  ``std * Phi^-1((j + 0.5) / 65536)`` rounded to the nearest-even bf16.  The
  65 536 quantiles are finer than bf16 resolution over the range, so this is
  N(0, std) sampled at bf16 precision, with no floating point in the per-element
  path (integer hash + table lookup), hence identical on CPU and GPU.
* token ids: ``(h(i) >> 1) % vocab``.
* uniform doubles in [0, 1): ``(h(i) >> 11) * 2**-53``.

The hash is written with torch int64 tensor ops (two's-complement wrap-around
equals arithmetic mod 2**64), so the same code runs on ``cpu`` and ``cuda``.
"""
from __future__ import annotations

import functools
import math
from statistics import NormalDist

import numpy as np
import torch

_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK64 = (1 << 64) - 1

# stream ids: one per tensor kind; layer index is folded in by `stream_id`
SEED_WEIGHTS, SEED_PROMPTS, SEED_FORCED, SEED_ARRIVALS, SEED_SPLIT = 0, 1, 2, 3, 4
T_EMBED, T_LMHEAD, T_FINAL_NORM = 1, 2, 3
T_WQKV, T_WO, T_WGU, T_WD, T_G1, T_G2 = 10, 11, 12, 13, 14, 15


def stream_id(tensor: int, layer: int = 0) -> int:
    """Distinct stream per (tensor kind, layer)."""
    return tensor + 64 * (layer + 1)


def _signed(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _mix64_int(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def _key(seed: int, stream: int) -> int:
    return _mix64_int(seed * _GOLDEN + stream)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _signed(_M1)
    z = (z ^ _lsr(z, 27)) * _signed(_M2)
    return z ^ _lsr(z, 31)


def hash_u64(seed: int, stream: int, start: int, n: int, device="cpu") -> torch.Tensor:
    """h(i) for i in [start, start+n) as int64 bit patterns on `device`."""
    i = torch.arange(start + 1, start + n + 1, dtype=torch.int64, device=device)
    return _mix64_t(i * _signed(_GOLDEN) + _signed(_key(seed, stream)))


def hash_u64_numpy(seed: int, stream: int, start: int, n: int) -> np.ndarray:
    """Same hash with numpy uint64 (an independent spelling, used to cross-check)."""
    with np.errstate(over="ignore"):
        i = np.arange(start + 1, start + n + 1, dtype=np.uint64)
        z = i * np.uint64(_GOLDEN) + np.uint64(_key(seed, stream))
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_M1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_M2)
        return z ^ (z >> np.uint64(31))


def _bf16_round_bits(x: float) -> int:
    """float -> nearest-even bf16 bit pattern (finite inputs)."""
    b = np.array([x], dtype=np.float32).view(np.uint32)[0].item()
    b += 0x7FFF + ((b >> 16) & 1)
    return (b >> 16) & 0xFFFF


@functools.lru_cache(maxsize=8)
def normal_table_bits(std: float) -> np.ndarray:
    """65 536 bf16 bit patterns: std * Phi^-1((j + .5) / 65536)."""
    nd = NormalDist()
    out = np.empty(65536, dtype=np.uint16)
    for j in range(65536):
        out[j] = _bf16_round_bits(std * nd.inv_cdf((j + 0.5) / 65536.0))
    return out


_TABLE_CACHE: dict = {}


def _table_on(std: float, device) -> torch.Tensor:
    k = (std, str(device))
    if k not in _TABLE_CACHE:
        bits = torch.from_numpy(normal_table_bits(std).astype(np.int16).copy())
        _TABLE_CACHE[k] = bits.view(torch.bfloat16).to(device)
    return _TABLE_CACHE[k]


def normal_bf16(seed: int, stream: int, shape, std: float = 0.02, device="cpu",
                chunk: int = 1 << 26) -> torch.Tensor:
    """bf16 tensor ~ N(0, std), element i (row-major) drawn from h(i)."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    table = _table_on(std, device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        idx = _lsr(hash_u64(seed, stream, s, m, device), 48)
        out[s:s + m] = table[idx]
    return out.view(*shape)


def uniform_bf16(seed: int, stream: int, shape, lo: float, hi: float, device="cpu") -> torch.Tensor:
    """bf16 tensor ~ U[lo, hi) (used for norm gains that exercise the multiply)."""
    n = int(math.prod(shape))
    u = _lsr(hash_u64(seed, stream, 0, n, "cpu"), 11).to(torch.float64) * (2.0 ** -53)
    return (lo + (hi - lo) * u).to(torch.bfloat16).view(*shape).to(device)


def token_ids(seed: int, stream: int, n: int, vocab: int, device="cpu") -> torch.Tensor:
    """int32 ids uniform in [0, vocab)."""
    return (_lsr(hash_u64(seed, stream, 0, n, device), 1) % vocab).to(torch.int32)


def uniform_f64(seed: int, stream: int, n: int) -> np.ndarray:
    """float64 uniforms in [0, 1)."""
    return (_lsr(hash_u64(seed, stream, 0, n), 11).to(torch.float64) * (2.0 ** -53)).numpy()


def bf16_bits_to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact up-conversion of a bf16 tensor to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()


# ----------------------------------------------------------------------------
# model-shaped bundles
# ----------------------------------------------------------------------------
class ModelShape:
    """Decoder shape; mirrors the library's configuration record field for field."""

    def __init__(self, n_layers_total, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab,
                 rms_eps=1e-5, rope_theta=10000.0, kv_block_size=16):
        self.n_layers_total = n_layers_total
        self.hidden = hidden
        self.n_q_heads = n_q_heads
        self.n_kv_heads = n_kv_heads
        self.head_dim = head_dim
        self.ffn = ffn
        self.vocab = vocab
        self.rms_eps = rms_eps
        self.rope_theta = rope_theta
        self.kv_block_size = kv_block_size

    @property
    def qkv_rows(self):
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def layer_linear_params(self):
        h, f = self.hidden, self.ffn
        return self.qkv_rows * h + h * self.n_q_heads * self.head_dim + 2 * f * h + h * f

    def __repr__(self):
        return (f"ModelShape(L={self.n_layers_total}, H={self.hidden}, Hq={self.n_q_heads}, "
                f"Hkv={self.n_kv_heads}, D={self.head_dim}, F={self.ffn}, V={self.vocab})")


def tiny_shape(n_layers=2):
    return ModelShape(n_layers, 256, 4, 2, 64, 688, 1024)


def phi3_medium_shape(n_layers=40):
    return ModelShape(n_layers, 5120, 40, 10, 128, 17920, 32064)


def llama3_8b_shape(n_layers=32):
    """The paper's second evaluation model (its hardware / model table): 32 blocks, hidden 4096, grouped-query
    attention with 32 query and 8 KV heads of 128, SwiGLU width 14336, vocabulary 128256, rotary base 500000."""
    return ModelShape(n_layers, 4096, 32, 8, 128, 14336, 128256, rope_theta=500000.0)


def layer_weights(shape: ModelShape, layer: int, seed: int = SEED_WEIGHTS, device="cpu",
                  random_gains: bool = False) -> dict:
    """bf16 tensors of one decoder layer, each stored [out, in] row-major.

    wqkv rows = [Q (Hq*D); K (Hkv*D); V (Hkv*D)]; wgu rows = [gate (F); up (F)].
    Norm gains are 1.0 unless `random_gains` (then U[0.5, 1.5))."""
    h, f, qd = shape.hidden, shape.ffn, shape.n_q_heads * shape.head_dim
    w = {
        "wqkv": normal_bf16(seed, stream_id(T_WQKV, layer), (shape.qkv_rows, h), device=device),
        "wo": normal_bf16(seed, stream_id(T_WO, layer), (h, qd), device=device),
        "wgu": normal_bf16(seed, stream_id(T_WGU, layer), (2 * f, h), device=device),
        "wd": normal_bf16(seed, stream_id(T_WD, layer), (h, f), device=device),
    }
    if random_gains:
        w["g1"] = uniform_bf16(seed, stream_id(T_G1, layer), (h,), 0.5, 1.5, device)
        w["g2"] = uniform_bf16(seed, stream_id(T_G2, layer), (h,), 0.5, 1.5, device)
    else:
        w["g1"] = torch.ones(h, dtype=torch.bfloat16, device=device)
        w["g2"] = torch.ones(h, dtype=torch.bfloat16, device=device)
    return w


def embed_weights(shape: ModelShape, seed: int = SEED_WEIGHTS, device="cpu"):
    return normal_bf16(seed, stream_id(T_EMBED), (shape.vocab, shape.hidden), device=device)


def head_weights(shape: ModelShape, seed: int = SEED_WEIGHTS, device="cpu", random_gains=False):
    """(final norm gain [H], LM head [V, H]); the head is untied from the embedding."""
    if random_gains:
        gf = uniform_bf16(seed, stream_id(T_FINAL_NORM), (shape.hidden,), 0.5, 1.5, device)
    else:
        gf = torch.ones(shape.hidden, dtype=torch.bfloat16, device=device)
    return gf, normal_bf16(seed, stream_id(T_LMHEAD), (shape.vocab, shape.hidden), device=device)


def split_instance(N: int, T: int, seed: int = SEED_SPLIT, stream: int = 0, integer: bool = False,
                   tight_memory: bool = False):
    """Seeded partitioning instance (f, m, C, Mcap) as float64 arrays.

    Tier capacities cycle through the ratios 67 : 157 : 200 and memory limits
    through 8 : 16 : 32 (the paper's hardware table), scaled so limits can bind."""
    u = uniform_f64(seed, stream, 2 * N + 2 * T)
    if integer:
        f = np.floor(1 + 9 * u[:N])
        m = np.floor(1 + 3 * u[N:2 * N])
    else:
        f = 1.0 + u[:N]
        m = 0.5 + u[N:2 * N]
    caps = np.array([67.0, 157.0, 200.0])
    mems = np.array([8.0, 16.0, 32.0])
    C = np.array([caps[j % 3] for j in range(T)])
    scale = (m.sum() / T) / 8.0 * (1.05 if tight_memory else 2.5)
    Mcap = np.array([mems[j % 3] * scale for j in range(T)])
    if not integer:
        C = C * (0.9 + 0.2 * u[2 * N:2 * N + T])
    return f, m, C, Mcap


def poisson_arrivals(n: int, rate: float, seed: int = SEED_ARRIVALS, stream: int = 0):
    """Arrival times (s) of a Poisson process: cumulative Exp(1/rate) gaps."""
    u = uniform_f64(seed, stream, n)
    return np.cumsum(-np.log1p(-u) / rate)


def uniform_lengths(n: int, lo: int, hi: int, seed: int = SEED_ARRIVALS, stream: int = 1):
    """Integer lengths uniform in [lo, hi]."""
    u = uniform_f64(seed, stream, n)
    return (lo + np.floor(u * (hi - lo + 1))).astype(np.int64)
