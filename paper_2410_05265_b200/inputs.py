"""Seeded synthetic inputs shared by the tests, the smoke check and the bench.

Holds none of the method's arithmetic: only a counter-based random generator and the recipes
for Llama-shaped activations, weights, KV tensors and queries. A value depends only on
(seed, stream, flat index), so any slice can be regenerated. Tensors are produced on the
requested device; a test that needs the same bytes on host and device generates once and
copies (transcendentals may differ in the last bit between devices).
"""
from __future__ import annotations

import math

import torch

# stream ids: one per kind of tensor, so tensors with equal seeds never share random numbers
STREAM_SIGMA = 1  # per-channel spread of a layer input, shared by the eval and calibration batches
STREAM_ACT = 2
STREAM_WEIGHT = 3
STREAM_K = 4
STREAM_V = 5
STREAM_Q = 6
STREAM_PREFIX_K = 7
STREAM_PREFIX_V = 8
STREAM_GAIN = 9

_M64 = (1 << 64) - 1


def _s64(v: int) -> int:
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    """64-bit finalizer (splitmix64 style); int64 arithmetic wraps identically on every device."""
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def _mix_int(v: int) -> int:
    v &= _M64
    v = ((v ^ (v >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    v = ((v ^ (v >> 27)) * 0x94D049BB133111EB) & _M64
    return v ^ (v >> 31)


def _key(seed: int, stream: int) -> int:
    return _s64(_mix_int(_mix_int(seed * 0x9E3779B97F4A7C15 + 0x1234567) ^ (stream * 0xD1B54A32D192ED03)))


def normal(seed: int, stream: int, shape, device="cpu", dtype=torch.float64, scale: float = 1.0,
           offset: int = 0, chunk: int = 1 << 24) -> torch.Tensor:
    """N(0, scale^2) samples, Box-Muller in float64 on two hashed counters per element."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    key = _key(seed, stream)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(lo + offset, hi + offset, dtype=torch.int64, device=device)
        h1 = _mix((idx * 2) * _GOLDEN + key)
        h2 = _mix((idx * 2 + 1) * _GOLDEN + key)
        u1 = (_lsr(h1, 11).to(torch.float64) + 0.5) * (1.0 / (1 << 53))
        u2 = (_lsr(h2, 11).to(torch.float64) + 0.5) * (1.0 / (1 << 53))
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[lo:hi] = (z * scale).to(dtype)
    return out.reshape(tuple(shape))


def channel_sigma(K: int, layer: int = 0, device="cpu") -> torch.Tensor:
    """sigma_c ~ LogNormal(0, 0.5): the channel-wise spread of one layer's input (float64 [K])."""
    return torch.exp(0.5 * normal(layer, STREAM_SIGMA, (K,), device))


def outlier_channels(K: int):
    """The four fixed channels that carry the ~1000-magnitude values of a prefixed token."""
    return [(K * 3) // 17, (K * 7) // 17 + 1, (K * 11) // 17 + 2, (K * 15) // 17 + 3]


def activations(M: int, K: int, seed: int, n_prefix: int = 0, layer: int = 0, device="cpu") -> torch.Tensor:
    """Layer input bf16 [M,K]: x[t,c] = N(0,1) * sigma_c. Rows < n_prefix stand for the prefixed
    outlier tokens: same distribution, with four channels forced to +-1000."""
    sig = channel_sigma(K, layer, device)
    out = torch.empty((M, K), dtype=torch.bfloat16, device=device)
    rows = max(1, (1 << 24) // K)
    for r0 in range(0, M, rows):
        r1 = min(M, r0 + rows)
        z = normal(seed, STREAM_ACT + 16 * layer, (r1 - r0, K), device, offset=r0 * K)
        out[r0:r1] = (z * sig).to(torch.bfloat16)
    if n_prefix > 0:
        ch = outlier_channels(K)
        for t in range(min(n_prefix, M)):
            for i, c in enumerate(ch):
                out[t, c] = 1000.0 * (1.0 if (t + i) % 2 == 0 else -1.0) * (1.0 + 0.0625 * i)
    return out


def weights(N: int, K: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    """Linear weight bf16 [N out, K in] ~ N(0, std^2)."""
    return normal(seed, STREAM_WEIGHT, (N, K), device, dtype=torch.bfloat16, scale=std)


def kv_tensor(B: int, T: int, H: int, D: int, seed: int, which: str, device="cpu") -> torch.Tensor:
    """Keys or values bf16 [B,T,H,D] ~ N(0,1)."""
    return normal(seed, STREAM_K if which == "k" else STREAM_V, (B, T, H, D), device, dtype=torch.bfloat16)


def prefix_kv(Hkv: int, n_prefix: int, D: int, seed: int, which: str, magnitude: float = 50.0, device="cpu") -> torch.Tensor:
    """Full-precision K or V of the prefixed tokens, fp16 [Hkv, n_prefix, D] = magnitude * N(0,1)."""
    st = STREAM_PREFIX_K if which == "k" else STREAM_PREFIX_V
    return normal(seed, st, (Hkv, n_prefix, D), device, dtype=torch.float16, scale=magnitude)


def queries(B: int, Hq: int, D: int, seed: int, device="cpu") -> torch.Tensor:
    """Decode queries bf16 [B,Hq,D] ~ N(0,1)."""
    return normal(seed, STREAM_Q, (B, Hq, D), device, dtype=torch.bfloat16)


def bits(t: torch.Tensor):
    """Raw 16-bit patterns of a bf16/fp16 tensor as a host numpy uint16 array (what the oracle takes)."""
    assert t.dtype in (torch.bfloat16, torch.float16)
    return t.detach().contiguous().cpu().view(torch.uint16).numpy()


def from_bits(a, dtype=torch.bfloat16, device="cpu") -> torch.Tensor:
    """Inverse of bits()."""
    return torch.from_numpy(a.copy()).view(dtype).to(device)


# Llama-shaped linear sets: (name, N out, K in, block width of the online rotation)
def linear_set(hidden: int, kv_dim: int, ffn: int):
    had = lambda k: k if (k & (k - 1)) == 0 else 2048
    return [
        ("q", hidden, hidden, had(hidden)),
        ("k", kv_dim, hidden, had(hidden)),
        ("v", kv_dim, hidden, had(hidden)),
        ("o", hidden, hidden, had(hidden)),
        ("gate", ffn, hidden, had(hidden)),
        ("up", ffn, hidden, had(hidden)),
        ("down", hidden, ffn, had(ffn)),
    ]


LLAMA3_8B = dict(hidden=4096, kv_dim=1024, ffn=14336, n_q_heads=32, n_kv_heads=8, head_dim=128)
LLAMA3_70B = dict(hidden=8192, kv_dim=1024, ffn=28672, n_q_heads=64, n_kv_heads=8, head_dim=128)
