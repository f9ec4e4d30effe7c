"""Shared helpers of the GPU parity tests: tolerances stated once, oracle/GPU data shuttling."""
import numpy as np
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs

TIE_WINDOW = 1e-4          # a code may differ from the oracle only within this distance of a rounding tie
ATTN_REL_TOL = 2e-3        # per (sequence, head) vector: max|diff| <= 2e-3 * max|ref|


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def bf16_ulp(ref: np.ndarray) -> np.ndarray:
    a = np.abs(ref).astype(np.float64)
    e = np.floor(np.log2(np.maximum(a, 2.0**-126)))
    return 2.0 ** (e - 7)


def assert_bf16_close(gpu_bits: np.ndarray, ref_bits: np.ndarray, what: str):
    """|gpu - ref| <= 1 bf16 ulp (relative) + 1e-3 (absolute)."""
    g = orc.bf16_to_f64(gpu_bits)
    r = orc.bf16_to_f64(ref_bits)
    tol = bf16_ulp(r) + 1e-3
    bad = np.abs(g - r) > tol
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside 1 ulp + 1e-3; worst {np.abs(g - r).max()}"
    return float(np.mean(gpu_bits == ref_bits))


def assert_codes_tie_tolerant(gpu_packed: np.ndarray, ref_packed: np.ndarray, tie_dist: np.ndarray, what: str) -> int:
    """Codes equal the oracle's except at rounding ties: a mismatch must differ by exactly one and
    the oracle's pre-rounding value must lie within TIE_WINDOW of a tie. Returns the count."""
    g = orc.unpack_int4(gpu_packed).astype(np.int32)
    r = orc.unpack_int4(ref_packed).astype(np.int32)
    mism = g != r
    n = int(mism.sum())
    if n:
        assert np.all(np.abs(g[mism] - r[mism]) == 1), f"{what}: a code differs by more than one"
        assert np.all(tie_dist[mism] < TIE_WINDOW), f"{what}: mismatch away from a tie (max dist {tie_dist[mism].max()})"
    return n


def assert_attn_close(gpu_bits: np.ndarray, ref_f64: np.ndarray, what: str):
    """Attention tolerance: per (sequence, head) vector the computed values must lie within
    ATTN_REL_TOL * max|ref| of the oracle's unrounded (float64) result; the GPU stores bf16, so
    each element may in addition carry that store's own rounding, half a bf16 ulp."""
    g = orc.bf16_to_f64(gpu_bits)
    vmax = np.abs(ref_f64).max(axis=-1, keepdims=True)
    tol = ATTN_REL_TOL * vmax + 0.5 * bf16_ulp(g) + 1e-30
    err = np.abs(g - ref_f64)
    bad = err > tol
    rel = float(np.max(err / np.maximum(vmax, 1e-30)))
    assert not bad.any(), f"{what}: {bad.sum()} elements outside {ATTN_REL_TOL} relative (+ bf16 store rounding); worst {rel}"
    return rel


def rand_codes(rng, rows, K):
    """Packed uniform codes in [-8, 7] (every value, extremes included)."""
    return rng.integers(0, 256, (rows, K // 2)).astype(np.uint8)
