"""ctypes/numpy front end of the CPU oracle (test infrastructure, never on the product path).

bf16 and fp16 tensors travel as numpy uint16 bit patterns; packed INT4 as uint8; scales as
float32. The shared object is compiled from ``pq_oracle.cpp`` with g++ on first use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_int8, c_int32, c_int64, c_uint8, c_uint16

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pq_oracle.cpp")
_SO = os.path.join(_HERE, "libpq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no fast-math, no FP contraction)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread", _SRC, "-o", tmp]
        )
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_calib_act_scale.restype = c_float
        _lib.orc_gemm_i4.restype = c_int
        _lib.orc_kv4_append.restype = c_int
        _lib.orc_get_threads.restype = c_int
    return _lib


def _p(a: np.ndarray, ct):
    assert a.flags["C_CONTIGUOUS"], "oracle arguments must be C-contiguous"
    return a.ctypes.data_as(POINTER(ct))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16
    return a


def set_threads(n: int) -> None:
    lib().orc_set_threads(c_int(n))


def get_threads() -> int:
    return int(lib().orc_get_threads())


# ---- formats ---------------------------------------------------------------------------------
def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = _u16(bits)
    out = np.empty(bits.shape, np.float64)
    lib().orc_bf16_to_f64(_p(bits, c_uint16), _p(out, c_double), c_int64(bits.size))
    return out


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float64)
    out = np.empty(x.shape, np.uint16)
    lib().orc_f64_to_bf16(_p(x, c_double), _p(out, c_uint16), c_int64(x.size))
    return out


def fp16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = _u16(bits)
    out = np.empty(bits.shape, np.float64)
    lib().orc_fp16_to_f64(_p(bits, c_uint16), _p(out, c_double), c_int64(bits.size))
    return out


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, np.uint8)
    rows = int(np.prod(packed.shape[:-1])) if packed.ndim > 1 else 1
    K = packed.shape[-1] * 2
    out = np.empty(packed.shape[:-1] + (K,), np.int8)
    lib().orc_unpack_int4(_p(packed, c_uint8), _p(out, c_int8), c_int64(rows), c_int64(K))
    return out


def pack_int4(codes: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, np.int8)
    rows = int(np.prod(codes.shape[:-1])) if codes.ndim > 1 else 1
    K = codes.shape[-1]
    assert K % 2 == 0
    out = np.empty(codes.shape[:-1] + (K // 2,), np.uint8)
    lib().orc_pack_int4(_p(codes, c_int8), _p(out, c_uint8), c_int64(rows), c_int64(K))
    return out


# ---- rotation ----------------------------------------------------------------------------------
def rotate_f64(x: np.ndarray, block: int) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float64)
    M, K = x.shape
    assert block == 0 or K % block == 0
    y = np.empty_like(x)
    lib().orc_rotate_f64(_p(x, c_double), _p(y, c_double), c_int64(M), c_int64(K), c_int(block))
    return y


def rotate_bf16(x_bits: np.ndarray, block: int) -> np.ndarray:
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    assert block == 0 or K % block == 0
    y = np.empty((M, K), np.float64)
    lib().orc_rotate_bf16(_p(x_bits, c_uint16), c_int64(K), _p(y, c_double), c_int64(M), c_int64(K), c_int(block))
    return y


# ---- activations ---------------------------------------------------------------------------------
def calib_act_scale(x_bits: np.ndarray, block: int, row_begin: int = 0) -> np.float32:
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    return np.float32(
        lib().orc_calib_act_scale(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin))
    )


def quant_act(x_bits: np.ndarray, block: int, s_a, row_begin: int = 0, want_tie_dist: bool = False):
    """Returns packed codes [M,K/2] (rows < row_begin zero) and, optionally, the tie distances."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    xq = np.zeros((M, K // 2), np.uint8)
    tie = np.full((M, K), 0.5, np.float32) if want_tie_dist else None
    lib().orc_quant_act(
        _p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin),
        c_float(float(s_a)), _p(xq, c_uint8), _p(tie, c_float) if want_tie_dist else None,
    )
    return (xq, tie) if want_tie_dist else xq


def quant_f64(v: np.ndarray, s: float) -> np.ndarray:
    v = np.ascontiguousarray(v, np.float64)
    out = np.empty(v.shape, np.int8)
    lib().orc_quant_f64(_p(v, c_double), c_int64(v.size), c_double(float(s)), _p(out, c_int8))
    return out


def calib_act_scale8(x_bits: np.ndarray, block: int, row_begin: int = 0) -> np.float32:
    """Static per-tensor step of 8-bit activations: max |rotated x| / 127 over rows >= row_begin."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    f = lib().orc_calib_act_scale8
    f.restype = c_float
    return np.float32(f(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin)))


def quant_act8(x_bits: np.ndarray, block: int, s_a, row_begin: int = 0, want_tie_dist: bool = False):
    """Returns int8 codes [M,K] (rows < row_begin zero) and, optionally, the tie distances."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    xq = np.zeros((M, K), np.int8)
    tie = np.full((M, K), 0.5, np.float32) if want_tie_dist else None
    lib().orc_quant_act8(
        _p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin),
        c_float(float(s_a)), _p(xq, c_int8), _p(tie, c_float) if want_tie_dist else None,
    )
    return (xq, tie) if want_tie_dist else xq


def gemm_i8i4(xq8: np.ndarray, wq: np.ndarray) -> np.ndarray:
    """int8 activation codes [M,K] x packed 4-bit weight codes [N,K/2] -> exact int32 [M,N]."""
    xq8 = np.ascontiguousarray(xq8, np.int8)
    wq = np.ascontiguousarray(wq, np.uint8)
    M, K = xq8.shape
    N = wq.shape[0]
    assert wq.shape[1] * 2 == K
    acc = np.empty((M, N), np.int32)
    if lib().orc_gemm_i8i4(_p(xq8, c_int8), _p(wq, c_uint8), c_int64(M), c_int64(N), c_int64(K), _p(acc, c_int32)):
        raise OverflowError("accumulator does not fit int32")
    return acc


def dyn_act_scale(x_bits: np.ndarray, block: int, clip: float = 1.0, row_begin: int = 0) -> np.ndarray:
    """Per-token dynamic steps s[t] = clip * max |rotated x_t| / 7 (rows < row_begin: 0)."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    s = np.zeros(M, np.float32)
    lib().orc_dyn_act_scale(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin),
                            c_float(float(clip)), _p(s, c_float))
    return s


def quant_act_rows(x_bits: np.ndarray, block: int, s_tok: np.ndarray, row_begin: int = 0, want_tie_dist: bool = False):
    """Packed codes [M,K/2] with one step per row (rows < row_begin zero) and, optionally, the tie distances."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    s_tok = np.ascontiguousarray(s_tok, np.float32)
    assert s_tok.shape == (M,)
    xq = np.zeros((M, K // 2), np.uint8)
    tie = np.full((M, K), 0.5, np.float32) if want_tie_dist else None
    lib().orc_quant_act_rows(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin),
                             _p(s_tok, c_float), _p(xq, c_uint8), _p(tie, c_float) if want_tie_dist else None)
    return (xq, tie) if want_tie_dist else xq


def dequant_bf16_rows(acc: np.ndarray, s_tok: np.ndarray, s_w: np.ndarray) -> np.ndarray:
    acc = np.ascontiguousarray(acc, np.int32)
    M, N = acc.shape
    s_tok, s_w = np.ascontiguousarray(s_tok, np.float32), np.ascontiguousarray(s_w, np.float32)
    assert s_tok.shape == (M,) and s_w.shape == (N,)
    out = np.empty((M, N), np.uint16)
    lib().orc_dequant_bf16_rows(_p(acc, c_int32), c_int64(M), c_int64(N), _p(s_tok, c_float), _p(s_w, c_float), _p(out, c_uint16))
    return out


def outlier_tokens(x_bits: np.ndarray, eta1: float = 64.0, eta2: float = 8.0):
    """Token-wise maxima M, outlier degrees R = M / median(M), flags (1 upper, 2 lower, 0 neither) and the median."""
    x_bits = _u16(x_bits)
    T, C = x_bits.shape
    M, R = np.empty(T, np.float32), np.empty(T, np.float32)
    flags, med = np.empty(T, np.int32), np.zeros(1, np.float32)
    lib().orc_outlier_tokens(_p(x_bits, c_uint16), c_int64(C), c_int64(T), c_int64(C), c_float(eta1), c_float(eta2),
                             _p(M, c_float), _p(R, c_float), _p(flags, c_int32), _p(med, c_float))
    return M, R, flags, float(med[0])


def calib_act_minmax(x_bits: np.ndarray, block: int, row_begin: int = 0):
    """(min, max) of the rotated rows >= row_begin, as fp32."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    mn, mx = np.zeros(1, np.float32), np.zeros(1, np.float32)
    lib().orc_calib_act_minmax(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin),
                               _p(mn, c_float), _p(mx, c_float))
    return np.float32(mn[0]), np.float32(mx[0])


def asym_params(mn, mx, bits: int = 4):
    """Eq. 1 with gamma = beta = 1: step s = (mx - mn) / (2^bits - 1) and zero point z = -floor(mn / s)."""
    s, z = np.zeros(1, np.float32), np.zeros(1, np.int32)
    lib().orc_asym_params(c_float(float(mn)), c_float(float(mx)), c_int(bits), _p(s, c_float), _p(z, c_int32))
    return np.float32(s[0]), int(z[0])


def quant_act_asym(x_bits: np.ndarray, block: int, s_a, z: int, row_begin: int = 0, want_tie_dist: bool = False):
    """Unsigned codes [M,K] in 0..15 (rows < row_begin zero) and, optionally, the tie distances."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    u = np.zeros((M, K), np.uint8)
    tie = np.full((M, K), 0.5, np.float32) if want_tie_dist else None
    lib().orc_quant_act_asym(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin),
                             c_float(float(s_a)), c_int32(int(z)), _p(u, c_uint8), _p(tie, c_float) if want_tie_dist else None)
    return (u, tie) if want_tie_dist else u


def grid_candidates(mn, mx, n: int, lo: float, bits: int = 4):
    """The n x n candidates (s, z) of the clipping-factor grid gamma, beta in [lo, 1] (candidate i * n + j)."""
    s, z = np.zeros(n * n, np.float32), np.zeros(n * n, np.int32)
    lib().orc_grid_candidates(c_float(float(mn)), c_float(float(mx)), c_int(bits), c_int(n), c_float(float(lo)), _p(s, c_float), _p(z, c_int32))
    return s, z


def quant_sse_asym(x_bits: np.ndarray, block: int, s_a, z: int, row_begin: int = 0, bits: int = 4) -> float:
    """Squared error of quantizing and dequantizing the rotated rows >= row_begin with step s_a and zero point z."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    f = lib().orc_quant_sse_asym
    f.restype = c_double
    return float(f(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin), c_int(bits),
                   c_float(float(s_a)), c_int32(int(z))))


def grid_search_act(x_bits: np.ndarray, block: int, n: int, lo: float, row_begin: int = 0, bits: int = 4):
    """MSE grid search for the static (s, z): returns s, z and the squared errors of all n * n candidates."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    s, z, sse = np.zeros(1, np.float32), np.zeros(1, np.int32), np.zeros(n * n, np.float64)
    lib().orc_grid_search_act(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin), c_int(bits),
                              c_int(n), c_float(float(lo)), _p(s, c_float), _p(z, c_int32), _p(sse, c_double))
    return np.float32(s[0]), int(z[0]), sse


def grid_search_clip_dyn(x_bits: np.ndarray, block: int, n: int, lo: float, row_begin: int = 0):
    """MSE grid search for the clipping factor shared by the tokens of per-token dynamic quantization: returns the
    chosen factor, the n candidates and their squared errors."""
    x_bits = _u16(x_bits)
    M, K = x_bits.shape
    g, cand, sse = np.zeros(1, np.float32), np.zeros(n, np.float32), np.zeros(n, np.float64)
    lib().orc_grid_search_clip_dyn(_p(x_bits, c_uint16), c_int64(K), c_int64(M), c_int64(K), c_int(block), c_int64(row_begin), c_int(n),
                                   c_float(float(lo)), _p(g, c_float), _p(cand, c_float), _p(sse, c_double))
    return np.float32(g[0]), cand, sse


def gemm_asym(u: np.ndarray, z: int, wq: np.ndarray) -> np.ndarray:
    """sum_k (u[t,k] - z) * w[n,k] with unsigned activation codes and packed signed weight codes -> int32 [M,N]."""
    u = np.ascontiguousarray(u, np.uint8)
    wq = np.ascontiguousarray(wq, np.uint8)
    M, K = u.shape
    N = wq.shape[0]
    assert wq.shape[1] * 2 == K
    acc = np.empty((M, N), np.int32)
    if lib().orc_gemm_asym(_p(u, c_uint8), c_int32(int(z)), _p(wq, c_uint8), c_int64(M), c_int64(N), c_int64(K), _p(acc, c_int32)):
        raise OverflowError("accumulator does not fit int32")
    return acc


# ---- weights ---------------------------------------------------------------------------------------
def quant_weights(w_bits: np.ndarray, want_tie_dist: bool = False):
    """Packed codes [N,K/2], steps [N] and, optionally, the distance of each exact quotient from a rounding tie."""
    w_bits = _u16(w_bits)
    N, K = w_bits.shape
    wq = np.zeros((N, K // 2), np.uint8)
    s_w = np.empty((N,), np.float32)
    tie = np.full((N, K), 0.5, np.float32) if want_tie_dist else None
    lib().orc_quant_weights(_p(w_bits, c_uint16), c_int64(K), c_int64(N), c_int64(K), _p(wq, c_uint8), _p(s_w, c_float),
                            _p(tie, c_float) if want_tie_dist else None)
    return (wq, s_w, tie) if want_tie_dist else (wq, s_w)


# ---- GEMM --------------------------------------------------------------------------------------------
def gemm_i4(xq: np.ndarray, wq: np.ndarray) -> np.ndarray:
    xq = np.ascontiguousarray(xq, np.uint8)
    wq = np.ascontiguousarray(wq, np.uint8)
    M, K2 = xq.shape
    N, K2w = wq.shape
    assert K2 == K2w
    acc = np.empty((M, N), np.int32)
    ovf = lib().orc_gemm_i4(_p(xq, c_uint8), _p(wq, c_uint8), c_int64(M), c_int64(N), c_int64(K2 * 2), _p(acc, c_int32))
    assert ovf == 0, "int32 accumulator overflow in the oracle GEMM"
    return acc


def dequant_bf16(acc: np.ndarray, s_a, s_w: np.ndarray) -> np.ndarray:
    acc = np.ascontiguousarray(acc, np.int32)
    s_w = np.ascontiguousarray(s_w, np.float32)
    M, N = acc.shape
    out = np.empty((M, N), np.uint16)
    lib().orc_dequant_bf16(_p(acc, c_int32), c_int64(M), c_int64(N), c_float(float(s_a)), _p(s_w, c_float), _p(out, c_uint16))
    return out


# ---- KV cache ------------------------------------------------------------------------------------------
def calib_kv_scale(kv_bits: np.ndarray) -> np.ndarray:
    kv_bits = _u16(kv_bits)
    B, T, H, D = kv_bits.shape
    s = np.empty((H,), np.float32)
    lib().orc_calib_kv_scale(_p(kv_bits, c_uint16), c_int64(B), c_int64(T), c_int64(H), c_int64(D), _p(s, c_float))
    return s


def kv4_append(k_bits, v_bits, s_k, s_v, kq, vq, length, tie_k=None, tie_v=None) -> int:
    """In place on kq, vq [B,H,Tmax,D/2] and length [B] int32. Returns the oracle's status.
    tie_k, tie_v: optional float32 [B,T_new,H,D] outputs, distance of each exact quotient from a rounding tie."""
    k_bits, v_bits = _u16(k_bits), _u16(v_bits)
    B, T_new, H, D = k_bits.shape
    Tmax = kq.shape[2]
    assert kq.dtype == np.uint8 and vq.dtype == np.uint8 and length.dtype == np.int32
    s_k = np.ascontiguousarray(s_k, np.float32)
    s_v = np.ascontiguousarray(s_v, np.float32)
    return int(
        lib().orc_kv4_append(
            _p(k_bits, c_uint16), _p(v_bits, c_uint16), c_int64(B), c_int64(T_new), c_int64(H), c_int64(D),
            _p(s_k, c_float), _p(s_v, c_float), _p(kq, c_uint8), _p(vq, c_uint8), _p(length, c_int32), c_int64(Tmax),
            _p(tie_k, c_float) if tie_k is not None else None, _p(tie_v, c_float) if tie_v is not None else None,
        )
    )


def decode_attn(q_bits, prefix_k, prefix_v, kq, vq, s_k, s_v, length, sm_scale, want_f64: bool = False):
    q_bits = _u16(q_bits)
    B, Hq, D = q_bits.shape
    prefix_k, prefix_v = _u16(prefix_k), _u16(prefix_v)
    Hkv, n_prefix = prefix_k.shape[0], prefix_k.shape[1]
    Tmax = kq.shape[2]
    assert kq.shape == (B, Hkv, Tmax, D // 2)
    kq = np.ascontiguousarray(kq, np.uint8)
    vq = np.ascontiguousarray(vq, np.uint8)
    s_k = np.ascontiguousarray(s_k, np.float32)
    s_v = np.ascontiguousarray(s_v, np.float32)
    length = np.ascontiguousarray(length, np.int32)
    out = np.empty((B, Hq, D), np.uint16)
    out64 = np.empty((B, Hq, D), np.float64) if want_f64 else None
    lib().orc_decode_attn(
        _p(q_bits, c_uint16), _p(prefix_k, c_uint16), _p(prefix_v, c_uint16), _p(kq, c_uint8), _p(vq, c_uint8),
        _p(s_k, c_float), _p(s_v, c_float), _p(length, c_int32), c_int64(B), c_int64(Hq), c_int64(Hkv), c_int64(D),
        c_int64(n_prefix), c_int64(Tmax), c_double(float(sm_scale)), _p(out, c_uint16),
        _p(out64, c_double) if want_f64 else None,
    )
    return (out, out64) if want_f64 else out


def kv4_append_dyn(k_bits, v_bits, kq, vq, sk_tok, sv_tok, length) -> int:
    """Group-wise dynamic KV4 (group = one 128-wide (token, head) vector): in place on kq, vq [B,H,Tmax,D/2], the
    per-vector steps sk_tok, sv_tok f32 [B,H,Tmax] and length [B]. Returns the oracle's status."""
    k_bits, v_bits = _u16(k_bits), _u16(v_bits)
    B, T_new, H, D = k_bits.shape
    Tmax = kq.shape[2]
    assert kq.dtype == np.uint8 and vq.dtype == np.uint8 and length.dtype == np.int32
    assert sk_tok.dtype == np.float32 and sv_tok.dtype == np.float32 and sk_tok.shape == (B, H, Tmax) == sv_tok.shape
    f = lib().orc_kv4_append_dyn
    f.restype = c_int
    return int(f(_p(k_bits, c_uint16), _p(v_bits, c_uint16), c_int64(B), c_int64(T_new), c_int64(H), c_int64(D), _p(kq, c_uint8),
                 _p(vq, c_uint8), _p(sk_tok, c_float), _p(sv_tok, c_float), _p(length, c_int32), c_int64(Tmax)))


def decode_attn_dyn(q_bits, prefix_k, prefix_v, kq, vq, sk_tok, sv_tok, length, sm_scale):
    """Decode attention with per-key steps; returns (bf16 bits, float64)."""
    q_bits = _u16(q_bits)
    B, Hq, D = q_bits.shape
    prefix_k, prefix_v = _u16(prefix_k), _u16(prefix_v)
    Hkv, n_prefix = prefix_k.shape[0], prefix_k.shape[1]
    Tmax = kq.shape[2]
    kq, vq = np.ascontiguousarray(kq, np.uint8), np.ascontiguousarray(vq, np.uint8)
    sk_tok, sv_tok = np.ascontiguousarray(sk_tok, np.float32), np.ascontiguousarray(sv_tok, np.float32)
    assert kq.shape == (B, Hkv, Tmax, D // 2) and sk_tok.shape == (B, Hkv, Tmax)
    length = np.ascontiguousarray(length, np.int32)
    out, out64 = np.empty((B, Hq, D), np.uint16), np.empty((B, Hq, D), np.float64)
    lib().orc_decode_attn_dyn(_p(q_bits, c_uint16), _p(prefix_k, c_uint16), _p(prefix_v, c_uint16), _p(kq, c_uint8), _p(vq, c_uint8),
                              _p(sk_tok, c_float), _p(sv_tok, c_float), _p(length, c_int32), c_int64(B), c_int64(Hq), c_int64(Hkv),
                              c_int64(D), c_int64(n_prefix), c_int64(Tmax), c_double(float(sm_scale)), _p(out, c_uint16), _p(out64, c_double))
    return out, out64


def prefill_attn_dyn(q_bits, prefix_k, prefix_v, kq, vq, sk_tok, sv_tok, sm_scale):
    """Causal prefill attention of one sequence with per-key steps [Hkv,Tmax]; returns (bf16 bits, float64)."""
    q_bits = _u16(q_bits)
    T, Hq, D = q_bits.shape
    prefix_k, prefix_v = _u16(prefix_k), _u16(prefix_v)
    Hkv, n_prefix = prefix_k.shape[0], prefix_k.shape[1]
    Tmax = kq.shape[1]
    kq, vq = np.ascontiguousarray(kq, np.uint8), np.ascontiguousarray(vq, np.uint8)
    sk_tok, sv_tok = np.ascontiguousarray(sk_tok, np.float32), np.ascontiguousarray(sv_tok, np.float32)
    assert kq.shape == (Hkv, Tmax, D // 2) and sk_tok.shape == (Hkv, Tmax) and T <= Tmax
    out, out64 = np.empty((T, Hq, D), np.uint16), np.empty((T, Hq, D), np.float64)
    lib().orc_prefill_attn_dyn(_p(q_bits, c_uint16), _p(prefix_k, c_uint16), _p(prefix_v, c_uint16), _p(kq, c_uint8), _p(vq, c_uint8),
                               _p(sk_tok, c_float), _p(sv_tok, c_float), c_int64(T), c_int64(Hq), c_int64(Hkv), c_int64(D),
                               c_int64(n_prefix), c_int64(Tmax), c_double(float(sm_scale)), _p(out, c_uint16), _p(out64, c_double))
    return out, out64


def prefill_attn(q_bits, prefix_k, prefix_v, kq, vq, s_k, s_v, sm_scale, want_f64: bool = False):
    q_bits = _u16(q_bits)
    T, Hq, D = q_bits.shape
    prefix_k, prefix_v = _u16(prefix_k), _u16(prefix_v)
    Hkv, n_prefix = prefix_k.shape[0], prefix_k.shape[1]
    Tmax = kq.shape[1]
    assert kq.shape == (Hkv, Tmax, D // 2) and T <= Tmax
    kq = np.ascontiguousarray(kq, np.uint8)
    vq = np.ascontiguousarray(vq, np.uint8)
    s_k = np.ascontiguousarray(s_k, np.float32)
    s_v = np.ascontiguousarray(s_v, np.float32)
    out = np.empty((T, Hq, D), np.uint16)
    out64 = np.empty((T, Hq, D), np.float64) if want_f64 else None
    lib().orc_prefill_attn(
        _p(q_bits, c_uint16), _p(prefix_k, c_uint16), _p(prefix_v, c_uint16), _p(kq, c_uint8), _p(vq, c_uint8),
        _p(s_k, c_float), _p(s_v, c_float), c_int64(T), c_int64(Hq), c_int64(Hkv), c_int64(D), c_int64(n_prefix),
        c_int64(Tmax), c_double(float(sm_scale)), _p(out, c_uint16), _p(out64, c_double) if want_f64 else None,
    )
    return (out, out64) if want_f64 else out


# ---- block glue --------------------------------------------------------------------------------------------
def rmsnorm(x_bits, g_bits, eps: float = 1e-5):
    x_bits, g_bits = _u16(x_bits), _u16(g_bits)
    M, K = x_bits.shape
    y = np.empty((M, K), np.uint16)
    lib().orc_rmsnorm(_p(x_bits, c_uint16), _p(g_bits, c_uint16), c_int64(M), c_int64(K), c_double(eps), _p(y, c_uint16))
    return y


def rope(x_bits, pos0: int, theta: float):
    x_bits = _u16(x_bits)
    T, H, D = x_bits.shape
    y = np.empty((T, H, D), np.uint16)
    lib().orc_rope(_p(x_bits, c_uint16), c_int64(T), c_int64(H), c_int64(D), c_int64(pos0), c_double(theta), _p(y, c_uint16))
    return y


def rope_rotate(x_bits, pos0: int, theta: float):
    """RoPE, then the head-wise Hadamard rotation R3 (x H_D / sqrt(D)), one rounding to bf16. x [T,H,D]."""
    x_bits = _u16(x_bits)
    T, H, D = x_bits.shape
    y = np.empty_like(x_bits)
    lib().orc_rope_rotate(_p(x_bits, c_uint16), c_int64(T), c_int64(H), c_int64(D), c_int64(pos0), c_double(theta), _p(y, c_uint16))
    return y


def silu_mul(gate_bits, up_bits):
    gate_bits, up_bits = _u16(gate_bits), _u16(up_bits)
    y = np.empty(gate_bits.shape, np.uint16)
    lib().orc_silu_mul(_p(gate_bits, c_uint16), _p(up_bits, c_uint16), c_int64(gate_bits.size), _p(y, c_uint16))
    return y


def add(a_bits, b_bits):
    a_bits, b_bits = _u16(a_bits), _u16(b_bits)
    y = np.empty(a_bits.shape, np.uint16)
    lib().orc_add(_p(a_bits, c_uint16), _p(b_bits, c_uint16), c_int64(a_bits.size), _p(y, c_uint16))
    return y
