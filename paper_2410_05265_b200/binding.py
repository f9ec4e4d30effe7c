"""Thin ctypes binding over the C-ABI CUDA library (argument marshalling only).

Functions take torch CUDA tensors, pass their device pointers and the current torch stream to
the library and raise ``PQError`` on a non-zero status. No step of the path runs in Python or
torch; there is no CPU fallback: without the compiled library every call fails.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_double, c_float, c_int32, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpq_b200.so")

STATUS_NAMES = {
    0: "PQ_OK", 1: "PQ_ERR_INVALID_ARG", 2: "PQ_ERR_SHAPE", 3: "PQ_ERR_ALIGN", 4: "PQ_ERR_WORKSPACE",
    5: "PQ_ERR_CUDA", 6: "PQ_ERR_TIMEOUT", 7: "PQ_ERR_UNSUPPORTED",
}

EXPORTS = [
    "pq_status_string", "pq_create", "pq_destroy", "pq_check", "pq_quant_weights", "pq_hadamard_quant_act",
    "pq_calib_act_scale", "pq_w4a4_gemm_workspace_bytes", "pq_w4a4_gemm", "pq_kv4_append",
    "pq_decode_attn_workspace_bytes", "pq_decode_attn_kv4_prefix", "pq_decode_attn_kv4_prefix_noalloc",
    "pq_rmsnorm", "pq_rope", "pq_silu_mul", "pq_residual_add", "pq_prefill_attn_kv4_prefix", "pq_kv4_append_strided", "pq_calib_kv_scale",
    "pq_hadamard_quant_act8", "pq_hadamard_quant_act_c8", "pq_calib_act_scale8", "pq_w4a8_gemm", "pq_rope_rotate",
    "pq_dyn_act_scale", "pq_dyn_hadamard_quant_act", "pq_hadamard_quant_act_rows", "pq_w4a4_gemm_rows", "pq_outlier_tokens",
    "pq_calib_act_asym", "pq_hadamard_quant_act_asym", "pq_weight_code_sums", "pq_w4a4_gemm_asym",
    "pq_swiglu_hadamard_quant_act", "pq_kv4_append_decode_attn", "pq_set_wait_limit", "pq_probe_i8_mma", "pq_grid_search_act_asym", "pq_grid_search_clip_dyn", "pq_rmsnorm_hadamard_quant_act", "pq_rope_kv4_append", "pq_selftest_wait",
]


class PQError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class KV4CacheStruct(Structure):
    _fields_ = [
        ("prefix_k", c_void_p), ("prefix_v", c_void_p), ("kq", c_void_p), ("vq", c_void_p),
        ("s_k", c_void_p), ("s_v", c_void_p), ("len", c_void_p),
        ("B", c_int32), ("Hq", c_int32), ("Hkv", c_int32), ("D", c_int32), ("n_prefix", c_int32), ("Tmax", c_int32),
        ("sk_tok", c_void_p), ("sv_tok", c_void_p),
    ]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the compiled library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2410_05265_b200.build` first")
    lib = ctypes.CDLL(LIB_PATH)
    lib.pq_status_string.restype = c_char_p
    lib.pq_status_string.argtypes = [c_int32]
    lib.pq_create.argtypes = [POINTER(c_void_p)]
    lib.pq_destroy.argtypes = [c_void_p]
    lib.pq_check.argtypes = [c_void_p, c_void_p]
    lib.pq_set_wait_limit.argtypes = [c_void_p, c_int64]
    lib.pq_selftest_wait.argtypes = [c_void_p, c_void_p, c_void_p]
    lib.pq_probe_i8_mma.argtypes = [c_void_p, c_int32, c_void_p, c_int32, c_void_p]
    lib.pq_quant_weights.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_void_p]
    lib.pq_hadamard_quant_act.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_void_p,
                                          c_void_p, c_void_p]
    lib.pq_calib_act_scale.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_void_p,
                                       c_void_p]
    lib.pq_w4a4_gemm_workspace_bytes.restype = c_size_t
    lib.pq_w4a4_gemm_workspace_bytes.argtypes = [c_int64, c_int64, c_int64]
    lib.pq_w4a4_gemm.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64,
                                 c_int64, c_int64, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.pq_kv4_append.argtypes = [c_void_p, POINTER(KV4CacheStruct), c_void_p, c_void_p, c_int32, c_void_p]
    lib.pq_decode_attn_workspace_bytes.restype = c_size_t
    lib.pq_decode_attn_workspace_bytes.argtypes = [POINTER(KV4CacheStruct)]
    lib.pq_decode_attn_kv4_prefix.argtypes = [c_void_p, POINTER(KV4CacheStruct), c_void_p, c_void_p, c_float, c_void_p,
                                              c_size_t, c_void_p]
    lib.pq_decode_attn_kv4_prefix_noalloc.argtypes = [POINTER(KV4CacheStruct), c_void_p, c_void_p, c_float, c_void_p]
    lib.pq_calib_kv_scale.argtypes = [c_void_p, c_void_p, c_int64, c_int32, c_int32, c_int64, c_void_p, c_void_p]
    lib.pq_kv4_append_strided.argtypes = [c_void_p, POINTER(KV4CacheStruct), c_void_p, c_void_p, c_int32, c_int64, c_void_p]
    lib.pq_prefill_attn_kv4_prefix.argtypes = [c_void_p, POINTER(KV4CacheStruct), c_int32, c_void_p, c_int64, c_int32, c_void_p, c_float,
                                               c_void_p]
    lib.pq_rmsnorm.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_float, c_void_p, c_int64, c_void_p]
    lib.pq_rope.argtypes = [c_void_p, c_void_p, c_int64, c_int32, c_int32, c_int64, c_int64, c_double, c_void_p, c_void_p]
    lib.pq_rope_rotate.argtypes = lib.pq_rope.argtypes
    lib.pq_silu_mul.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p]
    lib.pq_residual_add.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_void_p]
    lib.pq_hadamard_quant_act8.argtypes = lib.pq_hadamard_quant_act.argtypes
    lib.pq_hadamard_quant_act_c8.argtypes = lib.pq_hadamard_quant_act.argtypes
    lib.pq_calib_act_scale8.argtypes = lib.pq_calib_act_scale.argtypes
    lib.pq_w4a8_gemm.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int64,
                                 c_int64, c_void_p, c_void_p]
    lib.pq_dyn_act_scale.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_float, c_void_p, c_void_p]
    lib.pq_hadamard_quant_act_rows.argtypes = lib.pq_hadamard_quant_act.argtypes
    lib.pq_dyn_hadamard_quant_act.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_float, c_void_p, c_void_p,
                                              c_void_p]
    lib.pq_w4a4_gemm_rows.argtypes = lib.pq_w4a8_gemm.argtypes
    lib.pq_outlier_tokens.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_float, c_float, c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_void_p]
    lib.pq_calib_act_asym.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_void_p, c_void_p, c_void_p]
    lib.pq_rmsnorm_hadamard_quant_act.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_float, c_int64, c_void_p,
                                                  c_void_p, c_void_p]
    lib.pq_rope_kv4_append.argtypes = [c_void_p, POINTER(KV4CacheStruct), c_int32, c_void_p, c_int64, c_int64, c_int64, c_double, c_int32,
                                       c_void_p]
    lib.pq_grid_search_clip_dyn.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_int32, c_float, c_void_p,
                                            c_void_p, c_void_p, c_void_p, c_void_p]
    lib.pq_grid_search_act_asym.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_int32, c_float, c_void_p,
                                            c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.pq_hadamard_quant_act_asym.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_void_p, c_void_p,
                                               c_void_p, c_void_p]
    lib.pq_weight_code_sums.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_void_p]
    lib.pq_w4a4_gemm_asym.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64,
                                      c_int64, c_int64, c_int64, c_void_p, c_void_p]
    lib.pq_swiglu_hadamard_quant_act.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int32, c_int64, c_void_p,
                                                 c_void_p, c_void_p]
    lib.pq_kv4_append_decode_attn.argtypes = [c_void_p, POINTER(KV4CacheStruct), c_void_p, c_void_p, c_void_p, c_void_p, c_float,
                                              c_void_p, c_size_t, c_void_p]
    for name in EXPORTS:
        getattr(lib, name)
        if name not in ("pq_status_string", "pq_w4a4_gemm_workspace_bytes", "pq_decode_attn_workspace_bytes"):
            getattr(lib, name).restype = c_int32
    _lib = lib
    return lib


def _ptr(t):
    return c_void_p(t.data_ptr()) if t is not None else c_void_p(0)


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _ok(status: int, where: str):
    if status != 0:
        raise PQError(status, where)


def _dev(t: torch.Tensor, dtype, name: str):
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError(f"{name} must be a CUDA tensor of dtype {dtype}")
    return t


class KV4Cache:
    """Caller-owned buffers of one layer's KV cache: fp16 prefix region + packed INT4 region."""

    def __init__(self, prefix_k, prefix_v, kq, vq, s_k, s_v, length, Hq: int, sk_tok=None, sv_tok=None):
        """Static setting: s_k, s_v [Hkv]. Group-wise dynamic setting: sk_tok, sv_tok f32 [B, Hkv, Tmax] (s_k, s_v may be None)."""
        B, Hkv, Tmax, D2 = kq.shape
        self.prefix_k, self.prefix_v, self.kq, self.vq = prefix_k, prefix_v, kq, vq
        self.s_k, self.s_v, self.length, self.sk_tok, self.sv_tok = s_k, s_v, length, sk_tok, sv_tok
        _dev(kq, torch.uint8, "kq"), _dev(vq, torch.uint8, "vq"), _dev(length, torch.int32, "length")
        if sk_tok is not None:
            _dev(sk_tok, torch.float32, "sk_tok"), _dev(sv_tok, torch.float32, "sv_tok")
            assert sk_tok.shape == (B, Hkv, Tmax) == sv_tok.shape and sk_tok.is_contiguous() and sv_tok.is_contiguous()
        else:
            _dev(s_k, torch.float32, "s_k"), _dev(s_v, torch.float32, "s_v")
        n_prefix = 0 if prefix_k is None else prefix_k.shape[1]
        if n_prefix:
            _dev(prefix_k, torch.float16, "prefix_k"), _dev(prefix_v, torch.float16, "prefix_v")
            assert prefix_k.is_contiguous() and prefix_v.is_contiguous()
        assert kq.is_contiguous() and vq.is_contiguous() and vq.shape == kq.shape
        self.B, self.Hq, self.Hkv, self.D, self.n_prefix, self.Tmax = B, Hq, Hkv, D2 * 2, n_prefix, Tmax
        self.struct = KV4CacheStruct(
            prefix_k.data_ptr() if n_prefix else 0, prefix_v.data_ptr() if n_prefix else 0, kq.data_ptr(), vq.data_ptr(),
            s_k.data_ptr() if s_k is not None else 0, s_v.data_ptr() if s_v is not None else 0, length.data_ptr(), B, Hq, Hkv, D2 * 2,
            n_prefix, Tmax, sk_tok.data_ptr() if sk_tok is not None else 0, sv_tok.data_ptr() if sv_tok is not None else 0,
        )


class Context:
    """Owns one pq_ctx on the current CUDA device."""

    def __init__(self):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2410_05265_b200 needs a CUDA device (sm_100a); there is no CPU path")
        torch.cuda.init()
        torch.empty(1, device="cuda")  # make sure the primary context exists
        h = c_void_p()
        _ok(self.lib.pq_create(ctypes.byref(h)), "pq_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.pq_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check(self):
        """Synchronizes the current stream and raises if a kernel reported an error."""
        _ok(self.lib.pq_check(self.h, _stream()), "pq_check")

    def check_status(self) -> int:
        return int(self.lib.pq_check(self.h, _stream()))

    def set_wait_limit(self, sm_clocks: int) -> None:
        """Bound of the device-side waits of later launches, in SM clocks (0: the default of about a second)."""
        _ok(self.lib.pq_set_wait_limit(self.h, int(sm_clocks)), "pq_set_wait_limit")

    def selftest_wait(self) -> torch.Tensor:
        """Launches a wait that nothing satisfies (bounded by the context's limit); returns the clocks it took (int64 [1])."""
        waited = torch.zeros(1, dtype=torch.int64, device="cuda")
        _ok(self.lib.pq_selftest_wait(self.h, _ptr(waited), _stream()), "pq_selftest_wait")
        return waited

    def probe_i8_mma(self, iters: int = 4096, n_ctas: int | None = None) -> torch.Tensor:
        """SM clocks each of n_ctas CTAs needed for `iters` resident-operand 128x256x32 kind::i8 MMAs (int64 [n_ctas])."""
        n = n_ctas or torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
        cycles = torch.zeros(n, dtype=torch.int64, device="cuda")
        _ok(self.lib.pq_probe_i8_mma(self.h, int(iters), _ptr(cycles), n, _stream()), "pq_probe_i8_mma")
        return cycles

    # ---- offline -----------------------------------------------------------------------------
    def quant_weights(self, W: torch.Tensor, out=None):
        _dev(W, torch.bfloat16, "W")
        N, K = W.shape
        assert W.stride(1) == 1
        if out is None:
            wq = torch.empty((N, K // 2), dtype=torch.uint8, device=W.device)
            s_w = torch.empty((N,), dtype=torch.float32, device=W.device)
        else:
            wq, s_w = out
            _dev(wq, torch.uint8, "wq"), _dev(s_w, torch.float32, "s_w")
            assert wq.shape == (N, K // 2) and wq.is_contiguous() and s_w.shape == (N,)
        _ok(self.lib.pq_quant_weights(self.h, _ptr(W), N, K, W.stride(0), _ptr(wq), _ptr(s_w), _stream()), "pq_quant_weights")
        return wq, s_w

    def calib_act_scale(self, x: torch.Tensor, had_block: int, row_begin: int = 0, s_a: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x")
        M, K = x.shape
        if s_a is None:
            s_a = torch.zeros((1,), dtype=torch.float32, device=x.device)
        _ok(self.lib.pq_calib_act_scale(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_a), _stream()),
            "pq_calib_act_scale")
        return s_a

    # ---- hot path ------------------------------------------------------------------------------
    def hadamard_quant_act(self, x: torch.Tensor, had_block: int, s_a: torch.Tensor, row_begin: int = 0,
                           out: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x"), _dev(s_a, torch.float32, "s_a")
        M, K = x.shape
        assert x.stride(1) == 1
        if out is None:
            out = torch.zeros((M, K // 2), dtype=torch.uint8, device=x.device)
        _ok(self.lib.pq_hadamard_quant_act(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_a), _ptr(out),
                                           _stream()), "pq_hadamard_quant_act")
        return out

    def swiglu_hadamard_quant_act(self, gate: torch.Tensor, up: torch.Tensor, had_block: int, s_a: torch.Tensor, row_begin: int = 0,
                                  out: torch.Tensor | None = None):
        """pq_silu_mul followed by pq_hadamard_quant_act in one launch; gate and up are the halves of a gate|up output."""
        _dev(gate, torch.bfloat16, "gate"), _dev(up, torch.bfloat16, "up"), _dev(s_a, torch.float32, "s_a")
        M, K = gate.shape
        assert up.shape == (M, K) and gate.stride(1) == 1 and up.stride(1) == 1 and gate.stride(0) == up.stride(0)
        if out is None:
            out = torch.zeros((M, K // 2), dtype=torch.uint8, device=gate.device)
        _ok(self.lib.pq_swiglu_hadamard_quant_act(self.h, _ptr(gate), _ptr(up), M, K, gate.stride(0), had_block, row_begin, _ptr(s_a),
                                                  _ptr(out), _stream()), "pq_swiglu_hadamard_quant_act")
        return out

    def w4a4_gemm(self, xq: torch.Tensor, wq: torch.Tensor, s_a: torch.Tensor, s_w: torch.Tensor, row_begin: int = 0,
                  out: torch.Tensor | None = None, acc_dbg: torch.Tensor | None = None):
        _dev(xq, torch.uint8, "xq"), _dev(wq, torch.uint8, "wq")
        _dev(s_a, torch.float32, "s_a"), _dev(s_w, torch.float32, "s_w")
        M, K2 = xq.shape
        N = wq.shape[0]
        assert wq.shape[1] == K2 and xq.is_contiguous() and wq.is_contiguous()
        if out is None:
            out = torch.zeros((M, N), dtype=torch.bfloat16, device=xq.device)
        if acc_dbg is not None:
            _dev(acc_dbg, torch.int32, "acc_dbg")
            assert acc_dbg.shape == (M, N) and acc_dbg.is_contiguous()
        _ok(self.lib.pq_w4a4_gemm(self.h, _ptr(xq), _ptr(wq), _ptr(s_a), _ptr(s_w), _ptr(out), out.stride(0), M, N, K2 * 2,
                                  row_begin, _ptr(acc_dbg), c_void_p(0), 0, _stream()), "pq_w4a4_gemm")
        return out

    def rmsnorm_hadamard_quant_act(self, x: torch.Tensor, g: torch.Tensor, eps: float, s_a: torch.Tensor, row_begin: int = 0,
                                   out: torch.Tensor | None = None):
        """RMSNorm, rotation over the whole row and static quantizer in one launch (K a power of two up to 8192)."""
        _dev(x, torch.bfloat16, "x"), _dev(g, torch.bfloat16, "g"), _dev(s_a, torch.float32, "s_a")
        M, K = x.shape
        assert x.stride(1) == 1 and g.numel() == K
        if out is None:
            out = torch.zeros((M, K // 2), dtype=torch.uint8, device=x.device)
        _ok(self.lib.pq_rmsnorm_hadamard_quant_act(self.h, _ptr(x), M, K, x.stride(0), _ptr(g), float(eps), row_begin, _ptr(s_a),
                                                   _ptr(out), _stream()), "pq_rmsnorm_hadamard_quant_act")
        return out

    # ---- Eq. 1 as printed: asymmetric activation quantizer with a zero point ---------------------------
    def calib_act_asym(self, x: torch.Tensor, had_block: int, row_begin: int = 0):
        """Returns device scalars (s_a f32, z_a int32) from the range of the rotated rows >= row_begin."""
        _dev(x, torch.bfloat16, "x")
        M, K = x.shape
        s_a = torch.zeros((1,), dtype=torch.float32, device=x.device)
        z_a = torch.zeros((1,), dtype=torch.int32, device=x.device)
        _ok(self.lib.pq_calib_act_asym(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_a), _ptr(z_a), _stream()),
            "pq_calib_act_asym")
        return s_a, z_a

    def grid_search_act_asym(self, x: torch.Tensor, had_block: int, n_grid: int, lo: float, row_begin: int = 0):
        """MSE grid search for the static (s, z). Returns device tensors s_a [1], z_a [1], cand_s [n^2], cand_z [n^2], sse [n^2]."""
        _dev(x, torch.bfloat16, "x")
        M, K = x.shape
        n2 = max(1, n_grid * n_grid)
        s_a = torch.zeros((1,), dtype=torch.float32, device=x.device)
        z_a = torch.zeros((1,), dtype=torch.int32, device=x.device)
        cand_s = torch.zeros((n2,), dtype=torch.float32, device=x.device)
        cand_z = torch.zeros((n2,), dtype=torch.int32, device=x.device)
        sse = torch.zeros((n2,), dtype=torch.float64, device=x.device)
        _ok(self.lib.pq_grid_search_act_asym(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, int(n_grid), float(lo), _ptr(s_a),
                                             _ptr(z_a), _ptr(cand_s), _ptr(cand_z), _ptr(sse), _stream()), "pq_grid_search_act_asym")
        return s_a, z_a, cand_s, cand_z, sse

    def grid_search_clip_dyn(self, x: torch.Tensor, had_block: int, n_grid: int, lo: float, row_begin: int = 0):
        """MSE grid search for the clipping factor shared by the tokens of per-token dynamic quantization. Returns device
        tensors gamma [1], s_tok [M] (unclipped steps), cand [n], sse [n]."""
        _dev(x, torch.bfloat16, "x")
        M, K = x.shape
        n = max(1, n_grid)
        gamma = torch.zeros((1,), dtype=torch.float32, device=x.device)
        s_tok = torch.zeros((M,), dtype=torch.float32, device=x.device)
        cand = torch.zeros((n,), dtype=torch.float32, device=x.device)
        sse = torch.zeros((n,), dtype=torch.float64, device=x.device)
        _ok(self.lib.pq_grid_search_clip_dyn(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, int(n_grid), float(lo), _ptr(gamma),
                                             _ptr(s_tok), _ptr(cand), _ptr(sse), _stream()), "pq_grid_search_clip_dyn")
        return gamma, s_tok, cand, sse

    def hadamard_quant_act_asym(self, x: torch.Tensor, had_block: int, s_a: torch.Tensor, z_a: torch.Tensor, row_begin: int = 0,
                                out: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x"), _dev(s_a, torch.float32, "s_a"), _dev(z_a, torch.int32, "z_a")
        M, K = x.shape
        assert x.stride(1) == 1
        if out is None:
            out = torch.zeros((M, K // 2), dtype=torch.uint8, device=x.device)
        _ok(self.lib.pq_hadamard_quant_act_asym(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_a), _ptr(z_a),
                                                _ptr(out), _stream()), "pq_hadamard_quant_act_asym")
        return out

    def weight_code_sums(self, wq: torch.Tensor) -> torch.Tensor:
        _dev(wq, torch.uint8, "wq")
        N, K2 = wq.shape
        assert wq.is_contiguous()
        wsum = torch.empty((N,), dtype=torch.int32, device=wq.device)
        _ok(self.lib.pq_weight_code_sums(self.h, _ptr(wq), N, K2 * 2, _ptr(wsum), _stream()), "pq_weight_code_sums")
        return wsum

    def w4a4_gemm_asym(self, xq: torch.Tensor, wq: torch.Tensor, s_a: torch.Tensor, z_a: torch.Tensor, s_w: torch.Tensor,
                       wsum: torch.Tensor, row_begin: int = 0, out: torch.Tensor | None = None, acc_dbg: torch.Tensor | None = None):
        _dev(xq, torch.uint8, "xq"), _dev(wq, torch.uint8, "wq"), _dev(z_a, torch.int32, "z_a"), _dev(wsum, torch.int32, "wsum")
        _dev(s_a, torch.float32, "s_a"), _dev(s_w, torch.float32, "s_w")
        M, K2 = xq.shape
        N = wq.shape[0]
        assert wq.shape[1] == K2 and xq.is_contiguous() and wq.is_contiguous() and wsum.shape == (N,)
        if out is None:
            out = torch.zeros((M, N), dtype=torch.bfloat16, device=xq.device)
        if acc_dbg is not None:
            _dev(acc_dbg, torch.int32, "acc_dbg")
            assert acc_dbg.shape == (M, N) and acc_dbg.is_contiguous()
        _ok(self.lib.pq_w4a4_gemm_asym(self.h, _ptr(xq), _ptr(wq), _ptr(s_a), _ptr(z_a), _ptr(s_w), _ptr(wsum), _ptr(out),
                                       out.stride(0), M, N, K2 * 2, row_begin, _ptr(acc_dbg), _stream()), "pq_w4a4_gemm_asym")
        return out

    # ---- offline analysis: outlier tokens (Sec. 4.1, Eq. 2) -------------------------------------------
    def outlier_tokens(self, x: torch.Tensor, eta1: float = 64.0, eta2: float = 8.0):
        """Returns (M, R, flags, median) for x bf16 [T, C]: token maxima, outlier degrees, 1/2/0 flags."""
        _dev(x, torch.bfloat16, "x")
        T, C = x.shape
        assert x.stride(1) == 1
        M = torch.empty((T,), dtype=torch.float32, device=x.device)
        R = torch.empty_like(M)
        flags = torch.empty((T,), dtype=torch.int32, device=x.device)
        med = torch.empty((1,), dtype=torch.float32, device=x.device)
        _ok(self.lib.pq_outlier_tokens(self.h, _ptr(x), T, C, x.stride(0), float(eta1), float(eta2), _ptr(M), _ptr(R), _ptr(flags),
                                       _ptr(med), _stream()), "pq_outlier_tokens")
        return M, R, flags, med

    # ---- per-token dynamic activations (Table 1, O1) ---------------------------------------------------
    def dyn_act_scale(self, x: torch.Tensor, had_block: int, clip: float = 1.0, row_begin: int = 0, out: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x")
        M, K = x.shape
        if out is None:
            out = torch.zeros((M,), dtype=torch.float32, device=x.device)
        _dev(out, torch.float32, "out")
        _ok(self.lib.pq_dyn_act_scale(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, float(clip), _ptr(out), _stream()),
            "pq_dyn_act_scale")
        return out

    def dyn_hadamard_quant_act(self, x: torch.Tensor, had_block: int, clip: float = 1.0, row_begin: int = 0,
                               s_tok: torch.Tensor | None = None, out: torch.Tensor | None = None):
        """pq_dyn_act_scale followed by pq_hadamard_quant_act_rows in one call; returns (s_tok, xq)."""
        _dev(x, torch.bfloat16, "x")
        M, K = x.shape
        assert x.stride(1) == 1
        if s_tok is None:
            s_tok = torch.zeros((M,), dtype=torch.float32, device=x.device)
        if out is None:
            out = torch.zeros((M, K // 2), dtype=torch.uint8, device=x.device)
        _dev(s_tok, torch.float32, "s_tok"), _dev(out, torch.uint8, "out")
        _ok(self.lib.pq_dyn_hadamard_quant_act(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, float(clip), _ptr(s_tok),
                                               _ptr(out), _stream()), "pq_dyn_hadamard_quant_act")
        return s_tok, out

    def hadamard_quant_act_rows(self, x: torch.Tensor, had_block: int, s_tok: torch.Tensor, row_begin: int = 0,
                                out: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x"), _dev(s_tok, torch.float32, "s_tok")
        M, K = x.shape
        assert x.stride(1) == 1 and s_tok.shape == (M,) and s_tok.is_contiguous()
        if out is None:
            out = torch.zeros((M, K // 2), dtype=torch.uint8, device=x.device)
        _ok(self.lib.pq_hadamard_quant_act_rows(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_tok), _ptr(out),
                                                _stream()), "pq_hadamard_quant_act_rows")
        return out

    def w4a4_gemm_rows(self, xq: torch.Tensor, wq: torch.Tensor, s_tok: torch.Tensor, s_w: torch.Tensor, row_begin: int = 0,
                       out: torch.Tensor | None = None, acc_dbg: torch.Tensor | None = None):
        _dev(xq, torch.uint8, "xq"), _dev(wq, torch.uint8, "wq")
        _dev(s_tok, torch.float32, "s_tok"), _dev(s_w, torch.float32, "s_w")
        M, K2 = xq.shape
        N = wq.shape[0]
        assert wq.shape[1] == K2 and xq.is_contiguous() and wq.is_contiguous() and s_tok.shape == (M,) and s_tok.is_contiguous()
        if out is None:
            out = torch.zeros((M, N), dtype=torch.bfloat16, device=xq.device)
        if acc_dbg is not None:
            _dev(acc_dbg, torch.int32, "acc_dbg")
            assert acc_dbg.shape == (M, N) and acc_dbg.is_contiguous()
        _ok(self.lib.pq_w4a4_gemm_rows(self.h, _ptr(xq), _ptr(wq), _ptr(s_tok), _ptr(s_w), _ptr(out), out.stride(0), M, N, K2 * 2,
                                       row_begin, _ptr(acc_dbg), _stream()), "pq_w4a4_gemm_rows")
        return out

    # ---- W4A8: 8-bit activation codes, one signed byte per element (Sec. 5.1) -------------------------
    def calib_act_scale8(self, x: torch.Tensor, had_block: int, row_begin: int = 0, s_a: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x")
        M, K = x.shape
        if s_a is None:
            s_a = torch.zeros((1,), dtype=torch.float32, device=x.device)
        _ok(self.lib.pq_calib_act_scale8(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_a), _stream()),
            "pq_calib_act_scale8")
        return s_a

    def hadamard_quant_act8(self, x: torch.Tensor, had_block: int, s_a: torch.Tensor, row_begin: int = 0,
                            out: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x"), _dev(s_a, torch.float32, "s_a")
        M, K = x.shape
        assert x.stride(1) == 1
        if out is None:
            out = torch.zeros((M, K), dtype=torch.int8, device=x.device)
        _dev(out, torch.int8, "out")
        _ok(self.lib.pq_hadamard_quant_act8(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_a), _ptr(out),
                                            _stream()), "pq_hadamard_quant_act8")
        return out

    def hadamard_quant_act_c8(self, x: torch.Tensor, had_block: int, s_a: torch.Tensor, row_begin: int = 0,
                              out: torch.Tensor | None = None):
        """The 4-bit codes of hadamard_quant_act, one per byte (operand of w4a8_gemm)."""
        _dev(x, torch.bfloat16, "x"), _dev(s_a, torch.float32, "s_a")
        M, K = x.shape
        assert x.stride(1) == 1
        if out is None:
            out = torch.zeros((M, K), dtype=torch.int8, device=x.device)
        _dev(out, torch.int8, "out")
        _ok(self.lib.pq_hadamard_quant_act_c8(self.h, _ptr(x), M, K, x.stride(0), had_block, row_begin, _ptr(s_a), _ptr(out),
                                              _stream()), "pq_hadamard_quant_act_c8")
        return out

    def w4a8_gemm(self, xq8: torch.Tensor, wq: torch.Tensor, s_a: torch.Tensor, s_w: torch.Tensor, row_begin: int = 0,
                  out: torch.Tensor | None = None, acc_dbg: torch.Tensor | None = None):
        _dev(xq8, torch.int8, "xq8"), _dev(wq, torch.uint8, "wq")
        _dev(s_a, torch.float32, "s_a"), _dev(s_w, torch.float32, "s_w")
        M, K = xq8.shape
        N = wq.shape[0]
        assert wq.shape[1] * 2 == K and xq8.is_contiguous() and wq.is_contiguous()
        if out is None:
            out = torch.zeros((M, N), dtype=torch.bfloat16, device=xq8.device)
        if acc_dbg is not None:
            _dev(acc_dbg, torch.int32, "acc_dbg")
            assert acc_dbg.shape == (M, N) and acc_dbg.is_contiguous()
        _ok(self.lib.pq_w4a8_gemm(self.h, _ptr(xq8), _ptr(wq), _ptr(s_a), _ptr(s_w), _ptr(out), out.stride(0), M, N, K,
                                  row_begin, _ptr(acc_dbg), _stream()), "pq_w4a8_gemm")
        return out

    def kv4_append(self, cache: KV4Cache, k: torch.Tensor, v: torch.Tensor):
        _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v")
        B, T_new, Hkv, D = k.shape
        assert (B, Hkv, D) == (cache.B, cache.Hkv, cache.D) and v.shape == k.shape
        if k.is_contiguous() and v.is_contiguous():
            _ok(self.lib.pq_kv4_append(self.h, ctypes.byref(cache.struct), _ptr(k), _ptr(v), T_new, _stream()), "pq_kv4_append")
            return
        # column slices of a wider matrix (the k and v parts of a q|k|v projection output)
        ld = k.stride(1)
        for t in (k, v):
            assert t.stride(3) == 1 and t.stride(2) == D and t.stride(1) == ld and (B == 1 or t.stride(0) == T_new * ld)
        _ok(self.lib.pq_kv4_append_strided(self.h, ctypes.byref(cache.struct), _ptr(k), _ptr(v), T_new, ld, _stream()),
            "pq_kv4_append_strided")

    def calib_kv_scale(self, x: torch.Tensor, s: torch.Tensor | None = None) -> torch.Tensor:
        """x bf16 [n_tok, Hkv, D] (token stride free): folds max|x|/7 per head into s (created as zeros)."""
        _dev(x, torch.bfloat16, "x")
        n_tok, Hkv, D = x.shape
        assert x.stride(2) == 1 and x.stride(1) == D
        if s is None:
            s = torch.zeros((Hkv,), dtype=torch.float32, device=x.device)
        _ok(self.lib.pq_calib_kv_scale(self.h, _ptr(x), n_tok, Hkv, D, x.stride(0), _ptr(s), _stream()), "pq_calib_kv_scale")
        return s

    def decode_attn_workspace(self, cache: KV4Cache) -> torch.Tensor:
        n = int(self.lib.pq_decode_attn_workspace_bytes(ctypes.byref(cache.struct)))
        return torch.empty((max(n, 16),), dtype=torch.uint8, device=cache.kq.device)

    def decode_attn(self, cache: KV4Cache, q: torch.Tensor, sm_scale: float, ws: torch.Tensor,
                    out: torch.Tensor | None = None):
        _dev(q, torch.bfloat16, "q")
        assert q.shape == (cache.B, cache.Hq, cache.D) and q.is_contiguous()
        if out is None:
            out = torch.empty_like(q)
        _ok(self.lib.pq_decode_attn_kv4_prefix(self.h, ctypes.byref(cache.struct), _ptr(q), _ptr(out), float(sm_scale),
                                               _ptr(ws), ws.numel(), _stream()), "pq_decode_attn_kv4_prefix")
        return out

    def kv4_append_decode_attn(self, cache: KV4Cache, k: torch.Tensor, v: torch.Tensor, q: torch.Tensor, sm_scale: float,
                               ws: torch.Tensor, out: torch.Tensor | None = None):
        """kv4_append of one token per sequence and decode_attn in one launch (k, v bf16 [B, 1, Hkv, D], dense)."""
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v")
        assert q.shape == (cache.B, cache.Hq, cache.D) and q.is_contiguous()
        assert k.shape == (cache.B, 1, cache.Hkv, cache.D) and v.shape == k.shape and k.is_contiguous() and v.is_contiguous()
        if out is None:
            out = torch.empty_like(q)
        _ok(self.lib.pq_kv4_append_decode_attn(self.h, ctypes.byref(cache.struct), _ptr(k), _ptr(v), _ptr(q), _ptr(out),
                                               float(sm_scale), _ptr(ws), ws.numel(), _stream()), "pq_kv4_append_decode_attn")
        return out


    def prefill_attn(self, cache: KV4Cache, seq: int, q: torch.Tensor, sm_scale: float, out: torch.Tensor | None = None):
        _dev(q, torch.bfloat16, "q")
        T = q.shape[0]
        assert q.shape == (T, cache.Hq, cache.D) and q.stride(2) == 1 and q.stride(1) == cache.D
        if out is None:
            out = torch.empty((T, cache.Hq, cache.D), dtype=q.dtype, device=q.device)
        assert out.is_contiguous()
        _ok(self.lib.pq_prefill_attn_kv4_prefix(self.h, ctypes.byref(cache.struct), int(seq), _ptr(q), q.stride(0), T, _ptr(out),
                                                float(sm_scale), _stream()), "pq_prefill_attn_kv4_prefix")
        return out

    def rope_kv4_append(self, cache: KV4Cache, seq: int, qkv: torch.Tensor, pos0: int, theta: float, rotate: bool = False):
        """Rotary embedding (+ R3) of the q and k heads of qkv [T, (Hq + 2 Hkv) * D] in place and KV4 append of k, v."""
        _dev(qkv, torch.bfloat16, "qkv")
        T = qkv.shape[0]
        assert qkv.dim() == 2 and qkv.stride(1) == 1 and qkv.shape[1] == (cache.Hq + 2 * cache.Hkv) * cache.D
        _ok(self.lib.pq_rope_kv4_append(self.h, ctypes.byref(cache.struct), int(seq), _ptr(qkv), T, qkv.stride(0), int(pos0), float(theta),
                                        1 if rotate else 0, _stream()), "pq_rope_kv4_append")

    # ---- transformer-block glue -----------------------------------------------------------------
    def rmsnorm(self, x: torch.Tensor, g: torch.Tensor, eps: float = 1e-5, out: torch.Tensor | None = None):
        _dev(x, torch.bfloat16, "x"), _dev(g, torch.bfloat16, "g")
        M, K = x.shape
        assert x.stride(1) == 1 and g.numel() == K
        if out is None:
            out = torch.empty((M, K), dtype=torch.bfloat16, device=x.device)
        _ok(self.lib.pq_rmsnorm(self.h, _ptr(x), M, K, x.stride(0), _ptr(g), float(eps), _ptr(out), out.stride(0),
                                _stream()), "pq_rmsnorm")
        return out

    def rope(self, x: torch.Tensor, pos0: int, theta: float, out: torch.Tensor | None = None, rotate: bool = False):
        """Rotary embedding of x [T, H, D]; with rotate=True followed by the head-wise Hadamard rotation R3."""
        _dev(x, torch.bfloat16, "x")
        T, H, D = x.shape
        assert x.stride(2) == 1 and x.stride(1) == D
        if out is None:
            out = torch.empty((T, H, D), dtype=x.dtype, device=x.device)
        assert out.stride() == x.stride() or (out.is_contiguous() and x.is_contiguous())
        fn, name = (self.lib.pq_rope_rotate, "pq_rope_rotate") if rotate else (self.lib.pq_rope, "pq_rope")
        _ok(fn(self.h, _ptr(x), T, H, D, x.stride(0), int(pos0), float(theta), _ptr(out), _stream()), name)
        return out

    def silu_mul(self, gate: torch.Tensor, up: torch.Tensor, out: torch.Tensor | None = None):
        _dev(gate, torch.bfloat16, "gate"), _dev(up, torch.bfloat16, "up")
        M, F = gate.shape
        assert up.shape == (M, F) and gate.stride(1) == 1 and up.stride(1) == 1 and gate.stride(0) == up.stride(0)
        if out is None:
            out = torch.empty((M, F), dtype=torch.bfloat16, device=gate.device)
        _ok(self.lib.pq_silu_mul(self.h, _ptr(gate), _ptr(up), M, F, gate.stride(0), _ptr(out), out.stride(0), _stream()),
            "pq_silu_mul")
        return out

    def residual_add(self, a: torch.Tensor, b: torch.Tensor, out: torch.Tensor | None = None):
        _dev(a, torch.bfloat16, "a"), _dev(b, torch.bfloat16, "b")
        assert a.shape == b.shape and a.is_contiguous() and b.is_contiguous()
        if out is None:
            out = torch.empty_like(a)
        _ok(self.lib.pq_residual_add(self.h, _ptr(a), _ptr(b), _ptr(out), a.numel(), _stream()), "pq_residual_add")
        return out


def decode_attn_noalloc(cache: KV4Cache, q: torch.Tensor, sm_scale: float, out: torch.Tensor) -> torch.Tensor:
    """Decode attention through the entry point that allocates nothing: no Context and no
    workspace are involved, the library's built-in scratch array is used instead. It exists for
    callers that are handed buffers but may not allocate device memory themselves; `out` must
    therefore be supplied. Calls on one device must not overlap on the GPU (they share the array).
    The first call on a device should come before any CUDA-graph capture."""
    _dev(q, torch.bfloat16, "q"), _dev(out, torch.bfloat16, "out")
    assert q.shape == (cache.B, cache.Hq, cache.D) and q.is_contiguous() and out.shape == q.shape and out.is_contiguous()
    _ok(load_library().pq_decode_attn_kv4_prefix_noalloc(ctypes.byref(cache.struct), _ptr(q), _ptr(out), float(sm_scale),
                                                       _stream()), "pq_decode_attn_kv4_prefix_noalloc")
    return out
