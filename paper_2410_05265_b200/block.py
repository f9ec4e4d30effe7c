"""A W4A4KV4 Llama transformer block at prefill as a fixed sequence of library calls.

Nothing is computed here: the class owns the device buffers of one block (packed weights, static
scales, the KV cache with its full-precision prefix) and issues the C-ABI calls in the order of the
block in App. B of the paper: [RMSNorm + rotate + quantize, one launch] -> q|k|v GEMM -> [rotary embedding
(optionally followed by the head-wise rotation R3 of q and k) + KV4 append, one launch] -> causal attention over
[prefix || INT4 cache] -> [rotate + quantize] -> o GEMM -> residual -> [RMSNorm + rotate + quantize] -> gate|up
GEMM -> [SwiGLU + block rotate + quantize, one launch] -> down GEMM -> residual. When every stage is looked at
(tap) or calibrated, the fused launches are replaced by the calls they stand for, which give the same bits. The tokens that enter are ordinary tokens: the prefixed outlier tokens are
never run through the quantized path, their K/V sit in the cache in fp16 (Sec. 4.2).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

from . import binding


@dataclass
class BlockShape:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    ffn: int
    head_dim: int = 128
    rope_theta: float = 500000.0
    eps: float = 1e-5
    r3: bool = False  # online head-wise Hadamard rotation of q and k after RoPE (App. B, R3)

    @property
    def q_dim(self):
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self):
        return self.n_kv_heads * self.head_dim

    def had_block(self, width: int) -> int:
        """Rotation width of a linear input: the whole width when it is a power of two, else 2048."""
        return width if width & (width - 1) == 0 else 2048


class Block:
    """Device state of one block. Weights are bf16 [out, in]; q|k|v and gate|up are concatenated along
    the output dimension so that each pair of logical layers is one GEMM."""

    def __init__(self, ctx: binding.Context, shape: BlockShape, w_qkv, w_o, w_gate_up, w_down, g_attn, g_mlp, prefix_k,
                 prefix_v, t_max: int):
        self.ctx, self.shape = ctx, shape
        dev = w_qkv.device
        self.wq_qkv, self.sw_qkv = ctx.quant_weights(w_qkv)
        self.wq_o, self.sw_o = ctx.quant_weights(w_o)
        self.wq_gu, self.sw_gu = ctx.quant_weights(w_gate_up)
        self.wq_down, self.sw_down = ctx.quant_weights(w_down)
        self.g_attn, self.g_mlp = g_attn, g_mlp
        self.prefix_k, self.prefix_v = prefix_k, prefix_v
        self.n_prefix = 0 if prefix_k is None else prefix_k.shape[1]
        self.t_max = t_max
        # static scales, filled by calibrate()
        self.s_a = [torch.zeros(1, device=dev) for _ in range(4)]
        self.s_k = torch.zeros(shape.n_kv_heads, device=dev)
        self.s_v = torch.zeros(shape.n_kv_heads, device=dev)
        self.kq = torch.zeros((1, shape.n_kv_heads, t_max, shape.head_dim // 2), dtype=torch.uint8, device=dev)
        self.vq = torch.zeros_like(self.kq)
        self.length = torch.zeros(1, dtype=torch.int32, device=dev)
        self.cache = None
        self.buf = {}

    def _cache(self):
        if self.cache is None:
            self.cache = binding.KV4Cache(self.prefix_k, self.prefix_v, self.kq, self.vq, self.s_k, self.s_v, self.length,
                                          self.shape.n_q_heads)
        return self.cache

    def _buffers(self, T: int, dev):
        s = self.shape
        if self.buf.get("T") != T:
            z = lambda *sh, dt=torch.bfloat16: torch.empty(sh, dtype=dt, device=dev)
            self.buf = dict(
                T=T, h=z(T, s.hidden), xq_h=z(T, s.hidden // 2, dt=torch.uint8), qkv=z(T, s.q_dim + 2 * s.kv_dim),
                attn=z(T, s.n_q_heads, s.head_dim), xq_a=z(T, s.q_dim // 2, dt=torch.uint8), o=z(T, s.hidden),
                x2=z(T, s.hidden), gu=z(T, 2 * s.ffn), act=z(T, s.ffn), xq_f=z(T, s.ffn // 2, dt=torch.uint8),
                d=z(T, s.hidden), y=z(T, s.hidden))
        return self.buf

    def forward(self, x: torch.Tensor, calibrate: bool = False, tap=None) -> torch.Tensor:
        """x bf16 [T, hidden]: T ordinary tokens at positions n_prefix .. n_prefix + T - 1 of one sequence.
        With calibrate=True the same pass folds max|.|/7 of every quantizer input into the static scales
        before using them (a calibration batch; call it once with seed-1 data before timing anything).
        `tap(name, tensor)`, if given, is called after every stage with its output (buffers are reused
        later in the block, so a test that wants to look at one has to copy it there)."""
        staged = tap is not None  # a caller that looks at every stage gets the SwiGLU output as a tensor of its own
        tap = tap or (lambda name, t: None)
        ctx, s, T = self.ctx, self.shape, x.shape[0]
        b = self._buffers(T, x.device)
        self.length.zero_()
        fused_norm = not (calibrate or staged) and s.hidden & (s.hidden - 1) == 0 and 128 <= s.hidden <= 8192
        if fused_norm:  # RMSNorm inside the rotate+quantize launch: same bits, the normalised tensor stays on chip
            ctx.rmsnorm_hadamard_quant_act(x, self.g_attn, s.eps, self.s_a[0], out=b["xq_h"])
        else:
            ctx.rmsnorm(x, self.g_attn, s.eps, out=b["h"])
            tap("h1", b["h"])
            if calibrate:
                ctx.calib_act_scale(b["h"], s.had_block(s.hidden), 0, s_a=self.s_a[0])
            ctx.hadamard_quant_act(b["h"], s.had_block(s.hidden), self.s_a[0], out=b["xq_h"])
        tap("xq1", b["xq_h"])
        ctx.w4a4_gemm(b["xq_h"], self.wq_qkv, self.s_a[0], self.sw_qkv, out=b["qkv"])
        tap("qkv", b["qkv"])
        q = b["qkv"][:, : s.q_dim].unflatten(1, (s.n_q_heads, s.head_dim))
        k = b["qkv"][:, s.q_dim: s.q_dim + s.kv_dim].unflatten(1, (s.n_kv_heads, s.head_dim))
        v = b["qkv"][:, s.q_dim + s.kv_dim:].unflatten(1, (s.n_kv_heads, s.head_dim))
        cache = self._cache()
        if calibrate or staged:
            qk = b["qkv"][:, : s.q_dim + s.kv_dim].unflatten(1, (s.n_q_heads + s.n_kv_heads, s.head_dim))
            ctx.rope(qk, self.n_prefix, s.rope_theta, out=qk, rotate=s.r3)
            tap("qkv_rope", b["qkv"])
            if calibrate:
                ctx.calib_kv_scale(k, self.s_k)
                ctx.calib_kv_scale(v, self.s_v)
            ctx.kv4_append(cache, k.unsqueeze(0), v.unsqueeze(0))
        else:  # rotary embedding (+ R3) and the KV4 append in one launch: same bits
            ctx.rope_kv4_append(cache, 0, b["qkv"], self.n_prefix, s.rope_theta, rotate=s.r3)
        tap("kq", self.kq)
        tap("vq", self.vq)
        ctx.prefill_attn(cache, 0, q, 1.0 / math.sqrt(s.head_dim), out=b["attn"])
        tap("attn", b["attn"])
        attn2d = b["attn"].view(T, s.q_dim)
        if calibrate:
            ctx.calib_act_scale(attn2d, s.had_block(s.q_dim), 0, s_a=self.s_a[1])
        ctx.hadamard_quant_act(attn2d, s.had_block(s.q_dim), self.s_a[1], out=b["xq_a"])
        tap("xq2", b["xq_a"])
        ctx.w4a4_gemm(b["xq_a"], self.wq_o, self.s_a[1], self.sw_o, out=b["o"])
        tap("o", b["o"])
        ctx.residual_add(x, b["o"], out=b["x2"])
        tap("x2", b["x2"])
        if fused_norm:
            ctx.rmsnorm_hadamard_quant_act(b["x2"], self.g_mlp, s.eps, self.s_a[2], out=b["xq_h"])
        else:
            ctx.rmsnorm(b["x2"], self.g_mlp, s.eps, out=b["h"])
            tap("h2", b["h"])
            if calibrate:
                ctx.calib_act_scale(b["h"], s.had_block(s.hidden), 0, s_a=self.s_a[2])
            ctx.hadamard_quant_act(b["h"], s.had_block(s.hidden), self.s_a[2], out=b["xq_h"])
        tap("xq3", b["xq_h"])
        ctx.w4a4_gemm(b["xq_h"], self.wq_gu, self.s_a[2], self.sw_gu, out=b["gu"])
        tap("gu", b["gu"])
        if calibrate or staged:
            ctx.silu_mul(b["gu"][:, : s.ffn], b["gu"][:, s.ffn:], out=b["act"])
            tap("act", b["act"])
            if calibrate:
                ctx.calib_act_scale(b["act"], s.had_block(s.ffn), 0, s_a=self.s_a[3])
            ctx.hadamard_quant_act(b["act"], s.had_block(s.ffn), self.s_a[3], out=b["xq_f"])
        else:  # the SwiGLU is formed inside the rotation kernel: same bits, the activation tensor stays on chip
            ctx.swiglu_hadamard_quant_act(b["gu"][:, : s.ffn], b["gu"][:, s.ffn:], s.had_block(s.ffn), self.s_a[3], out=b["xq_f"])
        tap("xq4", b["xq_f"])
        ctx.w4a4_gemm(b["xq_f"], self.wq_down, self.s_a[3], self.sw_down, out=b["d"])
        tap("d", b["d"])
        ctx.residual_add(b["x2"], b["d"], out=b["y"])
        tap("y", b["y"])
        return b["y"]

    LAUNCHES_PER_FORWARD = 12  # 16 when every stage is tapped (RMSNorm, rotary embedding and SwiGLU then are launches of their own)
