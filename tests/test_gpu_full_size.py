"""Parity at the full benchmark sizes, in the launch configuration bench.py times, on sampled outputs
that the CPU oracle computes one by one (rows of a GEMM, rows of the rotation, single queries of the
attention). Integer results bit-exact, floating-point results within the tolerances of helpers.py."""
import math

import numpy as np
import pytest
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs
from helpers import assert_attn_close, assert_bf16_close, assert_codes_tie_tolerant, bf16_ulp, to_np

pytestmark = pytest.mark.gpu

N_PREFIX = 4


@pytest.fixture(scope="module")
def ctx():
    from paper_2410_05265_b200 import binding

    c = binding.Context()
    yield c
    c.check()
    c.close()


def _sample_rows(M, n, seed):
    rng = np.random.default_rng(seed)
    rows = np.unique(np.concatenate([[N_PREFIX, M - 1, 127 + N_PREFIX, 128 + N_PREFIX, 255, 256], rng.integers(N_PREFIX, M, n)]))
    return rows[rows < M]


@pytest.mark.parametrize("name,N,K", [("q|k|v", 6144, 4096), ("gate|up", 28672, 4096), ("down", 4096, 14336)])
def test_gemm_llama8b_prefill_2048_sampled_rows(ctx, name, N, K):
    M = 2048
    g = torch.Generator(device="cuda").manual_seed(N + K)
    xq = torch.randint(0, 256, (M, K // 2), dtype=torch.uint8, device="cuda", generator=g)
    wq = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device="cuda", generator=g)
    s_a = torch.tensor([0.0173], device="cuda")
    s_w = torch.rand(N, device="cuda", generator=g) * 0.004 + 0.001
    acc = torch.full((M, N), -77, dtype=torch.int32, device="cuda")
    out = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    ctx.w4a4_gemm(xq, wq, s_a, s_w, N_PREFIX, out=out, acc_dbg=acc)
    ctx.check()
    assert int(acc[:N_PREFIX].min()) == int(acc[:N_PREFIX].max()) == -77 and float(out[:N_PREFIX].float().min()) == 3.0
    rows = _sample_rows(M, 10, seed=N)
    acc_ref = orc.gemm_i4(to_np(xq[rows]), to_np(wq))
    assert np.array_equal(to_np(acc[rows]), acc_ref), "sampled accumulator rows must be bit-exact"
    assert_bf16_close(inputs.bits(out[rows]), orc.dequant_bf16(acc_ref, np.float32(0.0173), to_np(s_w)), f"gemm {name}")
    # the launch without the debug dump (the one bench.py times) writes the same bf16 output
    out2 = torch.full_like(out, 3.0)
    ctx.w4a4_gemm(xq, wq, s_a, s_w, N_PREFIX, out=out2)
    ctx.check()
    assert torch.equal(out2, out)


@pytest.mark.parametrize("K,B", [(4096, 4096), (14336, 2048)])
def test_hadamard_quant_llama8b_prefill_2048_sampled_rows(ctx, K, B):
    M = 2048
    x = inputs.activations(M, K, seed=0, n_prefix=N_PREFIX, device="cuda")
    cal = inputs.activations(M, K, seed=1, n_prefix=N_PREFIX, device="cuda")
    s_gpu = ctx.calib_act_scale(cal, B, N_PREFIX)
    rows = _sample_rows(M, 10, seed=K)
    # the scale is a maximum over all rows: the oracle's maximum over a row sample can only be smaller
    s_part = orc.calib_act_scale(inputs.bits(cal[torch.from_numpy(rows).cuda()].cpu()), B, 0)
    assert float(s_part) <= float(s_gpu) * (1 + 2e-6)
    out = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.hadamard_quant_act(x, B, s_gpu, N_PREFIX, out=out)
    ctx.check()
    assert bool((out[:N_PREFIX] == 0x5A).all())
    xr = x[torch.from_numpy(rows).cuda()].cpu()
    ref, tie = orc.quant_act(inputs.bits(xr), B, np.float32(float(s_gpu)), 0, want_tie_dist=True)
    n = assert_codes_tie_tolerant(to_np(out)[rows], ref, tie, "hadamard_quant_act full size")
    assert n <= max(2, int(2e-4 * ref.size * 2))


def test_decode_attention_config3_sampled_queries(ctx):
    from paper_2410_05265_b200 import binding

    B, Hq, Hkv, D, P, T, Tmax = 8, 32, 8, 128, 4, 4092, 4096
    g = torch.Generator(device="cuda").manual_seed(7)
    kq = torch.randint(0, 256, (B, Hkv, Tmax, D // 2), dtype=torch.uint8, device="cuda", generator=g)
    vq = torch.randint(0, 256, (B, Hkv, Tmax, D // 2), dtype=torch.uint8, device="cuda", generator=g)
    pk, pv = inputs.prefix_kv(Hkv, P, D, 0, "k", 50.0), inputs.prefix_kv(Hkv, P, D, 0, "v", 50.0)
    s_k = np.full(Hkv, 4.5 / 7, np.float32)
    s_v = np.linspace(0.4, 0.8, Hkv).astype(np.float32)
    q = inputs.queries(B, Hq, D, 0)
    length = np.array([T, T - 1, 4000, 64, T, 1, 2049, T], np.int32)
    cache = binding.KV4Cache(pk.cuda(), pv.cuda(), kq, vq, torch.from_numpy(s_k).cuda(), torch.from_numpy(s_v).cuda(),
                             torch.from_numpy(length).cuda(), Hq)
    out = ctx.decode_attn(cache, q.cuda(), 1 / math.sqrt(D), ctx.decode_attn_workspace(cache))
    ctx.check()
    _, ref = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), to_np(kq), to_np(vq), s_k, s_v, length,
                             1 / math.sqrt(D), want_f64=True)
    assert_attn_close(inputs.bits(out), ref, "decode attention, prefix magnitude 50")
    # with the prefix out of the way the INT4 region decides the result
    cache0 = binding.KV4Cache(None, None, kq, vq, torch.from_numpy(s_k).cuda(), torch.from_numpy(s_v).cuda(),
                              torch.from_numpy(length).cuda(), Hq)
    out0 = ctx.decode_attn(cache0, q.cuda(), 1 / math.sqrt(D), ctx.decode_attn_workspace(cache0))
    ctx.check()
    z = np.zeros((Hkv, 0, D), np.uint16)
    _, ref0 = orc.decode_attn(inputs.bits(q), z, z, to_np(kq), to_np(vq), s_k, s_v, length, 1 / math.sqrt(D), want_f64=True)
    assert_attn_close(inputs.bits(out0), ref0, "decode attention, no prefix")


def test_prefill_attention_llama70b_4096_sampled_queries(ctx):
    """configs[4] attention shape: 4096 tokens, 64 query / 8 KV heads. Sampled query tokens are checked
    against the oracle's single-query attention over the keys 0..t they may see."""
    from paper_2410_05265_b200 import binding

    T, Hq, Hkv, D, P = 4096, 64, 8, 128, 4
    g = torch.Generator(device="cuda").manual_seed(11)
    kq = torch.randint(0, 256, (1, Hkv, T, D // 2), dtype=torch.uint8, device="cuda", generator=g)
    vq = torch.randint(0, 256, (1, Hkv, T, D // 2), dtype=torch.uint8, device="cuda", generator=g)
    pk, pv = inputs.prefix_kv(Hkv, P, D, 0, "k", 2.0), inputs.prefix_kv(Hkv, P, D, 0, "v", 2.0)
    s_k = np.full(Hkv, 0.3 / 7, np.float32)  # small steps keep the softmax from collapsing onto one key
    s_v = np.linspace(0.4, 0.8, Hkv).astype(np.float32)
    q = inputs.kv_tensor(1, T, Hq, D, 3, "k")[0].contiguous()
    cache = binding.KV4Cache(pk.cuda(), pv.cuda(), kq, vq, torch.from_numpy(s_k).cuda(), torch.from_numpy(s_v).cuda(),
                             torch.full((1,), T, dtype=torch.int32, device="cuda"), Hq)
    out = ctx.prefill_attn(cache, 0, q.cuda(), 1 / math.sqrt(D))
    ctx.check()
    toks = np.array([0, 1, 15, 16, 63, 64, 65, 1000, 2047, 2048, 4094, 4095])
    # the oracle's decode attention with len = t + 1 is the causal row t
    kq_h, vq_h = to_np(kq), to_np(vq)
    n = len(toks)
    kq_b = np.broadcast_to(kq_h, (n, Hkv, T, D // 2))
    vq_b = np.broadcast_to(vq_h, (n, Hkv, T, D // 2))
    _, ref = orc.decode_attn(inputs.bits(q[toks]), inputs.bits(pk), inputs.bits(pv), np.ascontiguousarray(kq_b),
                             np.ascontiguousarray(vq_b), s_k, s_v, (toks + 1).astype(np.int32), 1 / math.sqrt(D), want_f64=True)
    assert_attn_close(inputs.bits(out[toks]), ref, "prefill attention, sampled tokens")


def test_gemm_llama70b_prefill_4096_sampled_rows(ctx):
    """The long-K kernel (token operand in tensor memory) at the configs[4] down-projection shape."""
    M, N, K = 4096, 8192, 28672
    g = torch.Generator(device="cuda").manual_seed(5)
    xq = torch.randint(0, 256, (M, K // 2), dtype=torch.uint8, device="cuda", generator=g)
    wq = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device="cuda", generator=g)
    s_a, s_w = torch.tensor([0.01], device="cuda"), torch.full((N,), 0.002, device="cuda")
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    out = ctx.w4a4_gemm(xq, wq, s_a, s_w, acc_dbg=acc)
    ctx.check()
    rows = np.array([0, 127, 128, 255, 256, 2049, 4095])
    acc_ref = orc.gemm_i4(to_np(xq[rows]), to_np(wq))
    assert np.array_equal(to_np(acc[rows]), acc_ref)
    assert_bf16_close(inputs.bits(out[rows]), orc.dequant_bf16(acc_ref, np.float32(0.01), to_np(s_w)), "gemm 70B down")


def test_block_llama70b_4096_staged_sampled_rows():
    """configs[4] at full width (hidden 8192, 64 / 8 heads, FFN 28672, 4096 tokens after 4 prefixed ones): every stage
    of the block against the oracle applied to the GPU's own input of that stage, on sampled token rows; then the
    untapped pass (fused RMSNorm, rotary + append and SwiGLU launches) must reproduce the tapped one bit for bit."""
    from paper_2410_05265_b200 import binding, block

    ctx = binding.Context()
    c = inputs.LLAMA3_70B
    T, P, D = 4096, N_PREFIX, c["head_dim"]
    Hq, Hkv = c["n_q_heads"], c["n_kv_heads"]
    shape = block.BlockShape(hidden=c["hidden"], n_q_heads=Hq, n_kv_heads=Hkv, ffn=c["ffn"])
    qd, kvd, hidden, ffn = shape.q_dim, shape.kv_dim, shape.hidden, shape.ffn
    dev = "cuda"
    W = dict(qkv=inputs.weights(qd + 2 * kvd, hidden, seed=2, device=dev), o=inputs.weights(hidden, qd, seed=3, device=dev),
             gu=inputs.weights(2 * ffn, hidden, seed=4, device=dev), d=inputs.weights(hidden, ffn, seed=5, device=dev))
    g1 = torch.ones(hidden, dtype=torch.bfloat16, device=dev)
    pk, pv = inputs.prefix_kv(Hkv, P, D, 0, "k", 50.0), inputs.prefix_kv(Hkv, P, D, 0, "v", 50.0)
    blk = block.Block(ctx, shape, W["qkv"], W["o"], W["gu"], W["d"], g1, g1, pk.cuda(), pv.cuda(), t_max=T)
    blk.forward(inputs.activations(T, hidden, seed=1, device=dev), calibrate=True)
    x = inputs.activations(T, hidden, seed=0, device=dev)
    taps = {}
    y = blk.forward(x, tap=lambda name, t: taps.__setitem__(name, t.detach().clone()))
    ctx.check()
    s_a = [float(s.item()) for s in blk.s_a]
    s_k, s_v = to_np(blk.s_k), to_np(blk.s_v)
    rows = np.array([0, 1, 127, 128, 255, 256, 2047, 2048, 4095])
    ridx = torch.from_numpy(rows).cuda()
    rb = lambda t: inputs.bits(t[ridx].contiguous())           # sampled rows of a device tensor as bf16 bit patterns
    had = [shape.had_block(hidden), shape.had_block(qd), shape.had_block(hidden), shape.had_block(ffn)]

    def check_quant(name, src, blockw, s):
        ref, tie = orc.quant_act(rb(src), blockw, np.float32(s), 0, want_tie_dist=True)
        n = assert_codes_tie_tolerant(to_np(taps[name][ridx]), ref, tie, name)
        assert n <= max(2, int(2e-4 * ref.size * 2))

    def check_gemm(name, xq_name, wname, wq, sw, s):
        # weights: sampled output channels of the offline quantizer bit for bit, then the GEMM on the GPU's own codes
        ch = torch.tensor([0, 1, 255, 256, wq.shape[0] - 1], device=dev)
        wq_ref, sw_ref = orc.quant_weights(inputs.bits(W[wname][ch].contiguous()))
        assert np.array_equal(to_np(wq[ch]), wq_ref) and np.array_equal(to_np(sw[ch]), sw_ref)
        acc = orc.gemm_i4(to_np(taps[xq_name][ridx]), to_np(wq))
        assert_bf16_close(rb(taps[name]), orc.dequant_bf16(acc, np.float32(s), to_np(sw)), name)

    assert_bf16_close(rb(taps["h1"]), orc.rmsnorm(rb(x), inputs.bits(g1)), "rmsnorm 1")
    check_quant("xq1", taps["h1"], had[0], s_a[0])
    check_gemm("qkv", "xq1", "qkv", blk.wq_qkv, blk.sw_qkv, s_a[0])
    # rotary embedding at positions P + t, one sampled token at a time (the oracle takes a start position)
    for t in rows[[0, 3, 8]]:
        qk = taps["qkv"][t: t + 1, : qd + kvd].reshape(1, Hq + Hkv, D).contiguous()
        got = taps["qkv_rope"][t: t + 1, : qd + kvd].reshape(1, Hq + Hkv, D).contiguous()
        assert_bf16_close(inputs.bits(got), orc.rope(inputs.bits(qk), P + int(t), 500000.0), "rope")
    assert torch.equal(taps["qkv_rope"][:, qd + kvd:], taps["qkv"][:, qd + kvd:])
    # KV4 append of all 4096 tokens (the multi-CTA path): sampled tokens as a batch of one-token sequences
    n = len(rows)
    k_s = taps["qkv_rope"][ridx, qd: qd + kvd].reshape(n, 1, Hkv, D).contiguous()
    v_s = taps["qkv_rope"][ridx, qd + kvd:].reshape(n, 1, Hkv, D).contiguous()
    kq_ref, vq_ref = np.zeros((n, Hkv, 1, D // 2), np.uint8), np.zeros((n, Hkv, 1, D // 2), np.uint8)
    assert orc.kv4_append(inputs.bits(k_s), inputs.bits(v_s), s_k, s_v, kq_ref, vq_ref, np.zeros(n, np.int32)) == 0
    assert np.array_equal(to_np(taps["kq"][0][:, ridx]).transpose(1, 0, 2), kq_ref[:, :, 0])
    assert np.array_equal(to_np(taps["vq"][0][:, ridx]).transpose(1, 0, 2), vq_ref[:, :, 0])
    assert int(blk.length[0]) == T
    # causal attention of sampled tokens over the GPU's own cache
    toks = rows[[0, 2, 3, 6, 8]]
    q_s = taps["qkv_rope"][torch.from_numpy(toks).cuda(), :qd].reshape(len(toks), Hq, D).contiguous()
    kq_b = np.ascontiguousarray(np.broadcast_to(to_np(taps["kq"]), (len(toks), Hkv, T, D // 2)))
    vq_b = np.ascontiguousarray(np.broadcast_to(to_np(taps["vq"]), (len(toks), Hkv, T, D // 2)))
    _, ref = orc.decode_attn(inputs.bits(q_s), inputs.bits(pk), inputs.bits(pv), kq_b, vq_b, s_k, s_v, (toks + 1).astype(np.int32),
                             1 / math.sqrt(D), want_f64=True)
    assert_attn_close(inputs.bits(taps["attn"][torch.from_numpy(toks).cuda()].contiguous()), ref, "prefill attention in the block")
    check_quant("xq2", taps["attn"].reshape(T, qd), had[1], s_a[1])
    check_gemm("o", "xq2", "o", blk.wq_o, blk.sw_o, s_a[1])
    assert np.array_equal(rb(taps["x2"]), orc.add(rb(x), rb(taps["o"])))
    assert_bf16_close(rb(taps["h2"]), orc.rmsnorm(rb(taps["x2"]), inputs.bits(g1)), "rmsnorm 2")
    check_quant("xq3", taps["h2"], had[2], s_a[2])
    check_gemm("gu", "xq3", "gu", blk.wq_gu, blk.sw_gu, s_a[2])
    gu = taps["gu"][ridx]
    assert_bf16_close(rb(taps["act"]), orc.silu_mul(inputs.bits(gu[:, :ffn].contiguous()), inputs.bits(gu[:, ffn:].contiguous())), "silu_mul")
    check_quant("xq4", taps["act"], had[3], s_a[3])           # the 14-block rotation of the 28672-wide input
    check_gemm("d", "xq4", "d", blk.wq_down, blk.sw_down, s_a[3])
    assert np.array_equal(rb(taps["y"]), orc.add(rb(taps["x2"]), rb(taps["d"])))
    # the pass bench.py times (no taps: fused launches) gives the same bits, twice
    want = taps["y"]
    taps.clear()
    for _ in range(2):
        assert torch.equal(blk.forward(x), want)
    ctx.check()
    ctx.close()
