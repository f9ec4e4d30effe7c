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
