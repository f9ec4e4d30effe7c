"""GPU parity of the group-wise dynamic KV4 setting (Table 1, O1; group size 128 = one (token, head) vector) against
the CPU oracle, through the C ABI: per-vector steps and codes of the append bit for bit, decode and causal prefill
attention with per-key steps within the attention tolerance."""
import math

import numpy as np
import pytest
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs
from helpers import assert_attn_close, to_np

pytestmark = pytest.mark.gpu
D = 128


@pytest.fixture(scope="module")
def ctx():
    from paper_2410_05265_b200 import binding

    c = binding.Context()
    yield c
    c.check()
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _scaled_kv(B, T, Hkv, seed, which):
    """K or V whose vectors differ in magnitude by orders of magnitude: per-vector steps matter."""
    x = inputs.kv_tensor(B, T, Hkv, D, seed, which).float()
    mag = torch.exp2(torch.arange(B * T * Hkv).reshape(B, T, Hkv, 1) % 7 - 3.0)
    return (x * mag).to(torch.bfloat16)


def _setup(ctx, B, Hq, Hkv, P, T, Tmax, start):
    from paper_2410_05265_b200 import binding

    k, v = _scaled_kv(B, T, Hkv, 0, "k"), _scaled_kv(B, T, Hkv, 0, "v")
    if T > 2:
        k[0, 1, 0] = 0                                   # an all-zero vector: step 1, codes 0
    start = np.asarray(start, np.int32)
    kq_ref = np.full((B, Hkv, Tmax, D // 2), 0x11, np.uint8)
    vq_ref = np.full_like(kq_ref, 0x11)
    sk_ref, sv_ref = np.full((B, Hkv, Tmax), 0.5, np.float32), np.full((B, Hkv, Tmax), 0.5, np.float32)
    len_ref = start.copy()
    assert orc.kv4_append_dyn(inputs.bits(k), inputs.bits(v), kq_ref, vq_ref, sk_ref, sv_ref, len_ref) == 0
    kq = torch.full((B, Hkv, Tmax, D // 2), 0x11, dtype=torch.uint8, device="cuda")
    vq = torch.full_like(kq, 0x11)
    sk = torch.full((B, Hkv, Tmax), 0.5, device="cuda")
    sv = torch.full((B, Hkv, Tmax), 0.5, device="cuda")
    pk = inputs.prefix_kv(Hkv, max(P, 1), D, 0, "k", 1.0)[:, :P].contiguous()
    pv = inputs.prefix_kv(Hkv, max(P, 1), D, 0, "v", 1.0)[:, :P].contiguous()
    cache = binding.KV4Cache(pk.cuda() if P else None, pv.cuda() if P else None, kq, vq, None, None, dev(start), Hq, sk_tok=sk, sv_tok=sv)
    ctx.kv4_append(cache, k.cuda(), v.cuda())
    ctx.check()
    assert np.array_equal(to_np(cache.length), len_ref)
    assert np.array_equal(to_np(sk), sk_ref) and np.array_equal(to_np(sv), sv_ref), "per-vector steps must match bit for bit"
    assert np.array_equal(to_np(kq), kq_ref) and np.array_equal(to_np(vq), vq_ref), "codes must match bit for bit"
    return cache, pk, pv, kq_ref, vq_ref, sk_ref, sv_ref, len_ref


@pytest.mark.parametrize("B,Hq,Hkv,P,T,Tmax,start", [
    (1, 4, 1, 0, 16, 16, [0]), (2, 8, 2, 2, 100, 128, [0, 17]), (3, 32, 8, 4, 333, 400, [0, 5, 60]),
    (2, 16, 2, 4, 1000, 1024, [24, 0]), (1, 8, 8, 1, 5, 64, [0]), (8, 32, 8, 4, 2000, 2048, [0] * 8),
])
def test_dynamic_kv_append_and_decode_attention(ctx, B, Hq, Hkv, P, T, Tmax, start):
    cache, pk, pv, kq_ref, vq_ref, sk_ref, sv_ref, len_ref = _setup(ctx, B, Hq, Hkv, P, T, Tmax, start)
    q = inputs.queries(B, Hq, D, 0)
    sm = 1 / math.sqrt(D)
    _, ref = orc.decode_attn_dyn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_ref, vq_ref, sk_ref, sv_ref, len_ref, sm)
    ws = ctx.decode_attn_workspace(cache)
    out = ctx.decode_attn(cache, q.cuda(), sm, ws)
    ctx.check()
    assert_attn_close(inputs.bits(out), ref, f"dynamic-KV decode attention B{B} Hq{Hq} T{T} P{P}")
    assert torch.equal(out, ctx.decode_attn(cache, q.cuda(), sm, ws)), "a second call reproduces the first"
    # steps matter here: the static per-head reading of the same codes is far off
    _, wrong = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_ref, vq_ref, sk_ref[0, :, 0].copy(), sv_ref[0, :, 0].copy(),
                               len_ref, sm, want_f64=True)
    if T > 16:
        assert np.abs(wrong - ref).max() > 0.05 * np.abs(ref).max()


@pytest.mark.parametrize("T,Hq,Hkv,P", [(1, 8, 1, 4), (37, 8, 2, 4), (150, 4, 1, 0), (300, 16, 2, 3), (130, 2, 2, 64)])
def test_dynamic_kv_prefill_attention(ctx, T, Hq, Hkv, P):
    B, Tmax = 2, T + 11
    cache, pk, pv, kq_ref, vq_ref, sk_ref, sv_ref, _ = _setup(ctx, B, Hq, Hkv, P, T, Tmax, [0, 0])
    q = inputs.kv_tensor(1, T, Hq, D, 3, "k")[0].contiguous()
    sm = 1 / math.sqrt(D)
    _, ref = orc.prefill_attn_dyn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_ref[1], vq_ref[1], sk_ref[1], sv_ref[1], sm)
    out = ctx.prefill_attn(cache, 1, q.cuda(), sm)
    ctx.check()
    assert_attn_close(inputs.bits(out), ref, f"dynamic-KV prefill attention T{T} Hq{Hq} Hkv{Hkv} P{P}")


def test_dynamic_kv_refuses_overflow_and_the_static_only_calls(ctx):
    from paper_2410_05265_b200 import binding

    B, Hkv, Tmax = 2, 2, 8
    k = inputs.kv_tensor(B, 3, Hkv, D, 0, "k").cuda()
    kq = torch.zeros((B, Hkv, Tmax, D // 2), dtype=torch.uint8, device="cuda")
    sk = torch.zeros((B, Hkv, Tmax), device="cuda")
    length = torch.tensor([2, 6], dtype=torch.int32, device="cuda")
    cache = binding.KV4Cache(None, None, kq, torch.zeros_like(kq), None, None, length, 4, sk_tok=sk, sv_tok=torch.zeros_like(sk))
    ctx.kv4_append(cache, k, k)
    assert ctx.check_status() == 2 and length.tolist() == [2, 6] and int(kq.sum()) == 0 and float(sk.sum()) == 0.0
    q = torch.zeros((B, 4, D), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.PQError) as e:
        k1 = k[:, :1].contiguous()
        ctx.kv4_append_decode_attn(cache, k1, k1, q, 0.1, ctx.decode_attn_workspace(cache))
    assert e.value.status == 7  # PQ_ERR_UNSUPPORTED
    with pytest.raises(binding.PQError) as e:
        binding.decode_attn_noalloc(cache, q, 0.1, torch.empty_like(q))
    assert e.value.status == 7
