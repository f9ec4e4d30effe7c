"""The allocation-free decode-attention entry point against the regular one.

Some users of the library run where they cannot allocate device memory (no allocator handed to
them, or allocation forbidden at that point of their program), so they can build neither a
context nor a workspace. For them the library carries its own fixed scratch array. This test
drives that entry point through the C ABI, twice in a row on different inputs (the array keeps
the first call's contents, which must not leak into the second), and compares each result with
the regular entry point on the same inputs. Collected last on purpose.
"""
import math

import numpy as np
import pytest
import torch

from helpers import assert_attn_close, to_np
from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs

pytestmark = pytest.mark.gpu


def _cache(binding, B, Hq, Hkv, P, T, Tmax, seed):
    D = 128
    g = torch.Generator(device="cuda").manual_seed(seed)
    kq = torch.randint(0, 256, (B, Hkv, Tmax, D // 2), dtype=torch.uint8, device="cuda", generator=g)
    vq = torch.randint(0, 256, (B, Hkv, Tmax, D // 2), dtype=torch.uint8, device="cuda", generator=g)
    s_k = torch.full((Hkv,), 0.61, device="cuda")
    s_v = torch.full((Hkv,), 0.57, device="cuda")
    length = torch.tensor([T - 3 * b for b in range(B)], dtype=torch.int32, device="cuda")
    pk = inputs.prefix_kv(Hkv, P, D, seed, "k", 1.0, device="cuda")
    pv = inputs.prefix_kv(Hkv, P, D, seed, "v", 1.0, device="cuda")
    q = inputs.queries(B, Hq, D, seed, device="cuda")
    return binding.KV4Cache(pk, pv, kq, vq, s_k, s_v, length, Hq), q


def test_noalloc_entry_point_matches_regular_one_twice_in_a_row():
    from paper_2410_05265_b200 import binding

    sm = 1 / math.sqrt(128)
    # the last two cases: one (sequence, head) pair with a long cache = 32 splits merged through the array,
    # with a long and with a short sequence in it
    cases = [(_cache(binding, 4, 32, 8, 4, 700, 768, seed=3)), (_cache(binding, 2, 16, 2, 2, 333, 512, seed=4)),
             (_cache(binding, 1, 8, 1, 3, 8000, 8192, seed=5)), (_cache(binding, 1, 4, 1, 0, 200, 8192, seed=6))]
    # the new entry point first: it must work in a process that never created a context
    outs = []
    for cache, q in cases:
        out = torch.full_like(q, 7.0)
        binding.decode_attn_noalloc(cache, q, sm, out)
        outs.append(out)
    torch.cuda.synchronize()
    ctx = binding.Context()
    for (cache, q), out in zip(cases, outs):
        ref = ctx.decode_attn(cache, q, sm, ctx.decode_attn_workspace(cache))
        ctx.check()
        ref64 = orc.bf16_to_f64(inputs.bits(ref))
        assert_attn_close(inputs.bits(out), ref64, "noalloc vs regular entry point")
        # and against the CPU oracle's unrounded result, like every other attention test
        _, orc64 = orc.decode_attn(inputs.bits(q), inputs.bits(cache.prefix_k), inputs.bits(cache.prefix_v), to_np(cache.kq),
                                   to_np(cache.vq), to_np(cache.s_k), to_np(cache.s_v), to_np(cache.length), sm, want_f64=True)
        assert_attn_close(inputs.bits(out), orc64, "noalloc vs oracle")
        # and a repeat of the same call reproduces itself (nothing of the previous call survives)
        again = torch.empty_like(out)
        binding.decode_attn_noalloc(cache, q, sm, again)
        torch.cuda.synchronize()
        assert torch.equal(again, out)
    ctx.close()


def test_noalloc_entry_point_rejects_sizes_beyond_its_array():
    from paper_2410_05265_b200 import binding

    D, B, Hkv = 128, 4100, 1   # B * Hkv above the 4096 the built-in array is sized for
    kq = torch.zeros((B, Hkv, 64, D // 2), dtype=torch.uint8, device="cuda")
    s = torch.ones(Hkv, device="cuda")
    cache = binding.KV4Cache(None, None, kq, kq, s, s, torch.zeros(B, dtype=torch.int32, device="cuda"), 1)
    q = torch.zeros((B, 1, D), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.PQError) as e:
        binding.decode_attn_noalloc(cache, q, 0.1, torch.empty_like(q))
    assert e.value.status == 4  # PQ_ERR_WORKSPACE
