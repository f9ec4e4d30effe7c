"""Failure detection on the device: every wait inside a kernel is bounded, and a wait that runs out is reported
through the status word while the kernel winds down in order (copies in flight awaited, tensor memory released).
Nothing is made to fault or hang: a self-test kernel waits, with a short bound, on a barrier nothing completes; and
the bound of the real kernels is lowered to a few clocks, so that an ordinary first wait (for a copy that needs a
microsecond) may legitimately run out. Whether it does depends on how long one hardware try_wait suspends, so each
such call may report a timeout or succeed; either way the same context, with the default bound back, must then give
exact results."""
import math

import numpy as np
import pytest
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs
from helpers import assert_attn_close, rand_codes, to_np

pytestmark = pytest.mark.gpu
PQ_ERR_TIMEOUT = 6


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_selftest_wait_runs_out_after_the_limit_and_is_reported():
    from paper_2410_05265_b200 import binding

    ctx = binding.Context()
    ctx.set_wait_limit(200_000)                 # a tenth of a millisecond
    waited = ctx.selftest_wait()
    assert ctx.check_status() == PQ_ERR_TIMEOUT
    assert 200_000 < int(waited) < 50_000_000, "the wait ends soon after its bound"
    assert ctx.check_status() == 0
    ctx.set_wait_limit(0)
    x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    ctx.hadamard_quant_act(x, 128, torch.ones(1, device="cuda"))
    assert ctx.check_status() == 0              # the context works on
    ctx.close()


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    from paper_2410_05265_b200 import binding

    ctx = binding.Context()
    rng = np.random.default_rng(0)
    D = 128
    # operands of a one-tile GEMM with short K (token operand in shared memory) and with long K (in tensor memory)
    gemms = []
    for M, N, K in [(128, 256, 512), (128, 256, 32768)]:
        xq, wq = rand_codes(rng, M, K), rand_codes(rng, N, K)
        gemms.append((dev(xq), dev(wq), orc.gemm_i4(xq, wq)))
    s_a, s_w = torch.full((1,), 0.02, device="cuda"), torch.full((256,), 0.003, device="cuda")
    # a small KV4 cache for the decode and the prefill attention
    B, Hq, Hkv, T, Tmax, P = 2, 8, 2, 300, 320, 4
    kq_np, vq_np = rng.integers(0, 256, (B, Hkv, Tmax, D // 2)).astype(np.uint8), rng.integers(0, 256, (B, Hkv, Tmax, D // 2)).astype(np.uint8)
    s_k, s_v = np.full(Hkv, 0.3, np.float32), np.full(Hkv, 0.5, np.float32)
    pk, pv = inputs.prefix_kv(Hkv, P, D, 0, "k", 1.0), inputs.prefix_kv(Hkv, P, D, 0, "v", 1.0)
    length = np.full(B, T, np.int32)
    cache = binding.KV4Cache(pk.cuda(), pv.cuda(), dev(kq_np), dev(vq_np), dev(s_k), dev(s_v), dev(length), Hq)
    q = inputs.queries(B, Hq, D, 0)
    qp = inputs.kv_tensor(1, T, Hq, D, 3, "k")[0].contiguous()
    ws = ctx.decode_attn_workspace(cache)
    sm = 1 / math.sqrt(D)

    ctx.set_wait_limit(16)                      # a few clocks: no copy from memory is that fast
    seen = []
    for xq, wq, _ in gemms:
        ctx.w4a4_gemm(xq, wq, s_a, s_w)
        seen.append(ctx.check_status())
        assert ctx.check_status() == 0          # reading the status word clears it
    ctx.decode_attn(cache, q.cuda(), sm, ws)
    seen.append(ctx.check_status())
    ctx.prefill_attn(cache, 1, qp.cuda(), sm)
    seen.append(ctx.check_status())
    torch.cuda.synchronize()                    # the process and the CUDA context are alive
    assert all(st in (0, PQ_ERR_TIMEOUT) for st in seen), seen
    print("statuses under a 16-clock bound (GEMM short K, GEMM long K, decode attention, prefill attention):", seen)

    ctx.set_wait_limit(0)                       # the default bound again: exact results from the same context
    for xq, wq, acc_ref in gemms:
        acc = torch.zeros(acc_ref.shape, dtype=torch.int32, device="cuda")
        ctx.w4a4_gemm(xq, wq, s_a, s_w, acc_dbg=acc)
        assert ctx.check_status() == 0 and np.array_equal(to_np(acc), acc_ref)
    out = ctx.decode_attn(cache, q.cuda(), sm, ws)
    assert ctx.check_status() == 0
    _, ref = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_np, vq_np, s_k, s_v, length, sm, want_f64=True)
    assert_attn_close(inputs.bits(out), ref, "decode attention after a timed-out call")
    outp = ctx.prefill_attn(cache, 1, qp.cuda(), sm)
    assert ctx.check_status() == 0
    _, refp = orc.prefill_attn(inputs.bits(qp), inputs.bits(pk), inputs.bits(pv), kq_np[1], vq_np[1], s_k, s_v, sm, want_f64=True)
    assert_attn_close(inputs.bits(outp), refp, "prefill attention after a timed-out call")
    ctx.close()
