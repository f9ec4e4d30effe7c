"""GPU parity of the full W4A4KV4 transformer block (the Llama-3-70B-shaped config at reduced width):
every stage of the block is checked against the CPU oracle applied to the GPU's own input of that
stage, so one stage's rounding differences never hide another's; the chained output is then compared
loosely with the oracle chained end to end."""
import math

import numpy as np
import pytest
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs
from helpers import assert_attn_close, assert_bf16_close, assert_codes_tie_tolerant, to_np

pytestmark = pytest.mark.gpu


def _bits(t):
    return inputs.bits(t.detach().cpu().contiguous())


@pytest.mark.parametrize("T,hidden,Hq,Hkv,ffn,P,r3", [(40, 512, 4, 2, 6144, 4, False), (19, 256, 8, 1, 1024, 0, False),
                                                      (40, 512, 4, 2, 6144, 4, True)])
def test_block_stages_match_oracle(T, hidden, Hq, Hkv, ffn, P, r3):
    from paper_2410_05265_b200 import binding, block

    ctx = binding.Context()
    D = 128
    shape = block.BlockShape(hidden=hidden, n_q_heads=Hq, n_kv_heads=Hkv, ffn=ffn, r3=r3)
    qd, kvd = Hq * D, Hkv * D
    w_qkv = inputs.weights(qd + 2 * kvd, hidden, seed=2, std=0.05)
    w_o = inputs.weights(hidden, qd, seed=3, std=0.05)
    w_gu = inputs.weights(2 * ffn, hidden, seed=4, std=0.05)
    w_d = inputs.weights(hidden, ffn, seed=5, std=0.05)
    g1 = torch.ones(hidden, dtype=torch.bfloat16)
    g2 = torch.ones(hidden, dtype=torch.bfloat16)
    pk = inputs.prefix_kv(Hkv, P, D, 0, "k", 5.0) if P else None
    pv = inputs.prefix_kv(Hkv, P, D, 0, "v", 5.0) if P else None
    blk = block.Block(ctx, shape, w_qkv.cuda(), w_o.cuda(), w_gu.cuda(), w_d.cuda(), g1.cuda(), g2.cuda(),
                      pk.cuda() if P else None, pv.cuda() if P else None, t_max=T + 5)
    x_cal = inputs.activations(T, hidden, seed=1)
    x = inputs.activations(T, hidden, seed=0)
    blk.forward(x_cal.cuda(), calibrate=True)
    taps = {}
    y = blk.forward(x.cuda(), tap=lambda name, t: taps.__setitem__(name, t.detach().clone().cpu()))
    ctx.check()
    s_a = [float(s.item()) for s in blk.s_a]
    s_k, s_v = to_np(blk.s_k), to_np(blk.s_v)
    assert all(v > 0 for v in s_a) and (s_k > 0).all() and (s_v > 0).all()
    B = [shape.had_block(hidden), shape.had_block(qd), shape.had_block(hidden), shape.had_block(ffn)]

    def check_quant(name, src_bits, blockw, s):
        ref, tie = orc.quant_act(src_bits, blockw, np.float32(s), 0, want_tie_dist=True)
        n = assert_codes_tie_tolerant(to_np(taps[name]), ref, tie, name)
        assert n <= max(2, int(2e-4 * src_bits.size))

    def check_gemm(name, xq_name, w_bits, s):
        wq, sw = orc.quant_weights(w_bits)
        acc = orc.gemm_i4(to_np(taps[xq_name]), wq)
        assert_bf16_close(inputs.bits(taps[name]), orc.dequant_bf16(acc, np.float32(s), sw), name)

    # attention half
    assert_bf16_close(inputs.bits(taps["h1"]), orc.rmsnorm(inputs.bits(x), inputs.bits(g1)), "rmsnorm 1")
    check_quant("xq1", inputs.bits(taps["h1"]), B[0], s_a[0])
    check_gemm("qkv", "xq1", inputs.bits(w_qkv), s_a[0])
    qkv = taps["qkv"]
    qk = qkv[:, : qd + kvd].reshape(T, Hq + Hkv, D).contiguous()
    ref_rope = (orc.rope_rotate if r3 else orc.rope)(inputs.bits(qk), P, 500000.0)
    got_rope = taps["qkv_rope"][:, : qd + kvd].reshape(T, Hq + Hkv, D).contiguous()
    assert_bf16_close(inputs.bits(got_rope), ref_rope, "rope")
    assert torch.equal(taps["qkv_rope"][:, qd + kvd:], qkv[:, qd + kvd:]), "v must pass through the rotary step untouched"
    k_g = got_rope[:, Hq:].reshape(1, T, Hkv, D).contiguous()
    v_g = taps["qkv_rope"][:, qd + kvd:].reshape(1, T, Hkv, D).contiguous()
    kq_ref = np.zeros((1, Hkv, T + 5, D // 2), np.uint8)
    vq_ref = np.zeros_like(kq_ref)
    orc.kv4_append(inputs.bits(k_g), inputs.bits(v_g), s_k, s_v, kq_ref, vq_ref, np.zeros(1, np.int32))
    assert np.array_equal(to_np(taps["kq"])[:, :, :T], kq_ref[:, :, :T]) and np.array_equal(to_np(taps["vq"])[:, :, :T], vq_ref[:, :, :T])
    q_g = got_rope[:, :Hq].contiguous()
    pk_b = inputs.bits(pk) if P else np.zeros((Hkv, 0, D), np.uint16)
    pv_b = inputs.bits(pv) if P else np.zeros((Hkv, 0, D), np.uint16)
    _, ref_attn = orc.prefill_attn(inputs.bits(q_g), pk_b, pv_b, to_np(taps["kq"])[0], to_np(taps["vq"])[0], s_k, s_v,
                                   1 / math.sqrt(D), want_f64=True)
    assert_attn_close(inputs.bits(taps["attn"]).reshape(T, Hq, D), ref_attn, "prefill attention")
    check_quant("xq2", inputs.bits(taps["attn"].reshape(T, qd)), B[1], s_a[1])
    check_gemm("o", "xq2", inputs.bits(w_o), s_a[1])
    assert np.array_equal(inputs.bits(taps["x2"]), orc.add(inputs.bits(x), inputs.bits(taps["o"])))
    # MLP half
    assert_bf16_close(inputs.bits(taps["h2"]), orc.rmsnorm(inputs.bits(taps["x2"]), inputs.bits(g2)), "rmsnorm 2")
    check_quant("xq3", inputs.bits(taps["h2"]), B[2], s_a[2])
    check_gemm("gu", "xq3", inputs.bits(w_gu), s_a[2])
    gu = taps["gu"]
    assert_bf16_close(inputs.bits(taps["act"]), orc.silu_mul(inputs.bits(gu[:, :ffn].contiguous()), inputs.bits(gu[:, ffn:].contiguous())),
                      "silu_mul")
    check_quant("xq4", inputs.bits(taps["act"]), B[3], s_a[3])
    check_gemm("d", "xq4", inputs.bits(w_d), s_a[3])
    assert np.array_equal(inputs.bits(taps["y"]), orc.add(inputs.bits(taps["x2"]), inputs.bits(taps["d"])))
    assert torch.equal(y.cpu(), taps["y"])
    # a second pass over the same input reproduces the first bit for bit (no stale state, no races)
    y2 = blk.forward(x.cuda()).clone()
    assert torch.equal(y2.cpu(), taps["y"])
    ctx.check()
    ctx.close()
