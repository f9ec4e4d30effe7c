"""GPU parity: every entry point of the C-ABI library against the CPU oracle on the same seeded
inputs, element by element. Integer results bit-exact; tolerances as stated in helpers.py."""
import math

import numpy as np
import pytest
import torch

from oracle import pq_oracle as orc
from paper_2410_05265_b200 import inputs
from helpers import (assert_attn_close, assert_bf16_close, assert_codes_tie_tolerant, bf16_ulp, rand_codes, to_np)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2410_05265_b200 import binding

    c = binding.Context()
    yield c
    c.check()
    c.close()


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


# ------------------------------------------------------------------------------- a0 weights
@pytest.mark.parametrize("N,K", [(64, 256), (301, 4096), (16, 14336)])
def test_quant_weights_bit_exact(ctx, N, K):
    W = inputs.weights(N, K, seed=2)
    if N > 5:
        W[5] = 0
    wq_ref, sw_ref = orc.quant_weights(inputs.bits(W))
    wq, s_w = ctx.quant_weights(W.cuda())
    ctx.check()
    assert np.array_equal(to_np(s_w), sw_ref)
    assert np.array_equal(to_np(wq), wq_ref)


# ------------------------------------------------------------------------------- a1 rotation + quantizer
@pytest.mark.parametrize("M,K,B,row_begin", [
    (5, 128, 128, 0), (37, 768, 256, 0), (19, 1024, 1024, 3), (70, 6144, 2048, 4), (33, 4096, 4096, 0),
    (9, 8192, 8192, 1), (300, 4096, 4096, 4), (21, 384, 0, 2),
])
def test_hadamard_quant_act_matches_oracle(ctx, M, K, B, row_begin):
    x = inputs.activations(M, K, seed=0, n_prefix=row_begin)
    cal = inputs.activations(max(M, 16), K, seed=1, n_prefix=row_begin)
    s_ref = orc.calib_act_scale(inputs.bits(cal), B, row_begin)
    s_gpu = ctx.calib_act_scale(cal.cuda(), B, row_begin)
    ctx.check()
    assert abs(float(s_gpu[0]) - float(s_ref)) <= 2e-6 * float(s_ref)
    s_a = torch.tensor([s_ref], dtype=torch.float32, device="cuda")
    xq_ref, tie = orc.quant_act(inputs.bits(x), B, s_ref, row_begin, want_tie_dist=True)
    out = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.hadamard_quant_act(x.cuda(), B, s_a, row_begin, out=out)
    ctx.check()
    got = to_np(out)
    assert np.all(got[:row_begin] == 0x5A), "prefix rows must not be written"
    n_mis = assert_codes_tie_tolerant(got[row_begin:], xq_ref[row_begin:], tie[row_begin:], "hadamard_quant_act")
    assert n_mis <= max(2, int(2e-4 * x.numel()))
    # isolation: the same rows quantize identically when the prefix rows are absent
    if row_begin:
        out2 = ctx.hadamard_quant_act(x[row_begin:].cuda().contiguous(), B, s_a)
        assert torch.equal(out2, out[row_begin:])


@pytest.mark.parametrize("K,B", [(4096, 2048), (4096, 4096)])
def test_hadamard_quant_output_aligned_to_16_bytes_only(ctx, K, B):
    """The header asks for a 16-byte aligned output: a base that is not 32-byte aligned gives the same codes."""
    M = 9
    x = inputs.activations(M, K, seed=0).cuda()
    s_a = ctx.calib_act_scale(x, B)
    ref = ctx.hadamard_quant_act(x, B, s_a)
    buf = torch.zeros(M * (K // 2) + 64, dtype=torch.uint8, device="cuda")
    off = (16 - buf.data_ptr() % 32) % 32
    out = buf[off:off + M * (K // 2)].view(M, K // 2)
    assert out.data_ptr() % 32 == 16
    ctx.hadamard_quant_act(x, B, s_a, out=out)
    ctx.check()
    assert torch.equal(out, ref)
    assert int(buf[:off].sum()) == 0 and int(buf[off + M * (K // 2):].sum()) == 0


def test_hadamard_quant_prefix_outliers_never_set_scale(ctx):
    x = inputs.activations(64, 4096, seed=1, n_prefix=4)
    s1 = ctx.calib_act_scale(x.cuda(), 4096, 4)
    x2 = x.clone()
    x2[:4] *= 100.0
    s2 = ctx.calib_act_scale(x2.cuda(), 4096, 4)
    s0 = ctx.calib_act_scale(x.cuda(), 4096, 0)
    ctx.check()
    assert float(s1) == float(s2) and float(s0) > 5 * float(s1)


# ------------------------------------------------------------------------------- a2 / a3 GEMM
def _gemm_case(ctx, M, N, K, seed, row_begin=0, real_scales=True):
    rng = np.random.default_rng(seed)
    xq = rand_codes(rng, M, K)
    wq = rand_codes(rng, N, K)
    s_a = np.float32(0.0173)
    s_w = (rng.random(N) * 0.004 + 0.001).astype(np.float32)
    acc_ref = orc.gemm_i4(xq, wq)
    out_ref = orc.dequant_bf16(acc_ref, s_a, s_w)
    acc = torch.full((M, N), -77, dtype=torch.int32, device="cuda")
    out = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    ctx.w4a4_gemm(dev(xq), dev(wq), torch.tensor([s_a], device="cuda"), dev(s_w), row_begin, out=out, acc_dbg=acc)
    ctx.check()
    acc = to_np(acc)
    assert np.all(acc[:row_begin] == -77) and np.all(to_np(out[:row_begin].float()) == 3.0)
    assert np.array_equal(acc[row_begin:], acc_ref[row_begin:]), "int32 accumulators must be bit-exact"
    assert_bf16_close(inputs.bits(out)[row_begin:], out_ref[row_begin:], f"gemm {M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", [
    (128, 256, 128),     # one tile, one K block
    (128, 256, 512),     # one tile, ring wraps
    (256, 512, 4096),    # several tiles per CTA pipeline
    (200, 264, 416),     # ragged M, N and K (K % 128 != 0)
    (17, 40, 160),       # smallest tensor-core case, mostly padding
    (333, 1000, 2048),
    (300, 520, 8192),    # long K: the kernel that keeps the token operand in tensor memory
    (257, 256, 14336),
])
def test_gemm_prefill_shapes_bit_exact(ctx, M, N, K):
    _gemm_case(ctx, M, N, K, seed=M + N + K)


def test_gemm_many_tiles_persistent_schedule(ctx):
    _gemm_case(ctx, 1024, 6144, 1024, seed=5)      # 192 tiles: CTAs take a second tile


def test_gemm_row_begin_skips_prefix_rows(ctx):
    _gemm_case(ctx, 260, 256, 256, seed=11, row_begin=4)
    _gemm_case(ctx, 12, 64, 256, seed=12, row_begin=4)


@pytest.mark.parametrize("M", [1, 4, 8, 9, 16])
@pytest.mark.parametrize("N,K", [(48, 4096), (1024, 4096), (40, 160), (4096, 14336)])
def test_gemm_decode_shapes_bit_exact(ctx, M, N, K):
    if N * K > 1 << 24 and M not in (1, 16):
        pytest.skip("large shape covered at M=1 and M=16")
    _gemm_case(ctx, M, N, K, seed=M * 7 + N)


@pytest.mark.parametrize("M,N,K", [(1, 50, 1024), (2, 33, 2048), (3, 1000, 4096), (4, 264, 8192), (2, 72, 14336),
                                   (1, 96, 28672), (4, 20, 28672), (3, 7, 3072)])
def test_gemm_few_tokens_bit_exact(ctx, M, N, K):
    """One to four tokens over short and long K, ragged channel counts."""
    _gemm_case(ctx, M, N, K, seed=M * 13 + N)


def test_gemm_few_tokens_extreme_codes_fit_int32(ctx):
    N, K = 24, 28672
    for M in (1, 4):
        xq = np.full((M, K // 2), 0x88, np.uint8)   # every code -8
        wq = np.full((N, K // 2), 0x88, np.uint8)
        acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
        ctx.w4a4_gemm(dev(xq), dev(wq), torch.ones(1, device="cuda"), torch.ones(N, device="cuda"), acc_dbg=acc)
        ctx.check()
        assert int(acc.min()) == int(acc.max()) == 64 * K


def test_gemm_extreme_codes_fit_int32(ctx):
    M, N, K = 128, 256, 28672
    xq = np.full((M, K // 2), 0x88, np.uint8)   # every code -8
    wq = np.full((N, K // 2), 0x88, np.uint8)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    ctx.w4a4_gemm(dev(xq), dev(wq), torch.ones(1, device="cuda"), torch.ones(N, device="cuda"), acc_dbg=acc)
    ctx.check()
    assert int(acc.min()) == int(acc.max()) == 64 * K


# ------------------------------------------------------------------------------- a1 -> a2 (config 0)
def test_linear_end_to_end_config0(ctx):
    M, K, N = 256, 4096, 4096
    x = inputs.activations(M, K, seed=0)
    cal = inputs.activations(M, K, seed=1)
    W = inputs.weights(N, K, seed=2)
    s_ref = orc.calib_act_scale(inputs.bits(cal), K)
    xq_ref, tie = orc.quant_act(inputs.bits(x), K, s_ref, want_tie_dist=True)
    wq_ref, sw_ref = orc.quant_weights(inputs.bits(W))
    out_ref = orc.dequant_bf16(orc.gemm_i4(xq_ref, wq_ref), s_ref, sw_ref)
    s_a = torch.tensor([s_ref], device="cuda")
    wq, s_w = ctx.quant_weights(W.cuda())
    xq = ctx.hadamard_quant_act(x.cuda(), K, s_a)
    out = ctx.w4a4_gemm(xq, wq, s_a, s_w)
    ctx.check()
    assert np.array_equal(to_np(wq), wq_ref) and np.array_equal(to_np(s_w), sw_ref)
    n_mis = assert_codes_tie_tolerant(to_np(xq), xq_ref, tie, "config0 codes")
    rows_clean = ~(orc.unpack_int4(to_np(xq)) != orc.unpack_int4(xq_ref)).any(axis=1)
    assert rows_clean.sum() >= M - n_mis
    assert_bf16_close(inputs.bits(out)[rows_clean], out_ref[rows_clean], "config0 output")
    # a row with a counted tie mismatch moves by at most one product per mismatch
    if n_mis:
        g = orc.bf16_to_f64(inputs.bits(out)[~rows_clean])
        r = orc.bf16_to_f64(out_ref[~rows_clean])
        assert np.all(np.abs(g - r) <= n_mis * 8 * float(s_ref) * sw_ref.max() + 2e-3 + np.abs(r) * 2.0**-7)


# ------------------------------------------------------------------------------- a4 / a5 KV cache
def _kv_setup(B, Hq, Hkv, D, P, T, Tmax, mag, seed=0, lens=None):
    k = inputs.kv_tensor(B, T, Hkv, D, seed, "k")
    v = inputs.kv_tensor(B, T, Hkv, D, seed, "v")
    s_k = orc.calib_kv_scale(inputs.bits(inputs.kv_tensor(2, 64, Hkv, D, 1, "k")))
    s_v = orc.calib_kv_scale(inputs.bits(inputs.kv_tensor(2, 64, Hkv, D, 1, "v")))
    pk = inputs.prefix_kv(Hkv, P, D, seed, "k", mag)
    pv = inputs.prefix_kv(Hkv, P, D, seed, "v", mag)
    q = inputs.queries(B, Hq, D, seed)
    return k, v, s_k, s_v, pk, pv, q


def _run_attention(ctx, B, Hq, Hkv, P, T, Tmax, mag, seed=0, start=None):
    from paper_2410_05265_b200 import binding

    D = 128
    k, v, s_k, s_v, pk, pv, q = _kv_setup(B, Hq, Hkv, D, P, T, Tmax, mag, seed)
    start = np.zeros(B, np.int32) if start is None else np.asarray(start, np.int32)
    # oracle
    kq_ref = np.full((B, Hkv, Tmax, D // 2), 0x11, np.uint8)
    vq_ref = np.full((B, Hkv, Tmax, D // 2), 0x11, np.uint8)
    len_ref = start.copy()
    assert orc.kv4_append(inputs.bits(k), inputs.bits(v), s_k, s_v, kq_ref, vq_ref, len_ref) == 0
    _, out_ref = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_ref, vq_ref, s_k, s_v, len_ref,
                                 1 / math.sqrt(D), want_f64=True)
    # GPU
    kq = torch.full((B, Hkv, Tmax, D // 2), 0x11, dtype=torch.uint8, device="cuda")
    vq = torch.full((B, Hkv, Tmax, D // 2), 0x11, dtype=torch.uint8, device="cuda")
    length = dev(start)
    cache = binding.KV4Cache(pk.cuda() if P else None, pv.cuda() if P else None, kq, vq, dev(s_k), dev(s_v), length, Hq)
    ctx.kv4_append(cache, k.cuda(), v.cuda())
    ctx.check()
    assert np.array_equal(to_np(length), len_ref)
    assert np.array_equal(to_np(kq), kq_ref) and np.array_equal(to_np(vq), vq_ref), "KV4 codes must match bit for bit"
    ws = ctx.decode_attn_workspace(cache)
    out = ctx.decode_attn(cache, q.cuda(), 1 / math.sqrt(D), ws)
    ctx.check()
    worst = assert_attn_close(inputs.bits(out), out_ref, f"decode attention B{B} Hq{Hq} T{T} P{P} mag{mag}")
    # a second call on the same cache must give the same bits (ticket counters reset themselves)
    out2 = ctx.decode_attn(cache, q.cuda(), 1 / math.sqrt(D), ws)
    assert torch.equal(out, out2)
    return worst


@pytest.mark.parametrize("B,Hq,Hkv,P,T,Tmax,mag", [
    (1, 4, 1, 0, 16, 16, 1.0),       # one block, no prefix
    (2, 8, 2, 2, 100, 128, 1.0),     # ragged tail inside a 16-key block
    (3, 32, 8, 4, 333, 400, 1.0),    # GQA 4, several splits
    (2, 16, 2, 4, 1000, 1024, 50.0), # GQA 8, dominant prefix keys
    (1, 8, 8, 1, 5, 64, 1.0),        # fewer keys than one block, MHA
])
def test_kv4_append_and_decode_attention(ctx, B, Hq, Hkv, P, T, Tmax, mag):
    _run_attention(ctx, B, Hq, Hkv, P, T, Tmax, mag)


def test_decode_attention_config3_variants(ctx):
    # config 3 (prefix magnitude ~50 makes most heads one-hot on a prefix key), plus the variants
    # that put the weight on the INT4 region: magnitude 1 and no prefix at all
    for P, mag in [(4, 50.0), (4, 1.0), (0, 1.0)]:
        _run_attention(ctx, 8, 32, 8, P, 4092, 4096, mag)


def test_decode_attention_ragged_lengths_and_empty_cache(ctx):
    # appending one token to sequences of different lengths, one of them empty
    _run_attention(ctx, 4, 8, 2, 2, 1, 64, 1.0, start=[0, 5, 31, 63])
    _run_attention(ctx, 2, 8, 2, 0, 3, 64, 1.0, start=[0, 40])


def test_decode_attention_short_sequences_in_long_caches(ctx):
    """Most splits have nothing to do: their first round is requested before the length is known and must be
    waited for and ignored (32 splits through the workspace; 8 splits merged inside a cluster)."""
    _run_attention(ctx, 1, 8, 1, 2, 1, 8192, 1.0, start=[129])
    _run_attention(ctx, 1, 8, 1, 0, 1, 8192, 1.0, start=[0])
    _run_attention(ctx, 1, 4, 1, 3, 1, 8000, 1.0, start=[7935])   # the last rounds do not fit the allocation as a whole
    _run_attention(ctx, 8, 32, 8, 4, 1, 4096, 1.0, start=[0, 10, 200, 1000, 127, 128, 129, 4000])


@pytest.mark.parametrize("B,Hq,Hkv,P,Tmax,start", [
    (1, 4, 1, 0, 64, [0]),                      # empty cache, no prefix: the new key is the only key
    (2, 8, 2, 2, 128, [99, 0]),
    (3, 32, 8, 4, 400, [333, 17, 398]),
    (8, 32, 8, 4, 4096, [4091, 10, 200, 1000, 127, 128, 129, 4000]),   # cluster merge
    (1, 8, 1, 3, 8192, [129]),                  # 32 splits through the workspace
])
def test_fused_append_and_decode_attention_equals_the_two_calls(ctx, B, Hq, Hkv, P, Tmax, start):
    from paper_2410_05265_b200 import binding

    D = 128
    k, v, s_k, s_v, pk, pv, q = _kv_setup(B, Hq, Hkv, D, P, 1, Tmax, 1.0, 0)
    start = np.asarray(start, np.int32)
    kq_ref = np.full((B, Hkv, Tmax, D // 2), 0x11, np.uint8)
    vq_ref = np.full_like(kq_ref, 0x11)
    len_ref = start.copy()
    assert orc.kv4_append(inputs.bits(k), inputs.bits(v), s_k, s_v, kq_ref, vq_ref, len_ref) == 0
    _, out_ref = orc.decode_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_ref, vq_ref, s_k, s_v, len_ref,
                                 1 / math.sqrt(D), want_f64=True)

    def fresh():
        kq = torch.full((B, Hkv, Tmax, D // 2), 0x11, dtype=torch.uint8, device="cuda")
        vq = torch.full_like(kq, 0x11)
        return binding.KV4Cache(pk.cuda() if P else None, pv.cuda() if P else None, kq, vq, dev(s_k), dev(s_v), dev(start), Hq)

    cache = fresh()
    ws = ctx.decode_attn_workspace(cache)
    out = ctx.kv4_append_decode_attn(cache, k.cuda(), v.cuda(), q.cuda(), 1 / math.sqrt(D), ws)
    ctx.check()
    assert np.array_equal(to_np(cache.length), len_ref)
    assert np.array_equal(to_np(cache.kq), kq_ref) and np.array_equal(to_np(cache.vq), vq_ref), "appended codes must match bit for bit"
    assert_attn_close(inputs.bits(out), out_ref, "fused append + decode attention")
    # the two calls on a fresh cache agree with the fused one (same codes, same keys; both round to bf16, whose ulp
    # alone is 4e-3 of a value)
    cache2 = fresh()
    ctx.kv4_append(cache2, k.cuda(), v.cuda())
    out2 = ctx.decode_attn(cache2, q.cuda(), 1 / math.sqrt(D), ws)
    ctx.check()
    assert torch.equal(cache2.kq, cache.kq) and torch.equal(cache2.length, cache.length)
    assert float((out.float() - out2.float()).abs().max()) <= 8e-3 * float(out2.float().abs().max()) + 1e-6
    # a second fused call appends the next token
    out3 = ctx.kv4_append_decode_attn(cache, k.cuda(), v.cuda(), q.cuda(), 1 / math.sqrt(D), ws)
    ctx.check()
    assert np.array_equal(to_np(cache.length), len_ref + 1)


def test_fused_append_grid_larger_than_resident_with_a_sequence_that_fills_up(ctx):
    """More CTAs than the GPU holds at once, and one sequence whose append fills it exactly: CTAs that start late
    must not see a length this launch has already advanced (they would take the batch for full)."""
    from paper_2410_05265_b200 import binding

    B, Hq, Hkv, D, Tmax = 96, 8, 8, 128, 128          # 768 CTAs of one split each
    k, v, s_k, s_v, pk, pv, q = _kv_setup(B, Hq, Hkv, D, 0, 1, Tmax, 1.0, 0)
    start = (np.arange(B, dtype=np.int32) * 5) % (Tmax - 1)
    start[0] = Tmax - 1
    start[B - 1] = Tmax - 1
    kq_ref = np.random.default_rng(3).integers(0, 256, (B, Hkv, Tmax, D // 2)).astype(np.uint8)
    vq_ref = np.random.default_rng(4).integers(0, 256, (B, Hkv, Tmax, D // 2)).astype(np.uint8)
    kq, vq = dev(kq_ref), dev(vq_ref)
    len_ref = start.copy()
    assert orc.kv4_append(inputs.bits(k), inputs.bits(v), s_k, s_v, kq_ref, vq_ref, len_ref) == 0
    z = np.zeros((Hkv, 0, D), np.uint16)
    _, out_ref = orc.decode_attn(inputs.bits(q), z, z, kq_ref, vq_ref, s_k, s_v, len_ref, 1 / math.sqrt(D), want_f64=True)
    cache = binding.KV4Cache(None, None, kq, vq, dev(s_k), dev(s_v), dev(start), Hq)
    ws = ctx.decode_attn_workspace(cache)
    out = ctx.kv4_append_decode_attn(cache, k.cuda(), v.cuda(), q.cuda(), 1 / math.sqrt(D), ws)
    assert ctx.check_status() == 0
    assert np.array_equal(to_np(cache.length), len_ref) and int(len_ref[0]) == Tmax
    assert np.array_equal(to_np(kq), kq_ref) and np.array_equal(to_np(vq), vq_ref)
    assert_attn_close(inputs.bits(out), out_ref, "fused append, grid above residency")
    # the next call finds two full sequences: nothing moves, the verdict comes through the status word
    ctx.kv4_append_decode_attn(cache, k.cuda(), v.cuda(), q.cuda(), 1 / math.sqrt(D), ws)
    assert ctx.check_status() == 2
    assert np.array_equal(to_np(cache.length), len_ref) and np.array_equal(to_np(kq), kq_ref)
    # and after the full ones are emptied the counters are in order: the append goes through again
    cache.length[0] = 0
    cache.length[B - 1] = 0
    ctx.kv4_append_decode_attn(cache, k.cuda(), v.cuda(), q.cuda(), 1 / math.sqrt(D), ws)
    assert ctx.check_status() == 0
    len_ref[0] = len_ref[B - 1] = 0
    assert np.array_equal(to_np(cache.length), len_ref + 1)


def test_weights_quantized_in_the_same_stream_reach_the_streaming_gemm(ctx):
    """quantize weights -> rotate + quantize -> M = 1 GEMM enqueued back to back without a synchronisation: the
    weight-streaming kernel fetches its weights ahead of its predecessor's end, and they must be the new ones."""
    N, K = 4096, 4096
    x = inputs.activations(1, K, seed=0)
    s_a = torch.tensor([0.3], device="cuda")
    acc = torch.zeros((1, N), dtype=torch.int32, device="cuda")
    wq = torch.zeros((N, K // 2), dtype=torch.uint8, device="cuda")
    s_w = torch.zeros(N, device="cuda")
    xd = x.cuda()
    for seed in (2, 3, 4):                               # the same buffers are overwritten: stale weights would show
        W = inputs.weights(N, K, seed=seed).cuda()
        torch.cuda.synchronize()
        ctx.quant_weights(W, out=(wq, s_w))
        xq = ctx.hadamard_quant_act(xd, K, s_a)
        ctx.w4a4_gemm(xq, wq, s_a, s_w, acc_dbg=acc)
        ctx.check()
        assert np.array_equal(to_np(acc), orc.gemm_i4(to_np(xq), to_np(wq)))


def test_fused_append_refuses_a_full_sequence(ctx):
    from paper_2410_05265_b200 import binding

    B, Hq, Hkv, D, Tmax = 2, 4, 2, 128, 64
    k, v, s_k, s_v, pk, pv, q = _kv_setup(B, Hq, Hkv, D, 0, 1, Tmax, 1.0, 0)
    kq = torch.full((B, Hkv, Tmax, D // 2), 0x11, dtype=torch.uint8, device="cuda")
    vq = torch.full_like(kq, 0x11)
    length = torch.tensor([10, 64], dtype=torch.int32, device="cuda")   # the second sequence is full
    cache = binding.KV4Cache(None, None, kq, vq, dev(s_k), dev(s_v), length, Hq)
    ws = ctx.decode_attn_workspace(cache)
    out = ctx.kv4_append_decode_attn(cache, k.cuda(), v.cuda(), q.cuda(), 1 / math.sqrt(D), ws)
    assert ctx.check_status() == 2                                      # PQ_ERR_SHAPE through the status word
    assert length.tolist() == [10, 64] and bool((kq == 0x11).all()), "nothing is appended anywhere"
    ref = ctx.decode_attn(cache, q.cuda(), 1 / math.sqrt(D), ws)       # the attention ran over the cache as it was
    assert ctx.check_status() == 0
    assert float((out.float() - ref.float()).abs().max()) <= 1e-6


def test_kv4_append_refuses_overflow(ctx):
    from paper_2410_05265_b200 import binding

    B, Hkv, D, Tmax = 2, 2, 128, 8
    k = inputs.kv_tensor(B, 3, Hkv, D, 0, "k").cuda()
    kq = torch.zeros((B, Hkv, Tmax, D // 2), dtype=torch.uint8, device="cuda")
    vq = torch.zeros_like(kq)
    length = torch.tensor([2, 6], dtype=torch.int32, device="cuda")
    s = torch.ones(Hkv, device="cuda")
    cache = binding.KV4Cache(None, None, kq, vq, s, s, length, 4)
    ctx.kv4_append(cache, k, k)
    assert ctx.check_status() == 2  # PQ_ERR_SHAPE, reported through the status word
    assert length.tolist() == [2, 6] and int(kq.sum()) == 0
    assert ctx.check_status() == 0  # the status word was cleared


def test_argument_errors_are_synchronous(ctx):
    from paper_2410_05265_b200.binding import PQError

    x = torch.zeros((4, 96), dtype=torch.bfloat16, device="cuda")
    s = torch.ones(1, device="cuda")
    with pytest.raises(PQError):
        ctx.hadamard_quant_act(x, 0, s)            # K % 128 != 0
    x = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(PQError):
        ctx.hadamard_quant_act(x, 192, s)          # not a power of two
    xq = torch.zeros((4, 24), dtype=torch.uint8, device="cuda")
    with pytest.raises(PQError):
        ctx.w4a4_gemm(xq, xq, s, torch.ones(4, device="cuda"))   # K = 48 not a multiple of 32


def test_argument_errors_of_the_widened_entry_points(ctx):
    from paper_2410_05265_b200.binding import PQError

    s = torch.ones(1, device="cuda")
    x = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(PQError):
        ctx.hadamard_quant_act8(x, 192, s)                                  # not a power of two
    with pytest.raises(PQError):
        ctx.dyn_act_scale(x, 256, clip=1.5)                                 # clip must lie in (0, 1]
    with pytest.raises(PQError):
        ctx.dyn_act_scale(x, 256, clip=0.0)
    xq8 = torch.zeros((4, 48), dtype=torch.int8, device="cuda")
    wq = torch.zeros((4, 24), dtype=torch.uint8, device="cuda")
    with pytest.raises(PQError):
        ctx.w4a8_gemm(xq8, wq, s, torch.ones(4, device="cuda"))            # K = 48 not a multiple of 32
    with pytest.raises(PQError):
        ctx.outlier_tokens(torch.zeros((8193, 128), dtype=torch.bfloat16, device="cuda"))   # more than 8192 tokens
    with pytest.raises(PQError):
        ctx.outlier_tokens(torch.zeros((8, 100), dtype=torch.bfloat16, device="cuda"))      # C % 8 != 0
    with pytest.raises(PQError):
        ctx.rope(torch.zeros((2, 2, 64), dtype=torch.bfloat16, device="cuda"), 0, 500000.0, rotate=True)  # head_dim != 128
    ctx.check()


# ------------------------------------------------------------------------------- a6 block glue
@pytest.mark.parametrize("M,K", [(5, 128), (37, 4096), (9, 8192), (3, 16384)])
def test_rmsnorm_matches_oracle(ctx, M, K):
    x = inputs.activations(M, K, seed=0)
    g = (1.0 + 0.1 * inputs.weights(1, K, seed=7)[0] / 0.02 * 0.1).to(torch.bfloat16)
    ref = orc.rmsnorm(inputs.bits(x), inputs.bits(g))
    got = ctx.rmsnorm(x.cuda(), g.cuda())
    ctx.check()
    assert_bf16_close(inputs.bits(got), ref, "rmsnorm")


@pytest.mark.parametrize("M,K,row_begin", [(5, 128, 0), (37, 1024, 3), (70, 4096, 4), (19, 8192, 0), (300, 2048, 0)])
def test_rmsnorm_fused_into_rotate_quantize_changes_no_bit(ctx, M, K, row_begin):
    """RMSNorm formed inside the rotation kernel against the two-launch path bit for bit (each of whose stages the
    oracle checks on its own), and the fused codes against the oracle's rotation + quantizer on the GPU's own
    normalised rows."""
    x = inputs.activations(M, K, seed=0, n_prefix=row_begin)
    g = (1.0 + 0.1 * inputs.weights(1, K, seed=7)[0] / 0.02 * 0.1).to(torch.bfloat16)
    xd, gd = x.cuda(), g.cuda()
    h = ctx.rmsnorm(xd, gd, 1e-5)
    assert_bf16_close(inputs.bits(h), orc.rmsnorm(inputs.bits(x), inputs.bits(g), 1e-5), "rmsnorm feeding the rotation")
    s_a = ctx.calib_act_scale(h, K, row_begin)
    two = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    one = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.hadamard_quant_act(h, K, s_a, row_begin, out=two)
    ctx.rmsnorm_hadamard_quant_act(xd, gd, 1e-5, s_a, row_begin, out=one)
    ctx.check()
    assert torch.equal(one, two)
    ref, tie = orc.quant_act(inputs.bits(h), K, np.float32(float(s_a)), row_begin, want_tie_dist=True)
    n = assert_codes_tie_tolerant(to_np(one)[row_begin:], ref[row_begin:], tie[row_begin:], "fused rmsnorm codes")
    assert n <= max(2, int(2e-4 * x.numel()))


@pytest.mark.parametrize("T,H,pos0", [(3, 2, 0), (33, 9, 4), (5, 72, 4090)])
def test_rope_matches_oracle(ctx, T, H, pos0):
    x = inputs.kv_tensor(1, T, H, 128, 0, "k")[0]
    ref = orc.rope(inputs.bits(x), pos0, 500000.0)
    got = ctx.rope(x.cuda().contiguous(), pos0, 500000.0)
    ctx.check()
    assert_bf16_close(inputs.bits(got), ref, "rope")
    xin = x.cuda().contiguous()
    ctx.rope(xin, pos0, 500000.0, out=xin)  # in place
    assert torch.equal(xin, got)


@pytest.mark.parametrize("T,H,pos0", [(3, 2, 0), (33, 9, 4), (5, 72, 4090)])
def test_rope_rotate_matches_oracle(ctx, T, H, pos0):
    """Rotary embedding + head-wise rotation R3 in one call; strided (q|k of a q|k|v row) and in place."""
    x = inputs.kv_tensor(1, T, H, 128, 0, "k")[0]
    ref = orc.rope_rotate(inputs.bits(x), pos0, 500000.0)
    got = ctx.rope(x.cuda().contiguous(), pos0, 500000.0, rotate=True)
    ctx.check()
    assert_bf16_close(inputs.bits(got), ref, "rope + R3")
    wide = torch.zeros((T, H * 128 + 256), dtype=torch.bfloat16, device="cuda")
    wide[:, : H * 128] = x.cuda().reshape(T, H * 128)
    wide[:, H * 128:] = 7.0
    view = wide[:, : H * 128].unflatten(1, (H, 128))
    ctx.rope(view, pos0, 500000.0, out=view, rotate=True)
    ctx.check()
    assert torch.equal(view, got) and bool((wide[:, H * 128:] == 7.0).all())
    # the rotation keeps the scores: q' . k' == q . k up to the bf16 store
    plain = ctx.rope(x.cuda().contiguous(), pos0, 500000.0).double()
    s_plain, s_rot = torch.einsum("thd,shd->hts", plain, plain), torch.einsum("thd,shd->hts", got.double(), got.double())
    assert float((s_plain - s_rot).abs().max()) <= 2.0**-6 * float(s_plain.abs().max())


@pytest.mark.parametrize("T,Hq,Hkv,rotate,start", [(1, 4, 1, False, 0), (37, 8, 2, False, 5), (300, 8, 2, True, 11), (64, 64, 8, True, 0)])
def test_rope_fused_with_kv4_append_equals_the_two_calls(ctx, T, Hq, Hkv, rotate, start):
    """pq_rope_kv4_append against pq_rope (or pq_rope_rotate) followed by pq_kv4_append_strided: the q|k|v buffer, the
    appended codes and the length bit for bit (each of those calls is checked against the oracle on its own)."""
    from paper_2410_05265_b200 import binding

    D, Tmax, P = 128, T + start + 3, 4
    width = (Hq + 2 * Hkv) * D
    qkv = inputs.kv_tensor(1, T, Hq + 2 * Hkv, D, 5, "k")[0].reshape(T, width).contiguous()
    s_k = orc.calib_kv_scale(inputs.bits(inputs.kv_tensor(2, 64, Hkv, D, 1, "k")))
    s_v = orc.calib_kv_scale(inputs.bits(inputs.kv_tensor(2, 64, Hkv, D, 1, "v")))

    def cache(B):
        kq = torch.full((B, Hkv, Tmax, D // 2), 0x11, dtype=torch.uint8, device="cuda")
        return binding.KV4Cache(None, None, kq, torch.full_like(kq, 0x11), dev(s_k), dev(s_v),
                                torch.full((B,), start, dtype=torch.int32, device="cuda"), Hq)

    # the two calls
    a, ca = qkv.cuda(), cache(1)
    qk = a[:, : (Hq + Hkv) * D].unflatten(1, (Hq + Hkv, D))
    ctx.rope(qk, P, 500000.0, out=qk, rotate=rotate)
    k = a[:, Hq * D: (Hq + Hkv) * D].unflatten(1, (Hkv, D)).unsqueeze(0)
    v = a[:, (Hq + Hkv) * D:].unflatten(1, (Hkv, D)).unsqueeze(0)
    ctx.kv4_append(ca, k, v)
    # one call, on the second sequence of a two-sequence cache
    b, cb = qkv.cuda(), cache(2)
    ctx.rope_kv4_append(cb, 1, b, P, 500000.0, rotate=rotate)
    ctx.check()
    assert torch.equal(a, b), "rotated q and k (and the untouched v) must be the same bits"
    assert torch.equal(cb.kq[1], ca.kq[0]) and torch.equal(cb.vq[1], ca.vq[0])
    assert cb.length.tolist() == [start, start + T] and ca.length.tolist() == [start + T]
    assert bool((cb.kq[0] == 0x11).all()) and bool((cb.vq[0] == 0x11).all()), "the other sequence is not touched"
    # past the capacity: the rotation still happens, nothing is appended, the verdict comes through the status word
    c2 = cache(1)
    c2.length.fill_(Tmax - T + 1)
    b2 = qkv.cuda()
    ctx.rope_kv4_append(c2, 0, b2, P, 500000.0, rotate=rotate)
    assert ctx.check_status() == 2
    assert torch.equal(b2, a) and bool((c2.kq == 0x11).all()) and c2.length.tolist() == [Tmax - T + 1]
    # and the counters are in order afterwards
    c3 = cache(1)
    ctx.rope_kv4_append(c3, 0, qkv.cuda(), P, 500000.0, rotate=rotate)
    assert ctx.check_status() == 0 and torch.equal(c3.kq, ca.kq)


@pytest.mark.parametrize("M,F,B,row_begin", [(19, 1024, 1024, 0), (33, 14336, 2048, 4), (5, 256, 128, 1), (130, 4096, 4096, 0)])
def test_swiglu_fused_into_rotate_quantize_changes_no_bit(ctx, M, F, B, row_begin):
    """SiLU(gate) * up formed inside the rotation kernel against the two-launch path (which the oracle checks
    stage by stage elsewhere) and against the oracle chain itself."""
    gu = (inputs.activations(M, 2 * F, seed=3, n_prefix=row_begin) * 2).to(torch.bfloat16)
    gud = gu.cuda()
    gate, up = gud[:, :F], gud[:, F:]
    act = ctx.silu_mul(gate, up)
    s_a = ctx.calib_act_scale(act, B, row_begin)
    two = torch.full((M, F // 2), 0x5A, dtype=torch.uint8, device="cuda")
    one = torch.full((M, F // 2), 0x5A, dtype=torch.uint8, device="cuda")
    ctx.hadamard_quant_act(act, B, s_a, row_begin, out=two)
    ctx.swiglu_hadamard_quant_act(gate, up, B, s_a, row_begin, out=one)
    ctx.check()
    assert torch.equal(one, two)
    # the SwiGLU itself against the oracle (within one bf16 ulp), then the oracle's rotation + quantizer on the GPU's
    # own activation bits, so that an ulp of difference in the SwiGLU never hides the check of the codes
    act_ref = orc.silu_mul(inputs.bits(gu[:, :F].contiguous()), inputs.bits(gu[:, F:].contiguous()))
    assert_bf16_close(inputs.bits(act), act_ref, "silu_mul feeding the rotation")
    ref, tie = orc.quant_act(inputs.bits(act), B, np.float32(float(s_a)), row_begin, want_tie_dist=True)
    n = assert_codes_tie_tolerant(to_np(one)[row_begin:], ref[row_begin:], tie[row_begin:], "fused swiglu codes")
    assert n <= max(2, int(2e-4 * act.numel()))


def test_silu_mul_and_residual_match_oracle(ctx):
    M, F = 19, 1024
    gu = (inputs.activations(M, 2 * F, seed=3) * 2).to(torch.bfloat16)
    gate, up = gu[:, :F], gu[:, F:]
    ref = orc.silu_mul(inputs.bits(gate.contiguous()), inputs.bits(up.contiguous()))
    gud = gu.cuda()
    got = ctx.silu_mul(gud[:, :F], gud[:, F:])
    ctx.check()
    assert_bf16_close(inputs.bits(got), ref, "silu_mul")
    a, b = inputs.activations(M, F, seed=4), inputs.activations(M, F, seed=5)
    ref = orc.add(inputs.bits(a), inputs.bits(b))
    got = ctx.residual_add(a.cuda(), b.cuda())
    ctx.check()
    assert np.array_equal(inputs.bits(got), ref), "a + b in fp32 rounds exactly like the oracle"


@pytest.mark.parametrize("T,Hq,Hkv,P,mag", [(1, 8, 1, 4, 1.0), (37, 8, 2, 4, 50.0), (150, 4, 1, 0, 1.0), (200, 16, 2, 3, 1.0),
                                            (70, 2, 2, 64, 1.0), (96, 4, 2, 4, 1.0)])
def test_prefill_attention_matches_oracle(ctx, T, Hq, Hkv, P, mag):
    from paper_2410_05265_b200 import binding

    D, Tmax, B = 128, T + 11, 2
    k = inputs.kv_tensor(B, T, Hkv, D, 0, "k")
    v = inputs.kv_tensor(B, T, Hkv, D, 0, "v")
    s_k, s_v = orc.calib_kv_scale(inputs.bits(k)), orc.calib_kv_scale(inputs.bits(v))
    kq_ref = np.zeros((B, Hkv, Tmax, D // 2), np.uint8)
    vq_ref = np.zeros_like(kq_ref)
    orc.kv4_append(inputs.bits(k), inputs.bits(v), s_k, s_v, kq_ref, vq_ref, np.zeros(B, np.int32))
    pk = inputs.prefix_kv(Hkv, max(P, 1), D, 0, "k", mag)[:, :P].contiguous()
    pv = inputs.prefix_kv(Hkv, max(P, 1), D, 0, "v", mag)[:, :P].contiguous()
    seq = 1
    q = inputs.kv_tensor(1, T, Hq, D, 3, "k")[0].contiguous()
    _, ref64 = orc.prefill_attn(inputs.bits(q), inputs.bits(pk), inputs.bits(pv), kq_ref[seq], vq_ref[seq], s_k, s_v,
                                1 / math.sqrt(D), want_f64=True)
    cache = binding.KV4Cache(pk.cuda() if P else None, pv.cuda() if P else None, dev(kq_ref), dev(vq_ref), dev(s_k), dev(s_v),
                             torch.full((B,), T, dtype=torch.int32, device="cuda"), Hq)
    out = torch.full((T, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.prefill_attn(cache, seq, q.cuda(), 1 / math.sqrt(D), out=out)
    ctx.check()
    # the stated attention tolerance against the oracle's unrounded result (plus the bf16 store's own half ulp)
    assert_attn_close(inputs.bits(out), ref64, f"prefill attention T{T} Hq{Hq} Hkv{Hkv} P{P}")


# ------------------------------------------------------------------------------- outlier tokens (Sec. 4.1, Eq. 2)
@pytest.mark.parametrize("T,C", [(1, 128), (33, 256), (64, 4096), (2048, 4096), (8192, 128)])
def test_outlier_tokens_match_oracle_bit_for_bit(ctx, T, C):
    x = inputs.activations(T, C, seed=3, n_prefix=min(4, T - 1))
    if T > 20:
        x[17] *= 0.01   # a lower outlier
        x[9] = 0        # a silent token: 1 / R is infinite
    M_ref, R_ref, f_ref, med_ref = orc.outlier_tokens(inputs.bits(x))
    M, R, flags, med = ctx.outlier_tokens(x.cuda())
    ctx.check()
    assert np.array_equal(to_np(M), M_ref) and float(med) == med_ref
    assert np.array_equal(to_np(R), R_ref, equal_nan=True) and np.array_equal(to_np(flags), f_ref)
    if T > 20:
        assert to_np(flags)[:4].tolist() == [1, 1, 1, 1] and int(flags[17]) == 2 and int(flags[9]) == 2
    # a strided view (the first C columns of a wider matrix) gives the same answer
    wide = torch.zeros((T, C + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :C] = x.cuda()
    wide[:, C:] = 1e6
    _, R2, f2, _ = ctx.outlier_tokens(wide[:, :C])
    assert torch.equal(f2, flags) and np.array_equal(to_np(R2), R_ref, equal_nan=True)
