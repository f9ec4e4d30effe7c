"""The index-bit roles and the padded exchange layout of the rotation kernel for blocks of 2048, 4096 and 8192
(csrc/pq_hadamard_quant.cu, hadamard_quant_wide_kernel), restated on the CPU and checked for what the kernel relies on:
the thread roles of pass 1 cover every element of a block exactly once, the padded layout is injective and fits the
kernel's buffer, a warp's 8-byte stores (half-warp at a time) and 16-byte loads (quarter-warp at a time) touch every
bank at most once, and a warp's 4-byte loads cover whole 32-byte sectors of few 128-byte lines. No GPU needed."""
import pytest


def roles(logb):
    j = 13 - logb
    t0s = 6 if j == 0 else 1
    t1s = 2 if j == 2 else (6 if j == 1 else 7)
    return dict(J=j, T0=t0s, T1=t1s, G=j + 1, W=j + 4, M3=8 - j, K3=9 - j, TAU=10 - j,
                PADK={2: 4, 1: 20, 0: 28}[j], BLKF={2: 2176, 1: 4736, 0: 9088}[j], WPB=1 << (logb - 11))


def pad(i, r):
    extra = 0
    if r["J"] == 1:
        extra = 16 * ((i >> 6) & 1)
    elif r["J"] == 0:
        extra = 8 * ((i >> 6) & 1) + 16 * ((i >> 7) & 1)
    return r["PADK"] * (i >> r["M3"]) + extra


def writer_index(r, wv, lane, m3, nb, tau):
    g, t = lane >> 2, lane & 3
    return ((t & 1) << r["T0"]) | ((t >> 1) << r["T1"]) | (g << r["G"]) | (wv << r["W"]) | (m3 << r["M3"]) | (nb << r["K3"]) | (tau << r["TAU"])


@pytest.mark.parametrize("logb", [11, 12, 13])
def test_pass_one_roles_cover_the_block_and_the_padded_layout_is_conflict_free(logb):
    r = roles(logb)
    n = 1 << logb
    seen = set()
    top = 0
    for wv in range(r["WPB"]):
        for m3 in range(2):
            for nb in range(2):
                for tau in range(8):
                    for half in range(2):  # an 8-byte store is served one half-warp at a time
                        banks = {}
                        for lane in range(16 * half, 16 * half + 16):
                            i = writer_index(r, wv, lane, m3, nb, tau)
                            for k in range(2):  # the pair (index bit 0) leaves in one store
                                assert i + k not in seen
                                seen.add(i + k)
                                a = i + k + pad(i + k, r)
                                assert a == i + pad(i, r) + k, "a pair must stay adjacent"
                                top = max(top, a)
                                banks[a % 32] = banks.get(a % 32, 0) + 1
                        assert max(banks.values()) == 1
    assert seen == set(range(n))
    assert len({i + pad(i, r) for i in range(n)}) == n, "the padded layout must be injective"
    assert top < r["BLKF"], "the padded block must fit the kernel's buffer"
    assert r["BLKF"] % 4 == 0 and r["BLKF"] * (4 // r["WPB"]) <= 2 * 4736
    # pass 2: thread hi reads the 64 consecutive elements 64 hi .. 64 hi + 63 with 16-byte loads, a quarter-warp at a time
    for wv in range(r["WPB"]):
        for cc in range(16):
            for quarter in range(4):
                banks = {}
                for lane in range(8 * quarter, 8 * quarter + 8):
                    hi = lane | (wv << 5)
                    i = (hi << 6) | (cc << 2)
                    a = i + pad(i, r)
                    assert a % 4 == 0
                    for k in range(4):
                        assert i + k + pad(i + k, r) == a + k, "a thread's 64 elements must stay contiguous"
                        banks[(a + k) % 32] = banks.get((a + k) % 32, 0) + 1
                assert max(banks.values()) == 1


@pytest.mark.parametrize("logb,max_lines", [(11, 1), (12, 2), (13, 4)])
def test_a_warp_load_covers_whole_sectors_of_few_lines(logb, max_lines):
    r = roles(logb)
    for wv in range(r["WPB"]):
        for m3 in range(2):
            for k3 in range(2):
                for tau in range(8):
                    byte = [2 * writer_index(r, wv, lane, m3, k3, tau) for lane in range(32)]  # same roles at the load
                    sectors = {}
                    for b in byte:
                        sectors.setdefault(b // 32, set()).update(range(b % 32, b % 32 + 4))
                    assert all(len(v) == 32 for v in sectors.values()), "every touched sector is used in full"
                    assert len({s // 4 for s in sectors}) <= max_lines
