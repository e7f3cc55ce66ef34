"""Pins for the oracle's value codecs and the multi-worker sum."""
import struct

import numpy as np
import pytest

import oracle
from conftest import read_golden


def f32(x):
    """Round a Python float (double) to float32 and back, via struct."""
    return struct.unpack("<f", struct.pack("<f", x))[0]


def scalar_int8_block(vals):
    """Independent scalar restatement with Python doubles: a double quotient
    rounded to float32 equals the float32 quotient (double rounding is
    innocuous for division when 53 >= 2*24 + 2), and Python's round() is
    half-to-even."""
    maxabs = max(abs(float(v)) for v in vals)
    scale = f32(maxabs / 127.0)
    if scale == 0.0:
        return [0] * len(vals), scale
    codes = []
    for v in vals:
        q = f32(float(v) / scale)
        codes.append(int(max(-127, min(127, round(q)))))
    return codes, scale


def test_golden_int8_blocks():
    gold = read_golden("h2_int8.txt")
    for blk in "AB":
        v = np.array([float(x) for x in gold[f"block{blk}_val"][0]], dtype=np.float32)
        codes, scales = oracle.quantize_int8(v)
        assert codes.tolist() == [int(x) for x in gold[f"block{blk}_codes"][0]]
        assert int(scales.view(np.uint32)[0]) == int(gold[f"block{blk}_scale_bits"][0][0], 16)
    deq = oracle.dequantize_int8(*oracle.quantize_int8(np.array([0.5, -2.0, 2.0, 1.0], np.float32)))
    want = [float(x) for x in gold["blockB_dequant"][0]]
    assert np.allclose(deq, want, rtol=0, atol=5e-7)
    for blk in "CD":
        v = np.array([float(x) for x in gold[f"block{blk}_val"][0]], dtype=np.float32)
        codes, scales = oracle.quantize_int8(v)
        assert codes.tolist() == [int(x) for x in gold[f"block{blk}_codes"][0]]
        assert scales[0] == 0.0


@pytest.mark.parametrize("seed", range(6))
def test_int8_against_scalar_doubles(seed):
    rng = np.random.default_rng(seed)
    k = 2 * oracle.QBLOCK + 137  # two full blocks and a ragged one
    v = (rng.standard_normal(k) * 10.0 ** rng.uniform(-42, 3, k)).astype(np.float32)
    v[rng.random(k) < 0.05] = 0.0
    if seed == 0:  # a block of half-way quotients
        v[: oracle.QBLOCK] = 0.0
        v[0] = 127.0
        v[1:255] = np.arange(1, 255) * 0.5
    codes, scales = oracle.quantize_int8(v)
    for b in range(3):
        blk = v[b * oracle.QBLOCK:(b + 1) * oracle.QBLOCK]
        want_codes, want_scale = scalar_int8_block(blk)
        assert float(scales[b]) == want_scale
        assert codes[b * oracle.QBLOCK:(b + 1) * oracle.QBLOCK].tolist() == want_codes


def test_int8_invariants():
    rng = np.random.default_rng(11)
    k = 5 * oracle.QBLOCK + 3
    v = (rng.standard_normal(k) * 10.0 ** rng.uniform(-6, 0, k)).astype(np.float32)
    codes, scales = oracle.quantize_int8(v)
    assert scales.size == 6 and np.all(scales >= 0)
    assert codes.min() >= -127 and codes.max() <= 127
    deq = oracle.dequantize_int8(codes, scales).astype(np.float64)
    per = np.repeat(scales.astype(np.float64), oracle.QBLOCK)[:k]
    assert np.all(np.abs(v.astype(np.float64) - deq) <= per * (0.5 + 2.0 ** -20))
    for b in range(6):
        blk = v[b * oracle.QBLOCK:(b + 1) * oracle.QBLOCK]
        j = int(np.argmax(np.abs(blk)))
        assert abs(int(codes[b * oracle.QBLOCK + j])) == 127
        assert np.sign(codes[b * oracle.QBLOCK + j]) == np.sign(blk[j])


def test_golden_fp16_bits():
    gold = read_golden("fp16_bits.txt")
    vals = np.array([float(p[0]) for p in gold["pair"]], dtype=np.float32)
    want = [int(p[1], 16) for p in gold["pair"]]
    assert oracle.f32_to_f16_bits(vals).tolist() == want


def test_fp16_matches_library_casts_in_range():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(400000) * 10.0 ** rng.uniform(-10, 5, 400000)).astype(np.float32)
    x = x[np.abs(x) < 65520.0]
    got = oracle.f32_to_f16_bits(x)
    assert np.array_equal(got, x.astype(np.float16).view(np.uint16))
    # python's struct 'e' packer is a second, numpy-free implementation
    for v, h in zip(x[:3000].tolist(), got[:3000].tolist()):
        assert struct.unpack("<H", struct.pack("<e", v))[0] == h
    # exhaustively: every finite half converts back to itself
    allh = np.arange(0x10000, dtype=np.uint32).astype(np.uint16)
    finite = ((allh >> 10) & 0x1F) != 31
    back = oracle.f16_bits_to_f32(allh[finite])
    assert np.array_equal(back, allh[finite].view(np.float16).astype(np.float32))
    assert np.array_equal(oracle.f32_to_f16_bits(back), allh[finite])


def test_fp16_midpoints_round_to_even():
    # midpoints between neighbouring halves, built exactly in float32
    h = np.arange(0x0001, 0x7BFF, 97, dtype=np.uint32).astype(np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + np.uint16(1)).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (lo + hi) / 2)  # exact in float32
    got = oracle.f32_to_f16_bits(mid)
    want = np.where(h % 2 == 0, h, h + np.uint16(1))
    assert np.array_equal(got, want)


def test_fp16_saturates():
    v = np.array([65519.99, 65520.0, 3e38, -65520.0, -3e38], dtype=np.float32)
    assert oracle.f32_to_f16_bits(v).tolist() == [0x7BFF, 0x7BFF, 0x7BFF, 0xFBFF, 0xFBFF]


def _mk(n, idx, vals, bits=16):
    idx = np.array(idx, dtype=np.uint32)
    raw = np.array(vals, dtype=np.float32)
    p = oracle.Payload(n=n, k=idx.size, bits=bits, idx=idx, raw=raw)
    if bits == 16:
        p.half = oracle.f32_to_f16_bits(raw)
    else:
        p.codes, p.scales = oracle.quantize_int8(raw)
    return p


def test_sum_closed_forms():
    n = 50
    a = _mk(n, [1, 7, 20], [0.5, -1.25, 3.0])
    one = oracle.decompress_sum([a], n)
    assert one[[1, 7, 20]].tolist() == [0.5, -1.25, 3.0] and np.count_nonzero(one) == 3
    assert np.array_equal(oracle.decompress_sum([a] * 4, n), 4 * one)  # power of two: exact
    b = _mk(n, [2, 8, 49], [1.0, 2.0, -4.0])
    both = oracle.decompress_sum([a, b], n)
    assert np.array_equal(both, one + oracle.decompress_sum([b], n))  # disjoint
    twice = oracle.decompress_sum([a], n, dense_in=oracle.decompress_sum([a], n))
    assert np.array_equal(twice, 2 * one)


def test_sum_against_dense_loop():
    rng = np.random.default_rng(5)
    n, W = 300, 5
    payloads, dense = [], [0.0] * n
    base = rng.standard_normal(n).astype(np.float32)
    for w in range(W):
        g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-3, 0, n)).astype(np.float32)
        payloads.append(oracle.compress(g, 0.2, 8 if w % 2 else 16))
    want = [float(x) for x in base]
    for p in payloads:
        vals = p.values()
        for j in range(p.k):
            if p.bits == 8:
                assert float(vals[j]) == f32(float(p.codes[j]) * float(p.scales[j // oracle.QBLOCK]))
            want[int(p.idx[j])] += float(vals[j])
    got = oracle.decompress_sum(payloads, n, dense_in=base)
    assert got.tolist() == [f32(x) for x in want]


def test_round_trip_bounds():
    rng = np.random.default_rng(9)
    n = 40000
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-4, -1, n)).astype(np.float32)
    for bits in (8, 16):
        p = oracle.compress(g, 0.1, bits)
        d = oracle.decompress_sum([p], n)
        sel = np.zeros(n, bool)
        sel[p.idx] = True
        assert np.all(d[~sel] == 0.0) and not np.any(np.signbit(d[~sel]))
        err = np.abs(d[sel].astype(np.float64) - g[sel].astype(np.float64))
        if bits == 8:
            per = np.repeat(p.scales.astype(np.float64), oracle.QBLOCK)[: p.k]
            assert np.all(err <= per * (0.5 + 2.0 ** -20))
        else:
            assert np.all(err <= np.maximum(np.abs(g[sel]) * 2.0 ** -11, 2.0 ** -25))


def test_sum_rejects_bad_payload():
    with pytest.raises(ValueError):
        oracle.decompress_sum([_mk(10, [3, 3], [1.0, 1.0])], 10)
    with pytest.raises(ValueError):
        oracle.decompress_sum([_mk(10, [3, 10], [1.0, 1.0])], 10)
