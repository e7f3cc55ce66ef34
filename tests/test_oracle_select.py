"""Pins for the oracle's selection (Alg. 2 Steps 2-3): brute force, a library
partial sort on distinct keys, hand-worked examples and invariants."""
import itertools
import math

import numpy as np
import pytest

import oracle
from conftest import read_golden


def _dominates(g, i, j):
    """True if element i must be kept before element j: larger |g| first, then
    lower index.  Uses float abs, not bit patterns."""
    a, b = math.fabs(float(g[i])), math.fabs(float(g[j]))
    return a > b or (a == b and i < j)


def brute_force_topk(g, k):
    n = len(g)
    hits = []
    for subset in itertools.combinations(range(n), k):
        inside = set(subset)
        outside = [j for j in range(n) if j not in inside]
        if all(_dominates(g, i, j) for i in subset for j in outside):
            hits.append(list(subset))
    assert len(hits) == 1, "the tie-break makes the survivor set unique"
    return hits[0]


def test_golden_h1_and_k_rule():
    gold = read_golden("h1_select.txt")
    g = np.array([float(x) for x in gold["g"][0]], dtype=np.float32)
    for case in gold["case"]:
        ratio, k, idx = float(case[0]), int(case[1]), [int(x) for x in case[2:]]
        assert oracle.k_of(ratio, g.size) == k
        assert oracle.select_topk(g, k).tolist() == idx
    for n, ratio, k in gold["krule"]:
        assert oracle.k_of(float(ratio), int(n)) == int(k)


@pytest.mark.parametrize("seed", range(40))
def test_brute_force_small(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 11))
    # few distinct magnitudes -> many ties, signed zeros, both signs
    pool = np.array([0.0, -0.0, 0.5, -0.5, 1.0, -1.0, 2.0, 1e-40, -1e-40, 3.5], dtype=np.float32)
    g = pool[rng.integers(0, pool.size, n)]
    for k in range(1, n + 1):
        assert oracle.select_topk(g, k).tolist() == brute_force_topk(g, k)


@pytest.mark.parametrize("seed", range(20))
def test_brute_force_small_many_k_from_one_sort(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 10))
    pool = np.array([0.0, -0.0, 0.5, -0.5, 1.0, -1.0, 2.0, 1e-40, -1e-40, 3.5], dtype=np.float32)
    g = pool[rng.integers(0, pool.size, n)]
    ks = list(range(n, 0, -1))  # not in increasing order on purpose
    got = oracle.select_topk_many(g, ks)
    assert [s.tolist() for s in got] == [brute_force_topk(g, k) for k in ks]


def test_compress_many_payloads_carry_the_brute_force_sets():
    g = np.array([0.5, -2.0, 0.0, 2.0, -0.5, 1.0, -0.0, 0.5], dtype=np.float32)  # the worked example
    ratios = [1.0, 0.3, 0.75, 0.5]
    for bits in (8, 16, 32):
        for ratio, p in zip(ratios, oracle.compress_many(g, ratios, bits)):
            k = oracle.k_of(ratio, g.size)
            assert (p.n, p.k, p.bits) == (8, k, bits)
            assert p.idx.tolist() == brute_force_topk(g, k)
            assert np.array_equal(p.raw.view(np.uint32), g[p.idx].view(np.uint32))


def test_distinct_keys_match_partial_sort():
    rng = np.random.default_rng(7)
    mag = rng.permutation(5000).astype(np.float32) * np.float32(0.125) + np.float32(0.125)
    g = mag * rng.choice(np.array([-1.0, 1.0], dtype=np.float32), 5000)
    assert np.unique(np.abs(g)).size == g.size
    for k in (1, 17, 2500, 5000):
        part = np.argpartition(-np.abs(g).astype(np.float64), k - 1)[:k]
        assert oracle.select_topk(g, k).tolist() == sorted(part.tolist())


@pytest.mark.parametrize("seed", range(5))
def test_invariants_with_heavy_ties(seed):
    rng = np.random.default_rng(100 + seed)
    n = 20000
    g = (rng.integers(-6, 7, n) * 0.25).astype(np.float32)  # 7 magnitudes incl. 0
    for ratio in (0.001, 0.3, 0.77, 1.0):
        k = oracle.k_of(ratio, n)
        idx = oracle.select_topk(g, k).astype(np.int64)
        assert idx.size == k and np.all(np.diff(idx) > 0)
        a = np.abs(g)
        inside = np.zeros(n, bool)
        inside[idx] = True
        if k < n:
            thr = a[inside].min()
            assert thr >= a[~inside].max()
            tie_in = np.flatnonzero(inside & (a == thr))
            tie_out = np.flatnonzero(~inside & (a == thr))
            if tie_out.size:
                assert tie_in.max() < tie_out.min()


def test_mask_zeroes_before_selection():
    g = np.array([5.0, 4.0, 3.0, 2.0, 1.0, 0.5], dtype=np.float32)
    mask = np.array([1, 0, 0, 1, 0, 0], dtype=bool)
    p = oracle.compress(g, 0.5, 16, prune_mask=mask)  # k = 3
    assert p.idx.tolist() == [1, 2, 4]
    # pruned positions are picked only after all unpruned ones, lowest index first
    p = oracle.compress(g, 5 / 6, 16, prune_mask=mask)  # k = 5
    assert p.idx.tolist() == [0, 1, 2, 4, 5]
    assert p.raw[0] == 0.0 and not np.signbit(p.raw[0])


def test_fewer_nonzeros_than_k_keeps_sign_of_zero():
    g = np.array([0.0, -0.0, 3.0, -0.0, 0.0], dtype=np.float32)
    p = oracle.compress(g, 0.8, 16)  # k = 4
    assert p.idx.tolist() == [0, 1, 2, 3]
    assert np.signbit(p.raw).tolist() == [False, True, False, True]
    assert p.half.tolist() == [0x0000, 0x8000, 0x4200, 0x8000]


def test_denormals_order_above_zero():
    g = np.array([0.0, 1e-45, -3e-45, 0.0, 1e-38], dtype=np.float32)
    assert oracle.select_topk(g, 3).tolist() == [1, 2, 4]
    assert oracle.select_topk(g, 1).tolist() == [4]
    assert oracle.select_topk(g, 2).tolist() == [2, 4]


def test_nonfinite_rejected():
    for bad in (np.inf, -np.inf, np.nan):
        g = np.array([1.0, bad, 2.0], dtype=np.float32)
        with pytest.raises(oracle.NonFiniteGradient):
            oracle.compress(g, 0.5, 8)


def test_bf16_widening_is_exact():
    bits = np.array([0x3F80, 0xBF80, 0x0000, 0x8000, 0x0001, 0x7F7F, 0x3DCD], dtype=np.uint16)
    v = oracle.widen_bf16(bits)
    assert v.tolist()[:4] == [1.0, -1.0, 0.0, -0.0]
    assert v.view(np.uint32).tolist() == [int(b) << 16 for b in bits]


def test_argument_checks():
    with pytest.raises(ValueError):
        oracle.k_of(0.0, 10)
    with pytest.raises(ValueError):
        oracle.k_of(1.5, 10)
    with pytest.raises(ValueError):
        oracle.k_of(0.5, 0)
    with pytest.raises(ValueError):
        oracle.compress(np.ones(4, np.float32), 0.5, 4)
