"""Pins for the oracle's gate, pruning mask and local accumulation (Alg. 2
Steps 1-2, Section 4.2 Step 3): closed forms, brute force, a library partial
sort on distinct keys, hand-worked examples and invariants."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from conftest import read_golden


# ---------------------------------------------------------------- L2 norm
def test_l2_closed_forms():
    assert oracle.l2_norm(np.array([3.0, -4.0], dtype=np.float32)) == 5.0
    assert oracle.l2_norm(np.zeros(17, dtype=np.float32)) == 0.0
    # constant vector: sqrt(n) * |c|, exact for n a square and c a power of two
    assert oracle.l2_norm(np.full(1 << 20, -0.25, dtype=np.float32)) == 1024 * 0.25
    # a sign flip or a permutation changes nothing
    rng = np.random.default_rng(0)
    g = rng.standard_normal(1000).astype(np.float32)
    assert oracle.l2_norm(g) == pytest.approx(oracle.l2_norm(-g[::-1]), rel=1e-15)


@pytest.mark.parametrize("seed", range(5))
def test_l2_against_exact_rational_sum(seed):
    rng = np.random.default_rng(seed)
    g = (rng.standard_normal(300) * 10.0 ** rng.uniform(-6, 2, 300)).astype(np.float32)
    exact = sum(Fraction(float(x)) ** 2 for x in g)  # float32 values are exact rationals
    want = math.sqrt(float(exact))
    assert oracle.l2_norm(g) == pytest.approx(want, rel=1e-14)


def test_l2_matches_library_norm_in_float64():
    rng = np.random.default_rng(3)
    g = rng.standard_normal(100_000).astype(np.float32)
    assert oracle.l2_norm(g) == pytest.approx(float(np.linalg.norm(g.astype(np.float64))), rel=1e-13)


def test_l2_float32_would_not_do():
    # 2^24 ones and one more: a float32 running sum stalls at 2^24, the float64 one does not
    g = np.ones((1 << 24) + 9, dtype=np.float32)
    assert oracle.l2_norm(g) ** 2 == pytest.approx((1 << 24) + 9, rel=1e-15)


def test_l2_rejects_nonfinite():
    with pytest.raises(oracle.NonFiniteGradient):
        oracle.l2_norm(np.array([1.0, np.inf], dtype=np.float32))


# ---------------------------------------------------------------- gate (Alg. 2 Step 1)
def test_gate_branches():
    # ratio below tr_q and norm above tr_d: 16-bit values, ratio doubled
    assert oracle.quantize_gate(0.01, 3.0, 0.05, 1.0) == (True, 0.02)
    # norm not above tr_d (strict comparison): nothing changes
    assert oracle.quantize_gate(0.01, 1.0, 0.05, 1.0) == (False, 0.01)
    # ratio not below tr_q (strict comparison): nothing changes, whatever the norm
    assert oracle.quantize_gate(0.05, 1e9, 0.05, 1.0) == (False, 0.05)
    # the doubled ratio is a kept fraction: capped at 1
    assert oracle.quantize_gate(0.7, 2.0, 0.9, 1.0) == (True, 1.0)


def test_alg2_order_gate_then_mask_then_topk():
    # Step 1 doubles the ratio, and Steps 2 and 3 use the doubled one
    rng = np.random.default_rng(5)
    n = 400
    g = rng.standard_normal(n).astype(np.float32)
    w = rng.standard_normal(n).astype(np.float32)
    p, ratio, bits, l2, mask = oracle.netsense_compression(g, 0.05, tr_q=0.1, tr_d=1.0, weights=w)
    assert (ratio, bits) == (0.1, 16) and l2 == oracle.l2_norm(g) and l2 > 1.0
    assert p.k == 40 and int(mask.sum()) == oracle.pruned_count(0.1, n) == 180
    assert not mask[p.idx.astype(np.int64)].any(), "enough unpruned non-zeros: no pruned position is sent"
    # gate closed (ratio >= tr_q): plain floats, norm not even computed
    p, ratio, bits, l2, mask = oracle.netsense_compression(g, 0.2, tr_q=0.1, tr_d=1.0, weights=w)
    assert (ratio, bits, l2) == (0.2, 32, None) and p.k == 80 and int(mask.sum()) == 160
    assert np.array_equal(p.values().view(np.uint32), g[p.idx.astype(np.int64)].view(np.uint32))
    # gate open but the gradient is small: plain floats at the old ratio
    p, ratio, bits, l2, _ = oracle.netsense_compression(g * np.float32(1e-3), 0.05, tr_q=0.1, tr_d=1.0)
    assert (ratio, bits) == (0.05, 32) and l2 < 1.0 and p.k == 20


# ---------------------------------------------------------------- pruning mask (Alg. 2 Step 2)
def _prunes_before(w, i, j):
    a, b = math.fabs(float(w[i])), math.fabs(float(w[j]))
    return a < b or (a == b and i < j)


def brute_force_mask(w, m):
    n = len(w)
    hits = []
    for subset in itertools.combinations(range(n), m):
        inside = set(subset)
        if all(_prunes_before(w, i, j) for i in subset for j in range(n) if j not in inside):
            hits.append(sorted(subset))
    assert len(hits) == 1
    return hits[0]


def test_golden_h5_mask_and_count_rule():
    gold = read_golden("h5_prune_mask.txt")
    w = np.array([float(x) for x in gold["w"][0]], dtype=np.float32)
    for case in gold["case"]:
        ratio, rate, m, idx = float(case[0]), float(case[1]), int(case[2]), [int(x) for x in case[3:]]
        assert oracle.pruning_rate(ratio) == rate
        assert oracle.pruned_count(ratio, w.size) == m
        assert np.flatnonzero(oracle.prune_mask(w, ratio)).tolist() == idx
    for n, ratio, m in gold["count"]:
        assert oracle.pruned_count(float(ratio), int(n)) == int(m)


@pytest.mark.parametrize("seed", range(30))
def test_mask_brute_force_small(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 11))
    pool = np.array([0.0, -0.0, 0.5, -0.5, 1.0, -1.0, 2.0, 1e-40, -1e-40, 3.5], dtype=np.float32)
    w = pool[rng.integers(0, pool.size, n)]
    for ratio in (1.0, 0.9, 0.6, 0.3, 0.05):
        m = oracle.pruned_count(ratio, n)
        assert np.flatnonzero(oracle.prune_mask(w, ratio)).tolist() == brute_force_mask(w, m)


def test_mask_distinct_keys_match_partial_sort():
    rng = np.random.default_rng(11)
    mag = rng.permutation(5000).astype(np.float32) * np.float32(0.125) + np.float32(0.125)
    w = mag * rng.choice(np.array([-1.0, 1.0], dtype=np.float32), 5000)
    for ratio in (0.9, 0.5, 0.01):
        m = oracle.pruned_count(ratio, w.size)
        part = np.argpartition(np.abs(w).astype(np.float64), m - 1)[:m]
        assert np.array_equal(np.flatnonzero(oracle.prune_mask(w, ratio)), np.sort(part))


@pytest.mark.parametrize("seed", range(6))
def test_mask_invariants(seed):
    rng = np.random.default_rng(200 + seed)
    n = 3000
    w = np.round(rng.standard_normal(n) * 4).astype(np.float32) / 4  # heavy ties, zeros
    for ratio in (0.8, 0.3, 0.02):
        mask = oracle.prune_mask(w, ratio)
        m = oracle.pruned_count(ratio, n)
        assert int(mask.sum()) == m
        a = np.abs(w)
        if 0 < m < n:
            t = a[mask].max()
            assert t <= a[~mask].min()
            tied_in, tied_out = np.flatnonzero(mask & (a == t)), np.flatnonzero(~mask & (a == t))
            if tied_in.size and tied_out.size:
                assert tied_in.max() < tied_out.min(), "ties at the threshold: lower index pruned first"
        # Alg. 2: pruning never leaves fewer candidates than Step 3 keeps
        assert n - m >= oracle.k_of(ratio, n)


# ---------------------------------------------------------------- local accumulation (Section 4.2 Step 3)
def test_golden_h6_error_feedback():
    gold = read_golden("h6_error_feedback.txt")
    ratio = float(gold["ratio"][0][0])
    r = np.zeros(4, dtype=np.float32)
    for step in (1, 2, 3):
        g = np.array([float(x) for x in gold[f"g{step}"][0]], dtype=np.float32)
        p, r = oracle.error_feedback_step(g, r, ratio, 32)
        assert p.idx.tolist() == [int(gold[f"sent{step}"][0][0])]
        assert p.values().tolist() == [float(gold[f"sent{step}"][0][1])]
        assert r.tolist() == [float(x) for x in gold[f"r{step}"][0]]


@pytest.mark.parametrize("bits", [8, 16, 32])
def test_feedback_conserves_the_accumulated_gradient(bits):
    rng = np.random.default_rng(bits)
    n = 5000
    r = np.zeros(n, dtype=np.float32)
    total_in = np.zeros(n, dtype=np.float64)
    total_sent = np.zeros(n, dtype=np.float64)
    for step in range(6):
        g = (rng.standard_normal(n) * 0.01).astype(np.float32)
        acc = (g + r).astype(np.float32)
        p, r_new = oracle.error_feedback_step(g, r, 0.05, bits)
        idx = p.idx.astype(np.int64)
        # unsent positions keep the whole accumulated value
        keep = np.ones(n, dtype=bool)
        keep[idx] = False
        assert np.array_equal(r_new[keep].view(np.uint32), acc[keep].view(np.uint32))
        # sent positions keep exactly the part the receiver does not get
        sent = p.values().astype(np.float64)
        assert np.all(np.abs(sent + r_new[idx].astype(np.float64) - acc[idx].astype(np.float64))
                      <= np.spacing(np.abs(acc[idx])).astype(np.float64))
        if bits == 32:
            assert not r_new[idx].any()
        total_in += g.astype(np.float64)
        total_sent[idx] += sent
        r = r_new
    # nothing is lost over the steps: inputs = sent + still held, up to float32 rounding of each step
    assert np.max(np.abs(total_in - total_sent - r.astype(np.float64))) < 6 * 2.0 ** -24 * 0.1


def test_feedback_with_mask_keeps_accumulating_pruned_positions():
    g = np.array([4.0, 1.0, 2.0, 0.5], dtype=np.float32)
    mask = np.array([True, False, False, False])
    p, r = oracle.error_feedback_step(g, np.zeros(4, dtype=np.float32), 0.5, 32, mask)
    assert p.idx.tolist() == [1, 2]
    assert r.tolist() == [4.0, 0.0, 0.0, 0.5]  # the pruned gradient is not sent but not forgotten
