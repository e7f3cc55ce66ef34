"""Host arithmetic of Alg. 2 Steps 1-2 behind the C ABI (no GPU needed): the
quantisation gate and the pruned-parameter count, against the oracle and the
worked examples."""
import numpy as np
import pytest

import oracle
import paper_2506_16235_b200 as nsml
from conftest import read_golden


def test_gate_matches_oracle_on_a_grid():
    for ratio in (0.005, 0.01, 0.049999, 0.05, 0.3, 0.5, 0.75, 1.0):
        for l2 in (0.0, 0.5, 1.0, 1.0000001, 7.0):
            for tr_q, tr_d in ((0.05, 1.0), (0.9, 0.5), (0.0, 0.0), (2.0, -1.0)):
                want_q, want_ratio = oracle.quantize_gate(ratio, l2, tr_q, tr_d)
                got_ratio, got_bits = nsml.nsml_quantize_gate(ratio, l2, tr_q, tr_d, nsml.NSML_BITS_FP32)
                assert got_ratio == want_ratio
                assert got_bits == (16 if want_q else 32)
    # the codec used when the gate stays closed is the caller's
    assert nsml.nsml_quantize_gate(0.5, 9.0, 0.1, 1.0, nsml.NSML_BITS_INT8) == (0.5, 8)


def test_gate_rejects_bad_arguments():
    for args in ((0.0, 1.0, 0.1, 1.0, 32), (1.5, 1.0, 0.1, 1.0, 32), (0.1, -1.0, 0.1, 1.0, 32),
                 (0.1, 1.0, float("nan"), 1.0, 32), (0.1, 1.0, 0.1, 1.0, 7)):
        with pytest.raises(nsml.NsmlError) as e:
            nsml.nsml_quantize_gate(*args)
        assert e.value.status == nsml.NSML_ERR_ARG


def test_pruned_count_matches_oracle_and_golden():
    gold = read_golden("h5_prune_mask.txt")
    for n, ratio, m in gold["count"]:
        assert nsml.nsml_pruned_count(int(n), float(ratio)) == int(m)
    rng = np.random.default_rng(0)
    for _ in range(300):
        n = int(rng.integers(1, 10**9))
        ratio = float(rng.choice([1.0, 0.5, 0.1, 0.01, 0.001, rng.uniform(1e-6, 1.0)]))
        assert nsml.nsml_pruned_count(n, ratio) == oracle.pruned_count(ratio, n)
    assert nsml.nsml_pruned_count(0, 0.5) == 0 and nsml.nsml_pruned_count(10, 0.0) == 0


def test_adaptive_payload_capacity_covers_both_outcomes():
    n = 1 << 20
    for ratio, tr_q in ((0.01, 0.05), (0.2, 0.05), (0.6, 0.9)):
        cap = nsml.lib.nsml_adaptive_payload_bytes(n, ratio, tr_q, 32)
        assert cap >= nsml.nsml_payload_bytes(n, ratio, 32)
        if ratio < tr_q:
            assert cap >= nsml.nsml_payload_bytes(n, min(1.0, 2 * ratio), 16)
    assert nsml.nsml_payload_bytes(n, 0.01, 32) == 64 + 4 * 10486 + 8 + 4 * 10486 + 8
