"""GPU parity for the rest of Alg. 2: L2 norm and gate (Step 1), pruning mask
from the weights (Step 2), plain float32 values, local accumulation of the
filtered gradients (Section 4.2 Step 3) and the three steps in one call."""
import numpy as np
import pytest
import torch

import oracle
from conftest import read_golden
import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2506_16235_b200 as nsml
    from gpu_util import (CANARY, assert_payload_equal, check_accumulate, check_compress, mask_words,
                          payload_to_device, to_device_grad)

L2_RTOL = 1e-12  # float64 sums of exact squares in another order: ~sqrt(n) * 2^-53 at worst


# ------------------------------------------------------------------ Step 1
@pytest.mark.parametrize("n", [1, 3, 4, 5, 255, 4095, 4096, 4097, 100003, 1 << 20, 6_553_600])
def test_l2_norm(n):
    rng = np.random.default_rng(n)
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-4, 1, n)).astype(np.float32)
    want = oracle.l2_norm(g)
    got = nsml.nsml_grad_l2(to_device_grad(g))
    assert abs(got - want) <= L2_RTOL * want
    assert nsml.nsml_grad_l2(to_device_grad(g)) == got, "fixed summation order: reproducible"


def test_l2_norm_bf16_and_closed_forms():
    rng = np.random.default_rng(2)
    bits16 = (rng.standard_normal(300001).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    want = oracle.l2_norm(oracle.widen_bf16(bits16))
    got = nsml.nsml_grad_l2(to_device_grad(bits16))
    assert abs(got - want) <= L2_RTOL * want
    assert nsml.nsml_grad_l2(torch.full((1 << 22,), -0.25, device="cuda")) == 2048 * 0.25
    assert nsml.nsml_grad_l2(torch.zeros(777, device="cuda")) == 0.0
    # 2^24 + 9 ones: a float32 running sum would stall at 2^24
    assert nsml.nsml_grad_l2(torch.ones((1 << 24) + 9, device="cuda")) ** 2 == pytest.approx((1 << 24) + 9, rel=1e-15)


def test_l2_norm_reports_nonfinite():
    g = torch.ones(10000, device="cuda")
    g[7777] = float("inf")
    with pytest.raises(nsml.NsmlError) as e:
        nsml.nsml_grad_l2(g)
    assert e.value.status == nsml.NSML_ERR_NONFINITE


# ------------------------------------------------------------------ Step 2
def gpu_mask(w, ratio):
    n = w.size
    words = (n + 31) // 32
    buf = torch.full((words + 64,), -1515870811, dtype=torch.int32, device="cuda")  # 0xA5A5A5A5
    ws = nsml.alloc_bytes(nsml.nsml_prune_workspace_bytes(n), "cuda")
    nsml.nsml_prune_mask_build(torch.from_numpy(w).cuda(), ratio, prune_mask=buf, workspace=ws)
    status = nsml.nsml_last_status(ws)
    assert bool((buf[words:] == -1515870811).all()), "wrote past the end of the mask"
    return buf[:words].cpu().numpy().view(np.uint32), status


def check_mask(w, ratio):
    got, status = gpu_mask(w, ratio)
    assert status == 0, nsml.nsml_strerror(status)
    want = mask_words(oracle.prune_mask(w, ratio))
    assert np.array_equal(got, want), f"mask differs (n={w.size}, ratio={ratio})"


def make_weights(kind, n, rng):
    if kind == "normal":
        return (rng.standard_normal(n) * 0.05).astype(np.float32)
    if kind == "equal":
        return np.full(n, 1.0, dtype=np.float32)  # e.g. freshly initialised normalisation weights
    if kind == "zero":
        w = np.zeros(n, dtype=np.float32)
        w[rng.random(n) < 0.5] = -0.0
        return w
    if kind == "ties":
        return (rng.integers(-3, 4, n) * 0.5).astype(np.float32)
    if kind == "denormal":
        bits = rng.integers(0, 1 << 12, n).astype(np.uint32) | (rng.integers(0, 2, n).astype(np.uint32) << 31)
        return bits.view(np.float32)
    raise ValueError(kind)


@pytest.mark.parametrize("kind", ["normal", "equal", "zero", "ties", "denormal"])
@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 127, 4095, 4096, 4097, 8191, 12289, 100003])
def test_prune_mask_small(kind, n):
    rng = np.random.default_rng(n * 11 + len(kind))
    w = make_weights(kind, n, rng)
    for ratio in (1.0, 0.99, 0.5, 0.1, 0.01, 1e-9):
        check_mask(w, ratio)


def test_prune_mask_golden_h5():
    gold = read_golden("h5_prune_mask.txt")
    w = np.array([float(x) for x in gold["w"][0]], dtype=np.float32)
    for case in gold["case"]:
        got, status = gpu_mask(w, float(case[0]))
        assert status == 0
        assert [i for i in range(w.size) if (got[0] >> i) & 1] == [int(x) for x in case[3:]]


def test_prune_mask_ties_span_many_tiles():
    rng = np.random.default_rng(9)
    n = 60 * 4096 + 55
    w = np.full(n, 0.5, dtype=np.float32)
    w[rng.random(n) < 0.2] = 0.01
    w[rng.random(n) < 0.3] *= -1.0
    for ratio in (0.9, 0.5, 0.2, 0.01):
        check_mask(w, ratio)


@pytest.mark.parametrize("ratio", [0.5, 0.1, 0.01, 0.001])
def test_prune_mask_resnet50_bucket(ratio):
    rng = np.random.default_rng(4)
    w = (rng.standard_normal(6_553_600) * 0.03).astype(np.float32)
    w[rng.random(w.size) < 0.01] = 0.0
    check_mask(w, ratio)


def test_prune_mask_25m_bucket():
    rng = np.random.default_rng(5)
    w = (rng.standard_normal(25_000_000) * 10.0 ** rng.uniform(-3, -1, 25_000_000)).astype(np.float32)
    check_mask(w, 0.01)


def prune_sampled_positions(n, strata=8192):
    """Positions the mask build's stratified sampler reads (one per stratum, a hashed offset inside it),
    restated from its description so that a test can build weights on which the sample misleads."""
    s = np.arange(strata, dtype=np.uint64)
    width = np.uint64(n // strata)
    x = (s * np.uint64(0x9E3779B1) + np.uint64(0x85EBCA6B)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(16)
    x = (x * np.uint64(0x7FEB352D)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(15)
    x = (x * np.uint64(0x846CA68B)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(16)
    return (s * width + ((x * width) >> np.uint64(32))).astype(np.int64)


@pytest.mark.parametrize("n", [70_001, 1 << 20])
def test_prune_mask_misleading_sample_still_exact(n):
    # tiny (then huge) magnitudes exactly where the sampler looks: the sampled window misses the threshold and
    # the four-pass build has to produce the mask
    rng = np.random.default_rng(n)
    w = rng.standard_normal(n).astype(np.float32)
    pos = prune_sampled_positions(n)
    for fill in (1e-9, 1e9):
        w2 = w.copy()
        w2[pos] = (fill * (1.0 + rng.random(pos.size))).astype(np.float32)
        for ratio in (0.01, 0.5):
            check_mask(w2, ratio)


def test_prune_mask_two_pass_path_with_ties_in_the_threshold_bin():
    # Gaussian weights rounded to few mantissa bits: every key has many equals, the threshold's bin holds tens
    # of equal keys and only some of them (lowest indices first) are pruned
    rng = np.random.default_rng(77)
    n = 3_000_017
    w = rng.standard_normal(n).astype(np.float32)
    w = (w.view(np.uint32) & np.uint32(0xFFFFF000)).view(np.float32)  # 11 mantissa bits left
    for ratio in (0.2, 0.003):
        check_mask(w, ratio)


def test_prune_mask_reports_nonfinite():
    w = np.ones(5000, dtype=np.float32)
    w[123] = np.nan
    _, status = gpu_mask(w, 0.5)
    assert status == nsml.NSML_ERR_NONFINITE


@pytest.mark.parametrize("ratio", [0.01, 0.5])  # list strategy and dense strategy of Step 3
def test_whole_algorithm_keeps_the_mask_build_error_visible(ratio):
    # Steps 2 and 3 share one workspace: non-finite weights found while the mask is built (Step 2) must
    # still be reported after Step 3 has run on the same workspace
    n = 100_000
    rng = np.random.default_rng(17)
    g = rng.standard_normal(n).astype(np.float32)
    w = rng.standard_normal(n).astype(np.float32)
    w[4321] = np.inf
    ws = nsml.alloc_bytes(int(nsml.lib.nsml_adaptive_workspace_bytes(n, nsml.NSML_F32)), "cuda")
    nsml.nsml_compress_adaptive(to_device_grad(g), ratio, 0.0, 0.0, plain_bits=8, weights=torch.from_numpy(w).cuda(),
                                workspace=ws)
    assert nsml.nsml_last_status(ws) == nsml.NSML_ERR_NONFINITE
    # and the same workspace reports a clean run afterwards
    w[4321] = 0.25
    payload, _, _, _, mask = nsml.nsml_compress_adaptive(to_device_grad(g), ratio, 0.0, 0.0, plain_bits=8,
                                                         weights=torch.from_numpy(w).cuda(), workspace=ws)
    assert nsml.nsml_last_status(ws) == 0
    assert_payload_equal(payload, oracle.compress(g, ratio, 8, prune_mask=oracle.prune_mask(w, ratio)))


def test_mask_feeds_compress():
    rng = np.random.default_rng(6)
    n = 200_003
    g = rng.standard_normal(n).astype(np.float32)
    w = rng.standard_normal(n).astype(np.float32)
    mask = nsml.nsml_prune_mask_build(torch.from_numpy(w).cuda(), 0.05)
    payload = nsml.nsml_compress(to_device_grad(g), 0.05, 8, prune_mask=mask)
    assert_payload_equal(payload, oracle.compress(g, 0.05, 8, prune_mask=oracle.prune_mask(w, 0.05)))


# ------------------------------------------------------------------ plain float32 values
@pytest.mark.parametrize("n", [1, 5, 1023, 1024, 1025, 4097, 100003])
def test_fp32_values_small(n):
    rng = np.random.default_rng(n)
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-30, 30, n)).astype(np.float32)
    for ratio in (0.01, 0.3, 1.0):
        payload, want = check_compress(g, ratio, 32)
        check_accumulate([payload], [want], n, zero_first=True)


def test_fp32_values_mixed_with_other_codecs():
    g = synth.config1_bucket(n=300001, seed=4)
    pts, pos = [], []
    for w, bits in enumerate((32, 8, 16, 32)):
        gw = np.roll(g, 1000 * w)
        payload, want = check_compress(gw, 0.02, bits)
        pts.append(payload)
        pos.append(want)
    check_accumulate(pts, pos, g.size, zero_first=False)
    # a payload laid out by hand is read the same way
    check_accumulate([payload_to_device(pos[0])], [pos[0]], g.size, zero_first=True)


def test_fp32_values_dense_strategy_and_large_bucket():
    g = list(synth.resnet50_buckets(seed=1))[3]
    for ratio in (0.5, 0.01):
        check_compress(g, ratio, 32)


# ------------------------------------------------------------------ Section 4.2 Step 3
def run_feedback(gs, ratio, bits, mask_bool=None, dtype_bf16=False):
    n = gs[0].size
    residual = torch.zeros(n, device="cuda")
    r_want = np.zeros(n, dtype=np.float32)
    ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(n, nsml.NSML_F32), "cuda")
    mw = None if mask_bool is None else torch.from_numpy(mask_words(mask_bool).view(np.int32)).cuda()
    for g in gs:
        need = nsml.nsml_payload_bytes(n, ratio, bits)
        buf = torch.full((need + 256,), CANARY, dtype=torch.uint8, device="cuda")
        payload = nsml.nsml_compress_feedback(to_device_grad(g), residual, ratio, bits, prune_mask=mw, payload=buf,
                                              workspace=ws)
        assert nsml.nsml_last_status(ws) == 0
        assert bool((buf[need:] == CANARY).all())
        vals = oracle.widen_bf16(g) if g.dtype == np.uint16 else g
        want, r_want = oracle.error_feedback_step(vals, r_want, ratio, bits, mask_bool)
        assert_payload_equal(payload, want)
        # one float32 add and one float32 subtraction per element on both sides: bit for bit
        assert np.array_equal(residual.cpu().numpy().view(np.uint32), r_want.view(np.uint32)), "residual differs"


def test_feedback_golden_h6():
    gold = read_golden("h6_error_feedback.txt")
    gs = [np.array([float(x) for x in gold[f"g{s}"][0]], dtype=np.float32) for s in (1, 2, 3)]
    run_feedback(gs, float(gold["ratio"][0][0]), 32)


@pytest.mark.parametrize("bits", [8, 16, 32])
@pytest.mark.parametrize("n", [7, 4097, 300_001])
def test_feedback_steps(bits, n):
    rng = np.random.default_rng(n + bits)
    gs = [(rng.standard_normal(n) * 10.0 ** rng.uniform(-4, -1, n)).astype(np.float32) for _ in range(4)]
    run_feedback(gs, 0.03, bits)


def test_feedback_with_mask_bf16_and_dense_strategy():
    rng = np.random.default_rng(8)
    n = 150_001
    mask = rng.random(n) < 0.4
    gs = [(rng.standard_normal(n).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16) for _ in range(3)]
    run_feedback(gs, 0.02, 16, mask_bool=mask)
    run_feedback([oracle.widen_bf16(g) for g in gs], 0.5, 8, mask_bool=mask)


def test_feedback_resnet50_bucket():
    bucket = list(synth.resnet50_buckets(seed=1))[0]
    run_feedback([bucket, np.roll(bucket, 12345)], 0.01, 8)


# ------------------------------------------------------------------ Alg. 2 in one call
@pytest.mark.parametrize("case", ["quantise", "small_norm", "gate_closed"])
def test_adaptive_matches_oracle(case):
    rng = np.random.default_rng(12)
    n = 500_003
    g = rng.standard_normal(n).astype(np.float32)
    w = rng.standard_normal(n).astype(np.float32)
    ratio, tr_q, tr_d = {"quantise": (0.02, 0.05, 10.0), "small_norm": (0.02, 0.05, 1e6),
                         "gate_closed": (0.2, 0.05, 10.0)}[case]
    want, want_ratio, want_bits, want_l2, want_mask = oracle.netsense_compression(g, ratio, tr_q, tr_d, weights=w)
    payload, got_ratio, got_bits, got_l2, mask = nsml.nsml_compress_adaptive(
        to_device_grad(g), ratio, tr_q, tr_d, weights=torch.from_numpy(w).cuda())
    assert (got_ratio, got_bits) == (want_ratio, want_bits)
    assert (got_l2 is None) == (want_l2 is None)
    if want_l2 is not None:
        assert abs(got_l2 - want_l2) <= L2_RTOL * want_l2
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), mask_words(want_mask))
    assert_payload_equal(payload, want)
    assert {"quantise": (0.04, 16), "small_norm": (0.02, 32), "gate_closed": (0.2, 32)}[case] == (got_ratio, got_bits)


# ------------------------------------------------------------------ the exchange step around the path
def test_gradient_exchange_single_rank_follows_the_controller():
    # one rank (no process group): the all-gather is a copy, everything else is the real path
    from paper_2506_16235_b200 import dp

    n = 300_001
    rng = np.random.default_rng(21)
    ex = dp.GradientExchange(n, bits=16, startup_max_steps=0, ratio_init=0.05)
    ora = oracle.Controller(oracle.ControllerParams(startup_max_steps=0, ratio_init=0.05))
    dense = torch.empty(n, device="cuda")
    last = (0.0, 0.0)
    for step in range(4):
        g = rng.standard_normal(n).astype(np.float32)
        ratio = ex.step(to_device_grad(g), dense)
        assert ratio == ora.select_ratio(last[0], last[1], 4.0 * n)
        last = ex.last
        assert last[0] == nsml.nsml_payload_bytes(n, ratio, 16) and last[1] > 0
        want = oracle.compress(g, ratio, 16)
        got = dense.cpu().numpy()
        ref = oracle.decompress_sum([want], n)
        assert np.max(np.abs(got.astype(np.float64) - ref.astype(np.float64))) <= 1e-6 * float(np.abs(g).max())


# ------------------------------------------------------------------ corner paths of the new steps
def test_prune_mask_small_tie_group_at_the_threshold():
    # exactly three weights share the threshold magnitude and only some of them are pruned: decided by index
    n = 100_001
    rng = np.random.default_rng(31)
    w = ((rng.permutation(n).astype(np.float32) + 1.0) * np.float32(1e-4)) * rng.choice(np.array([-1.0, 1.0], np.float32), n)
    order = np.argsort(np.abs(w), kind="stable")
    for ratio, extra in ((0.5, 0), (0.5, 1), (0.5, 2), (0.2, 1)):
        m = oracle.pruned_count(ratio, n)
        v = w.copy()
        tied = order[m - 1 - extra:m + 2 - extra]  # three ranks around the m-th smallest
        v[tied] = np.abs(w[order[m - 1 - extra]]) * np.array([1.0, -1.0, 1.0], np.float32)
        check_mask(v, ratio)


def test_feedback_when_fewer_than_k_sums_are_nonzero():
    # list strategy whose candidate list comes out short: the list stage rebuilds it from the bucket, which
    # here is the residual buffer holding gradient + residual
    rng = np.random.default_rng(41)
    n = 300_001
    gs = []
    for _ in range(3):
        g = rng.standard_normal(n).astype(np.float32)
        g[rng.random(n) < 0.93] = 0.0
        gs.append(g)
    run_feedback(gs[:1], 0.2, 8)   # first step: 7 % non-zero, 20 % kept
    run_feedback(gs, 0.2, 16)      # later steps: the residual fills positions up


def test_adaptive_bf16_gradient_with_int8_as_the_plain_codec():
    rng = np.random.default_rng(51)
    n = 400_003
    bits16 = (rng.standard_normal(n).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    g = oracle.widen_bf16(bits16)
    w = rng.standard_normal(n).astype(np.float32)
    for ratio, tr_q in ((0.03, 0.1), (0.3, 0.1)):
        want, want_ratio, want_bits, _, want_mask = oracle.netsense_compression(g, ratio, tr_q, 5.0, weights=w, plain_bits=8)
        payload, got_ratio, got_bits, _, mask = nsml.nsml_compress_adaptive(
            to_device_grad(bits16), ratio, tr_q, 5.0, plain_bits=8, weights=torch.from_numpy(w).cuda())
        assert (got_ratio, got_bits) == (want_ratio, want_bits)
        assert np.array_equal(mask.cpu().numpy().view(np.uint32), mask_words(want_mask))
        assert_payload_equal(payload, want)
