"""GPU parity: nsml_compress against the oracle, bit-exact (index sets, int8
codes, scales, fp16 bit patterns), on small and adversarial buckets."""
import numpy as np
import pytest
import torch

import oracle
import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2506_16235_b200 as nsml
    from gpu_util import (assert_payload_equal, check_compress, gpu_compress, oracle_compress, to_device_grad)

SIZES = [1, 2, 3, 4, 5, 7, 31, 32, 33, 127, 128, 129, 511, 512, 513, 4095, 4096, 4097, 8191, 12289, 100003]


def make(kind, n, rng):
    if kind == "normal":
        return (rng.standard_normal(n) * 10.0 ** rng.uniform(-4, -1, n)).astype(np.float32)
    if kind == "equal":
        return np.full(n, -0.375, dtype=np.float32)
    if kind == "zero":
        g = np.zeros(n, dtype=np.float32)
        g[rng.random(n) < 0.5] = -0.0
        return g
    if kind == "ties":
        return (rng.integers(-3, 4, n) * 0.5).astype(np.float32)
    if kind == "sparse":
        g = rng.standard_normal(n).astype(np.float32)
        g[rng.random(n) < 0.9] = 0.0
        return g
    if kind == "denormal":
        bits = rng.integers(0, 1 << 12, n).astype(np.uint32)  # keys far below 2**19
        bits |= (rng.integers(0, 2, n).astype(np.uint32) << 31)
        return bits.view(np.float32)
    if kind == "wide":
        return (rng.standard_normal(n) * 10.0 ** rng.uniform(-38, 38, n)).astype(np.float32)
    raise ValueError(kind)


@pytest.mark.parametrize("kind", ["normal", "equal", "zero", "ties", "sparse", "denormal"])
@pytest.mark.parametrize("n", SIZES)
def test_small_buckets(kind, n):
    rng = np.random.default_rng(n * 7 + len(kind))
    g = make(kind, n, rng)
    for ratio in (1e-9, 0.01, 0.3, 0.5, 1.0):
        for bits in (8, 16):
            check_compress(g, ratio, bits)


def test_wide_range_saturates_fp16_and_keeps_int8_exact():
    rng = np.random.default_rng(1)
    g = make("wide", 50000, rng)
    for ratio in (0.02, 0.7):
        for bits in (8, 16):
            check_compress(g, ratio, bits)


def test_config1_full():
    g = synth.config1_bucket()
    payload, want = check_compress(g, 0.01, 8)
    assert want.k == 10486 and want.scales.size == 11
    check_compress(g, 0.01, 16)


@pytest.mark.parametrize("ratio", [0.001, 0.05, 0.25, 0.8, 0.81, 1.0])
def test_zero_heavy_bucket_all_ratios(ratio):
    # 20 % zeros: ratios above 0.8 must fill up with zeros, lowest index first
    g = synth.config1_bucket(n=300001, seed=3)
    check_compress(g, ratio, 8)


def test_threshold_ties_span_many_tiles():
    rng = np.random.default_rng(5)
    n = 40 * 4096 + 77
    g = np.full(n, 0.25, dtype=np.float32)
    g[rng.random(n) < 0.001] = 3.0
    g[rng.random(n) < 0.3] *= -1.0
    for ratio in (0.0005, 0.01, 0.5, 0.9999):
        check_compress(g, ratio, 16)


def test_prune_mask():
    rng = np.random.default_rng(8)
    for n in (37, 4096, 50001):
        g = (rng.standard_normal(n)).astype(np.float32)
        for ratio in (0.05, 0.5, 0.9):
            # the paper's pruning rate for this ratio: 0.5 * (1 - ratio)
            mask = rng.random(n) < 0.5 * (1.0 - ratio)
            check_compress(g, ratio, 8, mask_bool=mask)
            check_compress(g, ratio, 16, mask_bool=mask)
    # everything pruned: k zeros, lowest indices
    g = rng.standard_normal(1000).astype(np.float32)
    payload, want = check_compress(g, 0.1, 16, mask_bool=np.ones(1000, bool))
    assert want.idx.tolist() == list(range(100)) and not want.half.any()


@pytest.mark.parametrize("n", [5, 4096, 70001])
def test_bf16_buckets(n):
    rng = np.random.default_rng(n)
    g = synth.f32_to_bf16_bits((rng.standard_normal(n) * 10.0 ** rng.uniform(-6, -2, n)).astype(np.float32))
    for ratio in (0.001, 0.1, 0.6):
        for bits in (8, 16):
            check_compress(g, ratio, bits)


def sampled_positions(n, strata=8192):
    """Positions the library's stratified sampler reads (one per stratum, a
    hashed offset inside it), restated from its description so that a test can
    build a bucket on which the sample is misleading."""
    s = np.arange(strata, dtype=np.uint64)
    begin = s * np.uint64(n) // np.uint64(strata)
    end = (s + np.uint64(1)) * np.uint64(n) // np.uint64(strata)
    x = (s * np.uint64(0x9E3779B1) + np.uint64(0x85EBCA6B)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(16)
    x = (x * np.uint64(0x7FEB352D)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(15)
    x = (x * np.uint64(0x846CA68B)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(16)
    return (begin + x % (end - begin)).astype(np.int64)


@pytest.mark.parametrize("n", [20000, 200000, 1 << 20])
def test_misleading_sample_still_gives_the_exact_result(n):
    # large magnitudes exactly where the sampler looks, small ones elsewhere:
    # the sampled bracket then keeps far fewer than k elements and the repeat
    # pass has to produce the list
    rng = np.random.default_rng(n)
    g = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    pos = sampled_positions(n)
    g[pos] = (100.0 + rng.random(pos.size)).astype(np.float32) * rng.choice(np.array([-1.0, 1.0], np.float32), pos.size)
    for ratio in (0.1, 0.5):
        check_compress(g, ratio, 8)
    # and the opposite: zeros where the sampler looks (bracket starts at key 0)
    g = rng.standard_normal(n).astype(np.float32)
    g[pos] = 0.0
    check_compress(g, 0.05, 16)


def test_nonfinite_is_reported_not_trapped():
    rng = np.random.default_rng(2)
    for bad in (np.inf, -np.inf, np.nan):
        g = rng.standard_normal(9000).astype(np.float32)
        g[4321] = bad
        _, status = gpu_compress(g, 0.1, 8)
        assert status == nsml.NSML_ERR_NONFINITE
        with pytest.raises(oracle.NonFiniteGradient):
            oracle_compress(g, 0.1, 8)
    # the same workspace is usable afterwards
    check_compress(rng.standard_normal(9000).astype(np.float32), 0.1, 8)


def test_payload_is_bit_reproducible():
    g = synth.config1_bucket(n=777777, seed=4)
    a, _ = gpu_compress(g, 0.03, 8)
    b, _ = gpu_compress(g, 0.03, 8)
    assert torch.equal(a, b)


def test_workspace_reuse_across_calls_and_sizes():
    rng = np.random.default_rng(12)
    ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(200000), "cuda")
    for n, ratio, bits in ((200000, 0.01, 8), (1234, 0.5, 16), (199999, 0.2, 8), (4096, 1.0, 16)):
        g = rng.standard_normal(n).astype(np.float32)
        grad = to_device_grad(g)
        payload = nsml.nsml_compress(grad, ratio, bits, workspace=ws)
        assert nsml.nsml_last_status(ws) == 0
        assert_payload_equal(payload, oracle_compress(g, ratio, bits))


def test_runtime_argument_errors():
    grad = torch.zeros(1000, device="cuda")
    with pytest.raises(nsml.NsmlError) as e:
        nsml.nsml_compress(grad, 0.5, 8, payload=torch.zeros(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == nsml.NSML_ERR_CAPACITY
    with pytest.raises(nsml.NsmlError) as e:
        nsml.nsml_compress(grad, 0.5, 8, workspace=torch.zeros(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == nsml.NSML_ERR_CAPACITY
    with pytest.raises(nsml.NsmlError):
        nsml.nsml_compress(grad, 0.0, 8)
    with pytest.raises(nsml.NsmlError) as e:
        nsml.nsml_compress(grad[1:], 0.5, 8)  # 4-byte offset: not 16-byte aligned
    assert e.value.status == nsml.NSML_ERR_ARG


# ---- the dense strategy (high kept fractions; no sample, no bucket pass) at sizes that use the large
# kernel shape, with and without values beyond a block's shared-memory cache ----
@pytest.mark.parametrize("n,ratio", [(2_000_003, 0.5), (3_100_000, 0.26), (9_000_001, 0.3)])
def test_dense_strategy_large_buckets(n, ratio):
    assert nsml.nsml_compress_strategy(n, ratio) == 1
    rng = np.random.default_rng(n)
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-4, -1, n)).astype(np.float32)
    g[rng.random(n) < 0.2] = 0.0
    check_compress(g, ratio, 8)
    mask = rng.random(n) < 0.5 * (1.0 - ratio)
    check_compress(g, ratio, 16, mask_bool=mask)
    check_compress(synth.f32_to_bf16_bits(g), ratio, 8, mask_bool=mask)


@pytest.mark.parametrize("kind", ["equal", "zero", "ties", "sparse", "denormal"])
def test_dense_strategy_degenerate_values(kind):
    # every key equal / mostly zeros: the selection is decided by the index tie-break across blocks
    n = 2_500_000 + 13
    g = make(kind, n, np.random.default_rng(17))
    for ratio in (0.25, 0.6, 1.0):
        assert nsml.nsml_compress_strategy(n, ratio) == 1
        check_compress(g, ratio, 8)


def test_strategy_switch_is_invisible():
    # the same bucket just below and just above the kept fraction at which the strategy changes
    n = 1_500_000
    g = synth.config1_bucket(n=n, seed=11)
    seen = set()
    for ratio in (0.049, 0.051, 0.249, 0.2499, 0.25, 0.251):
        seen.add(nsml.nsml_compress_strategy(n, ratio))
        check_compress(g, ratio, 8)
    assert seen == {0, 1}


def test_buckets_on_concurrent_streams_and_replayed_from_a_graph():
    # independent buckets on eight streams with their own workspaces (as the benchmark runs them), nothing
    # synchronised in between; then one of the calls captured into a CUDA graph and replayed on new data
    rng = np.random.default_rng(77)
    cases = []
    for s in range(8):
        n = int(rng.integers(200_000, 900_000))
        g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-4, -1, n)).astype(np.float32)
        ratio, bits = [(0.01, 8), (0.001, 16), (0.1, 8), (0.5, 16), (0.03, 32), (0.01, 16), (0.3, 8), (0.002, 8)][s]
        cases.append((g, ratio, bits))
    streams = [torch.cuda.Stream() for _ in cases]
    grads = [to_device_grad(g) for g, _, _ in cases]
    wss = [nsml.alloc_bytes(nsml.nsml_workspace_bytes(g.size), "cuda") for g, _, _ in cases]
    torch.cuda.synchronize()
    payloads = []
    for rep in range(3):  # the same calls again and again, still without waiting
        payloads = [nsml.nsml_compress(grads[i], r, b, workspace=wss[i], stream=streams[i])
                    for i, (_, r, b) in enumerate(cases)]
    torch.cuda.synchronize()
    for i, (g, r, b) in enumerate(cases):
        assert nsml.nsml_last_status(wss[i]) == 0
        assert_payload_equal(payloads[i], oracle_compress(g, r, b))

    g, ratio, bits = cases[0]
    buf, ws = grads[0], wss[0]
    payload = nsml.alloc_bytes(nsml.nsml_payload_bytes(g.size, ratio, bits), "cuda")
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        nsml.nsml_compress(buf, ratio, bits, payload=payload, workspace=ws, stream=side)
    for rep in range(2):
        fresh = np.roll(g, 1234 * (rep + 1))
        buf.copy_(torch.from_numpy(fresh))
        graph.replay()
        torch.cuda.synchronize()
        assert_payload_equal(payload[:nsml.nsml_payload_bytes(g.size, ratio, bits)], oracle_compress(fresh, ratio, bits))


def test_bounded_wait_runs_out_and_reports_timeout():
    # a barrier that can never complete: the kernel gives up after the poll limit, returns by itself and
    # leaves NSML_ERR_TIMEOUT in the status word; the workspace then serves an ordinary call
    g = synth.config1_bucket(n=1 << 18, seed=3)
    n = g.size
    ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(n), "cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for polls in (1, 2000):
        assert nsml.lib.nsml_selftest_bounded_wait(ws.data_ptr(), ws.numel(), polls, stream) == 0
        assert nsml.nsml_last_status(ws) == nsml.NSML_ERR_TIMEOUT
    assert nsml.lib.nsml_selftest_bounded_wait(ws.data_ptr(), ws.numel(), 0, stream) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_selftest_bounded_wait(ws.data_ptr(), ws.numel(), 1 << 20, stream) == nsml.NSML_ERR_ARG
    assert "wait" in nsml.nsml_strerror(nsml.NSML_ERR_TIMEOUT)
    payload = nsml.nsml_compress(torch.from_numpy(g).cuda(), 0.01, 8, workspace=ws)
    assert nsml.nsml_last_status(ws) == 0
    assert_payload_equal(payload, oracle.compress(g, 0.01, 8))

# The bucket pass gives every warp 2 KB of the bucket (one float32 segment of 512 elements, two bfloat16
# segments) and every block eight warps: sizes at and around the segment, warp and block boundaries, with the
# ragged last segment falling to the first, a middle and the last warp of a block, with and without a mask.
PASS_EDGE_SIZES = [16384, 16385, 16384 + 511, 16384 + 512, 16384 + 513, 16384 + 1024 + 1, 20480 - 1, 20480, 20480 + 1,
                   24576 + 7 * 512 + 3, 8 * 4096 - 512 + 5, 8 * 4096 + 1]


@pytest.mark.parametrize("n", PASS_EDGE_SIZES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bucket_pass_tails(n, dtype):
    rng = np.random.default_rng(n)
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-5, -2, n)).astype(np.float32)
    g[-3:] = [3.0, -4.0, 5.0]  # the last elements are survivors: a dropped tail shows
    g[0] = -6.0
    if dtype == "bf16":
        g = synth.f32_to_bf16_bits(g)
    mask = rng.random(n) < 0.3
    mask[-2] = True
    for ratio in (0.003, 0.05):  # list strategy
        assert nsml.nsml_compress_strategy(n, ratio) == 0
        check_compress(g, ratio, 16)
        check_compress(g, ratio, 8, mask_bool=mask)


@pytest.mark.parametrize("candidates", [1024, 8192])
def test_list_block_candidates_knob_does_not_change_the_payload(candidates):
    rng = np.random.default_rng(77)
    n = 3_000_001
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-4, -1, n)).astype(np.float32)
    nsml.nsml_set_list_block_candidates(candidates)
    try:
        for ratio in (0.002, 0.02, 0.2):  # cluster shape and small shape of the list stage
            check_compress(g, ratio, 8)
            check_compress(g, ratio, 16)
        # the large shape (more than about 1.2M expected candidates): one block per SM above the default setting
        big = (rng.standard_normal(8_000_003) * 10.0 ** rng.uniform(-4, -1, 8_000_003)).astype(np.float32)
        check_compress(big, 0.2, 8)
    finally:
        nsml.nsml_set_list_block_candidates(4096)
