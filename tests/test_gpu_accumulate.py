"""GPU parity: nsml_decompress_accumulate against the oracle's fp64 sum, within
1e-6 of the bucket's largest magnitude; exact where the sum has one term."""
import numpy as np
import pytest
import torch

import oracle
import synth

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2506_16235_b200 as nsml
    from gpu_util import check_accumulate, check_compress, payload_to_device


def worker_grads(n, W, seed):
    rng = np.random.default_rng(seed)
    return [(rng.standard_normal(n) * 10.0 ** rng.uniform(-3, -1, n)).astype(np.float32) for _ in range(W)]


@pytest.mark.parametrize("n", [1, 5, 4097, 8192, 8193, 100003])
@pytest.mark.parametrize("W", [1, 2, 4, 8])
def test_compress_then_sum(n, W):
    pt, po = [], []
    for w, g in enumerate(worker_grads(n, W, n + W)):
        payload, want = check_compress(g, 0.07, 8 if w % 2 == 0 else 16)
        pt.append(payload)
        po.append(want)
    check_accumulate(pt, po, n, zero_first=True)
    rng = np.random.default_rng(0)
    check_accumulate(pt, po, n, zero_first=False, dense_init=rng.standard_normal(n).astype(np.float32))


def test_single_worker_round_trip_is_exact():
    n = 300007
    g = synth.config1_bucket(n=n, seed=9)
    for bits in (8, 16):
        payload, want = check_compress(g, 0.01, bits)
        got, ref = check_accumulate([payload], [want], n, zero_first=True)
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))  # one term per element: exact
        sel = np.zeros(n, bool)
        sel[want.idx] = True
        assert not got[~sel].any() and not np.signbit(got[~sel]).any()


def test_identical_payloads_sum_exactly():
    n = 50000
    g = worker_grads(n, 1, 3)[0]
    payload, want = check_compress(g, 0.2, 8)
    check_accumulate([payload] * 8, [want] * 8, n, zero_first=True)  # sequential float32 adds: within tolerance
    got, _ = check_accumulate([payload] * 2, [want] * 2, n, zero_first=True)
    one, _ = check_accumulate([payload], [want], n, zero_first=True)
    assert np.array_equal(got, 2 * one)  # v + v is exact
    twice, _ = check_accumulate([payload], [want], n, zero_first=False, dense_init=one)
    assert np.array_equal(twice, 2 * one)


@pytest.mark.parametrize("density", [0.0004, 0.05, 0.5])
def test_sparse_and_dense_tiles_in_accumulate_mode(density):
    # low density takes the touched-elements-only path, high density the staged path
    n, W = 200000, 3
    pt, po = [], []
    for w, g in enumerate(worker_grads(n, W, 77)):
        payload, want = check_compress(g, density, 8)
        pt.append(payload)
        po.append(want)
    rng = np.random.default_rng(1)
    check_accumulate(pt, po, n, zero_first=False, dense_init=rng.standard_normal(n).astype(np.float32))


def test_stress_style_payloads_with_overlap():
    n, k, W = 3_500_000, 175_000, 8
    pt, po = [], []
    for w in range(W):
        idx, codes, scales = synth.stress_payload_parts(n, k, 30 + w, shared_seed=99)
        p = oracle.Payload(n=n, k=k, bits=8, idx=idx, raw=oracle.dequantize_int8(codes, scales), codes=codes, scales=scales)
        po.append(p)
        pt.append(payload_to_device(p))
    overlap = np.intersect1d(po[0].idx, po[1].idx).size / k
    assert 0.2 < overlap < 0.4
    check_accumulate(pt, po, n, zero_first=True)


def test_empty_regions_and_last_tile():
    # all survivors sit in the last partial tile; every other tile is only zero-filled
    n = 3 * 8192 + 11
    g = np.zeros(n, dtype=np.float32)
    g[-7:] = np.arange(1, 8, dtype=np.float32)
    payload, want = check_compress(g, 7 / n, 16)
    got, _ = check_accumulate([payload], [want], n, zero_first=True)
    assert got[-7:].tolist() == [1, 2, 3, 4, 5, 6, 7] and not got[:-7].any()


def test_corrupt_payloads_are_reported():
    n = 20000
    g = worker_grads(n, 1, 5)[0]
    payload, want = check_compress(g, 0.1, 8)
    dense = torch.zeros(n, device="cuda")
    ws = nsml.alloc_bytes(nsml.nsml_accumulate_workspace_bytes(n, 1), "cuda")

    def run(p, size=n, d=dense):
        nsml.nsml_decompress_accumulate([p], d, zero_first=True, workspace=ws)
        return nsml.nsml_last_status(ws)

    assert run(payload) == 0
    bad = payload.clone()
    bad[0] ^= 0xFF  # magic
    assert run(bad) == nsml.NSML_ERR_PAYLOAD
    assert run(payload, d=torch.zeros(n + 1, device="cuda")) == nsml.NSML_ERR_PAYLOAD  # built for another n
    bad = payload.clone()
    bad[64:68] = torch.tensor([0xFF, 0xFF, 0xFF, 0x7F], dtype=torch.uint8, device="cuda")  # idx[0] far out of range
    canary = torch.zeros(n + 64, device="cuda")
    nsml.nsml_decompress_accumulate([bad], canary[:n], zero_first=True, workspace=ws)
    assert nsml.nsml_last_status(ws) == nsml.NSML_ERR_PAYLOAD  # reported, and never written out of range
    assert not canary[n:].any()
    assert run(payload) == 0  # workspace stays usable


def test_truncated_payload_is_refused_when_sizes_are_passed():
    n = 50000
    gs = worker_grads(n, 2, 9)
    p0, w0 = check_compress(gs[0], 0.05, 8)
    p1, w1 = check_compress(gs[1], 0.05, 16)
    ws = nsml.alloc_bytes(nsml.nsml_accumulate_workspace_bytes(n, 2), "cuda")
    dense = torch.full((n,), 5.0, device="cuda")
    # whole payloads with their sizes: the same sum as without sizes
    nsml.nsml_decompress_accumulate([p0, p1], dense, zero_first=True, workspace=ws, sized=True)
    assert nsml.nsml_last_status(ws) == 0
    assert np.array_equal(dense.cpu().numpy(), oracle.decompress_sum([w0, w1], n))
    # a buffer that ends before the payload its header describes: reported, its entries are not read
    cut = p0[: p0.numel() - 32].clone()
    nsml.nsml_decompress_accumulate([cut, p1], dense, zero_first=True, workspace=ws, sized=True)
    assert nsml.nsml_last_status(ws) == nsml.NSML_ERR_PAYLOAD
    assert np.array_equal(dense.cpu().numpy(), oracle.decompress_sum([w1], n))  # the intact worker's sum only
    # k corrupted upwards inside a buffer of the right size
    grown = p0.clone()
    grown[16:24] = torch.from_numpy(np.array([w0.k * 4], np.uint64).view(np.uint8)).cuda()
    nsml.nsml_decompress_accumulate([grown], dense, zero_first=True, workspace=ws, sized=True)
    assert nsml.nsml_last_status(ws) == nsml.NSML_ERR_PAYLOAD
    nsml.nsml_decompress_accumulate([p0, p1], dense, zero_first=True, workspace=ws, sized=True)
    assert nsml.nsml_last_status(ws) == 0


def test_host_buffer_variants():
    n = 123457
    g = worker_grads(n, 1, 21)[0]
    want = oracle.compress(g, 0.02, 8)
    grad_h = torch.from_numpy(g).pin_memory()
    need = nsml.nsml_payload_bytes(n, 0.02, 8)
    payload_h = torch.zeros(need, dtype=torch.uint8).pin_memory()
    scratch = nsml.alloc_bytes(nsml.lib.nsml_compress_host_scratch_bytes(n, 0, 0.02, 8), "cuda")
    nsml.nsml_compress_host(grad_h, 0.02, 8, payload_h, scratch)
    assert nsml.nsml_last_status(scratch) == 0
    from gpu_util import assert_payload_equal
    assert_payload_equal(payload_h, want)
    dense_h = torch.full((n,), 3.0).pin_memory()
    scratch2 = nsml.alloc_bytes(nsml.lib.nsml_accumulate_host_scratch_bytes(n, 2, 2 * need), "cuda")
    nsml.nsml_decompress_accumulate_host([payload_h, payload_h], dense_h, True, scratch2)
    assert nsml.nsml_last_status(scratch2) == 0
    assert np.array_equal(dense_h.numpy(), oracle.decompress_sum([want, want], n))


def test_host_variant_reports_a_truncated_payload():
    # the host-buffer variant passes the sizes it was given to the device check
    n = 40000
    g = worker_grads(n, 1, 33)[0]
    want = oracle.compress(g, 0.05, 8)
    raw = nsml.pack_payload(want.n, 8, want.idx, codes=want.codes, scales=want.scales)
    whole = torch.from_numpy(raw).pin_memory()
    cut = torch.from_numpy(raw[: raw.size - 48].copy()).pin_memory()
    dense_h = torch.zeros(n).pin_memory()
    scratch = nsml.alloc_bytes(nsml.lib.nsml_accumulate_host_scratch_bytes(n, 1, raw.size), "cuda")
    nsml.nsml_decompress_accumulate_host([cut], dense_h, True, scratch)
    assert nsml.nsml_last_status(scratch) == nsml.NSML_ERR_PAYLOAD
    assert not dense_h.numpy().any()  # nothing of the cut payload was added
    nsml.nsml_decompress_accumulate_host([whole], dense_h, True, scratch)
    assert nsml.nsml_last_status(scratch) == 0
    assert np.array_equal(dense_h.numpy(), oracle.decompress_sum([want], n))
