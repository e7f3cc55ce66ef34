"""nsml_decompress_accumulate_static: the entry point for callers that cannot
allocate device memory (its scratch is an array inside the library image).
Checked through the C ABI against nsml_decompress_accumulate on the same
payloads, twice in a row, because the array is shared by every call and keeps
the previous call's contents; against the CPU sum of CPU-built payloads; and
for leaving the device's free memory untouched.  Collected last on purpose."""
import ctypes

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2506_16235_b200 as nsml


def make_grads(n, W, seed):
    rng = np.random.default_rng(seed)
    return [(rng.standard_normal(n) * 10.0 ** rng.uniform(-3, -1, n)).astype(np.float32) for _ in range(W)]


def make_payloads(n, W, seed, ratio=0.03):
    ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(n), "cuda")
    out, max_abs = [], 0.0
    for w, g in enumerate(make_grads(n, W, seed)):
        max_abs = max(max_abs, float(np.abs(g).max()))
        bits = 8 if w % 2 == 0 else 16
        out.append(nsml.nsml_compress(torch.from_numpy(g).cuda(), ratio, bits, workspace=ws).clone())
        assert nsml.nsml_last_status(ws) == 0
    return out, max_abs


def reference_sum(payloads, n, zero_first, init):
    dense = init.clone()
    ws = nsml.alloc_bytes(nsml.nsml_accumulate_workspace_bytes(n, len(payloads)), "cuda")
    nsml.nsml_decompress_accumulate(payloads, dense, zero_first=zero_first, workspace=ws)
    assert nsml.nsml_last_status(ws) == 0
    return dense


def call_static(payloads, dense, zero_first):
    """Straight through the C ABI: pointers and sizes only."""
    W = len(payloads)
    ptrs = (ctypes.c_void_p * W)(*[p.data_ptr() for p in payloads])
    status = ctypes.c_int(-100)
    rc = nsml.lib.nsml_decompress_accumulate_static(ptrs, W, dense.data_ptr(), dense.numel(), int(zero_first),
                                                    torch.cuda.current_stream().cuda_stream, ctypes.byref(status))
    return rc, status.value


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    cases = [(1_000_003, 4, 11), (70_001, 8, 12)]  # the second call sees the first call's leftovers
    for n, W, seed in cases:
        payloads, max_abs = make_payloads(n, W, seed)
        init = torch.from_numpy(np.random.default_rng(seed).standard_normal(n).astype(np.float32)).cuda()
        for zero_first in (True, False):
            want = reference_sum(payloads, n, zero_first, init)
            got = init.clone()
            rc, status = call_static(payloads, got, zero_first)
            assert (rc, status) == (0, 0)
            err = (got.double() - want.double()).abs().max().item()
            assert err <= 1e-6 * max_abs  # the tolerance of the other accumulate tests
            assert torch.equal(got, want)  # and in fact bit-identical: same kernels, same order


def test_static_scratch_against_the_cpu_sum_and_without_allocating():
    # the payloads come from the CPU restatement of the compression, the expected sum from its plain
    # float64 sum: nothing of the CUDA path is on the expected side
    n, W, ratio = 300_007, 3, 0.02
    grads = make_grads(n, W, 21)
    wants = [oracle.compress(g, ratio, 8 if w % 2 == 0 else 16) for w, g in enumerate(grads)]
    payloads = [torch.from_numpy(nsml.pack_payload(p.n, p.bits, p.idx, codes=p.codes, scales=p.scales, half=p.half)).cuda()
                for p in wants]
    init = np.random.default_rng(5).standard_normal(n).astype(np.float32)
    tol = 1e-6 * max(float(np.abs(g).max()) for g in grads)
    got = torch.from_numpy(init.copy()).cuda()
    assert call_static(payloads, got, True) == (0, 0)  # also the set-up call: the array's address is known from here on
    err = np.abs(got.cpu().numpy().astype(np.float64) - oracle.decompress_sum(wants, n).astype(np.float64)).max()
    assert err <= tol
    # further calls leave the device's free memory as it is, also while per-kernel timing is switched on
    # (the static path never creates the events that timing uses)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    nsml.nsml_prof_enable(True)
    try:
        for zero_first in (False, True):  # accumulate on top of the first sum, then overwrite again
            assert call_static(payloads, got, zero_first) == (0, 0)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
    finally:
        nsml.nsml_prof_enable(False)
    want = oracle.decompress_sum(wants, n)  # the last call overwrote
    assert np.abs(got.cpu().numpy().astype(np.float64) - want.astype(np.float64)).max() <= tol


def test_static_scratch_limits_and_status():
    n = 10_000
    payloads, _ = make_payloads(n, 1, 3)
    dense = torch.zeros(n, device="cuda")
    ptrs = (ctypes.c_void_p * 9)(*([payloads[0].data_ptr()] * 9))
    stream = torch.cuda.current_stream().cuda_stream
    too_many = nsml.lib.nsml_decompress_accumulate_static(ptrs, 9, dense.data_ptr(), n, 1, stream, None)
    assert too_many == nsml.NSML_ERR_CAPACITY
    too_long = nsml.lib.nsml_decompress_accumulate_static(ptrs, 1, dense.data_ptr(), (1 << 24) + 1, 1, stream, None)
    assert too_long == nsml.NSML_ERR_CAPACITY
    assert "small" in nsml.nsml_strerror(too_long)
    # a corrupt payload is reported through status_out, and the next call starts clean
    bad = payloads[0].clone()
    bad[0] ^= 0xFF
    assert call_static([bad], dense, True) == (0, nsml.NSML_ERR_PAYLOAD)
    assert call_static(payloads, dense, True) == (0, 0)
    # asynchronous form through the binding
    assert nsml.nsml_decompress_accumulate_static(payloads, dense, zero_first=True) is None
    torch.cuda.synchronize()
    assert torch.equal(dense, reference_sum(payloads, n, True, torch.zeros(n, device="cuda")))
