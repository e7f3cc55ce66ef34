"""Helpers shared by the GPU parity tests: run the CUDA path through the
binding and compare it with the CPU oracle element by element."""
import numpy as np
import torch

import oracle
import paper_2506_16235_b200 as nsml

CANARY = 0xA5


def mask_words(mask_bool: np.ndarray) -> np.ndarray:
    """Pack a boolean prune mask into the library's bit layout (bit i&31 of word i>>5)."""
    n = mask_bool.size
    padded = np.zeros((n + 31) // 32 * 32, dtype=np.uint8)
    padded[:n] = mask_bool
    return np.packbits(padded.reshape(-1, 32), axis=1, bitorder="little").view(np.uint32).reshape(-1).copy()


def to_device_grad(g: np.ndarray) -> torch.Tensor:
    if g.dtype == np.uint16:  # bf16 bit patterns
        return torch.from_numpy(g.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(g, dtype=np.float32)).cuda()


def gpu_compress(g: np.ndarray, ratio: float, bits: int, mask_bool=None, check_canary=True):
    grad = to_device_grad(g)
    n = grad.numel()
    need = nsml.nsml_payload_bytes(n, ratio, bits)
    buf = torch.full((need + 256,), CANARY, dtype=torch.uint8, device="cuda")
    ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(n, nsml.NSML_BF16 if g.dtype == np.uint16 else nsml.NSML_F32), "cuda")
    mw = None
    if mask_bool is not None:
        mw = torch.from_numpy(mask_words(mask_bool).view(np.int32)).cuda()
    payload = nsml.nsml_compress(grad, ratio, bits, prune_mask=mw, payload=buf, workspace=ws)
    status = nsml.nsml_last_status(ws)
    if check_canary:
        assert bool((buf[need:] == CANARY).all()), "wrote past the end of the payload"
    return payload, status


def oracle_compress(g: np.ndarray, ratio: float, bits: int, mask_bool=None) -> oracle.Payload:
    vals = oracle.widen_bf16(g) if g.dtype == np.uint16 else g
    return oracle.compress(vals, ratio, bits, prune_mask=mask_bool)


def assert_payload_equal(payload, want: oracle.Payload):
    got = nsml.unpack_payload(payload)
    assert got["magic"] == nsml.NSML_PAYLOAD_MAGIC and got["version"] == 1
    assert (got["n"], got["k"], got["bits"], got["qblock"]) == (want.n, want.k, want.bits, 1024)
    assert np.array_equal(got["idx"], want.idx), "selected index set differs"
    if want.bits == 8:
        assert np.array_equal(got["scales"].view(np.uint32), want.scales.view(np.uint32)), "scales differ"
        assert np.array_equal(got["codes"], want.codes), "int8 codes differ"
    elif want.bits == 16:
        assert np.array_equal(got["half"], want.half), "fp16 bit patterns differ"
    else:
        assert np.array_equal(got["f32"].view(np.uint32), want.raw.view(np.uint32)), "float32 values differ"
    return got


def check_compress(g, ratio, bits, mask_bool=None):
    payload, status = gpu_compress(g, ratio, bits, mask_bool)
    assert status == 0, nsml.nsml_strerror(status)
    want = oracle_compress(g, ratio, bits, mask_bool)
    assert_payload_equal(payload, want)
    return payload, want


def payload_to_device(want: oracle.Payload) -> torch.Tensor:
    raw = nsml.pack_payload(want.n, want.bits, want.idx, codes=want.codes, scales=want.scales, half=want.half,
                            f32=want.raw if want.bits == 32 else None)
    return torch.from_numpy(raw).cuda()


def check_accumulate(payload_tensors, oracle_payloads, n, zero_first, dense_init=None, max_abs=None):
    """GPU sum vs oracle: within 1e-6 of the bucket's largest magnitude."""
    if dense_init is None:
        dense_init = np.full(n, 7.0, dtype=np.float32) if zero_first else np.zeros(n, dtype=np.float32)
    dense = torch.from_numpy(dense_init.copy()).cuda()
    ws = nsml.alloc_bytes(nsml.nsml_accumulate_workspace_bytes(n, len(payload_tensors)), "cuda")
    nsml.nsml_decompress_accumulate(payload_tensors, dense, zero_first=zero_first, workspace=ws)
    status = nsml.nsml_last_status(ws)
    assert status == 0, nsml.nsml_strerror(status)
    want = oracle.decompress_sum(oracle_payloads, n, dense_in=None if zero_first else dense_init)
    got = dense.cpu().numpy()
    if max_abs is None:
        max_abs = max([float(np.max(np.abs(p.raw))) if p.raw.size else 0.0 for p in oracle_payloads] +
                      [0.0 if zero_first else float(np.max(np.abs(dense_init)))])
    tol = 1e-6 * max_abs
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    assert float(err.max()) <= tol, f"max error {err.max()} > {tol}"
    return got, want
