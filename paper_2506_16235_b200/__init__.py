"""Python binding of libnsml (argument marshalling only).

Every operation runs in the CUDA library behind the C ABI declared in
include/nsml.h; this module converts tensors to pointers, allocates the
caller-owned buffers with torch when none are passed in, and turns status
codes into exceptions.  There is no CPU fallback: importing this module fails
if the library has not been built.

    import paper_2506_16235_b200 as nsml
    ctrl = nsml.Controller()
    ratio = ctrl.select_ratio(last_bytes, last_seconds, dense_bytes)
    payload = nsml.nsml_compress(grad, ratio, bits=8)
    nsml.nsml_decompress_accumulate([payload, ...], dense, zero_first=True)
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

NSML_OK = 0
NSML_ERR_ARG = -1
NSML_ERR_CAPACITY = -2
NSML_ERR_CUDA = -3
NSML_ERR_NONFINITE = -4
NSML_ERR_TIMEOUT = -5
NSML_ERR_PAYLOAD = -6
NSML_ERR_INTERNAL = -7
NSML_F32 = 0
NSML_BF16 = 1
NSML_BITS_INT8 = 8
NSML_BITS_FP16 = 16
NSML_BITS_FP32 = 32
NSML_QBLOCK = 1024
NSML_MAX_WORKERS = 64
NSML_PAYLOAD_MAGIC = 0x4C4D534E
HEADER_BYTES = 64


class NsmlError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {nsml_strerror(status)} (status {status})")


class CtrlParams(ctypes.Structure):
    _fields_ = [
        ("ratio_init", ctypes.c_double), ("ratio_min", ctypes.c_double), ("ratio_max", ctypes.c_double),
        ("alpha", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
        ("bdp_frac", ctypes.c_double), ("rtt_excess", ctypes.c_double),
        ("startup_max_steps", ctypes.c_int32), ("btlbw_window", ctypes.c_int32),
        ("rtprop_window", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]


class CtrlState(ctypes.Structure):
    _fields_ = [
        ("ratio", ctypes.c_double), ("ebb", ctypes.c_double), ("btlbw", ctypes.c_double),
        ("rtprop", ctypes.c_double), ("bdp", ctypes.c_double),
        ("phase", ctypes.c_int32), ("startup_steps", ctypes.c_int32), ("calls", ctypes.c_int64),
    ]


def _load() -> ctypes.CDLL:
    path = _build.LIB_PATH
    if _build.is_stale():
        # sources changed since the library was built (or it was never built):
        # rebuild when a compiler is at hand, otherwise use what is there
        try:
            _build.build()
        except RuntimeError:
            if not os.path.exists(path):
                raise
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2506_16235_b200.build` "
            "(needs nvcc; there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    vp, i64, dbl, sz, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_double, ctypes.c_size_t, ctypes.c_int
    sig = {
        "nsml_ctrl_default_params": (ci, [ctypes.POINTER(CtrlParams)]),
        "nsml_ctrl_create": (ci, [ctypes.POINTER(CtrlParams), ctypes.POINTER(vp)]),
        "nsml_ctrl_destroy": (None, [vp]),
        "nsml_select_ratio": (ci, [vp, dbl, dbl, dbl, ctypes.POINTER(dbl)]),
        "nsml_ctrl_get_state": (ci, [vp, ctypes.POINTER(CtrlState)]),
        "nsml_ctrl_save_bytes": (sz, [vp]),
        "nsml_ctrl_save": (ci, [vp, vp, sz]),
        "nsml_ctrl_load": (ci, [vp, vp, sz]),
        "nsml_k_of": (i64, [i64, dbl]),
        "nsml_compress_strategy": (ci, [i64, dbl]),
        "nsml_set_list_block_candidates": (ci, [ci]),
        "nsml_payload_bytes": (sz, [i64, dbl, ci]),
        "nsml_workspace_bytes": (sz, [i64, ci]),
        "nsml_accumulate_workspace_bytes": (sz, [i64, ci]),
        "nsml_compress": (ci, [vp, i64, ci, dbl, ci, vp, vp, sz, vp, sz, vp]),
        "nsml_decompress_accumulate": (ci, [ctypes.POINTER(vp), ci, vp, i64, ci, vp, sz, vp]),
        "nsml_decompress_accumulate_sized": (ci, [ctypes.POINTER(vp), ctypes.POINTER(sz), ci, vp, i64, ci, vp, sz, vp]),
        "nsml_decompress_accumulate_static": (ci, [ctypes.POINTER(vp), ci, vp, i64, ci, vp, ctypes.POINTER(ci)]),
        "nsml_compress_host_scratch_bytes": (sz, [i64, ci, dbl, ci]),
        "nsml_compress_host": (ci, [vp, i64, ci, dbl, ci, vp, vp, sz, vp, sz, vp]),
        "nsml_accumulate_host_scratch_bytes": (sz, [i64, ci, sz]),
        "nsml_decompress_accumulate_host": (ci, [ctypes.POINTER(vp), ctypes.POINTER(sz), ci, vp, i64, ci, vp, sz, vp]),
        "nsml_l2_workspace_bytes": (sz, []),
        "nsml_grad_l2": (ci, [vp, i64, ci, vp, sz, vp, ctypes.POINTER(dbl)]),
        "nsml_quantize_gate": (ci, [dbl, dbl, dbl, dbl, ci, ctypes.POINTER(dbl), ctypes.POINTER(ci)]),
        "nsml_pruned_count": (i64, [i64, dbl]),
        "nsml_prune_workspace_bytes": (sz, [i64]),
        "nsml_prune_mask_build": (ci, [vp, i64, dbl, vp, vp, sz, vp]),
        "nsml_compress_feedback": (ci, [vp, vp, i64, ci, dbl, ci, vp, vp, sz, vp, sz, vp]),
        "nsml_adaptive_payload_bytes": (sz, [i64, dbl, dbl, ci]),
        "nsml_adaptive_workspace_bytes": (sz, [i64, ci]),
        "nsml_compress_adaptive": (ci, [vp, i64, ci, dbl, dbl, dbl, ci, vp, vp, vp, sz, vp, sz, vp,
                                        ctypes.POINTER(dbl), ctypes.POINTER(ci), ctypes.POINTER(dbl)]),
        "nsml_selftest_bounded_wait": (ci, [vp, sz, ci, vp]),
        "nsml_last_status": (ci, [vp, vp, ctypes.POINTER(ci)]),
        "nsml_strerror": (ctypes.c_char_p, [ci]),
        "nsml_kernel_count": (ci, []),
        "nsml_kernel_name": (ctypes.c_char_p, [ci]),
        "nsml_launch_count": (i64, []),
        "nsml_prof_enable": (ci, [ci]),
        "nsml_prof_read": (ci, [ci, ctypes.POINTER(dbl), ctypes.POINTER(i64)]),
        "nsml_prof_reset": (ci, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


lib = _load()


def nsml_strerror(status: int) -> str:
    return lib.nsml_strerror(int(status)).decode()


def _check(rc: int, where: str) -> None:
    if rc != NSML_OK:
        raise NsmlError(rc, where)


# --------------------------------------------------------------------------
# controller (host)
# --------------------------------------------------------------------------
def default_params() -> CtrlParams:
    p = CtrlParams()
    _check(lib.nsml_ctrl_default_params(ctypes.byref(p)), "nsml_ctrl_default_params")
    return p


class Controller:
    """Owns one nsml_ctrl.  Keyword arguments override nsml_ctrl_params fields."""

    def __init__(self, **overrides):
        p = default_params()
        for key, val in overrides.items():
            if not hasattr(p, key):
                raise TypeError(f"unknown controller parameter {key!r}")
            setattr(p, key, val)
        self._h = ctypes.c_void_p()
        _check(lib.nsml_ctrl_create(ctypes.byref(p), ctypes.byref(self._h)), "nsml_ctrl_create")

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            lib.nsml_ctrl_destroy(h)

    def select_ratio(self, last_bytes: float, last_seconds: float, next_dense_bytes: float) -> float:
        return nsml_select_ratio(self, last_bytes, last_seconds, next_dense_bytes)

    def state(self) -> CtrlState:
        s = CtrlState()
        _check(lib.nsml_ctrl_get_state(self._h, ctypes.byref(s)), "nsml_ctrl_get_state")
        return s

    def save(self) -> bytes:
        nbytes = lib.nsml_ctrl_save_bytes(self._h)
        buf = ctypes.create_string_buffer(nbytes)
        _check(lib.nsml_ctrl_save(self._h, buf, nbytes), "nsml_ctrl_save")
        return buf.raw

    def load(self, blob: bytes) -> None:
        buf = ctypes.create_string_buffer(bytes(blob), len(blob))
        _check(lib.nsml_ctrl_load(self._h, buf, len(blob)), "nsml_ctrl_load")


def nsml_select_ratio(ctrl: Controller, last_bytes: float, last_seconds: float, next_dense_bytes: float) -> float:
    out = ctypes.c_double()
    _check(lib.nsml_select_ratio(ctrl._h, float(last_bytes), float(last_seconds), float(next_dense_bytes),
                                 ctypes.byref(out)), "nsml_select_ratio")
    return out.value


# --------------------------------------------------------------------------
# sizes
# --------------------------------------------------------------------------
def nsml_k_of(n: int, ratio: float) -> int:
    return int(lib.nsml_k_of(int(n), float(ratio)))


def nsml_set_list_block_candidates(candidates: int) -> None:
    """Tuning knob of the list stage (1024 ... 8192, default 4096); the results do not depend on it."""
    _check(lib.nsml_set_list_block_candidates(int(candidates)), "nsml_set_list_block_candidates")


def nsml_compress_strategy(n: int, ratio: float) -> int:
    """0 = sampled candidate list, 1 = dense select over the bucket (current device)."""
    rc = int(lib.nsml_compress_strategy(int(n), float(ratio)))
    if rc < 0:
        raise NsmlError(rc, "nsml_compress_strategy")
    return rc


def nsml_payload_bytes(n: int, ratio: float, bits: int) -> int:
    return int(lib.nsml_payload_bytes(int(n), float(ratio), int(bits)))


def nsml_workspace_bytes(n: int, grad_dtype: int = NSML_F32) -> int:
    return int(lib.nsml_workspace_bytes(int(n), int(grad_dtype)))


def nsml_accumulate_workspace_bytes(n: int, W: int) -> int:
    return int(lib.nsml_accumulate_workspace_bytes(int(n), int(W)))


# --------------------------------------------------------------------------
# device operations
# --------------------------------------------------------------------------
def _torch():
    import torch

    return torch


def _stream_ptr(stream) -> int:
    torch = _torch()
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _grad_dtype(t) -> int:
    torch = _torch()
    if t.dtype == torch.float32:
        return NSML_F32
    if t.dtype == torch.bfloat16:
        return NSML_BF16
    raise TypeError("gradient bucket must be float32 or bfloat16")


def alloc_bytes(nbytes: int, device):
    """Caller-owned device scratch (256-byte aligned by the torch allocator)."""
    torch = _torch()
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def nsml_compress(grad, ratio: float, bits: int = NSML_BITS_INT8, prune_mask=None, payload=None,
                  workspace=None, stream=None):
    """Compress one flat bucket on its device; returns the payload (uint8 tensor).

    grad: contiguous 1-D float32 / bfloat16 CUDA tensor.  prune_mask: int32
    CUDA tensor of ceil(n/32) words (bit set = pruned) or None.  payload /
    workspace: optional preallocated uint8 CUDA tensors.  Asynchronous on
    `stream` (default: torch's current stream).
    """
    if not (grad.is_cuda and grad.is_contiguous() and grad.dim() == 1):
        raise ValueError("grad must be a contiguous 1-D CUDA tensor")
    n = grad.numel()
    dtype = _grad_dtype(grad)
    need = nsml_payload_bytes(n, ratio, bits)
    if need == 0:
        raise NsmlError(NSML_ERR_ARG, "nsml_compress")
    if payload is None:
        payload = alloc_bytes(need, grad.device)
    if workspace is None:
        workspace = alloc_bytes(nsml_workspace_bytes(n, dtype), grad.device)
    mask_ptr = None
    if prune_mask is not None:
        if not (prune_mask.is_cuda and prune_mask.is_contiguous() and prune_mask.element_size() == 4
                and prune_mask.numel() >= (n + 31) // 32):
            raise ValueError("prune_mask must be a contiguous CUDA tensor of ceil(n/32) 32-bit words")
        mask_ptr = prune_mask.data_ptr()
    rc = lib.nsml_compress(grad.data_ptr(), n, dtype, float(ratio), int(bits), mask_ptr,
                           payload.data_ptr(), payload.numel(), workspace.data_ptr(), workspace.numel(),
                           _stream_ptr(stream))
    _check(rc, "nsml_compress")
    return payload[:need]


def nsml_decompress_accumulate(payloads: Sequence, dense, zero_first: bool = True, workspace=None, stream=None,
                               sized: bool = False):
    """dense (float32 CUDA tensor, n elements) = (0 or dense) + sum of the payloads.
    sized=True passes each payload tensor's size in bytes along, so that a
    truncated payload is refused on the device."""
    W = len(payloads)
    if not (dense.is_cuda and dense.is_contiguous() and dense.dim() == 1):
        raise ValueError("dense must be a contiguous 1-D CUDA float32 tensor")
    torch = _torch()
    if dense.dtype != torch.float32:
        raise TypeError("dense must be float32")
    n = dense.numel()
    if workspace is None:
        workspace = alloc_bytes(nsml_accumulate_workspace_bytes(n, max(1, min(W, NSML_MAX_WORKERS))), dense.device)
    ptrs = (ctypes.c_void_p * max(W, 1))(*[p.data_ptr() for p in payloads])
    if sized:
        sizes = (ctypes.c_size_t * max(W, 1))(*[p.numel() * p.element_size() for p in payloads])
        rc = lib.nsml_decompress_accumulate_sized(ptrs, sizes, W, dense.data_ptr(), n, 1 if zero_first else 0,
                                                  workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    else:
        rc = lib.nsml_decompress_accumulate(ptrs, W, dense.data_ptr(), n, 1 if zero_first else 0,
                                            workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "nsml_decompress_accumulate")
    return dense


NSML_STATIC_MAX_N = 1 << 24
NSML_STATIC_MAX_WORKERS = 8


def nsml_decompress_accumulate_static(payloads: Sequence, dense, zero_first: bool = True, stream=None,
                                      want_status: bool = False):
    """nsml_decompress_accumulate without a workspace argument: the scratch is
    an array inside the library (for callers that cannot allocate device
    memory).  Limited to n <= NSML_STATIC_MAX_N and W <= NSML_STATIC_MAX_WORKERS;
    calls on one device must not overlap.  With want_status the call
    synchronises the stream and returns the device-detected status."""
    W = len(payloads)
    ptrs = (ctypes.c_void_p * max(W, 1))(*[p.data_ptr() for p in payloads])
    status = ctypes.c_int(0)
    rc = lib.nsml_decompress_accumulate_static(ptrs, W, dense.data_ptr(), dense.numel(), 1 if zero_first else 0,
                                               _stream_ptr(stream), ctypes.byref(status) if want_status else None)
    _check(rc, "nsml_decompress_accumulate_static")
    return status.value if want_status else None


def _check_bucket(t, what="grad"):
    if not (t.is_cuda and t.is_contiguous() and t.dim() == 1):
        raise ValueError(f"{what} must be a contiguous 1-D CUDA tensor")


def nsml_grad_l2(grad, workspace=None, stream=None, sync: bool = True):
    """L2 norm of a bucket (Alg. 2 Step 1), float64.  sync=True synchronises the
    stream and returns the norm; sync=False only enqueues (the float64 sum of
    squares is then left at byte offset 8 of `workspace`) and returns None."""
    _check_bucket(grad)
    if workspace is None:
        workspace = alloc_bytes(lib.nsml_l2_workspace_bytes(), grad.device)
    out = ctypes.c_double()
    rc = lib.nsml_grad_l2(grad.data_ptr(), grad.numel(), _grad_dtype(grad), workspace.data_ptr(), workspace.numel(),
                          _stream_ptr(stream), ctypes.byref(out) if sync else None)
    _check(rc, "nsml_grad_l2")
    return out.value if sync else None


def nsml_quantize_gate(ratio: float, l2: float, tr_q: float, tr_d: float, plain_bits: int = NSML_BITS_FP32):
    """Alg. 2 Step 1 decision: (ratio to use, value codec to use)."""
    r, b = ctypes.c_double(), ctypes.c_int()
    _check(lib.nsml_quantize_gate(float(ratio), float(l2), float(tr_q), float(tr_d), int(plain_bits),
                                  ctypes.byref(r), ctypes.byref(b)), "nsml_quantize_gate")
    return r.value, b.value


def nsml_pruned_count(n: int, ratio: float) -> int:
    return int(lib.nsml_pruned_count(int(n), float(ratio)))


def nsml_prune_workspace_bytes(n: int) -> int:
    return int(lib.nsml_prune_workspace_bytes(int(n)))


def nsml_prune_mask_build(weights, ratio: float, prune_mask=None, workspace=None, stream=None):
    """Pruning mask from the weights (Alg. 2 Step 2): int32 CUDA tensor of ceil(n/32) words."""
    _check_bucket(weights, "weights")
    torch = _torch()
    if weights.dtype != torch.float32:
        raise TypeError("weights must be float32")
    n = weights.numel()
    if prune_mask is None:
        prune_mask = torch.empty((n + 31) // 32, dtype=torch.int32, device=weights.device)
    if workspace is None:
        workspace = alloc_bytes(nsml_prune_workspace_bytes(n), weights.device)
    rc = lib.nsml_prune_mask_build(weights.data_ptr(), n, float(ratio), prune_mask.data_ptr(), workspace.data_ptr(),
                                   workspace.numel(), _stream_ptr(stream))
    _check(rc, "nsml_prune_mask_build")
    return prune_mask


def nsml_compress_feedback(grad, residual, ratio: float, bits: int = NSML_BITS_INT8, prune_mask=None, payload=None,
                           workspace=None, stream=None):
    """nsml_compress of grad + residual; residual (float32 CUDA tensor) is updated in place."""
    _check_bucket(grad)
    _check_bucket(residual, "residual")
    torch = _torch()
    n = grad.numel()
    if residual.dtype != torch.float32 or residual.numel() != n:
        raise ValueError("residual must be float32 with one element per gradient element")
    need = nsml_payload_bytes(n, ratio, bits)
    if need == 0:
        raise NsmlError(NSML_ERR_ARG, "nsml_compress_feedback")
    if payload is None:
        payload = alloc_bytes(need, grad.device)
    if workspace is None:
        workspace = alloc_bytes(nsml_workspace_bytes(n, NSML_F32), grad.device)
    rc = lib.nsml_compress_feedback(grad.data_ptr(), residual.data_ptr(), n, _grad_dtype(grad), float(ratio), int(bits),
                                    None if prune_mask is None else prune_mask.data_ptr(), payload.data_ptr(),
                                    payload.numel(), workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "nsml_compress_feedback")
    return payload[:need]


def nsml_compress_adaptive(grad, ratio: float, tr_q: float, tr_d: float, plain_bits: int = NSML_BITS_FP32,
                           weights=None, prune_mask=None, payload=None, workspace=None, stream=None):
    """Alg. 2 as a whole.  Returns (payload, ratio used, bits used, L2 norm or None, prune mask or None)."""
    _check_bucket(grad)
    torch = _torch()
    n = grad.numel()
    dtype = _grad_dtype(grad)
    cap = int(lib.nsml_adaptive_payload_bytes(n, float(ratio), float(tr_q), int(plain_bits)))
    if cap == 0:
        raise NsmlError(NSML_ERR_ARG, "nsml_compress_adaptive")
    if payload is None:
        payload = alloc_bytes(cap, grad.device)
    if workspace is None:
        workspace = alloc_bytes(int(lib.nsml_adaptive_workspace_bytes(n, dtype)), grad.device)
    if weights is not None and prune_mask is None:
        prune_mask = torch.empty((n + 31) // 32, dtype=torch.int32, device=grad.device)
    r, b, l2 = ctypes.c_double(), ctypes.c_int(), ctypes.c_double()
    rc = lib.nsml_compress_adaptive(grad.data_ptr(), n, dtype, float(ratio), float(tr_q), float(tr_d), int(plain_bits),
                                    None if weights is None else weights.data_ptr(),
                                    None if prune_mask is None else prune_mask.data_ptr(),
                                    payload.data_ptr(), payload.numel(), workspace.data_ptr(), workspace.numel(),
                                    _stream_ptr(stream), ctypes.byref(r), ctypes.byref(b), ctypes.byref(l2))
    _check(rc, "nsml_compress_adaptive")
    need = nsml_payload_bytes(n, r.value, b.value)
    return payload[:need], r.value, b.value, (l2.value if l2.value >= 0.0 else None), prune_mask


def nsml_last_status(workspace, stream=None) -> int:
    out = ctypes.c_int()
    _check(lib.nsml_last_status(workspace.data_ptr(), _stream_ptr(stream), ctypes.byref(out)), "nsml_last_status")
    return out.value


def nsml_compress_host(grad_host, ratio: float, bits: int, payload_host, device_scratch, prune_mask_host=None,
                       stream=None) -> int:
    """Host-buffer compress: grad_host / payload_host are CPU tensors (pinned for
    asynchronous copies), device_scratch a uint8 CUDA tensor.  Returns the payload size."""
    n = grad_host.numel()
    dtype = _grad_dtype(grad_host)
    need = nsml_payload_bytes(n, ratio, bits)
    rc = lib.nsml_compress_host(grad_host.data_ptr(), n, dtype, float(ratio), int(bits),
                                None if prune_mask_host is None else prune_mask_host.data_ptr(),
                                payload_host.data_ptr(), payload_host.numel(),
                                device_scratch.data_ptr(), device_scratch.numel(), _stream_ptr(stream))
    _check(rc, "nsml_compress_host")
    return need


def nsml_decompress_accumulate_host(payloads_host: Sequence, dense_host, zero_first: bool, device_scratch,
                                    stream=None):
    W = len(payloads_host)
    ptrs = (ctypes.c_void_p * max(W, 1))(*[p.data_ptr() for p in payloads_host])
    sizes = (ctypes.c_size_t * max(W, 1))(*[p.numel() * p.element_size() for p in payloads_host])
    rc = lib.nsml_decompress_accumulate_host(ptrs, sizes, W, dense_host.data_ptr(), dense_host.numel(),
                                             1 if zero_first else 0, device_scratch.data_ptr(),
                                             device_scratch.numel(), _stream_ptr(stream))
    _check(rc, "nsml_decompress_accumulate_host")
    return dense_host


# --------------------------------------------------------------------------
# payload layout helpers (byte layout only; no arithmetic on the values)
# --------------------------------------------------------------------------
def _align16(x: int) -> int:
    return (x + 15) // 16 * 16


def unpack_payload(payload) -> dict:
    """Split a payload (CUDA/CPU uint8 tensor, bytes or uint8 ndarray) into its
    sections as numpy arrays: n, k, bits, idx, and codes+scales, half or f32."""
    if hasattr(payload, "detach"):
        raw = payload.detach().cpu().numpy()
    else:
        raw = np.frombuffer(bytes(payload), dtype=np.uint8) if not isinstance(payload, np.ndarray) else payload
    raw = np.ascontiguousarray(raw, dtype=np.uint8)
    magic, version = (int(x) for x in raw[0:8].view(np.uint32))
    n, k = (int(x) for x in raw[8:24].view(np.uint64))
    bits, qblock = (int(x) for x in raw[24:32].view(np.uint32))
    nblocks, idx_off, val_off, scale_off = (int(x) for x in raw[32:64].view(np.uint64))
    out = dict(magic=magic, version=version, n=n, k=k, bits=bits, qblock=qblock, nblocks=nblocks,
               idx_off=idx_off, val_off=val_off, scale_off=scale_off)
    out["idx"] = raw[idx_off:idx_off + 4 * k].view(np.uint32).copy()
    if bits == NSML_BITS_INT8:
        out["codes"] = raw[val_off:val_off + k].view(np.int8).copy()
        out["scales"] = raw[scale_off:scale_off + 4 * nblocks].view(np.float32).copy()
    elif bits == NSML_BITS_FP16:
        out["half"] = raw[val_off:val_off + 2 * k].view(np.uint16).copy()
    else:
        out["f32"] = raw[val_off:val_off + 4 * k].view(np.float32).copy()
    return out


def pack_payload(n: int, bits: int, idx, codes=None, scales=None, half=None, f32=None) -> np.ndarray:
    """Lay out payload sections as nsml_compress would (uint8 ndarray)."""
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    k = idx.size
    val_off = HEADER_BYTES + _align16(4 * k)
    if bits == NSML_BITS_INT8:
        nblocks = (k + NSML_QBLOCK - 1) // NSML_QBLOCK
        scale_off = val_off + _align16(k)
        total = scale_off + _align16(4 * nblocks)
    else:
        nblocks, scale_off = 0, 0
        total = val_off + _align16((4 if bits == NSML_BITS_FP32 else 2) * k)
    raw = np.zeros(total, dtype=np.uint8)
    raw[0:8].view(np.uint32)[:] = (NSML_PAYLOAD_MAGIC, 1)
    raw[8:24].view(np.uint64)[:] = (n, k)
    raw[24:32].view(np.uint32)[:] = (bits, NSML_QBLOCK)
    raw[32:64].view(np.uint64)[:] = (nblocks, HEADER_BYTES, val_off, scale_off)
    raw[HEADER_BYTES:HEADER_BYTES + 4 * k] = idx.view(np.uint8)
    if bits == NSML_BITS_INT8:
        raw[val_off:val_off + k] = np.ascontiguousarray(codes, dtype=np.int8).view(np.uint8)
        raw[scale_off:scale_off + 4 * nblocks] = np.ascontiguousarray(scales, dtype=np.float32).view(np.uint8)
    elif bits == NSML_BITS_FP16:
        raw[val_off:val_off + 2 * k] = np.ascontiguousarray(half, dtype=np.uint16).view(np.uint8)
    else:
        raw[val_off:val_off + 4 * k] = np.ascontiguousarray(f32, dtype=np.float32).view(np.uint8)
    return raw


# --------------------------------------------------------------------------
# instrumentation
# --------------------------------------------------------------------------
def kernel_names() -> List[str]:
    return [lib.nsml_kernel_name(i).decode() for i in range(lib.nsml_kernel_count())]


def nsml_launch_count() -> int:
    return int(lib.nsml_launch_count())


def nsml_prof_enable(on: bool) -> None:
    _check(lib.nsml_prof_enable(1 if on else 0), "nsml_prof_enable")


def nsml_prof_reset() -> None:
    _check(lib.nsml_prof_reset(), "nsml_prof_reset")


def nsml_prof_read() -> dict:
    """{kernel name: (total device ms, launches)} since the last reset."""
    out = {}
    for i, name in enumerate(kernel_names()):
        ms, cnt = ctypes.c_double(), ctypes.c_int64()
        _check(lib.nsml_prof_read(i, ctypes.byref(ms), ctypes.byref(cnt)), "nsml_prof_read")
        out[name] = (ms.value, cnt.value)
    return out
