"""Oracle for bucket compression and multi-worker decompress-sum.

TEST INFRASTRUCTURE ONLY (see the package docstring).

What is computed, and where the paper states it:

* Alg. 2 Step 2: gradients of pruned parameters are set to zero *before*
  sparsification.  Here the pruned set arrives as a boolean mask.
* Alg. 2 Step 3: top-k sparsification by absolute value at the given ratio
  (ratio = kept fraction).  The paper gives only "top_k(grads, ratio)"; the
  readings taken here are k = ceil(ratio * n) evaluated in IEEE double,
  ties broken by larger |g| first and then lower index, and a payload
  ordered by ascending index.  Exactly k entries survive even when fewer
  than k gradients are non-zero (zeros fill up by lowest index).
* Alg. 2 Step 1 "quantize": 32-bit to 16-bit floating point, round to
  nearest even; magnitudes that would round to infinity saturate to the
  largest finite half (65504).  The int8 codec (symmetric, one max-abs scale
  per block of 1024 consecutive survivors) is an addition to the paper.
  When Step 1 does not quantise, the survivors travel as the 32-bit floats
  they are (bits = 32).
* Section 4.2 Step 3 / Section 5.3: every worker receives all workers'
  sparse payloads (AllGather pattern) and sums them into a dense gradient.
  The sum is a plain sum (no averaging), taken in fp64 and rounded once.

The selection is written as its plain definition: a full sort of all n
elements on (magnitude bits descending, index ascending).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

QBLOCK = 1024  # survivors per int8 scale block, in payload order

_ABS_MASK = np.uint32(0x7FFFFFFF)
_INF_BITS = 0x7F800000


class NonFiniteGradient(ValueError):
    """Raised when a bucket holds NaN or +-Inf (inputs must be finite)."""


def k_of(ratio: float, n: int) -> int:
    """Number of survivors: ceil(ratio * n) in IEEE double, clamped to [1, n].

    The product is formed in double exactly as written, so that for instance
    ratio 0.07 and n 100 give 8 (the double product is slightly above 7).
    """
    if not (isinstance(n, (int, np.integer)) and n >= 1):
        raise ValueError("n must be a positive integer")
    ratio = float(ratio)
    if not (ratio > 0.0 and ratio <= 1.0):
        raise ValueError("ratio must lie in (0, 1]")
    k = int(math.ceil(ratio * float(n)))
    return max(1, min(int(n), k))


def widen_bf16(bits16: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> the exactly equal float32 values."""
    b = np.ascontiguousarray(bits16, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def keys_of(values: np.ndarray) -> np.ndarray:
    """Magnitude keys: the float32 bit pattern with the sign bit cleared.

    For finite floats (denormals and both zeros included) unsigned integer
    order of the key equals the order of |g|.
    """
    v = np.ascontiguousarray(values, dtype=np.float32)
    return v.view(np.uint32) & _ABS_MASK


def _apply_mask(grad: np.ndarray, prune_mask: Optional[np.ndarray]) -> np.ndarray:
    g = np.ascontiguousarray(grad, dtype=np.float32)
    if prune_mask is None:
        return g
    m = np.asarray(prune_mask, dtype=bool)
    if m.shape != g.shape:
        raise ValueError("prune_mask must have one flag per gradient element")
    v = g.copy()
    v[m] = np.float32(0.0)  # pruned gradients become +0.0 (Alg. 2 Step 2)
    return v


def select_topk(values: np.ndarray, k: int) -> np.ndarray:
    """Indices (ascending, uint32) of the k largest-magnitude elements.

    Full sort on (key descending, index ascending); the first k entries of
    that order are the survivors.  The composite sort key is the pair packed
    into one unsigned 64-bit integer: high word = (0x7FFFFFFF - key), so that
    ascending order of the word is descending order of the magnitude, low
    word = index.
    """
    key = keys_of(values)
    n = key.size
    if n >= 2**32:
        raise ValueError("n must be below 2**32")
    if not (1 <= k <= n):
        raise ValueError("k out of range")
    if key.size and int(key.max()) >= _INF_BITS:
        raise NonFiniteGradient("bucket holds NaN or Inf")
    hi = (np.uint64(0x7FFFFFFF) - key.astype(np.uint64)) << np.uint64(32)
    packed = hi | np.arange(n, dtype=np.uint64)
    packed.sort()  # the full sort
    survivors = (packed[:k] & np.uint64(0xFFFFFFFF)).astype(np.uint32)
    survivors.sort()  # payload order = ascending index
    return survivors


def select_topk_many(values: np.ndarray, ks: Sequence[int]):
    """select_topk for several k on the same bucket: the same full sort on
    (key descending, index ascending), taken once; the survivors for each k
    are the first k entries of that one order.  Returns a list of ascending
    uint32 index arrays, one per k."""
    key = keys_of(values)
    n = key.size
    if n >= 2**32:
        raise ValueError("n must be below 2**32")
    if any(not (1 <= int(k) <= n) for k in ks):
        raise ValueError("k out of range")
    if key.size and int(key.max()) >= _INF_BITS:
        raise NonFiniteGradient("bucket holds NaN or Inf")
    hi = (np.uint64(0x7FFFFFFF) - key.astype(np.uint64)) << np.uint64(32)
    packed = hi | np.arange(n, dtype=np.uint64)
    packed.sort()  # the full sort
    out = []
    for k in ks:
        survivors = (packed[: int(k)] & np.uint64(0xFFFFFFFF)).astype(np.uint32)
        survivors.sort()  # payload order = ascending index
        out.append(survivors)
    return out


def quantize_int8(val: np.ndarray):
    """Symmetric int8 codes with one max-abs scale per QBLOCK survivors.

    Per block: scale = maxabs / 127 (one IEEE float32 division); if the scale
    is zero every code is zero, otherwise code = clamp(rint(v / scale), +-127)
    with one IEEE float32 division and round-half-to-even.  Denormals are
    honoured (no flush to zero).  Written as a scalar loop over blocks.
    """
    v = np.ascontiguousarray(val, dtype=np.float32)
    k = v.size
    nblocks = (k + QBLOCK - 1) // QBLOCK
    codes = np.zeros(k, dtype=np.int8)
    scales = np.zeros(nblocks, dtype=np.float32)
    f127 = np.float32(127.0)
    with np.errstate(under="ignore", divide="ignore", invalid="ignore"):
        for b in range(nblocks):
            blk = v[b * QBLOCK:(b + 1) * QBLOCK]
            maxabs = np.float32(np.max(np.abs(blk)))
            scale = np.float32(maxabs / f127)
            scales[b] = scale
            if scale == np.float32(0.0):
                continue
            q = np.rint((blk / scale).astype(np.float32))
            q = np.clip(q, -127.0, 127.0)
            codes[b * QBLOCK:(b + 1) * QBLOCK] = q.astype(np.int8)
    return codes, scales


def dequantize_int8(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """v' = float(code) * scale of its block: one float32 multiply each."""
    c = np.ascontiguousarray(codes, dtype=np.int8)
    s = np.ascontiguousarray(scales, dtype=np.float32)
    per_entry = np.repeat(s, QBLOCK)[: c.size]
    with np.errstate(under="ignore"):
        return (c.astype(np.float32) * per_entry).astype(np.float32)


def f32_to_f16_bits(val: np.ndarray) -> np.ndarray:
    """float32 -> IEEE binary16 bit patterns, round to nearest even, with
    saturation: |v| >= 65520 (which a plain cast would round to infinity)
    becomes +-65504.  Written out on the bit patterns (integer arithmetic on
    the float32 fields), not via a library cast.
    """
    w = np.ascontiguousarray(val, dtype=np.float32).view(np.uint32).astype(np.int64)
    sign = (w >> 16) & 0x8000
    a = w & 0x7FFFFFFF
    if a.size and int(a.max()) >= _INF_BITS:
        raise NonFiniteGradient("NaN or Inf reached the fp16 codec")

    # normal halves, |v| >= 2**-14: re-bias the exponent from 127 to 15, drop
    # 13 mantissa bits with round-half-even (a carry into the exponent field
    # is the correct result)
    r = a - 0x38000000
    h_norm = r >> 13
    rem = r & 0x1FFF
    h_norm = h_norm + ((rem > 0x1000) | ((rem == 0x1000) & ((h_norm & 1) == 1)))

    # subnormal halves and zero, |v| < 2**-14: h = rint(|v| / 2**-24) where
    # |v| = m * 2**(e - 150), so h = m * 2**(e - 126) = m >> (126 - e)
    e = a >> 23
    m = (a & 0x7FFFFF) | 0x800000
    shift = np.clip(126 - e, 1, 25)  # shift 25 already gives 0 for every m
    h_sub = m >> shift
    rem_s = m & ((np.int64(1) << shift) - 1)
    half = np.int64(1) << (shift - 1)
    h_sub = h_sub + ((rem_s > half) | ((rem_s == half) & ((h_sub & 1) == 1)))
    h_sub = np.where(e == 0, 0, h_sub)  # float32 denormals are far below 2**-25

    h = np.where(a >= 0x38800000, h_norm, h_sub)
    h = np.where(a >= 0x477FF000, 0x7BFF, h)  # 65520.0f and above saturate
    return (sign | h).astype(np.uint16)


def f16_bits_to_f32(bits16: np.ndarray) -> np.ndarray:
    """binary16 bit patterns -> the exactly equal float32 values."""
    w = np.ascontiguousarray(bits16, dtype=np.uint16).astype(np.int64)
    e = (w >> 10) & 0x1F
    m = w & 0x3FF
    if e.size and int(e.max()) == 31:
        raise NonFiniteGradient("Inf or NaN half in a payload")
    sub = m.astype(np.float64) * 2.0 ** -24
    nrm = (1.0 + m.astype(np.float64) / 1024.0) * np.exp2((e - 15).astype(np.float64))
    mag = np.where(e == 0, sub, nrm)
    return np.where((w & 0x8000) != 0, -mag, mag).astype(np.float32)


@dataclass
class Payload:
    """One worker's compressed bucket, in payload order (ascending index)."""

    n: int
    k: int
    bits: int  # 8 -> int8 codes + per-block scales; 16 -> fp16 bit patterns; 32 -> the raw float32 values
    idx: np.ndarray  # uint32[k], strictly ascending
    raw: np.ndarray  # float32[k], survivor values before quantisation
    codes: Optional[np.ndarray] = None  # int8[k]       (bits == 8)
    scales: Optional[np.ndarray] = None  # float32[ceil(k/QBLOCK)] (bits == 8)
    half: Optional[np.ndarray] = None  # uint16[k]     (bits == 16)

    def values(self) -> np.ndarray:
        """Dequantised float32 values v'."""
        if self.bits == 8:
            return dequantize_int8(self.codes, self.scales)
        if self.bits == 32:
            return self.raw.copy()
        return f16_bits_to_f32(self.half)


def compress(
    grad: np.ndarray,
    ratio: float,
    bits: int,
    prune_mask: Optional[np.ndarray] = None,
) -> Payload:
    """Alg. 2 Steps 2-3 plus the value codec, for one flat float32 bucket.

    A bf16 bucket is widened with widen_bf16 first.  `prune_mask[i]` true
    means parameter i is pruned this step.
    """
    if bits not in (8, 16, 32):
        raise ValueError("bits must be 8 (int8), 16 (fp16) or 32 (float32 as is)")
    v = _apply_mask(grad, prune_mask)
    n = v.size
    k = k_of(ratio, n)
    idx = select_topk(v, k)
    raw = v[idx]
    p = Payload(n=n, k=k, bits=bits, idx=idx, raw=raw)
    if bits == 8:
        p.codes, p.scales = quantize_int8(raw)
    elif bits == 16:
        p.half = f32_to_f16_bits(raw)
    return p


def compress_many(
    grad: np.ndarray,
    ratios: Sequence[float],
    bits: int,
    prune_mask: Optional[np.ndarray] = None,
):
    """compress() of one bucket at several ratios (one full sort serves all
    of them: the survivors at ratio r are the first k_of(r, n) entries of the
    sorted order).  Returns one Payload per ratio."""
    if bits not in (8, 16, 32):
        raise ValueError("bits must be 8 (int8), 16 (fp16) or 32 (float32 as is)")
    v = _apply_mask(grad, prune_mask)
    n = v.size
    ks = [k_of(r, n) for r in ratios]
    out = []
    for k, idx in zip(ks, select_topk_many(v, ks)):
        raw = v[idx]
        p = Payload(n=n, k=k, bits=bits, idx=idx, raw=raw)
        if bits == 8:
            p.codes, p.scales = quantize_int8(raw)
        elif bits == 16:
            p.half = f32_to_f16_bits(raw)
        out.append(p)
    return out


def decompress_sum(
    payloads: Sequence[Payload],
    n: int,
    dense_in: Optional[np.ndarray] = None,
) -> np.ndarray:
    """Dense float32 gradient = (dense_in or 0) + sum over workers of their
    dequantised payloads scattered to their indices.  Accumulated in float64
    in worker order and rounded once to float32."""
    acc = np.zeros(n, dtype=np.float64)
    if dense_in is not None:
        d = np.ascontiguousarray(dense_in, dtype=np.float32)
        if d.size != n:
            raise ValueError("dense_in must have n elements")
        acc += d.astype(np.float64)
    for p in payloads:
        if p.n != n:
            raise ValueError("payload built for another bucket size")
        idx = p.idx.astype(np.int64)
        if idx.size and (idx[-1] >= n or np.any(np.diff(idx) <= 0)):
            raise ValueError("payload indices must be strictly ascending and < n")
        # indices are unique within one payload, so the indexed add is a
        # plain element-wise add
        acc[idx] += p.values().astype(np.float64)
    return acc.astype(np.float32)
