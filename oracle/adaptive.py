"""Oracle for the parts of Alg. 2 around the top-k step: the adaptive
quantisation gate (Step 1), the pruning mask built from the weights (Step 2)
and the local accumulation of what sparsification filtered out (Step 3).

TEST INFRASTRUCTURE ONLY (see the package docstring).

What is computed, and where the paper states it:

* Alg. 2 Step 1: if ratio < tr_q, the gradient's L2 norm is computed; if it
  exceeds tr_d the gradients are sent as 16-bit floats and the ratio is
  doubled.  The paper gives no values for tr_q and tr_d (they are inputs)
  and does not cap the doubled ratio; it is capped at 1 here because a kept
  fraction above 1 has no meaning.  The norm is sqrt(sum g_i^2) in float64.
* Alg. 2 Step 2: pruning_rate = 0.5 * (1 - ratio); the parameters with the
  smallest weights are pruned and their gradients set to zero before Step 3.
  The paper does not say how many parameters a rate stands for, nor how ties
  are broken: the readings taken are m = ceil(pruning_rate * n) evaluated in
  IEEE double, smaller |w| first, then lower index.  The mask is rebuilt
  from the weights whenever it is asked for (pruning is not permanent).
* Section 4.2 Step 3: the gradients that sparsification filters out are
  accumulated locally for later transmission.  Read as a residual: the
  bucket that is compressed is acc = g + residual (one float32 add), and the
  new residual is acc with what the payload carries taken out, acc[i] - v'_i
  (one float32 subtraction) at the selected positions, v' being the value
  the receiver reconstructs, so that quantisation error is carried over too.

Every function is its plain definition: a float64 sum, a full sort, an
element-wise update of the selected positions.
"""
from __future__ import annotations

import math
from typing import Optional, Tuple

import numpy as np

from .compress import Payload, NonFiniteGradient, compress, keys_of


def l2_norm(grad: np.ndarray) -> float:
    """sqrt(sum of squares), every square and the sum in float64."""
    g = np.ascontiguousarray(grad, dtype=np.float32).astype(np.float64)
    if g.size and not np.all(np.isfinite(g)):
        raise NonFiniteGradient("bucket holds NaN or Inf")
    return math.sqrt(float(np.sum(g * g)))


def quantize_gate(ratio: float, l2: float, tr_q: float, tr_d: float) -> Tuple[bool, float]:
    """Alg. 2 Step 1: (quantise to 16 bits?, ratio to use from here on)."""
    ratio = float(ratio)
    if ratio < float(tr_q) and float(l2) > float(tr_d):
        return True, min(1.0, 2.0 * ratio)
    return False, ratio


def pruning_rate(ratio: float) -> float:
    """Alg. 2 Step 2: 0.5 * (1 - ratio), in double as written."""
    ratio = float(ratio)
    if not (ratio > 0.0 and ratio <= 1.0):
        raise ValueError("ratio must lie in (0, 1]")
    return 0.5 * (1.0 - ratio)


def pruned_count(ratio: float, n: int) -> int:
    """Parameters pruned at this ratio: ceil(pruning_rate * n), at most n."""
    if not (isinstance(n, (int, np.integer)) and n >= 1):
        raise ValueError("n must be a positive integer")
    return min(int(n), int(math.ceil(pruning_rate(ratio) * float(n))))


def prune_mask(weights: np.ndarray, ratio: float) -> np.ndarray:
    """Boolean mask, true = pruned: the pruned_count(ratio, n) parameters of
    smallest magnitude, ties by lower index.  Full sort on (key ascending,
    index ascending), the pair packed into one unsigned 64-bit word."""
    key = keys_of(weights)
    n = key.size
    if n >= 2**32:
        raise ValueError("n must be below 2**32")
    if n and int(key.max()) >= 0x7F800000:
        raise NonFiniteGradient("weights hold NaN or Inf")
    m = pruned_count(ratio, n)
    packed = (key.astype(np.uint64) << np.uint64(32)) | np.arange(n, dtype=np.uint64)
    packed.sort()
    mask = np.zeros(n, dtype=bool)
    mask[(packed[:m] & np.uint64(0xFFFFFFFF)).astype(np.int64)] = True
    return mask


def netsense_compression(
    grads: np.ndarray,
    ratio: float,
    tr_q: float,
    tr_d: float,
    weights: Optional[np.ndarray] = None,
    plain_bits: int = 32,
):
    """Alg. 2 as a whole, in its order: Step 1 gate (may switch to 16-bit
    values and double the ratio), Step 2 mask from the weights at the ratio
    Step 1 left, Step 3 top-k at that ratio.  `plain_bits` is the value codec
    used when Step 1 does not quantise (32 = the paper's plain floats).
    Returns (payload, ratio used, bits used, L2 norm or None, mask or None).

    As in the rest of this oracle the survivors are chosen on the float32
    magnitudes and only they are converted to 16 bits."""
    ratio = float(ratio)
    l2 = None
    bits = plain_bits
    if ratio < float(tr_q):
        l2 = l2_norm(grads)
        quantise, ratio = quantize_gate(ratio, l2, tr_q, tr_d)
        if quantise:
            bits = 16
    mask = prune_mask(weights, ratio) if weights is not None else None
    return compress(grads, ratio, bits, prune_mask=mask), ratio, bits, l2, mask


def error_feedback_step(
    grad: np.ndarray,
    residual: np.ndarray,
    ratio: float,
    bits: int,
    prune_mask_: Optional[np.ndarray] = None,
) -> Tuple[Payload, np.ndarray]:
    """One step of local accumulation: returns (payload of acc = grad +
    residual, new residual)."""
    g = np.ascontiguousarray(grad, dtype=np.float32)
    r = np.ascontiguousarray(residual, dtype=np.float32)
    if g.shape != r.shape:
        raise ValueError("residual must have one element per gradient element")
    with np.errstate(under="ignore"):
        acc = (g + r).astype(np.float32)  # one float32 add per element
    p = compress(acc, ratio, bits, prune_mask=prune_mask_)
    sent = p.values()
    new_r = acc.copy()
    idx = p.idx.astype(np.int64)  # unique, so the indexed store is a plain element-wise one
    with np.errstate(under="ignore"):
        new_r[idx] = (acc[idx] - sent).astype(np.float32)  # one float32 subtraction
    return p, new_r
