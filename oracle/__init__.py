"""CPU oracle for the NetSenseML adaptive-compression hot path.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, obviously-correct
restatement of what the path computes (Alg. 1, Alg. 2 Steps 2-3, Eq. 1-3 of
the paper, plus the int8 / fp16 value codecs and the multi-worker sum).  It
shares no code with the CUDA library and never imports it.  Only the tests,
the smoke check and the CPU-baseline leg of the benchmark may import it; the
product path must never route through it.

Pins (what each function is checked against, independently of itself):
  select_topk        brute force over all k-subsets, partial-sort special
                     case, worked examples, invariants
  select_topk_many   the same brute force, for every k of one bucket at once
  quantize_int8      worked half-way examples, invariants, fractions.Fraction
                     exact arithmetic on small blocks
  f32_to_f16_bits    NumPy's float16 cast on finite in-range inputs, worked
                     bit patterns
  decompress_sum     closed forms (identical payloads, disjoint payloads),
                     dense brute-force loop
  l2_norm            closed forms (constant vectors, 3-4-5), math.fsum of exact
                     rational squares, the library norm in float64
  quantize_gate      the four branches of Alg. 2 Step 1 written out by hand
  prune_mask         brute force over all m-subsets, worked example, library
                     partial sort on distinct keys, the paper's rate formula,
                     invariants (count, order, tie rule)
  error_feedback_step  worked two-step example, conservation (what is sent
                     plus what is kept equals the accumulated gradient)
  Controller (NetSense phase)  hand trace from Eq. 1-3, closed forms for the
                     multiplicative-decrease / additive-increase recurrences
  Controller (start-up phase)  parity unpinned: the paper gives neither the
                     increment beta_1, the phase length nor the exit test, so
                     the start-up recurrence and its three exits (excessive
                     transfer time, step limit, ratio at its cap) are hand
                     traced only under the reading stated in this package.
"""
from .compress import (  # noqa: F401
    QBLOCK,
    NonFiniteGradient,
    k_of,
    widen_bf16,
    keys_of,
    select_topk,
    select_topk_many,
    quantize_int8,
    dequantize_int8,
    f32_to_f16_bits,
    f16_bits_to_f32,
    compress,
    compress_many,
    decompress_sum,
    Payload,
)
from .adaptive import (  # noqa: F401
    l2_norm,
    quantize_gate,
    pruning_rate,
    pruned_count,
    prune_mask,
    netsense_compression,
    error_feedback_step,
)
from .controller import Controller, ControllerParams  # noqa: F401
