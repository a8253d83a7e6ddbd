"""CPU oracle for the 8-bit case of the Lo-Bi quantiser applied to the LM head (test infrastructure).

The Lo-Bi Optimization section maps sub-blocks of a weight matrix to 4-, 8- or 16-bit precision with a quantiser
Q(.) that it does not spell out, and reports that over 70 % of the blocks end at 8 bits.  The reading taken here
for the LM head: every sub-block is one vocabulary row of W_lm, all rows at 8 bits, and Q is the plain symmetric
scheme - one fp32 scale per row, integers in [-127, 127], round half to even:

    scale_v = max_h |W[v, h]| / 127          (scale_v = 1 for an all-zero row)
    q[v, h] = clip(rint(W[v, h] / scale_v), -127, 127)
    W8[v, h] = scale_v * q[v, h]             (what the verifier's LM head multiplies with)

All three lines are evaluated in fp32, the precision in which the CUDA quantiser decides the integers, so that the
integers can be compared bit for bit.  The logits of the quantised head are then the ordinary definition
l[r, v] = sum_h hidden[r, h] * W8[v, h], taken in fp64 by oracle/hola_verify_ref.cpp on the dequantised matrix.
Nothing on the product path imports this module.
"""
from __future__ import annotations

import numpy as np


def quantize_rows_int8(W: np.ndarray):
    """W: float32 [V, H] (bf16 values widened exactly).  Returns (q int8 [V, H], scale float32 [V])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    amax = np.max(np.abs(W), axis=1).astype(np.float32)
    scale = (amax / np.float32(127.0)).astype(np.float32)
    scale[amax == 0] = np.float32(1.0)
    ratio = (W / scale[:, None]).astype(np.float32)          # fp32 division, correctly rounded
    q = np.clip(np.rint(ratio), -127, 127).astype(np.int8)   # rint: round half to even
    return q, scale


def dequantize_rows(q: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """W8 = scale_v * q[v, h] as float64 (each product of an fp32 scale and an 8-bit integer is exact in fp64)."""
    return q.astype(np.float64) * scale.astype(np.float64)[:, None]


# ---- 16-bit-class activations as two 8-bit planes -------------------------------------------------------------------
# With 8-bit weights, the verifier's hidden rows can stay close to their bf16 values and still run on the 8-bit
# tensor-core kind if each row is written as a coarse 8-bit plane plus an 8-bit plane of what the first one missed:
#
#     s1 = max_h |x[h]| / 127  (1 for an all-zero row)      q1 = clip(rint(x / s1), -127, 127)
#     r  = x - s1 * q1         (|r| <= s1 / 2)               s2 = s1 / 254
#     q2 = clip(rint(r / s2), -127, 127)                     x16 = s1 * q1 + s2 * q2
#
# so |x16 - x| <= s2 / 2 = max|x| / 64516: sixteen bits' worth against the row maximum.  (The Lo-Bi section keeps
# "16-bit" as its widest setting and says nothing about activations; this is the reading that lets the 8-bit head
# keep them at that width.)  Every step is one fp32 operation - division, rint, product, difference - so both sides
# can take the integers in the same precision and compare them bit for bit.


def quantize_rows_two_plane(x: np.ndarray):
    """x: float32 [R, H].  Returns (q1 int8 [R, H], q2 int8 [R, H], s1 float32 [R], s2 float32 [R])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    q1, s1 = quantize_rows_int8(x)
    coarse = (s1[:, None] * q1.astype(np.float32)).astype(np.float32)    # fp32 product, rounded once
    r = (x - coarse).astype(np.float32)                                  # fp32 difference, rounded once
    s2 = (s1 / np.float32(254.0)).astype(np.float32)
    q2 = np.clip(np.rint((r / s2[:, None]).astype(np.float32)), -127, 127).astype(np.int8)
    return q1, q2, s1, s2


def dequantize_two_plane(q1, q2, s1, s2) -> np.ndarray:
    """x16 = s1 * q1 + s2 * q2 as float64 (both products and their sum are exact in fp64)."""
    return (q1.astype(np.float64) * s1.astype(np.float64)[:, None]
            + q2.astype(np.float64) * s2.astype(np.float64)[:, None])
