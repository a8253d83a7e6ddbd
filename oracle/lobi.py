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
