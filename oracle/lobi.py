"""CPU oracle for the Lo-Bi quantiser applied to the LM head: 8-bit rows, 4-bit sub-blocks, mixed widths (test infrastructure).

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


# ---- 4-bit sub-blocks with per-sub-block scales -----------------------------------------------------------------------
# The Lo-Bi section maps SUB-BLOCKS of a weight matrix to 4, 8 or 16 bits.  Reading taken for the 4-bit case on the LM
# head: a sub-block is 128 consecutive hidden channels of one vocabulary row; its codes are symmetric 4-bit integers
# c in [-7, 7]; its scale is a power-of-two multiple of the row's fp32 scale (a shared exponent per sub-block on top of
# one fp32 number per row):
#
#     s_v      = max_h |W[v, h]| / 112                     (1 for an all-zero row; 112 = 7 * 2^4)
#     e_{v,b}  = the smallest e in {0, 1, 2, 3, 4} with 7 * 2^e * s_v >= max_{h in b} |W[v, h]|   (4 if none does)
#     c[v, h]  = clip(rint(W[v, h] / (s_v * 2^e)), -7, 7)  (round half to even)
#     W4[v, h] = s_v * (c[v, h] << e_{v,b})                (an integer of magnitude <= 112 times the row scale)
#
# Every line is one fp32 operation (the product s_v * 2^e is exact), so the device can decide the same integers bit for
# bit.  Two codes share a byte: byte j of a row holds c[2j] in its low nibble and c[2j+1] in its high nibble, both as
# 4-bit two's complement.
SUB_BLOCK = 128
W4_TOP = 112.0          # 7 * 2^4: the largest magnitude c << e


def quantize_rows_w4(W: np.ndarray):
    """W: float32 [V, H], H a multiple of 128.  Returns (codes int8 [V, H] in [-7, 7], shifts uint8 [V, H / 128],
    scale float32 [V])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    V, H = W.shape
    assert H % SUB_BLOCK == 0
    nb = H // SUB_BLOCK
    amax = np.max(np.abs(W), axis=1).astype(np.float32)
    scale = (amax / np.float32(W4_TOP)).astype(np.float32)
    scale[amax == 0] = np.float32(1.0)
    blocks = W.reshape(V, nb, SUB_BLOCK)
    bmax = np.max(np.abs(blocks), axis=2).astype(np.float32)                   # [V, nb]
    shifts = np.full((V, nb), 4, dtype=np.uint8)
    for e in (3, 2, 1, 0):                                                     # ends with the smallest e that covers
        reach = (scale * np.float32(7 * (1 << e))).astype(np.float32)[:, None]  # fp32 product, rounded once
        shifts[reach >= bmax] = e
    step = (scale[:, None] * np.exp2(shifts.astype(np.float32))).astype(np.float32)   # exact
    ratio = (blocks / step[:, :, None]).astype(np.float32)
    codes = np.clip(np.rint(ratio), -7, 7).astype(np.int8).reshape(V, H)
    return codes, shifts, scale


def dequantize_rows_w4(codes: np.ndarray, shifts: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """W4 = s_v * (c << e) as float64 (exact: an integer of at most 7 bits times an fp32 number)."""
    V, H = codes.shape
    ints = codes.astype(np.int64).reshape(V, -1, SUB_BLOCK) << shifts.astype(np.int64)[:, :, None]
    return ints.reshape(V, H).astype(np.float64) * scale.astype(np.float64)[:, None]


def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    """int8 [V, H] in [-8, 7] -> uint8 [V, H / 2]: even h in the low nibble, odd h in the high nibble."""
    u = codes.astype(np.uint8) & 0xF
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)


def unpack_nibbles(packed: np.ndarray) -> np.ndarray:
    lo = (packed & 0xF).astype(np.int8)
    hi = (packed >> 4).astype(np.int8)
    lo = np.where(lo > 7, lo - 16, lo).astype(np.int8)
    hi = np.where(hi > 7, hi - 16, hi).astype(np.int8)
    out = np.empty((packed.shape[0], packed.shape[1] * 2), dtype=np.int8)
    out[:, 0::2], out[:, 1::2] = lo, hi
    return out


# ---- vocabulary groups of mixed width ----------------------------------------------------------------------------------
# Widths are assigned per GROUP of 256 consecutive vocabulary rows (the rows one pair of CTAs multiplies at a time);
# inside a group every sub-block has the group's width.  16: the bf16 weights as they are (scale 1).  8: the per-row
# 8-bit form above (one sub-block scale per row).  4: the 4-bit form above.  The head that results is the matrix whose
# rows are the dequantised rows of their groups; the verify step on it is the ordinary definition.
GROUP_ROWS = 256


def dequantize_mixed(W: np.ndarray, widths) -> np.ndarray:
    """W float32 [V, H] (bf16 values widened), widths[g] in {4, 8, 16} for group g.  Returns float64 [V, H]."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    V = W.shape[0]
    out = np.empty(W.shape, dtype=np.float64)
    for g, width in enumerate(widths):
        lo, hi = g * GROUP_ROWS, min(V, (g + 1) * GROUP_ROWS)
        if lo >= hi:
            break
        if width == 16:
            out[lo:hi] = W[lo:hi].astype(np.float64)
        elif width == 8:
            out[lo:hi] = dequantize_rows(*quantize_rows_int8(W[lo:hi]))
        elif width == 4:
            out[lo:hi] = dequantize_rows_w4(*quantize_rows_w4(W[lo:hi]))
        else:
            raise ValueError(f"width {width} is not one of 4, 8, 16")
    return out
