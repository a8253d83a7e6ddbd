"""Pins for the 8-bit quantiser oracle (oracle/lobi.py): facts that any symmetric round-to-nearest int8 scheme with
a per-row scale must satisfy, none of them taken from the oracle's own output."""
import numpy as np

from oracle import lobi, ref


def test_integer_rows_with_maximum_127_are_reproduced_exactly():
    rng = np.random.default_rng(1)
    W = rng.integers(-127, 128, size=(9, 64)).astype(np.float32)
    W[:, 0] = 127.0                                        # every row reaches the top code: scale is exactly 1
    q, s = lobi.quantize_rows_int8(W)
    assert np.all(s == 1.0) and np.array_equal(q.astype(np.float32), W)
    assert np.array_equal(lobi.dequantize_rows(q, s), W.astype(np.float64))


def test_error_bound_extremes_sign_and_zero_rows():
    rng = np.random.default_rng(2)
    W = (rng.normal(size=(40, 96)) * 0.02).astype(np.float32)
    W[7] = 0.0
    q, s = lobi.quantize_rows_int8(W)
    deq = lobi.dequantize_rows(q, s)
    assert np.all(np.abs(deq - W) <= 0.5 * s[:, None] * (1 + 1e-6))      # round to nearest: at most half a step
    amax_at = np.argmax(np.abs(W), axis=1)
    rows = np.arange(40)
    assert np.all(np.abs(q[rows, amax_at])[np.arange(40) != 7] == 127)   # the largest entry of a row takes the top code
    assert np.all(q[7] == 0) and s[7] == 1.0                             # an all-zero row
    assert q.min() >= -127 and q.max() <= 127                           # -128 is never used (symmetric range)
    q2, s2 = lobi.quantize_rows_int8(-W)
    assert np.array_equal(q2, -q) and np.array_equal(s2, s)              # odd symmetry
    q3, s3 = lobi.quantize_rows_int8(W * np.float32(4.0))
    nz = np.arange(40) != 7
    assert np.array_equal(q3, q) and np.array_equal(s3[nz], s[nz] * np.float32(4.0))   # a power-of-two factor moves into the scale


def test_ties_round_to_even():
    # scale = 1 (row maximum 127): x.5 goes to the even neighbour
    W = np.array([[127.0, 0.5, 1.5, 2.5, -0.5, -1.5, 126.5]], np.float32)
    q, s = lobi.quantize_rows_int8(W)
    assert s[0] == 1.0 and q[0].tolist() == [127, 0, 2, 2, 0, -2, 126]


def test_quantised_head_logits_are_the_plain_definition_on_w8():
    # logits of the quantised head = sum_h hidden * (scale * q): an independent fp64 matmul agrees with the oracle
    rng = np.random.default_rng(3)
    hid = ref.bf16_bits_to_f64(ref.f32_to_bf16_bits(rng.normal(size=(6, 64)).astype(np.float32)))
    W = ref.bf16_bits_to_f64(ref.f32_to_bf16_bits((rng.normal(size=(50, 64)) * 0.05).astype(np.float32)))
    q, s = lobi.quantize_rows_int8(W.astype(np.float32))
    W8 = lobi.dequantize_rows(q, s)
    got = ref.logits(hid, W8)
    np.testing.assert_allclose(got, hid @ W8.T, rtol=1e-13, atol=1e-13)
    assert np.max(np.abs(got - hid @ W.T)) < 0.05           # and stays close to the unquantised head
