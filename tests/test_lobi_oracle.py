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


# ---- two 8-bit planes per activation row
def test_two_plane_rows_error_bound_and_first_plane():
    rng = np.random.default_rng(5)
    x = ref.bf16_bits_to_f64(ref.f32_to_bf16_bits(rng.normal(size=(30, 128)).astype(np.float32))).astype(np.float32)
    x[4] = 0.0
    q1, q2, s1, s2 = lobi.quantize_rows_two_plane(x)
    qa, sa = lobi.quantize_rows_int8(x)
    assert np.array_equal(q1, qa) and np.array_equal(s1, sa)            # the first plane is the plain 8-bit quantiser
    x16 = lobi.dequantize_two_plane(q1, q2, s1, s2)
    amax = np.max(np.abs(x), axis=1)
    # half a step of the second plane, plus the two fp32 roundings that produced the residual (each < 2^-24 of the row
    # maximum): sixteen bits against the row maximum, 250 times finer than one plane
    bound = 0.5 * s2.astype(np.float64) + 2.0 ** -22 * amax
    assert np.all(np.abs(x16 - x) <= bound[:, None])
    nz = amax > 0
    one_plane = np.max(np.abs(lobi.dequantize_rows(qa, sa) - x), axis=1)
    assert np.all(np.max(np.abs(x16 - x), axis=1)[nz] < one_plane[nz] / 100)
    assert np.abs(q2).max() <= 127 and np.all(q2[4] == 0) and np.all(q1[4] == 0)
    assert np.allclose(s2 * np.float32(254.0), s1, rtol=1e-6)


def test_two_plane_exact_cases_and_symmetry():
    # integers with row maximum 127: scale 1, the first plane is exact and the second one is zero
    rng = np.random.default_rng(6)
    x = rng.integers(-127, 128, size=(5, 64)).astype(np.float32)
    x[:, 0] = 127.0
    q1, q2, s1, s2 = lobi.quantize_rows_two_plane(x)
    assert np.all(s1 == 1.0) and np.array_equal(q1.astype(np.float32), x) and np.all(q2 == 0)
    # multiples of 1/254 between the integers: the second plane holds them exactly
    y = x.copy()
    y[:, 1:] += (rng.integers(-127, 128, size=(5, 63)) / 254.0).astype(np.float32) * 0.999
    y = np.clip(y, -127, 127).astype(np.float32)
    q1, q2, s1, s2 = lobi.quantize_rows_two_plane(y)
    assert np.max(np.abs(lobi.dequantize_two_plane(q1, q2, s1, s2) - y)) <= 0.5 / 254 + 1e-5
    # odd symmetry, and a power-of-two factor moves into both scales
    x = rng.normal(size=(8, 96)).astype(np.float32)
    a = lobi.quantize_rows_two_plane(x)
    b = lobi.quantize_rows_two_plane(-x)
    assert np.array_equal(b[0], -a[0]) and np.array_equal(b[1], -a[1]) and np.array_equal(b[2], a[2])
    c = lobi.quantize_rows_two_plane(x * np.float32(8.0))
    assert np.array_equal(c[0], a[0]) and np.array_equal(c[1], a[1])
    assert np.array_equal(c[2], a[2] * np.float32(8.0)) and np.array_equal(c[3], a[3] * np.float32(8.0))


def test_two_plane_head_logits_stay_close_to_bf16_activations():
    rng = np.random.default_rng(7)
    hid = ref.bf16_bits_to_f64(ref.f32_to_bf16_bits(rng.normal(size=(6, 256)).astype(np.float32)))
    W = ref.bf16_bits_to_f64(ref.f32_to_bf16_bits((rng.normal(size=(50, 256)) * 0.05).astype(np.float32)))
    q, s = lobi.quantize_rows_int8(W.astype(np.float32))
    W8 = lobi.dequantize_rows(q, s)
    h16 = lobi.dequantize_two_plane(*lobi.quantize_rows_two_plane(hid.astype(np.float32)))
    h8 = lobi.dequantize_rows(*lobi.quantize_rows_int8(hid.astype(np.float32)))
    exact = hid @ W8.T
    assert np.max(np.abs(h16 @ W8.T - exact)) < 2e-4                    # 16-bit-class rows: invisible next to ...
    assert np.max(np.abs(h8 @ W8.T - exact)) > 2e-3                     # ... what one 8-bit plane does to the logits


# ---- 4-bit sub-blocks with a shared power-of-two exponent per sub-block --------------------------------------------
def _w4_rows(seed, V=12, nb=3):
    """Rows that ARE of the 4-bit form with row scale 1: entry = c << e with c in [-7, 7], e per sub-block, and one
    entry equal to 112 so that the row maximum gives scale exactly 1."""
    rng = np.random.default_rng(seed)
    c = rng.integers(-7, 8, size=(V, nb, 128))
    e = rng.integers(0, 5, size=(V, nb))
    c[:, :, 0] = 7                                          # every sub-block reaches its top code: e is forced
    e[:, 0] = 4                                             # sub-block 0 holds 7 << 4 = 112, the row maximum
    W = (c << e[:, :, None]).reshape(V, nb * 128).astype(np.float32)
    return W, c.reshape(V, -1).astype(np.int8), e.astype(np.uint8)


def test_w4_rows_of_the_format_are_reproduced_exactly():
    W, c, e = _w4_rows(3)
    codes, shifts, scale = lobi.quantize_rows_w4(W)
    assert np.all(scale == 1.0)
    assert np.array_equal(shifts, e) and np.array_equal(codes, c)
    assert np.array_equal(lobi.dequantize_rows_w4(codes, shifts, scale), W.astype(np.float64))
    # a power-of-two factor moves into the row scale and changes neither codes nor exponents
    codes2, shifts2, scale2 = lobi.quantize_rows_w4(W * np.float32(0.125))
    assert np.array_equal(codes2, codes) and np.array_equal(shifts2, shifts) and np.all(scale2 == 0.125)


def test_w4_exponent_is_the_smallest_that_covers_the_sub_block():
    W = np.zeros((1, 4 * 128), np.float32)
    W[0, 0] = 112.0                                         # row scale 1; sub-block 0 needs e = 4
    W[0, 128] = 7.0                                         # sub-block 1: 7 * 2^0 covers it
    W[0, 256] = 7.5                                         # sub-block 2: just beyond 7, so e = 1
    W[0, 384] = 56.0                                        # sub-block 3: 7 * 2^3
    codes, shifts, scale = lobi.quantize_rows_w4(W)
    assert scale[0] == 1.0 and shifts[0].tolist() == [4, 0, 1, 3]
    assert codes[0, 0] == 7 and codes[0, 128] == 7 and codes[0, 384] == 7
    assert codes[0, 256] == 4                               # 7.5 / 2 = 3.75 -> 4


def test_w4_error_bound_symmetry_zero_rows_and_ties():
    rng = np.random.default_rng(4)
    W = (rng.normal(size=(30, 512)) * 0.02).astype(np.float32)
    W[:, 128:256] *= 0.1                                    # a quiet sub-block in every row: it gets a smaller exponent
    W[5] = 0.0
    codes, shifts, scale = lobi.quantize_rows_w4(W)
    deq = lobi.dequantize_rows_w4(codes, shifts, scale)
    step = scale[:, None].astype(np.float64) * np.exp2(shifts.astype(np.float64))          # [V, nb]
    err = np.abs(deq - W).reshape(30, 4, 128)
    assert np.all(err <= 0.5 * step[:, :, None] * (1 + 1e-6))          # nothing clips: at most half a step per sub-block
    assert np.all(shifts[np.arange(30) != 5, 1] < 4)                   # the quiet sub-block uses a finer step
    assert codes.min() >= -7 and codes.max() <= 7                      # -8 is never used
    assert np.all(codes[5] == 0) and scale[5] == 1.0
    c2, e2, s2 = lobi.quantize_rows_w4(-W)
    assert np.array_equal(c2, -codes) and np.array_equal(e2, shifts) and np.array_equal(s2, scale)
    # ties go to the even code: row scale 1 (maximum 112), second sub-block at e = 0 holds x.5 values
    T = np.zeros((1, 256), np.float32)
    T[0, 0] = 112.0
    T[0, 128:134] = [0.5, 1.5, 2.5, -0.5, -1.5, 6.5]
    T[0, 134] = 7.0
    c, e, s = lobi.quantize_rows_w4(T)
    assert s[0] == 1.0 and e[0].tolist() == [4, 0] and c[0, 128:135].tolist() == [0, 2, 2, 0, -2, 6, 7]


def test_nibble_packing_round_trip_and_layout():
    rng = np.random.default_rng(5)
    c = rng.integers(-8, 8, size=(7, 64)).astype(np.int8)
    p = lobi.pack_nibbles(c)
    assert p.shape == (7, 32) and p.dtype == np.uint8
    assert np.array_equal(lobi.unpack_nibbles(p), c)
    one = np.array([[3, -2]], np.int8)                      # low nibble 0x3, high nibble 0xE (-2 in 4-bit two's complement)
    assert lobi.pack_nibbles(one)[0, 0] == 0xE3


def test_mixed_width_head_takes_each_group_from_its_own_quantiser():
    rng = np.random.default_rng(6)
    V, H = 2 * 256 + 100, 256                               # three groups, the last one ragged
    W = ref.bf16_bits_to_f64(ref.f32_to_bf16_bits((rng.normal(size=(V, H)) * 0.02).astype(np.float32))).astype(np.float32)
    D = lobi.dequantize_mixed(W, [16, 4, 8])
    assert np.array_equal(D[:256], W[:256].astype(np.float64))                              # 16 bits: untouched
    assert np.array_equal(D[256:512], lobi.dequantize_rows_w4(*lobi.quantize_rows_w4(W[256:512])))
    assert np.array_equal(D[512:], lobi.dequantize_rows(*lobi.quantize_rows_int8(W[512:])))
    # wider is closer: the 8-bit group's error is well below the 4-bit group's
    e4 = np.abs(D[256:512] - W[256:512]).max() / np.abs(W[256:512]).max()
    e8 = np.abs(D[512:] - W[512:]).max() / np.abs(W[512:]).max()
    assert e8 < 0.005 and 0.02 < e4 < 0.08
