"""Pins for the CPU oracle: everything here is fixed by the paper or by mathematics, not by the oracle itself.

The paper prints no worked numerical example of the verify step, so the pins are closed forms of the entropy
definition (HSD section), invariants, exact-integer products, library routines on special cases, and the
brute-force statement that the emitted token's marginal equals the verifier's distribution p when the gate is
off (and the draft's q at a gated position), checked on 8- and 16-token vocabularies.
"""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import ref

INF = float("inf")


# ------------------------------------------------------------------ step 1: logits (the LM-head projection)

def test_logits_identity_weight_returns_hidden():
    # W = I (V = H)  =>  logits = hidden, exactly.
    rng = np.random.default_rng(1)
    hidden = rng.integers(-8, 9, size=(5, 16)).astype(np.float32)
    W = np.eye(16, dtype=np.float32)
    assert np.array_equal(ref.logits(hidden, W), hidden.astype(np.float64))


def test_logits_small_integers_are_exact_and_not_transposed():
    # |values| <= 8, H = 96: every product and partial sum is an integer below 2^24, exact in any precision.
    # M != V != H and asymmetric data, so a transposed operand or swapped index cannot pass.
    rng = np.random.default_rng(2)
    M, H, V = 7, 96, 37
    hid = rng.integers(-8, 9, size=(M, H))
    W = rng.integers(-8, 9, size=(V, H))
    want = np.zeros((M, V), dtype=np.int64)
    for r in range(M):
        for v in range(V):
            want[r, v] = sum(int(hid[r, h]) * int(W[v, h]) for h in range(H))
    for dt in (np.float32, np.float64):
        got = ref.logits(hid.astype(dt), W.astype(dt))
        assert np.array_equal(got, want.astype(np.float64))
    got = ref.logits(ref.f32_to_bf16_bits(hid.astype(np.float32)), ref.f32_to_bf16_bits(W.astype(np.float32)))
    assert np.array_equal(got, want.astype(np.float64))


def test_logits_match_blas_on_random_fp64():
    rng = np.random.default_rng(3)
    hid = rng.standard_normal((11, 200))
    W = rng.standard_normal((53, 200)) * 0.05
    np.testing.assert_allclose(ref.logits(hid, W), hid @ W.T, rtol=0, atol=1e-12)


def test_bf16_widening_is_exact():
    # 1.0, -2.5, 2^-10 and the largest bf16 below 1 are exactly representable; the oracle must see them unchanged.
    vals = np.array([[1.0, -2.5, 2.0 ** -10, 1.0 - 2.0 ** -8]], dtype=np.float32)
    bits = ref.f32_to_bf16_bits(vals)
    W = ref.f32_to_bf16_bits(np.eye(4, dtype=np.float32))
    assert np.array_equal(ref.logits(bits, W), vals.astype(np.float64))


# ------------------------------------------------------------------ steps 2-3: logZ and entropy

@pytest.mark.parametrize("V", [8, 16, 1000, 32000, 128256])
def test_uniform_distribution_has_entropy_ln_v(V):
    # W = 0  =>  every logit is 0  =>  p uniform  =>  logZ = ln V and H = ln V.
    logZ, H = ref.softmax_entropy(np.zeros((2, V)))
    assert np.allclose(logZ, math.log(V), rtol=0, atol=1e-12)
    assert np.allclose(H, math.log(V), rtol=0, atol=1e-10)


@pytest.mark.parametrize("V,G", [(128256, 15.0), (32000, 15.0), (16, 3.0), (1000, 40.0)])
def test_peaked_distribution_closed_form(V, G):
    # one logit G above V-1 equal others: p* = 1/(1+(V-1)e^-G), H = -p* ln p* - (1-p*) ln((1-p*)/(V-1)).
    l = np.full((1, V), -2.25)
    l[0, V // 3] += G
    tail = (V - 1) * math.exp(-G)
    p_star = 1.0 / (1.0 + tail)
    H_want = -p_star * math.log(p_star) - (1 - p_star) * math.log((1 - p_star) / (V - 1))
    logZ, H = ref.softmax_entropy(l)
    assert abs(logZ[0] - (-2.25 + G + math.log1p(tail))) < 1e-10   # V sequential fp64 additions
    assert abs(H[0] - H_want) < 1e-10


def test_peaked_values_quoted_for_the_large_vocab_shape():
    # gap 15 at V = 128256: p* = 0.9622477, H = 0.6047686 nats (closed form evaluated to 7 digits).
    l = np.zeros((1, 128256))
    l[0, 7] = 15.0
    logZ, H = ref.softmax_entropy(l)
    assert abs(math.exp(15.0 - logZ[0]) - 0.9622477) < 5e-8
    assert abs(H[0] - 0.6047686) < 5e-8


def test_one_hot_limit_has_zero_entropy_and_is_clamped():
    l = np.full((1, 50), -800.0)
    l[0, 3] = 0.0
    logZ, H = ref.softmax_entropy(l)
    assert logZ[0] == 0.0 and H[0] == 0.0


def test_two_level_distribution():
    # a tokens with mass 3w and b tokens with mass w: H has a two-term closed form.
    a, b = 5, 11
    w = 1.0 / (3 * a + b)
    l = np.log(np.array([[3 * w] * a + [w] * b]))
    want = -(a * 3 * w * math.log(3 * w) + b * w * math.log(w))
    _, H = ref.softmax_entropy(l + 4.0)
    assert abs(H[0] - want) < 1e-12


def test_entropy_and_logz_match_scipy_on_random_rows():
    rng = np.random.default_rng(5)
    l = rng.standard_normal((6, 777)) * 3.0
    logZ, H = ref.softmax_entropy(l)
    np.testing.assert_allclose(logZ, scipy.special.logsumexp(l, axis=1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(H, scipy.stats.entropy(scipy.special.softmax(l, axis=1), axis=1), rtol=0, atol=1e-11)


def test_shift_invariance():
    # adding c to every logit of a row adds c to logZ and changes nothing else.
    rng = np.random.default_rng(6)
    B, k, V = 9, 3, 40
    l = rng.standard_normal((B, k + 1, V)) * 2
    q = scipy.special.softmax(l[:, :k] + rng.standard_normal((B, k, V)), axis=-1)
    tok = rng.integers(0, V, size=(B, k))
    u = rng.random((B, k + 1)).astype(np.float32)
    a = ref.verify_from_logits(l, tok, q, u, 2.0)
    shift = rng.standard_normal((B, k + 1, 1)) * 10
    b = ref.verify_from_logits(l + shift, tok, q, u, 2.0)
    np.testing.assert_allclose(b.logZ, a.logZ + shift[..., 0], atol=1e-11)
    np.testing.assert_allclose(b.entropy, a.entropy, atol=1e-11)
    assert np.array_equal(a.accept_len, b.accept_len) and np.array_equal(a.next_tok, b.next_tok)


# ------------------------------------------------------------------ steps 4-5 on hand-computable cases

def _ln(p):
    return np.log(np.asarray(p, dtype=np.float64))


def test_hand_case_two_tokens():
    # p = (1/4, 3/4), q = (1/2, 1/2), draft token 0: ratio = 1/2.  Residual = (0, 1/4) -> token 1.
    l = np.tile(_ln([0.25, 0.75]), (1, 2, 1))
    q = np.array([[[0.5, 0.5]]])
    acc = ref.verify_from_logits(l, [[0]], q, [[0.3, 0.9]], 0.0)
    assert acc.accept_len[0] == 1 and abs(acc.margin_accept[0, 0] - 0.2) < 1e-7
    assert acc.next_tok[0] == 1           # bonus draw from p: c = (0.25, 1.0), 0.9 -> token 1
    rej = ref.verify_from_logits(l, [[0]], q, [[0.7, 0.0]], 0.0)
    assert rej.accept_len[0] == 0 and rej.next_tok[0] == 1 and abs(rej.margin_accept[0, 0] - 0.2) < 1e-7
    # draft token 1 has p > q: always accepted, whatever u
    top = ref.verify_from_logits(l, [[1]], q, [[0.999999, 0.1]], 0.0)
    assert top.accept_len[0] == 1 and top.next_tok[0] == 0   # bonus: 0.1 < 0.25 -> token 0


def test_inverse_cdf_boundaries_and_tie_break():
    # k = 0: pure draw from p = (0.1, 0, 0.2, 0.3, 0.4).  c = (.1, .1, .3, .6, 1).  First v with c(v) > u.
    p = [0.1, 0.0, 0.2, 0.3, 0.4]
    with np.errstate(divide="ignore"):
        l = _ln(p).reshape(1, 1, 5)
    q = np.zeros((1, 0, 5))
    for u, want in [(0.0, 0), (0.05, 0), (0.15, 2), (0.29, 2), (0.31, 3), (0.61, 4), (0.999, 4)]:
        got = ref.verify_from_logits(l, np.zeros((1, 0)), q, [[u]], 1.5)
        assert got.next_tok[0] == want, (u, got.next_tok[0])
    # zero-mass token 1 is never chosen even when u sits exactly on its (empty) interval
    got = ref.verify_from_logits(l, np.zeros((1, 0)), q, [[np.float32(0.1)]], 1.5)
    assert got.next_tok[0] in (0, 2)
    # margin: u = 0.15 is 0.05 above c(1) = 0.1 and 0.15 below c(2) = 0.3
    got = ref.verify_from_logits(l, np.zeros((1, 0)), q, [[0.15]], 1.5)
    assert abs(got.margin_cdf[0] - 0.05) < 1e-7


def test_q_equal_p_accepts_every_draft():
    rng = np.random.default_rng(8)
    B, k, V = 64, 5, 33
    l = rng.standard_normal((B, k + 1, V)) * 2.5
    p = scipy.special.softmax(l, axis=-1)
    tok = rng.integers(0, V, size=(B, k))
    u = rng.random((B, k + 1)).astype(np.float32)
    u[:, 0] = np.float32(1.0) - np.float32(2.0 ** -24)      # the largest float below 1
    # p/q is 1 up to one rounding of exp/log; keep u at least 2^-24 below 1 and the draw must still pass
    for tau in (0.0, 1.5, INF):
        out = ref.verify_from_logits(l, tok, p[:, :k] * (1.0 - 1e-9), u, tau)
        assert np.all(out.accept_len == k)


def test_residual_mass_and_support():
    rng = np.random.default_rng(9)
    B, V = 200, 24
    l = rng.standard_normal((B, 2, V)) * 2
    p = scipy.special.softmax(l, axis=-1)
    q = scipy.special.softmax(l[:, :1] + rng.standard_normal((B, 1, V)) * 1.5, axis=-1)
    tok = np.array([[int(np.argmax(q[b, 0] - p[b, 0]))] for b in range(B)])     # a token with q > p
    u = np.concatenate([np.full((B, 1), 0.999999, np.float32), rng.random((B, 1)).astype(np.float32)], axis=1)
    out = ref.verify_from_logits(l, tok, q, u, 0.0)
    rejected = out.accept_len == 0
    assert rejected.sum() > B // 2
    for b in np.nonzero(rejected)[0]:
        y = out.next_tok[b]
        assert p[b, 0, y] > q[b, 0, y]          # the replacement always comes from where p exceeds q
        assert y != tok[b, 0]
    # total-variation identity: sum max(0,p-q) = 1 - sum min(p,q) = 0.5 * sum |p-q|
    R = np.maximum(0, p[:, 0] - q[:, 0]).sum(-1)
    np.testing.assert_allclose(R, 1 - np.minimum(p[:, 0], q[:, 0]).sum(-1), atol=1e-12)


def test_one_hot_draft_residual_is_p_without_that_token():
    # q = one-hot at x  =>  residual = p with x removed, renormalised.  p = (.1,.2,.3,.4), x = 2:
    # residual CDF = (1/7, 3/7, 3/7, 1).
    l = np.tile(_ln([0.1, 0.2, 0.3, 0.4]), (1, 2, 1))
    q = np.array([[[0.0, 0.0, 1.0, 0.0]]])
    for u, want in [(0.10, 0), (0.20, 1), (0.42, 1), (0.44, 3), (0.99, 3)]:
        out = ref.verify_from_logits(l, [[2]], q, [[0.5, u]], 0.0)      # ratio = 0.3 < 0.5 -> rejected
        assert out.accept_len[0] == 0 and out.next_tok[0] == want, (u, out.next_tok[0])


def test_next_token_is_monotone_in_u_and_reproduces_the_residual_histogram():
    rng = np.random.default_rng(10)
    V, G = 16, 20000
    l = rng.standard_normal((1, 2, V)) * 1.5
    p = scipy.special.softmax(l, axis=-1)
    q = scipy.special.softmax(l[:, :1] + rng.standard_normal((1, 1, V)), axis=-1)
    x = int(np.argmax(q[0, 0] - p[0, 0]))
    us = ((np.arange(G) + 0.5) / G).astype(np.float32)
    u = np.stack([np.full(G, 0.9999999, np.float32), us], axis=1)
    out = ref.verify_from_logits(np.repeat(l, G, 0), np.full((G, 1), x), np.repeat(q, G, 0), u, 0.0)
    assert np.all(out.accept_len == 0)
    assert np.all(np.diff(out.next_tok) >= 0)
    r = np.maximum(0, p[0, 0] - q[0, 0])
    hist = np.bincount(out.next_tok, minlength=V) / G
    np.testing.assert_allclose(hist, r / r.sum(), atol=1.5 / G)


# ------------------------------------------------------------------ brute force: the emitted marginal

def _threshold(fn, lo, hi, steps=26):
    """Largest u (per batch element) for which fn(u) is True, by bisection; fn is monotone True -> False."""
    lo = np.array(lo, dtype=np.float64)
    hi = np.array(hi, dtype=np.float64)
    for _ in range(steps):
        mid = 0.5 * (lo + hi)
        ok = fn(mid.astype(np.float32))
        lo = np.where(ok, mid, lo)
        hi = np.where(ok, hi, mid)
    return 0.5 * (lo + hi)


def _tables(V, k, seed):
    """Explicit rational distributions: p_j(v) and q_j(v) are integer weights over their sum."""
    rng = np.random.default_rng(seed)
    pw = rng.integers(1, 30, size=(k + 1, V)).astype(np.float64)
    qw = rng.integers(1, 30, size=(k, V)).astype(np.float64)
    return pw / pw.sum(-1, keepdims=True), qw / qw.sum(-1, keepdims=True)


def _emitted_marginal_at(j, p, q, tau, through_full_entry):
    """Distribution of the token emitted at draft position j, given positions < j were accepted,
    measured by probing the oracle's decisions as functions of the uniforms."""
    k, V = q.shape
    shifts = np.arange(k + 1, dtype=np.float64)[:, None] * 0.75 - 1.0        # arbitrary per-row logit offsets
    logits = np.log(p) + shifts

    def run(tok, u):
        n = tok.shape[0]
        qq = np.repeat(q[None], n, 0)
        if through_full_entry:
            # hidden[b, j] = e_j and W[v, j] = logit_j(v): the projection reproduces the table exactly.
            hidden = np.repeat(np.eye(k + 1)[None], n, 0)
            return ref.verify(hidden, np.ascontiguousarray(logits.T), tok, qq, u, tau)
        return ref.verify_from_logits(np.repeat(logits[None], n, 0), tok, qq, u, tau)

    # tokens before j: one with p >= q (always accepted at u = 0); after j: irrelevant
    base_tok = np.array([int(np.argmax(p[i] - q[i])) for i in range(k)])
    # acceptance probability a(x) at position j for every candidate draft token x
    tok = np.repeat(base_tok[None], V, 0)
    tok[:, j] = np.arange(V)

    def accepted(uj):
        u = np.zeros((V, k + 1), np.float32)
        u[:, j] = uj
        return run(tok, u).accept_len > j

    always = accepted(np.full(V, np.float32(1.0) - np.float32(2.0 ** -24)))
    a = np.where(always, 1.0, _threshold(accepted, np.zeros(V), np.ones(V)))
    # residual distribution after a rejection at j: CDF boundaries by bisection on the sampling uniform
    x_rej = int(np.argmin(a))
    marg = np.zeros(V)
    if a[x_rej] < 1.0:
        tok_r = np.repeat(base_tok[None], V - 1, 0)
        tok_r[:, j] = x_rej

        def at_most(us):
            u = np.zeros((V - 1, k + 1), np.float32)
            u[:, j] = np.float32(1.0) - np.float32(2.0 ** -24)
            u[:, k] = us
            out = run(tok_r, u)
            assert np.all(out.accept_len == j)
            return out.next_tok <= np.arange(V - 1)

        cdf = np.concatenate([_threshold(at_most, np.zeros(V - 1), np.ones(V - 1)), [1.0]])
        rho = np.diff(np.concatenate([[0.0], cdf]))
    else:
        rho = np.zeros(V)
    for x in range(V):
        marg[x] += q[j, x] * a[x]
        marg += q[j, x] * (1.0 - a[x]) * rho
    return marg, a


@pytest.mark.parametrize("V", [8, 16])
@pytest.mark.parametrize("full_entry", [False, True])
def test_gate_off_emitted_marginal_equals_p(V, full_entry):
    k = 3
    p, q = _tables(V, k, seed=100 + V)
    reach = 1.0
    for j in range(k):
        marg, a = _emitted_marginal_at(j, p, q, tau=0.0, through_full_entry=full_entry)
        np.testing.assert_allclose(marg, p[j], atol=3e-6)
        # acceptance rate at j: alpha_j = sum_x q(x) a(x) = sum_v min(p, q) = 1 - TV(p, q)
        alpha = float((q[j] * a).sum())
        assert abs(alpha - np.minimum(p[j], q[j]).sum()) < 3e-6
        reach *= alpha
    assert 0.0 < reach < 1.0


@pytest.mark.parametrize("V", [8, 16])
def test_gated_position_emits_the_draft_marginal(V):
    # tau above every entropy (<= ln V): each position is gated, accepted for every u, marginal = q_j.
    k = 2
    p, q = _tables(V, k, seed=200 + V)
    for j in range(k):
        marg, a = _emitted_marginal_at(j, p, q, tau=math.log(V) + 0.1, through_full_entry=False)
        assert np.all(a == 1.0)
        np.testing.assert_allclose(marg, q[j], atol=1e-12)


def test_bonus_token_follows_p_k():
    # all k accepted -> one more token from p_k by the same inverse-CDF rule.
    V, k, G = 8, 2, 8000
    p, q = _tables(V, k, seed=300)
    logits = np.repeat(np.log(p)[None], G, 0)
    tok = np.repeat(np.array([[int(np.argmax(p[i] - q[i])) for i in range(k)]]), G, 0)
    u = np.zeros((G, k + 1), np.float32)
    u[:, k] = (np.arange(G) + 0.5) / G
    out = ref.verify_from_logits(logits, tok, np.repeat(q[None], G, 0), u, 0.0)
    assert np.all(out.accept_len == k)
    np.testing.assert_allclose(np.bincount(out.next_tok, minlength=V) / G, p[k], atol=1.5 / G)


# ------------------------------------------------------------------ the gate (HSD section, Eq. 1)

def test_gate_is_strict_and_tau_semantics():
    V, k = 8, 1
    p, q = _tables(V, k, seed=400)
    l = np.log(p)[None]
    x = int(np.argmax(q[0] - p[0]))                     # ratio < 1
    u = np.array([[0.9999999, 0.5]], np.float32)        # the ratio test would reject
    H0 = ref.softmax_entropy(l[0])[1][0]
    assert ref.verify_from_logits(l, [[x]], q[None], u, H0).accept_len[0] == 0              # H < tau is strict
    assert ref.verify_from_logits(l, [[x]], q[None], u, np.nextafter(H0, 10)).accept_len[0] == 1
    assert ref.verify_from_logits(l, [[x]], q[None], u, INF).accept_len[0] == 1             # +inf: all gated
    assert ref.verify_from_logits(l, [[x]], q[None], u, 0.0).accept_len[0] == 0             # 0: gate off
    assert ref.verify_from_logits(l, [[x]], q[None], u, float("nan")).accept_len[0] == 0    # NaN: gate off
    # the paper's threshold, tau = 1.5 nats: a 4-token uniform row (ln 4 = 1.386) is gated, an 8-token one is not
    for Vu, want in [(4, 1), (8, 0)]:
        lu = np.zeros((1, 2, Vu))
        qu = np.zeros((1, 1, Vu))
        qu[0, 0, 0] = 1.0                               # ratio = (1/Vu)/1 < u
        got = ref.verify_from_logits(lu, [[0]], qu, u, 1.5)
        assert got.accept_len[0] == want


def test_gate_stops_at_first_rejection_only():
    # position 0 gated (low entropy), position 1 rejected by ratio, position 2 never looked at.
    V = 8
    peaked = np.zeros(V); peaked[0] = 12.0              # H ~ 0
    flat = np.zeros(V)                                   # H = ln 8 = 2.08 > 1.5
    l = np.stack([peaked, flat, flat, flat])[None]
    q = np.zeros((1, 3, V)); q[0, :, 5] = 1.0            # draft always token 5 with q = 1: ratio = p(5)
    u = np.array([[0.99, 0.5, 0.0, 0.25]], np.float32)
    out = ref.verify_from_logits(l, [[5, 5, 5]], q, u, 1.5)
    assert out.accept_len[0] == 1                        # j=0 gated although p(5) ~ 0; j=1: 0.5 >= 1/8 rejects
    assert np.isinf(out.margin_accept[0, 0]) and abs(out.margin_accept[0, 1] - (0.5 - 0.125)) < 1e-7
    assert np.isinf(out.margin_gate[0, 2]) and np.isinf(out.margin_accept[0, 2])
    # residual at j=1: p = 1/8 each, q one-hot at 5 -> 7 tokens with 1/8 each; u = 0.25 -> c(v) > 0.21875 -> v = 1
    assert out.next_tok[0] == 1


# ------------------------------------------------------------------ degenerate inputs

def test_degenerate_inputs_are_flagged_not_fatal():
    V = 6
    l = np.zeros((1, 2, V))
    q = np.full((1, 1, V), 1.0 / V)
    ok = ref.verify_from_logits(l, [[2]], q, [[0.5, 0.5]], 0.0)
    assert ok.flags[0] == 0
    bad_tok = ref.verify_from_logits(l, [[V]], q, [[0.0, 0.5]], INF)
    assert bad_tok.accept_len[0] == 0 and bad_tok.flags[0] & ref.FLAG_BAD_TOKEN
    neg_tok = ref.verify_from_logits(l, [[-1]], q, [[0.0, 0.5]], INF)
    assert neg_tok.accept_len[0] == 0 and neg_tok.flags[0] & ref.FLAG_BAD_TOKEN
    big_u = ref.verify_from_logits(l, [[2]], q, [[0.5, 1.0]], INF)
    assert big_u.flags[0] & ref.FLAG_BAD_UNIFORM and big_u.next_tok[0] == V - 1
    # q > p everywhere (sum q = 2): zero residual mass -> draw from p, flagged
    q2 = np.full((1, 1, V), 2.0 / V)
    rz = ref.verify_from_logits(l, [[2]], q2, [[0.9, 0.5]], 0.0)
    assert rz.accept_len[0] == 0 and rz.flags[0] & ref.FLAG_R_ZERO and rz.next_tok[0] == 3
    # q(x) = 0: accepted when p(x) > 0
    q0 = np.zeros((1, 1, V)); q0[0, 0, 0] = 1.0
    assert ref.verify_from_logits(l, [[2]], q0, [[0.9999, 0.5]], 0.0).accept_len[0] == 1
    # empty batch
    e = ref.verify_from_logits(np.zeros((0, 2, V)), np.zeros((0, 1)), np.zeros((0, 1, V)), np.zeros((0, 2)), 1.0)
    assert e.accept_len.shape == (0,)


def test_full_entry_matches_from_logits_composition_on_bf16_inputs():
    # the full entry is step 1 followed by steps 2-6; bf16 q is widened exactly.
    rng = np.random.default_rng(12)
    B, k, H, V = 3, 2, 32, 50
    hid = ref.f32_to_bf16_bits(rng.standard_normal((B, k + 1, H)).astype(np.float32))
    W = ref.f32_to_bf16_bits((rng.standard_normal((V, H)) * 0.3).astype(np.float32))
    lg = (ref.bf16_bits_to_f64(hid).reshape(-1, H) @ ref.bf16_bits_to_f64(W).T).reshape(B, k + 1, V)
    qf = scipy.special.softmax(lg[:, :k] + rng.standard_normal((B, k, V)), axis=-1).astype(np.float32)
    qb = ref.f32_to_bf16_bits(qf)
    tok = rng.integers(0, V, size=(B, k))
    u = rng.random((B, k + 1)).astype(np.float32)
    full = ref.verify(hid, W, tok, qb, u, 1.5, keep_logits=True)
    np.testing.assert_allclose(full.logits, lg, atol=1e-12)
    part = ref.verify_from_logits(full.logits, tok, ref.bf16_bits_to_f64(qb), u, 1.5)
    assert np.array_equal(full.accept_len, part.accept_len) and np.array_equal(full.next_tok, part.next_tok)
    assert np.array_equal(full.entropy, part.entropy)


# ------------------------------------------------------------------ variants: draft-entropy gate, greedy verifier
def test_draft_entropy_matches_scipy_and_closed_forms():
    # H(q) = -sum q ln q: library routine on random rows, ln V on a uniform row, 0 on a one-hot row, and the
    # two-level closed form; bf16-stored rows are used as stored (no renormalisation).
    rng = np.random.default_rng(500)
    V, k = 37, 4
    q = rng.dirichlet(np.ones(V) * 0.3, size=k)
    q[1] = 1.0 / V
    q[2] = 0.0; q[2, 5] = 1.0
    q[3] = 0.25 / (V - 1); q[3, 9] = 0.75
    l = rng.normal(size=(1, k + 1, V))
    got = ref.verify_from_logits(l, [[0] * k], q[None], np.full((1, k + 1), 0.5, np.float32), 0.0,
                                 gate_source=ref.GATE_DRAFT)
    want = [scipy.stats.entropy(q[0]), math.log(V), 0.0, -0.75 * math.log(0.75) - 0.25 * math.log(0.25 / (V - 1))]
    np.testing.assert_allclose(got.draft_entropy[0], want, rtol=0, atol=1e-12)
    qb = ref.f32_to_bf16_bits(q.astype(np.float32))
    got_b = ref.verify_from_logits(l, [[0] * k], qb[None], np.full((1, k + 1), 0.5, np.float32), 0.0,
                                   gate_source=ref.GATE_DRAFT)
    qs = ref.bf16_bits_to_f64(qb)
    want_b = [-(r[r > 0] * np.log(r[r > 0])).sum() for r in qs]      # sum q != 1 after rounding: not scipy's normalised form
    np.testing.assert_allclose(got_b.draft_entropy[0], want_b, rtol=0, atol=1e-12)


def test_draft_entropy_gate_uses_q_not_p():
    # a peaked draft row under a flat target: gated only when the gate looks at the draft, and vice versa
    V = 16
    flat = np.zeros(V)
    peaked = np.zeros(V); peaked[3] = 12.0
    q_peaked = np.exp(peaked) / np.exp(peaked).sum()
    q_flat = np.full(V, 1.0 / V)
    u = np.array([[0.999999, 0.5]], np.float32)
    x = 7                                                   # p(7)/q(7) is tiny under the peaked draft: ratio test rejects
    # target flat (H = ln 16 = 2.77), draft peaked (H ~ 0.001), tau = 1.5
    a = ref.verify_from_logits(np.stack([flat, flat])[None], [[3]], q_peaked[None, None], u, 1.5)
    b = ref.verify_from_logits(np.stack([flat, flat])[None], [[3]], q_peaked[None, None], u, 1.5, gate_source=ref.GATE_DRAFT)
    assert a.accept_len[0] == 0 and b.accept_len[0] == 1   # p(3)/q(3) = (1/16)/0.9999 < u: only the draft gate accepts
    assert abs(b.margin_gate[0, 0] - abs(b.draft_entropy[0, 0] - 1.5)) < 1e-12
    # target peaked (H ~ 0), draft flat: only the target gate accepts the (wrong) draft token
    c = ref.verify_from_logits(np.stack([peaked, flat])[None], [[x]], q_flat[None, None], u, 1.5)
    d = ref.verify_from_logits(np.stack([peaked, flat])[None], [[x]], q_flat[None, None], u, 1.5, gate_source=ref.GATE_DRAFT)
    assert c.accept_len[0] == 1 and d.accept_len[0] == 0
    # the target entropy that is returned does not depend on which one gates
    np.testing.assert_array_equal(c.entropy, d.entropy)


def test_greedy_verifier_is_numpy_argmax():
    # gate off: a draft token survives iff it is the verifier's argmax; the next token is the argmax of the first
    # row that broke (or of row k).  Checked against numpy.argmax on random fp64 logits, ties included.
    rng = np.random.default_rng(501)
    B, k, V = 40, 4, 23
    l = rng.normal(size=(B, k + 1, V)).round(1)            # rounding makes exact ties appear
    am = l.argmax(-1)                                       # numpy: first maximal index = lowest token id
    tok = am[:, :k].copy()
    wrong = rng.random((B, k)) < 0.3
    tok[wrong] = (tok[wrong] + 1 + rng.integers(0, V - 1, wrong.sum())) % V
    q = rng.dirichlet(np.ones(V), size=(B, k))
    u = rng.random((B, k + 1)).astype(np.float32)
    got = ref.verify_from_logits(l, tok, q, u, 0.0, fallback=ref.FALLBACK_GREEDY)
    for b in range(B):
        n = next((j for j in range(k) if tok[b, j] != am[b, j]), k)
        assert got.accept_len[b] == n and got.next_tok[b] == am[b, n]
    assert 0 < got.accept_len.mean() < k
    top2 = np.sort(l, -1)[..., -2:]
    np.testing.assert_allclose(got.margin_argmax, top2[..., 1] - top2[..., 0], atol=1e-12)
    # uniforms play no part
    got2 = ref.verify_from_logits(l, tok, q, 1.0 - u, 0.0, fallback=ref.FALLBACK_GREEDY)
    assert np.array_equal(got.accept_len, got2.accept_len) and np.array_equal(got.next_tok, got2.next_tok)


def test_greedy_verifier_with_gate_keeps_gated_drafts():
    # tau = +inf gates everything: all k drafts kept whatever they are, next token = argmax p_k
    rng = np.random.default_rng(502)
    l = rng.normal(size=(3, 3, 11))
    tok = rng.integers(0, 11, (3, 2))
    q = rng.dirichlet(np.ones(11), size=(3, 2))
    got = ref.verify_from_logits(l, tok, q, np.zeros((3, 3), np.float32), INF, fallback=ref.FALLBACK_GREEDY)
    assert np.all(got.accept_len == 2) and np.array_equal(got.next_tok, l[:, 2].argmax(-1))
    # both variants together through the full entry point on bf16 inputs: same answers as the composition
    H, V, k = 24, 50, 3
    hid = ref.f32_to_bf16_bits(rng.normal(size=(2, k + 1, H)).astype(np.float32))
    W = ref.f32_to_bf16_bits((rng.normal(size=(V, H)) * 0.3).astype(np.float32))
    q = rng.dirichlet(np.ones(V) * 0.2, size=(2, k)).astype(np.float32)
    tok = rng.integers(0, V, (2, k))
    u = rng.random((2, k + 1)).astype(np.float32)
    full = ref.verify(hid, W, tok, q, u, 2.0, keep_logits=True, gate_source=ref.GATE_DRAFT, fallback=ref.FALLBACK_GREEDY)
    comp = ref.verify_from_logits(full.logits, tok, q, u, 2.0, gate_source=ref.GATE_DRAFT, fallback=ref.FALLBACK_GREEDY)
    assert np.array_equal(full.accept_len, comp.accept_len) and np.array_equal(full.next_tok, comp.next_tok)
    np.testing.assert_array_equal(full.draft_entropy, comp.draft_entropy)
