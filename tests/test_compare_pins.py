"""Pins for oracle/compare.py::compare, the bookkeeping every parity verdict goes through.

Each test hands `compare` an answer that is wrong in exactly one way and checks that the report says so, or an
answer that differs from the oracle's only inside one of the stated 1e-4 decision margins and checks that it is
counted as a margin case and not as a failure.  The "answers" are the oracle's own outputs with a planted
deviation: nothing here comes from the CUDA path.
"""
import numpy as np
import pytest

from oracle import compare, ref


def _case(seed=3, B=6, k=3, V=16, tau=0.0):
    """A small problem given directly by fp64 logits; the gate is off (tau = 0), so every position runs the ratio test."""
    rng = np.random.default_rng(seed)
    logits = rng.normal(0.0, 1.5, (B, k + 1, V))
    q = np.exp(logits[:, :k] + rng.normal(0.0, 0.7, (B, k, V)))
    q /= q.sum(-1, keepdims=True)
    tok = np.stack([[rng.choice(V, p=q[b, j]) for j in range(k)] for b in range(B)]).astype(np.int32)
    u = rng.random((B, k + 1)).astype(np.float32)
    return logits, tok, q.astype(np.float32), u, tau


def _oracle(logits, tok, q, u, tau):
    return ref.verify_from_logits(logits, tok, q, u, tau)


def _report(orc, q, u, **planted):
    got = dict(accept_len=orc.accept_len.copy(), next_tok=orc.next_tok.copy(),
               entropy=orc.entropy.astype(np.float32), logZ=orc.logZ.astype(np.float32),
               logits=orc.logits.astype(np.float32))
    got.update(planted)
    return compare.compare(orc, q, u, got["accept_len"], got["next_tok"], got["entropy"], got["logZ"], got["logits"])


def test_the_oracles_own_answer_passes():
    logits, tok, q, u, tau = _case()
    orc = _oracle(logits, tok, q, u, tau)
    rep = _report(orc, q, u)
    assert rep.ok and rep.accept_exact == 6 and rep.token_exact == 6
    assert rep.accept_margin_cases == 0 and rep.token_margin_cases == 0


@pytest.mark.parametrize("delta", [+1, -1])
def test_wrong_accept_len_outside_the_margin_fails(delta):
    logits, tok, q, u, tau = _case()
    orc = _oracle(logits, tok, q, u, tau)
    # a sequence whose deciding position is nowhere near a tie, and whose accept_len can move by delta
    for b in range(len(orc.accept_len)):
        n = int(orc.accept_len[b])
        if not 0 <= n + delta <= 3:
            continue
        j = min(n, n + delta)
        if min(orc.margin_gate[b, j], orc.margin_accept[b, j]) > 10 * compare.MARGIN:
            break
    else:
        pytest.skip("no suitable sequence in this draw")
    bad = orc.accept_len.copy()
    bad[b] += delta
    rep = _report(orc, q, u, accept_len=bad)
    assert not rep.ok and len(rep.accept_failures) == 1 and rep.accept_failures[0][0] == b
    assert rep.accept_margin_cases == 0


def test_wrong_token_far_from_the_uniform_fails():
    logits, tok, q, u, tau = _case()
    orc = _oracle(logits, tok, q, u, tau)
    bad = orc.next_tok.copy()
    b = int(np.argmax(orc.margin_cdf))                     # the draw furthest from any CDF edge
    assert orc.margin_cdf[b] > 10 * compare.MARGIN
    bad[b] = (bad[b] + 7) % 16
    rep = _report(orc, q, u, next_tok=bad)
    assert not rep.ok and len(rep.token_failures) == 1 and rep.token_failures[0][0] == b
    assert rep.token_margin_cases == 0


def test_token_out_of_range_fails():
    logits, tok, q, u, tau = _case()
    orc = _oracle(logits, tok, q, u, tau)
    for wrong in (-1, 16, 1 << 20):
        bad = orc.next_tok.copy()
        bad[0] = wrong
        assert not _report(orc, q, u, next_tok=bad).ok


def test_entropy_and_logZ_beyond_tolerance_fail():
    logits, tok, q, u, tau = _case()
    orc = _oracle(logits, tok, q, u, tau)
    e = orc.entropy.astype(np.float32)
    e[2, 1] += 3e-3
    rep = _report(orc, q, u, entropy=e)
    assert not rep.ok and rep.max_entropy_err > compare.ENTROPY_ATOL
    z = orc.logZ.astype(np.float32)
    z[4, 0] -= 3e-3
    rep = _report(orc, q, u, logZ=z)
    assert not rep.ok and rep.max_logZ_err > compare.ENTROPY_ATOL
    # and just inside the tolerance passes
    e = orc.entropy.astype(np.float32)
    e[2, 1] += 1e-3
    assert _report(orc, q, u, entropy=e).ok


def test_one_logit_off_by_five_per_cent_fails():
    logits, tok, q, u, tau = _case()
    orc = _oracle(logits, tok, q, u, tau)
    l = orc.logits.astype(np.float32)
    i = np.unravel_index(np.argmax(np.abs(l)), l.shape)     # |l| > 1 there, so 5 % is beyond 1e-2 relative
    assert abs(l[i]) > 1.0
    l[i] *= 1.05
    rep = _report(orc, q, u, logits=l)
    assert not rep.ok and rep.max_logit_rel_err > compare.LOGIT_RTOL


def test_accept_decision_inside_the_ratio_margin_is_counted_not_failed():
    """u placed 3e-5 below min(1, p/q) at position 0: the oracle accepts; an answer that rejects there is a margin case."""
    logits, tok, q, u, tau = _case(seed=11)
    base = _oracle(logits, tok, q, u, tau)
    b = 0
    p0 = np.exp(logits[b, 0] - base.logZ[b, 0])
    x = int(np.argmax(q[b, 0] - p0))                       # a token the draft over-weights: ratio < 1
    ratio = p0[x] / float(q[b, 0, x])
    assert ratio < 0.99
    tok = tok.copy()
    tok[b, 0] = x
    u = u.copy()
    u[b, 0] = np.float32(ratio - 3e-5)
    orc = _oracle(logits, tok, q, u, tau)
    assert orc.accept_len[b] >= 1 and orc.margin_accept[b, 0] < compare.MARGIN
    bad = orc.accept_len.copy()
    bad[b] = 0                                             # the other side of the near-tie
    rep = _report(orc, q, u, accept_len=bad)
    assert rep.ok and rep.accept_margin_cases == 1 and not rep.accept_failures
    # the same deviation with u well away from the ratio is a failure
    u[b, 0] = np.float32(ratio - 0.05) if ratio > 0.06 else np.float32(0.0)
    orc2 = _oracle(logits, tok, q, u, tau)
    if orc2.margin_accept[b, 0] > 10 * compare.MARGIN and orc2.accept_len[b] >= 1:
        bad = orc2.accept_len.copy()
        bad[b] = 0
        assert not _report(orc2, q, u, accept_len=bad).ok


def test_gate_decision_inside_the_entropy_margin_is_counted_not_failed():
    logits, tok, q, u, _ = _case(seed=5, B=12)
    plain = _oracle(logits, tok, q, u, 0.0)                # gate off everywhere
    rejected_at_0 = [b for b in range(12) if plain.accept_len[b] == 0 and plain.margin_accept[b, 0] > 10 * compare.MARGIN]
    assert rejected_at_0, "the draw holds no sequence whose first draft token is rejected"
    b = rejected_at_0[0]
    H0 = float(plain.entropy[b, 0])
    # every other position of every sequence stays clear of tau by construction of the draw (entropies differ by > 1e-3)
    tau = H0 + 4e-5                                        # the gate fires at (b, 0) by a hair: the oracle accepts there
    orc = _oracle(logits, tok, q, u, tau)
    assert orc.margin_gate[b, 0] < compare.MARGIN and orc.accept_len[b] >= 1
    other = orc.accept_len.copy()
    other[b] = 0                                           # the answer of a side whose H came out a hair above tau
    rep = _report(orc, q, u, accept_len=other)
    assert rep.ok and rep.accept_margin_cases == 1 and not rep.accept_failures
    # with tau clearly above H0 the same answer is an error
    orc = _oracle(logits, tok, q, u, H0 + 0.01)
    other = orc.accept_len.copy()
    other[b] = 0
    assert not _report(orc, q, u, accept_len=other).ok


def test_token_next_to_a_cdf_edge_is_a_margin_case_and_further_away_a_failure():
    logits, tok, q, u, tau = _case(seed=7)
    orc = _oracle(logits, tok, q, u, tau)
    b = 2
    n = int(orc.accept_len[b])
    k = 3
    p = np.exp(orc.logits[b, n] - orc.logZ[b, n])
    r = np.maximum(0.0, p - q[b, n].astype(np.float64)) if n < k else p
    c = np.cumsum(r) / r.sum()
    # put the uniform 2e-5 above an inner CDF edge: the oracle picks the token after the edge, the one before it is
    # within the margin, the one two places before is not
    cand = [v for v in range(1, 15) if r[v] > 1e-3 and r[v + 1] > 1e-3 and r[v - 1] > 1e-3]
    v = cand[0]
    u = u.copy()
    u[b, k] = np.float32(c[v] + 2e-5)
    orc = _oracle(logits, tok, q, u, tau)
    assert int(orc.accept_len[b]) == n and int(orc.next_tok[b]) == v + 1
    near = orc.next_tok.copy()
    near[b] = v
    rep = _report(orc, q, u, next_tok=near)
    assert rep.ok and rep.token_margin_cases == 1 and not rep.token_failures
    far = orc.next_tok.copy()
    far[b] = v - 1
    rep = _report(orc, q, u, next_tok=far)
    assert not rep.ok and len(rep.token_failures) == 1


def test_token_is_not_compared_where_accept_len_differs_inside_the_margin():
    logits, tok, q, u, tau = _case(seed=11)
    base = _oracle(logits, tok, q, u, tau)
    b = 0
    p0 = np.exp(logits[b, 0] - base.logZ[b, 0])
    x = int(np.argmax(q[b, 0] - p0))
    ratio = p0[x] / float(q[b, 0, x])
    tok = tok.copy(); tok[b, 0] = x
    u = u.copy(); u[b, 0] = np.float32(ratio - 3e-5)
    orc = _oracle(logits, tok, q, u, tau)
    bad_n = orc.accept_len.copy(); bad_n[b] = 0
    bad_t = orc.next_tok.copy(); bad_t[b] = (bad_t[b] + 5) % 16
    rep = _report(orc, q, u, accept_len=bad_n, next_tok=bad_t)
    assert rep.ok and rep.token_compared == len(orc.accept_len) - 1
