"""Parity bookkeeping between a result under test and the CPU oracle (test infrastructure).

The comparison rule:
  * entropy and logZ: absolute error <= 2e-3;
  * logits (when available): |l - l_ref| <= 1e-2 * max(|l_ref|, 1);
  * accept_len: equal, except where the oracle's own decision margin at a position that decided the outcome,
    |H - tau| or |u - min(1, p/q)|, is below 1e-4 - such cases are counted, not failed;
  * next_tok: compared only where accept_len agrees; equal, except where the supplied uniform lies within 1e-4
    (in probability mass) of the oracle's CDF interval of the token under test - counted separately;
  * greedy verifier: the accept decision's margin is the gap between the two largest logits of that row, and a
    next_tok mismatch is a margin case only where that gap is below 1e-4.
Nothing here is used by the product path.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import ref

ENTROPY_ATOL = 2e-3
LOGIT_RTOL = 1e-2
MARGIN = 1e-4


def torch_to_numpy(t):
    """torch tensor -> numpy; bf16 becomes uint16 bit patterns."""
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def run_oracle(w, keep_logits: bool = True, nthreads: int = 0, gate_source: int = 0,
               fallback: int = 0) -> ref.RefResult:
    """Runs the oracle on a workload object with torch tensors hidden, W_lm, draft_tok, draft_q, uniforms, tau."""
    return ref.verify(torch_to_numpy(w.hidden), torch_to_numpy(w.W_lm), torch_to_numpy(w.draft_tok),
                      torch_to_numpy(w.draft_q), torch_to_numpy(w.uniforms), w.tau, keep_logits=keep_logits,
                      nthreads=nthreads, gate_source=gate_source, fallback=fallback)


@dataclass
class ParityReport:
    n_seq: int = 0
    max_entropy_err: float = 0.0
    max_logZ_err: float = 0.0
    max_logit_rel_err: float = 0.0
    accept_exact: int = 0
    accept_margin_cases: int = 0
    accept_failures: list = field(default_factory=list)
    token_compared: int = 0
    token_exact: int = 0
    token_margin_cases: int = 0
    token_failures: list = field(default_factory=list)

    @property
    def ok(self) -> bool:
        return (self.max_entropy_err <= ENTROPY_ATOL and self.max_logZ_err <= ENTROPY_ATOL
                and self.max_logit_rel_err <= LOGIT_RTOL and not self.accept_failures and not self.token_failures)

    def summary(self) -> str:
        return (f"seq={self.n_seq} |dH|max={self.max_entropy_err:.2e} |dlogZ|max={self.max_logZ_err:.2e} "
                f"logit_rel_max={self.max_logit_rel_err:.2e} accept exact={self.accept_exact} "
                f"margin={self.accept_margin_cases} fail={len(self.accept_failures)} | token compared="
                f"{self.token_compared} exact={self.token_exact} margin={self.token_margin_cases} "
                f"fail={len(self.token_failures)}")


def _q_row_f64(q_np: np.ndarray, b: int, j: int) -> np.ndarray:
    row = q_np[b, j]
    return ref.bf16_bits_to_f64(row) if row.dtype == np.uint16 else row.astype(np.float64)


def compare(oracle: ref.RefResult, q_np: np.ndarray, uniforms: np.ndarray, accept_len, next_tok, entropy, logZ,
            logits=None) -> ParityReport:
    """All arguments after `oracle` are numpy arrays for the same sequences, in the same order."""
    B, k1 = oracle.entropy.shape
    k = k1 - 1
    rep = ParityReport(n_seq=B)
    if B == 0:
        return rep
    rep.max_entropy_err = float(np.max(np.abs(entropy.astype(np.float64) - oracle.entropy)))
    rep.max_logZ_err = float(np.max(np.abs(logZ.astype(np.float64) - oracle.logZ)))
    if logits is not None and oracle.logits is not None:
        denom = np.maximum(np.abs(oracle.logits), 1.0)
        rep.max_logit_rel_err = float(np.max(np.abs(logits.astype(np.float64) - oracle.logits) / denom))
    for b in range(B):
        n_ref, n_got = int(oracle.accept_len[b]), int(accept_len[b])
        if n_ref == n_got:
            rep.accept_exact += 1
        else:
            # the two runs part ways at position j = min(n): a margin case only if the oracle was near a tie there
            j = min(n_ref, n_got)
            m = min(oracle.margin_gate[b, j], oracle.margin_accept[b, j]) if j < k else np.inf
            if m < MARGIN:
                rep.accept_margin_cases += 1
            else:
                rep.accept_failures.append((b, n_ref, n_got, float(m)))
            continue
        rep.token_compared += 1
        t_ref, t_got = int(oracle.next_tok[b]), int(next_tok[b])
        if t_ref == t_got:
            rep.token_exact += 1
            continue
        ok = False
        if oracle.fallback == ref.FALLBACK_GREEDY:
            # greedy verifier: the two sides may differ only where the top two logits of that row nearly tie
            ok = 0 <= t_got < (oracle.logits.shape[2] if oracle.logits is not None else 1 << 30) and \
                oracle.margin_argmax[b, n_ref] < MARGIN
        elif oracle.logits is not None and 0 <= t_got < oracle.logits.shape[2]:
            p = np.exp(oracle.logits[b, n_ref] - oracle.logZ[b, n_ref])
            r = np.maximum(0.0, p - _q_row_f64(q_np, b, n_ref)) if n_ref < k else p
            R = r.sum()
            if R <= 0:
                r, R = p, p.sum()
            c = np.cumsum(r) / R
            lo = c[t_got - 1] if t_got > 0 else 0.0
            u = float(uniforms[b, k])
            ok = (lo - MARGIN) <= u <= (c[t_got] + MARGIN) and r[t_got] > 0
        if ok:
            rep.token_margin_cases += 1
        else:
            rep.token_failures.append((b, t_ref, t_got, float(oracle.margin_cdf[b])))
    return rep
