"""Seeded synthetic inputs for the verify step.

This module only *makes arrays*: it serves the CUDA path, the CPU oracle and the benchmark alike, and holds none
of the method's arithmetic (no accept test, no residual, no sampling).  It uses stock torch operations (matmul,
softmax, multinomial) to shape the inputs the way the workload descriptions ask: a draft distribution q that is
a noisy copy of the target softmax, draft tokens drawn from q, target rows with a prescribed entropy spread.

The paper evaluates on GSM8K and ARC with pretrained checkpoints; neither is used here.  Only LM-head shapes of
7B/8B-class models and a plausible entropy / acceptance structure are reproduced, from a fixed seed.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

SEED_BASE = 250618952 * 10
PAPER_TAU = 1.5          # entropy threshold, Hyperparameters section


@dataclass
class VerifyInputs:
    name: str
    B: int
    k: int
    H: int
    V: int
    tau: float
    hidden: torch.Tensor      # bf16 [B, k+1, H]
    W_lm: torch.Tensor        # bf16 [V, H]
    draft_tok: torch.Tensor   # int32 [B, k]
    draft_q: torch.Tensor     # bf16 or fp32 [B, k, V]
    uniforms: torch.Tensor    # fp32 [B, k+1]
    notes: dict = field(default_factory=dict)

    @property
    def M(self) -> int:
        return self.B * (self.k + 1)

    def slice(self, seqs) -> "VerifyInputs":
        """The same workload restricted to the given sequences (sequences are independent)."""
        idx = torch.as_tensor(list(seqs), device=self.hidden.device, dtype=torch.long)
        return VerifyInputs(self.name + "[subset]", len(idx), self.k, self.H, self.V, self.tau,
                            self.hidden[idx].contiguous(), self.W_lm, self.draft_tok[idx].contiguous(),
                            self.draft_q[idx].contiguous(), self.uniforms[idx].contiguous(), dict(self.notes))


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _target_logits(hidden_bf16: torch.Tensor, W_bf16: torch.Tensor) -> torch.Tensor:
    """fp32 logits of the rounded inputs, for shaping q only (input synthesis, not the product path)."""
    B, k1, H = hidden_bf16.shape
    h = hidden_bf16.reshape(B * k1, H).float()
    if hidden_bf16.is_cuda:
        prev = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = False
        try:
            out = h @ W_bf16.float().T
        finally:
            torch.backends.cuda.matmul.allow_tf32 = prev
    else:
        out = h @ W_bf16.float().T
    return out.reshape(B, k1, -1)


def _draft_from_logits(logits_k: torch.Tensor, sigma, temp: float, g: torch.Generator, q_dtype) -> tuple:
    """q = softmax((logits + sigma * N(0,1)) / temp); tokens ~ q.  sigma may be a per-sequence column."""
    noise = torch.randn(logits_k.shape, generator=g, device=logits_k.device, dtype=torch.float32)
    q = torch.softmax((logits_k + noise * sigma) / temp, dim=-1)
    B, k, V = q.shape
    if k == 0:
        tok = torch.zeros((B, 0), dtype=torch.int32, device=q.device)
    else:
        q_store = q.to(q_dtype)
        # tokens are drawn from the distribution as stored, so that q(x) > 0 for every draft token
        tok = torch.multinomial(q_store.float().reshape(B * k, V).clamp_min(0), 1, generator=g).reshape(B, k).int()
        q = q_store
    return q.to(q_dtype).contiguous(), tok.contiguous()


def _uniforms(B: int, k: int, g: torch.Generator, device) -> torch.Tensor:
    return torch.rand((B, k + 1), generator=g, device=device, dtype=torch.float32)


def _row_entropy(logits: torch.Tensor) -> torch.Tensor:
    lp = torch.log_softmax(logits.double(), dim=-1)
    return -(lp.exp() * lp).sum(-1)


def gaussian_head(name: str, B: int, k: int, H: int, V: int, *, seed: int, device="cpu", w_std=0.02, h_std=1.0,
                  sigma=1.0, temp=1.0, q_dtype=torch.bfloat16, tau: float | None = PAPER_TAU,
                  sigma_far: float | None = None) -> VerifyInputs:
    """hidden ~ N(0, h_std), W ~ N(0, w_std), both rounded to bf16; q a noisy copy of the target softmax.

    With sigma_far set, the first half of the sequences uses noise `sigma` (q close to p, long accepted runs)
    and the second half `sigma_far` (early rejection).  tau=None picks the median target entropy over the k
    draft positions of sequence 0 (midpoint of the two middle values when k is even).
    """
    g = _gen(seed, device)
    hidden = (torch.randn((B, k + 1, H), generator=g, device=device) * h_std).to(torch.bfloat16)
    W = (torch.randn((V, H), generator=g, device=device) * w_std).to(torch.bfloat16)
    logits = _target_logits(hidden, W)
    sig = sigma
    if sigma_far is not None:
        sig = torch.full((B, 1, 1), float(sigma), device=device)
        sig[B // 2:] = float(sigma_far)
    q, tok = _draft_from_logits(logits[:, :k], sig, temp, g, q_dtype)
    u = _uniforms(B, k, g, device)
    notes = {}
    if tau is None:
        ent = _row_entropy(logits[0, :k]) if k > 0 else _row_entropy(logits[0, :1])
        tau = float(ent.median()) if ent.numel() % 2 else float(ent.sort().values[ent.numel() // 2 - 1:ent.numel() // 2 + 1].mean())
        notes["tau_rule"] = "median target entropy over the k draft positions"
    return VerifyInputs(name, B, k, H, V, float(tau), hidden.contiguous(), W.contiguous(), tok, q, u, notes)


def entropy_spread_head(name: str, B: int, k: int, H: int, V: int, *, seed: int, device="cpu", w_std=0.02,
                        h_lo=0.5, h_hi=8.0, sigma=1.0, tau=PAPER_TAU, q_dtype=torch.bfloat16) -> VerifyInputs:
    """Each hidden row is N(0,1) scaled by a factor found by bisection (entropy falls as the scale grows) so
    that target entropies are spread evenly over [h_lo, h_hi] nats, in a seeded random order over the rows."""
    g = _gen(seed, device)
    M = B * (k + 1)
    base = torch.randn((M, H), generator=g, device=device)
    W = (torch.randn((V, H), generator=g, device=device) * w_std).to(torch.bfloat16)
    z = _target_logits(base.to(torch.bfloat16).reshape(B, k + 1, H), W).reshape(M, V)
    want = torch.linspace(h_lo, min(h_hi, 0.95 * torch.log(torch.tensor(float(V))).item()), M, device=device)
    want = want[torch.randperm(M, generator=g, device=device)].double()
    lo = torch.full((M, 1), 1e-3, device=device)
    hi = torch.full((M, 1), 64.0, device=device)
    for _ in range(40):
        mid = 0.5 * (lo + hi)
        too_flat = (_row_entropy(z * mid) > want).unsqueeze(1)
        lo = torch.where(too_flat, mid, lo)
        hi = torch.where(too_flat, hi, mid)
    gamma = 0.5 * (lo + hi)
    hidden = (base * gamma).to(torch.bfloat16).reshape(B, k + 1, H)
    logits = _target_logits(hidden, W)
    q, tok = _draft_from_logits(logits[:, :k], sigma, 1.0, g, q_dtype)
    u = _uniforms(B, k, g, device)
    notes = {"entropy_target_lo": h_lo, "entropy_target_hi": float(want.max())}
    return VerifyInputs(name, B, k, H, V, float(tau), hidden.contiguous(), W.contiguous(), tok, q, u, notes)


def peaked_flat_head(name: str, B: int, k: int, H: int, V: int, *, seed: int, device="cpu", w_std=0.02,
                     gap=15.0, flat_std=0.05, sigma=1.0, tau=PAPER_TAU, q_dtype=torch.bfloat16) -> VerifyInputs:
    """Even rows peaked (hidden = a * W[v*], a chosen so the top logit leads the runner-up by `gap`), odd rows
    flat (hidden ~ flat_std * N(0,1), near-uniform target), so both branches of the entropy gate are taken."""
    g = _gen(seed, device)
    M = B * (k + 1)
    W = (torch.randn((V, H), generator=g, device=device) * w_std).to(torch.bfloat16)
    hidden = torch.randn((M, H), generator=g, device=device) * flat_std
    peaked_rows = torch.arange(0, M, 2, device=device)
    vstar = torch.randint(0, V, (peaked_rows.numel(),), generator=g, device=device)
    Wf = W.float()
    step = 256
    for s in range(0, peaked_rows.numel(), step):
        vs = vstar[s:s + step]
        dots = Wf[vs] @ Wf.T                                  # [n, V]
        top = dots.gather(1, vs[:, None]).squeeze(1)
        dots.scatter_(1, vs[:, None], float("-inf"))
        a = gap / (top - dots.max(dim=1).values)
        hidden[peaked_rows[s:s + step]] = Wf[vs] * a[:, None]
    hidden = hidden.to(torch.bfloat16).reshape(B, k + 1, H)
    logits = _target_logits(hidden, W)
    q, tok = _draft_from_logits(logits[:, :k], sigma, 1.0, g, q_dtype)
    u = _uniforms(B, k, g, device)
    return VerifyInputs(name, B, k, H, V, float(tau), hidden.contiguous(), W.contiguous(), tok, q, u,
                        {"gap": gap})


CONFIG_SHAPES = {
    "tiny":        dict(B=1, k=4, H=64, V=1000),
    "edge":        dict(B=1, k=4, H=4096, V=32000),
    "batched":     dict(B=64, k=5, H=4096, V=32000),
    "large_vocab": dict(B=64, k=5, H=4096, V=128256),
    "wide":        dict(B=256, k=8, H=8192, V=128256),
    "large_vocab_b32": dict(B=32, k=5, H=4096, V=128256),
}


def make_config(name: str, device="cpu", *, tau: float | None = None, seed_offset: int = 0,
                **shape_override) -> VerifyInputs:
    """The five named workloads (plus the B=32 large-vocab variant).  shape_override shrinks a recipe for CPU
    tests (e.g. V=4096, H=256) without changing how the arrays are made."""
    if name not in CONFIG_SHAPES:
        raise KeyError(f"unknown workload {name!r}; known: {sorted(CONFIG_SHAPES)}")
    shp = dict(CONFIG_SHAPES[name])
    shp.update(shape_override)
    idx = list(CONFIG_SHAPES).index(name) + 1
    seed = SEED_BASE + idx + seed_offset
    if name == "tiny":
        w = gaussian_head(name, **shp, seed=seed, device=device, w_std=0.05, sigma=0.5, q_dtype=torch.float32,
                          tau=tau)
    elif name == "edge":
        w = gaussian_head(name, **shp, seed=seed, device=device, sigma=1.0, temp=1.2,
                          tau=PAPER_TAU if tau is None else tau)
    elif name == "batched":
        w = gaussian_head(name, **shp, seed=seed, device=device, sigma=0.1, sigma_far=2.0,
                          tau=PAPER_TAU if tau is None else tau)
    elif name in ("large_vocab", "large_vocab_b32"):
        w = entropy_spread_head(name, **shp, seed=seed, device=device, tau=2.0 if tau is None else tau)
    else:
        w = peaked_flat_head(name, **shp, seed=seed, device=device, tau=PAPER_TAU if tau is None else tau)
    return w
