"""Multi-round HSD decode loop around hola_verify (the HSD part of Algorithm 1, run as a loop).

Each round: the draft model proposes k tokens with their distributions q, the verifier's hidden states for the
k+1 positions are formed, ONE hola_verify call decides how many drafts survive (entropy gate, Eq. 1, then the
verifier's test) and which token follows them, and the context grows by accept_len + 1 tokens.  The HSD section's
claim is that verifier invocations drop from one per token to one per round; the loop reports exactly that ratio
(tokens emitted per verifier call) together with the time spent inside the verify step.

The two models are seeded synthetic stand-ins (the paper's trained draft / verifier checkpoints are not used): both
read the context through embedding tables and share the LM head; the verifier sees two tokens back, the draft only
one, so q is close to p but not equal.  They are harness code in stock torch; every step of the verify path itself
runs in the CUDA library.  Everything stays on the device: no host read-back inside the loop.
"""
from __future__ import annotations

import argparse
import json
import math
from dataclasses import dataclass, field

import torch

from . import binding


class SyntheticPair:
    """Seeded draft / verifier stand-ins over a vocabulary V with hidden size H."""

    def __init__(self, V: int, H: int, seed: int, device, sharpness: float = 3.0, w_std: float = 0.02):
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        self.V, self.H, self.device = V, H, device
        self.W_lm = (torch.randn((V, H), generator=g, device=device) * w_std).to(torch.bfloat16).contiguous()
        self.E1 = torch.randn((V, H), generator=g, device=device)
        self.E2 = torch.randn((V, H), generator=g, device=device)
        # unit-norm hidden states times `gain`: logits then have a standard deviation of gain * w_std, here spread
        # over about 0.75 .. 5.25 by context, so that some positions are peaked (entropy below tau, the gate fires)
        # and others flat
        self.gain = (sharpness / w_std) * (0.25 + 1.5 * torch.rand((V,), generator=g, device=device))

    def _norm(self, h, prev1):
        return h / h.norm(dim=-1, keepdim=True) * self.gain[prev1].unsqueeze(-1)

    def target_hidden(self, prev1: torch.Tensor, prev2: torch.Tensor) -> torch.Tensor:
        """Verifier trunk stand-in: hidden state for the position that follows (..., prev2, prev1).  bf16 [..., H]."""
        return self._norm(self.E1[prev1] + 0.35 * self.E2[prev2], prev1).to(torch.bfloat16)

    def draft_probs(self, prev1: torch.Tensor) -> torch.Tensor:
        """Draft model stand-in: q(. | prev1), fp32 [..., V]."""
        h = self._norm(self.E1[prev1], prev1).to(torch.bfloat16).float()
        return torch.softmax(h @ self.W_lm.float().T, dim=-1)


@dataclass
class RoundRecord:
    """What one round handed to hola_verify and got back (device tensors)."""
    hidden: torch.Tensor
    draft_tok: torch.Tensor
    draft_q: torch.Tensor
    uniforms: torch.Tensor
    out: binding.VerifyOutputs


@dataclass
class DecodeResult:
    tokens: torch.Tensor        # int64 [B, 2 + rounds * (k + 1)], first two are the prompt
    lengths: torch.Tensor       # int64 [B]: tokens present per sequence
    rounds: int
    verify_ms: float            # CUDA-event time of all hola_verify calls
    total_ms: float             # CUDA-event time of the whole loop (draft + trunk stand-ins included)
    accepted: torch.Tensor      # int64 [B]: draft tokens kept, summed over the rounds
    records: list = field(default_factory=list)


def hsd_decode(ctx: binding.HolaVerify, models: SyntheticPair, prompt: torch.Tensor, k: int, tau: float, rounds: int,
               seed: int, gate_source: int = 0, fallback: int = 0, keep_records: bool = False) -> DecodeResult:
    """Runs `rounds` draft-and-verify rounds for a batch of sequences.  prompt: int64 [B, 2] (two context tokens)."""
    dev = prompt.device
    B = prompt.shape[0]
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    cap = 2 + rounds * (k + 1)
    tokens = torch.zeros((B, cap), dtype=torch.int64, device=dev)
    tokens[:, :2] = prompt
    lengths = torch.full((B,), 2, dtype=torch.int64, device=dev)
    accepted = torch.zeros((B,), dtype=torch.int64, device=dev)
    rows = torch.arange(B, device=dev)
    steps = torch.arange(k + 1, device=dev)
    out = ctx.alloc_outputs(B, k, False)
    records = []
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * rounds + 2)]
    ev[-2].record()
    for r in range(rounds):
        last1 = tokens[rows, lengths - 1]
        last2 = tokens[rows, lengths - 2]
        # draft: k tokens, each drawn from the distribution as stored (bf16), conditioned on the previous one
        draft_tok = torch.empty((B, k), dtype=torch.int64, device=dev)
        draft_q = torch.empty((B, k, models.V), dtype=torch.bfloat16, device=dev)
        prev = last1
        for j in range(k):
            q = models.draft_probs(prev).to(torch.bfloat16)
            draft_q[:, j] = q
            prev = torch.multinomial(q.float(), 1, generator=g).squeeze(1)
            draft_tok[:, j] = prev
        # verifier hidden states for the k + 1 positions: position j follows (.., c2, c1) = context + drafts < j
        c1 = torch.cat([last1[:, None], draft_tok], dim=1)                       # [B, k+1]
        c2 = torch.cat([last2[:, None], last1[:, None], draft_tok[:, :-1]], dim=1) if k > 0 else last2[:, None]
        hidden = models.target_hidden(c1, c2).contiguous()                      # [B, k+1, H]
        uniforms = torch.rand((B, k + 1), generator=g, device=dev, dtype=torch.float32)
        tok32 = draft_tok.to(torch.int32).contiguous()
        ev[2 * r].record()
        ctx.hola_verify(hidden, models.W_lm, tok32, draft_q, uniforms, tau, out=out, gate_source=gate_source,
                        fallback=fallback)
        ev[2 * r + 1].record()
        # the context grows by the accepted drafts and the verifier's token (no host read-back)
        n = out.accept_len.to(torch.int64)
        new = torch.cat([draft_tok, torch.zeros((B, 1), dtype=torch.int64, device=dev)], dim=1)
        new[rows, n] = out.next_tok.to(torch.int64)
        keep = steps[None, :] <= n[:, None]
        pos = (lengths[:, None] + steps[None, :]).clamp_max(cap - 1)
        tokens[rows[:, None].expand(-1, k + 1)[keep], pos[keep]] = new[keep]
        lengths = lengths + n + 1
        accepted += n
        if keep_records:
            records.append(RoundRecord(hidden, tok32, draft_q, uniforms, binding.VerifyOutputs(
                out.accept_len.clone(), out.next_tok.clone(), out.entropy.clone(), out.logZ.clone(), None,
                out.status.clone(), out.draft_entropy.clone())))
    ev[-1].record()
    torch.cuda.synchronize()
    verify_ms = sum(ev[2 * r].elapsed_time(ev[2 * r + 1]) for r in range(rounds))
    return DecodeResult(tokens, lengths, rounds, verify_ms, ev[-2].elapsed_time(ev[-1]), accepted, records)


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--B", type=int, default=16)
    ap.add_argument("--k", type=int, default=5)
    ap.add_argument("--H", type=int, default=4096)
    ap.add_argument("--V", type=int, default=32000)
    ap.add_argument("--rounds", type=int, default=40)
    ap.add_argument("--tau", type=float, default=1.5)
    ap.add_argument("--gate", default="target", choices=["target", "draft"])
    ap.add_argument("--fallback", default="sample", choices=["sample", "greedy"])
    ap.add_argument("--seed", type=int, default=2506189520)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("driver: no CUDA device; the verify path has no CPU fallback")
    dev = torch.device("cuda", torch.cuda.current_device())
    models = SyntheticPair(args.V, args.H, args.seed, dev)
    prompt = torch.randint(0, args.V, (args.B, 2), device=dev, generator=torch.Generator(device=dev).manual_seed(args.seed + 1))
    gs, fb = int(args.gate == "draft"), int(args.fallback == "greedy")
    with binding.HolaVerify(args.B, args.k, args.H, args.V) as ctx:
        hsd_decode(ctx, models, prompt, args.k, args.tau, 3, args.seed, gs, fb)          # warm-up
        res = hsd_decode(ctx, models, prompt, args.k, args.tau, args.rounds, args.seed, gs, fb)
    emitted = int((res.lengths - 2).sum().item())
    print(json.dumps({
        "workload": f"multi-round HSD decode: B={args.B} k={args.k} H={args.H} V={args.V}, synthetic draft/verifier pair",
        "tau": args.tau, "gate": args.gate, "fallback": args.fallback, "rounds": res.rounds,
        "verifier_calls_per_sequence": res.rounds, "tokens_emitted": emitted,
        "tokens_per_verifier_call": emitted / (args.B * res.rounds),
        "draft_acceptance": float(res.accepted.sum().item()) / (args.B * res.rounds * max(1, args.k)),
        "verify_ms_per_round": res.verify_ms / res.rounds,
        "tokens_per_s_verify_only": emitted / (res.verify_ms * 1e-3),
        "loop_ms_per_round": res.total_ms / res.rounds,
        "tokens_per_s_whole_loop": emitted / (res.total_ms * 1e-3),
        "data": "synthetic"}))


if __name__ == "__main__":
    main()
