"""Vocabulary-parallel form of the verify step: every rank (normally one GPU) holds a contiguous range of the
vocabulary rows of W_lm and of the vocabulary axis of draft_q; hidden states, draft tokens, uniforms and the k draft
probabilities q_j(x_j) are the same everywhere.  A step is three library calls with two small all-gathers between
them and a max over ranks at the end:

    hola_shard_lm_head  -> all-gather of the per-row statistics records (16 bytes per verify row and rank)
    hola_shard_accept   -> all-gather of the two masses of row accept_len per sequence (16 bytes per sequence and rank)
    hola_shard_sample   -> max over ranks of next_tok (the one rank that holds the point u * R wrote a token, the
                           others -1)

Everything numeric runs in the library's kernels; this module marshals arguments and moves the records.
`ShardedHolaVerify.step` does it for one rank over torch.distributed (NCCL on device tensors); `run_ranks_in_turn` runs
all ranks of a group one after the other in ONE process, which is how a single GPU checks the multi-rank path - and
how one GPU runs a head whose vocabulary ranges are stored at different widths (each range is a "rank" with its own
weight mode; the merges are exact, so the result is the verify step on the mixed-width matrix).
"""
from __future__ import annotations

import ctypes

import torch
import torch.distributed as dist

from . import binding


def shard_range(V: int, rank: int, world: int) -> tuple[int, int]:
    """(first row, rows) of `rank`'s contiguous share of V vocabulary rows; shares are multiples of 8 rows (16-byte
    rows of a bf16 draft tensor) except the last one."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("rank outside the group")
    per = -(-V // world)
    per = -(-per // 8) * 8
    lo = min(V, rank * per)
    hi = min(V, lo + per)
    if hi <= lo:
        raise ValueError(f"rank {rank} of {world} gets no vocabulary rows of {V}")
    return lo, hi - lo


class TorchDistExchange:
    """The three collectives of a step over a torch.distributed group (NCCL for device tensors, gloo for host ones)."""

    def __init__(self, group=None):
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        flat = t.contiguous().view(-1)
        out = torch.empty(self.world * flat.numel(), dtype=t.dtype, device=t.device)
        dist.all_gather_into_tensor(out, flat, group=self.group)
        return out.view((self.world,) + tuple(t.shape))

    def all_reduce_max_(self, t: torch.Tensor) -> torch.Tensor:
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=self.group)
        return t


class LocalExchange:
    """The exchange of a group of one: every collective is the identity."""

    world, rank = 1, 0

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        return t.contiguous().unsqueeze(0)

    def all_reduce_max_(self, t: torch.Tensor) -> torch.Tensor:
        return t


class ShardedHolaVerify:
    """One rank of the vocabulary-parallel verify step."""

    def __init__(self, maxB: int, maxK: int, H: int, V_global: int, rank: int, world: int, device: int | None = None):
        self.rank, self.world, self.V_global = rank, world, V_global
        self.v_offset, self.V_local = shard_range(V_global, rank, world)
        self.ctx = binding.HolaVerify(maxB, maxK, H, self.V_local, device)
        self._live = None

    def close(self):
        self.ctx.close()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # ---- the three calls.  W_lm / draft_q / w_scale are this rank's parts; draft_tok holds global token ids.
    def lm_head(self, hidden, W_lm, draft_tok, draft_q, q_tok, uniforms, tau, fallback=binding.HOLA_FALLBACK_SAMPLE,
                w_scale=None, a8=False, out=None, stream=None) -> torch.Tensor:
        """Call 1.  Returns this rank's record (uint8 device tensor) for the first all-gather."""
        B, k = hidden.shape[0], hidden.shape[1] - 1
        if W_lm.shape[0] != self.V_local or (k > 0 and draft_q.shape[-1] != self.V_local):
            raise binding.HolaError("W_lm and draft_q must be this rank's vocabulary range")
        out = out or self.ctx.alloc_outputs(B, k, False)
        a = self.ctx._args(hidden, W_lm, draft_tok, draft_q, uniforms, tau, out, B, k,
                           binding.HOLA_GATE_TARGET_ENTROPY, fallback, w_scale, a8)
        sh = binding.hola_shard_args()
        sh.world, sh.rank, sh.v_offset, sh.V_global = self.world, self.rank, self.v_offset, self.V_global
        qt = q_tok.to(torch.float32).contiguous() if k > 0 else None
        sh.q_tok = binding._dptr(qt)
        record = torch.empty(int(self.ctx.lib.hola_shard_record_bytes(B, k)), dtype=torch.uint8, device=hidden.device)
        sh.record_out = binding._dptr(record)
        mass = torch.zeros((B, 2), dtype=torch.float64, device=hidden.device)
        sh.mass_out = binding._dptr(mass)
        self.ctx.hola_shard_call("hola_shard_lm_head", a, sh, stream)
        # the argument structs point into these tensors: keep them until the step is over
        self._live = dict(a=a, sh=sh, out=out, record=record, mass=mass, qt=qt, stream=stream,
                          keep=(hidden, W_lm, draft_tok, draft_q, uniforms, w_scale), greedy=bool(fallback))
        return record

    def accept(self, records: torch.Tensor) -> torch.Tensor | None:
        """Call 2, given all ranks' records [world, bytes].  Returns this rank's masses [B, 2] for the second
        all-gather, or None when the greedy fallback has already fixed next_tok."""
        L = self._live
        L["records"] = records.contiguous()
        L["sh"].records = binding._dptr(L["records"])
        self.ctx.hola_shard_call("hola_shard_accept", L["a"], L["sh"], L["stream"])
        return None if L["greedy"] else L["mass"]

    def sample(self, masses: torch.Tensor) -> binding.VerifyOutputs:
        """Call 3, given all ranks' masses [world, B, 2].  next_tok holds the global token where this rank's range has
        the point u * R, -1 elsewhere."""
        L = self._live
        L["masses"] = masses.contiguous()
        L["sh"].masses = binding._dptr(L["masses"])
        self.ctx.hola_shard_call("hola_shard_sample", L["a"], L["sh"], L["stream"])
        return L["out"]

    def outputs(self) -> binding.VerifyOutputs:
        return self._live["out"]

    def step(self, hidden, W_lm, draft_tok, draft_q, q_tok, uniforms, tau, exchange: TorchDistExchange, **kw):
        """One whole step of this rank; the collectives run on the current stream's device tensors."""
        record = self.lm_head(hidden, W_lm, draft_tok, draft_q, q_tok, uniforms, tau, **kw)
        mass = self.accept(exchange.all_gather(record))
        if mass is None:
            return self.outputs()
        out = self.sample(exchange.all_gather(mass))
        exchange.all_reduce_max_(out.next_tok)
        return out


def split_inputs(W_lm, draft_q, draft_tok, world: int, w_scale=None):
    """Per-rank parts of a whole problem (test and demo helper): rows of W_lm (and of its scales), the vocabulary axis
    of draft_q, and q_j(x_j) gathered from the whole draft tensor."""
    V = W_lm.shape[0]
    B, k = draft_tok.shape if draft_tok is not None and draft_tok.dim() == 2 else (0, 0)
    q_tok = None
    if k > 0:
        idx = draft_tok.clamp(0, V - 1).to(torch.int64).unsqueeze(-1)
        q_tok = torch.gather(draft_q, 2, idx).squeeze(-1).to(torch.float32)
        bad = (draft_tok < 0) | (draft_tok >= V)
        q_tok = torch.where(bad, torch.zeros_like(q_tok), q_tok)
    parts = []
    for r in range(world):
        lo, n = shard_range(V, r, world)
        parts.append(dict(W_lm=W_lm[lo:lo + n].contiguous(),
                          draft_q=draft_q[:, :, lo:lo + n].contiguous() if k > 0 else None,
                          w_scale=w_scale[lo:lo + n].contiguous() if w_scale is not None else None))
    return parts, q_tok


def run_ranks_in_turn(ranks: list[ShardedHolaVerify], hidden, parts, draft_tok, q_tok, uniforms, tau, **kw):
    """All ranks of a group in one process, one after the other (no kernel waits for another): call 1 on every rank,
    the records side by side, call 2 on every rank, the masses side by side, call 3 on every rank, the max."""
    a8 = kw.pop("a8", False)                                 # (a part may carry its own "a8": ranges of mixed width)
    records = torch.stack([r.lm_head(hidden, p["W_lm"], draft_tok, p["draft_q"], q_tok, uniforms, tau,
                                     w_scale=p["w_scale"], a8=p.get("a8", a8) if p["w_scale"] is not None else False,
                                     **kw) for r, p in zip(ranks, parts)])
    masses = [r.accept(records) for r in ranks]
    if masses[0] is None:
        return ranks[0].outputs(), [r.outputs() for r in ranks]
    masses = torch.stack(masses)
    outs = [r.sample(masses) for r in ranks]
    next_tok = torch.stack([o.next_tok for o in outs]).max(dim=0).values
    first = outs[0]
    merged = binding.VerifyOutputs(first.accept_len, next_tok, first.entropy, first.logZ, None, first.status,
                                   first.draft_entropy)
    return merged, outs


def main():
    """Times ONE rank's three calls on its share of a named workload (the other ranks' records come from a run of all
    ranks in turn on the same device; the collectives themselves need several GPUs and are not timed here)."""
    import argparse
    import json

    from . import workloads

    ap = argparse.ArgumentParser(description=main.__doc__)
    ap.add_argument("--workload", default="large_vocab")
    ap.add_argument("--world", type=int, default=8)
    ap.add_argument("--steps", type=int, default=50)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("vocab_parallel: no CUDA device; the verify path has no CPU fallback")
    w = workloads.make_config(args.workload, device="cuda")
    parts, q_tok = split_inputs(w.W_lm, w.draft_q, w.draft_tok, args.world)
    ranks = [ShardedHolaVerify(w.B, w.k, w.H, w.V, r, args.world) for r in range(args.world)]
    merged, _ = run_ranks_in_turn(ranks, w.hidden, parts, w.draft_tok, q_tok, w.uniforms, w.tau)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        one = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for _ in range(5):
            ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau, out=one)
        ev[0].record()
        for _ in range(args.steps):
            ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau, out=one)
        ev[1].record()
        torch.cuda.synchronize()
        whole_ms = ev[0].elapsed_time(ev[1]) / args.steps
    same_accept = bool(torch.equal(merged.accept_len, one.accept_len))
    token_diffs = int((merged.next_tok != one.next_tok).sum())
    r0, p0 = ranks[0], parts[0]
    records = torch.stack([r._live["record"] for r in ranks])
    masses = torch.stack([r._live["mass"] for r in ranks])
    e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    t = [0.0, 0.0, 0.0]
    for it in range(args.steps + 5):
        e[0].record()
        r0.lm_head(w.hidden, p0["W_lm"], w.draft_tok, p0["draft_q"], q_tok, w.uniforms, w.tau)
        e[1].record()
        r0.accept(records)
        e[2].record()
        r0.sample(masses)
        e[3].record()
        torch.cuda.synchronize()
        if it >= 5:
            for i in range(3):
                t[i] += e[i].elapsed_time(e[i + 1]) / args.steps
    for r in ranks:
        r.close()
    print(json.dumps({
        "workload": f"{w.name}: B={w.B} k={w.k} H={w.H} V={w.V}, vocabulary split over {args.world} ranks",
        "rank0_vocabulary_rows": r0.V_local, "unsharded_ms_per_step": whole_ms,
        "rank0_ms": {"lm_head": t[0], "accept": t[1], "sample": t[2], "sum": sum(t)},
        "exchange_bytes_per_rank": {"records": int(records[0].numel()), "masses": int(masses[0].numel() * 8),
                                    "next_tok": int(w.B * 4)},
        "same_accept_len_as_unsharded": same_accept, "next_tok_differences": token_diffs,
        "note": "collectives not timed (one device); each call of a rank synchronised for timing"}))


if __name__ == "__main__":
    main()
