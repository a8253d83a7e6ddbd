"""Vocabulary-parallel form of the verify step.

CPU: the split itself, and the exchange protocol run by two gloo ranks whose three "calls" are plain numpy written
here from the definitions (statistics of a vocabulary range, masses of a row inside a range, inverse-CDF search over
ranges in rank order) — the result must be the unsharded oracle's, which pins the claim that the split changes nothing.
GPU: the library's three calls for 2-4 ranks run one after the other on one device, against the same oracle.
"""
import json
import math
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import compare, ref                                  # noqa: E402
from paper_2506_18952_b200 import workloads                      # noqa: E402
from paper_2506_18952_b200 import vocab_parallel as vp           # noqa: E402


def test_shard_range_is_a_partition():
    for V, world in [(5000, 2), (5000, 3), (128256, 8), (37, 4), (1001, 2)]:
        cover = []
        for r in range(world):
            try:
                lo, n = vp.shard_range(V, r, world)
            except ValueError:
                continue                                         # tiny vocabularies leave the last ranks empty
            assert n > 0 and (lo % 8 == 0)
            cover.extend(range(lo, lo + n))
        assert cover == list(range(V))
    with pytest.raises(ValueError):
        vp.shard_range(100, 2, 2)


def test_split_inputs_gathers_the_draft_probabilities():
    w = workloads.gaussian_head("split", 5, 3, 64, 1000, seed=3, w_std=0.3)
    tok = w.draft_tok.clone()
    tok[0, 0] = -4
    tok[1, 2] = 1000
    parts, q_tok = vp.split_inputs(w.W_lm, w.draft_q, tok, 3)
    assert sum(p["W_lm"].shape[0] for p in parts) == 1000
    assert torch.equal(torch.cat([p["draft_q"] for p in parts], dim=2), w.draft_q)
    for b in range(5):
        for j in range(3):
            x = int(tok[b, j])
            want = float(w.draft_q[b, j, x]) if 0 <= x < 1000 else 0.0
            assert float(q_tok[b, j]) == want


RANK_SCRIPT = r'''
import sys, json, math
sys.path.insert(0, {root!r})
import numpy as np, torch
import torch.distributed as dist
from oracle import ref
from paper_2506_18952_b200 import dist as hdist, workloads
from paper_2506_18952_b200 import vocab_parallel as vp

rank, world, _ = hdist.init("gloo")
w = workloads.gaussian_head("vp", 9, 4, 64, 3000, seed=21, w_std=0.3, sigma=1.0, tau={tau})
B, k, V = w.B, w.k, w.V
lo, n = vp.shard_range(V, rank, world)
hid = ref.bf16_bits_to_f64(w.hidden.view(torch.int16).numpy().view(np.uint16))
Wl = ref.bf16_bits_to_f64(w.W_lm.view(torch.int16).numpy().view(np.uint16))[lo:lo + n]
q = w.draft_q.float().numpy().astype(np.float64)
tok = w.draft_tok.numpy()
u = w.uniforms.numpy().astype(np.float64)
logits = hid.reshape(-1, w.H) @ Wl.T                         # this rank's range only, [M, n]
M = B * (k + 1)

class NumpyRank:
    """The three calls, from the definitions, on this rank's vocabulary range."""
    def lm_head(self):
        m = logits.max(axis=1); e = np.exp(logits - m[:, None])
        s = e.sum(axis=1); t = (e * (logits - m[:, None])).sum(axis=1)
        lx = np.full((B, k), -np.inf)
        for b in range(B):
            for j in range(k):
                x = tok[b, j] - lo
                if 0 <= x < n: lx[b, j] = logits[b * (k + 1) + j, x]
        return torch.from_numpy(np.concatenate([m, s, t, lx.reshape(-1)]))
    def accept(self, records):
        r = records.numpy()
        m, s, t = r[:, :M], r[:, M:2 * M], r[:, 2 * M:3 * M]
        lx = r[:, 3 * M:].reshape(world, B, k).max(axis=0)
        mg = m.max(axis=0); sc = np.exp(m - mg)
        S = (sc * s).sum(axis=0); T = (sc * (t + (m - mg) * s)).sum(axis=0)
        self.logZ = (mg + np.log(S)).reshape(B, k + 1); self.H = (np.log(S) - T / S).reshape(B, k + 1)
        self.n = np.full(B, k)
        for b in range(B):
            for j in range(k):
                if self.H[b, j] < {tau}: continue
                px = math.exp(lx[b, j] - self.logZ[b, j]); qx = q[b, j, tok[b, j]]
                if not (u[b, j] * qx < px): self.n[b] = j; break
        mass = np.zeros((B, 2))
        self.res = []
        for b in range(B):
            nb = self.n[b]
            p = np.exp(logits[b * (k + 1) + nb] - self.logZ[b, nb])
            r_ = np.maximum(0.0, p - q[b, nb, lo:lo + n]) if nb < k else p
            self.res.append((r_, p)); mass[b] = (r_.sum(), p.sum())
        return torch.from_numpy(mass)
    def sample(self, masses):
        mm = masses.numpy()
        out = np.full(B, -1, dtype=np.int64)
        for b in range(B):
            idx = 0 if mm[:, b, 0].sum() > 0 else 1
            target = u[b, k] * mm[:, b, idx].sum()
            before = mm[:rank, b, idx].sum()
            if before <= target < before + mm[rank, b, idx]:
                c = before + np.cumsum(self.res[b][idx])
                out[b] = lo + int(np.argmax(c > target))
        return torch.from_numpy(out)

ex = vp.TorchDistExchange()
me = NumpyRank()
mass = me.accept(ex.all_gather(me.lm_head()))
nxt = ex.all_reduce_max_(me.sample(ex.all_gather(mass)))
print(json.dumps(dict(rank=rank, accept=me.n.tolist(), next=nxt.tolist(), H=me.H.tolist(), logZ=me.logZ.tolist())))
hdist.shutdown()
'''


@pytest.mark.parametrize("tau", [0.0, 5.0])
def test_protocol_two_ranks_gloo_matches_the_unsharded_oracle(tmp_path, tau):
    script = tmp_path / "rank.py"
    script.write_text(RANK_SCRIPT.format(root=ROOT, tau=tau))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(29641 + int(tau)), WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs[0][1][-2000:] + outs[1][1][-2000:]
    recs = [json.loads(o[0].strip().splitlines()[-1]) for o in outs]
    w = workloads.gaussian_head("vp", 9, 4, 64, 3000, seed=21, w_std=0.3, sigma=1.0, tau=tau)
    orc = compare.run_oracle(w)
    for r in recs:                                               # every rank ends with the whole answer
        assert r["accept"] == orc.accept_len.tolist()
        assert r["next"] == orc.next_tok.tolist()
        assert np.max(np.abs(np.array(r["H"]) - orc.entropy)) < 1e-9
        assert np.max(np.abs(np.array(r["logZ"]) - orc.logZ)) < 1e-9
    if tau == 0.0:
        assert len(set(recs[0]["accept"])) >= 3                  # the case spreads over several accept lengths


# ------------------------------------------------------------------------------------------------ GPU
gpu = pytest.mark.gpu
DEV = "cuda"


def _np(t):
    t = t.detach().cpu()
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()


def _run_sharded(w, world, fallback=0, quant=False):
    from paper_2506_18952_b200 import binding
    W, scale = (binding.hola_quantize_w8(w.W_lm) if quant else (w.W_lm, None))
    parts, q_tok = vp.split_inputs(W, w.draft_q, w.draft_tok, world, w_scale=scale)
    ranks = [vp.ShardedHolaVerify(w.B, w.k, w.H, w.V, r, world) for r in range(world)]
    try:
        merged, outs = vp.run_ranks_in_turn(ranks, w.hidden, parts, w.draft_tok, q_tok, w.uniforms, w.tau,
                                            fallback=fallback, a8=quant)
        torch.cuda.synchronize()
        merged = type(merged)(merged.accept_len.clone(), merged.next_tok.clone(), merged.entropy.clone(),
                              merged.logZ.clone(), None, merged.status.clone(), None)
        per_rank = [(o.accept_len.clone(), o.next_tok.clone(), o.entropy.clone(), int(o.status.item())) for o in outs]
    finally:
        for r in ranks:
            r.close()
    return merged, per_rank


@gpu
@pytest.mark.parametrize("world", [1, 2, 3, 4])
@pytest.mark.parametrize("tau", [0.0, None, 100.0])
def test_sharded_step_matches_the_oracle(world, tau):
    w = workloads.gaussian_head("vp_gpu", 21, 4, 128, 5000, seed=31 + world, device=DEV, w_std=0.3, sigma=1.0, tau=tau,
                                sigma_far=0.2)
    merged, per_rank = _run_sharded(w, world)
    orc = compare.run_oracle(w)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(merged.accept_len), _np(merged.next_tok),
                          _np(merged.entropy), _np(merged.logZ), None)
    print(world, tau, rep.summary())
    assert rep.ok, rep.summary()
    assert rep.accept_margin_cases <= 1 and rep.token_margin_cases <= 2
    # every rank reaches the same accept lengths and statistics; exactly one rank wrote each token
    for a, t, h, st in per_rank:
        assert torch.equal(a, per_rank[0][0]) and torch.equal(h, per_rank[0][2])
    wrote = torch.stack([t for _, t, _, _ in per_rank]) >= 0
    assert torch.all(wrote.sum(dim=0) == 1)
    toks = merged.next_tok
    assert int(toks.min()) >= 0 and int(toks.max()) < w.V


@gpu
def test_sharded_step_equals_the_unsharded_call():
    from paper_2506_18952_b200 import binding
    w = workloads.gaussian_head("vp_same", 33, 5, 128, 20000, seed=77, device=DEV, w_std=0.3, sigma=1.0, tau=None,
                                sigma_far=0.2)
    with binding.HolaVerify(w.B, w.k, w.H, w.V) as ctx:
        one = ctx.hola_verify(w.hidden, w.W_lm, w.draft_tok, w.draft_q, w.uniforms, w.tau)
        torch.cuda.synchronize()
    merged, _ = _run_sharded(w, 4)
    assert torch.equal(merged.accept_len, one.accept_len)
    assert float((merged.entropy - one.entropy).abs().max()) < 1e-4
    assert float((merged.logZ - one.logZ).abs().max()) < 1e-4
    assert int((merged.next_tok != one.next_tok).sum()) <= 1     # at most a margin case of the fp64 chunk sums


@gpu
@pytest.mark.parametrize("world", [2, 3])
def test_sharded_greedy_verifier(world):
    w = workloads.gaussian_head("vp_greedy", 17, 4, 128, 4000, seed=5, device=DEV, w_std=0.3, sigma=1.0, tau=None)
    merged, per_rank = _run_sharded(w, world, fallback=1)
    orc = compare.run_oracle(w, fallback=1)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(merged.accept_len), _np(merged.next_tok),
                          _np(merged.entropy), _np(merged.logZ), None)
    assert rep.ok, rep.summary()
    for a, t, h, st in per_rank:                                 # greedy: every rank already holds the token
        assert torch.equal(t, per_rank[0][1])


@gpu
def test_sharded_step_when_the_residual_vanishes():
    """q = 1 everywhere: p - q <= 0 on every range, so all ranks switch to drawing from p, flag it, and still agree."""
    w = workloads.gaussian_head("vp_rzero", 6, 3, 64, 3000, seed=9, device=DEV, w_std=0.3, tau=0.0)
    w.draft_q = torch.ones_like(w.draft_q)
    merged, per_rank = _run_sharded(w, 3)
    orc = compare.run_oracle(w)
    from paper_2506_18952_b200 import binding
    assert any(st & binding.FLAG_R_ZERO for *_, st in per_rank)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(merged.accept_len), _np(merged.next_tok),
                          _np(merged.entropy), _np(merged.logZ), None)
    assert rep.ok, rep.summary()


@gpu
def test_sharded_step_with_the_8bit_head():
    from oracle import lobi
    from paper_2506_18952_b200 import binding
    w = workloads.gaussian_head("vp_w8a8", 12, 4, 128, 6000, seed=13, device=DEV, w_std=0.3, sigma=1.0, tau=None)
    merged, _ = _run_sharded(w, 2, quant=True)
    q8, scale = binding.hola_quantize_w8(w.W_lm)
    hid = ref.bf16_bits_to_f64(_np(w.hidden))
    hq, hs = lobi.quantize_rows_int8(hid.reshape(-1, w.H).astype(np.float32))
    hid = lobi.dequantize_rows(hq, hs).reshape(w.B, w.k + 1, w.H)
    W8 = lobi.dequantize_rows(_np(q8), _np(scale))
    orc = ref.verify(hid, W8, _np(w.draft_tok), _np(w.draft_q), _np(w.uniforms), w.tau, keep_logits=True)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(merged.accept_len), _np(merged.next_tok),
                          _np(merged.entropy), _np(merged.logZ), None)
    assert rep.ok, rep.summary()


@gpu
def test_ranges_of_mixed_width_on_one_device():
    """A head whose first vocabulary range stays bf16 and whose second range is 8-bit (weights, and rows as two planes):
    the ranges run as two "ranks" in turn and merge exactly, so the result is the verify step on the mixed matrix."""
    from oracle import lobi
    from paper_2506_18952_b200 import binding
    w = workloads.gaussian_head("vp_mixed", 14, 4, 128, 6000, seed=17, device=DEV, w_std=0.3, sigma=1.0, tau=None)
    parts, q_tok = vp.split_inputs(w.W_lm, w.draft_q, w.draft_tok, 2)
    lo1, n1 = vp.shard_range(w.V, 1, 2)
    q8, scale = binding.hola_quantize_w8(parts[1]["W_lm"])
    parts[1].update(W_lm=q8, w_scale=scale, a8="a16")
    ranks = [vp.ShardedHolaVerify(w.B, w.k, w.H, w.V, r, 2) for r in range(2)]
    try:
        merged, _ = vp.run_ranks_in_turn(ranks, w.hidden, parts, w.draft_tok, q_tok, w.uniforms, w.tau)
        torch.cuda.synchronize()
        got = [t.clone() for t in (merged.accept_len, merged.next_tok, merged.entropy, merged.logZ)]
    finally:
        for r in ranks:
            r.close()
    # oracle: logits of range 0 from the bf16 operands, of range 1 from the two-plane rows and the dequantised weights
    hid = ref.bf16_bits_to_f64(_np(w.hidden))
    B, k1, H = hid.shape
    h16 = lobi.dequantize_two_plane(*lobi.quantize_rows_two_plane(hid.reshape(B * k1, H).astype(np.float32)))
    W0 = ref.bf16_bits_to_f64(_np(w.W_lm))[:lo1]
    W1 = lobi.dequantize_rows(_np(q8), _np(scale))
    logits = np.concatenate([hid.reshape(B * k1, H) @ W0.T, h16 @ W1.T], axis=1).reshape(B, k1, w.V)
    orc = ref.verify_from_logits(logits, _np(w.draft_tok), _np(w.draft_q), _np(w.uniforms), w.tau)
    rep = compare.compare(orc, _np(w.draft_q), _np(w.uniforms), _np(got[0]), _np(got[1]), _np(got[2]), _np(got[3]), None)
    assert rep.ok, rep.summary()


@gpu
def test_shard_calls_validate_their_arguments():
    from paper_2506_18952_b200 import binding
    w = workloads.gaussian_head("vp_args", 3, 2, 64, 1000, seed=1, device=DEV, w_std=0.3)
    parts, q_tok = vp.split_inputs(w.W_lm, w.draft_q, w.draft_tok, 2)
    with vp.ShardedHolaVerify(w.B, w.k, w.H, w.V, 0, 2) as r0:
        with pytest.raises(binding.HolaError):                   # the whole matrix is not rank 0's range
            r0.lm_head(w.hidden, w.W_lm, w.draft_tok, parts[0]["draft_q"], q_tok, w.uniforms, w.tau)
        r0.lm_head(w.hidden, parts[0]["W_lm"], w.draft_tok, parts[0]["draft_q"], q_tok, w.uniforms, w.tau)
        r0._live["sh"].rank = 5                                  # outside the group
        with pytest.raises(binding.HolaError):
            r0.accept(torch.zeros((2, 256), dtype=torch.uint8, device=DEV))
        torch.cuda.synchronize()
