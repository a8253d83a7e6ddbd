"""Seeded input generators and the replica plumbing, on CPU."""
import math
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest
import torch

from oracle import compare
from paper_2506_18952_b200 import dist as hdist
from paper_2506_18952_b200 import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_tiny_config_is_deterministic_and_well_formed():
    a = workloads.make_config("tiny")
    b = workloads.make_config("tiny")
    assert (a.B, a.k, a.H, a.V) == (1, 4, 64, 1000)
    for x, y in [(a.hidden, b.hidden), (a.W_lm, b.W_lm), (a.draft_q, b.draft_q), (a.draft_tok, b.draft_tok),
                 (a.uniforms, b.uniforms)]:
        assert torch.equal(x, y)
    assert a.hidden.dtype == torch.bfloat16 and a.W_lm.dtype == torch.bfloat16 and a.draft_q.dtype == torch.float32
    assert torch.allclose(a.draft_q.sum(-1), torch.ones(1, 4), atol=1e-5)
    assert a.draft_tok.min() >= 0 and a.draft_tok.max() < 1000
    assert a.uniforms.min() >= 0 and a.uniforms.max() < 1
    # tau is the midpoint of the two middle target entropies of the 4 draft positions: two below, two above
    orc = compare.run_oracle(a)
    H = orc.entropy[0, :4]
    assert (H < a.tau).sum() == 2 and (H > a.tau).sum() == 2
    assert 6.0 < H.mean() < math.log(1000)


def test_scaled_down_recipes_hit_their_targets():
    w = workloads.make_config("batched", B=8, H=64, V=512)
    orc = compare.run_oracle(w)
    assert orc.accept_len[:4].mean() > orc.accept_len[4:].mean()          # near-p half vs far half
    w = workloads.make_config("large_vocab", B=6, k=3, H=64, V=2048)
    H = compare.run_oracle(w).entropy.reshape(-1)
    assert H.min() < 1.0 and H.max() > 5.0                                # prescribed entropy spread
    w = workloads.make_config("wide", B=4, k=3, H=128, V=1024)
    orc = compare.run_oracle(w, keep_logits=True)
    H = orc.entropy.reshape(-1)
    assert np.all(H[0::2] < 1.5) and np.all(H[1::2] > math.log(1024) - 0.1)
    top2 = np.sort(orc.logits.reshape(-1, 1024)[0::2], axis=1)[:, -2:]
    assert np.all(np.abs((top2[:, 1] - top2[:, 0]) - 15.0) < 0.5)         # the prescribed logit gap
    sub = w.slice([2, 0])
    assert sub.B == 2 and torch.equal(sub.hidden[0], w.hidden[2])


def test_replica_plumbing_two_ranks_gloo(tmp_path):
    # two CPU processes: different seeds per rank, max over ranks for time, sum over ranks for units
    script = tmp_path / "rank.py"
    script.write_text(textwrap.dedent(f"""
        import sys, json
        sys.path.insert(0, {ROOT!r})
        import torch
        from paper_2506_18952_b200 import dist as hdist, workloads
        rank, world, local = hdist.init("gloo")
        w = workloads.make_config("tiny", seed_offset=hdist.rank_seed_offset(rank))
        hdist.barrier()
        value, ms = hdist.aggregate_throughput(units_this_rank=w.M * 10, ms_this_rank=2.0 + rank)
        print(json.dumps(dict(rank=rank, world=world, value=value, ms=ms, first=float(w.uniforms[0, 0]))))
        hdist.shutdown()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29617", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs)
    import json
    recs = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert {r["rank"] for r in recs} == {0, 1} and all(r["world"] == 2 for r in recs)
    assert all(abs(r["ms"] - 3.0) < 1e-9 for r in recs)                   # the slower rank's time
    assert all(abs(r["value"] - (2 * 5 * 10) / 3e-3) < 1e-6 for r in recs)  # all ranks' units over that time
    assert recs[0]["first"] != recs[1]["first"]                           # replicas verify different batches


def test_single_process_defaults():
    assert hdist.env_world()[1] >= 1
    assert hdist.max_over_ranks(3.5) == 3.5 and hdist.sum_over_ranks(2.0) == 2.0


def _bench(*argv, timeout=300):
    """Runs bench.py as a user would, with no launcher variables in the environment; returns its JSON lines."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], env=env, capture_output=True, text=True,
                       timeout=timeout)
    assert p.returncode == 0, p.stderr[-2000:]
    return [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]


@pytest.mark.parametrize("mode,scaling", [("replicas", "weak"), ("vocab", "strong")])
def test_bench_starts_its_own_ranks(mode, scaling):
    """`python bench.py --gpus 2` without a launcher starts two ranks itself; they meet on the loopback address, make the
    collectives of the chosen parallelism (gloo, no GPU work) and rank 0 alone prints the one line, with n_gpus = 2."""
    lines = _bench("--gpus", "2", "--dry-run", "--steps", "2", "--parallelism", mode)
    assert len(lines) == 1
    assert lines[0]["n_gpus"] == 2 and lines[0]["scaling"] == scaling and lines[0]["parallelism"] == mode


def test_bench_reference_arm_runs_on_rank_zero_only():
    lines = _bench("--gpus", "2", "--impl", "reference", "--workload", "tiny", "--steps", "2", "--warmup", "1")
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and "1 of 1 sequences" in line["config"]["sample"]
