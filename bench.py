#!/usr/bin/env python
"""Benchmark of the HSD verify step (LM-head projection + entropy + gate / accept / resample).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                    [--parallelism replicas|vocab] [--repeats R]

One step = one pass of the whole hot path (hola_verify) over one synthetic batch that is already resident in HBM.
Prints ONE JSON line.  `value` is verify positions per second over all ranks; `e2e` is the same metric through
hola_verify_host with pinned HOST buffers (copies inside the timed region); `roofline` describes the dominant
kernel (the LM-head GEMM with fused softmax statistics); `cpu_baseline` is the CPU oracle timed on a bounded
sample of the same workload.  With --impl reference the oracle itself is the timed program.
The timed region (exactly K steps between two synchronisations) is repeated R times; the line reports the median
region, with the fastest and slowest beside it.
N > 1: one process per GPU, started by a launcher (torchrun: RANK / WORLD_SIZE in the environment) or, without one,
by this script itself.  --parallelism replicas (default): N independent replicas, one batch each, no data-path
collective ("weak" scaling).  --parallelism vocab: ONE batch, W_lm split by vocabulary rows over the N GPUs, three
small NCCL collectives per step ("strong" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2506_18952_b200 import dist as hdist  # noqa: E402
from paper_2506_18952_b200 import workloads  # noqa: E402

METRIC = "verify_positions_per_s"
UNIT = "positions/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# the nominal figures of the part (HBM3e bandwidth, dense bf16 tensor rate): the second denominator of every fraction
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of lm_head_entropy_kernel<0>, from the ncu captures
# summarised under profiles/: "batched" (--set full capture), "large_vocab" and "wide" (captures of the three DRAM /
# time counters on the full-size launch; their logits are stored with the streaming hint, so most of them reach DRAM
# inside the kernel; "wide" is the one launch that holds all six passes).  Other workloads, and the other weight modes,
# report null.
NCU_TRAFFIC = {"batched": 265923328 + 8595200, "large_vocab": 1055559936 + 172039680,
               "wide": 2809281024 + 1177498112}


def ncu_traffic_bytes(w):
    return NCU_TRAFFIC.get(w.name)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while the benchmark runs."""

    def __init__(self, cuda_index: int, period_s: float = 0.004):
        self.period, self.samples, self._stop = period_s, [], threading.Event()
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:        # CUDA ordinals follow CUDA_VISIBLE_DEVICES, NVML's do not: go through the UUID
                uuid = "GPU-" + str(torch.cuda.get_device_properties(cuda_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None
        self.t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv:
            self.t.start()

    def stop(self):
        self._stop.set()
        if self.nv and self.t.is_alive():
            self.t.join(timeout=2)

    def summary(self, t0: float, t1: float) -> dict:
        if not self.nv:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable"]}
        inside = [s for s in self.samples if t0 <= s[0] <= t1] or self.samples
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        seen = sorted(n for n, bit in names.items() if any(s[2] & bit for s in inside))
        return {"sm_mhz": statistics.median(s[1] for s in inside) if inside else None, "sm_max_mhz": self.max_mhz,
                "reasons": seen, "samples": len(inside)}


def algorithmic_work(w, w_bytes: int = 2) -> dict:
    """Strict algorithmic bytes and FLOPs of one step and of one launch of the dominant kernel."""
    M = w.M
    q_elem = w.draft_q.element_size()
    gemm_bytes = w.V * w.H * w_bytes + (w.V * 4 if w_bytes == 1 else 0) + M * w.H * 2     # W_lm (+ scales) + hidden, once
    sample_bytes = w.B * w.V * q_elem + w.B * w.k * (4 + q_elem)  # one q row + k gathers per sequence
    out_bytes = w.B * 8 + M * 8
    flops = 2.0 * M * w.V * w.H
    return {"gemm_bytes": gemm_bytes, "step_bytes": gemm_bytes + sample_bytes + out_bytes, "flops": flops}


def oracle_sample_size(w, steps: int, warmup: int) -> tuple[int, float]:
    """How many sequences of the workload the CPU oracle verifies per step, for both places that time it (the
    `cpu_baseline` leg and --impl reference), so that one record holds one oracle rate: all of them when
    (steps + warmup) such steps end within about four minutes, else as many as do.  Returns (n, seconds per sequence)."""
    from oracle import compare, ref
    ref.build()
    compare.run_oracle(w.slice([0]), keep_logits=False)            # builds, loads, spins up threads
    probe = min(w.B, 4)
    t0 = time.perf_counter()
    compare.run_oracle(w.slice(range(probe)), keep_logits=False)
    per_seq = (time.perf_counter() - t0) / probe
    per_step_budget = min(12.0, 240.0 / max(1, steps + warmup))
    n = int(max(1, min(w.B, per_step_budget / max(per_seq, 1e-4))))
    if n > 0.8 * w.B:                                               # the whole batch when it nearly fits anyway
        n = w.B
    elif n >= 8:                                                    # (a multiple of 8: the probe's jitter must not move it)
        n -= n % 8
    return n, per_seq


def oracle_positions_per_s(w, n: int):
    """Times the CPU oracle, as it stands, once on the first n sequences of the workload."""
    from oracle import compare, ref
    t0 = time.perf_counter()
    compare.run_oracle(w.slice(range(n)), keep_logits=False)
    dt = time.perf_counter() - t0
    return n * (w.k + 1) / dt, dt, ref.max_threads()


L2_BYTES = 126 * 1024 * 1024       # B200; replaced by the device's own figure when a GPU is present


def wants_flush(w, weight_bytes_per_element: int, mode: str = "auto") -> bool:
    """An L2-sized buffer is rewritten between steps unless the weights streamed per step exceed the L2 (every named
    workload does: the smallest, 8-bit weights at V = 32000, streams 131 MB, and forcing the flush costs it the same
    10-12 us as it costs the 262 MB bf16 case - the flush kernel breaks the launch chain and leaves dirty lines -
    so nothing of W_lm survives in L2 from one step to the next)."""
    if mode != "auto":
        return mode == "on"
    return w.V * w.H * weight_bytes_per_element <= L2_BYTES


def config_block(w, extra=None, weight_bytes_per_element: int = 2, flush: bool | None = None) -> dict:
    mb = w.V * w.H * weight_bytes_per_element / 1e6
    flush = wants_flush(w, weight_bytes_per_element) if flush is None else flush
    cfg = {"workload": f"{w.name}: B={w.B} k={w.k} H={w.H} V={w.V}, bf16 hidden/W_lm, q {str(w.draft_q.dtype).split('.')[-1]}",
           "tau": w.tau,
           "l2": (f"flush: a 256 MB buffer is rewritten between steps (W_lm streams {mb:.0f} MB per step; the time of the "
                  "rewrites alone is measured and taken out)") if flush else
                 f"no flush: every step streams W_lm ({mb:.0f} MB) which is larger than the {L2_BYTES / 1e6:.0f} MB L2"}
    cfg.update(extra or {})
    return cfg


def run_reference(args, rank: int, world: int):
    """--impl reference: the CPU oracle, unchanged, timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = workloads.make_config(args.workload, dev)
    from oracle import compare, ref
    n, _ = oracle_sample_size(w, args.steps, args.warmup)
    sub = w.slice(range(n))
    for _ in range(args.warmup):
        compare.run_oracle(sub, keep_logits=False)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        compare.run_oracle(sub, keep_logits=False)
    dt = time.perf_counter() - t0
    value = n * (w.k + 1) * args.steps / dt
    sample = f"{n} of {w.B} sequences ({n * (w.k + 1)} positions) per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_block(w, {"sample": sample}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": ref.max_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def spawn_ranks(n: int, argv: list[str]) -> int:
    """No launcher in sight and --gpus N > 1: start the N ranks here, one process per GPU (LOCAL_RANK picks the
    device), rendezvous on the loopback address.  Rank 0's JSON line goes to this process's standard output."""
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *argv], env=env))
    rcs = [p.wait() for p in procs]
    return max(abs(rc) for rc in rcs)


def timed_regions(step, steps: int, repeats: int, barrier) -> list[float]:
    """`repeats` timed regions of exactly `steps` steps each; every region sits between a barrier + synchronise on both
    sides and is timed with CUDA events on the launching stream.  Returns the regions' durations in ms."""
    out = []
    for _ in range(repeats):
        torch.cuda.synchronize()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(steps):
            step()
        ev1.record()
        torch.cuda.synchronize()
        barrier()
        out.append(ev0.elapsed_time(ev1))
    return out


def fractions(work, peaks, t_kernel_s, t_step_s, tensor_scale):
    """Roofline block of the dominant kernel: the bound (the slower of bytes / HBM bandwidth and FLOPs / tensor rate, at
    the measured peaks), what the kernel achieved on it, and the same against the part's nominal figures."""
    t_mem = work["gemm_bytes"] / (peaks["hbm_gbs"] * 1e9)
    tensor_peak = peaks["bf16_tflops"] * tensor_scale
    t_flop = work["flops"] / (tensor_peak * 1e12)
    nom_mem = work["gemm_bytes"] / (NOMINAL_PEAKS["hbm_gbs"] * 1e9)
    nom_flop = work["flops"] / (NOMINAL_PEAKS["bf16_tflops"] * tensor_scale * 1e12)
    if t_flop >= t_mem:
        roof = {"bound": "tensor", "achieved": work["flops"] / t_kernel_s / 1e12, "peak": tensor_peak, "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": work["gemm_bytes"] / t_kernel_s / 1e9, "peak": peaks["hbm_gbs"],
                "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["frac_of_nominal"] = max(nom_mem, nom_flop) / t_kernel_s
    roof["nominal_peaks"] = {"hbm_gbs": NOMINAL_PEAKS["hbm_gbs"], "bf16_tflops": NOMINAL_PEAKS["bf16_tflops"] * tensor_scale}
    if roof["bound"] == "tensor" and "bf16_tflops_sustained" in peaks:
        # context: the same against the seconds-long sustained GEMM figure (long loops here sit at the power cap too)
        sustained = peaks["bf16_tflops_sustained"] * tensor_scale
        roof["peak_sustained"] = sustained
        roof["frac_of_sustained"] = roof["achieved"] / sustained
    roof.update({"hbm_gbs_achieved": work["gemm_bytes"] / t_kernel_s / 1e9,
                 "hbm_frac": work["gemm_bytes"] / t_kernel_s / 1e9 / peaks["hbm_gbs"],
                 "tflops_achieved": work["flops"] / t_kernel_s / 1e12,
                 # the target's figure: whole call against max(bytes / HBM bandwidth, FLOPs / tensor peak)
                 "step_frac_of_roofline": max(t_mem, t_flop) / t_step_s,
                 "step_frac_of_nominal": max(nom_mem, nom_flop) / t_step_s})
    return roof


def run_dry(args, rank: int, world: int):
    """--dry-run: everything of a multi-rank run except the GPU work, on the gloo backend: the ranks start, meet, make
    the collectives of the chosen parallelism on tensors of the real sizes, and rank 0 prints the line."""
    hdist.init("gloo")
    shp = workloads.CONFIG_SHAPES[args.workload]
    B, k = shp["B"], shp["k"]
    hdist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        if args.parallelism == "vocab" and world > 1:
            from paper_2506_18952_b200 import vocab_parallel as vp
            ex = vp.TorchDistExchange()
            rec = ex.all_gather(torch.full((B * (k + 1) * 16 + B * k * 4,), rank, dtype=torch.uint8))
            mass = ex.all_gather(torch.full((B, 2), float(rank), dtype=torch.float64))
            tok = ex.all_reduce_max_(torch.full((B,), rank, dtype=torch.int32))
            assert rec.shape[0] == world and mass.shape[0] == world and int(tok.max()) == world - 1
    ms = (time.perf_counter() - t0) * 1e3
    value, ms_max = hdist.aggregate_throughput(B * (k + 1) * args.steps, max(ms, 1e-6))
    if rank == 0:
        print(json.dumps({"metric": METRIC, "dry_run": True, "n_gpus": world, "steps": args.steps,
                          "parallelism": args.parallelism, "value": None, "unit": UNIT,
                          "scaling": "strong" if args.parallelism == "vocab" else "weak",
                          "config": {"workload": args.workload}}), flush=True)
    hdist.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=9, help="timed regions of --steps steps each; the median is reported")
    ap.add_argument("--workload", default="large_vocab", choices=sorted(workloads.CONFIG_SHAPES))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--parallelism", default="replicas", choices=["replicas", "vocab"],
                    help="several GPUs: independent replicas (default), or one batch with W_lm split by vocabulary rows")
    ap.add_argument("--dry-run", action="store_true",
                    help="start the ranks and make the collectives on the gloo backend, without any GPU work")
    ap.add_argument("--gate", default="target", choices=["target", "draft"],
                    help="which entropy feeds the gate: the verifier's softmax (default) or the draft row")
    ap.add_argument("--fallback", default="sample", choices=["sample", "greedy"],
                    help="what the gate-off branch does: speculative-sampling test (default) or greedy verifier")
    ap.add_argument("--weights", default="bf16", choices=["bf16", "int8", "w8a8", "w8a16", "mixed", "w4"],
                    help="bf16 (default); int8: 8-bit W_lm from hola_quantize_w8, expanded exactly on chip; "
                         "w8a8: 8-bit W_lm and hidden rows quantised on the fly, 8-bit tensor-core kind; "
                         "w8a16: the same with the hidden rows as two 8-bit planes (16-bit-class activations); "
                         "mixed: groups of 256 vocabulary rows at 4 / 8 / 16 bits in the proportions 20 / 70 / 10 %% "
                         "(seeded), expanded on chip; w4: every group at 4 bits")
    ap.add_argument("--flush-l2", default="auto", choices=["auto", "on", "off"],
                    help="rewrite a 256 MB buffer between timed steps (auto: when the weights streamed per step do not "
                         "clearly exceed the L2)")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    args.repeats = max(1, args.repeats)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank, world, local = hdist.env_world()
    if world != args.gpus and world > 1:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}")
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.dry_run:
        run_dry(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the verify path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    hdist.init("nccl")
    if args.parallelism == "vocab":
        run_vocab_parallel(args, rank, world, local, dev)
        hdist.shutdown()
        return

    from paper_2506_18952_b200 import binding
    w = workloads.make_config(args.workload, dev, seed_offset=hdist.rank_seed_offset(rank))
    ctx = binding.HolaVerify(w.B, w.k, w.H, w.V, device=local)
    plan = ctx.hola_plan(w.B, w.k, {"bf16": binding.HOLA_W_BF16, "int8": binding.HOLA_W_INT8,
                                    "w8a8": binding.HOLA_W8A8, "w8a16": binding.HOLA_W8A16,
                                    "mixed": binding.HOLA_W_MIXED, "w4": binding.HOLA_W_MIXED}[args.weights])
    out = ctx.alloc_outputs(w.B, w.k, False)
    global L2_BYTES
    L2_BYTES = int(getattr(torch.cuda.get_device_properties(dev), "L2_cache_size", L2_BYTES)) or L2_BYTES
    w_elem = 2 if args.weights == "bf16" else 1
    do_flush = wants_flush(w, w_elem, args.flush_l2)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if do_flush else None

    W_dev, w_scale = w.W_lm, None
    a8 = {"w8a8": True, "w8a16": "a16"}.get(args.weights, False)
    head_bytes = None
    if args.weights in ("mixed", "w4"):
        import numpy as np
        ng = -(-w.V // binding.GROUP_ROWS)
        widths = ([4] * ng if args.weights == "w4" else
                  np.random.default_rng(250618952).choice([4, 8, 16], size=ng, p=[0.2, 0.7, 0.1]).tolist())
        W_dev = binding.hola_quantize_mixed(w.W_lm, widths)
        head_bytes = W_dev.weight_bytes()
        torch.cuda.synchronize()
    elif args.weights != "bf16":
        W_dev, w_scale = binding.hola_quantize_w8(w.W_lm)
        torch.cuda.synchronize()
    gate_source = 1 if args.gate == "draft" else 0
    fallback = 1 if args.fallback == "greedy" else 0

    def step():
        if flush is not None:
            flush.zero_()
        ctx.hola_verify(w.hidden, W_dev, w.draft_tok, w.draft_q, w.uniforms, w.tau, out=out,
                        gate_source=gate_source, fallback=fallback, w_scale=w_scale, a8=a8)

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        step()
    t_wall0 = time.perf_counter()
    regions = timed_regions(step, args.steps, args.repeats, hdist.barrier)
    t_wall1 = time.perf_counter()
    flush_ms = 0.0
    if flush is not None:
        # the flush is not part of the step: time it alone and take it out
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(args.steps):
            flush.zero_()
        f1.record()
        torch.cuda.synchronize()
        flush_ms = f0.elapsed_time(f1)
    # every rank's regions, the slowest rank per region, then the median region
    per_region = [hdist.max_over_ranks(r - flush_ms, dev) for r in regions]
    ms_total = statistics.median(per_region)
    status = int(out.status.item())
    if status & binding.FLAG_TIMEOUT:
        raise SystemExit("bench.py: a device-side wait timed out; outputs invalid")
    accepted = float(out.accept_len.sum().item())
    units_all = hdist.sum_over_ranks(w.M * args.steps, dev)
    value, ms_max = units_all / (ms_total * 1e-3), ms_total
    accepted_all = hdist.sum_over_ranks(accepted, dev)

    # per-kernel durations, live, with events around the GEMM launches inside hola_verify
    ctx.hola_profile_begin(args.steps)
    for _ in range(args.steps):
        step()
    prof = ctx.hola_profile_end()
    clocks = sampler.summary(t_wall0, t_wall1)
    k1_launches = plan["kernels_per_call"] - 1            # one per pass, or one in all when the passes share a launch
    k1_ms = prof["lm_head_ms"] / max(1, prof["calls"]) / k1_launches
    k3_ms = prof["accept_sample_ms"] / max(1, prof["calls"])

    # end to end through hola_verify_host: pinned host inputs, copies and read-back inside the timed region
    host = {n: getattr(w, n).cpu().pin_memory() for n in ("hidden", "draft_tok", "draft_q", "uniforms")}
    hout = ctx.alloc_outputs(w.B, w.k, False, device=torch.device("cpu"))
    for f in ("accept_len", "next_tok", "entropy", "logZ", "status"):
        setattr(hout, f, getattr(hout, f).pin_memory())

    def e2e_step():
        ctx.hola_verify_host(host["hidden"], W_dev, host["draft_tok"], host["draft_q"], host["uniforms"], w.tau,
                             out=hout, gate_source=gate_source, fallback=fallback, w_scale=w_scale, a8=a8)

    for _ in range(3):
        e2e_step()
    e2e_regions = timed_regions(e2e_step, args.e2e_steps, min(args.repeats, 5), hdist.barrier)
    e2e_total = statistics.median([hdist.max_over_ranks(r, dev) for r in e2e_regions])
    e2e_value = hdist.sum_over_ranks(w.M * args.e2e_steps, dev) / (e2e_total * 1e-3)
    sampler.stop()
    # bytes the library copied in the last step (every step has the same inputs): counted inside hola_verify_host,
    # which sends only the rows of the draft tensor that the step reads while the target entropy gates
    h2d, d2h = ctx.hola_host_traffic()
    e2e_ms = e2e_total / args.e2e_steps
    host_bytes = sum(t.numel() * t.element_size() for t in host.values())

    if rank == 0:
        peaks, peak_kind = load_peaks()
        work = algorithmic_work(w, 2 if args.weights == "bf16" else 1)
        if head_bytes is not None:                          # mixed widths: the bytes of the stored head, as they are
            delta = head_bytes - (work["gemm_bytes"] - w.M * w.H * 2)
            work["gemm_bytes"] += delta
            work["step_bytes"] += delta
        # the 8-bit tensor-core kinds have twice the nominal rate of bf16: measured bf16 peak x 2 for --weights w8a8
        # (w8a16 runs two 8-bit rows per verify row: per algorithmic flop its peak is the bf16 one again)
        roof = fractions(work, peaks, k1_ms * 1e-3 * k1_launches, ms_max / args.steps * 1e-3,
                         2.0 if a8 is True else 1.0)
        traffic = ncu_traffic_bytes(w) if args.weights == "bf16" else None
        roof["traffic"] = traffic
        roof["traffic_source"] = ("ncu capture summarised under profiles/ (a constant of this file, not measured by this "
                                  "run)") if traffic is not None else None
        roof.update({"kernel": "lm_head_entropy_kernel", "kernel_ms": k1_ms, "launches_per_step": k1_launches,
                     "peak_source": f"of {peak_kind}", "accept_sample_ms": k3_ms,
                     "kernel_ms_note": "events between the launches of a separate loop: they keep the accept/sample "
                                       "kernel from starting under the GEMM kernel's tail as it does in the timed steps"})
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int8" if a8 else "bf16", "data": "synthetic",
                "weight_bytes": head_bytes if head_bytes is not None else w.V * w.H * w_elem,
                "repeats": {"regions": len(per_region), "ms_per_step_min": min(per_region) / args.steps,
                            "ms_per_step_median": ms_total / args.steps, "ms_per_step_max": max(per_region) / args.steps},
                "config": config_block(w, {"plan": plan, "parallelism": f"replicas x{world}", "gate": args.gate,
                                           "fallback": args.fallback, "weights": args.weights}, w_elem, do_flush),
                "clocks": clocks,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "ms_per_step": e2e_ms, "host_input_bytes": host_bytes},
                "gpu_launches": (plan["kernels_per_call"] + (1 if gate_source and w.k > 0 else 0) + (1 if a8 else 0))
                * args.steps,
                "accepted_tokens_per_s": accepted_all * args.steps / (ms_max * 1e-3),
                "roofline": roof}
        if world == 1 and not args.no_cpu_baseline:
            n, _ = oracle_sample_size(w, args.steps, args.warmup)
            v, dt, cores = oracle_positions_per_s(w, n)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{n} of {w.B} sequences ({n * (w.k + 1)} positions) per step"}
        print(json.dumps(line), flush=True)
    ctx.close()
    hdist.shutdown()


def run_vocab_parallel(args, rank: int, world: int, local: int, dev):
    """--parallelism vocab: ONE batch; rank r holds rows [v_r, v_r + V_r) of W_lm and the same range of the vocabulary
    axis of the draft tensor; a step is the three shard calls with two all-gathers and a max between and after them
    (NCCL on device tensors; with one rank the exchange is the identity).  Total work is fixed as N grows."""
    from paper_2506_18952_b200 import binding, vocab_parallel as vp
    if args.weights != "bf16" or args.gate != "target":
        raise SystemExit("bench.py: --parallelism vocab is timed with bf16 weights and the target-entropy gate")
    w = workloads.make_config(args.workload, dev)              # the same batch on every rank
    parts, q_tok = vp.split_inputs(w.W_lm, w.draft_q, w.draft_tok, world)
    mine = parts[rank]
    del parts
    sh = vp.ShardedHolaVerify(w.B, w.k, w.H, w.V, rank, world, device=local)
    exchange = vp.TorchDistExchange() if world > 1 else vp.LocalExchange()
    fallback = 1 if args.fallback == "greedy" else 0
    out = sh.ctx.alloc_outputs(w.B, w.k, False)

    def step():
        return sh.step(w.hidden, mine["W_lm"], w.draft_tok, mine["draft_q"], q_tok, w.uniforms, w.tau, exchange,
                       fallback=fallback, out=out)

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        step()
    t_wall0 = time.perf_counter()
    regions = timed_regions(step, args.steps, args.repeats, hdist.barrier)
    t_wall1 = time.perf_counter()
    per_region = [hdist.max_over_ranks(r, dev) for r in regions]
    ms_total = statistics.median(per_region)
    res = step()
    torch.cuda.synchronize()
    if int(res.status.item()) & binding.FLAG_TIMEOUT:
        raise SystemExit("bench.py: a device-side wait timed out; outputs invalid")
    accepted = float(res.accept_len.sum().item())
    value = w.M * args.steps / (ms_total * 1e-3)               # one batch, whatever the number of ranks

    # end to end: the per-step inputs start in pinned host memory, the results end there
    host = {n: getattr(w, n).cpu().pin_memory() for n in ("hidden", "draft_tok", "uniforms")}
    host["draft_q"] = mine["draft_q"].cpu().pin_memory() if w.k > 0 else None
    host["q_tok"] = q_tok.cpu().pin_memory() if w.k > 0 else None
    d_in = {n: (torch.empty_like(t, device=dev) if t is not None else None) for n, t in host.items()}
    h_out = {n: torch.empty_like(getattr(out, n), device="cpu").pin_memory() for n in ("accept_len", "next_tok", "entropy", "logZ")}

    def e2e_step():
        for n, t in host.items():
            if t is not None:
                d_in[n].copy_(t, non_blocking=True)
        r = sh.step(d_in["hidden"], mine["W_lm"], d_in["draft_tok"], d_in["draft_q"], d_in["q_tok"], d_in["uniforms"],
                    w.tau, exchange, fallback=fallback, out=out)
        for n, t in h_out.items():
            t.copy_(getattr(r, n), non_blocking=True)
        torch.cuda.current_stream().synchronize()

    for _ in range(3):
        e2e_step()
    e2e_regions = timed_regions(e2e_step, args.e2e_steps, min(args.repeats, 5), hdist.barrier)
    e2e_total = statistics.median([hdist.max_over_ranks(r, dev) for r in e2e_regions])
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)
    h2d = sum(t.numel() * t.element_size() for t in host.values() if t is not None)
    d2h = sum(t.numel() * t.element_size() for t in h_out.values())
    if rank == 0:
        peaks, peak_kind = load_peaks()
        whole = algorithmic_work(w, 2)
        # one rank's share of the dominant kernel: its rows of W_lm, all hidden rows, its share of the FLOPs
        share = {"gemm_bytes": sh.V_local * w.H * 2 + w.M * w.H * 2, "flops": 2.0 * w.M * sh.V_local * w.H,
                 "step_bytes": whole["step_bytes"]}
        t_step = ms_total / args.steps * 1e-3
        roof = fractions(share, peaks, t_step, t_step, 1.0)
        roof.update({"kernel": "lm_head_entropy_kernel (one rank's vocabulary range)", "kernel_ms": None,
                     "traffic": None, "peak_source": f"of {peak_kind}",
                     "note": "achieved = one rank's algorithmic bytes or FLOPs over the WHOLE step's time (three shard "
                             "calls and three collectives): the shard calls record no per-kernel events"})
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "repeats": {"regions": len(per_region), "ms_per_step_min": min(per_region) / args.steps,
                            "ms_per_step_median": ms_total / args.steps, "ms_per_step_max": max(per_region) / args.steps},
                "config": config_block(w, {"parallelism": f"vocab x{world}", "rows_of_W_lm_per_rank": sh.V_local,
                                           "collectives_per_step": 3 if world > 1 else 0, "gate": args.gate,
                                           "fallback": args.fallback, "weights": args.weights}, 2, False),
                "clocks": clocks,
                "e2e": {"value": w.M * args.e2e_steps / (e2e_total * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": e2e_total / args.e2e_steps},
                "gpu_launches": (sh.ctx.hola_plan(w.B, w.k)["kernels_per_call"] + 2) * args.steps,
                "accepted_tokens_per_s": accepted * args.steps / (ms_total * 1e-3),
                "roofline": roof}
        print(json.dumps(line), flush=True)
    sh.close()


if __name__ == "__main__":
    main()
