#!/usr/bin/env python
"""Benchmark of the HSD verify step (LM-head projection + entropy + gate / accept / resample).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole hot path (hola_verify) over one synthetic batch that is already resident in HBM.
Prints ONE JSON line.  `value` is verify positions per second over all ranks; `e2e` is the same metric through
hola_verify_host with pinned HOST buffers (copies inside the timed region); `roofline` describes the dominant
kernel (the LM-head GEMM with fused softmax statistics); `cpu_baseline` is the CPU oracle timed on a bounded
sample of the same workload.  With --impl reference the oracle itself is the timed program.
N > 1 (under torchrun): independent replicas, one per GPU, no data-path collective ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of lm_head_entropy_kernel<0>, from the ncu captures
# summarised under profiles/: "batched" (--set full capture) and "large_vocab" (a capture of the three DRAM / time
# counters on the full-size launch; its logits are stored with the streaming hint, so most of the 197 MB reach DRAM
# inside the kernel).  Other workloads, and the other weight modes, report null.
NCU_TRAFFIC = {"batched": 265883392 + 7073536, "large_vocab": 1055344896 + 165309952}


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


def oracle_positions_per_s(w, budget_s: float, nthreads: int = 0):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload's sequences."""
    from oracle import compare, ref
    compare.run_oracle(w.slice([0]), keep_logits=False, nthreads=nthreads)        # builds, loads, spins up threads
    n, dt = 1, 0.0
    while True:
        t0 = time.perf_counter()
        compare.run_oracle(w.slice(range(n)), keep_logits=False, nthreads=nthreads)
        dt = time.perf_counter() - t0
        if dt >= 0.6 * budget_s or n >= w.B:
            break
        n = int(min(w.B, max(n + 1, n * min(8.0, budget_s / max(dt, 1e-3)))))
    return n * (w.k + 1) / dt, n, dt, ref.max_threads()


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
    ref.build()
    # size the per-step sample so that (steps + warmup) steps end within a few minutes
    t0 = time.perf_counter()
    compare.run_oracle(w.slice([0]), keep_logits=False)
    t_one = time.perf_counter() - t0
    per_step_budget = min(4.0, 150.0 / max(1, args.steps + args.warmup))
    n = int(max(1, min(w.B, per_step_budget // max(t_one, 1e-3))))
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="large_vocab", choices=sorted(workloads.CONFIG_SHAPES))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--gate", default="target", choices=["target", "draft"],
                    help="which entropy feeds the gate: the verifier's softmax (default) or the draft row")
    ap.add_argument("--fallback", default="sample", choices=["sample", "greedy"],
                    help="what the gate-off branch does: speculative-sampling test (default) or greedy verifier")
    ap.add_argument("--weights", default="bf16", choices=["bf16", "int8", "w8a8", "w8a16"],
                    help="bf16 (default); int8: 8-bit W_lm from hola_quantize_w8, expanded exactly on chip; "
                         "w8a8: 8-bit W_lm and hidden rows quantised on the fly, 8-bit tensor-core kind; "
                         "w8a16: the same with the hidden rows as two 8-bit planes (16-bit-class activations)")
    ap.add_argument("--flush-l2", default="auto", choices=["auto", "on", "off"],
                    help="rewrite a 256 MB buffer between timed steps (auto: when the weights streamed per step do not "
                         "clearly exceed the L2)")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-budget-s", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank, world, local = hdist.env_world()
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the verify path has no CPU fallback")
    if world != args.gpus and world > 1:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    hdist.init("nccl")

    from paper_2506_18952_b200 import binding
    w = workloads.make_config(args.workload, dev, seed_offset=hdist.rank_seed_offset(rank))
    ctx = binding.HolaVerify(w.B, w.k, w.H, w.V, device=local)
    plan = ctx.hola_plan(w.B, w.k, {"bf16": binding.HOLA_W_BF16, "int8": binding.HOLA_W_INT8,
                                    "w8a8": binding.HOLA_W8A8, "w8a16": binding.HOLA_W8A16}[args.weights])
    out = ctx.alloc_outputs(w.B, w.k, False)
    global L2_BYTES
    L2_BYTES = int(getattr(torch.cuda.get_device_properties(dev), "L2_cache_size", L2_BYTES)) or L2_BYTES
    w_elem = 2 if args.weights == "bf16" else 1
    do_flush = wants_flush(w, w_elem, args.flush_l2)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if do_flush else None

    W_dev, w_scale = w.W_lm, None
    a8 = {"w8a8": True, "w8a16": "a16"}.get(args.weights, False)
    if args.weights != "bf16":
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
    torch.cuda.synchronize()
    hdist.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.perf_counter()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    t_wall1 = time.perf_counter()
    hdist.barrier()
    ms_total = ev0.elapsed_time(ev1)
    if flush is not None:
        # the flush is not part of the step: time it alone and take it out
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(args.steps):
            flush.zero_()
        f1.record()
        torch.cuda.synchronize()
        ms_total -= f0.elapsed_time(f1)
    status = int(out.status.item())
    if status & binding.FLAG_TIMEOUT:
        raise SystemExit("bench.py: a device-side wait timed out; outputs invalid")
    accepted = float(out.accept_len.sum().item())
    value, ms_max = hdist.aggregate_throughput(w.M * args.steps, ms_total, dev)
    accepted_all = hdist.sum_over_ranks(accepted, dev)

    # per-kernel durations, live, with events around the GEMM launches inside hola_verify
    ctx.hola_profile_begin(args.steps)
    for _ in range(args.steps):
        step()
    prof = ctx.hola_profile_end()
    clocks = sampler.summary(t_wall0, t_wall1)
    k1_ms = prof["lm_head_ms"] / max(1, prof["calls"]) / plan["passes"]
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
    torch.cuda.synchronize()
    hdist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    e2e_value, _ = hdist.aggregate_throughput(w.M * args.e2e_steps, e0.elapsed_time(e1), dev)
    sampler.stop()
    # bytes the library copied in the last step (every step has the same inputs): counted inside hola_verify_host,
    # which sends only the rows of the draft tensor that the step reads while the target entropy gates
    h2d, d2h = ctx.hola_host_traffic()
    e2e_ms = e0.elapsed_time(e1) / args.e2e_steps
    host_bytes = sum(t.numel() * t.element_size() for t in host.values())

    if rank == 0:
        peaks, peak_kind = load_peaks()
        work = algorithmic_work(w, 2 if args.weights == "bf16" else 1)
        t_mem = work["gemm_bytes"] / (peaks["hbm_gbs"] * 1e9)
        # the 8-bit tensor-core kinds have twice the nominal rate of bf16: measured bf16 peak x 2 for --weights w8a8
        # (w8a16 runs two 8-bit rows per verify row: per algorithmic flop its peak is the bf16 one again)
        tensor_peak = peaks["bf16_tflops"] * (2.0 if a8 is True else 1.0)
        t_flop = work["flops"] / (tensor_peak * 1e12)
        t_k1 = k1_ms * 1e-3 * plan["passes"]
        if t_flop >= t_mem:
            roof = {"bound": "tensor", "achieved": work["flops"] / t_k1 / 1e12, "peak": tensor_peak,
                    "unit": "TFLOP/s"}
        else:
            roof = {"bound": "hbm", "achieved": work["gemm_bytes"] / t_k1 / 1e9, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s"}
        roof["frac"] = roof["achieved"] / roof["peak"]
        if roof["bound"] == "tensor" and "bf16_tflops_sustained" in peaks:
            # context: the same against the seconds-long sustained GEMM figure (the loop here runs at the power cap too)
            sustained = peaks["bf16_tflops_sustained"] * (2.0 if a8 is True else 1.0)
            roof["peak_sustained"] = sustained
            roof["frac_of_sustained"] = roof["achieved"] / sustained
        roof["traffic"] = ncu_traffic_bytes(w) if args.weights == "bf16" else None
        roof.update({"kernel": "lm_head_entropy_kernel", "kernel_ms": k1_ms, "launches_per_step": plan["passes"],
                     "peak_source": f"of {peak_kind}", "hbm_gbs_achieved": work["gemm_bytes"] / t_k1 / 1e9,
                     "hbm_frac": work["gemm_bytes"] / t_k1 / 1e9 / peaks["hbm_gbs"],
                     "tflops_achieved": work["flops"] / t_k1 / 1e12,
                     "step_frac_of_roofline": max(t_mem, t_flop) / (ms_max / args.steps * 1e-3),
                     "accept_sample_ms": k3_ms})
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int8" if a8 else "bf16", "data": "synthetic",
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
            v, n, dt, cores = oracle_positions_per_s(w, args.cpu_budget_s)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{n} of {w.B} sequences ({n * (w.k + 1)} positions) in {dt:.1f} s"}
        print(json.dumps(line), flush=True)
    ctx.close()
    hdist.shutdown()


if __name__ == "__main__":
    main()
