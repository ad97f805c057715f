#!/usr/bin/env python
"""Benchmark: LSTM BPTT sequence-steps/s under a memory budget m, on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--mode msm] [--m 100]
    python bench.py --impl reference ...      # times the fp64 CPU oracle instead

A "step" is one whole training step: every forward, recomputed forward and backward operation
the plan dictates over the workload's t time steps.  One JSON line is printed by rank 0.

* value / ms_per_step: device-resident inputs, CUDA events around each step.
* e2e: the same step through the host-buffer entry point, host<->device copies included.
* roofline: the dominant kernel (a run of forward operations), timed launch by launch with CUDA
  events on the launching stream in three extra steps: flops of the recurrent gate contraction
  per launch over the mean launch duration, against the measured bf16 peak.
* cpu_baseline: the oracle on the host cores, on a truncated sequence.
* budgets: the other budgets of the workload, with the time ratio against full-memory BPTT
  beside the paper's model (C/t + 2) / 3.

With several GPUs every rank runs an independent replica of the workload (the recurrence does
not shard; no collective is on the data path) and the job's value is the sum.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

WORKLOADS = {
    # name: (mode, headline m, other budgets)
    "c1": ("hsm", 8, []),
    "c2": ("hsm", 64, [("hsm", 16), ("hsm", 256), ("ism", 16), ("ism", 64), ("ism", 256)]),
    # "chen": Chen's sqrt(t) schedule (Section 2.2) on the same executor; it needs 127 units at
    # t = 1000 (alpha = 4, beta = 3), so MSM at m = 127 is the like-for-like DP policy
    # "chenrec": Chen's recursive schedule with k = 3 cuts per level (22 units at t = 1000), beside
    # MSM at the same 22 units
    # "msmx": BPTT-MSM planned over the byte sizes of the layout's states (bf16: hidden : internal :
    # without input state = 3 : 10 : 7) at the bytes of m hidden states, beside "msm3" = the same
    # bytes with internal states rounded up to 4 (3 without input state) hidden states
    "c3": ("msm", 100, [("msm", 10), ("msm", 22), ("chenrec", 3), ("msm", 32), ("msm3", 100), ("msmx", 100),
                        ("msm", 127), ("chen", 0), ("msm", 1000)]),
    "c4": ("ism", 50, [("ism", 20), ("ism", 200), ("msm", 80), ("msm", 200), ("msm", 800)]),
    "c5": ("msm", 341, [("msm3", 341), ("msmx", 341), ("msm", 1365), ("msm", 5461)]),
    "p0": ("hsm", 100, [("hsm", 10), ("hsm", 50), ("hsm", 500), ("hsm", 1000)]),
}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--mode", default=None)
    ap.add_argument("--m", type=int, default=None)
    ap.add_argument("--t", type=int, default=None, help="override the sequence length")
    ap.add_argument("--no-budgets", action="store_true", help="skip the other budgets")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--kernel-breakdown", action="store_true",
                    help="also print device time per kernel for one step (CUPTI via torch.profiler) to stderr")
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thr = threading.Thread(target=self._read, daemon=True)
            self.thr.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx = float(r[2])
                for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                                  ("sw_power_cap", 8)):
                    if r[col].lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        busy = [v for v in sm if mx and v > 0.3 * mx] or sm
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


def kernel_breakdown(dp, plans):
    """Device time per kernel over one training step of each plan, measured with CUPTI
    (kernels run back to back as in production, unlike under ncu)."""
    import collections
    import torch
    from torch.profiler import ProfilerActivity, profile
    for label, plan in plans:
        for _ in range(2):
            dp.enqueue(plan)
        torch.cuda.synchronize()
        with profile(activities=[ProfilerActivity.CUDA]) as prof:
            dp.enqueue(plan)
            torch.cuda.synchronize()
        agg = collections.OrderedDict()
        for ev in prof.events():
            if ev.device_type == torch.autograd.DeviceType.CUDA:
                name = ev.name.replace("mebptt::tc::(anonymous namespace)::", "").replace("void ", "")
                name = name.split("(")[0][:48]
                a = agg.setdefault(name, [0, 0.0])
                a[0] += 1
                a[1] += ev.device_time
        tot = sum(a[1] for a in agg.values())
        print(f"\n### {label}: C = {plan.cost}, t = {plan.t}; sum of device times {tot / 1e3:.2f} ms\n", file=sys.stderr)
        print("| kernel | launches | total us | avg us | share |\n|---|---:|---:|---:|---:|", file=sys.stderr)
        for k, (n, v) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
            print(f"| {k} | {n} | {v:.1f} | {v / n:.2f} | {100 * v / tot:.1f}% |", file=sys.stderr)


def profiled_traffic(kernel_source: str, summary: str):
    """DRAM bytes per forward operation from the committed ncu summary of the dominant kernel, or
    None if the kernel's source has changed since the counters were taken (the summary records the
    hash of the source file it was taken from)."""
    import hashlib
    import re
    try:
        text = open(os.path.join(ROOT, summary)).read()
        sha = hashlib.sha256(open(os.path.join(ROOT, kernel_source), "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    m_sha = re.search(r"kernel source sha256\[:16\]:\s*([0-9a-f]{16})", text)
    m_b = re.search(r"DRAM bytes per forward operation:\s*([0-9.eE+]+)", text)
    if not m_sha or not m_b or m_sha.group(1) != sha:
        return None
    return float(m_b.group(1))


def max_over_ranks(v: float, world: int, device) -> float:
    """Slowest rank's time: the job is done when the last replica is."""
    if world == 1:
        return v
    import torch
    import torch.distributed as dist
    tns = torch.tensor([v], dtype=torch.float64, device=device)
    dist.all_reduce(tns, op=dist.ReduceOp.MAX)
    return float(tns.item())


def job_value(world: int, t: int, ms: float) -> float:
    """Whole-job sequence-steps per second: every replica advances t steps in ms milliseconds."""
    return world * t / (ms * 1e-3)


def oracle_sample(cfg, seconds: float):
    """Time the oracle, as it stands, on a truncated copy of the workload."""
    from oracle import lstm_bptt as O
    from paper_1606_03401_b200 import synth
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count()
    t_s, dt, tried = 2, 0.0, []
    while True:
        c = synth.with_overrides(cfg, t=t_s)
        pr = synth.make_problem(c)
        t0 = time.perf_counter()
        O.lstm_bptt(pr["W"], pr["b"], pr["W_out"], pr["b_out"], pr["x"], pr["targets"], pr["h0"], pr["c0"])
        dt = time.perf_counter() - t0
        tried.append((t_s, dt))
        if dt >= seconds / 3 or t_s >= cfg.t:
            break
        t_s = min(cfg.t, max(t_s * 2, int(t_s * seconds / max(dt, 1e-3) * 0.8)))
    return {"value": t_s / dt, "unit": "seq-steps/s", "cores": cores, "kind": "oracle",
            "sample": f"fp64 full-memory BPTT of the same layer sizes on the first {t_s} of {cfg.t} time steps "
                      f"({dt:.1f} s; cost per step is constant in t)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_1606_03401_b200 import synth
    cfg = synth.CONFIGS[args.workload]
    if args.t:
        cfg = synth.with_overrides(cfg, t=args.t)
    per = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals = []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(cfg, per)
        if i >= args.warmup:
            vals.append(r)
    v = statistics.mean(x["value"] for x in vals)
    mode, m, _ = WORKLOADS[args.workload]
    line = {"impl": "reference", "metric": "lstm_bptt_seq_steps_per_s", "value": v, "unit": "seq-steps/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cfg.t / v,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{cfg.name}: L{cfg.layers} I{cfg.input} H{cfg.hidden} B{cfg.batch} t{cfg.t}",
                       "mode": "full-memory BPTT (oracle)", "m": None},
            "cpu_baseline": {"value": v, "unit": "seq-steps/s", "cores": vals[-1]["cores"], "kind": "oracle",
                             "sample": vals[-1]["sample"]},
            "e2e": {"value": v, "unit": "seq-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    args = parse()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_1606_03401_b200 import binding as B
    from paper_1606_03401_b200 import harness, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cfg = synth.CONFIGS[args.workload]
    if args.t:
        cfg = synth.with_overrides(cfg, t=args.t)
    cfg = synth.with_overrides(cfg, seed=cfg.seed + 1000 * rank)   # independent replicas
    mode0, m0, others = WORKLOADS[args.workload]
    mode = args.mode or mode0
    m = args.m or m0

    dp = harness.DeviceProblem(cfg, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > L2 (126 MB)
    stream = torch.cuda.current_stream()

    def timed(plan, steps, warmup, sample_clocks=False):
        # the sampler starts before the warm-up so that short timed regions still get samples;
        # the warm-up runs the same kernels at the same load
        sampler = ClockSampler(local) if sample_clocks else None
        if sampler:
            sampler.start()
            time.sleep(0.3)
        for _ in range(warmup):
            dp.enqueue(plan)
        barrier()
        evs = []
        for _ in range(steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            dp.enqueue(plan)
            e1.record(stream)
            evs.append((e0, e1))
        barrier()
        clocks = sampler.stop() if sampler else None
        ms = [a.elapsed_time(b) for a, b in evs]
        return sum(ms) / len(ms), clocks

    def max_over(v):
        return max_over_ranks(v, world, dev)

    plan = dp.plan(mode, m)
    full = dp.full_memory_plan()
    if args.kernel_breakdown and rank == 0:
        kernel_breakdown(dp, [(f"{mode} m={plan.m}", plan), ("full memory", full)])
    W = max(3, args.warmup)
    ms, clocks = timed(plan, args.steps, W, sample_clocks=True)
    ms = max_over(ms)
    # host time of one enqueue (the call returns before the device has started on the step)
    torch.cuda.synchronize()
    host_ms = []
    for _ in range(5):
        t0 = time.perf_counter()
        dp.enqueue(plan)
        host_ms.append((time.perf_counter() - t0) * 1e3)
        torch.cuda.synchronize()
    host_enqueue_ms = statistics.median(host_ms)
    counters = dp.out["counters"].cpu().numpy()
    assert int(counters[0]) == plan.cost and int(counters[3]) == 0, counters

    # full-memory BPTT: the denominator of the time ratio, and (by difference) the duration of
    # one forward operation
    ms_full, _ = timed(full, max(2, args.steps // 2), 2)
    ms_full = max_over(ms_full)
    K = cfg.input + cfg.hidden
    flops_fwd_op = 0
    for l in range(cfg.layers):
        K_l = (cfg.input if l == 0 else cfg.hidden) + cfg.hidden
        flops_fwd_op += 2 * cfg.batch * K_l * 4 * cfg.hidden
    pk = peaks()
    extra_ops = plan.cost - cfg.t
    peak_tf = pk["bf16_tflops_sustained"] if cfg.dtype == "bf16" else pk["bf16_tflops_sustained"] / 2.0
    runs = None
    if B.mebptt_lstm_launch_count(dp.desc, plan) and cfg.dtype == "bf16":
        # the dominant kernel, timed launch by launch with CUDA events on the launching stream
        # (separate steps: the event pairs cost stream time, so the whole-step figure above has none)
        B.mebptt_lstm_run_times()
        dp.desc.flags |= B.MEBPTT_FLAG_TIME_RUNS
        for _ in range(3):
            flush.fill_(1)
            dp.enqueue(plan)
        torch.cuda.synchronize()
        dp.desc.flags &= ~B.MEBPTT_FLAG_TIME_RUNS
        runs = B.mebptt_lstm_run_times()
        if runs["forward"][1] == 0:
            runs = None     # the shape runs on the CUDA-core path
    if runs:
        f_ms, f_n, f_ops = runs["forward"]
        b_ms, b_n, b_ops = runs["backward"]
        flops_rec = 2 * cfg.batch * cfg.hidden * 4 * cfg.hidden      # the recurrent contraction of one operation
        per_op_traffic = (profiled_traffic("paper_1606_03401_b200/csrc/tc_lstm.cu",
                                           "profiles/ncu_full_fwd_run_kernel_c3_shapes_t64.md")
                          if (cfg.name == "c3" and cfg.input == 1024) else None)
        achieved = f_ops * flops_rec / (f_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": achieved / peak_tf,
                    "traffic": (per_op_traffic * (f_ops / f_n)) if per_op_traffic else None,
                    "kernel": "fwd_run_kernel (a run of forward operations: recurrent gate contraction + cell update)",
                    "launches": f_n // 3, "ops_per_launch": f_ops / f_n, "us_per_launch": f_ms * 1e3 / f_n,
                    "us_per_op": f_ms * 1e3 / f_ops,
                    "share_of_step": (f_ms / 3) / ms,
                    "backward_runs": {"kernel": "bwd_run_group_kernel (bwd_run_cluster_kernel where B <= 32)", "launches": b_n // 3,
                                      "us_per_op": b_ms * 1e3 / max(1, b_ops), "share_of_step": (b_ms / 3) / ms},
                    "traffic_note": ("DRAM bytes per launch = bytes per operation (ncu capture of a 32-operation launch, "
                                     "config 3's layer sizes) x mean operations per launch; null when the kernel's "
                                     "source has changed since the capture"),
                    "how": f"CUDA events around each launch, 3 steps; {flops_rec} flops per operation x operations per launch / mean "
                           f"launch duration; peak = bf16 sustained ({pk['source']})"}
    else:
        if extra_ops > 0 and ms > ms_full:
            fwd_op_ms = (ms - ms_full) / extra_ops
        else:
            fwd_op_ms = None
        achieved = flops_fwd_op / (fwd_op_ms * 1e-3) / 1e12 if fwd_op_ms else None
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": (achieved / peak_tf) if achieved else None, "traffic": None,
                    "kernel": ("forward operation, step by step (per layer: two tensor-core GEMMs and a cell kernel)"
                               if cfg.dtype == "bf16" and not (cfg.batch % 32) else
                               "forward operation on the CUDA-core path (gate contraction + cell update in one launch per layer)"),
                    "how": "(T(m) - T(full memory)) / (C(t,m) - t) = duration of one forward operation; "
                           f"{flops_fwd_op} flops per operation; peak = bf16 sustained ({pk['source']})"
                           + ("" if cfg.dtype == "bf16" else " / 2: float32 storage takes three bf16 MMAs per product, so the "
                              "rate of useful float32-product flops is at most a third of the bf16 peak; half of it "
                              "(the nominal tf32 : bf16 ratio) is the denominator used here")}

    # the whole step against the tensor peak: forward operations executed, backward operations
    # (dh and dW products, dx is not asked for here), readout with its two gradients
    flops_step = plan.cost * flops_fwd_op + cfg.t * flops_fwd_op + cfg.t * (flops_fwd_op - 2 * cfg.batch * cfg.input * 4 * cfg.hidden) \
        + cfg.t * 6 * cfg.batch * cfg.hidden * cfg.readout
    roofline["step_frac"] = flops_step / (ms * 1e-3) / 1e12 / peak_tf
    roofline["step_flops"] = flops_step

    budgets = []
    if not args.no_budgets and rank == 0 or (not args.no_budgets and world > 1):
        for omode, om in others:
            unit_b = B.mebptt_lstm_unit_bytes(dp.desc)
            op = (B.mebptt_plan_chen_sqrt(cfg.t, 4, 3) if omode == "chen" else
                  B.mebptt_plan_chen_recursive(cfg.t, om, 4, 3) if omode == "chenrec" else
                  B.mebptt_plan_bytes_exact(dp.desc, om * unit_b, True) if omode == "msmx" else
                  dp.plan("msm", om, beta=3) if omode == "msm3" else dp.plan(omode, om))
            om = op.m if omode != "msmx" else om
            oms, _ = timed(op, max(2, args.steps // 2), 1)
            oms = max_over(oms)
            budgets.append({"mode": omode, "m": om, "C": op.cost, "ms_per_step": oms,
                            "seq_steps_per_s": world * cfg.t / (oms * 1e-3),
                            "ratio_vs_full": oms / ms_full, "paper_model_ratio": (op.cost / cfg.t + 2) / 3,
                            "arena_bytes": op.arena_units * unit_b // op.sigma})

    # end to end: host buffers in, host buffers out
    e2e = None
    if not args.no_e2e:
        h = dp.host
        pin = {k: torch.from_numpy(v.view(np.int16) if v.dtype == np.uint16 else v).pin_memory() for k, v in h.items()}
        outs = {k: torch.empty(v.numel(), dtype=v.dtype).pin_memory() for k, v in dp.out.items() if v is not None}
        hws = torch.empty(B.mebptt_lstm_host_workspace_bytes(dp.desc, plan), dtype=torch.uint8, device=dev)
        h2d = sum(v.numel() * v.element_size() for v in pin.values())
        d2h = sum(v.numel() * v.element_size() for v in outs.values())

        def e2e_step():
            B.mebptt_lstm_train_step_host(dp.desc, plan, pin["W"], pin["b"], pin["W_out"], pin["b_out"], pin["x"],
                                          pin["targets"], pin["h0"], pin["c0"], hws, stream.cuda_stream,
                                          outs["loss"], outs["dW"], outs["db"], outs["dW_out"], outs["db_out"],
                                          None, outs["counters"])
        e2e_step()
        barrier()
        n_e2e = max(2, args.steps // 2)
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
            torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / n_e2e
        dt = max_over(dt)
        e2e = {"value": world * cfg.t / dt, "unit": "seq-steps/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": dt * 1e3}
        del hws

    # slot save / restore as an explicit copy: one internal state of this workload, and a large
    # block, against the measured HBM copy rate (bytes read + bytes written)
    slot_io = None
    if rank == 0:
        unit_b = B.mebptt_lstm_unit_bytes(dp.desc)
        slot_io = []
        for label, nbytes in (("one internal state (4 units)", 4 * unit_b), ("1 GiB", 1 << 30)):
            a = torch.empty(nbytes, dtype=torch.uint8, device=dev)
            b_ = torch.empty(nbytes, dtype=torch.uint8, device=dev)
            reps = 20 if nbytes < (64 << 20) else 5
            for _ in range(3):
                B.mebptt_slot_copy(b_, a, nbytes, stream.cuda_stream)
            ms_c = []
            for _ in range(reps):
                flush.fill_(1)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                B.mebptt_slot_copy(b_, a, nbytes, stream.cuda_stream)
                e1.record(stream)
                torch.cuda.synchronize()
                ms_c.append(e0.elapsed_time(e1))
            med = statistics.median(ms_c)
            gbs = 2 * nbytes / (med * 1e-3) / 1e9
            slot_io.append({"what": label, "bytes": nbytes, "us": med * 1e3, "GB_s": gbs,
                            "frac_of_hbm_peak": gbs / pk["hbm_gbs"], "peak_GB_s": pk["hbm_gbs"]})
            del a, b_

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = oracle_sample(synth.with_overrides(cfg, seed=cfg.seed), args.cpu_seconds)

    if rank == 0:
        unit = B.mebptt_lstm_unit_bytes(dp.desc)
        line = {
            "metric": "lstm_bptt_seq_steps_per_s", "value": job_value(world, cfg.t, ms), "unit": "seq-steps/s",
            "n_gpus": world, "steps": args.steps, "warmup": W, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "host_enqueue_ms": host_enqueue_ms,
            "config": {"workload": f"{cfg.name}: L{cfg.layers} I{cfg.input} H{cfg.hidden} B{cfg.batch} t{cfg.t} O{cfg.readout}",
                       "mode": mode, "m": plan.m, "alpha": plan.alpha, "C": plan.cost,
                       "train_steps_per_s": world / (ms * 1e-3),
                       "ratio_vs_full": ms / ms_full, "paper_model_ratio": (plan.cost / cfg.t + 2) / 3,
                       "full_memory_ms": ms_full,
                       "arena_bytes": plan.arena_units * unit,
                       "working_bytes_outside_budget": B.mebptt_lstm_working_bytes(dp.desc, plan),
                       "full_memory_arena_bytes": full.arena_units * unit,
                       "l2": "256 MiB buffer written between timed steps; x alone (131 MB at c3) exceeds L2",
                       "replicas": world, "budgets": budgets, "slot_io": slot_io},
            "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * B.mebptt_lstm_launch_count(dp.desc, plan),
            "roofline": roofline, "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
