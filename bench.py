#!/usr/bin/env python
"""Throughput of the PBT hot path on synthetic data: population member-samples per second.

One "step" = one lockstep pass of the whole hot path over one batch per member: batch
window, forward, loss, backward, fused optimiser.  The timed region is K such steps plus
exactly ONE ready point (evaluation, exploit / explore) whatever K is; it is repeated R
times and the headline is the median repeat.  `ms_per_step` and `value` come from that
whole region; `train_ms_per_step` is the K steps alone and `amortised_ms_per_step` adds
the ready point at the workload's own ready interval.  After the headline the other
benchmark populations are timed in compact form (`workloads`).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl ours|reference]

N > 1 (under torch.distributed.run) runs N independent replicas of the population, one per
GPU, with no data-path collective ("replicas only"); the value is the sum over replicas
divided by the slowest replica's time.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "population member-samples/sec"
UNIT = "member-samples/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def max_over_ranks(x: float, device=None) -> float:
    """Slowest rank's time: the population replicas are independent, the job is as slow as its slowest replica."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(cfg, world: int, steps: int, ms: float) -> float:
    """member-samples/s of the whole job: every rank trains its own replica of the population."""
    return world * cfg.n_members * max(cfg.batch, 1) * steps / (ms * 1e-3)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# DRAM bytes per parameter of the fused weight-gradient + Adam kernel, from one `ncu --set full` capture of an
# 8-member case (the traffic is proportional to the members), valid for the source file with this sha1 only.
_NCU_TRAFFIC = {"wgrad_adam": {"bytes_per_param": 25.37, "source": "paper_1711_09846_b200/csrc/wgrad_adam_tcgen05.cu",
                               "sha1": "4f3a44b941b70cfe935a561e5010283c3990f8bd"}}


def _ncu_traffic(name, params_per_launch):
    """Measured DRAM traffic of one launch, scaled from the captured small case; None once the kernel changed."""
    import hashlib
    rec = _NCU_TRAFFIC.get(name)
    if not rec:
        return None
    try:
        sha = hashlib.sha1(open(os.path.join(ROOT, rec["source"]), "rb").read()).hexdigest()
    except OSError:
        return None
    return rec["bytes_per_param"] * params_per_launch if sha == rec["sha1"] else None


def _tc_layer(fan_in, fan_out, rows):
    """Layers whose weight gradient qualifies for the tensor-core kernel (the library's own rule)."""
    return fan_in >= 128 and fan_out >= 128 and rows >= 64 and fan_in % 8 == 0 and fan_out % 8 == 0


def _algorithmic_work(cfg):
    """Algorithmic work of ONE lockstep step of the whole population: GEMM FLOPs, optimiser traffic."""
    B = cfg.batch
    fused_flops = fused_params = 0.0
    if cfg.model == "toy_quadratic":
        return {"flops": 0.0, "fused_flops": 0.0, "fused_params": 0.0, "opt_params": 0.0, "opt_bytes_per_param": 0}
    adam_bf16 = cfg.optimizer == "adam" and cfg.dtype == "bf16_fp32master"
    if cfg.model == "gan_pair":
        g, d = cfg.widths
        wg = sum(g[i] * g[i + 1] for i in range(len(g) - 1))
        wd = sum(d[i] * d[i + 1] for i in range(len(d) - 1))
        K = cfg.gan_d_steps
        # K discriminator updates: G forward (B rows), D forward + wgrad on 2B rows, D dgrad above layer 0
        flops = K * (2 * B * wg + 2 * (2 * B) * wd * 2 + 2 * (2 * B) * (wd - d[0] * d[1]))
        rows_d = 2 * B
        if cfg.loss == "wgan_gp":
            # critic update on real, generated and interpolated rows: forward, data-gradient chain and weight gradient
            # over 3B rows; input gradient of the interpolates; the penalty's second chain up to the last hidden layer
            rows_d = 3 * B
            flops = K * (2 * B * wg + 2 * (3 * B) * wd * 2 + 2 * (3 * B) * (wd - d[0] * d[1]) + 2 * B * d[0] * d[1]
                         + 2 * B * (wd - d[-2] * d[-1]))
        # generator update: G fwd, D fwd, D dgrad to the input, G dgrad + wgrad
        flops += 2 * B * wg + 2 * B * wd + 2 * B * wd + 2 * B * (wg - g[0] * g[1]) + 2 * B * wg
        opt_params = (wg + sum(g[1:])) + K * (wd + sum(d[1:]))
        if adam_bf16:
            for i in range(len(g) - 1):
                if _tc_layer(g[i], g[i + 1], B):
                    fused_params += g[i] * g[i + 1]
                    fused_flops += 2 * B * g[i] * g[i + 1]
            for i in range(len(d) - 1):
                if _tc_layer(d[i], d[i + 1], rows_d):
                    fused_params += K * d[i] * d[i + 1]
                    fused_flops += K * 2 * rows_d * d[i] * d[i + 1]
    else:
        w = cfg.widths[0]
        W = sum(w[i] * w[i + 1] for i in range(len(w) - 1))
        flops = 2 * B * W + 2 * B * (W - w[0] * w[1]) + 2 * B * W
        opt_params = W + sum(w[1:])
        if adam_bf16:
            for i in range(len(w) - 1):
                if _tc_layer(w[i], w[i + 1], B):
                    fused_params += w[i] * w[i + 1]
                    fused_flops += 2 * B * w[i] * w[i + 1]
    bpp = {"adam": 16 + 12, "sgdm": 12 + 8, "rmsprop": 12 + 8, "sgd_plain": 8 + 4}[cfg.optimizer] + \
        (2 if cfg.dtype == "bf16_fp32master" else 0)
    n = cfg.n_members
    return {"flops": n * flops, "fused_flops": n * fused_flops, "fused_params": n * fused_params,
            "opt_params": n * opt_params, "opt_bytes_per_param": bpp}


def _cpu_count_used():
    try:
        from threadpoolctl import threadpool_info
        n = max((i.get("num_threads", 1) for i in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def _oracle_sample(cfg, inp, members, steps):
    """Time the CPU oracle, as it stands, on `members` members for `steps` steps."""
    from oracle import pbt_oracle as O
    sub = cfg.replace(n_members=members)
    sub_inp = type(inp)(**{**inp.__dict__, "init_hparams": inp.init_hparams[:members]})
    pop = O.Population(sub, sub_inp)
    t0 = time.perf_counter()
    pop.step(steps)
    dt = time.perf_counter() - t0
    return members * max(cfg.batch, 1) * steps / dt, dt


def _oracle_budget(cfg):
    """(members, steps) of the bounded oracle sample: roughly 10-30 s of CPU work."""
    per_member = _algorithmic_work(cfg)["flops"] / cfg.n_members
    target = 10.0 * 3e10          # ~10 s at an assumed ~30 GFLOP/s effective float64 rate
    if per_member <= 0:
        return cfg.n_members, 50
    members = max(1, min(cfg.n_members, int(target // max(per_member, 1))))
    steps = max(1, min(50, int(target // max(per_member * members, 1))))
    return members, steps


def run_reference(args, cfg, inp):
    """The oracle as the reference arm: every step is a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import pbt_oracle as O
    members, _ = _oracle_budget(cfg)
    members = max(1, min(members, 4))
    sub = cfg.replace(n_members=members)
    sub_inp = type(inp)(**{**inp.__dict__, "init_hparams": inp.init_hparams[:members]})
    pop = O.Population(sub, sub_inp)
    for _ in range(args.warmup):
        pop.step(1)
    t0 = time.perf_counter()
    for i in range(args.steps):
        pop.step(1)
    dt = time.perf_counter() - t0
    value = members * max(cfg.batch, 1) * args.steps / dt
    cores = _cpu_count_used()
    sample = f"{members} of {cfg.n_members} members x {args.steps} steps, float64 NumPy oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "members": cfg.n_members, "batch": cfg.batch, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def _time_population(pop, cfg, steps, repeats, torch, barrier, two_pass):
    """R timed repeats of [K training steps + ONE ready point (eval, exploit/explore)], CUDA events on the
    library's stream.  Returns per-repeat totals, the split into training and ready-point time, launches of one
    repeat and (from the last repeat when profiled in place, else from an extra profiled pass) per-class times."""
    totals, trains, readys = [], [], []
    launches = 0
    prof = None
    for r in range(repeats):
        profiled = (not two_pass) and r == repeats - 1
        barrier()
        if profiled:
            pop.profile_begin()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        n = 0
        e0.record(pop.stream)
        pop.step(steps)
        n += pop.launch_count()
        e1.record(pop.stream)
        pop.eval()
        n += pop.launch_count()
        pop.exploit_explore()
        n += pop.launch_count()
        e2.record(pop.stream)
        if profiled:
            prof = pop.profile_end()
        barrier()
        totals.append(e0.elapsed_time(e2))
        trains.append(e0.elapsed_time(e1))
        readys.append(e1.elapsed_time(e2))
        launches = n
    if prof is None:
        pop.profile_begin()
        pop.step(steps)
        pop.eval()
        pop.exploit_explore()
        prof = pop.profile_end()
    return {"total_ms": totals, "train_ms": trains, "ready_ms": readys, "launches": launches, "prof": prof}


def _class_rooflines(cfg, prof, steps, peaks):
    """Achieved rate of every kernel class against its roofline: algorithmic work of `steps` steps / summed event
    time of the class (the ready point's few launches are in the class times too; its GEMM and loss work is not in
    the numerator, which makes the fractions slightly conservative)."""
    work = _algorithmic_work(cfg)
    kern = {}

    def add(name, bound, amount, unit, peak, src):
        if prof[name]["launches"] and amount > 0 and prof[name]["ms"] > 0:
            ach = amount * steps / (prof[name]["ms"] * 1e-3) / (1e12 if unit == "TFLOP/s" else 1e9)
            nominal = {"TFLOP/s": 2250.0 if bound == "tensor" else None, "GB/s": 8000.0}[unit]
            kern[name] = {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                          "frac_of_nominal": (ach / nominal) if nominal else None, "nominal_peak": nominal, "traffic": None,
                          "ms_per_step": prof[name]["ms"] / steps,
                          "launches_per_step": prof[name]["launches"] / steps, "peak_source": src}

    fused = prof["wgrad_adam"]["launches"] > 0
    tensor = cfg.dtype == "bf16_fp32master"
    gemm_flops = work["flops"] - (work["fused_flops"] if fused else 0.0)
    add("gemm", "tensor" if tensor else "alu", gemm_flops, "TFLOP/s",
        peaks["bf16_tflops_sustained"] if tensor else 2 * 148 * 128 * 1.965e9 / 1e12,
        peaks["source"] + (" sustained bf16" if tensor else ": n/a, 148 SM x 128 FMA x 2 x 1.965 GHz fp32"))
    if fused:
        # HBM-bound: 12 B read + 14 B written per weight (master, two moments, bf16 shadow); the gradient stays on chip
        add("wgrad_adam", "hbm", work["fused_params"] * 26.0, "GB/s", peaks["hbm_gbs"], peaks["source"])
        if "wgrad_adam" in kern:
            k = kern["wgrad_adam"]
            per_step = prof["wgrad_adam"]["launches"] / steps
            k["tflops"] = work["fused_flops"] * steps / (prof["wgrad_adam"]["ms"] * 1e-3) / 1e12
            k["algorithmic_bytes_per_launch"] = work["fused_params"] * 26.0 / per_step
            k["traffic"] = _ncu_traffic("wgrad_adam", work["fused_params"] / per_step)
    opt_params = work["opt_params"] - (work["fused_params"] if fused else 0)
    add("optimizer", "hbm", opt_params * work["opt_bytes_per_param"], "GB/s", peaks["hbm_gbs"], peaks["source"])
    return kern


def _median_spread(xs):
    return statistics.median(xs), [min(xs), max(xs)]


def _side_workload(pkg, torch, name, steps, repeats, peaks, device):
    """One of the other benchmark populations: K graph-replayed steps + one ready point, R repeats; compact record."""
    from workloads import get_config, make_inputs
    cfg = get_config(name)
    pop = pkg.Population(cfg, make_inputs(cfg), device=device)

    def barrier():
        torch.cuda.synchronize()
    for _ in range(3):
        pop.step(5)
    pop.eval()
    pop.exploit_explore()
    t = _time_population(pop, cfg, steps, repeats, torch, barrier, two_pass=True)
    train, spread = _median_spread([x / steps for x in t["train_ms"]])
    ready = statistics.median(t["ready_ms"])
    amort = train + ready / cfg.ready_interval
    kern = _class_rooflines(cfg, t["prof"], steps, peaks)
    cls_ms = {k: v["ms"] for k, v in t["prof"].items() if v["ms"] > 0}
    tot = sum(cls_ms.values()) or 1.0
    dom = max(cls_ms, key=cls_ms.get) if cls_ms else None
    out = {"workload": cfg.name, "members": cfg.n_members, "batch": cfg.batch, "steps": steps, "repeats": repeats,
           "train_ms_per_step": train, "train_ms_per_step_spread": spread, "ready_point_ms": ready,
           "amortised_ms_per_step": amort, "ready_interval": cfg.ready_interval,
           "member_samples_per_s": cfg.n_members * max(cfg.batch, 1) / (amort * 1e-3),
           "launches_per_step": sum(v["launches"] for v in t["prof"].values()) / steps,
           "dominant_class": dom, "dominant_share_of_kernel_time": (cls_ms[dom] / tot) if dom else None,
           "dominant_frac_of_roofline": kern.get(dom, {}).get("frac") if dom else None,
           "dominant_bound": kern.get(dom, {}).get("bound") if dom else None}
    pop.close()
    del pop
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--repeats", type=int, default=5, help="the timed region (K steps + one ready point) is run this often; the headline is the median")
    ap.add_argument("--workload", default="c5")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the compact figures of the other benchmark populations")
    ap.add_argument("--fuse-adam", type=int, default=-1, help="1/0: apply Adam inside the weight-gradient GEMM (default: the library's choice)")
    ap.add_argument("--graph", type=int, default=-1, help="1: time CUDA-graph replays and profile in a second pass; 0: profile the timed region; -1: by step length")
    ap.add_argument("--backward-streams", type=int, default=0, help="0: the library's choice; 1: one stream; 2: weight and bias gradients beside the data gradient on a second stream")
    ap.add_argument("--members", type=int, default=0, help="override the population size (profiling a small case)")
    ap.add_argument("--pool-rows", type=int, default=0, help="override the training-pool size (default: the workload's)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    args.repeats = max(args.repeats, 1)

    from workloads import get_config, make_inputs
    cfg = get_config(args.workload)
    if args.pool_rows:
        cfg = cfg.replace(pool_rows=args.pool_rows)
    if args.members:
        cfg = cfg.replace(n_members=args.members, name=f"{cfg.name}[members={args.members}]")

    if args.impl == "reference":
        if args.steps == 50:
            args.steps = 3
        if args.warmup >= 3:
            args.warmup = 1
        small = cfg.replace(pool_rows=min(cfg.pool_rows, 4096), eval_batch=min(cfg.eval_batch, 512))
        run_reference(args, small, make_inputs(small))
        return

    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    import paper_1711_09846_b200 as pkg
    inp = make_inputs(cfg)
    kw = {} if args.fuse_adam < 0 else {"fuse_adam": bool(args.fuse_adam)}
    kw["backward_streams"] = args.backward_streams
    pop = pkg.Population(cfg, inp, device=f"cuda:{local}", **kw)
    interval = cfg.ready_interval

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        pop.step(1)
    # one ready point in the warm-up regardless of its length
    pop.eval()
    pop.exploit_explore()

    # Launch-bound workloads (a step of a few hundred microseconds) replay the step as a CUDA graph, which the
    # per-launch event records of the profiler would prevent: for those the timed region runs unprofiled and the
    # per-kernel times come from an extra, profiled pass of the same K steps.  Long steps are profiled in place
    # (in the last repeat only, so the other repeats show what the event records cost).
    t_probe0 = time.perf_counter()
    pop.step(3)
    pop.synchronize()
    probe_ms = (time.perf_counter() - t_probe0) / 3 * 1e3
    two_pass = args.graph == 1 or (args.graph < 0 and probe_ms < 6.0)

    # ---- timed region: device-resident inputs; K steps and exactly one ready point, R times ----
    sampler = ClockSampler(local)
    sampler.start()
    t = _time_population(pop, cfg, args.steps, args.repeats, torch, barrier, two_pass)
    clocks = sampler.stop()
    prof = t["prof"]
    total_ms, total_spread = _median_spread(t["total_ms"])
    total_ms = max_over_ranks(total_ms, f"cuda:{local}")
    train_ms, train_spread = _median_spread([x / args.steps for x in t["train_ms"]])
    ready_ms = statistics.median(t["ready_ms"])
    value = job_value(cfg, world, args.steps, total_ms)

    # ---- end to end: host buffers in, loss out, through the C ABI (MLP populations) ----
    e2e = None
    if cfg.model == "mlp":
        op = torch.bfloat16 if cfg.dtype == "bf16_fp32master" else torch.float32
        ydt = {"mse": torch.float32, "ce_hard": torch.int32, "ce_soft": op}[cfg.loss]
        n_host = 2
        xs, ys = [], []
        for j in range(n_host):
            off = 128 * j
            xs.append(torch.from_numpy(inp.x_pool[off:off + cfg.batch]).to(op).unsqueeze(0)
                      .repeat(cfg.n_members, 1, 1).contiguous().pin_memory())
            yb = torch.from_numpy(inp.y_pool[off:off + cfg.batch]).to(ydt).unsqueeze(0)
            ys.append(yb.repeat(cfg.n_members, *([1] * (yb.dim() - 1))).contiguous().pin_memory())
        loss_out = np.zeros((cfg.n_members, 2), dtype=np.float64)
        e2e_steps = max(3, min(args.steps, 50))
        for j in range(2):
            pop.step_host(xs[j % n_host], ys[j % n_host], loss_out)
        barrier()
        # every step: upload of that step's rows from pinned host memory (on the library's copy stream, overlapping
        # the previous step), the step, and the read-back of the losses; one ready point at the end
        t0 = time.perf_counter()
        pop.prefetch_host_batch(xs[0], ys[0])
        for j in range(e2e_steps):
            pop.step_prefetched(wait=False)
            if j + 1 < e2e_steps:
                pop.prefetch_host_batch(xs[(j + 1) % n_host], ys[(j + 1) % n_host])
            loss_out = pop.last_loss()
        pop.eval()
        pop.exploit_explore()
        pop.synchronize()
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, f"cuda:{local}")
        e2e = {"value": world * cfg.n_members * cfg.batch * e2e_steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": int(xs[0].numel() * xs[0].element_size() + ys[0].numel() * ys[0].element_size()),
               "d2h_bytes_per_step": int(cfg.n_members * 2 * 4), "steps": e2e_steps,
               "timing": "host wall clock; per step: H2D of the batch (pbt_prefetch_host_batch, overlapping the previous step), pbt_step_prefetched, D2H of the losses; one ready point (pbt_eval + pbt_exploit_explore) after the last step"}
    else:
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
               "note": "host-fed steps exist for MLP populations only"}

    # ---- roofline per kernel class, from CUDA events recorded around every launch ----
    peaks = _peaks()
    kern = _class_rooflines(cfg, prof, args.steps, peaks)
    shares = {k: v["ms"] for k, v in prof.items()}
    dominant = max(kern, key=lambda k: kern[k]["ms_per_step"]) if kern else None
    roofline = dict(kern[dominant], kernel=dominant) if dominant else None

    # ---- exploit-copy bandwidth (once, outside the timed region) ----
    copy_gbs = None
    if cfg.model != "toy_quadratic":
        f = np.arange(cfg.n_members, dtype=np.float64)
        pop.set_fitness(f)
        pop.profile_begin()
        pop.exploit_explore()
        pr = pop.profile_end()
        n_cut = max(1, cfg.n_members * cfg.trunc_num // cfg.trunc_den)
        per_member = pop.n_params * (12 if cfg.optimizer == "adam" else 8) + \
            (pop.n_params * 2 if cfg.dtype == "bf16_fp32master" else 0)
        if pr["copy"]["ms"] > 0:
            copy_gbs = 2 * n_cut * per_member / (pr["copy"]["ms"] * 1e-3) / 1e9

    # ---- the two phases of a ready point on their own (CUDA events on the library's stream, median of 5) ----
    def phase_ms(fn):
        ts = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(pop.stream)
            fn()
            b.record(pop.stream)
            pop.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    def ready_point():
        pop.set_fitness(np.arange(cfg.n_members, dtype=np.float64))   # the same n_cut copies every time
        pop.exploit_explore()
    phases = {"eval_ms": phase_ms(pop.eval), "exploit_explore_ms": phase_ms(ready_point),
              "note": "one pbt_eval / one pbt_exploit_explore of the whole population, timed on their own after the "
                      "timed region; the timed region itself contains exactly one ready point (ready_point_ms)"}

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"bf16_fp32master": "bf16", "fp32": "f32", "fp64_toy": "f64"}[cfg.dtype], "data": "synthetic",
        "config": {"workload": cfg.name, "members": cfg.n_members, "batch": cfg.batch, "widths": [list(w) for w in cfg.widths],
                   "optimizer": cfg.optimizer, "ready_interval": interval, "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "timed_region": f"{args.steps} lockstep steps + 1 ready point (pbt_eval, pbt_exploit_explore); "
                                   f"median of {args.repeats} repeats",
                   "timing": ("CUDA-graph replay; per-kernel times from an extra profiled pass" if two_pass else "per-launch events in the last repeat")
                             + "; profiled launches run one at a time, while unprofiled steps run bias gradients beside data gradients on a second stream, so class times can add up to slightly more than the step",
                   "l2": "inputs larger than L2: population state %.1f GB" % (pop.workspace_bytes / 1e9)},
        "repeats": args.repeats, "ms_per_step_spread": [x / args.steps for x in total_spread],
        "train_ms_per_step": train_ms, "train_ms_per_step_spread": train_spread, "ready_point_ms": ready_ms,
        "amortised_ms_per_step": train_ms + ready_ms / interval,
        "amortised_value": world * cfg.n_members * max(cfg.batch, 1) / ((train_ms + ready_ms / interval) * 1e-3),
        "e2e": e2e, "gpu_launches": int(t["launches"]), "clocks": clocks, "roofline": roofline,
        "kernels": kern, "class_ms": shares, "phases": phases,
        "exploit_copy": {"achieved": copy_gbs, "unit": "GB/s", "peak": peaks["hbm_gbs"],
                         "frac": (copy_gbs / peaks["hbm_gbs"]) if copy_gbs else None},
    }
    pop.close()
    del pop
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_workloads:
        side = {}
        for name in ("c1", "c2", "c3", "c4", "c4_wgan", "c5"):
            if get_config(name).name == cfg.name:
                continue
            try:
                side[name] = _side_workload(pkg, torch, name, 200 if name != "c5" else 25, 3, peaks, f"cuda:{local}")
            except Exception as ex:      # a side figure must not take the headline down with it
                side[name] = {"error": repr(ex)}
        result["workloads"] = side

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        members, steps = _oracle_budget(cfg)
        small = cfg.replace(pool_rows=min(cfg.pool_rows, 4096), eval_batch=min(cfg.eval_batch, 512))
        small_inp = make_inputs(small)
        v, dt = _oracle_sample(small, small_inp, members, steps)
        result["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": _cpu_count_used(), "kind": "oracle",
                                  "sample": f"{members} of {cfg.n_members} members x {steps} step(s), {dt:.1f} s, "
                                            f"float64 NumPy oracle, training step only"}
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                m1 = max(1, members // 8)
                v1, dt1 = _oracle_sample(small, small_inp, m1, 1)
            result["cpu_baseline"]["single_thread"] = {"value": v1, "unit": UNIT, "cores": 1,
                                                       "sample": f"{m1} member(s) x 1 step, {dt1:.1f} s"}
        except Exception as ex:
            result["cpu_baseline"]["single_thread"] = {"error": repr(ex)}
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
