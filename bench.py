#!/usr/bin/env python
"""Benchmark of the mixed-precision neural-ODE hot path (Alg. 1 forward + Alg. 2 backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

One "step" is one whole pass of the hot path over one synthetic batch: mpode_forward, the caller-side loss head,
mpode_backward.  The metric is forward+adjoint RK step*samples per second (n_steps * batch / time of a pass),
summed over all ranks.  Default workload: c3, the MLP ODE block (d=256, 257->1024->1024->256 softplus, batch
8192, RK4, 64 steps, bf16), the largest tensor-bound configuration that fits one GPU.

N > 1 (launched by torchrun, one rank per GPU): the batch dimension shards, every rank integrates its own
batch of the same size (weak scaling) and the parameter gradient is summed with one NCCL all-reduce per pass.

--impl reference times the CPU oracle (numpy, fp64 with emulated rounding) on a bounded batch slice of the same
workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2510_23498_b200 import dp, inputs  # noqa: E402

METRIC = "fwd+adjoint RK step*samples/s"
UNIT = "step*samples/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for k, nm in enumerate(names):
                if f[4 + k].lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))


def make_workload(name: str, n_steps=None):
    """The full-size configuration; `n_steps` shortens the time grid only (profiling captures), every launch keeps
    its full-size shape."""
    if not n_steps:
        return inputs.FULL_CONFIGS[name]()
    if name == "n2":
        return inputs.FULL_CONFIGS[name](n_steps=n_steps, n_intervals=min(4, n_steps))
    return inputs.FULL_CONFIGS[name](n_steps=n_steps)


def loss_head_device(torch, wl, yT, target):
    """Caller-side loss head on the device (not part of the RK loop): value and dL/dy_T."""
    if wl.name.startswith("c3") or wl.name.startswith("parabolic"):
        r = yT - target
        return (r * r).mean(), r * (2.0 / r.numel())
    if wl.name.startswith("c2") or wl.name.startswith("c1"):
        r = yT - target
        return 0.5 * (r * r).sum() / yT.shape[0], r / yT.shape[0]
    if wl.name.startswith("c5") or wl.name.startswith("n4"):
        d = wl.vel["d"]
        B = yT.shape[0]
        z, ell = yT[:, :d], yT[:, d]
        loss = (0.5 * (z * z).sum(dim=1) + 0.5 * d * float(np.log(2 * np.pi)) + ell).mean()
        g = torch.cat([z / B, torch.full((B, 1), 1.0 / B, device=yT.device)], dim=1)
        return loss, g.contiguous()
    if wl.name.startswith("c4"):
        H, W, C = wl.vel["H"], wl.vel["W"], wl.vel["C"]
        B = yT.shape[0]
        Wh, labels = target
        feat = yT.view(B, H * W, C).mean(dim=1)
        logp = torch.log_softmax(feat @ Wh.T, dim=1)
        loss = -logp[torch.arange(B, device=yT.device), labels].mean()
        dlog = logp.exp()
        dlog[torch.arange(B, device=yT.device), labels] -= 1.0
        dfeat = (dlog / B) @ Wh
        g = (dfeat[:, None, :] / (H * W)).expand(B, H * W, C).reshape(B, H * W * C).contiguous()
        return loss, g
    raise ValueError(wl.name)


def loss_target(torch, wl, dev):
    if wl.name.startswith("c3") or wl.name.startswith("parabolic"):
        return torch.from_numpy(wl.extra["target"].astype(np.float32)).to(dev)
    if wl.name.startswith("c2"):
        return torch.zeros((wl.batch, wl.vel["d"]), device=dev)
    if wl.name.startswith("c1"):
        R = np.array([[0.0, -1.0], [1.0, 0.0]])
        return torch.from_numpy((wl.y0.astype(np.float64) @ R.T).astype(np.float32)).to(dev)
    if wl.name.startswith("c4"):
        return (torch.from_numpy(wl.extra["Wh"].astype(np.float32)).to(dev), torch.from_numpy(wl.extra["labels"]).to(dev))
    return None


def oracle_rate(wl, sample_batch: int, repeats: int = 1):
    """Forward+adjoint step*samples/s of the CPU oracle on the first `sample_batch` samples (all time steps)."""
    import threadpoolctl
    from oracle import BY_NAME, Policy, make_velocity, odeint_backward, odeint_forward
    vel = make_velocity(wl.vel)
    pol = Policy(low=wl.low, scaling=wl.scaling)
    tab = BY_NAME[wl.solver]
    y0 = wl.y0[:sample_batch]
    aux = None if wl.probe is None else wl.probe[:sample_batch].astype(np.float64)
    cores = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        traj, yT = odeint_forward(vel, wl.theta, y0, wl.tgrid, tab, pol, aux)
        dl = np.ones_like(yT) / yT.size
        odeint_backward(vel, wl.theta, traj, wl.tgrid, tab, pol, dl, aux)
        times.append(time.perf_counter() - t0)
    t = float(np.median(times))
    return wl.n_steps * sample_batch / t, cores, t


# dram__bytes_read.sum + dram__bytes_write.sum per launch (profiles/rk_fused_kernel_c3_mlp_block.md)
MEASURED_TRAFFIC = {("c3", "fused_backward"): 748.6e6}

ORACLE_SAMPLE = {"c1": 512, "c2": 1024, "c3": 128, "c4": 2, "c5": 32, "n2": 1}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload(args.workload, args.n_steps)
    sb = min(ORACLE_SAMPLE[args.workload], wl.batch)
    for _ in range(min(args.warmup, 1)):
        oracle_rate(wl, max(1, sb // 8))
    vals = []
    t_tot = 0.0
    for _ in range(args.steps):
        v, cores, t = oracle_rate(wl, sb)
        vals.append(v)
        t_tot += t
    value = float(np.mean(vals))
    sample = "first %d of %d samples, all %d time steps, per step" % (sb, wl.batch, wl.n_steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wl.low, "data": "synthetic",
        "config": {"workload": wl.name, "batch_per_gpu": wl.batch, "d": int(wl.vel["d"]), "n_steps": wl.n_steps, "solver": wl.solver,
                   "scaling_policy": wl.scaling, "parallelism": "dp%d" % max(args.gpus, 1)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def fp32_mode_bytes(binding, wl, B, N, D, p):
    """Size of the same solve with every buffer in float32 (host-side query: nothing is allocated or run)."""
    import ctypes as C
    lib = binding.load_library()
    widths = wl.vel.get("widths")
    if wl.vel["kind"] == "cnf_hyper":
        widths = [int(wl.vel["hidden"]), int(wl.vel["w"])]
    wa = (C.c_int * len(widths))(*widths) if widths else None
    desc = binding.VelocityDesc(binding.KINDS[wl.vel["kind"]], int(wl.vel["d"]), (len(widths) - 1) if widths else 0,
                                C.cast(wa, C.POINTER(C.c_int)) if widths else None, binding.ACTS[wl.vel.get("act", "none")],
                                int(bool(wl.vel.get("append_time", False))), int(bool(wl.vel.get("bias", wl.vel["kind"] != "linear"))),
                                int(wl.vel.get("H", 0)), int(wl.vel.get("W", 0)), int(wl.vel.get("C", 0)),
                                int(wl.vel.get("n_intervals", 0)), int(bool(wl.vel.get("norm", True))))
    pol32 = binding.Policy(binding.DTYPES["f32"], binding.SCALINGS["none"], 10, 0, 0, binding.NO_OVERRIDE)
    h32 = C.c_void_p()
    if lib.mpode_create(C.byref(h32), C.byref(desc), B, N, C.byref(pol32)) != 0:
        return None, None
    fp32_lib = int(lib.mpode_workspace_bytes(h32)) + int(lib.mpode_trajectory_bytes(h32, N))
    lib.mpode_destroy(h32)
    return fp32_lib + 3 * B * D * 4 + 2 * p * 4, fp32_lib


KERNEL_NAMES = {
    "fused_backward": "rk_fused_kernel<T, true> (one launch per time step: input-gradient chains + weight gradients of all stages)",
    "forward_fused": "rk_fused_kernel<T, false> (forward loop in one launch; one recompute launch per step)",
    "forward": "gemm_tc_kernel (forward layers)", "dgrad": "gemm_tc_kernel (input-gradient layers)",
    "wgrad": "gemm_tc_kernel (weight-gradient layers)"}


def measure_config(torch, binding, name, steps, warmup, dev, n_steps=None):
    """Device-timed passes of one configuration on one GPU, its per-class contraction timing, launch counts and memory."""
    wl = make_workload(name, n_steps)
    B, N = wl.batch, wl.n_steps
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats(dev)
    base_alloc = torch.cuda.memory_allocated(dev)
    ctx = binding.Context(wl.vel, B, N, low=wl.low, scaling=wl.scaling, k_max=wl.k_max, device=str(dev))
    theta = torch.from_numpy(wl.theta).to(dev)
    y0 = torch.from_numpy(wl.y0).to(dev)
    probe = None if wl.probe is None else torch.from_numpy(wl.probe).to(dev)
    target = loss_target(torch, wl, dev)

    def one_pass():
        _, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver, probe)
        loss, dl = loss_head_device(torch, wl, yT, target)
        a0, gg, _, status = ctx.backward(dl, want_log=False)
        if status != 0:
            raise RuntimeError("backward pass of %s returned status %d" % (wl.name, status))
        return loss

    for _ in range(max(warmup, 3)):
        one_pass()
    torch.cuda.synchronize()
    peak_measured = torch.cuda.max_memory_allocated(dev) - base_alloc
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        loss = one_pass()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / steps
    st = ctx.stats()
    ctx.set_profiling(True)
    one_pass()
    prof = ctx.collect_profile()
    ctx.set_profiling(False)
    peaks = measured_peaks()
    tot_ms = sum(v["ms"] for v in prof.values())
    per_class = {k: {"tflops": (v["flops"] / (v["ms"] * 1e-3) / 1e12 if v["ms"] > 0 else 0.0), "launches": v["launches"], "ms": v["ms"]}
                 for k, v in prof.items()}
    top = max(prof, key=lambda k: prof[k]["ms"]) if tot_ms > 0 else None
    roof = None
    if top is not None:
        ach = per_class[top]["tflops"]
        key = "forward_fused" if (top == "forward" and st["fused_launches"] > 0) else top
        roof = {"bound": "tensor", "kernel": KERNEL_NAMES[key], "achieved": ach, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": ach / peaks["bf16_tflops_sustained"], "contraction_share_of_pass": tot_ms / ms if ms > 0 else None,
                "per_class_tflops": {k: round(v["tflops"], 1) for k, v in per_class.items() if v["launches"]}}
    model_bytes = ctx.workspace_bytes + (N + 1) * B * ctx.d * (4 if wl.low == "f32" else 2) + 3 * B * ctx.D * 4 + 2 * ctx.p * 4
    f32_bytes, _ = fp32_mode_bytes(binding, wl, B, N, ctx.D, ctx.p)
    out = {"workload": wl.name, "value": N * B / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "dtype": wl.low, "scaling_policy": wl.scaling,
           "batch": B, "n_steps": N, "launches_per_pass": st["kernel_launches"], "host_syncs_per_pass": st["host_syncs"],
           "paths": {k: st[k] for k in ("tc_contractions", "simt_contractions", "fused_launches", "whole_solve_launches")},
           "roofline": roof, "memory": {"mixed_mode_bytes": int(model_bytes), "measured_peak_bytes": int(peak_measured),
                                        "fp32_mode_bytes": f32_bytes, "ratio": (model_bytes / f32_bytes) if f32_bytes else None},
           "loss": float(loss.item())}
    ctx.close()
    del ctx, theta, y0, probe, target
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2510_23498_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = make_workload(args.workload, args.n_steps)
    B, N = wl.batch, wl.n_steps
    torch.cuda.reset_peak_memory_stats(dev)
    base_alloc = torch.cuda.memory_allocated(dev)
    ctx = binding.Context(wl.vel, B, N, low=wl.low, scaling=wl.scaling, k_max=wl.k_max, device=str(dev))
    theta = torch.from_numpy(wl.theta).to(dev)
    y0 = torch.from_numpy(wl.y0).to(dev)
    probe = None if wl.probe is None else torch.from_numpy(wl.probe).to(dev)
    target = loss_target(torch, wl, dev)
    g = torch.empty(ctx.p, dtype=torch.float32, device=dev)

    def one_pass():
        _, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver, probe)
        loss, dl = loss_head_device(torch, wl, yT, target)
        a0, gg, _, status = ctx.backward(dl, want_log=False)
        if status != 0:
            raise RuntimeError("backward pass of %s returned status %d" % (wl.name, status))
        dp.allreduce_sum_(gg, world)                # data-parallel sum of dL/dtheta over the batch shards
        return loss, a0, gg

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        one_pass()
    barrier()
    # what torch's allocator held at most during a pass on top of what was there before: workspace, trajectory, state, adjoint,
    # parameters, gradient, loss-head temporaries
    peak_measured = torch.cuda.max_memory_allocated(dev) - base_alloc
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        loss, a0, gg = one_pass()
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    launches = ctx.stats()["kernel_launches"] * args.steps
    tmax = torch.tensor([ms], device=dev)
    if world > 1:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    ms = float(tmax.item())
    value = world * N * B * args.steps / (ms * 1e-3)

    # ---- per-class contraction timing (CUDA events around every contraction launch), one extra pass
    ctx.set_profiling(True)
    one_pass()
    prof = ctx.collect_profile()
    ctx.set_profiling(False)
    peaks = measured_peaks()
    tot_ms = sum(v["ms"] for v in prof.values())
    n_l = sum(v["launches"] for v in prof.values())
    per_class = {k: {"tflops": (v["flops"] / (v["ms"] * 1e-3) / 1e12 if v["ms"] > 0 else 0.0),
                     "launches": v["launches"], "ms": v["ms"]} for k, v in prof.items()}
    # the dominant kernel is the class with the largest share of the device time
    top = max(prof, key=lambda k: prof[k]["ms"]) if tot_ms > 0 else "forward"
    ach = per_class[top]["tflops"]
    peak = peaks["bf16_tflops_sustained"]
    fused = prof.get("fused_backward", {}).get("launches", 0) > 0
    kernel_names = dict(KERNEL_NAMES)
    if fused:
        kernel_names["forward"] = KERNEL_NAMES["forward_fused"]
    # DRAM bytes per launch of that kernel from the ncu capture summarised in profiles/ (c3 shapes only; null otherwise)
    traffic = MEASURED_TRAFFIC.get((args.workload, top))
    roofline = {
        "bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
        "traffic": traffic, "peak_source": "bf16_tflops_sustained, " + peaks["source"],
        "kernel": kernel_names[top],
        "avg_launch_ms": prof[top]["ms"] / max(prof[top]["launches"], 1),
        "per_class": per_class,
        "all_contractions_tflops": (sum(v["flops"] for v in prof.values()) / (tot_ms * 1e-3) / 1e12 if tot_ms > 0 else 0.0),
        "contraction_share_of_pass": tot_ms / (ms / args.steps) if ms > 0 else None,
        "launches_per_pass": n_l,
    }

    # ---- end to end through the host-buffer entry points: pinned host inputs, host loss head, host outputs
    e2e = None
    if not args.skip_e2e:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        th_h, y0_h = pin(wl.theta), pin(wl.y0)
        pr_h = None if wl.probe is None else pin(wl.probe)
        yT_h = torch.empty((B, ctx.D), dtype=torch.float32).pin_memory()
        dl_h = torch.empty((B, ctx.D), dtype=torch.float32).pin_memory()
        a0_h = torch.empty((B, ctx.D), dtype=torch.float32).pin_memory()
        g_h = torch.empty(ctx.p, dtype=torch.float32).pin_memory()
        tgt_h = None if target is None or isinstance(target, tuple) else target.cpu()

        def host_pass():
            ctx.forward_host(th_h, y0_h, wl.tgrid, yT_h, wl.solver, pr_h)
            if tgt_h is not None and wl.name.startswith("c3"):
                torch.sub(yT_h, tgt_h, out=dl_h)
                lossv = float((dl_h * dl_h).mean())
                dl_h.mul_(2.0 / dl_h.numel())
            else:
                lossv, gnp = wl.loss(yT_h.numpy().astype(np.float64))
                dl_h.copy_(torch.from_numpy(gnp.astype(np.float32)))
            ctx.backward_host(dl_h, a0_h, g_h)
            return lossv

        host_pass()
        barrier()
        e_steps = max(1, min(args.steps, 3))
        t0 = time.perf_counter()
        for _ in range(e_steps):
            host_pass()
        torch.cuda.synchronize()
        te = time.perf_counter() - t0
        tt = torch.tensor([te], device=dev)
        if world > 1:
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        te = float(tt.item())
        h2d = ctx.p * 4 + B * ctx.d * 4 + (0 if wl.probe is None else B * ctx.d) + B * ctx.D * 4
        d2h = B * ctx.D * 4 + B * ctx.D * 4 + ctx.p * 4
        e2e = {"value": world * N * B * e_steps / te, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "steps": e_steps}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        sb = min(ORACLE_SAMPLE[args.workload], B)
        v, cores, t = oracle_rate(wl, sb)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "first %d of %d samples, all %d time steps (%.1f s)" % (sb, B, N, t)}

    peak_bytes = ctx.workspace_bytes + (N + 1) * B * ctx.d * (4 if wl.low == "f32" else 2) + 3 * B * ctx.D * 4 + 2 * ctx.p * 4
    try:
        fp32_bytes, fp32_lib = fp32_mode_bytes(binding, wl, B, N, ctx.D, ctx.p)
    except Exception:
        fp32_bytes = fp32_lib = None
    mixed_lib = ctx.workspace_bytes + (N + 1) * B * ctx.d * (4 if wl.low == "f32" else 2)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.low, "data": "synthetic",
        "config": {"workload": wl.name, "batch_per_gpu": B, "d": ctx.d, "n_steps": N, "solver": wl.solver,
                   "scaling_policy": wl.scaling, "l2": "working set (%.0f MB) larger than the 126 MB L2" % (peak_bytes / 1e6),
                   "parallelism": "dp%d" % world},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "cpu_baseline": cpu,
        "peak_hbm_bytes": int(peak_measured),
        "memory": {"mixed_mode_bytes": int(peak_bytes), "measured_peak_bytes": int(peak_measured), "fp32_mode_bytes": fp32_bytes,
                   "ratio": (peak_bytes / fp32_bytes) if fp32_bytes else None,
                   # mixed mode is meant to need at most 0.55 of float32 mode's memory; the whole c3 solve is above that (known
                   # shortfall: buffers that only the fused backward has), workspace + trajectory alone below
                   "target": 0.55, "meets_target": bool(fp32_bytes and peak_bytes / fp32_bytes <= 0.55),
                   # workspace + trajectory only (the caller's fp32 state, adjoint, parameters and gradient are the same in both modes)
                   "ratio_workspace_and_trajectory": (mixed_lib / fp32_lib) if fp32_lib else None},
        "loss": float(loss.item()),
    }
    if world == 1 and not args.no_configs:
        # the other configurations (parity-test cases, not the headline): a few device-timed passes each, same measurement
        ctx.close()
        del ctx
        torch.cuda.empty_cache()
        others = {}
        for name in sorted(inputs.FULL_CONFIGS):
            if name == args.workload:
                continue
            try:
                others[name] = measure_config(torch, binding, name, steps=3, warmup=3, dev=dev)
            except Exception as ex:      # a failing side configuration must not lose the headline line
                others[name] = {"error": "%s: %s" % (type(ex).__name__, ex)}
        line["configs"] = others
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1,
                    help="number of ranks; this script does not start them: for N > 1 launch it with torch.distributed.run "
                         "(--nproc-per-node N), which sets WORLD_SIZE / RANK / LOCAL_RANK")
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c3", choices=sorted(inputs.FULL_CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true", help="profiling runs: skip the host-buffer leg")
    ap.add_argument("--no-configs", action="store_true", help="skip the short measurements of the other configurations")
    ap.add_argument("--n-steps", type=int, default=0, help="profiling runs: shorten the time grid (launch shapes unchanged)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
