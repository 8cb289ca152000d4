#!/usr/bin/env python
"""Benchmark of the SpecKV speculation-step hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload b256]

A step = one pass of the whole hot path (draft signals, controller, verification: a memset of the
tickets, then the sweep kernel, whose grid also draws the fresh tokens for bf16 logits; for fp32
logits the ring sweep and the resample kernel) over one synthetic batch whose logits are resident
in HBM.
Prints ONE JSON line: verified speculation rows/s (whole job), the roofline of the dominant
kernel against the measured HBM peak, the end-to-end figure with host buffers, and the CPU
oracle timed on the host cores as a reported baseline.  With --impl reference the oracle
itself is the timed arm (rank 0 only).
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
for _p in (ROOT, os.path.join(ROOT, "tests")):
    if _p not in sys.path:
        sys.path.insert(0, _p)

METRIC = "verified_speculation_rows_per_sec"
UNIT = "rows/s"
FALLBACK_HBM_GBS = 6650.0  # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent


def _env_int(k, d):
    try:
        return int(os.environ.get(k, d))
    except ValueError:
        return d


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def ncu_traffic_bytes(kernel: str, workload: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, if there is one."""
    p = os.path.join(ROOT, "profiles", f"{kernel}_{workload}.txt")
    try:
        with open(p) as f:
            for line in f:
                if line.startswith("dram_bytes_per_launch:"):
                    return float(line.split(":")[1].split()[0])
    except Exception:
        pass
    return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, torch_index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons = period_s, [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:  # NVML numbers physical devices; find ours by UUID
                uuid = "GPU-" + str(torch.cuda.get_device_properties(torch_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def run_reference(args, w):
    """The oracle as the timed arm: each step is a bounded sample of rows of the workload."""
    import numpy as np
    import torch
    import oracle
    from paper_2605_02888_b200 import synth
    from parity import oracle_batch

    rank = _env_int("RANK", 0)
    if rank != 0:
        return
    cores = host_cores()
    # rows per step: sized from a short calibration so that warm-up + timed steps take about two minutes at most
    cal_rows = min(w.B, max(cores, 16))
    wc = synth.scaled(w, B=cal_rows)
    sc = synth.make_step(wc, 0, "cpu")
    mc = synth.make_mlp(wc, "cpu")
    t0 = time.perf_counter()
    oracle.step(oracle_batch(sc, n_threads=cores), sc["comp"].numpy(),
                oracle.Mlp(*(mc[k].numpy() for k in ("W1", "b1", "W2", "b2"))))
    rate = cal_rows / max(time.perf_counter() - t0, 1e-6)
    budget_s = 120.0
    rows = int(max(8, min(w.B, rate * budget_s / max(1, args.steps + args.warmup))))
    ws = synth.scaled(w, B=rows)
    s = synth.make_step(ws, 0, "cpu")
    mw = synth.make_mlp(ws, "cpu")
    om = oracle.Mlp(*(mw[k].numpy() for k in ("W1", "b1", "W2", "b2")))
    ob = oracle_batch(s, n_threads=cores)
    comp = s["comp"].numpy()
    for _ in range(args.warmup):
        oracle.step(ob, comp, om)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.step(ob, comp, om)
    dt = (time.perf_counter() - t0) / args.steps
    val = rows / dt
    sample = f"{rows} rows of workload {w.name} per step (gamma per row as in the workload), all host cores"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "gamma_max": w.gamma_max, "V": w.V, "logits": w.dtype,
                   "rows_per_step_sampled": rows},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="b256")
    ap.add_argument("--rows", type=int, default=None, help="override the workload's batch rows (profiling captures)")
    ap.add_argument("--lib", default=None, help="path of a libspeckv.so build to load instead of the in-tree one")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()

    from paper_2605_02888_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.rows:
        w = synth.scaled(w, B=args.rows)

    if args.impl == "reference":
        args.steps = args.steps or 3
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, w)
        return

    args.steps = args.steps or 2000
    args.warmup = 20 if args.warmup is None else max(3, args.warmup)

    import torch
    import paper_2605_02888_b200 as speckv
    if args.lib:
        from paper_2605_02888_b200 import binding
        binding._lib = binding.load_library(args.lib)

    def gpu_batch(s):
        return speckv.Batch(draft_logits=s["draft"], target_logits=s["target"], draft_tokens=s["draft_tokens"],
                            gamma=s["gamma"], temperature=s["temperature"], uniforms=s["uniforms"])

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    world = _env_int("WORLD_SIZE", 1)
    rank = _env_int("RANK", 0)
    local = _env_int("LOCAL_RANK", 0)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # every rank runs the full workload on its own seed (weak scaling; rows never interact)
    wr = synth.scaled(w, seed=w.seed + rank)
    attrs = synth.row_attrs(wr)
    n_batches = 2                                  # alternate so that no step re-reads a batch still in L2
    steps_in = [synth.make_step(wr, i, dev, attrs=attrs) for i in range(n_batches)]
    mw_dev = synth.make_mlp(wr, dev)
    gm = speckv.Mlp(mw_dev["W1"], mw_dev["b1"], mw_dev["W2"], mw_dev["b2"])
    batches = [gpu_batch(s) for s in steps_in]
    outs = [speckv.StepOutputs.allocate(b, gm.n_out) for b in batches]
    bytes_step = [synth.logit_bytes(wr, s["gamma"]) for s in steps_in]
    torch.cuda.synchronize()

    def one(i, events=None):
        k = i % n_batches
        speckv.speckv_step(batches[k], steps_in[k]["comp"], gm, out=outs[k], events=events)

    for i in range(args.warmup):
        one(i)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(args.steps):
        one(i)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    if dist:
        t = torch.tensor([ms_total], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
        dist.barrier()
    ms_step = ms_total / args.steps
    value = w.B * world / (ms_step * 1e-3)

    # dominant kernel alone: events recorded by the library around the sweep kernel
    n_prof = min(args.steps, 200)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_prof)]
    for i in range(n_prof):
        one(i, events=evs[i])
    torch.cuda.synchronize()
    sweep_ms = [e[0].elapsed_time(e[1]) for e in evs]
    resample_ms = [e[1].elapsed_time(e[2]) for e in evs]
    sweep_avg = sum(sweep_ms) / n_prof
    bytes_avg = sum(bytes_step[i % n_batches] for i in range(n_prof)) / n_prof
    peak, peak_kind = measured_hbm_peak()
    achieved = bytes_avg / (sweep_avg * 1e-3) / 1e9
    # the library picks by logit type and batch: fp32, 384..1024 rows -> ring sweep, then a resample kernel (two launches per step);
    # bf16 -> register-staged sweep whose grid also carries the resample CTAs (one launch per step, so
    # its duration is that of the whole pass over the batch, second read of the stop positions included)
    kernel = "pipe_sweep_kernel" if (w.dtype == "fp32" and 384 <= wr.B <= 1024) else "sweep_kernel"
    one_launch = kernel == "sweep_kernel"
    roofline = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": ncu_traffic_bytes(kernel, w.name) if not args.rows else None,
                "algorithmic_bytes_per_launch": bytes_avg, "kernel_ms": sweep_avg,
                "kernel_ms_min": min(sweep_ms),
                "kernel_covers": "sweep + row epilogues + fresh-token draw" if one_launch else "sweep + row epilogues",
                "resample_kernel_ms": None if one_launch else sum(resample_ms) / n_prof,
                "timed_over": f"{n_prof} steps after the timed region, CUDA events recorded inside the library call",
                "frac_of_8TBps": achieved / 8000.0,
                "step_GBps": sum(bytes_step[i % n_batches] for i in range(args.steps)) / args.steps / (ms_step * 1e-3) / 1e9}

    # end to end: pinned host buffers in, results out, every step
    e2e = None
    if not args.no_e2e:
        k = 0
        s = steps_in[k]
        names = ("draft", "target", "draft_tokens", "uniforms", "gamma", "temperature", "comp")
        host = {n: s[n].cpu().pin_memory() for n in names}
        devbuf = {n: torch.empty_like(s[n]) for n in names}
        o = outs[k]
        res_names = ("feat", "scores", "gamma_next", "n_accepted", "out_tokens", "row_status")
        host_out = {n: torch.empty_like(getattr(o, n), device="cpu").pin_memory() for n in res_names}
        h2d = sum(host[n].numel() * host[n].element_size() for n in names)
        d2h = sum(host_out[n].numel() * host_out[n].element_size() for n in res_names)
        bt = speckv.Batch(draft_logits=devbuf["draft"], target_logits=devbuf["target"],
                          draft_tokens=devbuf["draft_tokens"], gamma=devbuf["gamma"],
                          temperature=devbuf["temperature"], uniforms=devbuf["uniforms"])

        def e2e_step():
            for n in names:
                devbuf[n].copy_(host[n], non_blocking=True)
            speckv.speckv_step(bt, devbuf["comp"], gm, out=o)
            for n in res_names:
                host_out[n].copy_(getattr(o, n), non_blocking=True)

        n_e2e = 5
        e2e_step()
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n_e2e):
            e2e_step()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / n_e2e
        if dist:
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        e2e = {"value": w.B * world / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": n_e2e}
        del host, devbuf

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        from parity import oracle_batch
        cores = host_cores()
        # bounded sample: whole batches of the resident steps, repeated until about 12 s of CPU work
        # are done (rows per batch capped so that one call stays near a second)
        rows = list(range(min(w.B, 256)))
        obs = [oracle_batch(s_, rows=rows, n_threads=cores) for s_ in steps_in]
        mw = synth.make_mlp(wr, "cpu")
        om = oracle.Mlp(*(mw[k2].numpy() for k2 in ("W1", "b1", "W2", "b2")))
        comps = [s_["comp"].cpu().numpy()[rows] for s_ in steps_in]
        calls, t0 = 0, time.perf_counter()
        while calls < 3 or (time.perf_counter() - t0 < 12.0 and calls < 200):
            oracle.step(obs[calls % n_batches], comps[calls % n_batches], om)
            calls += 1
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": calls * len(rows) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"{calls} calls of {len(rows)} rows (steps 0/1 of workload {w.name} in turn), {dt:.1f} s"}

    if rank == 0:
        gam = steps_in[0]["gamma"]
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "B_per_gpu": w.B, "gamma_max": w.gamma_max, "V": w.V,
                       "logits": w.dtype, "temperature": w.temperature,
                       "gamma_per_row": {"choices": "hash-uniform over {2,4,6,8}", "ragged": "hash-uniform over 1..gamma_max"}.get(
                           w.gamma_mode, f"{min(w.gamma_fixed, w.gamma_max)} for every row"),
                       "temperature_mode": w.temperature_mode, "mean_gamma": float(gam.float().mean()),
                       "l2": f"{n_batches} resident batches of {bytes_step[0] / 1e6:.0f} MB alternate (each larger than L2)",
                       "parallelism": f"dp{world} (rows sharded, no collective)"},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "clocks": clocks,
            "gpu_launches": (1 if one_launch else 2) * args.steps,
            "tokens_per_step_mean": float(outs[0].n_accepted.float().mean()) + 1.0,
        }))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
