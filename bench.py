#!/usr/bin/env python
"""Benchmark of the batched FSD verification step.

One "step" is one fsd_verify_chain call (every kernel of the hot path) over one batch of
synthetic logits of the headline workload: chain, B=64, gamma=8, V=152064, bf16, JS, T=0.2.
Prints ONE JSON line.  `value` is verified draft positions per second with inputs resident in
HBM; `e2e` is the same through the host-buffer entry point with the copies inside the timed
region; `roofline` relates the algorithmic bytes (each needed logit read once) to the measured
HBM copy bandwidth; `cpu_baseline` times the double-precision CPU oracle on a bounded sample.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (under torchrun) every rank runs an independent replica of the workload on its own
GPU (the path has no exchange step), the timed region is bracketed by barriers and the time is
the maximum over ranks.
"""

from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import fsd_inputs as gi  # noqa: E402

WORKLOAD = "c4"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + written) of one pair-kernel launch on the headline workload, from the ncu
# capture summarised under profiles/; set to None whenever that kernel changes after the capture.
PAIR_KERNEL_DRAM_BYTES = 311_719_936
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def aggregate_over_ranks(local_ms: float, local_units: float, world: int, reduce_max, reduce_sum):
    """Whole-job throughput from per-rank numbers: units of all ranks over the slowest rank's time.
    `reduce_max` / `reduce_sum` are the collectives (identity functions when world == 1)."""
    t = reduce_max(local_ms)
    units = reduce_sum(local_units)
    return units / (t * 1e-3), t


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read only)."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _once(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        except Exception:
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
        names = {
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "hw_power_brake": getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80),
        }
        for k, bit in names.items():
            if r & bit:
                self.reasons.add(k)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
            try:
                self._once()
            except Exception:
                pass

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_sample_rate(c, rows: int, T: float, nthreads: int = 0):
    """Times the CPU oracle (as it stands) on the first `rows` batch rows; returns (positions/s, seconds, cores)."""
    from oracle import fsd_oracle as orc
    orc.lib()
    cores = orc.max_threads() if nthreads <= 0 else nthreads
    t0 = time.perf_counter()
    orc.verify_chain(c.target[:rows], c.draft[:rows], None, None, c.u_sample[:rows], dtype=c.dtype, div="js",
                     mode="fsd", T=T, nthreads=nthreads)
    dt = time.perf_counter() - t0
    return rows * c.gamma / dt, dt, cores


def run_reference(args, rank: int, world: int):
    """The reference arm: the CPU oracle on the host cores, each step a bounded sample of the workload."""
    if rank != 0:
        return
    rows = args.ref_rows
    c = gi.make_config(WORKLOAD, B=rows)
    T = float(gi.CONFIGS[WORKLOAD].thresholds[0])
    for _ in range(max(args.warmup, 1)):
        oracle_sample_rate(c, rows, T)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_rate(c, rows, T)
    dt = time.perf_counter() - t0
    from oracle import fsd_oracle as orc
    value = rows * c.gamma * args.steps / dt
    sample = f"first {rows} of 64 batch rows of the workload per step ({rows * c.gamma} positions)"
    line = {
        "impl": "reference", "metric": "verified draft positions/sec", "value": value, "unit": "positions/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(c, rows, sampled=True),
        "cpu_baseline": {"value": value, "unit": "positions/s", "cores": orc.max_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "positions/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(c, B, sampled=False):
    spec = gi.CONFIGS[WORKLOAD].params
    same = (B if not sampled else spec["B"], c.gamma, c.V, c.dtype) == (spec["B"], spec["gamma"], spec["V"], spec["dtype"])
    mb = c.elem_size * B * (2 * c.gamma + 1) * c.V / 1e6
    return {"workload": f"chain FSD verify B={B} gamma={c.gamma} V={c.V} {c.dtype} JS T=0.2 "
                        + ("(config 4)" if same else "(config 4's recipe, other shape)"),
            "B": B, "gamma": c.gamma, "V": c.V, "divergence": "js", "mode": "fsd", "threshold": 0.2,
            "parallelism": "independent replicas",
            "l2": f"inputs ({mb:.0f} MB) exceed L2 (126 MB); 3 input copies rotated between steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=12)
    ap.add_argument("--copies", type=int, default=3)
    ap.add_argument("--ref-rows", type=int, default=16, help="batch rows per step of the reference arm")
    # extra rows (not the headline): the headline recipe with another vocabulary, length, batch or dtype
    ap.add_argument("--V", type=int, default=None, help="vocabulary size instead of 152064 (e.g. 256000)")
    ap.add_argument("--gamma", type=int, default=None, help="candidate length instead of 8 (e.g. 10, 15, 20)")
    ap.add_argument("--B", type=int, default=None, help="batch rows instead of 64")
    ap.add_argument("--dtype", default=None, choices=["bf16", "f32"], help="logit type instead of bf16")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import paper_2502_20704_b200 as fsd

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def reduce_sum(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    # ---- workload (same seeded inputs on every rank: replicas) ----
    overrides = {k: v for k, v in (("V", args.V), ("gamma", args.gamma), ("B", args.B), ("dtype", args.dtype))
                 if v is not None}
    headline = not overrides
    c = gi.make_config(WORKLOAD, **overrides)
    T = float(gi.CONFIGS[WORKLOAD].thresholds[0])
    B, gamma, V = c.B, c.gamma, c.V
    opts = fsd.make_opts(div="js", mode="fsd", cmp="lt", sample="invcdf", dtype=c.dtype, T=T)
    if c.dtype == "bf16":
        h_target = torch.from_numpy(c.target.view(np.int16)).view(torch.bfloat16).pin_memory()
        h_draft = torch.from_numpy(c.draft.view(np.int16)).view(torch.bfloat16).pin_memory()
    else:
        h_target = torch.from_numpy(c.target).pin_memory()
        h_draft = torch.from_numpy(c.draft).pin_memory()
    h_us = torch.from_numpy(c.u_sample).pin_memory()
    copies = [(h_target.cuda(), h_draft.cuda()) for _ in range(max(args.copies, 1))]
    us = h_us.cuda()
    acc = torch.empty(B, dtype=torch.int32, device="cuda")
    tok = torch.empty(B, dtype=torch.int32, device="cuda")
    D = torch.empty(B, gamma, dtype=torch.float32, device="cuda")
    st = torch.empty(B, dtype=torch.int32, device="cuda")
    wsb = fsd.fsd_workspace_bytes(B, gamma, V, opts)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    sptr = stream.cuda_stream
    launches_per_step = 2

    def step(i):
        t, d = copies[i % len(copies)]
        rc = fsd.fsd_verify_chain(t, d, None, None, us, B, gamma, V, opts, acc, tok, D, st, ws, wsb, sptr)
        if rc != 0:
            raise RuntimeError(fsd.fsd_status_string(rc))

    for i in range(args.warmup):
        step(i)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        ev0.record(stream)
        for i in range(args.steps):
            step(i)
        ev1.record(stream)
        barrier()
    local_ms = ev0.elapsed_time(ev1)
    value, total_ms = aggregate_over_ranks(local_ms, float(B * gamma * args.steps), world, reduce_max, reduce_sum)
    ms_per_step = total_ms / args.steps
    res_acc, res_D = acc.cpu().numpy(), D.cpu().numpy()

    # ---- which kernel takes the time: a short second loop with an event recorded by the library
    #      between the pair kernel and the finish kernel (the calls are queued back to back, so
    #      the intervals are kernel durations, not launch gaps) ----
    n_attr = max(1, min(args.steps, 50))
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_attr)]
    for e3 in ev:
        e3[1].record(stream)                      # creates the handle the library will re-record
    for i in range(n_attr):
        ev[i][0].record(stream)
        fsd.fsd_set_stage_event(ev[i][1])
        step(i)
        ev[i][2].record(stream)
    fsd.fsd_set_stage_event(None)
    torch.cuda.synchronize()
    pair_ms = float(np.median([e3[0].elapsed_time(e3[1]) for e3 in ev]))
    finish_ms = float(np.median([e3[1].elapsed_time(e3[2]) for e3 in ev]))

    # ---- end to end: host buffers in, host results out, copies inside the timed region ----
    stg_b = fsd.fsd_host_staging_bytes(B, gamma, V, opts)
    staging = torch.empty(stg_b, dtype=torch.uint8, device="cuda")
    h_acc = torch.empty(B, dtype=torch.int32).pin_memory()
    h_tok = torch.empty(B, dtype=torch.int32).pin_memory()
    h_D = torch.empty(B, gamma, dtype=torch.float32).pin_memory()
    h_st = torch.empty(B, dtype=torch.int32).pin_memory()

    def e2e_step():
        rc = fsd.fsd_verify_chain_host(h_target, h_draft, None, None, h_us, B, gamma, V, opts,
                                       h_acc, h_tok, h_D, h_st, staging, stg_b, sptr)
        if rc != 0:
            raise RuntimeError(fsd.fsd_status_string(rc))

    for _ in range(3):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_value, e2e_ms = aggregate_over_ranks(e0.elapsed_time(e1), float(B * gamma * args.e2e_steps), world,
                                             reduce_max, reduce_sum)
    h2d = (h_target.numel() + h_draft.numel()) * c.elem_size + h_us.numel() * 4
    d2h = (h_acc.numel() + h_tok.numel() + h_D.numel() + h_st.numel()) * 4
    assert np.array_equal(h_acc.numpy(), res_acc)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the pair kernel): its algorithmic bytes (both rows of
    #      every pair read once) over its own duration; the whole call is given beside it ----
    peak, peak_kind = measured_hbm_peak()
    ideal = c.ideal_bytes
    pair_bytes = c.elem_size * B * gamma * 2 * V
    achieved = pair_bytes / (pair_ms * 1e-3) / 1e9
    call_achieved = ideal / (ms_per_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": PAIR_KERNEL_DRAM_BYTES if headline else None, "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
                "kernel": "pair kernel (fsd_pair_stream_kernel<bf16, JS> on the headline workload; includes the "
                          "256-byte flag memset in front of it)",
                "algorithmic_bytes_per_launch": pair_bytes, "ms_per_launch": pair_ms,
                "finish_kernel_ms": finish_ms,
                "whole_call": {"achieved": call_achieved, "frac": call_achieved / peak,
                               "algorithmic_bytes_per_call": ideal, "ms_per_call": ms_per_step}}

    # ---- CPU baseline: the oracle on a bounded sample, rank 0, N = 1 only ----
    cpu = None
    if world == 1:
        rows = 16
        v, secs, cores = oracle_sample_rate(c, rows, T)
        if secs < 5.0:
            reps = int(min(20, max(1, 10.0 / max(secs, 1e-3))))
            t0 = time.perf_counter()
            for _ in range(reps):
                oracle_sample_rate(c, rows, T)
            v = rows * gamma * reps / (time.perf_counter() - t0)
        cpu = {"value": v, "unit": "positions/s", "cores": cores, "kind": "oracle",
               "sample": f"first {rows} of {B} batch rows ({rows * gamma} positions per pass), repeated for ~10 s"}

    hist = np.bincount(res_acc, minlength=gamma + 1).tolist()
    line = {
        "metric": "verified draft positions/sec", "value": value, "unit": "positions/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(c, B),
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": "positions/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / args.e2e_steps, "steps": args.e2e_steps},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks.summary(),
        "workload_stats": {"accept_len_hist": hist, "D_min": float(np.nanmin(res_D)),
                           "D_median": float(np.nanmedian(res_D)), "D_max": float(np.nanmax(res_D))},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
