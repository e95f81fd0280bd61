#!/usr/bin/env python
"""Benchmark of the TensorGRaD optimizer step (Algorithm 1) on synthetic FNO-shaped gradients.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg3]

One "step" = one tgrad_step call on one weight tensor, following the refresh
schedule (Omega and the factors are re-selected when t mod T = 0).  Metric:
effective HBM GB/s = algorithmic bytes of a step / time (steps/s alongside).
Prints one JSON line (rank 0).
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

from paper_2501_02379_b200 import replicas, synth  # noqa: E402

METRIC = "tgrad_step effective HBM GB/s"
FALLBACK_HBM_GBS = 6650.0

NOMINAL_HBM_GBS = 8000.0      # the nominal HBM3e figure fractions are also quoted against

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the two streaming kernels as one ncu capture
# of this build's kernels counted them (bytes); None where no capture of the current kernel exists.
# (back_tail: 304.1 MB read + 218.1 MB written -- the rest of the 277 MB it writes is still in L2 when the
# kernel ends.  The 545 M-entry configuration: captured on 96x96x128x65 and scaled by the slab count, 7.11.)
NCU_TRAFFIC_BYTES = {("cfg3", "proj_tail"): 280.5e6 + 19.1e6, ("cfg3", "back_tail"): 304.1e6 + 218.2e6,
                     ("cfg5", "proj_tail"): 7.111 * (309.9e6 + 36.4e6), ("cfg5", "back_tail"): 7.111 * (353.8e6 + 248.0e6)}


def step_bytes(wl: synth.Workload) -> int:
    """Algorithmic bytes of one non-refresh step: G read once, W read + written once, the sparse
    side (index, gather, zero, both sparse moments read+written, W read-modify-write at Omega),
    the core side (core, moments, normalised core) and the factor matrices."""
    i = wl.numel
    eb = 4 if wl.half_storage else 8
    p = int(np.prod(wl.ranks, dtype=np.int64))
    fac = sum(a * b for a, b in zip(wl.shape, wl.ranks))
    return 3 * eb * i + 60 * wl.k + 40 * p + 8 * fac


def stage_bytes(wl: synth.Workload):
    """Algorithmic bytes per launch of the two streaming kernels (entries x bytes per entry)."""
    i = wl.numel
    eb = 4 if wl.half_storage else 8
    fac_tail = sum(a * b for a, b in zip(wl.shape[-2:], wl.ranks[-2:]))
    proj = eb * i + 36 * wl.k + 8 * fac_tail        # G read; idx 4 + M_S 16 + V_S 8 + N_S 8 per sparse entry
    back = 2 * eb * i + 12 * wl.k + 8 * fac_tail    # W read + write; idx 4 + N_S 8 per sparse entry
    return {"proj_tail": proj, "back_tail": back}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Reads SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self.active = False
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            if self.active:
                try:
                    self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                    try:
                        r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                    except Exception:
                        r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                    for bit, name in names.items():
                        if r & bit:
                            self.reasons.add(name)
                except Exception:
                    pass
            time.sleep(self.period)

    def stop(self):
        self._stop.set()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_sample(wl: synth.Workload, budget_s: float, n_steps: int):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the leading
    slices of mode 1 (ranks clipped to the sample's extents), sized for the time budget."""
    import dataclasses
    from oracle import tgrad_oracle as orc
    # a non-refresh oracle step handles roughly 1.5e7 entries per second on 8 cores and its refresh costs about
    # a dozen steps; size the sample for the budget (the whole tensor where that fits)
    per_step = budget_s / max(1, n_steps + 12)
    entries = max(200_000, int(1.2e7 * per_step))
    rest = wl.numel // wl.shape[0]
    i1 = int(min(wl.shape[0], max(4, entries // rest)))
    shape = (i1,) + tuple(wl.shape[1:])
    ranks = tuple(min(r, s) for r, s in zip(wl.ranks, shape))
    sub = dataclasses.replace(wl, shape=shape, ranks=ranks, signal_ranks=ranks, name=wl.name + "_sample")
    src = synth.GradientSource(sub)
    cfg = orc.OracleConfig(shape=shape, ranks=ranks, k=sub.k, T=sub.T, lr=sub.lr, half_storage=sub.half_storage)
    st = orc.OracleState(cfg)
    w = src.weight()
    grads = [src.gradient(t) for t in range(2)]
    if sub.half_storage:
        w = synth.from_half_pairs(synth.to_half_pairs(w))
        grads = [synth.from_half_pairs(synth.to_half_pairs(g)) for g in grads]
    t0 = time.perf_counter()
    w = orc.oracle_step(st, w, grads[0])            # includes the refresh (t = 0)
    t_refresh_step = time.perf_counter() - t0
    times = []
    for t in range(n_steps):
        t0 = time.perf_counter()
        w = orc.oracle_step(st, w, grads[(t + 1) % 2], refresh=False)
        times.append(time.perf_counter() - t0)
    return sub, times, t_refresh_step


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [int(i.get("num_threads", 1)) for i in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def config_of(wl: synth.Workload, world: int, ring: int):
    eb = 4 if wl.half_storage else 8
    return {"workload": wl.name, "tensors_per_gpu": wl.n_tensors, "shape": list(wl.shape), "ranks": list(wl.ranks),
            "k": wl.k, "T": wl.T, "storage": "2xfp16" if wl.half_storage else "complex64", "warm_refresh": True,
            "parallelism": "replicas only" if world > 1 else "single GPU",
            "l2": f"inputs larger than L2: ring of {ring} gradient buffers of {wl.numel * eb / 1e6:.0f} MB each "
                  f"plus the weight"}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_timed = args.steps
    sub, times, t_refresh = oracle_sample(wl, budget_s=150.0, n_steps=args.warmup + n_timed)
    timed = times[args.warmup:]
    total = float(sum(timed))
    b = step_bytes(sub)
    val = b * len(timed) / total / 1e9
    cores = blas_threads()
    sample = (f"oracle step on the leading {sub.shape[0]} of {wl.shape[0]} mode-1 slices of {wl.name} "
              f"(shape {'x'.join(map(str, sub.shape))}, ranks {sub.ranks}, k={sub.k}); refresh step {t_refresh:.2f}s")
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": len(timed),
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(timed), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, 1, args.ring),
        "sample_shape": list(sub.shape),
        "steps_per_s": len(timed) / total,
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def run_ours(args, wl):
    import torch
    from paper_2501_02379_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    B.lib()                                          # fails loudly if the CUDA library is missing
    half = wl.half_storage

    def dev(x):
        if half:
            return torch.from_numpy(synth.to_half_pairs(x)).cuda()
        return torch.from_numpy(np.ascontiguousarray(x).view(np.float32).reshape(x.shape + (2,))).cuda()

    # replicas only: every rank owns independent tensors (layers); no data-path collective
    n_t = wl.n_tensors
    srcs = [synth.GradientSource(wl, i) for i in replicas.tensor_ids_for_rank(rank, world, n_t)]
    ring = args.ring
    grads_host = [[s.gradient(r) for r in range(ring)] for s in srcs]
    if half:
        grads_host = [[synth.from_half_pairs(synth.to_half_pairs(g)) for g in gl] for gl in grads_host]
    grads = [[dev(g) for g in gl] for gl in grads_host]
    w0 = [s.weight() for s in srcs]
    weights = [dev(w) for w in w0]
    cfgs = [B.make_config(wl.shape, wl.ranks, wl.k, wl.T, lr=wl.lr, half_storage=half, auto_refresh=True,
                          warm_refresh=True)
            for _ in srcs]
    if wl.T < 2:
        raise SystemExit("the benchmark separates refresh steps from the others: T >= 2")
    states = [B.TgradState(c) for c in cfgs]
    stream = torch.cuda.current_stream()

    def one_step(t):
        if n_t == 1:
            states[0].step(weights[0], grads[0][t % ring], stream)
        else:
            B.step_batched(states, weights, [g[t % ring] for g in grads], stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    t = 0
    for _ in range(args.warmup):
        one_step(t); t += 1
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    l0 = B.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.active = True
    e0.record(stream)
    n_refresh = 0
    for _ in range(args.steps):
        if t % wl.T == 0:
            n_refresh += 1
        one_step(t); t += 1
    e1.record(stream)
    barrier()
    sampler.active = False
    launches = B.launch_count() - l0
    ms = e0.elapsed_time(e1)
    ms = replicas.max_over_ranks(ms, dist, "cuda")
    flags = [s.query_status()[0] for s in states]

    # ---- non-refresh steps alone, for at least a second of device time so that the clock sampler sees the
    #      GPU under this load (runs of T-1 steps; the counter is set back to 1 before each run, which keeps
    #      them off the refresh schedule and changes nothing but the bias-correction scalars) ----
    st0 = states[0]
    sampler.active = True
    run_len = min(wl.T - 1, 200)
    nonrefresh_total_ms, nonrefresh_steps = 0.0, 0
    while nonrefresh_total_ms < args.min_clock_ms and nonrefresh_steps < 20000:
        st0.set_step(1)
        e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2.record(stream)
        for _ in range(run_len):
            st0.step(weights[0], grads[0][t % ring], stream); t += 1
        e3.record(stream)
        torch.cuda.synchronize()
        nonrefresh_total_ms += e2.elapsed_time(e3); nonrefresh_steps += run_len
    sampler.active = False
    nonrefresh_ms = nonrefresh_total_ms / nonrefresh_steps
    # ---- per-stage device times (events on the launching stream between the stages) ----
    n_stage_steps = min(30, run_len)
    st0.set_step(1)
    st0.set_stage_timing(True)                       # the events between the stages add a few microseconds per stage
    for _ in range(n_stage_steps):
        st0.step(weights[0], grads[0][t % ring], stream); t += 1
    torch.cuda.synchronize()
    stage_ms, n_rec = st0.stage_times(stream)
    st0.set_stage_timing(False)
    # the counter of tensor 0 ran ahead of the others; irrelevant from here on
    stage_us = {name: 1e3 * v / max(1, n_rec) for name, v in zip(B.STAGE_NAMES, stage_ms)}

    # ---- steps that carry a refresh (t mod T = 0), timed alone: each on another gradient than the refresh
    #      before it, so that the warm start of the eigensolver meets a changed matrix ----
    refresh_step_list = []
    for i in range(3):
        st0.set_step(wl.T)
        e4, e5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e4.record(stream)
        st0.step(weights[0], grads[0][(i + 1) % ring], stream)
        e5.record(stream)
        torch.cuda.synchronize()
        refresh_step_list.append(e4.elapsed_time(e5))
    refresh_step_ms = float(np.median(refresh_step_list))
    refresh_ms = refresh_step_ms - nonrefresh_ms
    amortised_ms = ((wl.T - 1) * nonrefresh_ms + refresh_step_ms) / wl.T
    flags += [st0.query_status()[0]]

    # ---- end to end with host buffers: W and G go up, W comes back, every step ----
    n_e2e = max(1, min(args.steps, args.e2e_steps))
    eb = 4 if half else 8
    hw = [torch.from_numpy(np.ascontiguousarray(synth.to_half_pairs(w) if half else
                                                  w.view(np.float32).reshape(w.shape + (2,)))).pin_memory() for w in w0]
    hg = [[torch.from_numpy(np.ascontiguousarray(synth.to_half_pairs(g) if half else
                                                   g.view(np.float32).reshape(g.shape + (2,)))).pin_memory()
           for g in gl[:2]] for gl in grads_host]
    dw = [torch.empty_like(w) for w in weights]
    dg = [torch.empty_like(w) for w in weights]
    for s in states:
        s.set_step(1)            # keep the timed end-to-end steps off the refresh schedule
    barrier()
    # the gradient of step i+1 goes up on a copy stream while step i runs and its weight comes back (two device
    # gradient buffers, as an input pipeline would hold); the weight itself makes the round trip every step
    cs = torch.cuda.Stream()
    dgb = [dg, [torch.empty_like(w) for w in weights]]
    ev_up = [torch.cuda.Event(), torch.cuda.Event()]
    ev_done = [torch.cuda.Event(), torch.cuda.Event()]

    ev_wup = torch.cuda.Event()

    def upload(it):
        b = it % 2
        with torch.cuda.stream(cs):
            if it >= 1:
                cs.wait_event(ev_wup)                # after the weight upload of the step before: this copy then
                                                     # shares the link with that step's download, not with its upload
            if it >= 2:
                cs.wait_event(ev_done[b])            # the step that last read this buffer has finished
            for i in range(n_t):
                dgb[b][i].copy_(hg[i][b], non_blocking=True)
            ev_up[b].record(cs)

    e6, e7 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e6.record(stream)
    cs.wait_event(e6)
    upload(0)
    for it in range(n_e2e):
        b = it % 2
        for i in range(n_t):
            dw[i].copy_(hw[i], non_blocking=True)
        ev_wup.record(stream)
        if it + 1 < n_e2e:
            upload(it + 1)
        stream.wait_event(ev_up[b])
        if n_t == 1:
            states[0].step(dw[0], dgb[b][0], stream)
        else:
            B.step_batched(states, dw, dgb[b], stream)
        ev_done[b].record(stream)
        for i in range(n_t):
            hw[i].copy_(dw[i], non_blocking=True)
        stream.synchronize()
    e7.record(stream)
    barrier()
    e2e_ms = e6.elapsed_time(e7)
    e2e_ms = replicas.max_over_ranks(e2e_ms, dist, "cuda")
    sampler.stop()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    if any(flags):
        raise SystemExit(f"sticky device flags set during the benchmark: {flags}")
    bstep = step_bytes(wl) * n_t
    value = bstep * args.steps * world / (ms * 1e-3) / 1e9
    e2e_val = bstep * n_e2e * world / (e2e_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    sb = stage_bytes(wl)
    dom = max(("proj_tail", "back_tail"), key=lambda k: stage_us[k])
    ach = sb[dom] / (stage_us[dom] * 1e-6) / 1e9
    traffic = NCU_TRAFFIC_BYTES.get((wl.name, dom))
    out = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, world, ring),
        "steps_per_s": args.steps * world / (ms * 1e-3),
        "refreshes_in_timed_region": n_refresh,
        "step_bytes": bstep,
        # one tensor, from the separately timed regions above: a non-refresh step (mean over >= 1 s), a step that
        # carries a refresh (median of 3), and the schedule's mean ((T-1) t_step + t_refresh_step) / T
        "nonrefresh_step_us": 1e3 * nonrefresh_ms, "nonrefresh_steps_timed": nonrefresh_steps,
        "refresh_step_us": 1e3 * refresh_step_ms, "refresh_us": 1e3 * refresh_ms,
        "nonrefresh_gbs": step_bytes(wl) / (nonrefresh_ms * 1e-3) / 1e9,
        "frac_of_peak_nonrefresh": step_bytes(wl) / (nonrefresh_ms * 1e-3) / 1e9 / peak,
        "frac_of_nominal_8tbs_nonrefresh": step_bytes(wl) / (nonrefresh_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "amortised_ms_per_step": amortised_ms,
        "amortised_gbs": step_bytes(wl) / (amortised_ms * 1e-3) / 1e9,
        "frac_of_peak_amortised": step_bytes(wl) / (amortised_ms * 1e-3) / 1e9 / peak,
        "frac_of_nominal_8tbs_amortised": step_bytes(wl) / (amortised_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "peak_gbs": peak, "peak_kind": peak_kind, "nominal_gbs": NOMINAL_HBM_GBS,
        "stage_us": stage_us,
        "clocks": sampler.summary(),
        "e2e": {"value": e2e_val, "unit": "GB/s", "h2d_bytes_per_step": 2 * wl.numel * eb * n_t,
                "d2h_bytes_per_step": wl.numel * eb * n_t, "steps": n_e2e, "ms_per_step": e2e_ms / n_e2e,
                "pipeline": "gradient of step i+1 uploaded on a copy stream during step i; weight up and down every step"},
        "gpu_launches": int(launches),
        "sticky_flags": flags,
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                     "frac_of_nominal_8tbs": ach / NOMINAL_HBM_GBS,
                     "peak_kind": peak_kind, "bytes_per_launch": sb[dom], "us_per_launch": stage_us[dom],
                     "traffic": traffic},
    }
    if world == 1 and not args.no_cpu_baseline:
        sub, times, t_refresh = oracle_sample(wl, budget_s=45.0, n_steps=2)
        tm = float(np.median(times))
        out["cpu_baseline"] = {
            "value": step_bytes(sub) / tm / 1e9, "unit": "GB/s", "cores": blas_threads(), "kind": "oracle",
            "sample": f"oracle non-refresh step on the leading {sub.shape[0]} of {wl.shape[0]} mode-1 slices "
                      f"(shape {'x'.join(map(str, sub.shape))}, ranks {sub.ranks}, k={sub.k}): "
                      f"{tm:.2f}s per step, {t_refresh:.2f}s for the refresh step",
        }
    print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--ring", type=int, default=3, help="distinct gradient buffers cycled through")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-clock-ms", type=float, default=1200.0,
                    help="device time of the separately timed non-refresh region (the clock sampler runs over it)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    wl = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
