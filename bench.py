#!/usr/bin/env python
"""Benchmark of the FDA hot path on B200: one step = local states -> combine/estimate ->
K-way model average (in-place sync) over one synthetic workload resident in HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..7] [--impl reference]

Prints ONE JSON line.  ``value`` is params*workers/s of the whole step (K*d elements per
step / device time per step, CUDA events on the launching stream); ``roofline`` describes
the dominant kernel (the fused local-state pass); ``e2e`` is the same metric through
``fda_round_host`` (pinned host buffers, copies inside the timed region); ``cpu_baseline``
is the CPU oracle timed on a bounded sample of the same workload; ``also`` (default workload
only) holds the step, kernel times and roofline of the 20M-parameter workload, measured in the
same process after the main one is freed.

With ``--impl reference`` the CPU oracle itself is the timed arm (rank 0 only).
Under torchrun every rank runs an independent replica of the workload on its own GPU (the
path has no inter-GPU exchange); the time is the max over ranks and the value the sum.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import fda_synth as S  # noqa: E402

METRIC = "FDA local-state+sketch throughput (local state -> estimate -> K-way average)"
UNIT = "params*workers/s"
SKETCH_STATE = 1 | 4      # SketchFDA local state (Theorem 1): squared norm + AMS sketch
LINEAR_STATE = 1 | 2      # LinearFDA local state (Theorem 2): squared norm + projection
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 << 20
NOMINAL_HBM_GBS = 8000.0               # the data-sheet figure, quoted beside the measured copy rate
SMEM_CAS_UPDATES_PER_CLK_SM = 6.8     # measured on B200: bare fp32 shared-memory atomicAdd loop, 1024 threads
SMEM_GATHER_UPDATES_PER_CLK_SM = 32.0  # one 4-byte shared-memory read per update at 128 bytes per clock and SM

# dram__bytes_read.sum + dram__bytes_write.sum of one sketch-pass launch come from the ncu launch
# lists summarised under profiles/: profiles/traffic.json names, per workload, the bytes, the
# summary file and the sha256 of the kernel sources the capture was taken with.  When the sources
# have changed since, the figure is stale and the bench line says null.
KERNEL_SOURCES = ("paper_2405_20988_b200/csrc/fda_local_state_gather.cu", "paper_2405_20988_b200/csrc/fda_list_kernel.cuh",
                  "paper_2405_20988_b200/csrc/fda_sched.cu", "paper_2405_20988_b200/csrc/fda_internal.h")


def kernel_sources_sha256() -> str:
    import hashlib
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_traffic(workload: int):
    """(bytes per launch or None, where the figure comes from)"""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            tab = json.load(f)
        ent = tab["workloads"].get(str(workload))
        if ent is None:
            return None, "no capture for this workload"
        if tab["sources_sha256"] != kernel_sources_sha256():
            return None, "kernel sources changed since %s was captured" % ent["profile"]
        return ent["bytes"], ent["profile"]
    except (OSError, KeyError, ValueError):
        return None, "profiles/traffic.json missing"


def secondary_roofline(kernel, updates_per_s, n_sm, sm_mhz):
    gather = kernel == "k_local_state_gather"
    per_clk = SMEM_GATHER_UPDATES_PER_CLK_SM if gather else SMEM_CAS_UPDATES_PER_CLK_SM
    peak = per_clk * n_sm * sm_mhz * 1e6
    return {"bound": "smem_gather" if gather else "smem_cas", "unit": "updates/s", "achieved": updates_per_s,
            "peak": peak, "frac": updates_per_s / peak,
            "note": ("peak = one 4-byte shared-memory read per update, 128 bytes per clock and SM" if gather else
                     "peak = microbenchmarked fp32 atomicAdd rate on lane-private columns")}


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    """nvidia-smi sampler (100 ms) running beside the timed region; read-only queries."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines, self.thread = index, None, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax,
                "samples": len(sm), "reasons": sorted(reasons)}


def clocks_rejected(c) -> bool:
    bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(c.get("reasons", []))
    stuck = (c.get("sm_mhz") and c.get("sm_max_mhz") and not c.get("reasons")
             and c["sm_mhz"] < 0.6 * c["sm_max_mhz"])
    return bool(bad) or bool(stuck)


# ------------------------------------------------------------------- multi-rank plumbing
def max_over_ranks(value: float, dist, device="cpu") -> float:
    """Slowest rank's time: every multi-GPU number is the max over ranks."""
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world: int, units_per_rank: float, step_seconds: float) -> float:
    """Whole-job throughput of `world` independent replicas (weak scaling)."""
    return world * units_per_rank / step_seconds


# ----------------------------------------------------------------------- CPU baseline
def oracle_step_on_sample(wl, w_host, w_t0, xi, coeffs, d_sample, threads):
    """One whole step of the CPU oracle on the first d_sample indices of every worker."""
    import oracle
    t0 = time.perf_counter()
    st = oracle.local_state(w_host[:, :d_sample], w_t0[:d_sample], None, coeffs, wl.l, wl.m,
                            threads=threads)
    est = oracle.combine(st, wl.l, wl.m, 1, wl.epsilon, wl.thetas[-1])
    if est["trigger"]:
        oracle.average(w_host[:, :d_sample])
    dt = time.perf_counter() - t0
    return dt, est


def cpu_sample_size(wl, cores):
    # about 10-30 s of CPU work: the oracle does roughly 1e8 element*workers per second on 8-16 cores
    budget_elems = 1.5e9
    return int(min(wl.d, max(4096, budget_elems // wl.K)))


# ---------------------------------------------------------------------------- own arm
def run_ours(args, rank, world, local_rank):
    import torch
    import paper_2405_20988_b200 as F

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback exists)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    cores = host_cores()
    gen_threads = max(1, cores // max(1, world))

    class Run:
        """One workload resident in HBM with its context, and the timed steps on it."""

    def setup_and_time(workload, steps, warmup):
        r = Run()
        wl = S.WORKLOADS[workload]
        d, K = wl.d, wl.K
        r.wl, r.d, r.K = wl, d, K
        r.w_t0_np = S.last_global_model(wl)
        r.xi_np = S.unit_direction(wl)
        r.coeffs = S.hash_coefficients(wl.seed, wl.l)
        stride = S.row_stride(d)
        r.stride = stride
        r.w_pin = torch.empty((K, stride), dtype=torch.float32).pin_memory()
        S.worker_models(wl, r.w_t0_np, out=r.w_pin.numpy(), threads=gen_threads)
        r.w0_pin = torch.from_numpy(r.w_t0_np).pin_memory()
        xi_pin = torch.from_numpy(r.xi_np).pin_memory()

        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ctx = F.FdaContext(wl.l, wl.m, r.coeffs, d_max=d, K_max=K, device=local_rank)
        r.create_ms = (time.perf_counter() - t0) * 1e3
        r.ctx = ctx
        r.w_src = r.w_pin.to(dev, non_blocking=True)          # pristine copies (restored before each step)
        r.w0_src = r.w0_pin.to(dev, non_blocking=True)
        r.xi = xi_pin.to(dev, non_blocking=True)
        r.w = torch.empty_like(r.w_src)
        r.w0 = torch.empty_like(r.w0_src)
        r.states = torch.empty((K, ctx.state_len), dtype=torch.float32, device=dev)
        r.est_buf = ctx.new_estimate_buffer(dev)
        r.theta, r.eps = float(wl.thetas[-1]), float(np.float32(wl.epsilon))
        r.ls_kernel = ""       # the kernel the library picked for the sketch pass (asked after each launch)
        r.ls_launches = 2
        w, w0, states, est_buf = r.w, r.w0, r.states, r.est_buf

        def step_events():
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev[0].record(stream)
            ctx.fda_local_state(w[:, :d], w0, None, SKETCH_STATE, states)
            r.ls_kernel = ctx.fda_debug_last_kernel()
            r.ls_launches = ctx.fda_debug_last_launches()
            ev[1].record(stream)
            ctx.fda_combine_estimate(states, K, F.FDA_VARIANT_SKETCH, r.eps, r.theta, est_buf, want_host=False)
            ev[2].record(stream)
            ctx.fda_average_models(w[:, :d], w0, est_buf, F.FDA_AVG_BROADCAST)
            ev[3].record(stream)
            return ev

        def step(timed):
            # the sync of the previous step made all models equal: put the drifted models back
            w.copy_(r.w_src)
            w0.copy_(r.w0_src)
            return step_events()

        r.step, r.step_events = step, step_events

        def timed_run():
            sampler = ClockSampler(local_rank)      # spans warm-up and timed steps (all under load)
            sampler.start()
            for _ in range(warmup):
                step(False)
            torch.cuda.synchronize()
            if dist:
                dist.barrier()
            torch.cuda.synchronize()
            evs = [step(True) for _ in range(steps)]
            torch.cuda.synchronize()
            if dist:
                dist.barrier()
            late = False
            if not sampler.lines:
                # the timed region was shorter than one sampling period: keep the same load running
                # (untimed) until the sampler has seen it
                late = True
                t_end = time.perf_counter() + 1.5
                while len(sampler.lines) < 2 and time.perf_counter() < t_end:
                    for _ in range(20):
                        step(False)
                    torch.cuda.synchronize()
            clocks = sampler.stop()
            if late:
                clocks["sampled"] = "under the same load right after the timed steps (they took less than one sample period)"
            parts = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(3)] for e in evs])
            return parts, clocks

        parts, clocks = timed_run()
        if clocks_rejected(clocks):
            parts, clocks = timed_run()
            clocks["remeasured"] = True
        r.parts, r.clocks = parts, clocks
        r.est = F.Estimate.from_buffer_copy(bytes(est_buf.cpu().numpy()))
        if not r.est.trigger:
            raise SystemExit("bench: the round did not trigger; the average was not timed")
        r.info = ctx.fda_context_info()
        return r

    def roofline_of(r, peak, peak_kind):
        """The sketch pass of a run against the HBM roofline (algorithmic bytes: w, w_t0 read; states written)."""
        ls_ms = float(r.parts[:, 0].mean())
        algo_bytes = 4.0 * (r.K * r.d + r.d + r.K * r.ctx.state_len)
        achieved = algo_bytes / (ls_ms * 1e-3) / 1e9
        traffic, traffic_src = measured_traffic(r.wl_id)
        return {"kernel": r.ls_kernel, "bound": "hbm", "achieved": achieved, "peak": peak,
                "peak_kind": peak_kind + " copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                "algorithmic_bytes": algo_bytes, "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
                "traffic": traffic, "traffic_source": traffic_src}

    stream = torch.cuda.current_stream()
    run = setup_and_time(args.workload, args.steps, args.warmup)
    run.wl_id = args.workload
    wl, d, K, ctx = run.wl, run.d, run.K, run.ctx
    w, w0, w_src, w0_src, xi, states, est_buf = run.w, run.w0, run.w_src, run.w0_src, run.xi, run.states, run.est_buf
    w_pin, w0_pin, w_t0_np, xi_np, coeffs, stride = run.w_pin, run.w0_pin, run.w_t0_np, run.xi_np, run.coeffs, run.stride
    theta, eps, parts, clocks, est = run.theta, run.eps, run.parts, run.clocks, run.est
    ls_kernel = [run.ls_kernel]
    step_events = run.step_events

    # ---- the LinearFDA flavour of the local-state pass, timed beside the headline step ----
    w.copy_(w_src)
    w0.copy_(w0_src)
    lin_ms = []
    for it in range(3 + 10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.fda_local_state(w[:, :d], w0, xi, LINEAR_STATE, states)
        e1.record(stream)
        torch.cuda.synchronize()
        if it >= 3:
            lin_ms.append(e0.elapsed_time(e1))
    lin_ms = float(np.mean(lin_ms))
    lin_est = ctx.fda_combine_estimate(states, K, F.FDA_VARIANT_LINEAR, eps, theta, est_buf).as_dict()

    # ---- the one-pass averaged state (sketch of the mean drift, by linearity) ----
    mean_state = torch.empty((ctx.state_len,), dtype=torch.float32, device=dev)
    mean_ms = []
    for it in range(3 + 10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.fda_mean_state(w[:, :d], w0, None, SKETCH_STATE, mean_state)
        e1.record(stream)
        torch.cuda.synchronize()
        if it >= 3:
            mean_ms.append(e0.elapsed_time(e1))
    mean_ms = float(np.mean(mean_ms))
    mean_kernel = ctx.fda_debug_last_kernel()
    mean_est = ctx.fda_combine_estimate(mean_state.view(1, -1), 1, F.FDA_VARIANT_SKETCH, eps, theta, est_buf).as_dict()
    # ---- a kernel that only reads, on the same tensor (yardstick for the streaming kernels) ----
    probe_out = torch.zeros(1, dtype=torch.float32, device=dev)
    probe_ms = []
    for it in range(3 + 10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.fda_debug_read_probe(w, probe_out)
        e1.record(stream)
        torch.cuda.synchronize()
        if it >= 3:
            probe_ms.append(e0.elapsed_time(e1))
    probe_gbs = 4.0 * w.numel() / (float(np.mean(probe_ms)) * 1e-3) / 1e9

    # ---- cold-L2 timing for models that fit in L2 (the restoring copy leaves them cached) ----
    cold = None
    if 4 * K * stride < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        cold_parts = []
        for it in range(3 + 10):
            w.copy_(w_src)
            w0.copy_(w0_src)
            flush.zero_()
            ev = step_events()
            torch.cuda.synchronize()
            if it >= 3:
                cold_parts.append([ev[i].elapsed_time(ev[i + 1]) for i in range(3)])
        cp = np.array(cold_parts).mean(axis=0)
        cold = {"local_state": float(cp[0]), "combine": float(cp[1]), "average": float(cp[2]),
                "note": "a %d MB buffer written between the restoring copy and the step" % (2 * L2_BYTES >> 20)}
        del flush

    step_ms = float(parts.sum(axis=1).mean())
    step_all = parts.sum(axis=1)
    if dist:
        step_ms = max_over_ranks(step_ms, dist, dev)
    ls_ms, cb_ms, av_ms = (float(x) for x in parts.mean(axis=0))

    # ---- end to end through the host entry point (pinned buffers, copies timed) ----------
    slen = ctx.state_len
    st_pin = torch.empty((K, slen), dtype=torch.float32).pin_memory()
    e2e_steps = 0 if args.skip_e2e else max(1, min(args.steps, 5))
    e2e_times = []
    for it in range(2 + e2e_steps if e2e_steps else 0):
        w0_pin.copy_(torch.from_numpy(w_t0_np))
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e = ctx.fda_round_host(w_pin[:, :d], w0_pin, None, SKETCH_STATE, F.FDA_VARIANT_SKETCH, eps, theta,
                               0, st_pin)           # result: states, estimate, new global model
        dt = time.perf_counter() - t0
        if it >= 2:
            e2e_times.append(dt)
        assert e.trigger == 1
    e2e_s = float(np.mean(e2e_times)) if e2e_times else float('nan')
    if dist:
        e2e_s = max_over_ranks(e2e_s, dist, dev)
    h2d = 4 * (K * d + d)
    d2h = 4 * (d + K * slen) + 88

    out = None
    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
        algo_bytes = 4.0 * (K * d + d + K * slen)            # w, w_t0 read; states written
        lin_bytes = 4.0 * (K * d + 2 * d + K * slen)         # + xi
        achieved = algo_bytes / (ls_ms * 1e-3) / 1e9
        cpu = None
        if world == 1 and not args.skip_cpu_baseline:
            d_s = cpu_sample_size(wl, cores)
            threads = min(cores, K)
            dt, _ = oracle_step_on_sample(wl, w_pin.numpy(), w_t0_np, xi_np, coeffs, d_s, threads)
            d_1 = max(4096, d_s // max(1, threads))
            dt1, _ = oracle_step_on_sample(wl, w_pin.numpy(), w_t0_np, xi_np, coeffs, d_1, 1)
            cpu = {"value": K * d_s / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": "all %d workers x first %d of %d indices, one whole step, %.1f s" % (K, d_s, d, dt),
                   "single_thread": {"value": K * d_1 / dt1, "cores": 1,
                                     "sample": "first %d indices, %.1f s" % (d_1, dt1)}}
        out = {
            "metric": METRIC, "value": job_value(world, K * d, step_ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
            "ms_per_step_median": float(np.median(step_all)), "ms_per_step_best": float(step_all.min()),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": "%d:%s d=%d K=%d sketch=%dx%d eps=%.4f theta=%g" %
                                   (args.workload, wl.name, d, K, wl.l, wl.m, wl.epsilon, theta),
                       "state": "SketchFDA: norm+sketch", "variant": "sketch", "average": "broadcast in place",
                       "l2": "inputs (%.1f GB) larger than L2; models restored from a pristine copy before "
                             "each step, outside the timed events" % (4 * K * d / 1e9),
                       "multi_gpu": "replicas only"},
            "kernels_ms": {"local_state": ls_ms, "combine": cb_ms, "average": av_ms},
            "kernels_ms_cold_l2": cold,
            "read_probe": {"gbs": probe_gbs, "frac_of_peak": probe_gbs / peak,
                           "note": "fda_debug_read_probe over the model tensor: a kernel that only reads"},
            "local_state_only": {"value": K * d / (ls_ms * 1e-3), "unit": UNIT},
            "average_only": {"gbs": 4.0 * (2 * K * d + d) / (av_ms * 1e-3) / 1e9,
                             "frac_of_peak": 4.0 * (2 * K * d + d) / (av_ms * 1e-3) / 1e9 / peak,
                             "frac_of_nominal_8tbs": 4.0 * (2 * K * d + d) / (av_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
            "linear_local_state": {"ms": lin_ms, "value": K * d / (lin_ms * 1e-3), "unit": UNIT,
                                   "gbs": lin_bytes / (lin_ms * 1e-3) / 1e9,
                                   "frac_of_peak": lin_bytes / (lin_ms * 1e-3) / 1e9 / peak, "H": lin_est["H"]},
            "mean_state": {"ms": mean_ms, "value": K * d / (mean_ms * 1e-3), "unit": UNIT,
                           "gbs": 4.0 * (K * d + d + slen) / (mean_ms * 1e-3) / 1e9,
                           "frac_of_peak": 4.0 * (K * d + d + slen) / (mean_ms * 1e-3) / 1e9 / peak,
                           "H": mean_est["H"], "kernel": mean_kernel,
                           "note": "fda_mean_state: S-bar without the per-worker sketches"},
            "estimate": {"H": est.H, "trigger": int(est.trigger)},
            "roofline": roofline_of(run, peak, peak_kind),
            # what binds the sketch pass next to HBM: the shared-memory traffic of the l updates per
            # element (gather kernel: one 4-byte read each, 32 per clock and SM at best; the
            # compare-and-swap kernels: a measured 6.8 adds per clock and SM)
            "secondary_roofline": secondary_roofline(ls_kernel[0], K * d * wl.l / (ls_ms * 1e-3), n_sm,
                                                     clocks.get("sm_mhz") or 1965.0),
            "cpu_baseline": cpu,
            "e2e": None if not e2e_times else
                   {"value": job_value(world, K * d, e2e_s), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3, "api": "fda_round_host"},
            "gpu_launches": (run.ls_launches + 2) * args.steps,     # the state pass, its finalize, combine, average
            "clocks": clocks,
            "context": {"device_bytes": run.info["device_bytes"], "schedule_bytes": run.info["schedule_bytes"],
                        "tile_indices": run.info["tile_indices"], "table_bytes": run.info["table_bytes"],
                        "schedule_dropped_bytes": run.info["schedule_dropped_bytes"],
                        "fda_create_ms": run.create_ms, "schedule_build_ms": run.info["schedule_build_us"] / 1e3,
                        "note": "as reported by fda_context_info after the timed steps (before the lazily "
                                "allocated scratch of fda_mean_state and fda_round_host)"},
            "also": None,
        }
    ctx.close()
    # ---- the other roofline workload named by the target (20M parameters, K = 60, sketch 7 x 500),
    # measured in the same process once the main workload is freed ----
    if rank == 0 and world == 1 and args.workload == 5 and not args.skip_also:
        del run, w, w0, w_src, w0_src, xi, states, est_buf, w_pin, w0_pin, st_pin, mean_state
        torch.cuda.empty_cache()
        r4 = setup_and_time(4, max(3, min(args.steps, 20)), 3)
        r4.wl_id = 4
        p4 = r4.parts.mean(axis=0)
        mean4 = torch.empty((r4.ctx.state_len,), dtype=torch.float32, device=dev)
        mean4_ms = []
        for it in range(3 + 10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            r4.ctx.fda_mean_state(r4.w_src[:, :r4.d], r4.w0_src, None, SKETCH_STATE, mean4)
            e1.record(stream)
            torch.cuda.synchronize()
            if it >= 3:
                mean4_ms.append(e0.elapsed_time(e1))
        mean4_ms = float(np.mean(mean4_ms))
        out["also"] = {
            "config": {"workload": "4:%s d=%d K=%d sketch=%dx%d eps=%.4f theta=%g" %
                                   (r4.wl.name, r4.d, r4.K, r4.wl.l, r4.wl.m, r4.wl.epsilon, r4.theta)},
            "steps": int(r4.parts.shape[0]), "warmup": 3,
            "ms_per_step": float(r4.parts.sum(axis=1).mean()),
            "value": r4.K * r4.d / (float(r4.parts.sum(axis=1).mean()) * 1e-3), "unit": UNIT,
            "kernels_ms": {"local_state": float(p4[0]), "combine": float(p4[1]), "average": float(p4[2])},
            "roofline": roofline_of(r4, peak, peak_kind),
            "average_only": {"gbs": 4.0 * (2 * r4.K * r4.d + r4.d) / (float(p4[2]) * 1e-3) / 1e9,
                             "frac_of_peak": 4.0 * (2 * r4.K * r4.d + r4.d) / (float(p4[2]) * 1e-3) / 1e9 / peak},
            "secondary_roofline": secondary_roofline(r4.ls_kernel, r4.K * r4.d * r4.wl.l / (float(p4[0]) * 1e-3), n_sm,
                                                     r4.clocks.get("sm_mhz") or 1965.0),
            "mean_state": {"ms": mean4_ms, "value": r4.K * r4.d / (mean4_ms * 1e-3), "unit": UNIT,
                           "kernel": r4.ctx.fda_debug_last_kernel()},
            "estimate": {"H": r4.est.H, "trigger": int(r4.est.trigger)},
            "context": {"device_bytes": r4.info["device_bytes"], "schedule_bytes": r4.info["schedule_bytes"],
                        "tile_indices": r4.info["tile_indices"], "fda_create_ms": r4.create_ms},
            "clocks": r4.clocks,
        }
        out["gpu_launches"] += (r4.ls_launches + 2) * int(r4.parts.shape[0])
        r4.ctx.close()
    if dist:
        dist.barrier()
        dist.destroy_process_group()
    return out


# ---------------------------------------------------------------------- reference arm
def run_reference(args, rank, world):
    """The CPU oracle as it stands, timed on the host cores on a bounded sample per step."""
    if rank != 0:
        return None
    wl = S.WORKLOADS[args.workload]
    cores = host_cores()
    threads = min(cores, wl.K)
    d_s = cpu_sample_size(wl, cores)
    sub = S.small_workload(wl.seed, d_s, wl.K, wl.l, wl.m, wl.drift, wl.sigma, wl.epsilon)
    w_t0 = S.last_global_model(sub)
    w = S.worker_models(sub, w_t0, threads=cores)
    xi = S.unit_direction(sub)
    coeffs = S.hash_coefficients(wl.seed, wl.l)
    for _ in range(min(args.warmup, 1)):
        oracle_step_on_sample(sub, w, w_t0, xi, coeffs, d_s, threads)
    times = [oracle_step_on_sample(sub, w, w_t0, xi, coeffs, d_s, threads)[0] for _ in range(args.steps)]
    dt = float(np.mean(times))
    value = wl.K * d_s / dt
    sample = "all %d workers x %d of %d indices per step (same recipe)" % (wl.K, d_s, wl.d)
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%d:%s d=%d K=%d sketch=%dx%d" % (args.workload, wl.name, wl.d, wl.K, wl.l, wl.m),
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=5, choices=sorted(S.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="omit the oracle timing (profiling runs)")
    ap.add_argument("--skip-e2e", action="store_true", help="omit the host-buffer leg (profiling runs)")
    ap.add_argument("--skip-also", action="store_true", help="omit the second roofline workload (profiling runs)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        out = run_reference(args, rank, world)
    else:
        args.warmup = max(args.warmup, 3)
        out = run_ours(args, rank, world, local_rank)
    if out is not None:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
