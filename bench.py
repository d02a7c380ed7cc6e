#!/usr/bin/env python
"""Benchmark of the fused Non-blocking SGD step (masked accumulate + mix + momentum + update).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of synthetic mini-batch gradients:
the host straggler simulator draws the finished counts, then nb_step_fused runs (for MATCHA the
device-side W builder runs first).  Prints ONE JSON line (rank 0).

  value     K*P*N / t_step  (params*learners/s), gradient stream already resident in HBM
  e2e       the same metric through nb_step_fused_host: pinned HOST gradient buffers, the H2D copies
            of the finished rows and the D2H copy of the mean model inside the timed region
  roofline  algorithmic bytes of one fused-step launch / its mean CUDA-event duration, against
            the measured HBM copy bandwidth of this machine's B200s; `sustained` repeats the same step
            for at least two seconds and reports it against the clocks sampled meanwhile
  workloads the other configurations, variants and entry points, one short run each (N = 1 only)
  cpu_baseline  the CPU oracle, as it stands, timed on a bounded column slice of the same workload:
            on one core and on every core the process may use (columns split over processes)

With N > 1 (torchrun) every rank owns its own column shard of the same shape (weak scaling): the
path is independent per column, so there is no data-path collective; ranks only meet in the
barrier and the max-over-ranks of the device time.
"""
import argparse
import json
import os
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused NB-SGD step throughput (params*learners/s)"
UNIT = "params*learners/s"
DEFAULT_WORKLOAD = "cfg3_dpsgd_ring_resnet50"
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes per algorithmic byte of one step, per workloads-table entry (and for the headline: the
# entry of the same name): dram__bytes_read.sum + dram__bytes_write.sum of all kernels of a step
# over the algorithmic bytes of that step, from ncu captures of a narrower column range of the same
# workload (profiles/dram_traffic_per_workload_and_entry.md; traffic grows in proportion to the
# columns).  No entry: no capture exists and `traffic` is reported as null.
TRAFFIC_PER_ALGORITHMIC_BYTE = {
    "cfg3_dpsgd_ring_resnet50": 0.988,
    "cfg3_dpsgd_ring_resnet50[P+1, rows not 16-byte aligned]": 0.989,
    "cfg3_dpsgd_ring_resnet50[update_then_mix]": 0.987,
    "cfg3_dpsgd_ring_resnet50[unfused]": 1.283,
    "cfg3_dpsgd_ring_resnet50[streaming_hold]": 0.988,
    "cfg3_dpsgd_ring_resnet50[centralized]": 0.996,
    "cfg2_allreduce_resnet18": 0.990,
    "cfg4_matcha_vgg16": 0.980,
    "cfg5_scale_allreduce": 0.990,
    "cfg5_scale_ring": 0.990,
    "ring_K64_P12.8M": 0.987,
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default="", choices=["", "allreduce", "dpsgd", "centralized"],
                    help="run the workload's sizes with another variant (dpsgd = ring)")
    ap.add_argument("--order", default="mix_then_update", choices=["mix_then_update", "update_then_mix"])
    ap.add_argument("--entry", default="fused", choices=["fused", "unfused", "streaming", "streaming_hold"],
                    help="fused: nb_step_fused; unfused: nb_accumulate + nb_step; streaming: one "
                         "nb_accumulate_minibatch per finished mini-batch, then nb_step")
    ap.add_argument("--unfused", action="store_true", help="same as --entry unfused")
    ap.add_argument("--kernel", default="auto", choices=["auto", "direct"],
                    help="direct: the direct-load kernels only (NB_OPT_KERNEL), for comparison with the bulk-copy pipeline")
    ap.add_argument("--cols", type=int, default=0, help="profiling aid: run the workload on this many columns instead of its P")
    ap.add_argument("--learners", type=int, default=0, help="profiling aid: run the workload with this many learners instead of its K")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the table of other workloads / entries")
    ap.add_argument("--no-sustained", action="store_true", help="skip the >= 2 s repetition of the headline step")
    ap.add_argument("--workload-steps", type=int, default=20, help="timed steps of every `workloads` entry")
    ap.add_argument("--sustained-seconds", type=float, default=2.5)
    ap.add_argument("--coverage-map", action="store_true",
                    help="instead of the benchmark: the fused step over a grid of K, M, dtype, variant and order")
    ap.add_argument("--cpu-sample-cols", type=int, default=4_000_000)
    ap.add_argument("--cpu-sample-steps", type=int, default=8)
    a = ap.parse_args()
    if a.unfused:
        a.entry = "unfused"
    return a


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def host_threads():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


ENTRY_NAMES = {"fused": "nb_step_fused", "unfused": "nb_accumulate+nb_step",
               "streaming": "nb_accumulate_minibatch x sum(n_i) + nb_step",
               "streaming_hold": "nb_accumulate_minibatch x sum(n_i) [NB_STREAMING_HOLD] + nb_step"}


def config_of(w, order, entry, world):
    """Description of the timed workload; the same keys and values in both arms."""
    es = 4 if w.grad_dtype == "f32" else 2
    return {"workload": w.name, "K": w.K, "P": w.P, "M": w.M, "grad_dtype": w.grad_dtype, "variant": w.variant,
            "topology": w.topology, "order": order, "entry": ENTRY_NAMES[entry],
            "parallelism": "column-shard x%d" % world,
            "l2": "inputs larger than L2 (%.1f GB gradient stream + %.1f GB state per step; no flush needed)"
                  % (w.K * w.M * w.P * es / 1e9, 2 * w.K * w.P * 4 / 1e9)}


# ---------------------------------------------------------------------------------------------
# clocks: sampled through NVML while a timed region runs (read-only)
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, index, period=0.01):
        self.index, self.samples, self.times, self.reasons, self.max_mhz = index, [], [], set(), None
        self.period = period
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

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                self.times.append(time.perf_counter())
                self.samples.append(mhz)
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr:
            self._stop.set()
            self._thr.join()
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ---------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline legs and --impl reference)
# ---------------------------------------------------------------------------------------------
def _oracle_worker(job):
    """Runs in a worker process (or inline): times oracle.step on columns [0, cols) of a workload
    whose seed is offset per worker.  Returns the seconds of the timed steps, one per step."""
    (wdict, cols, steps, warmup, worker) = job
    for k in ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS"):
        os.environ[k] = "1"
    import numpy as np
    from oracle import nb_oracle as O
    from paper_2211_00889_b200 import workloads as WL
    w = WL.Workload(**wdict)
    ws = replace(WL.scaled(w, cols), seed=w.seed + 7919 * worker)
    central = w.variant == "centralized"
    if w.variant in ("allreduce", "centralized"):
        orc = O.Oracle(ws.K, ws.P, ws.M, ws.lr, ws.mom, "allreduce")
    elif w.variant == "dpsgd":
        orc = O.Oracle(ws.K, ws.P, ws.M, ws.lr, ws.mom, "dpsgd", W=O.ring_W(ws.K))
    else:
        partner = O.greedy_matchings(O.random_regular_graph(w.seed, ws.K, ws.degree)[0], ws.K)
        orc = O.Oracle(ws.K, ws.P, ws.M, ws.lr, ws.mom, "matcha", partner=partner, alpha=ws.alpha,
                       prob=ws.act_prob, seed=w.seed)
    x0 = WL.init_params(ws)
    orc.set_params(x0)
    x_ps, v_ps = x0.astype(np.float64), np.zeros(ws.P)
    G = WL.gradients_np(ws, 0)[1]                      # one block, reused (drawing it is not timed)
    out = []
    for t in range(warmup + steps):
        n = O.straggler_counts(w.straggler_model, w.seed, t, ws.K, ws.M, ws.straggler_params)
        t0 = time.perf_counter()
        if central:
            x_ps, v_ps = O.step_centralized(x_ps, v_ps, G, n, ws.lr, ws.mom)
        else:
            orc.step(G, n)
        dt = time.perf_counter() - t0
        if t >= warmup:
            out.append((t0, t0 + dt))
    return out


def time_oracle(w, sample_cols, steps, warmup=0, procs=1):
    """Times oracle.step on a column slice of workload w (exact: columns are independent), the
    columns split evenly over `procs` worker processes, each running the oracle untouched on one
    thread.  Returns (params*learners/s, seconds per step, description)."""
    from dataclasses import asdict
    cols = min(sample_cols, w.P)
    per = max(1, cols // procs)
    jobs = [(asdict(w), per, steps, warmup, r) for r in range(procs)]
    if procs == 1:
        spans = [_oracle_worker(jobs[0])]
    else:
        import multiprocessing as mp
        with mp.get_context("spawn").Pool(procs) as pool:
            spans = pool.map(_oracle_worker, jobs)
    # Workers run concurrently but not in lock step: the sample's duration is the busiest worker's
    # total over its timed steps (every worker does the same number of steps on the same width).
    total = max(sum(b - a for a, b in s) for s in spans)
    per_step = total / steps
    desc = ("oracle.step (NumPy fp64) on a %d-column slice of %s, %d steps, %d worker process%s of one thread each"
            % (per * procs, w.name, steps, procs, "" if procs == 1 else "es (%d columns each)" % per))
    return w.K * per * procs / per_step, per_step, desc


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = host_threads()
    # a bounded sample per step: 125k columns per core keeps 25 steps within about a minute
    cols = min(w.P, 125_000 * cores)
    value, per_step, desc = time_oracle(w, cols, args.steps, args.warmup, procs=cores)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, args.order, args.entry, max(1, args.gpus)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------
class Runner:
    """One workload resident on the device: context, gradient buffers, and the timed loop."""

    def __init__(self, B, WL, w, dev, order="mix_then_update", seed_offset=0, bufs=None, row_shift=0, pitch=0,
                 kernel="auto"):
        import torch
        self.B, self.WL, self.w, self.dev, self.torch = B, WL, w, dev, torch
        self.es = 4 if w.grad_dtype == "f32" else 2
        g_bytes = w.K * w.M * w.P * self.es
        wr = replace(w, seed=w.seed + seed_offset)
        if bufs is None:
            free, _ = torch.cuda.mem_get_info()
            n_buf = 2 if free > 2 * g_bytes + 3 * w.K * w.P * 4 + (8 << 30) else 1
            bufs = [WL.gradients_torch(wr, b, dev) for b in range(n_buf)]
            if pitch:          # rows `pitch` elements apart (a view of a wider buffer; the binding passes its strides)
                wide = []
                for b in bufs:
                    t = torch.empty((w.K, w.M, pitch), dtype=b.dtype, device=dev)
                    t[:, :, :w.P].copy_(b)
                    wide.append(t[:, :, :w.P])
                bufs = wide
            if row_shift:      # the same stream `row_shift` elements off its allocation's 16-byte boundary
                shifted = []
                for b in bufs:
                    flat = torch.empty(b.numel() + row_shift, dtype=b.dtype, device=dev)
                    v = flat[row_shift:].view_as(b)
                    v.copy_(b)
                    shifted.append(v)
                bufs = shifted
        self.bufs = bufs
        gen = torch.Generator(device=dev)
        gen.manual_seed(wr.seed)
        x0 = torch.randn(w.P, generator=gen, device=dev, dtype=torch.float32) * w.init_sigma
        self.ctx = B.context_for(w)
        self.ctx.set_params(x0)
        if order == "update_then_mix":
            self.ctx.set_option(B.NB_OPT_ORDER, B.NB_ORDER_UPDATE_THEN_MIX)
        if kernel == "direct":
            self.ctx.set_option(B.NB_OPT_KERNEL, B.NB_KERNEL_DIRECT)
        self.order = order

    def counts(self, t):
        w = self.w
        return self.B.straggler_sample(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)[0]

    def one_step(self, entry, g, n):
        ctx = self.ctx
        if entry == "fused":
            ctx.step_fused(g, n)
        elif entry == "unfused":
            ctx.accumulate(g, n)
            ctx.step()
        else:
            # Alg. 1 inner loop as the gradients arrive: round m delivers mini-batch m of every learner
            # that finished it; the fastest learner's M-th delivery raises the terminal signal last
            if entry == "streaming_hold" and not getattr(self, "_hold_set", False):
                ctx.set_option(self.B.NB_OPT_STREAMING, self.B.NB_STREAMING_HOLD)
                self._hold_set = True
            ctx.begin_iteration()
            for m in range(self.w.M):
                for i in range(self.w.K):
                    if m < n[i]:
                        ctx.accumulate_minibatch(i, g[i, m])
            ctx.step()

    def own_bytes(self, entry, n):
        """Bytes the entry point itself must move in one step (its accumulator round trips included)."""
        w, es = self.w, self.es
        rows = 1 if w.variant == "centralized" else w.K
        alg = w.P * (es * int(n.sum()) + 16 * rows)
        if entry == "unfused":
            return alg + 8 * w.K * w.P                                   # acc written once, read once
        if entry == "streaming":                                           # acc read-modify-write per delivery
            rmw = sum((2 * int(k) - 1) * 4 for k in n if k > 0) + 4 * w.K  # + the step's read of acc
            return alg + w.P * rmw
        return alg

    def timed(self, entry, steps, warmup, t_first=0, sampler=None, barrier=None, per_step_events=True):
        torch = self.torch
        ctx, bufs = self.ctx, self.bufs
        nb = len(bufs)
        for t in range(t_first, t_first + warmup):
            self.one_step(entry, bufs[t % nb], self.counts(t))
        if barrier:
            barrier()
        else:
            torch.cuda.synchronize()
        launches0 = ctx.get_stats()["kernel_launches"]
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        alg, own, sum_n = [], 0.0, 0
        if sampler:
            sampler.start()
        host_t0 = time.perf_counter()
        e0.record()
        for s in range(steps):
            t = t_first + warmup + s
            n = self.counts(t)                 # S0: host straggler simulator, inside the timed step
            ev[s][0].record()
            self.one_step(entry, bufs[t % nb], n)
            ev[s][1].record()
            st = ctx.get_stats()
            alg.append(st["algorithmic_bytes"])
            sum_n += st["sum_finished"]
            own += self.own_bytes(entry, n)
        e1.record()
        if barrier:
            barrier()
        else:
            torch.cuda.synchronize()
        clocks = sampler.stop() if sampler else None
        total_ms = e0.elapsed_time(e1)
        step_ms = [a.elapsed_time(b) for a, b in ev]
        launch_ms = sum(step_ms) / steps
        return {"total_ms": total_ms, "launch_ms": launch_ms, "step_ms": step_ms, "alg_bytes": alg,
                "own_bytes_per_step": own / steps, "mean_sum_finished": sum_n / steps,
                "launches": ctx.get_stats()["kernel_launches"] - launches0, "clocks": clocks,
                "kernel_plan": ctx.get_kernel_plan(), "host_t0": host_t0,
                "step_start_ms": [e0.elapsed_time(a) for a, _ in ev]}

    def close(self):
        self.ctx.close()
        self.bufs = None


def table_entry(label, w, order, entry, r, peak, steps, note=None):
    alg = sum(r["alg_bytes"]) / len(r["alg_bytes"])
    ms = r["total_ms"] / steps
    achieved = alg / (r["launch_ms"] * 1e-3) / 1e9
    moved = r["own_bytes_per_step"] / (r["launch_ms"] * 1e-3) / 1e9
    tr = TRAFFIC_PER_ALGORITHMIC_BYTE.get(label)
    out = {"name": label, "K": w.K, "P": w.P, "M": w.M, "grad_dtype": w.grad_dtype, "variant": w.variant,
           "topology": w.topology, "order": order, "entry": ENTRY_NAMES[entry], "steps": steps,
           "ms_per_step": ms, "step_ms_device": r["launch_ms"], "value": w.K * w.P / (ms * 1e-3), "unit": UNIT,
           "algorithmic_bytes_per_step": alg, "achieved_hbm_gbs": achieved, "frac": achieved / peak,
           "entry_bytes_per_step": r["own_bytes_per_step"], "entry_moved_gbs": moved, "entry_moved_frac": moved / peak,
           "traffic": tr * alg if tr else None, "mean_sum_finished": r["mean_sum_finished"],
           "gpu_launches_per_step": r["launches"] / steps, "kernel_plan": r["kernel_plan"], "clocks": r["clocks"]}
    if note:
        out["note"] = note
    return out


def sustained_leg(runner, seconds, est_ms, t_first, local):
    """The headline step repeated back to back for at least `seconds`; GB/s against the SM clock
    sampled meanwhile (a 1 kW part settles below its maximum clock under sw_power_cap)."""
    steps = max(50, int(seconds * 1e3 / est_ms) + 1)
    sampler = ClockSampler(local, period=0.02)
    r = runner.timed("fused", steps, 3, t_first=t_first, sampler=sampler)
    alg = r["alg_bytes"]
    gbs = [a / (ms * 1e-3) / 1e9 for a, ms in zip(alg, r["step_ms"])]
    total_alg = sum(alg)
    ms_per_step = r["total_ms"] / steps
    # clock of every step: the sample nearest to the step's start (device time since the region's
    # first event, laid over the host clock at that event's record call)
    times = [(t - r["host_t0"]) * 1e3 for t in sampler.times]
    bins = {}
    j = 0
    for s, start in enumerate(r["step_start_ms"]):
        while j + 1 < len(times) and abs(times[j + 1] - start) <= abs(times[j] - start):
            j += 1
        if times:
            b = int(sampler.samples[j] // 100 * 100)
            bins.setdefault(b, []).append(gbs[s])
    med = lambda v: sorted(v)[len(v) // 2]
    c = r["clocks"] or {}
    return {"steps": steps, "seconds": r["total_ms"] * 1e-3, "ms_per_step": ms_per_step,
            "achieved": total_alg / (sum(r["step_ms"]) * 1e-3) / 1e9, "unit": "GB/s",
            "sm_mhz_median": c.get("sm_mhz"), "sm_max_mhz": c.get("sm_max_mhz"), "reasons": c.get("reasons"),
            "clock_samples": c.get("samples"),
            "ms_x_sm_mhz": (ms_per_step * c["sm_mhz"]) if c.get("sm_mhz") else None,
            "gbs_by_sm_mhz_bin": {"%d-%d" % (b, b + 99): {"steps": len(v), "median_gbs": med(v)}
                                  for b, v in sorted(bins.items())}}


def other_workloads(args, B, WL, dev, base_runner, peak, local, log):
    """One short run each of the other configurations, variants and entry points (N = 1)."""
    import torch
    out = []
    steps, warm = args.workload_steps, 3
    w3 = base_runner.w

    def run(label, w, order="mix_then_update", entry="fused", bufs=None, row_shift=0, note=None):
        t0 = time.time()
        try:
            r = Runner(B, WL, w, dev, order=order, bufs=bufs, row_shift=row_shift)
            res = r.timed(entry, steps, warm, sampler=ClockSampler(local))
            out.append(table_entry(label, w, order, entry, res, peak, steps, note))
            r.close()
            del r
        except Exception as e:                      # a workload that cannot run is reported, not hidden
            out.append({"name": label, "error": "%s: %s" % (type(e).__name__, e)})
        torch.cuda.empty_cache()
        log("%s: %.1f s" % (label, time.time() - t0))

    # variants and entry points on the headline workload's own sizes and gradient buffers
    shared = base_runner.bufs
    run(w3.name + "[centralized]", replace(w3, variant="centralized", topology="full", name=w3.name + "[centralized]"),
        bufs=shared, note="Alg. 3: one shared model, algorithmic bytes P*(e_g*sum n_i + 16)")
    run(w3.name + "[update_then_mix]", w3, order="update_then_mix", bufs=shared, note="Eq. 4-6 order")
    run(w3.name + "[unfused]", w3, entry="unfused", bufs=shared,
        note="nb_accumulate + nb_step: the accumulator round trip (8*K*P bytes) is moved but not algorithmic")
    run(w3.name + "[streaming]", w3, entry="streaming", bufs=shared,
        note="Alg. 1 inner loop as the gradients arrive: one launch per finished mini-batch, accumulator "
             "read-modify-write per delivery")
    run(w3.name + "[streaming_hold]", w3, entry="streaming_hold", bufs=shared,
        note="the same deliveries only recorded (NB_STREAMING_HOLD): nb_step runs the fused step on the delivered "
             "vectors where they lie, one bulk copy per row from a table of row pointers")
    out.append(mean_model_entry(base_runner, peak, steps, local))
    return out, shared


def mean_model_entry(runner, peak, steps, local):
    """S7, the output step: nb_get_mean_params into a device buffer (K model rows read, one written)."""
    torch, w, ctx = runner.torch, runner.w, runner.ctx
    for _ in range(3):
        ctx.get_mean_params(device=runner.dev)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    e0.record()
    for _ in range(steps):
        ctx.get_mean_params(device=runner.dev)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / steps
    alg = 4.0 * w.P * (w.K + 1)
    gbs = alg / (ms * 1e-3) / 1e9
    return {"name": w.name + "[mean model]", "entry": "nb_get_mean_params", "steps": steps, "ms_per_step": ms,
            "algorithmic_bytes_per_step": alg, "achieved_hbm_gbs": gbs, "frac": gbs / peak, "entry_moved_gbs": gbs,
            "entry_moved_frac": gbs / peak, "traffic": None, "gpu_launches_per_step": 1.0, "kernel_plan": None,
            "clocks": clocks,
            "note": "Alg. 1 / Alg. 2 output: mean of the K learners' models, 4*P*(K+1) bytes"}


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    from paper_2211_00889_b200 import workloads as WL

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; this path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2211_00889_b200 import sharding

    def barrier():
        sharding.barrier()
        torch.cuda.synchronize()

    def log(msg):
        if rank == 0:
            print("[bench] " + msg, file=sys.stderr, flush=True)

    # rank r owns columns [r*P, (r+1)*P) of an N*P-wide problem: same counts everywhere, own data
    runner = Runner(B, WL, w, dev, order=args.order, seed_offset=1000 * rank, kernel=args.kernel)
    es = runner.es
    if world > 1:   # every rank derives the counts by itself; they must coincide (checked outside the timed region)
        assert sharding.counts_agree(runner.counts(args.warmup), dev), "ranks disagree on the finished counts"
    r = runner.timed(args.entry, args.steps, args.warmup, sampler=ClockSampler(local), barrier=barrier)
    total_ms_max = sharding.max_over_ranks(r["total_ms"], dev)
    ms_per_step = total_ms_max / args.steps
    value = w.K * w.P * world / (ms_per_step * 1e-3)
    clocks, launches = r["clocks"], r["launches"]

    peak, peak_kind = measured_peak()
    bytes_per_launch = sum(r["alg_bytes"]) / args.steps
    achieved = bytes_per_launch / (r["launch_ms"] * 1e-3) / 1e9
    head_label = w.name
    if args.kernel != "auto" or args.cols or args.learners:
        head_label = None                                  # not a captured configuration
    elif args.variant:
        head_label = None if args.variant != "centralized" or args.entry != "fused" else w.name
    elif args.entry != "fused":
        head_label = "%s[%s]" % (w.name, args.entry)
    elif args.order != "mix_then_update":
        head_label = "%s[%s]" % (w.name, args.order)
    tr = TRAFFIC_PER_ALGORITHMIC_BYTE.get(head_label)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": tr * bytes_per_launch if tr else None,
                "peak_source": "of " + peak_kind,
                "kernel": ("nb_step_kernel (direct loads; fused accumulate+mix+momentum+update)" if args.kernel == "direct"
                           else "nb_step_pipeline_kernel (fused accumulate+mix+momentum+update)") if args.entry == "fused"
                          else ENTRY_NAMES[args.entry],
                "algorithmic_bytes_per_launch": bytes_per_launch, "launch_ms": r["launch_ms"],
                "frac_of_8TBps_nominal": achieved / 8000.0, "mean_sum_finished": r["mean_sum_finished"],
                "kernel_plan": r["kernel_plan"], "timed": "burst: the %d timed steps" % args.steps}
    t_next = args.warmup + args.steps
    single = rank == 0 and world == 1

    workloads = None
    if single and not args.no_workloads:
        workloads, _ = other_workloads(args, B, WL, dev, runner, peak, local, log)

    # ---- end to end: host gradient buffers through nb_step_fused_host -------------------------
    e2e = None
    if not args.no_e2e:
        ctx, bufs = runner.ctx, runner.bufs
        host = torch.empty((w.K, w.M, w.P), dtype=bufs[0].dtype, pin_memory=True)
        host.copy_(bufs[0])
        mean_out = torch.empty(w.P, dtype=torch.float32, pin_memory=True)
        torch.cuda.synchronize()
        t_e2e = 1_000_000
        ctx.step_fused_host(host, runner.counts(t_e2e), mean_out=mean_out)   # warm-up: allocates staging
        barrier()
        h2d = 0
        t0 = time.perf_counter()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for s in range(args.e2e_steps):
            n = runner.counts(t_e2e + 1 + s)
            ctx.step_fused_host(host, n, mean_out=mean_out)
            h2d += int(n.sum()) * w.P * es
        a1.record()
        barrier()
        wall = time.perf_counter() - t0
        dev_ms = a0.elapsed_time(a1)
        per = sharding.max_over_ranks(max(dev_ms, wall * 1e3), dev) / args.e2e_steps
        # the bus roof beside it: one plain pinned host-to-device copy of 1 GiB, timed the same way
        n_el = min(host.numel(), (1 << 30) // es)
        dst = torch.empty(n_el, dtype=host.dtype, device=dev)
        src = host.view(-1)[:n_el]
        dst.copy_(src, non_blocking=True)
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record()
        for _ in range(3):
            dst.copy_(src, non_blocking=True)
        b1.record()
        torch.cuda.synchronize()
        pcie = 3 * n_el * es / (b0.elapsed_time(b1) * 1e-3) / 1e9
        del dst, src
        h2d_step = h2d // args.e2e_steps
        e2e = {"value": w.K * w.P * world / (per * 1e-3), "unit": UNIT, "ms_per_step": per,
               "steps": args.e2e_steps, "h2d_bytes_per_step": h2d_step,
               "d2h_bytes_per_step": w.P * 4,
               "h2d_gbs": h2d_step / (per * 1e-3) / 1e9, "plain_pinned_h2d_copy_gbs": pcie,
               "bound": "host-to-device bus: only the finished rows cross it, overlapped with the kernels and the "
                        "device-to-host copy of the mean model",
               "api": "nb_step_fused_host (pinned host gradients in, mean model out)"}
        del host, mean_out
        log("e2e done")
    torch.cuda.empty_cache()

    if workloads is not None:
        workloads += larger_workloads(args, B, WL, dev, w, peak, local, log)

    # last of the device work, so that the seconds under the power cap do not colour the short runs above
    if single and not args.no_sustained and args.entry == "fused":
        roofline["sustained"] = sustained_leg(runner, args.sustained_seconds, r["launch_ms"], t_next, local)
        roofline["sustained"]["frac"] = roofline["sustained"]["achieved"] / peak
        log("sustained leg done")

    runner.close()
    del runner
    torch.cuda.empty_cache()

    cpu = None
    if single and not args.no_cpu_baseline:
        cores = host_threads()
        v1, _, d1 = time_oracle(w, args.cpu_sample_cols, args.cpu_sample_steps, procs=1)
        log("cpu baseline, one core, done")
        vn, _, dn = time_oracle(w, args.cpu_sample_cols, args.cpu_sample_steps, procs=cores)
        cpu = {"value": vn, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": dn,
               "one_core": {"value": v1, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": d1},
               "host_cores_available": cores}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_of(w, args.order, args.entry, world),
            "achieved_hbm_gbs": achieved, "frac_of_8TBps": achieved / 8000.0,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
            "workloads": workloads,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def larger_workloads(args, B, WL, dev, w_head, peak, local, log):
    """The configurations that need their own gradient streams, run after the headline's memory is free."""
    import torch
    out = []
    steps, warm = args.workload_steps, 3

    def run(label, w, order="mix_then_update", entry="fused", bufs=None, row_shift=0, note=None, keep=False, pitch=0):
        t0 = time.time()
        r = None
        try:
            r = Runner(B, WL, w, dev, order=order, bufs=bufs, row_shift=row_shift, pitch=pitch)
            res = r.timed(entry, steps, warm, sampler=ClockSampler(local))
            out.append(table_entry(label, w, order, entry, res, peak, steps, note))
        except Exception as e:
            out.append({"name": label, "error": "%s: %s" % (type(e).__name__, e)})
        kept = r.bufs if (r is not None and keep) else None
        if r is not None:
            r.close()
        del r
        torch.cuda.empty_cache()
        log("%s: %.1f s" % (label, time.time() - t0))
        return kept

    W = WL.WORKLOADS
    # the headline workload with one more column: every gradient row starts at a different byte
    # offset, none on a 16-byte boundary (per-row bulk copies instead of tensor-map boxes)
    odd = replace(w_head, P=w_head.P + 1, name=w_head.name + "[P+1, rows not 16-byte aligned]")
    run(odd.name, odd, note="dense odd row length: per-row bulk copies of the 16-byte aligned superset")
    for name in ("cfg2_allreduce_resnet18", "cfg4_matcha_vgg16"):
        if name != w_head.name:
            run(name, W[name])
    w4 = W["cfg4_matcha_vgg16"]
    if w4.name != w_head.name:
        import torch as _t
        pitch = B.recommended_pitch(w4.P, _t.bfloat16 if w4.grad_dtype == "bf16" else _t.float32)
        if pitch != w4.P:
            run(w4.name + "[rows at nb_recommended_pitch]", w4, pitch=pitch,
                note="same values, gradient rows %d elements apart instead of dense: every tile segment inside "
                     "one 2 KB block of device memory" % pitch)
    w5 = W["cfg5_scale_allreduce"]
    kept = run(w5.name, w5, keep=True)
    run("cfg5_scale_ring", W["cfg5_scale_ring"], bufs=kept)
    del kept
    torch.cuda.empty_cache()
    k64 = replace(W["cfg3_dpsgd_ring_resnet50"], K=64, P=12_800_000, name="ring_K64_P12.8M")
    run(k64.name, k64, note="the largest learner count the library takes (NB_MAX_K)")
    return out


def coverage_map(args):
    """`--coverage-map`: the fused step over a grid of K, M, gradient dtype, variant and order (10 timed
    steps each, sizes of 5-8 GB), as fractions of the measured copy bandwidth; one JSON line.  Shows
    where the planner's shapes hold and where they do not (profiles/planner_coverage_map.md)."""
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    from paper_2211_00889_b200 import workloads as WL
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak()
    base = WL.WORKLOADS[DEFAULT_WORKLOAD]
    cells = []
    for variant, topology in (("dpsgd", "ring"), ("allreduce", "full"), ("centralized", "full")):
        for order in ("mix_then_update", "update_then_mix"):
            if variant == "centralized" and order != "mix_then_update":
                continue
            for dtype in ("bf16", "f32"):
                es = 2 if dtype == "bf16" else 4
                for K in (1, 2, 4, 8, 16, 32, 64):
                    for M in (1, 2, 4, 8, 16):
                        P = int(min(base.P, 5e9 / (K * M * es), 8e9 / (K * 16)))
                        P -= P % 512
                        w = replace(base, K=K, M=M, P=P, grad_dtype=dtype, variant=variant, topology=topology,
                                    name="K%d_M%d" % (K, M))
                        r = Runner(B, WL, w, dev, order=order)
                        res = r.timed("fused", 10, 3, sampler=ClockSampler(0))
                        gbs = sum(res["alg_bytes"]) / 10 / (res["launch_ms"] * 1e-3) / 1e9
                        cells.append({"variant": variant, "topology": topology, "order": order, "grad_dtype": dtype,
                                      "K": K, "M": M, "P": P, "ms_per_step": res["launch_ms"], "achieved_hbm_gbs": gbs,
                                      "frac": gbs / peak, "kernel_plan": res["kernel_plan"]})
                        r.close()
                        del r
                        torch.cuda.empty_cache()
    print(json.dumps({"coverage_map": cells, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s"}))


def main():
    args = parse_args()
    from paper_2211_00889_b200 import workloads as WL
    if args.coverage_map:
        return coverage_map(args)
    w = WL.WORKLOADS[args.workload]
    if args.cols:
        w = replace(WL.scaled(w, args.cols), name="%s[P=%d]" % (w.name, args.cols))
    if args.learners:
        w = replace(w, K=args.learners, name="%s[K=%d]" % (w.name, args.learners))
    if args.variant:
        topo = {"allreduce": "full", "dpsgd": "ring", "centralized": "full"}[args.variant]
        w = replace(w, variant=args.variant, topology=topo, name="%s[%s]" % (w.name, args.variant))
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
