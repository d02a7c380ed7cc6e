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
            the measured HBM copy bandwidth of this machine's B200s
  cpu_baseline  the CPU oracle, as it stands, timed on a bounded column slice of the same workload

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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused NB-SGD step throughput (params*learners/s)"
UNIT = "params*learners/s"
DEFAULT_WORKLOAD = "cfg3_dpsgd_ring_resnet50"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per algorithmic byte of the fused step kernel: dram__bytes_read.sum + dram__bytes_write.sum
# of nb_step_pipeline_kernel over the algorithmic bytes of the same launch, from the ncu capture of an
# 8M-column case of the default workload (summarised under profiles/).
# Traffic grows in proportion to the columns a launch processes.
TRAFFIC_PER_ALGORITHMIC_BYTE = 0.988


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
    ap.add_argument("--unfused", action="store_true", help="time nb_accumulate + nb_step instead of nb_step_fused")
    ap.add_argument("--grad-pad", type=int, default=0, help="experiment: extra elements of row pitch in the gradient buffers")
    ap.add_argument("--cols", type=int, default=0, help="profiling aid: run the workload on this many columns instead of its P")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample-cols", type=int, default=2_000_000)
    ap.add_argument("--cpu-sample-steps", type=int, default=10)
    return ap.parse_args()


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


# ---------------------------------------------------------------------------------------------
# clocks: sampled through NVML while the timed region runs (read-only)
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, index):
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
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
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.01)

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
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------
def time_oracle(w, sample_cols, steps, warmup=0):
    """Times oracle.step on a column slice of workload w (exact: columns are independent).
    Returns (params*learners/s, seconds per step, description)."""
    import numpy as np
    from oracle import nb_oracle as O
    from paper_2211_00889_b200 import workloads as WL
    ws = WL.scaled(w, min(sample_cols, w.P))
    central = w.variant == "centralized"
    if w.variant in ("allreduce", "centralized"):
        orc = O.Oracle(ws.K, ws.P, ws.M, ws.lr, ws.mom, "allreduce")
    elif w.variant == "dpsgd":
        orc = O.Oracle(ws.K, ws.P, ws.M, ws.lr, ws.mom, "dpsgd", W=O.ring_W(ws.K))
    else:
        partner = O.greedy_matchings(O.random_regular_graph(ws.seed, ws.K, ws.degree)[0], ws.K)
        orc = O.Oracle(ws.K, ws.P, ws.M, ws.lr, ws.mom, "matcha", partner=partner, alpha=ws.alpha,
                       prob=ws.act_prob, seed=ws.seed)
    x0 = WL.init_params(ws)
    orc.set_params(x0)
    x_ps, v_ps = x0.astype(np.float64), np.zeros(ws.P)
    G = WL.gradients_torch(ws, 0, "cpu").float().numpy()     # one block, reused (not timed)
    total = 0.0
    for t in range(warmup + steps):
        n = O.straggler_counts(ws.straggler_model, ws.seed, t, ws.K, ws.M, ws.straggler_params)
        t0 = time.perf_counter()
        if central:
            x_ps, v_ps = O.step_centralized(x_ps, v_ps, G, n, ws.lr, ws.mom)
        else:
            orc.step(G, n)
        dt = time.perf_counter() - t0
        if t >= warmup:
            total += dt
    per_step = total / steps
    desc = "oracle.step (NumPy fp64, 1 thread) on a %d-column slice of %s, %d steps" % (ws.P, w.name, steps)
    return ws.K * ws.P / per_step, per_step, desc


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cols = max(1, args.cpu_sample_cols // 4)
    value, per_step, desc = time_oracle(w, cols, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "K": w.K, "P": w.P, "M": w.M, "grad_dtype": w.grad_dtype,
                   "variant": w.variant, "topology": w.topology},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------
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

    # rank r owns columns [r*P, (r+1)*P) of an N*P-wide problem: same counts everywhere, own data
    wr = WL.scaled(w, w.P)
    from dataclasses import replace
    wr = replace(wr, seed=w.seed + 1000 * rank)
    es = 4 if w.grad_dtype == "f32" else 2
    g_bytes = w.K * w.M * w.P * es
    free, _ = torch.cuda.mem_get_info()
    n_buf = 2 if free > 2 * g_bytes + 4 * w.K * w.P * 4 + (8 << 30) else 1
    bufs = [WL.gradients_torch(wr, b, dev) for b in range(n_buf)]
    ld = {}
    if args.grad_pad:
        wide = [torch.empty((w.K, w.M, w.P + args.grad_pad), dtype=b.dtype, device=dev) for b in bufs]
        for dst, src in zip(wide, bufs):
            dst[:, :, :w.P].copy_(src)
        bufs = [b[:, :, :w.P] for b in wide]
        ld = dict(ld_m=w.P + args.grad_pad, ld_k=w.M * (w.P + args.grad_pad))
    gen = torch.Generator(device=dev)
    gen.manual_seed(wr.seed)
    x0 = torch.randn(w.P, generator=gen, device=dev, dtype=torch.float32) * w.init_sigma
    ctx = B.context_for(w)
    ctx.set_params(x0)
    if args.order == "update_then_mix":
        ctx.set_option(B.NB_OPT_ORDER, B.NB_ORDER_UPDATE_THEN_MIX)

    def one_step(g, n):
        if args.unfused:
            ctx.accumulate(g, n, **ld)
            ctx.step()
        else:
            ctx.step_fused(g, n, **ld)

    def counts(t):
        return B.straggler_sample(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)[0]

    total_steps = args.warmup + args.steps
    for t in range(args.warmup):
        one_step(bufs[t % n_buf], counts(t))
    if world > 1:   # every rank derives the counts by itself; they must coincide (checked outside the timed region)
        assert sharding.counts_agree(counts(args.warmup), dev), "ranks disagree on the finished counts"
    barrier()
    launches0 = ctx.get_stats()["kernel_launches"]
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    alg_bytes = 0.0
    sum_n = 0
    sampler.start()
    e0.record()
    for s in range(args.steps):
        t = args.warmup + s
        n = counts(t)                      # S0: host straggler simulator, inside the timed step
        ev[s][0].record()
        one_step(bufs[t % n_buf], n)
        ev[s][1].record()
        st = ctx.get_stats()
        alg_bytes += st["algorithmic_bytes"]
        sum_n += st["sum_finished"]
    e1.record()
    barrier()
    clocks = sampler.stop()
    kernel_plan = ctx.get_kernel_plan()
    launches = ctx.get_stats()["kernel_launches"] - launches0
    total_ms = e0.elapsed_time(e1)
    launch_ms = sum(a.elapsed_time(b) for a, b in ev) / args.steps
    total_ms_max = sharding.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms_max / args.steps
    value = w.K * w.P * world / (ms_per_step * 1e-3)

    peak, peak_kind = measured_peak()
    bytes_per_launch = alg_bytes / args.steps
    achieved = bytes_per_launch / (launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": (TRAFFIC_PER_ALGORITHMIC_BYTE * bytes_per_launch) if TRAFFIC_PER_ALGORITHMIC_BYTE else None,
                "peak_source": "of " + peak_kind, "kernel": "nb_step_pipeline_kernel (fused accumulate+mix+momentum+update)",
                "algorithmic_bytes_per_launch": bytes_per_launch, "launch_ms": launch_ms,
                "frac_of_8TBps_nominal": achieved / 8000.0, "mean_sum_finished": sum_n / args.steps,
                "kernel_plan": kernel_plan}

    # ---- end to end: host gradient buffers through nb_step_fused_host -------------------------
    e2e = None
    if not args.no_e2e:
        host = torch.empty((w.K, w.M, w.P), dtype=bufs[0].dtype, pin_memory=True)
        host.copy_(bufs[0])
        mean_out = torch.empty(w.P, dtype=torch.float32, pin_memory=True)
        torch.cuda.synchronize()
        ctx.step_fused_host(host, counts(total_steps), mean_out=mean_out)   # warm-up: allocates staging
        barrier()
        h2d = 0
        t0 = time.perf_counter()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for s in range(args.e2e_steps):
            n = counts(total_steps + 1 + s)
            ctx.step_fused_host(host, n, mean_out=mean_out)
            h2d += int(n.sum()) * w.P * es
        a1.record()
        barrier()
        wall = time.perf_counter() - t0
        dev_ms = a0.elapsed_time(a1)
        per = sharding.max_over_ranks(max(dev_ms, wall * 1e3), dev) / args.e2e_steps
        e2e = {"value": w.K * w.P * world / (per * 1e-3), "unit": UNIT, "ms_per_step": per,
               "steps": args.e2e_steps, "h2d_bytes_per_step": h2d // args.e2e_steps,
               "d2h_bytes_per_step": w.P * 4,
               "api": "nb_step_fused_host (pinned host gradients in, mean model out)"}
        del host

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, per_step, desc = time_oracle(w, args.cpu_sample_cols, args.cpu_sample_steps)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc,
               "host_cores_available": host_threads()}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "K": w.K, "P": w.P, "M": w.M, "grad_dtype": w.grad_dtype,
                       "variant": w.variant, "topology": w.topology, "order": args.order,
                       "entry": "nb_accumulate+nb_step" if args.unfused else "nb_step_fused",
                       "parallelism": "column-shard x%d" % world,
                       "l2": "inputs larger than L2 (%.1f GB gradient stream x%d buffers + %.1f GB state per step)"
                             % (g_bytes / 1e9, n_buf, 2 * w.K * w.P * 4 / 1e9)},
            "achieved_hbm_gbs": achieved, "frac_of_8TBps": achieved / 8000.0,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_2211_00889_b200 import workloads as WL
    w = WL.WORKLOADS[args.workload]
    if args.cols:
        from dataclasses import replace
        w = replace(WL.scaled(w, args.cols), name="%s[P=%d]" % (w.name, args.cols))
    if args.variant:
        from dataclasses import replace
        topo = {"allreduce": "full", "dpsgd": "ring", "centralized": "full"}[args.variant]
        w = replace(w, variant=args.variant, topology=topo, name="%s[%s]" % (w.name, args.variant))
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
