#!/usr/bin/env python
"""Benchmark of the SlowMo hot path: replica-parameter updates per second and achieved HBM
bandwidth of the fused local-step and outer-step kernels.

    python bench.py --gpus N --steps K --warmup W            (this library)
    python bench.py --impl reference --steps K --warmup W    (the CPU oracle, as it stands)

One step = one outer iteration of Algorithm 1 on the ResNet-50-shaped workload: tau fused
local-step launches over the [m, P] replica tensor and one fused outer-step launch. With
N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the
workload on its own GPU: the path has no exchange step, so no collective is on the data
path; ranks only agree on the slowest time.
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

METRIC = "replica-param updates/sec (local + outer step)"
UNIT = "updates/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch divided by the
# algorithmic bytes, from ncu captures of small cases of the current kernels (profiles/);
# traffic grows in proportion to m*P, so the ratio carries to the full launch. None = no capture
# of the kernel as it stands.
NCU_TRAFFIC_RATIO = {("local_step", "generated"): 0.961, ("local_step", "supplied"): 0.980,
                     ("outer_step", "average"): 0.952, ("outer_step", "reset"): 0.973,
                     ("last_step_outer", "generated-average"): 0.975, ("last_step_outer", "supplied-reset"): 0.983,
                     ("last_step_outer", "lazy-generated-average"): 1.001, ("last_step_outer", "lazy-supplied-reset"): 0.994,
                     ("local_step", "virt-generated-average"): 0.940, ("local_step", "virt-supplied-reset"): 0.970}


# ----------------------------------------------------------------------------- bytes and peaks

def local_step_bytes(w):
    """Algorithmic HBM bytes of one fused local-step launch: x and h (and v) read and written,
    the per-worker gradient data (centres c, or the supplied gradient) read, and the curvature
    read once for all workers."""
    per_update = 8 + 8 + 4 + (8 if "adam" in w["base"] else 0)
    total = per_update * w["m"] * w["P"]
    if w["grad_mode"] == "generated":
        total += 4 * w["P"]
    return total


def outer_step_bytes(w):
    """Algorithmic HBM bytes of one fused outer-step launch: m rows read and written, anchor
    and u read and written, plus the buffer policy (reset: nb*m rows written; average: nb*m
    rows read and written)."""
    m, P = w["m"], w["P"]
    nb = 2 if "adam" in w["base"] else 1
    per_param = 8 * m + 16
    if w["buffer_policy"] == "reset":
        per_param += 4 * m * nb
    elif w["buffer_policy"] == "average":
        per_param += 8 * m * nb
    return per_param * P


def fused_outer_step_bytes(w):
    """Algorithmic HBM bytes of the outer-step kernel that also takes the last inner step.
    Per parameter: x, h [, v] and c-or-G of the m rows read, a, anchor, u read; u, anchor and
    the m rows of x written; the m rows of h [, v] written once under every policy (stepped
    values, zeros or means)."""
    m, P = w["m"], w["P"]
    nb = 2 if "adam" in w["base"] else 1
    per_param = m * (4 + 4 * nb + 4) + 8 + 8 + m * 4 + m * 4 * nb
    if w["grad_mode"] == "generated":
        per_param += 4
    return per_param * P


def lazy_outer_step_bytes(w):
    """Algorithmic bytes of the fused outer step in the lazy variant: as fused_outer_step_bytes
    without the m broadcast rows of x and without the reset / averaged buffer rows (the mean goes
    to one row)."""
    m, P = w["m"], w["P"]
    nb = 2 if "adam" in w["base"] else 1
    per_param = m * (4 + 4 * nb + 4) + 8 + 8
    if w["grad_mode"] == "generated":
        per_param += 4
    if w["buffer_policy"] == "maintain":
        per_param += 4 * m * nb
    elif w["buffer_policy"] == "average":
        per_param += 4 * nb
    return per_param * P


def virtual_first_step_bytes(w):
    """Algorithmic bytes of the first local step after a lazy outer step: c-or-G of the m rows
    and the anchor read (plus the buffer rows under "maintain", or the one row of means under
    "average"), x and the buffers of the m rows written."""
    m, P = w["m"], w["P"]
    nb = 2 if "adam" in w["base"] else 1
    per_param = 4 * m + 4 + 4 * m + 4 * m * nb
    if w["grad_mode"] == "generated":
        per_param += 4
    if w["buffer_policy"] == "maintain":
        per_param += 4 * m * nb
    elif w["buffer_policy"] == "average":
        per_param += 4 * nb
    return per_param * P


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------ clock sampling

class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons of one GPU through NVML (read-only) while running."""

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ------------------------------------------------------------------------- multi-rank plumbing

def max_over_ranks(value, device=None):
    """Largest `value` over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, device=None):
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate_throughput(units_this_rank, ms_this_rank, device=None):
    """Whole-job throughput: units of all ranks divided by the slowest rank's time."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


# --------------------------------------------------------------------------------- timed loops

def time_steps(s, w, steps, warmup, grad=None, fused=False, lazy=False):
    """Device-timed outer iterations. Returns total ms and the per-kernel mean launch ms.
    With the fused variant the last inner step runs inside the outer-step kernel, so an
    iteration has tau-1 local-step launches. With the lazy variant the first launch of an
    iteration (which reads the anchor instead of the rows) is timed apart and returned in
    time_steps.first_ms; the run ends with slowmo_materialize inside the timed region."""
    import torch
    tau = w["tau"]
    split_first = lazy and tau >= 3
    local_launches = (max(1, tau - 1) if fused else tau) - (1 if split_first else 0)
    for _ in range(warmup):
        s.local_steps(tau, grad)
        s.outer_step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    end = torch.cuda.Event(enable_timing=True)
    s.synchronize()
    barrier()
    torch.cuda.synchronize()
    for i in range(steps):
        ev[i][0].record(s.stream)
        if split_first:
            s.local_steps(1, grad)
        ev[i][1].record(s.stream)
        s.local_steps(tau - 1 if split_first else tau, grad)
        ev[i][2].record(s.stream)
        s.outer_step()
        ev[i][3].record(s.stream)
    s.materialize()
    end.record(s.stream)
    s.synchronize()
    torch.cuda.synchronize()
    barrier()
    total = ev[0][0].elapsed_time(end)
    time_steps.first_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / steps if split_first else None
    local = sum(e[1].elapsed_time(e[2]) for e in ev) / (steps * local_launches)
    outer = sum(e[2].elapsed_time(e[3]) for e in ev) / steps
    s.sync_status()
    return total, local, outer


def time_steps_e2e(s, w, steps, warmup, host_in, host_out, chunks=16):
    """The same step through the C ABI with host buffers: every step uploads that step's
    per-worker input data from pinned host memory and reads the new anchor back."""
    import torch

    def one():
        # H2D of the [m, P] centres, tau local steps + outer step, D2H of the new outer iterate,
        # pipelined over column windows inside the library call
        s.iteration_host(host_in, host_out, chunks)

    for _ in range(warmup):
        one()
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    start = torch.cuda.Event(enable_timing=True)
    stop = torch.cuda.Event(enable_timing=True)
    start.record(s.stream)
    for _ in range(steps):
        one()
    stop.record(s.stream)
    s.synchronize()
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3
    dev_ms = start.elapsed_time(stop)
    barrier()
    return max(wall_ms, dev_ms)


def roofline(kind, bytes_per_launch, ms, peak, peak_kind, case=None):
    achieved = bytes_per_launch / (ms * 1e-3) / 1e9
    ratio = NCU_TRAFFIC_RATIO.get((kind, case))
    return {"bound": "hbm", "kernel": kind, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
            "frac": round(achieved / peak, 4), "peak_kind": peak_kind + " copy bandwidth",
            "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
            "bytes_per_launch": bytes_per_launch, "ms_per_launch": round(ms, 4),
            "traffic": None if ratio is None else int(ratio * bytes_per_launch),
            "traffic_source": None if ratio is None else
            f"ncu small-case capture scaled by m*P (traffic / algorithmic = {ratio})"}


def cpu_baseline(w, budget_s=15.0):
    """The oracle, untouched, on a contiguous slice of the same workload sized for ~budget_s."""
    import oracle
    cfg = oracle.make_config(**w)
    n0 = 512
    t0 = time.perf_counter()
    oracle.run(cfg, j0=0, n=n0, precision="f32")
    dt = max(time.perf_counter() - t0, 1e-4)
    n = int(max(n0, min(w["P"], n0 * budget_s / dt)))
    t0 = time.perf_counter()
    oracle.run(cfg, j0=0, n=n, precision="f32")
    dt = time.perf_counter() - t0
    updates = n * w["m"] * w["tau"] * w["T"]
    return {"value": updates / dt, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"coordinates 0..{n - 1} of P={w['P']}, all m={w['m']} workers, tau={w['tau']}, "
                      f"T={w['T']} outer iterations, binary32 mode, {dt:.1f} s"}


def stress_extra(peak, peak_kind, tau=12, iters=2):
    """Largest configuration (supplied gradient, P = 1e9, m = 4): per-kernel bandwidth."""
    import torch
    from paper_1910_00643_b200 import SlowMo, workloads
    w = workloads.workload("stress_tau12", tau=tau)
    out = {"workload": "stress P=1e9 m=4 supplied gradient"}
    s = SlowMo(w)
    s.alloc_gradient()
    s.fill_gradient()
    for variant in ("direct", "staged", "fused", "lazy"):
        s.set_variant("outer", variant)
        total, local, outer = time_steps(s, w, iters, 1, s.grad, fused=variant in ("fused", "lazy"),
                                         lazy=variant == "lazy")
        if variant == "lazy":
            out["last_step_outer_lazy"] = roofline("last_step_outer", lazy_outer_step_bytes(w), outer, peak, peak_kind,
                                                   "lazy-supplied-reset")
            out["first_local_step_lazy"] = roofline("local_step", virtual_first_step_bytes(w), time_steps.first_ms,
                                                    peak, peak_kind, "virt-supplied-reset")
        elif variant == "fused":
            out["last_step_outer_fused"] = roofline("last_step_outer", fused_outer_step_bytes(w), outer, peak,
                                                    peak_kind, "supplied-reset")
        else:
            out["local_step"] = roofline("local_step", local_step_bytes(w), local, peak, peak_kind, "supplied")
            out["outer_step_" + variant] = roofline("outer_step", outer_step_bytes(w), outer, peak, peak_kind,
                                                    "reset" if variant == "direct" else None)
        out["updates_per_s_tau%d_%s" % (tau, variant)] = w["m"] * w["P"] * tau * iters / (total * 1e-3)
    s.close()
    del s
    torch.cuda.empty_cache()
    # the workload is defined as a sweep over tau: whole-run updates/s at tau = 1 and 48 too (T = 3)
    sweep = {str(tau): {v: out["updates_per_s_tau%d_%s" % (tau, v)] for v in ("direct", "fused", "lazy")}}
    for t_in in (1, 48):
        wt = workloads.workload("stress_tau12", tau=t_in)
        s = SlowMo(wt)
        s.alloc_gradient()
        s.fill_gradient()
        sweep[str(t_in)] = {}
        for variant in ("direct", "fused", "lazy"):
            s.set_variant("outer", variant)
            total, _, _ = time_steps(s, wt, wt["T"], 1, s.grad, fused=variant in ("fused", "lazy"),
                                     lazy=variant == "lazy")
            sweep[str(t_in)][variant] = wt["m"] * wt["P"] * t_in * wt["T"] / (total * 1e-3)
        s.close()
        del s
        torch.cuda.empty_cache()
    out["updates_per_s_by_tau"] = sweep
    return out


# -------------------------------------------------------------------------------------- arms

def size_overrides(args):
    """Optional smaller problem (for profiler captures); the default is the named workload."""
    over = {}
    for key in ("P", "m", "tau"):
        if getattr(args, key) is not None:
            over[key] = getattr(args, key)
    if "P" in over:
        over["n_tensors"] = 0
    return over


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1910_00643_b200 import SlowMo, workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    launched = "RANK" in os.environ and "MASTER_ADDR" in os.environ   # under torch.distributed.run
    if world > 1 or launched:
        # NCCL announces its version on stdout when the communicator is created: send that to
        # stderr so that stdout carries the one JSON line only
        sys.stdout.flush()
        saved = os.dup(1)
        os.dup2(2, 1)
        try:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
            dist.barrier()
            torch.cuda.synchronize()
        finally:
            os.dup2(saved, 1)
            os.close(saved)
    dev = torch.device("cuda", local_rank)

    w = workloads.workload(args.workload, **size_overrides(args))
    peak, peak_kind = measured_peak()
    s = SlowMo(w)
    s.set_variant("outer", args.outer_variant)
    fused = (args.outer_variant in ("fused", "lazy") and (w["grad_mode"] == "supplied" or w["m"] <= 64)
             and w["tau"] > 1 and not w["base"].startswith("sgp") and not w.get("no_average"))
    lazy = fused and args.outer_variant == "lazy"
    grad = None
    if w["grad_mode"] == "supplied":
        grad = s.alloc_gradient()
        s.fill_gradient()

    sampler = ClockSampler(local_rank)
    sampler.start()
    total_ms, local_ms, outer_ms = time_steps(s, w, args.steps, args.warmup, grad, fused=fused, lazy=lazy)
    first_ms = time_steps.first_ms
    clocks = sampler.stop()
    units = w["m"] * w["P"] * w["tau"] * args.steps
    value, ms = aggregate_throughput(units, total_ms, dev)

    # end to end: host buffers in and out through the C ABI
    e2e = None
    if w["grad_mode"] == "generated" and not args.no_e2e:
        host_in = torch.empty((w["m"], w["P"]), dtype=torch.float32, pin_memory=True)
        host_out = torch.empty((1, w["P"]), dtype=torch.float32, pin_memory=True)
        s.get_params("c", out=host_in)  # the same per-worker data the device-resident run used
        e2e_steps = max(1, min(args.steps, 5))
        e2e_ms = time_steps_e2e(s, w, e2e_steps, 1, host_in, host_out)
        e2e_value, _ = aggregate_throughput(w["m"] * w["P"] * w["tau"] * e2e_steps, e2e_ms, dev)
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": host_in.numel() * 4,
               "d2h_bytes_per_step": host_out.numel() * 4, "steps": e2e_steps,
               "ms_per_step": round(e2e_ms / e2e_steps, 3),
               "note": "each step is one slowmo_iteration_host call: uploads the per-worker centres c [m,P] "
                       "from pinned host memory and reads x_{t+1,0} back, pipelined with the kernels over "
                       "16 column windows"}
        del host_in, host_out
    s.close()
    del s
    torch.cuda.empty_cache()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: P={w['P']} m={w['m']} tau={w['tau']} "
                               f"base={w['base']} buffers={w['buffer_policy']} grad={w['grad_mode']}",
                   "step": ("one outer iteration = tau-1 local-step launches (the first reads the anchor in "
                            "place of the replica rows) + one launch of the outer step with the last inner "
                            "step fused in and the broadcast left to the next iteration (SLOWMO_OUTER_LAZY); "
                            "the timed region ends with slowmo_materialize") if lazy else
                           ("one outer iteration = tau-1 local-step launches + one launch of the outer step "
                            "with the last inner step fused in (SLOWMO_OUTER_FUSED)") if fused else
                           "one outer iteration = tau local-step launches + one outer-step launch",
                   "outer_variant": args.outer_variant,
                   "replicas": "independent replica of the workload per GPU, no collective on the data path",
                   "l2": "state tensors (>= 5 GB) are far larger than the 126 MB L2; no flush needed"},
        "gpu_launches": args.steps * (w["tau"] + (0 if fused else 1)) + (1 if lazy else 0),
        "clocks": clocks,
        "roofline": roofline("local_step", local_step_bytes(w), local_ms, peak, peak_kind,
                             w["grad_mode"] if w["base"] == "nesterov" else None),
        "roofline_outer_step": (
            roofline("last_step_outer", lazy_outer_step_bytes(w), outer_ms, peak, peak_kind,
                     f"lazy-{w['grad_mode']}-{w['buffer_policy']}" if w["base"] == "nesterov" else None) if lazy else
            roofline("last_step_outer", fused_outer_step_bytes(w), outer_ms, peak, peak_kind,
                     f"{w['grad_mode']}-{w['buffer_policy']}" if w["base"] == "nesterov" else None) if fused else
            roofline("outer_step", outer_step_bytes(w), outer_ms, peak, peak_kind,
                     w["buffer_policy"] if args.outer_variant == "direct" and w["base"] == "nesterov"
                     and w["buffer_policy"] != "maintain" else None)),
        "e2e": e2e,
    }
    if lazy and first_ms is not None:
        line["roofline_first_local_step"] = roofline(
            "local_step", virtual_first_step_bytes(w), first_ms, peak, peak_kind,
            f"virt-{w['grad_mode']}-{w['buffer_policy']}" if w["base"] == "nesterov" else None)
    if rank == 0 and world == 1:
        if not args.no_stress:
            try:
                line["stress"] = stress_extra(peak, peak_kind)
            except Exception as exc:  # out of memory on a smaller device: report, do not hide
                line["stress"] = {"error": repr(exc)}
        if not args.no_cpu:
            line["cpu_baseline"] = cpu_baseline(w, args.cpu_seconds)
    if rank == 0:
        print(json.dumps(line))
    if dist.is_initialized():
        dist.destroy_process_group()


def run_reference(args):
    """The oracle on the host cores, one bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_1910_00643_b200 import workloads
    w = workloads.workload(args.workload)
    cfg = oracle.make_config(**dict(w, T=1))
    n = args.reference_coords
    for _ in range(args.warmup):
        oracle.run(cfg, j0=0, n=n, precision="f32")
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle.run(cfg, j0=(i * n) % max(1, w["P"] - n), n=n, precision="f32")
    dt = time.perf_counter() - t0
    value = n * w["m"] * w["tau"] * args.steps / dt
    sample = (f"each step = one outer iteration (tau={w['tau']} local steps + outer step) on {n} "
              f"contiguous coordinates of P={w['P']}, all m={w['m']} workers, binary32 mode")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(dt / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: P={w['P']} m={w['m']} tau={w['tau']} base={w['base']} "
                               f"buffers={w['buffer_policy']} grad={w['grad_mode']}", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50")
    ap.add_argument("--outer-variant", default="lazy", choices=["direct", "staged", "fused", "lazy"])
    ap.add_argument("--P", type=int, default=None, help="override the workload's parameter count")
    ap.add_argument("--m", type=int, default=None, help="override the workload's worker count")
    ap.add_argument("--tau", type=int, default=None, help="override the workload's inner steps")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end measurement")
    ap.add_argument("--no-stress", action="store_true", help="skip the P=1e9 per-kernel measurement")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--reference-coords", type=int, default=1 << 17)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
