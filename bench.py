#!/usr/bin/env python
"""Benchmark of the SlowMo hot path: replica-parameter updates per second and achieved HBM
bandwidth of the fused local-step and outer-step kernels.

    python bench.py --gpus N --steps K --warmup W            (this library)
    python bench.py --impl reference --steps K --warmup W    (the CPU oracle, as it stands)

One step = one outer iteration of Algorithm 1 on the largest workload, the bandwidth stress
(P = 1e9 parameters, m = 4 workers, tau = 12, supplied gradient, 56 GB resident): tau fused
local-step launches over the [m, P] replica tensor and one fused outer-step launch. The headline
runs the byte-saving variant of the same step (last inner step inside the outer-step kernel,
broadcast left to the next iteration's first step); the plain tau + 1 launches are timed in the
same run and reported beside it, and so are the other workloads (ResNet-50-shaped, BMUF,
transformer-shaped with Adam, tau = 1 and tau = 48).

With N > 1 every rank runs an independent replica of the workload on its own GPU: the path has no
exchange step, so no collective is on the data path; ranks only agree on the slowest time. Started
without a launcher, `--gpus N` starts the N ranks itself (torch.distributed.run on 127.0.0.1).
"""
import argparse
import glob
import json
import os
import re
import socket
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
HEADLINE = "stress_tau12"
E2E_CHUNKS = 64


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
    rows read and written). Without the exact average (Section 6): x, anchor, u of every worker
    read and written, plus the reset rows."""
    m, P = w["m"], w["P"]
    nb = 2 if "adam" in w["base"] else 1
    if w.get("no_average"):
        return (24 + (4 * nb if w["buffer_policy"] == "reset" else 0)) * m * P
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


_TRAFFIC = None


def traffic_ratios():
    """DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch divided by the
    algorithmic bytes, per kernel case, read from the ncu summaries under profiles/: every line
    `traffic_ratio: case=<kernel case> ... ratio=<r> source=<hash of the kernel sources>`. A ratio
    counts only while the kernel sources are the ones the capture was taken on; otherwise the
    kernel has changed since and the traffic is reported as null."""
    global _TRAFFIC
    if _TRAFFIC is None:
        _TRAFFIC = {}
        now = kernel_source_hash()
        for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
            for line in open(path):
                if line.startswith("traffic_ratio:"):
                    kv = dict(p.split("=", 1) for p in line.split()[1:] if "=" in p)
                    if kv.get("source") == now:
                        _TRAFFIC[kv["case"]] = (float(kv["ratio"]), os.path.basename(path))
    return _TRAFFIC


def kernel_source_hash():
    """Short hash of the CUDA sources: ties an ncu summary to the kernels it was taken on."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1910_00643_b200", "csrc")
    for f in sorted(os.listdir(csrc)):
        if f.endswith((".cu", ".cuh")):
            h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:12]


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


def free_port():
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_command(n_ranks, argv):
    """The launcher command that starts n_ranks copies of this script on one node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *argv]


def ensure_ranks(args):
    """`--gpus N` without a launcher: start the N ranks and hand over to them. Under a launcher the
    rank count must agree with --gpus."""
    world = os.environ.get("WORLD_SIZE")
    if world is None:
        if args.gpus > 1:
            os.execv(sys.executable, spawn_command(args.gpus, sys.argv[1:]))
        return
    if int(world) != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started WORLD_SIZE={world} ranks")


def init_process_group(backend, local_rank):
    """Rendezvous of the ranks started by a launcher; NCCL's banner is kept off stdout, which
    carries the one JSON line only."""
    import torch
    import torch.distributed as dist
    sys.stdout.flush()
    saved = os.dup(1)
    os.dup2(2, 1)
    try:
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
            dist.barrier()
            torch.cuda.synchronize()
        else:
            dist.init_process_group("gloo")
            dist.barrier()
    finally:
        os.dup2(saved, 1)
        os.close(saved)


# --------------------------------------------------------------------------------- timed loops

def time_steps(s, w, steps, warmup, grad=None, fused=False, lazy=False):
    """Device-timed outer iterations. Returns total ms, the per-kernel mean launch ms of the local
    step and of the outer step, and (lazy variant) of the first local step of an iteration.
    With the fused variant the last inner step runs inside the outer-step kernel, so an iteration
    has tau-1 local-step launches. With the lazy variant the first launch of an iteration (which
    reads the anchor instead of the rows) is timed apart; the run ends with slowmo_materialize
    inside the timed region."""
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
    first = sum(e[0].elapsed_time(e[1]) for e in ev) / steps if split_first else None
    local = sum(e[1].elapsed_time(e[2]) for e in ev) / (steps * local_launches) if not (fused and tau == 1) else None
    outer = sum(e[2].elapsed_time(e[3]) for e in ev) / steps
    s.sync_status()
    return total, local, outer, first


def time_steps_e2e(s, w, steps, warmup, host_in, host_out, chunks=E2E_CHUNKS):
    """The same step through the C ABI with host buffers: every step uploads that step's
    per-worker input data from pinned host memory and reads the new anchor back."""
    import torch

    def one():
        # H2D of the [m, P] input, tau local steps + outer step, D2H of the new outer iterate,
        # pipelined over column windows inside the library call
        if w["grad_mode"] == "generated":
            s.iteration_host(host_in, host_out, chunks)
        else:
            s.iteration_host_supplied(host_in, host_out, chunks)

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
    ratio, source = traffic_ratios().get(case, (None, None))
    return {"bound": "hbm", "kernel": kind, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
            "frac": round(achieved / peak, 4), "peak_kind": peak_kind + " copy bandwidth",
            "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
            "bytes_per_launch": bytes_per_launch, "ms_per_launch": round(ms, 4),
            "traffic": None if ratio is None else int(ratio * bytes_per_launch),
            "achieved_dram_traffic": None if ratio is None else round(ratio * achieved, 1),
            "traffic_source": None if ratio is None else
            f"profiles/{source}: ncu small-case capture scaled by m*P (traffic / algorithmic = {ratio})",
            "case": case}


def kernel_case(w, kernel, variant):
    """Name of the kernel case as the ncu summaries under profiles/ key it."""
    base = "adam" if "adam" in w["base"] else "nesterov"
    if kernel == "local_step":
        return f"{'sgp_step' if w['base'].startswith('sgp') else 'local_step'}:{base}:{w['grad_mode']}"
    if kernel == "first_local_step":
        return f"local_step_virtual:{base}:{w['grad_mode']}:{w['buffer_policy']}"
    if w.get("no_average"):
        return f"outer_step_noaverage:{base}:{w['buffer_policy']}"
    if variant in ("fused", "lazy"):
        return f"last_step_outer_{variant}:{base}:{w['grad_mode']}:{w['buffer_policy']}"
    return f"outer_step_{variant}:{base}:{w['buffer_policy']}"


def measure(name, variant, steps, warmup, peak, peak_kind, overrides=None, context=None):
    """One workload in one outer-step variant: whole-step time and per-kernel rooflines. Returns
    (result dict, context) — the context is kept open when `context` was given or asked for."""
    import torch
    from paper_1910_00643_b200 import SlowMo, workloads
    w = workloads.workload(name, **(overrides or {}))
    s = context if context is not None else SlowMo(w)
    if context is None and w["grad_mode"] == "supplied":
        s.alloc_gradient()
        s.fill_gradient()
    s.set_variant("outer", variant)
    plain = w["base"].startswith("sgp") or w.get("no_average")
    fused = variant in ("fused", "lazy") and not plain
    lazy = fused and variant == "lazy" and w["tau"] >= 2
    total, local, outer, first = time_steps(s, w, steps, warmup, s.grad, fused=fused, lazy=lazy)
    out = {"workload": name, "outer_variant": variant, "steps": steps,
           "ms_per_step": round(total / steps, 4), "value": w["m"] * w["P"] * w["tau"] * steps / (total * 1e-3),
           "unit": UNIT, "launches_per_step": w["tau"] + (0 if fused else 1)}
    if local is not None:
        out["roofline_local_step"] = roofline("local_step", local_step_bytes(w), local, peak, peak_kind,
                                              kernel_case(w, "local_step", variant))
    nbytes = lazy_outer_step_bytes(w) if lazy else fused_outer_step_bytes(w) if fused else outer_step_bytes(w)
    out["roofline_outer_step"] = roofline("last_step_outer" if fused else "outer_step", nbytes, outer, peak, peak_kind,
                                          kernel_case(w, "outer_step", variant if (fused or not plain) else "direct"))
    if first is not None:
        out["roofline_first_local_step"] = roofline("local_step", virtual_first_step_bytes(w), first, peak, peak_kind,
                                                    kernel_case(w, "first_local_step", variant))
    return out, s, w


def release(s):
    import torch
    s.close()
    del s
    torch.cuda.empty_cache()


def cpu_baseline(w, budget_s=12.0):
    """The oracle, untouched, on a contiguous slice of the same workload: once on all host cores
    (the headline `value`), once on a single thread, each sized for about budget_s seconds."""
    import oracle
    cfg = oracle.make_config(**w)
    per_coord = w["m"] * w["tau"] * w["T"]

    def timed(threads):
        # grow the slice until a run takes long enough to extrapolate from, then size it for the budget
        n, dt = 4096, 0.0
        while True:
            t0 = time.perf_counter()
            oracle.run(cfg, j0=0, n=n, precision="f32", threads=threads)
            dt = time.perf_counter() - t0
            if dt >= 0.5 or n >= w["P"]:
                break
            n = min(w["P"], n * 8)
        n = int(max(4096, min(w["P"], 1 << 26, n * budget_s / max(dt, 1e-3))))
        t0 = time.perf_counter()
        oracle.run(cfg, j0=0, n=n, precision="f32", threads=threads)
        dt = time.perf_counter() - t0
        return n * per_coord / dt, n, dt

    cores = oracle.threads()
    v_all, n_all, dt_all = timed(None)
    v_one, n_one, dt_one = timed(1)
    what = f"all m={w['m']} workers, tau={w['tau']}, T={w['T']} outer iterations, binary32 mode"
    return {"value": v_all, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"coordinates 0..{n_all - 1} of P={w['P']}, {what}, {dt_all:.1f} s on {cores} threads",
            "single_thread": {"value": v_one, "unit": UNIT, "cores": 1,
                              "sample": f"coordinates 0..{n_one - 1} of P={w['P']}, {what}, {dt_one:.1f} s on 1 thread"}}


# -------------------------------------------------------------------------------------- arms

def host_memory_available():
    try:
        import psutil
        return psutil.virtual_memory().available
    except Exception:
        return 0


def size_overrides(args):
    """Optional smaller problem (for profiler captures); the default is the named workload."""
    over = {}
    for key in ("P", "m", "tau"):
        if getattr(args, key) is not None:
            over[key] = getattr(args, key)
    if "P" in over:
        over["n_tensors"] = 0
    if args.no_average:
        over["no_average"] = True
    return over


def describe(w, name):
    return (f"{name}: P={w['P']} m={w['m']} tau={w['tau']} base={w['base']} buffers={w['buffer_policy']} "
            f"grad={w['grad_mode']}")


STEP_TEXT = {
    "lazy": "one outer iteration = tau-1 local-step launches (the first reads the anchor in place of the replica "
            "rows) + one launch of the outer step with the last inner step fused in and the broadcast left to the "
            "next iteration (SLOWMO_OUTER_LAZY); the timed region ends with slowmo_materialize",
    "fused": "one outer iteration = tau-1 local-step launches + one launch of the outer step with the last inner "
             "step fused in (SLOWMO_OUTER_FUSED)",
    "direct": "one outer iteration = tau local-step launches + one outer-step launch",
    "staged": "one outer iteration = tau local-step launches + one outer-step launch (bulk-copy staging)",
}


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ):   # under a launcher
        init_process_group("nccl", local_rank)
    dev = torch.device("cuda", local_rank)
    peak, peak_kind = measured_peak()
    over = size_overrides(args)
    name, variant = args.workload, args.outer_variant

    # ---- headline: device-resident, timed between barriers, clocks sampled meanwhile
    sampler = ClockSampler(local_rank)
    sampler.start()
    head, s, w = measure(name, variant, args.steps, args.warmup, peak, peak_kind, over)
    clocks = sampler.stop()
    value, ms = aggregate_throughput(w["m"] * w["P"] * w["tau"] * args.steps, head["ms_per_step"] * args.steps, dev)

    # ---- the plain tau + 1 launches of the same workload, same context, same run
    plain = None
    if variant != "direct" and not args.no_extra:
        plain, _, _ = measure(name, "direct", max(2, args.steps // 4), 1, peak, peak_kind, over, context=s)
        staged, _, _ = measure(name, "staged", 2, 1, peak, peak_kind, over, context=s)
        plain["roofline_outer_step_staged"] = staged["roofline_outer_step"]
        s.set_variant("outer", variant)

    # ---- end to end: host buffers in and out through the C ABI
    e2e = None
    host_bytes = 4 * (w["m"] + 1) * w["P"]
    if not args.no_e2e and host_memory_available() < 2 * host_bytes:
        e2e = {"skipped": f"needs {host_bytes / 1e9:.1f} GB of pinned host memory; "
                          f"{host_memory_available() / 1e9:.1f} GB available"}
    elif not args.no_e2e:
        generated = w["grad_mode"] == "generated"
        host_in = torch.empty((w["m"], w["P"]), dtype=torch.float32, pin_memory=True)
        host_out = torch.empty((w["m"] if w.get("no_average") else 1, w["P"]), dtype=torch.float32, pin_memory=True)
        # the same per-worker data the device-resident run used
        if generated:
            s.get_params("c", out=host_in)
        else:
            s.synchronize()
            host_in.copy_(s.grad.view(w["m"], s.pitch)[:, :w["P"]])
        e2e_steps = max(1, min(args.steps, 4))
        e2e_ms = time_steps_e2e(s, w, e2e_steps, 1, host_in, host_out, args.e2e_chunks)
        e2e_value, _ = aggregate_throughput(w["m"] * w["P"] * w["tau"] * e2e_steps, e2e_ms, dev)
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": host_in.numel() * 4,
               "d2h_bytes_per_step": host_out.numel() * 4, "steps": e2e_steps,
               "ms_per_step": round(e2e_ms / e2e_steps, 3),
               "note": "each step is one slowmo_iteration_host%s call: uploads the per-worker %s [m,P] from pinned "
                       "host memory and reads x_{t+1,0} back, pipelined with the kernels over %d column windows"
                       % ("" if generated else "_supplied", "centres c" if generated else "gradient G", args.e2e_chunks)}
        del host_in, host_out
    release(s)

    fused = head["launches_per_step"] == w["tau"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": describe(w, name), "step": STEP_TEXT[variant if fused or variant == "staged" else "direct"],
                   "outer_variant": variant,
                   "replicas": "independent replica of the workload per GPU, no collective on the data path",
                   "l2": "state tensors (56 GB at the default workload) are far larger than the 126 MB L2; no flush needed"},
        "gpu_launches": args.steps * head["launches_per_step"] + (1 if variant == "lazy" and fused else 0),
        "clocks": clocks,
        "roofline": head.get("roofline_local_step") or head["roofline_outer_step"],
        "roofline_outer_step": head["roofline_outer_step"],
        "e2e": e2e,
    }
    if "roofline_first_local_step" in head:
        line["roofline_first_local_step"] = head["roofline_first_local_step"]
    if plain is not None:
        line["direct_variant"] = plain
    if rank == 0 and world == 1:
        if not args.no_extra:
            line["other_workloads"] = other_workloads(peak, peak_kind, skip=name)
        if not args.no_cpu:
            from paper_1910_00643_b200 import workloads
            line["cpu_baseline"] = cpu_baseline(workloads.workload(name, **over), args.cpu_seconds)
    if rank == 0:
        print(json.dumps(line))
    if dist.is_initialized():
        dist.destroy_process_group()


def other_workloads(peak, peak_kind, skip):
    """The remaining workloads, a few outer iterations each, in the lazy and the direct variant."""
    out = {}
    for name, steps in (("stress_tau1", 3), ("stress_tau48", 2), ("resnet50", 5), ("bmuf", 2), ("transformer_adam", 3)):
        if name == skip:
            continue
        try:
            res, s, _ = measure(name, "lazy", steps, 1, peak, peak_kind)
            direct, _, _ = measure(name, "direct", steps, 1, peak, peak_kind, context=s)
            release(s)
            res["direct_variant"] = direct
            out[name] = res
        except Exception as exc:  # e.g. out of memory on a smaller device: report, do not hide
            out[name] = {"error": repr(exc)}
    return out


def run_sharded(args):
    """Workers sharded over the GPUs (one process per GPU, m / N workers each): the local steps run on
    each GPU's own rows and the outer step is slowmo_outer_step_sharded, which does the exact average
    over peer-mapped memory. Reports the step time, the outer step's share of it and the NVLink bytes
    each GPU moves per outer step, beside the expectation (1 - 1/N) * m * (P/N) * 4 bytes each way
    for the x rows (buffer rows on top under the average policy)."""
    import torch
    import torch.distributed as dist
    from paper_1910_00643_b200 import workloads
    from paper_1910_00643_b200.sharded import ShardedSlowMo
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if "RANK" not in os.environ:       # one rank without a launcher still needs a process group
        os.environ.update(RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(free_port()))
    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")   # peer memory is touched with plain loads and stores only
    init_process_group("nccl", local_rank)
    dev = torch.device("cuda", local_rank)
    name = "resnet50" if args.workload == HEADLINE else args.workload
    w = workloads.workload(name, **size_overrides(args))
    s = ShardedSlowMo(w)
    tau, steps = w["tau"], args.steps
    for _ in range(args.warmup):
        s.local_steps(tau)
        s.outer_step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    s.local.synchronize()
    barrier()
    torch.cuda.synchronize()
    for i in range(steps):
        ev[i][0].record(s.local.stream)
        s.local_steps(tau)
        ev[i][1].record(s.local.stream)
        s.outer_step()                     # fence, sharded kernel, fence
        ev[i][2].record(s.local.stream)
    s.local.synchronize()
    torch.cuda.synchronize()
    barrier()
    total = ev[0][0].elapsed_time(ev[-1][2])
    outer = sum(e[1].elapsed_time(e[2]) for e in ev) / steps
    value, ms = aggregate_throughput(s.m_local * w["P"] * tau * steps, total, dev)
    outer_ms = max_over_ranks(outer, dev)
    nb = 2 if "adam" in w["base"] else 1
    rows = 1 + (nb if w["buffer_policy"] == "average" else 0)          # row sets read from peers
    wrows = 1 + (nb if w["buffer_policy"] != "maintain" else 0)        # row sets written to peers
    slice_cols = w["P"] / world
    remote = (world - 1) * s.m_local * slice_cols * 4
    line = {"mode": "sharded", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": args.warmup, "ms_per_step": round(ms / steps, 4), "higher_is_better": True, "scaling": "strong",
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(w, name), "workers_per_gpu": s.m_local,
                       "step": "tau local-step launches on each GPU's own rows + fence + one sharded outer-step kernel "
                               "per GPU (reduce-scatter, Eq. 2/3, all-gather over peer memory) + fence"},
            "outer_step_ms": round(outer_ms, 4), "outer_step_share": round(outer_ms * steps / ms, 4),
            "nvlink_bytes_per_gpu_per_outer_step": {
                "read_from_peers": int(rows * remote), "written_to_peers": int(wrows * remote + (world - 1) * 8 * slice_cols),
                "expected_for_x_rows_each_way": int(remote),
                "formula": "(1 - 1/N) * m * (P/N) * 4 bytes for each set of rows read or written, plus the anchor and u "
                           "slices written to every peer"},
            "peer_access": "plain loads and stores; no bulk copy, no multicast, no library kernel on peer memory"}
    s.close()
    if rank == 0:
        print(json.dumps(line))
    dist.destroy_process_group()


def run_selftest_ranks(args):
    """Host-only check of the rank plumbing (no GPU): gloo rendezvous, aggregation, one JSON line."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if "RANK" in os.environ:
        init_process_group("gloo", 0)
    value, ms = aggregate_throughput(1000.0 * (rank + 1), 10.0 * (rank + 1))
    barrier()
    if rank == 0:
        print(json.dumps({"selftest": "ranks", "n_gpus": world, "value": value, "ms": ms}))
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
        "config": {"workload": describe(w, args.workload), "sample": sample},
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
    ap.add_argument("--mode", default="replicas", choices=["replicas", "sharded"],
                    help="replicas: every GPU runs the whole workload (the default). sharded: the m workers of "
                         "the ResNet-50-shaped workload are spread over the GPUs and the outer step averages "
                         "over peer memory")
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--outer-variant", default="lazy", choices=["direct", "staged", "fused", "lazy"])
    ap.add_argument("--P", type=int, default=None, help="override the workload's parameter count")
    ap.add_argument("--m", type=int, default=None, help="override the workload's worker count")
    ap.add_argument("--tau", type=int, default=None, help="override the workload's inner steps")
    ap.add_argument("--no-average", action="store_true",
                    help="run the workload without the exact average (Section 6 of the paper)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end measurement")
    ap.add_argument("--e2e-chunks", type=int, default=E2E_CHUNKS,
                    help="column windows the end-to-end call pipelines its copies and kernels over")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the direct-variant figure of the same workload and the other workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--reference-coords", type=int, default=1 << 20)
    ap.add_argument("--selftest-ranks", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    ensure_ranks(args)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.selftest_ranks:
        run_selftest_ranks(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.mode == "sharded":
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
