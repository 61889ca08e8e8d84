#!/usr/bin/env python
"""Benchmark of the Jacobi hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c3_eigenmode_16384] [--mode auto] [--tsteps T]

One *step* is one whole job of the workload: its sweeps (every sweep with its halo exchange:
pack, unpack, update, in whatever form the schedule gives them) and the residual norm after every
group of sweeps the workload names (configs 2 and 5: every 10 sweeps; else after the last sweep).  The metric is Jacobi GLUP/s
(1e9 lattice-point updates per second); effective GB/s = GLUP/s x compulsory bytes per point
(16 B: read u, write u'; 24 B with f).

Prints exactly one JSON line on stdout.  With N > 1 (launched by torchrun) every rank runs an
independent replica of the job on its own GPU -- the path is a single-GPU library and has no
exchange between GPUs -- and rank 0 reports units of all ranks / max time over ranks.

``--impl reference`` times the CPU oracle (the plain C checker under oracle/) on the host
cores for the same metric; it is a deliberately slow program, reported for context.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2210_01238_b200 import inputs  # noqa: E402

METRIC = "jacobi_glups"
UNIT = "GLUP/s"
L2_BYTES = 126e6

# DRAM bytes per launch of the dominant kernel from an ncu capture (profiles/), and the hash of
# the sources that define that kernel and its launch geometry at the time of the capture; reported
# as null once any of them changed.
# key: (schedule, tsteps, ndim, has_f)
# bytes_per_point_per_launch: (dram__bytes_read.sum + dram__bytes_write.sum) / points of the captured
# launch (a smaller case of the same workload, named beside each entry), scaled to the workload by
# its points -- traffic is proportional to the points: every strip or tile reads and writes its own
# part of the grid once per launch.
SWEEP_SOURCES = ("jac_kernels.cuh", "jac_temporal3d.cuh", "jac_geom.h", "jac.cu")
CAPTURE_SHA = "22367cf9d08cf954"
RESIDENT_SOURCES = ("jac_resident.cuh", "jac_kernels.cuh", "jac_geom.h", "jac.cu")
RESIDENT_CAPTURE_SHA = "5bebd6c06a175820"
NCU_TRAFFIC = {
    # profiles/temporal2d_eigenmode_8192.md
    ("temporal", 8, 2, False): {"bytes_per_point_per_launch": (606.869248e6 + 494.355200e6) / 8192 ** 2},
    ("temporal", 4, 2, False): {"bytes_per_point_per_launch": (617.974528e6 + 489.620224e6) / 8192 ** 2},
    # profiles/temporal2d_poisson_4096.md (config 2 itself; its arrays are about the size of L2)
    ("temporal", 6, 2, True): {"bytes_per_point_per_launch": (322.085632e6 + 103.113216e6) / 4096 ** 2},
    # profiles/temporal3d_poisson_512.md
    ("temporal", 3, 3, True): {"bytes_per_point_per_launch": (2.514893e9 + 1.050443e9) / 512 ** 3},
    ("temporal", 2, 3, True): {"bytes_per_point_per_launch": (2.447718e9 + 1.050805e9) / 512 ** 3},
    # profiles/exchange_schedule_eigenmode_8192.md (the update launch alone)
    ("exchange", 1, 2, False): {"bytes_per_point_per_launch": (574.175488e6 + 494.808576e6) / 8192 ** 2},
    ("exchange", 1, 3, True): {"bytes_per_point_per_launch": (2.370464e9 + 1.048717e9) / 512 ** 3},
    # profiles/resident_heated_edge_256.md (config 1 itself: the grid is read once, the result stays in L2)
    ("resident", 0, 2, False): {"bytes_per_point_per_launch": 600.832e3 / 256 ** 2},
}
for _key, _rec in NCU_TRAFFIC.items():
    if _key[0] == "resident":
        _rec.update(src=RESIDENT_SOURCES, src_sha=RESIDENT_CAPTURE_SHA)
    else:
        _rec.update(src=SWEEP_SOURCES, src_sha=CAPTURE_SHA)
KERNEL_NAMES = {("temporal", 2): "temporal2d_kernel", ("temporal", 3): "temporal3d_kernel", ("fused", 2): "sweep2d_kernel (update pulling neighbour interiors)",
                ("exchange", 2): "sweep2d_kernel", ("pertask", 2): "sweep2d_kernel (one launch per block)",
                ("fused", 3): "sweep3d_kernel (update pulling neighbour interiors)", ("exchange", 3): "sweep3d_kernel",
                ("pertask", 3): "sweep3d_kernel (one launch per block)",
                ("resident", 2): "resident2d_kernel (one cluster, grid in shared memory)",
                ("wide", 2): "sweep2d_kernel (grown boxes between wide exchanges)",
                ("wide", 3): "sweep3d_kernel (grown boxes between wide exchanges)"}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def kernel_src_sha(names=SWEEP_SOURCES) -> str:
    h = hashlib.sha256()
    for name in names:
        h.update((ROOT / "paper_2210_01238_b200" / "csrc" / name).read_bytes())
    return h.hexdigest()[:16]


def measured_peak_gbs():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str | None):
        self.uuid, self.proc = uuid, None

    def start(self):
        cmd = ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"]
        if self.uuid:
            cmd += ["-i", self.uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # "under load": samples in the upper half of the clock range seen (idle samples sit low)
        load = [x for x in sm if x >= 0.5 * max(sm)] if sm else []
        return {"sm_mhz": statistics.median(load) if load else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- workloads
def make_inputs(w: inputs.Workload):
    u0 = inputs.initial_u(w)
    f = inputs.rhs(w)
    return u0, f


def job_updates(w: inputs.Workload, sweeps: int) -> float:
    return float(w.points) * sweeps


# ----------------------------------------------------------------------------- reference arm
def oracle_time_job(w: inputs.Workload, u0, f, target_seconds: float, max_sweeps: int):
    """Times the CPU oracle (blocked form: pack, unpack, update per sweep, then the residual) on a
    bounded number of sweeps of the same grid.  Returns (glups, sweeps, seconds, threads)."""
    from oracle import orc
    B = orc.Blocked(w.n, w.b, w.halo, w.has_f)
    for face, v in enumerate(w.boundary()):
        B.set_boundary(face, v)
    B.set_u(u0)
    if f is not None:
        B.set_f(f)
    t0 = time.perf_counter()
    B.sweep(1)
    t1 = time.perf_counter() - t0
    sweeps = int(max(1, min(max_sweeps, target_seconds / max(t1, 1e-9))))
    every = w.residual_every if w.residual_every > 0 else 0
    if every:
        sweeps = max(every, sweeps // every * every)     # whole groups: `every` sweeps, then the residual
    t0 = time.perf_counter()
    if every:
        for _ in range(sweeps // every):
            B.sweep(every)
            B.residual()
    else:
        B.sweep(sweeps)
        B.residual()
    dt = time.perf_counter() - t0
    B.close()
    return job_updates(w, sweeps) / dt / 1e9, sweeps, dt, orc.max_threads()


def run_reference(args, w: inputs.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    u0, f = make_inputs(w)
    vals, sweeps = [], 0
    per_step = max(2.0, min(20.0, 60.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        g, sweeps, dt, threads = oracle_time_job(w, u0, f, per_step, w.sweeps)
        log(f"[reference] step {i}: {sweeps} sweeps in {dt:.2f} s -> {g:.3f} GLUP/s on {threads} threads")
        if i >= args.warmup:
            vals.append((g, dt))
    total_updates = sum(g * dt for g, dt in vals)
    total_time = sum(dt for _, dt in vals)
    value = total_updates / total_time
    sample = f"{sweeps} of {w.sweeps} sweeps (+1 residual) of the full {'x'.join(map(str, w.n))} grid per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_time / len(vals),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "grid": list(w.n), "block": list(w.b), "halo": w.halo,
                   "sweeps_per_step": sweeps, "has_f": w.has_f},
        "effective_gbs": value * w.bytes_per_point,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- our arm
def reduce_max_over_ranks(ms: float, device: str) -> float:
    """The slowest rank's time: what a job of independent replicas takes as a whole."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replicated_glups(updates_per_rank: float, world: int, ms: float) -> float:
    """Whole-job throughput of `world` independent replicas that all finish within `ms`."""
    return updates_per_rank * world / (ms * 1e-3) / 1e9


def resident_fits(w: inputs.Workload) -> bool:
    """Does the library accept the resident schedule for this grid (pure host query)?"""
    from paper_2210_01238_b200 import jac
    try:
        jac.workspace_bytes(jac.make_desc(w.n, w.b, w.halo, w.has_f, "resident"))
        return True
    except jac.JacError:
        return False


def default_schedule(w: inputs.Workload):
    """Fastest schedule the library has for the workload (all schedules give identical bits)."""
    if resident_fits(w):
        return "resident", 0          # small 2D grids: all sweeps of a call in one launch
    if (w.ndim == 2 and w.b[0] % 4 == 0) or (w.ndim == 3 and w.b[0] % 2 == 0):
        return "temporal", 0          # 0: the library picks the sweeps per launch
    return "exchange", 1


def run_ours(args, w: inputs.Workload):
    import torch
    import torch.distributed as dist
    from paper_2210_01238_b200 import jac

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    distributed = world > 1
    if distributed:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms: float) -> float:
        return reduce_max_over_ranks(ms, "cuda") if distributed else ms

    stream = torch.cuda.current_stream()
    u0, f = make_inputs(w)
    sweeps = args.sweeps if args.sweeps > 0 else w.sweeps
    u0_dev = torch.from_numpy(u0).cuda()
    props = torch.cuda.get_device_properties(local)
    uuid = str(props.uuid) if hasattr(props, "uuid") else None
    if uuid and not uuid.startswith("GPU-"):
        uuid = "GPU-" + uuid
    peak, peak_kind = measured_peak_gbs()

    def make_ctx(mode, tsteps, on_stream=None):
        # the wide schedule needs as many ghost layers as sweeps per exchange
        halo = max(w.halo, tsteps) if mode == "wide" else w.halo
        J = jac.Jacobi(w.n, w.b, halo, w.has_f, mode, tsteps, stream=on_stream)
        for face, v in enumerate(w.boundary()):
            J.set_boundary(face, v)
        if f is not None:
            J.set_f(f)
        return J

    # the workload's cadence: a residual after every `every` sweeps (0: only after the last sweep)
    every = w.residual_every if 0 < w.residual_every <= sweeps else sweeps
    groups = [every] * (sweeps // every) + ([sweeps % every] if sweeps % every else [])
    norms = torch.zeros(len(groups), dtype=torch.float64).pin_memory()

    def one_job(J, pairs=None):
        """The sweeps of one step with the residual norm after every group (queued, nothing waits).
        The norm after group k comes out of the sweep that reads that state anyway, the first of
        group k + 1 (jac_sweep_norms_async; the temporal schedule does not even cut its launches
        there); only the last one needs a pass of its own."""
        if pairs is not None:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(J.stream)
        if len(groups) > 1:
            J.sweep_norms_async(sweeps, every, norms)
        else:
            J.sweep(sweeps)
        if pairs is not None:
            b.record(J.stream)
            pairs.append((a, b))
        J.residual_async(norms[len(groups) - 1:])

    def time_schedule(J, mode, tsteps, steps, warmup, sample_clocks):
        """K steps (each: input -> blocks, the sweeps, a residual after every group of sweeps the
        workload names) between two barriers, timed with CUDA events on the launch stream; the sweep
        calls are also timed on their own."""
        for _ in range(warmup):
            J.set_u_device(u0_dev)
            one_job(J)
        barrier()
        sampler = ClockSampler(uuid) if sample_clocks else None
        if sampler:
            sampler.start()
        l0 = J.launch_count()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        step_pairs = []
        ev0.record(stream)
        for _ in range(steps):
            J.set_u_device(u0_dev)
            pairs = []
            one_job(J, pairs)
            step_pairs.append(pairs)
        ev1.record(stream)
        barrier()
        launches = J.launch_count() - l0
        clocks = sampler.stop() if sampler else None
        ms_total = max_over_ranks(ev0.elapsed_time(ev1))
        per_step = sorted(sum(a.elapsed_time(b) for a, b in pairs) for pairs in step_pairs)
        sweep_ms = sum(per_step)
        if mode == "temporal" and every >= tsteps:
            n_launch = -(-sweeps // tsteps)          # launches run across the points where a norm is due
        elif mode == "temporal":
            n_launch = sum(-(-n_sw // tsteps) for n_sw in groups)
        else:
            n_launch = len(groups) if mode == "resident" else sweeps
        glups = replicated_glups(job_updates(w, sweeps) * steps, world, ms_total)
        return {"glups": glups, "ms_total": ms_total, "launch_ms": sweep_ms / (steps * n_launch),
                "launch_ms_best": per_step[0] / n_launch, "launch_ms_median": statistics.median(per_step) / n_launch,
                "sweeps_per_launch": sweeps / n_launch, "launches": int(launches), "residual": float(norms[-1]),
                "residuals_per_step": len(groups), "clocks": clocks}

    mode, tsteps = args.mode, args.tsteps
    if mode == "auto":
        mode, tsteps = default_schedule(w)
    if mode == "wide":
        tsteps = tsteps or 4
    elif mode not in ("temporal", "resident"):      # resident: tsteps is the cluster size (0 = library's)
        tsteps = 1
    try:
        J = make_ctx(mode, tsteps)
    except jac.JacError:
        if mode != "resident" or args.mode != "auto":
            raise
        mode, tsteps = "temporal", 0      # the device cannot co-schedule the cluster: next best schedule
        J = make_ctx(mode, tsteps)
    if mode not in ("wide", "resident"):
        tsteps = J.sweeps_per_launch()
    main_run = time_schedule(J, mode, tsteps, args.steps, args.warmup, True)
    value = main_run["glups"]

    # ---- roofline of the dominant kernel (the sweep): algorithmic bytes per launch / mean launch time
    alg_bytes_per_launch = w.points * w.bytes_per_point * main_run["sweeps_per_launch"]
    achieved = alg_bytes_per_launch / (main_run["launch_ms"] * 1e-3) / 1e9
    traffic = None
    rec = NCU_TRAFFIC.get((mode, tsteps, w.ndim, w.has_f))
    if rec and rec["src_sha"] == kernel_src_sha(rec["src"]):
        traffic = rec["bytes_per_point_per_launch"] * w.points
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                "kernel": KERNEL_NAMES.get((mode, w.ndim), "sweep"),
                "launch_ms": main_run["launch_ms"], "launch_ms_best": main_run["launch_ms_best"],
                "launch_ms_median": main_run["launch_ms_median"], "sweeps_per_launch": main_run["sweeps_per_launch"],
                "algorithmic_bytes_per_launch": alg_bytes_per_launch,
                "frac_of_nominal_8TBs": achieved / 8000.0,
                "dram_gbs": traffic / (main_run["launch_ms"] * 1e-3) / 1e9 if traffic else None,
                "note": ("one launch performs sweeps_per_launch sweeps: bytes are counted per sweep "
                         "(16 or 24 B/point), so frac > 1 means DRAM traffic per sweep is below the "
                         "compulsory bytes of a one-sweep-per-pass kernel; dram_gbs is the measured traffic rate"
                         if main_run["sweeps_per_launch"] > 1 else
                         "launch time is the mean over the timed jac_sweep calls"
                         + (" and includes the pack and unpack launches" if mode == "exchange" else ""))}

    # ---- end to end through the C ABI with HOST buffers: every step copies its input from pinned
    # host memory into the context (jac_set_u_async), runs the job, and copies the solution and
    # the residual norms back (jac_get_u_async, jac_residual_async) inside the timed region.  The
    # contexts carry JAC_FLAG_HOST_STAGING: one contiguous copy per direction plus a kernel
    # between the dense staging array and the blocks; the copy in runs on the context's own copy
    # stream and overlaps the previous step's sweeps and copy out.
    J.close()
    J = None
    e2e = None
    if not args.no_e2e:
        host_in = torch.from_numpy(u0).pin_memory()
        nbytes = int(u0.nbytes)

        def job_norms():
            return torch.zeros(len(groups), dtype=torch.float64).pin_memory()

        def staged_ctx(on_stream):
            halo = max(w.halo, tsteps) if mode == "wide" else w.halo
            Jc = jac.Jacobi(w.n, w.b, halo, w.has_f, mode, tsteps, stream=on_stream, flags=jac.FLAG_HOST_STAGING)
            for face, v in enumerate(w.boundary()):
                Jc.set_boundary(face, v)
            if f is not None:
                Jc.set_f(f)
            return Jc

        def e2e_step(Jc, out, nrm):
            Jc.set_u_async(host_in)
            if len(groups) > 1:
                Jc.sweep_norms_async(sweeps, every, nrm)
            else:
                Jc.sweep(sweeps)
            Jc.residual_async(nrm[len(groups) - 1:])
            Jc.get_u_async(out)

        def run_pipeline(depth, count):
            """`count` steps going round `depth` contexts on `depth` streams; host clock between
            synchronisations of all streams (fill and drain of the pipeline inside the timed region)."""
            streams = [torch.cuda.Stream() for _ in range(depth)]
            ctxs = [staged_ctx(st) for st in streams]
            outs = [torch.empty_like(host_in).pin_memory() for _ in range(depth)]
            nrms = [job_norms() for _ in range(depth)]
            for i in range(depth):                                   # warm every context
                e2e_step(ctxs[i], outs[i], nrms[i])
            for st in streams:
                st.synchronize()
            barrier()
            t0 = time.perf_counter()
            for k in range(count):
                i = k % depth
                e2e_step(ctxs[i], outs[i], nrms[i])
            for st in streams:
                st.synchronize()
            barrier()
            ms = max_over_ranks((time.perf_counter() - t0) * 1e3)
            last = float(nrms[(count - 1) % depth][-1])
            assert abs(last - main_run["residual"]) <= 1e-10 * main_run["residual"], (last, main_run["residual"])
            for Jc in ctxs:
                Jc.close()
            return ms

        def e2e_record(ms, count, what):
            return {"value": job_updates(w, sweeps) * count * world / (ms * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes + 8 * len(groups),
                    "steps": count, "ms_per_step": ms / count,
                    "pcie_gbs_per_direction": nbytes / (ms / count * 1e-3) / 1e9, "what": what}

        one_steps = max(3, min(args.steps, 6))
        one = e2e_record(run_pipeline(1, one_steps), one_steps,
                         "one context, steps queued back to back on one stream: jac_set_u_async(pinned host) + jac_sweep (jac_sweep_norms_async when the workload names a residual cadence) + "
                         "jac_residual_async after the last group + jac_get_u_async(pinned host)")
        e2e = one
        # several contexts on as many streams, steps going round them: the copy in of one step, the
        # sweeps of another and the copy out of a third run at the same time (the two copy directions
        # and the SMs are separate engines).  Single-process runs only: every rank of a multi-GPU run
        # would pin several more GiB of host memory.
        if nbytes <= 4 * 2 ** 30 and world == 1:
            depth = 3
            pipe_steps = max(2 * depth, args.steps)
            e2e = e2e_record(run_pipeline(depth, pipe_steps), pipe_steps,
                             f"{depth} contexts on {depth} streams, steps going round them; every step is jac_set_u_async(pinned "
                             "host) + jac_sweep (jac_sweep_norms_async when the workload names a residual cadence) + jac_residual_async + jac_get_u_async(pinned host); timed by the host "
                             "clock between synchronisations of all streams")
            e2e["one_context"] = one
        bound_ms = 2 * nbytes / 55e9 * 1e3
        e2e["note"] = ("bound by the host link when the copies take longer than the sweeps: at about 55 GB/s per direction "
                       f"{nbytes / 2 ** 30:.2f} GiB in and out are {bound_ms / 2:.1f} ms each against "
                       f"{main_run['ms_total'] / args.steps:.1f} ms of device work per step")
        del host_in

    # ---- the other schedules, briefly, for context (same job, fewer steps)
    others = {}
    if not args.no_others and world == 1:
        alts = [("exchange", 1), ("fused", 1), ("wide", 4)]   # wide: 4 ghost layers, 4 sweeps per exchange
        if resident_fits(w):
            alts += [("resident", 8), ("resident", 16)]   # cluster sizes
        if w.ndim == 2 and w.b[0] % 4 == 0:
            alts += [("temporal", 1), ("temporal", 2), ("temporal", 4), ("temporal", 8)]
        if w.ndim == 3 and w.b[0] % 2 == 0:
            alts += [("temporal", 1), ("temporal", 2)]
        for m, t in alts:
            if (m, t) == (mode, tsteps):
                continue
            if m == "resident":
                try:
                    jac.workspace_bytes(jac.make_desc(w.n, w.b, w.halo, w.has_f, m, t))
                except jac.JacError:
                    continue      # the grid does not fit a cluster of this size
            try:
                Jo = make_ctx(m, t)
            except jac.JacError:
                if m == "resident":
                    continue      # the device cannot co-schedule a cluster of this size
                raise
            r = time_schedule(Jo, m, t, 2, 1, False)
            Jo.close()
            others[f"{m}{t if m in ('temporal', 'wide', 'resident') else ''}"] = {
                "glups": r["glups"], "effective_gbs": r["glups"] * w.bytes_per_point,
                "launch_ms": r["launch_ms"], "launches": r["launches"]}
    del u0_dev
    torch.cuda.empty_cache()

    # ---- the oracle on the host cores, bounded sample (rank 0, single-GPU runs only)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        g, osw, dt, threads = oracle_time_job(w, u0, f, 20.0, w.sweeps)
        cpu_baseline = {"value": g, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": f"{osw} of {w.sweeps} sweeps (+1 residual) of the full "
                                  f"{'x'.join(map(str, w.n))} grid, {dt:.1f} s"}
        if w.points <= 2 ** 24:      # the small grids also on one core
            from oracle import orc
            orc.set_threads(1)
            g1, osw1, dt1, _ = oracle_time_job(w, u0, f, 5.0, w.sweeps)
            orc.set_threads(threads)
            cpu_baseline["one_core"] = {"value": g1, "sample": f"{osw1} sweeps, {dt1:.1f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": main_run["ms_total"] / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "grid": list(w.n), "block": list(w.b),
                       "halo": max(w.halo, tsteps) if mode == "wide" else w.halo,
                       "has_f": w.has_f, "sweeps_per_step": sweeps, "residuals_per_step": main_run["residuals_per_step"],
                       "schedule": mode, "tsteps": tsteps,
                       "l2": f"arrays of {w.points * 8 / 1e6:.0f} MB each exceed the {L2_BYTES / 1e6:.0f} MB L2"
                             if w.points * 8 > L2_BYTES else "arrays fit in L2 (no flush; latency-bound case)",
                       "replicas": world},
            "effective_gbs": value * w.bytes_per_point / world,
            "frac_of_8TBs": value * w.bytes_per_point / 8000.0 / world,
            "residual": main_run["residual"],
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e,
            "gpu_launches": main_run["launches"], "clocks": main_run["clocks"],
            "other_schedules": others,
        }
        print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- one domain over all ranks
def run_sharded(args, w: inputs.Workload):
    """--scaling strong: ONE job of the workload over all ranks.  The block grid is cut into slabs of
    whole block planes along the slowest axis, one slab context per rank (paper_2210_01238_b200.sharded);
    per sweep the faces on the cut planes travel to the neighbour ranks (NCCL send/recv between the
    contexts' cut buffers) while the rest of each slab is updated, and a residual costs one all-reduce
    of a double.  Every step copies the rank's part of the input in from pinned host memory and its
    part of the solution back (the timed region is the whole step); value = all points x sweeps /
    the slowest rank's time."""
    import torch
    import torch.distributed as dist
    from paper_2210_01238_b200 import jac, sharded

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    stream = torch.cuda.current_stream()
    sweeps = args.sweeps if args.sweeps > 0 else w.sweeps
    every = w.residual_every if 0 < w.residual_every <= sweeps else sweeps
    groups = [every] * (sweeps // every) + ([sweeps % every] if sweeps % every else [])
    mode = "fused" if world > 1 else ("temporal" if args.mode == "auto" else args.mode)
    u0, f = make_inputs(w)
    sl = sharded.slab_slice(w.n, w.b, rank, world)
    mine = torch.from_numpy(np.ascontiguousarray(u0[sl])).pin_memory()
    out = torch.empty_like(mine).pin_memory()
    J = sharded.slab_context(w.n, w.b, w.halo, w.has_f, mode, rank, world, stream=stream, flags=jac.FLAG_HOST_STAGING)
    sharded.set_slab_boundary(J, w.ndim, rank, world, w.boundary())
    if f is not None:
        J.set_f(np.ascontiguousarray(f[sl]))
    del u0, f

    def sumsq():
        return torch.tensor([J.residual_sumsq()], dtype=torch.float64, device="cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    norms = []

    def step():
        R = sharded.SlabRank(J, rank, world, dist, sumsq)
        J.set_u_async(mine)
        norms.clear()
        for n_sw in groups:
            R.sweep(n_sw)
            norms.append(R.residual())
        J.get_u_async(out)

    for _ in range(args.warmup):
        step()
    barrier()
    l0 = J.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    if world > 1:
        ms = reduce_max_over_ranks(ms, "cuda")
    launches = J.launch_count() - l0
    J.close()
    if rank == 0:
        value = job_updates(w, sweeps) * args.steps / (ms * 1e-3) / 1e9
        n_slab = sharded.slab_of(w.n, w.b, 0, world)[0]
        cut_bytes = 8 * w.halo * int(np.prod(w.n[:-1]))
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
                "dtype": "f64", "data": "synthetic",
                "config": {"workload": w.name, "grid": list(w.n), "block": list(w.b), "halo": w.halo, "has_f": w.has_f,
                           "sweeps_per_step": sweeps, "residuals_per_step": len(groups), "schedule": mode,
                           "slabs": world, "slab_of_rank_0": list(n_slab),
                           "cut_bytes_per_sweep_per_direction": cut_bytes if world > 1 else 0},
                "effective_gbs": value * w.bytes_per_point, "residual": norms[-1],
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": int(mine.numel() * 8) * world,
                        "d2h_bytes_per_step": int(mine.numel() * 8) * world + 8 * len(groups),
                        "what": "the timed step itself: jac_set_u_async(pinned host) + sweeps + residuals + jac_get_u_async"},
                "gpu_launches": int(launches), "roofline": None, "cpu_baseline": None}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- config 4
def run_halo_microbenchmark(args):
    """Config 4 (halo pack/unpack microbenchmark): the library's timings per block size and halo
    width with their roofline fractions, and beside each the CPU oracle's pack and unpack loops of the
    same decomposition timed on the host cores.  One JSON line."""
    import torch
    from paper_2210_01238_b200 import halo_bench
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    peak, peak_kind = measured_peak_gbs()
    total_gib = args.halo_gib
    rows = halo_bench.run(sorted(inputs.HALO_BENCH_SHAPES), list(inputs.HALO_BENCH_WIDTHS), total_gib, peak,
                          with_3d=not args.no_others)
    torch.cuda.empty_cache()
    if not args.no_cpu_baseline:
        from oracle import orc
        threads = orc.max_threads()
        for r in rows:
            n, b, h = r["grid"], r["block"], r["halo"]
            if len(n) == 3:
                continue            # 26 GB of oracle state for one number: the 2D cases carry the comparison
            O = orc.Blocked(n, b, h)
            O.set_u(inputs.uniform_field(n, inputs.HALO_BENCH_SEED))
            O.pack(); O.unpack()
            reps = max(3, min(200, int(2e8 / max(1, r["payload_bytes_per_call"]))))
            t0 = time.perf_counter()
            for _ in range(reps):
                O.pack()
            t_pack = (time.perf_counter() - t0) / reps
            t0 = time.perf_counter()
            for _ in range(reps):
                O.unpack()
            t_unpack = (time.perf_counter() - t0) / reps
            O.close()
            counted = 2 * r["payload_bytes_per_call"]
            r["cpu_baseline"] = {"kind": "oracle", "cores": threads, "unit": "GB/s",
                                 "pack_gbs": counted / t_pack / 1e9, "unpack_gbs": counted / t_unpack / 1e9,
                                 "pack_us": t_pack * 1e6, "unpack_us": t_unpack * 1e6,
                                 "sample": f"{reps} repetitions of pack and of unpack of all faces"}
    big = rows[-1]["all:exchange"]
    line = {"metric": "halo_exchange_gbs", "unit": "GB/s", "value": big["cold_gbs"], "n_gpus": 1, "higher_is_better": True,
            "dtype": "f64", "data": "synthetic", "vs_baseline": None,
            "config": {"workload": "c4_halo_microbenchmark", "value_is": "one-launch exchange of all faces, L2 evicted "
                       "between repetitions, of the last row", "gib_per_operation": total_gib},
            "roofline": dict(big["roofline"], peak_kind=f"of {peak_kind}"), "rows": rows}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3_eigenmode_16384", choices=sorted(inputs.CONFIGS) + ["c4_halo"])
    ap.add_argument("--halo-gib", type=float, default=1.0, help="c4_halo: GiB of face payload per operation")
    ap.add_argument("--mode", default="auto", choices=["auto", "fused", "exchange", "pertask", "temporal", "wide", "resident"],
                    help="schedule of jac_sweep; auto = the fastest one the library has for the workload")
    ap.add_argument("--tsteps", type=int, default=0)
    ap.add_argument("--sweeps", type=int, default=0, help="sweeps per step (default: the workload's)")
    ap.add_argument("--residual-every", type=int, default=-1,
                    help="residual norm after every N sweeps (default: the workload's; 0: only after the last sweep)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the brief runs of the other schedules")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="more than one GPU: weak = every rank runs a replica of the job; strong = one job, the "
                         "block grid cut into one slab per rank")
    ap.add_argument("--n", type=int, default=0,
                    help="profiling aid: same recipe on an n^d grid (block size unchanged)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        log("warning: fewer than 3 warm-up steps")
    if args.workload == "c4_halo":
        if args.impl == "ours" and int(os.environ.get("RANK", "0")) == 0:
            run_halo_microbenchmark(args)
        return
    w = inputs.CONFIGS[args.workload]
    if args.n:
        w = inputs.scaled(w, (args.n,) * w.ndim, name=f"{w.name}_at_{args.n}")
    if args.residual_every >= 0:
        import dataclasses
        w = dataclasses.replace(w, residual_every=args.residual_every)
    if args.impl == "reference":
        run_reference(args, w)
    elif args.scaling == "strong":
        run_sharded(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
