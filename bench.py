#!/usr/bin/env python
"""Benchmark of the batched corrected reduce / allreduce executor.

One step = one pass of the whole hot path (decode, up-correction, tree phase, root selection, allreduce
retry and broadcast bookkeeping, emit) over one resident batch of synthetic scenarios, i.e. one call of
ftc_allreduce_batch / ftc_reduce_batch = one kernel launch. Default workload: the P=4096 allreduce
configuration (f=4, k=32 int32, max, pre- and in-operation failures), a batch of 32768 scenarios
(16 GiB of inputs, far larger than L2, so no flush is needed between steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c4|c5|c5r] [--batch S]
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample of the same workload

Prints ONE JSON line (rank 0). With N > 1 (torchrun) every rank runs its own batch: scenarios are
independent, there is no collective on the data path ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_22445_b200 import scenarios as sc  # noqa: E402

ESZ = {"int32": 4, "int64": 8, "uint64": 8, "float32": 4}


def make_workload(name: str, S: int, first: int, rounds_attempt_c4: int):
    if name == "c3":
        return sc.config3(S=S, first=first)
    if name == "c4":
        return sc.config4(rounds_attempt_c4, S=S, first=first)
    if name == "c5":
        return sc.config5("allreduce", "sum", S=S, first=first)
    if name == "c5r":
        return sc.config5("reduce", "xor", S=S, first=first)
    raise SystemExit(f"unknown workload {name}")


DEFAULT_BATCH = {"c3": 1 << 18, "c4": 1 << 15, "c5": 1 << 13, "c5r": 1 << 13}     # 16 GiB of inputs each
DESCRIPTION = {
    "c3": "allreduce P=1024 f=3 k=16 float32 sum, 0..3 pre-operation failures",
    "c4": "allreduce P=4096 f=4 k=32 int32 max, 0..2 pre-operation + 0..2 in-operation failures",
    "c5": "allreduce P=65536 f=8 k=4 uint64 sum, 0..8 pre-operation failures, per-scenario first root",
    "c5r": "reduce P=65536 f=8 k=4 uint64 xor, 0..8 pre-operation failures, per-scenario root",
}


def bytes_per_scenario(w) -> int:
    """Algorithmic bytes of one scenario: inputs, failure mask, in-operation entries, root, result, status."""
    e = ESZ[np.dtype(w.dtype).name]
    b = w.P * w.k * e + sc.mask_words(w.P) * 4 + w.k * e + 16
    if w.inop is not None:
        b += w.inop.shape[1] * 8
    if w.roots is not None:
        b += 4
    return b


def rounds_of(w, sched) -> int:
    return sched["rounds_attempt"] if w.collective == "allreduce" else sched["rounds_reduce"]


# ------------------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.NamedTemporaryFile(prefix="ftc_clocks_", suffix=".csv", delete=False).name
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(gpu_index)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def lines(self) -> int:
        try:
            return sum(1 for _ in open(self.path))
        except OSError:
            return 0

    def wait_ready(self, timeout: float = 5.0) -> None:
        t0 = time.time()
        while self.proc is not None and self.lines() == 0 and time.time() - t0 < timeout:
            time.sleep(0.05)

    def mark(self) -> None:
        """Samples from here on count (the timed region starts)."""
        self.first = self.lines()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln, line in enumerate(open(self.path)):
            if ln < getattr(self, "first", 0):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
def prepare_oracle(w, n_scen: int, chunk: int):
    """Host inputs of the first n_scen scenarios of w, in chunks (prepared before any clock starts)."""
    ids = [np.arange(s, min(s + chunk, n_scen)) for s in range(0, n_scen, chunk)]
    return ids, [w.host_inputs(i) for i in ids]


def time_oracle(w, prepared):
    """Runs the oracle, as it stands, over the prepared scenarios on all host cores (threads; the C call releases
    the GIL). Returns (scenarios/s, seconds, threads used)."""
    from oracle import oracle as orc
    orc.lib()
    ids, xs = prepared
    cores = os.cpu_count() or 1
    allred = w.collective == "allreduce"

    def work(j):
        i = ids[j]
        orc.batch(xs[j], w.f, w.op, w.prefail[i], None if w.inop is None else w.inop[i],
                  None if w.roots is None else w.roots[i], max(w.root, 0), allred)

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as ex:
        list(ex.map(work, range(len(ids))))
    dt = time.perf_counter() - t0
    n_scen = sum(len(i) for i in ids)
    return n_scen / dt, dt, min(cores, len(ids))


ORACLE_SAMPLE = {"c3": (32768, 256), "c4": (8192, 64), "c5": (192, 2), "c5r": (192, 2)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    sched = orc.schedule(*{"c3": (1024, 3), "c4": (4096, 4), "c5": (65536, 8), "c5r": (65536, 8)}[args.workload])
    n_max, chunk = ORACLE_SAMPLE[args.workload]
    w = make_workload(args.workload, n_max, 0, sched["rounds_attempt"])
    cores = os.cpu_count() or 1
    # size one step so that the whole run stays near two minutes: probe the rate on one chunk per core first
    probe = prepare_oracle(w, min(n_max, chunk * cores), chunk)
    rate, _, _ = time_oracle(w, probe)
    n = int(rate * 120.0 / max(1, args.steps + args.warmup))
    n = max(chunk, min(n_max, (n // chunk) * chunk))
    prepared = prepare_oracle(w, n, chunk)
    times = []
    for it in range(args.warmup + args.steps):
        rate, dt, cores = time_oracle(w, prepared)
        if it >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = n / (ms / 1e3)
    line = {
        "impl": "reference", "metric": "scenarios_per_sec", "value": value, "unit": "scenarios/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"c3": "f32", "c4": "i32", "c5": "u64", "c5r": "u64"}[args.workload],
        "data": "synthetic", "process_rounds_per_sec": value * w.P * rounds_of(w, sched),
        "config": {"workload": f"{args.workload}: {DESCRIPTION[args.workload]}", "scenarios_per_step": n,
                   "note": "CPU oracle (literal message-by-message simulation) on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "scenarios/s", "cores": cores, "kind": "oracle",
                         "sample": f"{n} scenarios of the workload per step, threads over host cores"},
        "e2e": {"value": value, "unit": "scenarios/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def kernel_source_hash() -> str:
    """Hash of the sources of the staged kernel (the one the traffic figures belong to): ncu counters taken from
    an older kernel must not be quoted for a newer one."""
    import glob
    import hashlib
    h = hashlib.sha256()
    base = os.path.join(ROOT, "paper_2602_22445_b200", "csrc")
    files = glob.glob(os.path.join(base, "ftc_staged*.cu")) + glob.glob(os.path.join(base, "ftc_staged*.cuh")) + \
        [os.path.join(base, n) for n in ("ftc_tile_common.cuh", "ftc_device.cuh")]
    for f in sorted(files):
        h.update(open(f, "rb").read())
    return h.hexdigest()[:16]


def kernel_traffic(name: str, S: int):
    """DRAM read+write bytes of one launch over S scenarios, scaled from the committed ncu capture of a 2 GiB batch
    (traffic is proportional to the scenarios of a launch); None when there is no capture or the sources changed."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    rec = json.load(open(path))
    if rec.get("source_sha256_16") != kernel_source_hash() or name not in rec or not rec[name].get("valid"):
        return None
    return rec[name]["dram_bytes_per_scenario"] * S


def max_over_ranks(value: float, dist, device) -> float:
    """Largest value over all ranks (step times are reported as the slowest rank's)."""
    if dist is None:
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, scenarios_per_rank: int, ms_per_step: float) -> float:
    """Scenarios per second of the whole job: every rank processed its own scenarios in the slowest rank's time."""
    return world * scenarios_per_rank / (ms_per_step / 1e3)


def upload(w, torch):
    d_pf = torch.from_numpy(w.prefail.view(np.int32)).cuda()
    d_inop = None if w.inop is None else torch.from_numpy(np.ascontiguousarray(w.inop).view(np.int32)).cuda()
    d_roots = None if w.roots is None else torch.from_numpy(w.roots.view(np.int32)).cuda()
    return d_pf, d_inop, d_roots


def run_gpu(args):
    import torch
    from paper_2602_22445_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.load()

    name = args.workload
    S = args.batch or DEFAULT_BATCH[name]
    probe = make_workload(name, 1, 0, 28)
    tdt = getattr(torch, np.dtype(probe.dtype).name)
    desc0 = B.make_desc(probe.P, probe.f, probe.k, B.dtype_code(tdt), probe.op)
    sched = B.ftc_schedule_info(desc0)
    w = make_workload(name, S, rank * S, sched["rounds_attempt"])          # each rank its own scenarios
    if args.collective:
        w.collective = args.collective
    if args.failure_free:
        w.prefail[:] = 0
        if w.inop is not None:
            w.inop[:, :, 0] = sc.UNUSED
    allred = w.collective == "allreduce"
    kflags = {"auto": 0, "direct": B.FTC_KERNEL_DIRECT, "generic": B.FTC_KERNEL_GENERIC}[args.kernel]
    desc = B.make_desc(w.P, w.f, w.k, B.dtype_code(tdt), w.op, root=-1 if w.roots is not None else 0,
                       max_inop=0 if w.inop is None else w.inop.shape[1], flags=kflags)
    fn = B.ftc_allreduce_batch if allred else B.ftc_reduce_batch

    d_x = torch.empty((S, w.P, w.k), dtype=tdt, device="cuda")
    B.ftc_fill_inputs(w.kind, w.seed, w.first_scenario, S, w.P, w.k, d_x)
    d_pf, d_inop, d_roots = upload(w, torch)
    d_out = torch.empty((S, w.k), dtype=tdt, device="cuda")
    d_st = torch.empty((S, 4), dtype=torch.int32, device="cuda")
    wsb = B.ftc_workspace_bytes(desc, S, allred)
    d_ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()

    def step():
        fn(desc, S, d_x, d_pf, d_inop, d_roots, d_out, d_st, d_ws)

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.wait_ready()
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    if sampler:
        sampler.mark()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(args.steps):
        step()
        ev[i + 1].record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    clocks = sampler.stop() if sampler else None
    per_launch_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    total_ms = ev[0].elapsed_time(ev[-1])
    total_ms = max_over_ranks(total_ms, dist, torch.device("cuda", local))
    ms_per_step = total_ms / args.steps
    value = whole_job_value(world, S, ms_per_step)

    e2e = None
    if not args.kernel_only:
        # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region) ----
        Se = min(S, args.e2e_scenarios or max(64, (1 << 30) // (w.P * w.k * ESZ[np.dtype(w.dtype).name])))
        we = w
        h_x = torch.empty((Se, w.P, w.k), dtype=tdt).pin_memory()
        h_x.copy_(d_x[:Se])                                                   # same synthetic inputs, now resident on the host
        h_pf = torch.from_numpy(np.ascontiguousarray(we.prefail[:Se]).view(np.int32)).pin_memory()
        h_inop = None if we.inop is None else torch.from_numpy(np.ascontiguousarray(we.inop[:Se]).view(np.int32)).pin_memory()
        h_roots = None if we.roots is None else torch.from_numpy(np.ascontiguousarray(we.roots[:Se]).view(np.int32)).pin_memory()
        h_out = torch.empty((Se, w.k), dtype=tdt).pin_memory()
        h_st = torch.empty((Se, 4), dtype=torch.int32).pin_memory()
        staging = torch.empty(B.ftc_host_staging_bytes(desc, Se), dtype=torch.uint8, device="cuda")
        fn_host = B.ftc_allreduce_batch_host if allred else B.ftc_reduce_batch_host
        e2e_steps = max(2, min(args.steps, 5))
        fn_host(desc, Se, h_x, h_pf, h_inop, h_roots, h_out, h_st, staging)
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            fn_host(desc, Se, h_x, h_pf, h_inop, h_roots, h_out, h_st, staging)     # synchronises its stream itself
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        e2e_s = max_over_ranks(e2e_s, dist, torch.device("cuda", local))
        h2d = Se * (bytes_per_scenario(w) - w.k * ESZ[np.dtype(w.dtype).name] - 16)
        d2h = Se * (w.k * ESZ[np.dtype(w.dtype).name] + 16)
        same = bool((h_st.numpy() == d_st[:Se].cpu().numpy()).all() and
                    (h_out.view(torch.uint8).numpy() == d_out[:Se].cpu().view(torch.uint8).numpy()).all())

        e2e = {"value": world * Se / e2e_s, "unit": "scenarios/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "scenarios_per_step": Se, "matches_device_run": same}
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    # ---- roofline of the one kernel a step launches ----
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_kind = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_kind = 6650.0, "fallback"
    bytes_launch = S * bytes_per_scenario(w)
    avg_launch_ms = sum(per_launch_ms) / len(per_launch_ms)
    achieved = bytes_launch / (avg_launch_ms / 1e3) / 1e9
    traffic = kernel_traffic(name, S)

    # ---- the oracle beside it, on a bounded sample ----
    cpu = None
    if not (args.no_cpu_baseline or args.kernel_only):
        n, chunk = ORACLE_SAMPLE[name]
        wo = make_workload(name, n, 0, sched["rounds_attempt"])
        rate, dt, cores = time_oracle(wo, prepare_oracle(wo, n, chunk))
        cpu = {"value": rate, "unit": "scenarios/s", "cores": cores, "kind": "oracle",
               "sample": f"first {n} scenarios of the workload ({dt:.1f} s wall on {cores} threads)"}

    status = d_st.cpu().numpy().view(np.uint32)
    R = rounds_of(w, sched)
    line = {
        "metric": "scenarios_per_sec", "value": value, "unit": "scenarios/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"int32": "i32", "int64": "i64", "uint64": "u64", "float32": "f32"}[np.dtype(w.dtype).name],
        "data": "synthetic",
        "process_rounds_per_sec": value * w.P * R,
        "config": {"workload": f"{name}: {DESCRIPTION[name]}" + (f" [collective={args.collective}]" if args.collective else "")
                   + (" [failure-free]" if args.failure_free else ""), "scenarios_per_step_per_gpu": S,
                   "input_bytes_per_step_per_gpu": S * w.P * w.k * ESZ[np.dtype(w.dtype).name],
                   "cache": "inputs larger than L2, no flush", "kernel": B.ftc_kernel_name(desc, allred),
                   "rounds_per_scenario": R, "ok_scenarios": int(((status[:, 0] & 0xFF) == 0).sum())},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": peak_kind, "frac_of_nominal_8TBs": achieved / 8000.0, "traffic": traffic,
                     "bytes_per_launch": bytes_launch, "avg_launch_ms": avg_launch_ms,
                     "min_launch_ms": min(per_launch_ms)},
        "cpu_baseline": cpu,
        "e2e": e2e,
        "gpu_launches": args.steps,
        "clocks": clocks,
    }
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(DESCRIPTION))
    ap.add_argument("--batch", type=int, default=0, help="scenarios per step per GPU")
    ap.add_argument("--e2e-scenarios", type=int, default=0)
    ap.add_argument("--kernel", default="auto", choices=["auto", "direct", "generic"], help="force a kernel family")
    ap.add_argument("--collective", default="", choices=["", "reduce", "allreduce"], help="override the workload's collective")
    ap.add_argument("--failure-free", action="store_true", help="clear every failure of the workload (diagnostic)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel-only", action="store_true", help="skip the end-to-end and CPU legs (for profiler runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
