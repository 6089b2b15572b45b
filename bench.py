#!/usr/bin/env python
"""Benchmark of the batched corrected reduce / allreduce executor.

One step = one pass of the whole hot path (decode, up-correction, tree phase, root selection, allreduce
retry and broadcast bookkeeping, emit) over one resident batch of synthetic scenarios, i.e. one call of
ftc_allreduce_batch / ftc_reduce_batch = one kernel launch. Default workload: the P=4096 allreduce
configuration (f=4, k=32 int32, max, pre- and in-operation failures), a batch of 32768 scenarios
(16 GiB of inputs, far larger than L2, so no flush is needed between steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5|c5r] [--batch S]
    python bench.py --full-config [--workload cN]   # every batch of the configuration, every scenario checked
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample of the same workload

Beside the K timed steps of the headline workload the line carries: the same step repeated for about two seconds
with the SM clocks sampled meanwhile (roofline.sustained), the bandwidth of the library's read-only streaming
kernels over the same buffer (roofline.read_only_gbs), and one record per other configuration, timed the same way
(workloads: c5, c5r, c3, c2, and what every root child delivers on c4 and c5).

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
    if name == "c2":
        # all 2081 failure sets of size <= 2, each under S / 2081 input draws (the configuration has 16 draws: 33 296 scenarios)
        if S % 2081:
            raise SystemExit("a c2 batch is a multiple of 2081 scenarios (every failure set of size <= 2 once per draw)")
        w = sc.config2(draws=S // 2081)
        w.first_scenario = first
        return w
    if name == "c3":
        return sc.config3(S=S, first=first)
    if name == "c4":
        return sc.config4(rounds_attempt_c4, S=S, first=first)
    if name == "c5":
        return sc.config5("allreduce", "sum", S=S, first=first)
    if name == "c5r":
        return sc.config5("reduce", "xor", S=S, first=first)
    raise SystemExit(f"unknown workload {name}")


DEFAULT_BATCH = {"c3": 1 << 18, "c4": 1 << 15, "c5": 1 << 13, "c5r": 1 << 13,      # 16 GiB of inputs each
                 "c2": 2081 * 1024}                                                  # 8 GiB: the configuration's sets under 1024 draws
CONFIG_SCENARIOS = {"c3": 1 << 20, "c4": 1 << 18, "c5": 1 << 14, "c5r": 1 << 14, "c2": 2081 * 16}    # scenarios of the whole configuration
DESCRIPTION = {
    "c2": "reduce P=64 f=2 k=8 int64 sum, every pre-operation failure set of size <= 2, root 0 (64x the configuration's 16 input draws)",
    "c3": "allreduce P=1024 f=3 k=16 float32 (Irwin-Hall stand-in for N(0,1)) sum, 0..3 pre-operation failures",
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
        """Ends the sampling; returns the record of everything since mark()."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.proc = None
        rec = self.window(getattr(self, "first", 0), 1 << 60)
        os.unlink(self.path)
        return rec

    def window(self, lo: int, hi: int) -> dict:
        """Clock record of the samples lo <= line < hi (at least the last sample before hi)."""
        if not os.path.exists(self.path):
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        if hi <= lo:
            lo = max(0, hi - 1)
        sm, mx, reasons = [], [], set()
        for ln, line in enumerate(open(self.path)):
            if ln < lo or ln >= hi:
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


ORACLE_SAMPLE = {"c3": (32768, 256), "c4": (4096, 32), "c5": (192, 2), "c5r": (192, 2), "c2": (2081 * 128, 2081)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    sched = orc.schedule(*{"c2": (64, 2), "c3": (1024, 3), "c4": (4096, 4), "c5": (65536, 8), "c5r": (65536, 8)}[args.workload])
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
        "vs_baseline": None, "dtype": {"c2": "i64", "c3": "f32", "c4": "i32", "c5": "u64", "c5r": "u64"}[args.workload],
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
    """Hash of the sources of the staged and warp kernels (the ones the traffic figures belong to): ncu counters
    taken from an older kernel must not be quoted for a newer one."""
    import glob
    import hashlib
    h = hashlib.sha256()
    base = os.path.join(ROOT, "paper_2602_22445_b200", "csrc")
    files = [f for pat in ("ftc_staged*.cu", "ftc_staged*.cuh", "ftc_warp*.cu", "ftc_warp*.cuh") for f in glob.glob(os.path.join(base, pat))] + \
        [os.path.join(base, n) for n in ("ftc_tile_common.cuh", "ftc_device.cuh", "ftc_decode_warp.cuh")]
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


def measured_peak():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class Leg:
    """One workload resident on the device: inputs generated there, failure patterns uploaded, outputs and workspace."""

    def __init__(self, name, S, first, args, B, torch, sched_rounds, candidates=False, expanded=False):
        self.name, self.S, self.B, self.torch = name, S, B, torch
        self.candidates = candidates
        w = make_workload(name, S, first, sched_rounds)
        if args.collective:
            w.collective = args.collective
        if args.failure_free:
            w.prefail[:] = 0
            if w.inop is not None:
                w.inop[:, :, 0] = sc.UNUSED
        self.w = w
        self.allred = w.collective == "allreduce"
        self.tdt = getattr(torch, np.dtype(w.dtype).name)
        kflags = {"auto": 0, "direct": B.FTC_KERNEL_DIRECT, "generic": B.FTC_KERNEL_GENERIC, "levels": B.FTC_KERNEL_LEVELS}[args.kernel]
        if args.arity:
            kflags |= B.FTC_TREE_BINOMIAL if args.arity == 1 else B.FTC_TREE_ARITY(args.arity)
        if expanded:
            kflags |= B.FTC_OUT_EXPANDED            # allreduce: the value in the slot of every process that holds it, [S][P][k]
        self.desc = B.make_desc(w.P, w.f, w.k, B.dtype_code(self.tdt), w.op, root=-1 if w.roots is not None else 0,
                                max_inop=0 if w.inop is None else w.inop.shape[1], flags=kflags)
        self.fn = B.ftc_allreduce_batch if self.allred else B.ftc_reduce_batch
        self.d_x = torch.empty((S, w.P, w.k), dtype=self.tdt, device="cuda")
        B.ftc_fill_inputs(w.kind, w.seed, w.first_scenario, S, w.P, w.k, self.d_x)
        self.d_pf, self.d_inop, self.d_roots = upload(w, torch)
        self.d_out = torch.empty((S, w.k), dtype=self.tdt, device="cuda")
        self.d_st = torch.empty((S, 4), dtype=torch.int32, device="cuda")
        self.sched = B.ftc_schedule_info(self.desc)
        self.esz = ESZ[np.dtype(w.dtype).name]
        self.bytes_per_launch = S * bytes_per_scenario(w)
        if candidates:
            # every root child's delivery: f+1 values and (flag, list size) pairs per scenario instead of one result and status
            self.d_out = torch.empty((S, w.f + 1, w.k), dtype=self.tdt, device="cuda")
            self.d_st = torch.empty((S, w.f + 1, 2), dtype=torch.int32, device="cuda")
            self.d_ws = torch.empty(max(B.ftc_candidates_workspace_bytes(self.desc, S), 256), dtype=torch.uint8, device="cuda")
            self.bytes_per_launch += S * w.f * (w.k * self.esz + 8) - S * 8
        else:
            if expanded:
                self.d_out = torch.empty((S, w.P, w.k), dtype=self.tdt, device="cuda")
                self.bytes_per_launch += S * (w.P - 1) * w.k * self.esz
            self.d_ws = torch.empty(max(B.ftc_workspace_bytes(self.desc, S, self.allred), 16), dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()

    def regenerate(self, first, sched_rounds):
        """The next batch of the same workload in the same buffers (scenarios first .. first+S-1)."""
        w = make_workload(self.name, self.S, first, sched_rounds)
        w.collective = self.w.collective
        self.w = w
        self.B.ftc_fill_inputs(w.kind, w.seed, w.first_scenario, self.S, w.P, w.k, self.d_x)
        self.d_pf, self.d_inop, self.d_roots = upload(w, self.torch)
        self.torch.cuda.synchronize()

    def step(self):
        if self.candidates:
            self.B.ftc_candidates_batch(self.desc, self.S, self.allred, self.d_x, self.d_pf, self.d_inop, self.d_roots, self.d_out,
                                        self.d_st, self.d_ws)
        else:
            self.fn(self.desc, self.S, self.d_x, self.d_pf, self.d_inop, self.d_roots, self.d_out, self.d_st, self.d_ws)

    def rounds(self):
        return self.sched["rounds_attempt"] if self.allred else self.sched["rounds_reduce"]

    def status(self):
        return self.d_st.cpu().numpy().view(np.uint32)

    def free(self):
        for n in ("d_x", "d_pf", "d_inop", "d_roots", "d_out", "d_st", "d_ws"):
            setattr(self, n, None)
        self.torch.cuda.empty_cache()


def time_steps(torch, fn, steps):
    """CUDA events on the launching stream (torch's current stream: the binding passes exactly that stream to the
    library) around every step; returns (per-step ms, total ms)."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(steps):
        fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    return [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)], ev[0].elapsed_time(ev[-1])


def time_sustained(torch, fn, ms_per_step, seconds, sampler):
    """The same step back to back for about `seconds` of GPU time: (steps, ms per step, clocks during it)."""
    n = max(10, int(seconds * 1e3 / max(ms_per_step, 1e-3)))
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    m0 = sampler.lines() if sampler else 0
    a.record()
    for _ in range(n):
        fn()
    b.record()
    torch.cuda.synchronize()
    clocks = sampler.window(m0, sampler.lines()) if sampler else None
    return n, a.elapsed_time(b) / n, clocks


def roofline_record(name, bytes_launch, per_launch_ms, S, peak, peak_kind):
    avg = sum(per_launch_ms) / len(per_launch_ms)
    achieved = bytes_launch / (avg / 1e3) / 1e9
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_kind": peak_kind, "frac_of_nominal_8TBs": achieved / 8000.0, "traffic": kernel_traffic(name, S),
            "bytes_per_launch": bytes_launch, "avg_launch_ms": avg, "min_launch_ms": min(per_launch_ms)}


def add_sustained(roof, leg, torch, sampler, seconds):
    n, ms, clocks = time_sustained(torch, leg.step, roof["avg_launch_ms"], seconds, sampler)
    ach = leg.bytes_per_launch / (ms / 1e3) / 1e9
    mhz = clocks["sm_mhz"] if clocks else None
    roof["sustained"] = {"steps": n, "seconds": n * ms / 1e3, "ms_per_step": ms, "achieved": ach, "frac": ach / roof["peak"],
                         "sm_mhz_median": mhz, "ms_x_mhz": (ms * mhz) if mhz else None, "clocks": clocks}


def run_side_leg(name, args, B, torch, sampler, peak, peak_kind, candidates=False, arity=0, expanded=False):
    """One more workload, timed like the headline one: K steps, then a sustained run; its own roofline record.
    candidates: what every root child delivers (ftc_candidates_batch) instead of the batch call.
    arity: another subtree shape below the root's children (a-ary heaps; 1 = binomial trees) on the same inputs."""
    if arity:
        args = argparse.Namespace(**{**vars(args), "arity": arity})
    S = (args.batch if args.candidates and args.batch else 0) or DEFAULT_BATCH[name]
    leg = Leg(name, S, 0, args, B, torch, 28, candidates=candidates, expanded=expanded)
    for _ in range(max(args.warmup, 3)):
        leg.step()
    m0 = sampler.lines() if sampler else 0
    per_ms, total_ms = time_steps(torch, leg.step, args.steps)
    clocks = sampler.window(m0, sampler.lines()) if sampler else None
    roof = roofline_record(name, leg.bytes_per_launch, per_ms, S, peak, peak_kind)
    if candidates:
        roof["traffic"] = None
    add_sustained(roof, leg, torch, sampler, args.sustain_seconds / 2)
    ms = total_ms / args.steps
    shape = "" if not arity else " [subtrees: binomial trees]" if arity == 1 else f" [subtrees: {arity}-ary heaps]"
    if expanded:
        shape += " [expanded output: the value written into the slot of every process that holds it, zeros elsewhere]"
    rec = {"workload": f"{name}: {DESCRIPTION[name]}" + (" [what every root child delivers: all f+1 subtrees played]" if candidates else "") + shape,
           "value": S / (ms / 1e3), "unit": "scenarios/s", "ms_per_step": ms,
           "steps": args.steps, "scenarios_per_step": S, "process_rounds_per_sec": S / (ms / 1e3) * leg.w.P * leg.rounds(),
           "dtype": np.dtype(leg.w.dtype).name, "roofline": roof, "clocks": clocks}
    if candidates:
        info = leg.d_st.cpu().numpy()
        rec["kernel"] = "candidates/" + B.ftc_candidates_kernel_name(leg.desc)
        rec["subtrees_played"] = f"{leg.w.f + 1} of {leg.w.f + 1}"
        rec["children_delivering_clean"] = int((info[:, :, 0] == 0).sum())
        rec["children_with_failed_bit_or_silent"] = int((info[:, :, 0] != 0).sum())
    else:
        st = leg.status()
        rec["kernel"] = B.ftc_kernel_variant(leg.desc, leg.allred)
        rec["ok_scenarios"] = int(((st[:, 0] & 0xFF) == 0).sum())
    leg.free()
    return rec


def read_only_ceiling(B, torch, d_x, steps):
    """The library's streaming kernels over the same buffer: what a kernel that only reads can reach here."""
    nbytes = (d_x.numel() * d_x.element_size()) // 16384 * 16384
    sink = torch.zeros(2, dtype=torch.int64, device="cuda")
    out = {}
    for mode, label in ((0, "loads_128bit"), (1, "bulk_copies_to_shared")):
        for _ in range(3):
            B.ftc_read_bandwidth_probe(mode, d_x, nbytes, sink)
        per_ms, _ = time_steps(torch, lambda: B.ftc_read_bandwidth_probe(mode, d_x, nbytes, sink), max(5, min(steps, 20)))
        out[label] = nbytes / (sum(per_ms) / len(per_ms) / 1e3) / 1e9
    out["gave_up"] = int(sink[1].item())
    return out


def full_config_pass(name, args, B, torch, peak, peak_kind, steps, batch=0):
    """Every batch of configuration `name` at its stated scenario count: per batch the inputs are regenerated on the device,
    `steps` steps are timed, and the batch is checked against the any-size properties; times are summed over the batches.
    Returns (leg facts, sum of the batches' mean step times in ms, all step times, checks)."""
    from paper_2602_22445_b200 import verify
    total = CONFIG_SCENARIOS[name]
    S = batch or min(DEFAULT_BATCH[name], total)
    nb = (total + S - 1) // S
    leg = Leg(name, S, 0, args, B, torch, 28)
    sum_ms, all_ms, checks = 0.0, [], {"ok_scenarios": 0, "noop_scenarios": 0, "retried": 0, "excluded_pairs": 0}
    for b in range(nb):
        if b:
            leg.regenerate(b * S, 28)
        for _ in range(3):
            leg.step()
        per_ms, total_ms = time_steps(torch, leg.step, steps)
        sum_ms += total_ms / steps
        all_ms += per_ms
        st = leg.status()
        for k, v in verify.check_status_fields(leg.w, st).items():
            checks[k] += v
        rep = verify.check_results_by_definition(leg.w, leg.d_x, leg.d_out, st)
        checks["excluded_pairs"] += rep["excluded_pairs"]
        if "worst_relative_error" in rep:
            checks["worst_relative_error"] = max(checks.get("worst_relative_error", 0.0), rep["worst_relative_error"])
    facts = {"scenarios_total": nb * S, "batches": nb, "scenarios_per_batch": S, "bytes_per_launch": leg.bytes_per_launch,
             "kernel": B.ftc_kernel_variant(leg.desc, leg.allred), "rounds": leg.rounds(), "P": leg.w.P, "f": leg.w.f,
             "dtype": np.dtype(leg.w.dtype).name}
    leg.free()
    return facts, sum_ms, all_ms, checks


def run_full_config(args, B, torch, sampler, peak, peak_kind):
    """`--full-config`: one line for the whole configuration (see full_config_pass)."""
    name = args.workload
    facts, sum_ms, all_ms, checks = full_config_pass(name, args, B, torch, peak, peak_kind, args.steps, args.batch)
    clocks = sampler.stop() if sampler else None
    nb, S = facts["batches"], facts["scenarios_per_batch"]
    roof = roofline_record(name, facts["bytes_per_launch"], all_ms, S, peak, peak_kind)
    value = nb * S / (sum_ms / 1e3)
    line = {
        "metric": "scenarios_per_sec", "value": value, "unit": "scenarios/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": sum_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"int32": "i32", "int64": "i64", "uint64": "u64", "float32": "f32"}[facts["dtype"]], "data": "synthetic",
        "process_rounds_per_sec": value * facts["P"] * facts["rounds"],
        "config": {"workload": f"{name}: {DESCRIPTION[name]} [whole configuration]", "scenarios_total": nb * S, "batches": nb,
                   "scenarios_per_batch": S, "step": "one pass over all batches (times of the batches summed)",
                   "cache": "inputs larger than L2, no flush", "kernel": facts["kernel"],
                   "rounds_per_scenario": facts["rounds"], "subtrees_played": f"1 of {facts['f'] + 1}",
                   "checked": "every scenario: outcome and counts from the masks, result by the plain definition (torch)", **checks},
        "roofline": roof, "cpu_baseline": None, "e2e": None, "gpu_launches": args.steps * nb, "clocks": clocks,
    }
    print(json.dumps(line))


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
    peak, peak_kind = measured_peak()
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.wait_ready()
    if args.full_config:
        if world > 1:
            raise SystemExit("--full-config runs on one GPU")
        run_full_config(args, B, torch, sampler, peak, peak_kind)
        return
    if args.candidates:
        if world > 1:
            raise SystemExit("--candidates runs on one GPU")
        rec = run_side_leg(args.workload, args, B, torch, sampler, peak, peak_kind, candidates=True)
        sampler.stop()
        line = {"metric": "scenarios_per_sec", "value": rec["value"], "unit": "scenarios/s", "n_gpus": 1, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": rec["dtype"], "data": "synthetic", "process_rounds_per_sec": rec["process_rounds_per_sec"],
                "config": {"workload": rec["workload"], "scenarios_per_step_per_gpu": rec["scenarios_per_step"], "kernel": rec["kernel"],
                           "subtrees_played": rec["subtrees_played"], "cache": "inputs larger than L2, no flush"},
                "roofline": rec["roofline"], "cpu_baseline": None, "e2e": None, "gpu_launches": args.steps, "clocks": rec["clocks"]}
        print(json.dumps(line))
        return

    name = args.workload
    S = args.batch or DEFAULT_BATCH[name]
    leg = Leg(name, S, rank * S, args, B, torch, 28)                       # each rank its own scenarios
    w, desc, allred, tdt = leg.w, leg.desc, leg.allred, leg.tdt
    sched = leg.sched
    d_x, d_out, d_st = leg.d_x, leg.d_out, leg.d_st
    step = leg.step

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    if sampler:
        sampler.mark()
    per_launch_ms, total_ms = time_steps(torch, step, args.steps)
    if dist:
        dist.barrier()
    clocks = sampler.window(sampler.first, sampler.lines()) if sampler else None
    total_ms = max_over_ranks(total_ms, dist, torch.device("cuda", local))
    ms_per_step = total_ms / args.steps
    value = whole_job_value(world, S, ms_per_step)
    roof = roofline_record(name, leg.bytes_per_launch, per_launch_ms, S, peak, peak_kind)
    status = leg.status()

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
        del h_x, staging
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    launches = args.steps
    workloads, whole = {}, {}
    cpu = None
    if not args.kernel_only:
        # ---- the same step for seconds, with the clocks it ran at; and what a kernel that only reads can reach ----
        add_sustained(roof, leg, torch, sampler, args.sustain_seconds)
        launches += roof["sustained"]["steps"]
        roof["read_only_gbs"] = read_only_ceiling(B, torch, d_x, args.steps)
        roof["read_only_gbs"]["best"] = max(roof["read_only_gbs"]["loads_128bit"], roof["read_only_gbs"]["bulk_copies_to_shared"])
        roof["frac_of_read_only"] = roof["achieved"] / roof["read_only_gbs"]["best"]

        # ---- the oracle beside it, on a bounded sample played until about 4 s of wall time on all cores are done ----
        if not args.no_cpu_baseline:
            n, chunk = ORACLE_SAMPLE[name]
            n = min(n, S)
            ids = [np.arange(s, min(s + chunk, n)) for s in range(0, n, chunk)]
            xh = d_x[:n].cpu()
            xh = xh.view(torch.int64).numpy().view(np.uint64) if tdt == torch.uint64 else xh.numpy()
            prepared = (ids, [xh[i[0]:i[-1] + 1] for i in ids])
            plays, secs, cores = 0, 0.0, 1
            while secs < 4.0 and plays < 64:
                _, dt, cores = time_oracle(w, prepared)
                plays += 1
                secs += dt
            cpu = {"value": plays * n / secs, "unit": "scenarios/s", "cores": cores, "kind": "oracle",
                   "sample": f"first {n} scenarios of the workload, played {plays} times ({secs:.1f} s wall on {cores} threads)"}
        leg.free()
        del d_x, d_out, d_st

        # ---- the other configurations the target names, each timed the same way (one GPU only) ----
        if world == 1 and not args.no_legs:
            for other in [x for x in ("c5", "c5r", "c3", "c4", "c2") if x != name]:
                workloads[other] = run_side_leg(other, args, B, torch, sampler, peak, peak_kind)
                launches += args.steps + workloads[other]["roofline"]["sustained"]["steps"]
            for other, ar, tag in (("c4", 4, "c4_4ary"), ("c4", 1, "c4_binomial")):     # other I(f)-tree shapes on the same inputs
                workloads[tag] = run_side_leg(other, args, B, torch, sampler, peak, peak_kind, arity=ar)
                workloads[tag]["roofline"]["traffic"] = None
                launches += args.steps + workloads[tag]["roofline"]["sustained"]["steps"]
            workloads["c4_expanded"] = run_side_leg("c4", args, B, torch, sampler, peak, peak_kind, expanded=True)
            workloads["c4_expanded"]["roofline"]["traffic"] = None
            launches += 2 * (args.steps + workloads["c4_expanded"]["roofline"]["sustained"]["steps"])     # two kernels a step
            for other in ("c4", "c5"):                      # all f+1 root children played (integer configurations)
                key = other + "_all_children"
                workloads[key] = run_side_leg(other, args, B, torch, sampler, peak, peak_kind, candidates=True)
                launches += args.steps + workloads[key]["roofline"]["sustained"]["steps"]
        # ---- the configurations at their stated scenario counts: every batch played and checked, times summed ----
        if world == 1 and not args.no_legs and not args.no_whole:
            for cfg in ("c4", "c5", "c3"):
                facts, sum_ms, all_ms, checks = full_config_pass(cfg, args, B, torch, peak, peak_kind, 3)
                gbs = facts["bytes_per_launch"] * facts["batches"] / (sum_ms / 1e3) / 1e9
                whole[cfg] = {"scenarios_total": facts["scenarios_total"], "batches": facts["batches"], "steps_per_batch": 3,
                              "ms_all_batches": sum_ms, "scenarios_per_sec": facts["scenarios_total"] / (sum_ms / 1e3),
                              "achieved_gbs": gbs, "frac": gbs / peak, "kernel": facts["kernel"],
                              "checked": "every scenario: outcome and counts from the masks, result by the plain definition (torch)", **checks}
                launches += 6 * facts["batches"]
    if sampler:
        sampler.stop()

    R = leg.rounds()
    line = {
        "metric": "scenarios_per_sec", "value": value, "unit": "scenarios/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"int32": "i32", "int64": "i64", "uint64": "u64", "float32": "f32"}[np.dtype(w.dtype).name],
        "data": "synthetic",
        "process_rounds_per_sec": value * w.P * R,
        "config": {"workload": f"{name}: {DESCRIPTION[name]}" + (f" [collective={args.collective}]" if args.collective else "")
                   + (" [failure-free]" if args.failure_free else ""), "scenarios_per_step_per_gpu": S,
                   "input_bytes_per_step_per_gpu": S * w.P * w.k * ESZ[np.dtype(w.dtype).name],
                   "cache": "inputs larger than L2, no flush", "kernel": B.ftc_kernel_variant(desc, allred),
                   "rounds_per_scenario": R, "subtrees_played": f"1 of {w.f + 1} (the child the root selects; "
                   "process_rounds_per_sec counts P x rounds per scenario as the schedule has them)",
                   "scenarios_of_the_configuration": CONFIG_SCENARIOS[name],
                   "ok_scenarios": int(((status[:, 0] & 0xFF) == 0).sum())},
        "roofline": roof,
        "workloads": workloads,
        "cpu_baseline": cpu,
        "e2e": e2e,
        "gpu_launches": args.steps,
        "whole_configurations": whole, "launches_all_legs": launches,
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
    ap.add_argument("--kernel", default="auto", choices=["auto", "direct", "generic", "levels"], help="force a kernel family")
    ap.add_argument("--arity", type=int, default=0, help="subtrees below the root's children as a-ary heaps, 1 = binomial trees (diagnostic: 0 = the binary heap of the configurations)")
    ap.add_argument("--collective", default="", choices=["", "reduce", "allreduce"], help="override the workload's collective")
    ap.add_argument("--failure-free", action="store_true", help="clear every failure of the workload (diagnostic)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel-only", action="store_true", help="skip the end-to-end, sustained, CPU and other-workload legs (for profiler runs)")
    ap.add_argument("--no-legs", action="store_true", help="skip the legs over the other configurations")
    ap.add_argument("--no-whole", action="store_true", help="skip the pass over every batch of C3, C4 and C5 at their stated scenario counts")
    ap.add_argument("--sustain-seconds", type=float, default=2.0, help="GPU time of the sustained run of the headline workload")
    ap.add_argument("--candidates", action="store_true",
                    help="time ftc_candidates_batch (what every root child delivers: all f+1 subtrees) on the workload")
    ap.add_argument("--full-config", action="store_true",
                    help="play every batch of the configuration (its stated scenario count), checking every scenario")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
