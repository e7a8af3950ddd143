#!/usr/bin/env python
"""Benchmark of the batched schedule builder + evaluator (one step = one pass of the whole hot
path over one batch of seeded synthetic instances).  Prints ONE JSON line on rank 0.

    python bench.py --gpus 1 --steps 5 --warmup 3            # config 5, the workload the target is quoted on
    python bench.py --workload c1|c2|c3|c4|c5|c2d|c2s|bounds # the other configs: c4 = the (tau, k) sweep, c2d = dynamic refill, c2s = speculative runs
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference                         # the CPU oracle, as it stands, on a bounded sample
"""
from __future__ import annotations

import argparse
import csv
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_22996_b200 import workloads  # noqa: E402

METRIC, UNIT = "schedule_evaluation_job_steps_per_sec", "job-steps/s"
WORKLOADS = {
    # name: (generator, instances, jobs per instance, families, description)
    "c1": ("config1", 1, 1_000, ["GBA", "GSA", "SPS", "SIMS"], "config 1: one instance of 1,000 jobs, M = 200,000, four families, full outputs"),
    "c2": ("config2", 1024, 10_000, ["GBA", "GSA"], "config 2: 1,024 instances x 10,000 jobs, M in {2^17..2^24}, GBA+GSA"),
    "c3": ("config3", 256, 100_000, ["GBA", "GSA"], "config 3: 256 instances x 100,000 jobs, online arrivals, estimates, M=2^22"),
    "c4": ("config4", 1, 1_000_000, ["SPS", "SIMS"], "config 4: one instance of 1,000,000 jobs, 64 x 64 (tau, k) grid, SPS and SimS, scalars only"),
    "c5": ("config5", 16_384, 50_000, ["GBA", "GSA", "SPS", "SIMS"], "config 5 (stress): 16,384 instances x 50,000 jobs, mixed distributions, M per instance, four families"),
    "c2d": ("config2", 1024, 10_000, ["GBAD"], "config 2's instances and budgets under GBA with dynamic refill (GBA-D): batching schedule, then the refill kernel"),
    "c2s": ("config2", 1024, 10_000, ["GSAS"], "config 2's instances and budgets under GSA with speculative runs (GSA-Spec): slicing schedule, then the round-by-round kernel"),
    "bounds": ("config2", 1024, 10_000, ["GBA"], "class-size bounds (kvs_bounds) on config 2's instances and budgets"),
}
# The sweep is bound by integer arithmetic on inputs that stay in L2: per candidate round (one per run and
# setting) the kernel spends about this many integer instructions (counted in the inner loop of k_sweep: window
# update, two multiply-high divisions, compare and max), against the issue rate of the SMs.
SWEEP_OPS_PER_CANDIDATE = 40
SM_COUNT, WARP_ISSUE_PER_CLK, LANES = 148, 4, 32


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=sorted(WORKLOADS))
    ap.add_argument("--instances", type=int, default=0, help="override the number of instances (0 = the config's)")
    ap.add_argument("--families", default="", help="comma-separated subset of the workload's families (diagnostic)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--ncu-traffic", default=os.path.join(ROOT, "profiles", "k_fused_eval_c5_traffic.csv"),
                    help="csv of `ncu --csv --page raw` with dram__bytes_read.sum / dram__bytes_write.sum of the dominant kernel's launches on a "
                         "small case of config 5, headed by a line `# evaluations=<n> kvs_fused_sha256=<hash of csrc/kvs_fused.cu at the capture>`; "
                         "used only while that source file is unchanged")
    return ap.parse_args()


def make_instances(name: str, n_inst: int, device, first_instance: int = 0):
    """Seeded instances of the named config, generated in chunks to bound temporaries."""
    gen, _, n, _, _ = WORKLOADS[name]
    fn = getattr(workloads, gen)
    if gen in ("config1", "config4"):
        return fn(device=device)
    chunk = max(1, (1 << 25) // n)
    parts = []
    for lo in range(0, n_inst, chunk):
        c = min(chunk, n_inst - lo)
        parts.append(fn(n_inst=c, n=n, device=device, first_instance=first_instance + lo))
    cat = lambda f: None if getattr(parts[0], f) is None else torch.cat([getattr(p, f) for p in parts])
    off = torch.arange(n_inst + 1, dtype=torch.int64, device=device) * n
    meta = dict(parts[0].meta)
    if "M_per_instance" in meta:
        meta["M_per_instance"] = torch.cat([p.meta["M_per_instance"] for p in parts])
    return workloads.Instances(off, cat("s"), cat("o"), cat("o_est"), cat("arrival"), meta)


def make_settings(name: str, inst, fams=None):
    from paper_2601_22996_b200 import binding
    fams = fams or WORKLOADS[name][3]
    I = inst.n_instances
    if "M_per_instance" in inst.meta:
        Ms = inst.meta["M_per_instance"].cpu().numpy()[:, None]
    else:
        Ms = inst.meta["M"]
    return binding.settings_grid(range(I), fams, Ms), int(inst.meta.get("window", 0))


def stores_profile(name: str, family: int) -> bool:
    """Which evaluations of a workload get a per-round profile in the timed step.  The SPS / SimS schedules of
    config 5 reach 10^7 to 10^8 rounds each (tens of terabytes for all of them), so their peak comes from the
    run ends and no profile is stored; everything else stores its profile."""
    return not (name == "c5" and family >= 2)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.rows, self.proc, self.index = [], None, device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.rows.append([x.strip() for x in ln.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        mhz = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 9 for i in range(4) if r[5 + i].lower().startswith("active")})
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(mhz)}


# ---- the oracle as CPU baseline -------------------------------------------------------------------

def oracle_tasks(name: str, inst_cpu, settings, window: int):
    """The workload's evaluations as plain task dicts for oracle.timing (numpy views, no torch in the workers).
    An evaluation that stores no profile on the GPU takes the event evaluator here too: like for like."""
    npv = lambda t: None if t is None else t.numpy()
    s, o, est, arr, off = npv(inst_cpu.s), npv(inst_cpu.o), npv(inst_cpu.o_est), npv(inst_cpu.arrival), inst_cpu.job_off.numpy()
    if name == "c4":
        taus, ks = workloads.sweep_grids()
        M = inst_cpu.meta["M"][0]
        return [dict(family=fam, s=s, o=o, M=M, tau=t, k=k, s_bar=0, profile=False) for fam in ("SPS", "SIMS") for t in taus for k in ks]
    tasks = []
    for e in range(settings.shape[0]):
        st = settings[e]
        i = int(st["instance"])
        if i >= inst_cpu.n_instances:
            break
        a, b = int(off[i]), int(off[i + 1])
        tasks.append(dict(family=int(st["family"]), s=s[a:b], o=o[a:b], est=None if est is None else est[a:b],
                          arrival=None if arr is None else arr[a:b], window=window, M=int(st["M"]),
                          alpha=(int(st["alpha_num"]), int(st["alpha_den"])), profile=stores_profile(name, int(st["family"]))))
    return tasks


def cpu_baseline(name: str, inst_cpu, settings, window: int, budget_s: float) -> dict:
    """The oracle on one core, then the same single-threaded code on every host core over disjoint evaluations."""
    from oracle import timing
    tasks = oracle_tasks(name, inst_cpu, settings, window)
    steps1, ev1, dt1 = timing.run(tasks, budget_s / 3)
    cores = max(1, min(timing.host_cores(), len(tasks)))
    if name == "c4":
        rng = np.random.default_rng(4)       # cells differ a lot in cost: a seeded shuffle spreads them
        tasks = [tasks[i] for i in rng.permutation(len(tasks))]
    steps, ev, dt, used = timing.run_parallel([tasks[c::cores] for c in range(cores)], 2 * budget_s / 3)
    return {"value": steps / dt, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": f"{ev} evaluations of this workload spread over {used} processes (one per host core), {dt:.1f} s",
            "single_core": {"value": steps1 / dt1, "cores": 1, "sample": f"first {ev1} evaluations of this workload, {dt1:.1f} s"}}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def ncu_traffic(path: str, kernel_substr: str):
    """(dram__bytes_read.sum + dram__bytes_write.sum over the rows of an ncu raw csv whose kernel name contains
    `kernel_substr`, evaluations those launches processed), or None if the file is missing, holds no such row, or
    was captured from another state of the kernel's source."""
    import hashlib
    import re
    if not path or not os.path.exists(path):
        return None
    with open(path, newline="") as f:
        first = f.readline()
        m = re.match(r"#\s*evaluations=(\d+)\s+kvs_fused_sha256=([0-9a-f]+)", first)
        if not m:
            return None
        with open(os.path.join(ROOT, "paper_2601_22996_b200", "csrc", "kvs_fused.cu"), "rb") as src:
            if hashlib.sha256(src.read()).hexdigest() != m.group(2):
                return None                      # the kernel has changed since the counters were taken
        evals = int(m.group(1))
        rows = [r for r in csv.reader(f) if r]
    head = next((i for i, r in enumerate(rows) if "Kernel Name" in r), None)
    if head is None or head + 2 > len(rows):
        return None
    h, units = rows[head], rows[head + 1]
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    total, seen = 0.0, False
    for r in rows[head + 2:]:
        if len(r) != len(h) or kernel_substr not in r[h.index("Kernel Name")]:
            continue
        for col in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            if col in h:
                total += float(r[h.index(col)].replace(",", "")) * scale.get(units[h.index(col)], 1.0)
                seen = True
    return (total, evals) if seen and evals > 0 else None


def run_reference(args):
    """The CPU oracle on a bounded sample of the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import timing
    name = args.workload
    n_sample = {"c1": 1, "c3": 2, "c4": 1}.get(name, 32)
    inst = make_instances(name, n_sample, "cpu")
    settings, window = make_settings(name, inst)
    tasks = oracle_tasks(name, inst, settings, window)
    per = []
    steps_total = evals_total = 0
    for _ in range(args.warmup + args.steps):
        steps, evals, dt = timing.run(tasks, args.cpu_seconds)
        per.append(dt)
        steps_total, evals_total = steps, evals
    timed = per[args.warmup:]
    t = sum(timed)
    value = steps_total * len(timed) / t
    sample = f"first {evals_total} evaluations ({n_sample} instances) of {WORKLOADS[name][4]}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / len(timed), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic (seeded)",
        "config": {"workload": WORKLOADS[name][4], "sample": sample},
        "evaluations_per_sec": evals_total * len(timed) / t,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ---- the CUDA path ------------------------------------------------------------------------------------

def run_sweep(args, rank, world, dev, local, dist):
    """Config 4: one step = the 64 x 64 (tau, k) grid for SPS and for SimS on one instance of 10^6 jobs."""
    from paper_2601_22996_b200.api import Scheduler
    name = "c4"
    fams = [f for f in args.families.split(",") if f] or WORKLOADS[name][3]
    inst_cpu = make_instances(name, 1, "cpu")
    inst = inst_cpu.to(dev)
    taus, ks = workloads.sweep_grids()
    M = inst_cpu.meta["M"][0]
    n = int(inst.s.numel())
    sched = Scheduler(local)

    def step():
        return [sched.sweep(inst, 0, f, M, taus, ks) for f in fams]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        outs = step()
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = e0.elapsed_time(e1)
    job_steps = int(sum(int(o["job_steps"].sum()) for o in outs))
    cells = len(taus) * len(ks) * len(fams)
    e2e = None
    if not args.no_e2e:
        hs, ho, hoff = inst_cpu.s.pin_memory(), inst_cpu.o.pin_memory(), inst_cpu.job_off.pin_memory()
        ds, do_, doff = torch.empty_like(inst.s), torch.empty_like(inst.o), torch.empty_like(inst.job_off)
        dinst = workloads.Instances(doff, ds, do_)
        barrier()
        t0 = time.perf_counter()
        d2h = 0
        for _ in range(args.steps):
            ds.copy_(hs, non_blocking=True)
            do_.copy_(ho, non_blocking=True)
            doff.copy_(hoff, non_blocking=True)
            res = [sched.sweep(dinst, 0, f, M, taus, ks) for f in fams]
            host = [{k: v.cpu() for k, v in r.items()} for r in res]
            d2h = sum(v.numel() * v.element_size() for r in host for v in r.values())
        e2e = (time.perf_counter() - t0, 8 * n + 16, d2h)
    stats = torch.tensor([ms, e2e[0] if e2e else 0.0], dtype=torch.float64, device=dev)
    tot = torch.tensor([float(job_steps), float(cells)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(stats, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    if rank != 0:
        return
    ms, e2e_s = [float(x) for x in stats.tolist()]
    steps_all, cells_all = tot.tolist()
    sec = ms / 1e3 / args.steps
    sm_hz = (clocks.get("sm_mhz") or 1965.0) * 1e6
    peak_ops = SM_COUNT * WARP_ISSUE_PER_CLK * LANES * sm_hz
    achieved = cells * n * SWEEP_OPS_PER_CANDIDATE / sec
    line = {
        "metric": METRIC, "value": steps_all / sec, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * sec, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic (seeded)",
        "config": {"workload": WORKLOADS[name][4], "jobs_per_instance": n, "settings_per_gpu": cells, "M": M,
                   "profile": "none (scalars per setting; the peak comes from the run ends)",
                   "l2": "inputs (16 MB) stay in L2 by design: every setting re-reads them; outputs are 6 scalars per setting"},
        "evaluations_per_sec": cells_all / sec,
        "roofline": {"bound": "alu", "achieved": achieved / 1e12, "peak": peak_ops / 1e12, "unit": "T integer instructions/s",
                     "frac": achieved / peak_ops, "traffic": None, "kernel": "k_sweep",
                     "peak_kind": "148 SMs x 4 warp instructions per clock x 32 lanes at the sampled SM clock",
                     "ops_per_candidate": SWEEP_OPS_PER_CANDIDATE, "candidates_per_step": cells * n},
        "gpu_launches": 5 * len(fams) * args.steps, "clocks": clocks,
    }
    if e2e:
        line["e2e"] = {"value": steps_all / (e2e_s / args.steps), "unit": UNIT, "h2d_bytes_per_step": e2e[1], "d2h_bytes_per_step": e2e[2],
                       "result": "six scalars per setting"}
    if not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(name, inst_cpu, None, 0, args.cpu_seconds)
    print(json.dumps(line))


def run_bounds(args, rank, world, dev, local):
    """kvs_bounds on config 2's instances under its eight budgets (not on the benchmarked path; timed for the record)."""
    from paper_2601_22996_b200.api import Scheduler
    name = "bounds"
    I = args.instances or WORKLOADS[name][1]
    n = WORKLOADS[name][2]
    inst = make_instances(name, I, dev, first_instance=rank * I)
    settings, _ = make_settings(name, inst)
    sched = Scheduler(local)
    for _ in range(args.warmup):
        sched.bounds(inst, settings)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        out = sched.bounds(inst, settings)
    e1.record()
    torch.cuda.synchronize()
    sec = e0.elapsed_time(e1) / 1e3 / args.steps
    assert int((out["status"] != 0).sum()) == 0
    P = settings.shape[0]
    peak_gbs, peak_kind = load_peaks()
    alg = 4.0 * n * P + 8.0 * n * I            # the response lengths once per evaluation; s and o once for the statistics
    if rank == 0:
        print(json.dumps({"metric": "bound_evaluation_jobs_per_sec", "value": P * n / sec, "unit": "jobs/s", "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": 1e3 * sec, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "dtype": "int64/int128", "data": "synthetic (seeded)",
                          "config": {"workload": WORKLOADS[name][4], "instances_per_gpu": I, "jobs_per_instance": n, "evaluations_per_gpu": P},
                          "evaluations_per_sec": P / sec,
                          "roofline": {"bound": "hbm", "achieved": alg / sec / 1e9, "peak": peak_gbs, "unit": "GB/s", "frac": alg / sec / 1e9 / peak_gbs,
                                       "traffic": None, "peak_kind": peak_kind, "kernel": "k_bounds (+ statistics pass)", "algorithmic_bytes": alg},
                          "gpu_launches": 2 * args.steps}))


def run_ours(args):
    import torch.distributed as dist
    from paper_2601_22996_b200 import binding
    from paper_2601_22996_b200.api import Scheduler

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the schedule builder has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    try:
        if args.workload == "c4":
            return run_sweep(args, rank, world, dev, local, dist)
        if args.workload == "bounds":
            return run_bounds(args, rank, world, dev, local)
        return run_fused_workload(args, rank, world, dev, local, dist, binding, Scheduler)
    finally:
        if world > 1:
            dist.destroy_process_group()


def run_fused_workload(args, rank, world, dev, local, dist, binding, Scheduler):
    name = args.workload
    I = args.instances or WORKLOADS[name][1]
    n = WORKLOADS[name][2]
    fams = [f for f in args.families.split(",") if f] or WORKLOADS[name][3]

    # weak scaling: every rank gets its own I instances (different seeds), no data-path collective
    inst = make_instances(name, I, dev, first_instance=rank * I)
    settings, window = make_settings(name, inst, fams)
    P = settings.shape[0]
    N = I * n
    sched = Scheduler(local)
    ctx = sched.context(binding.workspace_bytes(N, I, n, P, host_staging=not args.no_e2e))

    # sizes: one scalar-only pass gives every horizon
    first = Scheduler.scalars(P, dev)
    ctx.build_schedule(inst, settings, dict(n_runs=torch.zeros(P, dtype=torch.int64, device=dev)), first, window=window, max_jobs=n)
    with_prof = torch.from_numpy(np.array([stores_profile(name, int(f)) for f in settings["family"]])).to(dev)
    cap = torch.where(with_prof, first["horizon"], torch.zeros_like(first["horizon"]))
    poff = torch.zeros(P + 1, dtype=torch.int64, device=dev)
    poff[1:] = torch.cumsum(cap, 0)
    job_off = torch.arange(P + 1, dtype=torch.int64, device=dev) * n
    out = dict(job_out_off=job_off, job_start=torch.empty(P * n, dtype=torch.int32, device=dev),
               job_completion=torch.empty(P * n, dtype=torch.int32, device=dev),
               n_runs=torch.zeros(P, dtype=torch.int64, device=dev))
    ev = Scheduler.scalars(P, dev)
    ev["profile_off"] = poff
    ev["profile"] = torch.empty(int(poff[-1]), dtype=torch.int32, device=dev)
    rounds = int(poff[-1])

    def step():
        ctx.evaluate_built(inst, settings, out, ev, window=window, max_jobs=n)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    ctx.set_timing(True)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = e0.elapsed_time(e1)
    # kernel durations (CUDA events recorded by the library on its stream around each kernel)
    sort_ms, build_ms, light_ms, full_ms = [], [], [], []
    for _ in range(args.steps):
        step()
        a, b = ctx.last_timing()
        _, c, d = ctx.last_timing_split()
        sort_ms.append(a)
        build_ms.append(b)
        light_ms.append(c)
        full_ms.append(d)
    ctx.set_timing(False)
    assert int((ev["status"] != 0).sum()) == 0, "an evaluation reported a non-zero status"
    job_steps = int(ev["job_steps"].sum())
    job_steps_prof = int(ev["job_steps"][with_prof].sum())

    # end to end through the host entry point: pinned host inputs in, scalars out
    e2e = None
    if not args.no_e2e:
        hin = workloads.Instances(inst.job_off.cpu().pin_memory(), inst.s.cpu().pin_memory(), inst.o.cpu().pin_memory(),
                                  None if inst.o_est is None else inst.o_est.cpu().pin_memory(),
                                  None if inst.arrival is None else inst.arrival.cpu().pin_memory())
        hev = {k: torch.zeros_like(v, device="cpu").pin_memory() for k, v in Scheduler.scalars(P, "cpu").items()}
        # The refill and the speculative runs work in the per-job results and the profile on the device, which the
        # host entry point does not allocate: their end-to-end step copies the pinned inputs to the device, calls
        # the device entry point and copies the scalars back.
        on_device = bool(np.isin(settings["family"], [binding.FAMILY[f] for f in ("GBAD", "GSAS") if f in binding.FAMILY]).any())

        def e2e_step():
            if not on_device:
                ctx.evaluate_built_host(hin, settings, hev, window=window, max_jobs=n)
                return
            din = workloads.Instances(*[None if x is None else x.to(dev, non_blocking=True)
                                        for x in (hin.job_off, hin.s, hin.o, hin.o_est, hin.arrival)])
            ctx.evaluate_built(din, settings, out, ev, window=window, max_jobs=n)
            for k2, v2 in hev.items():
                v2.copy_(ev[k2], non_blocking=True)
            torch.cuda.synchronize()

        e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            e2e_step()
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        assert int(hev["job_steps"].sum()) == job_steps
        h2d = sum(t.numel() * t.element_size() for t in (hin.job_off, hin.s, hin.o, hin.o_est, hin.arrival) if t is not None)
        h2d += settings.nbytes
        d2h = sum(t.numel() * t.element_size() for t in hev.values())
        e2e = (e2e_s, h2d, d2h)

    # max over ranks, totals over ranks
    stats = torch.tensor([ms, e2e[0] if e2e else 0.0, float(np.mean(build_ms)), float(np.mean(sort_ms)),
                          float(np.mean(light_ms)), float(np.mean(full_ms))], dtype=torch.float64, device=dev)
    tot = torch.tensor([float(job_steps), float(P), float(job_steps_prof)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(stats, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    if rank != 0:
        return
    ms, e2e_s, build_avg, sort_avg, light_avg, full_avg = [float(x) for x in stats.tolist()]
    steps_all, evals_all, steps_prof_all = tot.tolist()
    sec_per_step = ms / 1e3 / args.steps
    share = len(fams) * (len(inst.meta["M"]) if "M" in inst.meta and name == "c2" else 1)
    # Dominant kernel: the full variant of k_fused_eval, which takes the evaluations whose rounds are walked
    # (the GBA / GSA ones; with estimates or wanted profiles also SPS / SimS).  Its algorithmic bytes on this
    # rank: the instances once, start + completion per job and evaluation, one int32 per profile round,
    # scalars.  (`stage_algorithmic_bytes` adds the evaluations of the light variant.)
    walked = int(with_prof.sum())
    alg_bytes = (8 * N if walked else 0) + 8 * walked * n + 4 * rounds + 57 * walked
    stage_bytes = 8 * N + 8 * P * n + 4 * rounds + 57 * P
    peak_gbs, peak_kind = load_peaks()
    achieved = alg_bytes / (full_avg * 1e-3) / 1e9 if walked and full_avg > 0 else 0.0
    traffic = None
    captured = ncu_traffic(args.ncu_traffic, "k_fused_eval<0") if name == "c5" else None   # the full variant's launches of the captured small case
    if captured is not None:
        traffic = captured[0] / captured[1] * walked                  # traffic grows with the evaluations: each CTA holds one at a time
    # kernels of one kvs_evaluate_built call: ordering kernel; without estimates one launch of the light
    # variant per SPS / SimS family and one of the full variant per geometric family (with estimates one of
    # each for all families); the full variant for what the light one passes on; the general kernel on the
    # left-over list
    n_light_fams = sum(f in ("SPS", "SIMS") for f in fams)
    n_geo_fams = sum(f in ("GBA", "GSA", "GBAD", "GSAS") for f in fams)
    n_post = sum(f in fams for f in ("GBAD", "GSAS"))     # k_refill / k_spec after the fused kernels
    if inst.o_est is None:
        launches_per_step = 1 + n_light_fams + n_geo_fams + int(n_light_fams > 0) + 1 + n_post
    else:
        launches_per_step = 1 + int(n_light_fams > 0) + int(n_light_fams + n_geo_fams > 0) + 1
    prof_note = ("every evaluation stores its per-round profile" if walked == P else
                 "GBA/GSA evaluations store their per-round profile; the SPS/SimS schedules of this config reach 10^7-10^8 rounds each: "
                 "their peak comes from the run ends and no profile is stored")
    out_bytes = 8 * P * n + 4 * rounds
    line = {
        "metric": METRIC, "value": steps_all / sec_per_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sec_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32/int64", "data": "synthetic (seeded)",
        "config": {"workload": WORKLOADS[name][4], "instances_per_gpu": I, "jobs_per_instance": n,
                   "evaluations_per_gpu": P, "evaluations_sharing_an_instance": share, "alpha": "2/1",
                   "profile": prof_note, "profile_rounds_per_gpu": rounds,
                   "l2": ("inputs and outputs larger than L2" if 8 * N > 126e6 else
                          "outputs of a step larger than L2 (inputs smaller)" if out_bytes > 126e6 else
                          "working set of the config as specified is smaller than L2; no flush")},
        "evaluations_per_sec": evals_all / sec_per_step,
        "job_steps_per_sec_split": {"with_stored_profile": steps_prof_all / sec_per_step,
                                    "scalars_only_peak_from_run_ends": (steps_all - steps_prof_all) / sec_per_step},
        "kernels_ms": {"k_stats_sort": sort_avg, "k_fused_eval<light>": light_avg,
                       ("k_fused_eval<full>+k_build_eval+" + ("k_refill" if "GBAD" in fams else "k_spec") if n_post else
                        "k_fused_eval<full>+k_build_eval"): full_avg,
                       "builder_evaluator_stage": build_avg},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak_gbs, "unit": "GB/s", "frac": achieved / peak_gbs,
                     "traffic": traffic, "peak_kind": peak_kind, "kernel": "k_fused_eval<full>", "algorithmic_bytes": alg_bytes,
                     "stage_algorithmic_bytes": stage_bytes, "stage_frac": stage_bytes / (build_avg * 1e-3) / 1e9 / peak_gbs,
                     "step_frac": stage_bytes / sec_per_step / 1e9 / peak_gbs},
        "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
    }
    if traffic is not None and full_avg > 0:
        # the measured DRAM traffic of the same launches over their duration: what the memory system actually sustained
        line["roofline"]["dram_gbs"] = traffic / (full_avg * 1e-3) / 1e9
        line["roofline"]["dram_frac"] = line["roofline"]["dram_gbs"] / peak_gbs
    if n_post:
        post = "k_refill" if "GBAD" in fams else "k_spec"
        line["roofline"]["kernel"] = "k_fused_eval<full> + " + post + " (timed together)"
        line["roofline"]["note"] = (post + " applies a sequential rule per evaluation, one warp each: it is bound by the latency of "
                                    "dependent loads, and the HBM fraction is given for completeness only")
    if e2e:
        line["e2e"] = {"value": steps_all / (e2e_s / args.steps), "unit": UNIT, "h2d_bytes_per_step": e2e[1], "d2h_bytes_per_step": e2e[2],
                       "result": "scalars only (no per-job results and no profile leave the device on this path)"}
    if not args.no_cpu:
        n_s = {"c1": 1, "c3": 16}.get(name, 2048)    # upper bound; the time budget ends the sample earlier
        cpu_inst = inst.slice(0, min(n_s, I)).to("cpu")
        cpu_inst.meta = dict(inst.meta)
        line["cpu_baseline"] = cpu_baseline(name, cpu_inst, settings, window, args.cpu_seconds)
    print(json.dumps(line))


if __name__ == "__main__":
    a = parse_args()
    run_reference(a) if a.impl == "reference" else run_ours(a)
