#!/usr/bin/env python
"""Benchmark of the batched schedule builder + evaluator (one step = one pass of the whole hot
path over one batch of seeded synthetic instances).  Prints ONE JSON line on rank 0.

    python bench.py --gpus 1 --steps 5 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference      # the CPU oracle, as it stands, on a bounded sample
"""
from __future__ import annotations

import argparse
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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, the full variant of
# k_fused_eval (it takes the geometric evaluations), from the ncu capture summarised in
# profiles/k_fused_eval_c5.md (592 instances of config 5: 1,184 GBA/GSA evaluations, 3.418 GB, the launches of the two families together).
# Traffic grows with the number of evaluations (each CTA works on one at a time), so a launch is scaled
# by its evaluation count.  Valid for the kernel state named in that file; set to None when the kernel changes.
C5_TRAFFIC_BYTES_PER_GEOMETRIC_EVALUATION = 3.418012e9 / 1184
WORKLOADS = {
    # name: (generator, instances, jobs per instance, families, description)
    "c2": ("config2", 1024, 10_000, ["GBA", "GSA"], "config 2: 1,024 instances x 10,000 jobs, M in {2^17..2^24}, GBA+GSA"),
    "c3": ("config3", 256, 100_000, ["GBA", "GSA"], "config 3: 256 instances x 100,000 jobs, online arrivals, estimates, M=2^22"),
    "c5": ("config5", 16_384, 50_000, ["GBA", "GSA", "SPS", "SIMS"], "config 5 (stress): 16,384 instances x 50,000 jobs, mixed distributions, M per instance, four families"),
}


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
    return ap.parse_args()


def make_instances(name: str, n_inst: int, device, first_instance: int = 0):
    """Seeded instances of the named config, generated in chunks to bound temporaries."""
    gen, _, n, _, _ = WORKLOADS[name]
    fn = getattr(workloads, gen)
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


def oracle_sample(name: str, inst_cpu, settings, window: int, budget_s: float):
    """Times the oracle, as it stands, on the first evaluations of the workload until the budget is spent."""
    import oracle
    from tests.parity import oracle_eval
    t0 = time.perf_counter()
    steps = evals = 0
    for e in range(settings.shape[0]):
        if int(settings[e]["instance"]) >= inst_cpu.n_instances:
            break
        S = oracle_eval(inst_cpu, settings[e], window)
        if S.horizon <= 60_000_000:
            E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s, want_profile=False)
        else:
            E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
        assert E.job_steps == S.job_steps
        steps += S.job_steps
        evals += 1
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return steps, evals, dt


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def run_reference(args):
    """The CPU oracle on a bounded sample of the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    name = args.workload
    n_sample = 32 if name != "c3" else 2
    inst = make_instances(name, n_sample, "cpu")
    settings, window = make_settings(name, inst)
    per = []
    steps_total = evals_total = 0
    for _ in range(args.warmup + args.steps):
        steps, evals, dt = oracle_sample(name, inst, settings, window, budget_s=args.cpu_seconds)
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

    # sizes: one scalar-only pass gives every horizon; geometric families get their profile
    first = Scheduler.scalars(P, dev)
    ctx.build_schedule(inst, settings, dict(n_runs=torch.zeros(P, dtype=torch.int64, device=dev)), first, window=window, max_jobs=n)
    geo = torch.from_numpy(settings["family"] <= 1).to(dev)
    cap = torch.where(geo, first["horizon"], torch.zeros_like(first["horizon"]))
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

    # end to end through the host entry point: pinned host inputs in, scalars out
    e2e = None
    if not args.no_e2e:
        hin = workloads.Instances(inst.job_off.cpu().pin_memory(), inst.s.cpu().pin_memory(), inst.o.cpu().pin_memory(),
                                  None if inst.o_est is None else inst.o_est.cpu().pin_memory(),
                                  None if inst.arrival is None else inst.arrival.cpu().pin_memory())
        hev = {k: torch.zeros_like(v, device="cpu").pin_memory() for k, v in Scheduler.scalars(P, "cpu").items()}
        ctx.evaluate_built_host(hin, settings, hev, window=window, max_jobs=n)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            ctx.evaluate_built_host(hin, settings, hev, window=window, max_jobs=n)
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
    tot = torch.tensor([float(job_steps), float(P)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(stats, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    ms, e2e_s, build_avg, sort_avg, light_avg, full_avg = [float(x) for x in stats.tolist()]
    steps_all, evals_all = tot.tolist()
    sec_per_step = ms / 1e3 / args.steps
    share = len(fams) * (len(inst.meta["M"]) if "M" in inst.meta and name == "c2" else 1)
    # Dominant kernel: the full variant of k_fused_eval, which takes the geometric (GBA/GSA) evaluations.
    # Its algorithmic bytes on this rank: the instances once, start + completion per job and evaluation,
    # one int32 per profile round, scalars.  (The light variant does the same for SPS / SimS without
    # profile rounds; `stage_algorithmic_bytes` is the figure for both together.)
    geo = int((settings["family"] <= 1).sum())
    alg_bytes = (8 * N if geo else 0) + 8 * geo * n + 4 * rounds + 57 * geo
    stage_bytes = 8 * N + 8 * P * n + 4 * rounds + 57 * P
    peak_gbs, peak_kind = load_peaks()
    achieved = alg_bytes / (full_avg * 1e-3) / 1e9 if geo else 0.0
    traffic = None
    if name == "c5" and geo and C5_TRAFFIC_BYTES_PER_GEOMETRIC_EVALUATION:
        traffic = C5_TRAFFIC_BYTES_PER_GEOMETRIC_EVALUATION * geo
    # kernels of one kvs_evaluate_built call: ordering kernel; without estimates one launch of the light
    # variant per SPS / SimS family and one of the full variant per geometric family (with estimates one of
    # each for all families); the full variant for what the light one passes on; the general kernel on the
    # left-over list
    n_light_fams = sum(f in ("SPS", "SIMS") for f in fams)
    n_geo_fams = sum(f in ("GBA", "GSA") for f in fams)
    if inst.o_est is None:
        launches_per_step = 1 + n_light_fams + n_geo_fams + int(n_light_fams > 0) + 1
    else:
        launches_per_step = 1 + int(n_light_fams > 0) + int(n_light_fams + n_geo_fams > 0) + 1
    line = {
        "metric": METRIC, "value": steps_all / sec_per_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sec_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32/int64", "data": "synthetic (seeded)",
        "config": {"workload": WORKLOADS[name][4], "instances_per_gpu": I, "jobs_per_instance": n,
                   "evaluations_per_gpu": P, "evaluations_sharing_an_instance": share, "alpha": "2/1",
                   "profile_rounds_per_gpu": rounds, "l2": "inputs and outputs larger than L2"},
        "evaluations_per_sec": evals_all / sec_per_step,
        "kernels_ms": {"k_stats_sort": sort_avg, "k_fused_eval<light>": light_avg, "k_fused_eval<full>+k_build_eval": full_avg,
                       "builder_evaluator_stage": build_avg},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak_gbs, "unit": "GB/s", "frac": achieved / peak_gbs,
                     "traffic": traffic, "peak_kind": peak_kind, "kernel": "k_fused_eval<full>", "algorithmic_bytes": alg_bytes,
                     "stage_algorithmic_bytes": stage_bytes, "stage_frac": stage_bytes / (build_avg * 1e-3) / 1e9 / peak_gbs},
        "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
    }
    if e2e:
        line["e2e"] = {"value": steps_all / (e2e_s / args.steps), "unit": UNIT, "h2d_bytes_per_step": e2e[1], "d2h_bytes_per_step": e2e[2]}
    if not args.no_cpu:
        n_s = 512 if name != "c3" else 8      # upper bound; the time budget ends the sample earlier
        cpu_inst = inst.slice(0, min(n_s, I)).to("cpu")
        cpu_inst.meta = dict(inst.meta)
        st, ev_n, dt = oracle_sample(name, cpu_inst, settings, window, args.cpu_seconds)
        line["cpu_baseline"] = {"value": st / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"first {ev_n} evaluations of this workload, {dt:.1f} s"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    a = parse_args()
    run_reference(a) if a.impl == "reference" else run_ours(a)
