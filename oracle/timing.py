"""Times the oracle, as it stands, on a list of evaluations (the CPU baseline of the benchmark).

TEST INFRASTRUCTURE ONLY, like the rest of this package: used by bench.py's CPU baseline and reference
legs.  Imports numpy and the oracle only, so that worker processes started with `spawn` stay light.
The oracle itself is single-threaded code; `run_parallel` runs it on disjoint evaluations in one
process per host core.
"""
from __future__ import annotations

import multiprocessing
import os
import time

DENSE_LIMIT = 60_000_000   # rounds above which the dense array of the definition is not formed


def run(tasks, budget_s: float):
    """Works through `tasks` until the time budget is spent.  A task is a dict: family, s, o, M and optionally
    est, arrival, window, alpha, beta0, s_bar, tau, k, subroutine, per_class_s, and `profile` (True: the
    per-round memory of the definition, one update per job-step; False: the peak from sorted run events, as the
    CUDA path does for evaluations that store no profile).  Returns (job_steps, evaluations, seconds)."""
    import oracle
    t0 = time.perf_counter()
    steps = evals = 0
    for t in tasks:
        window = int(t.get("window", 0))
        S = oracle.build_schedule(t["family"], t["s"], t["o"], int(t["M"]), o_est=t.get("est"),
                                  arrival=t.get("arrival") if window else None, alpha=t.get("alpha", (2, 1)),
                                  beta0=int(t.get("beta0", 0)), s_bar=int(t.get("s_bar", -1)), tau=int(t.get("tau", 0)),
                                  k=int(t.get("k", 0)), window=window, subroutine=int(t.get("subroutine", 0)),
                                  per_class_s=int(t.get("per_class_s", 0)))
        if t.get("profile", True) and S.horizon <= DENSE_LIMIT:
            E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s, want_profile=False)
        else:
            E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
        assert E.job_steps == S.job_steps
        steps += S.job_steps
        evals += 1
        if time.perf_counter() - t0 > budget_s:
            break
    return steps, evals, time.perf_counter() - t0


def _worker(args):
    tasks, budget_s = args
    return run(tasks, budget_s)


def run_parallel(task_lists, budget_s: float):
    """One process per list (disjoint evaluations), all at once.  Returns (job_steps, evaluations, seconds of the
    slowest process, processes)."""
    n = len(task_lists)
    with multiprocessing.get_context("spawn").Pool(n) as pool:
        res = pool.map(_worker, [(tl, budget_s) for tl in task_lists], chunksize=1)
    return sum(r[0] for r in res), sum(r[1] for r in res), max(r[2] for r in res), n


def host_cores() -> int:
    return int(os.environ.get("KVS_ORACLE_WORKERS", "0")) or (os.cpu_count() or 1)
