"""Worker side of the multi-process oracle comparison.

The oracle is single-threaded code; the full-size parity checks run it on every host core at once,
one evaluation per task, in worker processes started with `spawn` (a process forked after the first
CUDA call would hang).  This module is what those workers import, so it pulls in numpy and the
oracle only - neither torch nor the CUDA binding.

A task carries the inputs of one evaluation together with what the CUDA path returned for it; the
worker builds the oracle's schedule, evaluates it by the definition and compares element by element
(all quantities are integers: the tolerance is zero).  It returns (job_steps, None) or (0, message).
"""
from __future__ import annotations

import multiprocessing
import os

import numpy as np

DENSE_LIMIT = 6_000_000   # rounds above which the oracle uses its event evaluator (no dense array)


def make_pool(n_workers: int | None = None):
    n = n_workers or int(os.environ.get("KVS_ORACLE_WORKERS", "0")) or (os.cpu_count() or 1)
    return multiprocessing.get_context("spawn").Pool(max(1, n)), max(1, n)


def check_evaluation(task: dict):
    """One (instance, setting, family) evaluation.  Keys: tag, s, o, est, arrival, window, st (dict of
    the setting's fields), got (dict: status flow horizon job_steps n_unfinished n_runs peak feasible,
    job_start, job_completion, profile or None, profile_capacity)."""
    import oracle
    st, got, tag = task["st"], task["got"], task["tag"]
    window = int(task.get("window", 0))
    arr = task.get("arrival") if window else None
    S = oracle.build_schedule(int(st["family"]), task["s"], task["o"], int(st["M"]), o_est=task.get("est"), arrival=arr,
                              alpha=(int(st["alpha_num"]), int(st["alpha_den"])), beta0=int(st["beta0"]),
                              s_bar=int(st["s_bar"]), tau=int(st["tau"]), k=int(st["k"]), window=window,
                              subroutine=int(st.get("subroutine", 0)), per_class_s=int(st.get("per_class_s", 0)))
    if S.status != 0:
        return (0, None) if int(got["status"]) & (1 | 8) else (0, f"{tag}: oracle status {S.status}, GPU status {got['status']}")
    if int(got["status"]) != 0:
        return 0, f"{tag}: GPU status {got['status']}"
    want = dict(flow=S.flow, horizon=S.horizon, job_steps=S.job_steps, n_unfinished=S.n_unfinished, n_runs=len(S.run_job))
    for name, v in want.items():
        if name in got and int(got[name]) != v:
            return 0, f"{tag}: {name} {int(got[name])} != {v}"
    for name, ref in (("job_start", S.job_start), ("job_completion", S.job_completion)):
        if got.get(name) is not None and not np.array_equal(np.asarray(got[name]).astype(np.int64), ref):
            bad = np.nonzero(np.asarray(got[name]).astype(np.int64) != ref)[0]
            return 0, f"{tag}: {name} differs at jobs {bad[:5].tolist()}"
    prof = got.get("profile")
    if prof is not None and int(got.get("profile_capacity", len(prof))) > 0:
        E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s)
        # the refill and the speculative runs work in a buffer sized by the schedule they start from, which ends
        # later: the rounds past the new horizon hold nothing
        later = int(st["family"]) >= 4
        if (len(prof) < S.horizon if later else len(prof) != S.horizon) or np.any(np.asarray(prof[S.horizon:])) or \
                not np.array_equal(np.asarray(prof[:S.horizon]).astype(np.int64), E.profile):
            return 0, f"{tag}: profile differs (length {len(prof)} vs horizon {S.horizon})"
    elif S.horizon <= DENSE_LIMIT:
        E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s, want_profile=False)
    else:
        E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
    if "peak" in got and int(got["peak"]) != E.peak:
        return 0, f"{tag}: peak {int(got['peak'])} != {E.peak}"
    if "feasible" in got and int(got["feasible"]) != int(E.peak <= int(st["M"])):
        return 0, f"{tag}: feasibility mask"
    return S.job_steps, None


def check_sweep_cell(task: dict):
    """One (tau, k) cell of a sweep.  Keys: tag, family, s, o, M, tau, k, got (peak flow horizon job_steps
    n_completed feasible)."""
    import oracle
    got, tag = task["got"], task["tag"]
    S = oracle.build_schedule(task["family"], task["s"], task["o"], int(task["M"]), tau=int(task["tau"]), k=int(task["k"]), s_bar=0)
    E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
    want = dict(peak=E.peak, flow=S.flow, horizon=S.horizon, job_steps=S.job_steps, n_completed=len(task["o"]) - S.n_unfinished,
                feasible=int(E.peak <= int(task["M"])))
    for name, v in want.items():
        if int(got[name]) != v:
            return 0, f"{tag}: {name} {int(got[name])} != {v}"
    return S.job_steps, None
