"""Shared helper of the GPU parity tests: run the CUDA path and the CPU oracle on the same
inputs and compare every output element by element (all quantities are integers: bit-exact)."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2601_22996_b200 import binding
from paper_2601_22996_b200.api import Scheduler
from paper_2601_22996_b200.workloads import Instances

FAM_NAME = {0: "GBA", 1: "GSA", 2: "SPS", 3: "SIMS", 4: "GBAD", 5: "GSAS"}
DENSE_LIMIT = 6_000_000   # rounds above which the oracle uses its event evaluator (no dense array)

_scheduler = None


def scheduler() -> Scheduler:
    global _scheduler
    if _scheduler is None:
        _scheduler = Scheduler()
    return _scheduler


def oracle_eval(inst: Instances, st, window=0):
    """Oracle schedule for one settings row (numpy record)."""
    i = int(st["instance"])
    a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
    est = None if inst.o_est is None else inst.o_est[a:b]
    arr = None if (inst.arrival is None or window == 0) else inst.arrival[a:b]
    return oracle.build_schedule(int(st["family"]), inst.s[a:b], inst.o[a:b], int(st["M"]), o_est=est, arrival=arr,
                                 alpha=(int(st["alpha_num"]), int(st["alpha_den"])), beta0=int(st["beta0"]),
                                 s_bar=int(st["s_bar"]), tau=int(st["tau"]), k=int(st["k"]), window=window,
                                 subroutine=int(st["subroutine"]), per_class_s=int(st["per_class_s"]))


def check_batch(inst_cpu: Instances, settings: np.ndarray, *, window=0, want_profile=True, want_runs=True,
                sample=None, label="", inst_gpu=None):
    """GPU (one batched call) against the oracle (one evaluation at a time).  Returns job-steps checked."""
    dev = torch.device("cuda:0")
    if inst_gpu is None:
        inst_gpu = inst_cpu.to(dev)
    # A call that asks for the explicit run list takes the general kernel, one that does not takes the
    # 32-bit fast kernel: both are checked against the oracle.
    variants = [want_runs] if not want_runs else [True, False]
    steps = 0
    for runs_wanted in variants:
        res = scheduler().evaluate(inst_gpu, settings, want_jobs=True, want_profile=want_profile,
                                   want_runs=runs_wanted, window=window)
        torch.cuda.synchronize()
        steps = _compare(res, inst_cpu, settings, window, want_profile, sample, f"{label} runs={int(runs_wanted)}")
    return steps


def _compare(res, inst_cpu, settings, window, want_profile, sample, label):
    g = {k: (v.cpu().numpy() if isinstance(v, torch.Tensor) else v) for k, v in vars(res).items() if k != "runs"}
    gruns = {k: v.cpu().numpy() for k, v in res.runs.items()} if res.runs else None
    P = settings.shape[0]
    todo = range(P) if sample is None else sample
    steps = 0
    for e in todo:
        st = settings[e]
        tag = f"{label} eval {e} fam {FAM_NAME[int(st['family'])]} M {int(st['M'])} inst {int(st['instance'])}"
        S = oracle_eval(inst_cpu, st, window)
        if S.status != 0:
            assert int(g["status"][e]) & (binding.EVAL_INFEASIBLE | binding.EVAL_BAD_INPUT), tag
            continue
        assert int(g["status"][e]) == 0, f"{tag}: status {int(g['status'][e])}"
        assert int(g["flow"][e]) == S.flow, tag
        assert int(g["horizon"][e]) == S.horizon, tag
        assert int(g["job_steps"][e]) == S.job_steps, tag
        assert int(g["n_unfinished"][e]) == S.n_unfinished, tag
        assert int(g["n_runs"][e]) == len(S.run_job), tag
        a, b = int(g["job_out_off"][e]), int(g["job_out_off"][e + 1])
        assert np.array_equal(g["job_start"][a:b].astype(np.int64), S.job_start), tag
        assert np.array_equal(g["job_completion"][a:b].astype(np.int64), S.job_completion), tag
        if gruns is not None:
            a, b = int(g["run_off"][e]), int(g["run_off"][e + 1])
            assert b - a == len(S.run_job), tag
            assert np.array_equal(gruns["run_job"][a:b], S.run_job), tag
            assert np.array_equal(gruns["run_phase"][a:b], S.run_phase), tag
            assert np.array_equal(gruns["run_start"][a:b], S.run_start), tag
            assert np.array_equal(gruns["run_len"][a:b], S.run_len), tag
            assert np.array_equal(gruns["run_s"][a:b], S.run_s), tag
        if S.horizon <= DENSE_LIMIT:
            E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s, want_profile=want_profile)
        else:
            E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
        assert int(g["peak"][e]) == E.peak, f"{tag}: peak {int(g['peak'][e])} vs {E.peak}"
        assert int(g["feasible"][e]) == int(E.peak <= int(st["M"])), tag
        if want_profile and E.profile is not None:
            a, b = int(g["profile_off"][e]), int(g["profile_off"][e + 1])
            assert b - a >= S.horizon, tag                   # a refilled schedule ends before the batching one that sized it
            assert not np.any(g["profile"][a + S.horizon:b]), tag
            got = g["profile"][a:a + S.horizon].astype(np.int64)
            if not np.array_equal(got, E.profile):
                bad = np.nonzero(got != E.profile)[0]
                raise AssertionError(f"{tag}: profile differs at {bad[:5]} got {got[bad[:5]]} want {E.profile[bad[:5]]}")
        steps += S.job_steps
    return steps
