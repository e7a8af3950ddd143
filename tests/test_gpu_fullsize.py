"""Parity at the benchmark's sizes, in the launch configuration bench.py times: the whole batch goes
through one fused call, a seeded sample of evaluations is compared with the oracle element by
element (scalars, every job's start and completion, the full profile), and size-independent
properties are checked on all evaluations."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_22996_b200 import binding, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def par():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import parity
    return parity


def _bench_call(par, name, n_inst):
    """Same tensors and the same single kvs_evaluate_built call as bench.py's step."""
    import bench
    from paper_2601_22996_b200.api import Scheduler
    dev = torch.device("cuda:0")
    inst = bench.make_instances(name, n_inst, dev)
    settings, window = bench.make_settings(name, inst)
    n = bench.WORKLOADS[name][2]
    P = settings.shape[0]
    ctx = par.scheduler().context(binding.workspace_bytes(n_inst * n, n_inst, n, P))
    first = Scheduler.scalars(P, dev)
    ctx.build_schedule(inst, settings, dict(n_runs=torch.zeros(P, dtype=torch.int64, device=dev)), first,
                       window=window, max_jobs=n)
    geo = torch.from_numpy(settings["family"] <= 1).to(dev)
    cap = torch.where(geo, first["horizon"], torch.zeros_like(first["horizon"]))
    poff = torch.zeros(P + 1, dtype=torch.int64, device=dev)
    poff[1:] = torch.cumsum(cap, 0)
    out = dict(job_out_off=torch.arange(P + 1, dtype=torch.int64, device=dev) * n,
               job_start=torch.full((P * n,), -2, dtype=torch.int32, device=dev),
               job_completion=torch.full((P * n,), -2, dtype=torch.int32, device=dev),
               n_runs=torch.zeros(P, dtype=torch.int64, device=dev))
    ev = Scheduler.scalars(P, dev)
    ev["profile_off"] = poff
    ev["profile"] = torch.full((int(poff[-1]),), -7, dtype=torch.int32, device=dev)
    ctx.evaluate_built(inst, settings, out, ev, window=window, max_jobs=n)
    torch.cuda.synchronize()
    return inst, settings, window, n, out, ev, first


def _check_sample(par, inst, settings, window, n, out, ev, sample):
    for e in sample:
        st = settings[e]
        i = int(st["instance"])
        one = inst.slice(i, i + 1).to("cpu")
        row = st.copy()
        row["instance"] = 0
        S = par.oracle_eval(one, row, window)
        tag = f"eval {e} family {int(st['family'])} M {int(st['M'])}"
        assert S.status == 0 and int(ev["status"][e]) == 0, tag
        assert (int(ev["flow"][e]), int(ev["horizon"][e]), int(ev["job_steps"][e]), int(ev["n_unfinished"][e])) == \
               (S.flow, S.horizon, S.job_steps, S.n_unfinished), tag
        assert int(out["n_runs"][e]) == len(S.run_job), tag
        assert np.array_equal(out["job_start"][e * n:(e + 1) * n].cpu().numpy().astype(np.int64), S.job_start), tag
        assert np.array_equal(out["job_completion"][e * n:(e + 1) * n].cpu().numpy().astype(np.int64), S.job_completion), tag
        a, b = int(ev["profile_off"][e]), int(ev["profile_off"][e + 1])
        if b > a:
            E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s)
            assert b - a == S.horizon and np.array_equal(ev["profile"][a:b].cpu().numpy().astype(np.int64), E.profile), tag
        elif S.horizon <= par.DENSE_LIMIT:
            E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s, want_profile=False)
        else:
            E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
        assert int(ev["peak"][e]) == E.peak and int(ev["feasible"][e]) == int(E.peak <= int(st["M"])), tag


def _check_properties(settings, n, out, ev, inst):
    """Hold for every evaluation at any size: all jobs complete, completion = start + o, memory fits
    (every schedule is built with s_bar = max s and the maximal feasible parallelism), flow = sum."""
    P = settings.shape[0]
    assert int((ev["status"] != 0).sum()) == 0
    assert int(ev["n_unfinished"].sum()) == 0
    M = torch.from_numpy(np.ascontiguousarray(settings["M"])).to(ev["peak"].device)
    assert bool((ev["peak"] <= M).all()) and bool((ev["feasible"] == 1).all())
    o = inst.o.view(inst.n_instances, n)
    inst_of = torch.from_numpy(np.ascontiguousarray(settings["instance"])).to(o.device)
    for lo in range(0, P, 2048):
        hi = min(P, lo + 2048)
        st = out["job_start"][lo * n:hi * n].view(hi - lo, n).to(torch.int64)
        cp = out["job_completion"][lo * n:hi * n].view(hi - lo, n).to(torch.int64)
        assert torch.equal(cp, st + o[inst_of[lo:hi]].to(torch.int64))
        arr = 0 if inst.arrival is None else inst.arrival.view(inst.n_instances, n)[inst_of[lo:hi]].sum(1)
        assert torch.equal(cp.sum(1) - arr, ev["flow"][lo:hi])
        assert bool((cp.max(1).values == ev["horizon"][lo:hi]).all())


def test_config2_full_size_sampled(par):
    inst, settings, window, n, out, ev, _ = _bench_call(par, "c2", 1024)
    _check_properties(settings, n, out, ev, inst)
    rng = np.random.default_rng(2)
    _check_sample(par, inst, settings, window, n, out, ev, sorted(rng.choice(settings.shape[0], 24, replace=False)))


def test_config5_full_size_sampled(par):
    """The whole stress config (16,384 instances, 65,536 evaluations) in one call, as bench.py times it."""
    inst, settings, window, n, out, ev, _ = _bench_call(par, "c5", 16384)
    _check_properties(settings, n, out, ev, inst)
    rng = np.random.default_rng(5)
    _check_sample(par, inst, settings, window, n, out, ev, sorted(rng.choice(settings.shape[0], 24, replace=False)))


def test_config3_online_sampled(par):
    inst, settings, window, n, out, ev, _ = _bench_call(par, "c3", 256)
    assert int((ev["status"] != 0).sum()) == 0 and int(ev["n_unfinished"].sum()) == 0
    rng = np.random.default_rng(3)
    _check_sample(par, inst, settings, window, n, out, ev, sorted(rng.choice(settings.shape[0], 8, replace=False)))


def test_config4_sweep_full_size_sampled(par):
    """One instance of 10^6 jobs, the 64 x 64 grid, both families; sampled cells against the oracle."""
    inst = workloads.config4()
    taus, ks = workloads.sweep_grids()
    dev_inst = inst.to("cuda:0")
    rng = np.random.default_rng(4)
    cells = [(int(rng.integers(64)), int(rng.integers(64))) for _ in range(5)] + [(0, 0), (63, 63)]
    for fam in ("SPS", "SIMS"):
        out = {f: t.cpu().numpy() for f, t in par.scheduler().sweep(dev_inst, 0, fam, inst.meta["M"][0], taus, ks).items()}
        # properties on the whole grid: job-steps and completed counts do not depend on k
        assert np.all(out["job_steps"] == out["job_steps"][:, :1]) and np.all(out["n_completed"] == out["n_completed"][:, :1])
        assert np.all(np.diff(out["n_completed"][:, 0]) >= 0) and np.all(out["feasible"] == (out["peak"] <= inst.meta["M"][0]))
        for i, j in cells:
            S = oracle.build_schedule(fam, inst.s, inst.o, inst.meta["M"][0], tau=taus[i], k=ks[j], s_bar=0)
            E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
            got = (int(out["peak"][i, j]), int(out["flow"][i, j]), int(out["horizon"][i, j]), int(out["job_steps"][i, j]),
                   int(out["n_completed"][i, j]))
            assert got == (E.peak, S.flow, S.horizon, S.job_steps, 1_000_000 - S.n_unfinished), (fam, taus[i], ks[j])
