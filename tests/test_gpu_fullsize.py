"""Parity at the benchmark's sizes, in the launch configuration bench.py times: the whole batch goes
through one fused call, a stratified seeded sample of evaluations is compared with the oracle element
by element (scalars, every job's start and completion, the full profile) - the oracle side running
on all host cores, one evaluation per worker task - and size-independent properties are checked on
all evaluations.  The pass over every evaluation of every config is tests/test_full_verify.py."""
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


@pytest.fixture(scope="module")
def pool():
    """Worker processes for the oracle side, started with spawn (CUDA is already initialised here)."""
    from tests import oracle_worker
    p, _ = oracle_worker.make_pool()
    yield p
    p.close()
    p.join()


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
    geo = torch.from_numpy(np.array([bench.stores_profile(name, int(f)) for f in settings["family"]])).to(dev)
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


def _eval_tasks(inst, settings, window, n, out, ev, sample, label):
    """Tasks for tests/oracle_worker.check_evaluation: inputs and CUDA results of the sampled evaluations."""
    cache = {}
    for e in sample:
        st = settings[e]
        i = int(st["instance"])
        if i not in cache:
            cache.clear()
            cache[i] = inst.slice(i, i + 1).to("cpu")
        one = cache[i]
        a, b = int(ev["profile_off"][e]), int(ev["profile_off"][e + 1])
        got = {k: int(ev[k][e]) for k in ("status", "flow", "horizon", "job_steps", "n_unfinished", "peak", "feasible")}
        got["n_runs"] = int(out["n_runs"][e])
        got["job_start"] = out["job_start"][e * n:(e + 1) * n].cpu().numpy()
        got["job_completion"] = out["job_completion"][e * n:(e + 1) * n].cpu().numpy()
        got["profile"] = ev["profile"][a:b].cpu().numpy() if b > a else None
        got["profile_capacity"] = b - a
        yield dict(tag=f"{label} eval {e} family {int(st['family'])} M {int(st['M'])} inst {i}",
                   s=one.s.numpy(), o=one.o.numpy(), est=None if one.o_est is None else one.o_est.numpy(),
                   arrival=None if one.arrival is None else one.arrival.numpy(), window=window,
                   st={f: int(st[f]) for f in st.dtype.names}, got=got)


def _check_sample(pool, inst, settings, window, n, out, ev, sample, label):
    """Every sampled evaluation element by element against the oracle, the oracle side on all host cores."""
    from tests import oracle_worker
    steps = 0
    for st, msg in pool.imap_unordered(oracle_worker.check_evaluation,
                                       _eval_tasks(inst, settings, window, n, out, ev, sorted(sample), label), chunksize=1):
        assert msg is None, msg
        steps += st
    assert steps > 0
    return steps


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


def test_config2_full_size_stratified(par, pool):
    """All 1,024 instances x 8 budgets x 2 families in one call; compared in full: 16 instances under
    every budget and both families (256 evaluations), the rest by properties."""
    inst, settings, window, n, out, ev, _ = _bench_call(par, "c2", 1024)
    _check_properties(settings, n, out, ev, inst)
    rng = np.random.default_rng(2)
    chosen = set(int(i) for i in rng.choice(1024, 16, replace=False))
    sample = [e for e in range(settings.shape[0]) if int(settings[e]["instance"]) in chosen]
    budgets = {(int(settings[e]["M"]), int(settings[e]["family"])) for e in sample}
    assert len(sample) == 256 and len(budgets) == 16
    _check_sample(pool, inst, settings, window, n, out, ev, sample, "config 2")


@pytest.mark.parametrize("name", ["c2d", "c2s"])
def test_config2_refill_and_speculation_full_size_stratified(par, pool, name):
    """Config 2's 1,024 instances x 8 budgets under the dynamic refill / under speculative runs, one call as
    bench.py times it; 8 instances under every budget compared in full (64 evaluations), the rest by properties
    (every job completes, completion = start + o for the run that completed it, every round fits)."""
    inst, settings, window, n, out, ev, first = _bench_call(par, name, 1024)
    _check_properties(settings, n, out, ev, inst)
    assert bool((ev["horizon"] <= first["horizon"]).all()) and bool((ev["flow"] <= first["flow"]).all())
    rng = np.random.default_rng(22)
    chosen = set(int(i) for i in rng.choice(1024, 8, replace=False))
    sample = [e for e in range(settings.shape[0]) if int(settings[e]["instance"]) in chosen]
    assert len(sample) == 64 and len({int(settings[e]["M"]) for e in sample}) == 8
    _check_sample(pool, inst, settings, window, n, out, ev, sample, name)


def test_config5_full_size_stratified(par, pool):
    """The whole stress config (16,384 instances, 65,536 evaluations) in one call, as bench.py times it.
    Compared in full: for each of the nine (prompt, response) distribution mixes the instances with the
    five smallest and the five largest budgets and five more, under all four families (540 evaluations:
    every (mix, family) combination and both ends of the budget range); the rest by properties."""
    inst, settings, window, n, out, ev, _ = _bench_call(par, "c5", 16384)
    _check_properties(settings, n, out, ev, inst)
    kinds = np.array([workloads.stream_key(workloads.BASE_SEED, 5, 3, i) % 9 for i in range(16384)])
    M = inst.meta["M_per_instance"].cpu().numpy()
    rng = np.random.default_rng(5)
    chosen = set()
    for mix in range(9):
        ids = np.nonzero(kinds == mix)[0]
        by_m = ids[np.argsort(M[ids], kind="stable")]
        chosen.update(int(i) for i in by_m[:5])
        chosen.update(int(i) for i in by_m[-5:])
        chosen.update(int(i) for i in rng.choice(by_m[5:-5], 5, replace=False))
    sample = [e for e in range(settings.shape[0]) if int(settings[e]["instance"]) in chosen]
    combos = {(int(kinds[int(settings[e]["instance"])]), int(settings[e]["family"])) for e in sample}
    assert len(sample) == 540 and len(combos) == 36
    _check_sample(pool, inst, settings, window, n, out, ev, sample, "config 5")


def test_config3_online_stratified(par, pool):
    """Online arrivals with estimates: 32 of the 256 instances under both families (64 evaluations)."""
    inst, settings, window, n, out, ev, _ = _bench_call(par, "c3", 256)
    assert int((ev["status"] != 0).sum()) == 0 and int(ev["n_unfinished"].sum()) == 0
    rng = np.random.default_rng(3)
    chosen = set(int(i) for i in rng.choice(256, 32, replace=False))
    sample = [e for e in range(settings.shape[0]) if int(settings[e]["instance"]) in chosen]
    assert len(sample) == 64
    _check_sample(pool, inst, settings, window, n, out, ev, sample, "config 3")


def test_config4_sweep_full_size_stratified(par, pool):
    """One instance of 10^6 jobs, the 64 x 64 grid, both families; 128 cells per family against the
    oracle: two permutations of the grid, so that every row and every column is hit twice."""
    from tests import oracle_worker
    inst = workloads.config4()
    taus, ks = workloads.sweep_grids()
    dev_inst = inst.to("cuda:0")
    rng = np.random.default_rng(4)
    cells = [(i, int(j)) for i, j in enumerate(rng.permutation(64))] + [(i, int(j)) for i, j in enumerate(rng.permutation(64))]
    cells[0], cells[63] = (0, 0), (63, 63)
    s_np, o_np = inst.s.numpy(), inst.o.numpy()
    for fam in ("SPS", "SIMS"):
        out = {f: t.cpu().numpy() for f, t in par.scheduler().sweep(dev_inst, 0, fam, inst.meta["M"][0], taus, ks).items()}
        # properties on the whole grid: job-steps and completed counts do not depend on k
        assert np.all(out["job_steps"] == out["job_steps"][:, :1]) and np.all(out["n_completed"] == out["n_completed"][:, :1])
        assert np.all(np.diff(out["n_completed"][:, 0]) >= 0) and np.all(out["feasible"] == (out["peak"] <= inst.meta["M"][0]))
        tasks = [dict(tag=f"config 4 {fam} tau {taus[i]} k {ks[j]}", family=fam, s=s_np, o=o_np, M=inst.meta["M"][0],
                      tau=taus[i], k=ks[j], got={f: int(out[f][i, j]) for f in out}) for i, j in cells]
        for _, msg in pool.imap_unordered(oracle_worker.check_sweep_cell, tasks, chunksize=2):
            assert msg is None, msg
