"""One full pass per config: EVERY evaluation of configs 2, 3 and 5 (chunk of instances by chunk), of config 2
under the dynamic refill and under speculative runs, and EVERY cell of config 4's two sweeps against the oracle,
element by element.

This takes tens of minutes of host time (the oracle is single-threaded code, run here on all host
cores over disjoint evaluations), so it is not part of the `-m gpu` suite: it is selected with
`-m full` and runs only when KVS_FULL_VERIFY=1:

    KVS_FULL_VERIFY=1 python -m pytest tests/test_full_verify.py -m full -s -q

Each test prints, and appends to KVS_FULL_VERIFY_LOG if that is set, one line with the number of
evaluations (cells) compared, the job-steps they cover and the number of mismatches (which must be 0).
KVS_FULL_VERIFY_LIMIT=<instances> bounds the pass for a quick check.
"""
import os
import time

import numpy as np
import pytest
import torch

from paper_2601_22996_b200 import binding, workloads

pytestmark = pytest.mark.full

CHUNK = {"c2": 128, "c3": 16, "c5": 256, "c2d": 128, "c2s": 128}     # instances per call


def _need():
    if os.environ.get("KVS_FULL_VERIFY") != "1":
        pytest.skip("full verification runs only with KVS_FULL_VERIFY=1")
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")


def _report(line):
    print(line, flush=True)
    path = os.environ.get("KVS_FULL_VERIFY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(line + "\n")


@pytest.fixture(scope="module")
def pool():
    _need()
    from tests import oracle_worker
    p, n = oracle_worker.make_pool()
    yield p, n
    p.close()
    p.join()


def _chunk_tasks(name, inst_cpu, settings, window, n, out, ev, first_instance):
    """Tasks of one chunk from host copies of the call's outputs."""
    poff = ev["profile_off"]
    for e in range(settings.shape[0]):
        st = settings[e]
        i = int(st["instance"])
        a, b = i * n, (i + 1) * n
        pa, pb = int(poff[e]), int(poff[e + 1])
        got = {k: int(ev[k][e]) for k in ("status", "flow", "horizon", "job_steps", "n_unfinished", "peak", "feasible")}
        got["n_runs"] = int(out["n_runs"][e])
        got["job_start"] = out["job_start"][e * n:(e + 1) * n]
        got["job_completion"] = out["job_completion"][e * n:(e + 1) * n]
        got["profile"] = ev["profile"][pa:pb] if pb > pa else None
        got["profile_capacity"] = pb - pa
        yield dict(tag=f"{name} instance {first_instance + i} eval {e} family {int(st['family'])} M {int(st['M'])}",
                   s=inst_cpu.s[a:b], o=inst_cpu.o[a:b], est=None if inst_cpu.o_est is None else inst_cpu.o_est[a:b],
                   arrival=None if inst_cpu.arrival is None else inst_cpu.arrival[a:b], window=window,
                   st={f: int(st[f]) for f in st.dtype.names}, got=got)


def _verify_config(name, pool):
    import bench
    from paper_2601_22996_b200.api import Scheduler
    from tests import oracle_worker
    pool, workers = pool
    dev = torch.device("cuda:0")
    _, I_all, n, fams, desc = bench.WORKLOADS[name]
    I_all = min(I_all, int(os.environ.get("KVS_FULL_VERIFY_LIMIT", I_all)))
    sched = Scheduler(0)
    t0 = time.time()
    evals = steps = bad = 0
    first_msg = None
    for lo in range(0, I_all, CHUNK[name]):
        c = min(CHUNK[name], I_all - lo)
        inst = bench.make_instances(name, c, dev, first_instance=lo)
        settings, window = bench.make_settings(name, inst)
        P = settings.shape[0]
        ctx = sched.context(binding.workspace_bytes(c * n, c, n, P))
        first = Scheduler.scalars(P, dev)
        ctx.build_schedule(inst, settings, dict(n_runs=torch.zeros(P, dtype=torch.int64, device=dev)), first, window=window, max_jobs=n)
        geo = torch.from_numpy(np.array([bench.stores_profile(name, int(f)) for f in settings["family"]])).to(dev)
        cap = torch.where(geo, first["horizon"], torch.zeros_like(first["horizon"]))   # as bench.py sizes them
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
        h_out = {k: v.cpu().numpy() for k, v in out.items()}
        h_ev = {k: v.cpu().numpy() for k, v in ev.items()}
        ic = inst.to("cpu")
        npv = lambda t: None if t is None else t.numpy()
        inst_cpu = workloads.Instances(ic.job_off.numpy(), ic.s.numpy(), ic.o.numpy(), npv(ic.o_est), npv(ic.arrival))
        for st, msg in pool.imap_unordered(oracle_worker.check_evaluation,
                                           _chunk_tasks(name, inst_cpu, settings, window, n, h_out, h_ev, lo), chunksize=4):
            evals += 1
            steps += st
            if msg is not None:
                bad += 1
                first_msg = first_msg or msg
        del out, ev, inst
    _report(f"full verify {name}: {desc}: {evals} evaluations of {I_all} instances compared with the oracle, "
            f"{steps} job-steps, {bad} mismatches, {workers} oracle workers, {time.time() - t0:.0f} s"
            + (f"; first: {first_msg}" if first_msg else ""))
    assert bad == 0, first_msg


def test_full_config2(pool):
    _need()
    _verify_config("c2", pool)


def test_full_config3(pool):
    _need()
    _verify_config("c3", pool)


def test_full_config5(pool):
    _need()
    _verify_config("c5", pool)


def test_full_config2_dynamic_refill(pool):
    _need()
    _verify_config("c2d", pool)


def test_full_config2_speculative_runs(pool):
    _need()
    _verify_config("c2s", pool)


def test_full_config1_and_config4(pool):
    """Config 1 (one instance, four families, full outputs) and every cell of the 64 x 64 sweep, both families."""
    _need()
    from tests import oracle_worker, parity
    pool, workers = pool
    t0 = time.time()
    inst = workloads.config1()
    st = binding.settings_grid([0], ["GBA", "GSA", "SPS", "SIMS"], inst.meta["M"])
    steps1 = parity.check_batch(inst, st, label="config 1")
    _report(f"full verify c1: 4 evaluations compared with the oracle (both kernels), {steps1} job-steps, 0 mismatches")
    inst = workloads.config4()
    taus, ks = workloads.sweep_grids()
    if "KVS_FULL_VERIFY_LIMIT" in os.environ:
        taus, ks = taus[::16], ks[::16]
    dev_inst = inst.to("cuda:0")
    s_np, o_np = inst.s.numpy(), inst.o.numpy()
    cells = bad = steps = 0
    first_msg = None
    for fam in ("SPS", "SIMS"):
        out = {f: t.cpu().numpy() for f, t in parity.scheduler().sweep(dev_inst, 0, fam, inst.meta["M"][0], taus, ks).items()}
        tasks = (dict(tag=f"config 4 {fam} tau {taus[i]} k {ks[j]}", family=fam, s=s_np, o=o_np, M=inst.meta["M"][0],
                      tau=taus[i], k=ks[j], got={f: int(out[f][i, j]) for f in out})
                 for i in range(len(taus)) for j in range(len(ks)))
        for stp, msg in pool.imap_unordered(oracle_worker.check_sweep_cell, tasks, chunksize=2):
            cells += 1
            steps += stp
            if msg is not None:
                bad += 1
                first_msg = first_msg or msg
    _report(f"full verify c4: {cells} cells (both families) compared with the oracle, {steps} job-steps, {bad} mismatches, "
            f"{workers} oracle workers, {time.time() - t0:.0f} s" + (f"; first: {first_msg}" if first_msg else ""))
    assert bad == 0, first_msg
