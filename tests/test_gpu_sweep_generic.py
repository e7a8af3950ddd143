"""Parity of the sweep and of the generic run evaluator against the CPU oracle (bit-exact)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2601_22996_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def par():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import parity
    return parity


def _oracle_setting(inst, fam, M, tau, k):
    S = oracle.build_schedule(fam, inst.s, inst.o, M, tau=tau, k=k, s_bar=0)
    E = oracle.evaluate_events(S.run_start, S.run_len, S.run_s)
    return dict(peak=E.peak, flow=S.flow, n_completed=len(inst.o) - S.n_unfinished, horizon=S.horizon,
                job_steps=S.job_steps, feasible=int(E.peak <= M))


def _check_sweep(par, inst, fam, M, taus, ks, sample=None):
    out = par.scheduler().sweep(inst.to("cuda:0"), 0, fam, M, taus, ks)
    got = {f: t.cpu().numpy() for f, t in out.items()}
    cells = [(i, j) for i in range(len(taus)) for j in range(len(ks))] if sample is None else sample
    for i, j in cells:
        want = _oracle_setting(inst, fam, M, taus[i], ks[j])
        for f, v in want.items():
            assert int(got[f][i, j]) == v, f"{fam} tau={taus[i]} k={ks[j]} {f}: {int(got[f][i, j])} vs {v}"


@pytest.mark.parametrize("fam", ["SPS", "SIMS"])
def test_sweep_small_full_grid(par, fam):
    inst = workloads.config4(n=3000)
    taus = [1, 2, 3, 7, 16, 100, 257, 1024, 16384, 40000]
    ks = [1, 2, 3, 5, 16, 33, 100, 1000, 2999, 3000, 3001, 50000]
    _check_sweep(par, inst, fam, 1 << 20, taus, ks)


@pytest.mark.parametrize("fam", ["SPS", "SIMS"])
def test_sweep_ragged_and_tiny(par, fam):
    for n in (1, 2, 63, 64, 65, 8191, 8193):
        inst = workloads.config1(n=n)
        _check_sweep(par, inst, fam, 5000, [1, 5, 64, 1024, 2000], [1, 4, 64, 1000])


def test_sweep_paper_grid_sampled(par):
    """The 64 x 64 grid on a 200,000-job instance; a sample of cells against the oracle."""
    inst = workloads.config4(n=200_000)
    taus, ks = workloads.sweep_grids()
    rng = np.random.default_rng(4)
    cells = [(int(rng.integers(64)), int(rng.integers(64))) for _ in range(24)] + [(0, 0), (63, 63), (0, 63), (63, 0)]
    for fam in ("SPS", "SIMS"):
        _check_sweep(par, inst, fam, inst.meta["M"][0], taus, ks, sample=cells)


def test_sweep_agrees_with_fused_path(par):
    """Same (tau, k) through kvs_sweep and through kvs_evaluate_built (dense profile)."""
    from paper_2601_22996_b200 import binding
    inst = workloads.config2(n_inst=1, n=5000)
    taus, ks = [16, 90, 700], [2, 17, 300]
    for fam in ("SPS", "SIMS"):
        out = par.scheduler().sweep(inst.to("cuda:0"), 0, fam, 1 << 22, taus, ks)
        rows = [dict(instance=0, family=fam, M=1 << 22, tau=t, k=k) for t in taus for k in ks]
        res = par.scheduler().evaluate(inst.to("cuda:0"), binding.make_settings(rows), want_profile=True)
        assert torch.equal(res.peak.view(3, 3), out["peak"]) and torch.equal(res.flow.view(3, 3), out["flow"])
        assert torch.equal(res.horizon.view(3, 3), out["horizon"]) and torch.equal(res.job_steps.view(3, 3), out["job_steps"])


def _runs_to_gpu(batches, dev):
    off = np.zeros(len(batches) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(b[0]) for b in batches])
    cat = lambda i, dt: torch.tensor(np.concatenate([np.asarray(b[i], dtype=dt) for b in batches]) if batches else [], dtype=getattr(torch, np.dtype(dt).name)).to(dev)
    return torch.tensor(off).to(dev), cat(0, np.int64), cat(1, np.int32), cat(2, np.int32)


def test_generic_evaluator_random_runs(par):
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(9)
    batches = []
    for e in range(40):
        R = int(rng.integers(0, 3000)) if e else 0
        batches.append((rng.integers(0, 20000, R), rng.integers(1, 900, R), rng.integers(0, 4000, R)))
    off, st, ln, ss = _runs_to_gpu(batches, dev)
    want = [oracle.evaluate_dense(*b) for b in batches]
    cap = torch.tensor([w.horizon for w in want], dtype=torch.int64, device=dev)
    M = torch.tensor([w.peak - (i % 2) for i, w in enumerate(want)], dtype=torch.int64, device=dev)
    res = par.scheduler().evaluate_runs(off, st, ln, ss, cap, M=M)
    prof, poff = res.profile.cpu().numpy(), res.profile_off.cpu().numpy()
    for e, w in enumerate(want):
        assert int(res.status[e]) == 0
        assert (int(res.peak[e]), int(res.horizon[e]), int(res.job_steps[e])) == (w.peak, w.horizon, w.job_steps)
        assert np.array_equal(prof[poff[e]:poff[e + 1]].astype(np.int64), w.profile)
        assert int(res.feasible[e]) == int(w.peak <= int(M[e]))


def test_generic_evaluator_paper_examples(par, golden_dir):
    """Example 1's two schedules as explicit runs, and the staggered schedule of the SimS lower bound."""
    dev = torch.device("cuda:0")
    batches, want = [], []
    for ln in open(os.path.join(golden_dir, "example1_memory.txt")):
        if ln.startswith("#") or not ln.strip():
            continue
        head, cells = ln.split(":")
        fam, k, tau, _ = head.split()
        k, tau = int(k), int(tau)
        starts = [(i * tau) // k if fam == "SPS" else (i // k) * tau for i in range(15)]
        batches.append((starts, [5] * 15, [0] * 15))
        want.append([int(x) for x in cells.split()])
    o, d, n = 60, 23, 12
    batches.append(([i * d for i in range(n)], [o] * n, [0] * n))
    off, st, ln_, ss = _runs_to_gpu(batches, dev)
    cap = torch.tensor([19, 25, (n - 1) * d + o], dtype=torch.int64, device=dev)
    res = par.scheduler().evaluate_runs(off, st, ln_, ss, cap)
    prof, poff = res.profile.cpu().numpy(), res.profile_off.cpu().numpy()
    assert list(prof[poff[0]:poff[1]]) == want[0] and list(prof[poff[1]:poff[2]]) == want[1]
    assert res.peak.cpu().tolist() == [15, 15, 3 * o - 3 * d]


def test_generic_evaluator_clips_at_capacity(par):
    dev = torch.device("cuda:0")
    off, st, ln, ss = _runs_to_gpu([([0, 4], [10, 3], [2, 1])], dev)
    res = par.scheduler().evaluate_runs(off, st, ln, ss, torch.tensor([6], dtype=torch.int64, device=dev))
    from paper_2601_22996_b200 import binding
    assert res.status.cpu().tolist() == [binding.EVAL_CAPACITY] and int(res.horizon[0]) == 10
    assert res.profile.cpu().tolist() == [3, 4, 5, 6, 7 + 2, 8 + 3]
