"""Speculative runs on top of the slicing schedule (GSA-Spec) on the GPU against the oracle: every job's start and
completion, the per-round memory, peak, flow, horizon, executed runs and job-steps, bit for bit."""
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


def test_hand_worked_instance(par):
    """The instance of tests/golden/speculative_runs_hand_example.txt."""
    inst = workloads.Instances(torch.tensor([0, 3]), torch.zeros(3, dtype=torch.int32), torch.tensor([4, 4, 2], dtype=torch.int32))
    st = binding.make_settings([dict(instance=0, family="GSAS", M=6), dict(instance=0, family="GSA", M=6)])
    res = par.scheduler().evaluate(inst.to("cuda:0"), st, want_jobs=True, want_profile=True)
    assert res.job_start[:3].tolist() == [6, 8, 1] and res.job_completion[:3].tolist() == [10, 12, 3]
    assert res.job_completion[3:].tolist() == [10, 16, 5]
    assert res.flow.tolist() == [25, 31] and res.horizon.tolist() == [12, 16] and res.peak.tolist() == [6, 6]
    assert res.n_runs.tolist() == [11, 8] and res.job_steps.tolist() == [25, 19]
    a = int(res.profile_off[0])
    assert res.profile[a:a + 16].tolist() == [3, 3, 5, 5, 4, 3, 3, 5, 4, 6, 3, 4, 0, 0, 0, 0]


def test_tiny_instances(par):
    inst = workloads.random_small(6100, 80, 60, 30, 90)
    rows = []
    for i in range(inst.n_instances):
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        if b == a:
            continue
        M = int(inst.s[a:b].max() + inst.o[a:b].max()) + 9 * i
        for alpha in ((2, 1), (3, 2), (4, 3)):
            rows.append(dict(instance=i, family="GSAS", M=M, alpha=alpha))
        rows.append(dict(instance=i, family="GSAS", M=M, beta0=4))
        rows.append(dict(instance=i, family="GSAS", M=4 * M))
        rows.append(dict(instance=i, family="GSA", M=M))          # other families beside it in one call
        rows.append(dict(instance=i, family="GBAD", M=M))
    par.check_batch(inst, binding.make_settings(rows), want_runs=False, label="spec tiny")


def test_single_prompt_length_and_edges(par):
    """Equal prompt lengths (the paper's model), one job, a budget that one job fills, an empty instance."""
    rng = np.random.default_rng(6200)
    offs, s, o = [0], [], []
    for n, sv in ((1, 3), (0, 0), (40, 0), (200, 7), (3, 7), (64, 1)):
        s += [sv] * n
        o += rng.integers(1, 50, n).tolist()
        offs.append(offs[-1] + n)
    inst = workloads.Instances(torch.tensor(offs), torch.tensor(s, dtype=torch.int32), torch.tensor(o, dtype=torch.int32))
    rows = []
    for i in range(inst.n_instances):
        for M in (57, 64, 300, 5000):
            rows.append(dict(instance=i, family="GSAS", M=M))
    par.check_batch(inst, binding.make_settings(rows), want_runs=False, label="spec edges")


def test_config2_subset(par):
    """Thousands of jobs, profiles of several tiles, speculative runs by the hundred at the larger budgets; the
    pipeline is kept, so no job completes later than in the slicing schedule."""
    inst = workloads.config2(n_inst=2, n=3_000)
    st = binding.settings_grid(range(2), ["GSAS"], [1 << 17, 1 << 19])
    par.check_batch(inst, st, want_runs=False, label="spec config 2")
    res_s = par.scheduler().evaluate(inst.to("cuda:0"), st, want_jobs=True, want_profile=True)
    st_b = st.copy()
    st_b["family"] = binding.GSA
    res_b = par.scheduler().evaluate(inst.to("cuda:0"), st_b, want_jobs=True, want_profile=True)
    assert bool((res_s.job_completion <= res_b.job_completion).all()) and bool((res_s.flow < res_b.flow).all())
    M = torch.from_numpy(np.ascontiguousarray(st["M"])).to(res_s.peak.device)
    assert bool((res_s.peak <= M).all()) and bool((res_s.feasible == 1).all())


def test_rejects_what_speculation_is_not_defined_on(par):
    est = workloads.random_small(6300, 3, 20, 10, 30, with_est=True).to("cuda:0")
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(est, binding.make_settings([dict(instance=0, family="GSAS", M=500)]), want_profile=True)
    one = workloads.config1().to("cuda:0")
    with pytest.raises(binding.KvsError):      # no profile: no working storage
        par.scheduler().evaluate(one, binding.make_settings([dict(instance=0, family="GSAS", M=200_000)]), want_profile=False)
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(one, binding.make_settings([dict(instance=0, family="GSAS", M=200_000, subroutine=1)]), want_profile=True)
