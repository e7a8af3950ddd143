"""Dynamic refill of the batching schedule (GBA-D) on the GPU against the oracle: every job's start and
completion, the refilled profile, peak, flow and horizon, bit for bit."""
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
    inst = workloads.Instances(torch.tensor([0, 6]), torch.full((6,), 2, dtype=torch.int32), torch.tensor([1, 1, 2, 3, 5, 8], dtype=torch.int32))
    st = binding.make_settings([dict(instance=0, family="GBAD", M=10), dict(instance=0, family="GBA", M=10)])
    res = par.scheduler().evaluate(inst.to("cuda:0"), st, want_jobs=True, want_profile=True)
    assert res.job_start[:6].tolist() == [0, 0, 0, 1, 1, 5] and res.job_start[6:].tolist() == [0, 0, 1, 3, 7, 15]
    assert res.flow.tolist() == [27, 46] and res.horizon.tolist() == [13, 23] and res.peak.tolist() == [10, 10]
    a = int(res.profile_off[0])
    assert res.profile[a:a + 13].tolist() == [9, 10, 8, 10, 6, 10, 4, 5, 6, 7, 8, 9, 10]


def test_tiny_instances(par):
    inst = workloads.random_small(5100, 80, 60, 30, 90)
    rows = []
    for i in range(inst.n_instances):
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        if b == a:
            continue
        M = int(inst.s[a:b].max() + inst.o[a:b].max()) + 9 * i
        for alpha in ((2, 1), (3, 2), (4, 3)):
            rows.append(dict(instance=i, family="GBAD", M=M, alpha=alpha))
        rows.append(dict(instance=i, family="GBAD", M=M, beta0=4, per_class_s=1))
        rows.append(dict(instance=i, family="GBA", M=M))          # other families beside it in one call
        rows.append(dict(instance=i, family="GSA", M=M))
    par.check_batch(inst, binding.make_settings(rows), want_runs=False, label="refill tiny")


def test_config2_subset(par):
    """Several tiles of profile, thousands of admissions per evaluation, dense and sparse classes."""
    inst = workloads.config2(n_inst=3, n=10_000)
    st = binding.settings_grid(range(3), ["GBAD"], [1 << 17, 1 << 19, 1 << 22])
    par.check_batch(inst, st, want_runs=False, label="refill config 2")
    res_d = par.scheduler().evaluate(inst.to("cuda:0"), st, want_jobs=True, want_profile=True)
    st_b = st.copy()
    st_b["family"] = binding.GBA
    res_b = par.scheduler().evaluate(inst.to("cuda:0"), st_b, want_jobs=True, want_profile=True)
    assert bool((res_d.job_start <= res_b.job_start).all()) and bool((res_d.flow < res_b.flow).all())
    M = torch.from_numpy(np.ascontiguousarray(st["M"])).to(res_d.peak.device)
    assert bool((res_d.peak <= M).all()) and bool((res_d.feasible == 1).all())


def test_rejects_what_the_refill_is_not_defined_on(par):
    est = workloads.random_small(5200, 3, 20, 10, 30, with_est=True).to("cuda:0")
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(est, binding.make_settings([dict(instance=0, family="GBAD", M=500)]), want_profile=True)
    one = workloads.config1().to("cuda:0")
    with pytest.raises(binding.KvsError):      # no profile: the refill has no working storage
        par.scheduler().evaluate(one, binding.make_settings([dict(instance=0, family="GBAD", M=200_000)]), want_profile=False)
