"""kvs_bounds against the oracle's literal sums: UpperGBA, the GSA bound and the area lower bound are
integers that depend on an instance only through its class sizes, so the comparison is bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_22996_b200 import binding, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sched():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import parity
    return parity.scheduler()


def _check(sched, inst, settings, sample=None):
    got = {k: v.cpu().numpy() for k, v in sched.bounds(inst.to("cuda:0"), settings).items()}
    for e in (range(settings.shape[0]) if sample is None else sample):
        st = settings[e]
        i = int(st["instance"])
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        B = oracle.bounds(inst.s[a:b], inst.o[a:b], int(st["M"]), alpha=(int(st["alpha_num"]), int(st["alpha_den"])),
                          beta0=int(st["beta0"]), s_bar=int(st["s_bar"]))
        tag = f"eval {e} inst {i} M {int(st['M'])}"
        if B.status == 1:
            assert int(got["status"][e]) == binding.EVAL_INFEASIBLE, tag
        elif B.status == 2:
            assert int(got["status"][e]) == 2, tag
        else:
            assert B.status == 0 and int(got["status"][e]) == 0, tag
            assert (int(got["upper_gba"][e]), int(got["upper_gsa"][e]), int(got["lower_2m"][e])) == \
                   (B.upper_gba, B.upper_gsa, B.lower_2m), tag
    return got


def test_worked_example(sched):
    off = torch.tensor([0, 6], dtype=torch.int64)
    inst = workloads.Instances(off, torch.full((6,), 2, dtype=torch.int32), torch.tensor([1, 1, 2, 3, 5, 8], dtype=torch.int32))
    got = _check(sched, inst, binding.make_settings([dict(instance=0, family="GBA", M=10)]))
    assert (int(got["upper_gba"][0]), int(got["upper_gsa"][0]), int(got["lower_2m"][0])) == (57, 93, 174)


@pytest.mark.parametrize("alpha", [(2, 1), (3, 2), (4, 3), (7, 4)])
def test_random_small_instances(sched, alpha):
    inst = workloads.config2(n_inst=24, n=257)
    I = inst.n_instances
    Ms = [int(inst.s.max()) + int(inst.o.max()) + 3, 1 << 15, 1 << 20]
    st = binding.settings_grid(range(I), ["GBA"], Ms, alpha=alpha)
    _check(sched, inst, st)
    st2 = st.copy()
    st2["beta0"] = 3
    st2["s_bar"] = 7            # a caller-chosen prompt length for the ladder
    _check(sched, inst, st2)


def test_config1_and_config2_settings(sched):
    inst = workloads.config1()
    _check(sched, inst, binding.settings_grid(range(1), ["GBA"], inst.meta["M"]))
    inst = workloads.config2(n_inst=16, n=10_000)
    _check(sched, inst, binding.settings_grid(range(16), ["GSA"], inst.meta["M"]))


def test_empty_infeasible_and_large(sched):
    off = torch.tensor([0, 0, 2], dtype=torch.int64)
    inst = workloads.Instances(off, torch.tensor([3, 3], dtype=torch.int32), torch.tensor([4, 90], dtype=torch.int32))
    got = _check(sched, inst, binding.make_settings([dict(instance=0, family="GBA", M=50), dict(instance=1, family="GBA", M=50),
                                                     dict(instance=1, family="GBA", M=500)]))
    assert got["status"].tolist() == [0, binding.EVAL_INFEASIBLE, 0] and int(got["upper_gba"][0]) == 0
    # one instance of a million jobs: the sums stay below 2^63 and the floor sums are closed forms
    big = workloads.config4()
    _check(sched, big, binding.settings_grid(range(1), ["GBA"], [1 << 22, 1 << 24]))
    with pytest.raises(binding.KvsError):
        sched.bounds(big.to("cuda:0"), binding.make_settings([dict(instance=0, family="GBA", M=1 << 22, alpha=(2, 2))]))


def test_config5_sampled(sched):
    import bench
    inst = bench.make_instances("c5", 2048, torch.device("cuda:0"))
    settings, _ = bench.make_settings("c5", inst, ["GBA"])
    cpu = inst.to("cpu")
    got = _check(sched, cpu, settings, sample=sorted(np.random.default_rng(9).choice(settings.shape[0], 16, replace=False)))
    assert int((torch.from_numpy(got["status"]) != 0).sum()) == 0
    assert bool((got["upper_gba"] <= got["upper_gsa"]).all()) and bool((got["lower_2m"] > 0).all())
