"""Variants inside the geometric classes on the GPU against the oracle: simultaneous batches as the
subroutine of every phase, the parallelism of a phase sized by the longest prompt among its participants,
and the sweep over tunable initial slices.  Bit-exact, every output."""
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


@pytest.mark.parametrize("sub,pc", [(1, 0), (0, 1), (1, 1)])
def test_tiny_instances_all_variants(par, sub, pc):
    inst = workloads.random_small(4100 + 10 * sub + pc, 60, 48, 30, 90)
    sizes = (inst.job_off[1:] - inst.job_off[:-1]).numpy()
    rows = []
    for i in range(inst.n_instances):
        if sizes[i] == 0:
            continue
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        M = int(inst.s[a:b].max() + inst.o[a:b].max()) + 7 * i
        for fam in ("GBA", "GSA"):
            for alpha in ((2, 1), (3, 2)):
                rows.append(dict(instance=i, family=fam, M=M, alpha=alpha, subroutine=sub, per_class_s=pc))
            rows.append(dict(instance=i, family=fam, M=M, beta0=3, subroutine=sub, per_class_s=pc))
    par.check_batch(inst, binding.make_settings(rows), label=f"variants sub={sub} pc={pc}")


def test_variants_with_estimates_and_windows(par):
    inst = workloads.random_small(4200, 24, 64, 25, 80, with_est=True)
    # arrivals: nondecreasing per instance, a few windows each
    arr = torch.zeros_like(inst.o, dtype=torch.int64)
    for i in range(inst.n_instances):
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        arr[a:b] = torch.arange(b - a, dtype=torch.int64) * 3
    inst.arrival = arr
    rows = []
    for i in range(inst.n_instances):
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        if b == a:
            continue
        M = int(inst.s[a:b].max() + max(int(inst.o[a:b].max()), 1)) + 40
        for fam in ("GBA", "GSA"):
            for sub, pc in ((1, 0), (0, 1), (1, 1)):
                rows.append(dict(instance=i, family=fam, M=M, subroutine=sub, per_class_s=pc))
    par.check_batch(inst, binding.make_settings(rows), window=37, label="variants est+windows")


def test_config2_subset_variants(par):
    inst = workloads.config2(n_inst=4, n=10_000)
    st = np.concatenate([binding.settings_grid(range(4), ["GBA", "GSA"], [1 << 17, 1 << 21], subroutine=1),
                         binding.settings_grid(range(4), ["GBA", "GSA"], [1 << 18, 1 << 24], per_class_s=1),
                         binding.settings_grid(range(4), ["GBA", "GSA"], [1 << 19], subroutine=1, per_class_s=1)])
    par.check_batch(inst, st, want_runs=False, label="config 2 variants")


def test_uniform_experiment_both_subroutines(par):
    """The uniform experiment of the paper (n = 200, o = 16, s = 0, M = 256, alpha = 2): the batching algorithm
    gives 14083 with the staggered pipeline and, with simultaneous batches inside the same class, the
    simultaneous number 21632."""
    inst = workloads.Instances(torch.tensor([0, 200]), torch.zeros(200, dtype=torch.int32), torch.full((200,), 16, dtype=torch.int32))
    st = binding.make_settings([dict(instance=0, family="GBA", M=256), dict(instance=0, family="GBA", M=256, subroutine=1)])
    res = par.scheduler().evaluate(inst.to("cuda:0"), st, want_jobs=False)
    assert res.flow.tolist() == [14083, 21632] and res.status.tolist() == [0, 0]


def test_rejects_variants_on_other_families(par):
    inst = workloads.config1().to("cuda:0")
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(inst, binding.make_settings([dict(instance=0, family="SPS", M=200_000, subroutine=1)]))


@pytest.mark.parametrize("fam", ["GBA", "GSA"])
def test_sweep_over_initial_slices(par, fam):
    inst = workloads.config2(n_inst=2, n=3000)
    one = inst.slice(1, 2)
    beta0 = [0, 1, 5, 64, 256, 5000]
    M = 1 << 18
    for sub in (0, 1):
        out = {f: t.cpu().numpy() for f, t in par.scheduler().sweep_beta0(inst.to("cuda:0"), 1, fam, M, beta0, subroutine=sub).items()}
        for i, b0 in enumerate(beta0):
            S = oracle.build_schedule(fam, one.s, one.o, M, beta0=b0, subroutine=sub)
            E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s, want_profile=False)
            got = tuple(int(out[f][i]) for f in ("peak", "flow", "horizon", "job_steps", "n_completed", "feasible"))
            assert got == (E.peak, S.flow, S.horizon, S.job_steps, 3000 - S.n_unfinished, int(E.peak <= M)), (fam, b0, sub)
    # an infeasible budget: nothing is scheduled and the cell says so
    out = par.scheduler().sweep_beta0(inst.to("cuda:0"), 1, fam, 100, [0, 64])
    assert out["feasible"].tolist() == [0, 0] and out["n_completed"].tolist() == [0, 0] and out["peak"].tolist() == [-1, -1]
