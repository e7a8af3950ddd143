"""Parity of the CUDA path against the CPU oracle, through the C ABI.  Bit-exact: every
quantity is an int32/int64 token or round count."""
import numpy as np
import pytest
import torch

from paper_2601_22996_b200 import binding, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def par():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import parity
    return parity


def _all_settings(inst, M_of, families=("GBA", "GSA", "SPS", "SIMS"), alpha=(2, 1), **extra):
    rows = []
    for i in range(inst.n_instances):
        for fam in families:
            rows.append(dict(instance=i, family=fam, M=M_of(i), alpha=alpha, **extra))
    return binding.make_settings(rows)


def _tight_M(inst, slack):
    """Budget per instance: largest s + largest o + slack (so that every job fits alone)."""
    out = []
    for i in range(inst.n_instances):
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        out.append((int(inst.s[a:b].max()) + int(inst.o[a:b].max()) if b > a else 2) + slack)
    return out


@pytest.mark.parametrize("alpha", [(2, 1), (3, 2), (4, 3), (7, 4)])
@pytest.mark.parametrize("seed", [1, 2])
def test_tiny_random_instances_all_families(par, alpha, seed):
    inst = workloads.random_small(seed * 100 + alpha[0], n_inst=150, n_max=64, s_max=40, o_max=90,
                                  equal_s=(seed == 2))
    M = _tight_M(inst, slack=17 * seed + 40)
    st = _all_settings(inst, lambda i: M[i], alpha=alpha)
    par.check_batch(inst, st, label=f"tiny a={alpha}")


def test_tiny_tight_budget_and_explicit_parameters(par):
    inst = workloads.random_small(7, n_inst=120, n_max=48, s_max=9, o_max=30)
    M = _tight_M(inst, slack=0)                       # k* = 1 in the last phases
    rows = []
    for i in range(inst.n_instances):
        rows += [dict(instance=i, family="GBA", M=M[i]), dict(instance=i, family="GSA", M=M[i]),
                 dict(instance=i, family="SPS", M=M[i] + 50, tau=1 + i % 7, k=1 + i % 5),       # unfinished jobs
                 dict(instance=i, family="SIMS", M=M[i] + 50, tau=3 + i % 11, k=1 + i % 4),
                 dict(instance=i, family="SPS", M=M[i] + 9, tau=35, k=200),                     # infeasible on purpose
                 dict(instance=i, family="GSA", M=M[i] + 100, s_bar=3),                         # s_bar below max s
                 dict(instance=i, family="GBA", M=M[i] + 300, beta0=4, alpha=(3, 2)),
                 dict(instance=i, family="GSA", M=M[i] + 300, beta0=64)]
    par.check_batch(inst, binding.make_settings(rows), label="explicit")


def test_estimates_and_windows(par):
    inst = workloads.random_small(11, n_inst=60, n_max=200, s_max=30, o_max=120, with_est=True)
    M = _tight_M(inst, slack=200)
    st = _all_settings(inst, lambda i: M[i], alpha=(2, 1))
    par.check_batch(inst, st, label="estimates")
    par.check_batch(inst, _all_settings(inst, lambda i: M[i], families=("GBA", "GSA"), alpha=(3, 2)), label="estimates 3/2")
    g = torch.Generator().manual_seed(5)               # arrivals: nondecreasing per instance
    arr = torch.zeros_like(inst.s, dtype=torch.int64)
    for i in range(inst.n_instances):
        a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
        arr[a:b] = torch.sort(torch.randint(0, 900, (b - a,), generator=g)).values
    inst.arrival = arr
    for W in (1, 37, 256, 5000):
        par.check_batch(inst, st, window=W, label=f"window {W}")
    inst.o_est = None
    par.check_batch(inst, st, window=64, label="window exact")


def test_config1_single_instance(par):
    inst = workloads.config1()
    for alpha in [(2, 1), (4, 3), (3, 2)]:
        st = _all_settings(inst, lambda i: 200_000, alpha=alpha)
        assert par.check_batch(inst, st, label="config1") > 0


def test_config2_subset_full_compare(par):
    inst = workloads.config2(n_inst=6)
    st = binding.settings_grid(range(6), ["GBA", "GSA"], inst.meta["M"])
    par.check_batch(inst, st, label="config2")


def test_config3_subset_online(par):
    inst = workloads.config3(n_inst=2, n=100_000)
    st = binding.settings_grid(range(2), ["GBA", "GSA"], inst.meta["M"])
    par.check_batch(inst, st, window=inst.meta["window"], label="config3")
    st = binding.settings_grid(range(2), ["SPS", "SIMS"], inst.meta["M"])
    par.check_batch(inst, st, window=inst.meta["window"], want_runs=False, label="config3 sps")


def test_config5_subset_mixed(par):
    inst = workloads.config5(n_inst=12)
    M = inst.meta["M_per_instance"].numpy()
    st = binding.settings_grid(range(12), ["GBA", "GSA"], M[:, None])
    par.check_batch(inst, st, want_runs=False, label="config5 geo")
    st = binding.settings_grid(range(12), ["SPS", "SIMS"], M[:, None])
    par.check_batch(inst, st, want_runs=False, want_profile=False, label="config5 sps")


def test_large_single_instance(par):
    inst = workloads.config4(n=300_000)
    st = binding.settings_grid([0], ["GBA", "GSA"], [1 << 22, 1 << 19])
    par.check_batch(inst, st, want_runs=False, label="big")


def test_many_runs_per_round_over_several_tiles(par):
    """Short prompts and a budget of some ten thousand tokens: the early phases of the geometric
    families start eight or more runs per round (k >= 8 tau) and, with 150,000 jobs, still last
    several tiles of rounds; with estimates both families carry killed jobs over."""
    g = torch.Generator().manual_seed(77)
    n = 150_000
    s = torch.randint(0, 4, (n,), generator=g, dtype=torch.int32)
    short = torch.randint(1, 41, (n,), generator=g, dtype=torch.int32)
    long_ = torch.randint(41, 401, (n,), generator=g, dtype=torch.int32)
    o = torch.where(torch.rand(n, generator=g) < 0.6, short, long_)
    inst = workloads.Instances(torch.tensor([0, n], dtype=torch.int64), s, o)
    st = binding.settings_grid([0], ["GBA", "GSA"], [35_003, 9_001, 300_007])
    par.check_batch(inst, st, want_runs=False, label="many runs per round")
    noise = torch.exp(0.5 * torch.randn(n, generator=g, dtype=torch.float64))
    inst.o_est = torch.clamp(torch.round(o.to(torch.float64) * noise), 1, 400).to(torch.int32)
    par.check_batch(inst, binding.settings_grid([0], ["GBA", "GSA"], [35_003]), want_runs=False, label="many runs per round, estimates")


def test_empty_and_degenerate(par):
    off = torch.tensor([0, 0, 1, 1, 4], dtype=torch.int64)
    inst = workloads.Instances(off, torch.tensor([5, 0, 0, 0], dtype=torch.int32), torch.tensor([3, 1, 1, 1], dtype=torch.int32))
    rows = [dict(instance=i, family=f, M=20) for i in range(4) for f in ("GBA", "GSA", "SPS", "SIMS")]
    rows += [dict(instance=3, family="GBA", M=1), dict(instance=1, family="GSA", M=8), dict(instance=1, family="GSA", M=7)]
    par.check_batch(inst, binding.make_settings(rows), label="degenerate")


def test_status_reports(par):
    dev = torch.device("cuda:0")
    off = torch.tensor([0, 3, 6, 9], dtype=torch.int64)
    s = torch.tensor([1, 2, 3, 1, 2, 3, 1, -2, 3], dtype=torch.int32)
    o = torch.tensor([4, 90, 6, 4, 0, 6, 4, 5, 6], dtype=torch.int32)
    inst = workloads.Instances(off, s, o).to(dev)
    st = binding.make_settings([dict(instance=0, family="GBA", M=50), dict(instance=1, family="GBA", M=50),
                                dict(instance=2, family="GSA", M=50), dict(instance=0, family="GBA", M=200)])
    res = par.scheduler().evaluate(inst, st, want_profile=True)
    status = res.status.cpu().tolist()
    assert status[0] == binding.EVAL_INFEASIBLE          # o = 90 > M - s_bar
    assert status[1] == binding.EVAL_BAD_INPUT           # o = 0
    assert status[2] == binding.EVAL_BAD_INPUT           # s < 0
    assert status[3] == 0 and res.feasible.cpu().tolist() == [0, 0, 0, 1]
    # capacity: a profile shorter than the horizon is clipped and flagged, scalars stay exact
    full = par.scheduler().evaluate(inst, st[3:], want_profile=True)
    cap = torch.tensor([5], dtype=torch.int64, device=dev)
    clip = par.scheduler().evaluate(inst, st[3:], want_profile=True, profile_capacity=cap)
    assert clip.status.cpu().tolist() == [binding.EVAL_CAPACITY]
    assert torch.equal(clip.profile, full.profile[:5]) and torch.equal(clip.peak, full.peak)
    # argument errors are found on the host, before any launch
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(inst, binding.make_settings([dict(instance=5, family="GBA", M=50)]))
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(inst, binding.make_settings([dict(instance=0, family="GBA", M=50, alpha=(2, 2))]))
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(inst, binding.make_settings([dict(instance=0, family="GBA", M=1 << 24, alpha=(11, 10))]))
    with pytest.raises(binding.KvsError):
        par.scheduler().evaluate(inst, binding.make_settings([dict(instance=0, family=7, M=50)]))


def test_int64_times(par):
    """Horizon beyond 2^31: 32-bit outputs are flagged, 64-bit outputs are exact."""
    import oracle
    dev = torch.device("cuda:0")
    n = 3000
    inst = workloads.Instances(torch.tensor([0, n], dtype=torch.int64), torch.zeros(n, dtype=torch.int32),
                               torch.full((n,), 1_000_000, dtype=torch.int32))
    st = binding.make_settings([dict(instance=0, family="SPS", M=1_000_000)])      # k* = 1: horizon 3e9
    r32 = par.scheduler().evaluate(inst.to(dev), st)
    assert r32.status.cpu().tolist() == [binding.EVAL_RANGE]
    r64 = par.scheduler().evaluate(inst.to(dev), st, time64=True)
    S = oracle.build_schedule("SPS", inst.s, inst.o, 1_000_000)
    assert r64.status.cpu().tolist() == [0] and int(r64.horizon[0]) == S.horizon == 3_000_000_000
    assert np.array_equal(r64.job_completion.cpu().numpy(), S.job_completion) and int(r64.flow[0]) == S.flow
    assert int(r64.peak[0]) == oracle.evaluate_events(S.run_start, S.run_len, S.run_s).peak


def test_host_entry_point(par):
    """kvs_evaluate_built_host (host buffers in, scalars out, copies pipelined with the kernels over chunks of
    instances) against the oracle, with the evaluations in instance order and in a shuffled order."""
    import oracle
    from paper_2601_22996_b200.api import Scheduler
    cases = [(workloads.config2(n_inst=37, n=1500), 0, ("GBA", "GSA", "SPS", "SIMS")),
             (workloads.config3(n_inst=5, n=6000), None, ("GBA", "GSA"))]
    for inst, window, fams in cases:
        if window is None:
            window = inst.meta["window"]
        I = inst.n_instances
        st = binding.settings_grid(range(I), fams, [inst.meta["M"][len(inst.meta["M"]) // 2]])
        n = int((inst.job_off[1:] - inst.job_off[:-1]).max())
        sched = par.scheduler()
        for order in (np.arange(st.shape[0]), np.random.default_rng(7).permutation(st.shape[0])):
            s2 = np.ascontiguousarray(st[order])
            P = s2.shape[0]
            ctx = sched.context(binding.workspace_bytes(int(inst.s.numel()), I, n, P, host_staging=True))
            hev = {k: torch.full_like(v, -5, device="cpu").pin_memory() for k, v in Scheduler.scalars(P, "cpu").items()}
            hin = workloads.Instances(inst.job_off, inst.s.pin_memory(), inst.o.pin_memory(),
                                      None if inst.o_est is None else inst.o_est.pin_memory(),
                                      None if inst.arrival is None else inst.arrival.pin_memory())
            ctx.evaluate_built_host(hin, s2, hev, window=window, max_jobs=n)
            for e in range(0, P, max(1, P // 40)):
                S = par.oracle_eval(inst, s2[e], window)
                assert S.status == 0 and int(hev["status"][e]) == 0
                assert (int(hev["flow"][e]), int(hev["horizon"][e]), int(hev["job_steps"][e]), int(hev["n_unfinished"][e])) == \
                       (S.flow, S.horizon, S.job_steps, S.n_unfinished)
                E = oracle.evaluate_dense(S.run_start, S.run_len, S.run_s, want_profile=False)
                assert int(hev["peak"][e]) == E.peak and int(hev["feasible"][e]) == int(E.peak <= int(s2[e]["M"]))
