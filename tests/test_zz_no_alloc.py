"""The allocation-free evaluator entry point against the workspace-based one.

Some users of this library run inside a process that owns all GPU memory through its own pool,
or inside a loop that must never touch the CUDA allocator; they cannot hand the library a
workspace.  kvs_evaluate_schedule_noalloc serves them from a fixed array inside the library.
This test calls it through the C ABI twice in a row, with different run lists, and requires the
same outputs, bit for bit, as kvs_evaluate_schedule and as the CPU oracle's literal evaluation
of the same runs (all outputs are integers, so the tolerance is zero, as everywhere in the GPU
tests).  The second call checks that nothing left in the shared array by the first call leaks
into the result.  A third test hands the kernel device offsets that disagree with the size the
host stated: the evaluation concerned must come back with a status and without a single write.
The file name sorts last on purpose.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _random_runs(seed, P, dev):
    rng = np.random.default_rng(seed)
    counts = rng.integers(0, 2500, P)
    counts[0], counts[P - 1] = 0, 1000
    off = np.zeros(P + 1, dtype=np.int64)
    off[1:] = np.cumsum(counts)
    R = int(off[-1])
    start = rng.integers(0, 15000, R).astype(np.int64)
    length = rng.integers(1, 700, R).astype(np.int32)
    s = rng.integers(0, 3000, R).astype(np.int32)
    cap = np.zeros(P, dtype=np.int64)
    for e in range(P):
        a, b = off[e], off[e + 1]
        cap[e] = int((start[a:b] + length[a:b]).max()) if b > a else 0
    cap[P - 1] = max(0, cap[P - 1] - 40)          # one evaluation clipped at its capacity
    t = lambda x: torch.from_numpy(x).to(dev)
    return dict(run_off=t(off), run_start=t(start), run_len=t(length), run_s=t(s),
                M=t(rng.integers(1000, 400000, P).astype(np.int64))), t(cap)


def test_noalloc_matches_workspace_entry_point_twice():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2601_22996_b200 import binding
    from paper_2601_22996_b200.api import Scheduler
    dev = torch.device("cuda:0")
    sched = Scheduler()
    for seed, P in ((101, 30), (202, 17)):         # two calls in a row on the shared array
        runs, cap = _random_runs(seed, P, dev)
        ref = sched.evaluate_runs(runs["run_off"], runs["run_start"], runs["run_len"], runs["run_s"], cap, M=runs["M"])
        ev = Scheduler.scalars(P, dev)
        ev["profile_off"] = ref.profile_off.clone()
        total = int(ref.profile_off[-1])
        ev["profile"] = torch.full((total,), -7, dtype=torch.int32, device=dev)
        binding.evaluate_schedule_noalloc(runs, ev, total)
        torch.cuda.synchronize()
        for name in ("status", "peak", "horizon", "job_steps", "flow", "feasible"):
            assert torch.equal(ev[name], getattr(ref, name)), name
        assert torch.equal(ev["profile"], ref.profile)
        assert int(ev["status"][P - 1]) == binding.EVAL_CAPACITY and int(ev["status"][1]) == 0
        # and against the oracle's definition, evaluation by evaluation (the clipped one excepted)
        import oracle
        off = runs["run_off"].cpu().numpy()
        poff = ev["profile_off"].cpu().numpy()
        start, length, s_ = (runs[k].cpu().numpy() for k in ("run_start", "run_len", "run_s"))
        prof = ev["profile"].cpu().numpy()
        for e in range(P - 1):
            a, b = int(off[e]), int(off[e + 1])
            E = oracle.evaluate_dense(start[a:b], length[a:b], s_[a:b])
            assert (int(ev["peak"][e]), int(ev["horizon"][e]), int(ev["job_steps"][e])) == (E.peak, E.horizon, E.job_steps), e
            assert np.array_equal(prof[int(poff[e]):int(poff[e + 1])].astype(np.int64), E.profile), e


def test_noalloc_device_offsets_beyond_the_stated_capacity_are_reported_not_written():
    """The host says 4,000 rounds in all; on the device the last evaluation claims 9,000 more and the
    one before it has offsets that run backwards.  Both lie far inside the built-in array either way,
    so no access could leave it; the kernel must still refuse them (status, no writes) and evaluate
    the honest ones."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2601_22996_b200 import binding
    from paper_2601_22996_b200.api import Scheduler
    dev = torch.device("cuda:0")
    t = lambda x, d: torch.tensor(x, dtype=d, device=dev)
    runs = dict(run_off=t([0, 2, 4, 6, 8], torch.int64), run_start=t([0, 5, 0, 3, 1, 2, 0, 10], torch.int64),
                run_len=t([10, 20, 7, 9, 4, 4, 30, 50], torch.int32), run_s=t([3, 1, 4, 1, 5, 9, 2, 6], torch.int32),
                M=t([100, 100, 100, 100], torch.int64))
    ev = Scheduler.scalars(4, dev)
    ev["profile_off"] = t([0, 1000, 3000, 2500, 13000], torch.int64)      # host copy below: 4,000
    ev["profile"] = torch.full((13000,), -7, dtype=torch.int32, device=dev)
    binding.evaluate_schedule_noalloc(runs, ev, 4000)
    torch.cuda.synchronize()
    bad = binding.EVAL_CAPACITY | binding.EVAL_BAD_INPUT
    assert ev["status"].tolist() == [0, 0, bad, bad]
    assert ev["peak"].tolist()[2:] == [-1, -1] and ev["job_steps"].tolist() == [30, 16, 0, 0]
    assert bool((ev["profile"][2500:] == -7).all())                       # nothing of the refused ones written
    import oracle
    E = oracle.evaluate_dense(np.array([0, 5]), np.array([10, 20]), np.array([3, 1]))
    assert int(ev["peak"][0]) == E.peak and np.array_equal(ev["profile"][:25].cpu().numpy(), E.profile)


def test_noalloc_rejects_sizes_beyond_the_built_in_array():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2601_22996_b200 import binding
    from paper_2601_22996_b200.api import Scheduler
    dev = torch.device("cuda:0")
    runs, _ = _random_runs(5, 3, dev)
    ev = Scheduler.scalars(3, dev)
    ev["profile_off"] = torch.tensor([0, 1 << 20, 1 << 20, 1 << 20], dtype=torch.int64, device=dev)
    with pytest.raises(binding.KvsError) as info:
        binding.evaluate_schedule_noalloc(runs, ev, 1 << 20)       # 2^20 rounds + 3 evaluations > 2^20 slots
    assert info.value.code == -3 and "1,048,576" in str(info.value)
