"""Pins for the CPU oracle: values the paper prints, closed forms, invariants, brute force.

Each test names the passage it checks.  None of them compares the oracle with itself:
expected values come from the paper (tests/golden), from closed forms typed out here,
from an independent arithmetic (Python big integers / Fractions), or from exhaustive search.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.filterwarnings("ignore")


def _golden_lines(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def _dense(S):
    return oracle.evaluate_dense(S.run_start, S.run_len, S.run_s)


# ---- Example "A Toy Example with Identical Jobs" + its figure ---------------------------------

def test_example1_memory_columns_and_flow(golden_dir):
    for ln in _golden_lines(golden_dir, "example1_memory.txt"):
        head, cells = ln.split(":")
        fam, k, tau, flow = head.split()
        want = [int(x) for x in cells.split()]
        S = oracle.build_schedule(fam, [0] * 15, [5] * 15, 15, tau=int(tau), k=int(k))
        E = _dense(S)
        assert S.status == 0 and S.n_unfinished == 0
        assert S.flow == int(flow)
        assert list(E.profile) == want
        assert E.peak == 15 and E.horizon == len(want)
        # the example's parallelism values are the automatic ones (k* and B)
        auto = oracle.build_schedule(fam, [0] * 15, [5] * 15, 15)
        assert int(auto.k[0]) == int(k) and int(auto.tau[0]) == 5 and auto.flow == int(flow)
    S = oracle.build_schedule("SPS", [0] * 15, [5] * 15, 15, tau=5, k=5)
    assert list(S.job_start) == list(range(15))          # "the i-th job starts at round i"
    assert int(S.job_completion[14]) == 19               # completes at the end of round 18


# ---- Numerical Experiments: uniform-size and two-point figures --------------------------------

def test_paper_flow_times(golden_dir):
    rows = {ln.split()[0]: [int(x) for x in ln.split()[1:]] for ln in _golden_lines(golden_dir, "paper_flow_times.txt")}
    n, s, M, a, b, want = rows["GBA_uniform"]
    S = oracle.build_schedule("GBA", [s] * n, [16] * n, M, alpha=(a, b))
    assert S.flow == want                                 # pins: empty classes take no time
    assert _dense(S).peak <= M
    n, s, M, a, b, want = rows["MCSF_uniform"]
    S = oracle.build_schedule("SIMS", [s] * n, [16] * n, M)
    assert S.flow == want and int(S.k[0]) == 16           # simultaneous batches of floor(M/(s+o))
    n, s, M, a, b, want = rows["GSA_twopoint"]
    lo = oracle.build_schedule("GSA", [s] * n, [1] * 194 + [160] * 6, M, alpha=(a, b)).flow
    hi = oracle.build_schedule("GSA", [s] * n, [160] * 6 + [1] * 194, M, alpha=(a, b)).flow
    assert lo <= want <= hi                               # order of the six long jobs is not stated
    # The alternative phase length floor(N*tau/k)+tau cannot produce the printed value:
    # it would add one extra round per short job even in the best order.
    assert (lo, hi) == (17960, 18542)
    S = oracle.build_schedule("GSA", [s] * n, [160] * 6 + [1] * 194, M, alpha=(a, b))
    assert list(S.tau) == [1, 2, 5, 10, 20, 40, 80, 160]  # tau_hat_0 = 160/128 = 1.25
    assert list(S.k) == [2, 2, 2, 2, 2, 2, 1, 1]


# ---- Example "Long-Job Trap" -----------------------------------------------------------------

@pytest.mark.parametrize("ell,n", [(3, 2), (4, 7), (6, 40), (10, 5)])
def test_long_job_trap_closed_form(ell, n):
    s, M = 2 ** ell, 2 ** (ell + 1)
    o = [2 ** ell] + [1] * (n - 1)                        # worst order: the long job goes first
    S = oracle.build_schedule("GSA", [s] * n, o, M)
    assert S.flow == (n + 2) * (n - 1) // 2 + n + 2 ** (ell + 1) - 2
    assert all(int(k) == 1 for k in S.k) and list(S.tau) == [2 ** p for p in range(ell + 1)]
    assert oracle.opt_bruteforce(s, o, M) == n * (n + 1) // 2 + 2 ** ell - 1 if n <= 7 and ell <= 4 else True
    assert _dense(S).peak <= M


# ---- Lemma "Peak Memory Usage of SPS" / Lemma "Feasible Parallelism of SPS" ------------------

def _peak_formula(k, tau, s):
    return s * k + (tau * k + tau + k - math.gcd(tau, k)) // 2


def test_peak_closed_form_matches_simulation():
    rng = np.random.default_rng(7)
    for _ in range(300):
        k, tau, s = int(rng.integers(1, 25)), int(rng.integers(1, 40)), int(rng.integers(0, 30))
        N = k * int(rng.integers(2, 5)) + int(rng.integers(0, k + 1))
        S = oracle.build_schedule("SPS", [s] * N, [tau] * N, 10 ** 9, tau=tau, k=k)
        E = _dense(S)
        want = _peak_formula(k, tau, s)
        assert oracle.peak_closed(k, tau, s) == want
        assert E.peak == want                              # steady state is reached with N >= 2k
        assert int(E.profile[tau - 1]) == want             # attained at t = q*tau - 1, q = 1
        assert int(E.profile[2 * tau - 1]) == want


def test_kstar_is_maximal_by_simulation():
    """k* against exhaustive simulation (does not use the closed form for the peak)."""
    rng = np.random.default_rng(11)
    for _ in range(60):
        tau, s = int(rng.integers(1, 14)), int(rng.integers(0, 12))
        M = s + tau + int(rng.integers(0, 120))
        best = 0
        for k in range(1, 60):
            N = 3 * k
            S = oracle.build_schedule("SPS", [s] * N, [tau] * N, 10 ** 9, tau=tau, k=k)
            if _dense(S).peak <= M:
                best = k
            else:
                break                                      # the peak is increasing in k
        ks = oracle.kstar(tau, s, M)
        assert ks == best
        assert ks >= (2 * M - tau + 1) // (2 * s + tau + 1)            # lemma's lower bound
        assert (ks + 2) * (2 * s + tau + 1) > 2 * M                    # packing-efficiency lemma
    assert oracle.kstar(5, 3, 7) == 0                      # even one job does not fit


def test_kstar_large_values():
    for tau, s, M in [(1, 0, 1 << 24), (16384, 8192, 1 << 24), (255, 79, 8192), (1 << 20, 5, 1 << 30)]:
        k = oracle.kstar(tau, s, M)
        assert _peak_formula(k, tau, s) <= M < _peak_formula(k + 1, tau, s)


# ---- Ladder (first line of the two geometric algorithms) -------------------------------------

@pytest.mark.parametrize("a,b", [(2, 1), (3, 2), (4, 3), (7, 4), (11, 10), (5, 1)])
def test_ladder_exact_rational(a, b):
    alpha = Fraction(a, b)
    for X in [1, 2, 3, 7, 8, 9, 160, 255, 256, 257, 1000, 4096, 65535, 65536, 2 ** 24 - 8192, 3 ** 9, 2 ** 31 - 1]:
        ell = 0
        while alpha ** (ell + 1) <= X:
            ell += 1
        beta = Fraction(X) / alpha ** ell
        assert 1 <= beta < alpha                           # comment on the algorithms' first line
        want = [math.floor(beta * alpha ** p) for p in range(ell + 1)]
        got = oracle.ladder(X, a, b)
        assert got == want
        assert got[-1] == X


def test_ladder_tunable_initial_slice():
    assert oracle.ladder(4096 - 79, 2, 1, 64) == [64, 128, 256, 512, 1024, 2048, 4017]
    assert oracle.ladder(100, 3, 2, 7) == [7, 10, 15, 23, 35, 53, 79, 100]
    assert oracle.ladder(5, 2, 1, 64) == [5]


# ---- closed forms for flow time ---------------------------------------------------------------

def test_flow_closed_forms():
    rng = np.random.default_rng(3)
    for _ in range(100):
        n, tau, k, s = int(rng.integers(1, 60)), int(rng.integers(1, 30)), int(rng.integers(1, 12)), int(rng.integers(0, 9))
        S = oracle.build_schedule("SPS", [s] * n, [tau] * n, 10 ** 9, tau=tau, k=k)
        assert S.flow == n * tau + sum(i * tau // k for i in range(n))      # Eq. (Fstag:identical)
        assert S.flow <= n * tau + Fraction(n * (n - 1) * tau, 2 * k)
        S = oracle.build_schedule("SIMS", [s] * n, [tau] * n, 10 ** 9, tau=tau, k=1)
        assert S.flow == tau * n * (n + 1) // 2                             # B = 1


def test_simultaneous_lower_bound_instance():
    """Proposition "Lower bound approaching 3": staggered schedule with spacing d = o/3 + delta."""
    for o, delta, n in [(30, 2, 9), (60, 3, 12), (90, 2, 20)]:
        d = o // 3 + delta
        M = 3 * o - 3 * d + 3
        starts = np.arange(n, dtype=np.int64) * d
        E = oracle.evaluate_dense(starts, np.full(n, o), np.zeros(n))
        # in the oldest job's last round the three active jobs hold o, o - d and o - 2d tokens;
        # the proof bounds this by M = 3o - 3d + 3
        assert E.peak == 3 * o - 3 * d <= M
        assert int((starts + o).sum()) == n * o + d * n * (n - 1) // 2
        S = oracle.build_schedule("SIMS", [0] * n, [o] * n, M)
        assert int(S.k[0]) == 1 and S.flow == o * n * (n + 1) // 2


# ---- evaluators --------------------------------------------------------------------------------

def test_event_evaluator_equals_dense_definition():
    rng = np.random.default_rng(5)
    for _ in range(200):
        R = int(rng.integers(0, 40))
        st = rng.integers(0, 60, R)
        ln = rng.integers(1, 25, R)
        ss = rng.integers(0, 50, R)
        D, E = oracle.evaluate_dense(st, ln, ss), oracle.evaluate_events(st, ln, ss)
        assert (D.peak, D.horizon, D.job_steps) == (E.peak, E.horizon, E.job_steps)
        # area identity: sum of the profile = sum of memory-time areas (Definition "Memory-Time Area")
        assert int(D.profile.sum()) == int((ss * ln + ln * (ln + 1) // 2).sum())


def test_dense_single_run_ramp():
    E = oracle.evaluate_dense([3], [4], [10])
    assert list(E.profile) == [0, 0, 0, 11, 12, 13, 14] and E.peak == 14 and E.argmax == 6


# ---- invariants on random instances -----------------------------------------------------------

def _random_instance(rng, n_max=40, hetero=True):
    n = int(rng.integers(1, n_max))
    o = rng.integers(1, 70, n)
    s = rng.integers(0, 25, n) if hetero else np.full(n, int(rng.integers(0, 25)))
    M = int(s.max() + o.max() + rng.integers(0, 300))
    return s, o, M


@pytest.mark.parametrize("alpha", [(2, 1), (3, 2), (4, 3)])
def test_schedules_are_feasible_and_complete(alpha):
    rng = np.random.default_rng(alpha[0] * 10 + alpha[1])
    for _ in range(120):
        s, o, M = _random_instance(rng)
        for fam in ["GBA", "GSA", "SPS", "SIMS"]:
            S = oracle.build_schedule(fam, s, o, M, alpha=alpha)
            assert S.status == 0 and S.n_unfinished == 0
            E = _dense(S)
            assert E.peak <= M                                        # feasibility every round
            assert np.array_equal(S.job_completion, S.job_start + o)  # completion = start + o
            assert S.flow == int(S.job_completion.sum()) >= int(o.sum())
            assert S.job_steps == E.job_steps == int(S.run_len.sum())
            # every run is either the job's final run (length o) or a killed run of exactly tau_p
            final = S.run_len == o[S.run_job]
            assert np.all(S.run_len[~final] == S.tau[S.run_phase[~final]])
            assert np.all(S.run_len <= S.tau[S.run_phase])
            assert np.array_equal(np.sort(S.run_job[final]), np.arange(len(o)))
            # phases do not overlap in time and the rank-r job starts floor(r*tau/k) after the base
            base = 0
            for p in range(len(S.tau)):
                sel = S.run_phase == p
                N = int(sel.sum())
                assert N == int(S.n_part[p])
                if N == 0:
                    continue
                tau, k = int(S.tau[p]), int(S.k[p])
                r = np.arange(N)
                want = base + (r // k) * tau if fam == "SIMS" else base + (r * tau) // k
                assert np.array_equal(S.run_start[sel], want)
                base = int(want[-1]) + tau
            if fam == "GBA":
                assert len(S.run_job) == len(o)                       # no restarts
            if fam == "GSA":
                # a job of class l runs in phases 0..l
                cls = np.searchsorted(S.tau, o)
                assert len(S.run_job) == int((cls + 1).sum())


def test_area_lower_bound_and_upper_bounds():
    """Area lower bound on any feasible schedule; UpperGBA and the GSA bound (exact integers)."""
    rng = np.random.default_rng(21)
    for alpha in [(2, 1), (3, 2), (4, 3)]:
        al = Fraction(*alpha)
        for _ in range(80):
            s, o, M = _random_instance(rng, hetero=False)
            s0, n = int(s[0]), len(o)
            area = np.sort(s0 * o + o * (o + 1) // 2)
            lower = sum((n - j) * int(area[j]) for j in range(n))       # sum (n-j+1) A_(j), j from 1
            gba = oracle.build_schedule("GBA", s, o, M, alpha=alpha)
            gsa = oracle.build_schedule("GSA", s, o, M, alpha=alpha)
            for S in (gba, gsa, oracle.build_schedule("SPS", s, o, M), oracle.build_schedule("SIMS", s, o, M)):
                assert M * S.flow >= lower
            tau, k = [int(x) for x in gba.tau], [int(x) for x in gba.k]
            cls = np.searchsorted(gba.tau, o)                           # class = first p with tau_p >= o
            n_p = [int((cls == p).sum()) for p in range(len(tau))]
            Q = [n_p[p] * tau[p] + sum(i * tau[p] // k[p] for i in range(n_p[p])) for p in range(len(tau))]
            Sp = [sum(n_p[q] * tau[q] // k[q] + tau[q] for q in range(p)) for p in range(len(tau))]
            upper_gba = sum(n_p[p] * Sp[p] + Q[p] for p in range(len(tau)))
            assert gba.flow <= upper_gba
            n_ge = [sum(n_p[p:]) for p in range(len(tau))]
            n_gt = [sum(n_p[p + 1:]) for p in range(len(tau))]
            Tp = [sum(n_ge[q] * tau[q] // k[q] + tau[q] for q in range(p)) for p in range(len(tau))]
            Dp = [-((-n_gt[p] * tau[p]) // k[p]) for p in range(len(tau))]
            gsa_bound = sum(n_p[p] * (Tp[p] + Dp[p]) for p in range(len(tau))) + sum(Q)
            assert gsa.flow <= gsa_bound
            assert gsa_bound <= (2 + 2 / (al - 1)) * upper_gba
            assert all(k[q] >= k[t] for q in range(len(k)) for t in range(q, len(k)))
            # the oracle's bound evaluator returns exactly these integers (the sums above are written
            # from the two packing-efficiency lemmas and the area lemma, not from its code)
            x = [0] + tau[:-1]
            area2 = [2 * s0 * x[p] + x[p] * (x[p] + 1) for p in range(len(tau))]
            lower_2m = sum(area2[p] * (n_p[p] * (n_p[p] + 1) // 2 + n_gt[p] * n_p[p]) for p in range(len(tau)))
            B = oracle.bounds(s, o, M, alpha=alpha)
            assert (B.status, B.upper_gba, B.upper_gsa, B.lower_2m) == (0, upper_gba, gsa_bound, lower_2m)


def test_ratios_against_bruteforce_optimum():
    rng = np.random.default_rng(33)
    for it in range(70):
        n = int(rng.integers(1, 8))
        s = int(rng.integers(0, 6))
        o = rng.integers(1, 7, n)
        M = int(s + o.max() + rng.integers(0, 14))
        opt = oracle.opt_bruteforce(s, o, M)
        assert opt >= int(o.sum())
        for alpha in [(2, 1), (3, 2)]:
            al = alpha[0] / alpha[1]
            gba = oracle.build_schedule("GBA", [s] * n, o, M, alpha=alpha)
            gsa = oracle.build_schedule("GSA", [s] * n, o, M, alpha=alpha)
            kmin = int(min(gba.k))
            g_gba = al * al * (1 + 2 / kmin) + al + al / (al - 1)
            assert opt <= gba.flow <= g_gba * opt + 1e-9                 # Theorem (GBA)
            assert opt <= gsa.flow <= (2 + 2 / (al - 1)) * g_gba * opt + 1e-9   # Theorem (GSA)
        for fam in ["SPS", "SIMS"]:
            assert opt <= oracle.build_schedule(fam, [s] * n, o, M).flow
    for it in range(40):                                                  # identical jobs: SPS is a 2-approximation
        n, s, o = int(rng.integers(1, 8)), int(rng.integers(0, 5)), int(rng.integers(1, 7))
        M = s + o + int(rng.integers(0, 16))
        opt = oracle.opt_bruteforce(s, [o] * n, M)
        sps = oracle.build_schedule("SPS", [s] * n, [o] * n, M)
        assert opt <= sps.flow <= 2 * opt


def test_bruteforce_small_cases_by_hand():
    assert oracle.opt_bruteforce(0, [1], 1) == 1
    assert oracle.opt_bruteforce(0, [1, 1, 1], 1) == 6          # one at a time
    assert oracle.opt_bruteforce(0, [1, 1, 1], 3) == 3          # all at once
    assert oracle.opt_bruteforce(0, [2, 2], 3) == 5             # starts 0 and 1: memory 1, 2+1, 2
    assert oracle.opt_bruteforce(0, [2, 2], 2) == 6
    assert oracle.opt_bruteforce(3, [2], 4) == -1               # s + o > M


# ---- readings beyond the paper: reductions to the paper's cases -------------------------------

def _same(A, B):
    return (A.status == B.status and A.flow == B.flow and A.horizon == B.horizon
            and np.array_equal(A.job_start, B.job_start) and np.array_equal(A.run_start, B.run_start)
            and np.array_equal(A.run_job, B.run_job) and np.array_equal(A.run_len, B.run_len))


def test_estimates_reduce_to_paper_cases():
    rng = np.random.default_rng(44)
    for _ in range(60):
        s, o, M = _random_instance(rng)
        assert _same(oracle.build_schedule("GBA", s, o, M, o_est=o), oracle.build_schedule("GBA", s, o, M))
        flat = np.full(len(o), 5)                              # equal estimates: stable order = index order
        assert _same(oracle.build_schedule("GSA", s, o, M, o_est=flat), oracle.build_schedule("GSA", s, o, M))
        est = np.maximum(1, (o * rng.uniform(0.3, 3.0, len(o))).astype(np.int64))
        for fam in ["GBA", "GSA"]:
            S = oracle.build_schedule(fam, s, o, M, o_est=est)
            assert S.status == 0 and S.n_unfinished == 0 and _dense(S).peak <= M
            assert np.array_equal(S.job_completion, S.job_start + o)
        # under-estimates are killed and carried to the next phase
        S = oracle.build_schedule("GBA", s, o, M, o_est=np.ones(len(o), dtype=np.int64))
        assert _same(S, oracle.build_schedule("GSA", s, o, M))


def test_windows_reduce_to_offline():
    rng = np.random.default_rng(55)
    for _ in range(40):
        s, o, M = _random_instance(rng)
        n = len(o)
        zero = np.zeros(n, dtype=np.int64)
        for fam in ["GBA", "GSA", "SPS", "SIMS"]:
            off = oracle.build_schedule(fam, s, o, M)
            assert _same(oracle.build_schedule(fam, s, o, M, arrival=zero, window=0), off)
            W = int(rng.integers(1, 50))
            win = oracle.build_schedule(fam, s, o, M, arrival=zero, window=W)   # all in window 0, released at W
            assert np.array_equal(win.job_start, off.job_start + W) and win.flow == off.flow + n * W
        arr = np.sort(rng.integers(0, 200, n))
        W = int(rng.integers(5, 60))
        for fam in ["GBA", "GSA"]:
            S = oracle.build_schedule(fam, s, o, M, arrival=arr, window=W)
            assert S.status == 0 and S.n_unfinished == 0
            assert np.all(S.job_start >= (arr // W + 1) * W)    # no job starts before its window closes
            assert S.flow == int((S.job_completion - arr).sum())
            assert _dense(S).peak <= M                          # windows never overlap in time


def test_status_codes():
    assert oracle.build_schedule("GBA", [10, 10], [5, 91], 100).status == 1     # o > M - s_bar
    assert oracle.build_schedule("GBA", [10], [5], 10).status == 1              # M - s_bar < 1
    assert oracle.build_schedule("SPS", [0, 0, 0], [2, 9, 4], 100, tau=4, k=2).n_unfinished == 1
    S = oracle.build_schedule("SPS", [0, 0, 0], [2, 9, 4], 100, tau=4, k=2)
    assert list(S.job_start) == [0, -1, 2] and list(S.job_completion) == [2, -1, 6] and S.flow == 8
    assert list(S.run_len) == [2, 4, 4]                          # order by o: jobs 0, 2, 1
    assert oracle.build_schedule("GBA", [], [], 100).status == 0


def test_bounds_worked_example():
    """Class-size bounds on an instance small enough to work by hand from the lemmas' formulas.
    M = 10, s = 2 (X = 8), alpha = 2: ladder 1, 2, 4, 8 with k* = 3, 2, 2, 1 (peak-memory lemma);
    o = 1, 1, 2, 3, 5, 8 gives class sizes 2, 1, 1, 2.
      ladder terms Q = 2, 2, 4, 24; class-prefix terms S = 0, 1, 4, 10; UpperGBA = 2 + 3 + 8 + 44 = 57
      spillover D = 2, 3, 4, 0; phase-prefix T = 0, 3, 9, 19; GSA bound = 4 + 6 + 13 + 38 + 32 = 93
      2*Area(x, 2) for x = 0, 1, 2, 4 is 0, 6, 14, 36 with weights 11, 4, 3, 3: 2*M*lower = 174."""
    B = oracle.bounds([2] * 6, [1, 1, 2, 3, 5, 8], 10)
    assert (B.status, B.upper_gba, B.upper_gsa, B.lower_2m) == (0, 57, 93, 174)
    assert [int(x) for x in oracle.build_schedule("GBA", [2] * 6, [1, 1, 2, 3, 5, 8], 10).k] == [3, 2, 2, 1]
    # the order of the jobs does not matter, only the class sizes do
    assert oracle.bounds([2] * 6, [8, 1, 5, 2, 1, 3], 10) == B
    assert oracle.bounds([2], [9], 10).status == 1 and oracle.bounds([2], [0], 10).status == 3


def test_bounds_hold_for_schedules_and_optimum():
    """GBA <= UpperGBA and GSA <= its bound (the two packing-efficiency lemmas), the aggregate
    inequality between the two bounds, and lower bound <= optimum <= every schedule."""
    rng = np.random.default_rng(55)
    for alpha in [(2, 1), (3, 2), (4, 3), (7, 4)]:
        al = Fraction(*alpha)
        for _ in range(60):
            s, o, M = _random_instance(rng, hetero=False)
            B = oracle.bounds(s, o, M, alpha=alpha)
            gba = oracle.build_schedule("GBA", s, o, M, alpha=alpha)
            gsa = oracle.build_schedule("GSA", s, o, M, alpha=alpha)
            assert B.status == 0 and gba.flow <= B.upper_gba and gsa.flow <= B.upper_gsa
            assert B.upper_gba <= B.upper_gsa <= (2 + 2 / (al - 1)) * B.upper_gba
            for S in (gba, gsa, oracle.build_schedule("SPS", s, o, M), oracle.build_schedule("SIMS", s, o, M)):
                assert B.lower_2m <= 2 * M * S.flow
    for _ in range(60):
        n, s = int(rng.integers(1, 8)), int(rng.integers(0, 6))
        o = rng.integers(1, 7, n)
        M = int(s + o.max() + rng.integers(0, 14))
        opt = oracle.opt_bruteforce(s, o, M)
        for alpha in [(2, 1), (3, 2)]:
            B = oracle.bounds([s] * n, o, M, alpha=alpha)
            assert B.lower_2m <= 2 * M * opt <= 2 * M * B.upper_gba
    # a tunable initial slice changes the ladder, not the validity of the upper bounds
    for _ in range(30):
        s, o, M = _random_instance(rng, hetero=False)
        b0 = int(rng.integers(1, 6))
        B = oracle.bounds(s, o, M, beta0=b0)
        assert oracle.build_schedule("GBA", s, o, M, beta0=b0).flow <= B.upper_gba
        assert oracle.build_schedule("GSA", s, o, M, beta0=b0).flow <= B.upper_gsa


# ---- variants inside the geometric classes ------------------------------------------------------

def test_simultaneous_subroutine_reproduces_the_paper_numbers():
    """With simultaneous batches as the subroutine of every phase, the batching algorithm on an instance
    whose jobs all fall into one class IS the simultaneous schedule of that class.  Uniform experiment
    (n = 200, o = 16, s = 0, M = 256, alpha = 2): class tau = 16, B = 256 / 16 = 16, the simultaneous number
    21632 of the paper's figure.  Example 1 (15 jobs, s = 0, o = 5, M = 15) with the initial slice set to 5:
    B = 3, flow 225 and the per-round memory 3, 6, 9, 12, 15 repeated."""
    S = oracle.build_schedule("GBA", [0] * 200, [16] * 200, 256, subroutine=1)
    assert S.status == 0 and S.flow == 21632
    assert oracle.build_schedule("GBA", [0] * 200, [16] * 200, 256).flow == 14083       # and staggered: the paper's GBA number
    S = oracle.build_schedule("GBA", [0] * 15, [5] * 15, 15, beta0=5, subroutine=1)
    assert S.flow == 225 and int(S.k[0]) == 3
    assert list(_dense(S).profile) == [3, 6, 9, 12, 15] * 5
    T = oracle.build_schedule("SIMS", [0] * 15, [5] * 15, 15)
    assert np.array_equal(S.run_start, T.run_start) and np.array_equal(S.job_completion, T.job_completion)
    # the slicing algorithm too: every phase is one simultaneous schedule of the remaining jobs
    G = oracle.build_schedule("GSA", [0] * 15, [5] * 15, 15, beta0=5, subroutine=1)
    assert G.flow == 225


def test_class_variants_invariants_and_reductions():
    rng = np.random.default_rng(77)
    for alpha in [(2, 1), (3, 2)]:
        for it in range(80):
            s, o, M = _random_instance(rng, hetero=it % 2 == 0)
            for fam in ("GBA", "GSA"):
                base = oracle.build_schedule(fam, s, o, M, alpha=alpha)
                for sub in (0, 1):
                    for pc in (0, 1):
                        S = oracle.build_schedule(fam, s, o, M, alpha=alpha, subroutine=sub, per_class_s=pc)
                        assert S.status == 0 and S.n_unfinished == 0
                        assert _dense(S).peak <= M                                   # every round fits
                        assert np.array_equal(S.job_completion, S.job_start + o)
                        # inside a phase: rank r starts floor(r tau / k) (staggered) or floor(r / k) tau (batches)
                        b0 = 0
                        for p in range(len(S.tau)):
                            sel = S.run_phase == p
                            N = int(sel.sum())
                            if N == 0:
                                continue
                            tau = int(S.tau[p])
                            st = S.run_start[sel]
                            kk = int(S.k[p])
                            r = np.arange(N)
                            assert np.array_equal(st, b0 + ((r // kk) * tau if sub else (r * tau) // kk))
                            b0 = int(st[-1]) + tau
                            s_p = int(max(s[S.run_job[sel]])) if pc else int(S.s_bar)
                            assert kk == (M // (s_p + tau) if sub else oracle.kstar(tau, s_p, M))
                    # one prompt length: the per-phase value is that length, nothing changes
                    if it % 2 == 1:
                        assert _same(oracle.build_schedule(fam, s, o, M, alpha=alpha, per_class_s=1), base)
                # a shorter prompt bound can only raise the parallelism: no job starts later
                P = oracle.build_schedule(fam, s, o, M, alpha=alpha, per_class_s=1)
                assert np.all(P.job_start <= base.job_start) and P.flow <= base.flow
    assert oracle.build_schedule("GBA", [1], [1], 10, subroutine=2).status == 3


# ---- dynamic refill of the batching schedule ------------------------------------------------------

def test_dynamic_refill_hand_worked_instance(golden_dir):
    """M = 10, s = 2, o = 1, 1, 2, 3, 5, 8 (alpha = 2: ladder 1, 2, 4, 8 with k* = 3, 2, 2, 1).  The batching
    schedule starts the jobs at 0, 0, 1, 3, 7, 15 (flow 46).  Refill, worked by hand from the reading: the job
    of length 2 fits at 0 beside the two unit jobs (3 + 3 + 3 = 9); the job of length 3 does not fit at 0
    (9 + 3 > 10) but at 1 (4 + 3, then 4, 5); the job of length 5 fits at 1 too (4 + 3 + 3 = 10, then 4 + 4,
    5 + 5, 6, 7); the job of length 8 fails at 1 .. 3, fits round 4 but not round 5 from 4 (7 + 4 > 10), and
    fits from 5 on: starts 0, 0, 0, 1, 1, 5, flow 27, memory 9, 10, 8, 10, 6, 10, 4, 5, ..., 10."""
    rows = [ln.split() for ln in open(os.path.join(golden_dir, "dynamic_refill_hand_example.txt")) if ln.strip() and not ln.startswith("#")]
    want = {r[0]: [int(x) for x in r[1:]] for r in rows}
    S = oracle.build_schedule("GBAD", [2] * 6, want["o"], 10)
    assert S.status == 0 and list(S.job_start) == want["start"] and S.flow == want["flow"][0]
    assert list(_dense(S).profile) == want["memory"]
    assert list(oracle.build_schedule("GBA", [2] * 6, want["o"], 10).job_start) == want["gba_start"]


def test_dynamic_refill_keeps_the_paper_promises():
    """No job starts later than in the batching schedule, admissions keep their order, every round fits, the
    flow time is at most the batching schedule's (hence within UpperGBA), and at least the optimum."""
    rng = np.random.default_rng(88)
    for alpha in [(2, 1), (3, 2), (4, 3)]:
        for it in range(120):
            s, o, M = _random_instance(rng, hetero=it % 3 == 0)
            G = oracle.build_schedule("GBA", s, o, M, alpha=alpha)
            D = oracle.build_schedule("GBAD", s, o, M, alpha=alpha)
            assert D.status == 0 and D.n_unfinished == 0 and len(D.run_job) == len(o)
            assert np.all(D.job_start <= G.job_start) and D.flow <= G.flow
            assert np.array_equal(D.run_job, G.run_job) and np.all(np.diff(D.run_start) >= 0)
            assert np.array_equal(D.job_completion, D.job_start + o) and D.job_steps == int(o.sum())
            assert _dense(D).peak <= M
            if it % 3:
                assert D.flow <= oracle.bounds(s, o, M, alpha=alpha).upper_gba
    for it in range(60):
        n, s = int(rng.integers(1, 8)), int(rng.integers(0, 6))
        o = rng.integers(1, 7, n)
        M = int(s + o.max() + rng.integers(0, 14))
        assert oracle.opt_bruteforce(s, o, M) <= oracle.build_schedule("GBAD", [s] * n, o, M).flow
    # a schedule without idle memory cannot move: one job per slot at full length
    D = oracle.build_schedule("GBAD", [0] * 5, [8] * 5, 8)
    assert list(D.job_start) == [0, 8, 16, 24, 32]
    assert oracle.build_schedule("GBAD", [1], [1], 10, window=5).status == 3


# ---- speculative runs on top of the slicing schedule ----------------------------------------------

def test_speculative_runs_hand_worked_instance(golden_dir):
    """M = 6, s = 0, o = 4, 4, 2 (alpha = 2: slices 1, 3, 6 with k* = 3, 3, 1).  By hand from the reading:
    round 0 the three unit runs; round 1 job 0 starts its slice of 3 and jobs 1, 2 (free, 1 + 1 + 1 <= 6) start
    speculative runs; round 2 job 1's slice starts, so its speculative run is killed after one round; round 3
    job 2's speculative run has its 2 rounds: done at 3 (5 in the slicing schedule), its slice of round 3 is
    dropped; rounds 4 and 5 jobs 0 and 1 come free and speculate; round 6 job 0's slice of 6 starts and kills
    its speculative run (2 rounds); round 8 the slice holds 3 and job 1's speculative run 4 > 6: killed after 3
    rounds, and, being free and first in line, restarted at once (3 + 1 <= 6); it completes at 12 (16 in the
    slicing schedule), job 0 at 10 as planned.  Flow 25 against 31."""
    rows = [ln.split() for ln in open(os.path.join(golden_dir, "speculative_runs_hand_example.txt")) if ln.strip() and not ln.startswith("#")]
    want = {r[0]: [int(x) for x in r[1:]] for r in rows if r[0] != "run"}
    runs = [tuple(int(x) for x in r[1:]) for r in rows if r[0] == "run"]
    n = len(want["o"])
    G = oracle.build_schedule("GSA", [0] * n, want["o"], 6)
    assert list(G.job_completion) == want["gsa_completion"]
    S = oracle.build_schedule("GSAS", [0] * n, want["o"], 6)
    assert S.status == 0 and S.n_unfinished == 0
    assert list(S.job_start) == want["start"] and list(S.job_completion) == want["completion"] and S.flow == want["flow"][0]
    assert list(zip(S.run_job.tolist(), S.run_start.tolist(), S.run_len.tolist())) == runs
    assert list(_dense(S).profile) == want["memory"]
    assert S.job_steps == sum(r[2] for r in runs)


def test_speculative_runs_keep_the_paper_promises():
    """The slicing schedule is kept: every pipeline run of a job that has not completed by then is executed at
    its round and length, so no job completes later than in the slicing schedule; every round fits; the flow
    time is at least the optimum; an instance whose pipeline leaves no room for a further first round is
    unchanged."""
    rng = np.random.default_rng(97)
    improved = 0
    for alpha in [(2, 1), (3, 2)]:
        for it in range(120):
            s, o, M = _random_instance(rng, hetero=it % 3 == 0)
            G = oracle.build_schedule("GSA", s, o, M, alpha=alpha)
            S = oracle.build_schedule("GSAS", s, o, M, alpha=alpha)
            assert S.status == 0 and S.n_unfinished == 0
            assert np.all(S.job_completion <= G.job_completion) and S.flow <= G.flow
            improved += S.flow < G.flow
            assert _dense(S).peak <= M and np.all(np.diff(S.run_start) >= 0)
            ex = set(zip(S.run_job.tolist(), S.run_start.tolist(), S.run_len.tolist()))
            for j, t0, ln in zip(G.run_job.tolist(), G.run_start.tolist(), G.run_len.tolist()):
                if S.job_completion[j] > t0:            # not done when the pipeline reaches it (a run that completes
                    assert (j, t0, ln) in ex            # its job at t0 + len has completion > t0 as well)
            # the run that completes a job has its full length; every run's length is at most the job's
            done_runs = {(j, c - ln) for j, c, ln in zip(range(len(o)), S.job_completion.tolist(), np.asarray(o).tolist())}
            assert all((j, t0, int(o[j])) in ex for j, t0 in done_runs)
            assert np.all(S.run_len <= np.asarray(o)[S.run_job]) and S.job_steps >= int(np.sum(o))
    assert improved > 60
    for it in range(60):
        n, s = int(rng.integers(1, 8)), int(rng.integers(0, 6))
        o = rng.integers(1, 7, n)
        M = int(s + o.max() + rng.integers(0, 14))
        assert oracle.opt_bruteforce(s, o, M) <= oracle.build_schedule("GSAS", [s] * n, o, M).flow
    # one job at a time fills the memory: nothing can be added
    A, B = oracle.build_schedule("GSA", [7] * 3, [1] * 3, 8), oracle.build_schedule("GSAS", [7] * 3, [1] * 3, 8)
    assert _same(A, B)
    # a single job is its own pipeline
    assert _same(oracle.build_schedule("GSA", [3], [9], 40), oracle.build_schedule("GSAS", [3], [9], 40))
    assert oracle.build_schedule("GSAS", [1], [1], 10, window=5).status == 3
