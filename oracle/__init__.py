"""ctypes front end of the CPU oracle (``kvs_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the CPU
baseline leg of the benchmark.  The CUDA package never imports this module and
this module never imports the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvs_oracle.cpp")
_LIB = os.path.join(_HERE, "libkvs_oracle.so")

GBA, GSA, SPS, SIMS, GBAD, GSAS = 0, 1, 2, 3, 4, 5
FAMILY = {"GBA": GBA, "GSA": GSA, "SPS": SPS, "SIMS": SIMS, "GBAD": GBAD, "GSAS": GSAS}


def build(force: bool = False) -> str:
    """Compile the oracle with the host compiler (plain C++17, single thread)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, i32, p = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p
        L.kvo_peak_closed.restype = i64
        L.kvo_peak_closed.argtypes = [i64, i64, i64]
        L.kvo_kstar.restype = i64
        L.kvo_kstar.argtypes = [i64, i64, i64]
        L.kvo_ladder.restype = i64
        L.kvo_ladder.argtypes = [i64, i32, i32, i64, p, i64]
        L.kvo_build.restype = p
        L.kvo_build.argtypes = [i32, i64, p, p, p, p, i64, i32, i32, i64, i64, i64, i64, i64]
        L.kvo_build_variant.restype = p
        L.kvo_build_variant.argtypes = [i32, i64, p, p, p, p, i64, i32, i32, i64, i64, i64, i64, i64, i32, i32]
        L.kvo_free.argtypes = [p]
        L.kvo_scalars.argtypes = [p, p]
        L.kvo_jobs.argtypes = [p, p, p]
        L.kvo_runs.argtypes = [p, p, p, p, p, p]
        L.kvo_phases.argtypes = [p, p, p, p]
        L.kvo_eval_dense.argtypes = [i64, p, p, p, p, i64, p]
        L.kvo_eval_events.argtypes = [i64, p, p, p, p]
        L.kvo_bounds.argtypes = [i64, p, p, i64, i32, i32, i64, i64, p]
        L.kvo_opt_bruteforce.restype = i64
        L.kvo_opt_bruteforce.argtypes = [i32, i64, p, i64]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _arr(x, dtype):
    if x is None:
        return None
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(np.asarray(x), dtype=dtype)


def peak_closed(k: int, tau: int, s: int) -> int:
    return int(lib().kvo_peak_closed(k, tau, s))


def kstar(tau: int, s: int, M: int) -> int:
    return int(lib().kvo_kstar(tau, s, M))


def ladder(X: int, alpha_num: int = 2, alpha_den: int = 1, beta0: int = 0) -> list[int]:
    buf = np.zeros(512, dtype=np.int64)
    n = int(lib().kvo_ladder(X, alpha_num, alpha_den, beta0, _ptr(buf), buf.size))
    return [int(v) for v in buf[:n]]


@dataclass
class Schedule:
    status: int
    s_bar: int
    job_start: np.ndarray          # int64 [n], -1 = never completed
    job_completion: np.ndarray     # int64 [n]
    run_job: np.ndarray            # int64 [R], order: window, phase, rank
    run_phase: np.ndarray
    run_start: np.ndarray
    run_len: np.ndarray
    run_s: np.ndarray
    tau: np.ndarray                # phase table
    k: np.ndarray
    n_part: np.ndarray             # participants per phase
    flow: int
    horizon: int
    job_steps: int
    n_unfinished: int


def build_schedule(family, s, o, M, *, o_est=None, arrival=None, alpha=(2, 1), beta0=0,
                   s_bar=-1, tau=0, k=0, window=0, subroutine=0, per_class_s=0) -> Schedule:
    """Build one schedule for one instance (see ``kvo_build``).  ``subroutine=1`` runs the simultaneous
    schedule inside every geometric phase, ``per_class_s=1`` sizes each phase's parallelism by the
    longest prompt among its participants (see ``build`` in kvs_oracle.cpp)."""
    fam = FAMILY[family] if isinstance(family, str) else int(family)
    s_, o_ = _arr(s, np.int32), _arr(o, np.int32)
    e_, a_ = _arr(o_est, np.int32), _arr(arrival, np.int64)
    n = int(s_.shape[0])
    L = lib()
    h = L.kvo_build_variant(fam, n, _ptr(s_), _ptr(o_), _ptr(e_), _ptr(a_), int(M), int(alpha[0]),
                            int(alpha[1]), int(beta0), int(s_bar), int(tau), int(k), int(window),
                            int(subroutine), int(per_class_s))
    try:
        sc = np.zeros(8, dtype=np.int64)
        L.kvo_scalars(h, _ptr(sc))
        R, P = int(sc[1]), int(sc[2])
        js, jc = np.zeros(n, np.int64), np.zeros(n, np.int64)
        L.kvo_jobs(h, _ptr(js), _ptr(jc))
        rj, rp, rs, rl, rr = (np.zeros(R, np.int64) for _ in range(5))
        L.kvo_runs(h, _ptr(rj), _ptr(rp), _ptr(rs), _ptr(rl), _ptr(rr))
        tau_, k_, np_ = (np.zeros(P, np.int64) for _ in range(3))
        L.kvo_phases(h, _ptr(tau_), _ptr(k_), _ptr(np_))
    finally:
        L.kvo_free(h)
    return Schedule(int(sc[0]), int(sc[7]), js, jc, rj, rp, rs, rl, rr, tau_, k_, np_,
                    int(sc[4]), int(sc[3]), int(sc[5]), int(sc[6]))


@dataclass
class Evaluation:
    peak: int
    horizon: int
    job_steps: int
    argmax: int
    profile: np.ndarray | None


def evaluate_dense(run_start, run_len, run_s, want_profile: bool = True) -> Evaluation:
    """Per-round memory by the definition: one update per job-step."""
    st, ln, ss = _arr(run_start, np.int64), _arr(run_len, np.int64), _arr(run_s, np.int64)
    R = int(st.shape[0])
    T = int((st + ln).max()) if R else 0
    prof = np.zeros(T, dtype=np.int64) if want_profile else None
    out = np.zeros(4, dtype=np.int64)
    lib().kvo_eval_dense(R, _ptr(st), _ptr(ln), _ptr(ss), _ptr(prof), T, _ptr(out))
    return Evaluation(int(out[0]), int(out[1]), int(out[2]), int(out[3]), prof)


def evaluate_events(run_start, run_len, run_s) -> Evaluation:
    """Peak / horizon / job-steps from sorted start and end events (no dense array)."""
    st, ln, ss = _arr(run_start, np.int64), _arr(run_len, np.int64), _arr(run_s, np.int64)
    out = np.zeros(4, dtype=np.int64)
    lib().kvo_eval_events(int(st.shape[0]), _ptr(st), _ptr(ln), _ptr(ss), _ptr(out))
    return Evaluation(int(out[0]), int(out[1]), int(out[2]), -1, None)


@dataclass
class Bounds:
    status: int
    upper_gba: int        # GBA flow <= upper_gba
    upper_gsa: int        # GSA flow <= upper_gsa
    lower_2m: int         # 2 * M * (lower bound on the optimal flow), see kvo_bounds


def bounds(s, o, M, *, alpha=(2, 1), beta0=0, s_bar=-1) -> Bounds:
    """Bounds computed from the class sizes alone (see ``kvo_bounds``)."""
    s_, o_ = _arr(s, np.int32), _arr(o, np.int32)
    out = np.zeros(4, dtype=np.int64)
    lib().kvo_bounds(int(s_.shape[0]), _ptr(s_), _ptr(o_), int(M), int(alpha[0]), int(alpha[1]), int(beta0),
                     int(s_bar), _ptr(out))
    return Bounds(int(out[0]), int(out[1]), int(out[2]), int(out[3]))


def opt_bruteforce(s: int, o, M: int) -> int:
    """Minimum total flow time over all kill-free schedules (n <= 10, identical s)."""
    o_ = _arr(o, np.int32)
    return int(lib().kvo_opt_bruteforce(int(o_.shape[0]), int(s), _ptr(o_), int(M)))
