"""Thin ctypes binding of ``libkvs.so`` (declarations in ``include/kvs.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels.  Tensors are
PyTorch CUDA tensors used as device memory; the context runs on the CUDA stream that is
current when it is created.  There is no CPU fallback: loading fails if the library is
missing and ``Context`` fails without a CUDA device.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_float, c_int32, c_int64, c_uint64, c_void_p

import numpy as np
import torch

from . import build as _build
from .workloads import Instances

GBA, GSA, SPS, SIMS, GBAD, GSAS = 0, 1, 2, 3, 4, 5
FAMILY = {"GBA": GBA, "GSA": GSA, "SPS": SPS, "SIMS": SIMS, "GBAD": GBAD, "GSAS": GSAS}
EVAL_OK, EVAL_INFEASIBLE, EVAL_RANGE, EVAL_CAPACITY, EVAL_BAD_INPUT = 0, 1, 2, 4, 8

SETTING_DTYPE = np.dtype([("instance", "<i8"), ("family", "<i4"), ("alpha_num", "<i4"), ("alpha_den", "<i4"),
                          ("s_bar", "<i4"), ("M", "<i8"), ("beta0", "<i8"), ("tau", "<i8"), ("k", "<i8"),
                          ("subroutine", "<i4"), ("per_class_s", "<i4")],
                         align=True)


class KvsError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"kvs error {code}: {message}")
        self.code = code


class _InitParams(Structure):
    _fields_ = [("device", c_int32), ("stream", c_void_p), ("workspace", c_void_p), ("workspace_bytes", c_uint64)]


class _Instances(Structure):
    _fields_ = [("n_instances", c_int64), ("n_jobs_total", c_int64), ("max_jobs_per_instance", c_int64),
                ("job_off", c_void_p), ("s", c_void_p), ("o", c_void_p), ("o_est", c_void_p),
                ("arrival", c_void_p), ("window", c_int64)]


class _ScheduleOut(Structure):
    _fields_ = [("job_out_off", c_void_p), ("job_start", c_void_p), ("job_completion", c_void_p),
                ("job_start64", c_void_p), ("job_completion64", c_void_p), ("run_off", c_void_p),
                ("run_job", c_void_p), ("run_phase", c_void_p), ("run_start", c_void_p), ("run_len", c_void_p),
                ("run_s", c_void_p), ("n_runs", c_void_p)]


class _EvalOut(Structure):
    _fields_ = [("profile_off", c_void_p), ("profile", c_void_p), ("peak", c_void_p), ("flow", c_void_p),
                ("job_steps", c_void_p), ("horizon", c_void_p), ("n_unfinished", c_void_p),
                ("feasible", c_void_p), ("status", c_void_p)]


class _Runs(Structure):
    _fields_ = [("P", c_int64), ("run_off", c_void_p), ("run_start", c_void_p), ("run_len", c_void_p),
                ("run_s", c_void_p), ("run_flow", c_void_p), ("M", c_void_p)]


class _SweepParams(Structure):
    _fields_ = [("instance", c_int64), ("M", c_int64), ("tau", c_void_p), ("k", c_void_p),
                ("n_tau", c_int32), ("n_k", c_int32), ("family", c_int32), ("n_beta0", c_int32), ("beta0", c_void_p),
                ("alpha_num", c_int32), ("alpha_den", c_int32), ("subroutine", c_int32), ("per_class_s", c_int32)]


class _SweepOut(Structure):
    _fields_ = [("peak", c_void_p), ("flow", c_void_p), ("n_completed", c_void_p), ("horizon", c_void_p),
                ("job_steps", c_void_p), ("feasible", c_void_p)]


class _BoundsOut(Structure):
    _fields_ = [("upper_gba", c_void_p), ("upper_gsa", c_void_p), ("lower_2m", c_void_p), ("status", c_void_p)]


EXPORTS = ["kvs_init", "kvs_destroy", "kvs_last_error", "kvs_set_timing", "kvs_last_timing", "kvs_last_timing_split", "kvs_debug_check_word", "kvs_workspace_bytes",
           "kvs_build_schedule", "kvs_evaluate_built", "kvs_evaluate_built_host", "kvs_evaluate_schedule", "kvs_sweep",
           "kvs_evaluate_schedule_noalloc", "kvs_bounds"]

_lib = None


def load(path: str | None = None):
    """Load libkvs.so (building it in-tree with nvcc if it is missing or stale)."""
    global _lib
    if _lib is None:
        if path is None:
            path = _build.LIB_PATH
            if not os.path.exists(path) or _build._stale():
                path = _build.build()
        L = ctypes.CDLL(path)
        L.kvs_init.argtypes = [POINTER(_InitParams), POINTER(c_void_p)]
        L.kvs_destroy.argtypes = [c_void_p]
        L.kvs_last_error.argtypes = [c_void_p]
        L.kvs_last_error.restype = c_char_p
        L.kvs_set_timing.argtypes = [c_void_p, c_int32]
        L.kvs_last_timing.argtypes = [c_void_p, POINTER(c_float), POINTER(c_float)]
        L.kvs_last_timing_split.argtypes = [c_void_p, POINTER(c_float), POINTER(c_float), POINTER(c_float)]
        L.kvs_debug_check_word.argtypes = [POINTER(c_uint64), POINTER(c_int32), c_int32]
        L.kvs_workspace_bytes.argtypes = [c_int64, c_int64, c_int64, c_int64, c_int64, c_int32, POINTER(c_uint64)]
        L.kvs_build_schedule.argtypes = [c_void_p, POINTER(_Instances), c_void_p, c_int64, POINTER(_ScheduleOut), POINTER(_EvalOut)]
        L.kvs_evaluate_built.argtypes = L.kvs_build_schedule.argtypes
        L.kvs_evaluate_built_host.argtypes = [c_void_p, POINTER(_Instances), c_void_p, c_int64, POINTER(_EvalOut)]
        L.kvs_evaluate_schedule.argtypes = [c_void_p, POINTER(_Runs), POINTER(_EvalOut)]
        L.kvs_sweep.argtypes = [c_void_p, POINTER(_Instances), POINTER(_SweepParams), POINTER(_SweepOut)]
        L.kvs_bounds.argtypes = [c_void_p, POINTER(_Instances), c_void_p, c_int64, POINTER(_BoundsOut)]
        L.kvs_evaluate_schedule_noalloc.argtypes = [c_int32, c_void_p, POINTER(_Runs), POINTER(_EvalOut), c_int64,
                                                    ctypes.c_char_p, c_uint64]
        _lib = L
    return _lib


def debug_check_word(reset: bool = False) -> tuple[int, bool]:
    """(first index violation recorded by a checked build, 0 = none; whether the loaded library is a checked build)."""
    w, c = c_uint64(0), c_int32(0)
    rc = load().kvs_debug_check_word(ctypes.byref(w), ctypes.byref(c), 1 if reset else 0)
    if rc:
        raise KvsError(rc, "kvs_debug_check_word")
    return int(w.value), bool(c.value)


def evaluate_schedule_noalloc(runs: dict, ev: dict, capacity_total: int, device: int | None = None):
    """kvs_evaluate_schedule_noalloc: evaluates explicit runs without a context or a workspace.

    For callers that may not allocate on the GPU: the scratch is a fixed array inside the library
    (capacity_total + P <= 1,048,576).  Runs on the current CUDA stream; calls on one device must
    not overlap.  ``runs`` / ``ev`` as in ``Context.evaluate_schedule``."""
    dev = torch.cuda.current_device() if device is None else device
    P = int(runs["run_off"].numel()) - 1
    cr = _Runs(P, _p(runs["run_off"]), _p(runs["run_start"]), _p(runs["run_len"]), _p(runs["run_s"]),
               _p(runs.get("run_flow")), _p(runs.get("M")))
    eo = _EvalOut(*[_p(ev.get(f[0])) for f in _EvalOut._fields_])
    msg = ctypes.create_string_buffer(256)
    rc = load().kvs_evaluate_schedule_noalloc(dev, c_void_p(torch.cuda.current_stream(dev).cuda_stream),
                                              ctypes.byref(cr), ctypes.byref(eo), capacity_total, msg, 256)
    if rc:
        raise KvsError(rc, msg.value.decode())


def make_settings(rows) -> np.ndarray:
    """Settings array from dicts: instance, family, M [, alpha, s_bar, beta0, tau, k, subroutine, per_class_s]."""
    out = np.zeros(len(rows), dtype=SETTING_DTYPE)
    for i, r in enumerate(rows):
        fam = r["family"]
        out[i]["instance"] = r["instance"]
        out[i]["family"] = FAMILY[fam] if isinstance(fam, str) else fam
        out[i]["alpha_num"], out[i]["alpha_den"] = r.get("alpha", (2, 1))
        out[i]["s_bar"] = r.get("s_bar", -1)
        out[i]["M"] = r["M"]
        out[i]["beta0"] = r.get("beta0", 0)
        out[i]["tau"] = r.get("tau", 0)
        out[i]["k"] = r.get("k", 0)
        out[i]["subroutine"] = r.get("subroutine", 0)
        out[i]["per_class_s"] = r.get("per_class_s", 0)
    return out


def settings_grid(instances, families, Ms, alpha=(2, 1), subroutine=0, per_class_s=0) -> np.ndarray:
    """Vectorised settings: every (instance, M, family) combination, instance-major.

    ``Ms`` is either one list shared by all instances or an array [n_instances, n_M]."""
    inst = np.asarray(list(instances), dtype=np.int64)
    fams = np.asarray([FAMILY[f] if isinstance(f, str) else f for f in families], dtype=np.int32)
    Ms = np.asarray(Ms, dtype=np.int64)
    n_M = Ms.shape[0] if Ms.ndim == 1 else Ms.shape[1]
    out = np.zeros((inst.size, n_M, fams.size), dtype=SETTING_DTYPE)
    out["instance"] = inst[:, None, None]
    out["family"] = fams[None, None, :]
    out["M"] = Ms[None, :, None] if Ms.ndim == 1 else Ms[:, :, None]
    out["alpha_num"], out["alpha_den"] = alpha
    out["s_bar"] = -1
    geo = (out["family"] <= GSA) | (out["family"] >= GBAD)
    out["subroutine"] = np.where(geo, subroutine, 0)
    out["per_class_s"] = np.where(geo, per_class_s, 0)
    return out.reshape(-1)


def _p(t):
    return None if t is None else c_void_p(t.data_ptr())


def workspace_bytes(n_jobs_total, n_instances, max_jobs, n_evaluations, generic_capacity=0, host_staging=False) -> int:
    out = c_uint64(0)
    rc = load().kvs_workspace_bytes(n_jobs_total, n_instances, max_jobs, n_evaluations, generic_capacity,
                                    1 if host_staging else 0, ctypes.byref(out))
    if rc:
        raise KvsError(rc, "kvs_workspace_bytes")
    return int(out.value)


class Context:
    """kvs_ctx bound to a device, the current CUDA stream and a caller-owned workspace tensor."""

    def __init__(self, workspace: torch.Tensor, device: int | None = None):
        if not torch.cuda.is_available():
            raise KvsError(-2, "no CUDA device: the schedule builder has no CPU path")
        self._lib = load()
        self.device = torch.cuda.current_device() if device is None else device
        self.workspace = workspace
        self.stream = torch.cuda.current_stream(self.device)
        prm = _InitParams(self.device, c_void_p(self.stream.cuda_stream), c_void_p(workspace.data_ptr()),
                          workspace.numel() * workspace.element_size())
        self._ctx = c_void_p()
        rc = self._lib.kvs_init(ctypes.byref(prm), ctypes.byref(self._ctx))
        if rc:
            raise KvsError(rc, "kvs_init failed")

    def close(self):
        if getattr(self, "_ctx", None):
            self._lib.kvs_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        self.close()

    def _check(self, rc):
        if rc:
            raise KvsError(rc, self._lib.kvs_last_error(self._ctx).decode())

    def set_timing(self, enabled: bool):
        self._check(self._lib.kvs_set_timing(self._ctx, 1 if enabled else 0))

    def last_timing(self) -> tuple[float, float]:
        """(ordering kernel ms, builder/evaluator kernel ms) of the most recent fused call."""
        a, b = c_float(0), c_float(0)
        self._check(self._lib.kvs_last_timing(self._ctx, ctypes.byref(a), ctypes.byref(b)))
        return float(a.value), float(b.value)

    def last_timing_split(self) -> tuple[float, float, float]:
        """Device milliseconds of the ordering kernel, the light variant and the full variant (+ general kernel)."""
        a, b, c = c_float(0), c_float(0), c_float(0)
        self._check(self._lib.kvs_last_timing_split(self._ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
        return float(a.value), float(b.value), float(c.value)

    @staticmethod
    def _instances(inst: Instances, window: int = 0, max_jobs: int | None = None):
        I = inst.n_instances
        N = int(inst.s.numel())
        if max_jobs is None:
            max_jobs = int((inst.job_off[1:] - inst.job_off[:-1]).max()) if I else 0
        return _Instances(I, N, max_jobs, _p(inst.job_off), _p(inst.s), _p(inst.o), _p(inst.o_est),
                          _p(inst.arrival) if window > 0 else None, window)

    def _fused(self, fn, inst, settings, out, ev, window, max_jobs):
        ci = self._instances(inst, window, max_jobs)
        so = _ScheduleOut(*[_p(out.get(f[0])) for f in _ScheduleOut._fields_]) if out else None
        eo = _EvalOut(*[_p(ev.get(f[0])) for f in _EvalOut._fields_]) if ev else None
        settings = np.ascontiguousarray(settings, dtype=SETTING_DTYPE)
        self._keep = (settings, inst, out, ev)   # alive until the stream has consumed them
        self._check(fn(self._ctx, ctypes.byref(ci), settings.ctypes.data_as(c_void_p), settings.shape[0],
                       ctypes.byref(so) if so else None, ctypes.byref(eo) if eo else None))

    def build_schedule(self, inst: Instances, settings: np.ndarray, out: dict, ev: dict | None = None,
                       window: int = 0, max_jobs: int | None = None):
        """kvs_build_schedule: ``out`` / ``ev`` map field names of the C structs to CUDA tensors."""
        self._fused(self._lib.kvs_build_schedule, inst, settings, out, ev, window, max_jobs)

    def evaluate_built(self, inst: Instances, settings: np.ndarray, out: dict | None, ev: dict,
                       window: int = 0, max_jobs: int | None = None):
        """kvs_evaluate_built: builder and evaluator fused."""
        self._fused(self._lib.kvs_evaluate_built, inst, settings, out, ev, window, max_jobs)

    def evaluate_built_host(self, inst: Instances, settings: np.ndarray, ev: dict, window: int = 0,
                            max_jobs: int | None = None):
        """kvs_evaluate_built_host: ``inst`` and ``ev`` hold HOST (ideally pinned) tensors."""
        ci = self._instances(inst, window, max_jobs)
        eo = _EvalOut(*[_p(ev.get(f[0])) for f in _EvalOut._fields_])
        settings = np.ascontiguousarray(settings, dtype=SETTING_DTYPE)
        self._check(self._lib.kvs_evaluate_built_host(self._ctx, ctypes.byref(ci), settings.ctypes.data_as(c_void_p),
                                                      settings.shape[0], ctypes.byref(eo)))

    def bounds(self, inst: Instances, settings: np.ndarray, out: dict, max_jobs: int | None = None):
        """kvs_bounds: ``out`` maps upper_gba, upper_gsa, lower_2m (int64 [P]) and status (int32 [P]) to CUDA tensors."""
        ci = self._instances(inst, 0, max_jobs)
        bo = _BoundsOut(*[_p(out.get(f[0])) for f in _BoundsOut._fields_])
        settings = np.ascontiguousarray(settings, dtype=SETTING_DTYPE)
        self._keep = (settings, inst, out)
        self._check(self._lib.kvs_bounds(self._ctx, ctypes.byref(ci), settings.ctypes.data_as(c_void_p), settings.shape[0],
                                         ctypes.byref(bo)))

    def evaluate_schedule(self, runs: dict, ev: dict):
        """kvs_evaluate_schedule: ``runs`` maps run_off, run_start, run_len, run_s [, run_flow, M]."""
        P = int(runs["run_off"].numel()) - 1
        cr = _Runs(P, _p(runs["run_off"]), _p(runs["run_start"]), _p(runs["run_len"]), _p(runs["run_s"]),
                   _p(runs.get("run_flow")), _p(runs.get("M")))
        eo = _EvalOut(*[_p(ev.get(f[0])) for f in _EvalOut._fields_])
        self._keep = (runs, ev)
        self._check(self._lib.kvs_evaluate_schedule(self._ctx, ctypes.byref(cr), ctypes.byref(eo)))

    def sweep(self, inst: Instances, instance: int, family, M: int, tau, k, out: dict, max_jobs: int | None = None,
              beta0=(), alpha=(2, 1), subroutine=0, per_class_s=0):
        """kvs_sweep over the grid tau x k (SPS / SIMS) or over the initial slices beta0 (GBA / GSA); host lists;
        ``out`` maps field names to CUDA tensors."""
        ci = self._instances(inst, 0, max_jobs)
        tau = np.ascontiguousarray(tau, dtype=np.int64)
        k = np.ascontiguousarray(k, dtype=np.int64)
        b0 = np.ascontiguousarray(beta0, dtype=np.int64)
        fam = FAMILY[family] if isinstance(family, str) else family
        sp = _SweepParams(instance, M, tau.ctypes.data_as(c_void_p), k.ctypes.data_as(c_void_p), tau.size, k.size, fam,
                          b0.size, b0.ctypes.data_as(c_void_p), alpha[0], alpha[1], subroutine, per_class_s)
        so = _SweepOut(*[_p(out.get(f[0])) for f in _SweepOut._fields_])
        self._keep = (tau, k, b0, inst, out)
        self._check(self._lib.kvs_sweep(self._ctx, ctypes.byref(ci), ctypes.byref(sp), ctypes.byref(so)))
