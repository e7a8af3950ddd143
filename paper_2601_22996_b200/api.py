"""Convenience layer over the binding: allocates outputs as CUDA tensors and sizes them.

Only allocation and call sequencing live here; all arithmetic is in the CUDA library.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import binding
from .workloads import Instances


@dataclass
class Result:
    """Device tensors of one batched call (P evaluations)."""
    status: torch.Tensor
    flow: torch.Tensor
    peak: torch.Tensor
    horizon: torch.Tensor
    job_steps: torch.Tensor
    n_unfinished: torch.Tensor
    feasible: torch.Tensor
    job_out_off: torch.Tensor | None = None
    job_start: torch.Tensor | None = None
    job_completion: torch.Tensor | None = None
    profile_off: torch.Tensor | None = None
    profile: torch.Tensor | None = None
    n_runs: torch.Tensor | None = None
    run_off: torch.Tensor | None = None
    runs: dict | None = None


class Scheduler:
    """Owns a workspace tensor and a context; grows the workspace when a call needs more."""

    def __init__(self, device: int | None = None):
        if not torch.cuda.is_available():
            raise binding.KvsError(-2, "no CUDA device: the schedule builder has no CPU path")
        self.device = torch.cuda.current_device() if device is None else device
        self._ws = None
        self._ctx = None

    def context(self, need: int) -> binding.Context:
        if self._ws is None or self._ws.numel() < need:
            if self._ctx is not None:
                torch.cuda.synchronize(self.device)
                self._ctx.close()
            self._ws = torch.empty(max(need, 1 << 20), dtype=torch.uint8, device=f"cuda:{self.device}")
            self._ctx = binding.Context(self._ws, self.device)
        return self._ctx

    @staticmethod
    def _sizes(inst: Instances):
        n_per = (inst.job_off[1:] - inst.job_off[:-1])
        return int(inst.s.numel()), inst.n_instances, int(n_per.max()) if inst.n_instances else 0, n_per

    @staticmethod
    def scalars(P, dev):
        z64 = lambda: torch.zeros(P, dtype=torch.int64, device=dev)
        return dict(peak=z64(), flow=z64(), job_steps=z64(), horizon=z64(), n_unfinished=z64(),
                    feasible=torch.zeros(P, dtype=torch.uint8, device=dev),
                    status=torch.zeros(P, dtype=torch.int32, device=dev))

    def evaluate(self, inst: Instances, settings: np.ndarray, *, want_jobs=True, want_profile=False,
                 want_runs=False, window=0, profile_capacity: torch.Tensor | None = None,
                 time64=False) -> Result:
        """Build and evaluate P schedules.  Profiles and run lists are sized by a first scalar-only pass."""
        dev = inst.s.device
        N, I, max_n, n_per = self._sizes(inst)
        P = int(settings.shape[0])
        if P and (settings["instance"].min() < 0 or settings["instance"].max() >= I):
            raise binding.KvsError(-1, "settings: instance out of range")   # before any device indexing
        ctx = self.context(binding.workspace_bytes(N, I, max_n, P))
        out, ev = {}, self.scalars(P, dev)
        if want_jobs:
            eval_inst = torch.from_numpy(np.ascontiguousarray(settings["instance"])).to(dev)
            off = torch.zeros(P + 1, dtype=torch.int64, device=dev)
            off[1:] = torch.cumsum(n_per[eval_inst], 0)
            total = int(off[-1])
            out["job_out_off"] = off
            tdt = torch.int64 if time64 else torch.int32
            suffix = "64" if time64 else ""
            out["job_start" + suffix] = torch.full((total,), -2, dtype=tdt, device=dev)
            out["job_completion" + suffix] = torch.full((total,), -2, dtype=tdt, device=dev)
        if want_profile or want_runs:
            first = self.scalars(P, dev)
            sizes = dict(n_runs=torch.zeros(P, dtype=torch.int64, device=dev))
            ctx.build_schedule(inst, settings, sizes, first, window=window, max_jobs=max_n)
            if want_profile:
                cap = first["horizon"] if profile_capacity is None else profile_capacity
                poff = torch.zeros(P + 1, dtype=torch.int64, device=dev)
                poff[1:] = torch.cumsum(cap, 0)
                ev["profile_off"] = poff
                ev["profile"] = torch.full((int(poff[-1]),), -7, dtype=torch.int32, device=dev)
            if want_runs:
                roff = torch.zeros(P + 1, dtype=torch.int64, device=dev)
                roff[1:] = torch.cumsum(sizes["n_runs"], 0)
                R = int(roff[-1])
                out["run_off"] = roff
                out["run_job"] = torch.empty(R, dtype=torch.int32, device=dev)
                out["run_phase"] = torch.empty(R, dtype=torch.int32, device=dev)
                out["run_start"] = torch.empty(R, dtype=torch.int64, device=dev)
                out["run_len"] = torch.empty(R, dtype=torch.int32, device=dev)
                out["run_s"] = torch.empty(R, dtype=torch.int32, device=dev)
        out["n_runs"] = torch.zeros(P, dtype=torch.int64, device=dev)
        ctx.evaluate_built(inst, settings, out, ev, window=window, max_jobs=max_n)
        runs = {k: out[k] for k in ("run_job", "run_phase", "run_start", "run_len", "run_s")} if want_runs else None
        sfx = "64" if time64 else ""
        return Result(ev["status"], ev["flow"], ev["peak"], ev["horizon"], ev["job_steps"], ev["n_unfinished"],
                      ev["feasible"], out.get("job_out_off"), out.get("job_start" + sfx), out.get("job_completion" + sfx),
                      ev.get("profile_off"), ev.get("profile"), out["n_runs"], out.get("run_off"), runs)

    def evaluate_runs(self, run_off, run_start, run_len, run_s, capacity, run_flow=None, M=None, want_profile=True):
        """Evaluate explicit runs (kvs_evaluate_schedule).  ``capacity`` is an int64 tensor [P]."""
        dev = run_start.device
        P = int(run_off.numel()) - 1
        poff = torch.zeros(P + 1, dtype=torch.int64, device=dev)
        poff[1:] = torch.cumsum(capacity, 0)
        total = int(poff[-1])
        ctx = self.context(binding.workspace_bytes(0, 0, 0, P, generic_capacity=max(total, 1)))
        ev = self.scalars(P, dev)
        ev["profile_off"] = poff
        if want_profile:
            ev["profile"] = torch.full((total,), -7, dtype=torch.int32, device=dev)
        runs = dict(run_off=run_off, run_start=run_start, run_len=run_len, run_s=run_s, run_flow=run_flow, M=M)
        ctx.evaluate_schedule(runs, ev)
        return Result(ev["status"], ev["flow"], ev["peak"], ev["horizon"], ev["job_steps"], ev["n_unfinished"],
                      ev["feasible"], profile_off=poff, profile=ev.get("profile"))

    def bounds(self, inst: Instances, settings: np.ndarray) -> dict:
        """Class-size bounds (kvs_bounds) of P (instance, setting) pairs; returns device tensors [P]."""
        dev = inst.s.device
        N, I, max_n, _ = self._sizes(inst)
        P = int(settings.shape[0])
        if P and (settings["instance"].min() < 0 or settings["instance"].max() >= I):
            raise binding.KvsError(-1, "settings: instance out of range")
        ctx = self.context(binding.workspace_bytes(N, I, max_n, P))
        out = {f: torch.zeros(P, dtype=torch.int64, device=dev) for f in ("upper_gba", "upper_gsa", "lower_2m")}
        out["status"] = torch.zeros(P, dtype=torch.int32, device=dev)
        ctx.bounds(inst, settings, out, max_jobs=max_n)
        return out

    def sweep_beta0(self, inst: Instances, instance: int, family, M: int, beta0, alpha=(2, 1), subroutine=0,
                    per_class_s=0) -> dict:
        """GBA / GSA over a list of initial slices on one instance; returns device tensors [n_beta0]."""
        dev = inst.s.device
        N, I, max_n, _ = self._sizes(inst)
        n_set = len(beta0)
        ctx = self.context(binding.workspace_bytes(N, I, max_n, n_set))
        out = {f: torch.zeros(n_set, dtype=torch.int64, device=dev)
               for f in ("peak", "flow", "n_completed", "horizon", "job_steps")}
        out["feasible"] = torch.zeros(n_set, dtype=torch.uint8, device=dev)
        ctx.sweep(inst, instance, family, M, [], [], out, max_jobs=max_n, beta0=beta0, alpha=alpha,
                  subroutine=subroutine, per_class_s=per_class_s)
        return out

    def sweep(self, inst: Instances, instance: int, family, M: int, tau, k) -> dict:
        """SPS / SimS over a (tau, k) grid on one instance; returns device tensors [n_tau, n_k]."""
        dev = inst.s.device
        N, I, max_n, _ = self._sizes(inst)
        ctx = self.context(binding.workspace_bytes(N, I, max_n, 0))
        n_set = len(tau) * len(k)
        out = {f: torch.zeros(n_set, dtype=torch.int64, device=dev)
               for f in ("peak", "flow", "n_completed", "horizon", "job_steps")}
        out["feasible"] = torch.zeros(n_set, dtype=torch.uint8, device=dev)
        ctx.sweep(inst, instance, family, M, tau, k, out, max_jobs=max_n)
        return {f: t.view(len(tau), len(k)) for f, t in out.items()}
