"""Seeded synthetic workloads for the schedule builder / evaluator.

This module only draws inputs (prompt lengths ``s``, response lengths ``o``,
estimates ``o_est``, arrival times, budgets ``M``, sweep grids).  It contains
none of the scheduling arithmetic, so that the CUDA path and the CPU oracle can
both be fed from it without sharing any of the method's code.

Every draw is a pure function of ``(seed, stream, counter)``: a splitmix64
finaliser is applied to a 64-bit counter, uniforms use the top 53 bits, normals
use Box-Muller.  All integer hashing is exact on CPU and CUDA tensors alike;
the floating-point transforms may differ by an ulp between devices, which can
move a rounded draw by one but never affects parity because both sides always
read the same generated arrays.

The shapes stand in for the right-skewed response-length trace the paper
measures on (Numerical Experiments, trace-driven part), which is not available
offline.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

BASE_SEED = 20260122

_MASK64 = (1 << 64) - 1


def _i64(x: int) -> int:
    """Wrap an unsigned 64-bit constant into the signed range torch uses."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _i64(0x9E3779B97F4A7C15)
_MIX1 = _i64(0xBF58476D1CE4E5B9)
_MIX2 = _i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def _splitmix64(z: torch.Tensor) -> torch.Tensor:
    z = z + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MIX1
    z = (z ^ _lsr(z, 27)) * _MIX2
    return z ^ _lsr(z, 31)


def _splitmix64_int(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, *tags: int) -> int:
    """Derive a 64-bit stream key from a seed and integer tags."""
    h = _splitmix64_int(seed & _MASK64)
    for t in tags:
        h = _splitmix64_int(h ^ (t & _MASK64))
    return h


def bits(key: int, counter: torch.Tensor) -> torch.Tensor:
    """64 random bits per counter value (int64 tensor in, int64 tensor out)."""
    return _splitmix64(counter * _GOLDEN + _i64(key))


def uniform01(key: int, counter: torch.Tensor) -> torch.Tensor:
    """Uniform doubles in (0, 1): top 53 bits plus half an ulp."""
    b = _lsr(bits(key, counter), 11).to(torch.float64)
    return (b + 0.5) * (1.0 / 9007199254740992.0)


def normal(key: int, counter: torch.Tensor) -> torch.Tensor:
    """Standard normal doubles (Box-Muller on two independent streams)."""
    u1 = uniform01(key, counter)
    u2 = uniform01(_splitmix64_int(key ^ 0x5851F42D4C957F2D), counter)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)


def _round_clip(x: torch.Tensor, lo: int, hi: int) -> torch.Tensor:
    return torch.clamp(torch.floor(x + 0.5), lo, hi).to(torch.int32)


# ---- marginal distributions ------------------------------------------------

def uniform_int(key: int, counter: torch.Tensor, lo: int, hi: int) -> torch.Tensor:
    u = uniform01(key, counter)
    return torch.clamp(torch.floor(u * (hi - lo + 1)) + lo, lo, hi).to(torch.int32)


def lognormal_int(key, counter, median: float, sigma: float, lo: int, hi: int):
    return _round_clip(median * torch.exp(sigma * normal(key, counter)), lo, hi)


def pareto_int(key, counter, x_m: float, alpha: float, lo: int, hi: int):
    u = uniform01(key, counter)
    return _round_clip(x_m * torch.pow(u, -1.0 / alpha), lo, hi)


def geometric_int(key, counter, mean: float, lo: int, hi: int):
    """Geometric on {1, 2, ...} with success probability 1/mean."""
    u = uniform01(key, counter)
    p = 1.0 / mean
    x = torch.floor(torch.log(u) / math.log1p(-p)) + 1.0
    return torch.clamp(x, lo, hi).to(torch.int32)


# ---- workload containers ---------------------------------------------------

@dataclass
class Instances:
    """Batched instances in CSR form (tensors on one device)."""
    job_off: torch.Tensor                 # int64 [I+1]
    s: torch.Tensor                       # int32 [N]
    o: torch.Tensor                       # int32 [N]
    o_est: torch.Tensor | None = None     # int32 [N]
    arrival: torch.Tensor | None = None   # int64 [N], nondecreasing per instance
    meta: dict = field(default_factory=dict)

    @property
    def n_instances(self) -> int:
        return self.job_off.numel() - 1

    def to(self, device) -> "Instances":
        mv = lambda t: None if t is None else t.to(device)
        return Instances(mv(self.job_off), mv(self.s), mv(self.o), mv(self.o_est),
                         mv(self.arrival), dict(self.meta))

    def slice(self, lo: int, hi: int) -> "Instances":
        """Instances lo..hi-1 as a new batch (offsets rebased to zero)."""
        off = self.job_off[lo:hi + 1]
        a, b = int(off[0]), int(off[-1])
        cut = lambda t: None if t is None else t[a:b]
        return Instances(off - a, self.s[a:b], self.o[a:b], cut(self.o_est),
                         cut(self.arrival), dict(self.meta))


def _counters(first_instance: int, n_inst: int, n: int, device) -> torch.Tensor:
    """Global job counter: instance * 2^32 + position (unique per job)."""
    inst = torch.arange(first_instance, first_instance + n_inst, dtype=torch.int64, device=device)
    pos = torch.arange(n, dtype=torch.int64, device=device)
    return (inst[:, None] * (1 << 32) + pos[None, :]).reshape(-1)


def _uniform_offsets(n_inst: int, n: int, device) -> torch.Tensor:
    return torch.arange(n_inst + 1, dtype=torch.int64, device=device) * n


S_LOGNORMAL = dict(median=256.0, sigma=1.0, lo=1, hi=8192)
O_PARETO = dict(x_m=64.0, alpha=1.5, lo=1, hi=16384)


def config1(seed: int = BASE_SEED, n: int = 1000, device="cpu") -> Instances:
    """One instance, uniform prompt and response lengths, M = 200,000."""
    c = _counters(0, 1, n, device)
    s = uniform_int(stream_key(seed, 1, 1), c, 16, 512)
    o = uniform_int(stream_key(seed, 1, 2), c, 1, 1024)
    return Instances(_uniform_offsets(1, n, device), s, o,
                     meta=dict(config=1, M=[200_000], families=["GBA", "GSA", "SPS", "SIMS"]))


def config2(seed: int = BASE_SEED, n_inst: int = 1024, n: int = 10_000, device="cpu",
            first_instance: int = 0) -> Instances:
    """Lognormal prompts, Pareto responses, M swept over 2^17..2^24."""
    c = _counters(first_instance, n_inst, n, device)
    s = lognormal_int(stream_key(seed, 2, 1), c, **S_LOGNORMAL)
    o = pareto_int(stream_key(seed, 2, 2), c, **O_PARETO)
    return Instances(_uniform_offsets(n_inst, n, device), s, o,
                     meta=dict(config=2, M=[1 << e for e in range(17, 25)], families=["GBA", "GSA"]))


def config3(seed: int = BASE_SEED, n_inst: int = 256, n: int = 100_000, device="cpu",
            M: int = 1 << 22, load: float = 0.9, window: int = 1024,
            first_instance: int = 0) -> Instances:
    """Online arrivals at a given load, geometric responses, noisy estimates."""
    c = _counters(first_instance, n_inst, n, device)
    s = lognormal_int(stream_key(seed, 3, 1), c, **S_LOGNORMAL)
    o = geometric_int(stream_key(seed, 3, 2), c, 512.0, 1, 16384)
    noise = torch.exp(0.5 * normal(stream_key(seed, 3, 3), c))
    o_est = _round_clip(o.to(torch.float64) * noise, 1, M - 8192)
    # Poisson arrivals: exponential gaps with rate = load * M / mean memory-time footprint.
    sd, od = s.to(torch.float64).view(n_inst, n), o.to(torch.float64).view(n_inst, n)
    footprint = (sd * od + od * (od + 1.0) / 2.0).mean(dim=1, keepdim=True)
    rate = load * M / footprint
    gaps = -torch.log(uniform01(stream_key(seed, 3, 4), c)).view(n_inst, n) / rate
    arrival = torch.floor(torch.cumsum(gaps, dim=1)).to(torch.int64).reshape(-1)
    return Instances(_uniform_offsets(n_inst, n, device), s, o, o_est, arrival,
                     meta=dict(config=3, M=[M], window=window, families=["GBA", "GSA"]))


def sweep_grids() -> tuple[list[int], list[int]]:
    """64 geometric slice lengths 16..2^14 and 64 parallelism values 2..2^14."""
    tau = [int(math.floor(16.0 * 2.0 ** (10.0 * j / 63.0) + 0.5)) for j in range(64)]
    k = [int(math.ceil(2.0 ** (14.0 * (j + 1) / 64.0) - 1e-9)) for j in range(64)]
    return tau, k


def config4(seed: int = BASE_SEED, n: int = 1_000_000, device="cpu") -> Instances:
    """One large instance for the (tau, k) sweep; M = 2^22 for the feasibility mask."""
    c = _counters(0, 1, n, device)
    s = lognormal_int(stream_key(seed, 4, 1), c, **S_LOGNORMAL)
    o = pareto_int(stream_key(seed, 4, 2), c, **O_PARETO)
    tau, k = sweep_grids()
    return Instances(_uniform_offsets(1, n, device), s, o,
                     meta=dict(config=4, M=[1 << 22], tau=tau, k=k, families=["SPS", "SIMS"]))


def config5(seed: int = BASE_SEED, n_inst: int = 16_384, n: int = 50_000, device="cpu",
            first_instance: int = 0) -> Instances:
    """Stress: per-instance mix of uniform / lognormal / Pareto marginals, M per instance."""
    inst_ids = list(range(first_instance, first_instance + n_inst))
    c = _counters(first_instance, n_inst, n, device).view(n_inst, n)
    ks, ko = stream_key(seed, 5, 1), stream_key(seed, 5, 2)
    kinds = torch.tensor([stream_key(seed, 5, 3, i) % 9 for i in inst_ids], device=device)
    s = torch.empty((n_inst, n), dtype=torch.int32, device=device)
    o = torch.empty((n_inst, n), dtype=torch.int32, device=device)
    s_gen = [lambda cc: uniform_int(ks, cc, 16, 512),
             lambda cc: lognormal_int(ks, cc, **S_LOGNORMAL),
             lambda cc: pareto_int(ks, cc, 32.0, 1.5, 1, 8192)]
    o_gen = [lambda cc: uniform_int(ko, cc, 1, 1024),
             lambda cc: lognormal_int(ko, cc, 128.0, 1.0, 1, 16384),
             lambda cc: pareto_int(ko, cc, **O_PARETO)]
    for d in range(3):
        rows = torch.nonzero(kinds // 3 == d).flatten()
        if rows.numel():
            s[rows] = s_gen[d](c[rows].reshape(-1)).view(rows.numel(), n)
        rows = torch.nonzero(kinds % 3 == d).flatten()
        if rows.numel():
            o[rows] = o_gen[d](c[rows].reshape(-1)).view(rows.numel(), n)
    um = uniform01(stream_key(seed, 5, 4), torch.tensor(inst_ids, dtype=torch.int64, device=device))
    M = torch.floor(torch.pow(2.0, 18.0 + 6.0 * um)).to(torch.int64)
    return Instances(_uniform_offsets(n_inst, n, device), s.reshape(-1), o.reshape(-1),
                     meta=dict(config=5, M_per_instance=M, families=["GBA", "GSA", "SPS", "SIMS"]))


def random_small(seed: int, n_inst: int, n_max: int, s_max: int, o_max: int, device="cpu",
                 with_est: bool = False, equal_s: bool = False) -> Instances:
    """Ragged batch of tiny instances (sizes 0..n_max) for exhaustive parity tests."""
    key = stream_key(seed, 99)
    sizes = [(_splitmix64_int(key ^ i) % (n_max + 1)) for i in range(n_inst)]
    off = torch.zeros(n_inst + 1, dtype=torch.int64)
    off[1:] = torch.cumsum(torch.tensor(sizes, dtype=torch.int64), 0)
    N = int(off[-1])
    c = torch.arange(N, dtype=torch.int64)
    s = uniform_int(stream_key(seed, 99, 1), c, 0, s_max)
    o = uniform_int(stream_key(seed, 99, 2), c, 1, o_max)
    if equal_s:
        inst_of = torch.repeat_interleave(torch.arange(n_inst), torch.tensor(sizes))
        s = uniform_int(stream_key(seed, 99, 4), inst_of.to(torch.int64), 0, s_max)
    est = None
    if with_est:
        noise = torch.exp(0.7 * normal(stream_key(seed, 99, 3), c))
        est = _round_clip(o.to(torch.float64) * noise, 1, 4 * o_max)
    out = Instances(off, s, o, est, meta=dict(config=0))
    return out.to(device)
