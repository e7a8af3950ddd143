"""The checked build of the library (-DKVS_DEBUG): every computed index of the fast fused kernel and of the
refill and speculative-run kernels is tested against its bound before the access, a violation is recorded in one device word and the access skipped.
compute-sanitizer is not available on the GPU pool, so this is the memory-safety evidence: the tiny, edge,
window and estimate parity cases run against the checked library in a child process (the binding keeps one
library per process) and must leave the word at 0 while still matching the oracle bit for bit."""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, {root!r})
import numpy as np, torch
from paper_2601_22996_b200 import binding, build, workloads
binding.load(path=build.build(debug=True))
word, checked = binding.debug_check_word(reset=True)
assert checked, "the library loaded is not the checked build"
from tests import parity
# tiny ragged instances, all families, three alphas (incl. empty and one-job instances)
inst = workloads.random_small(911, 70, 60, 40, 120)
sizes = (inst.job_off[1:] - inst.job_off[:-1]).numpy()
rows = []
for i in range(inst.n_instances):
    a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
    M = (int(inst.s[a:b].max() + inst.o[a:b].max()) if b > a else 10) + 5 * i
    for fam in ("GBA", "GSA", "SPS", "SIMS"):
        rows.append(dict(instance=i, family=fam, M=M, alpha=((2, 1), (3, 2), (7, 4))[i % 3]))
parity.check_batch(inst, binding.make_settings(rows), want_runs=False, label="checked tiny")
# estimates and arrival windows
inst = workloads.random_small(912, 20, 300, 60, 200, with_est=True)
arr = torch.zeros_like(inst.o, dtype=torch.int64)
for i in range(inst.n_instances):
    a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
    arr[a:b] = torch.arange(b - a, dtype=torch.int64) * 2
inst.arrival = arr
rows = []
for i in range(inst.n_instances):
    a, b = int(inst.job_off[i]), int(inst.job_off[i + 1])
    if b > a:
        M = int(inst.s[a:b].max() + inst.o[a:b].max()) + 300
        rows += [dict(instance=i, family=f, M=M) for f in ("GBA", "GSA", "SPS", "SIMS")]
parity.check_batch(inst, binding.make_settings(rows), window=37, want_runs=False, label="checked est+windows")
# several tiles, a ragged tail, dense and sparse phases: config 2 and config 5 subsets
c2 = workloads.config2(n_inst=3, n=10_000)
parity.check_batch(c2, binding.settings_grid(range(3), ["GBA", "GSA", "SPS", "SIMS"], [1 << 17, 1 << 20, 1 << 24]), want_runs=False, label="checked config 2")
c5 = workloads.config5(n_inst=4, n=50_000)
st = binding.settings_grid(range(4), ["GBA", "GSA"], c5.meta["M_per_instance"].numpy()[:, None])
parity.check_batch(c5, st, want_runs=False, label="checked config 5")
# the kernels of the two heuristics: hand-sized, ragged and config-2 cases
heur = workloads.random_small(913, 40, 60, 30, 90)
rows = []
for i in range(heur.n_instances):
    a, b = int(heur.job_off[i]), int(heur.job_off[i + 1])
    if b > a:
        M = int(heur.s[a:b].max() + heur.o[a:b].max()) + 11 * i
        rows += [dict(instance=i, family=f, M=M, alpha=((2, 1), (3, 2))[i % 2]) for f in ("GBAD", "GSAS")]
parity.check_batch(heur, binding.make_settings(rows), want_runs=False, label="checked heuristics tiny")
parity.check_batch(c2, binding.settings_grid(range(3), ["GBAD", "GSAS"], [1 << 17, 1 << 20, 1 << 24]), want_runs=False, label="checked heuristics config 2")
torch.cuda.synchronize()
word, _ = binding.debug_check_word()
print("CHECK_WORD", hex(word))
assert word == 0, f"index violation: code {{word >> 56}}, index {{word & ((1 << 56) - 1)}}"
"""


def test_checked_build_records_no_violation():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    r = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT)], capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "CHECK_WORD 0x0" in r.stdout
