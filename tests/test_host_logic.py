"""CPU-only checks: the library builds, loads and exports every declared symbol; the seeded
generators are deterministic and shard consistently; the multi-rank reporting path (gloo, 2 ranks)."""
import os
import re

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from paper_2601_22996_b200 import binding, sharding, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "kvs.h")).read()
    declared = set(re.findall(r"\b(kvs_[a-z_0-9]+)\s*\(", header))
    declared -= {"kvs_status", "kvs_family", "kvs_eval_status"}
    lib = binding.load()
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_the_header():
    import ctypes
    assert binding.SETTING_DTYPE.itemsize == 64 and binding.SETTING_DTYPE.fields['subroutine'][1] == 56
    assert ctypes.sizeof(binding._Instances) == 72 and ctypes.sizeof(binding._ScheduleOut) == 96
    assert ctypes.sizeof(binding._EvalOut) == 72 and ctypes.sizeof(binding._Runs) == 56
    assert ctypes.sizeof(binding._SweepParams) == 72 and binding._SweepParams.beta0.offset == 48 and ctypes.sizeof(binding._SweepOut) == 48


def test_family_and_status_codes_match_the_header():
    """The binding and the oracle number the schedule families like `enum kvs_family`; the status bits the tests
    read are those of `enum kvs_eval_status`."""
    import oracle
    header = open(os.path.join(ROOT, "include", "kvs.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    fam = dict((k, int(v)) for k, v in re.findall(r"KVS_(GBA|GSA|SPS|SIMS|GBAD|GSAS)\s*=\s*(\d+)", header))
    assert fam == binding.FAMILY == oracle.FAMILY and len(fam) == 6
    bits = dict((k, int(v, 0)) for k, v in re.findall(r"KVS_EVAL_([A-Z_]+)\s*=\s*(0x[0-9a-fA-F]+|\d+)", header))
    assert bits["INFEASIBLE"] == binding.EVAL_INFEASIBLE and bits["BAD_INPUT"] == binding.EVAL_BAD_INPUT


def test_no_gpu_means_a_loud_failure():
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.KvsError):
        binding.Context(torch.zeros(1024, dtype=torch.uint8))
    assert binding.workspace_bytes(10_000, 4, 5_000, 16) > 0        # host-only entry point still works


def test_generators_are_deterministic_and_in_range():
    a, b = workloads.config2(n_inst=3, n=500), workloads.config2(n_inst=3, n=500)
    assert torch.equal(a.s, b.s) and torch.equal(a.o, b.o)
    assert int(a.s.min()) >= 1 and int(a.s.max()) <= 8192 and int(a.o.min()) >= 1 and int(a.o.max()) <= 16384
    c3 = workloads.config3(n_inst=2, n=2000)
    arr = c3.arrival.view(2, 2000)
    assert bool((arr[:, 1:] >= arr[:, :-1]).all()) and int(c3.o_est.min()) >= 1
    c5 = workloads.config5(n_inst=9, n=300)
    M = c5.meta["M_per_instance"]
    assert int(M.min()) >= 1 << 18 and int(M.max()) < 1 << 24
    tau, k = workloads.sweep_grids()
    assert (tau[0], tau[-1], len(tau)) == (16, 16384, 64) and (k[0], k[-1], len(k)) == (2, 16384, 64)
    assert workloads.config2(seed=1, n_inst=1, n=50).o.tolist() != workloads.config2(seed=2, n_inst=1, n=50).o.tolist()


def test_shards_tile_the_seeded_stream():
    whole = workloads.config5(n_inst=6, n=200)
    for rank in range(2):
        part = workloads.config5(n_inst=3, n=200, first_instance=sharding.shard_first_instance(rank, 3))
        assert torch.equal(part.s, whole.s[rank * 600:(rank + 1) * 600])
        assert torch.equal(part.o, whole.o[rank * 600:(rank + 1) * 600])
        assert torch.equal(part.meta["M_per_instance"], whole.meta["M_per_instance"][rank * 3:(rank + 1) * 3])


def _rank_main(rank, world, port, q):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    inst = workloads.config2(n_inst=2, n=100, first_instance=sharding.shard_first_instance(rank, 2))
    times, counts = sharding.reduce_report([10.0 + rank, 5.0 - rank], [float(inst.o.sum()), 2.0], "cpu", world)
    q.put((rank, times, counts, int(inst.o.sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_reporting_over_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    total = got[0][3] + got[1][3]
    for _, times, counts, _ in got:
        assert times == [11.0, 5.0] and counts == [float(total), 4.0]     # max over ranks, sum over ranks
    whole = workloads.config2(n_inst=4, n=100)
    assert int(whole.o.sum()) == total                                    # the two shards are the 4-instance stream


def test_reference_arm_prints_one_json_line():
    """bench.py --impl reference times the oracle on the host and prints the contract's JSON line."""
    import json
    import subprocess
    import sys
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                          "--cpu-seconds", "0.5"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["value"] > 0 and d["unit"] == "job-steps/s" and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
