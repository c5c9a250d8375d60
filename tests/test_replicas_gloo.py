"""Multi-process (world_size 2, gloo, CPU) tests of the replica plumbing the benchmark uses for N > 1.

The path has no data-path collective: ranks are independent replicas.  What is shared is the
launcher environment, the per-replica seed, the barrier, the max-over-ranks time and the
aggregate -- all host logic, so it runs here without a GPU.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

import workloads as wl
from paper_2609_12330_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys, time
sys.path.insert(0, os.environ["EF_ROOT"])
import numpy as np
import workloads as wl
from paper_2609_12330_b200 import replicas

info = replicas.rank_info()
made = replicas.init_process_group(info, "gloo")
seed = replicas.replica_seed(info, base_seed=5)
p, t = wl.make_inputs("rmsnorm_matmul", seed=seed, size="small")
checksum = int(t["X"].astype(np.uint64).sum())
# rank r pretends its timed region took 10*(r+1) ms; rank 1 also arrives late at the barrier
if info.rank == 1:
    time.sleep(0.3)
t_before = time.time()
replicas.barrier(info)
t_after = time.time()
slowest = replicas.max_over_ranks(info, 10.0 * (info.rank + 1))
rate = replicas.aggregate_rate(info, 1000.0, slowest)
out = dict(rank=info.rank, world=info.world, local=info.local, made=made, seed=seed, checksum=checksum,
           slowest=slowest, rate=rate, left_barrier=t_after, entered_barrier=t_before, root=info.is_root)
with open(os.path.join(os.environ["EF_OUT"], f"rank{info.rank}.json"), "w") as f:
    json.dump(out, f)
replicas.destroy_process_group(info)
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(world, script, tmp_path, extra_env=None):
    port = _free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE=str(world), LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), EF_ROOT=ROOT, EF_OUT=str(tmp_path), OMP_NUM_THREADS="1")
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for pr in procs:
        try:
            o, e = pr.communicate(timeout=120)
        except subprocess.TimeoutExpired:
            pr.kill()
            o, e = pr.communicate()
        outs.append((pr.returncode, o, e))
    return outs


def test_two_replicas_over_gloo(tmp_path):
    outs = _launch(2, WORKER, tmp_path)
    for rc, o, e in outs:
        assert rc == 0, e[-2000:]
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(2)]
    assert [r["rank"] for r in res] == [0, 1] and all(r["world"] == 2 and r["made"] for r in res)
    assert res[0]["root"] and not res[1]["root"]
    # each replica draws its own inputs
    assert [r["seed"] for r in res] == [5, 6]
    assert res[0]["checksum"] != res[1]["checksum"]
    for r in res:
        _, t = wl.make_inputs("rmsnorm_matmul", seed=r["seed"], size="small")
        assert int(t["X"].astype(np.uint64).sum()) == r["checksum"]
    # the job's time is the slowest rank's, on every rank; the aggregate counts both replicas' units
    assert all(r["slowest"] == 20.0 for r in res)
    assert all(r["rate"] == pytest.approx(2 * 1000.0 / 20e-3) for r in res)
    # nobody leaves the barrier before the late rank has entered it
    assert res[0]["left_barrier"] >= res[1]["entered_barrier"] - 1e-3


def test_single_process_needs_no_group():
    info = replicas.rank_info({})
    assert (info.rank, info.world, info.local, info.is_root) == (0, 1, 0, True)
    assert replicas.init_process_group(info, "gloo") is False
    replicas.barrier(info)                                  # no group: returns at once
    assert replicas.max_over_ranks(info, 3.5) == 3.5
    assert replicas.aggregate_rate(info, 10.0, 2.0) == pytest.approx(5000.0)
    assert replicas.replica_seed(info, 7) == 7


def test_rank_info_rejects_inconsistent_environment():
    with pytest.raises(ValueError):
        replicas.rank_info({"RANK": "2", "WORLD_SIZE": "2"})
    with pytest.raises(ValueError):
        replicas.rank_info({"RANK": "0", "WORLD_SIZE": "0"})
    info = replicas.rank_info({"RANK": "3", "WORLD_SIZE": "8"})
    assert info.local == 3                                  # local rank defaults to the rank on one node


def test_reference_arm_runs_on_rank_zero_only():
    """Under a 2-rank launch the oracle arm's non-root rank exits 0 without work or output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=60)
    assert r.returncode == 0, r.stderr[-2000:]
    assert r.stdout.strip() == ""


def test_our_arm_fails_loudly_without_a_gpu():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0
    assert "no CPU path" in r.stderr
