"""The N > 1 launch of bench.py on CPU: two gloo ranks, no GPU.

The path shards by replication (every rank compresses its own copy of the workload, no data-path collective),
so what the ranks share is the timing: the slowest rank's time and the whole-job aggregate; the reference arm
runs on rank 0 alone.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
my_ms = [10.0, 14.5][rank]
slowest = bench.max_over_ranks(my_ms, dist, "cpu")
specs = bench.workload_specs("small_bf16")[1]
seeds = [s.seed + bench.rank_seed_offset(rank) for s in specs]
gathered = [None] * world
dist.all_gather_object(gathered, seeds)
dist.barrier()
if rank == 0:
    print(json.dumps({"slowest": slowest, "value": bench.whole_job_gbs(world, 10**9, slowest),
                      "disjoint": len(set(gathered[0]) & set(gathered[1])) == 0, "n": len(seeds)}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_args, world=2, extra_env=None):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), **(extra_env or {}))
        procs.append(subprocess.Popen([sys.executable] + code_or_args, env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    return [(p.returncode, o, e) for p, (o, e) in zip(procs, outs)]


def test_two_ranks_share_the_slowest_time_and_use_their_own_seeds():
    res = _spawn(["-c", WORKER, ROOT])
    for rc, out, err in res:
        assert rc == 0, err
    line = json.loads(res[0][1].strip().splitlines()[-1])
    assert res[1][1].strip() == ""                                   # only rank 0 prints
    assert line["slowest"] == 14.5
    assert line["value"] == pytest.approx(2 * 1e9 / 14.5 / 1e6)      # both ranks' bytes over the slowest rank's time
    assert line["disjoint"] and line["n"] > 0


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25, None, "cpu") == 3.25
    assert bench.rank_seed_offset(0) == 0
    assert bench.whole_job_gbs(1, 2 * 10**9, 1000.0) == pytest.approx(2.0)


def test_reference_arm_runs_on_rank_zero_only(monkeypatch):
    """`bench.py --impl reference` under a 2-rank launch: rank 1 exits 0 without work or output; rank 0 prints
    the line with the keys the contract asks for (a tiny sample keeps it short)."""
    res = _spawn([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                  "--workload", "small_bf16"], extra_env={"ZC_ORACLE_SAMPLE_BYTES": str(1 << 20)})
    for rc, out, err in res:
        assert rc == 0, err
    assert res[1][1].strip() == ""
    line = json.loads(res[0][1].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
