"""The N > 1 plumbing of bench.py on CPU: two gloo ranks on 127.0.0.1.  The path shards by replicas (no
data-path collective), so what has to be right is the whole-job view: max time over ranks, summed units, the
barrier, and that only rank 0 of the reference arm does any work."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["MRL_ROOT"])
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
bench.barrier(world)
ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), world)
bench.barrier(world)
dist.destroy_process_group()
print(json.dumps({"rank": rank, "ms": ms, "units": units}))
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _env(rank, world, port):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port), MRL_ROOT=ROOT, OMP_NUM_THREADS="2")
    return env


def test_two_gloo_ranks_agree_on_max_time_and_total_units():
    port = _free_port()
    procs = [subprocess.Popen([sys.executable, "-c", WORKER], env=_env(r, 2, port), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    res = [json.loads(o.strip().splitlines()[-1]) for o, _ in outs]
    for r in res:
        assert r["ms"] == 15.0          # the slower rank's time
        assert r["units"] == 3000.0     # the units of both ranks


def test_single_rank_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0, 1) == (3.5, 7.0)


def test_reference_arm_runs_on_rank_zero_only():
    """Under a 2-rank launch rank 1 of `--impl reference` exits 0 without printing or working."""
    port = _free_port()
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=_env(1, 2, port), capture_output=True, text=True,
                       timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""
