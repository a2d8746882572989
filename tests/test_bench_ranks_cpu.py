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


LAUNCHED = r"""
import os, sys, json
sys.path.insert(0, os.environ["MRL_ROOT"])
import torch.distributed as dist
import bench
rank, world, local = bench.resolve_world(int(sys.argv[1]))
dist.init_process_group("gloo")
ms, units = bench.aggregate_over_ranks(1.0 + rank, 10.0, world)
dist.destroy_process_group()
if rank == 0:
    print(json.dumps({"n_gpus": world, "ms": ms, "units": units}), flush=True)
if len(sys.argv) > 2 and int(sys.argv[2]) == rank:
    sys.exit(3)
"""


def _run_launcher(tmp_path, n, fail_rank=None):
    script = tmp_path / "worker.py"
    script.write_text(LAUNCHED)
    code = ("import sys, os; sys.path.insert(0, os.environ['MRL_ROOT']); import bench; "
            f"sys.exit(bench.launch_ranks({n}, {[str(n)] + ([str(fail_rank)] if fail_rank is not None else [])!r}, "
            f"script={str(script)!r}))")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    env.update(MRL_ROOT=ROOT, OMP_NUM_THREADS="2")
    return subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=180)


def test_launcher_starts_one_gloo_rank_per_gpu_asked_for(tmp_path):
    """`bench.py --gpus N` without a launcher's environment starts N ranks itself: here two gloo ranks on CPU."""
    res = _run_launcher(tmp_path, 2)
    assert res.returncode == 0, res.stderr
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line == {"n_gpus": 2, "ms": 2.0, "units": 20.0}


def test_launcher_reports_a_failed_rank(tmp_path):
    res = _run_launcher(tmp_path, 2, fail_rank=1)
    assert res.returncode != 0


def test_world_size_must_match_gpus():
    """A launcher that started a different number of ranks than --gpus says is an error, never a silent N = 1."""
    sys.path.insert(0, ROOT)
    import bench
    import pytest
    saved = {k: os.environ.pop(k, None) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    try:
        assert bench.resolve_world(1) == (0, 1, 0)
        assert bench.resolve_world(4) is None                 # nothing launched yet: the caller starts the ranks
        os.environ.update(WORLD_SIZE="2", RANK="1", LOCAL_RANK="1")
        assert bench.resolve_world(2) == (1, 2, 1)
        with pytest.raises(SystemExit):
            bench.resolve_world(8)
        with pytest.raises(SystemExit):
            bench.resolve_world(1)
    finally:
        for k, v in saved.items():
            os.environ.pop(k, None)
            if v is not None:
                os.environ[k] = v


def test_plain_invocation_with_gpus_two_runs_two_ranks_of_the_reference_arm():
    """End to end on CPU: `python bench.py --gpus 2 --impl reference` (no torchrun) prints one line that says 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    env.update(OMP_NUM_THREADS="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--workload", "C1", "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                         text=True, timeout=300)
    assert res.returncode == 0, res.stderr
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert json.loads(lines[0])["n_gpus"] == 2 and json.loads(lines[0])["impl"] == "reference"
