"""The N > 1 path of the benchmark on CPU: two gloo ranks run independent replicas (the path
does not shard across GPUs; there is no collective on the data path), agree on the slowest
rank's time through a MAX all-reduce and rank 0 reports the whole-job value."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import torch
    import torch.distributed as dist
    from bench import aggregate_replicas, replica_job_value
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group(backend="gloo")
    # every rank 'measured' its own step time for the same per-rank work
    my_ms = 10.0 + 5.0 * rank
    slowest = aggregate_replicas(my_ms, dist, torch.device("cpu"))
    assert abs(slowest - 15.0) < 1e-9, slowest          # MAX over ranks, on every rank
    value = replica_job_value(batch=32, world=world, ms_per_step=slowest)
    if rank == 0:
        print(json.dumps({{"value": value, "ms": slowest, "world": world}}))
    dist.barrier()
    dist.destroy_process_group()
""")


def test_two_gloo_ranks_report_max_time_and_whole_job_value(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29631")
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29631", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    import json
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["world"] == 2 and out["ms"] == 15.0
    # two replicas of 32 sequences each, one token per sequence per step, at the slowest rank's pace
    assert abs(out["value"] - 2 * 32 / 0.015) < 1e-6


def test_peer_tier_workload_says_unavailable_without_two_gpus():
    """The peer-GPU second tier needs two GPUs in one process; anywhere else the workload must say
    so in one JSON line and exit 0 instead of touching a device."""
    import json
    import pytest
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        pytest.skip("this box has two GPUs: the workload would run")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "peer_tier"],
                         capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    out = json.loads([l for l in res.stdout.splitlines() if l.startswith("{")][-1])
    assert out["workload"] == "peer_gpu_second_tier" and "two GPUs" in out["unavailable"]
