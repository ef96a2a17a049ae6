"""N > 1 plumbing on CPU: the path has no exchange step (one replica per rank), so the only
multi-rank logic is the reduction of the timings -- max over ranks of the device time, sum over
ranks of the bytes processed.  Run here with the gloo backend, world size 2, on 127.0.0.1."""
import json
import os
import socket
import subprocess
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist  # noqa: E402
import torch.multiprocessing as mp  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    local_ms = 10.0 + 5.0 * rank          # rank 1 is the slow one
    local_units = 1.0e9 * (rank + 1)      # bytes this rank processed
    t, u = bench.reduce_over_ranks(local_ms, local_units, dist, torch.device("cpu"))
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"t": t, "u": u}, f)
    dist.destroy_process_group()


def test_timing_reduction_over_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        got = json.load(open(tmp_path / f"r{rank}.json"))
        assert got == {"t": 15.0, "u": 3.0e9}  # max of the times, sum of the units, on every rank
    # whole-job throughput = all ranks' bytes / slowest rank's time
    assert 3.0e9 / 15.0 == pytest.approx(2.0e8)


def test_single_process_reduction_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.reduce_over_ranks(7.5, 42.0) == (7.5, 42.0)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""  # other ranks exit 0 without work
