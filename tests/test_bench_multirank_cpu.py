"""Host-side logic of the N > 1 benchmark path, on CPU with the gloo backend and world_size 2: the step time is
the maximum over ranks, the value is all ranks' images over that time, and under `--impl reference` only rank 0
prints a line."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = [2.0 + rank, 10.0 - 3 * rank]          # rank 0: (2, 10), rank 1: (3, 7)
    got = bench.max_over_ranks(local_ms, world, "cpu")
    val = bench.whole_job_value(128, world, got[0])
    out.put((rank, got, val))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, val in res:
        assert got == [3.0, 10.0]                        # max over ranks, element-wise
        assert val == pytest.approx(2 * 128 / 3e-3)      # both ranks' images over the slowest rank's step


def test_reference_arm_only_rank0_prints():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    outs = []
    for rank in (0, 1):
        e = dict(env, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank))
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--steps", "1", "--warmup", "0", "--config", "0"], env=e, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-500:]
        outs.append(r.stdout.strip())
    line = json.loads(outs[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert outs[1] == ""
