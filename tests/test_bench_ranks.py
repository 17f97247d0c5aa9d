"""The multi-replica arithmetic of bench.py on two CPU processes (gloo): the job's time is the slowest replica's,
its throughput the images of all replicas over that time; replicas draw different synthetic batches; the
reference arm runs on rank 0 only.  No GPU, no data-path collective: images are independent through every layer."""
import os
import socket
import subprocess
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    import dr_synth as S
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 40.0 + 10.0 * rank                       # rank 1 is the slow replica
    ms = bench.max_over_ranks(local_ms, world, device="cpu")
    value = bench.whole_job_images_per_s(ms, 256, 10, world)
    x = S.stream(rank, "bench.x").standard_normal(8, dtype=np.float32)
    out.put((rank, ms, value, x.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, v0, x0), (r1, ms1, v1, x1) = res
    assert ms0 == ms1 == 50.0                            # max over ranks, the same on every rank
    assert v0 == v1 == 2 * 256 * 10 / 0.050              # whole-job images per second
    assert x0 != x1                                      # per-rank seed: the replicas see different images


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, 1) == 12.5
    assert bench.whole_job_images_per_s(4.0, 256, 100, 1) == 256 * 100 / 0.004
