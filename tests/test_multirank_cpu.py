"""The N > 1 path of bench.py on CPU: two gloo ranks, max-over-ranks step time, whole-job
throughput (heads are independent, so ranks exchange nothing but the timing)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    value, ms = bench.job_throughput(2.0e12, ms_local, world)
    assert ms == 15.0
    assert abs(value - world * 2.0e12 / 15e-3 / 1e12) < 1e-9
    assert bench.max_over_ranks(float(rank)) == world - 1
    dist.barrier()
    out.put((rank, value, ms))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_job_throughput():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0][1:] == results[1][1:]
    assert abs(results[0][1] - 2 * 2.0 / 15e-3) < 1e-6


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.job_throughput(1.0e12, 20.0, 1)
    assert ms == 20.0 and abs(value - 50.0) < 1e-9
