"""The exchange in front of and behind the head-sharded path (sequence shards <-> head shards),
on two gloo ranks: each rank must end up with every token of its own heads, in token order, and
the way back must restore its token slice of every head."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
B, H, N, D = 2, 6, 40, 8


def _full():
    return torch.arange(B * H * N * D, dtype=torch.float32).reshape(B, H, N, D)


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_15810_b200 import sequence_parallel as SP
    x = _full()
    n, h = N // world, H // world
    mine = x[:, :, rank * n:(rank + 1) * n].contiguous()                  # my token slice of every head
    heads = SP.seq_to_head_shard(mine)
    ok = torch.equal(heads, x[:, rank * h:(rank + 1) * h])               # every token of my heads, in order
    back = SP.head_to_seq_shard(heads * 2.0)
    ok = ok and torch.equal(back, 2.0 * mine)
    try:
        SP.seq_to_head_shard(mine[:, :5])                                 # 5 heads on 2 ranks
        ok = False
    except ValueError:
        pass
    dist.barrier()
    out.put((rank, bool(ok)))
    dist.destroy_process_group()


def test_exchange_on_two_gloo_ranks():
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
    assert results == [(0, True), (1, True)]


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    from paper_2609_15810_b200 import sequence_parallel as SP
    x = _full()
    assert torch.equal(SP.seq_to_head_shard(x), x) and torch.equal(SP.head_to_seq_shard(x), x)
