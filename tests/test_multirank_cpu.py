"""The N > 1 plumbing of bench.py on the CPU: two gloo ranks, each with its own batch (sharding by
sequence, no data-path collective); the job's time is the slowest rank's and its bytes are the sum."""
import os
import socket
import sys
from pathlib import Path

import torch
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, str(ROOT))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    import bench
    from paper_2512_05033_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shape = wl.DRAFT_DECODE

    def kv_bytes(r):
        g = torch.Generator().manual_seed(bench.rank_seed(shape, r))
        prefix = wl.draw_prefix_lens(shape, g)
        return bench.attn_bytes(shape, prefix + 1, torch.ones_like(prefix))["kv"], prefix

    mine, my_prefix = kv_bytes(rank)
    ms_max, total = bench.reduce_over_ranks(10.0 + rank, float(mine), dist, "cpu")
    dist.barrier()
    expected = sum(kv_bytes(r)[0] for r in range(world))
    q.put((rank, ms_max, total, expected, my_prefix.tolist()))
    dist.destroy_process_group()


def test_two_ranks_shard_by_sequence_and_reduce():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms_max, total, expected, _ in res:
        assert ms_max == 11.0            # the slowest rank
        assert total == expected          # bytes of both ranks
    assert res[0][4] != res[1][4]         # every rank drew its own batch
    single = __import__("bench").reduce_over_ranks(3.0, 5.0, None, "cpu")
    assert single == (3.0, 5.0)
