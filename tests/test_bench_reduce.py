"""The multi-rank reduction of bench.py (max of times, sum of counts), on CPU with gloo and two ranks."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    out = bench.reduce_over_ranks({"max_total_ms": 10.0 + 5 * rank, "sum_swaps": 100 + rank, "max_search_ms": 3.0 - rank},
                                  world, torch.device("cpu"))
    q.put((rank, out))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_reduction():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(2):
        assert got[r] == {"max_total_ms": 15.0, "sum_swaps": 201.0, "max_search_ms": 3.0}


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    vals = {"max_total_ms": 1.5, "sum_swaps": 7}
    assert bench.reduce_over_ranks(vals, 1, torch.device("cpu")) == vals
    assert bench.swap_bytes(8602, 20070, 7168) == 3222668576
    # fused y pass, inverse kept in fp64: 16 n_I^2 instead of 12 n_I^2
    assert bench.swap_bytes(8602, 20070, 7168, True) == 3222668576 + 4 * 8602 * 8602
