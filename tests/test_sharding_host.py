"""Host side of the multi-device layer solve, on CPU: how columns and token chunks are dealt to ranks, and the reduce
hook over torch.distributed with two gloo ranks (the device kernels it serves are covered by the GPU tests)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def test_columns_and_chunks_tile_the_layer():
    from paper_2403_12983_b200 import sharding
    for m, world in [(7168, 8), (301, 2), (5, 8), (2048, 3)]:
        ranges = [sharding.column_range(m, r, world) for r in range(world)]
        assert ranges[0][0] == 0 and ranges[-1][1] == m
        assert all(ranges[r][1] == ranges[r + 1][0] for r in range(world - 1))             # contiguous, no gap, no overlap
        sizes = [b - a for a, b in ranges]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    for n_chunks, world in [(16, 8), (16, 3), (1, 2), (5, 4)]:
        owned = [list(sharding.chunk_indices(n_chunks, r, world)) for r in range(world)]
        assert sorted(i for o in owned for i in o) == list(range(n_chunks))                # every chunk exactly once
        assert max(len(o) for o in owned) - min(len(o) for o in owned) <= 1


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2403_12983_b200 import sharding
    hook = sharding.dist_reduce_hook()
    # what the library hands to the hook: a view into the workspace holding this rank's partial sums
    ws = torch.zeros(64, dtype=torch.uint8)
    norms = ws[8:8 + 4 * 6].view(torch.float32)
    norms.copy_(torch.arange(6, dtype=torch.float32) * (rank + 1))
    scalar = ws[40:48].view(torch.float64)
    scalar.fill_(0.25 + rank)
    hook(norms, 0)
    hook(scalar, 0)
    q.put((rank, norms.tolist(), scalar.item(), ws[:8].tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_reduce_hook_sums_views_in_place_over_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, norms, scalar, head in got:
        assert norms == [0.0, 3.0, 6.0, 9.0, 12.0, 15.0] and scalar == 1.5 and head == [0] * 8
