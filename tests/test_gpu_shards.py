"""Column-sharded swap search and token-split Gram, proved on ONE device: two contexts in one process, each with half of
the output columns and half of the token chunks, one host thread and one stream per shard.  The reduce hook that an
NCCL all-reduce fills on several devices is replaced by a device-side add of the two shards' buffers, ordered with
stream events (no kernel ever waits for another kernel).  The sharded walk must follow the strict oracle of the whole
layer under the usual tie protocol, both shards must report identical traces, and the columns they return must put
together the oracle's weights.
"""
import threading

import numpy as np
import pytest
import torch

import workloads
from oracle import osscar_oracle as orc
from tests.parity import follow_trace, oracle_problem, rel_fro

pytestmark = pytest.mark.gpu


class LocalExchange:
    """In-place sum of one buffer per shard, all on one device; every shard calls `reduce` from its own host thread
    with its own stream current.  The sum is taken in shard order by everyone, so all shards get the same bits."""

    def __init__(self, n, max_elems, device):
        self.n = n
        self.host = threading.Barrier(n)
        self.slots = {torch.float32: [torch.empty(max_elems, dtype=torch.float32, device=device) for _ in range(n)],
                      torch.float64: [torch.empty(max_elems, dtype=torch.float64, device=device) for _ in range(n)]}
        self.written = [torch.cuda.Event() for _ in range(n)]
        self.read = [torch.cuda.Event() for _ in range(n)]
        self.rounds = 0

    def reduce(self, rank, view):
        stream = torch.cuda.current_stream()
        flat = view.reshape(-1)
        n_el = flat.numel()
        for j in range(self.n):                      # nobody still reads my slot from the previous round
            if j != rank:
                stream.wait_event(self.read[j])
        slot = self.slots[flat.dtype][rank]
        slot[:n_el].copy_(flat)
        self.written[rank].record(stream)
        self.host.wait()                             # every shard has enqueued its copy and recorded its event
        for j in range(self.n):
            if j != rank:
                stream.wait_event(self.written[j])
        total = self.slots[flat.dtype][0][:n_el].clone()
        for j in range(1, self.n):
            total += self.slots[flat.dtype][j][:n_el]
        flat.copy_(total)
        self.read[rank].record(stream)
        self.host.wait()                             # the read events exist before anyone's next round waits on them


def run_shards(pkg, wl, n_shards, max_swaps, accept_always=False, refresh_every=0):
    from paper_2403_12983_b200 import sharding
    b = pkg.binding
    dev = torch.device("cuda", 0)
    chunks = [c.cuda() for c in wl.x_chunks()]
    W = wl.weight().cuda()
    ex = LocalExchange(n_shards, wl.d1 * wl.d1, dev)
    results, errors = [None] * n_shards, []

    def work(rank):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream(dev)
            with torch.cuda.stream(stream):
                solver = pkg.Solver(0, stream=stream)
                c0, c1 = sharding.column_range(wl.m, rank, n_shards)
                mine = [chunks[i] for i in sharding.chunk_indices(len(chunks), rank, n_shards)]
                for c in mine:
                    c.record_stream(stream)
                W_local = W[:, c0:c1].contiguous()
                res = sharding.solve_layer_sharded(
                    solver, mine, W_local, wl.d1, wl.g, wl.k, max_swaps,
                    reduce_hook=lambda view, sptr: ex.reduce(rank, view), reduce_H=lambda H: ex.reduce(rank, H),
                    damp=wl.damp, accept_mode=b.ACCEPT_ALWAYS if accept_always else b.ACCEPT_IMPROVING,
                    accept_rel_tol=wl.eps_acc, refresh_every=refresh_every)
                stream.synchronize()
                results[rank] = (res, (c0, c1))
                solver.close()
        except Exception as exc:                     # a failed shard must not leave the other one at the barrier
            errors.append(exc)
            ex.host.abort()

    torch.cuda.synchronize()
    threads = [threading.Thread(target=work, args=(r,)) for r in range(n_shards)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    if errors:
        raise errors[0]
    return results


@pytest.mark.parametrize("name,over,seed,max_swaps,always,refresh", [
    ("c2", dict(n=6144, d1=520, m=150, k=207, chunk_rows=2048), 0, 60, False, 0),       # 3 chunks, 75 columns per shard
    ("c5", dict(n=8192, d1=1000, m=301, k=300, chunk_rows=2048), 1, 40, True, 0),       # odd column count: 151 + 150
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 2, 30, True, 12),       # one chunk (one shard has none), refresh
])
def test_two_column_shards_follow_the_oracle(name, over, seed, max_swaps, always, refresh):
    import paper_2403_12983_b200 as pkg
    wl = workloads.config(name, seed=seed, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    results = run_shards(pkg, wl, 2, max_swaps, accept_always=always, refresh_every=refresh)
    (r0, (a0, a1)), (r1, (b0, b1)) = results
    assert (a0, a1, b0, b1) == (0, (wl.m + 1) // 2, (wl.m + 1) // 2, wl.m)
    # both shards hold the same Gram (sum of their token shares), the same kept set and the same traces
    assert torch.equal(r0.H, r1.H)
    scale = np.sqrt(np.outer(np.diag(H64), np.diag(H64)))
    assert np.max(np.abs(r0.H.cpu().numpy() - H64) / scale) < 5e-6
    assert torch.equal(r0.support, r1.support) and torch.equal(r0.swap_trace, r1.swap_trace)
    assert torch.equal(r0.obj_trace, r1.obj_trace) and r0.obj_final == r1.obj_final and r0.n_swaps == r1.n_swaps
    if always:
        assert r0.n_swaps == max_swaps
    # the walk against the strict oracle of the whole layer (fed the device's H and the two halves of G)
    Hr = r0.H.cpu().numpy().astype(np.float64)
    Gr = np.concatenate([r0.G.cpu().numpy(), r1.G.cpu().numpy()], axis=1).astype(np.float64)
    const_r = float(np.sum(W * Gr))
    assert r0.const_term + r1.const_term == pytest.approx(const_r, rel=1e-9)
    S0, _ = orc.init_support(Hr, W, wl.g, wl.k)
    swaps = [tuple(int(v) for v in r) for r in r0.swap_trace.cpu().numpy()]
    srch, _ = follow_trace(Hr, Gr, const_r, wl.g, S0, swaps, r0.obj_trace.cpu().numpy(), accept="always" if always else "improving",
                           gpu_stop=r0.stop_reason, max_swaps=max_swaps, eps_acc=wl.eps_acc)
    S_or, W_or, _, _ = srch.result()
    assert np.array_equal(r0.support.cpu().numpy(), S_or)
    assert r0.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    Wg = np.concatenate([r0.W.cpu().numpy(), r1.W.cpu().numpy()], axis=1)
    assert rel_fro(Wg, W_or) < 1e-3


def test_shard_mode_rejects_what_it_does_not_cover():
    import paper_2403_12983_b200 as pkg
    b = pkg.binding
    wl = workloads.config("c4", n=49 * 20, d1=9 * 30, m=40, k=10, chunk_rows=49 * 20)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    solver = pkg.Solver()
    H, G, Wd = (torch.as_tensor(x, dtype=torch.float32).cuda() for x in (H64, G64, W))
    solver.ensure_workspace(wl.d1, wl.m, wl.g, wl.k)
    solver.set_shard_reduce(lambda view, sptr: None)
    with pytest.raises(pkg.OsscarError) as ei:
        solver.init_support(H, G, Wd, wl.g, wl.k)              # groups of nine rows
    assert ei.value.status == b.E_ARG
    solver.set_shard_reduce(None)
    solver.init_support(H, G, Wd, wl.g, wl.k)
    solver.close()
