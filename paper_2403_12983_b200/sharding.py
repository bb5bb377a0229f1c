"""One layer solved by several devices: calibration tokens split for the Gram, output columns split for the search.

The columns of W_hat are independent given the kept set (Section 2, convolutional-layer paragraph), so rank r keeps
columns [c0, c1) of W_hat, G, the optimal weights V and the residual R -- the matrices that dominate the traffic of a
swap -- while the kept set, (H_II)^-1, H and the Schur complements are replicated.  What a decision needs from all
columns (group energies, row norms of V and R, the cross term of the chosen pair, the objective) is summed over ranks
by a hook that the library calls in stream order (include/osscar.h, osscar_set_shard_reduce): here an NCCL all-reduce
through torch.distributed.  H itself is the sum over token chunks (Appendix B.1: H is accumulated segment by segment),
so every rank accumulates the chunks it owns and one all-reduce of H follows.

Only argument marshalling and torch.distributed plumbing live here; all arithmetic runs in libosscar's kernels.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch

from . import binding as b
from .pipeline import LayerResult


def column_range(m: int, rank: int, world: int) -> Tuple[int, int]:
    """Columns [c0, c1) of rank `rank`: contiguous, sizes differ by at most one, earlier ranks take the remainder."""
    base, rem = divmod(m, world)
    c0 = rank * base + min(rank, rem)
    return c0, c0 + base + (1 if rank < rem else 0)


def chunk_indices(n_chunks: int, rank: int, world: int) -> range:
    """Token chunks of rank `rank`: every world-th chunk, so that ranks finish their Gram share together."""
    return range(rank, n_chunks, world)


def dist_reduce_hook(group=None):
    """Hook for Solver.set_shard_reduce: in-place sum over the ranks of `group` on the current stream."""
    import torch.distributed as dist

    def hook(view: torch.Tensor, stream_ptr: int):
        dist.all_reduce(view, op=dist.ReduceOp.SUM, group=group)
    return hook


def solve_layer_sharded(solver: b.Solver, x_chunks_local: Sequence[torch.Tensor], W_local: torch.Tensor, d1: int, g: int, k: int,
                        max_swaps: int, reduce_hook, reduce_H, damp: float = 0.0, init_mode: int = b.INIT_ENERGY,
                        accept_mode: int = b.ACCEPT_IMPROVING, accept_rel_tol: float = -1.0, refresh_every: int = 0,
                        H: Optional[torch.Tensor] = None) -> LayerResult:
    """This rank's part of one layer solve.

    x_chunks_local: the token chunks this rank owns (device tensors, possibly none); W_local: d1 x m_local fp32, this
    rank's columns of W_hat.  reduce_hook: see Solver.set_shard_reduce.  reduce_H(H): in-place sum of the d1 x d1 fp32
    Gram over ranks, on the current stream (e.g. torch.distributed.all_reduce).  Every rank returns the same support,
    traces and (whole-layer) objectives; LayerResult.W holds this rank's columns.
    """
    if g != 1:
        raise ValueError("column shards support single-row groups")
    dev = torch.device("cuda", solver.device)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
    m_local = W_local.shape[1]
    solver.ensure_workspace(d1, m_local, g, k)
    ev[0].record()
    if H is None:
        H = torch.zeros(d1, d1, dtype=torch.float32, device=dev)
    else:
        H.zero_()
    G = torch.empty(d1, m_local, dtype=torch.float32, device=dev)
    empty = torch.empty(0, d1, dtype=x_chunks_local[0].dtype if len(x_chunks_local) else torch.bfloat16, device=dev)
    if len(x_chunks_local) == 0:
        solver.gram_chunk(empty, H, b.GRAM_BEGIN)
    for c, Xc in enumerate(x_chunks_local):
        solver.gram_chunk(Xc, H, b.GRAM_BEGIN if c == 0 else 0)
    reduce_H(H)                                   # upper-triangle tiles of every rank's share; END mirrors the sum
    ev[1].record()
    const_local = solver.gram_chunk(empty, H, b.GRAM_END, W_local, G, damp)
    ev[2].record()
    solver.set_shard_reduce(reduce_hook)
    try:
        support0, obj0 = solver.init_support(H, G, W_local, g, k, init_mode)
        ev[3].record()
        out = solver.local_search(max_swaps, b.SCORE_INDEPENDENT, accept_mode, refresh_every, accept_rel_tol=accept_rel_tol,
                                  loop_mode=b.LOOP_LAUNCHES)
    finally:
        solver.set_shard_reduce(None)
    ev[4].record()
    ev[4].synchronize()
    ms = {n: ev[i].elapsed_time(ev[i + 1]) for i, n in enumerate(["gram", "gram_end", "init", "search"])}
    ms["search_loop"] = out.ms_search
    res = LayerResult(out.support, out.W, out.obj_trace, out.swap_trace, out.n_swaps, out.stop_reason,
                      out.obj_init, out.obj_final, const_local, ms, out.ms_kernel, H, G)
    res.loop_driver = out.loop_driver
    res.io = {"h2d": 0, "d2h": 0}
    return res
