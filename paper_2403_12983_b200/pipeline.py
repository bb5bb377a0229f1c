"""Whole per-layer solve as one call: Gram over token chunks -> starting support -> swap search.

`solve_layer` is the call a user makes.  Chunks of X may live on the device or in (pinned) host
memory; host chunks are copied on a side stream into two device staging buffers so that the copy of
chunk c+1 overlaps the Gram kernel of chunk c.  All arithmetic runs in libosscar's kernels.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional, Sequence

import torch

from . import binding as b


@dataclass
class LayerResult:
    support: torch.Tensor
    W: torch.Tensor
    obj_trace: torch.Tensor
    swap_trace: torch.Tensor
    n_swaps: int
    stop_reason: str
    obj_init: float
    obj_final: float
    const_term: float
    ms: dict                 # device milliseconds per phase: gram, gram_end, init, search
    ms_kernel: dict
    H: torch.Tensor
    G: torch.Tensor


def _gram_stream_host(solver: b.Solver, chunks: Sequence[torch.Tensor], H, dev):
    """H = sum_c Xc^T Xc with Xc read from host memory through two staging buffers."""
    main = torch.cuda.current_stream(dev)
    copy = getattr(solver, "_copy_stream", None)
    if copy is None:
        copy = solver._copy_stream = torch.cuda.Stream(dev)
    rows = max(c.shape[0] for c in chunks)
    d1 = chunks[0].shape[1]
    stage = getattr(solver, "_stage", None)
    if stage is None or stage[0].shape[0] < rows or stage[0].shape[1] != d1 or stage[0].dtype != chunks[0].dtype:
        stage = solver._stage = [torch.empty(rows, d1, dtype=chunks[0].dtype, device=dev) for _ in range(2)]
    copied = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]
    nbytes = 0
    for c, Xc in enumerate(chunks):
        s = c & 1
        with torch.cuda.stream(copy):
            if c >= 2:
                copy.wait_event(consumed[s])
            stage[s][:Xc.shape[0]].copy_(Xc, non_blocking=True)
            copied[s].record(copy)
        nbytes += Xc.numel() * Xc.element_size()
        main.wait_event(copied[s])
        solver.gram_chunk(stage[s][:Xc.shape[0]], H, b.GRAM_BEGIN if c == 0 else 0)
        consumed[s].record(main)
    return nbytes


def solve_layer(solver: b.Solver, x_chunks: Sequence[torch.Tensor], W: torch.Tensor, g: int, k: int,
                max_swaps: int, damp: float = 0.0, init_mode: int = b.INIT_ENERGY,
                score_mode: int = b.SCORE_INDEPENDENT, accept_mode: int = b.ACCEPT_IMPROVING,
                refresh_every: int = 0, profile_samples: int = 0, accept_rel_tol: float = -1.0,
                H: Optional[torch.Tensor] = None, G: Optional[torch.Tensor] = None,
                greedy_t_hat: int = 0, block_pairs: int = 0, loop_mode: int = b.LOOP_AUTO) -> LayerResult:
    """Prunes one layer to k groups of g rows.  W: d1 x m fp32 (device or host); x_chunks: row blocks of X
    (bf16 or fp32; all on the device, or all on the host).  block_pairs > 1 exchanges that many groups per iteration.  greedy_t_hat > 0 starts from the nested phase with
    that many groups pruned per iteration instead of the energy ranking."""
    dev = torch.device("cuda", solver.device)
    host_x = not x_chunks[0].is_cuda
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
    io = {"h2d": 0, "d2h": 0}
    ev[0].record()
    if not W.is_cuda:
        io["h2d"] += W.numel() * 4
        W = W.to(dev, non_blocking=True)
    d1, m = W.shape
    solver.ensure_workspace(d1, m, g, k)          # also lets the cross term G = H W run on the tensor cores
    if H is None:
        H = torch.empty(d1, d1, dtype=torch.float32, device=dev)
    if G is None:
        G = torch.empty(d1, m, dtype=torch.float32, device=dev)
    if host_x:
        io["h2d"] += _gram_stream_host(solver, x_chunks, H, dev)
    else:
        for c, Xc in enumerate(x_chunks):
            solver.gram_chunk(Xc, H, b.GRAM_BEGIN if c == 0 else 0)
    ev[1].record()
    const = solver.gram_chunk(x_chunks[0][:0] if not host_x else solver._stage[0][:0], H, b.GRAM_END, W, G, damp)
    ev[2].record()
    if greedy_t_hat > 0:          # the paper's own start: nested phase of Algorithm 1 from the dense layer
        support0, _, obj0, _ = solver.init_support_greedy(H, G, W, g, k, greedy_t_hat)
    else:
        support0, obj0 = solver.init_support(H, G, W, g, k, init_mode)
    ev[3].record()
    out = solver.local_search(max_swaps, score_mode, accept_mode, refresh_every, accept_rel_tol=accept_rel_tol,
                              profile_samples=profile_samples, block_pairs=block_pairs, loop_mode=loop_mode)
    ev[4].record()
    ev[4].synchronize()
    names = ["gram", "gram_end", "init", "search"]
    ms = {n: ev[i].elapsed_time(ev[i + 1]) for i, n in enumerate(names)}
    ms["search_loop"] = out.ms_search
    res = LayerResult(out.support, out.W, out.obj_trace, out.swap_trace, out.n_swaps, out.stop_reason,
                      out.obj_init, out.obj_final, const, ms, out.ms_kernel, H, G)
    res.io = io
    res.loop_driver = out.loop_driver
    return res


def result_to_host(res: LayerResult, pinned: Optional[dict] = None) -> dict:
    """Device -> host read of a layer's result (weights, support, traces); returns tensors and the byte count."""
    out, nbytes = {}, 0
    for name in ("W", "support", "obj_trace", "swap_trace"):
        t = getattr(res, name)
        if pinned is not None and name in pinned and pinned[name].numel() >= t.numel():
            dst = pinned[name].view(-1)[:t.numel()].view(t.shape)
            dst.copy_(t, non_blocking=True)
        else:
            dst = t.to("cpu", non_blocking=False)
        out[name] = dst
        nbytes += t.numel() * t.element_size()
    torch.cuda.current_stream().synchronize()
    out["bytes"] = nbytes
    return out
