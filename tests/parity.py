"""Shared helpers of the GPU parity tests: oracle problems and the step-by-step comparison of a
GPU swap trace with the fp64 oracle (re-basing the oracle at non-decisive steps).

Which oracle mode walks beside the GPU.  `strict` (every step re-solved from H and G with a fresh Cholesky
factorisation; nothing is carried from step to step) is the default and is used by every case whose strict step
takes under about a second: all reduced-size cases, the c1, c3, c4 and c6 layers at full size.  `lowrank` (the
oracle's own fp64 update identities) is used only for the full-size c2 and c5 layers, where one strict step costs
3 s and 30 s of host time; there the walk re-solves from scratch every `refactor_every` steps, compares the carried
state with the fresh one and continues from the fresh one.
"""
import contextlib

import numpy as np
import torch
from threadpoolctl import threadpool_limits

import workloads
from oracle import osscar_oracle as orc

GAP = 1e-5      # relative best-vs-second-best gap above which the oracle's choice is binding


def blas_threads(H, g):
    """Small problems run faster on one BLAS thread than on a pool that spins up for every tiny call; large layers
    use every core."""
    small = H.shape[0] <= 3000
    return threadpool_limits(1) if small else contextlib.nullcontext()


def assert_states_agree(a, b, tol=1e-8):
    """The carried low-rank state `a` against the freshly solved `b` (same support, same slot order)."""
    assert np.array_equal(a.S, b.S)
    assert rel_fro(a.Hinv, b.Hinv) < tol and rel_fro(a.V, b.V) < tol
    scale = np.linalg.norm(b.R) + 1e-300
    assert np.linalg.norm(a.R - b.R) / scale < tol
    assert abs(a.obj - b.obj) <= tol * abs(b.obj)
    for q, cq in b.c.items():
        assert np.allclose(a.c[q], cq, rtol=1e-6, atol=1e-9 * np.abs(cq).max())


def oracle_problem(wl):
    chunks = [c.float().numpy().astype(np.float64) for c in wl.x_chunks()]
    W = wl.weight().numpy().astype(np.float64)
    H, G, const = orc.gram_chunked(chunks, W, wl.damp)
    return chunks, W, H, G, const


def follow_trace(H, G, const, g, S0, swaps, gpu_obj, score_mode="independent", accept="improving",
                 mode="strict", max_swaps=None, gpu_stop=None, obj_rtol=1e-4, eps_acc=orc.EPS_ACC, refactor_every=25):
    """Walks the GPU's swap sequence with the oracle.  Returns (search, n_rebased).

    At each step the oracle proposes its swap from its own fp64 state.  If the GPU made the same
    swap, fine.  Otherwise the step must be non-decisive for the oracle (runner-up within GAP) and
    the GPU's choice must itself be within GAP of the oracle's best scores; the oracle is then moved
    to the GPU's support and the walk continues.  The running objective must agree throughout.
    """
    with blas_threads(np.asarray(H), g):
        return _follow_trace(H, G, const, g, S0, swaps, gpu_obj, score_mode, accept, mode, max_swaps, gpu_stop, obj_rtol,
                             eps_acc, refactor_every)


def _follow_trace(H, G, const, g, S0, swaps, gpu_obj, score_mode, accept, mode, max_swaps, gpu_stop, obj_rtol, eps_acc,
                  refactor_every):
    # the oracle's own periodic re-factorisation is switched off: the walk does it below and checks the carried state
    srch = orc.Search(H, G, const, g, S0, mode=mode, score_mode=score_mode, accept=accept, eps_acc=eps_acc,
                      refactor_every=1 << 30)
    rebased = 0
    assert gpu_obj[0] == __import__("pytest").approx(srch.st.obj, rel=obj_rtol)
    for step, (i_out, j_in) in enumerate(swaps):
        if mode == "lowrank" and step > 0 and step % refactor_every == 0:
            fresh = orc.fresh_state(srch.H, srch.G, srch.const, srch.st.S, g)
            assert_states_agree(srch.st, fresh)
            srch.st = fresh
        info = srch.propose(keep_scores=True)
        assert info is not None, f"step {step}: oracle has no candidate"
        slot = int(np.nonzero(srch.st.S == i_out)[0][0]) if i_out in srch.st.S else None
        assert slot is not None and j_in in srch.st.c, f"step {step}: GPU swap ({i_out},{j_in}) not possible"
        if (info.i_out, info.j_in) != (i_out, j_in):
            if score_mode == "independent":
                Dbest, Abest = info.D[info.slot], info.A[info.j_in]
                ok_out = info.D[slot] <= Dbest * (1 + GAP) + 1e-300
                ok_in = info.A[j_in] >= Abest * (1 - GAP) - 1e-300
                assert ok_out and ok_in, (
                    f"step {step}: GPU ({i_out},{j_in}) vs oracle ({info.i_out},{info.j_in}); "
                    f"D {info.D[slot]:.9g} vs {Dbest:.9g}, A {info.A[j_in]:.9g} vs {Abest:.9g}")
            else:
                pruned = np.array(sorted(srch.st.c.keys()))
                dgpu = info.pair_delta[slot, int(np.nonzero(pruned == j_in)[0][0])]
                assert abs(dgpu - info.delta) <= GAP * abs(info.delta), f"step {step}: pair not admissible"
            rebased += 1
            delta = srch.exact_delta(slot, j_in) if mode == "strict" else orc.swap_delta_closed_form(srch.H, srch.st, g, slot, j_in)
        else:
            delta = info.delta
        if accept == "improving":
            # the GPU accepted this swap: the oracle must agree unless the margin is tiny
            # (delta is a difference of two scores, each known to about GAP relative: that sets the tie band)
            thr = -srch.eps_acc * srch.st.obj
            band = GAP * (abs(info.D[slot]) + abs(info.D[slot] - delta)) if info.D is not None else GAP * srch.st.obj
            assert delta <= thr or abs(delta - thr) <= band, f"step {step}: accepted a non-improving swap"
        srch.apply(slot, j_in)
        assert gpu_obj[step + 1] == __import__("pytest").approx(srch.st.obj, rel=obj_rtol), f"step {step}: objective drifted"
    if mode == "lowrank" and len(swaps) > 0:      # the carried state at the end of the walk, against a fresh solve
        fresh = orc.fresh_state(srch.H, srch.G, srch.const, srch.st.S, g)
        assert_states_agree(srch.st, fresh)
        srch.st = fresh
    # after the GPU's last swap: it either hit max_swaps or stopped because the next swap did not improve
    if gpu_stop == "no_improvement":
        info = srch.propose(keep_scores=True)
        if info is not None and info.accepted:
            near_tie = info.gap_out <= GAP or info.gap_in <= GAP
            Dsel = info.D[info.slot] if info.D is not None else srch.st.obj
            band = GAP * (abs(Dsel) + abs(Dsel - info.delta))
            assert abs(info.delta + srch.eps_acc * srch.st.obj) <= band or near_tie, \
                f"GPU stopped but the oracle would go on (delta {info.delta}, obj {srch.st.obj})"
    elif gpu_stop == "max_swaps":
        assert len(swaps) == max_swaps
    return srch, rebased


def follow_block(H, G, const, g, S0, s, swaps, gpu_obj, accept="improving", gpu_stop=None, max_iters=None,
                 obj_rtol=1e-4, eps_acc=orc.EPS_ACC):
    """Walks the GPU's block exchanges (s pairs per iteration) with the oracle.  Per iteration the groups the GPU took
    out must be the s cheapest drops and the groups it brought in the s best adds by the oracle's fresh scores, up
    to ties within GAP at the cut; the oracle then makes the GPU's exchange and the objectives must agree."""
    import pytest
    with blas_threads(np.asarray(H), g):
        return _follow_block(H, G, const, g, S0, s, swaps, gpu_obj, accept, gpu_stop, max_iters, obj_rtol, eps_acc)


def _follow_block(H, G, const, g, S0, s, swaps, gpu_obj, accept, gpu_stop, max_iters, obj_rtol, eps_acc):
    import pytest
    srch = orc.BlockSearch(H, G, const, g, S0, s, accept=accept, eps_acc=eps_acc)
    assert gpu_obj[0] == pytest.approx(srch.st.obj, rel=obj_rtol)
    assert len(swaps) % s == 0 and len(gpu_obj) == len(swaps) // s + 1
    for it in range(len(swaps) // s):
        out = [o for o, _ in swaps[it * s:(it + 1) * s]]
        inn = [i for _, i in swaps[it * s:(it + 1) * s]]
        info = srch.propose()
        assert info is not None, f"iteration {it}: oracle has no candidate"
        assert len(set(out)) == s and len(set(inn)) == s, f"iteration {it}: repeated group"
        S = srch.st.S
        assert all(o in S for o in out) and all(i in srch.st.c for i in inn), f"iteration {it}: impossible exchange"
        slots = [int(np.nonzero(S == o)[0][0]) for o in out]
        thrD = np.sort(info.D)[s - 1]
        finiteA = info.A[np.isfinite(info.A)]
        thrA = np.sort(finiteA)[::-1][s - 1]
        for sl in slots:
            assert info.D[sl] <= thrD * (1 + GAP) + 1e-300, f"iteration {it}: group {S[sl]} is not among the {s} cheapest"
        for sl in range(len(S)):
            if sl not in slots:
                assert info.D[sl] >= thrD * (1 - GAP) - 1e-300, f"iteration {it}: kept group {S[sl]} is cheaper than a dropped one"
        for q in inn:
            assert info.A[q] >= thrA * (1 - GAP) - 1e-300, f"iteration {it}: group {q} is not among the {s} best adds"
        for q in srch.st.c:
            if q not in inn and np.isfinite(info.A[q]):
                assert info.A[q] <= thrA * (1 + GAP) + 1e-300, f"iteration {it}: pruned group {q} beats an added one"
        same = sorted(out) == sorted(info.out) and sorted(inn) == sorted(info.inn)
        delta = info.delta if same else srch.exchange_delta(slots, inn)
        if accept == "improving":
            thr = -srch.eps_acc * srch.st.obj
            Dsum = float(np.sum(info.D[slots]))
            band = GAP * (abs(Dsum) + abs(Dsum - delta))
            assert delta <= thr or abs(delta - thr) <= band, f"iteration {it}: accepted a non-improving exchange"
        srch.apply(slots, inn)
        assert gpu_obj[it + 1] == pytest.approx(srch.st.obj, rel=obj_rtol), f"iteration {it}: objective drifted"
    if gpu_stop == "no_improvement":
        info = srch.propose()
        if info is not None and info.accepted:
            Dsum = float(np.sum(info.D[info.slots]))
            band = GAP * (abs(Dsum) + abs(Dsum - info.delta))
            sD = np.sort(info.D); sA = np.sort(info.A[np.isfinite(info.A)])[::-1]
            tie = (len(sD) > s and sD[s] - sD[s - 1] <= GAP * abs(sD[s - 1])) or \
                  (len(sA) > s and sA[s - 1] - sA[s] <= GAP * abs(sA[s - 1]))
            assert abs(info.delta + srch.eps_acc * srch.st.obj) <= band or tie, \
                f"GPU stopped but the oracle would go on (delta {info.delta}, obj {srch.st.obj})"
    elif gpu_stop == "max_swaps":
        assert len(swaps) // s == max_iters
    return srch


def rel_fro(a, b):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def follow_greedy(H, G, const, g, k, t_hat, drops):
    """Walks the GPU's nested (greedy) phase with the oracle: per iteration the groups the GPU pruned must be the
    t cheapest by the oracle's fresh scores, up to ties within GAP; the oracle then continues from the GPU's set."""
    import scipy.linalg as sla
    ng = H.shape[0] // g
    S = np.arange(ng)
    pos = 0
    while len(S) > k:
        t = min(t_hat, len(S) - k)
        I = orc.rows_of(S, g)
        L = sla.cho_factor(H[np.ix_(I, I)], lower=True, check_finite=False)
        Hinv = sla.cho_solve(L, np.eye(len(I)), check_finite=False)
        V = sla.cho_solve(L, G[I], check_finite=False)
        D = orc.drop_scores(orc.State(S=S, Hinv=0.5 * (Hinv + Hinv.T), V=V, R=None, c={}, obj=0.0), g)
        out = [int(q) for q in drops[pos:pos + t]]
        assert len(set(out)) == t and all(q in S for q in out), f"iteration at {pos}: bad drop set {out}"
        thr = np.sort(D)[t - 1]
        idx = {int(q): i for i, q in enumerate(S)}
        for q in out:
            assert D[idx[q]] <= thr * (1 + GAP) + 1e-300, f"pruned group {q} is not among the {t} cheapest"
        for q in S:
            if int(q) not in out:
                assert D[idx[int(q)]] >= thr * (1 - GAP) - 1e-300, f"group {q} is cheaper than the pruned ones"
        keep = np.array([q for q in S if int(q) not in set(out)])
        S = keep
        pos += t
    return np.sort(S)
