"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests calls the oracle to check itself: every expected value comes from the
definition of the quantity (least squares on X, enumeration of supports, numpy.linalg.inv,
closed forms for orthogonal columns), so a dropped term, a wrong sign or a transposed operand
in the oracle fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest

import workloads
from oracle import osscar_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def problem(wl):
    X = wl.x_full().float().numpy().astype(np.float64)
    W = wl.weight().numpy().astype(np.float64)
    H, G, const = orc.gram(X, W, wl.damp)
    return X, W, H, G, const


# ----------------------------------------------------------------------------- Gram (Section 2)
def test_gram_definition_and_symmetry():
    wl = workloads.config("c1")
    X, W, H, G, const = problem(wl)
    assert np.allclose(H, H.T, rtol=0, atol=1e-12 * np.abs(H).max())
    # H_ii is the squared norm of column i; H_ij the inner product of columns i and j
    for i, j in [(0, 0), (3, 17), (63, 5)]:
        assert H[i, j] == pytest.approx(float(np.dot(X[:, i], X[:, j])), rel=1e-12)
    # G = X^T (X W_hat) and const = ||X W_hat||_F^2
    Y = X @ W
    assert np.allclose(G, X.T @ Y, rtol=1e-11, atol=1e-9)
    assert const == pytest.approx(float(np.sum(Y * Y)), rel=1e-12)
    # quadratic form of a Gram matrix is non-negative
    rng = np.random.default_rng(0)
    for _ in range(5):
        v = rng.standard_normal(H.shape[0])
        assert v @ H @ v >= 0


def test_gram_chunked_equals_whole_and_damping():
    wl = workloads.config("c2", n=600, d1=48, m=8, k=24, chunk_rows=256)
    W = wl.weight().numpy()
    chunks = [c.float().numpy() for c in wl.x_chunks()]
    assert [c.shape[0] for c in chunks] == [256, 256, 88]
    Hc, Gc, cc = orc.gram_chunked(chunks, W, damp=0.0)
    H, G, c0 = orc.gram(np.concatenate(chunks), W, damp=0.0)
    assert np.allclose(Hc, H, rtol=1e-12) and np.allclose(Gc, G, rtol=1e-10, atol=1e-9)
    Hd, Gd, cd = orc.gram(np.concatenate(chunks), W, damp=0.05)
    lam = 0.05 * np.trace(H) / H.shape[0]
    assert np.allclose(Hd - H, lam * np.eye(48), atol=1e-9 * lam)
    assert np.allclose(Gd, Hd @ W.astype(np.float64), rtol=1e-12)


# ----------------------------------------------------------------------------- f(S) (Eq. deff / Eq. optf)
@pytest.mark.parametrize("g,p,k", [(1, 12, 6), (3, 6, 3)])
def test_closed_form_objective_equals_least_squares_for_every_support(g, p, k):
    """Eq. optf against the definition Eq. deff: enumerate all supports (p=12, k=6 -> 924)."""
    wl = workloads.tiny(p=p, m=4, g=g, k=k, n=50, seed=3)
    X, W, H, G, const = problem(wl)
    bf = orc.brute_force(H, G, const, g, k)
    assert len(bf) == math.comb(p, k)
    for S, obj in bf.items():
        W_ls, obj_ls = orc.solve_support_lstsq(X, W, S, g)
        assert obj == pytest.approx(obj_ls, rel=1e-9, abs=1e-9)
        W_cf, _ = orc.solve_support(H, G, const, S, g)
        assert np.allclose(W_cf, W_ls, rtol=1e-7, atol=1e-9)
        # pruned rows are exactly zero and the quadratic form agrees with the X-space error
        I = orc.rows_of(S, g)
        mask = np.ones(p * g, bool)
        mask[I] = False
        assert np.all(W_cf[mask] == 0)
        assert orc.objective_quadratic(H, W, W_cf) == pytest.approx(orc.objective_from_X(X, W, W_cf), rel=1e-9)


def test_enumerator_count_matches_paper_example():
    """Section 3.1: C(32, 16), the supports that keep half of 32 channels, exceeds the bound the paper prints."""
    with open(os.path.join(GOLDEN, "paper_support_count.txt")) as fh:
        rows = [l.split() for l in fh if l.strip() and not l.startswith("#")]
    (p, k, lower_bound), = [(int(a), int(b), int(c)) for a, b, c in rows]
    assert math.comb(p, k) > lower_bound
    assert sum(1 for _ in itertools.combinations(range(12), 6)) == 924


def test_full_support_reproduces_dense_weight():
    wl = workloads.tiny(p=10, m=3, g=2, k=10, n=60)
    X, W, H, G, const = problem(wl)
    W_all, obj = orc.solve_support(H, G, const, range(10), 2)
    assert np.allclose(W_all, W, atol=1e-9)
    assert abs(obj) < 1e-8 * const


def test_sign_of_linear_term():
    """L(W) = 1/2 Tr(W^T H W) - Tr(G^T W) (Eq. MIQP): its minimiser over all W is W_hat itself."""
    wl = workloads.tiny(p=8, m=3, g=1, k=8, n=40)
    X, W, H, G, const = problem(wl)
    W_min = np.linalg.solve(H, G)           # stationary point of the minus-sign form
    assert np.allclose(W_min, W, atol=1e-9)
    # with a plus sign the stationary point would be -W_hat, whose reconstruction error is 4 * const
    assert orc.objective_from_X(X, W, -W_min) == pytest.approx(4 * const, rel=1e-9)


def test_residual_identity():
    """obj(S) = Tr(W_hat_J^T R_J) with R = H (W_hat - W^(S)); R vanishes on kept rows."""
    wl = workloads.tiny(p=9, m=4, g=2, k=4, n=70, seed=5)
    X, W, H, G, const = problem(wl)
    S = np.array([1, 4, 6, 7])
    st = orc.fresh_state(H, G, const, S, 2)
    W_S, obj = orc.solve_support(H, G, const, S, 2)
    R_def = H @ (W - W_S)
    I = orc.rows_of(S, 2)
    assert np.abs(R_def[I]).max() < 1e-9 * np.abs(R_def).max()
    R_def[I] = 0
    assert np.allclose(st.R, R_def, atol=1e-9 * np.abs(R_def).max())
    assert float(np.sum(W * st.R)) == pytest.approx(obj, rel=1e-10)
    assert st.obj == pytest.approx(obj, rel=1e-12)


# ----------------------------------------------------------------------------- scores (Eq. impact)
@pytest.mark.parametrize("g", [1, 3])
def test_scores_equal_objective_differences(g):
    """Eq. impact by its definition: re-solve with the group removed / added."""
    p, k = 9, 4
    wl = workloads.tiny(p=p, m=5, g=g, k=k, n=80, seed=7)
    X, W, H, G, const = problem(wl)
    S = np.array([0, 3, 4, 8])
    st = orc.fresh_state(H, G, const, S, g)
    D = orc.drop_scores(st, g)
    A = orc.add_scores(st, g, p, H)
    obj_S = orc.solve_support_lstsq(X, W, S, g)[1]
    for s, i in enumerate(S):
        obj_less = orc.solve_support_lstsq(X, W, [x for x in S if x != i], g)[1]
        assert D[s] == pytest.approx(obj_less - obj_S, rel=1e-8)
        assert D[s] >= 0
    for q in range(p):
        if q in S:
            assert A[q] == -np.inf
        else:
            obj_more = orc.solve_support_lstsq(X, W, list(S) + [q], g)[1]
            assert A[q] == pytest.approx(obj_S - obj_more, rel=1e-8)
            assert A[q] >= 0


def test_single_row_drop_score_is_obs_saliency():
    """g = 1: the drop score is ||V_i||^2 / [H_II^-1]_ii, with the inverse from numpy.linalg.inv."""
    wl = workloads.config("c1")
    X, W, H, G, const = problem(wl)
    S, _ = orc.init_support(H, W, 1, 32)
    st = orc.fresh_state(H, G, const, S, 1)
    Hinv = np.linalg.inv(H[np.ix_(S, S)])
    V = Hinv @ G[S]
    expect = np.sum(V * V, axis=1) / np.diag(Hinv)
    assert np.allclose(orc.drop_scores(st, 1), expect, rtol=1e-9)


@pytest.mark.parametrize("g", [1, 2])
def test_swap_delta_closed_form_equals_fresh_difference(g):
    p, k = 8, 4
    wl = workloads.tiny(p=p, m=3, g=g, k=k, n=60, seed=11)
    X, W, H, G, const = problem(wl)
    S = np.array([1, 2, 5, 7])
    st = orc.fresh_state(H, G, const, S, g)
    obj_S = orc.solve_support_lstsq(X, W, S, g)[1]
    D = orc.drop_scores(st, g)
    A = orc.add_scores(st, g, p, H)
    interact = False
    for s in range(k):
        for q in set(range(p)) - set(S):
            S2 = S.copy()
            S2[s] = q
            expect = orc.solve_support_lstsq(X, W, S2, g)[1] - obj_S
            got = orc.swap_delta_closed_form(H, st, g, s, q)
            assert got == pytest.approx(expect, rel=1e-7, abs=1e-9 * obj_S)
            interact |= abs((D[s] - A[q]) - expect) > 1e-6 * obj_S
    assert interact     # the two moves interact: delta is not simply D - A


# ----------------------------------------------------------------------------- selection rule and search
def test_orthogonal_columns_closed_form():
    """X with orthogonal columns: H is diagonal, every score is H_ii ||W_i||^2, the energy
    support is optimal, so the search makes no swap and obj is the sum over pruned rows."""
    rng = np.random.default_rng(4)
    n, p, m, k = 40, 10, 3, 4
    Q, _ = np.linalg.qr(rng.standard_normal((n, p)))
    s = rng.uniform(0.5, 3.0, p)
    X = Q * s
    W = rng.standard_normal((p, m))
    H, G, const = orc.gram(X, W)
    e_expect = s ** 2 * np.sum(W * W, axis=1)
    S0, e = orc.init_support(H, W, 1, k)
    assert np.allclose(e, e_expect, rtol=1e-10)
    assert set(S0) == set(np.argsort(-e_expect)[:k])
    run = orc.Search(H, G, const, 1, S0).run(20)
    assert run.swap_trace == [] and run.stop_reason == "no_improvement"
    pruned = sorted(set(range(p)) - set(S0))
    assert run.obj_trace[0] == pytest.approx(float(np.sum(e_expect[pruned])), rel=1e-9)
    D, A = run.scores()
    assert np.allclose(D, e_expect[S0], rtol=1e-9)
    assert np.allclose(A[pruned], e_expect[pruned], rtol=1e-9)
    bf = orc.brute_force(H, G, const, 1, k)
    assert min(bf, key=bf.get) == tuple(S0)


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_search_is_monotone_and_bounded_by_brute_force(seed):
    wl = workloads.tiny(p=12, m=5, g=1, k=6, n=40, seed=seed)
    X, W, H, G, const = problem(wl)
    bf = orc.brute_force(H, G, const, 1, 6)
    best = min(bf.values())
    S0, _ = orc.init_support(H, W, 1, 6)
    run = orc.Search(H, G, const, 1, S0).run(50)
    S, W_out, obj, swaps = run.result()
    assert np.all(np.diff(obj) < 0)                      # every accepted swap lowers obj
    assert obj[-1] >= best - 1e-9 * best
    assert obj[-1] == pytest.approx(bf[tuple(S)], rel=1e-10)
    assert obj[0] == pytest.approx(bf[tuple(S0)], rel=1e-10)
    # each step took the cheapest group out and the most valuable group in, as re-solved from X
    Scur = list(S0)
    for (i_out, j_in), o_next in zip(swaps, obj[1:]):
        base = bf[tuple(sorted(Scur))]
        drop_cost = {i: orc.solve_support_lstsq(X, W, [x for x in Scur if x != i], 1)[1] - base for i in Scur}
        add_gain = {q: base - orc.solve_support_lstsq(X, W, Scur + [q], 1)[1]
                    for q in range(12) if q not in Scur}
        assert i_out == min(drop_cost, key=lambda i: (drop_cost[i], i))
        assert j_in == max(add_gain, key=lambda q: (add_gain[q], -q))
        Scur[Scur.index(i_out)] = j_in
        assert o_next == pytest.approx(bf[tuple(sorted(Scur))], rel=1e-10)


def test_pair_exact_picks_best_neighbour():
    g, p, k = 2, 8, 4
    wl = workloads.tiny(p=p, m=4, g=g, k=k, n=70, seed=2)
    X, W, H, G, const = problem(wl)
    bf = orc.brute_force(H, G, const, g, k)
    S0, _ = orc.init_support(H, W, g, k)
    srch = orc.Search(H, G, const, g, S0, score_mode="pair_exact")
    while True:
        info = srch.propose()
        Scur = sorted(srch.st.S)
        neigh = {}
        for i in Scur:
            for q in set(range(p)) - set(Scur):
                neigh[(i, q)] = bf[tuple(sorted(set(Scur) - {i} | {q}))]
        (bi, bq) = min(neigh, key=lambda t: (neigh[t], t))
        assert (info.i_out, info.j_in) == (bi, bq)
        assert info.delta == pytest.approx(neigh[(bi, bq)] - bf[tuple(Scur)], rel=1e-8, abs=1e-10)
        if not info.accepted:
            break
        srch.apply(info.slot, info.j_in)
    # a pair-exact search ends in a support no single swap can improve (by more than the threshold)
    assert min(neigh.values()) - bf[tuple(Scur)] > -orc.EPS_ACC * bf[tuple(Scur)]


def test_accept_always_runs_fixed_number_of_iterations():
    """The paper's Algorithm 1 runs T iterations with no test; 'always' reproduces that."""
    wl = workloads.tiny(p=12, m=5, g=1, k=6, n=40, seed=0)
    X, W, H, G, const = problem(wl)
    S0, _ = orc.init_support(H, W, 1, 6)
    run = orc.Search(H, G, const, 1, S0, accept="always").run(7)
    assert len(run.swap_trace) == 7 and run.stop_reason == "max_swaps"
    for o, S_hist in zip(run.obj_trace[-1:], [run.st.S]):
        assert o == pytest.approx(orc.solve_support_lstsq(X, W, S_hist, 1)[1], rel=1e-9)


# ----------------------------------------------------------------------------- update algebra (Prop. 1)
@pytest.mark.parametrize("g,score_mode", [(1, "independent"), (3, "independent"), (2, "pair_exact")])
def test_lowrank_updates_match_fresh_state(g, score_mode):
    p, k = 14, 6
    wl = workloads.tiny(p=p, m=6, g=g, k=k, n=120, seed=9)
    X, W, H, G, const = problem(wl)
    S0, _ = orc.init_support(H, W, g, k)
    lr = orc.Search(H, G, const, g, S0, mode="lowrank", score_mode=score_mode, accept="always",
                    refactor_every=10 ** 9)
    for step in range(12):
        info = lr.propose()
        lr.apply(info.slot, info.j_in)
        st = lr.st
        I = orc.rows_of(st.S, g)
        HII = H[np.ix_(I, I)]
        assert np.abs(st.Hinv @ HII - np.eye(len(I))).max() < 1e-9       # still the inverse
        assert np.allclose(st.Hinv, np.linalg.inv(HII), rtol=1e-8, atol=1e-12)
        V_def = np.linalg.lstsq(X[:, I], X @ W, rcond=None)[0]
        assert np.allclose(st.V, V_def, rtol=1e-6, atol=1e-9)
        W_S = np.zeros_like(W)
        W_S[I] = V_def
        R_def = H @ (W - W_S)
        R_def[I] = 0
        assert np.allclose(st.R, R_def, atol=1e-8 * np.abs(R_def).max())
        assert np.all(st.R[I] == 0)
        for q, cq in st.c.items():
            rq = slice(q * g, q * g + g)
            assert np.allclose(cq, H[rq, rq] - H[rq][:, I] @ np.linalg.inv(HII) @ H[I][:, rq], atol=1e-8 * H.max())
        assert set(st.c.keys()) == set(range(p)) - set(st.S)
        assert st.obj == pytest.approx(orc.objective_from_X(X, W, W_S), rel=1e-9)   # running == fresh


def test_dropped_rows_vanish_case1():
    """Eq. tmp4: applying the Case-1 correction zeroes the dropped rows of W and leaves the optimum
    of the smaller support on the remaining rows."""
    wl = workloads.tiny(p=7, m=3, g=2, k=4, n=50, seed=1)
    X, W, H, G, const = problem(wl)
    S = np.array([0, 2, 3, 6])
    I = orc.rows_of(S, 2)
    Hinv = np.linalg.inv(H[np.ix_(I, I)])
    V = Hinv @ G[I]
    r = np.array([2, 3])                 # slot 1 -> group 2
    full = V - Hinv[:, r] @ np.linalg.solve(Hinv[np.ix_(r, r)], V[r])
    assert np.abs(full[r]).max() < 1e-12
    W_small = orc.solve_support_lstsq(X, W, [0, 3, 6], 2)[0]
    keep = np.setdiff1d(np.arange(8), r)
    assert np.allclose(full[keep], W_small[I[keep]], rtol=1e-7, atol=1e-10)


@pytest.mark.parametrize("name,over", [
    ("c1", {}),
    ("c2", dict(n=2048, d1=256, m=64, k=128, chunk_rows=2048)),
    ("c5", dict(n=2048, d1=256, m=64, k=77, chunk_rows=2048)),
    ("c4", dict(n=49 * 16, d1=9 * 48, m=32, k=24, chunk_rows=49 * 16)),
    ("c6", dict(n=49 * 40, d1=128, m=48, k=64, chunk_rows=49 * 10)),
])
def test_strict_and_lowrank_follow_the_same_sequence(name, over):
    wl = workloads.config(name, **over)
    X, W, H, G, const = problem(wl)
    S0, _ = orc.init_support(H, W, wl.g, wl.k)
    a = orc.Search(H, G, const, wl.g, S0, mode="strict").run(60)
    b = orc.Search(H, G, const, wl.g, S0, mode="lowrank", refactor_every=25).run(60)
    assert a.swap_trace == b.swap_trace and a.stop_reason == b.stop_reason
    assert len(a.swap_trace) >= 2
    assert np.allclose(a.obj_trace, b.obj_trace, rtol=1e-10)
    assert np.all(np.diff(a.obj_trace) < 0)
    Sa, Wa, _, _ = a.result()
    Sb, Wb, _, _ = b.result()
    assert np.array_equal(Sa, Sb) and np.allclose(Wa, Wb, rtol=1e-7, atol=1e-10)
    # with damping the objective lives on the damped H: ||X E||^2 + lambda ||E||^2
    lam = wl.damp * np.mean(np.sum(X * X, axis=0))
    expect = orc.objective_from_X(X, W, Wa) + lam * float(np.sum((W - Wa) ** 2))
    assert a.obj_trace[-1] == pytest.approx(expect, rel=1e-8)


def test_c1_golden_trace():
    """Regression pin: the stored trace was written by tests/golden/make_golden.py from the oracle."""
    import json
    with open(os.path.join(GOLDEN, "c1_seed0_trace.json")) as fh:
        gold = json.load(fh)
    wl = workloads.config("c1")
    X, W, H, G, const = problem(wl)
    S0, _ = orc.init_support(H, W, 1, 32)
    run = orc.Search(H, G, const, 1, S0).run(wl.max_swaps)
    assert list(S0) == gold["init_support"]
    assert [list(t) for t in run.swap_trace] == gold["swap_trace"]
    assert np.allclose(run.obj_trace, gold["obj_trace"], rtol=1e-9)
    assert list(run.result()[0]) == gold["final_support"]


# ----------------------------------------------------------------------------- initial support
def test_init_support_modes_and_ties():
    H = np.diag([1.0, 4.0, 1.0, 1.0])
    W = np.array([[2.0], [1.0], [2.0], [0.5]])
    S, e = orc.init_support(H, W, 1, 2, "energy")          # energies 4, 4, 4, .25 -> ids 0, 1 by tie rule
    assert list(S) == [0, 1] and np.allclose(e, [4, 4, 4, 0.25])
    S, e = orc.init_support(H, W, 1, 2, "magnitude")       # 4, 1, 4, .25 -> ids 0, 2
    assert list(S) == [0, 2]
    # group energy is ||X_q W_q||_F^2
    wl = workloads.tiny(p=5, m=3, g=3, k=2, n=30)
    X, Wt, Hh, G, const = problem(wl)
    _, e = orc.init_support(Hh, Wt, 3, 2)
    for q in range(5):
        r = slice(3 * q, 3 * q + 3)
        assert e[q] == pytest.approx(float(np.sum((X[:, r] @ Wt[r]) ** 2)), rel=1e-10)


# ----------------------------------------------------------------------------- workload generators
def test_workloads_are_reproducible_and_shaped():
    a = workloads.config("c2", n=700, d1=64, m=16, k=32, chunk_rows=256)
    b = workloads.config("c2", n=700, d1=64, m=16, k=32, chunk_rows=256)
    assert a.n_chunks == 3
    for c in range(3):
        assert np.array_equal(a.x_chunk(c).float().numpy(), b.x_chunk(c).float().numpy())
    x = a.x_full().float().numpy()
    assert x.shape == (700, 64) and 0.35 < np.mean(x == 0) < 0.65 and x.min() >= 0
    c3 = workloads.config("c3", n=4096, d1=8 * 16, m=8, g=16, k=4, chunk_rows=4096,
                          params={"outlier_frac": 0.0})
    x3 = c3.x_full().float().numpy()
    cc = np.corrcoef(x3[:, :16].T)
    assert abs(np.mean(cc[np.triu_indices(16, 1)]) - 0.5) < 0.05      # within-head correlation
    assert abs(np.corrcoef(x3[:, 0], x3[:, 16])[0, 1]) < 0.06          # heads independent
    c4 = workloads.config("c4", n=49 * 4, d1=9 * 6, m=5, k=3, chunk_rows=49 * 4)
    x4 = c4.x_full().numpy()
    assert x4.shape == (196, 54)
    # column c*9 + 4 is the centre tap of channel c: a plain copy of the feature map
    assert np.mean(x4[:, 4] == 0) == pytest.approx(0.5, abs=0.12)
    # zero padding: the top-left tap of the first patch of an image is outside the map
    assert x4[0, 0] == 0 and x4[49, 0] == 0
    c6 = workloads.config("c6", n=49 * 6, d1=32, m=8, k=16, chunk_rows=49 * 2)
    x6 = c6.x_full().numpy()
    assert x6.shape == (294, 32) and x6.min() >= 0 and 0.3 < np.mean(x6 == 0) < 0.7 and c6.n_chunks == 3
    assert np.array_equal(x6[98:196], c6.x_chunk(1).numpy())


# ----------------------------------------------------------------------------- nested (greedy) phase
@pytest.mark.parametrize("g,t_hat", [(1, 1), (1, 3), (2, 2)])
def test_greedy_phase_prunes_the_cheapest_groups(g, t_hat):
    """Each iteration of the nested phase removes the kept groups whose individual removal raises the
    reconstruction error least, as re-solved from X; the objective is non-decreasing and ends at obj of the result."""
    p, k = 9, 4
    wl = workloads.tiny(p=p, m=4, g=g, k=k, n=80, seed=13)
    X, W, H, G, const = problem(wl)
    S, dropped, obj = orc.greedy_prune(H, G, const, g, k, t_hat)
    assert len(S) == k and sum(len(d) for d in dropped) == p - k
    assert abs(obj[0]) < 1e-8 * const                      # full support reproduces the dense layer
    assert np.all(np.diff(obj) >= -1e-9 * const)
    cur = list(range(p))
    for out in dropped:
        base = orc.solve_support_lstsq(X, W, cur, g)[1]
        cost = {i: orc.solve_support_lstsq(X, W, [x for x in cur if x != i], g)[1] - base for i in cur}
        expect = sorted(cur, key=lambda i: (cost[i], i))[:len(out)]
        assert list(out) == expect
        cur = [x for x in cur if x not in out]
    assert sorted(cur) == list(S)
    assert obj[-1] == pytest.approx(orc.solve_support_lstsq(X, W, list(S), g)[1], rel=1e-8)


def test_greedy_phase_on_orthogonal_columns_keeps_the_largest_energies():
    rng = np.random.default_rng(8)
    n, p, m, k = 30, 8, 2, 3
    Q, _ = np.linalg.qr(rng.standard_normal((n, p)))
    sc = rng.uniform(0.5, 3.0, p)
    X = Q * sc
    W = rng.standard_normal((p, m))
    H, G, const = orc.gram(X, W)
    e = sc ** 2 * np.sum(W * W, axis=1)
    S, dropped, obj = orc.greedy_prune(H, G, const, 1, k, 2)
    assert set(S) == set(np.argsort(-e)[:k])
    assert [q for d in dropped for q in d] == list(np.argsort(e)[:p - k])
    assert obj[-1] == pytest.approx(float(np.sum(np.sort(e)[:p - k])), rel=1e-9)


# ----------------------------------------------------------------------------- cross term (sequential layer-wise form)
def test_cross_term_objective_is_least_squares_against_dense_output():
    wl = workloads.tiny(p=9, m=4, g=1, k=4, n=70, seed=21)
    Xd = wl.x_chunk(0).numpy().astype(np.float64)
    Xp = wl.x_pruned_chunk(0, noise=0.3).numpy().astype(np.float64)
    W = wl.weight().numpy().astype(np.float64)
    Y = wl.dense_output_chunk(0).numpy().astype(np.float64)
    assert np.allclose(Y, Xd @ W, rtol=1e-6, atol=1e-6) and not np.allclose(Xp, Xd)
    H, G, const = orc.gram_cross(Xp, Y)
    for S in [(0, 2, 5, 8), (1, 3, 4, 6), tuple(range(9))]:
        W_S, obj = orc.solve_support(H, G, const, S, 1)
        V, res, *_ = np.linalg.lstsq(Xp[:, list(S)], Y, rcond=None)
        assert obj == pytest.approx(float(np.sum((Y - Xp[:, list(S)] @ V) ** 2)), rel=1e-8)
        assert np.allclose(W_S[list(S)], V, rtol=1e-6, atol=1e-9)
    # the search works on (H, G, const) unchanged: every accepted swap lowers ||Y - X W||^2
    S0, _ = orc.init_support(H, W, 1, 4)
    run = orc.Search(H, G, const, 1, S0).run(20)
    assert np.all(np.diff(run.obj_trace) < 0)
    Wf = run.result()[1]
    assert run.obj_trace[-1] == pytest.approx(float(np.sum((Y - Xp @ Wf) ** 2)), rel=1e-8)


# ----------------------------------------------------------------------------- block exchanges (t_hat = 2 s, p_hat = 0)
def _tiny_problem(p=14, m=4, g=1, k=6, n=90, seed=5):
    wl = workloads.tiny(p=p, m=m, g=g, k=k, n=n, seed=seed)
    X = wl.x_chunk(0).numpy().astype(np.float64)
    W = wl.weight().numpy().astype(np.float64)
    H, G, const = orc.gram(X, W)
    return X, W, H, G, const


def test_block_search_with_one_pair_is_the_swap_search():
    X, W, H, G, const = _tiny_problem()
    S0, _ = orc.init_support(H, W, 1, 6)
    a = orc.Search(H, G, const, 1, S0, mode="strict").run(20)
    b = orc.BlockSearch(H, G, const, 1, S0, 1).run(20)
    assert [(o[0], i[0]) for o, i in b.block_trace] == a.swap_trace and len(a.swap_trace) > 0
    assert np.allclose(a.obj_trace, b.obj_trace, rtol=1e-12)
    assert a.stop_reason == b.stop_reason


@pytest.mark.parametrize("g,s", [(1, 2), (1, 3), (2, 2)])
def test_block_exchange_takes_the_s_lowest_and_highest_impacts_from_definitions(g, s):
    """Eq. impact by brute force: B_j from re-solved supports; the exchange is the s extremes on each side and its
    change of obj is the re-solved difference measured on X."""
    X, W, H, G, const = _tiny_problem(p=10, m=3, g=g, k=5, n=80, seed=8)
    S0, _ = orc.init_support(H, W, g, 5)
    srch = orc.BlockSearch(H, G, const, g, S0, s, accept="always")
    for _ in range(3):
        S = [int(v) for v in srch.st.S]
        obj = orc.solve_support_lstsq(X, W, S, g)[1]
        drop = {i: orc.solve_support_lstsq(X, W, [j for j in S if j != i], g)[1] - obj for i in S}
        add = {q: obj - orc.solve_support_lstsq(X, W, S + [q], g)[1] for q in range(10) if q not in S}
        want_out = sorted(drop, key=lambda i: (drop[i], i))[:s]
        want_in = sorted(add, key=lambda q: (-add[q], q))[:s]
        info = srch.propose()
        assert info.out == want_out and info.inn == want_in
        S_new = sorted(set(S) - set(want_out) | set(want_in))
        assert info.delta == pytest.approx(orc.solve_support_lstsq(X, W, S_new, g)[1] - obj, rel=1e-7, abs=1e-9)
        srch.apply(info.slots, info.inn)
        assert sorted(int(v) for v in srch.st.S) == S_new
        assert srch.st.obj == pytest.approx(orc.solve_support_lstsq(X, W, S_new, g)[1], rel=1e-8)


def test_block_exchange_on_orthogonal_columns_adds_up():
    """H diagonal: impacts do not interact, so the exchange changes obj by sum(D_out) - sum(A_in) and the search
    reaches the top-k energies in one iteration when s covers every misplaced group."""
    rng = np.random.default_rng(3)
    h = rng.uniform(0.5, 2.0, 12)
    W = rng.normal(size=(12, 3))
    H = np.diag(h); G = H @ W; const = float(np.sum(W * G))
    e = h * np.sum(W * W, axis=1)
    best = np.argsort(-e)[:6]
    S0 = np.sort(np.concatenate([best[:3], np.argsort(-e)[9:]]))       # three right, three wrong
    srch = orc.BlockSearch(H, G, const, 1, S0, 3)
    info = srch.propose()
    assert sorted(info.out) == sorted(int(v) for v in np.argsort(-e)[9:])
    assert sorted(info.inn) == sorted(int(v) for v in best[3:])
    assert info.delta == pytest.approx(np.sum(e[info.out]) - np.sum(e[info.inn]), rel=1e-10)
    srch.run(5)
    assert sorted(int(v) for v in srch.st.S) == sorted(int(v) for v in best)
    assert srch.stop_reason == "no_improvement" and len(srch.block_trace) == 1


def test_block_search_stops_when_the_exchange_does_not_improve_and_rejects_bad_sizes():
    X, W, H, G, const = _tiny_problem(p=12, m=4, g=1, k=6, n=100, seed=11)
    S0, _ = orc.init_support(H, W, 1, 6)
    run = orc.BlockSearch(H, G, const, 1, S0, 2).run(50)
    assert run.stop_reason == "no_improvement" and np.all(np.diff(run.obj_trace) < 0)
    info = run.propose()
    assert info.delta > -run.eps_acc * run.st.obj
    with pytest.raises(ValueError):
        orc.BlockSearch(H, G, const, 1, S0, 7)
    with pytest.raises(ValueError):
        orc.BlockSearch(H, G, const, 1, S0, 0)


# ----------------------------------------------------------------------------- candidate guard (Proposition 1, Case 2)
def duplicated_problem(g, k, m=5, n=80, seed=0):
    """A layer whose last k groups are copies of its first k groups (columns of X repeated): with the first k groups
    kept, every pruned group lies in the span of the kept columns."""
    rng = np.random.default_rng(seed)
    Xk = rng.standard_normal((n, k * g))
    X = np.concatenate([Xk, Xk], axis=1)
    W = rng.standard_normal((2 * k * g, m))
    H, G, const = orc.gram(X, W)
    return X, W, H, G, const


@pytest.mark.parametrize("g", [1, 3])
def test_dependent_group_is_ineligible_and_adds_nothing(g):
    """A pruned group that repeats kept columns has Schur complement 0 (the C^-1 of Case 2 is H_qq - H_qI H_II^-1 H_Iq,
    the squared distance of its columns from the kept span), bringing it back cannot lower the least-squares error,
    and the oracle must score it -inf (single rows) / report no inverse (groups) instead of dividing by it."""
    k = 4
    X, W, H, G, const = duplicated_problem(g, k)
    ng = 2 * k
    # one independent extra candidate so that the step still has somewhere to go: replace the last copy by fresh columns
    rng = np.random.default_rng(5)
    X[:, (ng - 1) * g:] = rng.standard_normal((X.shape[0], g))
    H, G, const = orc.gram(X, W)
    S = np.arange(k)
    st = orc.fresh_state(H, G, const, S, g)
    _, obj_S = orc.solve_support_lstsq(X, W, S, g)
    for q in range(k, ng - 1):
        assert np.abs(st.c[q]).max() <= 1e-9 * np.abs(H).max()                       # Schur complement vanishes
        _, obj_add = orc.solve_support_lstsq(X, W, list(S) + [q], g)                 # the definition: nothing gained
        assert obj_add == pytest.approx(obj_S, rel=1e-9)
        if g > 1:
            assert orc._quad_inv(st.c[q], st.R[q * g:(q + 1) * g], float(np.max(np.diag(H[q * g:(q + 1) * g, q * g:(q + 1) * g])))) is None
    A = orc.add_scores(st, g, ng, H)
    assert np.all(np.isneginf(A[:ng - 1])) and np.isfinite(A[ng - 1]) and A[ng - 1] > 0
    # the eligible candidate's score is the true gain
    _, obj_new = orc.solve_support_lstsq(X, W, list(S) + [ng - 1], g)
    assert A[ng - 1] == pytest.approx(obj_S - obj_new, rel=1e-8)
    # the search never brings a group in while its twin (the group with the same columns) is kept
    twin = {q: q + k for q in range(k - 1)}
    twin.update({q + k: q for q in range(k - 1)})
    srch = orc.Search(H, G, const, g, S, accept="always")
    for _ in range(4):
        info = srch.propose(keep_scores=True)
        assert info is not None
        kept = set(int(v) for v in srch.st.S)
        assert twin.get(info.j_in) not in kept
        srch.apply(info.slot, info.j_in)
        assert len(set(int(v) for v in srch.st.S)) == k


@pytest.mark.parametrize("g", [1, 2])
def test_search_stops_with_guard_when_every_candidate_is_dependent(g):
    k = 5
    X, W, H, G, const = duplicated_problem(g, k, seed=2)
    srch = orc.Search(H, G, const, g, np.arange(k), accept="always").run(10)
    assert srch.stop_reason == "guard" and len(srch.swap_trace) == 0
    assert srch.propose() is None
    blk = orc.BlockSearch(H, G, const, g, np.arange(k), 2, accept="always").run(3)
    assert blk.stop_reason == "guard" and len(blk.block_trace) == 0
