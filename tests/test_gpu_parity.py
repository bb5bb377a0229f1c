"""Parity of the CUDA path (through the C ABI) with the fp64 CPU oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

import workloads
from oracle import osscar_oracle as orc
from tests.parity import GAP, follow_block, follow_greedy, follow_trace, oracle_problem, rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def osscar():
    import paper_2403_12983_b200 as pkg
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    pkg.lib()          # fails loudly if libosscar.so cannot be built / loaded
    return pkg


@pytest.fixture()
def solver(osscar):
    s = osscar.Solver()
    yield s
    s.close()


def dev(x, dtype=torch.float32):
    return torch.as_tensor(np.ascontiguousarray(x), dtype=dtype).cuda()


# ------------------------------------------------------------------------------------ Gram
GRAM_CASES = [
    # name, overrides: several 128x256 tiles, ragged column tail, token count not a multiple of 64
    ("c2", dict(n=1000, d1=840, m=72, k=400, chunk_rows=384)),
    ("c5", dict(n=700, d1=264, m=40, k=80, chunk_rows=700)),
    ("c3", dict(n=2100, d1=8 * 80, m=96, g=80, k=4, chunk_rows=1024)),
    ("c2", dict(n=130, d1=8, m=3, k=4, chunk_rows=64)),
]


@pytest.mark.parametrize("name,over", GRAM_CASES)
def test_gram_bf16_tensor_core(solver, name, over):
    wl = workloads.config(name, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, const = solver.gram([c.cuda() for c in wl.x_chunks()], wl.weight().cuda(), wl.damp)
    Hg, Gg = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    scale = np.sqrt(np.outer(np.diag(H64), np.diag(H64)))
    # bf16 products are exact in fp32; the tensor core adds each 16-token partial sum to its fp32 accumulator
    # with truncation, so chains are cut at 2048 tokens (128 MMAs, bias <= ~2e-6) and summed in registers
    assert np.max(np.abs(Hg - H64) / scale) < 4e-6
    assert np.array_equal(Hg, Hg.T)
    gs = np.linalg.norm(G64, axis=1, keepdims=True) + 1e-300
    assert np.max(np.abs(Gg - G64) / gs) < 1e-5
    assert const == pytest.approx(const64, rel=1e-5)


@pytest.mark.parametrize("name,over", [("c1", {}), ("c4", dict(n=49 * 12, d1=9 * 37, m=50, k=12, chunk_rows=49 * 5))])
def test_gram_fp32(solver, name, over):
    wl = workloads.config(name, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, const = solver.gram([c.cuda() for c in wl.x_chunks()], wl.weight().cuda(), wl.damp)
    Hg = H.cpu().numpy().astype(np.float64)
    scale = np.sqrt(np.outer(np.diag(H64), np.diag(H64)))
    assert np.max(np.abs(Hg - H64) / scale) < 5e-6
    assert np.array_equal(Hg, Hg.T)
    assert rel_fro(G.cpu().numpy(), G64) < 1e-5
    assert const == pytest.approx(const64, rel=1e-5)


@pytest.mark.parametrize("name,over,ws_rows", [
    ("c1", {}, None),
    ("c4", dict(n=49 * 12, d1=9 * 37, m=50, k=12, chunk_rows=49 * 5), None),         # d1 = 333: ragged tiles, odd row length
    ("c4", dict(n=49 * 24, d1=9 * 64, m=64, k=20, chunk_rows=49 * 10), 200),          # workspace holds 192-row panels only
    ("c6", dict(n=49 * 40, d1=520, m=96, k=260, chunk_rows=49 * 16), None),
])
def test_gram_fp32_on_tensor_cores(solver, osscar, name, over, ws_rows):
    """With a workspace lent to the context, fp32 activations are split into three bf16 terms and accumulated on the
    tensor cores (in row panels when the workspace is small); the result must be as accurate as the fp32 product."""
    wl = workloads.config(name, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    if ws_rows is None:
        solver.ensure_workspace(wl.d1, wl.m, wl.g, wl.k)
    else:
        solver.lend_workspace(6 * ws_rows * ((wl.d1 + 7) // 8 * 8) + 4096)
    launches0 = osscar.binding.launch_count()
    H, G, const = solver.gram([c.cuda() for c in wl.x_chunks()], wl.weight().cuda(), wl.damp)
    Hg = H.cpu().numpy().astype(np.float64)
    scale = np.sqrt(np.outer(np.diag(H64), np.diag(H64)))
    assert np.max(np.abs(Hg - H64) / scale) < 5e-6
    assert np.array_equal(Hg, Hg.T)
    assert rel_fro(G.cpu().numpy(), G64) < 1e-5
    assert const == pytest.approx(const64, rel=1e-5)
    if ws_rows is not None:       # panels of 192 rows (whole multiples of 64 that fit): one split and one product each
        panels = sum(-(-c.shape[0] // (ws_rows // 64 * 64)) for c in chunks)
        assert panels > len(chunks) and osscar.binding.launch_count() - launches0 >= 2 * panels


@pytest.mark.parametrize("name,over", [GRAM_CASES[0], GRAM_CASES[2], ("c2", dict(n=600, d1=200, m=37, k=100, chunk_rows=600))])
def test_cross_term_on_tensor_cores(solver, name, over):
    """With a workspace lent to the context, G = H W runs as a three-term bf16 split on the tensor cores;
    it must be as accurate as the fp32 product (ragged sizes: m not a multiple of 4, d1 not of 64)."""
    wl = workloads.config(name, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    Wd = wl.weight().cuda()
    solver.ensure_workspace(wl.d1, wl.m, wl.g, wl.k)
    H, G, const = solver.gram([c.cuda() for c in wl.x_chunks()], Wd, wl.damp)
    Hg = H.cpu().numpy().astype(np.float64)
    Gref = Hg @ W                        # the product itself, from the GPU's own H: isolates the GEMM
    gs = np.linalg.norm(Gref, axis=1, keepdims=True) + 1e-300
    assert np.max(np.abs(G.cpu().numpy() - Gref) / gs) < 2e-6
    assert const == pytest.approx(float(np.sum(W * Gref)), rel=3e-6)
    assert rel_fro(G.cpu().numpy(), G64) < 1e-5


def test_gram_empty_and_single_chunk_flags(solver, osscar):
    wl = workloads.config("c2", n=256, d1=64, m=8, k=32, chunk_rows=256)
    X = wl.x_chunk(0).cuda(); W = wl.weight().cuda()
    H = torch.full((64, 64), 7.0, device="cuda"); G = torch.empty(64, 8, device="cuda")
    b = osscar.binding
    # an empty first block clears H, the data then accumulates, END mirrors and builds G
    solver.gram_chunk(X[:0], H, b.GRAM_BEGIN)
    solver.gram_chunk(X, H, 0)
    const = solver.gram_chunk(X[:0], H, b.GRAM_END, W, G, 0.0)
    H2, G2, const2 = solver.gram([X], W, 0.0)
    assert torch.equal(H, H2) and torch.equal(G, G2) and const == const2


# ------------------------------------------------------------------------------------ state after init
STATE_CASES = [
    ("c1", {}, 0),
    ("c2", dict(n=3000, d1=520, m=150, k=207, chunk_rows=2048), 0),
    ("c5", dict(n=3000, d1=520, m=150, k=156, chunk_rows=2048), 1),
    ("c4", dict(n=49 * 30, d1=9 * 70, m=100, k=33, chunk_rows=49 * 30), 0),
    ("c3", dict(n=4096, d1=10 * 24, m=90, g=24, k=5, chunk_rows=4096), 2),
]


@pytest.mark.parametrize("name,over,seed", STATE_CASES)
def test_init_support_and_state(solver, name, over, seed):
    wl = workloads.config(name, seed=seed, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    # feed the oracle's own H and G (rounded to fp32) so that only the state construction is compared
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    S0, e = orc.init_support(Hr, W, wl.g, wl.k)
    support, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
    assert np.array_equal(support.cpu().numpy(), S0)
    st = orc.fresh_state(Hr, Gr, const_r, S0, wl.g)
    perm = solver.debug_state(4).cpu().numpy()
    assert np.array_equal(perm[:wl.k], S0) and np.array_equal(np.sort(perm), np.arange(wl.ngroups))
    assert obj0 == pytest.approx(st.obj, rel=1e-5)
    assert rel_fro(solver.debug_state(0).cpu().numpy(), st.Hinv) < 1e-4      # fp32 inverse: ~cond * 2^-24
    assert rel_fro(solver.debug_state(1).cpu().numpy(), st.V) < 5e-5
    rows_J = orc.rows_of(perm[wl.k:], wl.g)
    assert rel_fro(solver.debug_state(2).cpu().numpy(), st.R[rows_J]) < 5e-5
    c = solver.debug_state(3).cpu().numpy()
    for t, q in enumerate(perm[wl.k:]):
        assert np.allclose(c[t], st.c[int(q)], rtol=1e-4, atol=1e-5 * np.abs(st.c[int(q)]).max())
    D, A = orc.drop_scores(st, wl.g), orc.add_scores(st, wl.g, wl.ngroups, Hr)
    assert np.allclose(solver.debug_state(5).cpu().numpy(), D, rtol=1e-4)
    assert np.allclose(solver.debug_state(6).cpu().numpy(), A[perm[wl.k:]], rtol=1e-4)


def test_init_user_and_magnitude_modes(solver, osscar):
    wl = workloads.config("c2", n=2048, d1=96, m=24, k=40, chunk_rows=2048)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    b = osscar.binding
    Sm, _ = orc.init_support(H64, W, 1, 40, "magnitude")
    s, _ = solver.init_support(H, G, Wd, 1, 40, mode=b.INIT_MAGNITUDE)
    assert np.array_equal(s.cpu().numpy(), Sm)
    user = np.array(sorted(np.random.default_rng(0).choice(96, 40, replace=False)))[::-1].copy()
    s, obj = solver.init_support(H, G, Wd, 1, 40, mode=b.INIT_USER, support=torch.as_tensor(user))
    assert np.array_equal(s.cpu().numpy(), np.sort(user))
    assert obj == pytest.approx(orc.solve_support(H64, G64, const64, user, 1)[1], rel=1e-4)


# ------------------------------------------------------------------------------------ search
SEARCH_CASES = [
    ("c1", {}, 0, 50),
    ("c1", {}, 1, 50),
    ("c1", {}, 2, 50),
    ("c2", dict(n=8192, d1=1000, m=300, k=437, chunk_rows=4096), 0, 200),
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 1, 200),
    ("c5", dict(n=8192, d1=1000, m=300, k=300, chunk_rows=4096), 0, 200),
    ("c5", dict(n=4096, d1=520, m=150, k=156, chunk_rows=4096), 2, 200),
    ("c4", dict(n=49 * 40, d1=9 * 100, m=130, k=50, chunk_rows=49 * 40), 0, 100),
    ("c4", dict(n=49 * 40, d1=9 * 100, m=130, k=50, chunk_rows=49 * 40), 1, 100),
    ("c3", dict(n=8192, d1=12 * 40, m=200, g=40, k=6, chunk_rows=8192, score_mode="independent"), 0, 30),
    ("c6", dict(n=49 * 60, d1=320, m=136, k=160, chunk_rows=49 * 20), 0, 150),
]


def run_gpu_search(solver, wl, H, G, Wd, max_swaps, accept_always=False, S0=None):
    import paper_2403_12983_b200.binding as b
    if S0 is None:
        support, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
    else:
        support, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k, mode=b.INIT_USER, support=torch.as_tensor(S0))
    out = solver.local_search(max_swaps, accept_mode=b.ACCEPT_ALWAYS if accept_always else b.ACCEPT_IMPROVING,
                              accept_rel_tol=wl.eps_acc)
    return support.cpu().numpy(), obj0, out


@pytest.mark.parametrize("name,over,seed,max_swaps", SEARCH_CASES)
def test_search_matches_oracle_given_H(solver, name, over, seed, max_swaps):
    """Search parity with H, G handed over from the oracle (fp32-rounded): isolates the swap loop."""
    wl = workloads.config(name, seed=seed, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    S0, obj0, out = run_gpu_search(solver, wl, H, G, Wd, max_swaps)
    S0o, _ = orc.init_support(Hr, W, wl.g, wl.k)
    assert np.array_equal(S0, S0o)
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    gobj = out.obj_trace.cpu().numpy()
    srch, rebased = follow_trace(Hr, Gr, const_r, wl.g, S0, swaps, gobj, gpu_stop=out.stop_reason, max_swaps=max_swaps,
                                 eps_acc=wl.eps_acc)
    S_or, W_or, _, _ = srch.result()
    assert np.array_equal(out.support.cpu().numpy(), S_or)                       # identical final support
    assert np.all(np.diff(gobj) < 0)                                             # accepted swaps lower obj
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    assert gobj[-1] == pytest.approx(out.obj_final, rel=1e-4)                    # running == recomputed
    assert rel_fro(out.W.cpu().numpy(), W_or) < 1e-3
    Wg = out.W.cpu().numpy()
    pruned_rows = np.setdiff1d(np.arange(wl.d1), orc.rows_of(S_or, wl.g))
    assert np.all(Wg[pruned_rows] == 0)
    # state-independent cross-check of the objective through its own entry point
    assert solver.objective(H, Wd, out.W) == pytest.approx(srch.st.obj, rel=2e-4)
    assert len(swaps) >= 1 or wl.g > 1


@pytest.mark.parametrize("name,over,seed", [
    ("c3", dict(n=8192, d1=12 * 40, m=200, g=40, k=6, chunk_rows=8192), 0),
    ("c4", dict(n=49 * 40, d1=9 * 100, m=130, k=50, chunk_rows=49 * 40), 2),
    ("c3", dict(n=4096, d1=7 * 80, m=72, g=80, k=3, chunk_rows=4096), 1),
])
def test_group_updates_follow_oracle_with_forced_swaps(solver, osscar, name, over, seed):
    """Groups of several rows, every proposed swap applied (the paper's fixed-iteration form): the
    rank-2g updates must keep tracking the oracle's fp64 state."""
    wl = workloads.config(name, seed=seed, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    S0, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
    out = solver.local_search(12, accept_mode=osscar.binding.ACCEPT_ALWAYS)
    assert out.n_swaps == 12
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch, _ = follow_trace(Hr, Gr, const_r, wl.g, S0.cpu().numpy(), swaps, out.obj_trace.cpu().numpy(),
                           accept="always", gpu_stop="max_swaps", max_swaps=12)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    assert rel_fro(out.W.cpu().numpy(), srch.result()[1]) < 1e-3
    perm = solver.debug_state(4).cpu().numpy()
    st = orc.fresh_state(Hr, Gr, const_r, perm[:wl.k], wl.g)
    assert rel_fro(solver.debug_state(0).cpu().numpy(), st.Hinv) < 2e-4
    c = solver.debug_state(3).cpu().numpy()
    for t, q in enumerate(perm[wl.k:]):
        assert np.allclose(c[t], st.c[int(q)], rtol=1e-3, atol=1e-4 * np.abs(st.c[int(q)]).max())


PAIR_CASES = [
    ("c3", dict(n=8192, d1=12 * 40, m=200, g=40, k=6, chunk_rows=8192), 0, 12, False),
    ("c3", dict(n=8192, d1=12 * 40, m=200, g=40, k=6, chunk_rows=8192), 1, 8, True),
    ("c3", dict(n=16384, d1=32 * 80, m=384, g=80, k=16, chunk_rows=16384), 0, 6, True),     # c3's own head layout
    ("c4", dict(n=49 * 40, d1=9 * 40, m=130, k=20, chunk_rows=49 * 40, score_mode="pair_exact"), 0, 10, False),
    ("c1", dict(score_mode="pair_exact"), 0, 20, False),                                    # single-row groups
]


@pytest.mark.parametrize("name,over,seed,max_swaps,always", PAIR_CASES)
def test_pair_exact_search_matches_oracle(solver, osscar, name, over, seed, max_swaps, always):
    """Exhaustive pair scoring (Eq. local solved exactly for one swap): every step must take the oracle's best pair."""
    b = osscar.binding
    wl = workloads.config(name, seed=seed, **over)
    assert wl.score_mode == "pair_exact"
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    S0, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
    out = solver.local_search(max_swaps, score_mode=b.SCORE_PAIR_EXACT,
                              accept_mode=b.ACCEPT_ALWAYS if always else b.ACCEPT_IMPROVING, accept_rel_tol=wl.eps_acc)
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch, rebased = follow_trace(Hr, Gr, const_r, wl.g, S0.cpu().numpy(), swaps, out.obj_trace.cpu().numpy(),
                                 score_mode="pair_exact", accept="always" if always else "improving",
                                 gpu_stop=out.stop_reason, max_swaps=max_swaps, eps_acc=wl.eps_acc)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    assert rel_fro(out.W.cpu().numpy(), srch.result()[1]) < 1e-3
    if always:
        assert out.n_swaps == max_swaps
    else:
        assert np.all(np.diff(out.obj_trace.cpu().numpy()) < 0)


@pytest.mark.parametrize("name,over,seed,max_swaps", [SEARCH_CASES[0], SEARCH_CASES[4], SEARCH_CASES[6], SEARCH_CASES[7]])
def test_end_to_end_from_X(solver, name, over, seed, max_swaps):
    """Whole path from X: Gram on the GPU, then init and search; compared with the oracle run from X."""
    wl = workloads.config(name, seed=seed, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    Wd = wl.weight().cuda()
    H, G, const = solver.gram([c.cuda() for c in wl.x_chunks()], Wd, wl.damp)
    S0, obj0, out = run_gpu_search(solver, wl, H, G, Wd, max_swaps)
    S0o, e = orc.init_support(H64, W, wl.g, wl.k)
    if not np.array_equal(S0, S0o):
        # only groups whose energies tie within GAP at the selection boundary may differ
        diff = np.setxor1d(S0, S0o)
        thr = np.sort(e)[-wl.k]
        assert np.all(np.abs(e[diff] - thr) <= GAP * thr)
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    gobj = out.obj_trace.cpu().numpy()
    srch, rebased = follow_trace(H64, G64, const64, wl.g, S0, swaps, gobj, gpu_stop=out.stop_reason, max_swaps=max_swaps,
                                 eps_acc=wl.eps_acc)
    S_or, W_or, _, _ = srch.result()
    assert np.array_equal(out.support.cpu().numpy(), S_or)
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    assert rel_fro(out.W.cpu().numpy(), W_or) < 1e-3


def test_accept_always_runs_fixed_iterations_and_refresh(solver, osscar):
    wl = workloads.config("c2", n=4096, d1=520, m=150, k=207, chunk_rows=4096)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    b = osscar.binding
    S0, obj0 = solver.init_support(H, G, Wd, 1, wl.k)
    out = solver.local_search(40, accept_mode=b.ACCEPT_ALWAYS, refresh_every=16)
    assert out.n_swaps == 40 and out.stop_reason == "max_swaps" and out.n_refresh == 2
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch, _ = follow_trace(Hr, Gr, const_r, 1, S0.cpu().numpy(), swaps, out.obj_trace.cpu().numpy(),
                           accept="always", gpu_stop="max_swaps", max_swaps=40)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)


def test_state_after_search_is_consistent(solver):
    """After many swaps the updated (H_II)^-1 is still the inverse and V, R match a fresh solve."""
    wl = workloads.config("c5", n=4096, d1=520, m=150, k=156, chunk_rows=4096, seed=3)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    import paper_2403_12983_b200.binding as b
    solver.init_support(H, G, Wd, 1, wl.k)
    out = solver.local_search(60, accept_mode=b.ACCEPT_ALWAYS)
    perm = solver.debug_state(4).cpu().numpy()
    I = perm[:wl.k]
    Hinv = solver.debug_state(0).cpu().numpy().astype(np.float64)
    assert np.abs(Hinv @ Hr[np.ix_(I, I)] - np.eye(wl.k)).max() < 1e-3
    st = orc.fresh_state(Hr, Gr, float(np.sum(W * Gr)), I, 1)
    assert rel_fro(solver.debug_state(1).cpu().numpy(), st.V) < 1e-4
    assert rel_fro(solver.debug_state(2).cpu().numpy(), st.R[perm[wl.k:]]) < 1e-4
    c = solver.debug_state(3).cpu().numpy().reshape(-1)
    assert np.allclose(c, [st.c[int(q)][0, 0] for q in perm[wl.k:]], rtol=1e-3)


# ------------------------------------------------------------------------------------ block exchanges (t_hat = 2 s, p_hat = 0)
BLOCK_CASES = [
    # name, overrides, seed, pairs per iteration, max_swaps, accept always
    ("c1", {}, 0, 2, 50, False),
    ("c1", {}, 1, 5, 50, True),
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 1, 4, 200, False),
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 0, 16, 160, False),
    ("c5", dict(n=8192, d1=1000, m=300, k=300, chunk_rows=4096), 0, 50, 500, False),
    ("c5", dict(n=4096, d1=520, m=150, k=156, chunk_rows=4096), 2, 96, 960, True),
    ("c6", dict(n=49 * 60, d1=320, m=136, k=160, chunk_rows=49 * 20), 0, 8, 160, False),
    ("c2", dict(n=1024, d1=64, m=16, k=60, chunk_rows=1024), 0, 4, 8, True),        # every pruned group enters
    ("c2", dict(n=1024, d1=64, m=16, k=3, chunk_rows=1024), 0, 3, 6, True),         # every kept group leaves
    ("c4", dict(n=49 * 40, d1=9 * 100, m=130, k=50, chunk_rows=49 * 40), 0, 2, 60, False),
    ("c4", dict(n=49 * 40, d1=9 * 100, m=130, k=50, chunk_rows=49 * 40), 1, 5, 40, True),
    ("c3", dict(n=8192, d1=12 * 40, m=200, g=40, k=6, chunk_rows=8192, score_mode="independent"), 0, 2, 12, True),
]


@pytest.mark.parametrize("name,over,seed,s,max_swaps,always", BLOCK_CASES)
def test_block_exchange_matches_oracle(solver, name, over, seed, s, max_swaps, always):
    """s groups out and s groups in per iteration: sets, exact change, objective, final support and weights."""
    import paper_2403_12983_b200.binding as b
    wl = workloads.config(name, seed=seed, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    support, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
    S0 = support.cpu().numpy()
    max_swaps = min(max_swaps, 6 * s) if always else max_swaps
    out = solver.local_search(max_swaps, accept_mode=b.ACCEPT_ALWAYS if always else b.ACCEPT_IMPROVING,
                              accept_rel_tol=wl.eps_acc, block_pairs=s)
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    gobj = out.obj_trace.cpu().numpy()
    assert out.n_swaps % s == 0 and (out.n_swaps >= s or not always)
    srch = follow_block(Hr, Gr, const_r, wl.g, S0, s, swaps, gobj, accept="always" if always else "improving",
                        gpu_stop=out.stop_reason, max_iters=max_swaps // s, eps_acc=wl.eps_acc)
    S_or, W_or, _, _ = srch.result()
    assert np.array_equal(out.support.cpu().numpy(), S_or)
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    assert gobj[-1] == pytest.approx(out.obj_final, rel=1e-4)
    assert rel_fro(out.W.cpu().numpy(), W_or) < 1e-3
    # the maintained state against a fresh solve of the final support (slot order of the device)
    perm = solver.debug_state(4).cpu().numpy()
    st = orc.fresh_state(Hr, Gr, const_r, perm[:wl.k], wl.g)
    assert rel_fro(solver.debug_state(0).cpu().numpy(), st.Hinv) < 1e-3
    assert rel_fro(solver.debug_state(1).cpu().numpy(), st.V) < 1e-3
    pr = orc.rows_of(perm[wl.k:], wl.g)
    assert rel_fro(solver.debug_state(2).cpu().numpy(), st.R[pr]) < 1e-3
    c = solver.debug_state(3).cpu().numpy()
    cref = np.stack([st.c[int(q)] for q in perm[wl.k:]])
    assert np.allclose(c, cref, rtol=2e-3, atol=2e-3 * np.abs(cref).max())


def test_block_exchange_breaks_exact_ties_at_the_cut_by_group_id(solver, osscar):
    """Sixteen kept features that are uncorrelated with everything else and carry no weight have V_i = 0, hence drop
    scores that are exactly zero on both sides: more ties than the s = 5 places.  The rule (ties to the smaller id) then
    fixes which five leave in each iteration, and in which order they are listed."""
    b = osscar.binding
    rng = np.random.default_rng(5)
    nA, nZ, m, s = 72, 24, 24, 5
    d1 = nA + nZ
    X = rng.standard_normal((400, nA))
    H64 = np.zeros((d1, d1))
    H64[:nA, :nA] = X.T @ X
    H64[nA:, nA:] = np.diag(rng.uniform(50.0, 150.0, nZ))
    W = np.zeros((d1, m))
    W[:nA] = rng.standard_normal((nA, m))
    H64 = H64.astype(np.float32).astype(np.float64)
    W = W.astype(np.float32).astype(np.float64)
    G64 = H64 @ W
    assert not G64[nA:].any()
    keptZ = np.array([95, 73, 80, 76, 90, 74, 88, 79, 93, 72, 85, 91, 77, 83, 94, 81])
    keptA = rng.permutation(nA)[:32]
    S0 = rng.permutation(np.concatenate([keptA, keptZ])).astype(np.int32)      # the slot order must not matter
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    support, obj0 = solver.init_support(H, G, Wd, 1, len(S0), mode=b.INIT_USER, support=torch.as_tensor(S0))
    out = solver.local_search(3 * s, accept_mode=b.ACCEPT_ALWAYS, block_pairs=s)
    assert out.n_swaps == 3 * s
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    order = sorted(int(z) for z in keptZ)
    for it in range(3):
        assert [o for o, _ in swaps[it * s:(it + 1) * s]] == order[it * s:(it + 1) * s], f"iteration {it}"
    # the oracle, which breaks ties the same way, takes the same groups out
    srch = orc.BlockSearch(Hr, Gr, const_r, 1, np.sort(S0), s, accept="always")
    for it in range(3):
        info = srch.propose()
        assert sorted(int(o) for o in info.out) == order[it * s:(it + 1) * s]
        slots = [int(np.nonzero(srch.st.S == o)[0][0]) for o, _ in swaps[it * s:(it + 1) * s]]
        srch.apply(slots, [i for _, i in swaps[it * s:(it + 1) * s]])
    follow_block(Hr, Gr, const_r, 1, np.sort(S0), s, swaps, out.obj_trace.cpu().numpy(), accept="always", gpu_stop=out.stop_reason,
                 max_iters=3)


@pytest.mark.parametrize("name,over,s,greedy", [
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 8, 0),
    ("c4", dict(n=49 * 40, d1=9 * 100, m=130, k=50, chunk_rows=49 * 40), 3, 0),
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 8, 16),
])
def test_block_exchange_with_refresh_and_greedy_start(solver, osscar, name, over, s, greedy):
    """Block exchanges with the state rebuilt from H every second iteration, from the energy start and after the
    nested phase: the rebuilt state must continue the same walk."""
    b = osscar.binding
    wl = workloads.config(name, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    if greedy:
        support, _, obj0, _ = solver.init_support_greedy(H, G, Wd, wl.g, wl.k, greedy)
    else:
        support, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
    S0 = support.cpu().numpy()
    out = solver.local_search(5 * s, accept_mode=b.ACCEPT_ALWAYS, refresh_every=2, block_pairs=s)
    assert out.n_swaps == 5 * s and out.n_refresh == 2          # before iterations 2 and 4
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch = follow_block(Hr, Gr, const_r, wl.g, S0, s, swaps, out.obj_trace.cpu().numpy(), accept="always",
                        gpu_stop=out.stop_reason, max_iters=5, eps_acc=wl.eps_acc)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    assert rel_fro(out.W.cpu().numpy(), srch.result()[1]) < 1e-3


def test_block_exchange_argument_checks(solver, osscar):
    import paper_2403_12983_b200.binding as b
    wl = workloads.config("c1")
    chunks, W, H64, G64, _ = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    solver.init_support(H, G, Wd, 1, wl.k)
    for bad in (33, 97):                      # more pairs than pruned / kept groups, more rows than the limit
        with pytest.raises(osscar.OsscarError) as ei:
            solver.local_search(100, block_pairs=bad)
        assert ei.value.status == b.E_ARG
    with pytest.raises(osscar.OsscarError):
        solver.local_search(10, score_mode=b.SCORE_PAIR_EXACT, block_pairs=2)
    out = solver.local_search(3, block_pairs=4)           # fewer swaps allowed than one iteration exchanges
    assert out.n_swaps == 0 and out.stop_reason == "max_swaps"
    out = solver.local_search(50, block_pairs=1)          # one pair per iteration is the plain swap search
    ref = orc.Search(H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64),
                     float(np.sum(W * G.cpu().numpy().astype(np.float64))), 1,
                     orc.init_support(H.cpu().numpy().astype(np.float64), W, 1, wl.k)[0]).run(50)
    assert out.n_swaps == len(ref.swap_trace)


# ------------------------------------------------------------------------------------ nested (greedy) phase
GREEDY_CASES = [
    ("c1", {}, 1),
    ("c1", {}, 5),
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 10),
    ("c5", dict(n=4096, d1=264, m=72, k=80, chunk_rows=4096), 7),
    ("c4", dict(n=49 * 40, d1=9 * 60, m=130, k=25, chunk_rows=49 * 40), 2),
    ("c3", dict(n=8192, d1=12 * 40, m=200, g=40, k=6, chunk_rows=8192), 2),
    ("c2", dict(n=4096, d1=520, m=150, k=207, chunk_rows=4096), 64),          # wide steps: tensor-core downdates
    ("c5", dict(n=8192, d1=1000, m=300, k=300, chunk_rows=4096), 100),
]


@pytest.mark.parametrize("name,over,t_hat", GREEDY_CASES)
def test_greedy_phase_matches_oracle(solver, name, over, t_hat):
    """Nested phase of Algorithm 1 from the dense layer down to k groups, then the swap search from there."""
    wl = workloads.config(name, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    support, drops, obj0, iters = solver.init_support_greedy(H, G, Wd, wl.g, wl.k, t_hat)
    npr = wl.ngroups - wl.k
    assert iters == -(-npr // t_hat) and len(drops) == npr
    S_or = follow_greedy(Hr, Gr, const_r, wl.g, wl.k, t_hat, drops.cpu().numpy())
    assert np.array_equal(support.cpu().numpy(), S_or)
    assert obj0 == pytest.approx(orc.solve_support(Hr, Gr, const_r, S_or, wl.g)[1], rel=1e-4)
    # the state handed over is the regular one: the swap search continues from it and follows the oracle
    out = solver.local_search(20, accept_rel_tol=wl.eps_acc)
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch, _ = follow_trace(Hr, Gr, const_r, wl.g, S_or, swaps, out.obj_trace.cpu().numpy(), gpu_stop=out.stop_reason,
                           max_swaps=20, eps_acc=wl.eps_acc)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)


# ------------------------------------------------------------------------------------ cross term (sequential layer-wise form)
@pytest.mark.parametrize("name,over,ydt,lend", [
    ("c2", dict(n=3000, d1=520, m=152, k=207, chunk_rows=1024), torch.bfloat16, False),
    ("c2", dict(n=3000, d1=520, m=150, k=207, chunk_rows=1024), torch.float32, False),
    ("c4", dict(n=49 * 30, d1=9 * 37, m=50, k=12, chunk_rows=49 * 10), torch.float32, False),
    ("c4", dict(n=49 * 30, d1=9 * 37, m=50, k=12, chunk_rows=49 * 10), torch.float32, True),    # fp32 X: H on the tensor cores
])
def test_cross_term_gram_and_search(solver, name, over, ydt, lend):
    """Pruned-model inputs X, dense-model outputs Y: H = X^T X, G = X^T Y, const = ||Y||^2, then init and search."""
    wl = workloads.config(name, **over)
    if lend:
        solver.ensure_workspace(wl.d1, wl.m, wl.g, wl.k)
    W = wl.weight().numpy().astype(np.float64)
    xs = [wl.x_pruned_chunk(c) for c in range(wl.n_chunks)]
    ys = [wl.dense_output_chunk(c, dtype=ydt) for c in range(wl.n_chunks)]
    H64, G64, const64 = orc.gram_cross(np.concatenate([x.float().numpy() for x in xs]),
                                       np.concatenate([y.float().numpy() for y in ys]), wl.damp)
    H, G, const = solver.gram_cross([x.cuda() for x in xs], [y.cuda() for y in ys], wl.damp)
    scale = np.sqrt(np.outer(np.diag(H64), np.diag(H64)))
    assert np.max(np.abs(H.cpu().numpy() - H64) / scale) < 5e-6
    gs = np.linalg.norm(G64, axis=1, keepdims=True) + 1e-300
    assert np.max(np.abs(G.cpu().numpy() - G64) / gs) < 5e-6
    assert const == pytest.approx(const64, rel=1e-9)
    Wd = wl.weight().cuda()
    support, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
    S0 = support.cpu().numpy()
    assert obj0 == pytest.approx(orc.solve_support(H64, G64, const64, S0, wl.g)[1], rel=1e-4)
    out = solver.local_search(40, accept_rel_tol=wl.eps_acc)
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch, _ = follow_trace(H64, G64, const64, wl.g, S0, swaps, out.obj_trace.cpu().numpy(), gpu_stop=out.stop_reason,
                           max_swaps=40, eps_acc=wl.eps_acc)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
    assert rel_fro(out.W.cpu().numpy(), srch.result()[1]) < 1e-3


# ------------------------------------------------------------------------------------ candidate guard
def duplicated_layer(g, k, m, n, seed, free_last):
    """H, G (fp64) of a layer whose groups k .. 2k-1 repeat the columns of groups 0 .. k-1 exactly (H is assembled from
    one k*g-wide Gram block, so the copies are bit-identical); with `free_last` the last group gets fresh columns."""
    rng = np.random.default_rng(seed)
    Xk = rng.standard_normal((n, k * g))
    X = np.concatenate([Xk, Xk], axis=1)
    if free_last:
        X[:, (2 * k - 1) * g:] = rng.standard_normal((n, g))
    Hk = Xk.T @ Xk
    H = np.block([[Hk, Hk], [Hk, Hk]])
    if free_last:
        last = slice((2 * k - 1) * g, 2 * k * g)
        H[:, last] = X.T @ X[:, last]
        H[last, :] = H[:, last].T
    W = rng.standard_normal((2 * k * g, m)) / 8.0
    return H, H @ W, W


@pytest.mark.parametrize("g", [1, 3])
def test_dependent_groups_never_enter(solver, osscar, g):
    """Pruned groups that repeat kept columns have a vanishing Schur complement: both sides must leave them out of the
    add scores (the oracle by its 1e-12 pivot test in fp64, the device by 1e-6 on its fp32-built state), and the forced
    walk must still follow the oracle."""
    b = osscar.binding
    k = 12
    H64, G64, W = duplicated_layer(g, k, m=40, n=240, seed=3 + g, free_last=True)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    S0 = np.arange(k)
    support, obj0 = solver.init_support(H, G, Wd, g, k, mode=b.INIT_USER, support=torch.as_tensor(S0))
    A = solver.debug_state(6).cpu().numpy()                  # add scores by pruned slot (slot t holds group k + t)
    assert np.all(np.isneginf(A[:k - 1])) and np.isfinite(A[k - 1])
    st = orc.fresh_state(Hr, Gr, const_r, S0, g)
    A_or = orc.add_scores(st, g, 2 * k, Hr)
    assert np.all(np.isneginf(A_or[k:2 * k - 1])) and A[k - 1] == pytest.approx(A_or[2 * k - 1], rel=1e-4)
    out = solver.local_search(4, accept_mode=b.ACCEPT_ALWAYS)
    assert out.n_swaps == 4
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    twin = {q: q + k for q in range(k - 1)}
    twin.update({q + k: q for q in range(k - 1)})
    kept = set(range(k))
    for i_out, j_in in swaps:                                 # no group enters while the group with the same columns is kept
        assert twin.get(j_in) not in kept
        kept.remove(i_out); kept.add(j_in)
    srch, _ = follow_trace(Hr, Gr, const_r, g, S0, swaps, out.obj_trace.cpu().numpy(), accept="always",
                           gpu_stop="max_swaps", max_swaps=4)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])


@pytest.mark.parametrize("g,pairs", [(1, 0), (2, 0), (1, 3)])
def test_guard_stop_when_every_candidate_is_dependent(solver, osscar, g, pairs):
    b = osscar.binding
    k = 10
    H64, G64, W = duplicated_layer(g, k, m=24, n=200, seed=11, free_last=False)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    support, obj0 = solver.init_support(H, G, Wd, g, k, mode=b.INIT_USER, support=torch.arange(k, dtype=torch.int32))
    assert np.all(np.isneginf(solver.debug_state(6).cpu().numpy()))
    out = solver.local_search(12, accept_mode=b.ACCEPT_ALWAYS, block_pairs=pairs)
    assert out.n_swaps == 0 and out.stop_reason == "guard"
    assert out.obj_final == pytest.approx(obj0, rel=1e-6)
    assert np.array_equal(out.support.cpu().numpy(), np.arange(k))
    ref = orc.Search(H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64),
                     float(np.sum(W * G.cpu().numpy().astype(np.float64))), g, np.arange(k), accept="always").run(12)
    assert ref.stop_reason == "guard" and len(ref.swap_trace) == 0


# ------------------------------------------------------------------------------------ the two drivers of the swap loop
@pytest.mark.parametrize("name,over,seed,max_swaps", [
    SEARCH_CASES[0],                                                                  # 64 rows: fewer rows than blocks
    SEARCH_CASES[3],                                                                  # four / two rows per pass
    ("c2", dict(n=8192, d1=2600, m=1100, k=1300, chunk_rows=4096), 0, 10),            # two rows and one row per pass
    ("c5", dict(n=8192, d1=4200, m=2300, k=2100, chunk_rows=4096), 1, 8),            # one row per pass, two passes per row of V
])
def test_persistent_loop_and_launch_chain_follow_the_oracle(solver, osscar, name, over, seed, max_swaps):
    """Single-row groups have two drivers: one cooperative kernel with grid-wide barriers, or five launches per step.
    Both must follow the strict oracle; where no choice is a near-tie they make the same swaps."""
    b = osscar.binding
    wl = workloads.config(name, seed=seed, **over)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    runs = {}
    for mode in (b.LOOP_PERSISTENT, b.LOOP_LAUNCHES):
        S0, obj0 = solver.init_support(H, G, Wd, wl.g, wl.k)
        launches0 = b.launch_count()
        out = solver.local_search(max_swaps, accept_rel_tol=wl.eps_acc, loop_mode=mode, profile_samples=2)
        launched = b.launch_count() - launches0
        swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
        srch, rebased = follow_trace(Hr, Gr, const_r, wl.g, S0.cpu().numpy(), swaps, out.obj_trace.cpu().numpy(),
                                     gpu_stop=out.stop_reason, max_swaps=max_swaps, eps_acc=wl.eps_acc)
        assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
        assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)
        assert rel_fro(out.W.cpu().numpy(), srch.result()[1]) < 1e-3
        # the maintained state after the run against a fresh solve of the final support
        perm = solver.debug_state(4).cpu().numpy()
        st = orc.fresh_state(Hr, Gr, const_r, perm[:wl.k], wl.g)
        assert rel_fro(solver.debug_state(0).cpu().numpy(), st.Hinv) < 2e-4
        assert rel_fro(solver.debug_state(1).cpu().numpy(), st.V) < 1e-4
        assert rel_fro(solver.debug_state(2).cpu().numpy(), st.R[perm[wl.k:]]) < 1e-4
        runs[mode] = (swaps, rebased, launched, out)
    # the persistent driver is a handful of launches however many swaps it makes
    assert runs[b.LOOP_PERSISTENT][2] < 20 <= runs[b.LOOP_LAUNCHES][2]
    assert runs[b.LOOP_PERSISTENT][3].ms_kernel and runs[b.LOOP_LAUNCHES][3].ms_kernel
    if runs[b.LOOP_PERSISTENT][1] == 0 and runs[b.LOOP_LAUNCHES][1] == 0:
        assert runs[b.LOOP_PERSISTENT][0] == runs[b.LOOP_LAUNCHES][0]


def test_persistent_loop_with_refresh_and_forced_swaps(solver, osscar):
    b = osscar.binding
    wl = workloads.config("c2", n=4096, d1=520, m=150, k=207, chunk_rows=4096)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    const_r = float(np.sum(W * Gr))
    S0, obj0 = solver.init_support(H, G, Wd, 1, wl.k)
    out = solver.local_search(40, accept_mode=b.ACCEPT_ALWAYS, refresh_every=16, loop_mode=b.LOOP_PERSISTENT)
    assert out.n_swaps == 40 and out.stop_reason == "max_swaps" and out.n_refresh == 2
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch, _ = follow_trace(Hr, Gr, const_r, 1, S0.cpu().numpy(), swaps, out.obj_trace.cpu().numpy(),
                           accept="always", gpu_stop="max_swaps", max_swaps=40)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0])
    assert out.obj_final == pytest.approx(srch.st.obj, rel=1e-4)


# ------------------------------------------------------------------------------------ bounded waits
def test_grid_barrier_that_runs_out_returns_a_status(solver, osscar):
    """With a budget of a few cycles the first block to reach the first grid barrier of the persistent loop gives up:
    every block returns, the call reports OSSCAR_E_TIMEOUT, nothing hangs, and the same context then solves the same
    layer with the default budget."""
    b = osscar.binding
    wl = workloads.config("c2", n=4096, d1=1000, m=300, k=437, chunk_rows=4096)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    solver.init_support(H, G, Wd, 1, wl.k)
    with pytest.raises(osscar.OsscarError) as ei:
        solver.local_search(50, accept_rel_tol=wl.eps_acc, loop_mode=b.LOOP_PERSISTENT, wait_limit_cycles=4)
    assert ei.value.status == b.E_TIMEOUT
    with pytest.raises(osscar.OsscarError) as ei:               # the state of a failed search is not trusted
        solver.local_search(50, accept_rel_tol=wl.eps_acc)
    assert ei.value.status == b.E_STATE
    S0, obj0 = solver.init_support(H, G, Wd, 1, wl.k)
    out = solver.local_search(50, accept_rel_tol=wl.eps_acc, loop_mode=b.LOOP_PERSISTENT)
    Hr, Gr = H.cpu().numpy().astype(np.float64), G.cpu().numpy().astype(np.float64)
    swaps = [tuple(int(v) for v in r) for r in out.swap_trace.cpu().numpy()]
    srch, _ = follow_trace(Hr, Gr, float(np.sum(W * Gr)), 1, S0.cpu().numpy(), swaps, out.obj_trace.cpu().numpy(),
                           gpu_stop=out.stop_reason, max_swaps=50, eps_acc=wl.eps_acc)
    assert np.array_equal(out.support.cpu().numpy(), srch.result()[0]) and out.n_swaps > 0


def test_wait_that_runs_out_in_a_gram_chunk_is_reported_at_the_end(solver, osscar):
    """A wait budget of one cycle makes the first pipeline wait of the first chunk run out; the kernel drains its
    copies, returns, and the error must survive the second chunk and come back from the END call.  The context then
    works as before."""
    b = osscar.binding
    wl = workloads.config("c2", n=1024, d1=512, m=64, k=200, chunk_rows=512)
    X = [c.cuda() for c in wl.x_chunks()]
    W = wl.weight().cuda()
    H = torch.empty(wl.d1, wl.d1, device="cuda"); G = torch.empty(wl.d1, wl.m, device="cuda")
    solver.set_wait_limit(1)
    solver.gram_chunk(X[0], H, b.GRAM_BEGIN)
    solver.set_wait_limit(0)                                  # back to the default before the second chunk
    with pytest.raises(osscar.OsscarError) as ei:
        solver.gram_chunk(X[1], H, b.GRAM_END, W, G, wl.damp)
    assert ei.value.status == b.E_TIMEOUT
    chunks, Wh, H64, G64, const64 = oracle_problem(wl)
    H2, G2, const = solver.gram(X, W, wl.damp)
    scale = np.sqrt(np.outer(np.diag(H64), np.diag(H64)))
    assert np.max(np.abs(H2.cpu().numpy() - H64) / scale) < 4e-6
    assert const == pytest.approx(const64, rel=1e-5)


# ------------------------------------------------------------------------------------ edge cases and errors
def test_edge_cases(solver, osscar):
    b = osscar.binding
    wl = workloads.config("c2", n=1024, d1=64, m=16, k=64, chunk_rows=1024)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    # every group kept: nothing to swap, the dense weights come back and obj is ~0
    S, obj0 = solver.init_support(H, G, Wd, 1, 64)
    out = solver.local_search(10)
    assert out.n_swaps == 0 and np.array_equal(out.support.cpu().numpy(), np.arange(64))
    assert rel_fro(out.W.cpu().numpy(), W) < 1e-4 and abs(out.obj_final) < 1e-4 * const64
    # a single kept group and max_swaps = 0
    S, obj0 = solver.init_support(H, G, Wd, 1, 1)
    out = solver.local_search(0)
    assert out.n_swaps == 0 and out.stop_reason == "max_swaps"
    assert obj0 == pytest.approx(orc.solve_support(H64, G64, const64, S.cpu().numpy(), 1)[1], rel=1e-5)


def test_errors_are_reported_not_raised_on_device(solver, osscar):
    b = osscar.binding
    wl = workloads.config("c2", n=512, d1=64, m=16, k=32, chunk_rows=512)
    chunks, W, H64, G64, const64 = oracle_problem(wl)
    H, G, Wd = dev(H64), dev(G64), dev(W)
    with pytest.raises(osscar.OsscarError) as ei:
        solver.init_support(H, G, Wd, 5, 3)                 # 64 % 5 != 0
    assert ei.value.status == b.E_SHAPE
    with pytest.raises(osscar.OsscarError) as ei:
        solver.init_support(H, G, Wd, 1, 65)                # k > groups
    assert ei.value.status == b.E_SHAPE
    fresh = osscar.Solver()
    with pytest.raises(osscar.OsscarError) as ei:
        fresh._shape = (64, 16, 1, 32); fresh._keep = [H, G, Wd]
        fresh.local_search(5)                                # no state yet
    assert ei.value.status == b.E_STATE
    fresh.close()
    # duplicated column -> H_II singular -> E_NOTPD, and the context stays usable afterwards
    Hs = H64.copy(); Hs[:, 1] = Hs[:, 0]; Hs[1, :] = Hs[0, :]
    user = torch.arange(32, dtype=torch.int32)
    with pytest.raises(osscar.OsscarError) as ei:
        solver.init_support(dev(Hs), G, Wd, 1, 32, mode=b.INIT_USER, support=user)
    assert ei.value.status == b.E_NOTPD
    S, obj0 = solver.init_support(H, G, Wd, 1, 32)
    assert obj0 > 0
    with pytest.raises(osscar.OsscarError) as ei:
        solver.init_support(H, G, Wd, 1, 32, mode=b.INIT_USER, support=torch.zeros(32, dtype=torch.int32))
    assert ei.value.status == b.E_ARG
