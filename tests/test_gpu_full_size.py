"""Full-size checks (the c2, c5 and c6 shapes, in the launch configuration bench.py times).

The oracle cannot form H at these sizes in test time, so the checks are properties that hold at any size,
evaluated on the oracle side from X itself on sampled outputs:
  * sampled entries of H against fp64 inner products of the corresponding columns of X;
  * optimality of the returned weights for the returned support: for sampled kept rows i and sampled output
    columns j,  X_i^T (X e_j) + lambda e_ij = 0  with e = W_hat - W_out and lambda the damping term;
  * the objective: per sampled column, ||X e_j||^2 + lambda ||e_j||^2 against the same column of the GPU's
    quadratic form, and the search's running objective against its recomputed value and against the
    state-independent osscar_objective entry point;
  * the trace: every accepted swap lowered the objective by more than the accept threshold; the support has k
    distinct groups; pruned rows of W_out are exactly zero.
"""
import numpy as np
import pytest
import torch

import workloads

pytestmark = [pytest.mark.gpu, pytest.mark.slow]


def _run(name, n_cols, max_swaps, block_pairs=0):
    import paper_2403_12983_b200 as pkg
    wl = workloads.config(name)
    dev = torch.device("cuda", 0)
    solver = pkg.Solver(0)
    W = wl.weight(dev)
    x_dev = [wl.x_chunk(c, dev) for c in range(wl.n_chunks)]
    res = pkg.solve_layer(solver, x_dev, W, wl.g, wl.k, max_swaps, damp=wl.damp, accept_rel_tol=wl.eps_acc,
                          block_pairs=block_pairs)
    rng = np.random.default_rng(0)
    support = res.support.cpu().numpy()
    assert len(np.unique(support)) == wl.k and support.min() >= 0 and support.max() < wl.ngroups
    assert np.all(np.diff(support) > 0)
    obj = res.obj_trace.cpu().numpy()
    per_it = max(block_pairs, 1)                 # block exchanges record one objective per iteration
    assert res.n_swaps % per_it == 0 and len(obj) == res.n_swaps // per_it + 1 and res.n_swaps > 0
    assert np.all(np.diff(obj) <= -wl.eps_acc * obj[:-1] * (1 - 1e-6))
    assert obj[-1] == pytest.approx(res.obj_final, rel=1e-4)
    swaps = res.swap_trace.cpu().numpy()
    kept = set(int(s) for s in support)
    assert all(int(j) != int(i) for i, j in swaps)
    for it in range(res.n_swaps // per_it):       # an exchange moves distinct groups
        blk = swaps[it * per_it:(it + 1) * per_it]
        assert len(set(int(v) for v in blk.reshape(-1))) == 2 * per_it
    Wout = res.W
    pruned_mask = torch.ones(wl.d1, dtype=torch.bool, device=dev)
    pruned_mask[res.support.long()] = False
    assert torch.count_nonzero(Wout[pruned_mask]).item() == 0
    # ---- oracle side, from X: sampled columns of X and E, accumulated chunk by chunk in fp64
    E = (W - Wout)
    cols_j = np.sort(rng.choice(wl.m, n_cols, replace=False))
    rows_i = np.sort(rng.choice(support, 24, replace=False))
    hpairs = rng.integers(0, wl.d1, size=(48, 2))
    hcols = np.unique(hpairs.reshape(-1))
    E_s = E[:, torch.as_tensor(cols_j, device=dev)].double().cpu().numpy()
    colsq = np.zeros(wl.d1)
    a_ij = np.zeros((len(rows_i), n_cols))
    rr = np.zeros(n_cols)
    hsub = np.zeros((len(hcols), len(hcols)))
    for Xc in x_dev:
        Xh = Xc.float().cpu().numpy().astype(np.float64)
        colsq += np.einsum("ij,ij->j", Xh, Xh)
        r = Xh @ E_s
        a_ij += Xh[:, rows_i].T @ r
        rr += np.einsum("ij,ij->j", r, r)
        Xs = Xh[:, hcols]
        hsub += Xs.T @ Xs
        del Xh
    lam = wl.damp * colsq.mean()
    # sampled H entries (damping sits on the diagonal)
    Hg = res.H[torch.as_tensor(hcols, device=dev)][:, torch.as_tensor(hcols, device=dev)].double().cpu().numpy()
    href = hsub + lam * np.eye(len(hcols))
    scale = np.sqrt(np.outer(np.diag(href), np.diag(href)))
    assert np.max(np.abs(Hg - href) / scale) < 4e-6
    # optimality on kept rows: X_i^T r_j + lam e_ij = 0, relative to |X_i| |r_j|
    resid = a_ij + lam * E_s[rows_i]
    denom = np.sqrt(np.outer(colsq[rows_i] + lam, rr + 1e-300))
    assert np.max(np.abs(resid) / denom) < 2e-4
    # per-column objective of the GPU's quadratic form vs ||X e_j||^2 + lam ||e_j||^2
    HE = res.H @ E[:, torch.as_tensor(cols_j, device=dev)]
    obj_cols_gpu = (E[:, torch.as_tensor(cols_j, device=dev)] * HE).sum(0).double().cpu().numpy()
    obj_cols = rr + lam * np.sum(E_s * E_s, axis=0)
    assert np.allclose(obj_cols_gpu, obj_cols, rtol=2e-4)
    # state-independent objective entry point (independent of the search state)
    H, Wd, Wo = res.H, W, res.W.clone()
    total = solver.objective(H, Wd, Wo)
    assert total == pytest.approx(res.obj_final, rel=2e-4)
    solver.close()
    return res


def test_c2_full_size_properties():
    res = _run("c2", n_cols=4, max_swaps=2000)
    assert res.stop_reason in ("no_improvement", "max_swaps")


def test_c5_full_size_properties():
    res = _run("c5", n_cols=2, max_swaps=300)
    assert res.n_swaps == 300 or res.stop_reason == "no_improvement"


def test_c2_full_size_block_exchange_properties():
    res = _run("c2", n_cols=4, max_swaps=2000, block_pairs=50)
    assert res.stop_reason in ("no_improvement", "max_swaps")


def test_c5_full_size_block_exchange_properties():
    res = _run("c5", n_cols=2, max_swaps=600, block_pairs=50)
    assert res.n_swaps == 600 or res.stop_reason == "no_improvement"


def test_c6_pointwise_conv_full_size_properties():
    res = _run("c6", n_cols=4, max_swaps=500)
    assert res.stop_reason in ("no_improvement", "max_swaps")
