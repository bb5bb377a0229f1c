"""CPU oracle for the OSSCAR per-layer solve.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 NumPy restatement of what the paper's per-layer problem
computes, written to be checked against the paper by eye.  It shares no code,
tables or helpers with the CUDA path and must never be imported by it: only the
test-suite, the smoke check and the benchmark's CPU-baseline leg call it.

Conventions (kept-set form of the paper's notation)
---------------------------------------------------
* W_hat is the dense weight, d1 x m; its rows are split into equal contiguous
  groups of g rows (Section 2, "Structured pruning as a MIQP": one group per
  input neuron, per conv input channel, or per attention head); group q holds
  rows q*g .. q*g+g-1 (0-based).
* `S` here is the set of KEPT groups (|S| = k) and I = I(S) its rows; the
  paper's S (Eq. deff) is the complementary, pruned set and its I_S (Eq. indexS)
  is our I.  J denotes the pruned rows.
* H = X^T X and G = H W_hat (Section 2, dense-layer paragraph).  The loss is the
  un-normalised reconstruction error  obj(S) = min_W ||X W_hat - X W||_F^2 over
  W with pruned rows zero;  obj = 2 f(S) + const with f from Eq. optf and
  const = Tr(W_hat^T H W_hat).

Readings of the paper taken here (each pinned by a CPU test)
------------------------------------------------------------
* Linear term has a minus sign (Eq. MIQP / Eq. deff), not the plus of
  Eq. obj-ver2.
* Dropping a kept group RAISES obj by Tr(V_r^T C^-1 V_r) (Case 1, Eq. tmp6 read
  with the sign monotonicity forces); adding a pruned group LOWERS obj by
  Tr(R_q^T c_q^-1 R_q) (Case 2, last display).
* Selection (text after Eq. impact, with t_hat = 2, p_hat = 0 so s1 = s2 = 1):
  the kept group whose removal costs least leaves, the pruned group whose
  return gains most enters.  Ties go to the smallest group id.
* Larger local-search steps (t_hat = 2 s, p_hat = 0, `BlockSearch`): s_1 = s_2 = s groups are exchanged per
  iteration, all chosen from the scores at the current support; the acceptance test applies to the whole exchange.
* The paper has no acceptance test; `accept="improving"` (stop at the first swap
  that does not lower obj by more than eps_acc * obj) and damping of H are
  choices of this build: parity unpinned by the paper.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass, field
from typing import Iterable, List, Optional, Sequence, Tuple

import numpy as np
import scipy.linalg as sla

EPS_ACC = 1e-5          # relative improvement a swap must bring to be accepted
PIVOT_TOL = 1e-12       # relative pivot below which a group is ineligible


# --------------------------------------------------------------------------- problem data
def gram(X: np.ndarray, W_hat: np.ndarray, damp: float = 0.0):
    """H = X^T X (+ damp * mean(diag H) * I), G = H W_hat, const = Tr(W_hat^T G).

    Section 2, dense-layer paragraph (H = X^T X, G = X^T X W_hat).  The damping
    term is not in the paper; it is applied before G so that the objective is
    defined on the damped H.
    """
    X = np.asarray(X, dtype=np.float64)
    W_hat = np.asarray(W_hat, dtype=np.float64)
    H = X.T @ X
    if damp:
        H = H + damp * np.mean(np.diag(H)) * np.eye(H.shape[0])
    G = H @ W_hat
    const = float(np.sum(W_hat * G))
    return H, G, const


def gram_cross(X, Y, damp: float = 0.0):
    """Sequential layer-wise objective (Appendix B.1, "Pruning strategies"): the target is the dense model's output
    Y = X_hat W_hat, the input the pruned model's activations X, so L(W) = ||Y - X W||_F^2 and
    H = X^T X (+ damping), G = X^T Y, const = ||Y||_F^2."""
    X = np.asarray(X, np.float64); Y = np.asarray(Y, np.float64)
    H = X.T @ X
    if damp:
        H = H + damp * np.mean(np.diag(H)) * np.eye(H.shape[0])
    return H, X.T @ Y, float(np.sum(Y * Y))


def gram_chunked(chunks: Iterable[np.ndarray], W_hat: np.ndarray, damp: float = 0.0):
    """Same as `gram` with X given as an iterable of row blocks."""
    H = None
    for Xc in chunks:
        Xc = np.asarray(Xc, dtype=np.float64)
        H = Xc.T @ Xc if H is None else H + Xc.T @ Xc
    if damp:
        H = H + damp * np.mean(np.diag(H)) * np.eye(H.shape[0])
    W_hat = np.asarray(W_hat, dtype=np.float64)
    G = H @ W_hat
    return H, G, float(np.sum(W_hat * G))


def rows_of(S: Sequence[int], g: int) -> np.ndarray:
    """Row indices I(S) of the groups in S, in the order of S (Eq. indexS)."""
    S = np.asarray(S, dtype=np.int64)
    return (S[:, None] * g + np.arange(g)[None, :]).reshape(-1)


def objective_from_X(X: np.ndarray, W_hat: np.ndarray, W: np.ndarray) -> float:
    """||X W_hat - X W||_F^2: the layer-wise reconstruction error (Eq. obj-ver1, un-normalised)."""
    X = np.asarray(X, dtype=np.float64)
    return float(np.sum((X @ (np.asarray(W_hat, np.float64) - np.asarray(W, np.float64))) ** 2))


def objective_quadratic(H: np.ndarray, W_hat: np.ndarray, W: np.ndarray) -> float:
    """Tr((W_hat - W)^T H (W_hat - W)) for any candidate W (Eq. obj-ver2 re-centred)."""
    E = np.asarray(W_hat, np.float64) - np.asarray(W, np.float64)
    return float(np.sum(E * (np.asarray(H, np.float64) @ E)))


def solve_support(H, G, const, S, g):
    """Optimal weights and objective for a fixed kept set S.

    W^(S)_I = H_II^-1 G_I, other rows zero (Eq. tmp5); obj = const - Tr(G_I^T H_II^-1 G_I)
    (Eq. optf times two, plus const).  Fresh Cholesky solve.
    """
    I = rows_of(sorted(S), g)
    L = sla.cho_factor(H[np.ix_(I, I)], lower=True, check_finite=False)
    V = sla.cho_solve(L, G[I], check_finite=False)
    W = np.zeros_like(G)
    W[I] = V
    return W, const - float(np.sum(G[I] * V))


def solve_support_lstsq(X, W_hat, S, g):
    """The same optimum straight from its definition: least squares on the kept columns of X."""
    X = np.asarray(X, np.float64)
    W_hat = np.asarray(W_hat, np.float64)
    I = rows_of(sorted(S), g)
    Y = X @ W_hat
    V, *_ = np.linalg.lstsq(X[:, I], Y, rcond=None)
    W = np.zeros_like(W_hat)
    W[I] = V
    return W, float(np.sum((Y - X[:, I] @ V) ** 2))


# --------------------------------------------------------------------------- initial support
def init_support(H, W_hat, g, k, mode="energy"):
    """k groups kept at the start, sorted.

    "energy":    e_q = Tr(W_q^T H_qq W_q) = ||X_q W_q||_F^2 (for g = 1: H_qq ||W_q||^2);
    "magnitude": e_q = ||W_q||_F^2 (the paper's MP baseline, Appendix B.1).
    The k largest are kept; equal energies go to the smaller group id.
    """
    W_hat = np.asarray(W_hat, np.float64)
    ng = W_hat.shape[0] // g
    e = np.empty(ng)
    for q in range(ng):
        r = slice(q * g, q * g + g)
        if mode == "energy":
            e[q] = np.sum(W_hat[r] * (H[r, r] @ W_hat[r]))
        elif mode == "magnitude":
            e[q] = np.sum(W_hat[r] ** 2)
        else:
            raise ValueError(mode)
    order = np.lexsort((np.arange(ng), -e))      # by -e, then id
    return np.sort(order[:k]).astype(np.int64), e


# --------------------------------------------------------------------------- state for a support
@dataclass
class State:
    S: np.ndarray            # kept groups, slot order (slot s holds rows s*g..s*g+g-1 of Hinv and V)
    Hinv: np.ndarray         # (H_II)^-1
    V: np.ndarray            # W^(S)_I = Hinv G_I
    R: np.ndarray            # G - H[:, I] V   (d1 x m; rows in I are exactly 0)
    c: dict                  # pruned group q -> Schur complement H_qq - H_qI Hinv H_Iq  (g x g)
    obj: float


def fresh_state(H, G, const, S, g) -> State:
    """Everything a search step needs, recomputed from scratch for the kept groups S (slot order kept)."""
    S = np.asarray(S, dtype=np.int64)
    I = rows_of(S, g)
    HII = H[np.ix_(I, I)]
    L = sla.cho_factor(HII, lower=True, check_finite=False)      # raises LinAlgError if not PD
    Hinv = sla.cho_solve(L, np.eye(len(I)), check_finite=False)
    Hinv = 0.5 * (Hinv + Hinv.T)
    V = sla.cho_solve(L, G[I], check_finite=False)
    R = G - H[:, I] @ V
    R[I] = 0.0
    ng = H.shape[0] // g
    kept = np.zeros(ng, dtype=bool)
    kept[S] = True
    c = {}
    HinvHIq = sla.cho_solve(L, H[I], check_finite=False)          # n_I x d1
    for q in np.nonzero(~kept)[0]:
        r = slice(q * g, q * g + g)
        c[int(q)] = H[r, r] - H[r][:, I] @ HinvHIq[:, r]
    obj = const - float(np.sum(G[I] * V))
    return State(S=S, Hinv=Hinv, V=V, R=R, c=c, obj=obj)


def _quad_inv(Mat, Rows, scale=None):
    """Tr(Rows^T Mat^-1 Rows) for a small SPD Mat; None if Mat is not safely positive definite
    (smallest Cholesky pivot <= PIVOT_TOL * scale, scale defaulting to the largest diagonal entry)."""
    try:
        L = np.linalg.cholesky(Mat)
    except np.linalg.LinAlgError:
        return None
    if scale is None:
        scale = max(np.max(np.diag(Mat)), 0.0)
    if np.min(np.diag(L)) ** 2 <= PIVOT_TOL * scale:
        return None
    Y = sla.solve_triangular(L, Rows, lower=True, check_finite=False)
    return float(np.sum(Y * Y))


def drop_scores(st: State, g: int) -> np.ndarray:
    """D[s] for every kept slot s: rise of obj when that group is pruned.

    Case 1 of Proposition 1 / Lemma A.1 with C = Hinv_rr and W_r = V_r:
    D = Tr(V_r^T C^-1 V_r)  (g = 1: ||V_s||^2 / Hinv_ss).
    """
    k = len(st.S)
    D = np.full(k, np.inf)
    if g == 1:                       # scalar case written out: ||V_s||^2 / Hinv_ss
        hd = np.diag(st.Hinv)
        ok = hd > 0
        D[ok] = np.sum(st.V[ok] ** 2, axis=1) / hd[ok]
        return D
    for s in range(k):
        r = slice(s * g, s * g + g)
        val = _quad_inv(st.Hinv[r, r], st.V[r])
        if val is not None:
            D[s] = val
    return D


def add_scores(st: State, g: int, ngroups: int, H=None) -> np.ndarray:
    """A[q] for every pruned group q (-inf for kept or ineligible groups): fall of obj when q returns.

    Case 2 of Proposition 1: the new rows of W are C (G_r - H_rI Hinv G_I) = c_q^-1 R_q with
    C^-1 = c_q the Schur complement, so the gain is Tr(R_q^T c_q^-1 R_q)  (g = 1: ||R_q||^2 / c_q).
    """
    A = np.full(ngroups, -np.inf)
    if g == 1:                       # scalar case written out: ||R_q||^2 / c_q
        for q, cq in st.c.items():
            scale = float(cq[0, 0]) if H is None else float(H[q, q])
            if cq[0, 0] > PIVOT_TOL * scale:
                A[q] = float(np.sum(st.R[q] ** 2)) / float(cq[0, 0])
        return A
    for q, cq in st.c.items():
        rq = slice(q * g, q * g + g)
        scale = None if H is None else float(np.max(np.diag(H[rq, rq])))
        val = _quad_inv(cq, st.R[rq], scale)
        if val is not None:
            A[q] = val
    return A


def swap_delta_closed_form(H, st: State, g: int, s: int, q: int) -> Optional[float]:
    """obj(S - {S[s]} + {q}) - obj(S) from the current state (Case 3 = Case 1 then Case 2).

    With r the rows of slot s:  C = Hinv_rr, K = C^-1 V_r, P = H_qI Hinv_Ir,
    R1_q = R_q + P K, c1 = c_q + P C^-1 P^T  and  delta = D_s - Tr(R1_q^T c1^-1 R1_q).
    """
    I = rows_of(st.S, g)
    r = slice(s * g, s * g + g)
    rq = slice(q * g, q * g + g)
    C = st.Hinv[r, r]
    Ds = _quad_inv(C, st.V[r])
    if Ds is None:
        return None
    K = np.linalg.solve(C, st.V[r])
    P = H[rq][:, I] @ st.Hinv[:, r]
    R1 = st.R[rq] + P @ K
    c1 = st.c[q] + P @ np.linalg.solve(C, P.T)
    gain = _quad_inv(0.5 * (c1 + c1.T), R1)
    if gain is None:
        return None
    return Ds - gain


# --------------------------------------------------------------------------- the search
@dataclass
class StepInfo:
    slot: int                 # slot of the leaving group
    i_out: int                # leaving group id
    j_in: int                 # entering group id
    delta: float              # exact change of obj for this swap (fresh evaluation)
    obj_before: float
    gap_out: float            # (second best - best) / best for the leaving choice (inf if unique)
    gap_in: float             # same for the entering choice
    accept_margin: float      # |delta + eps_acc * obj| / obj
    accepted: bool
    D: Optional[np.ndarray] = None
    A: Optional[np.ndarray] = None
    pair_delta: Optional[np.ndarray] = None


def _rel_gap_min(vals, ids):
    """index of the minimum (ties -> smallest id) and relative gap to the runner-up."""
    order = np.lexsort((ids, vals))
    best = order[0]
    if len(order) < 2 or not np.isfinite(vals[order[1]]):
        return best, np.inf
    denom = abs(vals[best]) if vals[best] != 0 else 1.0
    return best, (vals[order[1]] - vals[best]) / denom


class Search:
    """Algorithm 1 restricted to swaps (t_hat = 2, p_hat = 0), one step at a time.

    `mode="strict"` rebuilds the whole state from H, G with a fresh Cholesky factorisation at
    every step.  `mode="lowrank"` moves (Hinv, V, R, c) with the block-inverse identities of
    Proposition 1 (Cases 1-3) in fp64 and re-factorises every `refactor_every` swaps; it exists
    so that large layers can be followed for thousands of swaps and is itself tested step by
    step against the strict mode.
    """

    def __init__(self, H, G, const, g, S0, mode="strict", score_mode="independent",
                 accept="improving", eps_acc=EPS_ACC, refactor_every=250):
        self.H = np.asarray(H, np.float64)
        self.G = np.asarray(G, np.float64)
        self.const = float(const)
        self.g = int(g)
        self.ngroups = self.H.shape[0] // self.g
        self.mode, self.score_mode, self.accept, self.eps_acc = mode, score_mode, accept, eps_acc
        self.refactor_every = refactor_every
        self.st = fresh_state(self.H, self.G, self.const, np.asarray(S0, np.int64), self.g)
        self.obj_trace = [self.st.obj]
        self.swap_trace: List[Tuple[int, int]] = []
        self.stop_reason: Optional[str] = None
        self._since_refactor = 0

    # ---- scoring -------------------------------------------------------
    def scores(self):
        return drop_scores(self.st, self.g), add_scores(self.st, self.g, self.ngroups, self.H)

    def exact_delta(self, slot: int, q: int) -> float:
        """Change of obj for swapping slot's group with q, by fresh solves of both supports."""
        S_new = self.st.S.copy()
        S_new[slot] = q
        _, obj_new = solve_support(self.H, self.G, self.const, S_new, self.g)
        _, obj_old = solve_support(self.H, self.G, self.const, self.st.S, self.g)
        return obj_new - obj_old

    def propose(self, keep_scores=False) -> Optional[StepInfo]:
        st, g = self.st, self.g
        if len(st.c) == 0:
            return None
        D, A = self.scores()
        pair = None
        if self.score_mode == "independent":
            slot, gap_out = _rel_gap_min(D, st.S)
            neg = -A
            q, gap_in = _rel_gap_min(neg, np.arange(self.ngroups))
            if not np.isfinite(D[slot]) or not np.isfinite(A[q]):
                return None
        elif self.score_mode == "pair_exact":
            pruned = np.array(sorted(st.c.keys()))
            pair = np.full((len(st.S), len(pruned)), np.inf)
            for s in range(len(st.S)):
                for t, qq in enumerate(pruned):
                    val = swap_delta_closed_form(self.H, st, g, s, int(qq))
                    if val is not None:
                        pair[s, t] = val
            # ties: smallest leaving id, then smallest entering id
            ids_out = np.repeat(st.S, len(pruned))
            ids_in = np.tile(pruned, len(st.S))
            flat = pair.reshape(-1)
            order = np.lexsort((ids_in, ids_out, flat))
            best = order[0]
            if not np.isfinite(flat[best]):
                return None
            slot, q = int(best // len(pruned)), int(pruned[best % len(pruned)])
            if len(order) > 1 and np.isfinite(flat[order[1]]):
                denom = abs(flat[best]) if flat[best] != 0 else 1.0
                gap_out = gap_in = (flat[order[1]] - flat[best]) / denom
            else:
                gap_out = gap_in = np.inf
        else:
            raise ValueError(self.score_mode)
        if self.mode == "strict":
            delta = self.exact_delta(int(slot), int(q))
        else:
            delta = swap_delta_closed_form(self.H, st, g, int(slot), int(q))
            if delta is None:
                return None
        obj = st.obj
        if self.accept == "improving":
            accepted = delta <= -self.eps_acc * obj
        elif self.accept == "always":
            accepted = True
        else:
            raise ValueError(self.accept)
        margin = abs(delta + self.eps_acc * obj) / obj if obj > 0 else np.inf
        return StepInfo(slot=int(slot), i_out=int(st.S[slot]), j_in=int(q), delta=float(delta),
                        obj_before=obj, gap_out=float(gap_out), gap_in=float(gap_in),
                        accept_margin=float(margin), accepted=bool(accepted),
                        D=D if keep_scores else None, A=A if keep_scores else None,
                        pair_delta=pair if keep_scores else None)

    # ---- moving to the next support -------------------------------------
    def apply(self, slot: int, q: int):
        """Replace the group in `slot` by the pruned group q (the newcomer takes the slot)."""
        i_out = int(self.st.S[slot])
        if self.mode == "strict":
            S_new = self.st.S.copy()
            S_new[slot] = q
            self.st = fresh_state(self.H, self.G, self.const, S_new, self.g)
        else:
            self._since_refactor += 1
            if self._since_refactor >= self.refactor_every:
                S_new = self.st.S.copy()
                S_new[slot] = q
                self.st = fresh_state(self.H, self.G, self.const, S_new, self.g)
                self._since_refactor = 0
            else:
                self.st = lowrank_swap(self.H, self.st, self.g, slot, q)
        self.obj_trace.append(self.st.obj)
        self.swap_trace.append((i_out, int(q)))

    def run(self, max_swaps: int):
        while len(self.swap_trace) < max_swaps:
            info = self.propose()
            if info is None:
                self.stop_reason = "guard"
                break
            if not info.accepted:
                self.stop_reason = "no_improvement"
                break
            self.apply(info.slot, info.j_in)
        else:
            self.stop_reason = "max_swaps"
        return self

    def result(self):
        W = np.zeros_like(self.G)
        W[rows_of(self.st.S, self.g)] = self.st.V
        return np.sort(self.st.S), W, np.array(self.obj_trace), list(self.swap_trace)


@dataclass
class BlockStepInfo:
    slots: List[int]          # slots of the leaving groups, cheapest first
    out: List[int]            # leaving group ids (same order)
    inn: List[int]            # entering group ids, most valuable first; inn[t] takes slots[t]
    delta: float              # exact change of obj for the whole exchange (fresh evaluation)
    obj_before: float
    accepted: bool
    D: np.ndarray             # drop scores by slot
    A: np.ndarray             # add scores by group id (-inf for kept / ineligible groups)


class BlockSearch:
    """Local-search iterations of Algorithm 1 with p_hat = 0 and t_hat = 2 s (Eq. local, Eq. impact): the s kept
    groups with the lowest impact leave and the s pruned groups with the highest impact enter, all scored at the
    current support (s_1 = s_2 = s).  The exchange is kept iff it lowers obj by more than eps_acc * obj (or always).
    s = 1 is `Search` with independent scores.  Everything is recomputed from H, G at each iteration."""

    def __init__(self, H, G, const, g, S0, s, accept="improving", eps_acc=EPS_ACC):
        self.H = np.asarray(H, np.float64)
        self.G = np.asarray(G, np.float64)
        self.const = float(const)
        self.g, self.s = int(g), int(s)
        self.ngroups = self.H.shape[0] // self.g
        self.accept, self.eps_acc = accept, eps_acc
        S0 = np.asarray(S0, np.int64)
        if not (1 <= self.s <= min(len(S0), self.ngroups - len(S0))):
            raise ValueError("block size must be between 1 and min(k, ngroups - k)")
        self.st = fresh_state(self.H, self.G, self.const, S0, self.g)
        self.obj_trace = [self.st.obj]
        self.block_trace: List[Tuple[Tuple[int, ...], Tuple[int, ...]]] = []
        self.stop_reason: Optional[str] = None

    def exchange_delta(self, slots, inn) -> float:
        S_new = self.st.S.copy()
        S_new[np.asarray(slots)] = np.asarray(inn)
        return solve_support(self.H, self.G, self.const, S_new, self.g)[1] - \
            solve_support(self.H, self.G, self.const, self.st.S, self.g)[1]

    def propose(self) -> Optional[BlockStepInfo]:
        st = self.st
        D = drop_scores(st, self.g)
        A = add_scores(st, self.g, self.ngroups, self.H)
        slots = np.lexsort((st.S, D))[: self.s]
        inn = np.lexsort((np.arange(self.ngroups), -A))[: self.s]
        if not (np.all(np.isfinite(D[slots])) and np.all(np.isfinite(A[inn]))):
            return None
        delta = self.exchange_delta(slots, inn)
        accepted = True if self.accept == "always" else bool(delta <= -self.eps_acc * st.obj)
        return BlockStepInfo([int(v) for v in slots], [int(st.S[v]) for v in slots], [int(v) for v in inn],
                             float(delta), st.obj, accepted, D, A)

    def apply(self, slots, inn):
        out = tuple(int(self.st.S[v]) for v in slots)
        S_new = self.st.S.copy()
        S_new[np.asarray(slots)] = np.asarray(inn)
        self.st = fresh_state(self.H, self.G, self.const, S_new, self.g)
        self.obj_trace.append(self.st.obj)
        self.block_trace.append((out, tuple(int(v) for v in inn)))

    def run(self, max_iters: int):
        while len(self.block_trace) < max_iters:
            info = self.propose()
            if info is None:
                self.stop_reason = "guard"
                break
            if not info.accepted:
                self.stop_reason = "no_improvement"
                break
            self.apply(info.slots, info.inn)
        else:
            self.stop_reason = "max_swaps"
        return self

    def result(self):
        W = np.zeros_like(self.G)
        W[rows_of(self.st.S, self.g)] = self.st.V
        return np.sort(self.st.S), W, np.array(self.obj_trace), list(self.block_trace)


def lowrank_swap(H, st: State, g: int, slot: int, q: int) -> State:
    """State for S - {S[slot]} + {q} from the state for S, by Proposition 1 (Case 3).

    Case 1 (remove the rows r of `slot`): with [[A, B], [B^T, C]] the partition of Hinv,
    the inverse on the remaining rows is A - B C^-1 B^T and W loses [B C^-1; E] W_r.
    Case 2 (bring in the rows of q): C' = (H_qq - H_qI' Hinv' H_I'q)^-1, B' = -Hinv' H_I'q C',
    A' = Hinv' + B' C'^-1 B'^T, and the new rows of W are B'^T G_I' + C' G_q.
    The newcomer is stored in the slot that was vacated.
    """
    n_I = st.Hinv.shape[0]
    r = np.arange(slot * g, slot * g + g)
    keep = np.setdiff1d(np.arange(n_I), r)
    I = rows_of(st.S, g)
    rq = np.arange(q * g, q * g + g)
    i_out = int(st.S[slot])
    rout = np.arange(i_out * g, i_out * g + g)

    # ---- Case 1: drop rows r
    A_, B_, C_ = st.Hinv[np.ix_(keep, keep)], st.Hinv[np.ix_(keep, r)], st.Hinv[np.ix_(r, r)]
    Cinv_Bt = np.linalg.solve(C_, B_.T)
    Hinv1 = A_ - B_ @ Cinv_Bt                                  # inverse on I' = I minus r
    Wr = st.V[r]
    V1 = st.V[keep] - Cinv_Bt.T @ Wr                           # Eq. tmp4
    obj1 = st.obj + float(np.sum(Wr * np.linalg.solve(C_, Wr)))
    I1 = I[keep]
    U = H[:, I] @ st.Hinv[:, r]                                # H_{:,I} Hinv_{I,r}
    # residual after the drop, G - H[:, I'] V1: the rows of V changed by Hinv_{I,r} C^-1 W_r
    R1 = st.R + U @ np.linalg.solve(C_, Wr)
    R1[I1] = 0.0
    c1 = {}
    # Schur complements after the drop: every pruned group, plus the group that just left
    Cinv = np.linalg.inv(C_)
    for l, cl in st.c.items():
        rl = slice(l * g, l * g + g)
        c1[l] = cl + U[rl] @ Cinv @ U[rl].T
    c1[i_out] = Cinv.copy()

    # ---- Case 2: add rows of q
    hq = H[np.ix_(I1, rq)]
    y = Hinv1 @ hq
    cq = c1[q]
    Cn = np.linalg.inv(0.5 * (cq + cq.T))
    Bn = -y @ Cn
    An = Hinv1 + Bn @ cq @ Bn.T
    Vq = Cn @ R1[rq]                                           # = B'^T G_I' + C' G_q
    V2keep = V1 - y @ Vq
    obj2 = obj1 - float(np.sum(R1[rq] * Vq))
    Hinv2 = np.empty_like(st.Hinv)
    Hinv2[np.ix_(keep, keep)] = An
    Hinv2[np.ix_(keep, r)] = Bn
    Hinv2[np.ix_(r, keep)] = Bn.T
    Hinv2[np.ix_(r, r)] = Cn
    V2 = np.empty_like(st.V)
    V2[keep] = V2keep
    V2[r] = Vq
    dcol = H[:, rq] - H[:, I1] @ y                             # H_{:,q} - H_{:,I'} Hinv' H_{I',q}
    R2 = R1 - dcol @ Vq
    S2 = st.S.copy()
    S2[slot] = q
    R2[rows_of(S2, g)] = 0.0
    c2 = {}
    for l, cl in c1.items():
        if l == q:
            continue
        rl = slice(l * g, l * g + g)
        c2[l] = cl - dcol[rl] @ Cn @ dcol[rl].T
    return State(S=S2, Hinv=Hinv2, V=V2, R=R2, c=c2, obj=obj2)


# --------------------------------------------------------------------------- nested (greedy) phase
def greedy_prune(H, G, const, g, k, t_hat=1):
    """Nested phase of Algorithm 1 (t_i = p_i = t_hat): start from all groups kept (S_0 in the paper is the empty
    pruned set, with H^-1 and W* = H^-1 G) and, per iteration, prune the t_hat kept groups whose removal costs
    least (Eq. impact by Case 1 / Lemma A.1), all chosen from the scores at the current support, until k remain;
    the last iteration prunes only what is left to prune.  Everything is recomputed by fresh solves.

    Returns (kept groups sorted, list of the group tuples pruned per iteration in order of increasing score,
    objective after each iteration with entry 0 = obj of the full support).
    """
    H = np.asarray(H, np.float64); G = np.asarray(G, np.float64)
    ng = H.shape[0] // g
    S = np.arange(ng)
    obj = [solve_support(H, G, const, S, g)[1]]
    dropped = []
    while len(S) > k:
        I = rows_of(S, g)
        L = sla.cho_factor(H[np.ix_(I, I)], lower=True, check_finite=False)
        Hinv = sla.cho_solve(L, np.eye(len(I)), check_finite=False)
        V = sla.cho_solve(L, G[I], check_finite=False)
        st = State(S=S, Hinv=0.5 * (Hinv + Hinv.T), V=V, R=None, c={}, obj=obj[-1])
        D = drop_scores(st, g)
        t = min(t_hat, len(S) - k)
        order = np.lexsort((S, D))[:t]            # smallest score first, ties -> smaller id
        out = tuple(int(S[i]) for i in order)
        dropped.append(out)
        S = np.array([q for q in S if q not in set(out)])
        obj.append(solve_support(H, G, const, S, g)[1])
    return np.sort(S), dropped, np.array(obj)


# --------------------------------------------------------------------------- exhaustive reference
def brute_force(H, G, const, g, k):
    """Objective of every support of k groups (Eq. struc by enumeration).  Tiny inputs only."""
    ng = H.shape[0] // g
    out = {}
    for S in itertools.combinations(range(ng), k):
        _, obj = solve_support(H, G, const, S, g)
        out[S] = obj
    return out
