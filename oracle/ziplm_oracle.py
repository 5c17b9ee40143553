"""Float64 CPU oracle for the ZipLM layer-wise structured-OBS solver (arXiv 2302.04089, Sec. 3.1).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the method computes.
It is used by the tests, by the smoke check and by the CPU-baseline leg of the benchmark; the
product path never calls it and it never calls the product path (no shared code, no shared
constants).  Everything is numpy float64; inputs in fp32 / bf16 are widened exactly.

Notation follows the paper: W is d_row x d_col, X is d_col x N (one calibration token per
column), H = 2 X X^T (caption of Algorithm 1), a structure S is a set of g consecutive columns
("Pruned structures" paragraph: d_head consecutive columns of the attention out-matrix, single
columns of the second FFN matrix), R is the set of remaining structures.

Readings taken where the paper leaves a choice (each is also listed in the design notes):
  * H = 2 X X^T + lambda I with lambda = damp_frac * mean(diag(2 X X^T)); the paper's text writes
    H = X X^T once and 2 X X^T + lambda I in Algorithm 1's caption, and gives no lambda.
  * The row sum in Eq. 2 runs over all d_row rows once each.
  * The matrix norm in Eq. 1 is the squared Frobenius norm.
  * The final mask of Algorithm 1 zeroes the columns of the *removed* structures.
  * argmin ties go to the lowest structure index.
  * The reported loss is ||(W - W_hat) X||_F^2 without the damping term.
  * A level is the number of structures that remain; level 0 removes the whole module.

Pins (tests/test_oracle_pins.py): brute-force least-squares refits for every candidate on tiny
inputs, the direct inverse of the damped Hessian restricted to the survivors, the directly
computed reconstruction loss, the sum-of-saliencies identity, group-vs-single-column
equivalence, the diagonal-Hessian closed form, the duplicated-feature example, permutation and
scaling invariances.  The paper prints no worked numeric example of Algorithm 1, so no value is
pinned to a number printed there.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np


def as_f64(a) -> np.ndarray:
    """Widen a numpy array or a torch tensor (fp32 / bf16 / fp64, any device) to float64."""
    if hasattr(a, "detach"):
        a = a.detach().to("cpu").double().numpy()
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------------------------
# Hessian (caption of Algorithm 1; "Saliency scores and weight update" paragraph)
# --------------------------------------------------------------------------------------------
def hessian(X, alpha: float = 2.0) -> np.ndarray:
    """H = alpha * X X^T with alpha = 2 (Algorithm 1 caption).  X: [d_col, N]."""
    X = as_f64(X)
    return alpha * (X @ X.T)


def hessian_from_token_batches(batches, alpha: float = 2.0) -> np.ndarray:
    """H = alpha * sum over all calibration tokens x of x x^T (Algorithm 1 caption with X written
    column by column: X X^T is the sum of the outer products of its columns).  ``batches`` is a
    sequence of token-major matrices [n_b, d_col], one token per row, as a forward pass emits the
    layer inputs; the result does not depend on how the tokens are cut into batches."""
    H = None
    for A in batches:
        A = as_f64(A)
        part = np.zeros((A.shape[1], A.shape[1]))
        for x in A:
            part += np.outer(x, x)
        H = part if H is None else H + part
    return alpha * H


def damped(H, damp_frac: float):
    """(H + lambda I, lambda) with lambda = damp_frac * mean(diag H) (Algorithm 1 caption)."""
    H = as_f64(H)
    lam = damp_frac * float(np.mean(np.diag(H)))
    return H + lam * np.eye(H.shape[0]), lam


def inverse_spd(H_lam) -> np.ndarray:
    """Inverse of a symmetric positive definite matrix through its Cholesky factor.

    Raises numpy.linalg.LinAlgError when the matrix is not positive definite.
    """
    H_lam = as_f64(H_lam)
    Lc = np.linalg.cholesky(H_lam)                 # H_lam = Lc Lc^T
    Li = np.linalg.solve(Lc, np.eye(Lc.shape[0]))  # Lc^-1
    return Li.T @ Li


def reconstruction_loss(W0, W_hat, X) -> float:
    """||(W0 - W_hat) X||_F^2, the objective of Eq. 1, computed directly from X."""
    D = (as_f64(W0) - as_f64(W_hat)) @ as_f64(X)
    return float(np.sum(D * D))


def quadratic_loss(W0, W_hat, H) -> float:
    """1/2 tr(dW H dW^T), equal to reconstruction_loss when H = 2 X X^T (undamped)."""
    D = as_f64(W0) - as_f64(W_hat)
    return 0.5 * float(np.sum((D @ as_f64(H)) * D))


# --------------------------------------------------------------------------------------------
# Algorithm 1, one structure at a time
# --------------------------------------------------------------------------------------------
class GreedyOBS:
    """State of Algorithm 1: current W, current H^-1, remaining structures R."""

    def __init__(self, W, Hinv, group_size: int):
        self.W = as_f64(W).copy()
        self.Hinv = as_f64(Hinv).copy()
        self.g = int(group_size)
        self.d_row, self.d_col = self.W.shape
        if self.d_col % self.g != 0:
            raise ValueError("d_col must be a multiple of the group size")
        self.G = self.d_col // self.g
        self.remaining = np.ones(self.G, dtype=bool)      # R

    def live_groups(self) -> np.ndarray:
        return np.nonzero(self.remaining)[0]

    def saliencies(self):
        """Eq. 2 for every S in R:  rho_S = sum_i W[i,S] ((H^-1)[S,S])^-1 W[i,S]^T.

        Returns (live group indices ascending, rho of each).  The g x g block inverse is formed
        once per structure and shared by all rows (remark after Algorithm 1).
        """
        g, live = self.g, self.live_groups()
        Hb = self.Hinv.reshape(self.G, g, self.G, g)
        blocks = Hb[live, :, live, :]                                   # [n, g, g]
        Ws = self.W.reshape(self.d_row, self.G, g)[:, live, :]          # [r, n, g]
        Ws = np.transpose(Ws, (1, 2, 0))                                # [n, g, r]
        sol = np.linalg.solve(blocks, Ws)                               # B^-1 W_S^T
        rho = np.sum(Ws * sol, axis=(1, 2))
        return live, rho

    def best_two(self):
        """(best group, its rho, runner-up group, its rho); ties -> lowest index."""
        live, rho = self.saliencies()
        o = np.argsort(rho, kind="stable")
        b = o[0]
        s = o[1] if len(o) > 1 else o[0]
        return int(live[b]), float(rho[b]), int(live[s]), float(rho[s])

    def remove(self, s: int) -> None:
        """Eq. 3 (compensate W), Eq. 4 (downdate H^-1), R <- R - {S}."""
        if not self.remaining[s]:
            raise ValueError(f"structure {s} was already removed")
        S = slice(s * self.g, (s + 1) * self.g)
        K = np.linalg.solve(self.Hinv[S, S], self.Hinv[S, :])   # ((H^-1)_SS)^-1 (H^-1)_S,:
        self.W = self.W - self.W[:, S] @ K                      # W <- W + delta_S
        self.Hinv = self.Hinv - self.Hinv[:, S] @ K
        self.remaining[s] = False

    def masked_weights(self) -> np.ndarray:
        """W (.) M_R: columns of removed structures set to exactly zero (last line of Alg. 1)."""
        keep = np.repeat(self.remaining, self.g)
        return self.W * keep[None, :]

    def remaining_columns(self) -> np.ndarray:
        return np.nonzero(np.repeat(self.remaining, self.g))[0]


def prune(W, H, group_size: int, damp_frac: float, levels: Sequence[int],
          forced_order: Optional[Sequence[int]] = None, X=None,
          max_steps: Optional[int] = None) -> Dict:
    """Run Algorithm 1 on one layer and snapshot at the requested levels.

    W [d_row, d_col]; H [d_col, d_col] = 2 X X^T undamped; levels = numbers of remaining
    structures, strictly decreasing.  The loop runs until min(levels) structures remain (or for
    max_steps steps).  If forced_order is given, step t removes forced_order[t] (lock-step mode
    for parity runs) while the oracle still records its own best and runner-up for that step.
    If X is given the loss is ||(W - W_hat) X||_F^2 from X itself, else 1/2 tr(dW H dW^T).

    Returns a dict with: order, saliency (rho of the removed structure), best, best_rho,
    runner_up, runner_up_rho (per step), snapshots {level: W_hat}, losses {level: loss},
    base_loss = ||W X||_F^2, lam.
    """
    W0 = as_f64(W)
    H = as_f64(H)
    g = int(group_size)
    G = W0.shape[1] // g
    levels = [int(v) for v in levels]
    if any(levels[i] <= levels[i + 1] for i in range(len(levels) - 1)):
        raise ValueError("levels must be strictly decreasing")
    if levels and (levels[0] > G or levels[-1] < 0):
        raise ValueError("levels must lie in [0, G]")
    H_lam, lam = damped(H, damp_frac)
    st = GreedyOBS(W0, inverse_spd(H_lam), g)

    def loss_of(W_hat):
        return reconstruction_loss(W0, W_hat, X) if X is not None else quadratic_loss(W0, W_hat, H)

    out = dict(order=[], saliency=[], best=[], best_rho=[], runner_up=[], runner_up_rho=[],
               snapshots={}, losses={}, lam=lam,
               base_loss=loss_of(np.zeros_like(W0)))
    n_steps = G - (min(levels) if levels else G)
    if max_steps is not None:
        n_steps = min(n_steps, max_steps)
    if G in levels:
        out["snapshots"][G] = st.masked_weights()
        out["losses"][G] = 0.0
    for t in range(n_steps):
        live, rho = st.saliencies()
        o = np.argsort(rho, kind="stable")
        b = int(live[o[0]])
        s = int(live[o[1]]) if len(o) > 1 else b
        pick = b if forced_order is None else int(forced_order[t])
        rho_pick = float(rho[np.searchsorted(live, pick)])
        out["best"].append(b)
        out["best_rho"].append(float(rho[o[0]]))
        out["runner_up"].append(s)
        out["runner_up_rho"].append(float(rho[o[1]]) if len(o) > 1 else float(rho[o[0]]))
        out["order"].append(pick)
        out["saliency"].append(rho_pick)
        st.remove(pick)
        left = G - (t + 1)
        if left in levels:
            W_hat = st.masked_weights()
            out["snapshots"][left] = W_hat
            out["losses"][left] = loss_of(W_hat)
    out["final_state"] = st
    return out


# --------------------------------------------------------------------------------------------
# The plain definition the greedy updates reach for a given surviving set
# --------------------------------------------------------------------------------------------
def refit_on_support(W0, H_lam, remaining_cols: Sequence[int]):
    """Compensated weights and downdated inverse for a surviving column set, from definitions.

    After any sequence of removals that leaves the columns ``remaining_cols``, the updates of
    Eq. 3 / Eq. 4 give (in exact arithmetic)
        H^-1 restricted to the survivors = inverse(H_lam[R, R])   ("fully recomputing H^-1
        relative to the remaining structures", Sec. 3.1), and
        W_hat[:, R] = (W0 H_lam)[:, R] . inverse(H_lam[R, R]),
    the minimiser of 1/2 tr(dW H_lam dW^T) over weights supported on R.  Returns
    (W_hat [d_row, d_col] with zeros off R, inverse(H_lam[R, R])).
    """
    W0 = as_f64(W0)
    H_lam = as_f64(H_lam)
    Rc = np.asarray(remaining_cols, dtype=np.int64)
    W_hat = np.zeros_like(W0)
    if Rc.size == 0:
        return W_hat, np.zeros((0, 0))
    Hrr_inv = inverse_spd(H_lam[np.ix_(Rc, Rc)])
    W_hat[:, Rc] = (W0 @ H_lam)[:, Rc] @ Hrr_inv
    return W_hat, Hrr_inv


def saliencies_on_support(W0, H_lam, remaining_groups: Sequence[int], group_size: int):
    """Eq. 2 for every remaining structure, starting from the refit state of that support.

    Used to check a single late greedy step of a large problem without replaying the steps
    before it.  Returns (remaining groups ascending, rho).
    """
    g = int(group_size)
    groups = np.sort(np.asarray(remaining_groups, dtype=np.int64))
    cols = (groups[:, None] * g + np.arange(g)[None, :]).reshape(-1)
    W_hat, Hrr_inv = refit_on_support(W0, H_lam, cols)
    Wc = W_hat[:, cols]
    n = len(groups)
    rho = np.empty(n)
    for k in range(n):
        S = slice(k * g, (k + 1) * g)
        rho[k] = np.sum(Wc[:, S].T * np.linalg.solve(Hrr_inv[S, S], Wc[:, S].T))
    return groups, rho


# --------------------------------------------------------------------------------------------
# Model reshaping ("Pruned structures" paragraph of Sec. 3.1)
# --------------------------------------------------------------------------------------------
def kept_structures(order: Sequence[int], G: int, level: int) -> np.ndarray:
    """The `level` structures that the first G - level removals leave, ascending."""
    removed = [int(s) for s in order[:G - level]]
    if len(set(removed)) != len(removed) or any(s < 0 or s >= G for s in removed):
        raise ValueError("order must list distinct structures in [0, G)")
    return np.array([s for s in range(G) if s not in set(removed)], dtype=np.int64)


def drop_pruned_columns(W_masked, kept: Sequence[int], group_size: int) -> np.ndarray:
    """This layer after reshaping: only the columns of the kept structures remain."""
    W_masked = np.asarray(W_masked)
    cols = [s * group_size + c for s in kept for c in range(group_size)]
    return W_masked[:, cols]


def drop_matching_rows(M_prev, kept: Sequence[int], group_size: int) -> np.ndarray:
    """The previous layer after reshaping: the rows that produced the removed columns' inputs are
    removed ("corresponding rows in previous layers can be safely removed")."""
    M_prev = np.asarray(M_prev)
    rows = [s * group_size + c for s in kept for c in range(group_size)]
    return M_prev[rows]


# --------------------------------------------------------------------------------------------
# Budgeted level selection (Sec. 3.2: "Runtime awareness", "Finding the optimal sparsity
# configuration", "Structured SPDY search")
# --------------------------------------------------------------------------------------------
def error_prior(loss, base_loss) -> np.ndarray:
    """p_s: the layer-wise squared error of level s relative to ||W X||^2 -- 1 for a dropped
    module, 0 for the unpruned one ("Structured SPDY search")."""
    return as_f64(loss) / as_f64(base_loss)


def time_units(time, budget: float, n_buckets: int) -> int:
    """Run time of one option in units of budget / n_buckets, rounded up so that a selection that
    fits in units also fits in real time."""
    import math
    return int(math.ceil(float(np.float64(time) * (np.float64(n_buckets) / np.float64(budget)))))


def select_levels(loss, base_loss, time, n_options: Sequence[int], coef, budget: float,
                  n_buckets: int):
    """One level per module minimising sum_m coef[m] * p[m][s_m] subject to
    sum_m time[m][s_m] <= budget, by dynamic programming over modules on the discretised time
    axis: f_{m+1}[b] = min_s f_m[b - units(m, s)] + coef[m] * p[m][s], ties to the lowest s.

    loss, time: [n_modules, max_options]; base_loss, coef: [n_modules].
    Returns (selected option per module, minimal cost, summed time), or (None, inf, 0.0) when even
    the fastest options exceed the budget."""
    loss, time, coef = as_f64(loss), as_f64(time), as_f64(coef)
    base_loss = as_f64(base_loss)
    n_mod = loss.shape[0]
    f = np.zeros(n_buckets + 1)
    choices, units = [], []
    for m in range(n_mod):
        best = np.full(n_buckets + 1, np.inf)
        arg = np.zeros(n_buckets + 1, dtype=np.int64)
        um = []
        for s in range(int(n_options[m])):
            cost = coef[m] * (loss[m, s] / base_loss[m])
            u = time_units(time[m, s], budget, n_buckets)
            um.append(u)
            if u < 0 or u > n_buckets:
                continue
            cand = np.full(n_buckets + 1, np.inf)
            cand[u:] = f[:n_buckets + 1 - u] + cost
            better = cand < best                      # strict: the lowest s wins a tie
            best[better] = cand[better]
            arg[better] = s
        f = best
        choices.append(arg)
        units.append(um)
    if not np.isfinite(f[n_buckets]):
        return None, float("inf"), 0.0
    b = n_buckets
    selected = [0] * n_mod
    t_sum = 0.0
    for m in range(n_mod - 1, -1, -1):
        s = int(choices[m][b])
        selected[m] = s
        t_sum += time[m, s]
        b -= units[m][s]
    return selected, float(f[n_buckets]), float(t_sum)


def search_levels(loss, base_loss, time, n_options, objective, coef0, budget: float, n_buckets: int,
                  mask, values):
    """The mutation search of "Structured SPDY search", step by step: score coef0; then for every
    step replace the marked coefficients by the given values, solve the selection problem, score
    the selection (sum over modules of objective[m][s_m], the stand-in for the stitched model's
    calibration loss) and keep the mutated vector if the score is strictly lower.  mask, values:
    [n_steps, n_modules], drawn by the caller.
    Returns (best selection or None, best coefficients, best score, number of accepted steps)."""
    objective = as_f64(objective)
    best_c = np.asarray(coef0, dtype=np.float32).copy()
    best_sel, best_score, accepted = None, float("inf"), 0
    for step in range(len(mask) + 1):
        c = best_c.copy()
        if step > 0:
            marked = np.asarray(mask[step - 1]) != 0
            c[marked] = np.asarray(values[step - 1], dtype=np.float32)[marked]
        sel, _, _ = select_levels(loss, base_loss, time, n_options, c, budget, n_buckets)
        if sel is None:
            continue
        score = 0.0
        for m, s in enumerate(sel):
            score += objective[m, s]
        if score < best_score:
            best_sel, best_score, best_c = sel, score, c
            accepted += step > 0
    return best_sel, best_c, best_score, int(accepted)
