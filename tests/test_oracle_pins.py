"""Pins for the float64 oracle: what the paper's equations and plain mathematics fix.

Each test names the passage it pins.  None of them compares the oracle with itself: expected
values come from brute-force least squares, direct library inverses, per-token loops, closed
forms or hand-worked fixtures under tests/golden/.
"""
import os

import numpy as np
import pytest

import workloads as wl
from oracle import ziplm_oracle as zo

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = [float(x) for x in v]
    return out


def tiny_problem(seed, d, r, N, recipe="ffn"):
    rng = np.random.default_rng(seed)
    W = rng.normal(size=(r, d))
    if recipe == "ffn":
        A = rng.normal(size=(d, max(2, d // 2))) / np.sqrt(max(2, d // 2))
        Z = rng.normal(size=(max(2, d // 2), N))
        X = np.maximum(A @ Z, 0.0) + 0.1 * rng.normal(size=(d, N))
    else:
        X = rng.normal(size=(d, N))
    return W, X


def brute_force_errors(W0, X, lam, remaining_cols):
    """Least-squares refit of the surviving columns on X_aug = [X, sqrt(lam/2) I].

    ||(W_hat - W0) X_aug||_F^2 = ||(W_hat - W0) X||_F^2 + lam/2 ||W_hat - W0||_F^2 and
    2 X_aug X_aug^T = 2 X X^T + lam I.  Returns (error, W_hat).
    """
    d = W0.shape[1]
    Xa = np.concatenate([X, np.sqrt(lam / 2.0) * np.eye(d)], axis=1)
    target = W0 @ Xa
    W_hat = np.zeros_like(W0)
    Rc = np.asarray(remaining_cols, dtype=int)
    if Rc.size:
        sol, *_ = np.linalg.lstsq(Xa[Rc, :].T, target.T, rcond=None)
        W_hat[:, Rc] = sol.T
    E = W_hat @ Xa - target
    return float(np.sum(E * E)), W_hat


# ------------------------------------------------------------------ hand-worked fixtures
def test_hand_worked_2x2_matches_eq2_eq3_eq4():
    gold = read_golden("hand_2x2.txt")
    H_lam = np.array([[2.0, 1.0], [1.0, 2.0]])
    W = np.array([[1.0, 2.0]])
    st = zo.GreedyOBS(W, zo.inverse_spd(H_lam), 1)
    live, rho = st.saliencies()
    assert np.allclose(rho, gold["rho_step0"], rtol=1e-13)
    b, rb, s, rs = st.best_two()
    assert b == int(gold["pick_step0"][0])
    st.remove(b)
    assert np.isclose(st.W[0, 1], gold["w_after_step0_col1"][0], rtol=1e-13)
    assert np.isclose(st.Hinv[1, 1], gold["hinv_after_step0_11"][0], rtol=1e-13)
    assert np.isclose(zo.quadratic_loss(W, st.masked_weights(), H_lam),
                      gold["objective_after_step0"][0], rtol=1e-13)
    live, rho = st.saliencies()
    assert np.allclose(rho, gold["rho_step1"], rtol=1e-13)
    st.remove(1)
    assert np.all(st.masked_weights() == 0.0)
    assert np.isclose(zo.quadratic_loss(W, st.masked_weights(), H_lam),
                      gold["objective_after_step1"][0], rtol=1e-13)


def test_hand_worked_group_fixture():
    gold = read_golden("hand_group.txt")
    H_lam = np.array([[2.0, 1, 0, 0], [1, 2, 0, 0], [0, 0, 4, 0], [0, 0, 0, 1]])
    W = np.array([[1.0, 2.0, 3.0, 1.0]])
    st = zo.GreedyOBS(W, zo.inverse_spd(H_lam), 2)
    live, rho = st.saliencies()
    assert np.allclose(rho, gold["rho_step0"], rtol=1e-13)
    b = st.best_two()[0]
    assert b == int(gold["pick_step0"][0])
    st.remove(b)
    assert np.allclose(st.W[0, 2:], gold["w_after_step0_cols23"], rtol=1e-13)
    assert np.allclose(np.diag(st.Hinv)[2:], gold["hinv_after_step0_22_33"], rtol=1e-13)
    assert np.all(st.masked_weights()[:, :2] == 0.0)


# ------------------------------------------------------------------ brute force (Eq. 2, Eq. 3)
@pytest.mark.parametrize("d,g,r,seed", [(6, 1, 3, 0), (8, 2, 4, 1), (12, 3, 5, 2), (9, 1, 2, 3),
                                        (10, 2, 1, 4), (16, 4, 3, 5)])
def test_every_greedy_step_against_brute_force_refit(d, g, r, seed):
    """Eq. 2 is the increase of the (damped) least-squares error when S is removed and the
    survivors are refitted; Eq. 3 is that refit.  Checked for EVERY candidate at EVERY step."""
    W0, X = tiny_problem(seed, d, r, 40)
    H = zo.hessian(X)
    H_lam, lam = zo.damped(H, 0.01)
    st = zo.GreedyOBS(W0, zo.inverse_spd(H_lam), g)
    G = d // g
    for step in range(G):
        live, rho = st.saliencies()
        cols_now = st.remaining_columns()
        err_now, W_now = brute_force_errors(W0, X, lam, cols_now)
        assert np.allclose(st.masked_weights(), W_now, rtol=1e-8, atol=1e-10)
        inc = []
        for s in live:
            cols = [c for c in cols_now if c // g != s]
            err_s, _ = brute_force_errors(W0, X, lam, cols)
            inc.append(err_s - err_now)
        inc = np.array(inc)
        assert np.allclose(rho / 2.0, inc, rtol=1e-7, atol=1e-9 * np.max(inc))
        b = st.best_two()[0]
        assert b == int(live[np.argmin(inc)])
        st.remove(b)
    assert np.all(st.masked_weights() == 0.0)


# ------------------------------------------------------------------ Eq. 4 vs direct inverse
@pytest.mark.parametrize("g", [1, 2, 4])
def test_downdated_inverse_equals_direct_inverse_on_survivors(g):
    d = 16
    W0, X = tiny_problem(7 + g, d, 5, 64)
    H_lam, lam = zo.damped(zo.hessian(X), 0.01)
    st = zo.GreedyOBS(W0, np.linalg.inv(H_lam), g)
    rng = np.random.default_rng(5)
    for s in rng.permutation(d // g)[:-1]:      # arbitrary (not greedy) removal order
        st.remove(int(s))
        Rc = st.remaining_columns()
        direct = np.linalg.inv(H_lam[np.ix_(Rc, Rc)])
        assert np.allclose(st.Hinv[np.ix_(Rc, Rc)], direct, rtol=1e-8, atol=1e-12)
        # path independence of the compensated weights (ridge refit on the survivors)
        W_ref = (W0 @ H_lam)[:, Rc] @ direct
        assert np.allclose(st.W[:, Rc], W_ref, rtol=1e-8, atol=1e-12)
        W_def, Hrr = zo.refit_on_support(W0, H_lam, Rc)
        assert np.allclose(W_def[:, Rc], W_ref, rtol=1e-9, atol=1e-13)
        assert np.allclose(Hrr, direct, rtol=1e-9, atol=1e-13)


def test_inverse_spd_against_library_inverse_and_identity():
    _, X = tiny_problem(3, 20, 2, 50)
    H_lam, _ = zo.damped(zo.hessian(X), 0.01)
    Hi = zo.inverse_spd(H_lam)
    assert np.allclose(Hi, np.linalg.inv(H_lam), rtol=1e-9, atol=1e-14)
    assert np.allclose(Hi @ H_lam, np.eye(20), atol=1e-9)
    with pytest.raises(np.linalg.LinAlgError):
        zo.inverse_spd(np.array([[1.0, 2.0], [2.0, 1.0]]))


# ------------------------------------------------------------------ loss (Eq. 1) and identities
@pytest.mark.parametrize("g", [1, 4])
def test_reported_loss_is_direct_reconstruction_error(g):
    d, r, N = 16, 6, 48
    W0, X = tiny_problem(11, d, r, N)
    G = d // g
    levels = list(range(G, -1, -1))
    res = zo.prune(W0, zo.hessian(X), g, 0.01, levels, X=X)
    res_h = zo.prune(W0, zo.hessian(X), g, 0.01, levels)          # loss from H instead of X
    prev = -1.0
    for lv in levels:
        W_hat = res["snapshots"][lv]
        direct = 0.0
        for t in range(N):                                         # token by token, Eq. 1
            e = (W0 - W_hat) @ X[:, t]
            direct += float(e @ e)
        assert np.isclose(res["losses"][lv], direct, rtol=1e-10, atol=1e-12)
        assert np.isclose(res_h["losses"][lv], direct, rtol=1e-9, atol=1e-12)
        assert res["losses"][lv] >= prev - 1e-9                    # non-decreasing along levels
        prev = res["losses"][lv]
        removed = sorted(res["order"][:G - lv])
        for s in removed:                                          # pruned columns exactly zero
            assert np.all(W_hat[:, s * g:(s + 1) * g] == 0.0)
    assert res["losses"][G] == 0.0
    full = float(np.sum((W0 @ X) ** 2))
    assert np.isclose(res["losses"][0], full, rtol=1e-12)          # p_s = 1 for a dropped layer
    assert np.isclose(res["base_loss"], full, rtol=1e-12)
    assert np.all(res["snapshots"][0] == 0.0)


@pytest.mark.parametrize("g", [1, 2])
def test_sum_of_saliencies_identity(g):
    """loss + lam/2 ||dW||_F^2 = 1/2 sum of the removed structures' rho (each Eq. 2 value is
    twice the increase of the damped objective)."""
    d, r = 12, 4
    W0, X = tiny_problem(21, d, r, 40)
    G = d // g
    res = zo.prune(W0, zo.hessian(X), g, 0.01, list(range(G - 1, -1, -1)), X=X)
    lam = res["lam"]
    assert all(v > 0 for v in res["saliency"])
    for lv in range(G - 1, -1, -1):
        dW = W0 - res["snapshots"][lv]
        lhs = res["losses"][lv] + 0.5 * lam * float(np.sum(dW * dW))
        rhs = 0.5 * float(np.sum(res["saliency"][:G - lv]))
        assert np.isclose(lhs, rhs, rtol=1e-9)


# ------------------------------------------------------------------ group == its columns in turn
def test_group_removal_equals_its_columns_removed_one_by_one():
    d, g, r = 12, 3, 4
    W0, X = tiny_problem(31, d, r, 50)
    H_lam, _ = zo.damped(zo.hessian(X), 0.01)
    Hinv = np.linalg.inv(H_lam)
    grp = zo.GreedyOBS(W0, Hinv, g)
    one = zo.GreedyOBS(W0, Hinv, 1)
    live, rho = grp.saliencies()
    s = 2
    seq = 0.0
    for c in range(s * g, (s + 1) * g):
        l1, r1 = one.saliencies()
        seq += float(r1[np.searchsorted(l1, c)])
        one.remove(c)
    grp.remove(s)
    assert np.isclose(rho[s], seq, rtol=1e-10)
    Rc = grp.remaining_columns()
    assert np.array_equal(Rc, one.remaining_columns())
    assert np.allclose(grp.W[:, Rc], one.W[:, Rc], rtol=1e-9, atol=1e-13)
    assert np.allclose(grp.Hinv[np.ix_(Rc, Rc)], one.Hinv[np.ix_(Rc, Rc)], rtol=1e-9, atol=1e-13)


def test_group_size_one_block_path_equals_scalar_formula():
    d, r = 10, 3
    W0, X = tiny_problem(41, d, r, 30)
    H_lam, _ = zo.damped(zo.hessian(X), 0.01)
    Hinv = np.linalg.inv(H_lam)
    st = zo.GreedyOBS(W0, Hinv, 1)
    live, rho = st.saliencies()
    assert np.allclose(rho, np.sum(W0 ** 2, axis=0) / np.diag(Hinv), rtol=1e-12)


# ------------------------------------------------------------------ special cases
def test_diagonal_hessian_closed_form():
    """Orthogonal feature rows: H diagonal, rho_j = H_lam[j,j] ||W[:,j]||^2, no compensation,
    and the greedy order is the ascending sort of that product."""
    d, r, N = 8, 3, 8
    rng = np.random.default_rng(0)
    Q, _ = np.linalg.qr(rng.normal(size=(N, N)))
    scales = np.linspace(0.5, 2.0, d)
    X = scales[:, None] * Q[:d, :]
    W0 = rng.normal(size=(r, d))
    H = zo.hessian(X)
    assert np.allclose(H, np.diag(2 * scales ** 2), atol=1e-12)
    res = zo.prune(W0, H, 1, 0.01, [0], X=X)
    H_lam, lam = zo.damped(H, 0.01)
    expect = np.diag(H_lam) * np.sum(W0 ** 2, axis=0)
    assert res["order"] == list(np.argsort(expect, kind="stable"))
    assert np.allclose(res["saliency"], np.sort(expect), rtol=1e-9)
    res1 = zo.prune(W0, H, 1, 0.01, [d - 3], X=X)
    keep = sorted(set(range(d)) - set(res1["order"]))
    assert np.allclose(res1["snapshots"][d - 3][:, keep], W0[:, keep], rtol=1e-9)


def test_redundant_pair_first_is_free_then_survivor_absorbs_it():
    """Two redundant structures: dropping one costs ~0, the other takes over its weight and is
    then expensive (the S1/S2 example of Sec. 3.1)."""
    rng = np.random.default_rng(2)
    d, r, N = 6, 3, 64
    X = rng.normal(size=(d, N))
    X[4] = X[1]                                   # feature 4 duplicates feature 1
    W0 = rng.normal(size=(r, d))
    H = zo.hessian(X)
    st = zo.GreedyOBS(W0, zo.inverse_spd(zo.damped(H, 1e-8)[0]), 1)
    live, rho0 = st.saliencies()
    b = st.best_two()[0]
    assert b in (1, 4)
    other = 4 if b == 1 else 1
    assert rho0[b] < 1e-4 * np.min(np.delete(rho0, [1, 4]))
    st.remove(b)
    assert np.allclose(st.W[:, other], W0[:, 1] + W0[:, 4], rtol=1e-5)
    live, rho1 = st.saliencies()
    assert rho1[np.searchsorted(live, other)] > 1e3 * rho0[other]


def test_argmin_tie_goes_to_lowest_index():
    H_lam = np.eye(4) * 2.0
    W = np.array([[1.0, 1.0, 1.0, 1.0], [2.0, 2.0, 2.0, 2.0]])
    res = zo.prune(W, H_lam, 1, 0.0, [0])
    assert res["order"] == [0, 1, 2, 3]


# ------------------------------------------------------------------ invariances
def test_permutation_and_scaling_invariance():
    d, r, N, g = 12, 4, 40, 2
    W0, X = tiny_problem(51, d, r, N)
    G = d // g
    levels = [4, 2]
    base = zo.prune(W0, zo.hessian(X), g, 0.01, levels, X=X)
    perm_g = np.random.default_rng(3).permutation(G)
    perm_c = (perm_g[:, None] * g + np.arange(g)[None, :]).reshape(-1)
    pr = zo.prune(W0[:, perm_c], zo.hessian(X[perm_c]), g, 0.01, levels, X=X[perm_c])
    assert [int(perm_g[s]) for s in pr["order"]] == base["order"]
    for lv in levels:
        assert np.allclose(pr["snapshots"][lv], base["snapshots"][lv][:, perm_c], rtol=1e-8,
                           atol=1e-12)
    c = 3.0
    sc = zo.prune(W0, zo.hessian(c * X), g, 0.01, levels, X=c * X)
    assert sc["order"] == base["order"]
    for lv in levels:
        assert np.allclose(sc["snapshots"][lv], base["snapshots"][lv], rtol=1e-8, atol=1e-12)
        assert np.isclose(sc["losses"][lv], c * c * base["losses"][lv], rtol=1e-8)


def test_factor_two_in_hessian_only_scales_saliency():
    d, r, N = 10, 3, 30
    W0, X = tiny_problem(61, d, r, N)
    a = zo.prune(W0, zo.hessian(X, 2.0), 1, 0.01, [3], X=X)
    b = zo.prune(W0, zo.hessian(X, 1.0), 1, 0.01, [3], X=X)
    assert a["order"] == b["order"]
    assert np.allclose(a["saliency"], 2.0 * np.array(b["saliency"]), rtol=1e-9)
    assert np.allclose(a["snapshots"][3], b["snapshots"][3], rtol=1e-9, atol=1e-13)


# ------------------------------------------------------------------ Hessian
def test_hessian_against_naive_triple_loop_and_symmetry():
    rng = np.random.default_rng(9)
    d, N = 5, 7
    X = rng.normal(size=(d, N))
    H = zo.hessian(X)
    naive = np.zeros((d, d))
    for i in range(d):
        for j in range(d):
            for t in range(N):
                naive[i, j] += 2.0 * X[i, t] * X[j, t]
    assert np.allclose(H, naive, rtol=1e-13, atol=1e-14)
    assert np.array_equal(H, H.T)
    assert np.all(np.diag(H) >= 0)
    H_lam, lam = zo.damped(H, 0.01)
    assert np.isclose(lam, 0.01 * np.trace(naive) / d, rtol=1e-13)
    assert np.allclose(H_lam - H, lam * np.eye(d), atol=1e-15)


def test_token_batch_hessian_is_the_hessian_of_the_layer_error():
    """Token-major, batch-by-batch form: independent of the cut into batches, equal entry by
    entry to a plain triple loop, equal to the feature-major form on the transposed matrix, and
    -- what makes it the Hessian of Eq. 1 -- w H w^T = 2 * sum_t (w . x_t)^2 for any row w."""
    rng = np.random.default_rng(10)
    d, N = 6, 11
    A = rng.normal(size=(N, d))                      # one token per row
    cuts = [A[:4], A[4:5], A[5:5], A[5:]]            # ragged batches, one of them empty
    H = zo.hessian_from_token_batches(cuts)
    naive = np.zeros((d, d))
    for t in range(N):
        for i in range(d):
            for j in range(d):
                naive[i, j] += 2.0 * A[t, i] * A[t, j]
    assert np.allclose(H, naive, rtol=1e-13, atol=1e-14)
    assert np.allclose(H, zo.hessian_from_token_batches([A]), rtol=1e-13, atol=1e-14)
    assert np.allclose(H, zo.hessian(A.T), rtol=1e-13, atol=1e-14)
    for _ in range(3):
        w = rng.normal(size=d)
        direct = 2.0 * sum(float(w @ A[t]) ** 2 for t in range(N))
        assert np.isclose(w @ H @ w, direct, rtol=1e-12)
    # a transposed operand (A A^T instead of A^T A) would not even have this shape
    assert H.shape == (d, d)


def test_level_grid_against_the_sizes_the_paper_prints():
    """The database's level grid (Sec. 3.2): the FFN sizes 0.9^i * d printed in the example
    latency table are met by the truncating grid (1814 is printed where the formula gives
    1813.98; 33 is the step after i = 42), and heads are pruned one at a time down to none."""
    vals = {}
    for line in open(os.path.join(GOLD, "latency_table_sizes.txt")):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            vals[k] = [int(x) for x in v]
    d = vals["intermediate_sizes"][0]
    grid = wl.ffn_size_grid(d)
    assert len(grid) == 43 and grid[0] == d
    assert abs(1.0 - grid[-1] / d - 0.99) < 0.003            # "until about 99 % sparsity"
    for i in range(1, 43):
        assert abs(grid[i] / grid[i - 1] - 0.9) < 0.02        # relative steps of 10 %
    for size in vals["intermediate_sizes"]:
        if size == 1814:
            assert 1813 in grid
        elif size == 33:
            assert wl.ffn_size_grid(d, 43)[-1] == 33 and 33 not in grid
        else:
            assert size in grid, size
    levels = wl.paper_level_grid(d, 1)
    assert levels[-1] == 0 and d not in levels
    assert all(a > b for a, b in zip(levels, levels[1:]))
    assert set(levels) - {0} == set(grid) - {d}
    G = vals["head_counts"][0]
    heads = wl.paper_level_grid(G, 64)
    assert heads == tuple(range(G - 1, -1, -1))
    assert set(vals["head_counts"]) - {G} <= set(heads)


def test_bf16_and_fp32_inputs_are_widened_exactly():
    import torch
    x = torch.tensor([[1.0, 0.333251953125, -2.5]], dtype=torch.bfloat16)
    assert np.array_equal(zo.as_f64(x), x.double().numpy())
    sh = wl.scaled(wl.CONFIGS["c5_gpt2"][1], d_col=32, d_latent=8, d_row=4, n_tokens=64,
                   n_layers=1)
    X = wl.make_activations(sh, 0)
    assert X.dtype == torch.bfloat16
    H = zo.hessian(X)
    Xd = X.double().numpy()
    assert np.allclose(H, 2 * Xd @ Xd.T, rtol=1e-14)


# ------------------------------------------------------------------ lock-step driving mode
def test_forced_order_reports_own_best_and_follows_the_given_pick():
    d, r, N = 10, 3, 40
    W0, X = tiny_problem(71, d, r, N)
    H = zo.hessian(X)
    free = zo.prune(W0, H, 1, 0.01, [5])
    forced = list(free["order"])
    forced[2] = free["runner_up"][2]                      # deviate once
    if forced[2] in forced[3:]:
        forced[forced.index(forced[2], 3)] = free["order"][2]
    res = zo.prune(W0, H, 1, 0.01, [5], forced_order=forced)
    assert res["order"] == forced
    assert res["best"][:3] == free["best"][:3]
    assert res["saliency"][2] == pytest.approx(free["runner_up_rho"][2], rel=1e-12)
    left = sorted(set(range(d)) - set(forced))
    H_lam, _ = zo.damped(H, 0.01)
    W_ref, _ = zo.refit_on_support(W0, H_lam, left)
    assert np.allclose(res["snapshots"][5], W_ref, rtol=1e-8, atol=1e-12)


def test_saliencies_on_support_match_replayed_state():
    d, g, r = 12, 2, 3
    W0, X = tiny_problem(81, d, r, 50)
    H_lam, _ = zo.damped(zo.hessian(X), 0.01)
    st = zo.GreedyOBS(W0, np.linalg.inv(H_lam), g)
    for s in (4, 0, 3):
        st.remove(s)
    live, rho = st.saliencies()
    groups, rho2 = zo.saliencies_on_support(W0, H_lam, live, g)
    assert np.array_equal(groups, live)
    # independent expectation: brute-force error increases
    lam = H_lam[0, 0] - zo.hessian(X)[0, 0]
    cols_now = st.remaining_columns()
    e0, _ = brute_force_errors(W0, X, lam, cols_now)
    inc = [brute_force_errors(W0, X, lam, [c for c in cols_now if c // g != s])[0] - e0
           for s in live]
    assert np.allclose(rho2 / 2, inc, rtol=1e-7)
    assert np.allclose(rho / 2, inc, rtol=1e-7)


def test_level_validation():
    W0, X = tiny_problem(91, 8, 2, 20)
    H = zo.hessian(X)
    with pytest.raises(ValueError):
        zo.prune(W0, H, 1, 0.01, [3, 5])
    with pytest.raises(ValueError):
        zo.prune(W0, H, 1, 0.01, [9])
    with pytest.raises(ValueError):
        zo.GreedyOBS(W0, np.eye(8), 3)


# ------------------------------------------------------------------ model reshaping
@pytest.mark.parametrize("g", [1, 2])
def test_reshaped_two_layer_block_computes_the_same_output(g):
    """"Pruned structures" (Sec. 3.1): with the removed columns of the second matrix zero, dropping
    them and the matching rows (and bias entries) of the first matrix changes no output -- checked
    on a small FC1 -> GELU -> FC2 block against the masked, full-shape block."""
    rng = np.random.default_rng(21)
    d_in, d_mid, d_out, N = 5, 12, 4, 9
    W1, b1 = rng.normal(size=(d_mid, d_in)), rng.normal(size=d_mid)
    W2 = rng.normal(size=(d_out, d_mid))
    inp = rng.normal(size=(d_in, N))
    import math
    erf = np.vectorize(math.erf)

    def act(v):                                                       # exact GELU
        return 0.5 * v * (1.0 + erf(v / np.sqrt(2.0)))

    X = act(W1 @ inp + b1[:, None])                                   # inputs of the pruned layer
    G = d_mid // g
    res = zo.prune(W2, zo.hessian(X), g, 0.01, [G // 2])
    W_masked = res["snapshots"][G // 2]
    kept = zo.kept_structures(res["order"], G, G // 2)
    assert len(kept) == G // 2 and list(kept) == sorted(set(range(G)) - set(res["order"][:G - G // 2]))
    W2c = zo.drop_pruned_columns(W_masked, kept, g)
    W1c = zo.drop_matching_rows(W1, kept, g)
    b1c = zo.drop_matching_rows(b1[:, None], kept, g)[:, 0]
    assert W2c.shape == (d_out, (G // 2) * g) and W1c.shape == ((G // 2) * g, d_in)
    full = W_masked @ X
    small = W2c @ act(W1c @ inp + b1c[:, None])
    assert np.allclose(full, small, rtol=1e-12, atol=1e-13)
    # a wrong index map (e.g. keeping the removed structures instead) does change the output
    wrong = [s for s in range(G) if s not in set(kept)]
    if len(wrong) == len(kept):
        W2w = zo.drop_pruned_columns(W_masked, wrong, g)
        assert not np.allclose(full, W2w @ act(zo.drop_matching_rows(W1, wrong, g) @ inp
                                               + zo.drop_matching_rows(b1[:, None], wrong, g)))
    with pytest.raises(ValueError):
        zo.kept_structures([0, 0], G, G - 2)


# ------------------------------------------------------------------ budgeted level selection
def random_database(rng, n_mod, max_opt):
    """Per module: decreasing run times, increasing losses (level 0 of the list = unpruned:
    loss 0; last = dropped: loss = base, time 0), as a pruning database looks."""
    n_opt = rng.integers(2, max_opt + 1, size=n_mod)
    loss = np.zeros((n_mod, max_opt), np.float32)
    time = np.zeros((n_mod, max_opt), np.float32)
    base = rng.uniform(1.0, 5.0, size=n_mod).astype(np.float32)
    for m in range(n_mod):
        k = n_opt[m]
        t = np.sort(rng.uniform(0.5, 8.0, size=k))[::-1].copy()
        t[-1] = 0.0
        e = np.sort(rng.uniform(0.0, 1.0, size=k))
        e[0], e[-1] = 0.0, 1.0
        time[m, :k] = t
        loss[m, :k] = e * base[m]
    return loss, base, time, n_opt


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_level_selection_against_exhaustive_search(seed):
    """Every combination of levels is enumerated: the dynamic programme must return a selection
    that fits the budget in units and attains the smallest cost among all that do; it must also
    fit in real time (options are rounded up)."""
    import itertools
    rng = np.random.default_rng(seed)
    n_mod, max_opt, n_buckets = 5, 4, 97
    loss, base, time, n_opt = random_database(rng, n_mod, max_opt)
    coef = rng.uniform(0.1, 3.0, size=n_mod).astype(np.float32)
    t_all = float(time[:, 0].sum())
    for frac in (1.2, 0.7, 0.45, 0.2, 0.02):
        budget = frac * t_all
        sel, cost, t_sum = zo.select_levels(loss, base, time, n_opt, coef, budget, n_buckets)
        best = np.inf
        for combo in itertools.product(*[range(k) for k in n_opt]):
            u = sum(zo.time_units(time[m, s], budget, n_buckets) for m, s in enumerate(combo))
            if u <= n_buckets:
                c = sum(float(coef[m]) * float(loss[m, s]) / float(base[m]) for m, s in enumerate(combo))
                best = min(best, c)
        assert sel is not None and np.isclose(cost, best, rtol=1e-12, atol=1e-15)
        assert t_sum <= budget * (1 + 1e-12)
        assert np.isclose(cost, sum(float(coef[m]) * float(loss[m, s]) / float(base[m])
                                    for m, s in enumerate(sel)), rtol=1e-12, atol=1e-15)
        if frac == 1.2:     # the unpruned model fits (even with every option rounded up): nothing is lost
            assert sel == [0] * n_mod and cost == 0.0


def test_level_selection_limits_and_monotonicity():
    rng = np.random.default_rng(7)
    loss, base, time, n_opt = random_database(rng, 6, 5)
    coef = np.ones(6, np.float32)
    # budget (almost) zero: only the dropped modules (time 0) fit; cost = sum of priors of 1
    sel, cost, t_sum = zo.select_levels(loss, base, time, n_opt, coef, 1e-3, 50)
    assert sel == [int(k) - 1 for k in n_opt] and np.isclose(cost, 6.0) and t_sum == 0.0
    assert np.allclose(zo.error_prior(loss[np.arange(6), n_opt - 1], base), 1.0)
    # more budget never costs more
    costs = [zo.select_levels(loss, base, time, n_opt, coef, b, 200)[1] for b in (2.0, 5.0, 9.0, 20.0, 60.0)]
    assert all(a >= b - 1e-12 for a, b in zip(costs, costs[1:]))
    # a module nobody cares about (coefficient 0) is dropped first when time is short
    coef2 = coef.copy()
    coef2[2] = 0.0
    sel2, _, _ = zo.select_levels(loss, base, time, n_opt, coef2, 0.5 * float(time[:, 0].sum()), 200)
    assert sel2[2] == n_opt[2] - 1
    # no option without run time 0 and a budget below the fastest configuration: infeasible
    time3 = time.copy()
    time3[np.arange(6), n_opt - 1] = 1.0
    assert zo.select_levels(loss, base, time3, n_opt, coef, 5.9, 60)[0] is None
    assert zo.select_levels(loss, base, time3, n_opt, coef, 6.0, 60)[0] == [int(k) - 1 for k in n_opt]


def test_mutation_search_pins():
    """No marks: nothing is ever accepted and the result is coef0's selection.  If the score is
    the cost under some coefficients c* and one step sets all coefficients to c*, that step's
    selection is optimal among everything that fits, so it is accepted (unless coef0 already
    reached that score) and no later mutation can be: final score = the optimum of c*."""
    rng = np.random.default_rng(5)
    n_mod, max_opt, n_buckets, steps = 6, 5, 120, 12
    loss, base, time, n_opt = random_database(rng, n_mod, max_opt)
    budget = 0.4 * float(time[:, 0].sum())
    coef0 = rng.uniform(0.1, 3.0, size=n_mod).astype(np.float32)
    c_star = rng.uniform(0.1, 3.0, size=n_mod).astype(np.float32)
    objective = (c_star[:, None].astype(np.float64) * (loss.astype(np.float64) / base[:, None])).astype(np.float32)
    values = rng.uniform(0.1, 3.0, size=(steps, n_mod)).astype(np.float32)
    none = np.zeros((steps, n_mod), np.uint8)
    sel0, _, _ = zo.select_levels(loss, base, time, n_opt, coef0, budget, n_buckets)
    score0 = sum(float(objective[m, s]) for m, s in enumerate(sel0))
    sel, c, score, acc = zo.search_levels(loss, base, time, n_opt, objective, coef0, budget, n_buckets,
                                          none, values)
    assert sel == sel0 and acc == 0 and np.array_equal(c, coef0) and np.isclose(score, score0)
    mask = (rng.uniform(size=(steps, n_mod)) < 0.3).astype(np.uint8)
    mask[3] = 1
    values[3] = c_star
    sel_star, cost_star, _ = zo.select_levels(loss, base, time, n_opt, c_star, budget, n_buckets)
    sel, c, score, acc = zo.search_levels(loss, base, time, n_opt, objective, coef0, budget, n_buckets,
                                          mask, values)
    assert np.isclose(score, cost_star, rtol=1e-6)        # objective was rounded to fp32
    t_sel = sum(float(time[m, s]) for m, s in enumerate(sel))
    assert t_sel <= budget
    # the score never goes up as steps are added
    scores = [zo.search_levels(loss, base, time, n_opt, objective, coef0, budget, n_buckets,
                               mask[:t], values[:t])[2] for t in range(steps + 1)]
    assert all(a >= b for a, b in zip(scores, scores[1:])) and np.isclose(scores[0], score0)
