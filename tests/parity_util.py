"""Comparison rules between the CUDA path and the float64 oracle (used by the gpu tests).

Order rule: at step t let b be the oracle's argmin, s its runner-up and p the structure the CUDA
path removed.  p == b passes; p == s passes as a near-tie when (rho_s - rho_b) < 1e-5 * rho_b;
anything else fails.  In every case the oracle then removes p, so later steps and all levels stay
comparable.  Snapshots: relative Frobenius error <= 1e-3 (exactly zero where the oracle's snapshot
is zero).  Losses: relative error <= 1e-3 (exactly zero at the unpruned level).
"""
import numpy as np

from oracle import ziplm_oracle as zo

NEAR_TIE = 1e-5
SNAP_TOL = 1e-3
LOSS_TOL = 1e-3


def compare_layer(W, H, group_size, damp_frac, levels, gpu, layer, X=None):
    """Replay the CUDA path's removal order of one layer through the oracle and compare.

    ``gpu`` is the dict returned by prune_layers (torch tensors).  Returns a report dict and
    raises AssertionError on any violation.
    """
    g = int(group_size)
    damp_frac = float(np.float32(damp_frac))       # the C ABI takes damp_frac as a float
    G = W.shape[1] // g
    n_steps = G - (min(levels) if len(levels) else G)
    order = gpu["order"][layer].cpu().numpy()
    assert int(gpu["layer_status"][layer]) == 0, f"layer_status {int(gpu['layer_status'][layer])}"
    assert np.all(order[n_steps:G] == -1)
    picked = order[:n_steps]
    assert len(set(picked.tolist())) == n_steps and picked.min(initial=0) >= 0 and picked.max(initial=0) < G
    res = zo.prune(W, H, g, damp_frac, levels, forced_order=picked, X=X)
    near, max_rho_err = 0, 0.0
    sal = gpu["saliency"][layer].cpu().numpy() if gpu.get("saliency") is not None else None
    for t in range(n_steps):
        p, b, s = int(picked[t]), res["best"][t], res["runner_up"][t]
        rb, rs = res["best_rho"][t], res["runner_up_rho"][t]
        if p != b:
            gap = (rs - rb) / rb
            assert p == s and gap < NEAR_TIE, (
                f"layer {layer} step {t}: CUDA removed {p}, oracle best {b} (rho {rb:.9g}), "
                f"runner-up {s} (rho {rs:.9g}), gap {gap:.3e}")
            near += 1
        if sal is not None:
            max_rho_err = max(max_rho_err, abs(sal[t] - res["saliency"][t]) / res["saliency"][t])
    if sal is not None:
        assert np.all(sal[n_steps:G] == 0)
        assert max_rho_err < 1e-4, f"saliency relative error {max_rho_err:.3e}"
    snap_err, loss_err = 0.0, 0.0
    for slot, lv in enumerate(levels):
        Wg = gpu["W_snap"][layer, slot].cpu().double().numpy()
        Wo = res["snapshots"][lv]
        removed = np.ones(G, bool)
        removed[picked[:G - lv]] = False
        dead_cols = np.repeat(~removed, g)
        assert np.all(Wg[:, dead_cols] == 0.0), f"level {lv}: pruned columns not exactly zero"
        no = np.linalg.norm(Wo)
        if no == 0.0:
            assert np.all(Wg == 0.0)
        else:
            e = np.linalg.norm(Wg - Wo) / no
            snap_err = max(snap_err, e)
            assert e <= SNAP_TOL, f"layer {layer} level {lv}: snapshot error {e:.3e}"
        lg, lo = float(gpu["loss"][layer, slot]), res["losses"][lv]
        if lv == G:
            assert lg == 0.0 and lo == 0.0
        else:
            e = abs(lg - lo) / lo
            loss_err = max(loss_err, e)
            assert e <= LOSS_TOL, f"layer {layer} level {lv}: loss {lg} vs oracle {lo} ({e:.3e})"
    if gpu.get("base_loss") is not None:
        bg, bo = float(gpu["base_loss"][layer]), res["base_loss"]
        assert abs(bg - bo) <= LOSS_TOL * bo, f"base loss {bg} vs {bo}"
    return dict(near_ties=near, max_rho_err=max_rho_err, snap_err=snap_err, loss_err=loss_err,
                steps=n_steps)
