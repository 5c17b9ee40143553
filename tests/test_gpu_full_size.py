"""Full-size workloads in the launch configuration the benchmark uses (needs a B200).

The float64 oracle cannot replay 3072 steps of a 3072-wide layer in test time (about 0.1 s per
step), so at full size the CUDA path is checked on
  * a lock-step replay of the first steps of some layers (identical order rule),
  * single late steps: the oracle rebuilds the exact state for the CUDA path's surviving set from
    its definition (ridge refit + direct inverse) and must agree on the pick,
  * snapshots and losses at sampled levels against the same definition,
  * properties that hold at any size: permutation order, exact zeros, monotone losses,
    loss(level 0) = ||W X||^2.
Layers that the oracle checks get the oracle's own fp32-rounded Hessian as input; the others run
on the Hessian kernel's output so that the full batch is launched.
"""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import ziplm_oracle as zo
from parity_util import NEAR_TIE, SNAP_TOL, LOSS_TOL, compare_layer

pytestmark = pytest.mark.gpu


def zb():
    import paper_2302_04089_b200 as z
    return z


HESSIAN_TOL = 2e-6      # relative to sqrt(H_ii H_jj), for fp32, bf16 and fp16 activations alike


def run_full(shape, check_layers):
    """GPU Hessian for all layers; oracle Hessian (fp32-rounded) swapped in for check_layers."""
    z = zb()
    L = shape.n_layers
    W = torch.stack([wl.make_weight(shape, l) for l in range(L)]).cuda()
    X = torch.stack([wl.make_activations(shape, l, "cuda") for l in range(L)])
    H = z.hessian_accumulate(X)
    torch.cuda.synchronize()
    H_or = {}
    for l in check_layers:
        Ho = zo.hessian(X[l])
        scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
        err = np.max(np.abs(H[l].cpu().double().numpy() - Ho) / scale)
        assert err < HESSIAN_TOL, f"Hessian layer {l}: {err:.3e}"
        H_or[l] = Ho.astype(np.float32)
        H[l].copy_(torch.from_numpy(H_or[l]))
    del X
    out = z.prune_layers(W, H, shape.group_size, shape.damp_frac, list(shape.levels))
    torch.cuda.synchronize()
    return W, H_or, out


@pytest.fixture
def neuron_variant():
    """Selects the neuron-path variant for one test and restores the default afterwards."""
    z = zb()

    def choose(path):
        z.set_option(z.Option.NEURON_PATH, 1 if path == "stream" else 0)
        z.set_option(z.Option.COMPACT_EVERY_BLOCK, 1 if path == "lazy_compact" else 0)

    yield choose
    choose("lazy")


def generic_properties(shape, out):
    G, L = shape.n_groups, shape.n_layers
    levels = list(shape.levels)
    n_steps = G - min(levels)
    assert torch.count_nonzero(out["layer_status"]) == 0
    order = out["order"].cpu().numpy()
    loss = out["loss"].cpu().double().numpy()
    base = out["base_loss"].cpu().double().numpy()
    for l in range(L):
        assert sorted(order[l, :n_steps].tolist()) == sorted(set(order[l, :n_steps].tolist()))
        assert order[l, :n_steps].min() >= 0 and order[l, :n_steps].max() < G
        assert np.all(order[l, n_steps:] == -1)
        assert np.all(np.diff(loss[l]) >= -1e-6 * np.abs(loss[l][1:]))      # levels decrease
        if levels[-1] == 0:
            assert abs(loss[l, -1] - base[l]) <= LOSS_TOL * base[l]
            assert torch.count_nonzero(out["W_snap"][l, -1]) == 0


def check_late_step(W, H32, shape, out, layer, t):
    """The CUDA path's pick at step t against Eq. 2 evaluated on the exact state of its own
    surviving set (refit definition), with the near-tie rule."""
    g, G = shape.group_size, shape.n_groups
    order = out["order"][layer].cpu().numpy()
    alive = np.ones(G, bool)
    alive[order[:t]] = False
    H_lam, _ = zo.damped(H32, float(np.float32(shape.damp_frac)))
    groups, rho = zo.saliencies_on_support(W, H_lam, np.nonzero(alive)[0], g)
    o = np.argsort(rho, kind="stable")
    b, s = int(groups[o[0]]), int(groups[o[1]]) if len(o) > 1 else int(groups[o[0]])
    p = int(order[t])
    if p != b:
        gap = (rho[o[1]] - rho[o[0]]) / rho[o[0]]
        assert p == s and gap < NEAR_TIE, f"layer {layer} step {t}: picked {p}, best {b}, gap {gap:.2e}"
    sal = float(out["saliency"][layer, t])
    rp = float(rho[np.searchsorted(groups, p)])
    assert abs(sal - rp) <= 1e-4 * rp, (sal, rp)


def check_level(W, H32, shape, out, layer, slot):
    g, G = shape.group_size, shape.n_groups
    lv = shape.levels[slot]
    order = out["order"][layer].cpu().numpy()
    alive = np.ones(G, bool)
    alive[order[:G - lv]] = False
    cols = np.nonzero(np.repeat(alive, g))[0]
    H_lam, _ = zo.damped(H32, float(np.float32(shape.damp_frac)))
    W_ref, _ = zo.refit_on_support(W, H_lam, cols)
    Wg = out["W_snap"][layer, slot].cpu().double().numpy()
    assert np.all(Wg[:, ~np.repeat(alive, g)] == 0.0)
    if lv > 0:
        e = np.linalg.norm(Wg - W_ref) / np.linalg.norm(W_ref)
        assert e <= SNAP_TOL, f"layer {layer} level {lv}: snapshot {e:.3e}"
    lo = zo.quadratic_loss(W, W_ref, H32)
    lg = float(out["loss"][layer, slot])
    assert abs(lg - lo) <= LOSS_TOL * lo, f"layer {layer} level {lv}: loss {lg} vs {lo}"


def lockstep_head(W, H32, shape, out, layer, n_steps):
    order = out["order"][layer].cpu().numpy()
    G = shape.n_groups
    res = zo.prune(W, H32, shape.group_size, float(np.float32(shape.damp_frac)), [G - n_steps],
                   forced_order=order[:n_steps])
    near = 0
    for t in range(n_steps):
        p, b, s = int(order[t]), res["best"][t], res["runner_up"][t]
        if p != b:
            gap = (res["runner_up_rho"][t] - res["best_rho"][t]) / res["best_rho"][t]
            assert p == s and gap < NEAR_TIE, f"layer {layer} step {t}: {p} vs {b}, gap {gap:.2e}"
            near += 1
        sal = float(out["saliency"][layer, t])
        assert abs(sal - res["saliency"][t]) <= 1e-5 * res["saliency"][t]
    return near


@pytest.mark.parametrize("path", ["lazy", "lazy_compact", "stream"])
def test_c3_bert_base_fc2_full_size_twelve_layers(path, neuron_variant):
    neuron_variant(path)
    shape = wl.CONFIGS["c3_bert_base_fc2"][0]
    checked = [0, 7]
    W, H_or, out = run_full(shape, checked)
    generic_properties(shape, out)
    for l in checked:
        Wl = W[l].cpu().numpy()
        lockstep_head(Wl, H_or[l], shape, out, l, 48)
        for t in (1800, 2700, 3040, 3069):
            check_late_step(Wl, H_or[l], shape, out, l, t)
        for slot in (0, 5, 10, 11):          # levels 2816, 1536, 256, 0
            check_level(Wl, H_or[l], shape, out, l, slot)


def test_c2_bert_base_attention_full_config_twelve_layers():
    shape = wl.CONFIGS["c2_bert_base_attn"][0]
    checked = [0, 4, 9]
    W, H_or, out = run_full(shape, checked)
    generic_properties(shape, out)
    for l in checked:
        compare_layer(W[l].cpu().numpy(), H_or[l], shape.group_size, shape.damp_frac,
                      list(shape.levels), out, l)


def test_c4_bert_large_both_shapes_twenty_four_layers():
    attn, fc2 = wl.CONFIGS["c4_bert_large"]
    W, H_or, out = run_full(attn, [3])
    generic_properties(attn, out)
    compare_layer(W[3].cpu().numpy(), H_or[3], attn.group_size, attn.damp_frac, list(attn.levels),
                  out, 3)
    del W, out
    torch.cuda.empty_cache()
    W, H_or, out = run_full(fc2, [11])
    generic_properties(fc2, out)
    Wl = W[11].cpu().numpy()
    lockstep_head(Wl, H_or[11], fc2, out, 11, 24)
    for t in (3000, 4000, 4093):
        check_late_step(Wl, H_or[11], fc2, out, 11, t)
    for slot in (7, 14, 15):               # levels 2048, 256, 0
        check_level(Wl, H_or[11], fc2, out, 11, slot)


def test_c5_gpt2_bf16_activations_both_shapes():
    attn, mlp = wl.CONFIGS["c5_gpt2"]
    W, H_or, out = run_full(attn, [2])
    generic_properties(attn, out)
    compare_layer(W[2].cpu().numpy(), H_or[2], attn.group_size, attn.damp_frac, list(attn.levels),
                  out, 2)
    del W, out
    torch.cuda.empty_cache()
    W, H_or, out = run_full(mlp, [6])
    generic_properties(mlp, out)
    Wl = W[6].cpu().numpy()
    lockstep_head(Wl, H_or[6], mlp, out, 6, 24)
    for t in (2000, 3050):
        check_late_step(Wl, H_or[6], mlp, out, 6, t)
    for slot in (1, 8, 9):                 # levels 2457, 307, 0
        check_level(Wl, H_or[6], mlp, out, 6, slot)


def stream_token_major(shape, n_batches):
    """The Hessian of all layers from token-major batches (one token per row, the layout a forward
    pass emits), accumulated batch by batch with beta = 1.  Returns (X [L, d, N] on the GPU, H)."""
    z = zb()
    L, N, d = shape.n_layers, shape.n_tokens, shape.d_col
    X = torch.stack([wl.make_activations(shape, l, "cuda") for l in range(L)])
    H = torch.empty(L, d, d, device="cuda")
    step = N // n_batches
    ws = None
    for b in range(n_batches):
        A = X[:, :, b * step:(b + 1) * step].transpose(1, 2).contiguous()      # [L, step, d]
        if ws is None:
            dt = 0 if A.dtype == torch.float32 else 1
            ws = torch.empty(z.hessian_tokens_workspace_bytes(L, d, step, dt) + 256,
                             dtype=torch.uint8, device="cuda")
        z.hessian_accumulate_tokens(A, H, beta=0.0 if b == 0 else 1.0, workspace=ws)
        del A
    torch.cuda.synchronize()
    return X, H


def test_paper_database_grid_from_streamed_token_major_batches():
    """The per-layer database as the paper builds it (Sec. 3.2): FFN sizes 0.9^i * 3072 down to
    about 99 % sparsity plus the dropped module, the Hessian accumulated batch by batch from
    token-major fp32 activations; and the same accumulation for bf16 activations of the GPT-2
    attention shape (131072 tokens in 16 batches)."""
    z = zb()
    base = wl.CONFIGS["c3_bert_base_fc2"][0]
    shape = wl.scaled(base, levels=wl.paper_level_grid(base.n_groups, 1))
    assert len(shape.levels) == 43
    X, H = stream_token_major(shape, 8)
    l = 5
    Ho = zo.hessian(X[l])
    scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
    err = np.max(np.abs(H[l].cpu().double().numpy() - Ho) / scale)
    assert err < HESSIAN_TOL, err
    # eight batches and one pass differ only by the rounding of seven more fp32 additions
    H1 = z.hessian_accumulate(X[l:l + 1])
    assert torch.allclose(H[l], H1[0], rtol=0, atol=4e-6 * float(H1[0].diagonal().max()))
    del X, H1
    H32 = Ho.astype(np.float32)
    H[l].copy_(torch.from_numpy(H32))
    W = torch.stack([wl.make_weight(shape, k) for k in range(shape.n_layers)]).cuda()
    out = z.prune_layers(W, H, 1, shape.damp_frac, list(shape.levels))
    torch.cuda.synchronize()
    generic_properties(shape, out)
    Wl = W[l].cpu().numpy()
    lockstep_head(Wl, H32, shape, out, l, 24)
    for slot in (0, 7, 21, 41, 42):          # sizes 2764, 1322, 302, 36, 0
        check_level(Wl, H32, shape, out, l, slot)
    # reshaping at full size: every layer's 302 survivors, columns of the snapshot (read in place)
    # and rows of a stand-in FC1, bit for bit against plain indexing
    lv, slot = 302, 21
    kept, status = z.kept_structures(out["order"], lv)
    fc1 = torch.randn(shape.n_layers, shape.d_col, 768, device="cuda",
                      generator=torch.Generator(device="cuda").manual_seed(3))
    Wc = z.gather_columns(out["W_snap"][:, slot], kept, 1)
    Fc = z.gather_rows(fc1, kept, 1)
    torch.cuda.synchronize()
    assert torch.count_nonzero(status) == 0
    order = out["order"].cpu().numpy()
    for k in range(shape.n_layers):
        ko = zo.kept_structures(order[k], shape.n_groups, lv)
        assert np.array_equal(kept[k].cpu().numpy(), ko)
        assert np.array_equal(Wc[k].cpu().numpy(),
                              zo.drop_pruned_columns(out["W_snap"][k, slot].cpu().numpy(), ko, 1))
        assert np.array_equal(Fc[k].cpu().numpy(), zo.drop_matching_rows(fc1[k].cpu().numpy(), ko, 1))
        assert int(torch.count_nonzero(Wc[k])) == int(torch.count_nonzero(out["W_snap"][k, slot]))
    del W, out, H, fc1, Wc, Fc
    torch.cuda.empty_cache()

    attn = wl.CONFIGS["c5_gpt2"][0]
    X, H = stream_token_major(attn, 16)
    for l in (0, 11):
        Ho = zo.hessian(X[l])
        scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
        err = np.max(np.abs(H[l].cpu().double().numpy() - Ho) / scale)
        assert err < HESSIAN_TOL, err
