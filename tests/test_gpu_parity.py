"""CUDA path vs float64 oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import ziplm_oracle as zo
from parity_util import compare_layer

pytestmark = pytest.mark.gpu


def zb():
    import paper_2302_04089_b200 as z
    return z


def oracle_h32(X):
    """fp32 rounding of the oracle's 2 X X^T: the H handed to both sides (never a CUDA result)."""
    return torch.from_numpy(zo.hessian(X).astype(np.float32))


def run_case(shape, levels=None, layers=None, check_layers=None, base=True):
    z = zb()
    levels = list(shape.levels if levels is None else levels)
    W, X = wl.make_layers(shape, "cpu", layers)
    H = torch.stack([oracle_h32(X[l]) for l in range(W.shape[0])])
    out = z.prune_layers(W.cuda(), H.cuda(), shape.group_size, shape.damp_frac, levels,
                         want_base_loss=base)
    torch.cuda.synchronize()
    reports = []
    for l in (range(W.shape[0]) if check_layers is None else check_layers):
        reports.append(compare_layer(W[l].numpy(), H[l].numpy(), shape.group_size, shape.damp_frac,
                                     levels, out, l))
    return out, reports


# ------------------------------------------------------------------ Hessian (a1)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("d,N,ldx", [(64, 256, 256), (200, 1000, 1000), (130, 77 * 8, 640), (96, 8, 8)])
def test_hessian_matches_oracle(dtype, d, N, ldx):
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=d, d_latent=32, n_tokens=ldx,
                   n_layers=2, x_dtype=dtype)
    _, X = wl.make_layers(sh, "cpu")
    Xd = X.cuda()[:, :, :N]                       # pitched view: ldx >= N
    H = z.hessian_accumulate(Xd)
    torch.cuda.synchronize()
    for l in range(2):
        Ho = zo.hessian(X[l][:, :N])
        scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
        err = np.max(np.abs(H[l].cpu().double().numpy() - Ho) / scale)
        assert err < 2e-6, err
        assert torch.equal(H[l], H[l].T)
    # beta = 1 adds a second batch: 2 X X^T accumulated twice = 4 X X^T
    H2 = z.hessian_accumulate(Xd, H.clone(), beta=1.0)
    torch.cuda.synchronize()
    assert torch.allclose(H2, 2 * H, rtol=1e-6, atol=0)


def test_hessian_zero_tokens_and_bad_args():
    z = zb()
    H = torch.ones(1, 8, 8, device="cuda")
    X = torch.zeros(1, 8, 0, device="cuda")
    assert torch.equal(z.hessian_accumulate(X, H.clone(), beta=1.0), H)
    assert torch.count_nonzero(z.hessian_accumulate(X, H.clone(), beta=0.0)) == 0
    Xb = torch.zeros(1, 8, 6, device="cuda")           # pitch 6 floats = 24 B: not 16-byte pitched
    with pytest.raises(z.ZiplmError) as e:
        z.hessian_accumulate(Xb)
    assert e.value.status == z.Status.ERR_INVALID_ARG
    with pytest.raises(z.ZiplmError):
        z.hessian_accumulate(torch.zeros(1, 8, 8, device="cuda"), H.clone(), beta=0.5)


# ------------------------------------------------------------------ Hessian from token-major batches
def token_major_case(dtype, d, N, lda, L=2):
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=d, d_latent=32, n_tokens=N,
                   n_layers=L, x_dtype=dtype)
    _, X = wl.make_layers(sh, "cpu")                      # [L, d, N]
    A = torch.zeros(L, N, lda, dtype=X.dtype)
    A[:, :, :d] = X.transpose(1, 2)
    if lda > d:
        A[:, :, d:] = 7.0                                  # pitch padding must never be read
    return X, A


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("d,N,lda", [(64, 256, 64), (200, 1000, 208), (130, 613, 131), (96, 8, 96),
                                     (33, 31, 40), (257, 4099, 257), (130, 613, 132), (257, 4099, 260)])
def test_hessian_from_token_major_activations_matches_oracle(dtype, d, N, lda):
    z = zb()
    X, A = token_major_case(dtype, d, N, lda)
    Ad = A.cuda()[:, :, :d]
    H = z.hessian_accumulate_tokens(Ad)
    torch.cuda.synchronize()
    for l in range(2):
        Ho = zo.hessian(X[l])
        scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
        err = np.max(np.abs(H[l].cpu().double().numpy() - Ho) / scale)
        assert err < 2e-6, err
        assert torch.equal(H[l], H[l].T)
    # same numbers, to the bit, as the token-contiguous entry point where that one accepts the
    # layout (16-byte row pitch) and both take the same route
    if (N * X.element_size()) % 16 == 0:
        assert torch.equal(H, z.hessian_accumulate(X.cuda()))


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_hessian_streamed_batch_by_batch(dtype):
    """beta = 1 over ragged calibration batches (one of them shorter than a K block, one empty)
    against the oracle's sum of outer products over all tokens."""
    z = zb()
    d, N = 160, 1500
    X, A = token_major_case(dtype, d, N, d, L=3)
    cuts = [0, 512, 512, 531, 1100, 1500]
    Ad = A.cuda()
    H = torch.full((3, d, d), float("nan"), device="cuda")
    for b in range(len(cuts) - 1):
        part = Ad[:, cuts[b]:cuts[b + 1], :].contiguous()
        z.hessian_accumulate_tokens(part, H, beta=0.0 if b == 0 else 1.0)
    torch.cuda.synchronize()
    for l in range(3):
        Ho = zo.hessian_from_token_batches([A[l, cuts[b]:cuts[b + 1]] for b in range(len(cuts) - 1)]) \
            if l == 0 else zo.hessian(X[l])
        scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
        err = np.max(np.abs(H[l].cpu().double().numpy() - Ho) / scale)
        assert err < 2e-6, err


def test_a_bounded_wait_that_runs_out_is_reported_and_the_device_stays_usable():
    """The Hessian kernel's producer is given a poll limit of one look for its wait on a free
    pipeline stage: on a healthy input with more K blocks than stages it gives up, every role
    leaves through the abort path (issued copies and MMAs complete inside the live CTA, tensor
    memory is freed), H[l][0][0] comes back NaN and the next stage reports ZIPLM_ERR_NONFINITE.
    Nothing faults and nothing hangs; the same call works again with the default limit."""
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=64, d_latent=16, n_tokens=2048, n_layers=2)
    _, X = wl.make_layers(sh, "cpu")
    Xd = X.cuda()
    z.set_option(z.Option.SPIN_LIMIT, 1)
    try:
        H = z.hessian_accumulate(Xd)
        torch.cuda.synchronize()
    finally:
        z.set_option(z.Option.SPIN_LIMIT, 0)
    assert torch.isnan(H[:, 0, 0]).all()
    _, status = z.damped_inverse(H, 0.01)
    torch.cuda.synchronize()
    assert status.tolist() == [int(z.Status.ERR_NONFINITE)] * 2
    H = z.hessian_accumulate(Xd)
    torch.cuda.synchronize()
    Ho = zo.hessian(X[1])
    scale = np.sqrt(np.outer(np.diag(Ho), np.diag(Ho)))
    assert np.max(np.abs(H[1].cpu().double().numpy() - Ho) / scale) < 2e-6


def test_hessian_tokens_bad_args():
    z = zb()
    H = torch.ones(1, 8, 8, device="cuda")
    A0 = torch.zeros(1, 0, 8, device="cuda")
    assert torch.equal(z.hessian_accumulate_tokens(A0, H.clone(), beta=1.0), H)
    assert torch.count_nonzero(z.hessian_accumulate_tokens(A0, H.clone(), beta=0.0)) == 0
    with pytest.raises(z.ZiplmError):
        z.hessian_accumulate_tokens(torch.zeros(1, 4, 8, device="cuda"), H.clone(), beta=0.5)
    lib = z.load_library()
    a = torch.zeros(4, 8, device="cuda")
    ws = torch.empty(z.hessian_tokens_workspace_bytes(1, 8, 4, 0) + 256, dtype=torch.uint8, device="cuda")
    # row pitch smaller than the feature count
    assert lib.ziplm_hessian_accumulate_tokens(H.data_ptr(), a.data_ptr(), 0, 1, 8, 4, 7, 2.0, 0.0,
                                               ws.data_ptr(), ws.numel(), None) == z.Status.ERR_INVALID_ARG
    # workspace too small on the tensor-core route
    need = z.hessian_tokens_workspace_bytes(1, 8, 64, 0)
    assert need > 0
    a64 = torch.zeros(64, 8, device="cuda")
    assert lib.ziplm_hessian_accumulate_tokens(H.data_ptr(), a64.data_ptr(), 0, 1, 8, 64, 8, 2.0, 0.0,
                                               ws.data_ptr(), need - 256, None) == z.Status.ERR_WORKSPACE


# ------------------------------------------------------------------ damped inverse (a2, a3)
@pytest.mark.parametrize("d,L", [(64, 1), (100, 2), (256, 3), (448, 1), (827, 1), (1100, 2)])
def test_damped_inverse_matches_oracle(d, L):
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=d, d_latent=max(8, d // 4),
                   n_tokens=4 * d, n_layers=L)
    _, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(L)])
    Hinv, status = z.damped_inverse(H.cuda(), 0.01)
    torch.cuda.synchronize()
    assert torch.count_nonzero(status) == 0
    for l in range(L):
        H_lam = zo.damped(H[l].numpy(), float(np.float32(0.01)))[0]
        ref = zo.inverse_spd(H_lam)
        got = Hinv[l].cpu().numpy()
        assert np.array_equal(got, got.T)
        # float64 on both sides: forward error of an inverse is bounded by ~ cond * unit roundoff
        tol = 50 * np.linalg.cond(H_lam) * 2.2e-16
        err = np.max(np.abs(got - ref)) / np.max(np.abs(ref))
        assert err < tol, (err, tol)
        assert np.max(np.abs(got @ H_lam - np.eye(d))) < tol * 10


def test_not_positive_definite_layer_is_flagged_and_others_finish():
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c1_tiny_ffn"][0], d_col=64, d_latent=64, d_row=16, n_tokens=256,
                   n_layers=3)
    W, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(3)])
    H[1, 0, 1] = H[1, 1, 0] = 100.0 * H[1, 0, 0]         # indefinite even after 1 % damping
    Hinv, status = z.damped_inverse(H.cuda(), 0.01)
    torch.cuda.synchronize()
    assert status.tolist() == [0, int(z.Status.ERR_NOT_PD), 0]
    out = z.prune_layers(W.cuda(), H.cuda(), 1, 0.01, [32])
    torch.cuda.synchronize()
    st = out["layer_status"].tolist()
    assert st[0] == 0 and st[2] == 0 and st[1] == int(z.Status.ERR_NOT_PD)
    for l in (0, 2):
        compare_layer(W[l].numpy(), H[l].numpy(), 1, 0.01, [32], out, l)
    Hn = H.clone()
    Hn[2, 3, 3] = float("nan")
    _, status = z.damped_inverse(Hn.cuda(), 0.01)
    assert status.tolist()[2] == int(z.Status.ERR_NONFINITE) and status.tolist()[0] == 0


# ------------------------------------------------------------------ neuron path (a4 - a10)
def choose_neuron_path(z, name):
    z.set_option(z.Option.NEURON_PATH, 1 if name == "stream" else 0)
    z.set_option(z.Option.COMPACT_EVERY_BLOCK, 1 if name == "lazy_compact" else 0)


@pytest.fixture(params=["lazy", "lazy_compact", "stream"])
def neuron_path(request):
    """Run a test once per neuron-path variant: delayed rank-B updates (default where the shape
    allows it; removed positions left in place between compactions, dense tensor-core update),
    the same with a compaction after every block (gathering FMA update only), and the per-step
    streaming update."""
    z = zb()
    choose_neuron_path(z, request.param)
    yield request.param
    choose_neuron_path(z, "lazy")


def test_c1_tiny_ffn_full_config(neuron_path):
    out, reports = run_case(wl.CONFIGS["c1_tiny_ffn"][0])
    assert reports[0]["steps"] == 192


@pytest.mark.parametrize("d,r,L,levels", [
    (203, 50, 2, [203, 150, 77, 1, 0]),        # ragged widths, unpruned level, down to nothing
    (64, 7, 1, [63, 0]),
    (130, 129, 3, [65]),
    (8, 4, 2, [4]),
    (132, 30, 2, [132, 100, 99, 35, 3, 0]),    # multiple of 4: both variants; uneven block lengths
    (4, 3, 1, [3, 2, 1, 0]),
])
def test_neuron_path_ragged_shapes(d, r, L, levels, neuron_path):
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=d, d_row=r, d_latent=max(4, d // 4),
                   n_tokens=4 * d + 8, n_layers=L, levels=tuple(levels))
    run_case(sh)


def test_neuron_path_mid_size_full_depth_three_layers(neuron_path):
    """Scaled BERT-base fc2: several row blocks per step, full greedy order 768 -> 0."""
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=768, d_row=192, d_latent=192,
                   n_tokens=4096, n_layers=3, levels=tuple(range(704, -1, -64)))
    out, reports = run_case(sh)
    print(reports)


@pytest.mark.parametrize("d,check,variant", [(1536, [0, 1], "lazy"), (1536, [1], "lazy_compact"),
                                             (2048, [1], "lazy")])
def test_clustered_steps_kernel_full_depth_every_step(d, check, variant):
    """Full greedy order d -> 0 of the default path in lock-step with the oracle at widths where
    the steps kernel runs on clusters of 2 (769..1536 live positions) and 4 (1537..2048) CTAs, and
    on one CTA from 768 down: every single pick is compared, and every level's snapshot and loss.
    Both update routes of the default path are covered (dense blocks on the tensor cores with
    occasional compaction, and compaction after every block), and the exact rebuild of the state
    at 64 survivors lies inside the compared range."""
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=d, d_row=256, d_latent=d // 4,
                   n_tokens=2 * d, n_layers=2, levels=tuple(range(d - d // 8, -1, -d // 8)))
    choose_neuron_path(z, variant)
    try:
        out, reports = run_case(sh, check_layers=check)
    finally:
        choose_neuron_path(z, "lazy")
    for rep in reports:
        assert rep["steps"] == d
    print(reports)


def test_full_width_every_step_one_layer_of_3072():
    """The complete order 3072 -> 0 at the width of the BERT-base fc2 layers (few weight rows, so
    that the oracle's replay stays within minutes): clusters of 4 CTAs with full slices of 768
    positions, dense and compaction blocks at full width, the exact rebuild at 64 survivors --
    every pick, every saliency and every level compared."""
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=3072, d_row=64, d_latent=768,
                   n_tokens=6144, n_layers=2, levels=tuple(range(2560, -1, -512)))
    out, reports = run_case(sh, check_layers=[1])
    assert reports[0]["steps"] == 3072
    assert reports[0]["max_rho_err"] < 2e-5
    print(reports)


def test_cluster_of_eight_every_step_down_to_3072():
    """Width 4096 (the BERT-large fc2 layers): the steps kernel runs on clusters of 8 CTAs while
    more than 3072 positions are live, with 64 candidates per pick.  The first 1024 picks, their
    saliencies and the two levels are compared one by one (few weight rows, so that the oracle's
    replay stays within two minutes)."""
    sh = wl.scaled(wl.CONFIGS["c4_bert_large"][1], d_col=4096, d_row=64, d_latent=1024,
                   n_tokens=8192, n_layers=2, levels=(3584, 3072))
    out, reports = run_case(sh, check_layers=[0])
    assert reports[0]["steps"] == 1024
    assert reports[0]["max_rho_err"] < 2e-5
    print(reports)


def test_neuron_path_is_deterministic(neuron_path):
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=256, d_row=64, d_latent=64,
                   n_tokens=1024, n_layers=2, levels=(128, 0))
    W, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(2)]).cuda()
    a = z.prune_layers(W.cuda(), H, 1, 0.01, [128, 0])
    b = z.prune_layers(W.cuda(), H, 1, 0.01, [128, 0])
    torch.cuda.synchronize()
    assert torch.equal(a["order"], b["order"])
    assert torch.equal(a["W_snap"], b["W_snap"])


@pytest.mark.parametrize("groups", ["1", "3", "8"])
def test_layer_groups_do_not_change_the_result(groups):
    """Layers are independent problems: how many groups of them run on internal streams must not
    change a single bit of any output."""
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=320, d_row=48, d_latent=80,
                   n_tokens=1280, n_layers=9, levels=(256, 100, 0))
    W, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(9)]).cuda()
    z.set_option(z.Option.LAYER_GROUPS, 0)
    ref = z.prune_layers(W.cuda(), H, 1, 0.01, [256, 100, 0])
    torch.cuda.synchronize()
    z.set_option(z.Option.LAYER_GROUPS, int(groups))
    try:
        got = z.prune_layers(W.cuda(), H, 1, 0.01, [256, 100, 0])
        torch.cuda.synchronize()
    finally:
        z.set_option(z.Option.LAYER_GROUPS, 0)
    assert torch.count_nonzero(got["layer_status"]) == 0
    for k in ("order", "W_snap", "loss", "base_loss", "saliency"):
        assert torch.equal(ref[k], got[k]), k


@pytest.mark.parametrize("groups", [0, 3])
def test_batches_in_flight_on_two_streams_give_the_results_of_one_at_a_time(groups):
    """Calls on different streams with their own Hessian, workspace and outputs overlap on the
    device (the Hessian and inverse of one batch under the loop of the other); every output must
    be bit-identical to the one the same batch gives on its own."""
    z = zb()
    shapes = [wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=320, d_row=48, d_latent=80,
                        n_tokens=1280, n_layers=6, levels=(256, 100, 0), seed_base=8100 + 50 * b)
              for b in range(2)]
    data = [wl.make_layers(sh, "cuda") for sh in shapes]
    levels = [256, 100, 0]
    z.set_option(z.Option.LAYER_GROUPS, groups)
    try:
        alone = []
        for W, X in data:
            H = z.hessian_accumulate(X)
            alone.append((H, z.prune_layers(W, H, 1, 0.01, levels)))
            torch.cuda.synchronize()
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        start = torch.cuda.Event()
        start.record()
        together = [None, None]
        for rep in range(2):                       # two rounds, so that calls queue behind calls
            for b, (W, X) in enumerate(data):
                with torch.cuda.stream(streams[b]):
                    streams[b].wait_event(start)
                    H = z.hessian_accumulate(X)
                    together[b] = (H, z.prune_layers(W, H, 1, 0.01, levels))
        torch.cuda.synchronize()
    finally:
        z.set_option(z.Option.LAYER_GROUPS, 0)
    for b in range(2):
        assert torch.count_nonzero(together[b][1]["layer_status"]) == 0
        assert torch.equal(alone[b][0], together[b][0])
        for k in ("order", "W_snap", "loss", "base_loss", "saliency"):
            assert torch.equal(alone[b][1][k], together[b][1][k]), (b, k)
    assert not torch.equal(alone[0][1]["order"], alone[1][1]["order"])      # the batches do differ


def test_workspace_is_not_assumed_clean(neuron_path):
    """Poison the workspace with NaN bit patterns: values of unused slots never feed live ones."""
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=100, d_row=20, d_latent=25,
                   n_tokens=512, n_layers=2, levels=(50, 10))
    W, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(2)])
    ws = torch.full((z.prune_workspace_bytes(2, 20, 100, 1, 2),), 0xFF, dtype=torch.uint8, device="cuda")
    out = z.prune_layers(W.cuda(), H.cuda(), 1, 0.01, [50, 10], workspace=ws)
    torch.cuda.synchronize()
    for l in range(2):
        compare_layer(W[l].numpy(), H[l].numpy(), 1, 0.01, [50, 10], out, l)


# ------------------------------------------------------------------ block path (a4', heads)
@pytest.mark.parametrize("d,g,r,L,levels", [
    (256, 64, 64, 2, [4, 3, 2, 1, 0]),          # four heads, every head count
    (96, 2, 20, 2, [48, 40, 17, 0]),            # tiny groups, many steps
    (120, 24, 33, 1, [4, 1]),                   # group size that is no power of two, ragged rows
    (192, 64, 200, 3, [2]),
    (512, 128, 96, 2, [4, 3, 2, 1, 0]),         # 128-wide heads: four structures, every head count
    (1024, 128, 160, 2, [8, 6, 3, 0]),          # eight 128-wide heads
    (768, 96, 64, 1, [8, 5, 0]),                # width between 64 and 128
    (1024, 128, 256, 2, [8, 7, 4, 1]),          # grouped-query shape: out-projection input of 8
                                                # heads of width 128 feeding a narrow output
])
def test_block_path_small_shapes(d, g, r, L, levels):
    sh = wl.scaled(wl.CONFIGS["c2_bert_base_attn"][0], d_col=d, d_row=r, group_size=g,
                   n_tokens=4 * d + 16, n_layers=L, levels=tuple(levels))
    run_case(sh)


def test_c2_bert_base_attention_shape_three_layers():
    """Full-size attention out-projection (768 x 768, 12 heads x 64), 3 of the 12 layers."""
    sh = wl.CONFIGS["c2_bert_base_attn"][0]
    run_case(sh, layers=[0, 5, 11])


def test_block_path_with_group_size_one_agrees_with_neuron_path(neuron_path):
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=128, d_row=40, d_latent=32,
                   n_tokens=600, n_layers=2, levels=(128, 64, 0))
    W, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(2)])
    a = z.prune_layers(W.cuda(), H.cuda(), 1, 0.01, [128, 64, 0])
    z.set_option(z.Option.FORCE_BLOCK_PATH, 1)
    try:
        b = z.prune_layers(W.cuda(), H.cuda(), 1, 0.01, [128, 64, 0])
        torch.cuda.synchronize()
    finally:
        z.set_option(z.Option.FORCE_BLOCK_PATH, 0)
    assert torch.equal(a["order"], b["order"])
    assert torch.allclose(a["W_snap"], b["W_snap"], rtol=1e-4, atol=1e-7)
    assert torch.allclose(a["loss"], b["loss"], rtol=1e-4)
    for l in range(2):
        compare_layer(W[l].numpy(), H[l].numpy(), 1, 0.01, [128, 64, 0], b, l)


# ------------------------------------------------------------------ exact ties, degenerate shapes
@pytest.mark.parametrize("g", [1, 4])
def test_exact_ties_go_to_the_lowest_index(g, neuron_path):
    """Diagonal H with equal entries and columns of equal norm: every saliency ties exactly, so
    the removal order must be 0, 1, 2, ... on every path (Eq. 2 gives rho = (h + lambda) ||W_S||^2)."""
    z = zb()
    d, r, L = 32, 8, 2
    H = (3.0 * torch.eye(d))[None].repeat(L, 1, 1).contiguous()
    W = torch.ones(L, r, d) * 0.5
    G = d // g
    out = z.prune_layers(W.cuda(), H.cuda(), g, 0.01, [G // 2, 0])
    torch.cuda.synchronize()
    assert out["layer_status"].tolist() == [0] * L
    for l in range(L):
        assert out["order"][l].tolist() == list(range(G))
        compare_layer(W[l].numpy(), H[l].numpy(), g, 0.01, [G // 2, 0], out, l)


def test_single_structure_and_no_levels():
    z = zb()
    sh = wl.scaled(wl.CONFIGS["c2_bert_base_attn"][0], d_col=64, d_row=16, group_size=64,
                   n_tokens=300, n_layers=2, levels=(1, 0))
    run_case(sh)                                   # G = 1: one step removes the whole module
    W, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(2)])
    for g in (1, 64):                              # no levels requested: nothing is removed
        out = z.prune_layers(W.cuda(), H.cuda(), g, 0.01, [])
        torch.cuda.synchronize()
        assert out["layer_status"].tolist() == [0, 0]
        assert torch.all(out["order"] == -1)


# ------------------------------------------------------------------ host-side argument checks
def test_invalid_arguments_are_rejected_on_the_host():
    z = zb()
    W = torch.zeros(1, 4, 8, device="cuda")
    H = torch.eye(8, device="cuda")[None].contiguous()
    for lv in ([3, 5], [9], [-1], [4, 4]):
        with pytest.raises(z.ZiplmError) as e:
            z.prune_layers(W, H, 1, 0.01, lv)
        assert e.value.status == z.Status.ERR_INVALID_ARG
    with pytest.raises(z.ZiplmError) as e:
        z.prune_layers(W, H, 3, 0.01, [1])              # 8 % 3 != 0
    assert e.value.status == z.Status.ERR_INVALID_ARG
    with pytest.raises(z.ZiplmError) as e:
        z.prune_layers(W, H, 1, -0.5, [1])
    assert e.value.status == z.Status.ERR_INVALID_ARG
    with pytest.raises(z.ZiplmError) as e:
        z.prune_layers(W, H, 1, 0.01, [4], workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == z.Status.ERR_WORKSPACE


# ------------------------------------------------------------------ model reshaping
@pytest.mark.parametrize("d,g,r,L,level", [(256, 1, 64, 2, 100), (384, 64, 96, 3, 2), (200, 4, 33, 2, 49),
                                           (3072, 1, 40, 2, 302), (128, 1, 16, 1, 0), (128, 1, 16, 1, 128)])
def test_reshaping_is_a_bit_exact_copy_of_the_kept_structures(d, g, r, L, level):
    """Survivor list and both gathers against plain indexing, bit for bit, on the output of a real
    pruning run (snapshot read in place through its strides) and on a stand-in previous layer."""
    z = zb()
    G = d // g
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2" if g == 1 else "c2_bert_base_attn"][0], d_row=r,
                   d_col=d, d_latent=min(d, 96), n_tokens=max(2 * d, 512), n_layers=L, group_size=g)
    W, X = wl.make_layers(sh, "cpu")
    H = torch.stack([oracle_h32(X[l]) for l in range(L)])
    levels = [lv for lv in (G - 1, level) if lv < G] or [level]
    levels = sorted(set(levels), reverse=True)
    out = z.prune_layers(W.cuda(), H.cuda(), g, sh.damp_frac, levels)
    slot = levels.index(level) if level in levels else None
    kept, status = z.kept_structures(out["order"], level)
    torch.cuda.synchronize()
    assert torch.count_nonzero(status) == 0
    order = out["order"].cpu().numpy()
    prev = torch.randn(L, d, 24, generator=torch.Generator().manual_seed(5))     # e.g. FC1 [d, d_in]
    for l in range(L):
        ko = zo.kept_structures(order[l], G, level)
        assert np.array_equal(kept[l].cpu().numpy(), ko)
    if level == G:
        snap = W.cuda()                                     # nothing removed: the layer itself
    else:
        snap = out["W_snap"][:, slot]                       # strided view, read in place
    Wc = z.gather_columns(snap, kept, g)
    Pc = z.gather_rows(prev.cuda(), kept, g)
    bias = z.gather_rows(prev.cuda()[:, :, :1].contiguous(), kept, g)
    torch.cuda.synchronize()
    assert Wc.shape == (L, r, level * g) and Pc.shape == (L, level * g, 24)
    for l in range(L):
        ko = kept[l].cpu().numpy()
        assert np.array_equal(Wc[l].cpu().numpy(), zo.drop_pruned_columns(snap[l].cpu().numpy(), ko, g))
        assert np.array_equal(Pc[l].cpu().numpy(), zo.drop_matching_rows(prev[l].numpy(), ko, g))
        assert np.array_equal(bias[l].cpu().numpy(), zo.drop_matching_rows(prev[l][:, :1].numpy(), ko, g))
        if level < G:
            # the dropped columns were exactly zero: nothing of the snapshot is lost
            assert int(torch.count_nonzero(Wc[l])) == int(torch.count_nonzero(snap[l]))


def test_reshaping_rejects_a_level_the_order_does_not_reach():
    z = zb()
    order = torch.tensor([[3, 1, -1, -1], [2, 2, 0, 1]], dtype=torch.int32, device="cuda")
    kept, status = z.kept_structures(order, 2)              # two removals: fine for layer 0 only
    torch.cuda.synchronize()
    assert status.tolist() == [0, int(z.Status.ERR_INVALID_ARG)]
    assert kept[0].tolist() == [0, 2]
    _, status = z.kept_structures(order, 1)                 # three removals: layer 0 ran only two
    assert status.tolist() == [int(z.Status.ERR_INVALID_ARG)] * 2
    with pytest.raises(z.ZiplmError):
        z.kept_structures(order, 5)
    # an index outside [0, G) in a caller-made list gives zeros, never an out-of-bounds read
    M = torch.ones(1, 2, 4, device="cuda")
    bad = torch.tensor([[1, 9]], dtype=torch.int32, device="cuda")
    assert z.gather_columns(M, bad, 1).tolist() == [[[1.0, 0.0], [1.0, 0.0]]]


# ------------------------------------------------------------------ budgeted level selection
def synthetic_database(seed, n_mod, max_opt):
    """Losses / run times shaped like a pruning database: option 0 unpruned (loss 0), the last one
    the dropped module (loss = base, time 0); ragged option counts."""
    g = torch.Generator().manual_seed(seed)
    n_opt = torch.randint(2, max_opt + 1, (n_mod,), generator=g, dtype=torch.int32)
    base = torch.rand(n_mod, generator=g) * 4 + 1
    loss = torch.zeros(n_mod, max_opt)
    time = torch.zeros(n_mod, max_opt)
    for m in range(n_mod):
        k = int(n_opt[m])
        t = torch.sort(torch.rand(k, generator=g) * 7.5 + 0.5, descending=True).values
        e = torch.sort(torch.rand(k, generator=g)).values
        t[-1], e[0], e[-1] = 0.0, 0.0, 1.0
        time[m, :k], loss[m, :k] = t, e * base[m]
        time[m, k:], loss[m, k:] = -5.0, float("nan")          # padding must never be read
    return loss, base, time, n_opt


@pytest.mark.parametrize("n_mod,max_opt,n_buckets,K", [(5, 4, 97, 3), (24, 44, 1000, 6), (24, 44, 10000, 2),
                                                      (1, 2, 1, 1), (7, 255, 12000, 1)])
def test_level_selection_matches_oracle_bit_for_bit(n_mod, max_opt, n_buckets, K):
    z = zb()
    loss, base, time, n_opt = synthetic_database(11 + n_mod, n_mod, max_opt)
    g = torch.Generator().manual_seed(99)
    coef = torch.rand(K, n_mod, generator=g) * 3 + 0.05
    t_all = float(sum(time[m, 0] for m in range(n_mod)))
    for frac in (1.3, 0.5, 0.11):
        budget = frac * t_all
        out = z.select_levels(loss.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), coef.cuda(), budget,
                              n_buckets)
        torch.cuda.synchronize()
        for k in range(K):
            sel, cost, t_sum = zo.select_levels(loss.numpy(), base.numpy(), time.numpy(), n_opt.numpy(),
                                                coef[k].numpy(), budget, n_buckets)
            assert int(out["status"][k]) == 0
            assert out["selected"][k].tolist() == sel
            assert float(out["cost"][k]) == cost                         # same float64 sums, same order
            assert abs(float(out["time_sum"][k]) - t_sum) <= 1e-12 * max(t_sum, 1.0)
            assert float(out["time_sum"][k]) <= budget * (1 + 1e-12)


def test_level_selection_infeasible_budget_nan_and_bad_args():
    z = zb()
    loss, base, time, n_opt = synthetic_database(3, 4, 3)
    time2 = time.clone()
    for m in range(4):
        time2[m, int(n_opt[m]) - 1] = 1.0                     # no free option any more
    coef = torch.ones(2, 4)
    out = z.select_levels(loss.cuda(), base.cuda(), time2.cuda(), n_opt.cuda(), coef.cuda(), 3.9, 40)
    assert out["status"].tolist() == [int(z.Status.ERR_INVALID_ARG)] * 2
    assert out["selected"].flatten().tolist() == [-1] * 8
    assert zo.select_levels(loss.numpy(), base.numpy(), time2.numpy(), n_opt.numpy(), coef[0].numpy(),
                            3.9, 40)[0] is None
    out = z.select_levels(loss.cuda(), base.cuda(), time2.cuda(), n_opt.cuda(), coef.cuda(), 4.0, 40)
    assert out["status"].tolist() == [0, 0]
    bad = loss.clone()
    bad[1, 0] = float("nan")
    out = z.select_levels(bad.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), coef.cuda(), 10.0, 40)
    assert out["status"].tolist() == [int(z.Status.ERR_NONFINITE)] * 2
    with pytest.raises(z.ZiplmError) as e:
        z.select_levels(loss.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), coef.cuda(), 10.0, 12001)
    assert e.value.status == z.Status.ERR_UNSUPPORTED
    with pytest.raises(z.ZiplmError) as e:
        z.select_levels(loss.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), coef.cuda(), 0.0, 40)
    assert e.value.status == z.Status.ERR_INVALID_ARG


def test_database_to_selection_end_to_end():
    """Prune two small modules (heads and neurons) on every level of the paper's grid, feed the
    library's own losses to the selection, and compare the chosen levels with the oracle's on the
    same numbers; then reshape the chosen levels."""
    z = zb()
    attn = wl.scaled(wl.CONFIGS["c2_bert_base_attn"][0], n_layers=2, d_row=64, d_col=256, n_tokens=1024,
                     levels=wl.paper_level_grid(4, 64))
    ffn = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], n_layers=2, d_row=64, d_col=256, d_latent=64,
                    n_tokens=1024, levels=wl.paper_level_grid(256, 1))
    rows_loss, rows_time, rows_base, n_opt, outs = [], [], [], [], []
    max_opt = 1 + max(len(attn.levels), len(ffn.levels))
    for sh, full_ms, ovh in ((attn, 7.9, 0.6), (ffn, 11.9, 0.6)):
        W, X = wl.make_layers(sh, "cuda")
        out = z.prune_layers(W, z.hessian_accumulate(X), sh.group_size, sh.damp_frac, list(sh.levels))
        sizes = (sh.n_groups,) + tuple(sh.levels)                     # option 0 = unpruned
        t = wl.make_latency_table(sizes, full_ms, ovh)
        for l in range(sh.n_layers):
            lo = torch.full((max_opt,), float("nan"))
            lo[0] = 0.0
            lo[1:len(sizes)] = out["loss"][l].cpu()
            ti = torch.full((max_opt,), -1.0)
            ti[:len(sizes)] = t
            rows_loss.append(lo); rows_time.append(ti); n_opt.append(len(sizes))
            rows_base.append(out["base_loss"][l].cpu())
        outs.append((sh, out))
    loss, time = torch.stack(rows_loss), torch.stack(rows_time)
    base, n_opt = torch.stack(rows_base), torch.tensor(n_opt, dtype=torch.int32)
    coef = torch.ones(1, 4)
    budget = 0.5 * float(time[:, 0].sum())                             # a 2x speedup target
    res = z.select_levels(loss.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), coef.cuda(), budget, 10000)
    sel, cost, t_sum = zo.select_levels(loss.numpy(), base.numpy(), time.numpy(), n_opt.numpy(),
                                        coef[0].numpy(), budget, 10000)
    assert res["status"].tolist() == [0] and res["selected"][0].tolist() == sel
    assert float(res["cost"][0]) == cost and float(res["time_sum"][0]) <= budget
    assert 0.0 < cost < 4.0 and any(s > 0 for s in sel)
    # reshape the FFN modules at their chosen levels
    sh, out = outs[1]
    for l in range(2):
        s = sel[2 + l]
        if s == 0:
            continue
        lv = sh.levels[s - 1]
        kept, status = z.kept_structures(out["order"][l:l + 1].contiguous(), lv)
        Wc = z.gather_columns(out["W_snap"][l:l + 1, s - 1], kept, 1)
        assert int(status[0]) == 0 and Wc.shape == (1, sh.d_row, lv)
        assert int(torch.count_nonzero(Wc)) == int(torch.count_nonzero(out["W_snap"][l, s - 1]))


@pytest.mark.parametrize("n_mod,max_opt,n_buckets,steps", [(24, 44, 1000, 40), (5, 4, 97, 25)])
def test_mutation_search_matches_oracle_bit_for_bit(n_mod, max_opt, n_buckets, steps):
    """Three speedup targets searched in one launch against the oracle's step-by-step loop on
    the same marks and values: same accepted steps, same coefficients, same selection, same
    float64 score."""
    z = zb()
    loss, base, time, n_opt = synthetic_database(40 + n_mod, n_mod, max_opt)
    g = torch.Generator().manual_seed(7)
    S = 3
    coef0 = torch.ones(S, n_mod)
    mask = (torch.rand(S, steps, n_mod, generator=g) < 0.1).to(torch.uint8)     # 10 % in expectation
    values = torch.rand(S, steps, n_mod, generator=g) * 3 + 0.05
    objective = torch.nan_to_num(loss / base[:, None] * (torch.rand(n_mod, 1, generator=g) + 0.5), nan=0.0)
    t_all = float(sum(time[m, 0] for m in range(n_mod)))
    budgets = torch.tensor([0.8 * t_all, 0.5 * t_all, 0.1 * t_all], dtype=torch.float64)
    out = z.search_levels(loss.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), objective.cuda(),
                          coef0.cuda(), budgets.cuda(), n_buckets, mask.cuda(), values.cuda())
    torch.cuda.synchronize()
    for k in range(S):
        sel, c, score, acc = zo.search_levels(loss.numpy(), base.numpy(), time.numpy(), n_opt.numpy(),
                                              objective.numpy(), coef0[k].numpy(), float(budgets[k]),
                                              n_buckets, mask[k].numpy(), values[k].numpy())
        assert int(out["status"][k]) == 0
        assert out["selected"][k].tolist() == sel
        assert int(out["n_accepted"][k]) == acc
        assert np.array_equal(out["coef"][k].cpu().numpy(), c)
        assert float(out["objective"][k]) == score
    # no steps: the selection of coef0 itself
    out0 = z.search_levels(loss.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), objective.cuda(),
                           coef0.cuda(), budgets.cuda(), n_buckets, mask[:, :0].contiguous().cuda(),
                           values[:, :0].contiguous().cuda())
    ref = z.select_levels(loss.cuda(), base.cuda(), time.cuda(), n_opt.cuda(), coef0[:1].cuda(),
                          float(budgets[1]), n_buckets)
    assert out0["selected"][1].tolist() == ref["selected"][0].tolist()
    assert out0["n_accepted"].tolist() == [0, 0, 0]
