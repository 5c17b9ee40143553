"""The allocation-free damped inverse agrees with the ordinary one (needs a B200).

ziplm_damped_inverse_noalloc serves callers that cannot get device memory at the point of the
call (an allocator that must not be re-entered from a hook, a device budget owned by someone
else, a loop that cannot afford cudaMalloc's implicit synchronisation): its scratch is an array
inside the library.  Here it is driven through the C ABI twice in a row -- a large request first,
a smaller one second, so the second call runs over the first call's leftovers -- and each result
is compared with ziplm_damped_inverse on the same input.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import ziplm_oracle as zo

pytestmark = pytest.mark.gpu


def make_h(d, L, seed_shift):
    sh = wl.scaled(wl.CONFIGS["c3_bert_base_fc2"][0], d_col=d, d_latent=max(8, d // 4),
                   n_tokens=4 * d, n_layers=L, seed_base=7000 + seed_shift)
    _, X = wl.make_layers(sh, "cpu")
    Xd = X.double()
    return (2.0 * Xd @ Xd.transpose(1, 2)).float().cuda()


def test_noalloc_inverse_matches_the_workspace_version_twice_in_a_row():
    import paper_2302_04089_b200 as z
    for d, L, shift in ((320, 4, 0), (200, 2, 50)):
        H = make_h(d, L, shift)
        assert z.inverse_workspace_bytes(L, d) <= 12 << 20
        ref, ref_status = z.damped_inverse(H, 0.01)
        got = torch.full((L, d, d), float("nan"), dtype=torch.float64, device="cuda")
        status = torch.full((L,), -7, dtype=torch.int32, device="cuda")
        z.damped_inverse_noalloc(H, 0.01, got, status)
        torch.cuda.synchronize()
        assert status.tolist() == ref_status.tolist() == [0] * L
        g, r = got.cpu().numpy(), ref.cpu().numpy()
        # same float64 tolerance as the inverse parity test: cond * unit roundoff
        Hl = H[0].double().cpu().numpy()
        Hl = Hl + float(np.float32(0.01)) * np.mean(np.diag(Hl)) * np.eye(d)
        tol = 50 * np.linalg.cond(Hl) * 2.2e-16
        assert np.max(np.abs(g - r)) / np.max(np.abs(r)) < tol
        # and directly against the float64 oracle, layer by layer
        for l in range(L):
            Hd = zo.damped(H[l].cpu().numpy(), float(np.float32(0.01)))[0]
            ref64 = zo.inverse_spd(Hd)
            assert np.max(np.abs(g[l] - ref64)) / np.max(np.abs(ref64)) < 50 * np.linalg.cond(Hd) * 2.2e-16


def test_noalloc_inverse_rejects_requests_beyond_its_scratch():
    import paper_2302_04089_b200 as z
    d, L = 768, 1
    assert z.inverse_workspace_bytes(L, d) > 12 << 20
    H = torch.eye(d, device="cuda")[None].contiguous()
    out = torch.zeros(L, d, d, dtype=torch.float64, device="cuda")
    status = torch.zeros(L, dtype=torch.int32, device="cuda")
    with pytest.raises(z.ZiplmError) as e:
        z.damped_inverse_noalloc(H, 0.01, out, status)
    assert e.value.status == z.Status.ERR_UNSUPPORTED
    assert torch.count_nonzero(out) == 0
