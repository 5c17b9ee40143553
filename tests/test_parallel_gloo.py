"""Multi-rank host logic on CPU (gloo, world_size 2): layer partition, max-over-ranks timing,
gathering per-layer results.  The float64 oracle stands in for the GPU solver, so the test checks
that a layer-sharded run reproduces the single-process result layer by layer."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _layer_result(l):
    import workloads as wl
    from oracle import ziplm_oracle as zo
    sh = wl.scaled(wl.CONFIGS["c1_tiny_ffn"][0], d_col=24, d_row=6, d_latent=8, n_tokens=96,
                   n_layers=5, levels=(12, 0))
    W = wl.make_weight(sh, l).numpy()
    X = wl.make_activations(sh, l).numpy()
    res = zo.prune(W, zo.hessian(X), 1, 0.01, [12, 0])
    return dict(layer=l, order=res["order"], loss=[res["losses"][12], res["losses"][0]])


def _worker(rank, world, port, n_layers, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import torch.distributed as dist
    from paper_2302_04089_b200 import parallel as par
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b, e = par.partition_layers(n_layers, world, rank)
        local = [_layer_result(l) for l in range(b, e)]
        full = par.gather_layer_results(local, n_layers)
        slowest = par.max_over_ranks(10.0 + rank)
        # token-sharded calibration pass of layer 0: partial Hessian of this rank's tokens (the
        # oracle stands in for the accumulation kernel), one all-reduce
        import workloads as wl
        from oracle import ziplm_oracle as zo
        sh = wl.scaled(wl.CONFIGS["c1_tiny_ffn"][0], d_col=24, d_row=6, d_latent=8, n_tokens=96)
        X = wl.make_activations(sh, 0)
        tb, te = par.token_shard(96, world, rank, multiple=16)
        H = torch.from_numpy(zo.hessian_from_token_batches([X[:, tb:te].T.contiguous()])).unsqueeze(0)
        H = par.allreduce_hessian(H)
        q.put((rank, (b, e), full, slowest, (tb, te), H.numpy()))
    finally:
        dist.destroy_process_group()


def test_partition_covers_every_layer_once():
    from paper_2302_04089_b200 import parallel as par
    for n in (0, 1, 5, 12, 24):
        for world in (1, 2, 3, 8):
            spans = [par.partition_layers(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        par.partition_layers(4, 2, 2)


def test_layer_sharded_run_matches_single_process_world_size_2():
    n_layers, world = 5, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_layers, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    expect = [_layer_result(l) for l in range(n_layers)]
    spans = sorted(g[1] for g in got)
    assert spans == [(0, 2), (2, 5)]
    import workloads as wl
    from oracle import ziplm_oracle as zo
    sh = wl.scaled(wl.CONFIGS["c1_tiny_ffn"][0], d_col=24, d_row=6, d_latent=8, n_tokens=96)
    H_all = zo.hessian(wl.make_activations(sh, 0))
    assert sorted(g[4] for g in got) == [(0, 48), (48, 96)]
    for g in got:
        assert np.allclose(g[5][0], H_all, rtol=1e-12, atol=1e-12)      # partial sums add up
    assert np.array_equal(got[0][5], got[1][5])                         # ranks agree bit for bit
    for rank, span, full, slowest, _, _ in got:
        assert slowest == 11.0                      # max over ranks of 10 + rank
        assert [f["layer"] for f in full] == list(range(n_layers))
        for f, e in zip(full, expect):
            assert f["order"] == e["order"]
            assert np.allclose(f["loss"], e["loss"], rtol=1e-12)


def test_token_shards_cover_every_token_once_and_respect_sequences():
    from paper_2302_04089_b200 import parallel as par
    for n, mult in ((0, 1), (96, 16), (100, 16), (131072, 1024), (7, 3)):
        for world in (1, 2, 3, 8):
            spans = [par.token_shard(n, world, r, mult) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            assert all(b % mult == 0 for b, _ in spans if b < n)
    with pytest.raises(ValueError):
        par.token_shard(10, 2, 2)


def test_single_rank_helpers_need_no_process_group():
    from paper_2302_04089_b200 import parallel as par
    t = torch.ones(1, 2, 2)
    assert par.allreduce_hessian(t) is t
    assert par.max_over_ranks(3.5) == 3.5
    assert par.gather_layer_results([1, 2, 3], 3) == [1, 2, 3]
    with pytest.raises(ValueError):
        par.gather_layer_results([1], 3)
