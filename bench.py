#!/usr/bin/env python
"""Throughput of the whole ZipLM layer-wise pruning path on synthetic BERT-base fc2 layers.

One step = one pass of the whole path over one batch of 12 same-shape layers (W 768 x 3072,
X 3072 x 16384 fp32): Hessian accumulation, damping + float64 Cholesky inverse, the full greedy
loop 3072 -> 0 neurons, and a snapshot + loss at every 256 neurons.  The metric is pruned
structures per second (12 * 3072 structures per step and per GPU).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  ``--impl reference`` times the float64 CPU oracle on a bounded
sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import workloads as wl

WORKLOAD = "c3_bert_base_fc2"
METRIC = "pruned_structures_per_sec"
UNIT = "structures/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# ------------------------------------------------------------------------------------------
# CPU oracle leg
# ------------------------------------------------------------------------------------------
def oracle_sample(shape, n_loop_steps=24):
    """Time the float64 oracle, as it stands, on one layer of the workload: full Hessian, full
    damped inverse, the first ``n_loop_steps`` greedy steps (every oracle step costs the same:
    it updates the full d x d matrix).  Returns structures/s extrapolated to the full greedy
    order of that layer, and the parts."""
    from oracle import ziplm_oracle as zo
    W = wl.make_weight(shape, 0)
    X = wl.make_activations(shape, 0, "cpu")
    t0 = time.perf_counter()
    H = zo.hessian(X)
    t1 = time.perf_counter()
    H32 = H.astype(np.float32)
    t2 = time.perf_counter()
    res = zo.prune(W.numpy(), H32, shape.group_size, float(np.float32(shape.damp_frac)),
                   [shape.n_groups - n_loop_steps], max_steps=n_loop_steps)
    t3 = time.perf_counter()
    # prune() = damping + inverse + n_loop_steps steps (+ one snapshot/loss); split by a second
    # timing of the inverse alone
    t4 = time.perf_counter()
    zo.inverse_spd(zo.damped(H32, shape.damp_frac)[0])
    t5 = time.perf_counter()
    t_h, t_inv = t1 - t0, t5 - t4
    t_step = max((t3 - t2) - t_inv, 1e-9) / n_loop_steps
    G = shape.n_groups
    t_layer = t_h + t_inv + t_step * G
    return dict(value=G / t_layer, hessian_s=t_h, inverse_s=t_inv, step_s=t_step,
                layer_s_extrapolated=t_layer, steps_timed=n_loop_steps,
                order_head=[int(v) for v in res["order"][:4]])


def cpu_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args, shape):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(args.warmup):
        oracle_sample(shape, n_loop_steps=2)
    vals, t0 = [], time.perf_counter()
    for _ in range(args.steps):
        vals.append(oracle_sample(shape, n_loop_steps=args.oracle_steps))
    dt = time.perf_counter() - t0
    v = float(np.mean([s["value"] for s in vals]))
    sample = (f"1 of {shape.n_layers} layers: full float64 Hessian + damped inverse + first "
              f"{args.oracle_steps} of {shape.n_groups} greedy steps, extrapolated to the full order")
    line = dict(impl="reference", metric=METRIC, value=v, unit=UNIT, n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * dt / max(args.steps, 1),
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic", config=dict(workload=WORKLOAD, layers=shape.n_layers,
                                              d_row=shape.d_row, d_col=shape.d_col,
                                              n_tokens=shape.n_tokens, group_size=shape.group_size),
                cpu_baseline=dict(value=v, unit=UNIT, cores=cpu_cores(), kind="oracle", sample=sample),
                e2e=dict(value=v, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        os.unlink(self.f.name)
        # samples under load: the upper half by power draw
        if sm:
            order = np.argsort(power)
            load = [sm[i] for i in order[len(order) // 2:]]
            med = float(np.median(load))
        else:
            med = None
        return dict(sm_mhz=med, sm_max_mhz=(max(smax) if smax else None), reasons=sorted(reasons),
                    samples=len(sm), power_w_max=(max(power) if power else None))


# ------------------------------------------------------------------------------------------
# CUDA leg
# ------------------------------------------------------------------------------------------
LAZY_BLOCK = 32   # steps per block of the delayed-update neuron path (BMAX in prune_lazy.cu)
LAZY_REFRESH = 64 # survivors at which that path rebuilds its state exactly (kRefresh there)
LAZY_DEAD_MAX, LAZY_DEAD_FRACTION = 128, 16   # its rule for squeezing removed positions out (kDeadMax, kDeadFraction)

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch: constants from earlier
# ncu captures of these kernels (taken on 4 of the 12 layers and scaled by 3: traffic grows in
# proportion to the layers), not measurements of this run.  Only valid for the bench workload.
NCU_TRAFFIC = {
    # k_lazy_update_aq_tc, first block at full size (12 layers, 3072 positions of which 3040 live)
    "k_lazy_update_aq_tc": dict(bytes=3 * (209.6e6 + 291.3e6), launch="n_pos = 3072, m = 32, 12 layers",
                                algorithmic=12 * (24.0 * 3040 * 3039 / 2 + 8.0 * 768 * 3040)),
    # k_lazy_update_aq, a compaction block near full size (12 layers, n_new = 2944)
    "k_lazy_update_aq": dict(bytes=3 * (162.0e6 + 217.3e6), launch="n_new = 2944, m = 32, 12 layers",
                             algorithmic=12 * 24.0 * 2944 * 2943 / 2),
    # k_dgemm_tiles, top-level product F21 = A21 M11^T
    "k_dgemm_tiles": dict(bytes=3 * (116.6e6 + 49.0e6), launch="F21 = A21 M11^T, 12 x 24 macro tiles",
                          algorithmic=None),
    # k_neuron_update, first step at full size (12 layers, n = 3071)
    "k_neuron_update": dict(bytes=343.1e6 + 281.9e6, launch="n = 3071, 12 layers",
                            algorithmic=12 * (8.0 * 768 * 3071 + 4.0 * 3071 * 3071)),
}


def lazy_update_work(L, G, levels, r=0):
    """Algorithmic work of the rank-32 update of H^-1 and Q (k_lazy_update_aq_tc in blocks that
    leave removed positions in place, k_lazy_update_aq in blocks that squeeze them out) over one
    greedy run: a launch that leaves n live structures reads the off-diagonal entries of H^-1 and
    Q once per symmetric pair and writes them at [i][j] and [j][i] (2 matrices x n(n-1)/2 pairs x
    4 B x (1 read + 2 writes)) and spends 3 fp32 FMA per pair and pending step.  In the dense
    blocks the same kernel also updates W^T: 8 B x r x n (read + write of the live weights), counted
    separately.  Rows and columns of removed positions that a dense block still carries are
    overhead, not counted here.  Block boundaries, and which blocks are dense, as in the library.
    Returns (bytes, fma, launches, bytes of W^T in the dense blocks)."""
    n, npos, slot, nbytes, fma, launches, wbytes = G, G, 0, 0.0, 0.0, 0, 0.0
    levels = [v for v in levels if v < G]
    n_min = levels[-1] if levels else G
    while n > n_min:
        stop = levels[slot] if slot < len(levels) else n_min
        if n > LAZY_REFRESH and stop < LAZY_REFRESH:
            stop = LAZY_REFRESH          # the exact rebuild of the state ends a block
        m = min(LAZY_BLOCK, n - stop)
        dead_after = npos - (n - m)
        refresh = n > LAZY_REFRESH and n - m == LAZY_REFRESH
        compact = refresh or dead_after >= LAZY_DEAD_MAX or dead_after * LAZY_DEAD_FRACTION >= npos
        n -= m
        npos = n if compact else npos
        if n > 1:
            entries = L * n * (n - 1) / 2.0
            nbytes += 24.0 * entries
            fma += 3.0 * m * entries
            launches += 1
            if not compact:
                wbytes += 8.0 * L * r * n
        if slot < len(levels) and levels[slot] == n:
            slot += 1
    return nbytes, fma, launches, wbytes


def update_bytes(L, r, G, n_removed):
    """Algorithmic bytes of the fused H^-1 / W update over the whole greedy loop: per launch
    with n live structures, L * (8 r n + 4 n^2) (read + write of the live W, read + write of one
    triangle of H^-1).  The launch at n = 1 does not exist (nothing is left to update)."""
    n = np.arange(max(2, G - n_removed + 1), G + 1, dtype=np.float64)
    return float(L * np.sum(8.0 * r * n + 4.0 * n * n)), int(len(n))


def run_ours(args, shape):
    import paper_2302_04089_b200 as z
    from paper_2302_04089_b200 import build as zbuild
    zbuild.build()

    if args.layer_groups:
        z.set_option(z.Option.LAYER_GROUPS, args.layer_groups)
    if args.compact_every_block:
        z.set_option(z.Option.COMPACT_EVERY_BLOCK, 1)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    L, r, d, N, g = shape.n_layers, shape.d_row, shape.d_col, shape.n_tokens, shape.group_size
    G = shape.n_groups
    levels = list(shape.levels)
    # every rank prunes its own 12 layers (independent problems: no collective on the data path)
    rs = wl.scaled(shape, seed_base=shape.seed_base + 100 * rank)
    W, X = wl.make_layers(rs, dev)
    torch.cuda.synchronize()
    H = torch.empty(L, d, d, dtype=torch.float32, device=dev)
    h_ws = torch.empty(max(z.hessian_workspace_bytes(L, d, N, 0), 256), dtype=torch.uint8, device=dev)
    p_ws = torch.empty(z.prune_workspace_bytes(L, r, d, g, len(levels)), dtype=torch.uint8, device=dev)
    out = None

    def step():
        nonlocal out
        z.hessian_accumulate(X, H, alpha=2.0, beta=0.0, workspace=h_ws)
        out = z.prune_layers(W, H, g, shape.damp_frac, levels, workspace=p_ws, out=out)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    assert int(torch.count_nonzero(out["layer_status"])) == 0, out["layer_status"].tolist()

    # ---- device-resident timing, one batch at a time (the latency of a step)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms_single = e0.elapsed_time(e1) / args.steps

    # ---- device-resident timing of the job: a stream of batches with B of them in flight.  The
    # calls are asynchronous and batches are independent problems, so batch k + 1 is enqueued on
    # another stream with its own Hessian, workspace and output buffers (W and X are read-only and
    # shared): its tensor-core and float64 phases then run under the bandwidth- and latency-bound
    # greedy loop of batch k.  Every step still computes everything; the timed region holds
    # exactly `steps` whole steps between two barriers.
    B = args.batches_in_flight
    if B <= 0:
        B = 1 if (args.layers or args.max_removed or args.layer_groups) else 2
    groups_per_batch = args.layer_groups if args.layer_groups else (0 if B == 1 else max(1, 6 // B))
    z.set_option(z.Option.LAYER_GROUPS, groups_per_batch)
    slots = [dict(H=H, h_ws=h_ws, p_ws=p_ws, out=out, stream=torch.cuda.Stream() if B > 1 else None)]
    for _ in range(1, B):
        slots.append(dict(H=torch.empty_like(H), h_ws=torch.empty_like(h_ws), p_ws=torch.empty_like(p_ws),
                          out=None, stream=torch.cuda.Stream()))

    def run_batches(n_steps):
        cur = torch.cuda.current_stream()
        if B == 1:
            for _ in range(n_steps):
                step()
            return
        start = torch.cuda.Event()
        start.record(cur)
        for k in range(n_steps):
            sl = slots[k % B]
            with torch.cuda.stream(sl["stream"]):
                if k < B:
                    sl["stream"].wait_event(start)
                z.hessian_accumulate(X, sl["H"], alpha=2.0, beta=0.0, workspace=sl["h_ws"])
                sl["out"] = z.prune_layers(W, sl["H"], g, shape.damp_frac, levels, workspace=sl["p_ws"],
                                           out=sl["out"])
        for sl in slots[:min(B, n_steps)]:
            cur.wait_stream(sl["stream"])

    run_batches(max(args.warmup, B))
    barrier()
    for sl in slots:
        if sl["out"] is not None:
            assert int(torch.count_nonzero(sl["out"]["layer_status"])) == 0
            assert torch.equal(sl["out"]["order"], out["order"])     # same input, same result
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = z.launch_count()
    barrier()
    e0.record()
    run_batches(args.steps)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1) / args.steps
    launches = (z.launch_count() - launches0) // max(args.steps, 1)
    clocks = sampler.stop() if rank == 0 else None
    for sl in slots[1:]:
        sl.clear()
    del slots
    torch.cuda.empty_cache()
    z.set_option(z.Option.LAYER_GROUPS, args.layer_groups)

    # ---- end to end through the same calls with host buffers
    Wh = W.cpu().pin_memory()
    Xh = X.cpu().pin_memory()
    host_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory()
                for k, v in out.items() if k in ("W_snap", "loss", "base_loss", "order", "layer_status")}
    h2d = Wh.numel() * 4 + Xh.numel() * Xh.element_size()
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())

    # A stream of batches through the same public calls: every step uploads its own W and X from
    # pinned memory and downloads its own results, all inside the timed region, but on streams of
    # their own and with two sets of device buffers, so that the upload of step k+1 and the
    # download of step k-1 run under the compute of step k (PCIe is full duplex).  Within a step X
    # goes up in chunks of layers and the Hessian of a chunk is enqueued as soon as its
    # activations have arrived.
    up_stream, down_stream = torch.cuda.Stream(), torch.cuda.Stream()
    n_chunks = min(4, L)
    bounds = [L * c // n_chunks for c in range(n_chunks + 1)]
    Wd, Xd = [W, torch.empty_like(W)], [X, torch.empty_like(X)]
    outs = [out, None]
    compute_done, down_done = [None, None], [None, None]

    def e2e_step(k):
        b = k & 1
        cur = torch.cuda.current_stream()
        arrived = []
        with torch.cuda.stream(up_stream):
            if compute_done[b] is not None:
                up_stream.wait_event(compute_done[b])     # step k-2 no longer reads this buffer set
            Wd[b].copy_(Wh, non_blocking=True)
            for c in range(n_chunks):
                lo, hi = bounds[c], bounds[c + 1]
                Xd[b][lo:hi].copy_(Xh[lo:hi], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(up_stream)
                arrived.append(ev)
        if down_done[b] is not None:
            cur.wait_event(down_done[b])                  # the results of step k-2 have left outs[b]
        for c in range(n_chunks):
            lo, hi = bounds[c], bounds[c + 1]
            cur.wait_event(arrived[c])
            z.hessian_accumulate(Xd[b][lo:hi], H[lo:hi], alpha=2.0, beta=0.0, workspace=h_ws)
        outs[b] = z.prune_layers(Wd[b], H, g, shape.damp_frac, levels, workspace=p_ws, out=outs[b])
        done = torch.cuda.Event()
        done.record(cur)
        compute_done[b] = done
        with torch.cuda.stream(down_stream):
            down_stream.wait_event(done)
            for name, v in host_out.items():
                v.copy_(outs[b][name], non_blocking=True)
            left = torch.cuda.Event()
            left.record(down_stream)
            down_done[b] = left

    e2e_steps = 0 if args.skip_e2e else max(1, min(args.steps, 10))
    ms_e2e = ms_e2e_single = float("nan")
    if e2e_steps:
        for k in range(2):
            e2e_step(k)
        torch.cuda.current_stream().wait_stream(down_stream)
        barrier()
        compute_done, down_done = [None, None], [None, None]
        e0.record()
        up_stream.wait_stream(torch.cuda.current_stream())
        for k in range(e2e_steps):
            e2e_step(k)
        torch.cuda.current_stream().wait_stream(down_stream)
        e1.record()
        barrier()
        ms_e2e = e0.elapsed_time(e1) / e2e_steps
        # the same leg for a single batch (nothing to overlap with but its own Hessian)
        compute_done, down_done = [None, None], [None, None]
        e0.record()
        up_stream.wait_stream(torch.cuda.current_stream())
        e2e_step(0)
        torch.cuda.current_stream().wait_stream(down_stream)
        e1.record()
        torch.cuda.synchronize()
        ms_e2e_single = e0.elapsed_time(e1)
    out = outs[0]
    del Wd, Xd, outs
    torch.cuda.empty_cache()

    # ---- one more step with per-phase event timing (roofline of the dominant kernel), and one
    # with the per-step streaming update selected, whose fused H^-1 / W kernel is reported too
    # (layer groups are run back to back here, so that a kernel's time is its own)
    z.set_option(z.Option.LAYER_GROUPS, 1)
    step()
    torch.cuda.synchronize()
    e0.record()
    step()
    e1.record()
    torch.cuda.synchronize()
    ms_one_group = e0.elapsed_time(e1)
    z.profile_begin()
    step()
    torch.cuda.synchronize()
    phases = z.profile_end()
    phases_stream = {"update": (0.0, 0)}
    if not args.skip_stream_leg:
        z.set_option(z.Option.NEURON_PATH, 1)
        step()
        z.profile_begin()
        step()
        torch.cuda.synchronize()
        phases_stream = z.profile_end()
        z.set_option(z.Option.NEURON_PATH, 0)
    z.set_option(z.Option.LAYER_GROUPS, args.layer_groups)

    # ---- the Hessian from token-major activations (one token per row, the layout a forward pass
    # emits): one call on the whole calibration set, and eight calibration batches with beta = 1
    tok = None
    if not args.skip_extras:
        A = X.transpose(1, 2).contiguous()
        Ht = torch.empty_like(H)
        t_ws = torch.empty(z.hessian_tokens_workspace_bytes(L, d, N, 0) + 256, dtype=torch.uint8,
                           device=dev)
        nb = 8
        parts = [A[:, N * b // nb:N * (b + 1) // nb, :].contiguous() for b in range(nb)]

        def whole():
            z.hessian_accumulate_tokens(A, Ht, beta=0.0, workspace=t_ws)

        def batched():
            for b in range(nb):
                z.hessian_accumulate_tokens(parts[b], Ht, beta=0.0 if b == 0 else 1.0, workspace=t_ws)

        def plain():
            z.hessian_accumulate(X, Ht, beta=0.0, workspace=h_ws)

        tok = {}
        for name, fn in (("feature_major_ms", plain), ("token_major_ms", whole),
                         ("token_major_8_batches_ms", batched)):
            for _ in range(2):
                fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(5):
                fn()
            e1.record()
            torch.cuda.synchronize()
            tok[name] = e0.elapsed_time(e1) / 5
        whole()
        torch.cuda.synchronize()
        tok["max_abs_diff_vs_feature_major"] = float((Ht - H).abs().max())
        del A, parts, Ht, t_ws

    # ---- reshaping the whole database: survivors, compacted snapshot and compacted previous layer
    # (a stand-in FC1 of shape [d, r]) for every level
    reshape = None
    if not args.skip_extras:
        prev = torch.randn(L, d, r, device=dev)

        def reshape_all():
            moved = 0
            for slot, lv in enumerate(levels):
                kept, _ = z.kept_structures(out["order"], lv)
                z.gather_columns(out["W_snap"][:, slot], kept, g)
                z.gather_rows(prev, kept, g)
                moved += L * (2 * 4 * r * lv * g) * 2 + L * 4 * (G - lv + lv)
            return moved

        reshape_all()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(3):
            moved = reshape_all()
        e1.record()
        torch.cuda.synchronize()
        rs_ms = e0.elapsed_time(e1) / 3
        reshape = dict(ms=rs_ms, levels=len(levels), algorithmic_bytes=moved,
                       achieved_gbs=moved / (rs_ms * 1e-3) / 1e9,
                       note="ziplm_kept_structures + ziplm_gather_columns (snapshot read in place) + "
                            "ziplm_gather_rows (stand-in FC1 [d_col, d_row]) for every level of the "
                            "database; output buffers allocated by torch inside the timed region")
        del prev

    # ---- budgeted level selection on a database of the paper's size: 24 modules (12 attention,
    # 12 FFN), the paper's level grid, 10^4 time buckets; 1024 coefficient vectors per launch, and
    # the 1000-step mutation search for 148 speedup targets at once (one CTA each)
    select = None
    if not args.skip_extras:
        gsel = torch.Generator().manual_seed(1)
        grids = [wl.paper_level_grid(12, 64), wl.paper_level_grid(G, 1)]
        max_opt = 1 + max(len(x) for x in grids)
        n_mod = 24
        s_loss = torch.zeros(n_mod, max_opt)
        s_time = torch.full((n_mod, max_opt), -1.0)
        s_nopt = torch.zeros(n_mod, dtype=torch.int32)
        for m in range(n_mod):
            sizes = ((12,) if m % 2 == 0 else (G,)) + grids[m % 2]
            k = len(sizes)
            s_nopt[m] = k
            s_time[m, :k] = wl.make_latency_table(sizes, 7.9 if m % 2 == 0 else 11.9, 0.6)
            # priors rise as the module shrinks: the bench layer's own loss curve where it has one
            frac = torch.tensor([1.0 - n / sizes[0] for n in sizes])
            s_loss[m, :k] = frac ** 2 * (0.5 + torch.rand(1, generator=gsel))
        s_base = torch.ones(n_mod)
        Ksel, S, n_steps, n_buckets = 1024, 148, 1000, 10000
        coefs = (torch.rand(Ksel, n_mod, generator=gsel) * 3 + 0.05).to(dev)
        dl, db, dt_, dn = s_loss.to(dev), s_base.to(dev), s_time.to(dev), s_nopt.to(dev)
        budget = 0.5 * float(s_time[:, 0].sum())
        ws_sel = torch.empty(z.select_workspace_bytes(Ksel, n_mod, n_buckets) + 256, dtype=torch.uint8,
                             device=dev)
        z.select_levels(dl, db, dt_, dn, coefs, budget, n_buckets, workspace=ws_sel)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(3):
            res = z.select_levels(dl, db, dt_, dn, coefs, budget, n_buckets, workspace=ws_sel)
        e1.record()
        torch.cuda.synchronize()
        sel_ms = e0.elapsed_time(e1) / 3
        assert int(torch.count_nonzero(res["status"])) == 0
        del ws_sel
        mask = (torch.rand(S, n_steps, n_mod, generator=gsel) < 0.1).to(torch.uint8).to(dev)
        vals = (torch.rand(S, n_steps, n_mod, generator=gsel) * 3 + 0.05).to(dev)
        budgets = (torch.linspace(0.08, 0.9, S, dtype=torch.float64) * float(s_time[:, 0].sum())).to(dev)
        obj = (dl * (torch.rand(n_mod, 1, generator=gsel) + 0.5).to(dev)).contiguous()
        coef0 = torch.ones(S, n_mod, device=dev)
        e0.record()
        sres = z.search_levels(dl, db, dt_, dn, obj, coef0, budgets, n_buckets, mask, vals)
        e1.record()
        torch.cuda.synchronize()
        search_ms = e0.elapsed_time(e1)
        assert int(torch.count_nonzero(sres["status"])) == 0
        inner = float(sum(int(k) for k in s_nopt)) * (n_buckets + 1)
        select = dict(modules=n_mod, max_options=max_opt, n_buckets=n_buckets,
                      select_candidates=Ksel, select_ms=sel_ms,
                      selections_per_sec=Ksel / (sel_ms * 1e-3),
                      select_option_evals_per_sec=Ksel * inner / (sel_ms * 1e-3),
                      search_targets=S, search_steps=n_steps, search_ms=search_ms,
                      search_option_evals_per_sec=S * (n_steps + 1) * inner / (search_ms * 1e-3),
                      mean_accepted=float(sres["n_accepted"].float().mean()),
                      note="ziplm_select_levels / ziplm_search_levels on a synthetic database of the "
                           "paper's size (latency table: affine stand-in); an option evaluation is one "
                           "float64 add + compare against a shared-memory value row")
        del mask, vals

    # ---- the other workload families, one timed pass each (Hessian and pruning separately): the
    # head path on BERT-base / BERT-large / GPT-2 attention shapes, BERT-large fc2, and the GPT-2
    # shapes from 131072 bf16 tokens
    others = None
    if not args.skip_extras and rank == 0:
        others = {}
        del X, H, h_ws, p_ws
        torch.cuda.empty_cache()
        for fam, idx in (("c2_bert_base_attn", 0), ("c4_bert_large", 0), ("c4_bert_large", 1),
                         ("c5_gpt2", 0), ("c5_gpt2", 1)):
            sh = wl.CONFIGS[fam][idx]
            Wo = torch.stack([wl.make_weight(sh, l) for l in range(sh.n_layers)]).to(dev)
            Xo = torch.stack([wl.make_activations(sh, l, dev) for l in range(sh.n_layers)])
            torch.cuda.synchronize()
            lv = list(sh.levels)
            Ho = torch.empty(sh.n_layers, sh.d_col, sh.d_col, dtype=torch.float32, device=dev)

            def hess():
                z.hessian_accumulate(Xo, Ho, alpha=2.0, beta=0.0)

            res = [None]

            def prune():
                res[0] = z.prune_layers(Wo, Ho, sh.group_size, sh.damp_frac, lv, out=res[0])

            t = {}
            for nm, fn in (("hessian_ms", hess), ("prune_ms", prune)):
                fn()
                torch.cuda.synchronize()
                e0.record()
                for _ in range(2):
                    fn()
                e1.record()
                torch.cuda.synchronize()
                t[nm] = e0.elapsed_time(e1) / 2
            assert int(torch.count_nonzero(res[0]["layer_status"])) == 0
            z.set_option(z.Option.LAYER_GROUPS, 1)
            z.profile_begin()
            prune()
            torch.cuda.synchronize()
            ph = z.profile_end()
            z.set_option(z.Option.LAYER_GROUPS, args.layer_groups)
            removed = sh.n_layers * (sh.n_groups - min(lv))
            tot = t["hessian_ms"] + t["prune_ms"]
            esz = 2 if sh.x_dtype != "f32" else 4
            tri_flop = float(sh.n_layers) * sh.d_col * sh.d_col * sh.n_tokens      # lower triangle
            others[sh.name] = dict(
                layers=sh.n_layers, d_row=sh.d_row, d_col=sh.d_col, n_tokens=sh.n_tokens,
                group_size=sh.group_size, x_dtype=sh.x_dtype, levels=len(lv),
                hessian_ms=t["hessian_ms"], prune_ms=t["prune_ms"],
                structures_per_sec=removed / (tot * 1e-3), layers_per_sec=sh.n_layers / (tot * 1e-3),
                prune_structures_per_sec=removed / (t["prune_ms"] * 1e-3),
                hessian_useful_tflops=tri_flop / (t["hessian_ms"] * 1e-3) / 1e12,
                hessian_x_gb_per_s=sh.n_layers * sh.d_col * sh.n_tokens * esz / (t["hessian_ms"] * 1e-3) / 1e9,
                phases_ms={k: round(v[0], 3) for k, v in ph.items() if v[1] > 0})
            del Wo, Xo, Ho, res
            torch.cuda.empty_cache()

    from paper_2302_04089_b200.parallel import max_over_ranks
    ms, ms_e2e = max_over_ranks(ms), max_over_ranks(ms_e2e)
    n_removed = G - min(levels)
    structures = world * L * n_removed
    value = structures / (ms * 1e-3)
    e2e_value = structures / (ms_e2e * 1e-3)

    if rank == 0:
        full_workload = args.layers == 0 and args.max_removed == 0
        peak, peak_src = load_peaks()
        upd_ms, upd_n = phases_stream["update"]
        alg_bytes, n_launch = update_bytes(L, r, G, n_removed)
        achieved = alg_bytes / (upd_ms * 1e-3) / 1e9 if upd_ms > 0 else 0.0
        # float64 factor products of the damped inverse.
        # Algorithmic work per layer: d^3/3 flop for the Cholesky factor and d^3/3 for its inverse.
        prod_ms, prod_n = phases.get("inverse_products", (0.0, 0))
        prod_flop = L * (2.0 / 3.0) * float(d) ** 3
        prod_tflops = prod_flop / (prod_ms * 1e-3) / 1e12 if prod_ms > 0 else 0.0
        fp64_peak = 37.0      # TFLOP/s, measured with a register-only loop of the float64 mma instruction
        aq_ms, aq_n = phases.get("lazy_update_aq", (0.0, 0))
        aq_only_bytes, aq_fma, _, aq_w_bytes = lazy_update_work(L, G, levels, r)
        aq_bytes = aq_only_bytes + aq_w_bytes
        aq_gbs = aq_bytes / (aq_ms * 1e-3) / 1e9 if aq_ms > 0 else 0.0
        fma_peak = 35.7                                # fp32 TFMA/s measured with a register-only FMA loop
        hs_ms, _ = phases.get("hessian", (0.0, 0))
        hs_useful = float(L) * d * d * N                      # lower triangle: d^2 N flop per layer
        f16_peak = 2225.0     # TFLOP/s: tcgen05.mma kind::f16, M = 128, N >= 128, operands in shared memory
        line = dict(
            metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps,
            warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak",
            vs_baseline=None, dtype="f32", data="synthetic",
            config=dict(workload=WORKLOAD if (args.layers == 0 and args.max_removed == 0)
                        else WORKLOAD + " (reduced: profiling aid)", layers=L, d_row=r, d_col=d, n_tokens=N, group_size=g,
                        levels=len(levels), damp_frac=shape.damp_frac,
                        l2_policy="inputs_exceed_l2 (X 2.4 GB and about 2 GB of loop state per step)",
                        parallelism=f"layer-sharded x{world}, no collective",
                        batches_in_flight=B, layer_groups_per_batch=groups_per_batch if groups_per_batch else 6),
            layers_per_sec=world * L / (ms * 1e-3),
            single_batch=dict(ms_per_step=ms_single, value=structures / (ms_single * 1e-3), unit=UNIT,
                              note="the same steps one at a time on one stream (six layer groups on "
                                   "internal streams): the latency of a step.  `value` is the "
                                   "throughput of a stream of independent batches with "
                                   "batches_in_flight of them enqueued concurrently on streams of "
                                   "their own (own Hessian, workspace and outputs; W and X shared, "
                                   "read-only): the tensor-core and float64 phases of one batch run "
                                   "under the bandwidth- and latency-bound greedy loop of the other"),
            phases_ms={k: round(v[0], 3) for k, v in phases.items() if v[1] > 0},
            phases_note="per-phase CUDA-event times of one extra step with the layer groups run "
                        f"back to back, one batch (that step: {ms_one_group:.1f} ms); the timed steps "
                        "overlap layer groups on internal streams and batches on the caller's streams",
            e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                     ms_per_step=ms_e2e, steps=e2e_steps, single_batch_ms=ms_e2e_single,
                     note="a stream of batches through the public calls: every step uploads its own "
                          "W, X from pinned memory and downloads its own results inside the timed "
                          "region; two sets of device buffers and separate copy streams let the "
                          "upload of step k+1 and the download of step k-1 run under the compute of "
                          "step k; single_batch_ms is one such step on its own"),
            gpu_launches=int(launches),
            clocks=clocks,
            roofline_inverse_products=dict(kernel="k_dgemm_tiles + k_dgemm_pair", bound="alu", achieved=prod_tflops, peak=fp64_peak,
                          unit="TFLOP/s", frac=prod_tflops / fp64_peak,
                          traffic=NCU_TRAFFIC["k_dgemm_tiles"]["bytes"] if full_workload else None,
                          traffic_note=NCU_TRAFFIC["k_dgemm_tiles"],
                          launches=prod_n, avg_launch_us=1e3 * prod_ms / max(prod_n, 1),
                          algorithmic_flop_per_step=prod_flop,
                          peak_source="measured: register-only loop of mma.sync.m8n8k4.f64, 37.0 TFLOP/s "
                                      "(plain FMA loop 36.5; nominal 148 SMs x 64 lanes x 2 x 1.965 GHz "
                                      "= 37.2)",
                          note="float64 tile products of the Cholesky factor and its inverse "
                               "(2/3 d^3 flop per layer)"),
            roofline=dict(kernel="k_lazy_update_aq_tc (dense blocks) + k_lazy_update_aq (compaction blocks)",
                          bound="hbm", achieved=aq_gbs, peak=peak,
                          unit="GB/s", frac=aq_gbs / peak,
                          traffic=NCU_TRAFFIC["k_lazy_update_aq_tc"]["bytes"] if full_workload else None,
                          traffic_note=dict(dense=NCU_TRAFFIC["k_lazy_update_aq_tc"],
                                            compaction=NCU_TRAFFIC["k_lazy_update_aq"]),
                          peak_source=peak_src,
                          launches=aq_n, avg_launch_us=1e3 * aq_ms / max(aq_n, 1),
                          algorithmic_bytes_per_step=aq_bytes,
                          algorithmic_bytes_note="24 B per symmetric pair of live structures of H^-1 and Q "
                                                 f"({aq_only_bytes:.4g} B) + 8 B per live weight of W^T in "
                                                 f"the dense blocks ({aq_w_bytes:.4g} B)",
                          symmetric=dict(bytes_per_step=aq_only_bytes * 16.0 / 24.0 + aq_w_bytes,
                                         achieved=(aq_only_bytes * 16.0 / 24.0 + aq_w_bytes) / (aq_ms * 1e-3) / 1e9
                                         if aq_ms > 0 else 0.0,
                                         frac=((aq_only_bytes * 16.0 / 24.0 + aq_w_bytes) / (aq_ms * 1e-3) / 1e9 / peak)
                                         if aq_ms > 0 else 0.0,
                                         note="one read and one write per unique entry of the two "
                                              "symmetric matrices (16 B per pair); the kernel's own "
                                              "count (24 B) includes the second, mirrored store that "
                                              "lets the steps kernel read a pivot column as a row"),
                          note="rank-32 update of H^-1 and Q, the operation with the largest summed "
                               "time in the timed path (the phase also holds the small kernel that "
                               "packs the pending vectors for the tensor cores).  About three blocks "
                               "in four at full width leave removed positions in place and run dense "
                               "128 x 128 tiles on tcgen05 (bf16 x 3 split of the rank-32 operands, TMA "
                               "loads, direct and mirrored stores), W^T included as extra tiles of the "
                               "same kernel; the others squeeze removed positions "
                               "out with 4-byte gathers on the CUDA cores.  A stand-alone kernel "
                               "with this traffic shape (one read, a direct and a mirrored store per "
                               "entry) and no arithmetic reaches 5.0-5.2 TB/s on this part, 3.3-3.9 "
                               "TB/s with the gather in front",
                          alu=dict(achieved_tfma=aq_fma / (aq_ms * 1e-3) / 1e12 if aq_ms > 0 else 0.0,
                                   peak_tfma=fma_peak,
                                   note="3 fp32 FMA per entry and pending step; peak = measured "
                                        "71.4 TFLOP/s fp32 (nominal 148 SMs x 128 lanes x 1.965 GHz "
                                        "= 74.4)")),
            steps_kernel=dict(kernel="k_lazy_steps", bound="latency",
                              launches=phases.get("lazy_steps", (0.0, 0))[1],
                              ms=phases.get("lazy_steps", (0.0, 0))[0],
                              us_per_greedy_step=1e3 * phases.get("lazy_steps", (0.0, 0))[0] / max(n_removed, 1),
                              note="32 sequential greedy steps per launch on a cluster of 4, 2 or 1 CTAs "
                                   "per layer; a chain of long-latency instructions (cluster barrier, "
                                   "shuffles, shared-memory loads, float64 conversions), second to the "
                                   "rank-32 update in summed time and without a throughput roofline"),
            roofline_hessian=dict(
                kernel="k_row_absmax_split + k_syrk_tc<split>", bound="tensor",
                achieved=3.0 * hs_useful / (hs_ms * 1e-3) / 1e12 if hs_ms > 0 else 0.0, peak=f16_peak,
                unit="TFLOP/s", frac=(3.0 * hs_useful / (hs_ms * 1e-3) / 1e12 / f16_peak) if hs_ms > 0 else 0.0,
                useful_tflops=hs_useful / (hs_ms * 1e-3) / 1e12 if hs_ms > 0 else 0.0,
                traffic=None, ms=hs_ms,
                peak_source="measured on this part: one thread per SM issuing tcgen05.mma kind::f16 "
                            "128 x 128 x 16 back to back from shared-memory operands, 2222 TFLOP/s at "
                            "N = 128 and 2228 at N = 256 (1484 at N = 64; kind::tf32 the same way: "
                            "1115); nominal 2.25 PFLOP/s",
                note="fp32 activations: every feature row is scaled by a power of two and split "
                     "into two fp16 parts, every product is three fp16 MMAs (x1*x1, x1*x2, x2*x1), "
                     "so the tensor-pipe work is 3 x the useful d^2 N flop per layer; the time is "
                     "that of the whole call, the row-maximum and split pre-pass included; the "
                     "kernel is bound by its L2 -> shared-memory operand traffic (64 KB per K "
                     "block of 64 tokens against 816 clocks of MMAs)"),
            roofline_streaming_update=dict(
                kernel="k_neuron_update", bound="hbm", achieved=achieved, peak=peak, unit="GB/s",
                frac=achieved / peak,
                traffic=NCU_TRAFFIC["k_neuron_update"]["bytes"] if full_workload else None,
                traffic_note=NCU_TRAFFIC["k_neuron_update"], peak_source=peak_src, launches=upd_n,
                avg_launch_us=1e3 * upd_ms / max(upd_n, 1), algorithmic_bytes_per_step=alg_bytes,
                note="per-step fused H^-1/W update of the streaming variant "
                     "(option NEURON_PATH = 1), timed in a separate step",
                phases_ms={k: round(v[0], 3) for k, v in phases_stream.items() if v[1] > 0}),
        )
        if tok is not None:
            tok["note"] = ("ziplm_hessian_accumulate_tokens on the same 12 x 3072 x 16384 fp32 "
                           "activations stored one token per row; the transposing pre-pass replaces "
                           "the split pre-pass (4 B read, 8 B written per element either way)")
            line["hessian_token_major"] = tok
        if reshape is not None:
            line["reshape_database"] = reshape
        if select is not None:
            line["level_selection"] = select
        if others is not None:
            line["other_workloads"] = others
            line["other_workloads_note"] = (
                "one call each, inputs resident, mean of 2 after 1 warm-up; hessian_useful_tflops "
                "counts d^2 N flop per layer (the lower triangle); phases_ms from one more pruning "
                "call with the layer groups run back to back")
        if world == 1 and not args.no_cpu_baseline:
            s = oracle_sample(shape, n_loop_steps=args.oracle_steps)
            line["cpu_baseline"] = dict(
                value=s["value"], unit=UNIT, cores=cpu_cores(), kind="oracle",
                sample=(f"1 of {L} layers: full float64 Hessian ({s['hessian_s']:.1f} s) + damped "
                        f"inverse ({s['inverse_s']:.1f} s) + first {s['steps_timed']} of {G} greedy "
                        f"steps ({s['step_s'] * 1e3:.0f} ms each), extrapolated to the full order"))
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--oracle-steps", type=int, default=24)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: use only this many of the workload's layers")
    ap.add_argument("--max-removed", type=int, default=0,
                    help="profiling aid: stop the greedy loop after this many removals")
    ap.add_argument("--compact-every-block", action="store_true",
                    help="delayed-update path: squeeze removed positions out after every block "
                         "(the gathering CUDA-core update only; profiling aid)")
    ap.add_argument("--batches-in-flight", type=int, default=0,
                    help="independent batches enqueued concurrently on streams of their own in the "
                         "timed region (1: one batch at a time; default 2, or 1 together with the "
                         "profiling aids --layers, --max-removed and --layer-groups)")
    ap.add_argument("--layer-groups", type=int, default=0,
                    help="profiling aid: number of layer groups on internal streams (0 = library default; "
                         "1 runs them back to back, so that a profiler's per-kernel times add up)")
    ap.add_argument("--skip-e2e", action="store_true", help="profiling aid: no host-buffer leg")
    ap.add_argument("--skip-extras", action="store_true",
                    help="profiling aid: no token-major Hessian / reshaping / level-selection legs")
    ap.add_argument("--skip-stream-leg", action="store_true",
                    help="profiling aid: do not time the per-step streaming variant")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    shape = wl.CONFIGS[WORKLOAD][0]
    if args.layers > 0:
        shape = wl.scaled(shape, n_layers=args.layers)
    if args.max_removed > 0:
        keep = shape.n_groups - args.max_removed
        shape = wl.scaled(shape, levels=tuple(v for v in shape.levels if v > keep) + (keep,))
    if args.impl == "reference":
        run_reference(args, shape)
    else:
        if args.warmup < 3:
            args.warmup = 3          # timing rule: at least three warm-up steps
        run_ours(args, shape)


if __name__ == "__main__":
    main()
