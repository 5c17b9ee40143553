"""Deep parity run (not collected by pytest: several minutes of oracle time per layer).

Replays the COMPLETE removal order of whole full-size layers through the float64 oracle in
lock-step and applies the identical-order rule at every one of the 3072 (or 4096) steps, plus
the snapshot / loss tolerances at every level.  Usage on a B200:

    python tests/full_order_check.py [workload] [layers ...]        # default: c3_bert_base_fc2 0

Set ZIPLM_NEURON_PATH=stream to check the per-step streaming variant instead of the default.
"""
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import numpy as np
import torch

import workloads as wl
from oracle import ziplm_oracle as zo
from parity_util import compare_layer


def main():
    import paper_2302_04089_b200 as z
    name = sys.argv[1] if len(sys.argv) > 1 else "c3_bert_base_fc2"
    layers = [int(a) for a in sys.argv[2:]] or [0]
    shape = [s for s in wl.CONFIGS[name] if s.group_size == 1][0]
    levels = list(shape.levels)
    W = torch.stack([wl.make_weight(shape, l) for l in layers])
    H = []
    for l in layers:
        X = wl.make_activations(shape, l, "cuda")
        H.append(torch.from_numpy(zo.hessian(X).astype(np.float32)))
        del X
    H = torch.stack(H)
    out = z.prune_layers(W.cuda(), H.cuda(), 1, shape.damp_frac, levels)
    torch.cuda.synchronize()
    for i, l in enumerate(layers):
        t0 = time.time()
        rep = compare_layer(W[i].numpy(), H[i].numpy(), 1, shape.damp_frac, levels, out, i)
        print(f"{name} layer {l} variant {os.environ.get('ZIPLM_NEURON_PATH', 'default')}: "
              f"all {rep['steps']} steps pass, near ties {rep['near_ties']}, "
              f"max saliency err {rep['max_rho_err']:.2e}, snapshot err {rep['snap_err']:.2e}, "
              f"loss err {rep['loss_err']:.2e}  ({time.time() - t0:.0f} s of oracle)", flush=True)


if __name__ == "__main__":
    main()
