"""Seeded synthetic inputs for the layer-wise structured-OBS solver.

This module only draws random tensors and shapes them like the calibration activations and
weights of transformer layers (FFN second linear layer, attention output projection).  It holds
none of the pruning method's arithmetic and is the single source of inputs for both the CUDA path
and the CPU oracle: one call produces the bytes, and both sides receive the same bytes.

The random draws always come from a CPU ``torch.Generator`` so a (config, layer) pair names the
same seed tensors on every machine; the deterministic shaping (matrix product, GELU, LayerNorm)
runs on the requested device.

Recipes (stand-ins for BERT-base / BERT-large / GPT-2 calibration activations):

``ffn``   X = GELU(A Z): Z [d_lat, N] ~ N(0,1) are pre-activations' latent sources, A [d, d_lat]
          ~ N(0, 1/d_lat) mixes them to width d, exact (erf) GELU.  The d x d second moment of X
          is rank-structured because d > d_lat.
``attn``  X = LN_feat(Z) + U V / sqrt(rank): Z [d, N] ~ N(0,1), LayerNorm over the feature axis
          per token (no affine, eps 1e-5), plus a per-layer random low-rank (64) correlation.
W is N(0, 0.02^2) in both.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class LayerShape:
    """One family of same-shape layers that are pruned together."""
    name: str
    recipe: str          # "ffn" or "attn"
    n_layers: int        # L
    d_row: int           # r: output features
    d_col: int           # d: input features = prunable columns
    n_tokens: int        # N: calibration tokens
    group_size: int      # g: 1 = FFN neuron, 64 = attention head
    levels: Tuple[int, ...]  # remaining-structure counts, strictly decreasing
    d_latent: int = 0    # ffn recipe: width of the pre-activation sources
    x_dtype: str = "f32"  # "f32", "bf16" or "f16"
    seed_base: int = 0
    damp_frac: float = 0.01

    @property
    def n_groups(self) -> int:
        return self.d_col // self.group_size


def _even_levels(G: int, parts: int) -> Tuple[int, ...]:
    """parts evenly spaced remaining counts floor(G*i/parts), i = parts-1 .. 0."""
    return tuple(sorted({(G * i) // parts for i in range(parts)}, reverse=True))


def ffn_size_grid(d: int, steps: int = 42) -> Tuple[int, ...]:
    """Intermediate sizes d * 0.9^i, i = 0 .. steps, truncated to integers (Sec. 3.2, "Runtime
    awareness": relative steps of 10 % up to about 99 % sparsity).  Truncation is a reading: of the
    sizes the latency-table appendix prints for d = 3072 it reproduces 1322, 302, 130 and 76
    exactly (rounding to nearest gives 303 and 77), 1814 is printed where 0.9^5 gives 1813.98, and
    33 is i = 43."""
    return tuple(int(d * 0.9 ** i) for i in range(steps + 1))


def paper_level_grid(G: int, group_size: int) -> Tuple[int, ...]:
    """Remaining-structure counts of the database the paper builds per module (Sec. 3.2, "Runtime
    awareness"; latency-table appendix): every head count G-1 .. 0 for an attention module; for an
    FFN module the sizes of ``ffn_size_grid`` below G, repeated sizes dropped, and the dropped
    module (0).  The unpruned size (i = 0) needs no pruning run and is left out."""
    if group_size > 1:
        return tuple(range(G - 1, -1, -1))
    sizes = set(ffn_size_grid(G))
    sizes.discard(G)
    sizes.add(0)
    return tuple(sorted(sizes, reverse=True))


# The five workload families.  Names follow the model the shapes are taken from.
CONFIGS = {
    # tiny single FFN-style layer, greedy to 75 % removed, snapshots at 25/50/75 %
    "c1_tiny_ffn": [LayerShape("c1_tiny_ffn", "ffn", 1, 64, 256, 2048, 1, (192, 128, 64),
                               d_latent=256, seed_base=0)],
    # BERT-base attention out-projection, 12 layers, 12 heads x 64, every head count
    "c2_bert_base_attn": [LayerShape("c2_bert_base_attn", "attn", 12, 768, 768, 16384, 64,
                                     tuple(range(11, -1, -1)), seed_base=2000)],
    # BERT-base FFN fc2, 12 layers, neurons, 3072 -> 0 with snapshots every 256
    "c3_bert_base_fc2": [LayerShape("c3_bert_base_fc2", "ffn", 12, 768, 3072, 16384, 1,
                                    tuple(range(2816, -1, -256)), d_latent=768, seed_base=3000)],
    # BERT-large, 24 layers: attention out-projection + fc2, snapshots every 1/16
    "c4_bert_large": [
        LayerShape("c4_bert_large_attn", "attn", 24, 1024, 1024, 32768, 64,
                   tuple(range(15, -1, -1)), seed_base=4000),
        LayerShape("c4_bert_large_fc2", "ffn", 24, 1024, 4096, 32768, 1,
                   tuple(range(3840, -1, -256)), d_latent=1024, seed_base=4500),
    ],
    # GPT-2 decoder, 12 layers, bf16 activations, 10 evenly spaced sizes per module
    "c5_gpt2": [
        LayerShape("c5_gpt2_attn", "attn", 12, 768, 768, 131072, 64, _even_levels(12, 10),
                   x_dtype="bf16", seed_base=5000),
        LayerShape("c5_gpt2_mlp", "ffn", 12, 768, 3072, 131072, 1, _even_levels(3072, 10),
                   d_latent=768, x_dtype="bf16", seed_base=5500),
    ],
}


def scaled(shape: LayerShape, **kw) -> LayerShape:
    """A copy of ``shape`` with some fields replaced (used for reduced-size parity cases)."""
    return dataclasses.replace(shape, **kw)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def make_weight(shape: LayerShape, layer: int) -> torch.Tensor:
    """W [d_row, d_col] fp32 ~ N(0, 0.02^2), on the CPU."""
    g = _gen(shape.seed_base + layer)
    return torch.randn(shape.d_row, shape.d_col, generator=g, dtype=torch.float32) * 0.02


def make_activations(shape: LayerShape, layer: int, device: str = "cpu",
                     n_tokens: Optional[int] = None) -> torch.Tensor:
    """X [d_col, N] (tokens contiguous) in ``shape.x_dtype`` on ``device``."""
    N = shape.n_tokens if n_tokens is None else n_tokens
    d = shape.d_col
    g = _gen(1_000_003 * (shape.seed_base + layer) + 17)
    if shape.recipe == "ffn":
        dl = shape.d_latent
        A = torch.randn(d, dl, generator=g, dtype=torch.float32) / (dl ** 0.5)
        Z = torch.randn(dl, N, generator=g, dtype=torch.float32)
        X = torch.nn.functional.gelu(A.to(device) @ Z.to(device))
    elif shape.recipe == "attn":
        rank = 64
        Z = torch.randn(d, N, generator=g, dtype=torch.float32)
        U = torch.randn(d, rank, generator=g, dtype=torch.float32)
        V = torch.randn(rank, N, generator=g, dtype=torch.float32)
        Zd = Z.to(device)
        mu = Zd.mean(dim=0, keepdim=True)
        var = Zd.var(dim=0, unbiased=False, keepdim=True)
        X = (Zd - mu) / torch.sqrt(var + 1e-5) + (U.to(device) @ V.to(device)) / (rank ** 0.5)
    else:
        raise ValueError(f"unknown recipe {shape.recipe!r}")
    if shape.x_dtype == "bf16":
        X = X.to(torch.bfloat16)
    elif shape.x_dtype == "f16":
        X = X.to(torch.float16)
    return X.contiguous()


def make_layers(shape: LayerShape, device: str = "cpu",
                layers: Optional[List[int]] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """(W [L, r, d] fp32, X [L, d, N]) for the listed layers (default: all) on ``device``."""
    idx = list(range(shape.n_layers)) if layers is None else list(layers)
    W = torch.stack([make_weight(shape, l) for l in idx]).to(device)
    X = torch.stack([make_activations(shape, l, device) for l in idx])
    return W, X


def make_latency_table(sizes: Tuple[int, ...], full_ms: float, overhead_ms: float) -> torch.Tensor:
    """Synthetic stand-in for one column of the paper's latency table (latency-table appendix):
    run time of a module against its remaining structures, affine in the size with a fixed
    overhead, 0 for the dropped module.  The paper measures these on the target device; only the
    shape of the table (monotone, overhead-dominated at small sizes) is kept."""
    top = float(max(sizes))
    return torch.tensor([0.0 if n == 0 else overhead_ms + (full_ms - overhead_ms) * n / top
                         for n in sizes], dtype=torch.float32)
