"""Seeded synthetic inputs shaped like the paper's sequence-model linear layers.

This module only draws random tensors; it contains none of the method's arithmetic.  Both
the CUDA tests/benchmark and the CPU oracle's harness get their inputs from here, so the two
sides always see the same bits (bf16 rounding happens once, here, with round-to-nearest-even).

Every generator takes a ``device`` and is deterministic for a given (seed, device type, torch
version).  Large layers are drawn in row chunks so the fp32 staging never exceeds ~1 GiB.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 0x25100236


@dataclass
class LayerInputs:
    """Activations and output cotangents of one linear layer, plus optional master weights."""
    name: str
    X: torch.Tensor            # [B, T, d_in]
    dY: torch.Tensor           # [B, T, d_out]
    W: torch.Tensor | None = None   # [d_out, d_in] fp32 master weights, W ~ N(0, 1/d_in)
    meta: dict = field(default_factory=dict)

    @property
    def shape(self):
        B, T, d_in = self.X.shape
        return B, T, d_in, self.dY.shape[2]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, g, device, dtype, scale=1.0, chunk_elems=1 << 28):
    """N(0, scale^2) of ``shape`` in ``dtype``, drawn in fp32 row chunks."""
    out = torch.empty(shape, dtype=dtype, device=device)
    flat = out.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        z = torch.randn(e - s, generator=g, device=device, dtype=torch.float32)
        if scale != 1.0:
            z.mul_(scale)
        flat[s:e] = z.to(dtype)
    return out


def _student_t3(shape, g, device, dtype, scale=1.0, chunk_elems=1 << 26):
    """Student-t with 3 degrees of freedom, Z / sqrt((Z1^2+Z2^2+Z3^2)/3), times ``scale``."""
    out = torch.empty(shape, dtype=dtype, device=device)
    flat = out.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        z = torch.randn(4, e - s, generator=g, device=device, dtype=torch.float32)
        chi = (z[1:] * z[1:]).sum(0).div_(3.0).sqrt_()
        flat[s:e] = (z[0] / chi * scale).to(dtype)
    return out


def master_weights(d_out, d_in, seed, device) -> torch.Tensor:
    """fp32 W ~ N(0, 1/d_in), shape [d_out, d_in]."""
    return _normal((d_out, d_in), _gen(seed, device), device, torch.float32, scale=d_in ** -0.5)


def gaussian_layer(B, T, d_in, d_out, *, dtype=torch.bfloat16, seed=BASE_SEED, device="cpu",
                   name="gaussian", dy_scale=1.0, with_weights=False) -> LayerInputs:
    """X ~ N(0,1), dY ~ N(0, dy_scale^2) (the shape-sweep layers)."""
    g = _gen(seed, device)
    X = _normal((B, T, d_in), g, device, dtype)
    dY = _normal((B, T, d_out), g, device, dtype, scale=dy_scale)
    W = master_weights(d_out, d_in, seed + 7919, device) if with_weights else None
    return LayerInputs(name, X, dY, W, {"dist": "gaussian"})


def config1(device="cpu", seed=BASE_SEED + 1) -> LayerInputs:
    """Small fp32 layer: B=8, T=16, d_in=d_out=64, X and dY i.i.d. N(0,1), W ~ N(0,1/d_in)."""
    li = gaussian_layer(8, 16, 64, 64, dtype=torch.float32, seed=seed, device=device, name="c1",
                        with_weights=True)
    return li


def heterogeneous_layer(B, T, d_in, d_out, *, seed, device="cpu", name="hetero", frac=0.1, boost=5.0,
                        with_weights=True) -> LayerInputs:
    """bf16 MLP-shaped layer: X ~ N(0,1), dY ~ N(0,1/T); a seeded ``frac`` of the sequences has its
    dY multiplied by ``boost`` so the per-example gradients are heterogeneous."""
    g = _gen(seed, device)
    X = _normal((B, T, d_in), g, device, torch.bfloat16)
    dY32_scale = T ** -0.5
    n_boost = int(round(frac * B))
    perm = torch.randperm(B, generator=_gen(seed + 1, "cpu"))
    boosted = sorted(int(i) for i in perm[:n_boost])
    dY = torch.empty((B, T, d_out), dtype=torch.bfloat16, device=device)
    for b in range(B):
        z = torch.randn(T, d_out, generator=g, device=device, dtype=torch.float32)
        z.mul_(dY32_scale * (boost if b in boosted else 1.0))
        dY[b] = z.to(torch.bfloat16)
    W = master_weights(d_out, d_in, seed + 7919, device) if with_weights else None
    return LayerInputs(name, X, dY, W, {"dist": "hetero", "boosted": boosted})


def config2(device="cpu", seed=BASE_SEED + 2) -> LayerInputs:
    """Transformer-MLP-shaped bf16 layer: B=64, T=256, d_in=512, d_out=2048, 10% of sequences x5."""
    return heterogeneous_layer(64, 256, 512, 2048, seed=seed, device=device, name="c2")


def heavy_tailed_layer(B, T, d_in, d_out, *, seed, device="cpu", name="heavy", with_weights=True) -> LayerInputs:
    """bf16 layer with X ~ N(0,1) and dY ~ Student-t(3)/sqrt(T)."""
    g = _gen(seed, device)
    X = _normal((B, T, d_in), g, device, torch.bfloat16)
    dY = _student_t3((B, T, d_out), g, device, torch.bfloat16, scale=T ** -0.5)
    W = master_weights(d_out, d_in, seed + 7919, device) if with_weights else None
    return LayerInputs(name, X, dY, W, {"dist": "student_t3"})


def config4(device="cpu", seed=BASE_SEED + 4) -> LayerInputs:
    """Large bf16 layer: B=256, T=1024, d_in=2048, d_out=8192 (5.4 GB of inputs)."""
    return heavy_tailed_layer(256, 1024, 2048, 8192, seed=seed, device=device, name="c4")


# (B, T) points of the shape sweep with B*T <= 2^19, and the two widths.
SWEEP_BT = [(16, 32), (16, 512), (16, 4096), (128, 32), (128, 512), (128, 4096), (1024, 32), (1024, 512)]
SWEEP_D = [1024, 4096]


def config5_point(B, T, d, device="cpu", seed=BASE_SEED + 5) -> LayerInputs:
    """One point of the bf16 shape sweep: d_in = d_out = d, X and dY ~ N(0,1)."""
    return gaussian_layer(B, T, d, d, seed=seed + 131 * B + 17 * T + d, device=device,
                          name=f"c5_B{B}_T{T}_d{d}")


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """Host copy for the oracle: bf16 -> uint16 bit patterns, fp32 -> float32; shape kept."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.float32:
        return t.numpy()
    raise TypeError(f"unsupported dtype {t.dtype}")


def gather_columns(li: LayerInputs, rows_out, cols_in) -> LayerInputs:
    """Sub-layer made of the chosen output rows (columns of dY) and input columns (columns of X).
    Entry (r, c) of its statistics is entry (rows_out[r], cols_in[c]) of the full layer's: every
    output entry only depends on one column of dY and one column of X."""
    ro = torch.as_tensor(rows_out, device=li.dY.device, dtype=torch.long)
    ci = torch.as_tensor(cols_in, device=li.X.device, dtype=torch.long)
    X = li.X.index_select(2, ci).contiguous()
    dY = li.dY.index_select(2, ro).contiguous()
    W = None if li.W is None else li.W.index_select(0, ro.to(li.W.device)).index_select(1, ci.to(li.W.device)).contiguous()
    return LayerInputs(li.name + "_sub", X, dY, W, dict(li.meta))


def sample_indices(n, k, seed) -> list[int]:
    """k distinct sorted indices in [0, n), seeded; always includes 0 and n-1 when k >= 2."""
    k = min(k, n)
    rng = np.random.default_rng(seed)
    idx = set(rng.choice(n, size=k, replace=False).tolist())
    if k >= 2:
        idx = set(list(idx)[: k - 2]) | {0, n - 1}
        while len(idx) < k:
            idx.add(int(rng.integers(0, n)))
    return sorted(idx)
