"""Shared test plumbing: shape conversion, planted candidates, comparisons.  No method arithmetic."""
import numpy as np
import torch

from oracle import cerberus_oracle as orc
from paper_2410_13344_b200 import synth


def oracle_shape(ms: synth.ModelShape) -> orc.Shape:
    return orc.Shape(ms.n_layers, ms.d_model, ms.n_heads, ms.head_dim, ms.mlp_dim, ms.vocab, ms.dtype,
                     ms.rope_base, ms.rms_eps)


def concat_src(layout: synth.HeadLayout):
    return [[b.concat_src_head for b in row] for row in layout.blocks]


def cpu(d):
    return {k: v.detach().cpu() for k, v in d.items()}


def deepest_path(tree: synth.Tree):
    deepest = max(range(tree.n), key=lambda v: (len(orc.root_path(tree.parent, v)), -v))
    return orc.root_path(tree.parent, deepest)


def plant_tokens(tree: synth.Tree, truth, n_emitted: int, want: int):
    """Candidate overrides (-1 = keep) that spell truth[n_emitted+1 ...] along the deepest path,
    so that `want` tokens (root included) match the true continuation."""
    out = [-1] * tree.n
    path = deepest_path(tree)
    for j, node in enumerate(path[1:want], start=1):
        if n_emitted + j < len(truth):
            out[node] = int(truth[n_emitted + j])
    return out


def oracle_planter(tree: synth.Tree, truth, lengths):
    def plant(tree_tok, step, emitted):
        ov = plant_tokens(tree, truth, len(emitted), lengths[step % len(lengths)])
        return [t if o < 0 else o for t, o in zip(tree_tok, ov)]
    return plant


def close(a: torch.Tensor, b: torch.Tensor, tol: float = 0.0) -> float:
    """Combined absolute/relative error max |a-b| / (1 + |b|); "within tol" means
    |a-b| <= tol + tol*|b| for every element (atol = rtol = tol)."""
    a, b = a.double().cpu(), b.double().cpu()
    return float(((a - b).abs() / (1.0 + b.abs())).max())


def assert_close_large(a: torch.Tensor, b: torch.Tensor, tol: float, what: str = "", outliers: float = 1e-3):
    """Comparison for tensors of 10^5..10^7 bf16-derived elements, where the per-element maximum
    sits in the far tail of the rounding noise (two correct implementations differ by a near-Gaussian
    error of sigma ~ 0.3-0.4 % of the tensor's rms, and the maximum over 10^6 elements is ~5 sigma):
      (i)   max |a-b| <= tol * max(1, max|b|)            (max-abs error relative to the tensor's scale)
      (ii)  at most `outliers` of the elements violate the per-element bound |a-b| <= tol * (1 + |b|)
      (iii) mean |a-b| <= tol/4 * max(1, rms(b))         (no systematic error)
    A wrong row, a dropped term or a mis-scaled operand breaks all three by orders of magnitude."""
    a, b = a.double().cpu(), b.double().cpu()
    e = (a - b).abs()
    scale = max(1.0, float(b.abs().max()))
    assert float(e.max()) <= tol * scale, (what, "max", float(e.max()), scale)
    frac = float((e > tol * (1.0 + b.abs())).double().mean())
    assert frac <= outliers, (what, "outlier fraction", frac)
    rms = max(1.0, float((b * b).mean().sqrt()))
    assert float(e.mean()) <= tol / 4 * rms, (what, "mean", float(e.mean()), rms)


def top2_margin(logits_row: torch.Tensor) -> float:
    v = torch.topk(logits_row.double(), 2).values
    return float(v[0] - v[1])
