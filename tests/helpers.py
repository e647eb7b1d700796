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


def top2_margin(logits_row: torch.Tensor) -> float:
    v = torch.topk(logits_row.double(), 2).values
    return float(v[0] - v[1])
