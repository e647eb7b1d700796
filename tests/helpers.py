"""Shared test plumbing: shape conversion, planted candidates, comparisons.  No method arithmetic."""
import json
import os

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


def parity_stats(a: torch.Tensor, b: torch.Tensor, tol: float) -> dict:
    """Raw figures of a comparison against the oracle value b:
      max_rel   max |a-b| / (1 + |b|)      (the combined absolute/relative error; "within tol" means <= tol)
      max_abs   max |a-b|                  mean_abs  mean |a-b|
      outliers  fraction of elements with |a-b| > tol * (1 + |b|)
      rms_ref   rms of b                   max_ref   max |b|        n  element count"""
    a, b = a.double().cpu(), b.double().cpu()
    e = (a - b).abs()
    return dict(max_rel=float((e / (1.0 + b.abs())).max()), max_abs=float(e.max()), mean_abs=float(e.mean()),
                outliers=float((e > tol * (1.0 + b.abs())).double().mean()), rms_ref=float((b * b).mean().sqrt()),
                max_ref=float(b.abs().max()), n=int(b.numel()))


def record(what: str, **figures) -> None:
    """Prints one line of raw parity figures (shown with `pytest -s`) and, when the environment variable
    CERB_PARITY_LOG names a file, appends it there as JSON, so that a run leaves the measured errors behind and
    not only pass/fail."""
    line = dict(what=what, **figures)
    print("PARITY", json.dumps(line))
    path = os.environ.get("CERB_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(line) + "\n")


def assert_close_large(a: torch.Tensor, b: torch.Tensor, tol: float, what: str = "", outliers: float = 1e-3):
    """Comparison for tensors of 10^5..10^7 bf16-derived elements, where the per-element maximum
    sits in the far tail of the rounding noise (two correct implementations differ by a near-Gaussian
    error of sigma ~ 0.3-0.4 % of the tensor's rms, and the maximum over 10^6 elements is ~5 sigma):
      (i)   max |a-b| <= tol * max(1, max|b|)            (max-abs error relative to the tensor's scale)
      (ii)  at most `outliers` of the elements violate the per-element bound |a-b| <= tol * (1 + |b|)
      (iii) mean |a-b| <= tol/4 * max(1, rms(b))         (no systematic error)
    A wrong row, a dropped term or a mis-scaled operand breaks all three by orders of magnitude.
    The raw figures are recorded (see record) whether or not the assertion holds."""
    st = parity_stats(a, b, tol)
    record(what, tol=tol, allowed_outliers=outliers, **st)
    scale = max(1.0, st["max_ref"])
    assert st["max_abs"] <= tol * scale, (what, "max", st["max_abs"], scale)
    assert st["outliers"] <= outliers, (what, "outlier fraction", st["outliers"])
    assert st["mean_abs"] <= tol / 4 * max(1.0, st["rms_ref"]), (what, "mean", st["mean_abs"], st["rms_ref"])
    return st


def check_argmax_flips(node_argmax, o_logits, margin_tol: float, max_flips: int, what: str = ""):
    """Token decisions of the CUDA path against the oracle's logits: a different token is admissible only where the
    oracle scores it within margin_tol of its own best token, and at most max_flips nodes may differ.  Records the
    number of differing nodes and the largest such margin."""
    o_arg = [int(a) for a in orc.argmax_f32(o_logits)]
    margins = []
    for v, gv in enumerate(int(t) for t in node_argmax):
        if gv != o_arg[v]:
            margins.append(float(o_logits[v].max() - o_logits[v][gv]))
    record(what + " argmax flips", nodes=len(o_arg), flips=len(margins), largest_margin=max(margins, default=0.0),
           margin_tol=margin_tol, allowed=max_flips)
    assert all(m < margin_tol for m in margins), (what, margins)
    assert len(margins) <= max_flips, (what, len(margins))
    return margins


def top2_margin(logits_row: torch.Tensor) -> float:
    v = torch.topk(logits_row.double(), 2).values
    return float(v[0] - v[1])
