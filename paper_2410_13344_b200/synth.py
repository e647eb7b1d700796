"""Seeded synthetic inputs for the Cerberus decoding step.

This module only *generates inputs*: random tensors, token ids, tree topologies
and page tables.  It holds none of the method's arithmetic (no attention, no
heads, no entropy, no acceptance, no ancestor masks) so that both the CUDA path
and the CPU oracle can be fed from it without sharing any of their own code.

Random numbers come from one counter-based generator:

    key   = splitmix64(splitmix64(seed) ^ (tensor_id << 40) ^ counter)
    u     = ((key >> 11) + 0.5) * 2**-53                 (uniform in (0, 1))
    z_i   = sqrt(-2 ln u(2i)) * cos(2 pi u(2i+1))        (Box-Muller, one per index)

so every element is addressable by (seed, tensor_id, index) and a tensor can be
produced in chunks, on any torch device, with identical bit patterns for the
integer part.  The floating-point tail (log / cos) is evaluated once, on one
device, and the resulting tensor is what both sides receive.

Seeds: base model 0, Cerberus heads 1, prompts 2 (+ sequence index), trees 3,
stand-alone attention tensors 4.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

SEED_MODEL = 0
SEED_HEADS = 1
SEED_PROMPT = 2
SEED_TREE = 3
SEED_ATTN = 4

_MASK64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Python int (mod 2**64) -> the same bit pattern as a signed 64-bit int."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLD = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of the 64-bit pattern held in an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix64_t(x: torch.Tensor) -> torch.Tensor:
    z = x + _GOLD
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def splitmix64(x: int) -> int:
    """Scalar splitmix64 finaliser on Python ints (for keys and small draws)."""
    z = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def _base_key(seed: int, tensor_id: int) -> int:
    return _s64(splitmix64(seed) ^ ((tensor_id << 40) & _MASK64))


def uniform_bits(seed: int, tensor_id: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """64 random bits (as int64 patterns) for counters start .. start+count-1."""
    ctr = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _splitmix64_t(ctr ^ _base_key(seed, tensor_id))


def uniform01(seed: int, tensor_id: int, start: int, count: int, device="cpu") -> torch.Tensor:
    bits = uniform_bits(seed, tensor_id, start, count, device)
    return (_lsr(bits, 11).to(torch.float64) + 0.5) * (2.0 ** -53)


def normal(seed: int, tensor_id: int, shape: Sequence[int], std: float = 1.0, mean: float = 0.0,
           dtype=torch.float32, device="cpu", out: Optional[torch.Tensor] = None,
           chunk: int = 1 << 24) -> torch.Tensor:
    """N(mean, std) tensor of the given shape; element i uses counters 2i, 2i+1."""
    n = int(np.prod(shape)) if len(shape) else 1
    if out is None:
        out = torch.empty(n, dtype=dtype, device=device)
    flat = out.view(-1)
    assert flat.numel() == n
    dev = flat.device
    for s in range(0, n, chunk):
        c = min(chunk, n - s)
        u = uniform01(seed, tensor_id, 2 * s, 2 * c, dev).view(c, 2)
        z = torch.sqrt(-2.0 * torch.log(u[:, 0])) * torch.cos((2.0 * math.pi) * u[:, 1])
        flat[s:s + c] = (z * std + mean).to(flat.dtype)
    return out.view(*shape)


def randint(seed: int, tensor_id: int, shape: Sequence[int], high: int, device="cpu") -> torch.Tensor:
    """Uniform integers in [0, high) as int32."""
    n = int(np.prod(shape)) if len(shape) else 1
    bits = uniform_bits(seed, tensor_id, 0, n, device)
    return (_lsr(bits, 11) % high).to(torch.int32).view(*shape)


def scalar_randint(seed: int, tensor_id: int, counter: int, high: int) -> int:
    key = splitmix64((_base_key(seed, tensor_id) ^ counter) & _MASK64)
    return (key >> 11) % high


# --------------------------------------------------------------------------
# Shapes
# --------------------------------------------------------------------------

@dataclass
class ModelShape:
    """LLaMA-architecture decoder shape (the paper's base model is Vicuna-7B)."""
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    mlp_dim: int
    vocab: int
    dtype: str = "bf16"            # "bf16" | "fp32"
    rope_base: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


def tiny_shape(dtype: str = "fp32") -> ModelShape:
    return ModelShape(4, 256, 4, 64, 688, 1024, dtype)


def shape_7b(n_layers: int = 32) -> ModelShape:
    return ModelShape(n_layers, 4096, 32, 128, 11008, 32000, "bf16")


def shape_13b(n_layers: int = 40) -> ModelShape:
    return ModelShape(n_layers, 5120, 40, 128, 13824, 32000, "bf16")


@dataclass
class HeadBlock:
    """One Resblock of a decoding head: plain, or the two-input (concat) block."""
    concat_src_head: int = -1      # -1: plain block; else the head whose same-level state is appended


@dataclass
class HeadLayout:
    """Which Resblocks each decoding head has; widths follow from the table."""
    blocks: List[List[HeadBlock]]  # [head][level]

    @property
    def n_heads(self) -> int:
        return len(self.blocks)

    @property
    def n_levels(self) -> int:
        return len(self.blocks[0])

    def widths(self, d: int) -> List[List[int]]:
        """widths[h][j] = width of head h's state entering level j (j = n_levels: FC input)."""
        L = self.n_levels
        w = [[d] * (L + 1) for _ in self.blocks]
        for j in range(L):
            for h, blks in enumerate(self.blocks):
                src = blks[j].concat_src_head
                w[h][j + 1] = w[h][j] + (w[src][j] if src >= 0 else 0)
        return w


def cerberus_layout(n_heads: int, n_levels: int = 4, concat_level: Optional[int] = None) -> HeadLayout:
    """Default layout: head 0 is plain; head i >= 1 has its two-input block at
    `concat_level` (default: the last level) reading head i-1's same-level state."""
    if concat_level is None:
        concat_level = n_levels - 1
    blocks = []
    for h in range(n_heads):
        row = [HeadBlock() for _ in range(n_levels)]
        if h >= 1:
            row[concat_level] = HeadBlock(concat_src_head=h - 1)
        blocks.append(row)
    return HeadLayout(blocks)


def medusa_layout(n_heads: int, n_levels: int = 4) -> HeadLayout:
    return HeadLayout([[HeadBlock() for _ in range(n_levels)] for _ in range(n_heads)])


# --------------------------------------------------------------------------
# Weights
# --------------------------------------------------------------------------

_T_EMBED, _T_FNORM, _T_LMHEAD = 1, 2, 3
_LAYER_BASE, _LAYER_STRIDE = 16, 16
(_L_ANORM, _L_WQ, _L_WK, _L_WV, _L_WO, _L_MNORM, _L_WG, _L_WU, _L_WD) = range(9)


def _lt(layer: int, k: int) -> int:
    return _LAYER_BASE + _LAYER_STRIDE * layer + k


def make_model(shape: ModelShape, device="cpu", seed: int = SEED_MODEL, std: float = 0.02) -> Dict[str, torch.Tensor]:
    """Random-init base model.  Projection weights N(0, std); norm gains N(1, 0.1).

    Layout (row-major, `[out][in]` like a torch Linear):
      embed [V][d]; lm_head [V][d]; final_norm [d];
      per layer l: attn_norm.l [d], wqkv.l [3d][d] (q rows, k rows, v rows),
      wo.l [d][d], mlp_norm.l [d], wgu.l [2F][d] (gate rows then up rows), wd.l [d][F].
    """
    dt = shape.torch_dtype
    d, F, V = shape.d_model, shape.mlp_dim, shape.vocab
    hd = shape.n_heads * shape.head_dim
    m: Dict[str, torch.Tensor] = {}
    m["embed"] = normal(seed, _T_EMBED, (V, d), std, dtype=dt, device=device)
    m["final_norm"] = normal(seed, _T_FNORM, (d,), 0.1, 1.0, dtype=dt, device=device)
    m["lm_head"] = normal(seed, _T_LMHEAD, (V, d), std, dtype=dt, device=device)
    for l in range(shape.n_layers):
        m[f"attn_norm.{l}"] = normal(seed, _lt(l, _L_ANORM), (d,), 0.1, 1.0, dtype=dt, device=device)
        wqkv = torch.empty(3 * hd, d, dtype=dt, device=device)
        for j, k in enumerate((_L_WQ, _L_WK, _L_WV)):
            normal(seed, _lt(l, k), (hd, d), std, out=wqkv[j * hd:(j + 1) * hd])
        m[f"wqkv.{l}"] = wqkv
        m[f"wo.{l}"] = normal(seed, _lt(l, _L_WO), (d, hd), std, dtype=dt, device=device)
        m[f"mlp_norm.{l}"] = normal(seed, _lt(l, _L_MNORM), (d,), 0.1, 1.0, dtype=dt, device=device)
        wgu = torch.empty(2 * F, d, dtype=dt, device=device)
        normal(seed, _lt(l, _L_WG), (F, d), std, out=wgu[:F])
        normal(seed, _lt(l, _L_WU), (F, d), std, out=wgu[F:])
        m[f"wgu.{l}"] = wgu
        m[f"wd.{l}"] = normal(seed, _lt(l, _L_WD), (d, F), std, dtype=dt, device=device)
    return m


def make_heads(shape: ModelShape, layout: HeadLayout, device="cpu", seed: int = SEED_HEADS,
               std: float = 0.02) -> Dict[str, torch.Tensor]:
    """Random-init decoding heads: per head h and level j a square `W.h.j [w][w]` and
    bias `b.h.j [w]` (w = the block's working width), then `fc.h [V][w_final]`.
    Biases are non-zero so that the bias path is exercised."""
    dt = shape.torch_dtype
    widths = layout.widths(shape.d_model)
    hw: Dict[str, torch.Tensor] = {}
    for h in range(layout.n_heads):
        for j in range(layout.n_levels):
            w = widths[h][j + 1]
            hw[f"W.{h}.{j}"] = normal(seed, 16 + 64 * h + 2 * j, (w, w), std, dtype=dt, device=device)
            hw[f"b.{h}.{j}"] = normal(seed, 16 + 64 * h + 2 * j + 1, (w,), std, dtype=dt, device=device)
        wf = widths[h][layout.n_levels]
        hw[f"fc.{h}"] = normal(seed, 16 + 64 * h + 63, (shape.vocab, wf), std, dtype=dt, device=device)
    return hw


def make_prompt(vocab: int, length: int, seq: int = 0, seed: int = SEED_PROMPT) -> torch.Tensor:
    return randint(seed + seq, 1, (length,), vocab)


# --------------------------------------------------------------------------
# Trees (topology is an input; both sides derive depth / ancestors themselves)
# --------------------------------------------------------------------------

@dataclass
class Tree:
    """Candidate tree.  Node 0 is the root (the LM head's own token); nodes are
    topologically ordered (parent[v] < v).  head[v] / rank[v] say which decoding
    head and which of its top-k outputs fills node v (-1 for the root)."""
    parent: np.ndarray            # int32 [n], parent[0] = -1
    head: np.ndarray              # int32 [n]
    rank: np.ndarray              # int32 [n]

    @property
    def n(self) -> int:
        return int(self.parent.shape[0])


def best_first_tree(n_nodes: int, caps: Sequence[int]) -> Tree:
    """Prefix-closed tree of rank tuples (r_1..r_m), r_l < caps[l-1], ordered by
    (sum of ranks, length, lexicographic) and cut after n_nodes - 1 candidates."""
    cands: List[Tuple[int, ...]] = []

    def rec(prefix: Tuple[int, ...]):
        m = len(prefix)
        if m == len(caps):
            return
        for r in range(caps[m]):
            t = prefix + (r,)
            cands.append(t)
            rec(t)

    rec(())
    cands.sort(key=lambda t: (sum(t), len(t), t))
    keep = cands[: max(0, n_nodes - 1)]
    index = {(): 0}
    parent, head, rank = [-1], [-1], [-1]
    for t in keep:
        index[t] = len(parent)
        parent.append(index[t[:-1]])
        head.append(len(t) - 1)
        rank.append(t[-1])
    return Tree(np.asarray(parent, np.int32), np.asarray(head, np.int32), np.asarray(rank, np.int32))


def chain_tree(n_nodes: int) -> Tree:
    p = np.arange(-1, n_nodes - 1, dtype=np.int32)
    return Tree(p, p.copy(), np.zeros(n_nodes, np.int32) - (p < 0))


def single_node_tree() -> Tree:
    return chain_tree(1)


def random_parent_tree(n_nodes: int, max_depth: int, seed: int = SEED_TREE, tree_id: int = 0,
                       n_heads: int = 0, kmax: int = 10) -> Tree:
    """Node v's parent is uniform among earlier nodes whose depth is < max_depth.
    (Depth is tracked here only to respect the cap.)  head = depth-1 and rank is a
    random index < kmax when n_heads > 0, so the tree can also be filled by a draft."""
    parent = [-1]
    depth = [0]
    for v in range(1, n_nodes):
        ok = [u for u in range(v) if depth[u] < max_depth]
        u = ok[scalar_randint(seed, 100 + tree_id, v, len(ok))]
        parent.append(u)
        depth.append(depth[u] + 1)
    head = [d - 1 for d in depth]
    rank = [-1] + [scalar_randint(seed, 200 + tree_id, v, kmax) for v in range(1, n_nodes)]
    if n_heads:
        assert max(head) < n_heads
    return Tree(np.asarray(parent, np.int32), np.asarray(head, np.int32), np.asarray(rank, np.int32))


# --------------------------------------------------------------------------
# Paged KV cache helpers (pure layout)
# --------------------------------------------------------------------------

PAGE = 16


def shuffled_page_table(n_logical: int, n_physical: int, seed: int = SEED_ATTN, table_id: int = 0,
                        first: int = 0) -> np.ndarray:
    """A permutation-based logical->physical page map: logical page i of this
    sequence lives in physical page table[i]; physical ids are distinct and drawn
    from [first, first + n_physical)."""
    assert n_logical <= n_physical
    keys = [(splitmix64((_base_key(seed, 300 + table_id) ^ i) & _MASK64), i) for i in range(n_physical)]
    perm = [i for _, i in sorted(keys)]
    return (np.asarray(perm[:n_logical], np.int32) + first).astype(np.int32)
