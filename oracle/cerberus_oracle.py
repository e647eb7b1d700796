"""CPU oracle for the Cerberus decoding step (arxiv 2410.13344).

THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  It is a plain, slow,
float64 restatement of what one decoding step computes, written from the
paper.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import it; the CUDA library never does, and the two share no code.

What each function follows:

  resblock / concat_resblock   Section 4.1, the two displayed equations
                               (SiLU applied to the sum  W h + b + h).
  heads_forward                Section 4.1 prose: every head is Resblocks plus
                               one FC layer; the two-input block reads the
                               neighbouring head's Resblock state; all heads
                               advance level by level ("start simultaneously").
  gate_entropy / gate_mode     Section 4.2 equations and Algorithm 1: softmax
                               over the components of the last hidden state,
                               entropy in bits, S > T selects auto-regression.
  forward_full                 Algorithm 1's embedding / TL_i / LH for a LLaMA-
                               architecture decoder (Section 5.1, "Models"),
                               textbook causal attention, no cache.
  tree_attention               Section 1 / 3.1 "tree verification": node i sees
                               the prefix and its own root-to-i path; written as
                               ordinary attention over that explicit sequence.
  accept_longest               Section 3.1: candidates are verified to find the
                               tokens to accept; the rule used is strict greedy
                               matching, by enumeration of every root-to-node path.
  step / cerberus_greedy       Algorithm 1, then commit of the accepted tokens.

Readings of points the paper leaves open (all shared with the CUDA path by
specification, not by code):
  * concat block: W is square over the concatenated width, so the head's width
    grows after it; which level holds it and whose state it reads come from a
    layout table (default: last level, previous head, same level).  The paper's
    only drawing of this wiring is not available, so these readings have no
    external pin: PARITY UNPINNED for the placement/width reading of the
    two-input block (its arithmetic is pinned by closed forms and by the
    no-concat case reducing to the plain block).
  * Resblocks have a bias, the heads' FC and the base model do not.
  * h_last is the final-norm output at the last committed position.
  * S == T takes the parallel path.
  * node 0 of the tree is the LM head's own token and is always accepted; the
    argmax at the last accepted node becomes the next step's root.
  * RoPE position of a node = committed length + depth; its KV slot = committed
    length + node index; accepted nodes are moved to consecutive slots.
  * bf16 models: values are rounded to bf16 exactly at: every norm output, q and
    k after RoPE, v, the attention output, the SwiGLU output.  Everything else
    (the residual stream, accumulation, softmax, logits, head states, entropy)
    is unrounded.  fp32 models: no rounding at all (the oracle stays in float64).
  * Integer decisions (argmax, top-k) are taken on logits cast to float32, the
    precision the kernels decide in; ties go to the lower token id.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

F64 = torch.float64

MODE_PAR = 0
MODE_AR = 1


def rb(x: torch.Tensor, act: str) -> torch.Tensor:
    """Round to the activation storage type at a rounding point ("bf16") or not at all."""
    if act == "bf16":
        return x.to(torch.bfloat16).to(F64)
    return x


def f64(t: torch.Tensor) -> torch.Tensor:
    return t.to(F64)


# --------------------------------------------------------------------------
# Elementary pieces
# --------------------------------------------------------------------------

def silu(x: torch.Tensor) -> torch.Tensor:
    return x / (1.0 + torch.exp(-x))


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    ms = (x * x).mean(dim=-1, keepdim=True)
    return x / torch.sqrt(ms + eps) * gain


def rope(x: torch.Tensor, pos: Sequence[int], base: float) -> torch.Tensor:
    """Rotate-half rotary embedding.  x: [T][H][Dh]; component i pairs with i + Dh/2."""
    T, H, Dh = x.shape
    half = Dh // 2
    inv_freq = torch.tensor([base ** (-2.0 * i / Dh) for i in range(half)], dtype=F64)
    ang = torch.tensor(list(pos), dtype=F64)[:, None] * inv_freq[None, :]      # [T][half]
    c, s = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * c - x2 * s, x2 * c + x1 * s], dim=-1)


def argmax_f32(logits: torch.Tensor) -> torch.Tensor:
    """Row-wise argmax decided in float32; ties -> lowest id."""
    return torch.argmax(logits.to(torch.float32), dim=-1)


def topk_ids(logits: torch.Tensor, k: int) -> np.ndarray:
    """Top-k token ids of one logit vector by a full sort on (value desc, id asc), in float32."""
    v = logits.to(torch.float32).numpy()
    ids = np.arange(v.shape[0])
    order = np.lexsort((ids, -v))
    return order[:k].astype(np.int64)


def linear(x: torch.Tensor, W: torch.Tensor) -> torch.Tensor:
    """A bias-free dense layer of the base model (Algorithm 1, TL_i / LH): x [M][K], W [N][K] -> x W^T."""
    return f64(x) @ f64(W).T


# --------------------------------------------------------------------------
# Decoding heads (Section 4.1)
# --------------------------------------------------------------------------

def resblock(h: torch.Tensor, W: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """Output = SiLU((W h + b) + h)."""
    return silu((W @ h + b) + h)


def concat_resblock(h_i: torch.Tensor, h_prev: torch.Tensor, W: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """h = Concat(h_i, h_{i-1});  Output = SiLU((W h + b) + h)."""
    h = torch.cat([h_i, h_prev], dim=-1)
    return silu((W @ h + b) + h)


def heads_forward(h_last: torch.Tensor, heads: Dict[str, torch.Tensor], concat_src: List[List[int]]) -> List[torch.Tensor]:
    """Logits of every decoding head from the last hidden state.

    concat_src[h][j] = -1 for a plain block at level j of head h, else the head
    whose state *entering level j* is concatenated.  All heads step through the
    levels together, so a two-input block never waits for another head to finish."""
    n_heads = len(concat_src)
    n_levels = len(concat_src[0])
    state = [f64(h_last).clone() for _ in range(n_heads)]
    for j in range(n_levels):
        new = []
        for h in range(n_heads):
            W, b = f64(heads[f"W.{h}.{j}"]), f64(heads[f"b.{h}.{j}"])
            src = concat_src[h][j]
            if src < 0:
                new.append(resblock(state[h], W, b))
            else:
                new.append(concat_resblock(state[h], state[src], W, b))
        state = new
    return [f64(heads[f"fc.{h}"]) @ state[h] for h in range(n_heads)]


# --------------------------------------------------------------------------
# Entropy gate (Section 4.2, Algorithm 1)
# --------------------------------------------------------------------------

def gate_entropy(h_last: torch.Tensor) -> float:
    """P = Softmax(h);  S = -sum_i P_i log2 P_i, with 0 log 0 = 0."""
    h = f64(h_last)
    e = torch.exp(h - h.max())
    p = e / e.sum()
    nz = p > 0
    return float(-(p[nz] * torch.log2(p[nz])).sum())


def gate_mode(S: float, T: float) -> int:
    """Algorithm 1: S > T -> auto-regressive decoding, otherwise parallel decoding."""
    return MODE_AR if S > T else MODE_PAR


# --------------------------------------------------------------------------
# Base model (Algorithm 1: embedding, TL_1..N, LH)
# --------------------------------------------------------------------------

@dataclass
class Shape:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    mlp_dim: int
    vocab: int
    act: str = "bf16"          # "bf16": round at the rounding points; "fp32": never
    rope_base: float = 10000.0
    rms_eps: float = 1e-5


def causal_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor) -> torch.Tensor:
    """Textbook causal attention.  q, k, v: [T][H][Dh] -> [T][H][Dh]."""
    T, H, Dh = q.shape
    s = torch.einsum("thd,uhd->htu", q, k) / math.sqrt(Dh)
    mask = torch.ones(T, T, dtype=torch.bool).tril()
    s = s.masked_fill(~mask, float("-inf"))
    p = torch.softmax(s, dim=-1)
    return torch.einsum("htu,uhd->thd", p, v)


def _qkv(x, model, l, sh: Shape, pos):
    T = x.shape[0]
    H, Dh = sh.n_heads, sh.head_dim
    xn = rb(rmsnorm(x, f64(model[f"attn_norm.{l}"]), sh.rms_eps), sh.act)
    qkv = xn @ f64(model[f"wqkv.{l}"]).T
    q, k, v = [t.reshape(T, H, Dh) for t in qkv.split(H * Dh, dim=-1)]
    q = rb(rope(q, pos, sh.rope_base), sh.act)
    k = rb(rope(k, pos, sh.rope_base), sh.act)
    v = rb(v, sh.act)
    return q, k, v


def _post_attention(x, a, model, l, sh: Shape):
    T = x.shape[0]
    F = sh.mlp_dim
    x = x + a.reshape(T, -1) @ f64(model[f"wo.{l}"]).T
    xn = rb(rmsnorm(x, f64(model[f"mlp_norm.{l}"]), sh.rms_eps), sh.act)
    gu = xn @ f64(model[f"wgu.{l}"]).T
    m = rb(silu(gu[:, :F]) * gu[:, F:], sh.act)
    return x + m @ f64(model[f"wd.{l}"]).T


def _final(x, model, sh: Shape, want_logits=True):
    hidden = rb(rmsnorm(x, f64(model["final_norm"]), sh.rms_eps), sh.act)
    logits = hidden @ f64(model["lm_head"]).T if want_logits else None
    return hidden, logits


def forward_full(model, sh: Shape, tokens: Sequence[int]):
    """Whole-sequence causal forward, no cache.  Returns (hidden [T][d] after the
    final norm, logits [T][V], per-layer list of (k, v) each [T][H][Dh])."""
    tok = torch.as_tensor(list(tokens), dtype=torch.long)
    T = tok.shape[0]
    pos = list(range(T))
    x = f64(model["embed"][tok])
    kv = []
    for l in range(sh.n_layers):
        q, k, v = _qkv(x, model, l, sh, pos)
        kv.append((k, v))
        a = rb(causal_attention(q, k, v), sh.act)
        x = _post_attention(x, a, model, l, sh)
    hidden, logits = _final(x, model, sh)
    return hidden, logits, kv


# --------------------------------------------------------------------------
# Tree verification
# --------------------------------------------------------------------------

def root_path(parent: Sequence[int], v: int) -> List[int]:
    """Node indices from the root down to v."""
    p = []
    while v >= 0:
        p.append(v)
        v = int(parent[v])
    return p[::-1]


def node_depth(parent: Sequence[int], v: int) -> int:
    return len(root_path(parent, v)) - 1


def tree_attention(q, k_prefix, v_prefix, k_tree, v_tree, parent, scale=None):
    """Attention of every tree node over (prefix ++ its own root-to-node path).

    q, k_tree, v_tree: [n][H][Dh]; k_prefix, v_prefix: [len][H][Dh].
    Returns (O [n][H][Dh], lse [H][n]) with lse = ln sum exp(scaled scores)."""
    n, H, Dh = q.shape
    if scale is None:
        scale = 1.0 / math.sqrt(Dh)
    O = torch.empty(n, H, Dh, dtype=F64)
    lse = torch.empty(H, n, dtype=F64)
    for i in range(n):
        path = root_path(parent, i)
        K = torch.cat([k_prefix, k_tree[path]], dim=0)          # explicit sequence, last position = node i
        V = torch.cat([v_prefix, v_tree[path]], dim=0)
        s = torch.einsum("hd,thd->ht", q[i], K) * scale          # [H][T]
        m = s.max(dim=-1, keepdim=True).values
        e = torch.exp(s - m)
        z = e.sum(dim=-1, keepdim=True)
        O[i] = torch.einsum("ht,thd->hd", e / z, V)
        lse[:, i] = (m + torch.log(z)).squeeze(-1)
    return O, lse


@dataclass
class State:
    """Decoding state of one sequence: contiguous per-layer K/V, committed length,
    last hidden state and the next root token."""
    k: List[torch.Tensor]          # per layer [cap][H][Dh] float64
    v: List[torch.Tensor]
    length: int
    h_last: torch.Tensor           # [d]
    root: int


def new_state(sh: Shape, capacity: int) -> State:
    z = lambda: torch.zeros(capacity, sh.n_heads, sh.head_dim, dtype=F64)
    return State([z() for _ in range(sh.n_layers)], [z() for _ in range(sh.n_layers)], 0,
                 torch.zeros(sh.d_model, dtype=F64), -1)


def verify_tree(model, sh: Shape, st: State, tree_tok: Sequence[int], parent: Sequence[int], want_logits=True):
    """One base-model forward over all tree nodes on top of the committed cache.
    Writes node v's K/V at slot length + v.  Returns (hidden [n][d], logits [n][V])."""
    n = len(tree_tok)
    tok = torch.as_tensor(list(tree_tok), dtype=torch.long)
    pos = [st.length + node_depth(parent, v) for v in range(n)]
    x = f64(model["embed"][tok])
    L = st.length
    for l in range(sh.n_layers):
        q, k, v = _qkv(x, model, l, sh, pos)
        st.k[l][L:L + n] = k
        st.v[l][L:L + n] = v
        a, _ = tree_attention(q, st.k[l][:L], st.v[l][:L], k, v, parent)
        x = _post_attention(x, rb(a, sh.act), model, l, sh)
    return _final(x, model, sh, want_logits)


def accept_longest(tree_tok: Sequence[int], node_argmax: Sequence[int], parent: Sequence[int]) -> List[int]:
    """Enumerate every root-to-node path; a path is valid iff each non-root token
    equals the model's argmax at its parent node.  Longest valid path wins, ties go
    to the lowest end-node index.  The root alone is always valid."""
    best = [0]
    for v in range(len(tree_tok)):
        path = root_path(parent, v)
        ok = all(int(tree_tok[c]) == int(node_argmax[p]) for p, c in zip(path[:-1], path[1:]))
        if ok and len(path) > len(best):
            best = path
    return best


def compact(st: State, path: Sequence[int]) -> None:
    """Move the accepted nodes' K/V from slot length + path[j] to slot length + j."""
    L = st.length
    src = [L + int(p) for p in path]
    for l in range(len(st.k)):
        ks, vs = st.k[l][src].clone(), st.v[l][src].clone()
        st.k[l][L:L + len(path)] = ks
        st.v[l][L:L + len(path)] = vs


def prefill(model, sh: Shape, prompt: Sequence[int], capacity: int) -> State:
    """Process the prompt with the textbook forward and load its K/V into a state."""
    hidden, logits, kv = forward_full(model, sh, prompt)
    st = new_state(sh, capacity)
    T = len(prompt)
    for l, (k, v) in enumerate(kv):
        st.k[l][:T] = k
        st.v[l][:T] = v
    st.length = T
    st.h_last = hidden[-1].clone()
    st.root = int(argmax_f32(logits[-1]))
    return st


@dataclass
class StepRecord:
    S: float
    mode: int
    tree_tok: List[int]
    node_argmax: List[int]
    path: List[int]
    tokens: List[int]
    topk: Optional[List[List[int]]] = None


def step(model, sh: Shape, st: State, heads, concat_src, parent, head_of, rank_of, topk_per_head: Sequence[int],
         T: float, plant: Optional[Callable[[List[int]], List[int]]] = None,
         return_values: bool = False):
    """One decoding step, Algorithm 1, followed by acceptance and commit."""
    S = gate_entropy(st.h_last)
    mode = gate_mode(S, T)
    root = int(argmax_f32(f64(model["lm_head"]) @ st.h_last))
    topk = None
    if mode == MODE_AR:
        par, tree_tok = [-1], [root]
    else:
        head_logits = heads_forward(st.h_last, heads, concat_src)
        topk = [list(map(int, topk_ids(head_logits[h], topk_per_head[h]))) for h in range(len(head_logits))]
        par = list(map(int, parent))
        tree_tok = [root] + [topk[int(head_of[v])][int(rank_of[v])] for v in range(1, len(par))]
        if plant is not None:
            tree_tok = list(plant(list(tree_tok)))
            assert tree_tok[0] == root
    hidden, logits = verify_tree(model, sh, st, tree_tok, par)
    node_argmax = list(map(int, argmax_f32(logits)))
    path = accept_longest(tree_tok, node_argmax, par)
    compact(st, path)
    st.length += len(path)
    st.h_last = hidden[path[-1]].clone()
    st.root = node_argmax[path[-1]]
    rec = StepRecord(S, mode, list(tree_tok), node_argmax, list(path), [int(tree_tok[p]) for p in path], topk)
    if return_values:
        return rec, hidden, logits
    return rec


def ar_greedy(model, sh: Shape, prompt: Sequence[int], n_new: int):
    """Plain auto-regressive greedy decoding, whole-sequence forward per token.
    Returns (new tokens, gate entropy of the hidden state each token was decoded from)."""
    seq = list(map(int, prompt))
    out, Ss = [], []
    for _ in range(n_new):
        hidden, logits, _ = forward_full(model, sh, seq)
        Ss.append(gate_entropy(hidden[-1]))
        t = int(argmax_f32(logits[-1]))
        out.append(t)
        seq.append(t)
    return out, Ss


def cerberus_greedy(model, sh: Shape, heads, concat_src, prompt, parent, head_of, rank_of, topk_per_head,
                    T: float, n_new: int, capacity: Optional[int] = None,
                    plant: Optional[Callable[[List[int], int, List[int]], List[int]]] = None):
    """Greedy Cerberus decoding until at least n_new tokens are emitted.
    `plant(tree_tok, step_index, emitted_so_far)` may overwrite candidate tokens
    (never the root).  Returns (tokens[:n_new], step records, final state)."""
    n = len(parent)
    if capacity is None:
        capacity = len(prompt) + n_new + 2 * n + 8
    st = prefill(model, sh, prompt, capacity)
    out: List[int] = []
    recs: List[StepRecord] = []
    while len(out) < n_new:
        i = len(recs)
        pl = (lambda tt: plant(tt, i, list(out))) if plant is not None else None
        rec = step(model, sh, st, heads, concat_src, parent, head_of, rank_of, topk_per_head, T, pl)
        recs.append(rec)
        out.extend(rec.tokens)
    return out[:n_new], recs, st


def calibrate_threshold(S_values: Sequence[float], q: float = 0.5, min_gap: float = 1e-4) -> float:
    """Threshold putting a fraction q of the observed gate values at or below it:
    the midpoint of the two neighbouring order statistics, moved to the nearest
    gap of at least min_gap so that rounding noise cannot flip a step."""
    s = sorted(S_values)
    k = min(max(int(round(q * len(s))), 1), len(s) - 1)
    cand = sorted(range(1, len(s)), key=lambda i: abs(i - k))
    for i in cand:
        if s[i] - s[i - 1] >= min_gap:
            return 0.5 * (s[i] + s[i - 1])
    return 0.5 * (s[k] + s[k - 1])
