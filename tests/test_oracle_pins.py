"""Pins for the CPU oracle: every check compares it with something other than
itself -- closed forms, library routines, brute force, or invariants of greedy
draft-then-verify decoding.  No GPU needed."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as Fn

from oracle import cerberus_oracle as orc
from paper_2410_13344_b200 import synth

F64 = torch.float64
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed, std=1.0):
    return synth.normal(77, seed, shape, std, dtype=F64)


# ------------------------------------------------------------------ gate

def test_gate_closed_forms_golden():
    for line in open(os.path.join(GOLDEN, "gate_closed_forms.txt")):
        if line.startswith("#") or not line.strip():
            continue
        case, K, m, gap, expect = line.split()
        K, m, gap, expect = int(K), int(m), float(gap), float(expect)
        h = torch.full((K,), -3.25, dtype=F64)
        h[:m] += gap
        assert abs(orc.gate_entropy(h) - expect) < 1e-9, line


def test_gate_matches_library_entropy_and_shift_invariance():
    from scipy.stats import entropy
    h = _rand((4096,), 1, 2.0)
    p = torch.softmax(h, dim=0).numpy()
    S = orc.gate_entropy(h)
    assert abs(S - entropy(p, base=2)) < 1e-10
    assert abs(orc.gate_entropy(h + 123.5) - S) < 1e-9
    # bits, not nats: a mistake in the log base would be off by ln 2
    assert abs(S - entropy(p)) > 0.1
    # bounded by log2 K, positive
    assert 0 < S < 12


def test_gate_mode_rule():
    assert orc.gate_mode(0.6, 0.59) == orc.MODE_AR
    assert orc.gate_mode(0.58, 0.59) == orc.MODE_PAR
    assert orc.gate_mode(0.59, 0.59) == orc.MODE_PAR   # only a strictly larger entropy goes auto-regressive


# ------------------------------------------------------------------ heads

def test_resblock_hand_example():
    h = torch.tensor([1.0, -2.0], dtype=F64)
    W = torch.tensor([[1.0, 2.0], [3.0, 4.0]], dtype=F64)
    b = torch.tensor([0.5, -0.5], dtype=F64)
    # W h = [-3, -5]; + b = [-2.5, -5.5]; + h = [-1.5, -7.5]; SiLU(x) = x / (1 + e^-x)
    expect = [-1.5 / (1 + math.exp(1.5)), -7.5 / (1 + math.exp(7.5))]
    out = orc.resblock(h, W, b)
    assert np.allclose(out.numpy(), expect, atol=1e-14)


def test_resblock_closed_forms_and_library():
    h = _rand((32,), 2)
    Z, z = torch.zeros(32, 32, dtype=F64), torch.zeros(32, dtype=F64)
    assert torch.allclose(orc.resblock(h, Z, z), Fn.silu(h), atol=1e-14)
    W, b = _rand((32, 32), 3, 0.2), _rand((32,), 4, 0.2)
    assert torch.allclose(orc.resblock(h, W, b), Fn.silu(Fn.linear(h, W, b) + h), atol=1e-13)
    # activation sits outside the residual sum: differs from h + SiLU(W h + b)
    assert not torch.allclose(orc.resblock(h, W, b), h + Fn.silu(Fn.linear(h, W, b)), atol=1e-3)


def test_concat_resblock_closed_forms():
    a, p = _rand((16,), 5), _rand((24,), 6)
    Z, z = torch.zeros(40, 40, dtype=F64), torch.zeros(40, dtype=F64)
    out = orc.concat_resblock(a, p, Z, z)
    assert out.shape == (40,)
    assert torch.allclose(out, Fn.silu(torch.cat([a, p])), atol=1e-14)      # own state first, neighbour second
    W, b = _rand((40, 40), 7, 0.2), _rand((40,), 8, 0.2)
    u = torch.cat([a, p])
    assert torch.allclose(orc.concat_resblock(a, p, W, b), Fn.silu(Fn.linear(u, W, b) + u), atol=1e-13)


def _toy_heads(d, V, layout, seed=9):
    sh = synth.ModelShape(1, d, 1, d, d, V, "fp32")
    hw = synth.make_heads(sh, layout, seed=seed, std=0.3)
    return {k: v.to(F64) for k, v in hw.items()}


def _concat_src(layout):
    return [[b.concat_src_head for b in row] for row in layout.blocks]


def test_heads_without_concat_are_medusa_heads():
    d, V = 24, 50
    layout = synth.medusa_layout(3, 4)
    hw = _toy_heads(d, V, layout)
    h = _rand((d,), 10)
    got = orc.heads_forward(h, hw, _concat_src(layout))
    for i in range(3):                      # each head on its own, sequentially, with library ops
        x = h
        for j in range(4):
            x = Fn.silu(Fn.linear(x, hw[f"W.{i}.{j}"], hw[f"b.{i}.{j}"]) + x)
        assert torch.allclose(got[i], Fn.linear(x, hw[f"fc.{i}"]), atol=1e-12)


@pytest.mark.parametrize("concat_level", [3, 1, 0])
def test_cerberus_heads_level_synchronous_wiring(concat_level):
    d, V, Hc, L = 16, 40, 3, 4
    layout = synth.cerberus_layout(Hc, L, concat_level)
    widths = layout.widths(d)
    hw = _toy_heads(d, V, layout)
    h = _rand((d,), 11)
    got = orc.heads_forward(h, hw, _concat_src(layout))
    # independent restatement: keep the whole history of every head's states
    hist = [[h] for _ in range(Hc)]
    for j in range(L):
        for i in range(Hc):
            x = hist[i][j]
            if i >= 1 and j == concat_level:
                x = torch.cat([x, hist[i - 1][j]])      # neighbour's state entering the same level
            assert x.shape[0] == widths[i][j + 1]
            hist[i].append(Fn.silu(Fn.linear(x, hw[f"W.{i}.{j}"], hw[f"b.{i}.{j}"]) + x))
    for i in range(Hc):
        assert torch.allclose(got[i], Fn.linear(hist[i][L], hw[f"fc.{i}"]), atol=1e-12)
    # head 0 has no predecessor: it is a plain head
    assert widths[0] == [d] * (L + 1)


def test_topk_ids_sort_rule():
    v = _rand((1000,), 12)
    ids = orc.topk_ids(v, 10)
    assert list(ids) == list(torch.topk(v.float(), 10).indices.numpy())
    t = torch.tensor([1.0, 5.0, 5.0, 0.0, 5.0, 2.0], dtype=F64)
    assert list(orc.topk_ids(t, 4)) == [1, 2, 4, 5]            # equal values: lower id first
    assert int(orc.argmax_f32(t)) == 1


# ------------------------------------------------------------------ base model pieces

def test_rmsnorm_and_silu_match_library():
    x, g = _rand((5, 64), 13), _rand((64,), 14)
    assert torch.allclose(orc.rmsnorm(x, g, 1e-5), Fn.rms_norm(x, (64,), g, 1e-5), atol=1e-13)
    assert torch.allclose(orc.silu(x), Fn.silu(x), atol=1e-14)


def test_rope_complex_form_and_relative_property():
    T, H, Dh, base = 7, 2, 16, 10000.0
    x = _rand((T, H, Dh), 15)
    pos = [0, 3, 4, 9, 100, 101, 5000]
    y = orc.rope(x, pos, base)
    assert torch.allclose(y[0], x[0], atol=1e-15)                          # position 0 is the identity
    half = Dh // 2
    z = torch.complex(x[..., :half], x[..., half:])                        # pair (i, i + Dh/2)
    freqs = torch.tensor([base ** (-2.0 * i / Dh) for i in range(half)], dtype=F64)
    rot = torch.polar(torch.ones(T, half, dtype=F64), torch.tensor(pos, dtype=F64)[:, None] * freqs)
    zz = z * rot[:, None, :]
    assert torch.allclose(y, torch.cat([zz.real, zz.imag], -1), atol=1e-12)
    # scores depend only on the position difference
    q, k = _rand((1, 1, Dh), 16), _rand((1, 1, Dh), 17)
    s1 = (orc.rope(q, [10], base) * orc.rope(k, [7], base)).sum()
    s2 = (orc.rope(q, [1003], base) * orc.rope(k, [1000], base)).sum()
    assert abs(float(s1 - s2)) < 1e-10


def test_causal_attention_matches_library():
    T, H, Dh = 9, 3, 8
    q, k, v = _rand((T, H, Dh), 18), _rand((T, H, Dh), 19), _rand((T, H, Dh), 20)
    ref = Fn.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1), is_causal=True)
    assert torch.allclose(orc.causal_attention(q, k, v), ref.transpose(0, 1), atol=1e-12)


# ------------------------------------------------------------------ tree attention

def test_chain_tree_is_causal_attention():
    Lp, n, H, Dh = 11, 6, 2, 8
    kp, vp = _rand((Lp, H, Dh), 21), _rand((Lp, H, Dh), 22)
    q, kt, vt = _rand((n, H, Dh), 23), _rand((n, H, Dh), 24), _rand((n, H, Dh), 25)
    chain = synth.chain_tree(n).parent
    O, lse = orc.tree_attention(q, kp, vp, kt, vt, chain)
    K, V = torch.cat([kp, kt]), torch.cat([vp, vt])
    qq = torch.cat([torch.zeros(Lp, H, Dh, dtype=F64), q])
    ref = Fn.scaled_dot_product_attention(qq.transpose(0, 1), K.transpose(0, 1), V.transpose(0, 1), is_causal=True)
    assert torch.allclose(O, ref.transpose(0, 1)[Lp:], atol=1e-12)
    s = torch.einsum("thd,uhd->htu", q, K) / math.sqrt(Dh)
    for i in range(n):
        assert torch.allclose(lse[:, i], torch.logsumexp(s[:, i, :Lp + i + 1], dim=-1), atol=1e-12)


def test_tree_attention_matches_masked_library_attention():
    Lp, n, H, Dh = 5, 12, 2, 8
    tree = synth.random_parent_tree(n, 4, tree_id=1)
    kp, vp = _rand((Lp, H, Dh), 26), _rand((Lp, H, Dh), 27)
    q, kt, vt = _rand((n, H, Dh), 28), _rand((n, H, Dh), 29), _rand((n, H, Dh), 30)
    O, lse = orc.tree_attention(q, kp, vp, kt, vt, tree.parent, scale=0.3)
    # mask from an independent ancestor closure (transitive closure by repeated squaring)
    A = np.eye(n, dtype=bool)
    for v in range(1, n):
        A[v, tree.parent[v]] = True
    for _ in range(n):
        A = A | ((A.astype(int) @ A.astype(int)) > 0)
    mask = torch.cat([torch.ones(n, Lp, dtype=torch.bool), torch.from_numpy(A)], dim=1)
    K, V = torch.cat([kp, kt]), torch.cat([vp, vt])
    ref = Fn.scaled_dot_product_attention(q.transpose(0, 1), K.transpose(0, 1), V.transpose(0, 1),
                                          attn_mask=mask, scale=0.3)
    assert torch.allclose(O, ref.transpose(0, 1), atol=1e-12)
    s = (torch.einsum("thd,uhd->htu", q, K) * 0.3).masked_fill(~mask, float("-inf"))
    assert torch.allclose(lse, torch.logsumexp(s, dim=-1), atol=1e-12)


# ------------------------------------------------------------------ acceptance

def _continuation(prefix_tokens, V):
    """A deterministic stand-in 'model': next token after a token sequence."""
    acc = 12345
    for t in prefix_tokens:
        acc = (acc * 1103515245 + t * 2654435761 + 12345) % (1 << 31)
    return (acc >> 7) % V


@pytest.mark.parametrize("tree_id", range(12))
def test_acceptance_is_longest_prefix_of_true_continuation(tree_id):
    V, n = 3, 8                                   # tiny vocabulary: matches are frequent
    tree = synth.random_parent_tree(n, 4, tree_id=50 + tree_id)
    tok = [int(t) for t in synth.randint(5, tree_id, (n,), V)]
    paths = [orc.root_path(tree.parent, v) for v in range(n)]
    node_argmax = [_continuation([tok[u] for u in paths[v]], V) for v in range(n)]
    got = orc.accept_longest(tok, node_argmax, tree.parent)
    # independent characterisation: the emitted tokens are the longest prefix of the
    # true greedy continuation (after the root) that some root-to-node path spells out
    truth = [tok[0]]
    for _ in range(n):
        truth.append(_continuation(truth, V))
    best_len = 1
    for v in range(n):
        toks = [tok[u] for u in paths[v]]
        if toks == truth[:len(toks)]:
            best_len = max(best_len, len(toks))
    assert [tok[u] for u in got] == truth[:best_len]
    assert got[0] == 0 and all(tree.parent[c] == p for p, c in zip(got[:-1], got[1:]))
    # lowest end node among equally long valid paths
    ends = [v for v in range(n) if len(paths[v]) == best_len and [tok[u] for u in paths[v]] == truth[:best_len]]
    assert got[-1] == min(ends)


def test_accept_root_only_and_full_chain():
    chain = synth.chain_tree(5).parent
    assert orc.accept_longest([7, 1, 2, 3, 4], [9, 9, 9, 9, 9], chain) == [0]
    assert orc.accept_longest([7, 1, 2, 3, 4], [1, 2, 3, 4, 5], chain) == [0, 1, 2, 3, 4]
    assert orc.accept_longest([7, 1, 2, 3, 4], [1, 2, 0, 4, 5], chain) == [0, 1, 2]   # a later match cannot revive a broken path


# ------------------------------------------------------------------ whole step on a small model

def _small(act, seed=0, layers=2):
    ms = synth.ModelShape(layers, 64, 4, 16, 176, 96, act)
    model = synth.make_model(ms, seed=seed, std=0.08)
    layout = synth.cerberus_layout(3, 2)
    heads = synth.make_heads(ms, layout, std=0.08)
    sh = orc.Shape(ms.n_layers, ms.d_model, ms.n_heads, ms.head_dim, ms.mlp_dim, ms.vocab, act)
    return ms, model, layout, heads, sh


@pytest.mark.parametrize("act", ["fp32", "bf16"])
def test_verify_tree_equals_full_forward_on_each_path(act):
    ms, model, layout, heads, sh = _small(act)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 9)]
    tree = synth.random_parent_tree(10, 4, tree_id=2)
    tok = [int(t) for t in synth.randint(6, 0, (10,), ms.vocab)]
    st = orc.prefill(model, sh, prompt, 64)
    hidden, logits = orc.verify_tree(model, sh, st, tok, tree.parent)
    tol = 1e-9 if act == "fp32" else 3e-2      # bf16: a rounding flip is one bf16 ulp of an O(1) value
    for v in range(10):
        seq = prompt + [tok[u] for u in orc.root_path(tree.parent, v)]
        h_ref, l_ref, kv = orc.forward_full(model, sh, seq)
        assert float((hidden[v] - h_ref[-1]).abs().max()) < tol
        assert float((logits[v] - l_ref[-1]).abs().max()) < tol
        # the node's K/V sits at slot len + node index and equals the sequence's last position
        assert float((st.k[1][len(prompt) + v] - kv[1][0][-1]).abs().max()) < tol


def _planter(truth, tree, lengths):
    """Overwrite one root-to-leaf path of the tree with the true continuation."""
    def plant(tree_tok, step, emitted):
        want = lengths[step % len(lengths)]
        pos = len(emitted)                       # truth[pos] is the root of this step
        deepest = max(range(tree.n), key=lambda v: (len(orc.root_path(tree.parent, v)), -v))
        path = orc.root_path(tree.parent, deepest)
        out = list(tree_tok)
        for j, node in enumerate(path[1:want], start=1):
            if pos + j < len(truth):
                out[node] = truth[pos + j]
        return out
    return plant


@pytest.mark.parametrize("act,thr", [("fp32", "median"), ("fp32", "always_par"), ("bf16", "median"), ("fp32", "always_ar")])
def test_greedy_cerberus_emits_the_autoregressive_sequence(act, thr):
    ms, model, layout, heads, sh = _small(act)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 12)]
    n_new = 20
    truth, Ss = orc.ar_greedy(model, sh, prompt, n_new + 6)
    T = {"median": orc.calibrate_threshold(Ss[:n_new]), "always_par": 1e9, "always_ar": -1.0}[thr]
    tree = synth.best_first_tree(12, [3, 2, 2])
    plant = _planter(truth, tree, [1, 3, 2, 4, 1, 2])
    toks, recs, st = orc.cerberus_greedy(model, sh, heads, _concat_src(layout), prompt, tree.parent, tree.head,
                                         tree.rank, [3, 2, 2], T, n_new, plant=plant)
    assert toks == truth[:n_new]
    modes = [r.mode for r in recs]
    for r in recs:                                   # S > T  <=>  auto-regressive step with a one-node tree
        assert (r.S > T) == (r.mode == orc.MODE_AR)
        assert (len(r.tree_tok) == 1) == (r.mode == orc.MODE_AR)
    if thr == "always_par":
        assert max(len(r.path) for r in recs) >= 3 and set(modes) == {orc.MODE_PAR}
    if thr == "always_ar":
        assert set(modes) == {orc.MODE_AR} and len(recs) == n_new
    if thr == "median":
        assert set(modes) == {orc.MODE_PAR, orc.MODE_AR}
    # the compacted cache equals the cache of a plain forward over the same tokens
    emitted = [t for r in recs for t in r.tokens]
    _, _, kv = orc.forward_full(model, sh, prompt + emitted)
    tol = 1e-9 if act == "fp32" else 3e-2
    L = len(prompt) + len(emitted)
    assert st.length == L
    for l in range(ms.n_layers):
        assert float((st.k[l][:L] - kv[l][0]).abs().max()) < tol
        assert float((st.v[l][:L] - kv[l][1]).abs().max()) < tol


def test_threshold_calibration_splits_in_half():
    S = [0.1 * i for i in range(32)]
    T = orc.calibrate_threshold(S)
    assert sum(s > T for s in S) == 16


# ------------------------------------------------------------------ decoder-layer wiring against an independent library model

def _hf_llama(ms, model):
    """The same weights inside the stock `transformers` LLaMA implementation, parameters in float64, eager
    attention.  That implementation takes its norms, rotation angles and softmax in float32 whatever the
    parameter type, so agreement is at float32 rounding (~1e-7 per operation), not float64."""
    tr = pytest.importorskip("transformers")
    cfg = tr.LlamaConfig(vocab_size=ms.vocab, hidden_size=ms.d_model, intermediate_size=ms.mlp_dim,
                         num_hidden_layers=ms.n_layers, num_attention_heads=ms.n_heads,
                         num_key_value_heads=ms.n_heads, head_dim=ms.head_dim, rms_norm_eps=ms.rms_eps,
                         rope_theta=ms.rope_base, attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
                         max_position_embeddings=256, hidden_act="silu", attn_implementation="eager")
    hf = tr.LlamaForCausalLM(cfg).to(torch.float64).eval()
    hd, F = ms.n_heads * ms.head_dim, ms.mlp_dim
    sd = {"model.embed_tokens.weight": model["embed"], "model.norm.weight": model["final_norm"],
          "lm_head.weight": model["lm_head"]}
    for l in range(ms.n_layers):
        p = f"model.layers.{l}."
        wqkv, wgu = model[f"wqkv.{l}"], model[f"wgu.{l}"]
        sd[p + "self_attn.q_proj.weight"] = wqkv[:hd]
        sd[p + "self_attn.k_proj.weight"] = wqkv[hd:2 * hd]
        sd[p + "self_attn.v_proj.weight"] = wqkv[2 * hd:]
        sd[p + "self_attn.o_proj.weight"] = model[f"wo.{l}"]
        sd[p + "mlp.gate_proj.weight"] = wgu[:F]
        sd[p + "mlp.up_proj.weight"] = wgu[F:]
        sd[p + "mlp.down_proj.weight"] = model[f"wd.{l}"]
        sd[p + "input_layernorm.weight"] = model[f"attn_norm.{l}"]
        sd[p + "post_attention_layernorm.weight"] = model[f"mlp_norm.{l}"]
    missing, unexpected = hf.load_state_dict({k: v.to(torch.float64) for k, v in sd.items()}, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return hf


def test_decoder_wiring_matches_transformers_llama():
    """forward_full (pre-norm, fused QKV split, rotate-half RoPE, causal attention, o-projection + residual,
    pre-norm SwiGLU with gate rows first, down-projection + residual, final norm, untied LM head) against the
    LLaMA decoder of the `transformers` package holding the same weights: Section 5.1 names the base model as
    a LLaMA fine-tune, and that package is an independent statement of the architecture."""
    ms = synth.ModelShape(3, 64, 4, 16, 176, 96, "fp32")
    model = synth.make_model(ms, seed=5, std=0.08)
    sh = orc.Shape(ms.n_layers, ms.d_model, ms.n_heads, ms.head_dim, ms.mlp_dim, ms.vocab, "fp32")
    tokens = [int(t) for t in synth.make_prompt(ms.vocab, 23, seq=3)]
    hidden, logits, kv = orc.forward_full(model, sh, tokens)
    hf = _hf_llama(ms, model)
    with torch.no_grad():
        out = hf(torch.tensor([tokens]), use_cache=True, output_hidden_states=True)
        h_ref = hf.model(torch.tensor([tokens])).last_hidden_state[0]
    tol = 3e-6          # the library's float32 norms, angles and softmax; a wiring mistake is > 1e-3 (next test)
    assert float((logits - out.logits[0]).abs().max()) < tol
    assert float((hidden - h_ref).abs().max()) < tol
    # the residual stream entering every layer (hidden_states[l], before the final norm) is implied by the above
    # for the last layer only; K and V of every layer pin the rest: post-rotation keys, unrotated values
    for l in range(ms.n_layers):
        layer = out.past_key_values.layers[l]
        k_ref, v_ref = layer.keys[0].transpose(0, 1), layer.values[0].transpose(0, 1)     # [T][H][Dh]
        assert float((kv[l][0] - k_ref).abs().max()) < tol
        assert float((kv[l][1] - v_ref).abs().max()) < tol
    assert float(logits.abs().max()) > 0.1      # the comparison is not between two near-zero tensors


@pytest.mark.parametrize("mistake", ["no_attn_residual", "no_mlp_residual", "swap_gate_up", "post_norm", "no_final_norm"])
def test_decoder_wiring_pin_catches_planted_mistakes(mistake, monkeypatch):
    """The library comparison must turn red for each plausible wiring mistake, planted in the oracle."""
    ms = synth.ModelShape(2, 64, 4, 16, 176, 96, "fp32")
    model = synth.make_model(ms, seed=5, std=0.08)
    sh = orc.Shape(ms.n_layers, ms.d_model, ms.n_heads, ms.head_dim, ms.mlp_dim, ms.vocab, "fp32")
    tokens = [int(t) for t in synth.make_prompt(ms.vocab, 11, seq=4)]
    hf = _hf_llama(ms, model)
    with torch.no_grad():
        ref = hf(torch.tensor([tokens])).logits[0]
    good = orc.forward_full(model, sh, tokens)[1]
    assert float((good - ref).abs().max()) < 3e-6

    F = ms.mlp_dim
    f64 = orc.f64

    def post(x, a, m, l, s):
        T = x.shape[0]
        o = a.reshape(T, -1) @ f64(m[f"wo.{l}"]).T
        x = o if mistake == "no_attn_residual" else x + o
        if mistake == "post_norm":
            xn = x
        else:
            xn = orc.rmsnorm(x, f64(m[f"mlp_norm.{l}"]), s.rms_eps)
        gu = xn @ f64(m[f"wgu.{l}"]).T
        g, u = (gu[:, F:], gu[:, :F]) if mistake == "swap_gate_up" else (gu[:, :F], gu[:, F:])
        y = (orc.silu(g) * u) @ f64(m[f"wd.{l}"]).T
        y = y if mistake == "no_mlp_residual" else x + y
        if mistake == "post_norm":
            y = orc.rmsnorm(y, f64(m[f"mlp_norm.{l}"]), s.rms_eps)
        return y

    def final(x, m, s, want_logits=True):
        h = x if mistake == "no_final_norm" else orc.rmsnorm(x, f64(m["final_norm"]), s.rms_eps)
        return h, h @ f64(m["lm_head"]).T

    if mistake == "no_final_norm":
        monkeypatch.setattr(orc, "_final", final)
    else:
        monkeypatch.setattr(orc, "_post_attention", post)
    bad = orc.forward_full(model, sh, tokens)[1]
    assert float((bad - ref).abs().max()) > 1e-3
