"""Parity at the benchmark's sizes.

* 7B-width model cut to two layers (every kernel runs in the launch configuration the benchmark
  times: same widths, same grids, 64-node tree): values and decisions against the CPU oracle.
* Full-depth 7B-shaped and 13B-width (batch 4) models, where the oracle is too slow to run:
  properties that hold at any size, checked step by step from a shared state (see
  _teacher_forced_steps), with candidates planted so that paths of several tokens are accepted."""
import numpy as np
import pytest
import torch

from oracle import cerberus_oracle as orc
from paper_2410_13344_b200 import synth
from tests.helpers import (assert_close_large, check_argmax_flips, close, concat_src, cpu, deepest_path, oracle_shape,
                           parity_stats, record, top2_margin)

pytestmark = pytest.mark.gpu
TOL = 2e-2
TIE = 1e-3
# Allowances of the large-tensor criterion, set to about twice what was measured (the raw figures are recorded by
# every run, see tests/helpers.py: record): fraction of elements outside |a-b| <= TOL * (1 + |b|), largest oracle
# margin of a node whose argmax differs, and how many of 64 nodes may differ.
# Measured (two-layer models at the 7B / 13B widths): K/V 9e-6, hidden states 1.5e-5 (3.8e-5 over 128 nodes), logits
# 4.2e-4 / 1.2e-3; one node of 64 differing with an oracle margin of 5e-3 (one of 128 with 1.5e-2).  At all 32 layers,
# against the depth-scaled bound: K/V 6.8e-4, hidden states 1.5e-4, logits 1.0e-3.
OUTLIERS_KV = 2e-5
OUTLIERS_HIDDEN = 8e-5
OUTLIERS_LOGITS = 2.5e-3
OUTLIERS_KV_DEEP = 1.4e-3
OUTLIERS_HIDDEN_DEEP = 3e-4
OUTLIERS_LOGITS_DEEP = 2e-3
FLIP_MARGIN = 2e-2
MAX_FLIPS_64 = 2


@pytest.fixture(scope="module")
def cb():
    from paper_2410_13344_b200 import binding
    return binding


def _engine(cb, ms, n_cheads, topk, max_tokens, max_batch=1):
    model = synth.make_model(ms, device="cuda")
    layout = synth.cerberus_layout(n_cheads, 4)
    heads = synth.make_heads(ms, layout, device="cuda")
    eng = cb.Cerberus(ms, model, layout, heads, topk, max_tokens=max_tokens, max_batch=max_batch, max_nodes=128)
    return model, layout, heads, eng


def _two_layer_width_against_oracle(cb, ms, n_cheads, prompt_len, seq, what, n_nodes=64):
    """Prefill, gate, draft, one verification forward over an n_nodes tree, acceptance: values and decisions against
    the oracle."""
    topk = [10] * n_cheads
    model, layout, heads, eng = _engine(cb, ms, n_cheads, topk, 512)
    cmodel, cheads, sh, csrc = cpu(model), cpu(heads), oracle_shape(ms), concat_src(layout)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, prompt_len, seq=seq)]
    tree = synth.best_first_tree(n_nodes, topk)
    th = eng.tree(tree)
    eng.prefill(torch.tensor([prompt], dtype=torch.int32, device="cuda"), [len(prompt)])
    st = orc.prefill(cmodel, sh, prompt, 512)
    lens, roots, h_last = eng.read_state()
    assert lens[0] == len(prompt)
    record(what + " h_last", tol=TOL, **parity_stats(h_last[0], st.h_last, TOL))
    assert close(h_last[0], st.h_last) < TOL
    for l in range(ms.n_layers):
        k, v = eng.gather_kv(0, l, len(prompt))
        assert_close_large(k, st.k[l][:len(prompt)], TOL, f"{what} K[{l}]", outliers=OUTLIERS_KV)
        assert_close_large(v, st.v[l][:len(prompt)], TOL, f"{what} V[{l}]", outliers=OUTLIERS_KV)
    lm = orc.linear(st.h_last[None], cmodel["lm_head"])[0]
    assert roots[0] == st.root or top2_margin(lm) < TIE
    if roots[0] != st.root:
        pytest.skip("argmax near-tie at the prompt's last position")
    S, _ = eng.gate(0.0)
    record(what + " gate S", gpu=float(S[0]), oracle=orc.gate_entropy(st.h_last))
    assert abs(float(S[0]) - orc.gate_entropy(st.h_last)) < 2e-2
    # draft: head logits from the GPU's own h_last (the inputs must be identical to compare decisions)
    tree_tok, topk_ids, hlog = eng.draft(th, want_logits=True)
    olog = orc.heads_forward(h_last[0].double(), cheads, csrc)
    for h in range(n_cheads):
        assert close(hlog[0, h], olog[h]) < 5e-3
        assert [int(t) for t in topk_ids[0, h, :10]] == list(orc.topk_ids(hlog[0, h].cpu().double(), 10))
    want_tok = [int(roots[0])] + [int(topk_ids[0, tree.head[v], tree.rank[v]]) for v in range(1, tree.n)]
    assert [int(t) for t in tree_tok[0]] == want_tok
    # verify: hidden states and logits of all nodes, every argmax
    node_argmax, logits, hidden = eng.verify(th, tree_tok, want_logits=True, want_hidden=True)
    o_hidden, o_logits = orc.verify_tree(cmodel, sh, st, want_tok, tree.parent)
    assert_close_large(hidden[0], o_hidden, TOL, what + " hidden", outliers=OUTLIERS_HIDDEN)
    assert_close_large(logits[0], o_logits, TOL, what + " logits", outliers=OUTLIERS_LOGITS)
    # decisions: exact on the kernel's own logits; against the oracle's logits a different token is
    # admissible only where the oracle itself scores it within FLIP_MARGIN of its best one
    assert torch.equal(node_argmax[0].long().cpu(), torch.argmax(logits[0], dim=-1).cpu())
    check_argmax_flips(node_argmax[0], o_logits, FLIP_MARGIN, MAX_FLIPS_64, what)
    # accept + compaction against the oracle on the GPU's own decisions
    n_acc, gpath, gtok = eng.accept(th, tree_tok, node_argmax)
    opath = orc.accept_longest(want_tok, [int(a) for a in node_argmax[0]], tree.parent)
    assert [int(p) for p in gpath[0, :int(n_acc[0])]] == opath
    assert eng.device_status() == 0


def test_7b_width_two_layers_against_oracle(cb):
    _two_layer_width_against_oracle(cb, synth.shape_7b(n_layers=2), 4, 200, 7, "7B width, 2 layers")


def test_7b_width_two_layers_twelve_node_tree_against_oracle(cb):
    """Steps of up to 16 rows at head_dim 128 take other kernels for the same arithmetic: RoPE and the cache append run
    in the QKV GEMM's epilogue, SwiGLU in the gate-up GEMM's, attention on the warp-MMA kernel."""
    _two_layer_width_against_oracle(cb, synth.shape_7b(n_layers=2), 4, 150, 9, "7B width, 2 layers, 12 nodes", n_nodes=12)


def test_13b_width_two_layers_against_oracle(cb):
    """d_model 5120, 40 heads, MLP 13824, five decoding heads: the widths of the 13B configuration."""
    _two_layer_width_against_oracle(cb, synth.shape_13b(n_layers=2), 5, 200, 11, "13B width, 2 layers")


@pytest.mark.slow
def test_7b_full_depth_prefill_and_verify_against_oracle(cb):
    """All 32 layers of the 7B shape against the oracle: a 64-token prompt through cerb_prefill, then one 64-node
    verification forward (about two minutes of host time for the oracle).  The raw error is recorded next to the
    depth-scaled bound; decisions are compared as for the two-layer models."""
    ms = synth.shape_7b()
    topk = [10, 10, 10, 10]
    model, layout, heads, eng = _engine(cb, ms, 4, topk, 256)
    cmodel, sh = cpu(model), oracle_shape(ms)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 64, seq=21)]
    tree = synth.best_first_tree(64, topk)
    th = eng.tree(tree)
    eng.prefill(torch.tensor([prompt], dtype=torch.int32, device="cuda"), [len(prompt)])
    tree_tok, _, _ = eng.draft(th)
    node_argmax, logits, hidden = eng.verify(th, tree_tok, want_logits=True, want_hidden=True)
    lens, roots, h_last = eng.read_state()
    kv = {l: eng.gather_kv(0, l, len(prompt)) for l in (0, 15, 31)}
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    st = orc.prefill(cmodel, sh, prompt, 256)
    tol = _depth_tol(ms.n_layers)
    record("7B, 32 layers h_last", tol=TOL, depth_tol=tol, **parity_stats(h_last[0], st.h_last, TOL))
    assert close(h_last[0], st.h_last) < tol
    for l, (k, v) in kv.items():
        assert_close_large(k, st.k[l][:len(prompt)], tol, f"7B, 32 layers K[{l}]", outliers=OUTLIERS_KV_DEEP)
        assert_close_large(v, st.v[l][:len(prompt)], tol, f"7B, 32 layers V[{l}]", outliers=OUTLIERS_KV_DEEP)
    want_tok = [int(t) for t in tree_tok[0]]
    # the oracle verifies the GPU's own tree (the root may sit at a near-tie after 32 layers; the candidates come
    # from the GPU's h_last): what is compared is the forward over identical tokens
    o_hidden, o_logits = orc.verify_tree(cmodel, sh, st, want_tok, tree.parent)
    assert_close_large(hidden[0], o_hidden, tol, "7B, 32 layers hidden", outliers=OUTLIERS_HIDDEN_DEEP)
    assert_close_large(logits[0], o_logits, tol, "7B, 32 layers logits", outliers=OUTLIERS_LOGITS_DEEP)
    assert torch.equal(node_argmax[0].long().cpu(), torch.argmax(logits[0], dim=-1).cpu())
    check_argmax_flips(node_argmax[0], o_logits, tol, 8, "7B, 32 layers")


def test_7b_width_one_node_step_against_oracle(cb):
    """The auto-regressive step (one row per sequence) takes its own code paths: the 16-row GEMM bucket
    with SwiGLU fused into the gate-up GEMM's epilogue, and the one-node attention layout."""
    ms = synth.shape_7b(n_layers=2)
    topk = [10, 10, 10, 10]
    model, layout, heads, eng = _engine(cb, ms, 4, topk, 512)
    cmodel, sh = cpu(model), oracle_shape(ms)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 150, seq=9)]
    th1 = eng.tree(synth.single_node_tree())
    eng.prefill(torch.tensor([prompt], dtype=torch.int32, device="cuda"), [len(prompt)])
    st = orc.prefill(cmodel, sh, prompt, 512)
    lens, roots, _ = eng.read_state()
    tok = torch.tensor([[int(roots[0])]], dtype=torch.int32, device="cuda")
    node_argmax, logits, hidden = eng.verify(th1, tok, want_logits=True, want_hidden=True)
    o_hidden, o_logits = orc.verify_tree(cmodel, sh, st, [int(roots[0])], synth.single_node_tree().parent)
    assert close(hidden[0], o_hidden) < TOL
    assert_close_large(logits[0], o_logits, TOL, "7B width, one-node step logits", outliers=OUTLIERS_LOGITS)
    assert int(node_argmax[0, 0]) == int(torch.argmax(logits[0, 0]))
    assert eng.device_status() == 0


def _depth_tol(n_layers: int) -> float:
    """Two bf16 forwards that differ only in summation order drift apart like a random walk: every
    rounding point re-quantises a tiny difference into one-ulp flips, about 0.2 % of the rms per
    layer, measured to grow with the square root of the depth (mean |dK| 0.0027 at layer 1, 0.0186
    at layer 31 of the 7B shape).  The 2e-2 bound that holds for two layers is scaled accordingly."""
    return TOL * max(1.0, (n_layers / 2.0) ** 0.5)


def _teacher_forced_steps(cb, eng, tree, prompts, n_steps, lengths):
    """At full depth a free-running comparison of two decoding runs is not meaningful (see _depth_tol:
    near-tied argmaxes flip), so the greedy-equivalence property is checked step by step from a shared
    state:
      * the tree forward and the one-node (auto-regressive) forward, run from the same committed state,
        give the same K/V for the root position (first layer tightly, last layer within the depth
        tolerance) and the same logits within the depth tolerance, and the same token whenever the
        top-2 margin is clear of that tolerance;
      * every argmax is exact on the kernel's own logits; acceptance equals the oracle's rule applied to
        those argmaxes (exact);
      * compaction moves the accepted nodes' K/V bit-exactly; len and the next root follow.
    Candidates are planted with the greedy continuation from the current state (obtained by chain-shaped
    forwards) so that paths of several tokens are accepted."""
    B = len(prompts)
    tol = _depth_tol(eng.shape.n_layers)
    maxlen = max(len(p) for p in prompts)
    tok = torch.zeros(B, maxlen, dtype=torch.int32, device="cuda")
    for b, p in enumerate(prompts):
        tok[b, :len(p)] = torch.tensor(p, dtype=torch.int32)
    lens0 = [len(p) for p in prompts]
    th, th1 = eng.tree(tree), eng.tree(synth.single_node_tree())
    max_want = max(lengths)
    chains = {j: eng.tree(synth.chain_tree(j)) for j in range(2, max_want)}
    eng.prefill(tok, lens0)
    layers = (0, eng.shape.n_layers - 1)
    emitted = [[] for _ in range(B)]
    accepted, agree, clear = [], 0, 0
    for step in range(n_steps):
        lens, roots, _ = eng.read_state()
        roots_t = torch.tensor(roots, dtype=torch.int32, device="cuda").reshape(B, 1)
        am1, lg1, _ = eng.verify(th1, roots_t, want_logits=True)
        kv1 = [[tuple(t[int(lens[b])].clone() for t in eng.gather_kv(b, l, int(lens[b]) + 1)) for l in layers] for b in range(B)]
        # the greedy continuation from this state, by chain-shaped forwards of growing length
        cont = [[int(roots[b]), int(am1[b, 0])] for b in range(B)]
        for j in range(2, max_want):
            ct = torch.tensor([c[:j] for c in cont], dtype=torch.int32, device="cuda")
            amc, _, _ = eng.verify(chains[j], ct)
            for b in range(B):
                cont[b].append(int(amc[b, j - 1]))
        tree_tok, _, _ = eng.draft(th)
        path = deepest_path(tree)
        for b in range(B):
            assert int(tree_tok[b, 0]) == int(roots[b])
            want = lengths[(step + b) % len(lengths)]
            for j, node in enumerate(path[1:want], start=1):
                tree_tok[b, node] = cont[b][j]
        am, lg, _ = eng.verify(th, tree_tok, want_logits=True)
        torch.cuda.synchronize()
        snap = [[tuple(t[int(lens[b]):].clone() for t in eng.gather_kv(b, l, int(lens[b]) + tree.n)) for l in layers] for b in range(B)]
        for b in range(B):
            assert_close_large(lg[b, 0], lg1[b, 0], tol, "root logits, tree vs one-node forward")
            assert close(snap[b][0][0][0], kv1[b][0][0]) < 1e-2 and close(snap[b][0][1][0], kv1[b][0][1]) < 1e-2
            assert_close_large(snap[b][1][0][0], kv1[b][1][0], tol, "last layer K of the root")
            assert_close_large(snap[b][1][1][0], kv1[b][1][1], tol, "last layer V of the root")
            if top2_margin(lg1[b, 0].cpu()) >= 2 * tol:
                clear += 1
                assert int(am[b, 0]) == int(am1[b, 0])
            agree += int(am[b, 0]) == int(am1[b, 0])
            assert torch.equal(am[b].long().cpu(), torch.argmax(lg[b], dim=-1).cpu())
        n_acc, path, toks = eng.accept(th, tree_tok, am)
        torch.cuda.synchronize()
        lens2, roots2, _ = eng.read_state()
        for b in range(B):
            opath = orc.accept_longest([int(t) for t in tree_tok[b]], [int(a) for a in am[b]], tree.parent)
            na = int(n_acc[b])
            assert [int(p) for p in path[b, :na]] == opath
            assert [int(t) for t in toks[b, :na]] == [int(tree_tok[b, p]) for p in opath]
            assert lens2[b] == lens[b] + na and roots2[b] == int(am[b, opath[-1]])
            for li, l in enumerate(layers):
                k, v = eng.gather_kv(b, l, int(lens2[b]))
                for j, pj in enumerate(opath):
                    assert torch.equal(k[int(lens[b]) + j], snap[b][li][0][pj]) and torch.equal(v[int(lens[b]) + j], snap[b][li][1][pj])
            emitted[b].extend(int(t) for t in toks[b, :na])
            accepted.append(na)
    assert eng.device_status() == 0
    return accepted, agree, clear, n_steps * B


def test_7b_full_depth_tree_and_autoregressive_paths_agree(cb):
    ms = synth.shape_7b()
    topk = [10, 10, 10, 10]
    model, layout, heads, eng = _engine(cb, ms, 4, topk, 1024)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 600, seq=8)]
    tree = synth.best_first_tree(64, topk)
    accepted, agree, clear, total = _teacher_forced_steps(cb, eng, tree, [prompt], 10, [1, 2, 3, 4, 5])
    assert max(accepted) >= 3 and min(accepted) >= 1
    assert agree >= 0.6 * total


def test_13b_width_batch_of_four_tree_and_autoregressive_paths_agree(cb):
    ms = synth.shape_13b(n_layers=3)
    topk = [10] * 5
    model, layout, heads, eng = _engine(cb, ms, 5, topk, 512, max_batch=4)
    prompts = [[int(t) for t in synth.make_prompt(ms.vocab, L, seq=10 + i)] for i, L in enumerate((300, 140, 257, 31))]
    tree = synth.best_first_tree(64, topk)
    accepted, agree, clear, total = _teacher_forced_steps(cb, eng, tree, prompts, 6, [2, 5, 1, 3])
    assert max(accepted) >= 4
    assert agree >= 0.8 * total


@pytest.mark.parametrize("M,N,K", [(2048, 22016, 4096), (2048, 4096, 11008), (1024, 12288, 4096), (512, 32000, 4096),
                                   (256, 27648, 5120)])
def test_gemm_at_the_batched_steps_sizes_on_sampled_outputs(cb, M, N, K):
    """The projections of the 7B shape (gate/up, down, QKV, LM head) at the row counts of the batched verify steps
    (16 sequences x 128 / 64 / 32 nodes) and the 13B gate/up at 256 rows: the 256 x 256 units and the row chunks that
    walk the weights side by side.  The oracle computes a sample of 96 output rows x 384 output columns (first and
    last rows of every row chunk and first and last columns included) from its definition."""
    X = synth.normal(12, 1, (M, K), 1.0, dtype=torch.bfloat16, device="cuda")
    W = synth.normal(12, 2, (N, K), 0.05, dtype=torch.bfloat16, device="cuda")
    out = cb.gemm(X, W)
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
    def sample(must, tensor_id, count, high):
        picked = list(dict.fromkeys(must))
        for v in synth.randint(12, tensor_id, (4 * count,), high):
            if len(picked) >= count:
                break
            if int(v) not in picked:
                picked.append(int(v))
        return sorted(picked)

    rows = sample([0, M - 1] + [c * 256 + d for c in range(M // 256) for d in (0, 255)], 3, 96, M)
    cols = sample([0, 1, 127, 128, 255, 256, N - 257, N - 256, N - 1], 4, 384, N)
    ri, ci = torch.tensor(rows), torch.tensor(cols)
    ref = orc.linear(X.cpu()[ri], W.cpu()[ci])
    got = out.cpu()[ri][:, ci]
    assert close(got, ref, 0) < 2e-4
    # every output element, against the sum of its row's products in another order (a property that holds at any
    # size): column sums of the whole matrix equal X^T-weighted sums computed from the sampled definition
    colsum = out.double().sum(dim=0).cpu()[ci]
    ref_colsum = orc.linear(X.double().sum(dim=0, keepdim=True).cpu(), W.cpu()[ci].double())[0]
    assert float(((colsum - ref_colsum).abs() / (1.0 + ref_colsum.abs())).max()) < 2e-3


def test_7b_width_batch_of_16_with_128_node_trees_against_oracle(cb):
    """The largest batched verify step (16 sequences x 128 nodes = 2048 rows) at the 7B width, two layers: GEMMs in
    row chunks walked side by side, the 128-row tensor-core attention, ragged prompts.  One sequence of the batch is
    checked against the oracle (prefill state, hidden states and logits of all its 128 nodes, every argmax decision)."""
    ms = synth.shape_7b(n_layers=2)
    topk = [10, 10, 10, 10]
    B, pick = 16, 5
    model, layout, heads, eng = _engine(cb, ms, 4, topk, 400, max_batch=B)
    cmodel, sh = cpu(model), oracle_shape(ms)
    lens = [60 + 17 * b for b in range(B)]
    prompts = [[int(t) for t in synth.make_prompt(ms.vocab, L, seq=80 + b)] for b, L in enumerate(lens)]
    tok = torch.zeros(B, max(lens), dtype=torch.int32, device="cuda")
    for b, p in enumerate(prompts):
        tok[b, :len(p)] = torch.tensor(p, dtype=torch.int32)
    eng.prefill(tok, lens)
    tree = synth.random_parent_tree(128, 6, tree_id=77)
    th = eng.tree(synth.Tree(tree.parent, np.clip(tree.head, 0, 3), tree.rank))
    tt = torch.stack([synth.make_prompt(ms.vocab, 128, seq=120 + b).to(torch.int32) for b in range(B)]).cuda().contiguous()
    node_argmax, logits, hidden = eng.verify(th, tt, want_logits=True, want_hidden=True)
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    assert torch.equal(node_argmax.long().cpu(), torch.argmax(logits, dim=-1).cpu())
    st = orc.prefill(cmodel, sh, prompts[pick], 600)
    _, _, h_last = eng.read_state()
    assert close(h_last[pick], st.h_last) < TOL
    o_hidden, o_logits = orc.verify_tree(cmodel, sh, st, [int(t) for t in tt[pick]], tree.parent)
    assert_close_large(hidden[pick], o_hidden, TOL, "7B width, batch 16 x 128 nodes hidden", outliers=OUTLIERS_HIDDEN)
    assert_close_large(logits[pick], o_logits, TOL, "7B width, batch 16 x 128 nodes logits", outliers=OUTLIERS_LOGITS)
    check_argmax_flips(node_argmax[pick], o_logits, FLIP_MARGIN, 2 * MAX_FLIPS_64, "7B width, batch 16 x 128 nodes")
