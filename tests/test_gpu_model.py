"""Parity of the whole decoding step (prefill, gate, draft, verify, accept, step) with the CPU
oracle on small models, through the C ABI, plus properties that hold at any size."""
import numpy as np
import pytest
import torch

from oracle import cerberus_oracle as orc
from paper_2410_13344_b200 import synth
from tests.helpers import close, concat_src, cpu, oracle_planter, oracle_shape, plant_tokens, top2_margin

pytestmark = pytest.mark.gpu

TOL = {"bf16": 2e-2, "fp32": 1e-4}
TIE = 1e-3


@pytest.fixture(scope="module")
def cb():
    from paper_2410_13344_b200 import binding
    return binding


class Rig:
    """A model on the GPU (library) and the same weights on the CPU (oracle)."""

    def __init__(self, cb, ms, n_cheads=4, n_levels=4, topk=(4, 2, 1, 1), concat_level=None, max_tokens=512,
                 max_batch=1, max_nodes=64, std=0.02, shuffled=True):
        self.ms = ms
        self.model = synth.make_model(ms, device="cuda", std=std)
        self.layout = (synth.medusa_layout(n_cheads, n_levels) if concat_level == "medusa"
                       else synth.cerberus_layout(n_cheads, n_levels, concat_level))
        self.heads = synth.make_heads(ms, self.layout, device="cuda", std=std)
        self.topk = list(topk)
        max_pages = (max_tokens + max_nodes + 15) // 16
        pt = None
        if shuffled:
            pt = np.stack([synth.shuffled_page_table(max_pages, max_pages, table_id=900 + b, first=b * max_pages)
                           for b in range(max_batch)])
        self.eng = cb.Cerberus(ms, self.model, self.layout, self.heads, self.topk, max_tokens=max_tokens,
                               max_batch=max_batch, max_nodes=max_nodes, page_table=pt)
        self.cmodel, self.cheads = cpu(self.model), cpu(self.heads)
        self.sh = oracle_shape(ms)
        self.csrc = concat_src(self.layout)


def _run_gpu(rig, th, T, prompt, n_new, plant_fn=None):
    eng = rig.eng
    tok = torch.tensor([prompt], dtype=torch.int32, device="cuda")
    eng.prefill(tok, [len(prompt)])
    out, recs = [], []
    while len(out) < n_new:
        plant = None
        if plant_fn is not None:
            plant = torch.tensor([plant_fn(len(recs), len(out))], dtype=torch.int32, device="cuda")
        eng.step(th, T, plant)
        torch.cuda.synchronize()
        na = int(eng.h_n_accept[0])
        toks = [int(t) for t in eng.h_tokens[0, :na]]
        recs.append(dict(S=float(eng.h_S[0]), mode=int(eng.h_mode[0]), n_accept=na, tokens=toks))
        out.extend(toks)
    assert eng.wait_diagnosis() == [0, 0, 0, 0]        # no bounded wait ran out: code, wait, block and launch all unset
    assert eng.device_status() == 0
    return out[:n_new], recs


def _compare_runs(rig, gpu_recs, orc_recs, tol_S, allow_tie_divergence):
    """Step-by-step comparison.  With bf16 a near-tie in an argmax may legitimately flip; from that
    step on the two runs decode different prefixes and are no longer comparable."""
    compared = 0
    for g, o in zip(gpu_recs, orc_recs):
        same = g["mode"] == o.mode and g["tokens"] == o.tokens
        if not same and allow_tie_divergence:
            return compared, False
        assert abs(g["S"] - o.S) < tol_S, (compared, g, o.S)
        assert g["mode"] == o.mode, (compared, g, o.S)
        assert g["tokens"] == o.tokens and g["n_accept"] == len(o.path), (compared, g, o.tokens)
        compared += 1
    return compared, True


@pytest.fixture(scope="module")
def tiny_fp32(cb):
    return Rig(cb, synth.tiny_shape("fp32"))


def test_config1_greedy_decoding_matches_oracle(cb, tiny_fp32):
    """Tiny fp32 decoder, 64-token prompt, 16-node tree from top-{4,2,1,1}, threshold at the
    median gate value over 32 auto-regressive steps, 32 decoded tokens."""
    rig = tiny_fp32
    prompt = [int(t) for t in synth.make_prompt(rig.ms.vocab, 64)]
    truth, Ss = orc.ar_greedy(rig.cmodel, rig.sh, prompt, 40)
    T = orc.calibrate_threshold(Ss[:32])
    tree = synth.best_first_tree(16, rig.topk)
    th = rig.eng.tree(tree)
    toks, recs = _run_gpu(rig, th, T, prompt, 32)
    otoks, orecs, ost = orc.cerberus_greedy(rig.cmodel, rig.sh, rig.cheads, rig.csrc, prompt, tree.parent, tree.head,
                                            tree.rank, rig.topk, T, 32)
    assert toks == truth[:32] == otoks
    n, ok = _compare_runs(rig, recs, orecs, 1e-4, False)
    assert ok and n == len(orecs) and {r["mode"] for r in recs} == {0, 1}
    lens, roots, h_last = rig.eng.read_state()
    assert lens[0] == ost.length and roots[0] == ost.root
    assert close(h_last[0], ost.h_last, 0) < TOL["fp32"]
    for l in range(rig.ms.n_layers):
        k, v = rig.eng.gather_kv(0, l, ost.length)
        assert close(k, ost.k[l][:ost.length], 0) < TOL["fp32"]
        assert close(v, ost.v[l][:ost.length], 0) < TOL["fp32"]
    rig.eng.free_tree(th)


@pytest.mark.parametrize("thr", ["median", "always_par"])
def test_config1_planted_candidates_are_accepted(cb, tiny_fp32, thr):
    rig = tiny_fp32
    prompt = [int(t) for t in synth.make_prompt(rig.ms.vocab, 64, seq=1)]
    truth, Ss = orc.ar_greedy(rig.cmodel, rig.sh, prompt, 48)
    T = orc.calibrate_threshold(Ss[:32]) if thr == "median" else 1e9
    tree = synth.best_first_tree(16, rig.topk)
    th = rig.eng.tree(tree)
    lengths = [1, 3, 5, 2, 4, 1, 2]
    toks, recs = _run_gpu(rig, th, T, prompt, 32,
                          lambda step, emitted: plant_tokens(tree, truth, emitted, lengths[step % len(lengths)]))
    otoks, orecs, ost = orc.cerberus_greedy(rig.cmodel, rig.sh, rig.cheads, rig.csrc, prompt, tree.parent, tree.head,
                                            tree.rank, rig.topk, T, 32, plant=oracle_planter(tree, truth, lengths))
    assert toks == truth[:32] == otoks
    n, ok = _compare_runs(rig, recs, orecs, 1e-4, False)
    assert ok and n == len(orecs)
    assert max(r["n_accept"] for r in recs) >= 4
    lens, _, _ = rig.eng.read_state()
    for l in range(rig.ms.n_layers):
        k, v = rig.eng.gather_kv(0, l, int(lens[0]))
        assert close(k, ost.k[l][:ost.length], 0) < TOL["fp32"] and close(v, ost.v[l][:ost.length], 0) < TOL["fp32"]
    rig.eng.free_tree(th)


@pytest.mark.parametrize("mode", ["cerberus", "no_gate", "medusa_heads", "autoregressive"])
def test_comparison_modes_all_emit_the_greedy_continuation(cb, mode):
    """The decoding variants the paper compares (Sec. 5: independent heads without the sequential link,
    the gate switched off, plain auto-regressive decoding) differ in speed, never in output: each emits
    the base model's greedy continuation, and each step matches the oracle run in the same mode."""
    ms = synth.tiny_shape("fp32")
    rig = Rig(cb, ms, concat_level="medusa" if mode == "medusa_heads" else None)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 48, seq=3)]
    truth, Ss = orc.ar_greedy(rig.cmodel, rig.sh, prompt, 40)
    T = {"cerberus": orc.calibrate_threshold(Ss[:24]), "no_gate": 1e9, "medusa_heads": 1e9, "autoregressive": -1.0}[mode]
    tree = synth.best_first_tree(16, rig.topk)
    th = rig.eng.tree(tree)
    lengths = [2, 4, 1, 3]
    toks, recs = _run_gpu(rig, th, T, prompt, 24,
                          lambda step, emitted: plant_tokens(tree, truth, emitted, lengths[step % len(lengths)]))
    otoks, orecs, _ = orc.cerberus_greedy(rig.cmodel, rig.sh, rig.cheads, rig.csrc, prompt, tree.parent, tree.head,
                                          tree.rank, rig.topk, T, 24, plant=oracle_planter(tree, truth, lengths))
    assert toks == truth[:24] == otoks
    n, ok = _compare_runs(rig, recs, orecs, 1e-4, False)
    assert ok and n == len(orecs)
    modes = {r["mode"] for r in recs}
    if mode == "autoregressive":
        assert modes == {1} and all(r["n_accept"] == 1 for r in recs)
    elif mode != "cerberus":
        assert modes == {0} and max(r["n_accept"] for r in recs) >= 3
    rig.eng.free_tree(th)


@pytest.mark.parametrize("dtype,concat_level", [("fp32", None), ("fp32", 1), ("bf16", None), ("fp32", "medusa")])
def test_each_call_matches_oracle(cb, dtype, concat_level):
    """cerb_gate / cerb_draft / cerb_verify / cerb_accept one by one, with values."""
    ms = synth.tiny_shape(dtype)
    rig = Rig(cb, ms, concat_level=concat_level, topk=(4, 3, 2, 2))
    tol = TOL[dtype]
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 37, seq=2)]
    eng = rig.eng
    eng.prefill(torch.tensor([prompt], dtype=torch.int32, device="cuda"), [len(prompt)])
    st = orc.prefill(rig.cmodel, rig.sh, prompt, 256)
    lens, roots, h_last = eng.read_state()
    assert lens[0] == len(prompt)
    assert close(h_last[0], st.h_last, 0) < tol
    if roots[0] != st.root:
        lg = orc.linear(st.h_last[None], rig.cmodel["lm_head"])[0]
        assert top2_margin(lg) < TIE
        pytest.skip("argmax tie at the prompt's last position")
    # gate
    S, mode = eng.gate(0.0)
    assert abs(float(S[0]) - orc.gate_entropy(st.h_last)) < (1e-4 if dtype == "fp32" else 2e-2)
    # draft
    tree = synth.best_first_tree(24, rig.topk)
    th = eng.tree(tree)
    tree_tok, topk, hlog = eng.draft(th, want_logits=True)
    olog = orc.heads_forward(st.h_last if dtype == "fp32" else h_last[0].double(), rig.cheads, rig.csrc)
    for h in range(4):
        assert close(hlog[0, h], olog[h], 0) < (1e-4 if dtype == "fp32" else 5e-3)
        want = list(orc.topk_ids(hlog[0, h].cpu().double(), rig.topk[h]))      # decision on the kernel's own logits
        assert [int(t) for t in topk[0, h, :rig.topk[h]]] == want
    want_tok = [int(roots[0])] + [int(topk[0, tree.head[v], tree.rank[v]]) for v in range(1, tree.n)]
    assert [int(t) for t in tree_tok[0]] == want_tok
    # verify
    node_argmax, logits, hidden = eng.verify(th, tree_tok, want_logits=True, want_hidden=True)
    o_hidden, o_logits = orc.verify_tree(rig.cmodel, rig.sh, st, want_tok, tree.parent)
    assert close(hidden[0], o_hidden, 0) < tol
    assert close(logits[0], o_logits, 0) < tol
    o_arg = [int(a) for a in orc.argmax_f32(o_logits)]
    for v in range(tree.n):
        if int(node_argmax[0, v]) != o_arg[v]:
            assert top2_margin(o_logits[v]) < TIE
        assert int(node_argmax[0, v]) == int(torch.argmax(logits[0, v]))
    # accept, with candidates planted so that something beyond the root is accepted
    fake_argmax = node_argmax.clone()
    path = [0]
    for _ in range(3):
        kids = [c for c in range(tree.n) if tree.parent[c] == path[-1]]
        if not kids:
            break
        fake_argmax[0, path[-1]] = tree_tok[0, kids[-1]]
        path.append(kids[-1])
    n_acc, gpath, gtok = eng.accept(th, tree_tok, fake_argmax)
    opath = orc.accept_longest(want_tok, [int(a) for a in fake_argmax[0]], tree.parent)
    assert int(n_acc[0]) == len(opath) >= 2
    assert [int(p) for p in gpath[0, :len(opath)]] == opath
    assert [int(t) for t in gtok[0, :len(opath)]] == [want_tok[p] for p in opath]
    orc.compact(st, opath)
    lens, roots, h_last = eng.read_state()
    assert lens[0] == len(prompt) + len(opath) and roots[0] == int(fake_argmax[0, opath[-1]])
    assert close(h_last[0], o_hidden[opath[-1]], 0) < tol
    L = int(lens[0])
    for l in range(ms.n_layers):
        k, v = eng.gather_kv(0, l, L)
        assert close(k, st.k[l][:L], 0) < tol and close(v, st.v[l][:L], 0) < tol
    assert eng.device_status() == 0


def test_tiny_bf16_greedy_decoding_matches_oracle(cb):
    """bf16 model, planted candidates: the run must follow the oracle's step by step.  Where the two part, the
    step at which they part must hinge on a near-tie: either the gate value within the entropy tolerance of the
    threshold, or the oracle's two best logits at the deciding node within the bf16 logit tolerance."""
    ms = synth.tiny_shape("bf16")
    rig = Rig(cb, ms)
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 64, seq=3)]
    truth, Ss = orc.ar_greedy(rig.cmodel, rig.sh, prompt, 40)
    T = orc.calibrate_threshold(Ss[:32], min_gap=0.05)
    tree = synth.best_first_tree(16, rig.topk)
    th = rig.eng.tree(tree)
    lengths = [2, 1, 4, 3, 1]
    toks, recs = _run_gpu(rig, th, T, prompt, 32,
                          lambda step, emitted: plant_tokens(tree, truth, emitted, lengths[step % len(lengths)]))
    # the oracle run, step by step, keeping every step's logits
    st = orc.prefill(rig.cmodel, rig.sh, prompt, len(prompt) + 32 + 2 * tree.n + 8)
    plant = oracle_planter(tree, truth, lengths)
    otoks, orecs, ologits = [], [], []
    last_logits = orc.forward_full(rig.cmodel, rig.sh, prompt)[1][-1]          # decides the first root
    deciding = [last_logits]                                                    # logits that decide step i's root
    while len(otoks) < 32:
        i, emitted = len(orecs), list(otoks)
        rec, _, logits = orc.step(rig.cmodel, rig.sh, st, rig.cheads, rig.csrc, tree.parent, tree.head, tree.rank,
                                  rig.topk, T, lambda tt: plant(tt, i, emitted), return_values=True)
        orecs.append(rec)
        ologits.append(logits)
        otoks.extend(rec.tokens)
        deciding.append(logits[rec.path[-1]])
    n, ok = _compare_runs(rig, recs, orecs, 2e-2, True)
    if ok:
        assert toks == otoks[:32]
        return
    g, o = recs[n], orecs[n]
    if g["mode"] != o.mode:
        assert abs(o.S - T) < 2e-2, (n, g, o.S, T)              # the gate value sits at the threshold
        return
    j = 0
    while j < min(len(g["tokens"]), len(o.tokens)) and g["tokens"][j] == o.tokens[j]:
        j += 1
    row = deciding[n] if j == 0 else ologits[n][o.path[j - 1]]   # the oracle's logits at the node that decided
    assert top2_margin(row) < 2e-2, (n, j, g, o.tokens, top2_margin(row))
    if j < len(g["tokens"]):                                     # the token the GPU took instead is the runner-up
        assert float(row.max() - row[g["tokens"][j]]) < 2e-2, (n, j, g, o.tokens)


@pytest.mark.parametrize("lens", [(150, 21), (33, 70, 5, 128)])
def test_batch_with_ragged_prompts_and_mixed_modes(cb, lens):
    """Every sequence of a batch is gated on its own (Algorithm 1 applied per sequence).  In a step where some
    sequences draft and others decode auto-regressively, the rows of the forward are ragged: n rows for a drafting
    sequence, one for an auto-regressive one.  Step by step and sequence by sequence: entropy, mode, accepted
    length and tokens against the oracle's run of that sequence alone; the forward's row count against the modes."""
    ms = synth.tiny_shape("fp32")
    B = len(lens)
    rig = Rig(cb, ms, max_batch=B, max_tokens=400)
    prompts = [[int(t) for t in synth.make_prompt(ms.vocab, L, seq=4 + i)] for i, L in enumerate(lens)]
    tok = torch.zeros(B, max(lens), dtype=torch.int32, device="cuda")
    for b, p in enumerate(prompts):
        tok[b, :len(p)] = torch.tensor(p, dtype=torch.int32)
    eng = rig.eng
    eng.prefill(tok, list(lens))
    tree = synth.best_first_tree(16, rig.topk)
    th = eng.tree(tree)
    n_steps = 12
    truths = [orc.ar_greedy(rig.cmodel, rig.sh, p, n_steps + 8) for p in prompts]
    T = orc.calibrate_threshold(sorted(sum((t[1][:n_steps] for t in truths), [])), 0.5)
    lengths = [3, 1, 4, 2]
    # the oracle decodes every sequence on its own, with the same planted candidates
    oruns = [orc.cerberus_greedy(rig.cmodel, rig.sh, rig.cheads, rig.csrc, prompts[b], tree.parent, tree.head, tree.rank,
                                 rig.topk, T, 5 * n_steps, plant=oracle_planter(tree, truths[b][0] + [0] * 64, lengths))[1]
             for b in range(B)]
    outs = [[] for _ in range(B)]
    modes, mixed = set(), 0
    for step in range(n_steps):
        plant = torch.tensor([plant_tokens(tree, truths[b][0] + [0] * 64, len(outs[b]), lengths[step % len(lengths)])
                              for b in range(B)], dtype=torch.int32, device="cuda")
        eng.step(th, T, plant)
        torch.cuda.synchronize()
        step_modes = [int(eng.h_mode[b]) for b in range(B)]
        want_rows = sum(1 if m == cb.MODE_AR else tree.n for m in step_modes) if 0 in step_modes else B
        assert eng.last_forward_rows() == want_rows, (step, step_modes)
        mixed += len(set(step_modes)) == 2
        for b in range(B):
            o = oruns[b][step]
            na = int(eng.h_n_accept[b])
            assert abs(float(eng.h_S[b]) - o.S) < 1e-4 and step_modes[b] == o.mode, (step, b)
            assert na == len(o.path) and [int(t) for t in eng.h_tokens[b, :na]] == o.tokens, (step, b)
            outs[b].extend(o.tokens)
            modes.add(step_modes[b])
    for b in range(B):
        k = min(len(outs[b]), n_steps + 8)
        assert outs[b][:k] == truths[b][0][:k]
    assert modes == {0, 1} and mixed >= 2
    assert eng.device_status() == 0


def test_bf16_mixed_mode_batch_at_head_dim_128(cb):
    """Ragged rows through the bf16 kernels (row offsets in the norm, RoPE, the keys-on-M attention kernel, argmax
    and accept).  A mixed-mode batch is decoded twice with its sequences in a different order (other row offsets,
    other page tables): every sequence must give the same entropies, modes, accepted lengths and tokens in both
    runs, must emit its own auto-regressive continuation (taken from single-sequence runs, the path the other tests
    hold against the oracle), and the forward's row count must follow the modes."""
    ms = synth.ModelShape(2, 256, 2, 128, 512, 1024, "bf16")
    lens = (40, 75, 9, 130)
    B = len(lens)
    rig = Rig(cb, ms, max_batch=B, max_tokens=400)
    eng = rig.eng
    tree = synth.best_first_tree(24, rig.topk)
    th, th1 = eng.tree(tree), eng.tree(synth.single_node_tree())
    prompts = [[int(t) for t in synth.make_prompt(ms.vocab, L, seq=40 + i)] for i, L in enumerate(lens)]
    n_steps, lengths = 10, [3, 1, 4, 2]

    def alone(b, n):
        """n auto-regressive steps of sequence b on its own (threshold below any entropy)."""
        eng.prefill(torch.tensor([prompts[b]], dtype=torch.int32, device="cuda"), [lens[b]])
        Ss, out = [], []
        for _ in range(n):
            eng.step(th1, -1.0, None)
            torch.cuda.synchronize()
            assert int(eng.h_mode[0]) == cb.MODE_AR and int(eng.h_n_accept[0]) == 1
            Ss.append(float(eng.h_S[0]))
            out.append(int(eng.h_tokens[0, 0]))
        return Ss, out

    runs = [alone(b, 5 * n_steps) for b in range(B)]
    truths = [r[1] + [0] * 64 for r in runs]
    # a threshold in the widest gap of the entropies seen on those paths, so that both modes occur
    Ss = sorted(S for r in runs for S in r[0][:n_steps])
    g, i = max((Ss[k + 1] - Ss[k], k) for k in range(len(Ss) // 4, 3 * len(Ss) // 4))
    T = 0.5 * (Ss[i] + Ss[i + 1])

    def batch(order):
        tok = torch.zeros(B, max(lens), dtype=torch.int32, device="cuda")
        for pos, b in enumerate(order):
            tok[pos, :lens[b]] = torch.tensor(prompts[b], dtype=torch.int32)
        eng.prefill(tok, [lens[b] for b in order])
        outs = {b: [] for b in order}
        recs = {b: [] for b in order}
        mixed = 0
        for step in range(n_steps):
            plant = torch.tensor([plant_tokens(tree, truths[b], len(outs[b]), lengths[step % len(lengths)]) for b in order],
                                 dtype=torch.int32, device="cuda")
            eng.step(th, T, plant)
            torch.cuda.synchronize()
            modes = [int(eng.h_mode[pos]) for pos in range(B)]
            want_rows = sum(1 if m == cb.MODE_AR else tree.n for m in modes) if cb.MODE_PAR in modes else B
            assert eng.last_forward_rows() == want_rows, (step, modes)
            mixed += len(set(modes)) == 2
            for pos, b in enumerate(order):
                na = int(eng.h_n_accept[pos])
                toks = [int(t) for t in eng.h_tokens[pos, :na]]
                recs[b].append((float(eng.h_S[pos]), modes[pos], toks))
                outs[b].extend(toks)
        assert eng.device_status() == 0
        return recs, outs, mixed

    recs_a, outs_a, mixed_a = batch((0, 1, 2, 3))
    recs_b, outs_b, mixed_b = batch((2, 0, 3, 1))
    seen = set()
    for b in range(B):
        for step, (ra, rb) in enumerate(zip(recs_a[b], recs_b[b])):
            assert ra[1] == rb[1] and ra[2] == rb[2] and abs(ra[0] - rb[0]) < 1e-5, (b, step, ra, rb)
            seen.add(ra[1])
        assert outs_a[b] == truths[b][:len(outs_a[b])] and len(outs_a[b]) >= n_steps, (b, outs_a[b], truths[b][:len(outs_a[b])])
    assert seen == {cb.MODE_AR, cb.MODE_PAR} and mixed_a >= 2 and mixed_a == mixed_b, (seen, mixed_a, mixed_b, g)


def test_batch_16_with_128_node_trees(cb):
    """Sweep corner at small width: 16 ragged sequences, a 128-node tree (two ancestor words, 2048 rows
    per forward), planted candidates; every sequence must emit its own auto-regressive continuation."""
    ms = synth.tiny_shape("fp32")
    rig = Rig(cb, ms, max_batch=16, max_tokens=400, max_nodes=128, topk=(10, 10, 10, 10))
    B = 16
    lens = [20 + 13 * b for b in range(B)]
    prompts = [[int(t) for t in synth.make_prompt(ms.vocab, L, seq=30 + b)] for b, L in enumerate(lens)]
    tok = torch.zeros(B, max(lens), dtype=torch.int32, device="cuda")
    for b, p in enumerate(prompts):
        tok[b, :len(p)] = torch.tensor(p, dtype=torch.int32)
    eng = rig.eng
    tree = synth.best_first_tree(128, rig.topk)
    th = eng.tree(tree)
    n_new = 8
    truths = [orc.ar_greedy(rig.cmodel, rig.sh, p, n_new + 6)[0] for p in prompts]
    eng.prefill(tok, lens)
    outs = [[] for _ in range(B)]
    best = 0
    for step in range(n_new):
        plant = torch.tensor([plant_tokens(tree, truths[b], len(outs[b]), 1 + (step + b) % 5) for b in range(B)],
                             dtype=torch.int32, device="cuda")
        eng.step(th, 1e9, plant)
        torch.cuda.synchronize()
        for b in range(B):
            na = int(eng.h_n_accept[b])
            best = max(best, na)
            outs[b].extend(int(t) for t in eng.h_tokens[b, :na])
    for b in range(B):
        k = min(len(outs[b]), n_new + 6)
        assert outs[b][:k] == truths[b][:k], b
    assert best >= 4
    assert eng.device_status() == 0


def test_threshold_calibration_helper(cb, tiny_fp32):
    """calibrate_threshold decodes auto-regressively and returns the gate value that splits the observed
    entropies at the requested fraction; replaying the same steps shows that fraction below it."""
    rig = tiny_fp32
    prompt = [int(t) for t in synth.make_prompt(rig.ms.vocab, 40, seq=5)]
    tok = torch.tensor([prompt], dtype=torch.int32, device="cuda")
    th = rig.eng.tree(synth.best_first_tree(16, rig.topk))
    rig.eng.prefill(tok, [len(prompt)])
    T = rig.eng.calibrate_threshold(th, 20, 0.6)
    _, Ss = orc.ar_greedy(rig.cmodel, rig.sh, prompt, 20)
    assert sum(1 for v in Ss[:20] if v <= T) == 12
    rig.eng.free_tree(th)


def test_profiling_modes(cb):
    """Mode 1 brackets every kernel family with events; mode 2 lets each bf16 GEMM launch stamp its own span
    with the device timer.  Both count the GEMMs of one verification forward: four per layer and the LM head."""
    ms = synth.tiny_shape("bf16")
    rig = Rig(cb, ms)
    eng = rig.eng
    prompt = [int(t) for t in synth.make_prompt(ms.vocab, 30, seq=6)]
    eng.prefill(torch.tensor([prompt], dtype=torch.int32, device="cuda"), [len(prompt)])
    th = eng.tree(synth.best_first_tree(16, rig.topk))
    tok = torch.zeros(1, 16, dtype=torch.int32, device="cuda")
    n_gemm = 4 * ms.n_layers + 1
    for mode in (1, 2):
        eng.profile(mode)
        eng.profile_read()
        eng.verify(th, tok)
        prof = eng.profile_read()
        assert prof["gemm"][1] == n_gemm and 0.0 < prof["gemm"][0] < 1e3, (mode, prof)
        if mode == 1:
            assert prof["attention"][1] == ms.n_layers and prof["glue"][1] > 0
        else:
            assert prof["attention"][1] == 0
    eng.profile(False)
    assert cb.lib().cerb_profile_enable(eng.ctx, 3) == cb.E_ARG
    assert eng.device_status() == 0


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_151_node_trees(cb, dtype):
    """The paper's widest setting (Sec. 5.1: top-10 per head, 150 candidate paths + the root): three ancestor
    words, attention in two launches of query rows.  Planted candidates; the run must emit the auto-regressive
    greedy continuation, and one verification forward must agree with the oracle node by node."""
    ms = synth.tiny_shape(dtype)
    rig = Rig(cb, ms, max_batch=2, max_tokens=400, max_nodes=160, topk=(10, 10, 10, 10))
    eng = rig.eng
    tree = synth.best_first_tree(151, rig.topk)
    th = eng.tree(tree)
    lens = [150, 37]
    prompts = [[int(t) for t in synth.make_prompt(ms.vocab, L, seq=60 + b)] for b, L in enumerate(lens)]
    tok = torch.zeros(2, max(lens), dtype=torch.int32, device="cuda")
    for b, p in enumerate(prompts):
        tok[b, :len(p)] = torch.tensor(p, dtype=torch.int32)
    eng.prefill(tok, lens)
    # one verification forward against the oracle's per-node definition (explicit root-to-node sequences)
    tt = torch.stack([synth.make_prompt(ms.vocab, 151, seq=70 + b).to(torch.int32) for b in range(2)]).cuda().contiguous()
    am, logits, _ = eng.verify(th, tt, want_logits=True)
    torch.cuda.synchronize()
    tol = 1e-4 if dtype == "fp32" else 2e-2
    for b in range(2):
        st = orc.prefill(rig.cmodel, rig.sh, prompts[b], 600)
        _, want = orc.verify_tree(rig.cmodel, rig.sh, st, [int(t) for t in tt[b]], tree.parent)
        assert close(logits[b], want, 0) < tol, b
        for v in (0, 63, 64, 127, 128, 150):
            assert int(am[b, v]) == int(orc.argmax_f32(logits[b, v].cpu().reshape(1, -1))[0]), (b, v)
    if dtype == "fp32":
        n_new = 8
        truths = [orc.ar_greedy(rig.cmodel, rig.sh, p, n_new + 6)[0] for p in prompts]
        eng.prefill(tok, lens)
        outs = [[], []]
        best = 0
        for step in range(n_new):
            plant = torch.tensor([plant_tokens(tree, truths[b], len(outs[b]), 1 + (step + b) % 5) for b in range(2)],
                                 dtype=torch.int32, device="cuda")
            eng.step(th, 1e9, plant)
            torch.cuda.synchronize()
            for b in range(2):
                na = int(eng.h_n_accept[b])
                best = max(best, na)
                outs[b].extend(int(t) for t in eng.h_tokens[b, :na])
        for b in range(2):
            k = min(len(outs[b]), n_new + 6)
            assert outs[b][:k] == truths[b][:k], b
        assert best >= 4
    assert eng.device_status() == 0


def test_verify_accept_loop_runs_to_the_true_capacity(cb):
    """The stand-alone calls keep only an upper bound of the committed length on the host (every cerb_accept adds
    the deepest possible path).  A loop of draft / verify / accept must still run until the sequence really fills
    its pages: the library fetches the true lengths once its bound reaches the end of the page table."""
    ms = synth.tiny_shape("fp32")
    rig = Rig(cb, ms, max_tokens=96, max_nodes=16)
    eng = rig.eng
    tree = synth.best_first_tree(16, rig.topk)
    th = eng.tree(tree)
    eng.prefill(torch.zeros(1, 8, dtype=torch.int32, device="cuda"), [8])
    capacity = 16 * eng.max_pages
    steps = 0
    while True:
        try:
            tree_tok, _, _ = eng.draft(th)
            am, _, _ = eng.verify(th, tree_tok)
            eng.accept(th, tree_tok, am)
        except cb.CerbError as e:
            assert e.code == cb.E_STATE
            break
        steps += 1
        assert steps < 200
    lens, _, _ = eng.read_state()
    # untrained heads: one token per step; the loop must have used the pages up, not stopped at the drifting bound
    assert int(lens[0]) + tree.n > capacity and int(lens[0]) >= capacity - tree.n - 4 and steps >= 60
    assert eng.device_status() == 0


def test_error_codes(cb):
    ms = synth.tiny_shape("fp32")
    rig = Rig(cb, ms, max_tokens=128)
    eng = rig.eng
    tree = synth.best_first_tree(16, rig.topk)
    with pytest.raises(cb.CerbError) as e:            # no sequence yet
        eng.gate(0.5)
    assert e.value.code == cb.E_STATE
    th = eng.tree(tree)
    eng.prefill(torch.zeros(1, 8, dtype=torch.int32, device="cuda"), [8])
    tt = torch.zeros(1, 16, dtype=torch.int32, device="cuda")
    with pytest.raises(cb.CerbError) as e:            # accept without verify
        eng.accept(th, tt, tt)
    assert e.value.code == cb.E_STATE
    bad = synth.Tree(np.array([-1, 0, 1, 0], np.int32), np.array([-1, 0, 1, 7], np.int32), np.zeros(4, np.int32))
    with pytest.raises(cb.CerbError) as e:            # head index outside the configuration
        eng.tree(bad)
    assert e.value.code == cb.E_ARG
    with pytest.raises(cb.CerbError) as e:            # prompt longer than the page table allows
        eng.prefill(torch.zeros(1, 4000, dtype=torch.int32, device="cuda"), [4000])
    assert e.value.code == cb.E_STATE
