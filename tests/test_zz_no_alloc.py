"""cerb_tree_attention_noalloc: the tree-attention entry point for callers that cannot allocate
device memory (allocator callbacks, plug-ins working in fixed buffers, processes with a device-memory
budget fixed at start-up).  Its split-KV scratch is a static array inside the library.  The check
is against the ordinary entry point on the same inputs, twice in a row, because the static array
keeps the previous call's contents and the second call must not be disturbed by them.

This file is named so that pytest collects it last."""
import math

import numpy as np
import pytest
import torch

from paper_2410_13344_b200 import synth

pytestmark = pytest.mark.gpu


def _inputs(cb, B, n, H, Dh, L, seed):
    max_len = L + n
    mp = (max_len + 15) // 16 + 1
    npool = B * mp
    tree = synth.random_parent_tree(n, 5, tree_id=seed)
    q = synth.normal(synth.SEED_ATTN, 500 + seed, (B, n, H, Dh), 1.0, dtype=torch.bfloat16, device="cuda")
    kp = synth.normal(synth.SEED_ATTN, 510 + seed, (npool, H, 16, Dh), 1.0, dtype=torch.bfloat16, device="cuda")
    vp = synth.normal(synth.SEED_ATTN, 520 + seed, (npool, H, 16, Dh), 1.0, dtype=torch.bfloat16, device="cuda")
    pt = torch.from_numpy(np.stack([synth.shuffled_page_table(mp, mp, table_id=700 + seed + b, first=b * mp)
                                    for b in range(B)])).cuda()
    anc = torch.from_numpy(cb.tree_ancestors(tree.parent).view(np.int64)).cuda()
    lens = torch.full((B,), L, dtype=torch.int32, device="cuda")
    return q, kp, vp, pt, lens, anc, 1.0 / math.sqrt(Dh), max_len


def _oracle_attention(q, kp, vp, pt, L, n, parent, scale, b):
    """The oracle's per-node definition for sequence b of the paged inputs."""
    from oracle import cerberus_oracle as orc
    H, Dh = q.shape[2], q.shape[3]
    pages = pt[b].cpu().long()
    kc = kp.cpu()[pages].permute(0, 2, 1, 3).reshape(-1, H, Dh).double()
    vc = vp.cpu()[pages].permute(0, 2, 1, 3).reshape(-1, H, Dh).double()
    return orc.tree_attention(q[b].cpu().double(), kc[:L], vc[:L], kc[L:L + n], vc[L:L + n], parent, scale)


def _compare_with_the_ordinary_entry(cb, cases):
    for B, n, H, Dh, L, seed in cases:
        q, kp, vp, pt, lens, anc, scale, max_len = _inputs(cb, B, n, H, Dh, L, seed)
        ref_out, ref_lse, _ = cb.tree_attention(q, kp, vp, pt, lens, anc, scale, max_len)
        out = torch.empty_like(q)
        lse = torch.empty(B, H, n, dtype=torch.float32, device="cuda")
        rc = cb.tree_attention_noalloc(q, kp, vp, pt, lens, anc, scale, max_len, out, lse)
        assert rc == cb.OK, cb.strerror(rc)
        torch.cuda.synchronize()
        # same kernel, same split plan, fixed-order merge: the tolerance of the other attention tests
        # (2e-2 combined abs/rel on bf16 outputs) is far from tight here
        err = float(((out.float() - ref_out.float()).abs() / (1 + ref_out.float().abs())).max())
        assert err < 2e-2, err
        assert float((lse - ref_lse).abs().max()) < 2e-3
        # ... and against the oracle's definition, for the last sequence of the batch
        tree = synth.random_parent_tree(n, 5, tree_id=seed)
        O, l = _oracle_attention(q, kp, vp, pt, L, n, tree.parent, scale, B - 1)
        assert float(((out[B - 1].double().cpu() - O).abs() / (1 + O.abs())).max()) < 2e-2
        assert float((lse[B - 1].double().cpu() - l).abs().max()) < 2e-3
        # no bounded wait ran out and no sequence was longer than announced
        assert cb.tree_attention_noalloc_status() == cb.OK


def test_noalloc_entry_matches_the_ordinary_one_twice_in_a_row():
    from paper_2410_13344_b200 import binding as cb
    # two different problems, back to back, both long enough to be split along the keys
    _compare_with_the_ordinary_entry(cb, [(1, 64, 8, 128, 3000, 1), (2, 33, 4, 128, 1500, 2)])


def test_noalloc_entry_with_partials_in_the_static_array():
    """By default the key splits of the head_dim-128 kernels merge inside a thread-block cluster and the static array
    only carries the status words.  With CERB_ATTN_CLUSTER=0 (read once per process) the splits write their partial
    results into the array and the last CTA to arrive merges them: run the comparison again in a child process with
    that switch, and once with head_dim 64 and a 150-node tree (two launches of query rows sharing the array)."""
    import os
    import subprocess
    import sys
    from paper_2410_13344_b200 import binding as cb
    _compare_with_the_ordinary_entry(cb, [(1, 150, 4, 64, 700, 3)])
    if os.environ.get("CERB_NOALLOC_CHILD"):
        return
    env = dict(os.environ, CERB_ATTN_CLUSTER="0", CERB_NOALLOC_CHILD="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_zz_no_alloc.py", "-q", "-x", "-m", "gpu"], cwd=root, env=env,
                       capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def _reject_or_accept(cb, B, n, H, Dh):
    q = torch.zeros(B, n, H, Dh, dtype=torch.bfloat16, device="cuda")
    pool = torch.zeros(B * 10, H, 16, Dh, dtype=torch.bfloat16, device="cuda")
    pt = torch.arange(B * 10, dtype=torch.int32, device="cuda").reshape(B, 10)
    lens = torch.zeros(B, dtype=torch.int32, device="cuda")
    anc = torch.from_numpy(cb.tree_ancestors(synth.chain_tree(n).parent).view(np.int64)).cuda()
    rc = cb.tree_attention_noalloc(q, pool, pool, pt, lens, anc, 1.0, n, torch.empty_like(q))
    torch.cuda.synchronize()
    return rc


def test_noalloc_entry_limits_are_the_documented_ones():
    """The bounds the header states for the 16 MiB array: 64-node trees at head_dim 128 up to B * n_heads = 168, no
    tree above 64 nodes at head_dim 128, 150-node trees at head_dim 64 up to B * n_heads = 153."""
    from paper_2410_13344_b200 import binding as cb
    assert _reject_or_accept(cb, 5, 64, 32, 128) == cb.OK
    assert _reject_or_accept(cb, 6, 64, 32, 128) == cb.E_NOMEM
    assert _reject_or_accept(cb, 1, 65, 1, 128) == cb.E_NOMEM
    assert _reject_or_accept(cb, 1, 150, 153, 64) == cb.OK
    assert _reject_or_accept(cb, 1, 150, 154, 64) == cb.E_NOMEM
    assert cb.tree_attention_noalloc_status() == cb.OK


def test_noalloc_entry_rejects_problems_beyond_its_static_scratch():
    from paper_2410_13344_b200 import binding as cb
    B, n, H, Dh = 16, 128, 32, 128
    nb = cb.C.c_size_t(0)
    assert cb.lib().cerb_attn_scratch_bytes(B, n, H, Dh, cb.C.byref(nb)) == cb.OK
    assert nb.value > cb.STATIC_ATTN_SCRATCH_BYTES
    q = torch.zeros(B, n, H, Dh, dtype=torch.bfloat16, device="cuda")
    pool = torch.zeros(B * 10, H, 16, Dh, dtype=torch.bfloat16, device="cuda")
    pt = torch.arange(B * 10, dtype=torch.int32, device="cuda").reshape(B, 10)
    lens = torch.zeros(B, dtype=torch.int32, device="cuda")
    anc = torch.from_numpy(cb.tree_ancestors(synth.chain_tree(n).parent).view(np.int64)).cuda()
    rc = cb.tree_attention_noalloc(q, pool, pool, pt, lens, anc, 1.0, n, torch.empty_like(q))
    assert rc == cb.E_NOMEM
