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


def test_noalloc_entry_matches_the_ordinary_one_twice_in_a_row():
    from paper_2410_13344_b200 import binding as cb
    # two different problems, back to back, both long enough to be split along the keys
    cases = [(1, 64, 8, 128, 3000, 1), (2, 33, 4, 128, 1500, 2)]
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
