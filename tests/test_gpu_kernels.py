"""Parity of the individual CUDA kernels with the CPU oracle, through the C ABI.

Tolerances: bf16 values within 2e-2 max-abs/rel, fp32 within 1e-4; integers exact."""
import math

import numpy as np
import pytest
import torch

from oracle import cerberus_oracle as orc
from paper_2410_13344_b200 import synth
from tests.helpers import close

pytestmark = pytest.mark.gpu

TOL_BF16, TOL_F32 = 2e-2, 1e-4


@pytest.fixture(scope="module")
def cb():
    from paper_2410_13344_b200 import binding
    return binding


@pytest.mark.parametrize("M,N,K", [(64, 256, 512), (1, 128, 64), (16, 688, 256), (64, 256, 688), (100, 1000, 1024),
                                   (300, 384, 320), (64, 4096, 4096), (7, 130, 72),
                                   (2048, 640, 512), (1000, 11008, 256), (129, 256, 11008),
                                   # row chunks of 256 walked side by side: 3 chunks (49 groups), 6 ragged chunks,
                                   # and more chunks than half the SMs (back to the plain unit list)
                                   (513, 1536, 384), (1281, 300, 1024), (19201, 128, 64),
                                   # CTA pairs (more than 128 rows) at their edges: one short k block, a ragged last
                                   # k block, weight rows that end inside the first CTA's / the second CTA's half of a
                                   # 512-row unit, exactly one full unit
                                   (130, 520, 72), (200, 1000, 688), (256, 512, 64), (255, 100, 4096), (257, 900, 136)])
def test_gemm_bf16_matches_definition(cb, M, N, K):
    X = synth.normal(11, 1, (M, K), 1.0, dtype=torch.bfloat16, device="cuda")
    W = synth.normal(11, 2, (N, K), 0.05, dtype=torch.bfloat16, device="cuda")
    out = cb.gemm(X, W)
    torch.cuda.synchronize()
    ref = orc.linear(X.cpu(), W.cpu())
    # exact bf16 products, fp32 accumulation: error ~ K * 2^-24 relative to the row's magnitude
    assert close(out, ref, 0) < 2e-4


@pytest.mark.parametrize("M,N,K", [(16, 688, 256), (70, 100, 50)])
def test_gemm_f32_matches_definition(cb, M, N, K):
    X = synth.normal(11, 3, (M, K), 1.0, dtype=torch.float32, device="cuda")
    W = synth.normal(11, 4, (N, K), 0.05, dtype=torch.float32, device="cuda")
    out = cb.gemm(X, W)
    torch.cuda.synchronize()
    assert close(out, orc.linear(X.cpu(), W.cpu()), 0) < 1e-5


def _attention_case(cb, dtype, B, n, H, Dh, lens, max_depth, seed_id, shuffled=True, n_active=None, k_growth=0.0):
    """Builds a paged cache + tree queries, runs the kernel and the oracle, returns the two results."""
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    max_len = max(lens) + n
    max_pages = (max_len + 15) // 16 + 1
    n_pool = B * max_pages + 3
    tree = synth.random_parent_tree(n, max_depth, tree_id=seed_id) if n > 1 else synth.single_node_tree()
    pt = np.stack([synth.shuffled_page_table(max_pages, max_pages, table_id=seed_id * 16 + b, first=b * max_pages)
                   if shuffled else np.arange(b * max_pages, (b + 1) * max_pages, dtype=np.int32) for b in range(B)])
    q = synth.normal(synth.SEED_ATTN, 10 + seed_id, (B, n, H, Dh), 1.0, dtype=tdt, device="cuda")
    kpool = synth.normal(synth.SEED_ATTN, 20 + seed_id, (n_pool, H, 16, Dh), 1.0, dtype=tdt, device="cuda")
    vpool = synth.normal(synth.SEED_ATTN, 30 + seed_id, (n_pool, H, 16, Dh), 1.0, dtype=tdt, device="cuda")
    if k_growth:
        # keys grow with their position, so that scores keep rising along the cache: the running reference of an
        # online softmax has to move many times, far beyond what N(0,1) keys ever ask for
        for b in range(B):
            slots = torch.arange(lens[b] + n)
            pages = torch.from_numpy(pt[b].astype(np.int64))[slots // 16].cuda()
            f = (1.0 + k_growth * slots.float() / float(lens[b] + n)).to(tdt).cuda()
            kpool[pages, :, (slots % 16).cuda()] = kpool[pages, :, (slots % 16).cuda()] * f[:, None, None]
    # the unused tail of the pool holds non-finite garbage: the kernel must never let it leak
    kpool[n_pool - 3:] = float("nan")
    vpool[n_pool - 3:] = float("inf")
    # so do the slots of mapped pages past the last tree key
    for b in range(B):
        nb = n if n_active is None else n_active[b]
        for slot in range(lens[b] + nb, min(max_pages * 16, lens[b] + nb + 40)):
            kpool[int(pt[b][slot // 16]), :, slot % 16] = float("nan")
            vpool[int(pt[b][slot // 16]), :, slot % 16] = float("inf")
    anc = torch.from_numpy(cb.tree_ancestors(tree.parent).view(np.int64)).cuda()
    lens_t = torch.tensor(lens, dtype=torch.int32, device="cuda")
    na_t = None if n_active is None else torch.tensor(n_active, dtype=torch.int32, device="cuda")
    pt_t = torch.from_numpy(pt).cuda()
    scale = 1.0 / math.sqrt(Dh)
    out, lse, _ = cb.tree_attention(q, kpool, vpool, pt_t, lens_t, anc, scale, max_len, n_active=na_t)
    torch.cuda.synchronize()
    results = []
    for b in range(B):
        nb = n if n_active is None else n_active[b]
        if nb == 0:
            continue
        L = lens[b]
        pages = torch.from_numpy(pt[b].astype(np.int64))
        kc = kpool.cpu()[pages].permute(0, 2, 1, 3).reshape(-1, H, Dh).double()
        vc = vpool.cpu()[pages].permute(0, 2, 1, 3).reshape(-1, H, Dh).double()
        O, l = orc.tree_attention(q[b, :nb].cpu().double(), kc[:L], vc[:L], kc[L:L + nb], vc[L:L + nb],
                                  tree.parent[:nb], scale)
        results.append((out[b, :nb], lse[b, :, :nb], O, l))
    return results


ATTN_CASES = [
    # B, n, H, Dh, lens, max_depth
    (1, 64, 32, 128, [1024], 5),        # Llama-7B layer shape, 1024-token prefix, 64-node tree
    (1, 16, 4, 128, [100], 4),
    (2, 33, 3, 128, [257, 63], 6),      # ragged lengths, node count between warp layouts
    (1, 128, 2, 128, [700], 6),         # two ancestor words
    (1, 1, 4, 128, [333], 1),           # auto-regressive step: one node
    (1, 20, 2, 128, [0], 4),            # empty prefix: the tree alone
    (3, 64, 4, 64, [15, 16, 17], 5),    # head_dim 64, lengths around a page boundary
    (1, 64, 2, 128, [5000], 5),         # long context: many tiles per split
    (16, 16, 32, 128, [40] * 16, 3),    # more (sequence, head) pairs than CTAs wanted: no split
    (16, 128, 2, 128, [8192 - 17 * i for i in range(16)], 6),   # sweep corner: batch 16, 128 nodes, 8K keys
    (5, 32, 3, 128, [511, 512, 513, 2047, 1], 6),
    (2, 64, 3, 128, [4100, 3991], 5),   # 64-node trees over long caches: tcgen05 kernel, eight splits in one cluster
    (3, 40, 2, 128, [3000, 2999, 1], 5),
    (1, 121, 4, 128, [1500], 4),        # 120 candidate paths + root (the paper's middle tree setting, Sec. 5.1)
    (1, 64, 32, 128, [8200], 5),
    (1, 64, 8, 128, [2500], 5),         # tcgen05 kernel, five key splits merged inside a thread-block cluster
    (4, 64, 2, 128, [2100, 2000, 1900, 2047], 5),   # ... batch of four, ragged
    (1, 128, 8, 128, [3000], 6),        # ... three splits
    (2, 100, 16, 128, [2500, 77], 5),   # ... ragged: the short sequence leaves most splits without keys
    (1, 151, 4, 128, [1500], 4),        # 150 candidate paths + root (the paper's widest tree, Sec. 5.1): three ancestor
                                        # words, two launches of query rows (128 + 23), both on the tcgen05 kernel
    (2, 192, 2, 128, [300, 77], 6),     # the largest tree the library takes; short caches: second window on the warp-MMA kernel
    (2, 151, 2, 64, [500, 100], 5),     # head_dim 64: warp-MMA kernel for both windows
    (3, 140, 3, 128, [2000, 1, 640], 6),
]


@pytest.mark.parametrize("case", ATTN_CASES, ids=[str(i) for i in range(len(ATTN_CASES))])
def test_tree_attention_bf16(cb, case):
    B, n, H, Dh, lens, md = case
    for got_o, got_l, O, l in _attention_case(cb, "bf16", B, n, H, Dh, lens, md, seed_id=ATTN_CASES.index(case)):
        assert torch.isfinite(got_o.float()).all()
        assert close(got_o, O, 0) < TOL_BF16
        assert close(got_l, l, 0) < 2e-3


@pytest.mark.parametrize("case", [(2, 64, 4, 128, [1500, 700], 5), (1, 128, 2, 128, [900], 6), (1, 16, 4, 128, [3000], 4),
                                  (1, 64, 2, 64, [600], 5)])
def test_tree_attention_bf16_rising_scores(cb, case):
    """Scores that grow by tens of bits along the cache: every kernel's running softmax reference must follow
    (rescaling what it has accumulated) without losing the early keys' share or overflowing."""
    B, n, H, Dh, lens, md = case
    for got_o, got_l, O, l in _attention_case(cb, "bf16", B, n, H, Dh, lens, md, seed_id=70 + n, k_growth=40.0):
        assert torch.isfinite(got_o.float()).all()
        assert close(got_o, O, 0) < TOL_BF16
        assert close(got_l, l, 0) < 2e-3


@pytest.mark.parametrize("switch", ["CERB_ATTN_CLUSTER=0", "CERB_ATTN_KT=1", "CERB_ATTN_KT=0"])
def test_other_attention_routes_in_a_child_process(switch):
    """Environment switches that are read once per process select other routes through the attention kernels: the
    key splits merged through partials in the scratch buffer instead of inside a thread-block cluster; the
    keys-on-M tensor-core kernel for every launch of up to 64 query rows (by default it takes 17..64); that kernel
    off.  Each route runs the bf16 attention cases again in a child process."""
    import os
    import subprocess
    import sys
    name, value = switch.split("=")
    env = dict(os.environ, **{name: value})
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_kernels.py", "-q", "-x", "-m", "gpu", "-k",
                        "test_tree_attention_bf16"], cwd=root, env=env, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def test_tree_attention_bf16_partial_activity(cb):
    res = _attention_case(cb, "bf16", 3, 32, 4, 128, [90, 10, 200], 4, seed_id=40, n_active=[32, 0, 5])
    assert len(res) == 2
    for got_o, got_l, O, l in res:
        assert close(got_o, O, 0) < TOL_BF16 and close(got_l, l, 0) < 2e-3


def test_tree_attention_bf16_partial_activity_on_the_tensor_core_path(cb):
    """Long caches take the tcgen05 kernel, whose key splits form clusters: a sequence without live nodes makes
    whole clusters leave at once, one with five live nodes leaves most query rows empty."""
    res = _attention_case(cb, "bf16", 3, 64, 8, 128, [1500, 1200, 2100], 5, seed_id=42, n_active=[64, 0, 5])
    assert len(res) == 2
    for got_o, got_l, O, l in res:
        assert close(got_o, O, 0) < TOL_BF16 and close(got_l, l, 0) < 2e-3


def test_tree_attention_bf16_partial_activity_beyond_128_nodes(cb):
    """151-node tree, live node counts on either side of the 128-row boundary between the two launches:
    the second launch has 23, 2 and no live rows."""
    res = _attention_case(cb, "bf16", 3, 151, 4, 128, [1400, 90, 1100], 5, seed_id=43, n_active=[151, 130, 5])
    assert len(res) == 3
    for got_o, got_l, O, l in res:
        assert close(got_o, O, 0) < TOL_BF16 and close(got_l, l, 0) < 2e-3


def test_tree_attention_bf16_is_deterministic(cb):
    a = _attention_case(cb, "bf16", 1, 64, 8, 128, [3000], 5, seed_id=41)[0]
    b = _attention_case(cb, "bf16", 1, 64, 8, 128, [3000], 5, seed_id=41)[0]
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


@pytest.mark.parametrize("case", [(1, 16, 4, 64, [64], 4), (2, 40, 2, 128, [33, 5], 5), (1, 128, 2, 64, [10], 6),
                                  (2, 151, 2, 64, [40, 3], 6)])
def test_tree_attention_f32(cb, case):
    B, n, H, Dh, lens, md = case
    for got_o, got_l, O, l in _attention_case(cb, "fp32", B, n, H, Dh, lens, md, seed_id=50 + n):
        assert close(got_o, O, 0) < TOL_F32 and close(got_l, l, 0) < TOL_F32


def test_bounded_wait_runs_out_cleanly_and_the_next_call_is_correct(cb):
    """Every device-side wait has a cycle budget.  With the budget set to a thousand cycles, the epilogue warps of
    a long GEMM (2048 rows x 256 x 262144: each CTA accumulates ~230 k blocks, about half a millisecond, before its
    epilogue may read) run out of it by the limit alone -- nothing is skipped or broken.  The launch must report CERB_E_TIMEOUT in its status word, come
    back (its CTAs stop issuing, see their copies and MMAs in flight retire, free their tensor memory), and the
    same call with the default budget must then give the right result."""
    L = cb.lib()
    M, N, K = 2048, 256, 262144
    X = synth.normal(13, 1, (M, K), 1.0, dtype=torch.bfloat16, device="cuda")
    W = synth.normal(13, 2, (N, K), 0.05, dtype=torch.bfloat16, device="cuda")
    nb = cb.C.c_size_t(0)
    assert L.cerb_gemm_scratch_bytes(M, N, K, cb.C.byref(nb)) == cb.OK
    scratch = torch.zeros(nb.value + 512, dtype=torch.uint8, device="cuda")
    off = (-scratch.data_ptr()) % 256                      # where the binding places the status word
    assert L.cerb_set_wait_cycles(100) == cb.E_ARG
    assert L.cerb_set_wait_cycles(1000) == cb.OK
    try:
        cb.gemm(X, W, scratch=scratch)
        torch.cuda.synchronize()
        status = int(scratch[off:off + 4].view(torch.int32).item())
    finally:
        assert L.cerb_set_wait_cycles(4_000_000_000) == cb.OK
    assert status == cb.E_TIMEOUT
    out = cb.gemm(X, W, scratch=scratch)
    torch.cuda.synchronize()
    assert int(scratch[off:off + 4].view(torch.int32).item()) == 0
    ri, ci = torch.arange(0, M, 197), torch.arange(0, N, 37)
    ref = orc.linear(X[ri].cpu(), W[ci].cpu())
    assert close(out[ri][:, ci].cpu(), ref, 0) < 2e-3          # 262144 products per element


@pytest.mark.parametrize("B,n,H,L", [(1, 64, 32, 6000), (1, 8, 32, 6000), (1, 128, 32, 6000), (4, 64, 32, 3000)])
def test_attention_after_a_timeout_comes_back_and_the_next_call_is_correct(cb, B, n, H, L):
    """A wait that runs out leaves CERB_E_TIMEOUT in the status word, and every kernel that finds the word set when
    it starts (the rest of a decoding step after a time-out) shortens its waits to microseconds, issues no copies
    and no MMAs, lets those waits run out -- nothing fills its barriers -- and leaves, tensor memory freed and its
    cluster partners met.  Here the caller sets the word before the launch, for the three bf16 kernels (keys-on-M
    with a cluster of splits and with one split, warp-MMA, query-rows-on-M): the launch must come back with the word
    still set, and the same call after the word has been cleared must match the oracle."""
    Dh = 128
    max_len = L + n
    mp = (max_len + 15) // 16 + 1
    tree = synth.random_parent_tree(n, 5, tree_id=77)
    q = synth.normal(synth.SEED_ATTN, 801, (B, n, H, Dh), 1.0, dtype=torch.bfloat16, device="cuda")
    kp = synth.normal(synth.SEED_ATTN, 802, (B * mp, H, 16, Dh), 1.0, dtype=torch.bfloat16, device="cuda")
    vp = synth.normal(synth.SEED_ATTN, 803, (B * mp, H, 16, Dh), 1.0, dtype=torch.bfloat16, device="cuda")
    pt = torch.from_numpy(np.stack([synth.shuffled_page_table(mp, mp, table_id=880 + b, first=b * mp) for b in range(B)])).cuda()
    anc = torch.from_numpy(cb.tree_ancestors(tree.parent).view(np.int64)).cuda()
    lens = torch.full((B,), L, dtype=torch.int32, device="cuda")
    scale = 1.0 / math.sqrt(Dh)
    nb = cb.C.c_size_t(0)
    assert cb.lib().cerb_attn_scratch_bytes(B, n, H, Dh, cb.C.byref(nb)) == cb.OK
    scratch = torch.zeros(nb.value, dtype=torch.uint8, device="cuda")
    status = scratch[4096 - 16:4096].view(torch.int32)            # the status words of this entry point
    status[0] = cb.E_TIMEOUT
    cb.tree_attention(q, kp, vp, pt, lens, anc, scale, max_len, scratch=scratch)
    torch.cuda.synchronize()
    assert int(status[0].item()) == cb.E_TIMEOUT
    scratch[:4096] = 0                                            # status and ticket counters, as before a first use
    out, lse, _ = cb.tree_attention(q, kp, vp, pt, lens, anc, scale, max_len, scratch=scratch)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0
    b = B - 1
    pages = pt[b].cpu().long()
    kc = kp.cpu()[pages].permute(0, 2, 1, 3).reshape(-1, H, Dh).double()
    vc = vp.cpu()[pages].permute(0, 2, 1, 3).reshape(-1, H, Dh).double()
    O, l = orc.tree_attention(q[b].cpu().double(), kc[:L], vc[:L], kc[L:L + n], vc[L:L + n], tree.parent, scale)
    assert close(out[b], O, 0) < TOL_BF16 and close(lse[b], l, 0) < 2e-3


def test_abi_rejects_bad_arguments(cb):
    L = cb.lib()
    assert L.cerb_tree_attention(None, None) == cb.E_ARG
    out = np.zeros((4, cb.ANC_WORDS), np.uint64)
    bad = np.array([-1, 0, 3, 1], np.int32)       # parent after child
    assert L.cerb_tree_ancestors(bad.ctypes.data, 4, out.ctypes.data) == cb.E_ARG
    good = np.array([-1, 0, 0, 1], np.int32)
    assert L.cerb_tree_ancestors(good.ctypes.data, 4, out.ctypes.data) == cb.OK
    assert [int(x) for x in out[:, 0]] == [1, 3, 5, 11]
