"""The seeded input generators: determinism, chunk invariance, distributions, tree recipes."""
import numpy as np
import torch

from paper_2410_13344_b200 import synth


def test_normal_is_deterministic_and_chunk_invariant():
    a = synth.normal(3, 9, (1000,), 1.0, dtype=torch.float64)
    b = synth.normal(3, 9, (1000,), 1.0, dtype=torch.float64, chunk=64)
    assert torch.equal(a, b)
    c = synth.normal(3, 10, (1000,), 1.0, dtype=torch.float64)
    assert not torch.equal(a, c)
    big = synth.normal(1, 1, (200000,), 0.02, dtype=torch.float64)
    assert abs(float(big.mean())) < 3e-4 and abs(float(big.std()) - 0.02) < 3e-4


def test_scalar_and_tensor_splitmix_agree():
    bits = synth.uniform_bits(5, 7, 0, 4)
    for i in range(4):
        want = synth.splitmix64((synth._base_key(5, 7) ^ i) & ((1 << 64) - 1))
        assert (int(bits[i]) & ((1 << 64) - 1)) == want


def test_best_first_tree_counts():
    t = synth.best_first_tree(16, [4, 2, 1, 1])
    assert t.n == 16 and t.parent[0] == -1
    depth = [0] * t.n
    sums = [0] * t.n
    for v in range(1, t.n):
        assert 0 <= t.parent[v] < v
        depth[v] = depth[t.parent[v]] + 1
        sums[v] = sums[t.parent[v]] + t.rank[v]
        assert t.head[v] == depth[v] - 1
    assert [sums[1:].count(s) for s in (0, 1, 2)] == [4, 7, 4]
    t = synth.best_first_tree(64, [10, 10, 10, 10])
    sums = [0] * t.n
    for v in range(1, t.n):
        sums[v] = sums[t.parent[v]] + t.rank[v]
    assert [sums[1:].count(s) for s in (0, 1, 2, 3)] == [4, 10, 20, 29]


def test_random_parent_tree_respects_depth_cap():
    t = synth.random_parent_tree(64, 5, tree_id=3)
    depth = [0] * 64
    for v in range(1, 64):
        assert 0 <= t.parent[v] < v
        depth[v] = depth[t.parent[v]] + 1
    assert max(depth) <= 5 and max(depth) >= 3


def test_page_table_is_a_shuffled_injection():
    pt = synth.shuffled_page_table(68, 80)
    assert len(set(pt.tolist())) == 68 and pt.max() < 80 and list(pt) != sorted(pt)


def test_layout_widths():
    lay = synth.cerberus_layout(4, 4)
    w = lay.widths(4096)
    assert w[0] == [4096] * 5
    assert w[1] == [4096] * 4 + [8192]
    lay = synth.cerberus_layout(3, 4, concat_level=1)
    w = lay.widths(8)
    assert w[1] == [8, 8, 16, 16, 16] and w[2] == [8, 8, 16, 16, 16]
