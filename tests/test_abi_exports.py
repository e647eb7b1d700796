"""The shared library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "cerb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cerb_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2410_13344_b200 import binding
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_host_only_calls_work_without_a_gpu():
    from paper_2410_13344_b200 import binding, synth
    import numpy as np
    assert binding.strerror(binding.E_TIMEOUT) == "a bounded device-side wait ran out"
    anc = binding.tree_ancestors(synth.chain_tree(70).parent)
    assert anc.shape == (70, binding.ANC_WORDS)
    assert int(anc[69, 0]) == (1 << 64) - 1 and int(anc[69, 1]) == (1 << 6) - 1 and int(anc[69, 2]) == 0
    wide = binding.tree_ancestors(synth.chain_tree(151).parent)       # 150 candidates + root (Sec. 5.1)
    assert [int(x) for x in wide[150]] == [(1 << 64) - 1, (1 << 64) - 1, (1 << 23) - 1]
    star = np.array([-1] + [0] * 191, np.int32)                       # the largest tree: every node a child of the root
    s = binding.tree_ancestors(star)
    assert [int(x) for x in s[191]] == [1, 0, 1 << 63] and [int(x) for x in s[64]] == [1, 1, 0]
    cfg = binding.make_config(synth.shape_7b(), synth.cerberus_layout(4), [10] * 4, 200, 200, 1, 64)
    nbytes = binding.workspace_bytes(cfg)
    assert 10 << 20 < nbytes < 2 << 30
    cfg.head_dim = 96
    try:
        binding.workspace_bytes(cfg)
        assert False
    except binding.CerbError as e:
        assert e.code == binding.E_SHAPE


def test_threshold_from_samples_splits_the_requested_fraction():
    from paper_2410_13344_b200 import binding
    S = [0.3, 7.9, 7.1, 6.5, 7.7, 2.0, 7.3, 6.9, 7.5, 5.0]
    for frac, below in ((0.5, 5), (0.7, 7), (0.1, 1), (0.0, 1), (1.0, 9)):
        T = binding.threshold_from_samples(S, frac)
        assert sum(1 for v in S if v <= T) == below and T not in S
