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


def _slots_by_the_stated_schedule(M, N, K, sms=148):
    """Partial slots per output element of the bf16 GEMM, from its schedule as documented.  Up to 128 rows: units are
    (256-row weight tile, 64-wide k block) pairs, cut into 148 contiguous shares, one per CTA.  More rows: the workers
    are the 74 CTA pairs, a tile has 512 weight rows, and the rows form chunks of 256; with 2..37 chunks the unit list
    of ONE chunk is cut into floor(74 / chunks) shares (one pair per chunk walks each share), otherwise the list over
    all chunks is cut into 74 shares.  A share has at least min(k blocks, 4) units; a tile's slots = shares it touches."""
    pairs = M > 128
    workers = sms // 2 if pairs else sms
    tiles, kb = -(-N // (512 if pairs else 256)), -(-K // 64)
    chunks = -(-M // 256) if pairs else 1
    grouped = 1 < chunks <= workers // 2
    jobs = tiles if grouped else tiles * chunks
    shares = workers // chunks if grouped else workers
    per = max(-(-jobs * kb // shares), min(kb, 4))
    return max((j * kb + kb - 1) // per - (j * kb) // per + 1 for j in range(jobs))


def test_gemm_scratch_size_follows_the_documented_schedule():
    import ctypes as C
    from paper_2410_13344_b200 import binding
    L = binding.lib()
    shapes = [(1, 128, 64), (16, 22016, 4096), (64, 4096, 4096), (64, 22016, 4096), (64, 12288, 4096), (64, 32000, 4096),
              (128, 4096, 11008), (256, 22016, 4096), (300, 384, 320), (512, 4096, 4096), (513, 1536, 384),
              (1024, 12288, 4096), (1281, 300, 1024), (2048, 22016, 4096), (2048, 4096, 11008), (2048, 32000, 4096),
              (19201, 128, 64), (64, 27648, 5120), (256, 5120, 13824)]
    for M, N, K in shapes:
        nb = C.c_size_t(0)
        assert L.cerb_gemm_scratch_bytes(M, N, K, C.byref(nb)) == binding.OK
        assert nb.value == 256 + _slots_by_the_stated_schedule(M, N, K) * M * N * 4, (M, N, K)
    # weights leave HBM once at 2048 rows: 8 row chunks share 9 groups of pairs, a 64-block tile touches at most 2 shares
    assert _slots_by_the_stated_schedule(2048, 22016, 4096) == 2


def _launch_table(variant):
    from paper_2410_13344_b200 import binding
    buf = ctypes.create_string_buffer(1 << 14)
    rc = binding.lib().cerb_launch_order_table(variant, buf, len(buf))
    rows = [line.split("|") for line in buf.value.decode().strip().split("\n")]
    return rc, [(int(r[0]), r[1], int(r[2]), int(r[3])) for r in rows]


def test_no_kernel_reads_before_its_wait_what_the_kernel_in_front_writes():
    """Kernels of the forward start while their predecessor still runs and wait before touching its output.  Ahead of
    the wait they may read only what is at least two launches old.  The library exports its launch sequence with,
    per kernel, the buffers written and the buffers read ahead of the wait; the rule is recomputed here."""
    from paper_2410_13344_b200 import binding
    CONST = 1 << 9
    for variant in (0, 1, 2):
        rc, rows = _launch_table(variant)
        assert rc == binding.OK
        names = [r[1] for r in rows]
        assert sum("gemm" in n for n in names) == 3 * 4 + 1 and sum(n == "tree attention" for n in names) == 3
        assert ("swiglu" in names) == (variant == 0) and ("rope_append" in names) == (variant < 2)
        for i, (_, name, _, reads) in enumerate(rows):
            for bit in range(9):
                if not reads >> bit & 1:
                    continue
                writers = [j for j in range(i) if rows[j][2] >> bit & 1]
                assert not writers or i - writers[-1] >= 2, (variant, name, bit, rows[writers[-1]][1])
        # nothing claims to write the constants, and every GEMM reads only constants (its weights) ahead of its wait
        assert all(not w & CONST for _, _, w, _ in rows)
        assert all(r == CONST for _, n, _, r in rows if n.startswith("gemm"))


def test_every_forward_kernel_releases_its_dependents_after_its_own_wait():
    """The two-launches rule above rests on every kernel calling griddepcontrol.launch_dependents only after its
    own griddepcontrol.wait: checked on the sources, kernel by kernel (first trigger after first wait)."""
    src = os.path.join(ROOT, "paper_2410_13344_b200", "csrc")
    seen = 0
    for fn in sorted(os.listdir(src)):
        if not fn.endswith((".cu", ".cuh")) or fn == "cerb_internal.cuh":
            continue
        text = open(os.path.join(src, fn)).read()
        text = re.sub(r"//[^\n]*", "", text)
        for body in re.split(r"__global__", text)[1:]:
            w, t = body.find("griddep_wait()"), body.find("griddep_launch()")
            if t >= 0:
                seen += 1
                assert 0 <= w < t, (fn, body[:80])
    assert seen >= 8
