"""Thin ctypes binding of libcerb.so (include/cerb.h): argument marshalling only.

Every step of the decoding path runs in the library's CUDA kernels; torch is used
here for device memory and streams.  Importing this module fails loudly if the
shared library has not been built -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import synth

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcerb.so")

OK = 0
E_ARG, E_SHAPE, E_NOMEM, E_STATE, E_NONFINITE, E_TIMEOUT, E_CUDA = -1, -2, -3, -4, -5, -6, -7
F32, BF16 = 0, 1
MODE_PAR, MODE_AR = 0, 1
PAGE, MAX_NODES, MAX_DEPTH, MAX_HEADS, MAX_LEVELS, MAX_TOPK, MAX_BATCH, MAX_TREES = 16, 192, 8, 8, 8, 16, 16, 8
ANC_WORDS = 3
PATH_MAX = MAX_DEPTH + 1

EXPORTS = [
    "cerb_workspace_bytes", "cerb_load", "cerb_free", "cerb_tree_create", "cerb_tree_free", "cerb_reset",
    "cerb_prefill", "cerb_gate", "cerb_draft", "cerb_verify", "cerb_accept", "cerb_step",
    "cerb_attn_scratch_bytes", "cerb_tree_attention", "cerb_tree_ancestors", "cerb_gemm_scratch_bytes", "cerb_gemm",
    "cerb_read_state", "cerb_device_status", "cerb_launch_count", "cerb_strerror", "cerb_profile_enable",
    "cerb_profile_read", "cerb_tree_attention_noalloc", "cerb_set_wait_cycles", "cerb_wait_diagnosis", "cerb_tree_attention_noalloc_status", "cerb_launch_order_table", "cerb_last_forward_rows",
]


class CerbError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {code} ({strerror(code)})")
        self.code = code


class Config(C.Structure):
    _fields_ = [
        ("dtype", C.c_int32), ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
        ("head_dim", C.c_int32), ("mlp_dim", C.c_int32), ("vocab", C.c_int32),
        ("rope_base", C.c_float), ("rms_eps", C.c_float),
        ("max_pages", C.c_int32), ("n_pool_pages", C.c_int32), ("max_batch", C.c_int32), ("max_nodes", C.c_int32),
        ("n_cheads", C.c_int32), ("n_levels", C.c_int32),
        ("concat_src", (C.c_int32 * MAX_LEVELS) * MAX_HEADS),
        ("topk", C.c_int32 * MAX_HEADS),
    ]


class Weights(C.Structure):
    _fields_ = [
        ("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
        ("attn_norm", C.POINTER(C.c_void_p)), ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
        ("mlp_norm", C.POINTER(C.c_void_p)), ("wgu", C.POINTER(C.c_void_p)), ("wd", C.POINTER(C.c_void_p)),
        ("head_W", C.POINTER(C.c_void_p)), ("head_b", C.POINTER(C.c_void_p)), ("head_fc", C.POINTER(C.c_void_p)),
        ("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("page_table", C.c_void_p),
    ]


class StepOut(C.Structure):
    _fields_ = [
        ("S_dev", C.c_void_p), ("mode_dev", C.c_void_p), ("n_accept_dev", C.c_void_p), ("tokens_dev", C.c_void_p),
        ("S_host", C.c_void_p), ("mode_host", C.c_void_p), ("n_accept_host", C.c_void_p), ("tokens_host", C.c_void_p),
    ]


class AttnArgs(C.Structure):
    _fields_ = [
        ("dtype", C.c_int32), ("B", C.c_int32), ("n", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("max_pages", C.c_int32),
        ("q", C.c_void_p), ("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("page_table", C.c_void_p),
        ("len", C.c_void_p), ("n_active", C.c_void_p), ("anc", C.c_void_p), ("out", C.c_void_p), ("lse", C.c_void_p),
        ("scale", C.c_float), ("max_len", C.c_int32), ("n_pool_pages", C.c_int32),
        ("scratch", C.c_void_p), ("scratch_bytes", C.c_size_t),
    ]


_lib = None


def lib():
    """The loaded shared library; raises if it is missing (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2410_13344_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.cerb_strerror.restype = C.c_char_p
        L.cerb_strerror.argtypes = [C.c_int]
        L.cerb_launch_count.restype = C.c_int64
        L.cerb_launch_count.argtypes = [C.c_void_p]
        L.cerb_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t)]
        L.cerb_load.argtypes = [C.POINTER(Config), C.POINTER(Weights), C.c_void_p, C.c_size_t, C.POINTER(C.c_void_p)]
        L.cerb_free.argtypes = [C.c_void_p]
        L.cerb_tree_create.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_void_p)]
        L.cerb_tree_free.argtypes = [C.c_void_p, C.c_void_p]
        L.cerb_reset.argtypes = [C.c_void_p, C.c_void_p]
        L.cerb_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
        L.cerb_gate.argtypes = [C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
        L.cerb_draft.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.cerb_verify.argtypes = [C.c_void_p] * 8
        L.cerb_accept.argtypes = [C.c_void_p] * 9
        L.cerb_step.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.POINTER(StepOut), C.c_void_p]
        L.cerb_attn_scratch_bytes.argtypes = [C.c_int32] * 4 + [C.POINTER(C.c_size_t)]
        L.cerb_tree_attention.argtypes = [C.POINTER(AttnArgs), C.c_void_p]
        L.cerb_tree_ancestors.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.cerb_tree_attention_noalloc.argtypes = [C.POINTER(AttnArgs), C.c_void_p]
        L.cerb_tree_attention_noalloc_status.argtypes = [C.c_void_p]
        L.cerb_gemm_scratch_bytes.argtypes = [C.c_int32] * 3 + [C.POINTER(C.c_size_t)]
        L.cerb_gemm.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                C.c_void_p, C.c_size_t, C.c_void_p]
        L.cerb_read_state.argtypes = [C.c_void_p] * 5
        L.cerb_device_status.argtypes = [C.c_void_p, C.c_void_p]
        L.cerb_profile_enable.argtypes = [C.c_void_p, C.c_int32]
        L.cerb_set_wait_cycles.argtypes = [C.c_int64]
        L.cerb_last_forward_rows.argtypes = [C.c_void_p]
        L.cerb_launch_order_table.argtypes = [C.c_int32, C.c_char_p, C.c_size_t]
        L.cerb_wait_diagnosis.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.cerb_profile_read.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().cerb_strerror(code).decode()


def _check(rc: int, what: str):
    if rc != OK:
        raise CerbError(rc, what)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_config(shape: synth.ModelShape, layout: Optional[synth.HeadLayout], topk: Sequence[int], max_pages: int,
                n_pool_pages: int, max_batch: int = 1, max_nodes: int = 64) -> Config:
    cfg = Config()
    cfg.dtype = BF16 if shape.dtype == "bf16" else F32
    cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.head_dim = shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim
    cfg.mlp_dim, cfg.vocab, cfg.rope_base, cfg.rms_eps = shape.mlp_dim, shape.vocab, shape.rope_base, shape.rms_eps
    cfg.max_pages, cfg.n_pool_pages, cfg.max_batch, cfg.max_nodes = max_pages, n_pool_pages, max_batch, max_nodes
    for h in range(MAX_HEADS):
        for j in range(MAX_LEVELS):
            cfg.concat_src[h][j] = -1
    if layout is not None:
        cfg.n_cheads, cfg.n_levels = layout.n_heads, layout.n_levels
        for h, row in enumerate(layout.blocks):
            for j, blk in enumerate(row):
                cfg.concat_src[h][j] = blk.concat_src_head
            cfg.topk[h] = topk[h]
    return cfg


def workspace_bytes(cfg: Config) -> int:
    out = C.c_size_t(0)
    _check(lib().cerb_workspace_bytes(C.byref(cfg), C.byref(out)), "cerb_workspace_bytes")
    return out.value


def threshold_from_samples(S: Sequence[float], parallel_fraction: float) -> float:
    """Midpoint of the two order statistics that leave `parallel_fraction` of the gate values at or below it."""
    s = sorted(S)
    k = min(max(int(round(parallel_fraction * len(s))), 1), len(s) - 1)
    return 0.5 * (s[k - 1] + s[k])


def tree_ancestors(parent: np.ndarray) -> np.ndarray:
    parent = np.ascontiguousarray(parent, np.int32)
    out = np.zeros((parent.shape[0], ANC_WORDS), np.uint64)
    _check(lib().cerb_tree_ancestors(parent.ctypes.data, parent.shape[0], out.ctypes.data), "cerb_tree_ancestors")
    return out


class TreeHandle:
    def __init__(self, owner: "Cerberus", handle: int, tree: synth.Tree):
        self.owner, self.handle, self.tree = owner, handle, tree

    @property
    def n(self) -> int:
        return self.tree.n


class Cerberus:
    """A loaded model + decoding heads + paged KV cache on the current CUDA device."""

    def __init__(self, shape: synth.ModelShape, model: Dict[str, torch.Tensor], layout: Optional[synth.HeadLayout] = None,
                 heads: Optional[Dict[str, torch.Tensor]] = None, topk: Sequence[int] = (), max_tokens: int = 4096,
                 max_batch: int = 1, max_nodes: int = 64, page_table: Optional[np.ndarray] = None,
                 n_pool_pages: Optional[int] = None):
        self.shape, self.model, self.layout, self.heads = shape, model, layout, heads
        dev = model["embed"].device
        assert dev.type == "cuda", "weights must live on the GPU"
        self.device = dev
        dt = shape.torch_dtype
        max_pages = (max_tokens + max_nodes + PAGE - 1) // PAGE
        if n_pool_pages is None:
            n_pool_pages = max_pages * max_batch
        if page_table is None:
            page_table = np.arange(max_batch * max_pages, dtype=np.int32).reshape(max_batch, max_pages)
        assert page_table.shape == (max_batch, max_pages)
        self.max_pages, self.n_pool_pages, self.max_batch, self.max_nodes = max_pages, n_pool_pages, max_batch, max_nodes
        self.page_table_host = np.ascontiguousarray(page_table, np.int32)
        self.page_table = torch.from_numpy(self.page_table_host).to(dev)
        pool_shape = (shape.n_layers, n_pool_pages, shape.n_heads, PAGE, shape.head_dim)
        self.k_pool = torch.zeros(pool_shape, dtype=dt, device=dev)
        self.v_pool = torch.zeros(pool_shape, dtype=dt, device=dev)
        self.cfg = make_config(shape, layout, topk, max_pages, n_pool_pages, max_batch, max_nodes)
        self.ws = torch.empty(workspace_bytes(self.cfg) + 256, dtype=torch.uint8, device=dev)
        ws_ptr = (self.ws.data_ptr() + 255) // 256 * 256
        L = shape.n_layers

        def arr(names):
            a = (C.c_void_p * len(names))()
            for i, nm in enumerate(names):
                t = (model if nm in model else heads)[nm]
                assert t.is_contiguous() and t.dtype == dt and t.device == dev, nm
                a[i] = t.data_ptr()
            return a

        self._arrays = {k: arr([f"{k}.{l}" for l in range(L)]) for k in ("attn_norm", "wqkv", "wo", "mlp_norm", "wgu", "wd")}
        w = Weights()
        w.embed, w.final_norm, w.lm_head = model["embed"].data_ptr(), model["final_norm"].data_ptr(), model["lm_head"].data_ptr()
        for k, a in self._arrays.items():
            setattr(w, k, C.cast(a, C.POINTER(C.c_void_p)))
        if layout is not None:
            Hc, Lv = layout.n_heads, layout.n_levels
            self._hW = arr([f"W.{h}.{j}" for h in range(Hc) for j in range(Lv)])
            self._hb = arr([f"b.{h}.{j}" for h in range(Hc) for j in range(Lv)])
            self._hfc = arr([f"fc.{h}" for h in range(Hc)])
            w.head_W = C.cast(self._hW, C.POINTER(C.c_void_p))
            w.head_b = C.cast(self._hb, C.POINTER(C.c_void_p))
            w.head_fc = C.cast(self._hfc, C.POINTER(C.c_void_p))
        w.k_pool, w.v_pool, w.page_table = self.k_pool.data_ptr(), self.v_pool.data_ptr(), self.page_table.data_ptr()
        self._weights = w
        handle = C.c_void_p()
        _check(lib().cerb_load(C.byref(self.cfg), C.byref(w), ws_ptr, self.ws.numel() - 256, C.byref(handle)), "cerb_load")
        self.ctx = handle
        self.B = 0
        i32 = dict(dtype=torch.int32, device=dev)
        self.S = torch.zeros(max_batch, dtype=torch.float32, device=dev)
        self.mode = torch.zeros(max_batch, **i32)
        self.n_accept = torch.zeros(max_batch, **i32)
        self.tokens = torch.zeros(max_batch, PATH_MAX, **i32)
        self.path = torch.zeros(max_batch, PATH_MAX, **i32)
        self.h_S = torch.zeros(max_batch, dtype=torch.float32).pin_memory()
        self.h_mode = torch.zeros(max_batch, dtype=torch.int32).pin_memory()
        self.h_n_accept = torch.zeros(max_batch, dtype=torch.int32).pin_memory()
        self.h_tokens = torch.zeros(max_batch, PATH_MAX, dtype=torch.int32).pin_memory()
        self._step_out = StepOut(self.S.data_ptr(), self.mode.data_ptr(), self.n_accept.data_ptr(), self.tokens.data_ptr(),
                                 self.h_S.data_ptr(), self.h_mode.data_ptr(), self.h_n_accept.data_ptr(),
                                 self.h_tokens.data_ptr())

    def close(self):
        if self.ctx:
            lib().cerb_free(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- trees
    def tree(self, t: synth.Tree) -> TreeHandle:
        h = C.c_void_p()
        p, hd, rk = (np.ascontiguousarray(a, np.int32) for a in (t.parent, t.head, t.rank))
        _check(lib().cerb_tree_create(self.ctx, p.ctypes.data, hd.ctypes.data, rk.ctypes.data, t.n, C.byref(h)), "cerb_tree_create")
        return TreeHandle(self, h, t)

    def free_tree(self, th: TreeHandle):
        _check(lib().cerb_tree_free(self.ctx, th.handle), "cerb_tree_free")

    # ---- calls
    def prefill(self, tokens: torch.Tensor, lens: Sequence[int]):
        """tokens: device int32 [B][max_len]."""
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.is_contiguous() and tokens.dim() == 2
        B, max_len = tokens.shape
        lens_a = np.ascontiguousarray(lens, np.int32)
        _check(lib().cerb_prefill(self.ctx, tokens.data_ptr(), lens_a.ctypes.data, B, max_len, _stream()), "cerb_prefill")
        self.B = B

    def gate(self, T: float):
        _check(lib().cerb_gate(self.ctx, T, self.S.data_ptr(), self.mode.data_ptr(), _stream()), "cerb_gate")
        return self.S[:self.B], self.mode[:self.B]

    def draft(self, th: TreeHandle, want_logits: bool = False):
        i32 = dict(dtype=torch.int32, device=self.device)
        tree_tok = torch.empty(self.B, th.n, **i32)
        topk = torch.empty(self.B, self.cfg.n_cheads, MAX_TOPK, **i32)
        logits = torch.empty(self.B, self.cfg.n_cheads, self.shape.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        _check(lib().cerb_draft(self.ctx, th.handle, tree_tok.data_ptr(), topk.data_ptr(), _ptr(logits), _stream()), "cerb_draft")
        return tree_tok, topk, logits

    def verify(self, th: TreeHandle, tree_tok: torch.Tensor, n_active: Optional[torch.Tensor] = None,
               want_logits: bool = False, want_hidden: bool = False):
        assert tree_tok.dtype == torch.int32 and tree_tok.is_contiguous() and tuple(tree_tok.shape) == (self.B, th.n)
        dev = self.device
        node_argmax = torch.empty(self.B, th.n, dtype=torch.int32, device=dev)
        logits = torch.empty(self.B, th.n, self.shape.vocab, dtype=torch.float32, device=dev) if want_logits else None
        hidden = torch.empty(self.B, th.n, self.shape.d_model, dtype=self.shape.torch_dtype, device=dev) if want_hidden else None
        _check(lib().cerb_verify(self.ctx, th.handle, tree_tok.data_ptr(), _ptr(n_active), node_argmax.data_ptr(),
                                 _ptr(logits), _ptr(hidden), _stream()), "cerb_verify")
        return node_argmax, logits, hidden

    def accept(self, th: TreeHandle, tree_tok: torch.Tensor, node_argmax: torch.Tensor, n_active: Optional[torch.Tensor] = None):
        _check(lib().cerb_accept(self.ctx, th.handle, tree_tok.data_ptr(), _ptr(n_active), node_argmax.data_ptr(),
                                 self.n_accept.data_ptr(), self.path.data_ptr(), self.tokens.data_ptr(), _stream()), "cerb_accept")
        return self.n_accept[:self.B], self.path[:self.B], self.tokens[:self.B]

    def step(self, th: TreeHandle, T: float, plant: Optional[torch.Tensor] = None):
        """One decoding step; results land in the pinned mirrors (h_S, h_mode, h_n_accept, h_tokens)
        once the stream is synchronised."""
        rc = lib().cerb_step(self.ctx, th.handle, T, _ptr(plant), C.byref(self._step_out), _stream())
        if rc != OK:
            raise CerbError(rc, "cerb_step (device status words %s)" % self.wait_diagnosis())

    def read_state(self):
        lens = np.zeros(self.B, np.int32)
        roots = np.zeros(self.B, np.int32)
        h = torch.empty(self.B, self.shape.d_model, dtype=self.shape.torch_dtype)
        _check(lib().cerb_read_state(self.ctx, lens.ctypes.data, roots.ctypes.data, h.data_ptr(), _stream()), "cerb_read_state")
        return lens, roots, h

    def calibrate_threshold(self, th: "TreeHandle", n_steps: int, parallel_fraction: float) -> float:
        """Host-side helper for the gate's threshold T (Sec. 4.2; the paper lists finding T by hand as a
        limitation): decodes `n_steps` auto-regressive steps from the current state, which changes that
        state like any decoding does, and returns the value that would have sent `parallel_fraction`
        of those steps down the parallel path (entropy at or below T).  Batch 1."""
        assert self.B == 1 and n_steps >= 2
        S = []
        for _ in range(n_steps):
            self.step(th, -1.0)
            torch.cuda.current_stream().synchronize()
            S.append(float(self.h_S[0]))
        return threshold_from_samples(S, parallel_fraction)

    def device_status(self) -> int:
        return lib().cerb_device_status(self.ctx, _stream())

    PROF_KINDS = ("gemm", "attention", "heads", "glue", "gate", "accept")

    def wait_diagnosis(self):
        out = (C.c_int32 * 4)()
        _check(lib().cerb_wait_diagnosis(self.ctx, out, _stream()), "cerb_wait_diagnosis")
        return list(out)

    def profile(self, on):
        """False / 0: off; True / 1: CUDA-event brackets per kernel family; 2: the GEMM kernels stamp their own
        spans with the device timer (the launch sequence stays as it is)."""
        _check(lib().cerb_profile_enable(self.ctx, int(on)), "cerb_profile_enable")

    def profile_read(self):
        """{family: (milliseconds, launch groups)} since the last read."""
        ms = (C.c_double * 6)()
        gr = (C.c_int64 * 6)()
        _check(lib().cerb_profile_read(self.ctx, ms, gr, _stream()), "cerb_profile_read")
        return {k: (ms[i], gr[i]) for i, k in enumerate(self.PROF_KINDS)}

    def last_forward_rows(self) -> int:
        return int(lib().cerb_last_forward_rows(self.ctx))

    def launch_count(self) -> int:
        return lib().cerb_launch_count(self.ctx)

    def gather_kv(self, b: int, layer: int, length: int):
        """Contiguous [length][H][Dh] copies of a sequence's K and V (layout marshalling for tests)."""
        pages = torch.from_numpy(self.page_table_host[b, :(length + PAGE - 1) // PAGE].astype(np.int64)).to(self.device)
        k = self.k_pool[layer][pages].permute(0, 2, 1, 3).reshape(-1, self.shape.n_heads, self.shape.head_dim)[:length]
        v = self.v_pool[layer][pages].permute(0, 2, 1, 3).reshape(-1, self.shape.n_heads, self.shape.head_dim)[:length]
        return k, v


def tree_attention(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor,
                   lens: torch.Tensor, anc: torch.Tensor, scale: float, max_len: int,
                   n_active: Optional[torch.Tensor] = None, want_lse: bool = True, scratch: Optional[torch.Tensor] = None):
    """q [B][n][H][Dh]; pools [pages][H][16][Dh]; page_table [B][max_pages] int32; lens [B] int32;
    anc [n][ANC_WORDS] int64 bit patterns.  Returns (out, lse)."""
    B, n, H, Dh = q.shape
    dt = BF16 if q.dtype == torch.bfloat16 else F32
    out = torch.empty_like(q)
    lse = torch.empty(B, H, n, dtype=torch.float32, device=q.device) if want_lse else None
    if scratch is None:
        nb = C.c_size_t(0)
        _check(lib().cerb_attn_scratch_bytes(B, n, H, Dh, C.byref(nb)), "cerb_attn_scratch_bytes")
        scratch = torch.zeros(nb.value, dtype=torch.uint8, device=q.device)
    a = AttnArgs(dt, B, n, H, Dh, page_table.shape[1], q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
                 page_table.data_ptr(), lens.data_ptr(), _ptr(n_active), anc.data_ptr(), out.data_ptr(), _ptr(lse),
                 scale, max_len, k_pool.shape[0], scratch.data_ptr(), scratch.numel())
    _check(lib().cerb_tree_attention(C.byref(a), _stream()), "cerb_tree_attention")
    return out, lse, scratch


STATIC_ATTN_SCRATCH_BYTES = 16 << 20


def tree_attention_noalloc(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor,
                           lens: torch.Tensor, anc: torch.Tensor, scale: float, max_len: int, out: torch.Tensor,
                           lse: Optional[torch.Tensor] = None, n_active: Optional[torch.Tensor] = None) -> int:
    """Same operation as tree_attention for callers that must not allocate device memory: the split-KV
    scratch is a static array inside the library and `out` / `lse` are passed in, so neither this
    wrapper nor the library allocates anything.  Returns the library's status code."""
    B, n, H, Dh = q.shape
    a = AttnArgs(BF16, B, n, H, Dh, page_table.shape[1], q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
                 page_table.data_ptr(), lens.data_ptr(), _ptr(n_active), anc.data_ptr(), out.data_ptr(), _ptr(lse),
                 scale, max_len, k_pool.shape[0], None, 0)
    return lib().cerb_tree_attention_noalloc(C.byref(a), _stream())


def tree_attention_noalloc_status() -> int:
    """Device-side status of the calls made through tree_attention_noalloc since the last read (synchronises)."""
    return lib().cerb_tree_attention_noalloc_status(_stream())


def gemm(X: torch.Tensor, W: torch.Tensor, scratch: Optional[torch.Tensor] = None) -> torch.Tensor:
    """out[M][N] fp32 = X[M][K] . W[N][K]^T on the library's GEMM path."""
    M, K = X.shape
    N = W.shape[0]
    dt = BF16 if X.dtype == torch.bfloat16 else F32
    out = torch.empty(M, N, dtype=torch.float32, device=X.device)
    if scratch is None:
        nb = C.c_size_t(0)
        _check(lib().cerb_gemm_scratch_bytes(M, N, K, C.byref(nb)), "cerb_gemm_scratch_bytes")
        scratch = torch.empty(nb.value + 256, dtype=torch.uint8, device=X.device)
    sp = (scratch.data_ptr() + 255) // 256 * 256
    _check(lib().cerb_gemm(dt, X.data_ptr(), W.data_ptr(), out.data_ptr(), M, N, K, sp, scratch.numel() - 256, _stream()), "cerb_gemm")
    return out
