#!/usr/bin/env python
"""Benchmark of the Cerberus decoding step on a 7B-shaped, random-init bf16 model.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl cerb|reference] [--workload 7b|13b|tiny]
    python bench.py --sweep            # verify step alone over batch x KV length x tree nodes

A "step" is one whole decoding step (gate, draft when the gate allows it, tree verification
through all layers, acceptance and KV compaction) of one sequence.  Prints ONE JSON line.
With N > 1 (launched by torch.distributed.run) every rank decodes its own sequence on its own
GPU with a full replica of the weights; there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2410_13344_b200 import synth

METRIC = "decoded tokens/s at 7B shape (verify-step latency in extra keys)"
UNIT = "tokens/s"
N_NODES = 64
TOPK = [10, 10, 10, 10]
PROMPT_LEN = 2048
HBM_NOMINAL_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one gemm_bf16_kernel launch (ncu --set full, M=64 N=22016 K=4096:
# profiles/gemm_bf16_kernel_M64_N22016_K4096.md); algorithmic bytes of that launch: 183.7 MB.
GEMM_TRAFFIC = 186.0e6
GEMM_TRAFFIC_NOTE = {"launch": "M=64 N=22016 K=4096", "algorithmic_bytes_per_launch": 183.7e6}


def draft_setup(name: str):
    """(decoding heads, top-k per head, tree nodes) of a workload."""
    if name == "7b":
        return 4, TOPK, N_NODES
    if name == "13b":
        return 5, [10] * 5, N_NODES
    return 4, [4, 2, 1, 1], 16


def workload(name: str):
    if name == "7b":
        return synth.shape_7b(), PROMPT_LEN, "7B-shaped bf16 model, 4 Cerberus heads, 64-node tree, 2048-token prompt, batch 1"
    if name == "13b":
        return synth.shape_13b(), 4096, "13B-shaped bf16 model, 5 Cerberus heads, 64-node tree, 4096-token prompt, batch 1"
    if name == "tiny":
        ms = synth.tiny_shape("bf16")
        return ms, 64, "tiny bf16 model (debug)"
    raise SystemExit("unknown workload " + name)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def sustained_tensor_peak():
    """bf16 TFLOP/s of a library GEMM run back to back for seconds (power-capped clocks): the denominator for GEMMs
    timed inside a long batched step; the burst figure of peaks() is the one for a kernel timed alone."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        if "bf16_tflops_sustained" in d:
            return float(d["bf16_tflops_sustained"]), "measured"
    return 1400.0, "fallback"


class ClockSampler:
    """nvidia-smi sampling of SM clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if val.strip().lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def init_dist():
    """One process per GPU (replicas, no data-path collective).  NCCL when CUDA is there, gloo otherwise."""
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if torch.cuda.is_available():
        dist.init_process_group("nccl", device_id=torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0))))
    else:
        dist.init_process_group("gloo")


def max_over_ranks(value: float, world: int) -> float:
    """The slowest rank's time: what the whole job waited for."""
    if world <= 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device="cuda" if torch.cuda.is_available() else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def rank_prompt(vocab: int, prompt_len: int, rank: int) -> torch.Tensor:
    """Every rank decodes its own sequence (weak scaling)."""
    return synth.make_prompt(vocab, prompt_len, seq=rank).to(torch.int32)


def algorithmic_bytes(ms: synth.ModelShape, M: int, kv_len: int, n: int, heads_bytes: int):
    """Bytes one step must move at least (weights once, activations in/out at storage precision)."""
    d, F, V, HD = ms.d_model, ms.mlp_dim, ms.vocab, ms.n_heads * ms.head_dim
    e = 2
    per_layer = [(3 * HD, d), (d, HD), (2 * F, d), (d, F)]
    gemm = sum((N * K + M * K + M * N) * e for N, K in per_layer) * ms.n_layers + (V * d + M * d) * e + M * V * 4
    attn = ((kv_len + n) * HD * 2 * e + 2 * n * HD * e) * ms.n_layers
    return gemm, attn, heads_bytes


def run_cerb(args, rank, world):
    from paper_2410_13344_b200 import binding as cb
    import __graft_entry__
    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    ms, prompt_len, wl_name = workload(args.workload)
    # comparison modes (Sec. 5): "medusa" = independent heads without the sequential link and no gate,
    # "no-gate" = Cerberus heads, every step parallel, "ar" = plain auto-regressive decoding
    n_ch, topk, n_nodes = draft_setup(args.workload)
    layout = synth.medusa_layout(n_ch, 4) if args.mode == "medusa" else synth.cerberus_layout(n_ch, 4)
    t_setup = time.time()
    model = synth.make_model(ms, device="cuda")
    heads = synth.make_heads(ms, layout, device="cuda")
    heads_bytes = sum(t.numel() * t.element_size() for t in heads.values())
    eng = cb.Cerberus(ms, model, layout, heads, topk, max_tokens=prompt_len + 9 * (args.steps + args.warmup + 160) + 64,
                      max_batch=1, max_nodes=128)
    tree = synth.best_first_tree(n_nodes, topk)
    th = eng.tree(tree)
    # every rank decodes its own prompt (weak scaling: one sequence per GPU)
    prompt = rank_prompt(ms.vocab, prompt_len, rank)
    h_prompt = prompt.reshape(1, -1).contiguous().pin_memory()
    d_prompt = torch.empty_like(h_prompt, device="cuda")

    def prefill():
        d_prompt.copy_(h_prompt, non_blocking=True)
        eng.prefill(d_prompt, [prompt_len])

    def sync():
        torch.cuda.current_stream().synchronize()

    # --- calibration: an auto-regressive run gives the gate values and the true greedy continuation
    prefill()
    cal_S, truth = [], []
    for _ in range(max(4, args.cal_steps)):
        eng.step(th, -1.0)
        sync()
        cal_S.append(float(eng.h_S[0]))
        truth.extend(int(t) for t in eng.h_tokens[0, :int(eng.h_n_accept[0])])
    T = cb.threshold_from_samples(cal_S, 0.7)          # about 70 % of the steps decode in parallel
    if args.mode in ("medusa", "no-gate"):
        T = 1e9
    elif args.mode == "ar":
        T = -1.0
    setup_s = time.time() - t_setup

    def decode(n_steps, plant_lengths=None, e2e=False, h_plant=None, d_plant=None):
        toks, modes, accepted, emitted = 0, [], [], 0
        for i in range(n_steps):
            plant = None
            if plant_lengths is not None:
                want = plant_lengths[i % len(plant_lengths)]
                ov = [-1] * tree.n
                path = deepest
                for j, node in enumerate(path[1:want], start=1):
                    if emitted + j < len(truth):
                        ov[node] = truth[emitted + j]
                h_plant[0, :] = torch.tensor(ov, dtype=torch.int32)
                d_plant.copy_(h_plant, non_blocking=True)
                plant = d_plant
            elif e2e:
                d_plant.copy_(h_plant, non_blocking=True)     # this step's host inputs (no overrides)
                plant = d_plant
            eng.step(th, T, plant)
            sync()                                             # results are in the pinned mirrors
            na = int(eng.h_n_accept[0])
            emitted += na
            toks += na
            modes.append(int(eng.h_mode[0]))
            accepted.append(na)
        return toks, modes, accepted

    depth = [0] * tree.n
    for v in range(1, tree.n):
        depth[v] = depth[tree.parent[v]] + 1
    leaf = max(range(tree.n), key=lambda v: (depth[v], -v))
    deepest = []
    while leaf >= 0:
        deepest.append(leaf)
        leaf = int(tree.parent[leaf])
    deepest = deepest[::-1]
    h_plant = torch.full((1, tree.n), -1, dtype=torch.int32).pin_memory()
    d_plant = torch.full((1, tree.n), -1, dtype=torch.int32, device="cuda")

    def barrier():
        sync()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        sync()

    def timed(n_steps, **kw):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = eng.launch_count()
        e0.record()
        out = decode(n_steps, **kw)
        e1.record()
        barrier()
        ms_total = max_over_ranks(e0.elapsed_time(e1), world)
        return ms_total, out, eng.launch_count() - l0

    # --- A: the headline run (device-resident inputs), natural acceptance
    prefill()
    decode(args.warmup)
    sampler = ClockSampler(local)
    ms_a, (tok_a, modes_a, acc_a), launches = timed(args.steps)
    clocks = sampler.stop()
    # --- B: same run with per-family device timing, for the roofline of the dominant kernel
    prof_steps = min(args.steps, 24)
    eng.profile(True)
    eng.profile_read()
    ms_b, (tok_b, modes_b, acc_b), _ = timed(prof_steps)
    prof = eng.profile_read()
    # --- B2: the same steps once more with the GEMM kernels stamping their own spans (first CTA past its
    # dependency wait .. last CTA done, device nanosecond timer): the launch sequence and its overlaps stay intact
    eng.profile(2)
    _, (_, modes_b2, _), _ = timed(prof_steps)
    prof_clk = eng.profile_read()
    eng.profile(False)
    # --- C: end to end through the public call with host buffers in the loop
    prefill()
    decode(args.warmup, e2e=True, h_plant=h_plant, d_plant=d_plant)
    ms_c, (tok_c, _, _), _ = timed(args.steps, e2e=True, h_plant=h_plant, d_plant=d_plant)
    # --- D: planted acceptance (synthetic).  Before each step the greedy continuation from the current
    # state is obtained with chain-shaped forwards (untimed) and written over one root-to-leaf path, so
    # that 1..5 tokens are accepted; only the steps themselves are timed (one event pair per step).
    prefill()
    th1 = eng.tree(synth.single_node_tree())
    chains = {j: eng.tree(synth.chain_tree(j)) for j in range(2, 5)}
    plant_lengths = [1, 2, 3, 4, 5]
    ms_d, tok_d, acc_d = 0.0, 0, []
    for i in range(min(args.steps, 20)):
        want = plant_lengths[i % len(plant_lengths)]
        _, roots, _ = eng.read_state()
        cont = [int(roots[0])]
        if want > 1:
            am1, _, _ = eng.verify(th1, torch.tensor([cont], dtype=torch.int32, device="cuda"))
            cont.append(int(am1[0, 0]))
            for j in range(2, want):
                amc, _, _ = eng.verify(chains[j], torch.tensor([cont[:j]], dtype=torch.int32, device="cuda"))
                cont.append(int(amc[0, j - 1]))
        ov = [-1] * tree.n
        for j, node in enumerate(deepest[1:want], start=1):
            ov[node] = cont[j]
        h_plant[0, :] = torch.tensor(ov, dtype=torch.int32)
        sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        d_plant.copy_(h_plant, non_blocking=True)
        eng.step(th, 1e9, d_plant)                 # always parallel: the planted path is there to be verified
        e1.record()
        sync()
        ms_d += e0.elapsed_time(e1)
        acc_d.append(int(eng.h_n_accept[0]))
        tok_d += acc_d[-1]
    h_plant[0, :] = -1
    # --- prefill alone
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); prefill(); e1.record(); sync()
    prefill_ms = e0.elapsed_time(e1)
    status = eng.device_status()

    agg = lambda x: x * world          # every rank runs the same amount of work
    hbm_peak, tf_peak, peak_kind = peaks()
    kv_len = prompt_len + 64 + sum(acc_a) // 2
    par_b = sum(1 for m in modes_b if m == 0)
    n_b = [n_nodes if m == 0 else 1 for m in modes_b]
    gemm_bytes = sum(algorithmic_bytes(ms, M, kv_len, M, 0)[0] for M in n_b)
    attn_bytes = sum(algorithmic_bytes(ms, M, kv_len, M, 0)[1] for M in n_b)
    gemm_ms, gemm_groups = prof["gemm"]
    attn_ms, attn_groups = prof["attention"]
    heads_ms, heads_groups = prof["heads"]
    gemm_gbs = gemm_bytes / gemm_ms / 1e6 if gemm_ms > 0 else None
    gemm_clk_ms, gemm_clk_n = prof_clk["gemm"]
    gemm_bytes_clk = sum(algorithmic_bytes(ms, n_nodes if m == 0 else 1, kv_len, 1, 0)[0] for m in modes_b2)
    gemm_clk_gbs = gemm_bytes_clk / gemm_clk_ms / 1e6 if gemm_clk_ms > 0 else None
    attn_gbs = attn_bytes / attn_ms / 1e6 if attn_ms > 0 else None
    heads_gbs = heads_bytes * par_b / heads_ms / 1e6 if heads_ms > 0 else None
    HD_ = ms.n_heads * ms.head_dim
    gemm_params = ms.n_layers * (3 * HD_ * ms.d_model + ms.d_model * HD_ + 3 * ms.mlp_dim * ms.d_model) + ms.vocab * ms.d_model
    gemm_flops = sum(2 * M * gemm_params for M in n_b)
    par_steps = [i for i, m in enumerate(modes_a) if m == 0]
    line = {
        "metric": METRIC.replace("7B", "13B") if args.workload == "13b" else METRIC, "value": agg(tok_a) / (ms_a / 1e3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_a / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl_name, "mode": args.mode, "parallelism": "replicas" if world > 1 else "single",
                   "l2": "every step streams the model's weights (13 GB at the 7B shape), far beyond the 126 MB L2",
                   "threshold": T, "tree_nodes": n_nodes, "topk": topk, "prompt_len": prompt_len,
                   "acceptance": "natural (random-init heads)"},
        "verify_step_latency_us": ms_a / args.steps * 1e3,
        "parallel_step_fraction": len(par_steps) / max(1, len(modes_a)),
        "mean_accepted_per_step": tok_a / max(1, args.steps),
        "gpu_launches": launches,
        "e2e": {"value": agg(tok_c) / (ms_c / 1e3), "unit": UNIT, "h2d_bytes_per_step": int(h_plant.numel() * 4),
                "d2h_bytes_per_step": int(4 + 4 + 4 + 4 * cb.PATH_MAX), "ms_per_step": ms_c / args.steps},
        "planted": {"value": agg(tok_d) / (ms_d / 1e3), "unit": UNIT, "mean_accepted_per_step": tok_d / max(1, len(acc_d)),
                    "note": "synthetic acceptance: one tree path overwritten with the greedy continuation (lengths 1..5 requested), every step parallel; only the steps are timed"},
        "prefill_ms": prefill_ms,
        "roofline": {"bound": "hbm", "kernel": "gemm_bf16_kernel (tcgen05 weight-streaming GEMM)",
                     "achieved": gemm_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": (gemm_gbs / hbm_peak) if gemm_gbs else None,
                     "peak_kind": peak_kind + " copy bandwidth", "frac_of_nominal_8TBs": (gemm_gbs / HBM_NOMINAL_GBS) if gemm_gbs else None,
                     "traffic": GEMM_TRAFFIC, "traffic_of": GEMM_TRAFFIC_NOTE, "launch_groups": gemm_groups, "ms_per_step": gemm_ms / prof_steps,
                     "timing": "CUDA events around every GEMM launch (they keep neighbouring kernels from overlapping)",
                     "device_clock": {"achieved": gemm_clk_gbs, "frac": (gemm_clk_gbs / hbm_peak) if gemm_clk_gbs else None,
                                      "ms_per_step": gemm_clk_ms / prof_steps, "launches": gemm_clk_n,
                                      "timing": "each GEMM's own span in the undisturbed step: first CTA past the dependency "
                                                "wait .. last CTA done, device timer"},
                     "tensor_tflops": (gemm_flops / gemm_ms / 1e9) if gemm_ms > 0 else None, "tensor_peak_tflops": tf_peak},
        "attention": {"achieved": attn_gbs, "unit": "GB/s", "frac_of_measured": (attn_gbs / hbm_peak) if attn_gbs else None,
                      "frac_of_nominal_8TBs": (attn_gbs / HBM_NOMINAL_GBS) if attn_gbs else None,
                      "ms_per_step": attn_ms / prof_steps, "kv_len": kv_len},
        "heads": {"achieved": heads_gbs, "unit": "GB/s", "ms_per_parallel_step": heads_ms / max(1, par_b)},
        "profile_ms_per_step": {k: v[0] / prof_steps for k, v in prof.items()},
        "profiled_ms_per_step": ms_b / prof_steps,
        "clocks": clocks, "device_status": status, "setup_s": setup_s,
    }
    if rank == 0 and world == 1 and args.workload == "7b" and not args.no_corner:
        eng.close()
        torch.cuda.empty_cache()
        line["batched_corner"] = batched_corner(cb, ms, model, hbm_peak, tf_peak)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(ms, model, heads, layout, tree, prompt_len, tok_a / max(1, args.steps),
                                            len(par_steps) / max(1, len(modes_a)), budget_s=20.0)
    if rank == 0:
        print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# CPU baseline / reference arm: the oracle, as it stands, on the host cores
# ------------------------------------------------------------------------------------------------

def _oracle_sample(ms, model, heads, layout, tree, prompt_len, n_sample_layers):
    """Builds what the oracle needs for one bounded sample: the first layers' weights in float64,
    a synthetic committed cache of prompt_len tokens, tree tokens."""
    from oracle import cerberus_oracle as orc
    sub = {"embed": model["embed"].cpu().double(), "final_norm": model["final_norm"].cpu().double(),
           "lm_head": model["lm_head"].cpu().double()}
    for l in range(n_sample_layers):
        for k in ("attn_norm", "wqkv", "wo", "mlp_norm", "wgu", "wd"):
            sub[f"{k}.{l}"] = model[f"{k}.{l}"].cpu().double()
    sh = orc.Shape(n_sample_layers, ms.d_model, ms.n_heads, ms.head_dim, ms.mlp_dim, ms.vocab, ms.dtype)
    st = orc.new_state(sh, prompt_len + tree.n + 8)
    g = torch.Generator().manual_seed(1234)
    for l in range(n_sample_layers):
        st.k[l][:prompt_len] = torch.randn(prompt_len, ms.n_heads, ms.head_dim, generator=g, dtype=torch.float64)
        st.v[l][:prompt_len] = torch.randn(prompt_len, ms.n_heads, ms.head_dim, generator=g, dtype=torch.float64)
    st.length = prompt_len
    tok = [int(t) for t in synth.randint(7, 1, (tree.n,), ms.vocab)]
    return orc, sub, sh, st, tok


def cpu_baseline(ms, model, heads, layout, tree, prompt_len, tokens_per_step, par_fraction, budget_s):
    t0 = time.time()
    ns = 4 if ms.n_layers >= 8 else ms.n_layers        # 4 layers in float64 = 6.5 GB of host memory at the 7B shape
    orc, sub, sh, st, tok = _oracle_sample(ms, model, heads, layout, tree, prompt_len, ns)
    reps = 2
    t1 = time.time()
    for _ in range(reps):
        orc.verify_tree(sub, sh, st, tok, tree.parent)
    t_sample = (time.time() - t1) / reps
    t2 = time.time()
    orc.linear(torch.zeros(tree.n, ms.d_model, dtype=torch.float64), sub["lm_head"])
    t_lm = time.time() - t2
    # decoding heads: time one head's FC on the host and scale by parameter count
    t3 = time.time()
    hW = heads["fc.0"].cpu().double()
    orc.linear(torch.zeros(1, hW.shape[1], dtype=torch.float64), hW)
    t_fc = time.time() - t3
    head_params = sum(t.numel() for t in heads.values())
    t_heads = t_fc * head_params / hW.numel()
    t_step = (t_sample - t_lm) * ms.n_layers / ns + t_lm + par_fraction * t_heads
    return {"value": tokens_per_step / t_step, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "sample": f"one 64-node verify step through {ns} of {ms.n_layers} layers plus the LM head on a synthetic "
                      f"{prompt_len}-token cache (mean of {reps} runs: {t_sample:.1f} s), layers scaled to {ms.n_layers}; heads scaled from one FC "
                      f"({t_fc:.2f} s); weight conversion to float64 excluded; extrapolated step {t_step:.1f} s",
            "seconds": time.time() - t0}


def run_reference(args, rank, world):
    if rank != 0:
        return
    ms, prompt_len, wl_name = workload(args.workload)
    n_ch, topk, n_nodes = draft_setup(args.workload)
    layout = synth.cerberus_layout(n_ch, 4)
    tree = synth.best_first_tree(n_nodes, topk)
    # four layers of the model (the sample) plus embedding / LM head, generated on the host
    # (values do not matter for timing; a seeded torch generator is much faster on the host than the
    # counter-based generator the parity tests use)
    # layers per step sample: four when the requested step count leaves room for it, one for long runs, so that the
    # whole run stays within a few minutes (a sample layer costs about 0.7 s on 16 cores)
    NS = min(ms.n_layers, 4 if args.steps + args.warmup <= 40 else 1)
    ms1 = synth.ModelShape(NS, ms.d_model, ms.n_heads, ms.head_dim, ms.mlp_dim, ms.vocab, ms.dtype)
    g = torch.Generator().manual_seed(0)
    d_, F_, V_, HD_ = ms.d_model, ms.mlp_dim, ms.vocab, ms.n_heads * ms.head_dim

    def rnd(*shape, std=0.02, mean=0.0):
        return (torch.randn(*shape, generator=g) * std + mean).to(ms.torch_dtype)

    model = {"embed": rnd(V_, d_), "final_norm": rnd(d_, std=0.1, mean=1.0), "lm_head": rnd(V_, d_)}
    for l in range(NS):
        model.update({f"attn_norm.{l}": rnd(d_, std=0.1, mean=1.0), f"wqkv.{l}": rnd(3 * HD_, d_), f"wo.{l}": rnd(d_, HD_),
                      f"mlp_norm.{l}": rnd(d_, std=0.1, mean=1.0), f"wgu.{l}": rnd(2 * F_, d_), f"wd.{l}": rnd(d_, F_)})
    orc, sub, sh, st, tok = _oracle_sample(ms1, model, {}, layout, tree, prompt_len, NS)
    lm_t0 = time.time()
    orc.linear(torch.zeros(tree.n, ms.d_model, dtype=torch.float64), sub["lm_head"])
    t_lm = time.time() - lm_t0
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.time()
        orc.verify_tree(sub, sh, st, tok, tree.parent, want_logits=False)
        if i >= args.warmup:
            times.append(time.time() - t0)
    t_sample = sum(times) / len(times)
    t_step = t_sample * ms.n_layers / NS + t_lm
    value = 1.0 / t_step
    sample = (f"per step: one {n_nodes}-node verify step of the oracle through {NS} of {ms.n_layers} layers on a "
              f"synthetic {prompt_len}-token cache ({t_sample:.2f} s), scaled to {ms.n_layers} layers, plus the LM head timed once ({t_lm:.2f} s); heads and gate excluded; "
              f"one token per step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": t_step * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl_name, "parallelism": "host cores"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_kernel(args):
    """One kernel alone, through its stand-alone entry point, on inputs that rotate over enough
    distinct buffers to exceed the L2; CUDA-event time per launch (includes the host-side call)."""
    from paper_2410_13344_b200 import binding as cb
    import __graft_entry__
    __graft_entry__.build()
    torch.cuda.set_device(0)
    hbm_peak, tf_peak, kind = peaks()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timeit(fn):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for i in range(args.iters):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.iters * 1e3

    if args.kernel == "gemm":
        M, N, K = args.M, args.N, args.K
        nrot = max(2, min(8, int(1.5e9 // (N * K * 2)) + 1))
        Ws = [synth.normal(9, 100 + i, (N, K), 0.02, dtype=torch.bfloat16, device="cuda") for i in range(nrot)]
        X = synth.normal(9, 1, (M, K), 1.0, dtype=torch.bfloat16, device="cuda")
        nb = cb.C.c_size_t(0)
        cb.lib().cerb_gemm_scratch_bytes(M, N, K, cb.C.byref(nb))
        scratch = torch.empty(nb.value + 256, dtype=torch.uint8, device="cuda")
        us = timeit(lambda i: cb.gemm(X, Ws[i % nrot], scratch))
        byts = (N * K + M * K) * 2 + M * N * 4
        out = {"kernel": "gemm", "M": M, "N": N, "K": K, "us": us, "GBs": byts / us / 1e3, "frac_hbm": byts / us / 1e3 / hbm_peak,
               "TFs": 2.0 * M * N * K / us / 1e6, "frac_tensor": 2.0 * M * N * K / us / 1e6 / tf_peak, "peaks": kind, "rotating_buffers": nrot,
               "note": "per-call time of cerb_gemm = the GEMM kernel plus the kernel that sums its fp32 partial slots into one "
                       "matrix; from a few hundred rows on the second one is a large part (the step's own consumers read the "
                       "slots directly) -- for the GEMM kernel alone see --sweep (device-clock spans) or the ncu summaries"}
    else:
        B, n, L, H, Dh = args.B, args.n, args.len, 32, 128
        max_len = L + n
        mp = (max_len + 15) // 16
        npool = B * mp
        per = npool * H * 16 * Dh * 2 * 2
        nrot = max(2, min(8, int(1.5e9 // per) + 1))
        pools = [(synth.normal(9, 200 + 2 * i, (npool, H, 16, Dh), 1.0, dtype=torch.bfloat16, device="cuda"),
                  synth.normal(9, 201 + 2 * i, (npool, H, 16, Dh), 1.0, dtype=torch.bfloat16, device="cuda")) for i in range(nrot)]
        q = synth.normal(9, 2, (B, n, H, Dh), 1.0, dtype=torch.bfloat16, device="cuda")
        tree = synth.random_parent_tree(n, 5) if n > 1 else synth.single_node_tree()
        anc = torch.from_numpy(cb.tree_ancestors(tree.parent).view(np.int64)).cuda()
        pt = torch.arange(B * mp, dtype=torch.int32, device="cuda").reshape(B, mp)
        lens = torch.full((B,), L, dtype=torch.int32, device="cuda")
        _, _, scratch = cb.tree_attention(q, pools[0][0], pools[0][1], pt, lens, anc, 1 / math.sqrt(Dh), max_len)
        us = timeit(lambda i: cb.tree_attention(q, pools[i % nrot][0], pools[i % nrot][1], pt, lens, anc,
                                                1 / math.sqrt(Dh), max_len, scratch=scratch))
        byts = B * (L + n) * H * Dh * 2 * 2 + 2 * B * n * H * Dh * 2
        out = {"kernel": "attention", "B": B, "n": n, "len": L, "heads": H, "head_dim": Dh, "us": us, "GBs": byts / us / 1e3,
               "frac_hbm": byts / us / 1e3 / hbm_peak, "frac_of_nominal_8TBs": byts / us / 1e3 / HBM_NOMINAL_GBS,
               "MB": byts / 1e6, "peaks": kind, "rotating_buffers": nrot}
    print(json.dumps(out))


def _verify_point(eng, ms, params, B, L, n, iters, hbm_peak, tf_peak):
    """One point of the verify-step sweep on an engine whose B sequences hold L committed tokens: step latency
    (undisturbed launch sequence), attention GB/s (event brackets), GEMM TFLOP/s (the kernels' own device-clock spans)."""
    ev = lambda: torch.cuda.Event(enable_timing=True)
    th = eng.tree(synth.random_parent_tree(n, 6, tree_id=n))
    tok = torch.stack([synth.make_prompt(ms.vocab, n, seq=1000 + b).to(torch.int32) for b in range(B)]).cuda().contiguous()
    run = lambda: eng.verify(th, tok)          # verify without accept leaves the committed state as it is
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record()
    for _ in range(iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    step_ms = e0.elapsed_time(e1) / iters
    k = max(2, iters // 2)
    eng.profile(1); eng.profile_read()
    for _ in range(k):
        run()
    prof = eng.profile_read()
    eng.profile(2)
    for _ in range(k):
        run()
    clk = eng.profile_read()
    eng.profile(False)
    M = B * n
    gemm_b, attn_b, _ = algorithmic_bytes(ms, M, L, n, 0)
    attn_b *= B
    attn_ms = prof["attention"][0] / k
    gemm_ev_ms, gemm_ck_ms = prof["gemm"][0] / k, clk["gemm"][0] / k
    flops = 2.0 * M * params
    bound_ms = max(flops / (tf_peak * 1e9), gemm_b / (hbm_peak * 1e6))
    pt = {"B": B, "len": L, "n": n, "rows": M, "step_us": step_ms * 1e3,
          "attn_us_per_layer": attn_ms / ms.n_layers * 1e3, "attn_GBs": attn_b / attn_ms / 1e6,
          "attn_frac_of_measured": attn_b / attn_ms / 1e6 / hbm_peak, "attn_frac_of_8TBs": attn_b / attn_ms / 1e6 / HBM_NOMINAL_GBS,
          "gemm_ms_events": gemm_ev_ms, "gemm_ms_device_clock": gemm_ck_ms,
          "gemm_TFs": flops / gemm_ck_ms / 1e9, "gemm_frac_of_tensor_peak": flops / gemm_ck_ms / 1e9 / tf_peak,
          "gemm_weight_GBs": gemm_b / gemm_ck_ms / 1e6, "gemm_bound": "tensor" if flops / (tf_peak * 1e9) > gemm_b / (hbm_peak * 1e6) else "hbm",
          "gemm_frac_of_binding_roofline": bound_ms / gemm_ck_ms, "glue_ms_events": prof["glue"][0] / k}
    sus, sus_kind = sustained_tensor_peak()
    pt["gemm_frac_of_sustained_tensor_peak"] = flops / gemm_ck_ms / 1e9 / sus
    pt["sustained_tensor_peak_TFs"] = sus
    pt["sustained_peak_kind"] = sus_kind
    eng.free_tree(th)
    return pt


def batched_corner(cb, ms, model, hbm_peak, tf_peak):
    """The batched corner of the verify step: 16 sequences x 128-node trees (2048 rows per GEMM) on 512-token caches.
    The batch-1 headline keeps the GEMMs HBM-bound; here they are bound by the tensor pipe."""
    B, L, n = 16, 512, 128
    HD = ms.n_heads * ms.head_dim
    params = ms.n_layers * (3 * HD * ms.d_model + ms.d_model * HD + 3 * ms.mlp_dim * ms.d_model) + ms.vocab * ms.d_model
    eng = cb.Cerberus(ms, model, None, None, (), max_tokens=L + 16, max_batch=B, max_nodes=128)
    prompts = torch.stack([synth.make_prompt(ms.vocab, L, seq=b).to(torch.int32) for b in range(B)]).cuda().contiguous()
    eng.prefill(prompts, [L] * B)
    torch.cuda.synchronize()
    pt = _verify_point(eng, ms, params, B, L, n, 4, hbm_peak, tf_peak)
    pt["device_status"] = eng.device_status()
    pt["note"] = ("one verify step, batch 16 x 128 nodes x 512 committed tokens; GEMM TFLOP/s from the kernels' own "
                  "device-clock spans, against the measured bf16 tensor peak (burst figure; the sustained one, which is what a "
                  "35 ms step of back-to-back GEMMs runs against, beside it)")
    eng.close()
    return pt


def run_sweep(args):
    """The verify step alone (row a5 + a6: embedding .. LM head + argmax over every tree node) at the 7B shape over
    batch x committed KV length x tree nodes, random-parent trees of depth <= 6, KV produced by a real prefill of
    random token ids.  One JSON line per point: step latency (undisturbed launch sequence, CUDA events), attention
    GB/s over its algorithmic bytes (event brackets around the attention launches), GEMM TFLOP/s from the kernels'
    own device-clock spans and its fraction of the binding roofline min(tensor peak, rows x HBM)."""
    from paper_2410_13344_b200 import binding as cb
    import __graft_entry__
    __graft_entry__.build()
    torch.cuda.set_device(0)
    hbm_peak, tf_peak, kind = peaks()
    ms = synth.shape_13b() if args.workload == "13b" else synth.shape_7b()
    model = synth.make_model(ms, device="cuda")
    HD = ms.n_heads * ms.head_dim
    params = ms.n_layers * (3 * HD * ms.d_model + ms.d_model * HD + 3 * ms.mlp_dim * ms.d_model) + ms.vocab * ms.d_model
    batches = [int(x) for x in args.sweep_B.split(",")]
    lens = [int(x) for x in args.sweep_len.split(",")]
    nodes = [int(x) for x in args.sweep_n.split(",")]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    points = []
    for B in batches:
        for L in lens:
            eng = cb.Cerberus(ms, model, None, None, (), max_tokens=L + 16, max_batch=B, max_nodes=max(128, max(nodes)))
            prompts = torch.stack([synth.make_prompt(ms.vocab, L, seq=b).to(torch.int32) for b in range(B)]).cuda().contiguous()
            eng.prefill(prompts, [L] * B)
            torch.cuda.synchronize()
            for n in nodes:
                pt = _verify_point(eng, ms, params, B, L, n, args.iters, hbm_peak, tf_peak)
                assert eng.device_status() == 0
                print(json.dumps(pt), flush=True)
                points.append(pt)
            eng.close()
            del eng, prompts
            torch.cuda.empty_cache()
    print(json.dumps({"sweep": "verify step, %s shape, bf16" % ("13B" if args.workload == "13b" else "7B"), "points": len(points), "peaks": kind, "hbm_GBs": hbm_peak,
                      "tensor_TFs": tf_peak, "iters": args.iters}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="cerb", choices=["cerb", "reference"])
    ap.add_argument("--workload", default="7b")
    ap.add_argument("--mode", default="cerberus", choices=["cerberus", "medusa", "no-gate", "ar"],
                    help="decoding variant: the method, or one of the comparison modes of Sec. 5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cal-steps", type=int, default=64, help="auto-regressive calibration steps before the timed runs")
    ap.add_argument("--kernel", default=None, choices=["gemm", "attention"], help="time one kernel alone instead of the step")
    ap.add_argument("--M", type=int, default=64)
    ap.add_argument("--N", type=int, default=22016)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--B", type=int, default=1)
    ap.add_argument("--n", type=int, default=64)
    ap.add_argument("--len", type=int, default=2048)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--no-corner", action="store_true", help="skip the batched corner (batch 16 x 128 nodes) of the default line")
    ap.add_argument("--sweep", action="store_true", help="verify step alone over batch x KV length x tree nodes (7B shape)")
    ap.add_argument("--sweep-B", default="1,2,4,8,16")
    ap.add_argument("--sweep-len", default="512,2048,8192")
    ap.add_argument("--sweep-n", default="16,32,64,128")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.kernel:
        run_kernel(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    if world > 1:
        init_dist()
    try:
        run_cerb(args, rank, world)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
