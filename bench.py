#!/usr/bin/env python
"""Benchmark of tree-causal prefix-shared attention, forward + backward.

Metric: fwd+bwd TFLOP/s over deduplicated FLOPs (14 * d * Hq * tree_pairs:
forward 4d, backward 10d per attended (query, key) pair and query head; exact
mask counts, no tile padding, no duplicated prefix work, no recompute).

  python bench.py --gpus N --steps K --warmup W [--config c2] [--impl reference]

Without --config the headline is c5 (the largest single-GPU configuration) and c1 (fp32), c2, c3, c4
and the small-suffix case c2s are measured in the same run and reported under `per_config`.

One step = one pass of the whole hot path (forward, D pre-pass, dQ, dK/dV) over
one synthetic batch.  N > 1 (torchrun): every rank runs an independent batch
(prefix groups never span workers), no data-path collective, weak scaling.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tree_attn_fwd_bwd_dedup_tflops"
UNIT = "TFLOP/s"

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel
# (dkv_kernel), from the ncu captures summarised under profiles/ ; None = not captured.
NCU_TRAFFIC_BYTES = {"c2": 353620000 + 24440000,       # profiles/dkv_kernel_c2.md
                     "c3": 1140000000 + 65560000,      # profiles/dram_traffic_c5_c3.md
                     "c5": 92590000000 + 835340000}    # profiles/dram_traffic_c5_c3.md (full size, one pass)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *a):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        # under load = the upper half of the samples (idle samples before/after the region are dropped)
        sm_sorted = sorted(sm)
        load = sm_sorted[len(sm_sorted) // 2:]
        return {"sm_mhz": float(np.median(load)), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def dedup_flops(d, Hq, pairs):
    return 14.0 * d * Hq * float(pairs)


# --------------------------------------------------------------------------- oracle legs
def sub_workload(w, n_keep):
    """The first `n_keep` samples of `w` (their root-to-end paths), as a workload."""
    from paper_2608_25683_b200.workloads import Workload

    n = len(w.parent)
    has_child = [False] * n
    for p in w.parent:
        if p >= 0:
            has_child[p] = True
    flags = w.seg_flags or [1 | (0 if has_child[s] else 2) for s in range(n)]
    ends = [s for s in range(n) if flags[s] & 2][:n_keep]
    keep = set()
    for e in ends:
        s = e
        while s != -1:
            keep.add(s)
            s = w.parent[s]
    order = sorted(keep)
    new = {s: i for i, s in enumerate(order)}
    parent = [(-1 if w.parent[s] == -1 else new[w.parent[s]]) for s in order]
    roots_all = [s for s in range(n) if w.parent[s] == -1]
    gbs = [w.group_block_size[roots_all.index(s)] for s in order if w.parent[s] == -1]
    fl = [flags[s] if s in ends or not (flags[s] & 2) else flags[s] & ~2 for s in order]
    # an interior segment whose kept children all vanished cannot happen: ends are kept whole paths
    return Workload(w.name + f"[first {len(ends)} samples]", parent, [w.seg_len[s] for s in order], gbs,
                    w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, seg_flags=fl, seed=w.seed)


def oracle_leg(w, n_keep, seed, steps=1, warmup=0, budget=1.5e12):
    """Times the fp64 oracle, as it stands, on KV head 0 of the first n_keep samples.
    budget: fp64 FLOP of unshared work per pass (1.5e12 = 10-30 s on the host cores of this pool)."""
    import torch
    from oracle import oracle_attn, oracle_plan
    from paper_2608_25683_b200.workloads import make_inputs

    # Bound the sample: the oracle materialises every sample unshared, so its cost follows the flat pair
    # count.  Fewer samples first; if one sample alone is too large (c5), an evenly spaced subset of the
    # query rows (exact for those rows: the other dO rows are taken as zero).
    G = w.n_q_heads // w.n_kv_heads
    while True:
        sw = sub_workload(w, n_keep)
        plan = oracle_plan(sw.parent, sw.seg_len, sw.group_block_size, sw.seg_flags, None)
        flat_flops = dedup_flops(sw.head_dim, G, plan["flat_pairs"])
        if flat_flops <= budget or n_keep == 1:
            break
        n_keep -= 1
    q, k, v, d_o = make_inputs(plan["T_q"], plan["pool_slots"], plan["tok_slot"], sw.n_q_heads, sw.n_kv_heads,
                               sw.head_dim, sw.dtype, seed, device="cpu")
    f = lambda t: t.float().numpy()
    q, k, v, d_o = f(q), f(k), f(v), f(d_o)
    q_rows, rows_note = None, ""
    if flat_flops > budget:
        stride = int(np.ceil(flat_flops / budget))
        q_rows = np.arange(0, plan["T_q"], stride, dtype=np.int64)
        q, d_o = q[q_rows], d_o[q_rows]
        seg_of = np.repeat(np.arange(plan["n_seg"]), np.where(plan["seg_q_off"] >= 0, plan["seg_len"], 0))
        pos = q_rows - plan["seg_q_off"][seg_of[q_rows]]
        pairs = int(np.sum(plan["seg_anc_tokens"][seg_of[q_rows]].astype(np.int64) + pos + 1))
        flops = dedup_flops(sw.head_dim, G, pairs)
        rows_note = f", every {stride}th query row ({len(q_rows)} rows)"
    else:
        flops = dedup_flops(sw.head_dim, G, plan["tree_pairs"])
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        oracle_attn(plan, q, k, v, d_o, sw.softmax_scale, kv_heads=[0], q_rows=q_rows)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    t = float(np.mean(times))
    cores = len(os.sched_getaffinity(0))
    return dict(value=flops / t / 1e12, unit=UNIT, cores=cores, kind="oracle",
                sample=f"KV head 0 ({G} query heads) of the first {plan['n_samples']} samples of {w.name} "
                       f"(seed {w.seed}){rows_note}: {plan['T']} tree tokens, {plan['flat_tokens']} unshared tokens, "
                       f"{flops:.3e} dedup FLOP, {t:.2f} s per pass (numpy fp64, torch threads "
                       f"{torch.get_num_threads()})"), t


def run_reference(args):
    from paper_2608_25683_b200.workloads import make_workload

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args.config, args.seed)
    # every step is a bounded sample; the whole run (warm-up + steps) stays near 4e12 FLOP of oracle work
    base, t = oracle_leg(w, args.ref_samples, args.seed + 1, steps=args.steps, warmup=args.warmup,
                         budget=min(1.5e12, 4e12 / max(1, args.steps + args.warmup)))
    line = dict(metric=METRIC, value=base["value"], unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=t * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=workload_config(w, None), cpu_baseline=base,
                e2e=dict(value=base["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line), flush=True)


def workload_config(w, view):
    c = {"workload": f"{w.name}: " + {
        "c1": "tiny fp32 tree, 64-token prefix + 4 branches of 32",
        "c2": "step-wise RL group, 8 samples sharing a 4096-token prefix, suffixes U{256..1024}",
        "c2s": "cached 4096-token prefix + 8 suffixes U{1..8} (HBM-bound case)",
        "c3": "depth-3 branching-4 tree, 64 leaves",
        "c4": "mixed batch of 32 prefix groups, per-group block size {16,64,256}, fragmented pool",
        "c5": "long-context group, 32768-token prefix + 64 branches U{1024..4096}",
    }.get(w.name, w.name),
        "seed": w.seed, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
        "block_sizes": sorted(set(w.group_block_size)),
        "l2": "per-step working set exceeds the 126 MB L2 (inputs larger than L2); no explicit flush"}
    if view is not None:
        c.update(tree_tokens=view["T"], unshared_tokens=view["flat_tokens"], tree_pairs=view["tree_pairs"],
                 unshared_pairs=view["flat_pairs"], n_segments=view["n_seg"], n_samples=view["n_samples"],
                 prefix_match_rate=round(1 - view["T"] / view["flat_tokens"], 4))
    return c


# --------------------------------------------------------------------------- GPU arm
class Runner:
    """Holds one workload's plan, device tensors and preallocated outputs."""

    def __init__(self, lib, w, seed, device, view_from=None, data=None):
        import torch

        self.lib, self.w = lib, w
        self.plan = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                             w.seg_flags, w.free_extents).upload(device)
        V = self.plan.view
        if data is None:
            from paper_2608_25683_b200.workloads import make_inputs
            cap = V["pool_slots"]
            if w.free_extents:
                cap = max(cap, max(a + c for a, c in w.free_extents))
            data = make_inputs(V["T_q"], cap, V["tok_slot"], w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, seed,
                               device=device)
        self.q, self.k, self.v, self.d_o = data
        self.o = torch.empty_like(self.q)
        self.lse = torch.empty((w.n_q_heads, V["T_q"]), dtype=torch.float32, device=device)
        self.dq = torch.empty_like(self.q)
        self.dk = torch.zeros_like(self.k)
        self.dv = torch.zeros_like(self.v)
        self.scale = w.softmax_scale

    def fwd(self):
        self.lib.psrl_tree_attn_fwd(self.plan, self.q, self.k, self.v, self.scale, o=self.o, lse=self.lse)

    def bwd(self):
        self.lib.psrl_tree_attn_bwd(self.plan, self.q, self.k, self.v, self.o, self.lse, self.d_o, self.scale,
                                    d_q=self.dq, dk_pool=self.dk, dv_pool=self.dv)

    def step(self):
        self.fwd()
        self.bwd()


L2_BYTES = 126 << 20
_flush_buf = None


def flush_l2(device):
    """Overwrites a buffer of twice the L2 size, so that the next kernel finds its inputs in HBM."""
    import torch

    global _flush_buf
    if _flush_buf is None:
        _flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)
    _flush_buf.add_(1)


def time_region(fn, iters, warmup=0, flush_device=None):
    """Mean time of fn over `iters` calls, CUDA events on the current stream.  With flush_device
    every call is timed on its own and the L2 is flushed before it (outside the timed part)."""
    import torch

    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if flush_device is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in ev:
        flush_l2(flush_device)
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in ev) / iters


def flat_runner(lib, r, device, head_slice=None):
    """The same kernels on the unshared layout: every sample a root of its own
    holding copies of its tokens; dO goes to the first copy of each token."""
    import torch
    from paper_2608_25683_b200.workloads import Workload, flatten_forest

    V = r.plan.view
    w = r.w
    parent, seg_len, gbs, tok_src, first = flatten_forest(V)
    Hq, Hkv = w.n_q_heads, w.n_kv_heads
    G = Hq // Hkv
    hs = slice(None) if head_slice is None else slice(head_slice * G, (head_slice + 1) * G)
    ks = slice(None) if head_slice is None else slice(head_slice, head_slice + 1)
    fw = Workload(w.name + "-flat", parent, seg_len, gbs, Hq if head_slice is None else G,
                  Hkv if head_slice is None else 1, w.head_dim, w.dtype)
    fplan = lib.Plan(fw.parent, fw.seg_len, fw.group_block_size, fw.n_q_heads, fw.n_kv_heads, fw.head_dim, fw.dtype)
    FV = fplan.view
    # token -> query row of the tree layout
    qrow = np.full(V["T"], -1, dtype=np.int64)
    for c in range(V["n_seg"]):
        if V["seg_q_off"][c] >= 0:
            qrow[V["seg_tok_off"][c]:V["seg_tok_off"][c] + V["seg_len"][c]] = np.arange(
                V["seg_q_off"][c], V["seg_q_off"][c] + V["seg_len"][c])
    assert (qrow[tok_src] >= 0).all(), "the unshared comparison needs queries on every segment"
    src_rows = torch.as_tensor(qrow[tok_src], device=device)
    src_slots = torch.as_tensor(V["tok_slot"][tok_src].astype(np.int64), device=device)
    dst_slots = torch.as_tensor(FV["tok_slot"].astype(np.int64), device=device)
    q = r.q[src_rows][:, hs].contiguous()
    d_o = r.d_o[src_rows][:, hs].contiguous()
    d_o[torch.as_tensor(~first, device=device)] = 0
    k = torch.zeros((fw.n_kv_heads, FV["pool_slots"], w.head_dim), dtype=r.k.dtype, device=device)
    v = torch.zeros_like(k)
    k[:, dst_slots] = r.k[ks][:, src_slots]
    v[:, dst_slots] = r.v[ks][:, src_slots]
    return Runner(lib, fw, 0, device, data=(q, k, v, d_o))


def library_context_leg(lib, w, V, device, ms_tree, flops, iters):
    """Context, not a target and not the oracle: a library's varlen causal attention (flash_attn's
    kernels as shipped in the image) forward + backward on the flattened, unshared layout: every
    sample a sequence of its own.  Timing does not depend on the values, so inputs are random."""
    import torch
    try:
        import flash_attn
        from flash_attn import flash_attn_varlen_func
    except Exception as ex:
        return {"unavailable": str(ex)[:120]}
    from paper_2608_25683_b200.workloads import flatten_forest
    _, lens, _, _, _ = flatten_forest(V)
    lens = [int(x) for x in lens]
    Hq, Hkv, d = w.n_q_heads, w.n_kv_heads, w.head_dim
    T = sum(lens)
    # Slices of heads keep every tensor below 2^31 elements: on c4's unshared layout (4.3e9 elements per
    # Q-shaped tensor) the library raised an illegal memory access, so it is never handed such a tensor.
    hq, hkv = Hq, Hkv
    if T * hq * d >= 2 ** 31 or T * Hq * d * 2 * 4 >= 60e9:
        hq, hkv = Hq // Hkv, 1
    while T * hq * d >= 2 ** 31 and hq > 1:
        hq //= 2
    if T * hq * d >= 2 ** 31:
        return {"skipped": "a single head of the unshared layout exceeds 2^31 elements"}
    slices = Hq // hq
    try:
        cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=device)
        q = torch.randn(T, hq, d, device=device, dtype=torch.bfloat16, requires_grad=True)
        k = torch.randn(T, hkv, d, device=device, dtype=torch.bfloat16, requires_grad=True)
        v = torch.randn(T, hkv, d, device=device, dtype=torch.bfloat16, requires_grad=True)
        d_o = torch.randn(T, hq, d, device=device, dtype=torch.bfloat16)

        def step():
            o = flash_attn_varlen_func(q, k, v, cu, cu, max(lens), max(lens), softmax_scale=w.softmax_scale, causal=True)
            o.backward(d_o)
            q.grad = k.grad = v.grad = None

        ms = time_region(step, iters, 2) * slices
    except Exception as ex:
        return {"library": "flash_attn " + flash_attn.__version__, "error": str(ex)[:200]}
    flat_flops = dedup_flops(d, Hq, V["flat_pairs"])
    return {"library": "flash_attn " + flash_attn.__version__ + " flash_attn_varlen_func, causal, fwd + autograd bwd",
            "layout": "flattened unshared: %d sequences, %d tokens" % (len(lens), T), "kv_head_slices": slices,
            "ms_per_step": round(ms, 3), "tflops_on_unshared_flops": round(flat_flops / (ms * 1e-3) / 1e12, 1),
            "dedup_tflops_equivalent": round(flops / (ms * 1e-3) / 1e12, 1),
            "tree_path_speedup_over_library": round(ms / ms_tree, 2)}


def forest_of_groups(w, groups):
    """The sub-forest of `w` made of the prefix groups `groups` (root indices counted in input order)."""
    from paper_2608_25683_b200.workloads import Workload

    root_rank, group_of = -1, []
    for s, p in enumerate(w.parent):
        if p == -1:
            root_rank += 1
            group_of.append(root_rank)
        else:
            group_of.append(group_of[p])
    keep = [s for s in range(len(w.parent)) if group_of[s] in set(groups)]
    new = {s: i for i, s in enumerate(keep)}
    parent = [-1 if w.parent[s] == -1 else new[w.parent[s]] for s in keep]
    gbs = [w.group_block_size[group_of[s]] for s in keep if w.parent[s] == -1]
    return Workload(w.name + "-part", parent, [w.seg_len[s] for s in keep], gbs, w.n_q_heads, w.n_kv_heads, w.head_dim,
                    w.dtype, seed=w.seed)


def schedule_leg(lib, device, seed):
    """Eq. 1 in practice (Sec. 4.2).  (1) The coefficients are fitted by least squares to measured forward +
    backward times of single prefix groups of varied shape.  (2) The 32 groups of c4 are placed on k workers
    by descending workload (psrl_place_groups) and, for comparison, round-robin in input order; every worker's
    share is then run on this GPU and timed: the imbalance is max / mean of the workers' measured times."""
    from paper_2608_25683_b200.workloads import Workload, make_workload

    Hq, Hkv, d = 32, 8, 128
    rng = np.random.default_rng(seed)

    def measure(w):
        r = Runner(lib, w, seed, device)
        t = time_region(r.step, 5, 2)
        del r
        return t

    # ---- (1) fit: T(group) = a1 * sum(l_suf * l) + a2 * sum(l_suf) + a3 * n_samples ----
    rows, times = [], []
    for prefix, n_br, br in ((512, 2, 256), (2048, 4, 512), (4096, 8, 512), (8192, 4, 1024), (1024, 16, 128),
                             (16384, 2, 2048), (256, 8, 1024), (4096, 1, 4096), (12288, 8, 256)):
        parent = [-1] + [0] * n_br
        seg_len = [prefix] + [int(br * (0.75 + 0.5 * rng.random())) for _ in range(n_br)]
        w = Workload("fit", parent, seg_len, [64], Hq, Hkv, d, "bf16", seed=seed)
        a = [lib.psrl_group_workloads(parent, seg_len, e)[0] for e in ((1, 0, 0), (0, 1, 0), (0, 0, 1))]
        rows.append(a)
        times.append(measure(w))
    A, t = np.asarray(rows), np.asarray(times)
    alpha, *_ = np.linalg.lstsq(A, t, rcond=None)
    alpha = np.maximum(alpha, 0.0)
    fit_err = float(np.max(np.abs(A @ alpha - t) / t))

    # ---- (2) placement of c4's groups ----
    w = make_workload("c4", 2000)
    w.free_extents = None
    workload = lib.psrl_group_workloads(w.parent, w.seg_len, alpha)
    n_groups = len(workload)
    out = {"alpha_ms": [float(a) for a in alpha], "fit_max_rel_err": round(fit_err, 4), "n_groups": n_groups, "workers": {}}
    for k in (2, 4, 8):
        lpt, load = lib.psrl_place_groups(workload, k)
        rr = np.arange(n_groups) % k
        res = {}
        for name, assign in (("load_balanced", lpt), ("round_robin", rr)):
            ms = []
            for worker in range(k):
                groups = [g for g in range(n_groups) if assign[g] == worker]
                ms.append(measure(forest_of_groups(w, groups)) if groups else 0.0)
            pred = [float(sum(workload[g] for g in range(n_groups) if assign[g] == worker)) for worker in range(k)]
            res[name] = {"measured_ms": [round(x, 2) for x in ms], "predicted_ms": [round(x, 2) for x in pred],
                         "imbalance_max_over_mean": round(max(ms) / (sum(ms) / k), 4)}
        out["workers"][str(k)] = res
    return out


def microbatch_leg(lib, w, device, flops, seed, iters):
    """The same forest run as an ordered list of micro-batches (Sec. 4.1): every root is computed with its
    first child, every further child of a root in a micro-batch of its own (deeper levels follow their
    parent's micro-batch or later, breadth first).  Cached prefixes are read in place; the Dynamic Block
    Caching manager (Sec. 5.2) assigns extents and releases blocks after their last use.  Timed: all
    forward + backward calls of the micro-batches; plans are built and uploaded beforehand."""
    import torch

    n = len(w.parent)
    children = [[] for _ in range(n)]
    for s, p in enumerate(w.parent):
        if p >= 0:
            children[p].append(s)
    mb = [0] * n
    for s in range(n):                      # parents come before children
        for i, c in enumerate(children[s]):
            mb[c] = mb[s] + i
    M = max(mb) + 1
    cache = lib.Cache(w.parent, w.seg_len, w.group_block_size, mb, M, seg_flags=w.seg_flags)
    arena = cache.stats()["total_slots"]
    Hq, Hkv, d = w.n_q_heads, w.n_kv_heads, w.head_dim
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    g = torch.Generator(device=device).manual_seed(seed)
    K = torch.randn(Hkv, arena, d, generator=g, device=device, dtype=torch.float32).to(dt)
    V = torch.randn(Hkv, arena, d, generator=g, device=device, dtype=torch.float32).to(dt)
    dK, dV = torch.zeros_like(K), torch.zeros_like(V)
    steps, trace, t_plan = [], [], 0.0
    for m in range(M):
        st = cache.begin(m)
        t0 = time.perf_counter()
        plan = lib.Plan(st["parent"], st["seg_len"], st["group_block_size"], Hq, Hkv, d, w.dtype,
                        seg_flags=st["seg_flags"], seg_slot_base=st["seg_slot_base"]).upload(device)
        t_plan += time.perf_counter() - t0
        T_q = plan.view["T_q"]
        q = torch.randn(T_q, Hq, d, generator=g, device=device, dtype=torch.float32).to(dt)
        d_o = torch.randn(T_q, Hq, d, generator=g, device=device, dtype=torch.float32).to(dt)
        o, dq = torch.empty_like(q), torch.empty_like(q)
        lse = torch.empty((Hq, T_q), dtype=torch.float32, device=device)
        steps.append((plan, q, d_o, o, lse, dq))
        after = cache.end(m)["live_slots"]
        trace.append([st["live_slots"], after])

    def run():
        for plan, q, d_o, o, lse, dq in steps:
            lib.psrl_tree_attn_fwd(plan, q, K, V, w.softmax_scale, o=o, lse=lse)
            lib.psrl_tree_attn_bwd(plan, q, K, V, o, lse, d_o, w.softmax_scale, d_q=dq, dk_pool=dK, dv_pool=dV)

    ms = time_region(run, iters, 2)
    for plan, *_ in steps:
        assert lib.psrl_device_status(plan, "bwd") == 0
    st = cache.stats()
    return {"n_microbatches": M, "ms_all_microbatches": round(ms, 4), "dedup_tflops": round(flops / (ms * 1e-3) / 1e12, 2),
            "plan_build_upload_ms": round(t_plan * 1e3, 2), "peak_kv_slots": st["peak_slots"],
            "kv_slots_without_caching_policy": st["total_slots"],
            "peak_reduction": round(1 - st["peak_slots"] / st["total_slots"], 4),
            "live_slots_during_after": trace if M <= 64 else trace[:64]}


def measure_config(args, lib, name, device, rank, world, local, headline):
    """All measurements of one configuration.  Returns None on ranks other than 0 once the timed
    region (which every rank takes part in) is over."""
    import torch
    import torch.distributed as dist

    from paper_2608_25683_b200 import dist_util
    from paper_2608_25683_b200.workloads import make_workload

    # every rank gets an independent batch of the same shape (groups never span workers)
    w = make_workload(name, dist_util.rank_seed(args.seed, rank), scale_len=args.length_scale)
    if args.block_size is not None:
        bs = 0 if args.block_size == "adaptive" else int(args.block_size)
        w.group_block_size = [bs] * len(w.group_block_size)
        w.free_extents = None
    t0 = time.perf_counter()
    _p = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                  w.seg_flags, w.free_extents)
    t1 = time.perf_counter()
    _p.upload(device)
    torch.cuda.synchronize()
    plan_ms = {"build_ms": round((t1 - t0) * 1e3, 3), "upload_ms": round((time.perf_counter() - t1) * 1e3, 3),
               "device_bytes": _p.device_bytes()}
    del _p
    r = Runner(lib, w, dist_util.rank_seed(args.seed, rank) + 1, device)
    V = r.plan.view
    flops = dedup_flops(w.head_dim, w.n_q_heads, V["tree_pairs"])
    # algorithmic bytes of one step (each tensor once per pass)
    es = 2 if w.dtype == "bf16" else 4
    qb = V["T_q"] * w.n_q_heads * w.head_dim * es            # one Q-shaped tensor
    kb = V["T"] * w.n_kv_heads * w.head_dim * es              # one K-shaped tensor (tokens, not slots)
    lb = 4 * V["T_q"] * w.n_q_heads                           # LSE or D
    kbytes = {"fwd_kernel": 2 * qb + 2 * kb + lb, "dq_kernel": 3 * qb + 2 * kb + 2 * lb,
              "dkv_kernel": 2 * qb + 4 * kb + 2 * lb, "delta_kernel": 2 * qb + lb}
    step_bytes = 5 * qb + 6 * kb + 2 * lb
    # a working set that fits in the L2 would be served from it after the first step: flush between steps
    flush = device if step_bytes < 2 * L2_BYTES else None
    steps = args.steps

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        # the sampler also sees the warm-up so that short timed regions still get samples under load
        t_w = time.perf_counter()
        n_w = 0
        while n_w < max(args.warmup, 3) or time.perf_counter() - t_w < 0.5:
            r.step()
            n_w += 1
            if n_w % 8 == 0:
                torch.cuda.synchronize()
        assert lib.psrl_device_status(r.plan, "bwd") == 0
        barrier()
        if flush is None:
            e0.record()
            for _ in range(steps):
                r.step()
            e1.record()
            barrier()
            ms = e0.elapsed_time(e1) / steps
        else:
            ms = time_region(r.step, steps, 0, flush)
            barrier()
    ms_max, flops_all = dist_util.aggregate(ms, flops, device)  # max over ranks, sum of work
    value = flops_all / (ms_max * 1e-3) / 1e12
    if rank != 0:
        return None

    # ---- per-kernel times INSIDE running steps, right behind the headline region (the same warmed, power-
    # capped state): a step is issued as forward | D pre-pass | dQ | dK/dV with a CUDA event between the parts,
    # so the parts add up to the step; the SM clock is sampled over exactly these steps ----
    phases = (("fwd_kernel", None), ("delta_kernel", 1), ("dq_kernel", 2), ("dkv_kernel", 4))
    n_ph = max(3, min(400, int(np.ceil(600.0 / ms))))       # >= 0.6 s of steps, so that the sampler sees them
    with ClockSampler(local) as kclocks:
        t_w = time.perf_counter()
        while time.perf_counter() - t_w < 0.4:              # back into the headline's state after the sampler restart
            r.step()
            torch.cuda.synchronize()
        marks = []
        for _ in range(n_ph):
            if flush is not None:
                flush_l2(flush)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
            ev[0].record()
            r.fwd()
            ev[1].record()
            for i, (_, mask) in enumerate(phases[1:]):
                lib.psrl_bench_bwd_phases(r.plan, r.q, r.k, r.v, r.o, r.lse, r.d_o, r.scale, r.dq, r.dk, r.dv, mask)
                ev[2 + i].record()
            marks.append(ev)
        torch.cuda.synchronize()
    kern = {nm: float(np.mean([m[i].elapsed_time(m[i + 1]) for m in marks])) for i, (nm, _) in enumerate(phases)}
    kclk = kclocks.summary()

    # ---- host time of a step's calls (argument checks, tensor-map lookups, launches), GPU idle at the start ----
    torch.cuda.synchronize()
    n_h = 10 if ms < 50 else 2
    th = time.perf_counter()
    for _ in range(n_h):
        r.step()
    host_ms = (time.perf_counter() - th) / n_h * 1e3
    torch.cuda.synchronize()

    # ---- launch-bound steps: the same step replayed from a CUDA graph (one submission instead of 6-7 launches) ----
    graph = None
    if ms < 1.0:
        try:
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream(device=device)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                r.step()                               # warm: attributes set, tensor maps encoded
                side.synchronize()
                with torch.cuda.graph(g, stream=side):
                    r.step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g_ms = time_region(g.replay, max(10, steps), 3, flush)
            graph = {"ms_per_step": round(g_ms, 4), "value": round(flops / (g_ms * 1e-3) / 1e12, 3),
                     "note": "forward + backward captured once into a CUDA graph and replayed (same kernels)"}
            del g
        except Exception as ex:
            graph = {"error": str(ex)[:200]}
            torch.cuda.synchronize()

    # ---- every step on its own (median, min) and bitwise reproducibility over three runs ----
    n_each = max(3, min(steps, 20)) if ms < 100 else 3
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_each + 1)]
    if flush is None:
        evs[0].record()
        for i in range(n_each):
            r.step()
            evs[i + 1].record()
        torch.cuda.synchronize()
        each = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_each)]
    else:
        each = [time_region(r.step, 1, 0, flush) for _ in range(n_each)]
    step_stats = {"n": n_each, "median_ms": round(float(np.median(each)), 4), "min_ms": round(min(each), 4),
                  "max_ms": round(max(each), 4)}
    outs = (r.o, r.lse, r.dq, r.dk, r.dv)
    first = [x.clone() for x in outs]
    same = True
    for _ in range(2):
        r.step()
        same = same and all(torch.equal(a.view(torch.int16 if a.element_size() == 2 else torch.int32),
                                        b.view(torch.int16 if b.element_size() == 2 else torch.int32))
                            for a, b in zip(first, outs))
    del first
    torch.cuda.empty_cache()

    pk = peaks()
    d, Hq, pairs = w.head_dim, w.n_q_heads, float(V["tree_pairs"])
    # contractions each kernel has to execute for its outputs (2*d flops per pair, head and contraction):
    # forward S, PV; dQ kernel S, dP, dQ; dK/dV kernel S^T, dP^T, dV, dK.  The step metric counts 14*d (S and dP once).
    kflops = {"fwd_kernel": 4 * d * Hq * pairs, "dq_kernel": 6 * d * Hq * pairs, "dkv_kernel": 8 * d * Hq * pairs}
    kernels = {}
    for nm, tms in kern.items():
        kernels[nm] = {"ms": round(tms, 4), "sm_mhz": kclk["sm_mhz"]}
        if nm in kflops:
            kernels[nm]["algorithmic_tflops"] = round(kflops[nm] / (tms * 1e-3) / 1e12, 2)
        kernels[nm]["algorithmic_gbs"] = round(kbytes[nm] / (tms * 1e-3) / 1e9, 1)
    sum_ms = sum(kern.values())
    dom = max(("fwd_kernel", "dq_kernel", "dkv_kernel"), key=lambda n: kern[n])
    ridge = pk["bf16_tflops"] * 1e12 / (pk["hbm_gbs"] * 1e9)
    hbm_bound = w.dtype == "bf16" and flops / step_bytes < ridge
    timing_note = ("each kernel timed inside running steps (events between the step's parts), mean of %d steps, "
                   "SM clock sampled over those steps; in a whole step of a small plan dQ and dK/dV run side by "
                   "side on two streams, so there the parts add up to more than the step" % n_ph)
    if hbm_bound:
        achieved = kbytes[dom] / (kern[dom] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dom, "achieved": round(achieved, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": round(achieved / pk["hbm_gbs"], 4), "traffic": NCU_TRAFFIC_BYTES.get(name),
                    "peak_source": f"{pk['source']} copy bandwidth", "kernels": kernels,
                    "step_algorithmic_bytes": step_bytes, "step_flop_per_byte": round(flops / step_bytes, 1),
                    "whole_step_gbs": round(step_bytes / (ms * 1e-3) / 1e9, 1),
                    "whole_step_frac": round(step_bytes / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], 4)}
    else:
        achieved = kflops[dom] / (kern[dom] * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": dom, "achieved": round(achieved, 2), "peak": pk["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": round(achieved / pk["bf16_tflops"], 4),
                    "traffic": NCU_TRAFFIC_BYTES.get(name),
                    "peak_source": f"{pk['source']} cuBLAS bf16 burst (the sustained figure, "
                                   f"{pk['bf16_tflops_sustained']}, was taken at a lower SM clock than this run's)",
                    "frac_of_sustained": round(achieved / pk["bf16_tflops_sustained"], 4), "kernels": kernels,
                    "whole_step_frac_of_burst": round(value / world / pk["bf16_tflops"], 4),
                    "whole_step_frac_of_sustained": round(value / world / pk["bf16_tflops_sustained"], 4)}
    roofline.update(kernel_timing=timing_note, kernel_clocks=kclk, sum_kernel_ms=round(sum_ms, 4),
                    sum_kernel_ms_over_step_ms=round(sum_ms / ms, 4))
    if w.dtype != "bf16":
        # fp32 SIMT path: plain FMA arithmetic.  Peak from the unit counts and the clock: 148 SMs x 128 fp32 lanes
        # x 2 flop x 1.965 GHz = 74.4 TFLOP/s (the path keeps its long sums in fp64, which runs far below that:
        # the figure is a ceiling, and the configuration it serves is launch-bound)
        alu_peak = 148 * 128 * 2 * 1.965e9 / 1e12
        roofline.update(bound="alu", peak=round(alu_peak, 1), frac=round(achieved / alu_peak, 6),
                        peak_source="derived: 148 SMs x 128 fp32 lanes x 2 flop x 1.965 GHz")
        roofline.pop("frac_of_sustained", None)

    # ---- end to end through the public call with host buffers ----
    hq, hk, hv, hdo = (x.cpu().pin_memory() for x in (r.q, r.k, r.v, r.d_o))
    ho, hl, hdq, hdk, hdv = (torch.empty_like(x, device="cpu").pin_memory() for x in (r.o, r.lse, r.dq, r.dk, r.dv))

    def e2e_step():
        r.q.copy_(hq, non_blocking=True); r.k.copy_(hk, non_blocking=True)
        r.v.copy_(hv, non_blocking=True); r.d_o.copy_(hdo, non_blocking=True)
        r.step()
        ho.copy_(r.o, non_blocking=True); hl.copy_(r.lse, non_blocking=True); hdq.copy_(r.dq, non_blocking=True)
        hdk.copy_(r.dk, non_blocking=True); hdv.copy_(r.dv, non_blocking=True)

    n_e2e = max(4, min(steps, 10)) if ms < 100 else 3
    e2e_serial_ms = time_region(e2e_step, n_e2e, 2 if ms < 100 else 1)

    # The same, software-pipelined the way a training loop feeds a device: three streams and two sets of device
    # buffers, so that step i+1's host->device copies and step i-1's device->host copies run beside step i.
    # Every step still copies all its inputs in and all its outputs out inside the timed region.
    r2 = Runner(lib, w, 0, device, data=tuple(x.clone() for x in (r.q, r.k, r.v, r.d_o)))
    pair = (r, r2)
    s_in, s_c, s_out = (torch.cuda.Stream(device=device) for _ in range(3))

    def e2e_pipelined(n):
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_c = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        cur = torch.cuda.current_stream()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(cur)
        for st in (s_in, s_c, s_out):
            st.wait_event(t0)
        for i in range(n):
            b = i & 1
            x = pair[b]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_c[b])        # the inputs of set b are free once step i-2 has run
                x.q.copy_(hq, non_blocking=True); x.k.copy_(hk, non_blocking=True)
                x.v.copy_(hv, non_blocking=True); x.d_o.copy_(hdo, non_blocking=True)
                ev_in[b].record(s_in)
            with torch.cuda.stream(s_c):
                s_c.wait_event(ev_in[b])
                if i >= 2:
                    s_c.wait_event(ev_out[b])       # the outputs of set b have been read back
                x.step()
                ev_c[b].record(s_c)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_c[b])
                ho.copy_(x.o, non_blocking=True); hl.copy_(x.lse, non_blocking=True); hdq.copy_(x.dq, non_blocking=True)
                hdk.copy_(x.dk, non_blocking=True); hdv.copy_(x.dv, non_blocking=True)
                ev_out[b].record(s_out)
        for st in (s_in, s_c, s_out):
            cur.wait_stream(st)
        t1.record(cur)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / n

    e2e_pipelined(2)
    e2e_ms = e2e_pipelined(n_e2e)
    del r2, pair
    nbytes = lambda *ts: int(sum(x.numel() * x.element_size() for x in ts))
    e2e = {"value": round(flops / (e2e_ms * 1e-3) / 1e12 * world, 3), "unit": UNIT, "ms_per_step": round(e2e_ms, 3),
           "h2d_bytes_per_step": nbytes(hq, hk, hv, hdo), "d2h_bytes_per_step": nbytes(ho, hl, hdq, hdk, hdv),
           "mode": "three streams, two sets of device buffers: copies of neighbouring steps overlap the kernels",
           "serial": {"value": round(flops / (e2e_serial_ms * 1e-3) / 1e12 * world, 3),
                      "ms_per_step": round(e2e_serial_ms, 3), "mode": "copy in, run, copy out on one stream"}}
    del hq, hk, hv, hdo, ho, hl, hdq, hdk, hdv
    torch.cuda.empty_cache()

    # ---- the same kernels on the unshared (flattened) layout ----
    print(f"[bench] {name}: tree path measured; unshared leg", file=sys.stderr, flush=True)
    unshared = None
    if not args.no_unshared and world == 1 and all((f & 1) for f in V["seg_flags"]):
        try:
            bytes_flat = V["flat_tokens"] * Hq * d * es * 4
            slices = 1 if bytes_flat < 60e9 else w.n_kv_heads
            t_flat = 0.0
            n_fl = max(3, min(steps, 10)) if ms < 100 else 2
            for sl in range(slices):
                fr = flat_runner(lib, r, device, head_slice=None if slices == 1 else sl)
                t_flat += time_region(fr.step, n_fl, 2 if ms < 100 else 1)
                del fr
                torch.cuda.empty_cache()
            unshared = {"ms_per_step": round(t_flat, 3), "speedup_vs_unshared": round(t_flat / ms, 3),
                        "flop_ratio_unshared_over_tree": round(V["flat_pairs"] / V["tree_pairs"], 3),
                        "kv_head_slices": slices}
        except Exception as ex:  # e.g. out of memory on the flattened tensors
            unshared = {"error": str(ex)[:200]}

    res = dict(value=round(value, 3), ms_per_step=round(ms_max, 4), unit=UNIT,
               dtype=("bf16" if w.dtype == "bf16" else "f32"),
               config=dict(workload_config(w, V), length_scale=args.length_scale, pool_slots=V["pool_slots"], l2=(
                   "per-step working set exceeds the 126 MB L2 (inputs larger than L2); no explicit flush" if flush is None
                   else "working set fits in the L2: a 252 MB buffer is overwritten before every timed step "
                        "(each step timed on its own, flush outside the timed part)")),
               clocks=clocks.summary(), e2e=e2e,
               gpu_launches=(lib.psrl_launch_count(r.plan, False) + lib.psrl_launch_count(r.plan, True)) * steps,
               roofline=roofline, step_ms=step_stats, bitwise_reproducible_3_runs=bool(same),
               plan=dict(plan_ms, host_ms_per_step_of_calls=round(host_ms, 4)), unshared=unshared, cuda_graph=graph,
               frac_of_bf16_peak={"burst": round(value / world / pk["bf16_tflops"], 4),
                                  "sustained": round(value / world / pk["bf16_tflops_sustained"], 4)})

    if headline:
        extra = {}
        if args.context and world == 1:
            torch.cuda.synchronize()
            print("[bench] library context leg", file=sys.stderr, flush=True)
            extra["library_context"] = library_context_leg(lib, w, V, device, ms, flops, max(3, min(steps, 10)))
            torch.cuda.synchronize()
            torch.cuda.empty_cache()
        if args.pack and world == 1:
            T = V["T"]
            k_tok = torch.randn(T, w.n_kv_heads, w.head_dim, device=device).to(r.k.dtype)
            v_tok = torch.randn(T, w.n_kv_heads, w.head_dim, device=device).to(r.k.dtype)
            nbytes_pack = 2 * 2 * k_tok.numel() * k_tok.element_size()      # K and V, read + write
            fl = device if nbytes_pack < 2 * L2_BYTES else None
            t_sc = time_region(lambda: lib.psrl_kv_scatter(r.plan, k_tok, v_tok, r.k, r.v), 10, 2, fl)
            t_ga = time_region(lambda: lib.psrl_kv_gather(r.plan, r.k, r.v, k_tok, v_tok), 10, 2, fl)
            extra["kv_pack"] = {
                "bytes_per_call": nbytes_pack, "scatter_ms": round(t_sc, 4), "gather_ms": round(t_ga, 4),
                "scatter_gbs": round(nbytes_pack / (t_sc * 1e-3) / 1e9, 1), "gather_gbs": round(nbytes_pack / (t_ga * 1e-3) / 1e9, 1),
                "hbm_peak_gbs": pk["hbm_gbs"], "scatter_frac": round(nbytes_pack / (t_sc * 1e-3) / 1e9 / pk["hbm_gbs"], 4),
                "gather_frac": round(nbytes_pack / (t_ga * 1e-3) / 1e9 / pk["hbm_gbs"], 4)}
        if args.schedule and world == 1:
            extra["schedule"] = schedule_leg(lib, device, args.seed + 11)
        if args.microbatch and world == 1:
            extra["microbatch"] = microbatch_leg(lib, w, device, flops, args.seed + 7, max(3, min(steps, 10)))
        res["extra"] = extra
        res["workload_obj"] = w
    del r
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=None,
                    help="one configuration (c1..c5, c2s).  Default: c5 is the headline (the largest single-GPU "
                         "configuration) and c1 (fp32), c2, c3, c4 and the small-suffix c2s are measured too, under per_config")
    ap.add_argument("--seed", type=int, default=2000)
    ap.add_argument("--cpu-samples", type=int, default=4, help="samples in the oracle's timed sample")
    ap.add_argument("--ref-samples", type=int, default=2, help="samples per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-unshared", action="store_true")
    ap.add_argument("--context", action="store_true",
                    help="also time a library's varlen attention (flash_attn) on the unshared layout, for context")
    ap.add_argument("--block-size", default=None,
                    help="override the page size of every group: 16|32|64|128|256, or 'adaptive' (one extent per span)")
    ap.add_argument("--length-scale", type=float, default=1.0,
                    help="scale every segment length (tree shape and prefix match rate unchanged, cf. Sec. 7.5)")
    ap.add_argument("--pack", action="store_true", help="also time K/V scatter into the pools and the gather back")
    ap.add_argument("--schedule", action="store_true",
                    help="also fit Eq. 1 to measured times and compare load-balanced with round-robin group placement")
    ap.add_argument("--microbatch", action="store_true",
                    help="also run the group as one micro-batch per branch with the Dynamic Block Caching manager")
    args = ap.parse_args()
    head_name = args.config or "c5"
    others = [] if args.config else ["c1", "c2", "c3", "c4", "c2s"]
    if args.impl == "reference":
        args.config = head_name
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    from paper_2608_25683_b200 import binding as lib, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))
    build.build()

    # the other configurations first (short), the headline last; with several ranks only the headline runs
    per_config = {}
    if world == 1:
        for name in others:
            print(f"[bench] {name}", file=sys.stderr, flush=True)
            try:
                res = measure_config(args, lib, name, device, rank, world, local, headline=False)
                res.pop("unit", None)
                per_config[name] = res
            except Exception as ex:   # one configuration must not take the headline down with it
                per_config[name] = {"error": str(ex)[:300]}
                torch.cuda.empty_cache()
    print(f"[bench] {head_name} (headline)", file=sys.stderr, flush=True)
    res = measure_config(args, lib, head_name, device, rank, world, local, headline=True)
    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    w = res.pop("workload_obj")
    extra = res.pop("extra")
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        cpu, _ = oracle_leg(w, args.cpu_samples, args.seed + 1)

    line = dict(metric=METRIC, value=res["value"], unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=res["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype=res["dtype"], data="synthetic", config=res["config"], clocks=res["clocks"], e2e=res["e2e"],
                gpu_launches=res["gpu_launches"], roofline=res["roofline"], cpu_baseline=cpu, step_ms=res["step_ms"],
                bitwise_reproducible_3_runs=res["bitwise_reproducible_3_runs"], plan=res["plan"],
                unshared=res["unshared"], cuda_graph=res.get("cuda_graph"), frac_of_bf16_peak=res["frac_of_bf16_peak"],
                per_config=per_config or None, library_context=extra.get("library_context"),
                microbatch=extra.get("microbatch"), schedule=extra.get("schedule"), kv_pack=extra.get("kv_pack"))
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
