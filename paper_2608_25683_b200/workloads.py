"""Seeded synthetic workloads: prefix forests and attention inputs.

This module only draws shapes and random values.  It holds none of the
method's arithmetic and imports neither the CUDA binding nor the oracle, so
both sides of a parity test can be fed from it.

The forests take the shapes of the paper's agentic workloads (Tab. 2: prompts
of 4K-40K tokens, generations of 512-20K tokens, 4-8 rollouts per prompt;
Tab. 1: step-mode prefix match rates of 72-95 %); the paper's production
traces themselves are not used.

Configurations
  c1   one 64-token prefix + 4 branches of 32; MHA 2/2 heads, d=64, fp32, bs=16
  c2   one 4096-token prefix + 8 branches U{256..1024}; GQA 32/8, d=128, bf16, bs=64
  c3   depth-3 tree, branching 4 (1 + 4 + 16 internal, 64 leaves); root 512,
       internal 256, leaves U{128..512}; GQA 28/4, d=128, bf16, bs=64;
       listed level by level so the canonical reordering is exercised
  c4   32 independent groups; prefix lognormal(median 2048, sigma 1) clipped to
       [256, 16384]; group size geometric(mean 8) clipped to [1, 32]; suffixes
       U{64..2048}; per-group bs from {16, 64, 256}; fragmented free list;
       GQA 32/8, d=128, bf16
  c5   one 32768-token prefix + 64 branches U{1024..4096}; GQA 64/8, d=128,
       bf16, bs=256
  c2s  c2 with the prefix cached (no queries on the root) and branches
       U{1..8}: the HBM-bound small-suffix case
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

SEG_HAS_Q = 1
SEG_SAMPLE_END = 2


@dataclass
class Workload:
    name: str
    parent: List[int]
    seg_len: List[int]
    group_block_size: List[int]
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str  # "f32" | "bf16"
    seg_flags: Optional[List[int]] = None
    free_extents: Optional[List[Tuple[int, int]]] = None
    seed: int = 0
    notes: dict = field(default_factory=dict)

    @property
    def softmax_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))


def star(prefix: int, branches: List[int]):
    parent = [-1] + [0] * len(branches)
    return parent, [int(prefix)] + [int(b) for b in branches]


def make_workload(name: str, seed: int = 0, scale_len: float = 1.0) -> Workload:
    """Build configuration `name` from `seed`.  `scale_len` multiplies every
    drawn length (kept >= 1) to give reduced copies of the same shape."""
    rng = np.random.default_rng([seed, sum(map(ord, name))])

    def sl(x):
        return max(1, int(round(x * scale_len)))

    if name == "c1":
        parent, seg_len = star(64, [32] * 4)
        return Workload(name, parent, seg_len, [16], 2, 2, 64, "f32", seed=seed)
    if name == "c2":
        br = rng.integers(256, 1024, size=8, endpoint=True)
        parent, seg_len = star(sl(4096), [sl(b) for b in br])
        return Workload(name, parent, seg_len, [64], 32, 8, 128, "bf16", seed=seed)
    if name == "c2s":
        br = rng.integers(1, 8, size=8, endpoint=True)
        parent, seg_len = star(sl(4096), [int(b) for b in br])
        flags = [0] + [SEG_HAS_Q | SEG_SAMPLE_END] * 8
        return Workload(name, parent, seg_len, [64], 32, 8, 128, "bf16", seg_flags=flags, seed=seed)
    if name == "c3":
        parent = [-1]
        seg_len = [sl(512)]
        level = [0]
        for depth in range(1, 4):
            nxt = []
            for p in level:
                for _ in range(4):
                    parent.append(p)
                    if depth < 3:
                        seg_len.append(sl(256))
                    else:
                        seg_len.append(sl(int(rng.integers(128, 512, endpoint=True))))
                    nxt.append(len(parent) - 1)
            level = nxt
        return Workload(name, parent, seg_len, [64], 28, 4, 128, "bf16", seed=seed)
    if name == "c4":
        parent, seg_len, gbs = [], [], []
        for _ in range(32):
            root_len = int(np.clip(np.round(np.exp(rng.normal(np.log(2048.0), 1.0))), 256, 16384))
            n_child = int(np.clip(rng.geometric(1.0 / 8.0), 1, 32))
            r = len(parent)
            parent.append(-1)
            seg_len.append(sl(root_len))
            gbs.append(int(rng.choice([16, 64, 256])))
            for _c in range(n_child):
                parent.append(r)
                seg_len.append(sl(int(rng.integers(64, 2048, endpoint=True))))
        # a pool recycled by block caching: 1.25 x the bump size, cut into
        # extents of 256..4096 slots (multiples of 256), listed in shuffled order
        bump, g = 0, -1
        for s, p in enumerate(parent):
            if p == -1:
                g += 1
            bump += -(-seg_len[s] // gbs[g]) * gbs[g]
        arena = int(bump * 1.25) // 256 * 256 + 4096
        extents = []
        at = 0
        while at < arena:
            size = int(rng.integers(1, 16, endpoint=True)) * 256
            size = min(size, arena - at)
            extents.append((at, size))
            at += size
        order = rng.permutation(len(extents))
        extents = [extents[i] for i in order]
        return Workload(name, parent, seg_len, gbs, 32, 8, 128, "bf16", free_extents=extents, seed=seed)
    if name == "c5":
        br = rng.integers(1024, 4096, size=64, endpoint=True)
        parent, seg_len = star(sl(32768), [sl(b) for b in br])
        return Workload(name, parent, seg_len, [256], 64, 8, 128, "bf16", seed=seed)
    raise KeyError(name)


def random_forest(rng: np.random.Generator, n_seg: int, max_len: int, n_roots: int = 1,
                  block_sizes=(16, 32, 64, 128, 256), cached_roots: bool = False,
                  step_samples: bool = False):
    """A random forest for property tests: parents drawn uniformly among earlier
    segments, lengths U{1..max_len}; optional KV-only roots and step-mode samples
    (every segment ends a sample)."""
    parent, seg_len = [], []
    for s in range(n_seg):
        if s < n_roots:
            parent.append(-1)
        else:
            parent.append(int(rng.integers(0, s)))
        seg_len.append(int(rng.integers(1, max_len, endpoint=True)))
    has_child = [False] * n_seg
    for s in range(n_seg):
        if parent[s] >= 0:
            has_child[parent[s]] = True
    flags = []
    for s in range(n_seg):
        f = SEG_HAS_Q
        if cached_roots and parent[s] == -1 and has_child[s]:
            f = 0
        if not has_child[s] or step_samples:
            f |= SEG_SAMPLE_END
        flags.append(f)
    gbs = [int(rng.choice(block_sizes)) for _ in range(n_roots)]
    return parent, seg_len, gbs, flags


def make_inputs(T_q: int, pool_slots: int, tok_slot, n_q_heads: int, n_kv_heads: int,
                head_dim: int, dtype: str, seed: int, device: str = "cpu", pad: str = "normal",
                sparse_do_rows=None):
    """Q, dO [T_q, Hq, d] and K, V pools [Hkv, pool_slots, d], iid N(0,1) drawn
    in fp32 from `seed`, rounded to `dtype` ("f32" | "bf16").

    pad            "normal": slots that hold no token keep their random draw;
                   "nan": they are set to NaN (a correct kernel never lets them
                   reach an output)
    sparse_do_rows if given, dO is zero except on these rows (the rest of dO
                   contributes exactly nothing to any gradient)
    Returns torch tensors on `device`.
    """
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16

    def draw(*shape):
        return torch.randn(*shape, generator=g, device=device, dtype=torch.float32).to(tdt)

    q = draw(T_q, n_q_heads, head_dim)
    k = draw(n_kv_heads, pool_slots, head_dim)
    v = draw(n_kv_heads, pool_slots, head_dim)
    d_o = draw(T_q, n_q_heads, head_dim)
    if pad == "nan":
        used = torch.zeros(pool_slots, dtype=torch.bool, device=device)
        used[torch.as_tensor(np.asarray(tok_slot), dtype=torch.long, device=device)] = True
        k[:, ~used, :] = float("nan")
        v[:, ~used, :] = float("nan")
    if sparse_do_rows is not None:
        keep = torch.zeros(T_q, dtype=torch.bool, device=device)
        keep[torch.as_tensor(np.asarray(sparse_do_rows), dtype=torch.long, device=device)] = True
        d_o[~keep] = 0
    return q, k, v, d_o


def flatten_forest(view: dict):
    """The unshared layout: every sample becomes a root segment of its own
    holding copies of its tokens (what a system without prefix sharing stores).

    Returns (parent, seg_len, group_block_size, tok_src, first_copy) where
    tok_src[i] is the tree token copied to flat token i and first_copy[i] says
    whether it is that token's first copy in canonical sample order (the copy
    that carries the token's upstream gradient row; the others get zero).
    """
    parent, seg_len, gbs, src = [], [], [], []
    for e in view["sample_end_seg"]:
        e = int(e)
        path = list(view["anc_list"][view["anc_off"][e]:view["anc_off"][e + 1]]) + [e]
        L = 0
        for c in path:
            t0 = int(view["seg_tok_off"][c])
            n = int(view["seg_len"][c])
            src.append(np.arange(t0, t0 + n, dtype=np.int64))
            L += n
        parent.append(-1)
        seg_len.append(L)
        gbs.append(int(view["seg_bs"][e]))
    tok_src = np.concatenate(src)
    _, first_idx = np.unique(tok_src, return_index=True)
    first_copy = np.zeros(len(tok_src), dtype=bool)
    first_copy[first_idx] = True
    return parent, seg_len, gbs, tok_src, first_copy
