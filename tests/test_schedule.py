"""Invariants of the device work schedule (host logic, no GPU).

The schedule is not part of the bit-exact plan; what must hold is that the work
items of each kernel cover every attended (query row, key) pair of the tree
exactly once (tree mask of Sec. 2.5: all ancestor tokens + the causal own
segment), and that every reduction (split dK/dV tiles, merged rows) is a fixed
total order over parts that are each produced exactly once.
"""
import os
import re
from collections import Counter

import numpy as np
import pytest

from paper_2608_25683_b200 import binding
from paper_2608_25683_b200.workloads import make_workload, random_forest

PLAN_H = os.path.join(os.path.dirname(binding.__file__), "csrc", "plan.h")


def header_fields():
    """Field names of the schedule header, in order, read from the struct definition."""
    src = open(PLAN_H).read()
    body = src[src.index("struct DeviceHeader {"):]
    body = body[:body.index("};")]
    body = re.sub(r"//[^\n]*", "", body)
    names = []
    for decl in re.findall(r"int32_t\s+([^;]+);", body):
        for item in decl.split(","):
            item = item.strip()
            m = re.match(r"(\w+)\[(\d+)\]", item)
            if m:
                names += [f"{m.group(1)}{i}" for i in range(int(m.group(2)))]
            else:
                names.append(item)
    return names


def decode(plan):
    w = plan.schedule()
    H = dict(zip(header_fields(), w.tolist()))
    assert H["magic"] == 0x5053524C
    rec = lambda off, n, k: w[off:off + n * k].reshape(n, k)
    S = {"H": H}
    S["kvt"] = rec(H["off_kvt"], H["n_kvt"], 12)
    S["qt"] = rec(H["off_qt"], H["n_qt"], 8)
    S["kvi"] = rec(H["off_kvi"], H["n_kvi"], 8)
    S["split"] = rec(H["off_split"], H["n_split"], 4)
    S["path_tiles"] = w[H["off_path_tiles"]:]
    S["path_nvalid"] = w[H["off_path_nvalid"]:]
    n = H["n_merge_rows"]
    S["merge_row"] = w[H["off_merge_row"]:H["off_merge_row"] + n]
    S["merge_off"] = w[H["off_merge_off"]:H["off_merge_off"] + n + 1]
    S["merge_parts"] = w[H["off_merge_parts"]:H["off_merge_parts"] + (int(S["merge_off"][-1]) if n else 0)]
    return S


def expected_pairs(V):
    """{(query row, key token)} of the tree mask."""
    exp = set()
    for c in range(V["n_seg"]):
        if V["seg_q_off"][c] < 0:
            continue
        anc = V["anc_list"][V["anc_off"][c]:V["anc_off"][c + 1]]
        anc_tok = [t for a in anc for t in range(V["seg_tok_off"][a], V["seg_tok_off"][a] + V["seg_len"][a])]
        for i in range(V["seg_len"][c]):
            r = V["seg_q_off"][c] + i
            for t in anc_tok:
                exp.add((r, t))
            for j in range(i + 1):
                exp.add((r, V["seg_tok_off"][c] + j))
    return exp


def check_schedule(plan):
    V, S = plan.view, decode(plan)
    H = S["H"]
    exp = expected_pairs(V)
    tile_tok0 = lambda kt: V["seg_tok_off"][kt[5]] + kt[6] * 128   # seg, tile_idx

    # ---- forward / dQ items ----
    got = Counter()
    final_rows, part_owner = Counter(), {}
    for seg, tidx, q_row0, n_rows, pt, n_tiles, causal, part_row0 in S["qt"].tolist():
        assert 1 <= n_rows <= 128 and n_tiles >= 1
        for row in range(n_rows):
            r = q_row0 + row
            if part_row0 >= 0:
                assert part_row0 + row not in part_owner, "partial row written twice"
                part_owner[part_row0 + row] = r
            else:
                final_rows[r] += 1
            for j in range(n_tiles):
                kt = S["kvt"][S["path_tiles"][pt + j]]
                n_valid = int(kt[4])
                assert n_valid == S["path_nvalid"][pt + j]
                limit = min(row + 1, n_valid) if (causal and j == n_tiles - 1) else n_valid
                t0 = tile_tok0(kt)
                for k in range(limit):
                    got[(r, t0 + k)] += 1
    assert set(got) == exp, "forward items do not cover the tree mask"
    assert max(got.values(), default=1) == 1, "a (row, key) pair is covered twice"
    # every row has one final writer: its own item, or the merge of its parts
    merged = S["merge_row"].tolist()
    assert len(set(merged)) == len(merged)
    used = []
    for i, r in enumerate(merged):
        parts = S["merge_parts"][S["merge_off"][i]:S["merge_off"][i + 1]].tolist()
        assert len(parts) >= 2
        assert all(part_owner[p] == r for p in parts)
        used += parts
    assert sorted(used) == sorted(part_owner), "a partial row is merged twice or never"
    assert len(part_owner) == H["n_part_rows"]
    merged_set = set(merged)
    assert all((final_rows[r] == 1) != (r in merged_set) for r in range(V["T_q"]))

    # ---- dK/dV items ----
    got = Counter()
    owners, slabs = Counter(), Counter()
    for kvt, own0, own_end, dqb, dqe, sb, se, slab in S["kvi"].tolist():
        kt = S["kvt"][kvt]
        t0, n_valid = tile_tok0(kt), int(kt[4])
        subs = []   # (first row, end row, causal offset or None)
        if own0 >= 0:
            for s0 in range(own0, own_end, 128):
                subs.append((s0, min(s0 + 128, own_end), s0 - own0))
        for s0 in range(dqb, dqe, 128):
            subs.append((s0, min(s0 + 128, dqe), None))
        assert 0 <= sb < se <= len(subs)
        if slab < 0:
            owners[kvt] += 1
            assert (sb, se) == (0, len(subs))
        else:
            slabs[slab] += 1
        for s0, s1, diag in subs[sb:se]:
            for r in range(s0, s1):
                for k in range(n_valid):
                    # own rows: row (own0 + x) is the query at the tile's key x
                    if diag is None or k <= (r - own0):
                        got[(r, t0 + k)] += 1
    assert set(got) == exp, "dK/dV items do not cover the tree mask"
    assert max(got.values(), default=1) == 1
    split_tiles = set()
    for kvt, slab0, n_parts, _ in S["split"].tolist():
        assert n_parts >= 2 and kvt not in split_tiles and owners[kvt] == 0
        split_tiles.add(kvt)
        assert all(slabs[s] == 1 for s in range(slab0, slab0 + n_parts))
    assert sum(slabs.values()) == H["n_slabs"]
    assert all(owners[k] == 1 for k in range(H["n_kvt"]) if k not in split_tiles)
    return S


def small_plan(parent, seg_len, bs, flags=None, Hq=4, Hkv=2):
    return binding.Plan(parent, seg_len, bs, Hq, Hkv, 128, "bf16", seg_flags=flags)


def test_schedule_covers_tree_small_cases(lib):
    # plain tree
    check_schedule(small_plan([-1, 0, 0, 1], [200, 130, 7, 40], [64]))
    # single sequence
    check_schedule(small_plan([-1], [300], [16]))
    # two groups with different page sizes
    check_schedule(small_plan([-1, 0, -1, 2, 2], [70, 20, 129, 1, 256], [16, 256]))
    # adaptive blocks
    check_schedule(small_plan([-1, 0, 0, 1], [200, 130, 7, 300], [0]))


def test_short_suffixes_are_packed_and_split(lib):
    """Long cached prefix (no queries) + 8 suffixes of 1..8 tokens: the prefix is cascaded."""
    flags = [0] + [3] * 8
    plan = small_plan([-1] + [0] * 8, [1100, 1, 2, 3, 4, 5, 6, 7, 8], [64], flags, Hq=8, Hkv=2)
    S = check_schedule(plan)
    packed = [q for q in S["qt"].tolist() if q[6] == 0]
    assert packed, "the prefix should be handled by packed items"
    assert len({q[1] for q in packed}) >= 2, "and split into chunks over CTAs"
    assert all(q[3] == 36 for q in packed)
    assert S["H"]["n_merge_rows"] == 36
    assert binding.psrl_launch_count(plan, False) == 2 and binding.psrl_launch_count(plan, True) == 4


def test_many_short_branches_nested(lib):
    """Two levels that both qualify: every row merges parts of two cascaded ancestors + its own."""
    parent = [-1] + [0] * 3
    seg_len = [600, 520, 9, 11]
    for p in (1, 1, 1, 1, 1, 1):
        parent.append(p)
        seg_len.append(5)
    plan = small_plan(parent, seg_len, [128], Hq=2, Hkv=1)
    S = check_schedule(plan)
    assert S["H"]["n_merge_rows"] > 0


def test_which_benchmark_trees_are_cascaded(lib):
    """c2, c3, c5: branches of hundreds or thousands of tokens fill their own tiles - no packed items, no
    merge.  c4 mixes long prefixes with suffixes down to 64 tokens: some of its groups are cascaded, so its
    forward and dQ are followed by the merge kernels; every merged row then has at least two parts and every
    partial row belongs to exactly one merged row."""
    for name in ("c2", "c3", "c5"):
        for seed in (7, 2000):
            w = make_workload(name, seed)
            plan = binding.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
            S = decode(plan)
            assert S["H"]["n_merge_rows"] == 0 and S["H"]["n_part_rows"] == 0
            assert all(q[6] == 1 and q[7] == -1 for q in S["qt"].tolist())
            assert binding.psrl_launch_count(plan, False) == 1
    w = make_workload("c4", 2000)
    plan = binding.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                        w.seg_flags, w.free_extents)
    S = decode(plan)
    H = S["H"]
    assert H["n_merge_rows"] > 0 and binding.psrl_launch_count(plan, False) == 2
    off = S["merge_off"]
    assert (np.diff(off) >= 2).all()
    parts = np.sort(S["merge_parts"])
    assert len(parts) == H["n_part_rows"] and (parts == np.arange(H["n_part_rows"])).all()
    # every work item of every kernel has at least one step wherever its kernel syncs on a named barrier
    assert all(q[5] >= 1 for q in S["qt"].tolist())
    assert all(k[6] > k[5] for k in S["kvi"].tolist())


def test_random_forests(lib):
    rng = np.random.default_rng(5)
    for it in range(16):
        n_roots = 1 + it % 2
        parent, seg_len, gbs, flags = random_forest(rng, n_seg=int(rng.integers(n_roots, 14)), max_len=[12, 150, 400][it % 3],
                                                    n_roots=n_roots, cached_roots=(it % 4 == 0))
        if it % 5 == 0:   # one long prefix above everything
            seg_len[0] = 1500
        plan = binding.Plan(parent, seg_len, gbs, 4, 2, 128, "bf16", seg_flags=flags)
        check_schedule(plan)
