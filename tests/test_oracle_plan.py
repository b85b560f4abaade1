"""Pins for the plan oracle: the paper's printed examples, closed forms, hand
counts and a brute-force token-by-token expansion."""
import os

import numpy as np
import pytest

from oracle import oracle_plan, PlanError
from paper_2608_25683_b200.workloads import make_workload, random_forest

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read(name):
    with open(os.path.join(GOLD, name)) as f:
        return [l.split() for l in f if l.strip() and not l.startswith("#")]


def test_refcount_example_from_paper():
    rows = _read("refcount_example.txt")
    parent = [int(r[1]) for r in rows if r[0] == "seg"]
    seg_len = [int(r[2]) for r in rows if r[0] == "seg"]
    p = oracle_plan(parent, seg_len, [16])
    for r in rows:
        if r[0] == "expect":
            c = int(p["canon_of_input"][int(r[1])])
            assert p["seg_refcount"][c] == int(r[2])
            pg = p["seg_first_page"][c]
            assert p["page_refcount"][pg] == int(r[2])
    assert p["n_samples"] == 4


def test_shared_28_tokens_example_from_paper():
    rows = _read("shared_28_tokens.txt")
    parent = [int(r[1]) for r in rows if r[0] == "seg"]
    seg_len = [int(r[2]) for r in rows if r[0] == "seg"]
    for r in rows:
        if r[0] == "bs":
            bs = int(r[1].rstrip(":"))
            want = [int(x) for x in r[3:]]
            p = oracle_plan(parent, seg_len, [bs])
            got = list(p["page_valid"][: p["seg_n_pages"][0]])
            assert got == want
            assert p["T"] == 36 and p["flat_tokens"] == 64
            assert p["seg_refcount"][0] == 2
            # the divergent tokens sit in pages of their own
            assert p["seg_n_pages"][1] == 1 and p["seg_n_pages"][2] == 1
            assert p["page_slot"][p["seg_first_page"][1]] != p["page_slot"][p["seg_first_page"][2]]


def test_c1_hand_counts():
    want = {r[0]: int(r[1]) for r in _read("c1_counts.txt")}
    w = make_workload("c1")
    p = oracle_plan(w.parent, w.seg_len, w.group_block_size)
    assert p["T"] == want["T"]
    assert p["flat_tokens"] == want["flat_tokens"]
    assert p["n_pages"] == want["n_pages"]
    assert len(p["bt_pages"]) == want["bt_entries"]
    assert p["tree_pairs"] == want["tree_pairs"]
    assert p["flat_pairs"] == want["flat_pairs"]


def _forests():
    rng = np.random.default_rng(7)
    out = []
    for i in range(40):
        n_roots = int(rng.integers(1, 4))
        n_seg = int(rng.integers(n_roots, 14))
        parent, seg_len, gbs, flags = random_forest(
            rng, n_seg, 70, n_roots, cached_roots=(i % 3 == 0), step_samples=(i % 4 == 1))
        out.append((parent, seg_len, gbs, flags))
    return out


@pytest.mark.parametrize("forest", _forests())
def test_closed_forms_and_brute_force(forest):
    parent, seg_len, gbs, flags = forest
    p = oracle_plan(parent, seg_len, gbs, flags)
    n = p["n_seg"]
    # closed forms
    assert int(p["page_valid"].sum()) == p["T"] == sum(seg_len)
    assert p["pool_slots"] == int((p["seg_n_pages"] * p["seg_bs"]).sum())  # bump allocation
    assert int((p["seg_len"].astype(np.int64) * p["seg_refcount"]).sum()) == p["flat_tokens"]
    # canonical order is a permutation and keeps parents before children
    assert sorted(p["input_of_canon"]) == list(range(n))
    for c in range(n):
        assert p["seg_parent"][c] < c
        s = p["input_of_canon"][c]
        assert p["seg_len"][c] == seg_len[s]
        want_parent = -1 if parent[s] == -1 else p["canon_of_input"][parent[s]]
        assert p["seg_parent"][c] == want_parent
    # brute force: expand every sample token by token (input indexing, no plan)
    ends = [s for s in range(n) if flags[s] & 2]
    count = np.zeros(n, dtype=np.int64)  # samples through each segment
    flat_tokens = 0
    flat_pairs = 0
    for e in ends:
        path = []
        s = e
        while s != -1:
            path.append(s)
            s = parent[s]
        path.reverse()
        L = 0
        for s in path:
            count[s] += 1
            for _ in range(seg_len[s]):
                L += 1
                flat_pairs += L
        flat_tokens += L
        # the block-table row of the end segment lists exactly the slots of the
        # sample's tokens, in order
        c = p["canon_of_input"][e]
        slots = []
        for pg in p["bt_pages"][p["bt_off"][c]:p["bt_off"][c + 1]]:
            slots.extend(range(p["page_slot"][pg], p["page_slot"][pg] + p["page_valid"][pg]))
        toks = []
        for s in path:
            cc = p["canon_of_input"][s]
            toks.extend(range(p["seg_tok_off"][cc], p["seg_tok_off"][cc] + p["seg_len"][cc]))
        assert slots == [int(p["tok_slot"][t]) for t in toks]
        assert p["sample_len"][list(p["sample_end_seg"]).index(c)] == L
    assert flat_tokens == p["flat_tokens"] and flat_pairs == p["flat_pairs"]
    for s in range(n):
        assert p["seg_refcount"][p["canon_of_input"][s]] == count[s]
    tree_pairs = 0
    for s in range(n):
        if flags[s] & 1:
            anc = 0
            a = parent[s]
            while a != -1:
                anc += seg_len[a]
                a = parent[a]
            for i in range(seg_len[s]):
                tree_pairs += anc + i + 1
            assert p["seg_anc_tokens"][p["canon_of_input"][s]] == anc
    assert tree_pairs == p["tree_pairs"]
    # every token has a slot of its own, inside a page of its segment
    assert len(set(p["tok_slot"].tolist())) == p["T"]
    for pg in range(p["n_pages"]):
        c = p["page_seg"][pg]
        i = pg - p["seg_first_page"][c]
        assert p["page_pos"][pg] == p["seg_anc_tokens"][c] + i * p["page_bs"][pg]
        assert p["page_slot"][pg] % 16 == 0
    # subtree ranges: descendants are exactly the canonical indices in (c, sub_end)
    for c in range(n):
        for e in range(n):
            a = e
            is_desc = False
            while a != -1:
                a = p["seg_parent"][a]
                if a == c:
                    is_desc = True
            assert is_desc == (c < e < p["seg_sub_end"][c])
    # q offsets pack the querying segments in canonical order
    tq = 0
    for c in range(n):
        if p["seg_flags"][c] & 1:
            assert p["seg_q_off"][c] == tq
            tq += p["seg_len"][c]
        else:
            assert p["seg_q_off"][c] == -1
    assert tq == p["T_q"]


def test_first_fit_over_free_extents():
    # pages of 16: extents are consumed front to back in list order
    p = oracle_plan([-1, 0], [40, 20], [16], free_extents=[(64, 32), (0, 16), (256, 64)])
    # root: 3 pages -> 64, 80 (first extent), then 0 (second extent)
    # child: 2 pages -> 256, 272
    assert p["page_slot"].tolist() == [64, 80, 0, 256, 272]
    assert p["pool_slots"] == 288
    with pytest.raises(PlanError) as e:
        oracle_plan([-1], [100], [64], free_extents=[(0, 64), (64, 32)])
    assert e.value.code == "POOL_FULL"
    # a page must lie wholly inside one extent
    p = oracle_plan([-1], [64], [64], free_extents=[(0, 32), (32, 32), (128, 64)])
    assert p["page_slot"].tolist() == [128]


def test_validation_errors():
    for args, code in [
        (([0], [4], [16]), "BAD_TREE"),            # parent not before child
        (([-1, 1], [4, 4], [16]), "BAD_TREE"),
        (([-1], [0], [16]), "BAD_TREE"),
        (([-1], [4], [24]), "BAD_BLOCK_SIZE"),
        (([-1], [4], [8]), "BAD_BLOCK_SIZE"),
        (([-1], [4], [512]), "BAD_BLOCK_SIZE"),
        (([-1], [4], [16, 16]), "INVALID_ARG"),
    ]:
        with pytest.raises(PlanError) as e:
            oracle_plan(*args)
        assert e.value.code == code
    with pytest.raises(PlanError) as e:
        oracle_plan([-1, 0], [4, 4], [16], seg_flags=[3, 1])  # leaf without SAMPLE_END
    assert e.value.code == "BAD_TREE"


def test_synthetic_configs_land_in_paper_ranges():
    # Tab. 1: step-mode prefix match rates 72.56 % .. 94.51 %; tree modes 54-62 %
    for name, lo, hi in [("c2", 0.70, 0.95), ("c5", 0.85, 0.95), ("c3", 0.5, 0.8), ("c4", 0.5, 0.8)]:
        w = make_workload(name, 0)
        p = oracle_plan(w.parent, w.seg_len, w.group_block_size, w.seg_flags, w.free_extents)
        pmr = 1 - p["T"] / p["flat_tokens"]
        assert lo <= pmr <= hi, (name, pmr)


def test_adaptive_blocks():
    """Block size 0 = Adaptive Block Allocation (Sec. 5.1): every segment gets one extent sized to its
    span at 16-slot granularity, so a 28-token shared span costs 32 slots whatever the page size of
    other groups, tokens sit at consecutive slots, and the pool is the sum of the rounded spans."""
    parent, seg_len = [-1, 0, 0, -1, 3], [28, 4, 300, 129, 16]
    p = oracle_plan(parent, seg_len, [0, 0])
    ceil16 = lambda x: -(-x // 16) * 16
    assert p["pool_slots"] == sum(ceil16(l) for l in seg_len)
    assert int(p["page_valid"].sum()) == sum(seg_len)
    for c in range(p["n_seg"]):
        t0, l = int(p["seg_tok_off"][c]), int(p["seg_len"][c])
        slots = p["tok_slot"][t0:t0 + l]
        assert np.array_equal(slots, slots[0] + np.arange(l))                 # one contiguous extent
        sizes = p["page_bs"][p["seg_first_page"][c]:p["seg_first_page"][c] + p["seg_n_pages"][c]].tolist()
        assert sizes == [128] * (l // 128) + [16] * (-(-(l % 128) // 16))
    assert p["seg_bs"].tolist() == [0] * 5
    # the shared 28-token span of the paper's example: 32 slots, stored once, whereas a fixed page of
    # 32 in a layout that pages whole sequences could not share it (Sec. 5.1)
    c0 = int(p["canon_of_input"][0])
    assert int(p["page_bs"][p["seg_first_page"][c0]]) == 16 and int(p["seg_n_pages"][c0]) == 2
    # mixed with a fixed-size group, fragmented pool: an adaptive extent is taken whole from one free extent
    q = oracle_plan([-1, -1], [200, 100], [0, 64], None, [(0, 128), (1024, 512)])
    assert q["page_slot"].tolist()[:3] == [1024, 1152, 1168]     # 200 -> 208 slots do not fit in the first extent
    assert q["page_slot"].tolist()[6:] == [0, 64]                # the 64-slot pages of the second group do
