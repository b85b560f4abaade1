"""Pins of the Dynamic Block Caching oracle (oracle/cache.py): the paper's worked example
(Sec. 5.2), a closed form for the live set, the farthest-next-use rule checked event by event,
and a brute-force search over eviction choices on tiny equal-size cases."""
import itertools
import os

import numpy as np
import pytest

from oracle.cache import CacheError, OracleCache

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "dbc_example.txt")


def read_golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = [int(x) for x in v]
    return out


def test_paper_example():
    g = read_golden()
    n = len(g["parent"])
    c = OracleCache(g["parent"], [40] * n, [64], g["mb_of_seg"], 4)
    assert c.refcount == g["refcount"]                      # root 4, leaves 1
    step = c.begin(0)
    assert step["seg_id"] == [0, 1, 2] and step["new"] == [0, 1, 2]
    assert step["seg_flags"] == [1, 1, 3]                   # all three issue queries; sample a ends at block2
    done = c.end(0)
    assert c.refcount == g["refcount_after_mb0"]
    assert [int(b >= 0) for b in c.base] == g["resident_after_mb0"]
    assert done["freed"] == g["freed_after_mb0"]
    # sample b: the two shared blocks are read in place (no queries on them), its own block is new
    step = c.begin(1)
    assert step["seg_id"] == [0, 1, 3] and step["seg_flags"] == [0, 0, 3] and step["new"] == [3]
    assert step["seg_slot_base"][:2] == [0, 64]
    c.end(1)
    c.begin(2); c.end(2)
    assert c.base[1] == -1 and c.base[0] >= 0               # block1 dies with c, the root waits for d
    c.begin(3)
    assert c.end(3)["live_slots"] == 0


def random_case(rng, n, M, max_len=200):
    parent, mb = [-1], [int(rng.integers(0, max(1, M // 2)))]
    for s in range(1, n):
        if rng.random() < 0.15:
            parent.append(-1)
            mb.append(int(rng.integers(0, M)))
        else:
            p = int(rng.integers(0, s))
            parent.append(p)
            mb.append(int(rng.integers(mb[p], M)))
    seg_len = [int(rng.integers(1, max_len + 1)) for _ in range(n)]
    n_roots = sum(p == -1 for p in parent)
    gbs = [int(rng.choice([16, 64, 256])) for _ in range(n_roots)]
    return parent, seg_len, gbs, mb


def subtree_uses(parent, mb):
    n = len(parent)
    uses = [set() for _ in range(n)]
    for s in range(n):
        a = s
        while a != -1:
            uses[a].add(mb[s])
            a = parent[a]
    return uses


def test_live_set_closed_form_without_cap():
    """Without a memory cap a block lives from the micro-batch that computes it to the last one
    that reads it: live(m) = sum of extents with first use <= m <= last use; nothing is evicted."""
    rng = np.random.default_rng(3)
    for _ in range(40):
        n, M = int(rng.integers(1, 30)), int(rng.integers(1, 9))
        parent, seg_len, gbs, mb = random_case(rng, n, M)
        c = OracleCache(parent, seg_len, gbs, mb, M)
        uses = subtree_uses(parent, mb)
        total = sum(c.extent)
        for m in range(M):
            step = c.begin(m)
            want = sum(c.extent[s] for s in range(n) if min(uses[s]) <= m <= max(uses[s]))
            assert step["live_slots"] == want
            assert sorted(step["seg_id"]) == [s for s in range(n) if m in uses[s]]
            assert not step["evict"] and not step["reload"]
            # extents of resident blocks are disjoint
            spans = sorted((c.base[s], c.base[s] + c.extent[s]) for s in range(n) if c.base[s] >= 0)
            assert all(a[1] <= b[0] for a, b in zip(spans, spans[1:]))
            # every block of the step is where the step says
            assert step["seg_slot_base"] == [c.base[s] for s in step["seg_id"]]
            after = c.end(m)
            assert after["live_slots"] == sum(c.extent[s] for s in range(n) if min(uses[s]) <= m < max(uses[s]))
        assert c.live_slots() == 0 and all(r == 0 for r in c.refcount)
        assert c.stats()["peak_slots"] <= total


def test_eviction_takes_the_farthest_next_use():
    rng = np.random.default_rng(4)
    seen_evictions = 0
    for _ in range(200):
        n, M = int(rng.integers(4, 24)), int(rng.integers(3, 9))
        parent, seg_len, gbs, mb = random_case(rng, n, M, max_len=64)
        free = OracleCache(parent, seg_len, gbs, mb, M)
        uses = subtree_uses(parent, mb)
        need_max = max(sum(free.extent[s] for s in range(n) if m in uses[s]) for m in range(M))
        for m in range(M):
            free.begin(m); free.end(m)
        cap = need_max + 16 * int(rng.integers(0, 3))
        c = OracleCache(parent, seg_len, gbs, mb, M, capacity_slots=cap)
        try:
            for m in range(M):
                resident_before = {s for s in range(n) if c.base[s] >= 0}
                step = c.begin(m)
                need = set(step["seg_id"])
                gone = set()
                for r, old_base in step["evict"]:
                    cands = [x for x in resident_before - need - gone]
                    nxt = lambda x: min(u for u in uses[x] if u > m)
                    assert r in cands and nxt(r) == max(nxt(x) for x in cands)
                    gone.add(r)
                    seen_evictions += 1
                assert step["live_slots"] <= cap
                spans = sorted((c.base[s], c.base[s] + c.extent[s]) for s in range(n) if c.base[s] >= 0)
                assert all(a[1] <= b[0] for a, b in zip(spans, spans[1:])) and (not spans or spans[-1][1] <= cap)
                for s in step["reload"]:
                    assert mb[s] < m
                c.end(m)
        except CacheError as e:   # fragmentation can defeat a cap that is only just large enough
            assert e.code == "POOL_FULL"
    assert seen_evictions > 8


def test_interleaved_groups_evict_and_reload():
    """Two prefix groups whose branches alternate between micro-batches, room for one group only:
    each root is evicted while the other group runs and brought back for its next branch."""
    parent = [-1, 0, 0, -1, 3, 3]
    mb = [0, 0, 2, 1, 1, 3]
    c = OracleCache(parent, [128, 64, 64, 128, 64, 64], [64, 64], mb, 4, capacity_slots=192)
    s0 = c.begin(0); c.end(0)
    assert s0["new"] == [0, 1] and not s0["evict"]
    s1 = c.begin(1); c.end(1)
    assert [r for r, _ in s1["evict"]] == [0] and s1["new"] == [3, 4]
    s2 = c.begin(2); c.end(2)
    assert [r for r, _ in s2["evict"]] == [3] and s2["reload"] == [0] and s2["new"] == [2]
    s3 = c.begin(3)
    assert s3["reload"] == [3] and s3["new"] == [5]
    assert c.end(3)["live_slots"] == 0
    st = c.stats()
    assert st["evicted_slots"] == 256 and st["reloaded_slots"] == 256 and st["peak_slots"] == 192


def brute_force_min_reloads(n, uses, M, slots):
    """Fewest reloads over all eviction choices; every block has the same size (one slot)."""
    best = [None]

    def go(m, resident, reloads, ever):
        if best[0] is not None and reloads >= best[0]:
            return
        if m == M:
            best[0] = reloads
            return
        need = {s for s in range(n) if m in uses[s]}
        missing = [s for s in need if s not in resident]
        room = slots - len(resident)
        k = max(0, len(missing) - room)
        cands = [r for r in resident if r not in need]
        if k > len(cands):
            return
        for out in itertools.combinations(cands, k):
            res = (resident - set(out)) | need
            rel = reloads + sum(1 for s in missing if s in ever)
            # blocks past their last use are dropped after the micro-batch
            res2 = {s for s in res if max(uses[s]) > m}
            go(m + 1, res2, rel, ever | need)

    go(0, set(), 0, set())
    return best[0]


def test_reloads_match_brute_force_on_equal_sizes():
    """With equal block sizes the farthest-next-use rule is optimal: the oracle's reload count
    equals the minimum over all eviction choices."""
    rng = np.random.default_rng(5)
    checked = 0
    for _ in range(40):
        n, M = int(rng.integers(4, 9)), int(rng.integers(3, 7))
        parent, _, _, mb = random_case(rng, n, M)
        n_roots = sum(p == -1 for p in parent)
        uses = subtree_uses(parent, mb)
        need_max = max(sum(1 for s in range(n) if m in uses[s]) for m in range(M))
        slots = need_max
        c = OracleCache(parent, [16] * n, [16] * n_roots, mb, M, capacity_slots=16 * slots)
        reloads = 0
        for m in range(M):
            reloads += len(c.begin(m)["reload"])
            c.end(m)
        assert reloads == brute_force_min_reloads(n, uses, M, slots)
        checked += reloads > 0
    assert checked >= 3


def test_errors():
    with pytest.raises(CacheError) as e:
        OracleCache([-1, 0], [10, 10], [16], [1, 0], 2)           # suffix before its prefix
    assert e.value.code == "BAD_TREE"
    with pytest.raises(CacheError) as e:
        OracleCache([-1, 0], [10, 10], [24], [0, 1], 2)
    assert e.value.code == "BAD_BLOCK_SIZE"
    c = OracleCache([-1, 0, 0], [100, 100, 100], [64], [0, 1, 2], 3, capacity_slots=128)
    with pytest.raises(CacheError) as e:
        c.begin(0); c.end(0); c.begin(1)                           # root (128) + child (128) > 128
    assert e.value.code == "POOL_FULL"
    c = OracleCache([-1], [10], [16], [0], 1)
    with pytest.raises(CacheError):
        c.end(0)
