"""The C++ Dynamic Block Caching manager against its oracle (oracle/cache.py): every step's tree,
slot bases, evictions, reloads, releases and counters must agree exactly (host logic, no GPU)."""
import numpy as np
import pytest

from oracle.cache import CacheError, OracleCache
from paper_2608_25683_b200 import binding

from test_oracle_cache import random_case, subtree_uses


def run_both(parent, seg_len, gbs, mb, M, flags=None, cap=0):
    sample_end = None if flags is None else [bool(f & 2) for f in flags]
    want = OracleCache(parent, seg_len, gbs, mb, M, sample_end=sample_end, capacity_slots=cap)
    got = binding.Cache(parent, seg_len, gbs, mb, M, seg_flags=flags, capacity_slots=cap)
    assert got.refcounts() == want.refcount
    for m in range(M):
        try:
            w = want.begin(m)
        except CacheError as e:
            with pytest.raises(binding.PsrlError) as g:
                got.begin(m)
            assert g.value.name == "PSRL_ERR_" + e.code
            return None
        g = got.begin(m)
        for key in ("seg_id", "parent", "seg_len", "seg_flags", "group_block_size", "seg_slot_base", "new", "reload",
                    "live_slots"):
            assert g[key] == w[key], (m, key)
        assert g["evict"] == [tuple(x) for x in w["evict"]]
        w2, g2 = want.end(m), got.end(m)
        assert g2 == w2
        assert got.refcounts() == want.refcount
    s = got.stats()
    ws = want.stats()
    assert (s["peak_slots"], s["evicted_slots"], s["reloaded_slots"], s["pool_high_water"]) == (
        ws["peak_slots"], ws["evicted_slots"], ws["reloaded_slots"], ws["high_water"])
    assert s["total_slots"] == sum(want.extent)
    return s


def test_paper_example(lib):
    s = run_both([-1, 0, 1, 1, 1, 0], [40] * 6, [64], [0, 0, 0, 1, 2, 3], 4)
    assert s["peak_slots"] == 192 and s["total_slots"] == 384 and s["evicted_slots"] == 0


def test_random_schedules_match_oracle(lib):
    rng = np.random.default_rng(11)
    for it in range(150):
        n, M = int(rng.integers(1, 30)), int(rng.integers(1, 9))
        parent, seg_len, gbs, mb = random_case(rng, n, M, max_len=[64, 300][it % 2])
        flags = None
        if it % 3 == 0:   # step-mode sampling: every segment ends a sample
            flags = [2] * n
        cap = 0
        if it % 2 == 1:
            probe = OracleCache(parent, seg_len, gbs, mb, M)
            uses = subtree_uses(parent, mb)
            need = max(sum(probe.extent[s] for s in range(n) if m in uses[s]) for m in range(M))
            cap = need + 16 * int(rng.integers(0, 8))
        run_both(parent, seg_len, gbs, mb, M, flags, cap)


def test_adaptive_extents(lib):
    s = run_both([-1, 0, 0], [28, 4, 300], [0], [0, 0, 1], 2)
    assert s["total_slots"] == 32 + 16 + 304


def test_interleaved_groups(lib):
    s = run_both([-1, 0, 0, -1, 3, 3], [128, 64, 64, 128, 64, 64], [64, 64], [0, 0, 2, 1, 1, 3], 4, cap=192)
    assert s["evicted_slots"] == 256 and s["reloaded_slots"] == 256


def test_errors(lib):
    for args, code in (
        (([-1, 0], [10, 10], [16], [1, 0], 2), "BAD_TREE"),
        (([-1, 0], [10, 10], [24], [0, 1], 2), "BAD_BLOCK_SIZE"),
        (([-1, 0], [10, 10], [16], [0, 2], 2), "INVALID_ARG"),
        (([-1, 0], [10, 0], [16], [0, 1], 2), "BAD_TREE"),
    ):
        with pytest.raises(CacheError) as e:
            OracleCache(*args)
        assert e.value.code == code
        with pytest.raises(binding.PsrlError) as g:
            binding.Cache(*args)
        assert g.value.name == "PSRL_ERR_" + code
    c = binding.Cache([-1], [10], [16], [0], 1)
    with pytest.raises(binding.PsrlError):
        c.end(0)                       # end without begin
    c.begin(0)
    with pytest.raises(binding.PsrlError):
        c.begin(0)                     # begin twice
    c.end(0)
    with pytest.raises(binding.PsrlError):
        c.begin(1)                     # past the last micro-batch
    L = binding.lib()
    assert L.psrl_cache_create(None, None) == 1
    L.psrl_cache_destroy(None)


def test_sawtooth_and_peak_reduction(lib):
    """Step-wise RL group: one long shared prefix per group, branches run in successive micro-batches,
    groups one after the other.  Releasing blocks after their last use bounds the live set by one
    group (a sawtooth), far below what keeping every block would take (cf. Sec. 7.4)."""
    parent, seg_len, mb, gbs = [], [], [], []
    M = 0
    for g in range(6):
        root = len(parent)
        parent.append(-1); seg_len.append(4096); mb.append(M); gbs.append(64)
        for b in range(4):
            parent.append(root); seg_len.append(512); mb.append(M + b)
        M += 4
    c = binding.Cache(parent, seg_len, gbs, mb, M)
    during, after = [], []
    for m in range(M):
        during.append(c.begin(m)["live_slots"])
        after.append(c.end(m)["live_slots"])
    s = c.stats()
    assert s["peak_slots"] == 4096 + 512 and s["total_slots"] == 6 * (4096 + 4 * 512)
    assert after[3::4] == [0] * 6                      # the live set falls to zero after every group
    assert all(d == 4096 + 512 for d in during)
