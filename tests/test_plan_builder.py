"""C++ plan builder vs the plan oracle, byte for byte; C-ABI surface checks (CPU only)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import oracle_plan, PlanError
from oracle.plan import PLAN_ARRAYS, PLAN_SCALARS
from paper_2608_25683_b200.workloads import flatten_forest, make_workload, random_forest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _same(view, want):
    for k in PLAN_SCALARS:
        assert view[k] == want[k], k
    for k in PLAN_ARRAYS:
        a, b = view[k], want[k]
        assert a.dtype == np.int32 and b.dtype == np.int32
        assert a.tobytes() == b.tobytes(), k


@pytest.mark.parametrize("name", ["c1", "c2", "c2s", "c3", "c4", "c5"])
@pytest.mark.parametrize("seed", [0, 1])
def test_configs_bit_exact(lib, name, seed):
    w = make_workload(name, seed)
    plan = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                    w.seg_flags, w.free_extents)
    _same(plan.view, oracle_plan(w.parent, w.seg_len, w.group_block_size, w.seg_flags, w.free_extents))


def test_random_forests_bit_exact(lib):
    rng = np.random.default_rng(11)
    for i in range(150):
        n_roots = int(rng.integers(1, 5))
        n_seg = int(rng.integers(n_roots, 40))
        parent, seg_len, gbs, flags = random_forest(rng, n_seg, 300, n_roots, cached_roots=(i % 3 == 0),
                                                    step_samples=(i % 4 == 1))
        extents = None
        if i % 2:
            need = oracle_plan(parent, seg_len, gbs, flags)["pool_slots"]
            extents, at = [], 0
            while at < 2 * need + 512:
                sz = int(rng.integers(1, 40)) * 16
                extents.append((at, sz))
                at += sz + int(rng.integers(0, 3)) * 16
            extents = [extents[j] for j in rng.permutation(len(extents))]
        try:
            want = oracle_plan(parent, seg_len, gbs, flags, extents)
        except PlanError as e:
            with pytest.raises(lib.PsrlError) as got:
                lib.Plan(parent, seg_len, gbs, 4, 2, 128, "bf16", flags, extents)
            assert got.value.name == "PSRL_ERR_" + e.code
            continue
        plan = lib.Plan(parent, seg_len, gbs, 4, 2, 128, "bf16", flags, extents)
        _same(plan.view, want)


def test_errors_match_oracle(lib):
    cases = [
        (([0], [4], [16]), {}, "BAD_TREE"),
        (([-1, 1], [4, 4], [16]), {}, "BAD_TREE"),
        (([-1], [0], [16]), {}, "BAD_TREE"),
        (([-1], [4], [24]), {}, "BAD_BLOCK_SIZE"),
        (([-1], [4], [8]), {}, "BAD_BLOCK_SIZE"),
        (([-1], [4], [512]), {}, "BAD_BLOCK_SIZE"),
        (([-1], [4], [16, 16]), {}, "INVALID_ARG"),
        (([-1, 0], [4, 4], [16]), dict(seg_flags=[3, 1]), "BAD_TREE"),
        (([-1], [100], [64]), dict(free_extents=[(0, 64), (64, 32)]), "POOL_FULL"),
        (([-1], [4], [16]), dict(free_extents=[(8, 64)]), "INVALID_ARG"),
    ]
    for args, kw, code in cases:
        with pytest.raises(PlanError) as e:
            oracle_plan(*args, **kw)
        assert e.value.code == code
        with pytest.raises(lib.PsrlError) as g:
            lib.Plan(*args, 2, 1, 128, "bf16", **kw)
        assert g.value.name == "PSRL_ERR_" + code
    # library-only argument errors
    for kw, name in [
        (dict(n_q_heads=3, n_kv_heads=2, head_dim=128, dtype="bf16"), "PSRL_ERR_SHAPE"),
        (dict(n_q_heads=2, n_kv_heads=2, head_dim=64, dtype="bf16"), "PSRL_ERR_UNSUPPORTED"),
        (dict(n_q_heads=2, n_kv_heads=2, head_dim=96, dtype="f32"), "PSRL_ERR_UNSUPPORTED"),
        (dict(n_q_heads=2, n_kv_heads=2, head_dim=64, dtype="f16"), "PSRL_ERR_UNSUPPORTED"),
    ]:
        with pytest.raises(lib.PsrlError) as g:
            lib.Plan([-1], [4], [16], **kw)
        assert g.value.name == name


def test_library_exports_every_declared_symbol(lib):
    hdr = open(os.path.join(ROOT, "include", "psrl.h")).read() + open(os.path.join(ROOT, "include", "psrl_cache.h")).read() + open(os.path.join(ROOT, "include", "psrl_sched.h")).read()
    declared = set(re.findall(r"\b(psrl_[a-z_0-9]+)\s*\(", hdr))
    assert declared, "no declarations found"
    L = lib.lib()
    for name in declared:
        assert hasattr(L, name), f"{name} declared in include/*.h but not exported"
    assert set(lib.EXPORTS) <= declared
    assert L.psrl_status_string(0) == b"PSRL_OK"
    assert L.psrl_status_string(10) == b"PSRL_ERR_TIMEOUT"
    # null handling never crashes
    assert L.psrl_plan_device_bytes(None) == 0
    assert L.psrl_plan_build(None, None) == 1
    L.psrl_plan_destroy(None)


def test_launch_argument_checks_need_no_gpu(lib):
    """The entry points reject bad arguments on the host, before any CUDA call."""
    plan = lib.Plan([-1, 0], [20, 5], [16], 2, 1, 64, "f32")
    L = lib.lib()
    buf = ctypes.create_string_buffer(4096)
    p = (ctypes.addressof(buf) + 255) // 256 * 256
    # not uploaded -> WORKSPACE; misaligned -> INVALID_ARG; small pool -> SHAPE
    st = L.psrl_tree_attn_fwd(plan.handle, p, p, p, 1024, p, p, 1.0, p, 4096 - 256, None)
    assert lib.STATUS_NAMES[st] == "PSRL_ERR_WORKSPACE"
    st = L.psrl_tree_attn_fwd(plan.handle, p + 4, p, p, 1024, p, p, 1.0, p, 4096 - 256, None)
    assert lib.STATUS_NAMES[st] == "PSRL_ERR_INVALID_ARG"
    st = L.psrl_tree_attn_fwd(plan.handle, p, p, p, 8, p, p, 1.0, p, 4096 - 256, None)
    assert lib.STATUS_NAMES[st] == "PSRL_ERR_SHAPE"
    st = L.psrl_tree_attn_bwd(plan.handle, p, p, p, 1024, p, p, None, p, p, p, 1.0, p, 4096 - 256, None)
    assert lib.STATUS_NAMES[st] == "PSRL_ERR_INVALID_ARG"
    assert plan.bwd_workspace_bytes() >= 256 + 4 * 2 * 25
    assert plan.device_bytes() % 256 == 0 and plan.device_bytes() > 0


def test_flatten_forest(lib):
    w = make_workload("c3", 0, scale_len=0.05)
    plan = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    parent, seg_len, gbs, src, first = flatten_forest(plan.view)
    V = plan.view
    assert sum(seg_len) == V["flat_tokens"] == len(src)
    assert first.sum() == V["T"]
    flat = lib.Plan(parent, seg_len, gbs, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    assert flat.view["tree_pairs"] == V["flat_pairs"] == flat.view["flat_pairs"]


def test_pinned_segments_bit_exact(lib):
    """Segments whose K/V already lives in the pool (cached by an earlier micro-batch) are pinned
    to their slots; everything else is allocated around them exactly as the oracle does."""
    rng = np.random.default_rng(77)
    for it in range(25):
        n_roots = 1 + it % 2
        parent, seg_len, gbs, flags = random_forest(rng, int(rng.integers(n_roots + 1, 12)), 300, n_roots,
                                                    cached_roots=(it % 3 == 0))
        # pin a random subset at non-overlapping bases far above the bump region
        base, pinned, at = [], rng.random(len(parent)) < 0.4, 1 << 16
        root_of = []
        for s, p in enumerate(parent):
            root_of.append(len([q for q in parent[:s + 1] if q == -1]) - 1 if p == -1 else root_of[p])
        for s in range(len(parent)):
            if pinned[s]:
                bs = gbs[root_of[s]]
                base.append(at)
                at += -(-seg_len[s] // bs) * bs + 16 * int(rng.integers(0, 4))
            else:
                base.append(-1)
        want = oracle_plan(parent, seg_len, gbs, flags, None, base)
        got = lib.Plan(parent, seg_len, gbs, 4, 2, 128, "bf16", seg_flags=flags, seg_slot_base=base).view
        for name in PLAN_ARRAYS:
            assert np.array_equal(got[name], want[name]), name
        for name in PLAN_SCALARS:
            assert int(got[name]) == int(want[name]), name
        # pinned pages sit where they were put
        for s in range(len(parent)):
            if base[s] >= 0:
                c = int(want["canon_of_input"][s])
                p0 = int(want["seg_first_page"][c])
                assert int(want["page_slot"][p0]) == base[s]
    # a base that is not a multiple of 16 is rejected by both
    with pytest.raises(PlanError) as e1:
        oracle_plan([-1, 0], [20, 5], [16], None, None, [8, -1])
    assert e1.value.code == "INVALID_ARG"
    with pytest.raises(lib.PsrlError) as e2:
        lib.Plan([-1, 0], [20, 5], [16], 4, 2, 128, "bf16", seg_slot_base=[8, -1])
    assert e2.value.name == "PSRL_ERR_INVALID_ARG"


def test_adaptive_blocks_bit_exact(lib):
    rng = np.random.default_rng(99)
    for it in range(30):
        n_roots = 1 + it % 3
        parent, seg_len, gbs, flags = random_forest(rng, int(rng.integers(n_roots, 14)), 500, n_roots,
                                                    block_sizes=(0, 0, 16, 64, 256), cached_roots=(it % 4 == 0))
        fe = None
        if it % 3 == 2:
            fe = [(4096 * i, 2048) for i in range(8)]
        want = oracle_plan(parent, seg_len, gbs, flags, fe)
        got = lib.Plan(parent, seg_len, gbs, 4, 2, 128, "bf16", seg_flags=flags, free_extents=fe).view
        for name in PLAN_ARRAYS:
            assert np.array_equal(got[name], want[name]), name
        for name in PLAN_SCALARS:
            assert int(got[name]) == int(want[name]), name
    with pytest.raises(lib.PsrlError) as e:     # adaptive blocks exist on the tensor-core path only
        lib.Plan([-1], [40], [0], 2, 2, 64, "f32")
    assert e.value.name == "PSRL_ERR_UNSUPPORTED"


def test_static_backward_limit_is_the_whole_workspace(lib):
    """The built-in scratch array of psrl_tree_attn_bwd_static stands in for the whole backward workspace: the
    header's constant equals the binding's, a plan under the D limit can still be over the array's size once the
    slabs of its split KV tiles are counted (c3), and small plans fit."""
    src = open(os.path.join(ROOT, "include", "psrl.h")).read()
    m = re.search(r"#define PSRL_BWD_STATIC_SCRATCH_BYTES \(\(size_t\)(\d+)\)", src)
    assert m and int(m.group(1)) == lib.BWD_STATIC_SCRATCH_BYTES == 16 * 1024 * 1024 + 256
    w = make_workload("c3", 2000)
    plan = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    assert plan.view["T_q"] * w.n_q_heads < 4 * 1024 * 1024
    assert plan.bwd_workspace_bytes() > lib.BWD_STATIC_SCRATCH_BYTES
    w = make_workload("c2", 2000)
    plan = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    assert plan.bwd_workspace_bytes() <= lib.BWD_STATIC_SCRATCH_BYTES
