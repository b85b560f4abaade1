"""GPU parity, bf16 tensor-core path, against the fp64 oracle on the same
bf16-rounded inputs.  Bars: max-abs 1e-2 on O (and on LSE), relative Frobenius
error 1e-2 on each of dQ, dK, dV; pad slots of the gradient pools are zeros."""
import numpy as np
import pytest
import torch

from oracle import oracle_attn
from paper_2608_25683_b200.workloads import Workload, make_inputs, make_workload, random_forest

from util import build_plan, page_masks, rel_fro, run_gpu, to_np

pytestmark = pytest.mark.gpu
O_TOL = 1e-2     # max-abs on O
G_TOL = 1e-2     # relative Frobenius on dQ, dK, dV


def check(lib, w, seed, pad="nan", extra_capacity=0, backward=True):
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    cap = V["pool_slots"] + extra_capacity
    q, k, v, d_o = make_inputs(V["T_q"], cap, V["tok_slot"], w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, seed,
                               device="cuda", pad=pad)
    got = run_gpu(lib, plan, q, k, v, d_o, w.softmax_scale, backward=backward)
    want = oracle_attn(V, to_np(q), to_np(k), to_np(v), to_np(d_o) if backward else None, w.softmax_scale)
    o = to_np(got["O"])
    assert np.isfinite(o).all()
    assert np.abs(o - want["O"]).max() <= O_TOL
    assert np.abs(to_np(got["LSE"]) - want["LSE"]).max() <= O_TOL
    if backward:
        tok, padm, outside = page_masks(V, cap)
        dq, dk, dv = to_np(got["dQ"]), to_np(got["dK"]), to_np(got["dV"])
        assert np.isfinite(dq).all()
        assert rel_fro(dq, want["dQ"]) <= G_TOL
        assert np.isfinite(dk[:, tok]).all() and np.isfinite(dv[:, tok]).all()
        assert rel_fro(dk[:, tok], want["dK"][:, tok]) <= G_TOL
        assert rel_fro(dv[:, tok], want["dV"][:, tok]) <= G_TOL
        assert np.all(dk[:, padm] == 0) and np.all(dv[:, padm] == 0)
        assert np.all(np.isnan(dk[:, outside])) and np.all(np.isnan(dv[:, outside]))
    return plan, (q, k, v, d_o), got


def test_single_tile(lib):
    check(lib, Workload("t", [-1], [128], [64], 2, 1, 128, "bf16"), seed=1)


def test_star_small(lib):
    # several KV tiles, ragged tails, pads inside pages; GQA group of 2 (one head pair per CTA)
    check(lib, Workload("s", [-1, 0, 0, 0], [300, 70, 129, 1], [64], 4, 2, 128, "bf16"), seed=2)


@pytest.mark.parametrize("bs", [16, 32, 64, 128, 256])
def test_every_block_size(lib, bs):
    check(lib, Workload("b", [-1, 0, 0], [333, 200, 45], [bs], 4, 2, 128, "bf16"), seed=3 + bs, extra_capacity=32)


def test_adaptive_blocks(lib):
    """Block size 0: one extent per segment sized to its span (Sec. 5.1); NaN in every slot that holds
    no token, next to mixed fixed-size groups."""
    check(lib, Workload("aba", [-1, 0, 0, 1], [333, 200, 45, 129], [0], 4, 2, 128, "bf16"), seed=71, extra_capacity=32)
    check(lib, Workload("aba2", [-1, 0, -1, 2, 2], [28, 4, 700, 16, 1], [0, 64], 8, 2, 128, "bf16"), seed=72)


def test_odd_group_and_mha(lib):
    # G = 3: one head pair + one single head per KV head; G = 1: MHA
    check(lib, Workload("g3", [-1, 0, 0], [150, 90, 260], [32], 6, 2, 128, "bf16"), seed=5)
    check(lib, Workload("mha", [-1, 0], [140, 130], [64], 2, 2, 128, "bf16"), seed=6)


def test_deep_tree_and_forest(lib):
    rng = np.random.default_rng(17)
    for i in range(4):
        n_roots = int(rng.integers(1, 4))
        parent, seg_len, gbs, flags = random_forest(rng, int(rng.integers(n_roots + 2, 14)), 400, n_roots,
                                                    cached_roots=(i % 2 == 0), step_samples=(i == 1))
        check(lib, Workload("rnd", parent, seg_len, gbs, 8, 2, 128, "bf16", seg_flags=flags), seed=30 + i,
              extra_capacity=64)


def test_fragmented_pool(lib):
    w = Workload("frag", [-1, 0, 0], [500, 140, 77], [16], 4, 1, 128, "bf16",
                 free_extents=[(2048, 256), (0, 160), (512, 512), (4096, 1024)])
    check(lib, w, seed=9, extra_capacity=128)


@pytest.mark.parametrize("name,scale_len", [("c2", 0.25), ("c3", 0.25), ("c4", 0.03)])
def test_reduced_configs(lib, name, scale_len):
    """The benchmark configurations at reduced lengths: every tile kind of the
    full-size runs (several tiles per segment, ragged tails, all block sizes,
    fragmented pool) at a size the oracle finishes in seconds."""
    w = make_workload(name, 0, scale_len=scale_len)
    if name == "c4":
        # keep a handful of groups: the oracle cost is what bounds this case
        keep, roots = [], 0
        for s, p in enumerate(w.parent):
            roots += p == -1
            if roots <= 6:
                keep.append(s)
        w.parent = [w.parent[s] for s in keep]
        w.seg_len = [w.seg_len[s] for s in keep]
        w.group_block_size = w.group_block_size[:6]
        w.n_q_heads, w.n_kv_heads = 8, 2
    check(lib, w, seed=100)


def test_small_suffixes_on_a_long_prefix(lib):
    """The memory-bound case: a cached prefix (no queries) and suffixes of a few tokens.  The
    prefix's KV tiles are visited by packed rows and split over CTAs; rows are assembled by
    the merge kernels (forward: log-sum-exp of the parts, backward: sum of the parts' dQ)."""
    flags = [0] + [3] * 8
    w = Workload("ss", [-1] + [0] * 8, [1100, 1, 2, 3, 4, 5, 6, 7, 8], [64], 8, 2, 128, "bf16", seg_flags=flags)
    plan, _, _ = check(lib, w, seed=40)
    assert lib.psrl_launch_count(plan, False) == 2
    # the same with queries on the prefix, G = 3 (a head pair + a single head)
    check(lib, Workload("ssq", [-1] + [0] * 8, [1100, 1, 2, 3, 4, 5, 6, 7, 8], [32], 6, 2, 128, "bf16"), seed=41)
    # full-size c2s
    w = make_workload("c2s", 3)
    plan, _, _ = check(lib, w, seed=42)
    assert lib.psrl_launch_count(plan, False) == 2


def test_nested_cascades(lib):
    """Two levels of long segments above many short leaves: rows merge the parts of two
    cascaded ancestors and their own item; more than 128 packed rows (two row blocks)."""
    parent, seg_len = [-1, 0, 0, 0], [600, 520, 9, 11]
    for _ in range(30):
        parent.append(1)
        seg_len.append(5)
    plan, _, _ = check(lib, Workload("nest", parent, seg_len, [128], 4, 2, 128, "bf16"), seed=43)
    assert lib.psrl_launch_count(plan, True) >= 4


def test_runs_are_bitwise_reproducible(lib):
    w = Workload("det", [-1, 0, 0, 1], [700, 300, 129, 50], [64], 8, 2, 128, "bf16")
    plan, (q, k, v, d_o), a = check(lib, w, seed=12)
    for _ in range(2):
        b = run_gpu(lib, plan, q, k, v, d_o, w.softmax_scale)
        for key in ("O", "LSE", "dQ"):
            assert torch.equal(a[key], b[key])
        for key in ("dK", "dV"):
            assert torch.equal(torch.nan_to_num(a[key]), torch.nan_to_num(b[key]))
    # and with merged rows (cascaded prefix, split over CTAs)
    w = make_workload("c2s", 5)
    plan, (q, k, v, d_o), a = check(lib, w, seed=13)
    for _ in range(2):
        b = run_gpu(lib, plan, q, k, v, d_o, w.softmax_scale)
        for key in ("O", "LSE", "dQ"):
            assert torch.equal(a[key], b[key])
        for key in ("dK", "dV"):
            assert torch.equal(torch.nan_to_num(a[key]), torch.nan_to_num(b[key]))


def test_no_queries_at_all(lib):
    """Degenerate input: every segment is a cached prefix (no queries anywhere).  Forward has nothing to
    write; backward still owns the gradient pools and writes zeros to every slot of every page."""
    w = Workload("nq", [-1, 0], [200, 70], [64], 4, 2, 128, "bf16", seg_flags=[0, 2])
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    assert V["T_q"] == 0
    cap = V["pool_slots"] + 64
    q = torch.zeros(0, 4, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.randn(2, cap, 128, device="cuda").to(torch.bfloat16)
    v = torch.randn(2, cap, 128, device="cuda").to(torch.bfloat16)
    o, lse = lib.psrl_tree_attn_fwd(plan, q, k, v, 0.1)
    assert o.shape[0] == 0 and lib.psrl_device_status(plan, "fwd") == 0
    dk = torch.full_like(k, float("nan")); dv = torch.full_like(v, float("nan"))
    dq, dk, dv = lib.psrl_tree_attn_bwd(plan, q, k, v, o, lse, q, 0.1, dk_pool=dk, dv_pool=dv)
    assert lib.psrl_device_status(plan, "bwd") == 0
    tok, padm, outside = page_masks(V, cap)
    dkn, dvn = to_np(dk), to_np(dv)
    assert np.all(dkn[:, tok] == 0) and np.all(dvn[:, tok] == 0)
    assert np.all(dkn[:, padm] == 0) and np.all(dvn[:, padm] == 0)
    assert np.all(np.isnan(dkn[:, outside]))
