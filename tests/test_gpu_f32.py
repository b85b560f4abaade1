"""GPU parity, fp32 path: element by element against the fp64 oracle, max-abs 1e-5."""
import numpy as np
import pytest
import torch

from oracle import oracle_attn
from paper_2608_25683_b200.workloads import Workload, make_inputs, make_workload, random_forest

from util import build_plan, page_masks, run_gpu, to_np

pytestmark = pytest.mark.gpu
TOL = 1e-5  # max-abs bound for fp32 inputs, on O, dQ, dK, dV


def _check(lib, w, seed, pad="nan", extra_capacity=0):
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    cap = V["pool_slots"] + extra_capacity
    q, k, v, d_o = make_inputs(V["T_q"], cap, V["tok_slot"], w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, seed,
                               device="cuda", pad=pad)
    got = run_gpu(lib, plan, q, k, v, d_o, w.softmax_scale)
    want = oracle_attn(V, to_np(q), to_np(k), to_np(v), to_np(d_o), w.softmax_scale)
    tok, padm, outside = page_masks(V, cap)
    assert np.abs(to_np(got["O"]) - want["O"]).max() <= TOL
    assert np.abs(to_np(got["LSE"]) - want["LSE"]).max() <= TOL
    assert np.abs(to_np(got["dQ"]) - want["dQ"]).max() <= TOL
    dk, dv = to_np(got["dK"]), to_np(got["dV"])
    assert np.abs(dk[:, tok] - want["dK"][:, tok]).max() <= TOL
    assert np.abs(dv[:, tok] - want["dV"][:, tok]).max() <= TOL
    # pad slots of pages are written as zeros; slots outside the plan's pages are untouched (still NaN)
    assert np.all(dk[:, padm] == 0) and np.all(dv[:, padm] == 0)
    assert np.all(np.isnan(dk[:, outside])) and np.all(np.isnan(dv[:, outside]))
    return plan, (q, k, v, d_o), got


def test_c1_tiny_tree(lib):
    _check(lib, make_workload("c1", 0), seed=1000)
    _check(lib, make_workload("c1", 0), seed=1001, pad="normal")


@pytest.mark.parametrize("d", [64, 128])
def test_random_forests(lib, d):
    rng = np.random.default_rng(5 + d)
    for i in range(6):
        n_roots = int(rng.integers(1, 4))
        parent, seg_len, gbs, flags = random_forest(rng, int(rng.integers(n_roots, 12)), 150, n_roots,
                                                    cached_roots=(i % 3 == 0), step_samples=(i % 3 == 1))
        w = Workload("rnd", parent, seg_len, gbs, 4, 2, d, "f32", seg_flags=flags)
        _check(lib, w, seed=i, extra_capacity=48)


def test_single_token_and_ragged_edges(lib):
    _check(lib, Workload("one", [-1], [1], [16], 1, 1, 64, "f32"), seed=3)
    _check(lib, Workload("ragged", [-1, 0, 1, 1], [129, 1, 17, 255], [64], 2, 1, 64, "f32"), seed=4)


def test_fragmented_pool(lib):
    w = Workload("frag", [-1, 0, 0], [100, 40, 7], [16], 2, 2, 64, "f32",
                 free_extents=[(512, 64), (0, 32), (128, 96), (1024, 256)])
    _check(lib, w, seed=5, extra_capacity=64)


def test_runs_are_bitwise_reproducible(lib):
    w = make_workload("c1", 0)
    plan, (q, k, v, d_o), a = _check(lib, w, seed=7)
    b = run_gpu(lib, plan, q, k, v, d_o, w.softmax_scale)
    for key in ("O", "LSE", "dQ"):
        assert torch.equal(a[key], b[key])
    for key in ("dK", "dV"):
        assert torch.equal(torch.nan_to_num(a[key]), torch.nan_to_num(b[key]))
