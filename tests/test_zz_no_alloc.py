"""psrl_tree_attn_bwd_static: the backward for callers that cannot allocate.

Some users of this library run where cudaMalloc is off limits (an allocation
synchronises the device, or the GPU memory belongs to someone else's pool), so
they cannot hand the regular backward its workspace.  The static variant keeps
that workspace inside the library image.  This test calls it through the C ABI
twice in a row (second call with a different upstream gradient, so leftovers of
the first call in the shared array would show) and checks each result against
the regular entry point on the same inputs: the two run the same kernels in
the same order, so the results must agree bit for bit (which is inside every
tolerance the other GPU tests use); the first call's result is also compared
with the fp64 oracle directly, at those tolerances.

The file name sorts last so that a run that stops at the first failure has
already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import oracle_attn
from paper_2608_25683_b200.workloads import Workload, make_inputs, make_workload

from util import build_plan, page_masks, rel_fro, to_np

pytestmark = pytest.mark.gpu


def _run_both(lib, w, seed):
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    cap = V["pool_slots"]
    q, k, v, d_o = make_inputs(V["T_q"], cap, V["tok_slot"], w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, seed,
                               device="cuda", pad="nan")
    o, lse = lib.psrl_tree_attn_fwd(plan, q, k, v, w.softmax_scale)
    tok, padm, _ = page_masks(V, cap)
    for call, grad in enumerate((d_o, (d_o * -0.5 + 0.25).to(d_o.dtype))):
        ref_dq, ref_dk, ref_dv = lib.psrl_tree_attn_bwd(plan, q, k, v, o, lse, grad, w.softmax_scale)
        assert lib.psrl_device_status(plan, "bwd") == 0
        # outputs are allocated here, by the test: the entry point itself allocates nothing
        dq = torch.full_like(q, float("nan"))
        dk = torch.full_like(k, float("nan"))
        dv = torch.full_like(v, float("nan"))
        ws = lib.psrl_tree_attn_bwd_static(plan, q, k, v, o, lse, grad, w.softmax_scale, dq, dk, dv)
        assert ws != 0
        assert lib.lib().psrl_device_status(ctypes.c_void_p(ws), None) == 0
        torch.cuda.synchronize()
        tok_t = torch.as_tensor(tok, device="cuda")
        assert torch.equal(dq, ref_dq), call
        assert torch.equal(dk[:, tok_t], ref_dk[:, tok_t]), call
        assert torch.equal(dv[:, tok_t], ref_dv[:, tok_t]), call
        assert np.all(to_np(dk)[:, padm] == 0) and np.all(to_np(dv)[:, padm] == 0)
        if call == 0:
            want = oracle_attn(V, to_np(q), to_np(k), to_np(v), to_np(grad), w.softmax_scale)
            if w.dtype == "f32":
                assert np.abs(to_np(dq) - want["dQ"]).max() <= 1e-5
                assert np.abs(to_np(dk)[:, tok] - want["dK"][:, tok]).max() <= 1e-5
                assert np.abs(to_np(dv)[:, tok] - want["dV"][:, tok]).max() <= 1e-5
            else:
                assert rel_fro(to_np(dq), want["dQ"]) <= 1e-2
                assert rel_fro(to_np(dk)[:, tok], want["dK"][:, tok]) <= 1e-2
                assert rel_fro(to_np(dv)[:, tok], want["dV"][:, tok]) <= 1e-2
    return plan


def test_static_backward_matches_regular_backward_bf16(lib):
    _run_both(lib, Workload("na", [-1, 0, 0, 1], [300, 140, 129, 60], [64], 4, 2, 128, "bf16"), seed=21)


def test_static_backward_matches_regular_backward_f32(lib):
    _run_both(lib, make_workload("c1", 0), seed=22)


def test_static_backward_with_split_tiles_and_partial_rows(lib):
    """Plans whose schedule needs the slabs of split KV tiles and partial dQ rows as well as D: all three
    live in the built-in array."""
    w = make_workload("c2s", 3)
    plan = _run_both(lib, w, seed=23)
    assert lib.psrl_launch_count(plan, True) >= 4
    assert plan.bwd_workspace_bytes() <= lib.BWD_STATIC_SCRATCH_BYTES


def test_static_backward_without_queries(lib):
    """A plan without any query row: the Q-shaped pointers may be NULL, as for the regular entry point;
    the gradient pools are still zeroed."""
    w = Workload("nq", [-1, 0], [200, 70], [64], 4, 2, 128, "bf16", seg_flags=[0, 2])
    plan = build_plan(lib, w)
    V = plan.oracle
    cap = V["pool_slots"]
    k = torch.randn(2, cap, 128, device="cuda").to(torch.bfloat16)
    v = torch.randn(2, cap, 128, device="cuda").to(torch.bfloat16)
    dk = torch.full_like(k, float("nan")); dv = torch.full_like(v, float("nan"))
    ws = ctypes.c_void_p()
    st = lib.lib().psrl_tree_attn_bwd_static(plan.handle, None, k.data_ptr(), v.data_ptr(), cap, None, None, None,
                                             None, dk.data_ptr(), dv.data_ptr(), 0.1, ctypes.byref(ws), None)
    assert lib.STATUS_NAMES[st] == "PSRL_OK"
    assert lib.lib().psrl_device_status(ws, None) == 0
    assert (dk == 0).all() and (dv == 0).all()


def test_size_limit_is_reported(lib):
    # 64 query heads x 70,000 rows = 4.48 M floats of D: over the 4,194,304 limit
    w = Workload("big", [-1], [70000], [256], 64, 8, 128, "bf16")
    plan = build_plan(lib, w)
    x = torch.zeros(1024, dtype=torch.bfloat16, device="cuda")
    ws = ctypes.c_void_p()
    st = lib.lib().psrl_tree_attn_bwd_static(plan.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                             plan.oracle["pool_slots"], x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                             x.data_ptr(), x.data_ptr(), x.data_ptr(), 1.0, ctypes.byref(ws), None)
    assert lib.STATUS_NAMES[st] == "PSRL_ERR_WORKSPACE"
    assert not ws.value
    # under the D limit (748,608 floats) but over the array's size once the slabs of its split KV tiles
    # are counted: the documented condition is bwd_workspace_bytes <= PSRL_BWD_STATIC_SCRATCH_BYTES
    w = make_workload("c3", 2000)
    plan = build_plan(lib, w)
    assert plan.oracle["T_q"] * w.n_q_heads < 4 * 1024 * 1024
    assert plan.bwd_workspace_bytes() > lib.BWD_STATIC_SCRATCH_BYTES
    st = lib.lib().psrl_tree_attn_bwd_static(plan.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                             plan.oracle["pool_slots"], x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                             x.data_ptr(), x.data_ptr(), x.data_ptr(), 1.0, ctypes.byref(ws), None)
    assert lib.STATUS_NAMES[st] == "PSRL_ERR_WORKSPACE"
    assert not ws.value
