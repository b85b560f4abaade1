"""psrl_tree_attn_bwd_static: the backward for callers that cannot allocate.

Some users of this library run where cudaMalloc is off limits (an allocation
synchronises the device, or the GPU memory belongs to someone else's pool), so
they cannot hand the regular backward its workspace.  The static variant keeps
that workspace inside the library image.  This test calls it through the C ABI
twice in a row (second call with a different upstream gradient, so leftovers of
the first call in the shared array would show) and checks each result against
the regular entry point on the same inputs, within the tolerances the other
GPU tests use (the two run the same kernels, so they agree bit for bit; the
assertion only requires the tolerance).

The file name sorts last so that a run that stops at the first failure has
already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2608_25683_b200.workloads import Workload, make_inputs, make_workload

from util import build_plan, page_masks, rel_fro, to_np

pytestmark = pytest.mark.gpu


def _run_both(lib, w, seed):
    plan = build_plan(lib, w)
    V = plan.view
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
        if w.dtype == "f32":
            assert np.abs(to_np(dq) - to_np(ref_dq)).max() <= 1e-5, call
            assert np.abs(to_np(dk)[:, tok] - to_np(ref_dk)[:, tok]).max() <= 1e-5, call
            assert np.abs(to_np(dv)[:, tok] - to_np(ref_dv)[:, tok]).max() <= 1e-5, call
        else:
            assert rel_fro(to_np(dq), to_np(ref_dq)) <= 1e-2, call
            assert rel_fro(to_np(dk)[:, tok], to_np(ref_dk)[:, tok]) <= 1e-2, call
            assert rel_fro(to_np(dv)[:, tok], to_np(ref_dv)[:, tok]) <= 1e-2, call
        assert np.all(to_np(dk)[:, padm] == 0) and np.all(to_np(dv)[:, padm] == 0)
    return plan


def test_static_backward_matches_regular_backward_bf16(lib):
    _run_both(lib, Workload("na", [-1, 0, 0, 1], [300, 140, 129, 60], [64], 4, 2, 128, "bf16"), seed=21)


def test_static_backward_matches_regular_backward_f32(lib):
    _run_both(lib, make_workload("c1", 0), seed=22)


def test_size_limit_is_reported(lib):
    # 64 query heads x 70,000 rows = 4.48 M floats of D: over the 4,194,304 limit
    w = Workload("big", [-1], [70000], [256], 64, 8, 128, "bf16")
    plan = build_plan(lib, w)
    x = torch.zeros(1024, dtype=torch.bfloat16, device="cuda")
    ws = ctypes.c_void_p()
    st = lib.lib().psrl_tree_attn_bwd_static(plan.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                             plan.view["pool_slots"], x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                             x.data_ptr(), x.data_ptr(), x.data_ptr(), 1.0, ctypes.byref(ws), None)
    assert lib.STATUS_NAMES[st] == "PSRL_ERR_WORKSPACE"
    assert not ws.value
