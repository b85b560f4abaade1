"""Shared helpers of the GPU parity tests (no arithmetic of the method here)."""
import numpy as np
import torch

from oracle import oracle_attn, oracle_plan
from oracle.plan import PLAN_ARRAYS, PLAN_SCALARS
from paper_2608_25683_b200.workloads import make_inputs


def checked_oracle_plan(view, parent, seg_len, group_block_size, seg_flags=None, free_extents=None,
                        seg_slot_base=None):
    """The plan of this forest built by the ORACLE, after asserting that the library's view of its own
    plan equals it byte for byte.  Parity tests hand this one to oracle_attn, so the checker never
    reads an index (tok_slot, anc_list, seg_q_off ...) that the product computed."""
    want = oracle_plan(parent, seg_len, group_block_size, seg_flags, free_extents, seg_slot_base)
    for key in PLAN_SCALARS:
        assert view[key] == want[key], key
    for key in PLAN_ARRAYS:
        assert view[key].dtype == np.int32 and want[key].dtype == np.int32, key
        assert view[key].tobytes() == want[key].tobytes(), key
    return want


def build_plan(lib, w, upload=True):
    """The library's plan of workload `w`; `plan.oracle` is the oracle's plan of the same forest."""
    plan = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                    w.seg_flags, w.free_extents)
    plan.oracle = checked_oracle_plan(plan.view, w.parent, w.seg_len, w.group_block_size, w.seg_flags, w.free_extents)
    if upload:
        plan.upload()
    return plan


def run_gpu(lib, plan, q, k, v, d_o, scale, backward=True):
    o, lse = lib.psrl_tree_attn_fwd(plan, q, k, v, scale)
    assert lib.psrl_device_status(plan, "fwd") == 0
    out = dict(O=o, LSE=lse)
    if backward:
        # poison the gradient pools: the library must overwrite every slot of every page
        dk = torch.full_like(k, float("nan"))
        dv = torch.full_like(v, float("nan"))
        dq, dk, dv = lib.psrl_tree_attn_bwd(plan, q, k, v, o, lse, d_o, scale, dk_pool=dk, dv_pool=dv)
        assert lib.psrl_device_status(plan, "bwd") == 0
        out.update(dQ=dq, dK=dk, dV=dv)
    torch.cuda.synchronize()
    return out


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def page_masks(view, capacity):
    """(token slots, pad slots of pages, slots outside every page) as boolean arrays."""
    tok = np.zeros(capacity, dtype=bool)
    tok[view["tok_slot"]] = True
    page = np.zeros(capacity, dtype=bool)
    for s, b in zip(view["page_slot"], view["page_bs"]):
        page[s:s + b] = True
    return tok, page & ~tok, ~page


def rel_fro(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))
