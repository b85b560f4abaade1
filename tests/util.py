"""Shared helpers of the GPU parity tests (no arithmetic of the method here)."""
import numpy as np
import torch

from oracle import oracle_attn
from paper_2608_25683_b200.workloads import make_inputs


def build_plan(lib, w, upload=True):
    plan = lib.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                    w.seg_flags, w.free_extents)
    if upload:
        plan.upload()
    return plan


def oracle_view(view):
    """The oracle functions take the plan as a dict of numpy arrays; the C++ plan
    is bit-identical to the oracle's (tests/test_plan_builder.py), so its view serves."""
    return view


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
