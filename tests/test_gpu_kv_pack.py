"""K/V scatter into the paged pools and gather back: byte-exact against plain indexing by tok_slot."""
import numpy as np
import pytest
import torch

from paper_2608_25683_b200.workloads import Workload, make_workload

from util import build_plan

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_scatter_gather_bit_exact(lib, dtype, d):
    w = Workload("p", [-1, 0, 0, -1, 3], [333, 200, 45, 17, 129], [64, 16], 4, 2, d, dtype,
                 free_extents=[(2048, 512), (0, 160), (512, 1024), (4096, 1024)])
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    T, cap = V["T"], 6000
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    g = torch.Generator(device="cuda").manual_seed(5)
    k_tok = torch.randn(T, 2, d, device="cuda", generator=g).to(tdt)
    v_tok = torch.randn(T, 2, d, device="cuda", generator=g).to(tdt)
    k_pool = torch.full((2, cap, d), float("nan"), device="cuda", dtype=tdt)
    v_pool = torch.full_like(k_pool, float("nan"))
    lib.psrl_kv_scatter(plan, k_tok, v_tok, k_pool, v_pool)
    torch.cuda.synchronize()
    slots = torch.as_tensor(V["tok_slot"].astype(np.int64), device="cuda")
    assert torch.equal(k_pool[:, slots].transpose(0, 1), k_tok) and torch.equal(v_pool[:, slots].transpose(0, 1), v_tok)
    untouched = torch.ones(cap, dtype=torch.bool, device="cuda")
    untouched[slots] = False
    assert torch.isnan(k_pool[:, untouched]).all() and torch.isnan(v_pool[:, untouched]).all()
    k2, v2 = lib.psrl_kv_gather(plan, k_pool, v_pool)
    torch.cuda.synchronize()
    assert torch.equal(k2, k_tok) and torch.equal(v2, v_tok)


def test_full_size_roundtrip_and_bandwidth(lib):
    w = make_workload("c5", 1)
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    T, cap = V["T"], V["pool_slots"]
    k_tok = torch.randn(T, w.n_kv_heads, 128, device="cuda").to(torch.bfloat16)
    v_tok = torch.randn(T, w.n_kv_heads, 128, device="cuda").to(torch.bfloat16)
    k_pool = torch.zeros(w.n_kv_heads, cap, 128, device="cuda", dtype=torch.bfloat16)
    v_pool = torch.zeros_like(k_pool)
    lib.psrl_kv_scatter(plan, k_tok, v_tok, k_pool, v_pool)
    k2, v2 = lib.psrl_kv_gather(plan, k_pool, v_pool)
    torch.cuda.synchronize()
    assert torch.equal(k2, k_tok) and torch.equal(v2, v_tok)
