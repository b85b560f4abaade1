"""GPU parity at the benchmark's full sizes (c2-c5), in the launch configuration
bench.py times.

c2 and c3 (dense): dO is dense on every head, as in the benchmark.  One seeded
KV head - all rows of all its query heads, every sample - is evaluated by the
oracle in full (heads are independent, so this is exact), which checks O and
LSE on every row and dQ, dK, dV element by element; in particular the prefix's
dK/dV summed over all branches (Sec. 6) with every split part and slab of the
full-size schedule contributing.

c4 and c5 (too large for a dense oracle pass): dO is non-zero on sampled rows
only.  Every other dO row contributes exactly nothing, so the oracle's
evaluation of just those rows gives the exact dQ (sampled rows), dK and dV (all
tokens) of one KV head; every other dQ row must be exactly zero.  The rows are
drawn from EVERY segment and every 128-row block of it (first, second, middle,
last row of the segment, the rows on either side of the first tile edge, and one
random row per block), so every work item and every split part of the three
kernels has a sampled row.

All configurations: properties that hold at any size - finite outputs, zero pads,
untouched slots outside the plan's pages, per-head sum of dV = sum of dO."""
import numpy as np
import pytest
import torch

from oracle import oracle_attn
from paper_2608_25683_b200.workloads import make_inputs, make_workload

from util import build_plan, page_masks, rel_fro, to_np

pytestmark = pytest.mark.gpu


def sample_rows(V, rng):
    rows = set()
    for c in range(V["n_seg"]):
        if V["seg_q_off"][c] < 0:
            continue
        n, q0 = int(V["seg_len"][c]), int(V["seg_q_off"][c])
        cand = [0, 1, 127, 128, n // 2, n - 1]
        cand += [b + int(rng.integers(0, min(128, n - b))) for b in range(0, n, 128)]
        rows.update(q0 + i for i in cand if 0 <= i < n)
    return np.array(sorted(rows), dtype=np.int64)


def run(lib, w, plan, V, sparse_rows):
    cap = V["pool_slots"]
    if w.free_extents:
        cap = max(cap, max(a + c for a, c in w.free_extents))
    q, k, v, d_o = make_inputs(V["T_q"], cap, V["tok_slot"], w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, 77,
                               device="cuda", pad="nan", sparse_do_rows=sparse_rows)
    o, lse = lib.psrl_tree_attn_fwd(plan, q, k, v, w.softmax_scale)
    assert lib.psrl_device_status(plan, "fwd") == 0
    dk = torch.full_like(k, float("nan"))
    dv = torch.full_like(v, float("nan"))
    dq, dk, dv = lib.psrl_tree_attn_bwd(plan, q, k, v, o, lse, d_o, w.softmax_scale, dk_pool=dk, dv_pool=dv)
    assert lib.psrl_device_status(plan, "bwd") == 0
    return cap, (q, k, v, d_o), (o, lse, dq, dk, dv)


def check_properties(w, V, cap, d_o, o, lse, dq, dk, dv):
    G = w.n_q_heads // w.n_kv_heads
    tok, padm, outside = page_masks(V, cap)
    assert torch.isfinite(o).all() and torch.isfinite(lse).all() and torch.isfinite(dq).all()
    tok_t = torch.as_tensor(tok, device="cuda")
    assert torch.isfinite(dk[:, tok_t]).all() and torch.isfinite(dv[:, tok_t]).all()
    assert (dk[:, torch.as_tensor(padm, device="cuda")] == 0).all()
    assert (dv[:, torch.as_tensor(padm, device="cuda")] == 0).all()
    assert torch.isnan(dk[:, torch.as_tensor(outside, device="cuda")]).all()
    assert torch.isnan(dv[:, torch.as_tensor(outside, device="cuda")]).all()
    # per KV head: sum over tokens of dV = sum over its query heads and rows of dO
    sum_dv = dv[:, tok_t].double().sum(dim=1)                                      # [Hkv, d]
    sum_do = d_o.double().sum(dim=0).view(w.n_kv_heads, G, w.head_dim).sum(dim=1)   # [Hkv, d]
    # dV is rounded to bf16 per token (relative 2^-9): the sum of T rounding errors of magnitude
    # ~2^-9 |dV| grows like sqrt(T)
    bound = 2e-2 * max(1.0, sum_do.abs().max().item()) + 2.0 ** -9 * float(np.sqrt(V["T"])) * 8
    assert (sum_dv - sum_do).abs().max().item() <= bound
    return tok


@pytest.mark.parametrize("name", ["c2", "c3"])
def test_full_size_dense(lib, name):
    w = make_workload(name, 2000)
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    cap, (q, k, v, d_o), (o, lse, dq, dk, dv) = run(lib, w, plan, V, None)
    tok = check_properties(w, V, cap, d_o, o, lse, dq, dk, dv)
    G = w.n_q_heads // w.n_kv_heads
    hk = int(np.random.default_rng(5).integers(0, w.n_kv_heads))
    hs = slice(hk * G, (hk + 1) * G)
    want = oracle_attn(V, to_np(q[:, hs]), to_np(k[hk:hk + 1]), to_np(v[hk:hk + 1]), to_np(d_o[:, hs]),
                       w.softmax_scale)
    assert np.abs(to_np(o[:, hs]) - want["O"]).max() <= 1e-2
    assert np.abs(to_np(lse[hs]) - want["LSE"]).max() <= 1e-2
    assert rel_fro(to_np(dq[:, hs]), want["dQ"]) <= 1e-2
    dk_h, dv_h = to_np(dk[hk]), to_np(dv[hk])
    assert rel_fro(dk_h[tok], want["dK"][0][tok]) <= 1e-2
    assert rel_fro(dv_h[tok], want["dV"][0][tok]) <= 1e-2
    # segment by segment as well: a fault confined to one short segment must not hide in the global norm
    for c in range(V["n_seg"]):
        t0, n, q0 = int(V["seg_tok_off"][c]), int(V["seg_len"][c]), int(V["seg_q_off"][c])
        slots = V["tok_slot"][t0:t0 + n].astype(np.int64)
        assert rel_fro(dk_h[slots], want["dK"][0][slots]) <= 2e-2, c
        assert rel_fro(dv_h[slots], want["dV"][0][slots]) <= 2e-2, c
        assert rel_fro(to_np(dq[q0:q0 + n, hs]), want["dQ"][q0:q0 + n]) <= 2e-2, c


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_full_size_sampled(lib, name):
    w = make_workload(name, 2000)
    plan = build_plan(lib, w)
    V = plan.oracle   # the oracle's own plan (asserted byte-equal to the library's view)
    rng = np.random.default_rng(5)
    rows = sample_rows(V, rng)
    cap, (q, k, v, d_o), (o, lse, dq, dk, dv) = run(lib, w, plan, V, rows)
    tok = check_properties(w, V, cap, d_o, o, lse, dq, dk, dv)
    G = w.n_q_heads // w.n_kv_heads
    hk = int(rng.integers(0, w.n_kv_heads))
    hs = slice(hk * G, (hk + 1) * G)
    rows_t = torch.as_tensor(rows, device="cuda")
    want = oracle_attn(V, to_np(q[rows_t][:, hs]), to_np(k[hk:hk + 1]), to_np(v[hk:hk + 1]),
                       to_np(d_o[rows_t][:, hs]), w.softmax_scale, q_rows=rows)
    assert np.abs(to_np(o[rows_t][:, hs]) - want["O"]).max() <= 1e-2
    assert np.abs(to_np(lse[hs][:, rows_t]) - want["LSE"]).max() <= 1e-2
    assert rel_fro(to_np(dq[rows_t][:, hs]), want["dQ"]) <= 1e-2
    dk_h, dv_h = to_np(dk[hk]), to_np(dv[hk])
    assert rel_fro(dk_h[tok], want["dK"][0][tok]) <= 1e-2
    assert rel_fro(dv_h[tok], want["dV"][0][tok]) <= 1e-2
    other = torch.ones(V["T_q"], dtype=torch.bool, device="cuda")
    other[rows_t] = False
    assert (dq[other] == 0).all(), "rows with zero dO must get exactly zero dQ"
