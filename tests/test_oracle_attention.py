"""Pins for the attention oracle: finite differences, copy invariants, library
special cases (torch CPU fp64 SDPA + autograd), closed forms, dO split."""
import numpy as np
import pytest
import torch

from oracle import oracle_plan, oracle_attn, oracle_rows, sample_paths
from paper_2608_25683_b200.workloads import random_forest


def _inputs(p, Hq, Hkv, d, seed, pad_nan=True):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((p["T_q"], Hq, d))
    d_o = rng.standard_normal((p["T_q"], Hq, d))
    k = rng.standard_normal((Hkv, p["pool_slots"], d))
    v = rng.standard_normal((Hkv, p["pool_slots"], d))
    return q, k, v, d_o


def _tree_mask(p):
    """Boolean [T_q, T]: which token each query row may attend to (built from
    parent links only, token by token)."""
    n = p["n_seg"]
    vis = np.zeros((p["T_q"], p["T"]), dtype=bool)
    for c in range(n):
        if p["seg_q_off"][c] < 0:
            continue
        for i in range(p["seg_len"][c]):
            r = p["seg_q_off"][c] + i
            a = p["seg_parent"][c]
            while a != -1:
                vis[r, p["seg_tok_off"][a]:p["seg_tok_off"][a] + p["seg_len"][a]] = True
                a = p["seg_parent"][a]
            vis[r, p["seg_tok_off"][c]:p["seg_tok_off"][c] + i + 1] = True
    return vis


def _torch_reference(p, q, k, v, d_o, scale, Hq, Hkv):
    """Dense attention over the packed tree tokens with an explicit tree mask,
    evaluated by torch's SDPA in fp64 with autograd."""
    G = Hq // Hkv
    slots = torch.as_tensor(p["tok_slot"].astype(np.int64))
    tq = torch.tensor(q, dtype=torch.float64, requires_grad=True)          # [T_q,Hq,d]
    tk = torch.tensor(k, dtype=torch.float64, requires_grad=True)          # pools
    tv = torch.tensor(v, dtype=torch.float64, requires_grad=True)
    K = tk[:, slots, :].repeat_interleave(G, dim=0)                        # [Hq,T,d]
    V = tv[:, slots, :].repeat_interleave(G, dim=0)
    Q = tq.permute(1, 0, 2)                                                # [Hq,T_q,d]
    mask = torch.as_tensor(_tree_mask(p))
    O = torch.nn.functional.scaled_dot_product_attention(
        Q[None], K[None], V[None], attn_mask=mask[None, None], scale=scale)[0]
    O = O.permute(1, 0, 2)
    O.backward(torch.tensor(d_o, dtype=torch.float64))
    return O.detach().numpy(), tq.grad.numpy(), tk.grad.numpy(), tv.grad.numpy()


CASES = [
    # parent, seg_len, gbs, flags, Hq, Hkv, d
    ([-1], [9], [16], None, 2, 1, 4),                                   # plain causal sequence
    ([-1, 0, 0], [3, 2, 2], [16], None, 2, 1, 4),                       # prefix 3 + branches 2, 2
    ([-1, 0, 0, 1, 1], [5, 3, 4, 2, 6], [16], None, 4, 2, 8),           # two levels
    ([-1, 0, 0, -1, 3], [20, 7, 18, 5, 33], [16, 32], None, 2, 2, 8),   # forest, pages with pads
    ([-1, 0, 0], [6, 3, 4], [16], [0, 3, 3], 2, 1, 4),                  # cached prefix (no root queries)
    ([-1, 0, 1], [4, 3, 5], [16], [3, 3, 3], 2, 1, 4),                  # step mode: every node a sample
]


@pytest.mark.parametrize("case", CASES)
def test_matches_torch_sdpa_with_tree_mask(case):
    parent, seg_len, gbs, flags, Hq, Hkv, d = case
    p = oracle_plan(parent, seg_len, gbs, flags)
    q, k, v, d_o = _inputs(p, Hq, Hkv, d, 1)
    scale = 0.37
    out = oracle_attn(p, q, k, v, d_o, scale)
    O, dQ, dK, dV = _torch_reference(p, q, k, v, d_o, scale, Hq, Hkv)
    assert np.abs(out["O"] - O).max() < 1e-12
    assert np.abs(out["dQ"] - dQ).max() < 1e-11
    assert np.abs(out["dK"] - dK).max() < 1e-11
    assert np.abs(out["dV"] - dV).max() < 1e-11
    # pad slots and unused slots get no gradient
    used = np.zeros(p["pool_slots"], dtype=bool)
    used[p["tok_slot"]] = True
    assert np.all(out["dK"][:, ~used] == 0) and np.all(out["dV"][:, ~used] == 0)


def test_single_sequence_is_textbook_causal_attention():
    p = oracle_plan([-1], [37], [16])
    q, k, v, d_o = _inputs(p, 2, 2, 8, 3)
    out = oracle_attn(p, q, k, v, d_o, 0.5)
    Q = torch.tensor(q).permute(1, 0, 2)[None]
    K = torch.tensor(k[:, p["tok_slot"]])[None]
    V = torch.tensor(v[:, p["tok_slot"]])[None]
    O = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True, scale=0.5)[0]
    assert np.abs(out["O"] - O.permute(1, 0, 2).numpy()).max() < 1e-12
    # LSE against a direct evaluation
    S = 0.5 * np.einsum("ihd,hjd->hij", q, k[:, p["tok_slot"]])
    S[:, np.triu(np.ones((37, 37), dtype=bool), 1)] = -np.inf
    assert np.abs(out["LSE"] - np.log(np.exp(S).sum(-1))).max() < 1e-12


@pytest.mark.parametrize("case", CASES[1:4])
def test_finite_differences(case):
    parent, seg_len, gbs, flags, Hq, Hkv, d = case
    p = oracle_plan(parent, seg_len, gbs, flags)
    q, k, v, d_o = _inputs(p, Hq, Hkv, d, 5)
    scale = 0.6
    base = oracle_attn(p, q, k, v, d_o, scale)

    def f(q_, k_, v_):
        return float((oracle_attn(p, q_, k_, v_, None, scale)["O"] * d_o).sum())

    rng = np.random.default_rng(0)
    h = 1e-6
    for name, arr, grad in (("q", q, base["dQ"]), ("k", k, base["dK"]), ("v", v, base["dV"])):
        idxs = list(np.ndindex(arr.shape))
        if name != "q":  # only slots that hold a token matter; check a few pads too
            used = set(p["tok_slot"].tolist())
            idxs = [i for i in idxs if i[1] in used] + [i for i in idxs if i[1] not in used][:3]
        pick = rng.choice(len(idxs), size=min(60, len(idxs)), replace=False)
        for t in pick:
            i = idxs[t]
            a = arr.copy(); a[i] += h
            b = arr.copy(); b[i] -= h
            args_p = dict(q=q, k=k, v=v); args_m = dict(q=q, k=k, v=v)
            args_p[name] = a; args_m[name] = b
            num = (f(args_p["q"], args_p["k"], args_p["v"]) - f(args_m["q"], args_m["k"], args_m["v"])) / (2 * h)
            assert abs(num - grad[i]) <= 1e-6 * max(1.0, abs(grad[i])), (name, i, num, grad[i])


@pytest.mark.parametrize("case", CASES[1:])
def test_copies_of_a_shared_token_agree_and_split_is_irrelevant(case):
    parent, seg_len, gbs, flags, Hq, Hkv, d = case
    p = oracle_plan(parent, seg_len, gbs, flags)
    q, k, v, d_o = _inputs(p, Hq, Hkv, d, 9)
    out = oracle_attn(p, q, k, v, d_o, 0.4, want_copies=True)
    # every copy of a shared token computes the same O and LSE as the recorded one
    n_copies = np.zeros(p["T_q"], dtype=int)
    for _k, h, rows, Oc, Lc in out["copies"]:
        assert np.abs(Oc - out["O"][rows, h]).max() < 1e-12
        assert np.abs(Lc - out["LSE"][h, rows]).max() < 1e-12
        if h == 0:
            n_copies[rows] += 1
    # number of copies of a query row = reference count of its segment
    for c in range(p["n_seg"]):
        if p["seg_q_off"][c] >= 0:
            r0 = p["seg_q_off"][c]
            assert np.all(n_copies[r0:r0 + p["seg_len"][c]] == p["seg_refcount"][c])
    # a random split of dO over the copies gives the same gradients
    rng = np.random.default_rng(2)
    paths = sample_paths(p)
    tok_lists = []
    for path in paths:
        toks = []
        for c in path:
            toks.extend(range(p["seg_tok_off"][c], p["seg_tok_off"][c] + p["seg_len"][c]))
        tok_lists.append(np.asarray(toks))
    raw = [rng.random(len(t)) + 0.1 for t in tok_lists]
    total = np.zeros(p["T"])
    for t, r in zip(tok_lists, raw):
        np.add.at(total, t, r)
    weights = [r / total[t] for t, r in zip(tok_lists, raw)]
    out2 = oracle_attn(p, q, k, v, d_o, 0.4, do_weights=weights)
    for key in ("dQ", "dK", "dV"):
        assert np.abs(out[key] - out2[key]).max() < 1e-12


def test_closed_forms():
    p = oracle_plan([-1, 0, 0], [11, 6, 9], [16])
    Hq, Hkv, d = 4, 2, 8
    q, k, v, d_o = _inputs(p, Hq, Hkv, d, 11)
    scale = 0.3
    # (a) all visible keys equal -> uniform P: O = mean of visible V, LSE = s + ln n, dQ = 0
    k_eq = np.broadcast_to(k[:, :1, :], k.shape).copy()
    out = oracle_attn(p, q, k_eq, v, d_o, scale)
    vis = np.zeros((p["T_q"], p["T"]), dtype=bool)
    vis[:] = _tree_mask(p)
    vt = v[:, p["tok_slot"]]
    for r in range(p["T_q"]):
        nvis = vis[r].sum()
        for h in range(Hq):
            assert np.abs(out["O"][r, h] - vt[h // 2][vis[r]].mean(0)).max() < 1e-12
            s = scale * float(q[r, h] @ k_eq[h // 2, 0])
            assert abs(out["LSE"][h, r] - (s + np.log(nvis))) < 1e-12
    assert np.abs(out["dQ"]).max() < 1e-12
    # (b) V constant per head -> O equals that constant
    v_c = np.broadcast_to(v[:, :1, :], v.shape).copy()
    out = oracle_attn(p, q, k, v_c, d_o, scale)
    for h in range(Hq):
        assert np.abs(out["O"][:, h] - v_c[h // 2, 0]).max() < 1e-12
    # (c) adding a constant vector to every key leaves O, dV unchanged and LSE shifts by scale*q.c
    cvec = np.random.default_rng(1).standard_normal(d)
    base = oracle_attn(p, q, k, v, d_o, scale)
    sh = oracle_attn(p, q, k + cvec, v, d_o, scale)
    assert np.abs(base["O"] - sh["O"]).max() < 1e-11
    assert np.abs(base["dV"] - sh["dV"]).max() < 1e-11
    assert np.abs((sh["LSE"] - base["LSE"]).T - scale * (q @ cvec)).max() < 1e-11
    # (d) per KV head, sum over tokens of dV = sum over its query heads and rows of dO
    for hk in range(Hkv):
        want = d_o[:, hk * 2:(hk + 1) * 2].sum(axis=(0, 1))
        assert np.abs(base["dV"][hk].sum(0) - want).max() < 1e-10
    # (e) rows of dS sum to zero  <=>  dQ is orthogonal to nothing in general, but
    #     with all keys equal to kk, dQ = scale * (sum_j dS_ij) kk = 0: checked in (a)
    # (f) log-sum-exp merge of a two-way key split equals the unsplit result
    qv = q[p["seg_q_off"][2] + 4, 1]
    O_full, L_full = oracle_rows(p, [qv], k, v, [p["seg_q_off"][2] + 4], [1], Hq, scale)
    toks = list(range(0, 11)) + list(range(p["seg_tok_off"][2], p["seg_tok_off"][2] + 5))
    sl = p["tok_slot"][toks]
    s_all = scale * (k[0, sl] @ qv)
    parts = []
    for idx in (slice(0, 7), slice(7, None)):
        s_ = s_all[idx]
        e = np.exp(s_ - s_.max())
        parts.append(((e / e.sum()) @ v[0, sl][idx], s_.max() + np.log(e.sum())))
    L = np.logaddexp(parts[0][1], parts[1][1])
    O = np.exp(parts[0][1] - L) * parts[0][0] + np.exp(parts[1][1] - L) * parts[1][0]
    assert abs(L - L_full[0]) < 1e-12 and np.abs(O - O_full[0]).max() < 1e-12
    assert np.abs(O_full[0] - base["O"][p["seg_q_off"][2] + 4, 1]).max() < 1e-12


def test_row_subset_is_exact_when_other_do_rows_are_zero():
    rng = np.random.default_rng(4)
    parent, seg_len, gbs, flags = random_forest(rng, 7, 25, 2)
    p = oracle_plan(parent, seg_len, gbs, flags)
    q, k, v, d_o = _inputs(p, 4, 2, 8, 6)
    rows = np.sort(rng.choice(p["T_q"], size=9, replace=False))
    d_sparse = np.zeros_like(d_o)
    d_sparse[rows] = d_o[rows]
    full = oracle_attn(p, q, k, v, d_sparse, 0.25)
    sub = oracle_attn(p, q[rows], k, v, d_sparse[rows], 0.25, q_rows=rows)
    assert np.abs(full["dK"] - sub["dK"]).max() < 1e-12
    assert np.abs(full["dV"] - sub["dV"]).max() < 1e-12
    assert np.abs(full["dQ"][rows] - sub["dQ"]).max() < 1e-12
    assert np.abs(full["O"][rows] - sub["O"]).max() < 1e-12
    # and a KV-head subset leaves the evaluated heads unchanged
    one = oracle_attn(p, q, k, v, d_o, 0.25, kv_heads=[1])
    allh = oracle_attn(p, q, k, v, d_o, 0.25)
    assert np.abs(one["dK"][1] - allh["dK"][1]).max() == 0
    assert np.abs(one["O"][:, 2:] - allh["O"][:, 2:]).max() == 0


def test_pad_slots_never_reach_an_output():
    p = oracle_plan([-1, 0, 0], [20, 5, 7], [16])
    q, k, v, d_o = _inputs(p, 2, 1, 4, 8)
    used = np.zeros(p["pool_slots"], dtype=bool)
    used[p["tok_slot"]] = True
    k2, v2 = k.copy(), v.copy()
    k2[:, ~used] = np.nan
    v2[:, ~used] = np.nan
    a = oracle_attn(p, q, k, v, d_o, 0.5)
    b = oracle_attn(p, q, k2, v2, d_o, 0.5)
    for key in ("O", "LSE", "dQ", "dK", "dV"):
        assert np.array_equal(a[key], b[key])
