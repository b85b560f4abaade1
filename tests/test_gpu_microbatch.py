"""GPU parity of multi-micro-batch execution (paper Sec. 4.1 inter-batch / self-sequence sharing with
the Dynamic Block Caching manager of Sec. 5.2): a forest is computed over several attention calls;
prefixes computed by an earlier micro-batch are read in place (no queries), their dK/dV contributions
are summed over the micro-batches (one accumulated backward on the shared prefix, Sec. 6).  The
result must equal the oracle's single evaluation of the whole forest."""
import numpy as np
import pytest
import torch

from oracle import oracle_attn

from util import checked_oracle_plan, rel_fro, to_np

pytestmark = pytest.mark.gpu
Hq, Hkv, D = 4, 2, 128


def run_forest(lib, parent, seg_len, gbs, mb, M, cap=0, seed=0, origin=None):
    """Runs the forest (parent, seg_len, gbs) as M attention calls, segment s in micro-batch mb[s], and
    compares with the oracle's single evaluation.  With origin = (parent, seg_len, gbs, piece_seg,
    piece_begin) the forest is a forest of PIECES of that original forest (piece i = tokens
    [piece_begin[i], piece_begin[i] + seg_len[i]) of original segment piece_seg[i]): the data are drawn
    per original segment, and the oracle evaluates the original, uncut forest."""
    n = len(parent)
    if origin is None:
        o_parent, o_len, o_gbs, piece_seg, piece_begin = parent, seg_len, gbs, list(range(n)), [0] * n
    else:
        o_parent, o_len, o_gbs, piece_seg, piece_begin = origin
    g = torch.Generator(device="cpu").manual_seed(seed)
    rnd = lambda *shape: torch.randn(*shape, generator=g).to(torch.bfloat16)
    Ko = [rnd(Hkv, l, D) for l in o_len]
    Vo = [rnd(Hkv, l, D) for l in o_len]
    Qo = [rnd(l, Hq, D) for l in o_len]
    Go = [rnd(l, Hq, D) for l in o_len]
    cut = lambda X, i, axis: X[piece_seg[i]].narrow(axis, piece_begin[i], seg_len[i])
    Kseg = [cut(Ko, i, 1) for i in range(n)]
    Vseg = [cut(Vo, i, 1) for i in range(n)]
    Qseg = [cut(Qo, i, 0) for i in range(n)]
    Gseg = [cut(Go, i, 0) for i in range(n)]
    scale = 1.0 / np.sqrt(D)

    # ---- the whole (original) forest in one evaluation by the oracle ----
    full = lib.Plan(o_parent, o_len, o_gbs, Hq, Hkv, D, "bf16")
    V = checked_oracle_plan(full.view, o_parent, o_len, o_gbs)   # the oracle's own plan of the whole forest
    q = torch.zeros(V["T_q"], Hq, D, dtype=torch.bfloat16)
    d_o = torch.zeros_like(q)
    k = torch.zeros(Hkv, V["pool_slots"], D, dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    for s in range(len(o_parent)):
        c = int(V["canon_of_input"][s])
        r0, t0 = int(V["seg_q_off"][c]), int(V["seg_tok_off"][c])
        q[r0:r0 + o_len[s]] = Qo[s]
        d_o[r0:r0 + o_len[s]] = Go[s]
        slots = torch.as_tensor(V["tok_slot"][t0:t0 + o_len[s]].astype(np.int64))
        k[:, slots] = Ko[s]
        v[:, slots] = Vo[s]
    want = oracle_attn(V, to_np(q), to_np(k), to_np(v), to_np(d_o), scale)

    # ---- the same over M attention calls ----
    cache = lib.Cache(parent, seg_len, gbs, mb, M, capacity_slots=cap)
    arena_slots = cap if cap else cache.stats()["total_slots"]
    dev = "cuda"
    K = torch.full((Hkv, arena_slots, D), float("nan"), dtype=torch.bfloat16, device=dev)
    Vp = torch.full_like(K, float("nan"))
    got_O = [None] * n; got_L = [None] * n; got_dQ = [None] * n
    dK = [torch.zeros(Hkv, l, D, dtype=torch.float64) for l in seg_len]
    dV = [torch.zeros(Hkv, l, D, dtype=torch.float64) for l in seg_len]
    saved = {}
    events = dict(evict=0, reload=0)
    for m in range(M):
        step = cache.begin(m)
        ext = lambda s: -(-seg_len[s] // gbs_of[s]) * gbs_of[s]
        for s, old in step["evict"]:                       # offload before anything overwrites it
            saved[s] = (K[:, old:old + seg_len[s]].clone(), Vp[:, old:old + seg_len[s]].clone())
            K[:, old:old + ext(s)] = float("nan"); Vp[:, old:old + ext(s)] = float("nan")
            events["evict"] += 1
        base_of = dict(zip(step["seg_id"], step["seg_slot_base"]))
        for s in step["reload"]:
            K[:, base_of[s]:base_of[s] + seg_len[s]], Vp[:, base_of[s]:base_of[s] + seg_len[s]] = saved.pop(s)
            events["reload"] += 1
        for s in step["new"]:                              # this micro-batch produces the segment's K/V
            K[:, base_of[s]:base_of[s] + seg_len[s]] = Kseg[s].to(dev)
            Vp[:, base_of[s]:base_of[s] + seg_len[s]] = Vseg[s].to(dev)
        plan = lib.Plan(step["parent"], step["seg_len"], step["group_block_size"], Hq, Hkv, D, "bf16",
                        seg_flags=step["seg_flags"], seg_slot_base=step["seg_slot_base"]).upload()
        PV = checked_oracle_plan(plan.view, step["parent"], step["seg_len"], step["group_block_size"],
                                 step["seg_flags"], None, step["seg_slot_base"])
        assert PV["pool_slots"] <= arena_slots
        qm = torch.zeros(PV["T_q"], Hq, D, dtype=torch.bfloat16)
        gm = torch.zeros_like(qm)
        for i, s in enumerate(step["seg_id"]):
            c = int(PV["canon_of_input"][i])
            assert int(PV["tok_slot"][int(PV["seg_tok_off"][c])]) == base_of[s]       # read in place
            if step["seg_flags"][i] & 1:
                r0 = int(PV["seg_q_off"][c])
                qm[r0:r0 + seg_len[s]] = Qseg[s]
                gm[r0:r0 + seg_len[s]] = Gseg[s]
        qm, gm = qm.to(dev), gm.to(dev)
        o, lse = lib.psrl_tree_attn_fwd(plan, qm, K, Vp, scale)
        assert lib.psrl_device_status(plan, "fwd") == 0
        dkp = torch.full_like(K, float("nan")); dvp = torch.full_like(K, float("nan"))
        dq, dkp, dvp = lib.psrl_tree_attn_bwd(plan, qm, K, Vp, o, lse, gm, scale, dk_pool=dkp, dv_pool=dvp)
        assert lib.psrl_device_status(plan, "bwd") == 0
        for i, s in enumerate(step["seg_id"]):
            c = int(PV["canon_of_input"][i])
            b = base_of[s]
            dK[s] += dkp[:, b:b + seg_len[s]].double().cpu()
            dV[s] += dvp[:, b:b + seg_len[s]].double().cpu()
            if step["seg_flags"][i] & 1:
                r0 = int(PV["seg_q_off"][c])
                got_O[s] = o[r0:r0 + seg_len[s]].float().cpu()
                got_L[s] = lse[:, r0:r0 + seg_len[s]].cpu()
                got_dQ[s] = dq[r0:r0 + seg_len[s]].float().cpu()
        cache.end(m)
    assert cache.stats()["peak_slots"] <= arena_slots

    # ---- compare per segment (per piece: its rows and tokens inside the original segment) ----
    for s in range(n):
        c = int(V["canon_of_input"][piece_seg[s]])
        r0, t0 = int(V["seg_q_off"][c]) + piece_begin[s], int(V["seg_tok_off"][c]) + piece_begin[s]
        rows = slice(r0, r0 + seg_len[s])
        slots = V["tok_slot"][t0:t0 + seg_len[s]].astype(np.int64)
        assert np.abs(got_O[s].numpy() - want["O"][rows]).max() <= 1e-2
        assert np.abs(got_L[s].numpy() - want["LSE"][:, rows]).max() <= 1e-2
        assert rel_fro(got_dQ[s].numpy(), want["dQ"][rows]) <= 1e-2
        assert rel_fro(dK[s].numpy(), want["dK"][:, slots]) <= 1e-2
        assert rel_fro(dV[s].numpy(), want["dV"][:, slots]) <= 1e-2
    return events, cache.stats()


gbs_of = {}


def setup_gbs(parent, gbs):
    gbs_of.clear()
    g = -1
    for s, p in enumerate(parent):
        if p == -1:
            g += 1
            gbs_of[s] = gbs[g]
        else:
            gbs_of[s] = gbs_of[p]


def test_prefix_reused_across_microbatches(lib):
    # a 300-token prefix computed with its first branch; two more branches and a grandchild later;
    # a second group whose long sequence is cut into three chunks (self-sequence sharing)
    parent = [-1, 0, 0, 0, 2, -1, 5, 6]
    seg_len = [300, 70, 129, 45, 33, 150, 150, 97]
    mb = [0, 0, 1, 2, 2, 0, 1, 2]
    gbs = [64, 32]
    setup_gbs(parent, gbs)
    events, stats = run_forest(lib, parent, seg_len, gbs, mb, 3, seed=1)
    assert events == dict(evict=0, reload=0)
    assert stats["peak_slots"] <= stats["total_slots"]


def test_eviction_and_reload_do_not_change_the_result(lib):
    # two groups whose branches alternate, arena with room for one group: each root is evicted while
    # the other group runs and restored for its next branch
    parent = [-1, 0, 0, -1, 3, 3]
    seg_len = [128, 60, 64, 100, 64, 50]
    mb = [0, 0, 2, 1, 1, 3]
    gbs = [64, 64]
    setup_gbs(parent, gbs)
    events, stats = run_forest(lib, parent, seg_len, gbs, mb, 4, cap=192, seed=2)
    assert events["evict"] == 2 and events["reload"] == 2
    assert stats["peak_slots"] == 192


def test_scheduler_output_runs_on_the_gpu(lib):
    """Sec. 4.2 + 4.3 end to end: the prefix groups of a forest are placed on two workers by descending
    Eq. 1 workload (psrl_place_groups); every worker's share is cut into micro-batches at the token level
    (psrl_microbatch_tokens: long sequences are cut in the middle of a segment and continue in the next
    micro-batch, reading their own earlier K/V from the cache); the pieces go through the cache manager and
    the attention calls as they are.  Every worker's multi-call result equals the oracle's single evaluation
    of that worker's uncut groups."""
    parent = [-1, 0, 0, -1, 3, -1, 5, 5, 6]
    seg_len = [420, 150, 97, 700, 64, 130, 200, 45, 33]
    gbs = [64, 32, 16]
    alpha = (1e-3, 1.0, 50.0)
    workload = lib.psrl_group_workloads(parent, seg_len, alpha)
    worker, load = lib.psrl_place_groups(workload, 2)
    assert sorted(set(worker.tolist())) == [0, 1] and abs(float(load.sum()) - float(workload.sum())) < 1e-9
    group_of, g = [], -1
    for s, p in enumerate(parent):
        g += p == -1
        group_of.append(g if p == -1 else group_of[p])
    n_cut_total = 0
    for wk in (0, 1):
        keep = [s for s in range(len(parent)) if worker[group_of[s]] == wk]
        new = {s: i for i, s in enumerate(keep)}
        w_parent = [-1 if parent[s] == -1 else new[parent[s]] for s in keep]
        w_len = [seg_len[s] for s in keep]
        w_gbs = [gbs[group_of[s]] for s in keep if parent[s] == -1]
        M = 3
        got = lib.psrl_microbatch_tokens(w_parent, w_len, alpha, M)
        p_parent, p_len = got["parent"].tolist(), got["seg_len"].tolist()
        p_mb, p_seg, p_begin = got["mb"].tolist(), got["seg"].tolist(), got["begin"].tolist()
        # the pieces partition every segment, in order, and micro-batches never decrease
        for s in range(len(w_parent)):
            mine = [(b, l) for sg, b, l in zip(p_seg, p_begin, p_len) if sg == s]
            assert mine[0][0] == 0 and sum(l for _, l in mine) == w_len[s]
            assert all(mine[i][0] + mine[i][1] == mine[i + 1][0] for i in range(len(mine) - 1))
        assert all(a <= b for a, b in zip(p_mb, p_mb[1:])) and max(p_mb) < M
        n_cut_total += len(p_parent) - len(w_parent)
        setup_gbs(p_parent, w_gbs)
        run_forest(lib, p_parent, p_len, w_gbs, p_mb, M, seed=10 + wk, origin=(w_parent, w_len, w_gbs, p_seg, p_begin))
    assert n_cut_total >= 2, "the case is meant to cut segments at the token level"
