"""GPU parity of multi-micro-batch execution (paper Sec. 4.1 inter-batch / self-sequence sharing with
the Dynamic Block Caching manager of Sec. 5.2): a forest is computed over several attention calls;
prefixes computed by an earlier micro-batch are read in place (no queries), their dK/dV contributions
are summed over the micro-batches (one accumulated backward on the shared prefix, Sec. 6).  The
result must equal the oracle's single evaluation of the whole forest."""
import numpy as np
import pytest
import torch

from oracle import oracle_attn

from util import rel_fro, to_np

pytestmark = pytest.mark.gpu
Hq, Hkv, D = 4, 2, 128


def run_forest(lib, parent, seg_len, gbs, mb, M, cap=0, seed=0):
    n = len(parent)
    g = torch.Generator(device="cpu").manual_seed(seed)
    rnd = lambda *shape: torch.randn(*shape, generator=g).to(torch.bfloat16)
    Kseg = [rnd(Hkv, l, D) for l in seg_len]
    Vseg = [rnd(Hkv, l, D) for l in seg_len]
    Qseg = [rnd(l, Hq, D) for l in seg_len]
    Gseg = [rnd(l, Hq, D) for l in seg_len]
    scale = 1.0 / np.sqrt(D)

    # ---- whole forest in one evaluation by the oracle ----
    full = lib.Plan(parent, seg_len, gbs, Hq, Hkv, D, "bf16")
    V = full.view
    q = torch.zeros(V["T_q"], Hq, D, dtype=torch.bfloat16)
    d_o = torch.zeros_like(q)
    k = torch.zeros(Hkv, V["pool_slots"], D, dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    for s in range(n):
        c = int(V["canon_of_input"][s])
        r0, t0 = int(V["seg_q_off"][c]), int(V["seg_tok_off"][c])
        q[r0:r0 + seg_len[s]] = Qseg[s]
        d_o[r0:r0 + seg_len[s]] = Gseg[s]
        slots = torch.as_tensor(V["tok_slot"][t0:t0 + seg_len[s]].astype(np.int64))
        k[:, slots] = Kseg[s]
        v[:, slots] = Vseg[s]
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
        PV = plan.view
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

    # ---- compare per segment ----
    for s in range(n):
        c = int(V["canon_of_input"][s])
        r0, t0 = int(V["seg_q_off"][c]), int(V["seg_tok_off"][c])
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
