"""Pins of the scheduling oracle (oracle/sched.py): Eq. 1 by hand, the classical LPT counter-example and
Graham's bound against brute force, token-wise micro-batching on a worked case and by invariants."""
import itertools

import numpy as np

from oracle.sched import (cost_sequence, group_workloads, microbatch_tokens, pieces_to_forest, place_groups)


def test_eq1_by_hand():
    # T = a1 * l_suf * l + a2 * l_suf + a3, l_suf = l - h   (Eq. 1)
    assert cost_sequence((2.0, 3.0, 5.0), 10, 4) == 2 * 6 * 10 + 3 * 6 + 5
    assert cost_sequence((1.0, 0.0, 0.0), 7, 7) == 0.0
    # a star: 4-token prefix, branches of 2 and 3 tokens.  First sample: l = 6, nothing cached;
    # second: l = 7 with the 4 prefix tokens cached.
    w = group_workloads([-1, 0, 0], [4, 2, 3], (1.0, 10.0, 100.0))
    assert w == [(6 * 6 + 10 * 6 + 100) + (3 * 7 + 10 * 3 + 100)]
    # without sharing (two roots) the second sequence pays for its whole length
    w2 = group_workloads([-1, -1], [6, 7], (1.0, 10.0, 100.0))
    assert w2 == [6 * 6 + 60 + 100, 7 * 7 + 70 + 100]
    # step-mode sampling: the interior node ends a sample too; the leaf then has it cached
    w3 = group_workloads([-1, 0], [4, 2], (1.0, 0.0, 0.0), sample_end=[True, True])
    assert w3 == [4 * 4 + 2 * 6]


def test_lpt_classical_example():
    # 7 jobs on 3 machines: LPT reaches 11 where 9 is optimal (5+4, 5+4, 3+3+3): the tight case of Graham's bound
    worker, load = place_groups([5, 5, 4, 4, 3, 3, 3], 3)
    assert worker == [0, 1, 2, 2, 0, 1, 0]
    assert load == [11, 8, 8]


def brute_force_makespan(w, m):
    best = float("inf")
    for assign in itertools.product(range(m), repeat=len(w)):
        load = [0.0] * m
        for g, k in enumerate(assign):
            load[k] += w[g]
        best = min(best, max(load))
    return best


def test_lpt_within_grahams_bound():
    rng = np.random.default_rng(8)
    for _ in range(60):
        m = int(rng.integers(2, 4))
        w = [float(x) for x in rng.integers(1, 30, size=int(rng.integers(1, 8)))]
        worker, load = place_groups(w, m)
        assert sorted(set(worker)) == sorted(set(worker) & set(range(m)))
        assert abs(sum(load) - sum(w)) < 1e-9
        for k in range(m):
            assert abs(load[k] - sum(w[g] for g in range(len(w)) if worker[g] == k)) < 1e-9
        assert max(load) <= (4 / 3 - 1 / (3 * m)) * brute_force_makespan(w, m) + 1e-9


def test_token_wise_split_worked_case():
    # cost = number of tokens (a2 = 1): sequences of 10 and 6 tokens, two micro-batches, budget 8:
    # the first sequence is cut after 8 tokens, its last 2 tokens travel with the second sequence
    pieces, budget = microbatch_tokens([-1, -1], [10, 6], (0.0, 1.0, 0.0), 2)
    assert budget == 8.0
    assert [(p["seg"], p["begin"], p["end"], p["mb"]) for p in pieces] == [(0, 0, 8, 0), (0, 8, 10, 1), (1, 0, 6, 1)]
    parent, seg_len, mb, origin = pieces_to_forest([-1, -1], [10, 6], pieces)
    assert parent == [-1, 0, -1] and seg_len == [8, 2, 6] and mb == [0, 1, 1]
    assert origin == [(0, 0), (0, 8), (1, 0)]
    # with the quadratic term a cut comes earlier in a long sequence: pieces of equal cost, not equal length
    pieces, budget = microbatch_tokens([-1], [100], (1.0, 0.0, 0.0), 2)
    cut = pieces[0]["end"]
    assert budget == 5000.0 and cut == 70            # 70 * 70 = 4900 <= 5000 < 71 * 71
    assert (pieces[1]["begin"], pieces[1]["end"], pieces[1]["mb"]) == (70, 100, 1)


def test_micro_batching_invariants():
    rng = np.random.default_rng(9)
    for it in range(60):
        n = int(rng.integers(1, 20))
        parent = [-1] + [int(rng.integers(-1, s)) for s in range(1, n)]
        seg_len = [int(rng.integers(1, 400)) for _ in range(n)]
        alpha = (float(rng.choice([0.0, 1e-3, 1.0])), float(rng.choice([0.0, 1.0, 7.0])), float(rng.choice([0.0, 50.0])))
        if alpha == (0.0, 0.0, 0.0):
            alpha = (0.0, 1.0, 0.0)
        M = int(rng.integers(1, 7))
        pieces, budget = microbatch_tokens(parent, seg_len, alpha, M)
        # every token of every segment exactly once, pieces of a segment in order
        cover = {s: [] for s in range(n)}
        for p in pieces:
            cover[p["seg"]].append((p["begin"], p["end"]))
        for s in range(n):
            assert cover[s][0][0] == 0 and cover[s][-1][1] == seg_len[s]
            assert all(a[1] == b[0] for a, b in zip(cover[s], cover[s][1:]))
        # micro-batch indices never decrease along the walk and stay in range
        mbs = [p["mb"] for p in pieces]
        assert mbs == sorted(mbs) and 0 <= mbs[0] and mbs[-1] < M
        # the forest of pieces is a valid input for the planner and the cache manager
        new_parent, new_len, mb, origin = pieces_to_forest(parent, seg_len, pieces)
        assert all(p < i for i, p in enumerate(new_parent))
        assert all(p == -1 or mb[p] <= mb[i] for i, p in enumerate(new_parent))
        assert sum(new_len) == sum(seg_len)
        # at most one segment is cut per micro-batch boundary
        assert len(pieces) <= n + (M - 1) * (max(1, n))
