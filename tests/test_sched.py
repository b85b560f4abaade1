"""The C++ scheduler (psrl_sched.h) against its oracle (oracle/sched.py): exact equality of workloads
(fp64, same order of operations), placements and pieces on random forests (host logic, no GPU)."""
import numpy as np
import pytest

from oracle.sched import cost_sequence, group_workloads, microbatch_tokens, pieces_to_forest, place_groups
from paper_2608_25683_b200 import binding


def random_tree(rng, n, max_len=400):
    parent = [-1] + [int(rng.integers(-1, s)) for s in range(1, n)]
    seg_len = [int(rng.integers(1, max_len)) for _ in range(n)]
    return parent, seg_len


def test_cost_and_workloads(lib):
    rng = np.random.default_rng(21)
    assert binding.psrl_cost_sequence((2.0, 3.0, 5.0), 10, 4) == cost_sequence((2.0, 3.0, 5.0), 10, 4) == 143.0
    for it in range(60):
        parent, seg_len = random_tree(rng, int(rng.integers(1, 30)))
        alpha = tuple(float(x) for x in rng.random(3) * [1e-3, 1.0, 50.0])
        flags = None
        if it % 3 == 0:
            flags = [2] * len(parent)      # step mode: every node ends a sample
        want = group_workloads(parent, seg_len, alpha, None if flags is None else [True] * len(parent))
        got = binding.psrl_group_workloads(parent, seg_len, alpha, flags)
        assert np.allclose(got, want, rtol=1e-12, atol=0)


def test_placement(lib):
    worker, load = binding.psrl_place_groups([5, 5, 4, 4, 3, 3, 3], 3)
    assert worker.tolist() == [0, 1, 2, 2, 0, 1, 0] and load.tolist() == [11, 8, 8]
    rng = np.random.default_rng(22)
    for _ in range(100):
        w = [float(x) for x in rng.integers(0, 50, size=int(rng.integers(0, 40)))]
        k = int(rng.integers(1, 9))
        want_w, want_l = place_groups(w, k)
        got_w, got_l = binding.psrl_place_groups(w, k)
        assert got_w.tolist() == want_w and got_l.tolist() == want_l
    with pytest.raises(binding.PsrlError):
        binding.psrl_place_groups([1.0, -2.0], 2)
    with pytest.raises(binding.PsrlError):
        binding.psrl_place_groups([1.0], 0)


def test_token_wise_micro_batching(lib):
    got = binding.psrl_microbatch_tokens([-1, -1], [10, 6], (0.0, 1.0, 0.0), 2)
    assert got["budget"] == 8.0
    assert got["parent"].tolist() == [-1, 0, -1] and got["seg_len"].tolist() == [8, 2, 6]
    assert got["mb"].tolist() == [0, 1, 1] and got["seg"].tolist() == [0, 0, 1] and got["begin"].tolist() == [0, 8, 0]
    rng = np.random.default_rng(23)
    for it in range(120):
        parent, seg_len = random_tree(rng, int(rng.integers(1, 25)))
        alpha = (float(rng.choice([0.0, 1e-3, 1.0])), float(rng.choice([0.0, 1.0, 7.0])), float(rng.choice([0.0, 50.0])))
        if alpha == (0.0, 0.0, 0.0):
            alpha = (1e-3, 0.0, 0.0)
        M = int(rng.integers(1, 8))
        flags = [2] * len(parent) if it % 4 == 0 else None
        pieces, budget = microbatch_tokens(parent, seg_len, alpha, M, None if flags is None else [True] * len(parent))
        want_parent, want_len, want_mb, origin = pieces_to_forest(parent, seg_len, pieces)
        got = binding.psrl_microbatch_tokens(parent, seg_len, alpha, M, flags)
        # the budget is a sum of doubles: equal to one unit in the last place; the cuts are integers: exact
        assert abs(got["budget"] - budget) <= np.spacing(max(abs(budget), abs(got["budget"])))
        assert got["parent"].tolist() == want_parent and got["seg_len"].tolist() == want_len
        assert got["mb"].tolist() == want_mb
        assert list(zip(got["seg"].tolist(), got["begin"].tolist())) == origin
        # the forest of pieces feeds the cache manager and the planner as it is
        n_roots = sum(p == -1 for p in want_parent)
        cache = binding.Cache(want_parent, want_len, [64] * n_roots, want_mb, M)
        for m in range(M):
            step = cache.begin(m)
            if step["seg_id"]:
                binding.Plan(step["parent"], step["seg_len"], step["group_block_size"], 4, 2, 128, "bf16",
                             seg_flags=step["seg_flags"], seg_slot_base=step["seg_slot_base"])
            cache.end(m)


def test_errors(lib):
    with pytest.raises(binding.PsrlError) as e:
        binding.psrl_group_workloads([-1, 5], [3, 3], (1, 1, 1))
    assert e.value.name == "PSRL_ERR_BAD_TREE"
    with pytest.raises(binding.PsrlError) as e:
        binding.psrl_microbatch_tokens([-1], [3], (-1.0, 0, 0), 2)
    assert e.value.name == "PSRL_ERR_INVALID_ARG"
