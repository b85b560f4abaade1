"""Host-side model check of the named-barrier hand-off protocol of the forward and dK/dV kernels.

A hardware named barrier (bar.arrive by the softmax warps, bar.sync by the MMA-issuing warp) has no
phases and no timeout: it completes whenever its count reaches the expected number of threads and then
starts over.  The kernels use it on two conditions (csrc/sm100.cuh): an arrival for step t+1 can never
reach a barrier before the consumer has synced on step t's arrivals, and every sync gets all its arrivals
in bounded time - also from warps that gave up on a wait of their own, and also when the consumer leaves
its loop early.  The path of a warp that gave up is only reached when a bounded wait runs out, which no
input provokes on a healthy GPU, so it is checked here instead: the protocol is replayed as a small state
machine under thousands of random interleavings, with warps giving up at arbitrary points and the consumer
leaving at arbitrary steps.  A negative control replays the protocol WITHOUT the lock-step rule (a warp
that gave up performs all its remaining arrivals at once) and must be caught.

The model is deliberately more hostile than the hardware: a warp may give up at any moment, not only when
the consumer stalls.
"""
import random

import pytest


class Barrier:
    """Count-based barrier: `expected` arrival units complete a generation (the consumer's sync is one)."""

    def __init__(self, expected):
        self.expected, self.count, self.generation = expected, 0, 0
        self.consumer_waiting = False
        self.log = []   # (generation the arrival was meant for, generation it landed in)

    def add(self, meant_for):
        self.log.append((meant_for, self.generation))
        self.count += 1
        if self.count == self.expected:
            self.count = 0
            self.generation += 1
            self.consumer_waiting = False


def run(seed, n_producers, n_steps, ids, lock_step=True, p_give_up=0.02, p_leave=0.01):
    """One random interleaving.  `ids` = barrier ids synced per step, in order.
    Returns ('ok' | 'deadlock', barriers)."""
    rng = random.Random(seed)
    bars = {b: Barrier(n_producers + 1) for b in ids}
    # consumer: position (t, k) = about to sync on ids[k] of step t; `passed[b]` = syncs completed on b
    cons = dict(t=0, k=0, waiting=None, left=False, at=-1)
    passed = {b: 0 for b in ids}
    prods = [dict(t=0, k=0, gave_up=False, done=False) for _ in range(n_producers)]
    for _ in range(200000):
        actors = []
        if not cons["left"]:
            actors.append("c")
        actors += [i for i, p in enumerate(prods) if not p["done"]]
        if not actors:
            return "ok", bars
        progressed = False
        rng.shuffle(actors)
        for a in actors:
            if a == "c":
                if cons["waiting"] is not None:
                    b = cons["waiting"]
                    if not bars[b].consumer_waiting:       # the generation completed
                        passed[b] += 1
                        cons["waiting"] = None
                        cons["k"] += 1
                        if cons["k"] == len(ids):
                            cons["k"], cons["t"] = 0, cons["t"] + 1
                        progressed = True
                    continue
                if cons["t"] == n_steps:
                    cons["left"] = True
                    progressed = True
                    continue
                if cons["k"] == 0:
                    if rng.random() < p_leave:             # its own bounded wait failed: only between steps
                        cons["left"] = True
                        progressed = True
                        continue
                    cons["at"] = cons["t"]                 # published before the step's syncs
                b = ids[cons["k"]]
                bars[b].consumer_waiting = True
                cons["waiting"] = b
                bars[b].add(cons["t"])
                progressed = True
                break
            p = prods[a]
            if p["t"] == n_steps:
                p["done"] = True
                progressed = True
                break
            b = ids[p["k"]]
            if not p["gave_up"] and rng.random() < p_give_up:
                p["gave_up"] = True
            if not p["gave_up"]:
                # normal path: the data this arrival follows is produced by MMAs that the consumer issues
                # after its sync on the previous step's arrival on the same barrier
                if passed[b] < p["t"]:
                    continue
            elif lock_step:
                if cons["left"]:
                    p["done"] = True                       # nobody syncs any more
                    progressed = True
                    break
                # dK/dV: the published step; forward: the completed MMAs of step t-1 (both imply that the
                # consumer is past every sync of step t-1)
                if cons["at"] < p["t"]:
                    continue
            bars[b].add(p["t"])
            p["k"] += 1
            if p["k"] == len(ids):
                p["k"], p["t"] = 0, p["t"] + 1
            progressed = True
            break
        if not progressed:
            if cons["waiting"] is not None and bars[cons["waiting"]].consumer_waiting:
                return "deadlock", bars
            if all(p["done"] or p["gave_up"] is False for p in prods) and cons["left"]:
                # producers on the normal path blocked on a consumer that left: their bounded waits end this
                for p in prods:
                    p["gave_up"] = True
                continue
            return "deadlock", bars
    raise AssertionError("the model did not terminate")


@pytest.mark.parametrize("name,n_producers,ids", [("forward, one head", 4, [1]), ("dK/dV", 8, [2, 3, 4, 5, 1])])
def test_lock_step_protocol_never_hangs_and_never_mixes_generations(name, n_producers, ids):
    for seed in range(1500):
        rng = random.Random(seed)
        status, bars = run(seed, n_producers, n_steps=rng.randint(1, 12), ids=ids,
                           p_give_up=rng.choice([0.0, 0.01, 0.05, 0.3]), p_leave=rng.choice([0.0, 0.02, 0.2]))
        assert status == "ok", (name, seed)
        for b in bars.values():
            assert all(meant == landed for meant, landed in b.log), (name, seed)


def test_the_model_catches_arrivals_that_run_ahead():
    """Negative control: without the lock-step rule a warp that gave up fires all its remaining arrivals at
    once; they wrap the barrier's count, and the consumer is left waiting for a residue (or generations mix)."""
    bad = 0
    for seed in range(300):
        status, bars = run(seed, 8, n_steps=10, ids=[2, 3, 4, 5, 1], lock_step=False, p_give_up=0.05, p_leave=0.0)
        mixed = any(meant != landed for b in bars.values() for meant, landed in b.log)
        bad += status == "deadlock" or mixed
    assert bad > 100
