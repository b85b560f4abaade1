"""ORACLE (test infrastructure, not product code): workload model and scheduling.

Written step by step from Sec. 4.2 (Eq. 1: execution time of a sequence with a
cached prefix; workload of a semantic group = sum over its sequences; groups are
sorted by workload in descending order and handed, one by one and never split,
to the worker with the smallest load) and Sec. 4.3 (token-wise micro-batching:
a per-micro-batch budget derived from the total workload; a sequence that would
exceed what is left of the budget is split at the token level and the rest goes
to the following micro-batches).  Plain Python floats (fp64).

Readings where the paper is silent:
  * inside a prefix group the samples (root-to-SAMPLE_END paths) are taken in
    canonical (DFS) order; the cached prefix h of a sample is the part of its
    path that earlier samples have already computed, its sequence length l the
    whole path;
  * ties: groups of equal workload keep their index order, the lower worker
    index wins among equally loaded workers;
  * micro-batching walks the samples in that order; a piece [a, b) of a
    sample's token range costs Eq. 1 with h = a and l = b; the overhead term
    alpha3 is paid by every piece; a split leaves at least one token on each
    side; an empty micro-batch takes at least one token; the last micro-batch
    takes whatever remains.
"""
from __future__ import annotations

import math


def cost_sequence(alpha, l, h):
    """Eq. 1: T(s) = a1 * l_suf * l + a2 * l_suf + a3 with l_suf = l - h."""
    a1, a2, a3 = alpha
    suf = l - h
    return a1 * suf * l + a2 * suf + a3


def _samples(parent, seg_len, sample_end=None):
    """Samples in canonical order as (path segments, h, l): h tokens of the path were computed
    by earlier samples.  Also returns the group of every segment."""
    n = len(parent)
    children = [[] for _ in range(n)]
    roots = []
    for s, p in enumerate(parent):
        (roots if p == -1 else children[p]).append(s)
    if sample_end is None:
        sample_end = [not children[s] for s in range(n)]
    group = [0] * n
    order = []
    for g, r in enumerate(roots):
        stack = [r]
        while stack:
            s = stack.pop()
            order.append(s)
            group[s] = g
            stack.extend(reversed(children[s]))
    done = [False] * n
    samples = []
    for e in order:
        if not sample_end[e]:
            continue
        path = []
        s = e
        while s != -1:
            path.append(s)
            s = parent[s]
        path.reverse()
        h = sum(seg_len[s] for s in path if done[s])
        l = sum(seg_len[s] for s in path)
        fresh = [s for s in path if not done[s]]
        for s in path:
            done[s] = True
        samples.append((fresh, h, l, group[e]))
    return samples, len(roots)


def group_workloads(parent, seg_len, alpha, sample_end=None):
    """Workload of every prefix group: the sum of Eq. 1 over its samples (cached prefixes accounted)."""
    samples, n_groups = _samples(parent, seg_len, sample_end)
    w = [0.0] * n_groups
    for _, h, l, g in samples:
        w[g] += cost_sequence(alpha, l, h)
    return w


def place_groups(workload, n_workers):
    """Longest-processing-time-first placement.  Returns (worker of every group, load of every worker)."""
    load = [0.0] * n_workers
    worker = [0] * len(workload)
    for g in sorted(range(len(workload)), key=lambda g: (-workload[g], g)):
        k = min(range(n_workers), key=lambda k: (load[k], k))
        worker[g] = k
        load[k] += workload[g]
    return worker, load


def _fit(alpha, c0, room, most):
    """Largest x in [0, most] with Eq. 1 cost of the piece [c0, c0 + x) <= room."""
    a1, a2, a3 = alpha
    if room <= a3:
        return 0
    if a1 > 0:
        bq = a1 * c0 + a2
        x = int(math.floor((-bq + math.sqrt(bq * bq + 4 * a1 * (room - a3))) / (2 * a1)))
    elif a2 > 0:
        x = int(math.floor((room - a3) / a2))
    else:
        x = most
    x = max(0, min(x, most))
    while x > 0 and cost_sequence(alpha, c0 + x, c0) > room:          # guard the rounding of the root
        x -= 1
    while x + 1 <= most and cost_sequence(alpha, c0 + x + 1, c0) <= room:
        x += 1
    return x


def microbatch_tokens(parent, seg_len, alpha, n_microbatches, sample_end=None):
    """Token-wise micro-batching of one worker's forest.

    Returns (pieces, budget): pieces in canonical order, each a dict
    (seg, begin, end, mb): tokens [begin, end) of input segment `seg` run in
    micro-batch `mb`; pieces of one segment are consecutive and form a chain
    (each is the cached prefix of the next)."""
    samples, _ = _samples(parent, seg_len, sample_end)
    total = 0.0
    for _, h, l, _ in samples:      # plain left-to-right fp64 accumulation (the built-in sum() compensates)
        total += cost_sequence(alpha, l, h)
    budget = total / n_microbatches
    pieces = []
    mb, used = 0, 0.0

    def emit(fresh, h, a, b, mb):
        # tokens [a, b) of the sample (positions along its path) -> pieces of its fresh segments
        pos = h
        for s in fresh:
            lo, hi = max(a, pos), min(b, pos + seg_len[s])
            if lo < hi:
                pieces.append(dict(seg=s, begin=lo - pos, end=hi - pos, mb=mb))
            pos += seg_len[s]

    for fresh, h, l, _ in samples:
        a = h
        while a < l:
            rest = cost_sequence(alpha, l, a)
            if mb == n_microbatches - 1 or used + rest <= budget:
                emit(fresh, h, a, l, mb)
                used += rest
                break
            x = _fit(alpha, a, budget - used, l - a - 1)
            if x == 0 and used == 0.0:
                x = 1
            if x > 0:
                emit(fresh, h, a, a + x, mb)
                a += x
            mb += 1
            used = 0.0
    return pieces, budget


def pieces_to_forest(parent, seg_len, pieces):
    """The forest of pieces: (parent, seg_len, mb_of_seg, origin) with pieces of a segment chained."""
    first, last = {}, {}
    new_parent, new_len, mb, origin = [], [], [], []
    for i, p in enumerate(pieces):
        s = p["seg"]
        if s not in first:
            first[s] = i
            new_parent.append(-1 if parent[s] == -1 else last[parent[s]])
        else:
            new_parent.append(last[s])
        last[s] = i
        new_len.append(p["end"] - p["begin"])
        mb.append(p["mb"])
        origin.append((s, p["begin"]))
    return new_parent, new_len, mb, origin
