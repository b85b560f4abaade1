"""ORACLE (test infrastructure, not product code): Dynamic Block Caching.

The liveness rules of the KV blocks of one worker over an ordered list of
micro-batches, written step by step from Sec. 5.2 (reference counts, removal of
reference entries after each micro-batch's backward pass, eviction of the block
with the farthest reuse distance when memory runs short) and Sec. 4.1 (a prefix
computed by an earlier micro-batch is reused by later ones; a long sequence may
be cut into chunks that run in successive micro-batches).  Plain Python, no
arithmetic of the attention itself.

Blocks are the segments of the prefix forest (Sec. 5.1: one block per reusable
prefix span); a segment occupies one contiguous extent of
ceil(len / block) * block slots of a per-worker arena.

Readings where the paper is silent:
  * a sample "completes" in the micro-batch that computes its last segment;
    the reference entries of all blocks on its path are removed after that
    micro-batch's backward pass;
  * the arena is managed first-fit in address order with coalescing;
  * a block evicted while its count is positive has to be brought back
    (offload / reload or recomputation) before its next use: the manager
    reports both events, it does not move data;
  * ties of the reuse distance are broken towards the larger segment index.
"""
from __future__ import annotations


class CacheError(Exception):
    def __init__(self, code, msg=""):
        super().__init__(f"{code}: {msg}")
        self.code = code


class OracleCache:
    def __init__(self, parent, seg_len, group_block_size, mb_of_seg, n_microbatches, sample_end=None,
                 capacity_slots=0):
        n = len(parent)
        self.n = n
        self.parent = [int(p) for p in parent]
        self.seg_len = [int(l) for l in seg_len]
        self.mb = [int(m) for m in mb_of_seg]
        self.M = int(n_microbatches)
        self.capacity = int(capacity_slots)
        if n < 1 or len(self.seg_len) != n or len(self.mb) != n or self.M < 1:
            raise CacheError("INVALID_ARG", "array lengths")
        children = [[] for _ in range(n)]
        roots = []
        for s, p in enumerate(self.parent):
            if p == -1:
                roots.append(s)
            elif 0 <= p < s:
                children[p].append(s)
            else:
                raise CacheError("BAD_TREE", f"parent[{s}]")
            if self.seg_len[s] < 1:
                raise CacheError("BAD_TREE", f"seg_len[{s}]")
            if not (0 <= self.mb[s] < self.M):
                raise CacheError("INVALID_ARG", f"mb_of_seg[{s}]")
            if p >= 0 and self.mb[p] > self.mb[s]:
                raise CacheError("BAD_TREE", "a prefix must be computed no later than what follows it")
        if len(group_block_size) != len(roots):
            raise CacheError("INVALID_ARG", "one block size per root")
        for b in group_block_size:
            if b != 0 and (b < 16 or b > 256 or (b & (b - 1))):
                raise CacheError("BAD_BLOCK_SIZE", str(b))
        if self.capacity < 0 or self.capacity % 16:
            raise CacheError("INVALID_ARG", "capacity")
        self.children = children
        self.roots = roots
        self.group = [0] * n
        for s in range(n):
            self.group[s] = roots.index(s) if self.parent[s] == -1 else self.group[self.parent[s]]
        self.gbs = [int(b) for b in group_block_size]
        self.bs = [self.gbs[self.group[s]] for s in range(n)]
        # block size 0 = adaptive (Sec. 5.1): the span at 16-slot granularity
        self.extent = [-(-self.seg_len[s] // (self.bs[s] or 16)) * (self.bs[s] or 16) for s in range(n)]
        if sample_end is None:
            self.sample_end = [not children[s] for s in range(n)]
        else:
            self.sample_end = [bool(x) for x in sample_end]
            for s in range(n):
                if not children[s] and not self.sample_end[s]:
                    raise CacheError("BAD_TREE", f"leaf {s} does not end a sample")
        # reference count = number of samples that will access the block (Sec. 5.2)
        self.path = []
        for s in range(n):
            self.path.append(([] if self.parent[s] == -1 else self.path[self.parent[s]]) + [s])
        self.refcount = [0] * n
        for e in range(n):
            if self.sample_end[e]:
                for s in self.path[e]:
                    self.refcount[s] += 1
        # micro-batches in which a block is read or written: those of its whole subtree
        self.uses = [set() for _ in range(n)]
        for s in range(n):
            for a in self.path[s]:
                self.uses[a].add(self.mb[s])
        self.uses = [sorted(u) for u in self.uses]
        self.base = [-1] * n          # resident extent, -1 = not resident
        self.evicted = [False] * n    # lost while still referenced
        self.free = [[0, self.capacity]] if self.capacity else [[0, 1 << 40]]
        self.next_mb = 0
        self.in_mb = False
        self.peak = 0
        self.evicted_slots = 0
        self.reloaded_slots = 0
        self.high_water = 0
        self.trace = []               # live slots (during, after) per micro-batch

    # ---- arena: first fit in address order, coalescing on release ----
    def _alloc(self, size):
        for e in self.free:
            if e[1] >= size:
                at = e[0]
                e[0] += size
                e[1] -= size
                if e[1] == 0:
                    self.free.remove(e)
                return at
        return -1

    def _release(self, at, size):
        self.free.append([at, size])
        self.free.sort()
        merged = []
        for e in self.free:
            if merged and merged[-1][0] + merged[-1][1] == e[0]:
                merged[-1][1] += e[1]
            else:
                merged.append(e)
        self.free = merged

    def live_slots(self):
        return sum(self.extent[s] for s in range(self.n) if self.base[s] >= 0)

    def _next_use(self, s, m):
        for u in self.uses[s]:
            if u > m:
                return u
        return None

    def begin(self, m):
        if m != self.next_mb or self.in_mb:
            raise CacheError("INVALID_ARG", "micro-batches run in order, begin then end")
        self.in_mb = True
        needed = [s for s in range(self.n) if m in self.uses[s]]
        need = set(needed)
        new, reload, evict = [], [], []
        for s in needed:
            if self.base[s] >= 0:
                continue
            while True:
                at = self._alloc(self.extent[s])
                if at >= 0:
                    break
                # evict the resident block, not used now, whose next use lies farthest ahead
                cand = [(self._next_use(r, m), r) for r in range(self.n) if self.base[r] >= 0 and r not in need]
                if not cand:
                    raise CacheError("POOL_FULL", f"micro-batch {m} does not fit")
                _, r = max(cand)
                evict.append((r, self.base[r]))
                self._release(self.base[r], self.extent[r])
                self.base[r] = -1
                self.evicted[r] = True
                self.evicted_slots += self.extent[r]
            self.base[s] = at
            self.high_water = max(self.high_water, at + self.extent[s])
            if self.evicted[s]:
                self.evicted[s] = False
                reload.append(s)
                self.reloaded_slots += self.extent[s]
            else:
                if self.mb[s] != m:
                    raise CacheError("INTERNAL", "a block is missing that was never evicted")
                new.append(s)
        live = self.live_slots()
        self.peak = max(self.peak, live)
        # the tree of this micro-batch: needed segments in forest order; active ones issue queries
        local = {s: i for i, s in enumerate(needed)}
        has_child = [False] * len(needed)
        for s in needed:
            if self.parent[s] >= 0:
                has_child[local[self.parent[s]]] = True
        flags = []
        for i, s in enumerate(needed):
            active = self.mb[s] == m
            f = 1 if active else 0
            if not has_child[i] or (active and self.sample_end[s]):
                f |= 2
            flags.append(f)
        step = dict(
            seg_id=needed,
            parent=[-1 if self.parent[s] == -1 else local[self.parent[s]] for s in needed],
            seg_len=[self.seg_len[s] for s in needed],
            seg_flags=flags,
            group_block_size=[self.gbs[self.group[s]] for s in needed if self.parent[s] == -1],
            seg_slot_base=[self.base[s] for s in needed],
            new=new, reload=reload, evict=evict, live_slots=live)
        self._live_during = live
        return step

    def end(self, m):
        if m != self.next_mb or not self.in_mb:
            raise CacheError("INVALID_ARG", "end without begin")
        # remove the reference entries of the samples that completed in this micro-batch
        for e in range(self.n):
            if self.sample_end[e] and self.mb[e] == m:
                for s in self.path[e]:
                    self.refcount[s] -= 1
        freed = []
        for s in range(self.n):
            if self.refcount[s] == 0 and self.base[s] >= 0:
                self._release(self.base[s], self.extent[s])
                self.base[s] = -1
                freed.append(s)
            if self.refcount[s] == 0:
                self.evicted[s] = False
        live = self.live_slots()
        self.trace.append((self._live_during, live))
        self.in_mb = False
        self.next_mb += 1
        return dict(freed=freed, live_slots=live)

    def stats(self):
        return dict(peak_slots=self.peak, evicted_slots=self.evicted_slots, reloaded_slots=self.reloaded_slots,
                    high_water=self.high_water)
