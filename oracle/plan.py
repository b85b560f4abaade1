"""Oracle for the canonical plan of a prefix forest.  TEST INFRASTRUCTURE ONLY.

The plan is an encoding, so this module takes the construction step by step,
in plain Python loops, in the order the specification lists the steps.

What the paper fixes:
  * Sec. 5.1 (Adaptive Block Allocation): a KV block covers a contiguous
    token span that is shared by one or more sequences; blocks never mix
    tokens whose sharing differs.  Here: pages never cross a segment boundary.
  * Sec. 6 (adaptive KV cache manager): per-block metadata = base address,
    block size, position of the token span in the full sequence, reference
    count.  Here: page_slot, page_bs (+ page_valid), page_pos, page_refcount.
  * Sec. 5.2 (Dynamic Block Caching): the reference count of a block is the
    number of training samples that will access it (root 4, leaf 1 in the
    paper's four-sample tree).
  * Sec. 2.5: prefix match rate = share of tokens in a batch that duplicate
    another sample's prefix; here 1 - T / flat_tokens.
  * Eq. 1: the attention term of a sequence's cost is l_suf * l; the exact
    integer form per segment is len * anc + len * (len + 1) / 2.
Everything else (canonical order, first-fit slot assignment, CSR layouts) is
this library's convention and is stated step by step below.

Pins (tests/test_oracle_plan.py): the paper's refcount example; the paper's
28-shared-token example; closed forms (sum page_valid == T, bump pool size,
sum len*refcount == flat_tokens, block-table row lengths); the hand-computed
counts of the tiny configuration; a brute-force token-by-token expansion of
every sample.
"""
from __future__ import annotations

import numpy as np

SEG_HAS_Q = 1
SEG_SAMPLE_END = 2


class PlanError(ValueError):
    """Raised with .code in {'INVALID_ARG','BAD_TREE','BAD_BLOCK_SIZE','POOL_FULL'}."""

    def __init__(self, code: str, msg: str = ""):
        super().__init__(f"{code}: {msg}")
        self.code = code


def _i32(x):
    return np.asarray(x, dtype=np.int32)


def oracle_plan(parent, seg_len, group_block_size, seg_flags=None, free_extents=None, seg_slot_base=None):
    """Build the canonical plan.

    parent[s]            -1 for a root, else an input index < s
    seg_len[s]           tokens in segment s (>= 1)
    group_block_size[g]  page size of the g-th root (roots counted in input
                         order); power of two in [16, 256], or 0 = adaptive
                         (Sec. 5.1): every segment of the group gets ONE
                         contiguous extent sized to its span at 16-slot
                         granularity, recorded as pages of 128 slots followed
                         by pages of 16 slots for the tail
    seg_flags[s]         bit 0 HAS_Q, bit 1 SAMPLE_END; None = HAS_Q everywhere,
                         SAMPLE_END on leaves
    free_extents         None = one unbounded extent starting at slot 0, else a
                         list of (start_slot, n_slots), all multiples of 16
    seg_slot_base[s]     None, or per segment: >= 0 (a multiple of 16) pins the
                         segment's pages to consecutive runs of block-size slots
                         from that slot on (K/V cached by an earlier micro-batch,
                         Sec. 4.1 / 5.2) and takes nothing from the free extents;
                         -1 allocates as usual

    Returns a dict of python ints and numpy int32 arrays (int64 where noted).
    """
    parent = [int(p) for p in parent]
    seg_len = [int(l) for l in seg_len]
    n = len(parent)

    # -- step 1: validate -----------------------------------------------------
    if n < 1 or len(seg_len) != n:
        raise PlanError("INVALID_ARG", "need >= 1 segment and matching arrays")
    for s in range(n):
        if not (parent[s] == -1 or 0 <= parent[s] < s):
            raise PlanError("BAD_TREE", f"parent[{s}]={parent[s]}")
        if seg_len[s] < 1:
            raise PlanError("BAD_TREE", f"seg_len[{s}]={seg_len[s]}")
    children = [[] for _ in range(n)]
    roots = []
    for s in range(n):
        if parent[s] == -1:
            roots.append(s)
        else:
            children[parent[s]].append(s)  # ascending input index by construction
    if seg_flags is None:
        flags = [SEG_HAS_Q | (SEG_SAMPLE_END if not children[s] else 0) for s in range(n)]
    else:
        flags = [int(f) for f in seg_flags]
        if len(flags) != n:
            raise PlanError("INVALID_ARG", "seg_flags length")
    for s in range(n):
        if flags[s] & ~(SEG_HAS_Q | SEG_SAMPLE_END):
            raise PlanError("INVALID_ARG", f"seg_flags[{s}]")
        if not children[s] and not (flags[s] & SEG_SAMPLE_END):
            raise PlanError("BAD_TREE", f"leaf {s} does not end a sample")
    gbs = [int(b) for b in group_block_size]
    if len(gbs) != len(roots):
        raise PlanError("INVALID_ARG", "one block size per root")
    for b in gbs:
        if b != 0 and (b < 16 or b > 256 or (b & (b - 1))):
            raise PlanError("BAD_BLOCK_SIZE", str(b))
    if free_extents is not None:
        free_extents = [(int(a), int(c)) for a, c in free_extents]
        for a, c in free_extents:
            if a < 0 or c < 0 or a % 16 or c % 16:
                raise PlanError("INVALID_ARG", "free extent not a multiple of 16")

    if seg_slot_base is not None:
        seg_slot_base = [int(b) for b in seg_slot_base]
        if len(seg_slot_base) != n:
            raise PlanError("INVALID_ARG", "seg_slot_base length")
        for b in seg_slot_base:
            if b < -1 or (b >= 0 and b % 16):
                raise PlanError("INVALID_ARG", "seg_slot_base not -1 or a multiple of 16")

    # -- step 2: canonical order = DFS preorder --------------------------------
    input_of_canon = []
    seg_group_in = [0] * n
    for g, r in enumerate(roots):
        stack = [r]
        while stack:
            s = stack.pop()
            input_of_canon.append(s)
            seg_group_in[s] = g
            for ch in reversed(children[s]):
                stack.append(ch)
    canon_of_input = [0] * n
    for c, s in enumerate(input_of_canon):
        canon_of_input[s] = c

    # -- step 3: per-segment arrays, canonical index ---------------------------
    c_parent = [(-1 if parent[s] == -1 else canon_of_input[parent[s]]) for s in input_of_canon]
    c_len = [seg_len[s] for s in input_of_canon]
    c_flags = [flags[s] for s in input_of_canon]
    c_group = [seg_group_in[s] for s in input_of_canon]
    c_bs = [gbs[g] for g in c_group]
    c_depth = [0] * n
    c_anc = [0] * n
    for c in range(n):
        p = c_parent[c]
        if p >= 0:
            c_depth[c] = c_depth[p] + 1
            c_anc[c] = c_anc[p] + c_len[p]
    c_sub_end = [c + 1 for c in range(n)]
    for c in range(n - 1, -1, -1):
        p = c_parent[c]
        if p >= 0 and c_sub_end[c] > c_sub_end[p]:
            c_sub_end[p] = c_sub_end[c]
    c_tok_off = [0] * n
    c_q_off = [0] * n
    t = 0
    tq = 0
    for c in range(n):
        c_tok_off[c] = t
        t += c_len[c]
        if c_flags[c] & SEG_HAS_Q:
            c_q_off[c] = tq
            tq += c_len[c]
        else:
            c_q_off[c] = -1
    T, T_q = t, tq
    c_ref = [0] * n
    for c in range(n):
        for e in range(c, c_sub_end[c]):
            if c_flags[e] & SEG_SAMPLE_END:
                c_ref[c] += 1

    # -- step 4: ancestor CSR, root -> parent ----------------------------------
    anc_off = [0]
    anc_list = []
    for c in range(n):
        chain = []
        p = c_parent[c]
        while p >= 0:
            chain.append(p)
            p = c_parent[p]
        chain.reverse()
        anc_list.extend(chain)
        anc_off.append(len(anc_list))

    # -- step 5: pages ----------------------------------------------------------
    c_first_page = [0] * n
    c_n_pages = [0] * n
    page_seg, page_bs, page_valid, page_pos, page_ref, page_slot = [], [], [], [], [], []
    extents = None if free_extents is None else [list(e) for e in free_extents]
    bump = 0
    def take(size):
        nonlocal bump
        if extents is None:
            slot = bump
            bump += size
            return slot
        for e in extents:
            if e[1] >= size:
                slot = e[0]
                e[0] += size
                e[1] -= size
                return slot
        raise PlanError("POOL_FULL", f"no extent fits {size} slots")

    for c in range(n):
        bs = c_bs[c]
        if bs:
            sizes = [bs] * (-(-c_len[c] // bs))
        else:  # adaptive: the span in 128-slot pages, its tail in 16-slot pages
            tail = c_len[c] % 128
            sizes = [128] * (c_len[c] // 128) + [16] * (-(-tail // 16))
        npg = len(sizes)
        c_first_page[c] = len(page_seg)
        c_n_pages[c] = npg
        pinned = -1 if seg_slot_base is None else seg_slot_base[input_of_canon[c]]
        at = pinned if pinned >= 0 else (take(sum(sizes)) if not bs else -1)  # adaptive: one extent
        tok = 0
        for i in range(npg):
            if at >= 0:
                slot = at
                at += sizes[i]
            else:
                slot = take(sizes[i])
            page_seg.append(c)
            page_bs.append(sizes[i])
            page_valid.append(min(sizes[i], c_len[c] - tok))
            page_pos.append(c_anc[c] + tok)
            page_ref.append(c_ref[c])
            page_slot.append(slot)
            tok += sizes[i]
    n_pages = len(page_seg)
    pool_slots = max(page_slot[p] + page_bs[p] for p in range(n_pages))

    # -- step 6: block table CSR: ancestors' pages root -> parent, then own -----
    bt_off = [0]
    bt_pages = []
    for c in range(n):
        for a in anc_list[anc_off[c]:anc_off[c + 1]]:
            bt_pages.extend(range(c_first_page[a], c_first_page[a] + c_n_pages[a]))
        bt_pages.extend(range(c_first_page[c], c_first_page[c] + c_n_pages[c]))
        bt_off.append(len(bt_pages))

    # -- step 7: token -> slot ---------------------------------------------------
    tok_slot = [0] * T
    for c in range(n):
        i = 0
        for pg in range(c_first_page[c], c_first_page[c] + c_n_pages[c]):
            for j in range(page_valid[pg]):
                tok_slot[c_tok_off[c] + i] = page_slot[pg] + j
                i += 1

    # -- step 8: samples ----------------------------------------------------------
    sample_end_seg = [c for c in range(n) if c_flags[c] & SEG_SAMPLE_END]
    sample_len = [c_anc[c] + c_len[c] for c in sample_end_seg]

    # -- step 9: statistics --------------------------------------------------------
    flat_tokens = sum(sample_len)
    tree_pairs = sum(
        c_len[c] * c_anc[c] + c_len[c] * (c_len[c] + 1) // 2
        for c in range(n)
        if c_flags[c] & SEG_HAS_Q
    )
    flat_pairs = sum(L * (L + 1) // 2 for L in sample_len)

    return dict(
        n_seg=n,
        n_groups=len(roots),
        n_pages=n_pages,
        n_samples=len(sample_end_seg),
        max_depth=max(c_depth),
        T=T,
        T_q=T_q,
        pool_slots=pool_slots,
        flat_tokens=int(flat_tokens),
        tree_pairs=int(tree_pairs),
        flat_pairs=int(flat_pairs),
        canon_of_input=_i32(canon_of_input),
        input_of_canon=_i32(input_of_canon),
        seg_group=_i32(c_group),
        seg_bs=_i32(c_bs),
        seg_parent=_i32(c_parent),
        seg_len=_i32(c_len),
        seg_flags=_i32(c_flags),
        seg_depth=_i32(c_depth),
        seg_anc_tokens=_i32(c_anc),
        seg_sub_end=_i32(c_sub_end),
        seg_tok_off=_i32(c_tok_off),
        seg_q_off=_i32(c_q_off),
        seg_refcount=_i32(c_ref),
        anc_off=_i32(anc_off),
        anc_list=_i32(anc_list),
        seg_first_page=_i32(c_first_page),
        seg_n_pages=_i32(c_n_pages),
        page_seg=_i32(page_seg),
        page_bs=_i32(page_bs),
        page_valid=_i32(page_valid),
        page_pos=_i32(page_pos),
        page_refcount=_i32(page_ref),
        page_slot=_i32(page_slot),
        bt_off=_i32(bt_off),
        bt_pages=_i32(bt_pages),
        tok_slot=_i32(tok_slot),
        sample_end_seg=_i32(sample_end_seg),
        sample_len=_i32(sample_len),
    )


PLAN_ARRAYS = (
    "canon_of_input", "input_of_canon", "seg_group", "seg_bs", "seg_parent", "seg_len",
    "seg_flags", "seg_depth", "seg_anc_tokens", "seg_sub_end", "seg_tok_off", "seg_q_off",
    "seg_refcount", "anc_off", "anc_list", "seg_first_page", "seg_n_pages", "page_seg",
    "page_bs", "page_valid", "page_pos", "page_refcount", "page_slot", "bt_off", "bt_pages",
    "tok_slot", "sample_end_seg", "sample_len",
)
PLAN_SCALARS = (
    "n_seg", "n_groups", "n_pages", "n_samples", "max_depth", "T", "T_q", "pool_slots",
    "flat_tokens", "tree_pairs", "flat_pairs",
)
