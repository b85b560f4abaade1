"""Oracle for tree-causal prefix-shared attention.  TEST INFRASTRUCTURE ONLY.

The method reaches, up to rounding order, a result with a plain definition
(Sec. 2.5, "Prefix sharing in training": with the sequence-specific mask the
shared computation gives the same attention results as computing every
sequence on its own; Sec. 6, "Prefix-sharing training runtime": the adjoints
of all consumers are accumulated on the shared prefix).  The oracle is that
definition written out:

  for every sample (a root-to-end path of segments)
      materialise its tokens as one unshared causal sequence, in fp64
      for every query head h (KV head h // G, G = Hq // Hkv)
          S = scale * Q K^T, S_ij = -inf for j > i
          P = softmax_j(S), O = P V, LSE_i = log sum_j exp(S_ij)
          dV = P^T dO, dP = dO V^T, D_i = sum_d dO_id O_id
          dS = P * (dP - D), dQ = scale * dS K, dK = scale * dS^T Q
  scatter: O, LSE of a shared token are taken from its copy in the first
  sample that contains it; dQ, dK, dV of a shared token are the sums over all
  of its copies (dK, dV also over the G query heads of the KV head).

A shared token has ONE upstream gradient row dO (already accumulated over its
consumers); in the materialisation that row is handed to the copy in the first
sample (canonical order) containing the token and the other copies get zero.
Backward is linear in dO, so any other split that sums to dO gives the same
totals; `do_weights` lets a test use one.

No blocking, fusion or reordering beyond the row chunking that bounds memory
(rows of one sample are evaluated `row_chunk` at a time; every row still sees
its full key range at once).

Pins (tests/test_oracle_attention.py): central finite differences on tiny
trees; equality of O/LSE across all copies of a shared token; torch CPU fp64
scaled_dot_product_attention + autograd on the single-sequence and explicit
tree-mask special cases; closed forms (equal keys -> uniform P; constant V;
key-shift invariance; sum_j dS_ij = 0; sum dV = sum dO); a random dO split.
"""
from __future__ import annotations

import numpy as np

SEG_HAS_Q = 1


def sample_paths(plan):
    """For each sample: list of canonical segment indices root -> end."""
    out = []
    for e in plan["sample_end_seg"]:
        e = int(e)
        anc = plan["anc_list"][plan["anc_off"][e]:plan["anc_off"][e + 1]]
        out.append([int(a) for a in anc] + [e])
    return out


def _sample_tokens(plan, path):
    """Token ids (canonical), q rows (-1 where the segment issues no query)."""
    toks, qrows = [], []
    for c in path:
        n = int(plan["seg_len"][c])
        t0 = int(plan["seg_tok_off"][c])
        toks.append(np.arange(t0, t0 + n, dtype=np.int64))
        if int(plan["seg_flags"][c]) & SEG_HAS_Q:
            q0 = int(plan["seg_q_off"][c])
            qrows.append(np.arange(q0, q0 + n, dtype=np.int64))
        else:
            qrows.append(np.full(n, -1, dtype=np.int64))
    return np.concatenate(toks), np.concatenate(qrows)


def oracle_attn(plan, q, k_pool, v_pool, d_o, scale, *, q_rows=None, kv_heads=None,
                do_weights=None, row_chunk=1024, want_copies=False):
    """Forward and backward of tree attention by per-sample materialisation.

    q, d_o   [T_q, Hq, d]   rows in canonical query order; or, with `q_rows`
                            (sorted global row ids), [len(q_rows), Hq, d]
                            holding just those rows: only they are evaluated,
                            which is exact when every other dO row is zero
    k_pool, v_pool [Hkv, pool_slots, d], token t at slot plan['tok_slot'][t]
    kv_heads optional subset of KV heads to evaluate (heads are independent)
    do_weights optional list, one float array per sample over its path tokens:
             the share of the token's dO row given to that copy
    Returns dict O, LSE [Hq, rows], dQ, dK, dV (pool layout, zeros elsewhere);
    with want_copies also 'copies': per sample (row ids, O, LSE) of every copy.
    d_o may be None (forward only).
    """
    q = np.asarray(q)
    Hq, d = q.shape[1], q.shape[2]
    Hkv = k_pool.shape[0]
    G = Hq // Hkv
    nrows = q.shape[0]
    if q_rows is None:
        row_of = None
    else:
        q_rows = np.asarray(q_rows, dtype=np.int64)
        row_of = np.full(int(plan["T_q"]), -1, dtype=np.int64)
        row_of[q_rows] = np.arange(len(q_rows))
    heads = list(range(Hkv)) if kv_heads is None else [int(h) for h in kv_heads]
    bwd = d_o is not None

    O = np.full((nrows, Hq, d), np.nan)
    LSE = np.full((Hq, nrows), np.nan)
    dQ = np.zeros((nrows, Hq, d)) if bwd else None
    dK = np.zeros(k_pool.shape) if bwd else None
    dV = np.zeros(v_pool.shape) if bwd else None
    seen = np.zeros(int(plan["T"]), dtype=bool)  # token already had its first copy
    copies = []
    tok_slot = plan["tok_slot"].astype(np.int64)

    for k_idx, path in enumerate(sample_paths(plan)):
        toks, qrows = _sample_tokens(plan, path)
        L = len(toks)
        slots = tok_slot[toks]
        first = ~seen[toks]
        seen[toks] = True
        if do_weights is None:
            w = first.astype(np.float64)
        else:
            w = np.asarray(do_weights[k_idx], dtype=np.float64)
        # positions of this sample that issue a query we were asked to evaluate
        if row_of is None:
            local = qrows
        else:
            local = np.where(qrows >= 0, row_of[np.maximum(qrows, 0)], -1)
        keep = local >= 0
        if not want_copies:
            # a copy that is neither recorded (not the first) nor carries any
            # dO contributes exactly nothing: skip it
            keep &= first | (w != 0.0)
        pos = np.nonzero(keep)[0]
        if len(pos) == 0:
            continue
        rows = local[pos]
        for hk in heads:
            K = k_pool[hk, slots, :].astype(np.float64)
            V = v_pool[hk, slots, :].astype(np.float64)
            dKs = np.zeros((L, d)) if bwd else None
            dVs = np.zeros((L, d)) if bwd else None
            for g in range(G):
                h = hk * G + g
                for a in range(0, len(pos), row_chunk):
                    p = pos[a:a + row_chunk]
                    r = rows[a:a + row_chunk]
                    Qc = q[r, h, :].astype(np.float64)
                    S = scale * (Qc @ K.T)
                    S[np.arange(L)[None, :] > p[:, None]] = -np.inf
                    m = S.max(axis=1, keepdims=True)
                    E = np.exp(S - m)
                    den = E.sum(axis=1, keepdims=True)
                    P = E / den
                    Oc = P @ V
                    Lc = (m + np.log(den))[:, 0]
                    fc = first[p]
                    O[r[fc], h, :] = Oc[fc]
                    LSE[h, r[fc]] = Lc[fc]
                    if want_copies:
                        copies.append((k_idx, h, r.copy(), Oc, Lc))
                    if not bwd:
                        continue
                    dOc = d_o[r, h, :].astype(np.float64) * w[p][:, None]
                    dVs += P.T @ dOc
                    dP = dOc @ V.T
                    D = (dOc * Oc).sum(axis=1, keepdims=True)
                    dS = P * (dP - D)
                    dQ[r, h, :] += scale * (dS @ K)
                    dKs += scale * (dS.T @ Qc)
            if bwd:
                np.add.at(dK[hk], slots, dKs)
                np.add.at(dV[hk], slots, dVs)
    out = dict(O=O, LSE=LSE, dQ=dQ, dK=dK, dV=dV)
    if want_copies:
        out["copies"] = copies
    return out


def oracle_rows(plan, q_vals, k_pool, v_pool, rows, heads, n_q_heads, scale):
    """O and LSE of single (query row, query head) pairs, one by one.

    q_vals[i] is the query vector [d] of pair i = (rows[i], heads[i]).  The row
    sees every token of its ancestors and the tokens of its own segment up to
    and including itself (Sec. 2.5: the original autoregressive dependency).
    Returns O [n, d] and LSE [n] in fp64.
    """
    G = n_q_heads // k_pool.shape[0]
    tok_slot = plan["tok_slot"].astype(np.int64)
    q_off = plan["seg_q_off"]
    res_o, res_l = [], []
    for qv, row, h in zip(q_vals, rows, heads):
        row, h = int(row), int(h)
        c = -1
        for s in range(int(plan["n_seg"])):
            if q_off[s] >= 0 and q_off[s] <= row < q_off[s] + plan["seg_len"][s]:
                c = s
        i = row - int(q_off[c])
        toks = []
        for a in plan["anc_list"][plan["anc_off"][c]:plan["anc_off"][c + 1]]:
            t0 = int(plan["seg_tok_off"][a])
            toks.extend(range(t0, t0 + int(plan["seg_len"][a])))
        t0 = int(plan["seg_tok_off"][c])
        toks.extend(range(t0, t0 + i + 1))
        slots = tok_slot[np.asarray(toks)]
        K = k_pool[h // G, slots, :].astype(np.float64)
        V = v_pool[h // G, slots, :].astype(np.float64)
        s_ = scale * (K @ np.asarray(qv, dtype=np.float64))
        m = s_.max()
        e = np.exp(s_ - m)
        res_o.append((e / e.sum()) @ V)
        res_l.append(m + np.log(e.sum()))
    return np.asarray(res_o), np.asarray(res_l)
