"""Full-matrix formulation of the HPD decode step in numpy (fp64).  TEST INFRASTRUCTURE ONLY.

An independent second statement of what the C oracle computes, used to pin it on small
inputs.  It follows the paper's own picture of the computation (Sec. 4.3.2, Fig. 3a): all
tokens of a prompt live in ONE sequence in memory -- the stacked documents first, then the
generated value tokens appended step after step, out of logical order -- and a boolean
mask over that whole sequence says what each new token may see.  Under the conditional
independence of Eq. 4-6 with document-local context, a new token of branch n may see the
tokens of its own document and the tokens of branch n that are not deeper than itself.

No blocking and no per-branch loops over keys: one score matrix, one mask, one softmax.
"""
from __future__ import annotations

import numpy as np


def rope_table(pos: np.ndarray, D: int, theta: float):
    """cos/sin [len(pos), D/2] of pos * theta^(-2i/D)."""
    i = np.arange(D // 2, dtype=np.float64)
    inv_freq = np.power(np.float64(theta), -2.0 * i / np.float64(D))
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang), np.sin(ang)


def rope_rows(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """x [n, H, D] rotated at pos[n]; pairs are (i, i + D/2)."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    c, s = rope_table(pos, D, theta)
    c, s = c[:, None, :], s[:, None, :]
    a, b = x[..., : D // 2], x[..., D // 2:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def full_matrix_step(Hq, Hkv, D, theta, scale, doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive,
                     suffix_cap, pos_gap, q_slot, k_new_slot, v_new_slot, prefix_k, prefix_v, suffix_k, suffix_v):
    """All arrays fp64/fp32 values; ``q_slot, k_new_slot, v_new_slot`` are indexed by SLOT.

    Returns (o [n_active,Hq,D], lse [n_active,Hq], active_slots) with rows in ascending slot id.
    """
    L = np.asarray(doc_prefix_len, dtype=np.int64)
    cnt = np.asarray(doc_branch_cnt, dtype=np.int64)
    depth = np.asarray(slot_depth, dtype=np.int64)
    alive = np.asarray(slot_alive).astype(bool)
    n_docs, n_slots = len(L), len(depth)
    slot_doc = np.repeat(np.arange(n_docs), cnt)
    slot_j = np.concatenate([np.arange(c) for c in cnt]) if n_slots else np.zeros(0, np.int64)
    kv_start = np.concatenate([[0], np.cumsum(L)])
    G = Hq // Hkv

    # ---- the sequence in memory: stacked documents, then appended value tokens step by step ----
    tok_doc, tok_slot, tok_depth, Krows, Vrows = [], [], [], [], []
    for d in range(n_docs):
        for t in range(L[d]):
            tok_doc.append(d); tok_slot.append(-1); tok_depth.append(-1)
            Krows.append(prefix_k[kv_start[d] + t]); Vrows.append(prefix_v[kv_start[d] + t])
    max_depth = int(depth.max()) if n_slots else 0
    for t in range(max_depth):                       # earlier steps' tokens, step-major
        for s in range(n_slots):
            if depth[s] > t:
                tok_doc.append(slot_doc[s]); tok_slot.append(s); tok_depth.append(t)
                Krows.append(suffix_k[s * suffix_cap + t]); Vrows.append(suffix_v[s * suffix_cap + t])
    act = np.nonzero(alive)[0]
    pos_new = L[slot_doc[act]] + slot_j[act] * pos_gap + depth[act]
    k_rot = rope_rows(np.asarray(k_new_slot, dtype=np.float64)[act], pos_new, theta)
    q_rot = rope_rows(np.asarray(q_slot, dtype=np.float64)[act], pos_new, theta)
    for i, s in enumerate(act):                      # this step's tokens, appended last
        tok_doc.append(slot_doc[s]); tok_slot.append(s); tok_depth.append(depth[s])
        Krows.append(k_rot[i]); Vrows.append(np.asarray(v_new_slot, dtype=np.float64)[s])
    tok_doc, tok_slot, tok_depth = map(np.asarray, (tok_doc, tok_slot, tok_depth))
    Kall = np.asarray(Krows, dtype=np.float64).reshape(-1, Hkv, D)
    Vall = np.asarray(Vrows, dtype=np.float64).reshape(-1, Hkv, D)

    # ---- mask [n_active, n_tokens] ----
    q_doc, q_depth = slot_doc[act], depth[act]
    is_prefix = tok_slot[None, :] < 0
    same_doc = tok_doc[None, :] == q_doc[:, None]
    same_branch = tok_slot[None, :] == act[:, None]
    not_deeper = tok_depth[None, :] <= q_depth[:, None]
    mask = (is_prefix & same_doc) | (same_branch & not_deeper)

    o = np.empty((len(act), Hq, D), dtype=np.float64)
    lse = np.empty((len(act), Hq), dtype=np.float64)
    for h in range(Hq):
        S = (q_rot[:, h, :] @ Kall[:, h // G, :].T) * scale
        S = np.where(mask, S, -np.inf)
        m = S.max(axis=1, keepdims=True)
        E = np.exp(S - m)
        den = E.sum(axis=1, keepdims=True)
        o[:, h, :] = (E / den) @ Vall[:, h // G, :]
        lse[:, h] = (m + np.log(den))[:, 0]
    return o, lse, act
