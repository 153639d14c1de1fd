"""ctypes front-end of the C oracle (``hpd_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Argument marshalling only: numpy arrays in, numpy arrays out; every number is computed by
the C file.  Floating inputs are fp32 arrays (bf16 values widened exactly by the caller).
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Optional

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.hpdo_decode_step.restype = C.c_int
        _lib.hpdo_build_meta.restype = C.c_int
        _lib.hpdo_alg2_value_position.restype = C.c_int32
        _lib.hpdo_build_meta_skeleton.restype = C.c_int
        _lib.hpdo_advance.restype = C.c_int
        _lib.hpdo_decode_step_shared3.restype = C.c_int
        _lib.hpdo_prefill.restype = C.c_int
        _lib.hpdo_decode_step_posorder.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def alg2_position_ids(len_s: int, attr_start, attr_end, k_max: int) -> np.ndarray:
    """Algorithm 2: position IDs of the model input with a K_max gap after every attribute."""
    st, en = _i32(attr_start), _i32(attr_end)
    out = np.empty(len_s, dtype=np.int32)
    lib().hpdo_alg2_position_ids(C.c_int(len_s), C.c_int(len(st)), _p(st), _p(en), C.c_int(k_max), _p(out))
    return out


def alg2_value_position(pos_id, attr_end, n: int, k: int) -> int:
    pi, en = _i32(pos_id), _i32(attr_end)
    return int(lib().hpdo_alg2_value_position(_p(pi), _p(en), C.c_int(n), C.c_int(k)))


@dataclass
class Meta:
    doc_kv_start: np.ndarray
    doc_slot_start: np.ndarray
    doc_active_start: np.ndarray
    active_slot: np.ndarray
    doc_id: np.ndarray
    branch_start: np.ndarray
    pos_id: np.ndarray
    suffix_off: np.ndarray
    suffix_len: np.ndarray
    n_active: int

    TABLES = ("doc_kv_start", "doc_slot_start", "doc_active_start", "active_slot", "doc_id",
              "branch_start", "pos_id", "suffix_off", "suffix_len")


def build_meta(doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive, suffix_cap: int, pos_gap: int = 0) -> Meta:
    L, cnt, dep = _i32(doc_prefix_len), _i32(doc_branch_cnt), _i32(slot_depth)
    alive = np.ascontiguousarray(slot_alive, dtype=np.uint8)
    nd, ns = len(L), len(dep)
    z = lambda n: np.full(n, -7, dtype=np.int32)
    m = Meta(z(nd + 1), z(nd + 1), z(nd + 1), z(ns), z(ns), z(ns), z(ns), z(ns), z(ns), 0)
    na = np.zeros(1, dtype=np.int32)
    rc = lib().hpdo_build_meta(C.c_int(nd), C.c_int(ns), _p(L), _p(cnt), _p(dep), _p(alive),
                               C.c_int32(suffix_cap), C.c_int32(pos_gap),
                               _p(m.doc_kv_start), _p(m.doc_slot_start), _p(m.doc_active_start),
                               _p(m.active_slot), _p(m.doc_id), _p(m.branch_start), _p(m.pos_id),
                               _p(m.suffix_off), _p(m.suffix_len), _p(na))
    if rc != 0:
        raise ValueError("oracle build_meta: inconsistent arguments")
    m.n_active = int(na[0])
    return m


def rope(x: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """x [n_heads, D] fp32 -> rotated fp64."""
    x = _f32(x)
    nh, D = x.shape
    out = np.empty((nh, D), dtype=np.float64)
    lib().hpdo_rope(C.c_int(nh), C.c_int(D), C.c_double(theta), C.c_int32(int(pos)), _p(x), _p(out))
    return out


def causal_attention_row(row: int, q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float):
    """q [Hq,D], K,V [n,Hkv,D] fp64; the query sits at index ``row``.  Returns (o [Hq,D], lse [Hq])."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    Hq, D = q.shape
    Hkv = K.shape[1]
    assert K.shape[0] >= row + 1 and V.shape == K.shape
    o = np.empty((Hq, D), dtype=np.float64)
    lse = np.empty(Hq, dtype=np.float64)
    sc = np.empty(row + 1, dtype=np.float64)
    lib().hpdo_causal_attention_row(C.c_int(row), C.c_int(Hq), C.c_int(Hkv), C.c_int(D), C.c_double(scale),
                                    _p(q), _p(K), _p(V), _p(o), _p(lse), _p(sc))
    return o, lse


@dataclass
class StepOut:
    o: np.ndarray
    lse: np.ndarray
    q_rot: np.ndarray
    k_rot: np.ndarray
    threads: int


def decode_step(geom, meta: Meta, doc_prefix_len, q, k_new, v_new, prefix_k, prefix_v, suffix_k, suffix_v,
                n_threads: int = 0, rows: Optional[np.ndarray] = None) -> StepOut:
    """One decode step for the live branches.  ``q, k_new, v_new`` are per ACTIVE ROW fp32 arrays.
    ``rows`` (optional) restricts the evaluation to a subset of active rows (sampling at full size)."""
    n = meta.n_active
    doc_id, pos_id = meta.doc_id[:n], meta.pos_id[:n]
    soff, slen = meta.suffix_off[:n], meta.suffix_len[:n]
    q, k_new, v_new = _f32(q), _f32(k_new), _f32(v_new)
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        doc_id, pos_id, soff, slen = (_i32(a[rows]) for a in (doc_id, pos_id, soff, slen))
        q, k_new, v_new = _f32(q[rows]), _f32(k_new[rows]), _f32(v_new[rows])
        n = len(rows)
    else:
        doc_id, pos_id, soff, slen = _i32(doc_id), _i32(pos_id), _i32(soff), _i32(slen)
    assert q.shape == (n, geom.Hq, geom.D) and k_new.shape == (n, geom.Hkv, geom.D)
    prefix_k, prefix_v, suffix_k, suffix_v = _f32(prefix_k), _f32(prefix_v), _f32(suffix_k), _f32(suffix_v)
    L = _i32(doc_prefix_len)
    o = np.empty((n, geom.Hq, geom.D), dtype=np.float32)
    lse = np.empty((n, geom.Hq), dtype=np.float32)
    q_rot = np.empty((n, geom.Hq, geom.D), dtype=np.float32)
    k_rot = np.empty((n, geom.Hkv, geom.D), dtype=np.float32)
    used = lib().hpdo_decode_step(C.c_int(geom.Hq), C.c_int(geom.Hkv), C.c_int(geom.D),
                                  C.c_double(geom.rope_theta), C.c_double(geom.sm_scale), C.c_int(n),
                                  _p(doc_id), _p(pos_id), _p(soff), _p(slen), _p(meta.doc_kv_start), _p(L),
                                  _p(q), _p(k_new), _p(v_new), _p(prefix_k), _p(prefix_v),
                                  _p(suffix_k), _p(suffix_v), _p(o), _p(lse), _p(q_rot), _p(k_rot),
                                  C.c_int(n_threads))
    if used < 0:
        raise MemoryError("oracle decode_step: allocation failed")
    return StepOut(o, lse, q_rot, k_rot, used)


def kv_append(geom, meta: Meta, k_rot, v_new, suffix_k: np.ndarray, suffix_v: np.ndarray) -> np.ndarray:
    """In-place append into fp32 branch caches; returns the per-row overflow flags."""
    n = meta.n_active
    assert suffix_k.dtype == np.float32 and suffix_k.flags.c_contiguous
    assert suffix_v.dtype == np.float32 and suffix_v.flags.c_contiguous
    k_rot, v_new = _f32(k_rot), _f32(v_new)
    soff, slen = _i32(meta.suffix_off[:n]), _i32(meta.suffix_len[:n])
    ovf = np.zeros(n, dtype=np.uint8)
    lib().hpdo_kv_append(C.c_int(geom.Hkv), C.c_int(geom.D), C.c_int(n), C.c_int32(geom.suffix_cap),
                         _p(soff), _p(slen), _p(k_rot), _p(v_new), _p(suffix_k), _p(suffix_v), _p(ovf))
    return ovf


# ------------------------------------------------------------------------------------------
# position-order mode (Sec. 4.3.2, Fig. 3, Sec. 4.4)
# ------------------------------------------------------------------------------------------
def build_meta_skeleton(doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive, slot_vis, suffix_cap: int, pos_gap: int):
    """Tables of the position-order mode: ``(Meta, prefix_vis)``; ``slot_vis[s]`` = prefix tokens of the group up to and
    including the slot's attribute key."""
    L, cnt, dep, vis = _i32(doc_prefix_len), _i32(doc_branch_cnt), _i32(slot_depth), _i32(slot_vis)
    alive = np.ascontiguousarray(slot_alive, dtype=np.uint8)
    nd, ns = len(L), len(dep)
    z = lambda n: np.full(n, -7, dtype=np.int32)
    m = Meta(z(nd + 1), z(nd + 1), z(nd + 1), z(ns), z(ns), z(ns), z(ns), z(ns), z(ns), 0)
    pv = z(ns)
    na = np.zeros(1, dtype=np.int32)
    rc = lib().hpdo_build_meta_skeleton(C.c_int(nd), C.c_int(ns), _p(L), _p(cnt), _p(dep), _p(alive), _p(vis),
                                        C.c_int32(suffix_cap), C.c_int32(pos_gap),
                                        _p(m.doc_kv_start), _p(m.doc_slot_start), _p(m.doc_active_start),
                                        _p(m.active_slot), _p(m.doc_id), _p(m.branch_start), _p(m.pos_id),
                                        _p(m.suffix_off), _p(m.suffix_len), _p(pv), _p(na))
    if rc != 0:
        raise ValueError("oracle build_meta_skeleton: inconsistent arguments")
    m.n_active = int(na[0])
    return m, pv


def decode_step_posorder(geom, meta: Meta, doc_prefix_len, slot_depth, slot_alive, slot_vis, k_max: int,
                         q, k_new, v_new, prefix_k, prefix_v, suffix_k, suffix_v, n_threads: int = 0):
    """One decode step under the position-order mask.  ``q, k_new, v_new`` per ACTIVE ROW (fp32).
    Returns (StepOut, positions of the rows' new tokens)."""
    n = meta.n_active
    q, k_new, v_new = _f32(q), _f32(k_new), _f32(v_new)
    assert q.shape == (n, geom.Hq, geom.D) and k_new.shape == (n, geom.Hkv, geom.D)
    prefix_k, prefix_v, suffix_k, suffix_v = _f32(prefix_k), _f32(prefix_v), _f32(suffix_k), _f32(suffix_v)
    L, dep, vis = _i32(doc_prefix_len), _i32(slot_depth), _i32(slot_vis)
    alive = np.ascontiguousarray(slot_alive, dtype=np.uint8)
    act, did = _i32(meta.active_slot[:n]), _i32(meta.doc_id[:n])
    o = np.empty((n, geom.Hq, geom.D), dtype=np.float32)
    lse = np.empty((n, geom.Hq), dtype=np.float32)
    q_rot = np.empty((n, geom.Hq, geom.D), dtype=np.float32)
    k_rot = np.empty((n, geom.Hkv, geom.D), dtype=np.float32)
    pos = np.empty(max(n, 1), dtype=np.int32)
    used = lib().hpdo_decode_step_posorder(
        C.c_int(geom.Hq), C.c_int(geom.Hkv), C.c_int(geom.D), C.c_double(geom.rope_theta), C.c_double(geom.sm_scale),
        _p(L), _p(meta.doc_kv_start), _p(meta.doc_slot_start), _p(dep), _p(alive), _p(vis),
        C.c_int32(geom.suffix_cap), C.c_int32(k_max), C.c_int(n), _p(act), _p(did),
        _p(q), _p(k_new), _p(v_new), _p(prefix_k), _p(prefix_v), _p(suffix_k), _p(suffix_v),
        _p(o), _p(lse), _p(q_rot), _p(k_rot), _p(pos), C.c_int(n_threads))
    if used < 0:
        raise MemoryError("oracle decode_step_posorder: allocation failed")
    return StepOut(o, lse, q_rot, k_rot, used), pos[:n]


def advance(meta: Meta, token_id, delimiter: int, k_max: int, slot_depth: np.ndarray, slot_alive: np.ndarray) -> int:
    """End of a step (Sec. 4.3.4), in place on int32 ``slot_depth`` / uint8 ``slot_alive``; returns rows still alive."""
    assert slot_depth.dtype == np.int32 and slot_alive.dtype == np.uint8
    n = meta.n_active
    act, tok = _i32(meta.active_slot[:n]), _i32(token_id)
    assert len(tok) >= n
    return int(lib().hpdo_advance(C.c_int(n), _p(act), _p(tok), C.c_int32(delimiter), C.c_int32(k_max),
                                  _p(slot_depth), _p(slot_alive)))


def decode_step_shared3(geom, meta: Meta, doc_prefix_len, doc_block, block_len, q, k_new, v_new, block_k, block_v,
                        prefix_k, prefix_v, suffix_k, suffix_v, n_threads: int = 0):
    """One decode step with three sharing levels (Sec. 4.3.5): block ``doc_block[d]`` of ``block_len`` tokens precedes
    document d.  ``meta`` are the ordinary tables of the documents.  Returns (StepOut, positions)."""
    n = meta.n_active
    q, k_new, v_new = _f32(q), _f32(k_new), _f32(v_new)
    blk, bl = _i32(doc_block), _i32(block_len)
    bstart = _i32(np.concatenate([[0], np.cumsum(bl)])[:-1])
    L = _i32(doc_prefix_len)
    did, soff, slen = _i32(meta.doc_id[:n]), _i32(meta.suffix_off[:n]), _i32(meta.suffix_len[:n])
    block_k, block_v, prefix_k, prefix_v = _f32(block_k), _f32(block_v), _f32(prefix_k), _f32(prefix_v)
    suffix_k, suffix_v = _f32(suffix_k), _f32(suffix_v)
    o = np.empty((n, geom.Hq, geom.D), dtype=np.float32)
    lse = np.empty((n, geom.Hq), dtype=np.float32)
    q_rot = np.empty((n, geom.Hq, geom.D), dtype=np.float32)
    k_rot = np.empty((n, geom.Hkv, geom.D), dtype=np.float32)
    pos = np.empty(max(n, 1), dtype=np.int32)
    used = lib().hpdo_decode_step_shared3(
        C.c_int(geom.Hq), C.c_int(geom.Hkv), C.c_int(geom.D), C.c_double(geom.rope_theta), C.c_double(geom.sm_scale),
        C.c_int(n), _p(did), _p(blk), _p(bstart), _p(bl), _p(soff), _p(slen), _p(meta.doc_kv_start), _p(L),
        _p(q), _p(k_new), _p(v_new), _p(block_k), _p(block_v), _p(prefix_k), _p(prefix_v), _p(suffix_k), _p(suffix_v),
        _p(o), _p(lse), _p(q_rot), _p(k_rot), _p(pos), C.c_int(n_threads))
    if used < 0:
        raise MemoryError("oracle decode_step_shared3: allocation failed")
    return StepOut(o, lse, q_rot, k_rot, used), pos[:n]


def merge_lse(o_a, lse_a, o_b, lse_b):
    """Combine two attention results over disjoint key sets; arrays [..., D] and [...]."""
    o_a = np.ascontiguousarray(o_a, dtype=np.float64); o_b = np.ascontiguousarray(o_b, dtype=np.float64)
    la = np.ascontiguousarray(lse_a, dtype=np.float64); lb = np.ascontiguousarray(lse_b, dtype=np.float64)
    D = o_a.shape[-1]
    n = la.size
    o = np.empty_like(o_a); lse = np.empty_like(la)
    lib().hpdo_merge_lse(C.c_int(n), C.c_int(D), _p(o_a), _p(la), _p(o_b), _p(lb), _p(o), _p(lse))
    return o, lse


def prefill(geom, doc_prefix_len, doc_branch_cnt, slot_vis, k_max: int, q, k, v, n_threads: int = 0):
    """First inference step (Sec. 4.3.2): causal attention of every prompt token with Algorithm 2's position IDs.
    ``q [T,Hq,D]``, ``k, v [T,Hkv,D]`` fp32 for the T prompt tokens.  Returns (StepOut over all T rows, positions [T])."""
    L, cnt, vis = _i32(doc_prefix_len), _i32(doc_branch_cnt), _i32(slot_vis)
    q, k, v = _f32(q), _f32(k), _f32(v)
    T = int(L.sum())
    assert q.shape == (T, geom.Hq, geom.D) and k.shape == (T, geom.Hkv, geom.D) and v.shape == k.shape
    o = np.empty((T, geom.Hq, geom.D), dtype=np.float32)
    lse = np.empty((T, geom.Hq), dtype=np.float32)
    q_rot = np.empty((T, geom.Hq, geom.D), dtype=np.float32)
    k_rot = np.empty((T, geom.Hkv, geom.D), dtype=np.float32)
    pos = np.empty(max(T, 1), dtype=np.int32)
    used = lib().hpdo_prefill(C.c_int(geom.Hq), C.c_int(geom.Hkv), C.c_int(geom.D), C.c_double(geom.rope_theta),
                              C.c_double(geom.sm_scale), C.c_int(len(L)), _p(L), _p(cnt), _p(vis), C.c_int32(k_max),
                              _p(q), _p(k), _p(v), _p(o), _p(lse), _p(q_rot), _p(k_rot), _p(pos), C.c_int(n_threads))
    if used < 0:
        raise MemoryError("oracle prefill: allocation failed")
    return StepOut(o, lse, q_rot, k_rot, used), pos[:T]
