"""Thin Python binding of ``libhpd.so`` (C ABI declared in ``include/hpd.h``).

Argument marshalling only: tensors are passed as raw device pointers together with the current
CUDA stream; every step of the path runs in the library's kernels.  PyTorch is used for device
memory and streams.  The library must be present -- there is no fallback; ``load()`` raises if
``libhpd.so`` has not been built (``python -m paper_2604_26209_b200.build``).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhpd.so")

EXPORTS = ("hpd_strerror", "hpd_last_cuda_error", "hpd_workspace_bytes", "hpd_build_meta", "hpd_rope",
           "hpd_kv_append", "hpd_rope_append", "hpd_attn_decode", "hpd_build_meta_skeleton", "hpd_attn_decode_posorder", "hpd_advance", "hpd_merge_lse", "hpd_prefill_meta", "hpd_prefill_attn", "hpd_attn_decode_shared", "std_workspace_bytes", "std_attn_decode",
           "std_attn_decode_static_max_bytes", "std_attn_decode_static")

HPD_S_OVERFLOW, HPD_S_BAD_TABLE, HPD_S_TIMEOUT = 1, 2, 4


class HpdGeom(C.Structure):
    _fields_ = [("Hq", C.c_int32), ("Hkv", C.c_int32), ("D", C.c_int32), ("rope_theta", C.c_float),
                ("sm_scale", C.c_float), ("suffix_cap", C.c_int32)]


class HpdError(RuntimeError):
    pass


_lib = None


def load() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise HpdError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_26209_b200.build` "
                           "(there is no CPU fallback)")
        lib = C.CDLL(LIB_PATH)
        lib.hpd_strerror.restype = C.c_char_p
        lib.hpd_strerror.argtypes = [C.c_int]
        lib.hpd_last_cuda_error.restype = C.c_int
        lib.hpd_workspace_bytes.restype = C.c_size_t
        lib.hpd_workspace_bytes.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, C.c_int]
        lib.std_workspace_bytes.restype = C.c_size_t
        lib.std_workspace_bytes.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int]
        vp = C.c_void_p
        lib.hpd_build_meta.restype = C.c_int
        lib.hpd_build_meta.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, vp, vp, vp, vp, C.c_int32] + [vp] * 10 + \
                                      [vp, C.c_size_t, vp, vp]
        lib.hpd_build_meta_skeleton.restype = C.c_int
        lib.hpd_build_meta_skeleton.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, vp, vp, vp, vp, vp, C.c_int32] + \
                                               [vp] * 11 + [vp, C.c_size_t, vp, vp]
        lib.hpd_attn_decode_posorder.restype = C.c_int
        lib.hpd_attn_decode_posorder.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, C.c_int, C.c_int] + [vp] * 15 + \
                                                [C.c_int, vp, vp, vp, C.c_size_t, vp, vp]
        lib.hpd_prefill_meta.restype = C.c_int
        lib.hpd_prefill_meta.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, C.c_int, vp, vp, vp, C.c_int32] + [vp] * 6 + \
                                        [vp, C.c_size_t, vp]
        lib.hpd_prefill_attn.restype = C.c_int
        lib.hpd_prefill_attn.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int] + [vp] * 10 + [vp, C.c_size_t, vp, vp]
        lib.hpd_attn_decode_shared.restype = C.c_int
        lib.hpd_attn_decode_shared.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, C.c_int, C.c_int] + [vp] * 7 + [C.c_int] + \
                                              [vp] * 10 + [C.c_int, vp, vp, vp, C.c_size_t, vp, vp]
        lib.hpd_merge_lse.restype = C.c_int
        lib.hpd_merge_lse.argtypes = [C.POINTER(HpdGeom), C.c_int] + [vp] * 8
        lib.hpd_advance.restype = C.c_int
        lib.hpd_advance.argtypes = [C.POINTER(HpdGeom), C.c_int, vp, vp, vp, C.c_int32, vp, vp, vp, vp]
        lib.hpd_rope.restype = C.c_int
        lib.hpd_rope.argtypes = [C.POINTER(HpdGeom), C.c_int, vp, vp, vp, vp, vp]
        lib.hpd_kv_append.restype = C.c_int
        lib.hpd_kv_append.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int] + [vp] * 9
        lib.hpd_rope_append.restype = C.c_int
        lib.hpd_rope_append.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int] + [vp] * 11
        lib.hpd_attn_decode.restype = C.c_int
        lib.hpd_attn_decode.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, C.c_int, C.c_int] + [vp] * 12 + \
                                       [C.c_int, vp, vp, vp, C.c_size_t, vp, vp]
        lib.std_attn_decode.restype = C.c_int
        lib.std_attn_decode.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, C.c_longlong] + [vp] * 8 + [vp, C.c_size_t, vp]
        lib.std_attn_decode_static_max_bytes.restype = C.c_size_t
        lib.std_attn_decode_static_max_bytes.argtypes = []
        lib.std_attn_decode_static.restype = C.c_int
        lib.std_attn_decode_static.argtypes = [C.POINTER(HpdGeom), C.c_int, C.c_int, C.c_longlong] + [vp] * 8 + [vp]
        _lib = lib
    return _lib


def make_geom(g) -> HpdGeom:
    return HpdGeom(int(g.Hq), int(g.Hkv), int(g.D), float(g.rope_theta), float(g.sm_scale), int(g.suffix_cap))


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, what: str):
    if rc != 0:
        lib = load()
        msg = lib.hpd_strerror(rc).decode()
        if rc == -5:
            msg += f" [cudaError {lib.hpd_last_cuda_error()}]"
        raise HpdError(f"{what}: {msg} ({rc})")


def hpd_workspace_bytes(geom, max_docs: int, max_slots: int, max_prefix_tokens: int) -> int:
    g = make_geom(geom)
    return int(load().hpd_workspace_bytes(C.byref(g), max_docs, max_slots, max_prefix_tokens))


def std_workspace_bytes(geom, max_rows: int, max_seq_len: int) -> int:
    g = make_geom(geom)
    return int(load().std_workspace_bytes(C.byref(g), max_rows, max_seq_len))


@dataclass
class MetaTables:
    """Device int32 tables written by ``hpd_build_meta`` (plus the workspace and status word)."""
    doc_kv_start: torch.Tensor
    doc_slot_start: torch.Tensor
    doc_active_start: torch.Tensor
    active_slot: torch.Tensor
    doc_id: torch.Tensor
    branch_start: torch.Tensor
    pos_id: torch.Tensor
    suffix_off: torch.Tensor
    suffix_len: torch.Tensor
    n_active: torch.Tensor
    workspace: torch.Tensor
    dev_status: torch.Tensor
    prefix_vis: Optional[torch.Tensor] = None      # position-order mode only

    NAMES = ("doc_kv_start", "doc_slot_start", "doc_active_start", "active_slot", "doc_id", "branch_start",
             "pos_id", "suffix_off", "suffix_len")

    @staticmethod
    def alloc(geom, n_docs: int, n_slots: int, total_prefix: int, device="cuda") -> "MetaTables":
        i32 = lambda n: torch.empty(max(n, 1), dtype=torch.int32, device=device)
        ws = torch.empty(max(hpd_workspace_bytes(geom, n_docs, n_slots, total_prefix), 256), dtype=torch.uint8, device=device)
        return MetaTables(i32(n_docs + 1), i32(n_docs + 1), i32(n_docs + 1), *[i32(n_slots) for _ in range(6)],
                          torch.zeros(1, dtype=torch.int32, device=device), ws,
                          torch.zeros(1, dtype=torch.int32, device=device), i32(n_slots))


def hpd_build_meta(geom, n_docs, n_slots, doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive, pos_gap, m: MetaTables):
    g = make_geom(geom)
    rc = load().hpd_build_meta(C.byref(g), n_docs, n_slots, _ptr(doc_prefix_len), _ptr(doc_branch_cnt), _ptr(slot_depth),
                               _ptr(slot_alive), int(pos_gap), _ptr(m.doc_kv_start), _ptr(m.doc_slot_start),
                               _ptr(m.doc_active_start), _ptr(m.active_slot), _ptr(m.doc_id), _ptr(m.branch_start),
                               _ptr(m.pos_id), _ptr(m.suffix_off), _ptr(m.suffix_len), _ptr(m.n_active),
                               _ptr(m.workspace), m.workspace.numel(), _ptr(m.dev_status), _stream())
    _check(rc, "hpd_build_meta")


def hpd_build_meta_skeleton(geom, n_docs, n_slots, doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive, slot_vis, pos_gap,
                            m: MetaTables):
    g = make_geom(geom)
    rc = load().hpd_build_meta_skeleton(C.byref(g), n_docs, n_slots, _ptr(doc_prefix_len), _ptr(doc_branch_cnt),
                                        _ptr(slot_depth), _ptr(slot_alive), _ptr(slot_vis), int(pos_gap),
                                        _ptr(m.doc_kv_start), _ptr(m.doc_slot_start), _ptr(m.doc_active_start),
                                        _ptr(m.active_slot), _ptr(m.doc_id), _ptr(m.branch_start), _ptr(m.pos_id),
                                        _ptr(m.suffix_off), _ptr(m.suffix_len), _ptr(m.prefix_vis), _ptr(m.n_active),
                                        _ptr(m.workspace), m.workspace.numel(), _ptr(m.dev_status), _stream())
    _check(rc, "hpd_build_meta_skeleton")


def hpd_attn_decode_posorder(geom, n_docs, max_rows, n_slots, total_prefix_tokens, q, prefix_k, prefix_v, suffix_k, suffix_v,
                             doc_prefix_len, slot_depth, slot_alive, m: MetaTables, suffix_includes_new, o, lse=None):
    g = make_geom(geom)
    rc = load().hpd_attn_decode_posorder(C.byref(g), n_docs, max_rows, n_slots, total_prefix_tokens, _ptr(q), _ptr(prefix_k),
                                         _ptr(prefix_v), _ptr(suffix_k), _ptr(suffix_v), _ptr(m.doc_kv_start),
                                         _ptr(doc_prefix_len), _ptr(m.doc_active_start), _ptr(m.doc_slot_start),
                                         _ptr(m.doc_id), _ptr(m.active_slot), _ptr(slot_depth), _ptr(slot_alive),
                                         _ptr(m.prefix_vis), _ptr(m.n_active), int(bool(suffix_includes_new)), _ptr(o),
                                         _ptr(lse), _ptr(m.workspace), m.workspace.numel(), _ptr(m.dev_status), _stream())
    _check(rc, "hpd_attn_decode_posorder")


@dataclass
class PrefillTables:
    """Device tables of the first inference step (``hpd_prefill_meta``)."""
    doc_kv_start: torch.Tensor
    doc_slot_start: torch.Tensor
    tok_doc: torch.Tensor
    tok_pos: torch.Tensor
    tok_vis: torch.Tensor
    n_tokens: torch.Tensor
    workspace: torch.Tensor
    dev_status: torch.Tensor

    @staticmethod
    def alloc(geom, n_docs: int, total_tokens: int, device="cuda") -> "PrefillTables":
        i32 = lambda n: torch.empty(max(n, 1), dtype=torch.int32, device=device)
        ws = torch.empty(max(hpd_workspace_bytes(geom, n_docs, total_tokens, total_tokens), 256), dtype=torch.uint8, device=device)
        return PrefillTables(i32(n_docs + 1), i32(n_docs + 1), i32(total_tokens), i32(total_tokens), i32(total_tokens),
                             torch.zeros(1, dtype=torch.int32, device=device), ws, torch.zeros(1, dtype=torch.int32, device=device))


def hpd_prefill_meta(geom, n_docs, n_slots, total_tokens, doc_prefix_len, doc_branch_cnt, slot_vis, pos_gap, t: PrefillTables):
    g = make_geom(geom)
    rc = load().hpd_prefill_meta(C.byref(g), n_docs, n_slots, total_tokens, _ptr(doc_prefix_len), _ptr(doc_branch_cnt),
                                 _ptr(slot_vis), int(pos_gap), _ptr(t.doc_kv_start), _ptr(t.doc_slot_start), _ptr(t.tok_doc),
                                 _ptr(t.tok_pos), _ptr(t.tok_vis), _ptr(t.n_tokens), _ptr(t.workspace), t.workspace.numel(),
                                 _stream())
    _check(rc, "hpd_prefill_meta")


def hpd_prefill_attn(geom, n_docs, total_tokens, q, prefix_k, prefix_v, doc_prefix_len, t: PrefillTables, o, lse=None):
    g = make_geom(geom)
    rc = load().hpd_prefill_attn(C.byref(g), n_docs, total_tokens, _ptr(q), _ptr(prefix_k), _ptr(prefix_v),
                                 _ptr(t.doc_kv_start), _ptr(doc_prefix_len), _ptr(t.tok_doc), _ptr(t.tok_vis), _ptr(t.n_tokens),
                                 _ptr(o), _ptr(lse), _ptr(t.workspace), t.workspace.numel(), _ptr(t.dev_status), _stream())
    _check(rc, "hpd_prefill_attn")


def hpd_attn_decode_shared(geom, n_docs, max_rows, n_slots, total_prefix_tokens, q, prefix_k, prefix_v, suffix_k, suffix_v,
                           block_k, block_v, total_block_tokens, doc_block, block_kv_start, block_len,
                           doc_prefix_len, m: MetaTables, suffix_includes_new, o, lse=None):
    g = make_geom(geom)
    rc = load().hpd_attn_decode_shared(C.byref(g), n_docs, max_rows, n_slots, total_prefix_tokens, _ptr(q), _ptr(prefix_k),
                                       _ptr(prefix_v), _ptr(suffix_k), _ptr(suffix_v), _ptr(block_k), _ptr(block_v),
                                       int(total_block_tokens), _ptr(doc_block), _ptr(block_kv_start), _ptr(block_len),
                                       _ptr(m.doc_kv_start), _ptr(doc_prefix_len), _ptr(m.doc_active_start), _ptr(m.doc_id),
                                       _ptr(m.suffix_off), _ptr(m.suffix_len), _ptr(m.n_active), int(bool(suffix_includes_new)),
                                       _ptr(o), _ptr(lse), _ptr(m.workspace), m.workspace.numel(), _ptr(m.dev_status), _stream())
    _check(rc, "hpd_attn_decode_shared")


def hpd_merge_lse(geom, max_rows, n_active, o_a, lse_a, o_b, lse_b, o, lse=None):
    g = make_geom(geom)
    rc = load().hpd_merge_lse(C.byref(g), max_rows, _ptr(n_active), _ptr(o_a), _ptr(lse_a), _ptr(o_b), _ptr(lse_b), _ptr(o),
                              _ptr(lse), _stream())
    _check(rc, "hpd_merge_lse")


def hpd_advance(geom, max_rows, n_active, active_slot, token_id, delimiter_id, slot_depth, slot_alive, n_alive):
    g = make_geom(geom)
    rc = load().hpd_advance(C.byref(g), max_rows, _ptr(n_active), _ptr(active_slot), _ptr(token_id), int(delimiter_id),
                            _ptr(slot_depth), _ptr(slot_alive), _ptr(n_alive), _stream())
    _check(rc, "hpd_advance")


def hpd_rope(geom, max_rows, n_active, pos_id, q, k_new):
    g = make_geom(geom)
    _check(load().hpd_rope(C.byref(g), max_rows, _ptr(n_active), _ptr(pos_id), _ptr(q), _ptr(k_new), _stream()), "hpd_rope")


def hpd_kv_append(geom, max_rows, n_slots, n_active, suffix_off, suffix_len, k_new, v_new, suffix_k, suffix_v, dev_status):
    g = make_geom(geom)
    rc = load().hpd_kv_append(C.byref(g), max_rows, n_slots, _ptr(n_active), _ptr(suffix_off), _ptr(suffix_len),
                              _ptr(k_new), _ptr(v_new), _ptr(suffix_k), _ptr(suffix_v), _ptr(dev_status), _stream())
    _check(rc, "hpd_kv_append")


def hpd_rope_append(geom, max_rows, n_slots, n_active, pos_id, suffix_off, suffix_len, q, k_new, v_new, suffix_k, suffix_v,
                    dev_status):
    g = make_geom(geom)
    rc = load().hpd_rope_append(C.byref(g), max_rows, n_slots, _ptr(n_active), _ptr(pos_id), _ptr(suffix_off),
                                _ptr(suffix_len), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(suffix_k), _ptr(suffix_v),
                                _ptr(dev_status), _stream())
    _check(rc, "hpd_rope_append")


def hpd_attn_decode(geom, n_docs, max_rows, n_slots, total_prefix_tokens, q, prefix_k, prefix_v, suffix_k, suffix_v,
                    doc_prefix_len, m: MetaTables, suffix_includes_new, o, lse=None):
    g = make_geom(geom)
    rc = load().hpd_attn_decode(C.byref(g), n_docs, max_rows, n_slots, total_prefix_tokens, _ptr(q), _ptr(prefix_k),
                                _ptr(prefix_v), _ptr(suffix_k), _ptr(suffix_v), _ptr(m.doc_kv_start),
                                _ptr(doc_prefix_len), _ptr(m.doc_active_start), _ptr(m.doc_id), _ptr(m.suffix_off),
                                _ptr(m.suffix_len), _ptr(m.n_active), int(bool(suffix_includes_new)), _ptr(o), _ptr(lse),
                                _ptr(m.workspace), m.workspace.numel(), _ptr(m.dev_status), _stream())
    _check(rc, "hpd_attn_decode")


def std_attn_decode(geom, max_rows, max_seq_len, n_active, q, dup_k, dup_v, seq_start, seq_len, o, lse=None,
                    workspace=None):
    g = make_geom(geom)
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().std_attn_decode(C.byref(g), max_rows, max_seq_len, int(dup_k.shape[0]), _ptr(n_active), _ptr(q), _ptr(dup_k), _ptr(dup_v),
                                _ptr(seq_start), _ptr(seq_len), _ptr(o), _ptr(lse), _ptr(workspace), wsb, _stream())
    _check(rc, "std_attn_decode")


def std_attn_decode_static_max_bytes() -> int:
    return int(load().std_attn_decode_static_max_bytes())


def std_attn_decode_static(geom, max_rows, max_seq_len, n_active, q, dup_k, dup_v, seq_start, seq_len, o, lse=None):
    """``std_attn_decode`` with the split-KV scratch inside the library (no workspace, no allocation).
    Returns the status code instead of raising when the problem exceeds the built-in scratch."""
    g = make_geom(geom)
    rc = load().std_attn_decode_static(C.byref(g), max_rows, max_seq_len, int(dup_k.shape[0]), _ptr(n_active), _ptr(q), _ptr(dup_k),
                                       _ptr(dup_v), _ptr(seq_start), _ptr(seq_len), _ptr(o), _ptr(lse), _stream())
    if rc != -3:
        _check(rc, "std_attn_decode_static")
    return rc
