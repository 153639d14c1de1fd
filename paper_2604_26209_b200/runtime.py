"""Device-side plumbing around the C-ABI calls: upload a synthetic batch and run decode steps.

Holds no arithmetic of the method: tensors are moved to the GPU with PyTorch and every step of
the path (bookkeeping, rope, append, attention) is a call into ``libhpd.so``.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding as B
from .synth import Structure


def _bf16(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    """bf16 device tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class DeviceBatch:
    """One layer's decode state of a synthetic batch on the GPU."""

    def __init__(self, s: Structure, t: Dict[str, np.ndarray], device="cuda", posorder: Optional[bool] = None):
        self.s, self.g, self.device = s, s.geom, device
        # a structure with per-slot anchors runs the position-order mask unless told that they are anchors only
        self.posorder = (s.slot_vis is not None) if posorder is None else posorder
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.doc_prefix_len = i32(s.doc_prefix_len) if s.n_docs else torch.zeros(1, dtype=torch.int32, device=device)
        self.doc_branch_cnt = i32(s.doc_branch_cnt) if s.n_docs else torch.zeros(1, dtype=torch.int32, device=device)
        self.slot_depth = i32(s.slot_depth) if s.n_slots else torch.zeros(1, dtype=torch.int32, device=device)
        self.slot_alive = (torch.from_numpy(np.ascontiguousarray(s.slot_alive, dtype=np.uint8)).to(device)
                           if s.n_slots else torch.zeros(1, dtype=torch.uint8, device=device))
        self.prefix_k = _bf16(t["prefix_k"], device) if s.total_prefix else torch.zeros(8, dtype=torch.bfloat16, device=device)
        self.prefix_v = _bf16(t["prefix_v"], device) if s.total_prefix else torch.zeros(8, dtype=torch.bfloat16, device=device)
        self.suffix_k = _bf16(t["suffix_k"], device) if s.n_slots else torch.zeros(8, dtype=torch.bfloat16, device=device)
        self.suffix_v = _bf16(t["suffix_v"], device) if s.n_slots else torch.zeros(8, dtype=torch.bfloat16, device=device)
        self.slot_vis = i32(s.slot_vis) if (s.slot_vis is not None and s.n_slots) else None     # position-order workloads
        self.meta = B.MetaTables.alloc(self.g, s.n_docs, s.n_slots, s.total_prefix, device)
        n = max(s.n_slots, 1)
        self.q = torch.zeros(n, self.g.Hq, self.g.D, dtype=torch.bfloat16, device=device)
        self.k_new = torch.zeros(n, self.g.Hkv, self.g.D, dtype=torch.bfloat16, device=device)
        self.v_new = torch.zeros(n, self.g.Hkv, self.g.D, dtype=torch.bfloat16, device=device)
        self.o = torch.zeros(n, self.g.Hq, self.g.D, dtype=torch.bfloat16, device=device)
        self.lse = torch.zeros(n, self.g.Hq, dtype=torch.float32, device=device)

    # -- the C-ABI calls, in the order of one step -------------------------------------------
    def build_meta(self):
        s = self.s
        if self.slot_vis is not None:
            B.hpd_build_meta_skeleton(self.g, s.n_docs, s.n_slots, self.doc_prefix_len, self.doc_branch_cnt, self.slot_depth,
                                      self.slot_alive, self.slot_vis, s.pos_gap, self.meta)
            return
        B.hpd_build_meta(self.g, s.n_docs, s.n_slots, self.doc_prefix_len, self.doc_branch_cnt, self.slot_depth,
                         self.slot_alive, s.pos_gap, self.meta)

    def set_step_inputs(self, q_rows: np.ndarray, k_rows: np.ndarray, v_rows: np.ndarray):
        """Copy the step's new-token activations (bf16 bits, one row per ACTIVE row) to the device."""
        n = q_rows.shape[0]
        if n:
            self.q[:n].copy_(_bf16(q_rows, self.device))
            self.k_new[:n].copy_(_bf16(k_rows, self.device))
            self.v_new[:n].copy_(_bf16(v_rows, self.device))

    def rope(self):
        B.hpd_rope(self.g, self.s.n_slots, self.meta.n_active, self.meta.pos_id, self.q, self.k_new)

    def kv_append(self):
        B.hpd_kv_append(self.g, self.s.n_slots, self.s.n_slots, self.meta.n_active, self.meta.suffix_off,
                        self.meta.suffix_len, self.k_new, self.v_new, self.suffix_k, self.suffix_v, self.meta.dev_status)

    def rope_append(self):
        B.hpd_rope_append(self.g, self.s.n_slots, self.s.n_slots, self.meta.n_active, self.meta.pos_id,
                          self.meta.suffix_off, self.meta.suffix_len, self.q, self.k_new, self.v_new, self.suffix_k,
                          self.suffix_v, self.meta.dev_status)

    def attn(self, suffix_includes_new=True, lse=True):
        s = self.s
        if self.posorder:
            B.hpd_attn_decode_posorder(self.g, s.n_docs, s.n_slots, s.n_slots, s.total_prefix, self.q, self.prefix_k,
                                       self.prefix_v, self.suffix_k, self.suffix_v, self.doc_prefix_len, self.slot_depth,
                                       self.slot_alive, self.meta, suffix_includes_new, self.o, self.lse if lse else None)
            return
        B.hpd_attn_decode(self.g, s.n_docs, s.n_slots, s.n_slots, s.total_prefix, self.q, self.prefix_k, self.prefix_v,
                          self.suffix_k, self.suffix_v, self.doc_prefix_len, self.meta, suffix_includes_new, self.o,
                          self.lse if lse else None)

    def step(self, with_meta=True, fused=True):
        """One decode step; ``fused`` rotates and appends in one launch (hpd_rope_append) instead of two."""
        if with_meta:
            self.build_meta()
        if fused:
            self.rope_append()
        else:
            self.rope()
            self.kv_append()
        self.attn(True)

    def capture_step(self, with_meta=True, fused=True):
        """The step's launches captured once in a CUDA graph (call step() at least once before: the first call sets
        kernel attributes and builds tensor maps).  replay() then runs the same kernels without a host call each."""
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            self.step(with_meta=with_meta, fused=fused)
        return g

    # -- read-back --------------------------------------------------------------------------
    def tables(self) -> Dict[str, np.ndarray]:
        s = self.s
        out = {}
        names = B.MetaTables.NAMES + (("prefix_vis",) if self.slot_vis is not None else ())
        for name in names:
            a = getattr(self.meta, name).cpu().numpy()
            n = s.n_docs + 1 if name.startswith("doc_") and name != "doc_id" else s.n_slots
            out[name] = a[:n].copy()
        out["n_active"] = int(self.meta.n_active.item())
        return out

    def status(self) -> int:
        return int(self.meta.dev_status.item())


class SharedBlockBatch:
    """Three sharing levels (Sec. 4.3.5): blocks of tokens common to several documents, the documents, the branches.
    ``attn()`` is one hpd_attn_decode_shared launch; ``attn_two_pass()`` is the same result from two hpd_attn_decode
    calls -- rows against their document and branch cache, rows against their block -- and hpd_merge_lse.  ``doc_block[d]`` = block of document d (blocks cover consecutive documents), ``block_len[b]`` tokens,
    ``block_k/v`` bf16 bits [sum block_len, Hkv, D]."""

    def __init__(self, s: Structure, t: Dict[str, np.ndarray], doc_block: np.ndarray, block_len: np.ndarray,
                 block_k: np.ndarray, block_v: np.ndarray, device="cuda"):
        from dataclasses import replace
        doc_block = np.asarray(doc_block, dtype=np.int64)
        assert np.all(np.diff(doc_block) >= 0), "blocks cover consecutive documents"
        self.n_blocks = int(len(block_len))
        anchor = (np.asarray(block_len, np.int64)[doc_block] + s.doc_prefix_len)[s.slot_doc()].astype(np.int32)
        self.db = DeviceBatch(replace(s, slot_vis=anchor, pos_gap=0), t, device, posorder=False)
        g = s.geom
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        cnt = np.zeros(self.n_blocks, np.int64)
        np.add.at(cnt, doc_block, s.doc_branch_cnt)
        self.block_len, self.block_cnt = i32(block_len), i32(cnt)
        self.doc_block = i32(doc_block)
        self.block_kv_start = i32(np.concatenate([[0], np.cumsum(block_len)])[:-1])
        self.total_block = int(np.sum(block_len))
        self.block_k = _bf16(block_k, device) if self.total_block else torch.zeros(8, dtype=torch.bfloat16, device=device)
        self.block_v = _bf16(block_v, device) if self.total_block else torch.zeros(8, dtype=torch.bfloat16, device=device)
        self.meta_b = B.MetaTables.alloc(g, self.n_blocks, s.n_slots, self.total_block, device)
        zeros = torch.zeros(max(s.n_slots, 1), dtype=torch.int32, device=device)
        self.meta_b_nosuffix = replace(self.meta_b, suffix_off=zeros, suffix_len=zeros)
        self.o_b = torch.zeros_like(self.db.o)
        self.lse_b = torch.zeros_like(self.db.lse)

    def build_meta(self):
        db, s = self.db, self.db.s
        db.build_meta()
        B.hpd_build_meta(self.db.g, self.n_blocks, s.n_slots, self.block_len, self.block_cnt, db.slot_depth, db.slot_alive, 0,
                         self.meta_b)

    def attn(self, lse=True):
        db, s, g = self.db, self.db.s, self.db.g
        B.hpd_attn_decode_shared(g, s.n_docs, s.n_slots, s.n_slots, s.total_prefix, db.q, db.prefix_k, db.prefix_v, db.suffix_k,
                                 db.suffix_v, self.block_k, self.block_v, self.total_block, self.doc_block, self.block_kv_start,
                                 self.block_len, db.doc_prefix_len, db.meta, True, db.o, db.lse if lse else None)

    def attn_two_pass(self):
        db, s, g = self.db, self.db.s, self.db.g
        db.attn(True, lse=True)
        B.hpd_attn_decode(g, self.n_blocks, s.n_slots, s.n_slots, self.total_block, db.q, self.block_k, self.block_v,
                          db.suffix_k, db.suffix_v, self.block_len, self.meta_b_nosuffix, False, self.o_b, self.lse_b)
        B.hpd_merge_lse(g, s.n_slots, db.meta.n_active, db.o, db.lse, self.o_b, self.lse_b, db.o, db.lse)

    def step(self, two_pass=False):
        if two_pass:
            self.build_meta()
        else:
            self.db.build_meta()
        self.db.rope_append()
        self.attn_two_pass() if two_pass else self.attn()


class DupBatch:
    """Duplicated-prefix layout for ``std_attn_decode``: every active row gets a private physical copy
    [its document's prefix ; its cached branch tokens (new token included)].  Built with torch gathers
    (data preparation for the comparison, not part of the timed path)."""

    def __init__(self, db: DeviceBatch, include_new: bool = True, rows: Optional[int] = None):
        g, dev = db.g, db.device
        t = db.tables()
        n = t["n_active"] if rows is None else min(rows, t["n_active"])
        self.n = n
        doc = t["doc_id"][:n].astype(np.int64)
        L = db.s.doc_prefix_len.astype(np.int64)[doc] if n else np.zeros(0, np.int64)
        sl = t["suffix_len"][:n].astype(np.int64) + (1 if include_new else 0)
        sl = np.minimum(sl, g.suffix_cap)
        lens = L + sl
        start = np.concatenate([[0], np.cumsum(lens)])[:-1] if n else np.zeros(0, np.int64)
        total = int(lens.sum())
        self.max_seq_len = int(lens.max()) if n else 0
        self.total_tokens = total
        self.seq_start = torch.from_numpy(start.astype(np.int64)).to(dev) if n else torch.zeros(1, dtype=torch.int64, device=dev)
        self.seq_len = torch.from_numpy(lens.astype(np.int32)).to(dev) if n else torch.zeros(1, dtype=torch.int32, device=dev)
        self.n_active = torch.tensor([n], dtype=torch.int32, device=dev)
        self.dup_k = torch.empty(max(total, 1), g.Hkv, g.D, dtype=torch.bfloat16, device=dev)
        self.dup_v = torch.empty(max(total, 1), g.Hkv, g.D, dtype=torch.bfloat16, device=dev)
        kv0 = t["doc_kv_start"].astype(np.int64)
        soff = t["suffix_off"][:n].astype(np.int64)
        # chunked gather: index tensors of a few million entries at a time
        CH = 2048
        for lo in range(0, n, CH):
            hi = min(n, lo + CH)
            src_p, src_s, dst_p, dst_s = [], [], [], []
            for r in range(lo, hi):
                src_p.append(np.arange(kv0[doc[r]], kv0[doc[r]] + L[r]))
                dst_p.append(np.arange(start[r], start[r] + L[r]))
                src_s.append(np.arange(soff[r], soff[r] + sl[r]))
                dst_s.append(np.arange(start[r] + L[r], start[r] + lens[r]))
            for src, dst, K, V in ((src_p, dst_p, db.prefix_k, db.prefix_v), (src_s, dst_s, db.suffix_k, db.suffix_v)):
                si = torch.from_numpy(np.concatenate(src)).to(dev)
                di = torch.from_numpy(np.concatenate(dst)).to(dev)
                if si.numel():
                    self.dup_k[di] = K.view(-1, g.Hkv, g.D)[si]
                    self.dup_v[di] = V.view(-1, g.Hkv, g.D)[si]
        wsb = B.std_workspace_bytes(g, max(n, 1), self.max_seq_len)
        self.workspace = torch.empty(max(wsb, 16), dtype=torch.uint8, device=dev)
        self.o = torch.zeros(max(n, 1), g.Hq, g.D, dtype=torch.bfloat16, device=dev)
        self.lse = torch.zeros(max(n, 1), g.Hq, dtype=torch.float32, device=dev)
        self.g = g

    def attn(self, q: torch.Tensor):
        B.std_attn_decode(self.g, self.n, self.max_seq_len, self.n_active, q, self.dup_k, self.dup_v, self.seq_start,
                          self.seq_len, self.o, self.lse, self.workspace)
