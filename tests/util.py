"""Shared helpers of the tests: marshal a synthetic workload into oracle inputs."""
from __future__ import annotations

import numpy as np

from paper_2604_26209_b200 import synth
from oracle import capi


def widen(t):
    """bf16-bit tensors -> fp32 arrays (exact)."""
    return {k: synth.bf16_bits_to_f32(v) for k, v in t.items()}


def oracle_step(s, t_bits, n_threads=0, rows=None):
    """Run the oracle on structure ``s`` with bf16-bit tensors ``t_bits`` (per-slot q/k_new/v_new)."""
    g = s.geom
    meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, g.suffix_cap, s.pos_gap)
    f = widen(t_bits)
    act = meta.active_slot[: meta.n_active]
    out = capi.decode_step(g, meta, s.doc_prefix_len, f["q"][act], f["k_new"][act], f["v_new"][act],
                           f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"],
                           n_threads=n_threads, rows=rows)
    return meta, out


def err_stats(got, want):
    d = np.abs(np.asarray(got, dtype=np.float64) - np.asarray(want, dtype=np.float64))
    return (float(d.max()) if d.size else 0.0, float(d.mean()) if d.size else 0.0)
