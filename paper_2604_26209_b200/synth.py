"""Seeded synthetic inputs for the HPD decode step (structure + bf16 tensors).

This module is the ONLY code shared by the CPU oracle's tests and the CUDA path.
It holds none of the method's arithmetic: it draws document lengths, branch
counts, branch depths / end-of-value lengths and standard-normal activations from
``numpy.random.default_rng(seed)`` and converts fp32 to bf16 bit patterns.  It
imports neither the oracle nor the CUDA binding.

The workloads stand in for the paper's product-attribute extraction prompts
(Sec. 4.3.5 stacks J documents per prompt; Sec. 4.3.6 batches b prompts; every
decode step carries b*J*N branch tokens).  The paper publishes no token-length
statistics, so prefix lengths, branch counts and depth distributions are the
ones the benchmark configuration states.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional

import numpy as np


# --------------------------------------------------------------------------------------
# bf16 <-> fp32 bit conversions (storage format only)
# --------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def randn_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    """Standard normal fp32 draws rounded to bf16 bits; generated in slabs to bound host memory."""
    shape = tuple(int(s) for s in np.atleast_1d(shape))
    n = int(np.prod(shape)) if len(shape) else 1
    out = np.empty(n, dtype=np.uint16)
    step = 1 << 24
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        out[lo:hi] = f32_to_bf16_bits(rng.standard_normal(hi - lo, dtype=np.float32))
    return out.reshape(shape)


# --------------------------------------------------------------------------------------
# Geometry and structure
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Geom:
    Hq: int
    Hkv: int
    D: int
    rope_theta: float
    sm_scale: float
    suffix_cap: int

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


LLAMA3_8B = dict(Hq=32, Hkv=8, D=128, rope_theta=500000.0)


@dataclass
class Structure:
    """Ragged description of one decode step's batch.

    Documents are numbered globally in prompt order; slots (branches ever admitted)
    are numbered globally, grouped by document.  ``slot_depth`` = branch tokens
    already cached before this step; ``slot_alive`` = 1 while the branch still decodes.
    """
    name: str
    geom: Geom
    doc_prefix_len: np.ndarray   # int32 [n_docs]
    doc_branch_cnt: np.ndarray   # int32 [n_docs]
    slot_depth: np.ndarray       # int32 [n_slots]
    slot_alive: np.ndarray       # uint8 [n_slots]
    pos_gap: int = 0
    n_prompts: int = 1
    docs_per_prompt: int = 1
    seed: int = 0
    eos_len: Optional[np.ndarray] = None  # int32 [n_slots], decode-loop workloads only
    slot_vis: Optional[np.ndarray] = None  # int32 [n_slots], position-order workloads: prefix tokens of the group up to
                                           # and including the slot's attribute key (the skeleton of Sec. 4.3.1)

    @property
    def n_docs(self) -> int:
        return int(self.doc_prefix_len.shape[0])

    @property
    def n_slots(self) -> int:
        return int(self.slot_depth.shape[0])

    @property
    def total_prefix(self) -> int:
        return int(self.doc_prefix_len.sum())

    @property
    def n_active(self) -> int:
        return int(self.slot_alive.astype(np.int64).sum())

    def slot_doc(self) -> np.ndarray:
        return np.repeat(np.arange(self.n_docs, dtype=np.int32), self.doc_branch_cnt)


def _structure(name, geom, n_prompts, docs_per_prompt, len_lo, len_hi, branches_per_doc,
               depth_lo, depth_hi, seed, pos_gap=0) -> Structure:
    """Lengths uniform on the integers [len_lo, len_hi]; depths uniform on [depth_lo, depth_hi)."""
    rng = np.random.default_rng(seed)
    n_docs = n_prompts * docs_per_prompt
    if len_lo == len_hi:
        L = np.full(n_docs, len_lo, dtype=np.int32)
    else:
        L = rng.integers(len_lo, len_hi + 1, size=n_docs, dtype=np.int32)
    cnt = np.full(n_docs, branches_per_doc, dtype=np.int32)
    n_slots = int(cnt.sum())
    depth = rng.integers(depth_lo, depth_hi, size=n_slots, dtype=np.int32)
    alive = np.ones(n_slots, dtype=np.uint8)
    return Structure(name, geom, L, cnt, depth, alive, pos_gap, n_prompts, docs_per_prompt, seed)


def config_tiny(seed: int = 0) -> Structure:
    """1 prompt, 1 document of 256 prefix tokens, 4 branches at depth 0..7, 4 q heads / 1 KV head, D=64."""
    g = Geom(Hq=4, Hkv=1, D=64, rope_theta=10000.0, sm_scale=1.0 / 8.0, suffix_cap=8)
    return _structure("tiny", g, 1, 1, 256, 256, 4, 0, 8, seed)


def config_main(n_prompts: int = 64, seed: int = 0, suffix_cap: int = 16) -> Structure:
    """Llama-3-8B attention geometry; each prompt stacks 4 documents of 512 prefix tokens with 24
    branches per document (96 branches/prompt); branch depths uniform in [0,16)."""
    g = Geom(**LLAMA3_8B, sm_scale=1.0 / np.sqrt(128.0), suffix_cap=suffix_cap)
    return _structure(f"main_p{n_prompts}", g, n_prompts, 4, 512, 512, 24, 0, 16, seed)


def config_long(n_prompts: int = 32, seed: int = 0) -> Structure:
    """Long documents: 8 documents per prompt, prefix lengths uniform on [1024,4096], 12 branches per
    document (96/prompt), depths uniform in [0,32)."""
    g = Geom(**LLAMA3_8B, sm_scale=1.0 / np.sqrt(128.0), suffix_cap=32)
    return _structure(f"long_p{n_prompts}", g, n_prompts, 8, 1024, 4096, 12, 0, 32, seed)


def config_loop(n_prompts: int = 64, seed: int = 0, mean_len: int = 8, cap: int = 32) -> Structure:
    """Decode-loop workload: the main structure at depth 0 with a per-branch end-of-value length
    drawn geometric (mean ``mean_len``) and capped at ``cap``; a branch is alive at steps 0..len-1."""
    g = Geom(**LLAMA3_8B, sm_scale=1.0 / np.sqrt(128.0), suffix_cap=cap)
    s = _structure(f"loop_p{n_prompts}", g, n_prompts, 4, 512, 512, 24, 0, 1, seed)
    rng = np.random.default_rng(seed + 1000003)
    s.eos_len = np.minimum(rng.geometric(1.0 / mean_len, size=s.n_slots), cap).astype(np.int32)
    return s


def config_custom(name, Hq, Hkv, D, theta, cap, prefix_lens, branch_cnts, depth_hi, seed=0,
                  pos_gap=0, alive_frac=1.0) -> Structure:
    """Arbitrary ragged structure for edge-case tests."""
    g = Geom(Hq=Hq, Hkv=Hkv, D=D, rope_theta=float(theta), sm_scale=float(1.0 / np.sqrt(D)), suffix_cap=cap)
    rng = np.random.default_rng(seed)
    L = np.asarray(prefix_lens, dtype=np.int32)
    cnt = np.asarray(branch_cnts, dtype=np.int32)
    n_slots = int(cnt.sum())
    depth = rng.integers(0, max(1, depth_hi), size=n_slots, dtype=np.int32) if n_slots else np.zeros(0, np.int32)
    alive = (rng.random(n_slots) < alive_frac).astype(np.uint8)
    return Structure(name, g, L, cnt, depth, alive, pos_gap, 1, int(L.shape[0]), seed)


def config_skeleton(name, Hq, Hkv, D, theta, k_max, prompt_lens, branch_cnts, key_len_hi=4, depth_hi=None, seed=0,
                    alive_frac=1.0) -> Structure:
    """Position-order workload: every group is one stacked prompt, its prefix = ``prompt_lens[d]`` prompt tokens followed
    by the skeleton, i.e. for each of its ``branch_cnts[d]`` branches an attribute key of 1..key_len_hi tokens (Sec.
    4.3.1).  ``slot_vis`` marks where each branch's key ends; slab size and position gap are both ``k_max``."""
    g = Geom(Hq=Hq, Hkv=Hkv, D=D, rope_theta=float(theta), sm_scale=float(1.0 / np.sqrt(D)), suffix_cap=k_max)
    rng = np.random.default_rng(seed)
    cnt = np.asarray(branch_cnts, dtype=np.int32)
    n_slots = int(cnt.sum())
    key_len = rng.integers(1, key_len_hi + 1, size=n_slots, dtype=np.int32)
    L, vis, at = [], np.zeros(n_slots, np.int32), 0
    for d, c in enumerate(cnt):
        end = int(prompt_lens[d]) + np.cumsum(key_len[at:at + c])
        vis[at:at + c] = end
        L.append(int(end[-1]) if c else int(prompt_lens[d]))
        at += c
    depth_hi = k_max if depth_hi is None else depth_hi
    depth = rng.integers(0, max(1, depth_hi), size=n_slots, dtype=np.int32)
    alive = (rng.random(n_slots) < alive_frac).astype(np.uint8)
    return Structure(name, g, np.asarray(L, dtype=np.int32), cnt, depth, alive, k_max, 1, len(cnt), seed, None, vis)


def loop_step_state(s: Structure, step: int) -> Structure:
    """Structure of decode step ``step`` of a loop workload: depth = step for every live branch."""
    assert s.eos_len is not None
    alive = (s.eos_len > step).astype(np.uint8)
    depth = np.minimum(s.eos_len, step).astype(np.int32)
    return replace(s, slot_depth=depth, slot_alive=alive)


# --------------------------------------------------------------------------------------
# Tensors
# --------------------------------------------------------------------------------------
def make_tensors(s: Structure, seed: Optional[int] = None, prefix: bool = True, suffix: bool = True,
                 step: bool = True, salt: int = 0) -> Dict[str, np.ndarray]:
    """bf16 (uint16 bit pattern) tensors of one step:

    prefix_k, prefix_v [total_prefix, Hkv, D]   cached keys/values of all documents (used as stored)
    suffix_k, suffix_v [n_slots*cap, Hkv, D]    branch slabs, every row filled (rows >= depth are junk
                                                that a correct implementation never reads)
    q [n_slots, Hq, D], k_new, v_new [n_slots, Hkv, D]  per-slot new-token activations; the step's
                                                active rows are gathered from them by the caller.
    Each group draws from its own child stream so that sub-sampling one does not disturb the others.
    """
    seed = s.seed if seed is None else seed
    g = s.geom
    out: Dict[str, np.ndarray] = {}
    ss = np.random.SeedSequence([int(seed), int(salt), 0x48504400])
    c_pre, c_suf, c_step = [np.random.default_rng(c) for c in ss.spawn(3)]
    if prefix:
        out["prefix_k"] = randn_bf16(c_pre, (s.total_prefix, g.Hkv, g.D))
        out["prefix_v"] = randn_bf16(c_pre, (s.total_prefix, g.Hkv, g.D))
    if suffix:
        out["suffix_k"] = randn_bf16(c_suf, (s.n_slots * g.suffix_cap, g.Hkv, g.D))
        out["suffix_v"] = randn_bf16(c_suf, (s.n_slots * g.suffix_cap, g.Hkv, g.D))
    if step:
        out["q"] = randn_bf16(c_step, (s.n_slots, g.Hq, g.D))
        out["k_new"] = randn_bf16(c_step, (s.n_slots, g.Hkv, g.D))
        out["v_new"] = randn_bf16(c_step, (s.n_slots, g.Hkv, g.D))
    return out


def shard_prompts(n_prompts: int, world_size: int, rank: int) -> range:
    """Contiguous, balanced split of prompt indices over ranks (prompts are independent units)."""
    base, rem = divmod(n_prompts, world_size)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))
