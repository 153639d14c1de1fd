"""Pins for the oracle's decode step: full-matrix brute force, library SDPA on the concatenated
sequence, independence invariants (Eq. 4), append/loop consistency.  No GPU."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import capi, brute
from paper_2604_26209_b200 import synth
from tests.util import oracle_step, widen


def _brute(s, tb):
    g = s.geom
    f = widen(tb)
    return brute.full_matrix_step(g.Hq, g.Hkv, g.D, g.rope_theta, g.sm_scale, s.doc_prefix_len, s.doc_branch_cnt,
                                  s.slot_depth, s.slot_alive, g.suffix_cap, s.pos_gap, f["q"], f["k_new"], f["v_new"],
                                  f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"])


def _ragged(seed, gap=0, alive_frac=0.7):
    return synth.config_custom("ragged", Hq=4, Hkv=2, D=16, theta=10000.0, cap=6,
                               prefix_lens=[7, 0, 13, 5], branch_cnts=[3, 2, 0, 4], depth_hi=6,
                               seed=seed, pos_gap=gap, alive_frac=alive_frac)


@pytest.mark.parametrize("make", [lambda: synth.config_tiny(0), lambda: _ragged(1), lambda: _ragged(2, gap=6),
                                  lambda: _ragged(3, alive_frac=1.0)])
def test_step_equals_full_matrix_masked_softmax(make):
    """The per-branch oracle equals one masked softmax over the whole stacked sequence held in the
    paper's memory order (documents, then value tokens appended step by step; Sec. 4.3.2, Fig. 3a)."""
    s = make()
    tb = synth.make_tensors(s)
    meta, out = oracle_step(s, tb)
    o, lse, act = _brute(s, tb)
    assert np.array_equal(act, meta.active_slot[: meta.n_active])
    assert np.allclose(out.o, o, atol=2e-6)
    assert np.allclose(out.lse, lse, atol=2e-6)


def test_one_branch_is_last_row_of_library_causal_sdpa():
    """1 document, 1 branch: the step output is the last row of torch's causal SDPA over
    [prefix ; cached branch tokens ; new token]."""
    s = synth.config_custom("one", Hq=4, Hkv=2, D=32, theta=10000.0, cap=8, prefix_lens=[19], branch_cnts=[1],
                            depth_hi=1, seed=4)
    s.slot_depth[:] = 5
    tb = synth.make_tensors(s)
    f = widen(tb)
    meta, out = oracle_step(s, tb)
    pos = 19 + 5
    k_rot = brute.rope_rows(f["k_new"][:1], [pos], 10000.0)[0]
    q_rot = brute.rope_rows(f["q"][:1], [pos], 10000.0)[0]
    K = np.concatenate([f["prefix_k"], f["suffix_k"][:5], k_rot[None]]).astype(np.float64)
    V = np.concatenate([f["prefix_v"], f["suffix_v"][:5], f["v_new"][:1]]).astype(np.float64)
    n = K.shape[0]
    Q = np.zeros((n, 4, 32))
    Q[-1] = q_rot
    qt = torch.from_numpy(Q).permute(1, 0, 2)[None]
    kt = torch.from_numpy(K).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    vt = torch.from_numpy(V).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=s.geom.sm_scale)
    assert np.allclose(out.o[0], ref[0, :, -1, :].numpy(), atol=2e-6)


def _permute_docs(s, tb, perm):
    """Re-stack the documents in another order (slots move with their documents)."""
    g = s.geom
    kv = np.concatenate([[0], np.cumsum(s.doc_prefix_len)])
    sl = np.concatenate([[0], np.cumsum(s.doc_branch_cnt)])
    tok = np.concatenate([np.arange(kv[d], kv[d + 1]) for d in perm]).astype(np.int64)
    slots = np.concatenate([np.arange(sl[d], sl[d + 1]) for d in perm]).astype(np.int64)
    srow = (slots[:, None] * g.suffix_cap + np.arange(g.suffix_cap)[None, :]).reshape(-1)
    s2 = replace(s, doc_prefix_len=s.doc_prefix_len[perm], doc_branch_cnt=s.doc_branch_cnt[perm],
                 slot_depth=s.slot_depth[slots], slot_alive=s.slot_alive[slots])
    t2 = dict(prefix_k=tb["prefix_k"][tok], prefix_v=tb["prefix_v"][tok], suffix_k=tb["suffix_k"][srow],
              suffix_v=tb["suffix_v"][srow], q=tb["q"][slots], k_new=tb["k_new"][slots], v_new=tb["v_new"][slots])
    return s2, t2, slots


def test_branch_output_is_independent_of_other_documents_and_order():
    """Eq. 4: values are conditionally independent given the prompt.  Re-ordering the stacked
    documents, dropping a document, or retiring other branches leaves each output bitwise unchanged."""
    s = _ragged(5, alive_frac=1.0)
    tb = synth.make_tensors(s)
    meta, out = oracle_step(s, tb)
    by_slot = {int(sl): out.o[r] for r, sl in enumerate(meta.active_slot[: meta.n_active])}

    perm = np.array([3, 0, 2, 1])
    s2, t2, slots = _permute_docs(s, tb, perm)
    m2, o2 = oracle_step(s2, t2)
    for r in range(m2.n_active):
        assert np.array_equal(o2.o[r], by_slot[int(slots[m2.active_slot[r]])])

    keep = np.array([0, 3])                                         # un-stack two documents
    s3, t3, slots3 = _permute_docs(s, tb, keep)
    m3, o3 = oracle_step(s3, t3)
    assert m3.n_active == 7
    for r in range(m3.n_active):
        assert np.array_equal(o3.o[r], by_slot[int(slots3[m3.active_slot[r]])])

    alive = s.slot_alive.copy()
    alive[[1, 4, 6]] = 0                                            # prune other branches
    m4, o4 = oracle_step(replace(s, slot_alive=alive), tb)
    for r in range(m4.n_active):
        assert np.array_equal(o4.o[r], by_slot[int(m4.active_slot[r])])


def test_branch_order_inside_a_document_does_not_matter():
    s = synth.config_custom("perm", Hq=2, Hkv=1, D=8, theta=100.0, cap=4, prefix_lens=[9], branch_cnts=[4],
                            depth_hi=4, seed=8)
    tb = synth.make_tensors(s)
    meta, out = oracle_step(s, tb)
    p = np.array([2, 0, 3, 1])
    srow = (p[:, None] * 4 + np.arange(4)[None, :]).reshape(-1)
    s2 = replace(s, slot_depth=s.slot_depth[p])
    t2 = dict(tb, suffix_k=tb["suffix_k"][srow], suffix_v=tb["suffix_v"][srow], q=tb["q"][p], k_new=tb["k_new"][p],
              v_new=tb["v_new"][p])
    _, o2 = oracle_step(s2, t2)
    assert np.array_equal(o2.o, out.o[p])


def test_junk_beyond_depth_and_other_slabs_is_never_read():
    s = _ragged(9, alive_frac=1.0)
    tb = synth.make_tensors(s)
    _, out = oracle_step(s, tb)
    t2 = {k: v.copy() for k, v in tb.items()}
    cap = s.geom.suffix_cap
    for sl in range(s.n_slots):
        t2["suffix_k"][sl * cap + s.slot_depth[sl]: (sl + 1) * cap] = 0x7FC0      # NaN
        t2["suffix_v"][sl * cap + s.slot_depth[sl]: (sl + 1) * cap] = 0x7FC0
    _, o2 = oracle_step(s, t2)
    assert np.array_equal(out.o, o2.o)


def test_decode_loop_equals_causal_attention_on_the_growing_sequence():
    """Sec. 4.3.3: run T steps (rope at the previous ID + 1, append, attend).  Step t's output must be
    row L+t of ordinary causal attention over the final sequence built in one go."""
    g = synth.Geom(Hq=2, Hkv=1, D=16, rope_theta=10000.0, sm_scale=0.25, suffix_cap=5)
    L, T = 11, 5
    rng = np.random.default_rng(10)
    f32 = lambda *sh: synth.bf16_bits_to_f32(synth.randn_bf16(rng, sh))
    pk, pv = f32(L, 1, 16), f32(L, 1, 16)
    qs, ks, vs = f32(T, 2, 16), f32(T, 1, 16), f32(T, 1, 16)
    cache_k = np.zeros((g.suffix_cap, 1, 16), np.float32)
    cache_v = np.zeros_like(cache_k)
    outs = []
    for t in range(T):
        meta = capi.build_meta([L], [1], [t], [1], g.suffix_cap, 0)
        assert meta.pos_id[0] == L + t
        so = capi.decode_step(g, meta, [L], qs[t:t + 1], ks[t:t + 1], vs[t:t + 1], pk, pv, cache_k, cache_v)
        ovf = capi.kv_append(g, meta, so.k_rot, vs[t:t + 1], cache_k, cache_v)
        assert not ovf.any()
        outs.append(so.o[0])
    # the cache now holds the rotated keys in branch order
    k_rot_all = brute.rope_rows(ks, np.arange(L, L + T), 10000.0)
    assert np.allclose(cache_k, k_rot_all, atol=1e-6)
    K = np.concatenate([pk.astype(np.float64), k_rot_all])
    V = np.concatenate([pv, vs]).astype(np.float64)
    Q = np.zeros((L + T, 2, 16))
    Q[L:] = brute.rope_rows(qs, np.arange(L, L + T), 10000.0)
    qt = torch.from_numpy(Q).permute(1, 0, 2)[None]
    kt = torch.from_numpy(K).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    vt = torch.from_numpy(V).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=0.25)[0]
    for t in range(T):
        assert np.allclose(outs[t], ref[:, L + t, :].numpy(), atol=2e-6)
    # a full slab refuses the next append (Sec. 4.3.4: values are truncated at K_max)
    meta = capi.build_meta([L], [1], [g.suffix_cap], [1], g.suffix_cap, 0)
    before = cache_k.copy()
    ovf = capi.kv_append(g, meta, qs[:1, :1], vs[:1], cache_k, cache_v)
    assert ovf.tolist() == [1] and np.array_equal(before, cache_k)


def test_zero_length_prefix_and_row_subset():
    s = synth.config_custom("zero", Hq=2, Hkv=2, D=8, theta=100.0, cap=3, prefix_lens=[0, 4], branch_cnts=[2, 1],
                            depth_hi=3, seed=11)
    tb = synth.make_tensors(s)
    meta, out = oracle_step(s, tb)
    o, lse, _ = _brute(s, tb)
    assert np.allclose(out.o, o, atol=2e-6)
    _, sub = oracle_step(s, tb, rows=np.array([2, 0]))
    assert np.array_equal(sub.o, out.o[[2, 0]])
