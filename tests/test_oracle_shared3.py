"""Pins of the oracle's three-level sharing (Sec. 4.3.5) and of its log-sum-exp merge.

Sharing is storage, not mathematics: a block stored once in front of several documents must give what the same
tokens stored in front of EVERY document give.  The merge must give what attention over the union of the keys gives."""
import numpy as np
import torch

from paper_2604_26209_b200 import synth
from oracle import capi
from tests.util import widen


def _case(seed):
    s = synth.config_custom("s3", Hq=4, Hkv=2, D=32, theta=10000.0, cap=6, prefix_lens=[9, 0, 14, 5, 7],
                            branch_cnts=[3, 2, 0, 4, 1], depth_hi=6, seed=seed, alive_frac=0.8)
    rng = np.random.default_rng(seed + 50)
    doc_block = np.array([0, 0, 1, 1, 2], np.int32)                      # three blocks shared by 2 / 2 / 1 documents
    block_len = np.array([11, 0, 6], np.int32)                           # one of them empty
    f = widen(synth.make_tensors(s))
    f["block_k"] = rng.standard_normal((int(block_len.sum()), 2, 32)).astype(np.float32)
    f["block_v"] = rng.standard_normal((int(block_len.sum()), 2, 32)).astype(np.float32)
    return s, f, doc_block, block_len


def test_shared_block_equals_the_block_stored_in_front_of_every_document():
    for seed in range(3):
        s, f, doc_block, block_len = _case(seed)
        meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap, 0)
        act = meta.active_slot[: meta.n_active]
        out, pos = capi.decode_step_shared3(s.geom, meta, s.doc_prefix_len, doc_block, block_len, f["q"][act], f["k_new"][act],
                                            f["v_new"][act], f["block_k"], f["block_v"], f["prefix_k"], f["prefix_v"],
                                            f["suffix_k"], f["suffix_v"])
        # the same tokens, two levels: every document's prefix physically preceded by its block
        bstart = np.concatenate([[0], np.cumsum(block_len)])
        kv0 = np.concatenate([[0], np.cumsum(s.doc_prefix_len)])
        pk, pv, L2 = [], [], []
        for d in range(s.n_docs):
            b = doc_block[d]
            pk += [f["block_k"][bstart[b]:bstart[b + 1]], f["prefix_k"][kv0[d]:kv0[d + 1]]]
            pv += [f["block_v"][bstart[b]:bstart[b + 1]], f["prefix_v"][kv0[d]:kv0[d + 1]]]
            L2.append(int(block_len[b] + s.doc_prefix_len[d]))
        meta2 = capi.build_meta(L2, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap, 0)
        ref = capi.decode_step(s.geom, meta2, L2, f["q"][act], f["k_new"][act], f["v_new"][act], np.concatenate(pk),
                               np.concatenate(pv), f["suffix_k"], f["suffix_v"])
        assert np.array_equal(pos, meta2.pos_id[: meta2.n_active])
        assert np.array_equal(out.o, ref.o) and np.array_equal(out.lse, ref.lse) and np.array_equal(out.k_rot, ref.k_rot)


def test_one_row_against_library_causal_attention():
    s, f, doc_block, block_len = _case(7)
    meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap, 0)
    act = meta.active_slot[: meta.n_active]
    out, pos = capi.decode_step_shared3(s.geom, meta, s.doc_prefix_len, doc_block, block_len, f["q"][act], f["k_new"][act],
                                        f["v_new"][act], f["block_k"], f["block_v"], f["prefix_k"], f["prefix_v"],
                                        f["suffix_k"], f["suffix_v"])
    r = int(np.argmax(meta.doc_id[: meta.n_active] == 0))               # a row of document 0 (block 0: 11 tokens)
    assert meta.doc_id[r] == 0
    d, sl = 0, act[r]
    kv0 = np.concatenate([[0], np.cumsum(s.doc_prefix_len)])
    K = np.concatenate([f["block_k"][0:11], f["prefix_k"][kv0[d]:kv0[d + 1]],
                        f["suffix_k"][sl * 6: sl * 6 + s.slot_depth[sl]], out.k_rot[r][None]]).astype(np.float64)
    V = np.concatenate([f["block_v"][0:11], f["prefix_v"][kv0[d]:kv0[d + 1]],
                        f["suffix_v"][sl * 6: sl * 6 + s.slot_depth[sl]], f["v_new"][sl][None]]).astype(np.float64)
    assert pos[r] == K.shape[0] - 1
    Q = torch.zeros(K.shape[0], 4, 32, dtype=torch.float64); Q[-1] = torch.from_numpy(out.q_rot[r].astype(np.float64))
    o = torch.nn.functional.scaled_dot_product_attention(
        Q.permute(1, 0, 2)[None], torch.from_numpy(K).repeat_interleave(2, 1).permute(1, 0, 2)[None],
        torch.from_numpy(V).repeat_interleave(2, 1).permute(1, 0, 2)[None], is_causal=True, scale=s.geom.sm_scale)[0, :, -1]
    assert np.allclose(o.numpy(), out.o[r], atol=2e-6)


def test_merge_equals_attention_over_the_union_of_the_keys():
    rng = np.random.default_rng(3)
    Hq, Hkv, D, n = 4, 2, 16, 23
    q = rng.standard_normal((Hq, D)); K = rng.standard_normal((n, Hkv, D)) * 2; V = rng.standard_normal((n, Hkv, D))
    full_o, full_l = capi.causal_attention_row(n - 1, q, K, V, 0.25)
    for cut in (1, 7, 22):
        oa, la = capi.causal_attention_row(cut - 1, q, K[:cut], V[:cut], 0.25)
        ob, lb = capi.causal_attention_row(n - cut - 1, q, K[cut:], V[cut:], 0.25)
        o, l = capi.merge_lse(oa, la, ob, lb)
        assert np.allclose(o, full_o, atol=1e-12) and np.allclose(l, full_l, atol=1e-12)
    # an empty side (lse = -inf) leaves the other untouched; two empty sides give zero
    o, l = capi.merge_lse(full_o, full_l, np.zeros_like(full_o), np.full(Hq, -np.inf))
    assert np.array_equal(o, full_o) and np.array_equal(l, full_l)
    o, l = capi.merge_lse(np.zeros_like(full_o), np.full(Hq, -np.inf), np.zeros_like(full_o), np.full(Hq, -np.inf))
    assert not o.any() and np.all(np.isneginf(l))
