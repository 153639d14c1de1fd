"""Pins of the oracle's position-order mode (Sec. 4.3.2, Fig. 3, Sec. 4.4, Algorithm 2): the mask the paper runs.

None of these re-types the oracle's visibility test.  They check it against (1) the position numbers the paper prints
and Algorithm 2 itself, (2) ordinary causal attention -- the library routine -- on the sequence sorted by position ID,
(3) the fine-tuning mask of Sec. 4.4 written out on the in-order training sequence, which the paper states gives the
identical pattern, (4) the branch-local mode where the two must coincide, (5) independence from later branches.
"""
from dataclasses import replace

import numpy as np
import torch

from paper_2604_26209_b200 import synth
from oracle import capi, brute
from tests.util import widen


def _skel(seed=0, **kw):
    d = dict(Hq=4, Hkv=2, D=32, theta=10000.0, k_max=7, prompt_lens=[10, 5], branch_cnts=[3, 4], key_len_hi=3, seed=seed)
    d.update(kw)
    return synth.config_skeleton("skel", **d)


def _run(s, f):
    meta, pvis = capi.build_meta_skeleton(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.slot_vis,
                                          s.geom.suffix_cap, s.pos_gap)
    act = meta.active_slot[: meta.n_active]
    out, pos = capi.decode_step_posorder(s.geom, meta, s.doc_prefix_len, s.slot_depth, s.slot_alive, s.slot_vis, s.pos_gap,
                                         f["q"][act], f["k_new"][act], f["v_new"][act], f["prefix_k"], f["prefix_v"],
                                         f["suffix_k"], f["suffix_v"])
    return meta, pvis, out, pos


def _alg2(s, d):
    """Algorithm 2 itself on group d: positions of its prefix tokens; attribute j spans (end of j-1, end of j]."""
    s0 = int(np.sum(s.doc_branch_cnt[:d])); c = int(s.doc_branch_cnt[d])
    end = s.slot_vis[s0:s0 + c] - 1
    start = np.concatenate([[0], end[:-1] + 1]) if c else np.zeros(0, np.int32)
    return capi.alg2_position_ids(int(s.doc_prefix_len[d]), start, end, s.pos_gap), end


def test_positions_are_the_papers_figure_2_numbers():
    # prompt of 10 tokens, three attributes of 3 tokens, K_max = 7: the first value tokens are read at positions
    # 12 / 22 / 32 and receive 13 / 23 / 33 (Sec. 4.3.1-4.3.2, numbers printed for the paper's figure)
    golden = [int(x) for x in open("tests/golden/alg2_fig2_positions.txt").read().split() if x.lstrip("-").isdigit()]
    s = synth.config_skeleton("fig2", 4, 1, 32, 1e4, 7, [10], [3], key_len_hi=1)
    s.slot_vis[:] = [13, 16, 19]; s.doc_prefix_len[:] = 19; s.slot_depth[:] = 0; s.slot_alive[:] = 1
    meta, pvis = capi.build_meta_skeleton(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.slot_vis, 7, 7)
    assert list(meta.pos_id[:3]) == [13, 23, 33] and list(meta.pos_id[:3] - 1) == [12, 22, 32]
    assert set([12, 22, 32, 13, 23, 33]) <= set(golden)
    assert list(pvis[:3]) == [13, 16, 19]
    s.slot_depth[:] = [2, 0, 5]                       # later steps: previous ID + 1 (Sec. 4.3.3)
    meta, _ = capi.build_meta_skeleton(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.slot_vis, 7, 7)
    assert list(meta.pos_id[:3]) == [15, 23, 38]


def test_positions_follow_algorithm_2_on_random_skeletons():
    for seed in range(5):
        s = _skel(seed, prompt_lens=[9, 0, 4], branch_cnts=[5, 2, 6], key_len_hi=4, alive_frac=0.7)
        meta, pvis = capi.build_meta_skeleton(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.slot_vis,
                                              s.geom.suffix_cap, s.pos_gap)
        slot0 = np.concatenate([[0], np.cumsum(s.doc_branch_cnt)])
        for r in range(meta.n_active):
            d, sl = meta.doc_id[r], meta.active_slot[r]
            pos, end = _alg2(s, d)
            j = sl - slot0[d]
            assert meta.pos_id[r] == capi.alg2_value_position(pos, end, j, int(s.slot_depth[sl]) + 1)
            assert pvis[r] == end[j] + 1
        # tables shared with the branch-local mode are the same function of the structure
        ref = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap, 0)
        for nm in ("doc_kv_start", "doc_slot_start", "doc_active_start", "active_slot", "doc_id", "suffix_off", "suffix_len"):
            assert np.array_equal(getattr(meta, nm), getattr(ref, nm)), nm


def _group_sequence(s, f, d, pos_new, k_rot, act):
    """All tokens of group d in the paper's memory order -- prompt and skeleton, then the value tokens appended step by
    step, then this step's new tokens -- with their position IDs.  Returns K, V [n,Hkv,D], pos [n], index of each row's
    new token."""
    g = s.geom
    kv0 = int(np.sum(s.doc_prefix_len[:d])); L = int(s.doc_prefix_len[d])
    s0 = int(np.sum(s.doc_branch_cnt[:d])); c = int(s.doc_branch_cnt[d])
    pos_pre, end = _alg2(s, d)
    K = [f["prefix_k"][kv0 + t] for t in range(L)]; V = [f["prefix_v"][kv0 + t] for t in range(L)]
    pos = list(pos_pre)
    for t in range(int(s.slot_depth[s0:s0 + c].max()) if c else 0):
        for j in range(c):
            if s.slot_depth[s0 + j] > t:
                K.append(f["suffix_k"][(s0 + j) * g.suffix_cap + t]); V.append(f["suffix_v"][(s0 + j) * g.suffix_cap + t])
                pos.append(capi.alg2_value_position(pos_pre, end, j, t + 1))
    where = {}
    for r, sl in enumerate(act):
        if s0 <= sl < s0 + c:
            where[r] = len(K)
            K.append(k_rot[r]); V.append(f["v_new"][sl]); pos.append(int(pos_new[r]))
    return np.asarray(K, np.float64), np.asarray(V, np.float64), np.asarray(pos), where


def test_equals_causal_attention_on_the_position_sorted_sequence():
    """'The triangular attention mask is computed using the position ID ordering': sort the group's tokens by position
    ID and the mask is the ordinary causal one, so the library's causal attention on the sorted sequence must give the
    oracle's rows."""
    for seed in range(4):
        s = _skel(seed, alive_frac=0.8)
        f = widen(synth.make_tensors(s))
        meta, _, out, pos_new = _run(s, f)
        act = meta.active_slot[: meta.n_active]
        g = s.geom
        k_rot = brute.rope_rows(f["k_new"][act], pos_new, g.rope_theta)
        q_rot = brute.rope_rows(f["q"][act], pos_new, g.rope_theta)
        for d in range(s.n_docs):
            K, V, pos, where = _group_sequence(s, f, d, pos_new, k_rot, act)
            if not where:
                continue
            assert len(set(pos.tolist())) == len(pos)                      # position IDs are unique inside a group
            order = np.argsort(pos)
            rank = np.empty_like(order); rank[order] = np.arange(len(order))
            Ks, Vs = torch.from_numpy(K[order]), torch.from_numpy(V[order])
            Q = torch.zeros(len(order), g.Hq, g.D, dtype=torch.float64)
            for r, idx in where.items():
                Q[rank[idx]] = torch.from_numpy(q_rot[r])
            rep = g.Hq // g.Hkv
            o = torch.nn.functional.scaled_dot_product_attention(
                Q.permute(1, 0, 2)[None], Ks.repeat_interleave(rep, 1).permute(1, 0, 2)[None],
                Vs.repeat_interleave(rep, 1).permute(1, 0, 2)[None], is_causal=True, scale=g.sm_scale)[0].permute(1, 0, 2)
            for r, idx in where.items():
                assert np.allclose(o[rank[idx]].numpy(), out.o[r], atol=2e-6), (seed, d, r)


def test_inference_pattern_equals_the_fine_tuning_mask():
    """Fig. 3: the attention pattern of (a) inference on the appended cache and (b) fine-tuning on the in-order sequence
    is identical.  (b) per Sec. 4.4: standard causal mask, plus value token (n,k) may not see value tokens (n',k') with
    n' < n and k' > k, plus attribute tokens see no value token.  The in-order sequence below also holds the value tokens
    that do not exist yet at step t (random data): the mask must hide them."""
    rng = np.random.default_rng(5)
    base = _skel(11, prompt_lens=[6], branch_cnts=[5], key_len_hi=3)
    g = base.geom
    K_n = np.array([3, 7, 1, 5, 4])                                    # final lengths of the five values
    f = widen(synth.make_tensors(base))
    L = int(base.doc_prefix_len[0]); end = base.slot_vis - 1
    for t in range(int(K_n.max())):                                    # decode step that generates token index t
        s = replace(base, slot_depth=np.minimum(K_n, t).astype(np.int32), slot_alive=(K_n > t).astype(np.uint8))
        meta, _, out, pos_new = _run(s, f)
        act = meta.active_slot[: meta.n_active]
        k_rot = brute.rope_rows(f["k_new"][act], pos_new, g.rope_theta)
        q_rot = brute.rope_rows(f["q"][act], pos_new, g.rope_theta)
        row_of = {int(sl): r for r, sl in enumerate(act)}
        # in-order training sequence: prompt, then for each attribute its key tokens followed by ALL its value tokens
        kind, K, V = [], [], []                                        # kind: ("p", t) | ("a", n) | ("v", n, k)
        tok = 0
        for n in range(5):
            while tok <= end[n]:
                kind.append(("a", n) if tok > (end[n - 1] if n else -1) and tok >= 6 else ("p", tok))
                K.append(f["prefix_k"][tok]); V.append(f["prefix_v"][tok]); tok += 1
            for k in range(int(K_n[n])):
                kind.append(("v", n, k))
                if k < t:
                    K.append(f["suffix_k"][n * g.suffix_cap + k]); V.append(f["suffix_v"][n * g.suffix_cap + k])
                elif k == t:
                    K.append(k_rot[row_of[n]]); V.append(f["v_new"][n])
                else:                                                  # not generated yet at this step
                    K.append(rng.standard_normal((g.Hkv, g.D)) * 50); V.append(rng.standard_normal((g.Hkv, g.D)) * 50)
        K, V = np.asarray(K, np.float64), np.asarray(V, np.float64)
        n_tok = len(kind)
        mask = np.tril(np.ones((n_tok, n_tok), bool))                  # standard causal mask on the in-order sequence
        for i, qi in enumerate(kind):
            for j2, kj in enumerate(kind):
                if qi[0] == "v" and kj[0] == "v" and kj[1] < qi[1] and kj[2] > qi[2]:
                    mask[i, j2] = False                                # (n', k') with n' < n and k' > k
                if qi[0] != "v" and kj[0] == "v":
                    mask[i, j2] = False                                # attributes never see values
        for n in range(5):
            if K_n[n] <= t:
                continue
            i = kind.index(("v", n, t)); r = row_of[n]
            for h in range(g.Hq):
                sc = (K[:, h // (g.Hq // g.Hkv)] @ q_rot[r, h]) * g.sm_scale
                sc = np.where(mask[i], sc, -np.inf)
                p = np.exp(sc - sc.max()); p /= p.sum()
                assert np.allclose(p @ V[:, h // (g.Hq // g.Hkv)], out.o[r, h], atol=2e-6), (t, n, h)


def test_single_branch_groups_reduce_to_the_branch_local_mode():
    s = synth.config_custom("n1", Hq=4, Hkv=2, D=32, theta=10000.0, cap=7, prefix_lens=[12, 0, 30, 7], branch_cnts=[1, 1, 1, 1],
                            depth_hi=7, seed=3, pos_gap=7)
    s.slot_vis = s.doc_prefix_len.copy()                                # no skeleton: the branch is anchored at the prefix end
    f = widen(synth.make_tensors(s))
    meta, _, out, _ = _run(s, f)
    ref_meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, 7, 7)
    act = ref_meta.active_slot[: ref_meta.n_active]
    ref = capi.decode_step(s.geom, ref_meta, s.doc_prefix_len, f["q"][act], f["k_new"][act], f["v_new"][act],
                           f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"])
    assert np.array_equal(meta.pos_id, ref_meta.pos_id)
    assert np.array_equal(out.o, ref.o) and np.array_equal(out.lse, ref.lse)


def test_earlier_branches_do_not_depend_on_later_ones_and_later_ones_do_on_earlier():
    s = _skel(21, prompt_lens=[8], branch_cnts=[6], alive_frac=1.0)
    s.slot_depth[:] = np.maximum(s.slot_depth, 1)
    f = widen(synth.make_tensors(s))
    _, _, base, _ = _run(s, f)
    f2 = {k: v.copy() for k, v in f.items()}
    f2["suffix_k"][3 * s.geom.suffix_cap] += 1.0                        # first cached key of branch 3
    f2["v_new"][3] += 1.0
    _, _, out, _ = _run(s, f2)
    assert np.array_equal(out.o[:3], base.o[:3])                        # branches 0-2 come before it in position order
    assert not np.array_equal(out.o[3], base.o[3])
    assert all(not np.array_equal(out.o[r], base.o[r]) for r in (4, 5)) # later branches see branch 3's tokens (Sec. 4.4)
    # a retired earlier branch stays visible: its cached tokens are never removed from the cache (Sec. 4.3.4)
    s2 = replace(s, slot_alive=np.array([1, 1, 1, 0, 1, 1], np.uint8))
    m2, _, out2, _ = _run(s2, f)
    keep = [0, 1, 2]
    assert np.array_equal(out2.o[:3], base.o[keep])
    assert not np.allclose(out2.o[3], base.o[4])                        # branch 4 no longer sees branch 3's NEW token...
    f3 = {k: v.copy() for k, v in f.items()}; f3["suffix_v"][3 * s.geom.suffix_cap] += 5.0
    _, _, out3, _ = _run(s2, f3)
    assert not np.array_equal(out3.o[3], out2.o[3])                     # ...but still its cached ones
