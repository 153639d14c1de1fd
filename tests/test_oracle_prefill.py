"""Pins of the oracle's first inference step (Sec. 4.3.2; the prefill of Algorithm 1)."""
import numpy as np
import torch

from paper_2604_26209_b200 import synth
from oracle import capi, brute
from tests.util import widen


def _case(seed, **kw):
    d = dict(Hq=4, Hkv=2, D=32, theta=10000.0, k_max=7, prompt_lens=[10, 0, 23], branch_cnts=[3, 2, 5], key_len_hi=3, seed=seed)
    d.update(kw)
    s = synth.config_skeleton("pf", **d)
    rng = np.random.default_rng(seed + 9)
    T = s.total_prefix
    q = rng.standard_normal((T, s.geom.Hq, s.geom.D)).astype(np.float32)
    k = rng.standard_normal((T, s.geom.Hkv, s.geom.D)).astype(np.float32)
    v = rng.standard_normal((T, s.geom.Hkv, s.geom.D)).astype(np.float32)
    return s, q, k, v


def test_positions_are_algorithm_2_and_the_papers_numbers():
    s = synth.config_skeleton("fig2", 4, 1, 32, 1e4, 7, [10], [3], key_len_hi=1)
    s.slot_vis[:] = [13, 16, 19]; s.doc_prefix_len[:] = 19
    z = np.zeros((19, 4, 32), np.float32)
    _, pos = capi.prefill(s.geom, s.doc_prefix_len, s.doc_branch_cnt, s.slot_vis, 7, z, z[:, :1], z[:, :1])
    # prompt 0..9, first attribute 10..12, second 20..22, third 30..32: predictions are read at 12 / 22 / 32 (Sec. 4.3.2)
    assert list(pos) == list(range(13)) + [20, 21, 22, 30, 31, 32]
    assert [int(pos[v - 1]) for v in s.slot_vis] == [12, 22, 32]


def test_prefill_equals_library_causal_attention_with_gapped_rotary_positions():
    for seed in range(3):
        s, q, k, v = _case(seed)
        g = s.geom
        out, pos = capi.prefill(g, s.doc_prefix_len, s.doc_branch_cnt, s.slot_vis, s.pos_gap, q, k, v)
        t0 = 0
        for d in range(s.n_docs):
            L = int(s.doc_prefix_len[d])
            if L == 0:
                continue
            sl = slice(t0, t0 + L)
            qr = torch.from_numpy(brute.rope_rows(q[sl], pos[sl], g.rope_theta))
            kr = torch.from_numpy(brute.rope_rows(k[sl], pos[sl], g.rope_theta))
            vv = torch.from_numpy(v[sl].astype(np.float64))
            rep = g.Hq // g.Hkv
            o = torch.nn.functional.scaled_dot_product_attention(
                qr.permute(1, 0, 2)[None], kr.repeat_interleave(rep, 1).permute(1, 0, 2)[None],
                vv.repeat_interleave(rep, 1).permute(1, 0, 2)[None], is_causal=True, scale=g.sm_scale)[0].permute(1, 0, 2)
            assert np.allclose(o.numpy(), out.o[sl], atol=2e-6), (seed, d)
            assert np.allclose(kr.numpy(), out.k_rot[sl], atol=1e-6)
            t0 += L


def test_prefill_feeds_the_position_order_decode_step():
    """The cache the prefill leaves (rotated keys, values) is the prefix of the decode steps: a depth-0 decode step on
    it must equal ordinary causal attention on [prefix up to the attribute key ; new token] with the same gapped IDs --
    i.e. the prefill of the sequence extended by that token, read at its last row."""
    s, q, k, v = _case(5, prompt_lens=[12], branch_cnts=[4])
    g = s.geom
    out, pos = capi.prefill(g, s.doc_prefix_len, s.doc_branch_cnt, s.slot_vis, s.pos_gap, q, k, v)
    s.slot_depth[:] = 0; s.slot_alive[:] = 1
    f = widen(synth.make_tensors(s))
    f["prefix_k"], f["prefix_v"] = out.k_rot, v
    meta, _ = capi.build_meta_skeleton(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.slot_vis, g.suffix_cap, s.pos_gap)
    dec, pos_new = capi.decode_step_posorder(g, meta, s.doc_prefix_len, s.slot_depth, s.slot_alive, s.slot_vis, s.pos_gap,
                                             f["q"], f["k_new"], f["v_new"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"])
    j = 0                                                               # first branch: nothing of other branches precedes it
    vis = int(s.slot_vis[j])
    assert pos_new[j] == pos[vis - 1] + 1                               # "pos_id[end(a_n)] + k" with k = 1
    K = np.concatenate([out.k_rot[:vis], dec.k_rot[j][None]]).astype(np.float64)
    V = np.concatenate([v[:vis], f["v_new"][j][None]]).astype(np.float64)
    o, _ = capi.causal_attention_row(vis, dec.q_rot[j].astype(np.float64), K, V, g.sm_scale)
    assert np.allclose(o, dec.o[j], atol=2e-6)
