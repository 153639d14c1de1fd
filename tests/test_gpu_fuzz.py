"""Randomised small structures through every attention entry point against the oracle: geometry, slab size, document
lengths, branch counts, depths and retirement drawn from a seeded generator, so that corner combinations nobody wrote
down by hand (a one-token slab next to a 33-token one, an empty first document, a single live branch) are exercised."""
import numpy as np
import pytest
import torch

from paper_2604_26209_b200 import synth
from oracle import capi
from tests.util import oracle_step, widen, err_stats

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    G = int(rng.choice([1, 2, 4, 8])); Hkv = int(rng.choice([1, 2, 4])); D = int(rng.choice([64, 128]))
    cap = int(rng.integers(1, 34))
    n_docs = int(rng.integers(1, 7))
    L = rng.integers(0, 700, size=n_docs); L[rng.random(n_docs) < 0.2] = 0
    cnt = rng.integers(0, 40, size=n_docs)
    if cnt.sum() == 0:
        cnt[0] = 3
    return rng, dict(Hq=G * Hkv, Hkv=Hkv, D=D, theta=float(rng.choice([1e4, 5e5])), cap=cap, prefix_lens=L.tolist(),
                     branch_cnts=cnt.tolist(), depth_hi=cap, seed=seed, alive_frac=float(rng.choice([1.0, 0.8, 0.3])))


@pytest.mark.parametrize("seed", range(12))
def test_random_structures_branch_local_and_shared_block(seed):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime as rt
    rng, kw = _draw(seed)
    s = synth.config_custom("fuzz", **kw)
    tb = synth.make_tensors(s)
    meta, want = oracle_step(s, tb)
    n = meta.n_active
    act = meta.active_slot[:n]
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    tabs = db.tables()
    for nm in capi.Meta.TABLES:
        assert np.array_equal(tabs[nm], getattr(meta, nm)), nm
    db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    db.rope_append(); db.attn(True)
    torch.cuda.synchronize()
    assert db.status() == 0
    if n:
        mx, mean = err_stats(synth.bf16_bits_to_f32(rt.bits_of(db.o))[:n], want.o)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (kw, mx, mean)
        assert np.max(np.abs(db.lse.cpu().numpy()[:n] - want.lse)) <= 2e-2
    # the same structure with random blocks shared by runs of consecutive documents
    n_blocks = int(rng.integers(1, s.n_docs + 1))
    doc_block = np.sort(rng.integers(0, n_blocks, size=s.n_docs)).astype(np.int32)
    block_len = rng.integers(0, 200, size=n_blocks).astype(np.int32)
    nb = int(block_len.sum())
    bk = synth.randn_bf16(rng, (nb, s.geom.Hkv, s.geom.D)); bv = synth.randn_bf16(rng, (nb, s.geom.Hkv, s.geom.D))
    f = widen(dict(tb, block_k=bk, block_v=bv))
    want3, _ = capi.decode_step_shared3(s.geom, meta, s.doc_prefix_len, doc_block, block_len, f["q"][act], f["k_new"][act],
                                        f["v_new"][act], f["block_k"], f["block_v"], f["prefix_k"], f["prefix_v"],
                                        f["suffix_k"], f["suffix_v"])
    sb = rt.SharedBlockBatch(s, tb, doc_block, block_len, bk, bv)
    sb.db.build_meta()
    sb.db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    sb.db.rope_append(); sb.attn()
    torch.cuda.synchronize()
    assert sb.db.status() == 0
    if n:
        mx, mean = err_stats(synth.bf16_bits_to_f32(rt.bits_of(sb.db.o))[:n], want3.o)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (kw, mx, mean)


@pytest.mark.parametrize("seed", range(8))
def test_random_structures_position_order_and_prefill(seed):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime as rt, binding as B
    rng = np.random.default_rng(2000 + seed)
    G = int(rng.choice([1, 2, 4, 8])); Hkv = int(rng.choice([1, 2, 4])); D = int(rng.choice([64, 128]))
    k_max = int(rng.integers(1, 25))
    n_docs = int(rng.integers(1, 5))
    s = synth.config_skeleton("fz", G * Hkv, Hkv, D, float(rng.choice([1e4, 5e5])), k_max, rng.integers(0, 400, size=n_docs).tolist(),
                              rng.integers(1, 100, size=n_docs).tolist(), key_len_hi=int(rng.integers(1, 5)), seed=seed,
                              alive_frac=float(rng.choice([1.0, 0.7])))
    g, dev = s.geom, "cuda"
    tb = synth.make_tensors(s)
    f = widen(tb)
    meta, pvis = capi.build_meta_skeleton(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.slot_vis, g.suffix_cap, s.pos_gap)
    n = meta.n_active
    act = meta.active_slot[:n]
    want, _ = capi.decode_step_posorder(g, meta, s.doc_prefix_len, s.slot_depth, s.slot_alive, s.slot_vis, s.pos_gap, f["q"][act],
                                        f["k_new"][act], f["v_new"][act], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"])
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    tabs = db.tables()
    assert np.array_equal(tabs["pos_id"], meta.pos_id) and np.array_equal(tabs["prefix_vis"], pvis)
    db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    db.rope_append(); db.attn(True)
    torch.cuda.synchronize()
    assert db.status() == 0
    if n:
        mx, mean = err_stats(synth.bf16_bits_to_f32(rt.bits_of(db.o))[:n], want.o)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (seed, mx, mean)
    # first inference step over the same prompts
    T = s.total_prefix
    qb = synth.randn_bf16(rng, (T, g.Hq, g.D)); kb = synth.randn_bf16(rng, (T, g.Hkv, g.D)); vb = synth.randn_bf16(rng, (T, g.Hkv, g.D))
    wantp, pos = capi.prefill(g, s.doc_prefix_len, s.doc_branch_cnt, s.slot_vis, s.pos_gap, *(synth.bf16_bits_to_f32(a) for a in (qb, kb, vb)))
    bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    q, pk, pv = bf(qb), bf(kb), bf(vb)
    t = B.PrefillTables.alloc(g, s.n_docs, T, dev)
    o = torch.zeros(max(T, 1), g.Hq, g.D, dtype=torch.bfloat16, device=dev)
    L, cnt, vis = i32(s.doc_prefix_len), i32(s.doc_branch_cnt), i32(s.slot_vis)
    B.hpd_prefill_meta(g, s.n_docs, s.n_slots, T, L, cnt, vis, s.pos_gap, t)
    B.hpd_rope(g, T, t.n_tokens, t.tok_pos, q, pk)
    B.hpd_prefill_attn(g, s.n_docs, T, q, pk, pv, L, t, o, None)
    torch.cuda.synchronize()
    assert int(t.dev_status.item()) == 0
    if T:
        assert np.array_equal(t.tok_pos.cpu().numpy()[:T], pos)
        mx, mean = err_stats(synth.bf16_bits_to_f32(rt.bits_of(o))[:T], wantp.o)
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (seed, mx, mean)
