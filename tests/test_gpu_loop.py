"""The decode loop on the GPU (Algorithm 1 for steps t >= 1; Sec. 4.3.3-4.3.4): branches retire raggedly, the
branch cache grows by one rotated key/value per live branch and step.  Every step's outputs are checked against
the oracle, which runs the same loop on its own fp32 caches."""
import numpy as np
import pytest
import torch

from paper_2604_26209_b200 import synth
from oracle import capi

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def test_loop_with_ragged_retirement_matches_oracle():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime
    s0 = synth.config_loop(n_prompts=1, seed=3, mean_len=4, cap=8)        # 4 documents x 24 branches, cap 8
    g = s0.geom
    tb = synth.make_tensors(s0, step=False)
    tb["suffix_k"][:] = 0x7FC0                                             # NaN: a stale or unwritten row would poison the output
    tb["suffix_v"][:] = 0x7FC0
    db = runtime.DeviceBatch(s0, dict(tb, q=None, k_new=None, v_new=None))
    f_pk, f_pv = synth.bf16_bits_to_f32(tb["prefix_k"]), synth.bf16_bits_to_f32(tb["prefix_v"])
    cache_k = np.zeros((s0.n_slots * g.suffix_cap, g.Hkv, g.D), np.float32)
    cache_v = np.zeros_like(cache_k)
    rng = np.random.default_rng(77)
    steps = int(s0.eos_len.max())
    assert steps == g.suffix_cap or steps < g.suffix_cap
    seen_tokens = 0
    for t in range(steps):
        st = synth.loop_step_state(s0, t)
        if st.n_active == 0:
            break
        db.slot_depth.copy_(torch.from_numpy(st.slot_depth))
        db.slot_alive.copy_(torch.from_numpy(st.slot_alive))
        db.build_meta()
        tabs = db.tables()
        n = tabs["n_active"]
        meta = capi.build_meta(st.doc_prefix_len, st.doc_branch_cnt, st.slot_depth, st.slot_alive, g.suffix_cap, 0)
        assert n == meta.n_active == st.n_active
        for nm in capi.Meta.TABLES:
            assert np.array_equal(tabs[nm], getattr(meta, nm)), (t, nm)
        q = synth.randn_bf16(rng, (n, g.Hq, g.D)); k = synth.randn_bf16(rng, (n, g.Hkv, g.D)); v = synth.randn_bf16(rng, (n, g.Hkv, g.D))
        db.set_step_inputs(q, k, v)
        db.rope(); db.kv_append(); db.attn(True)
        torch.cuda.synchronize()
        assert db.status() == 0
        fq, fk, fv = (synth.bf16_bits_to_f32(a) for a in (q, k, v))
        want = capi.decode_step(g, meta, st.doc_prefix_len, fq, fk, fv, f_pk, f_pv, cache_k, cache_v)
        assert not capi.kv_append(g, meta, want.k_rot, fv, cache_k, cache_v).any()
        got = synth.bf16_bits_to_f32(runtime.bits_of(db.o))[:n]
        d = np.abs(got - want.o)
        assert np.isfinite(got).all() and d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (t, d.max(), d.mean())
        seen_tokens += n
    # every branch decoded exactly its end-of-value length; the caches agree up to the bf16 rounding of the rotated keys
    assert seen_tokens == int(s0.eos_len.sum())
    gk = synth.bf16_bits_to_f32(runtime.bits_of(db.suffix_k)).reshape(cache_k.shape)
    gv = synth.bf16_bits_to_f32(runtime.bits_of(db.suffix_v)).reshape(cache_v.shape)
    for sl in range(s0.n_slots):
        lo, n = sl * g.suffix_cap, int(s0.eos_len[sl])
        assert np.all(np.abs(gk[lo:lo + n] - cache_k[lo:lo + n]) <= np.abs(cache_k[lo:lo + n]) * 2.0 ** -8 + 1e-6)
        assert np.array_equal(gv[lo:lo + n], cache_v[lo:lo + n])
        assert np.isnan(gk[lo + n: lo + g.suffix_cap]).all()                # rows beyond the value's length were never written


def test_fullsize_loop_two_layers_sampled_branches():
    """The loop workload at its real batch (64 prompts x 96 branches, cap 32, end-of-value lengths min(Geom(1/8), 32))
    over ALL steps and two layers with their own caches: tables bit-exact at every step, outputs of a fixed sample of
    branches against the oracle at every step and layer, final cache contents of those branches.  Under the
    branch-local mask of Eq. 5-6 a branch's history is its own, so the oracle keeps caches for the sampled branches only."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from dataclasses import replace
    from paper_2604_26209_b200 import runtime, binding as B
    L = 2
    s0 = synth.config_loop(n_prompts=64, seed=5)
    g, dev = s0.geom, "cuda"
    cap, kvw = g.suffix_cap, g.Hkv * g.D
    rng = np.random.default_rng(99)
    # sample: some long-lived branches (so late steps with few live rows per document are checked), some random ones
    order = np.argsort(-s0.eos_len, kind="stable")
    sample = np.unique(np.concatenate([order[:24], rng.choice(s0.n_slots, 72, replace=False), [0, s0.n_slots - 1]]))
    pools = {k: synth.randn_bf16(rng, (s0.n_slots, h, g.D)) for k, h in (("q", g.Hq), ("k", g.Hkv), ("v", g.Hkv))}
    pre = [synth.make_tensors(s0, suffix=False, step=False, salt=l) for l in range(L)]
    f_pre = [{k: synth.bf16_bits_to_f32(v) for k, v in p.items()} for p in pre]
    bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)
    pre_k = [bf(p["prefix_k"]) for p in pre]; pre_v = [bf(p["prefix_v"]) for p in pre]
    nan = lambda: torch.full((s0.n_slots * cap, g.Hkv, g.D), float("nan"), dtype=torch.bfloat16, device=dev)
    suf_k = [nan() for _ in range(L)]; suf_v = [nan() for _ in range(L)]
    cache_k = [np.zeros((s0.n_slots * cap, g.Hkv, g.D), np.float32) for _ in range(L)]      # oracle's, sampled slabs only
    cache_v = [np.zeros_like(cache_k[0]) for _ in range(L)]
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    L_d, cnt = i32(s0.doc_prefix_len), i32(s0.doc_branch_cnt)
    depth = torch.zeros(s0.n_slots, dtype=torch.int32, device=dev)
    alive = torch.ones(s0.n_slots, dtype=torch.uint8, device=dev)
    meta = B.MetaTables.alloc(g, s0.n_docs, s0.n_slots, s0.total_prefix, dev)
    q = torch.zeros(s0.n_slots, g.Hq, g.D, dtype=torch.bfloat16, device=dev)
    kn = torch.zeros(s0.n_slots, g.Hkv, g.D, dtype=torch.bfloat16, device=dev); vn = torch.zeros_like(kn)
    o = torch.zeros_like(q)
    steps = int(s0.eos_len.max())
    checked = 0
    for t in range(steps):
        st = synth.loop_step_state(s0, t)
        if st.n_active == 0:
            break
        depth.copy_(torch.from_numpy(st.slot_depth)); alive.copy_(torch.from_numpy(st.slot_alive))
        B.hpd_build_meta(g, s0.n_docs, s0.n_slots, L_d, cnt, depth, alive, 0, meta)
        om = capi.build_meta(st.doc_prefix_len, st.doc_branch_cnt, st.slot_depth, st.slot_alive, cap, 0)
        n = om.n_active
        assert int(meta.n_active.item()) == n
        for nm in capi.Meta.TABLES:
            assert np.array_equal(getattr(meta, nm).cpu().numpy()[: len(getattr(om, nm))], getattr(om, nm)), (t, nm)
        act = om.active_slot[:n]
        rows = np.nonzero(np.isin(act, sample))[0]
        for l in range(L):
            # the step's activations: the pools read through a permutation that changes with step and layer
            perm = (act.astype(np.int64) * 7919 + 104729 * (t * L + l + 1)) % s0.n_slots
            qb, kb, vb = pools["q"][perm], pools["k"][perm], pools["v"][perm]
            q[:n].copy_(bf(qb)); kn[:n].copy_(bf(kb)); vn[:n].copy_(bf(vb))
            B.hpd_rope(g, s0.n_slots, meta.n_active, meta.pos_id, q, kn)
            B.hpd_kv_append(g, s0.n_slots, s0.n_slots, meta.n_active, meta.suffix_off, meta.suffix_len, kn, vn,
                            suf_k[l], suf_v[l], meta.dev_status)
            B.hpd_attn_decode(g, s0.n_docs, s0.n_slots, s0.n_slots, s0.total_prefix, q, pre_k[l], pre_v[l], suf_k[l],
                              suf_v[l], L_d, meta, True, o, None)
            torch.cuda.synchronize()
            assert int(meta.dev_status.item()) == 0
            got_all = synth.bf16_bits_to_f32(runtime.bits_of(o))[:n]
            assert np.isfinite(got_all).all(), (t, l)
            if len(rows):
                fq, fk, fv = (synth.bf16_bits_to_f32(a) for a in (qb, kb, vb))
                want = capi.decode_step(g, om, st.doc_prefix_len, fq, fk, fv, f_pre[l]["prefix_k"], f_pre[l]["prefix_v"],
                                        cache_k[l], cache_v[l], rows=rows)
                d = np.abs(got_all[rows] - want.o)
                assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (t, l, d.max(), d.mean())
                dst = (om.suffix_off[:n][rows] + om.suffix_len[:n][rows]).astype(np.int64)
                cache_k[l][dst] = want.k_rot                     # the append rule of Sec. 4.3.2 for the sampled branches
                cache_v[l][dst] = fv[rows]
                checked += len(rows)
    assert checked == L * int(s0.eos_len[sample].sum())
    for l in range(L):
        gk = synth.bf16_bits_to_f32(runtime.bits_of(suf_k[l])).reshape(-1, g.Hkv, g.D)
        gv = synth.bf16_bits_to_f32(runtime.bits_of(suf_v[l])).reshape(-1, g.Hkv, g.D)
        written = np.zeros(s0.n_slots * cap, bool)
        for sl in range(s0.n_slots):
            written[sl * cap: sl * cap + int(s0.eos_len[sl])] = True
        assert np.isfinite(gk[written]).all() and np.isfinite(gv[written]).all()
        assert np.isnan(gk[~written]).all() and np.isnan(gv[~written]).all()      # nothing beyond a value's length
        for sl in sample:
            lo, m = sl * cap, int(s0.eos_len[sl])
            ck = cache_k[l][lo:lo + m]
            assert np.all(np.abs(gk[lo:lo + m] - ck) <= np.abs(ck) * 2.0 ** -8 + 1e-6)
            assert np.array_equal(gv[lo:lo + m], cache_v[l][lo:lo + m])


def test_device_side_retirement_drives_the_loop():
    """Algorithm 1 for steps t >= 1 without a host round trip per step: hpd_advance turns the sampled token ids into
    slot_alive / slot_depth on the device (Sec. 4.3.4), the next hpd_build_meta reads them.  The sampler is a stand-in:
    a table of token ids per (step, slot) with the delimiter where the value ends, gathered by row with a torch index op.
    Row counts of every step and the final slot tables must equal the oracle's loop, bit for bit."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import binding as B
    s0 = synth.config_loop(n_prompts=2, seed=9, mean_len=5, cap=12)
    g, dev, delim = s0.geom, "cuda", 3
    rng = np.random.default_rng(1)
    K = np.minimum(rng.geometric(1.0 / 5, size=s0.n_slots), 20).astype(np.int32)      # some values longer than K_max = 12
    steps = g.suffix_cap + 1
    tok_tab = np.full((steps, s0.n_slots), 17, np.int32)
    for sl in range(s0.n_slots):
        if K[sl] - 1 < steps:
            tok_tab[K[sl] - 1, sl] = delim                             # the token sampled at step K-1 ends the value
    tb = synth.make_tensors(s0)
    from paper_2604_26209_b200 import runtime
    db = runtime.DeviceBatch(s0, tb)
    db.slot_depth.zero_(); db.slot_alive.fill_(1)
    tok_dev = torch.from_numpy(tok_tab).to(dev)
    n_alive = torch.zeros(1, dtype=torch.int32, device=dev)
    hist = torch.zeros(steps, 2, dtype=torch.int32, device=dev)
    db.set_step_inputs(tb["q"], tb["k_new"], tb["v_new"])
    for t in range(steps):
        db.build_meta()
        rows_tok = tok_dev[t][db.meta.active_slot.clamp(min=0).long()].contiguous()
        db.rope_append()
        db.attn(True, lse=False)
        B.hpd_advance(g, s0.n_slots, db.meta.n_active, db.meta.active_slot, rows_tok, delim, db.slot_depth, db.slot_alive, n_alive)
        hist[t, 0].copy_(db.meta.n_active[0]); hist[t, 1].copy_(n_alive[0])
    torch.cuda.synchronize()
    assert db.status() == 0
    # the oracle's loop
    depth, alive = np.zeros(s0.n_slots, np.int32), np.ones(s0.n_slots, np.uint8)
    want = np.zeros((steps, 2), np.int32)
    for t in range(steps):
        meta = capi.build_meta(s0.doc_prefix_len, s0.doc_branch_cnt, depth, alive, g.suffix_cap, 0)
        stay = capi.advance(meta, tok_tab[t][meta.active_slot[: meta.n_active]], delim, g.suffix_cap, depth, alive) if meta.n_active else 0
        want[t] = (meta.n_active, stay)
    assert np.array_equal(hist.cpu().numpy(), want)
    assert np.array_equal(db.slot_depth.cpu().numpy(), depth) and np.array_equal(db.slot_alive.cpu().numpy(), alive)
    assert np.array_equal(depth, np.minimum(K, g.suffix_cap)) and want[-1, 0] == 0     # everything pruned or truncated at K_max
