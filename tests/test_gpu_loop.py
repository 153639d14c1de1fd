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
