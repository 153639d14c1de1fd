"""GPU parity of the position-order mode (Sec. 4.3.2, Fig. 3, Algorithm 2): hpd_build_meta_skeleton and
hpd_attn_decode_posorder through the C ABI against the oracle's position-order step on the same seeded inputs."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2604_26209_b200 import synth
from oracle import capi
from tests.util import widen, err_stats

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 2e-2, 2e-3

LLAMA = dict(Hq=32, Hkv=8, D=128, theta=500000.0)


def _lockstep(s, t, seed):
    """The state the loop of Algorithm 1 reaches at step t: every value has a final length; shorter ones are retired."""
    rng = np.random.default_rng(seed)
    K_n = np.minimum(rng.geometric(1.0 / 6, size=s.n_slots), s.geom.suffix_cap)
    return replace(s, slot_depth=np.minimum(K_n, t).astype(np.int32), slot_alive=(K_n > t).astype(np.uint8))


STRUCTS = {
    "tiny_two_groups": lambda: synth.config_skeleton("t", 4, 1, 64, 1e4, 7, [10, 5], [3, 4], key_len_hi=3, seed=0),
    # the paper's shape: one prompt stacking 6 documents x 16 attributes = 96 branches, K_max = 30 (Appendix B)
    "prompt_96": lambda: synth.config_skeleton("p96", **LLAMA, k_max=30, prompt_lens=[700], branch_cnts=[96], key_len_hi=4,
                                               seed=1, alive_frac=0.8),
    "prompt_96_lockstep_t5": lambda: _lockstep(synth.config_skeleton("p96l", **LLAMA, k_max=30, prompt_lens=[650],
                                                                     branch_cnts=[96], key_len_hi=4, seed=2), 5, 7),
    "prompts_batch": lambda: synth.config_skeleton("pb", **LLAMA, k_max=16, prompt_lens=[300, 0, 129, 512, 77],
                                                   branch_cnts=[24, 5, 0, 96, 33], key_len_hi=3, seed=3, alive_frac=0.7),
    "long_prompt_few_branches": lambda: synth.config_skeleton("lp", **LLAMA, k_max=8, prompt_lens=[3000, 2100],
                                                              branch_cnts=[6, 3], key_len_hi=5, seed=4),
    "g8_d64_full_group": lambda: synth.config_skeleton("g8", 8, 1, 64, 1e4, 5, [40], [128], key_len_hi=2, seed=5),
}


def _oracle(s, tb):
    f = widen(tb)
    meta, pvis = capi.build_meta_skeleton(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.slot_vis,
                                          s.geom.suffix_cap, s.pos_gap)
    act = meta.active_slot[: meta.n_active]
    out, _ = capi.decode_step_posorder(s.geom, meta, s.doc_prefix_len, s.slot_depth, s.slot_alive, s.slot_vis, s.pos_gap,
                                       f["q"][act], f["k_new"][act], f["v_new"][act], f["prefix_k"], f["prefix_v"],
                                       f["suffix_k"], f["suffix_v"])
    return meta, pvis, out


@pytest.mark.parametrize("name", list(STRUCTS))
def test_posorder_step_matches_oracle(name):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime as rt
    s = STRUCTS[name]()
    tb = synth.make_tensors(s)
    meta, pvis, want = _oracle(s, tb)
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    tabs = db.tables()
    n = meta.n_active
    assert tabs["n_active"] == n
    for nm in capi.Meta.TABLES:
        assert np.array_equal(tabs[nm], getattr(meta, nm)), nm
    assert np.array_equal(tabs["prefix_vis"], pvis)
    act = tabs["active_slot"][:n]
    db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    db.rope_append()
    db.attn(True)
    torch.cuda.synchronize()
    assert db.status() == 0
    q_gpu = synth.bf16_bits_to_f32(rt.bits_of(db.q))[:n]
    assert np.all(np.abs(q_gpu - want.q_rot) <= np.abs(want.q_rot) * (2.0 ** -8 + 1e-5) + 1e-6)
    o = synth.bf16_bits_to_f32(rt.bits_of(db.o))[:n]
    mx, mean = err_stats(o, want.o)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    assert np.max(np.abs(db.lse.cpu().numpy()[:n] - want.lse)) <= 2e-2


def test_posorder_group_beyond_128_slots_is_flagged():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime as rt, binding
    s = synth.config_skeleton("big", 8, 1, 64, 1e4, 4, [20], [130], key_len_hi=1, seed=6)
    tb = synth.make_tensors(s)
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    db.set_step_inputs(tb["q"], tb["k_new"], tb["v_new"])
    db.rope_append()
    db.attn(True)
    torch.cuda.synchronize()
    assert db.status() & binding.HPD_S_BAD_TABLE
    assert np.isfinite(synth.bf16_bits_to_f32(rt.bits_of(db.o))).all()
