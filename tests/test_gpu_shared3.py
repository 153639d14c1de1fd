"""GPU parity of three-level sharing (Sec. 4.3.5): block attention + document/branch attention + hpd_merge_lse
against the oracle, which attends the concatenated [block ; document ; branch] sequence directly."""
import numpy as np
import pytest
import torch

from paper_2604_26209_b200 import synth
from oracle import capi
from tests.util import widen, err_stats

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def _blocks(s, doc_block, block_len, seed):
    rng = np.random.default_rng(seed)
    n = int(np.sum(block_len))
    return (synth.randn_bf16(rng, (n, s.geom.Hkv, s.geom.D)), synth.randn_bf16(rng, (n, s.geom.Hkv, s.geom.D)))


CASES = {
    # instruction block of 160 tokens shared by all 8 documents of two prompts, 352-token documents
    "one_block_all_docs": lambda: (synth.config_custom("a", Hq=32, Hkv=8, D=128, theta=500000.0, cap=16, prefix_lens=[352] * 8,
                                                       branch_cnts=[24] * 8, depth_hi=16, seed=1, alive_frac=0.9),
                                   [0] * 8, [160]),
    # one block per prompt, ragged, an empty block, documents without prefix, D = 64
    "ragged": lambda: (synth.config_custom("b", Hq=8, Hkv=4, D=64, theta=10000.0, cap=6, prefix_lens=[90, 0, 140, 5, 70, 33],
                                           branch_cnts=[5, 3, 0, 40, 1, 7], depth_hi=6, seed=2, alive_frac=0.8),
                       [0, 0, 1, 1, 2, 2], [111, 0, 300]),
    # few rows and long documents: the prefix is split over several work items, the block goes with the first chunk
    "split_prefix": lambda: (synth.config_custom("c", Hq=32, Hkv=8, D=128, theta=500000.0, cap=8, prefix_lens=[3000, 2500],
                                                 branch_cnts=[2, 1], depth_hi=8, seed=3),
                             [0, 0], [200]),
    # documents without a prefix of their own: the block is all they share
    "block_only": lambda: (synth.config_custom("d", Hq=8, Hkv=2, D=128, theta=10000.0, cap=4, prefix_lens=[0, 0, 0],
                                               branch_cnts=[9, 30, 2], depth_hi=4, seed=4),
                           [0, 0, 1], [130, 64]),
}


@pytest.mark.parametrize("two_pass", [False, True], ids=["one_launch", "two_passes_and_merge"])
@pytest.mark.parametrize("name", list(CASES))
def test_shared_block_step_matches_oracle(name, two_pass):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime as rt
    s, doc_block, block_len = CASES[name]()
    doc_block, block_len = np.asarray(doc_block, np.int32), np.asarray(block_len, np.int32)
    tb = synth.make_tensors(s)
    bk, bv = _blocks(s, doc_block, block_len, 77)
    f = widen(dict(tb, block_k=bk, block_v=bv))
    meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap, 0)
    n = meta.n_active
    act = meta.active_slot[:n]
    want, pos = capi.decode_step_shared3(s.geom, meta, s.doc_prefix_len, doc_block, block_len, f["q"][act], f["k_new"][act],
                                         f["v_new"][act], f["block_k"], f["block_v"], f["prefix_k"], f["prefix_v"],
                                         f["suffix_k"], f["suffix_v"])
    sb = rt.SharedBlockBatch(s, tb, doc_block, block_len, bk, bv)
    sb.build_meta()
    tabs = sb.db.tables()
    assert tabs["n_active"] == n and np.array_equal(tabs["pos_id"][:n], pos)      # positions count the block
    for nm in ("doc_kv_start", "doc_slot_start", "doc_active_start", "active_slot", "doc_id", "suffix_off", "suffix_len"):
        assert np.array_equal(tabs[nm], getattr(meta, nm)), nm
    sb.db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    sb.db.rope_append()
    sb.attn_two_pass() if two_pass else sb.attn()
    torch.cuda.synchronize()
    assert sb.db.status() == 0
    o = synth.bf16_bits_to_f32(rt.bits_of(sb.db.o))[:n]
    mx, mean = err_stats(o, want.o)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    assert np.max(np.abs(sb.db.lse.cpu().numpy()[:n] - want.lse)) <= 2e-2
