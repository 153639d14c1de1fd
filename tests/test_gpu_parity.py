"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Bars: integer tables bit-exact; attention outputs max-abs <= 2e-2 and mean-abs <= 2e-3 against the
oracle; rope within bf16 rounding of the oracle's fp64 rotation; append bit-exact copies.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2604_26209_b200 import synth
from tests.util import oracle_step, err_stats, widen

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


@pytest.fixture(scope="module")
def rt():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime
    return runtime


def _ragged(seed, **kw):
    d = dict(Hq=32, Hkv=8, D=128, theta=500000.0, cap=16, prefix_lens=[300, 0, 129, 1000, 77, 512],
             branch_cnts=[5, 3, 0, 40, 1, 24], depth_hi=16, seed=seed, alive_frac=0.8)
    d.update(kw)
    return synth.config_custom("ragged", **d)


def _last_slot_full(s):
    """The last slot alive and one token short of its slab: after the step's append it is full, so the
    attention's rounded-up K boxes of that branch run past the slab and past the end of the cache tensor."""
    s.slot_depth[-1] = s.geom.suffix_cap - 1
    s.slot_alive[-1] = 1
    return s


def _odd_cap(cap, seed):
    return _last_slot_full(_ragged(seed, cap=cap, depth_hi=cap))


STRUCTS = {
    "tiny": lambda: synth.config_tiny(0),
    "main_p2": lambda: synth.config_main(n_prompts=2),
    "ragged": lambda: _ragged(1),
    "ragged_gap": lambda: _ragged(2, pos_gap=16),
    "ragged_d64_g2": lambda: _ragged(3, Hq=8, Hkv=4, D=64, theta=10000.0),
    "ragged_g8": lambda: _ragged(4, Hq=8, Hkv=1),
    "ragged_g1": lambda: _ragged(5, Hq=4, Hkv=4),
    "one_group_96": lambda: synth.config_custom("wide", Hq=32, Hkv=8, D=128, theta=500000.0, cap=8,
                                                prefix_lens=[700], branch_cnts=[96], depth_hi=8, seed=6),
    "few_alive": lambda: _ragged(7, alive_frac=0.1),
    # thousands of documents, many of them empty or without branches: several passes of the block-wide scans
    "many_docs": lambda: synth.config_custom("many", Hq=2, Hkv=1, D=64, theta=10000.0, cap=4,
                                             prefix_lens=[(7 * i) % 23 for i in range(4300)],
                                             branch_cnts=[(i % 3) for i in range(4300)], depth_hi=4, seed=10, alive_frac=0.7),
    # one query head per kv head: 128 branches per unit, four rounds of branch tables, dozens of suffix tiles per unit
    "g1_many_branches": lambda: synth.config_custom("g1", Hq=2, Hkv=2, D=128, theta=10000.0, cap=32,
                                                    prefix_lens=[200, 50, 0], branch_cnts=[200, 130, 70], depth_hi=32, seed=9),
    # slab sizes that are not a multiple of the four-column padding of packed branch tokens
    "cap1": lambda: _odd_cap(1, 20),
    "cap3": lambda: _odd_cap(3, 21),
    "cap5": lambda: _odd_cap(5, 22),
    "cap6": lambda: _odd_cap(6, 23),
    # the shape of the paper's experiments (Appendix B: J = 6 stacked documents, K_max = 30; 16 attributes per category)
    "paper_j6_n16_k30": lambda: _last_slot_full(synth.config_custom(
        "paper", Hq=32, Hkv=8, D=128, theta=500000.0, cap=30, prefix_lens=[700, 655, 811, 512, 903, 777],
        branch_cnts=[16] * 6, depth_hi=30, seed=24)),
    "paper_gap30": lambda: _last_slot_full(synth.config_custom(
        "paper_gap", Hq=32, Hkv=8, D=128, theta=500000.0, cap=30, prefix_lens=[300, 0, 411],
        branch_cnts=[16, 16, 16], depth_hi=30, seed=25, pos_gap=30)),
    # just below the largest slab the attention kernel indexes (16 branches x 4092 packed columns < 2^16)
    "cap_limit_g8": lambda: _last_slot_full(synth.config_custom(
        "caplimit", Hq=8, Hkv=1, D=64, theta=10000.0, cap=4092, prefix_lens=[100], branch_cnts=[16],
        depth_hi=4092, seed=26)),
    "long_small": lambda: synth.config_custom("long", Hq=32, Hkv=8, D=128, theta=500000.0, cap=32,
                                              prefix_lens=[4096, 1025, 3000], branch_cnts=[12, 12, 12], depth_hi=32, seed=8),
    # work lists around the size up to which the plan orders them longest unit first (2048 items): documents of very
    # different lengths, one or two branches each, every one alive so that each document is exactly one item
    "sorted_list_1500": lambda: _varied_docs(1500, 27),
    "sorted_list_2048": lambda: _varied_docs(2048, 28),
    "unsorted_list_2049": lambda: _varied_docs(2049, 29),
}


def _varied_docs(n, seed):
    lens = [(37 * i) % 331 + (900 if i % 97 == 0 else 0) for i in range(n)]
    return synth.config_custom("varied", Hq=4, Hkv=1, D=64, theta=10000.0, cap=4, prefix_lens=lens,
                               branch_cnts=[1 + (i % 2) for i in range(n)], depth_hi=4, seed=seed, alive_frac=1.0)


def _run_step(rt, s, tb):
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    tabs = db.tables()
    act = tabs["active_slot"][: tabs["n_active"]]
    db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    db.rope()
    db.kv_append()
    db.attn(True)
    torch.cuda.synchronize()
    return db, tabs


@pytest.mark.parametrize("name", list(STRUCTS))
def test_tables_bit_exact(rt, name):
    s = STRUCTS[name]()
    tb = synth.make_tensors(s, prefix=False, suffix=False, step=False)
    from oracle import capi
    meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap, s.pos_gap)
    t2 = dict(prefix_k=np.zeros((max(s.total_prefix, 1), s.geom.Hkv, s.geom.D), np.uint16))
    t2["prefix_v"] = t2["prefix_k"]
    t2["suffix_k"] = np.zeros((max(s.n_slots * s.geom.suffix_cap, 1), s.geom.Hkv, s.geom.D), np.uint16)
    t2["suffix_v"] = t2["suffix_k"]
    db = rt.DeviceBatch(s, t2)
    db.build_meta()
    torch.cuda.synchronize()
    tabs = db.tables()
    assert tabs["n_active"] == meta.n_active
    for nm in capi.Meta.TABLES:
        assert np.array_equal(tabs[nm], getattr(meta, nm)), nm
    assert db.status() == 0


def test_tables_empty_and_all_retired(rt):
    from oracle import capi
    s = _ragged(9, alive_frac=0.0)
    tb = synth.make_tensors(s)
    db, tabs = _run_step(rt, s, tb)            # every call must be a no-op with zero rows
    meta = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap, 0)
    assert tabs["n_active"] == 0
    for nm in capi.Meta.TABLES:
        assert np.array_equal(tabs[nm], getattr(meta, nm)), nm
    assert np.array_equal(rt.bits_of(db.suffix_k), tb["suffix_k"])     # nothing appended


@pytest.mark.parametrize("name", list(STRUCTS))
def test_step_matches_oracle(rt, name):
    s = STRUCTS[name]()
    tb = synth.make_tensors(s)
    meta, want = oracle_step(s, tb)
    db, tabs = _run_step(rt, s, tb)
    n = meta.n_active
    assert tabs["n_active"] == n and db.status() == 0

    # rope: bf16 rounding of the fp64 rotation (|x| <= ~6 -> half-ulp 2^-9 * 4 plus fp32 slack)
    q_gpu = synth.bf16_bits_to_f32(rt.bits_of(db.q))[:n]
    k_gpu = synth.bf16_bits_to_f32(rt.bits_of(db.k_new))[:n]
    for got, ref in ((q_gpu, want.q_rot), (k_gpu, want.k_rot)):
        tol = np.abs(ref) * (2.0 ** -8 + 1e-5) + 1e-6
        assert np.all(np.abs(got - ref) <= tol)

    # append: the rotated key and the value land at row off+len, bit-exact copies; nothing else moves
    sk, sv = rt.bits_of(db.suffix_k), rt.bits_of(db.suffix_v)
    dst = (meta.suffix_off[:n] + meta.suffix_len[:n]).astype(np.int64)
    assert np.array_equal(sk[dst], rt.bits_of(db.k_new)[:n])
    assert np.array_equal(sv[dst], tb["v_new"][meta.active_slot[:n]])
    untouched = np.ones(sk.shape[0], bool)
    untouched[dst] = False
    assert np.array_equal(sk[untouched], tb["suffix_k"][untouched])
    assert np.array_equal(sv[untouched], tb["suffix_v"][untouched])

    # attention
    o_gpu = synth.bf16_bits_to_f32(rt.bits_of(db.o))[:n]
    mx, mean = err_stats(o_gpu, want.o)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    lse_gpu = db.lse.cpu().numpy()[:n]
    assert np.max(np.abs(lse_gpu - want.lse)) <= 2e-2


@pytest.mark.parametrize("name", ["tiny", "main_p2", "ragged_gap", "ragged_d64_g2", "cap3", "paper_j6_n16_k30"])
def test_fused_rope_append_equals_the_two_calls(rt, name):
    """hpd_rope_append = hpd_rope then hpd_kv_append, bit for bit: rotated q and k, the whole branch cache, the status."""
    s = STRUCTS[name]()
    tb = synth.make_tensors(s)
    db, tabs = _run_step(rt, s, tb)
    n = tabs["n_active"]
    act = tabs["active_slot"][:n]
    db2 = rt.DeviceBatch(s, tb)
    db2.build_meta()
    db2.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    db2.rope_append()
    db2.attn(True)
    torch.cuda.synchronize()
    assert db2.status() == db.status() == 0
    for a in ("q", "k_new", "suffix_k", "suffix_v", "o"):
        assert np.array_equal(rt.bits_of(getattr(db2, a)), rt.bits_of(getattr(db, a))), a


def test_fused_rope_append_full_slab(rt):
    """A full slab: the fused call still rotates the row's q and k, writes nothing to the cache and raises the status bit."""
    from paper_2604_26209_b200 import binding
    s = synth.config_custom("ovf", Hq=4, Hkv=1, D=64, theta=10000.0, cap=4, prefix_lens=[16], branch_cnts=[3],
                            depth_hi=1, seed=14)
    s.slot_depth[:] = [0, 4, 2]
    tb = synth.make_tensors(s)
    out = []
    for fused in (False, True):
        db = rt.DeviceBatch(s, tb)
        db.build_meta()
        db.set_step_inputs(tb["q"], tb["k_new"], tb["v_new"])
        if fused:
            db.rope_append()
        else:
            db.rope(); db.kv_append()
        torch.cuda.synchronize()
        assert db.status() == binding.HPD_S_OVERFLOW
        out.append([rt.bits_of(getattr(db, a)).copy() for a in ("q", "k_new", "suffix_k", "suffix_v")])
    for a, b in zip(*out):
        assert np.array_equal(a, b)
    assert np.array_equal(out[1][2][4:8], tb["suffix_k"][4:8])


def test_graph_replay_equals_direct_calls(rt):
    """The step captured in a CUDA graph launches the same kernels on the same buffers: same bits."""
    s = synth.config_main(n_prompts=2)
    tb = synth.make_tensors(s)
    db, tabs = _run_step(rt, s, tb)
    n = tabs["n_active"]
    act = tabs["active_slot"][:n]
    o0 = rt.bits_of(db.o)[:n].copy()
    g = db.capture_step(with_meta=True)
    for _ in range(2):
        db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])     # rope rotates q and k in place
        db.o.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert db.status() == 0
        assert np.array_equal(rt.bits_of(db.o)[:n], o0)


def test_attention_is_bitwise_reproducible_across_launches(rt):
    """Work units are handed to the kernel's two pipelines per SM by a ticket counter, so which pipeline computes a
    row changes from launch to launch; the tiles of a unit are always taken in the same order, so the bits must not."""
    s = synth.config_main(n_prompts=8)                  # more units than pipelines: the ticket counter is in use
    tb = synth.make_tensors(s)
    db, tabs = _run_step(rt, s, tb)
    n = tabs["n_active"]
    o0, l0 = rt.bits_of(db.o)[:n].copy(), db.lse.cpu().numpy()[:n].copy()
    for _ in range(3):
        db.attn(True)
        torch.cuda.synchronize()
        assert db.status() == 0
        assert np.array_equal(rt.bits_of(db.o)[:n], o0)
        assert np.array_equal(db.lse.cpu().numpy()[:n], l0)


@pytest.mark.parametrize("name", ["tiny", "main_p2", "ragged", "ragged_d64_g2", "long_small"])
def test_std_decode_matches_oracle_and_hpd(rt, name):
    s = STRUCTS[name]()
    tb = synth.make_tensors(s)
    meta, want = oracle_step(s, tb)
    db, tabs = _run_step(rt, s, tb)
    n = meta.n_active
    dup = rt.DupBatch(db, include_new=True)
    dup.attn(db.q)
    torch.cuda.synchronize()
    o_std = synth.bf16_bits_to_f32(rt.bits_of(dup.o))[:n]
    mx, mean = err_stats(o_std, want.o)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    o_hpd = synth.bf16_bits_to_f32(rt.bits_of(db.o))[:n]
    mx, mean = err_stats(o_std, o_hpd)
    assert mx <= 2 * MAX_ABS and mean <= 2 * MEAN_ABS
    assert np.max(np.abs(dup.lse.cpu().numpy()[:n] - want.lse)) <= 2e-2


def test_std_decode_split_kv_small_batch(rt):
    """Few rows and long sequences: the split-KV path of the comparison kernel."""
    s = synth.config_custom("split", Hq=32, Hkv=8, D=128, theta=500000.0, cap=8, prefix_lens=[3000, 2500],
                            branch_cnts=[2, 1], depth_hi=8, seed=11)
    tb = synth.make_tensors(s)
    meta, want = oracle_step(s, tb)
    db, _ = _run_step(rt, s, tb)
    dup = rt.DupBatch(db)
    from paper_2604_26209_b200 import binding
    assert binding.std_workspace_bytes(s.geom, dup.n, dup.max_seq_len) > 0
    dup.attn(db.q)
    torch.cuda.synchronize()
    mx, mean = err_stats(synth.bf16_bits_to_f32(rt.bits_of(dup.o))[: dup.n], want.o)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


def test_gpu_output_independent_of_stacking_and_order(rt):
    """Eq. 4 on the GPU: re-ordering documents / retiring other branches leaves a branch's output
    within tolerance (the schedule may change the rounding order, not the value)."""
    s = _ragged(12, alive_frac=1.0)
    tb = synth.make_tensors(s)
    db, tabs = _run_step(rt, s, tb)
    n = tabs["n_active"]
    base = {int(sl): synth.bf16_bits_to_f32(rt.bits_of(db.o))[r] for r, sl in enumerate(tabs["active_slot"][:n])}
    alive = s.slot_alive.copy()
    alive[::3] = 0
    s2 = replace(s, slot_alive=alive)
    db2, tabs2 = _run_step(rt, s2, tb)
    o2 = synth.bf16_bits_to_f32(rt.bits_of(db2.o))
    for r, sl in enumerate(tabs2["active_slot"][: tabs2["n_active"]]):
        assert np.max(np.abs(o2[r] - base[int(sl)])) <= MAX_ABS


def test_attention_before_append_sees_depth_tokens_only(rt):
    """suffix_includes_new = 0: the branch sees exactly suffix_len cached tokens (oracle: depth-1 state)."""
    s = _ragged(13, alive_frac=1.0)
    s.slot_depth[:] = np.maximum(s.slot_depth, 1)
    tb = synth.make_tensors(s)
    # oracle view: the last cached token plays the role of the "new" token of a step at depth-1
    s_prev = replace(s, slot_depth=s.slot_depth - 1)
    from oracle import capi
    meta_prev = capi.build_meta(s_prev.doc_prefix_len, s_prev.doc_branch_cnt, s_prev.slot_depth, s_prev.slot_alive,
                                s.geom.suffix_cap, 0)
    f = widen(tb)
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    tabs = db.tables()
    n = tabs["n_active"]
    act = tabs["active_slot"][:n]
    db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    db.rope()
    db.attn(False)
    torch.cuda.synchronize()
    q_rot = synth.bf16_bits_to_f32(rt.bits_of(db.q))[:n]
    # reference by direct evaluation with the oracle's attention routine on the visible tokens
    o_gpu = synth.bf16_bits_to_f32(rt.bits_of(db.o))[:n]
    kv0 = np.concatenate([[0], np.cumsum(s.doc_prefix_len)])
    for r in range(0, n, 7):
        d, sl = tabs["doc_id"][r], act[r]
        K = np.concatenate([f["prefix_k"][kv0[d]:kv0[d + 1]], f["suffix_k"][sl * s.geom.suffix_cap: sl * s.geom.suffix_cap + s.slot_depth[sl]]])
        V = np.concatenate([f["prefix_v"][kv0[d]:kv0[d + 1]], f["suffix_v"][sl * s.geom.suffix_cap: sl * s.geom.suffix_cap + s.slot_depth[sl]]])
        o, _ = capi.causal_attention_row(K.shape[0] - 1, q_rot[r], K, V, s.geom.sm_scale)
        assert np.max(np.abs(o_gpu[r] - o)) <= MAX_ABS


def test_overflow_sets_status_and_suppresses_write(rt):
    s = synth.config_custom("ovf", Hq=4, Hkv=1, D=64, theta=10000.0, cap=4, prefix_lens=[16], branch_cnts=[3],
                            depth_hi=1, seed=14)
    s.slot_depth[:] = [0, 4, 2]                 # slot 1 is full
    tb = synth.make_tensors(s)
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    db.set_step_inputs(tb["q"], tb["k_new"], tb["v_new"])
    db.rope()
    db.kv_append()
    torch.cuda.synchronize()
    from paper_2604_26209_b200 import binding
    assert db.status() & binding.HPD_S_OVERFLOW
    sk = rt.bits_of(db.suffix_k)
    assert np.array_equal(sk[4:8], tb["suffix_k"][4:8])          # full slab untouched
    assert not np.array_equal(sk[0], tb["suffix_k"][0])          # slot 0 got its token
