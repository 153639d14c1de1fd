"""Pins for the oracle's position-ID and bookkeeping code (no GPU)."""
import os

import numpy as np
import pytest

from oracle import capi
from paper_2604_26209_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "alg2_fig2_positions.txt")


def _golden():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, a, b = line.split("|")
        return int(k), [int(x) for x in a.split()], [int(x) for x in b.split()]


def test_alg2_matches_the_numbers_printed_for_fig2():
    """Sec. 4.3.1-4.3.2: with K_max = 7 the first value tokens are read at positions 12/22/32 and
    receive IDs 13/23/33.  A 10-token prompt followed by three 3-token attributes reproduces them."""
    k_max, read_at, given = _golden()
    start, end = [10, 13, 16], [12, 15, 18]
    pos = capi.alg2_position_ids(19, start, end, k_max)
    assert [int(pos[e]) for e in end] == read_at
    assert [capi.alg2_value_position(pos, end, n, 1) for n in range(3)] == given
    # the prompt itself is untouched and IDs stay strictly increasing (ordering preserved)
    assert pos[:10].tolist() == list(range(10))
    assert np.all(np.diff(pos) > 0)


@pytest.mark.parametrize("k_max", [1, 7, 30])
def test_alg2_offsets_are_multiples_of_kmax(k_max):
    rng = np.random.default_rng(k_max)
    lens = rng.integers(1, 5, size=6)
    p = 11
    start = p + np.concatenate([[0], np.cumsum(lens)[:-1]])
    end = start + lens - 1
    pos = capi.alg2_position_ids(int(p + lens.sum()), start, end, k_max)
    for i in range(6):
        assert pos[start[i]] - start[i] == i * k_max
        assert pos[end[i]] - end[i] == i * k_max
    # consecutive attributes are separated by exactly K_max free IDs
    for i in range(5):
        assert pos[start[i + 1]] - pos[end[i]] - 1 == k_max


def _meta_by_numpy(L, cnt, depth, alive, cap, gap):
    """The same tables from array operations instead of loops."""
    L, cnt, depth = (np.asarray(a, dtype=np.int64) for a in (L, cnt, depth))
    alive = np.asarray(alive).astype(bool)
    nd, ns = len(L), len(depth)
    kv = np.concatenate([[0], np.cumsum(L)])
    sl = np.concatenate([[0], np.cumsum(cnt)])
    slot_doc = np.repeat(np.arange(nd), cnt)
    slot_j = np.arange(ns) - sl[slot_doc] if ns else np.zeros(0, np.int64)
    act = np.nonzero(alive)[0]
    per_doc = np.bincount(slot_doc[act], minlength=nd) if ns else np.zeros(nd, np.int64)
    ast = np.concatenate([[0], np.cumsum(per_doc)])
    pad = lambda a: np.concatenate([a, -np.ones(ns - len(a), dtype=np.int64)]).astype(np.int32)
    bs = L[slot_doc[act]] + slot_j[act] * gap
    return dict(doc_kv_start=kv.astype(np.int32), doc_slot_start=sl.astype(np.int32),
                doc_active_start=ast.astype(np.int32), active_slot=pad(act), doc_id=pad(slot_doc[act]),
                branch_start=pad(bs), pos_id=pad(bs + depth[act]), suffix_off=pad(act * cap),
                suffix_len=pad(depth[act])), len(act)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("gap", [0, 7])
def test_build_meta_against_array_formulation(seed, gap):
    rng = np.random.default_rng(seed)
    nd = int(rng.integers(1, 9))
    L = rng.integers(0, 50, size=nd)
    cnt = rng.integers(0, 6, size=nd)
    ns = int(cnt.sum())
    depth = rng.integers(0, 8, size=ns)
    alive = (rng.random(ns) < 0.6).astype(np.uint8)
    m = capi.build_meta(L, cnt, depth, alive, 8, gap)
    want, na = _meta_by_numpy(L, cnt, depth, alive, 8, gap)
    assert m.n_active == na
    for name in capi.Meta.TABLES:
        assert np.array_equal(getattr(m, name), want[name]), name


def test_counting_identity_b_times_J_times_N():
    """Sec. 4.3.6: with nothing pruned a step carries b*J*N tokens."""
    s = synth.config_main(n_prompts=3)
    m = capi.build_meta(s.doc_prefix_len, s.doc_branch_cnt, s.slot_depth, s.slot_alive, s.geom.suffix_cap)
    assert m.n_active == 3 * 4 * 24
    assert np.array_equal(m.active_slot, np.arange(3 * 96))
    assert np.all(np.diff(m.doc_active_start) == 24)


def test_positions_continue_the_document():
    """Contiguous mode: the branch continues its document, so pos = L_d + depth."""
    m = capi.build_meta([5, 9], [2, 3], [0, 3, 1, 0, 2], [1, 1, 1, 0, 1], 4, 0)
    assert m.pos_id[:4].tolist() == [5, 8, 10, 11]
    assert m.branch_start[:4].tolist() == [5, 5, 9, 9]
    assert m.suffix_off[:4].tolist() == [0, 4, 8, 16]
    assert m.doc_id[:4].tolist() == [0, 0, 1, 1]
    assert m.doc_active_start.tolist() == [0, 2, 4]


def test_gap_mode_uses_alg2_running_offset():
    """With pos_gap = K_max the j-th branch of a document is shifted by Algorithm 2's offset j*K_max."""
    k_max = 7
    m = capi.build_meta([10], [3], [1, 1, 1], [1, 1, 1], 8, k_max)
    start, end = [10, 13, 16], [12, 15, 18]
    pos = capi.alg2_position_ids(19, start, end, k_max)
    shift = [int(pos[s]) - s for s in start]                 # Algorithm 2's offsets 0, K, 2K
    assert (m.branch_start[:3] - 10).tolist() == shift
    assert (m.pos_id[:3] - m.branch_start[:3]).tolist() == [1, 1, 1]


def test_retired_and_empty():
    m = capi.build_meta([4, 4], [2, 2], [0, 0, 0, 0], [0, 0, 0, 0], 4, 0)
    assert m.n_active == 0 and np.all(m.active_slot == -1)
    assert m.doc_active_start.tolist() == [0, 0, 0]
    m = capi.build_meta([], [], [], [], 4, 0)
    assert m.n_active == 0 and m.doc_kv_start.tolist() == [0]
    with pytest.raises(ValueError):
        capi.build_meta([4], [3], [0, 0], [1, 1], 4, 0)      # branch counts do not add up


def test_advance_prunes_on_delimiter_and_truncates_at_k_max():
    """Sec. 4.3.4 on a hand-written case: K_max = 3, delimiter 9.  Slots 0..4; slot 3 is already retired."""
    depth = np.array([0, 2, 1, 1, 2], np.int32)
    alive = np.array([1, 1, 1, 0, 1], np.uint8)
    meta = capi.build_meta([5], [5], depth, alive, 3, 0)
    assert list(meta.active_slot[:4]) == [0, 1, 2, 4]
    stay = capi.advance(meta, [7, 7, 9, 9], 9, 3, depth, alive)
    # slot 0: 0 -> 1, goes on; slot 1: 2 -> 3 = K_max, truncated although no delimiter came; slot 2: delimiter;
    # slot 3: untouched; slot 4: delimiter (and full)
    assert list(depth) == [1, 3, 2, 1, 3] and list(alive) == [1, 0, 0, 0, 0] and stay == 1


def test_loop_ends_when_all_values_are_pruned_or_after_k_max_steps():
    """Algorithm 1's loop with the prune rule: a value of K tokens is alive for exactly min(K, K_max) steps, its slab ends
    up holding min(K, K_max) tokens, and the loop stops by itself after max(min(K, K_max)) <= K_max steps."""
    rng = np.random.default_rng(4)
    k_max, delim = 6, 0
    K = rng.integers(1, 11, size=40)                                   # value lengths, some longer than K_max
    depth, alive = np.zeros(40, np.int32), np.ones(40, np.uint8)
    steps = 0
    while True:
        meta = capi.build_meta([3, 9], [15, 25], depth, alive, k_max, 0)
        if meta.n_active == 0:
            break
        assert steps < k_max
        act = meta.active_slot[: meta.n_active]
        assert np.array_equal(act, np.nonzero(np.minimum(K, k_max) > steps)[0])
        tok = np.where(depth[act] + 1 == K[act], delim, 5)             # the token sampled at this step
        capi.advance(meta, tok, delim, k_max, depth, alive)
        steps += 1
    assert steps == int(np.minimum(K, k_max).max()) and np.array_equal(depth, np.minimum(K, k_max))
