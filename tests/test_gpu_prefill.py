"""GPU parity of the first inference step (Sec. 4.3.2): hpd_prefill_meta + hpd_rope (in place in the prefix cache) +
hpd_prefill_attn through the C ABI against the oracle's prefill on the same seeded inputs, every row."""
import numpy as np
import pytest
import torch

from paper_2604_26209_b200 import synth
from oracle import capi
from tests.util import err_stats

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 2e-2, 2e-3
LLAMA = dict(Hq=32, Hkv=8, D=128, theta=500000.0)

STRUCTS = {
    "tiny": lambda: synth.config_skeleton("t", 4, 1, 64, 1e4, 7, [10, 5], [3, 4], key_len_hi=3, seed=0),
    "prompt_96": lambda: synth.config_skeleton("p96", **LLAMA, k_max=30, prompt_lens=[700], branch_cnts=[96], key_len_hi=4, seed=1),
    "batch_ragged": lambda: synth.config_skeleton("pb", **LLAMA, k_max=16, prompt_lens=[300, 0, 129, 512, 31],
                                                  branch_cnts=[24, 5, 0, 96, 1], key_len_hi=3, seed=3),
    "long_prompt": lambda: synth.config_skeleton("lp", **LLAMA, k_max=8, prompt_lens=[3000], branch_cnts=[6], key_len_hi=5, seed=4),
    "g8_d64": lambda: synth.config_skeleton("g8", 8, 1, 64, 1e4, 5, [140, 77], [40, 9], key_len_hi=2, seed=5),
    "g1": lambda: synth.config_skeleton("g1", 4, 4, 128, 1e4, 5, [200], [10], key_len_hi=2, seed=6),
}


@pytest.mark.parametrize("name", list(STRUCTS))
def test_prefill_matches_oracle(name):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import binding as B, runtime as rt
    s = STRUCTS[name]()
    g, dev, T = s.geom, "cuda", s.total_prefix
    rng = np.random.default_rng(11)
    qb = synth.randn_bf16(rng, (T, g.Hq, g.D)); kb = synth.randn_bf16(rng, (T, g.Hkv, g.D)); vb = synth.randn_bf16(rng, (T, g.Hkv, g.D))
    want, pos = capi.prefill(g, s.doc_prefix_len, s.doc_branch_cnt, s.slot_vis, s.pos_gap,
                             *(synth.bf16_bits_to_f32(a) for a in (qb, kb, vb)))
    bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    q, pk, pv = bf(qb), bf(kb), bf(vb)                                   # k and v already sit in the prefix cache's rows
    L, cnt, vis = i32(s.doc_prefix_len), i32(s.doc_branch_cnt), i32(s.slot_vis)
    t = B.PrefillTables.alloc(g, s.n_docs, T, dev)
    o = torch.zeros(T, g.Hq, g.D, dtype=torch.bfloat16, device=dev)
    lse = torch.zeros(T, g.Hq, dtype=torch.float32, device=dev)
    B.hpd_prefill_meta(g, s.n_docs, s.n_slots, T, L, cnt, vis, s.pos_gap, t)
    B.hpd_rope(g, T, t.n_tokens, t.tok_pos, q, pk)
    B.hpd_prefill_attn(g, s.n_docs, T, q, pk, pv, L, t, o, lse)
    torch.cuda.synchronize()
    assert int(t.dev_status.item()) == 0 and int(t.n_tokens.item()) == T
    # tables: bit-exact (positions are Algorithm 2's)
    assert np.array_equal(t.tok_pos.cpu().numpy()[:T], pos)
    kv0 = np.concatenate([[0], np.cumsum(s.doc_prefix_len)])
    assert np.array_equal(t.doc_kv_start.cpu().numpy()[: s.n_docs + 1], kv0)
    assert np.array_equal(t.tok_doc.cpu().numpy()[:T], np.repeat(np.arange(s.n_docs), s.doc_prefix_len))
    assert np.array_equal(t.tok_vis.cpu().numpy()[:T], np.concatenate([np.arange(1, n + 1) for n in s.doc_prefix_len] + [np.zeros(0, int)]))
    # the rotated keys left in the prefix cache: bf16 rounding of the fp64 rotation
    k_gpu = synth.bf16_bits_to_f32(rt.bits_of(pk))
    assert np.all(np.abs(k_gpu - want.k_rot) <= np.abs(want.k_rot) * (2.0 ** -8 + 1e-5) + 1e-6)
    got = synth.bf16_bits_to_f32(rt.bits_of(o))
    mx, mean = err_stats(got, want.o)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    assert np.max(np.abs(lse.cpu().numpy() - want.lse)) <= 2e-2
