"""Pins for the oracle's rotary embedding and attention arithmetic (no GPU)."""
import numpy as np
import pytest
import torch

from oracle import capi, brute


# ----------------------------------------------------------------------------------- rope
def test_rope_position_zero_is_identity():
    x = np.random.default_rng(0).standard_normal((3, 16)).astype(np.float32)
    assert np.array_equal(capi.rope(x, 0, 10000.0), x.astype(np.float64))


def test_rope_d2_closed_form():
    """D = 2: a single pair with inverse frequency 1, i.e. a plane rotation by `pos` radians."""
    x = np.array([[0.75, -1.5]], dtype=np.float32)
    for p in (1, 5, 1000):
        r = capi.rope(x, p, 12345.0)[0]
        assert np.allclose(r, [0.75 * np.cos(p) + 1.5 * np.sin(p), -1.5 * np.cos(p) + 0.75 * np.sin(p)], atol=1e-12)


def test_rope_pairs_are_half_split_and_frequencies_decay():
    """A unit vector at index i moves only inside the pair (i, i + D/2), by the angle pos*theta^(-2i/D)."""
    D, theta, pos = 8, 100.0, 3
    for i in range(D // 2):
        e = np.zeros((1, D), dtype=np.float32)
        e[0, i] = 1.0
        r = capi.rope(e, pos, theta)[0]
        ang = pos * theta ** (-2.0 * i / D)
        want = np.zeros(D)
        want[i], want[i + D // 2] = np.cos(ang), np.sin(ang)
        assert np.allclose(r, want, atol=1e-12)


def test_rope_preserves_pair_norms_and_relative_position():
    rng = np.random.default_rng(1)
    D, theta = 64, 500000.0
    q = rng.standard_normal((1, D)).astype(np.float32)
    k = rng.standard_normal((1, D)).astype(np.float32)
    rq = capi.rope(q, 777, theta)[0]
    assert np.allclose(rq[: D // 2] ** 2 + rq[D // 2:] ** 2, q[0, : D // 2].astype(np.float64) ** 2 + q[0, D // 2:].astype(np.float64) ** 2)
    base = capi.rope(q, 40, theta)[0] @ capi.rope(k, 9, theta)[0]
    for shift in (1, 100, 4000):
        assert np.isclose(capi.rope(q, 40 + shift, theta)[0] @ capi.rope(k, 9 + shift, theta)[0], base, atol=1e-9)
    assert not np.isclose(capi.rope(q, 41, theta)[0] @ capi.rope(k, 9, theta)[0], base, atol=1e-6)


def test_rope_matches_transformers_rotate_half():
    """The decoder families the paper runs apply rope as x*cos + rotate_half(x)*sin with
    cos/sin = cat(freqs, freqs); compare with that library routine (fp64 tables)."""
    tf = pytest.importorskip("transformers.models.llama.modeling_llama")
    rng = np.random.default_rng(2)
    D, theta, pos = 128, 500000.0, 3011
    x = rng.standard_normal((4, D)).astype(np.float32)
    inv = 1.0 / (theta ** (torch.arange(0, D, 2, dtype=torch.float64) / D))
    freqs = pos * inv
    emb = torch.cat([freqs, freqs])[None, None, :]
    xt = torch.from_numpy(x).double()[None, :, None, :]            # [b, heads, seq, D]
    got, _ = tf.apply_rotary_pos_emb(xt, xt, emb.cos(), emb.sin())
    assert np.allclose(capi.rope(x, pos, theta), got[0, :, 0, :].numpy(), atol=1e-12)


def test_rope_c_and_numpy_agree():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 2, 32)).astype(np.float32)
    pos = np.array([0, 1, 17, 512, 4127])
    b = brute.rope_rows(x, pos, 10000.0)
    for n in range(5):
        assert np.allclose(capi.rope(x[n], int(pos[n]), 10000.0), b[n], atol=1e-12)


# ------------------------------------------------------------------------------ attention
def _rand(rng, *shape):
    return rng.standard_normal(shape)


@pytest.mark.parametrize("Hq,Hkv,D", [(4, 1, 64), (8, 2, 16), (3, 3, 8)])
def test_attention_rows_equal_library_causal_sdpa(Hq, Hkv, D):
    """Every row of ordinary causal attention, against torch's SDPA (fp64, CPU)."""
    rng = np.random.default_rng(Hq * 100 + D)
    n = 23
    Q, K, V = _rand(rng, n, Hq, D), _rand(rng, n, Hkv, D), _rand(rng, n, Hkv, D)
    scale = 1.0 / np.sqrt(D)
    G = Hq // Hkv
    qt = torch.from_numpy(Q).permute(1, 0, 2)[None]
    kt = torch.from_numpy(K).permute(1, 0, 2)[None].repeat_interleave(G, dim=1)
    vt = torch.from_numpy(V).permute(1, 0, 2)[None].repeat_interleave(G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=scale)[0].permute(1, 0, 2).numpy()
    for row in range(n):
        o, _ = capi.causal_attention_row(row, Q[row], K, V, scale)
        assert np.allclose(o, ref[row], atol=1e-12), row


def test_attention_closed_forms():
    rng = np.random.default_rng(5)
    Hq, Hkv, D, n = 4, 2, 8, 11
    q = _rand(rng, Hq, D)
    V = _rand(rng, n, Hkv, D)
    # all keys equal -> uniform weights -> o = mean of V
    K = np.tile(_rand(rng, 1, Hkv, D), (n, 1, 1))
    o, lse = capi.causal_attention_row(n - 1, q, K, V, 0.3)
    for h in range(Hq):
        assert np.allclose(o[h], V[:, h // 2].mean(axis=0), atol=1e-12)
        assert np.isclose(lse[h], 0.3 * q[h] @ K[0, h // 2] + np.log(n))
    # the query sees only indices <= row
    o5, _ = capi.causal_attention_row(5, q, K, V, 0.3)
    assert np.allclose(o5[0], V[:6, 0].mean(axis=0), atol=1e-12)
    # constant V -> o = that constant, whatever the scores
    K = _rand(rng, n, Hkv, D)
    c = _rand(rng, 1, Hkv, D)
    o, _ = capi.causal_attention_row(n - 1, q, K, np.tile(c, (n, 1, 1)), 1.0)
    for h in range(Hq):
        assert np.allclose(o[h], c[0, h // 2], atol=1e-12)
    # one dominant key -> o -> its V
    K2 = K.copy()
    K2[4, 0] = 50.0 * q[0] / np.linalg.norm(q[0])
    o, _ = capi.causal_attention_row(n - 1, q, K2, V, 1.0)
    assert np.allclose(o[0], V[4, 0], atol=1e-6)


def test_attention_lse_and_gqa_mapping():
    from scipy.special import logsumexp
    rng = np.random.default_rng(6)
    Hq, Hkv, D, n = 6, 3, 4, 9
    q, K, V = _rand(rng, Hq, D), _rand(rng, n, Hkv, D), _rand(rng, n, Hkv, D)
    o, lse = capi.causal_attention_row(n - 1, q, K, V, 0.5)
    for h in range(Hq):
        s = 0.5 * K[:, h // 2] @ q[h]                                # q heads 2j, 2j+1 -> kv head j
        assert np.isclose(lse[h], logsumexp(s), atol=1e-12)
        w = np.exp(s - logsumexp(s))
        assert np.allclose(o[h], w @ V[:, h // 2], atol=1e-12)
    # adding a constant to every score (q -> orthogonal shift impossible in general): use scale 0
    o0, lse0 = capi.causal_attention_row(n - 1, q, K, V, 0.0)
    assert np.allclose(o0[0], V[:, 0].mean(axis=0)) and np.isclose(lse0[0], np.log(n))


def test_attention_single_key():
    rng = np.random.default_rng(7)
    q, K, V = _rand(rng, 2, 4), _rand(rng, 1, 1, 4), _rand(rng, 1, 1, 4)
    o, lse = capi.causal_attention_row(0, q, K, V, 1.0)
    assert np.allclose(o, np.tile(V[0], (2, 1)))
    assert np.allclose(lse, K[0, 0] @ q.T)
