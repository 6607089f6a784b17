"""Pins of the attention / visual-mass oracle: things other than the oracle
itself fix every number checked here (torch SDPA in fp64, closed forms,
numpy brute force, invariances)."""
import numpy as np
import pytest
import torch

from paper_2604_05650_b200 import workloads as W


def _bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _rand_case(rng, B=2, gamma=3, Hq=4, Hkv=2, D=16, Lmax=40, kv_len=None, span=None):
    q = _bits(rng.standard_normal((B, gamma, Hq, D)))
    k = _bits(rng.standard_normal((B, Hkv, Lmax, D)))
    v = _bits(rng.standard_normal((B, Hkv, Lmax, D)))
    kv_len = np.asarray(kv_len if kv_len is not None else [Lmax] * B, dtype=np.int32)
    span = np.asarray(span if span is not None else [[3, Lmax // 2]] * B, dtype=np.int32)
    return q, k, v, kv_len, span


def _sdpa(q, k, v, kv_len):
    """torch's scaled_dot_product_attention in fp64 on CPU, GQA by repeating KV
    heads, causal tail as an explicit boolean mask."""
    qf = torch.from_numpy(W.bf16_bits_to_f32(q)).double()
    kf = torch.from_numpy(W.bf16_bits_to_f32(k)).double()
    vf = torch.from_numpy(W.bf16_bits_to_f32(v)).double()
    B, gamma, Hq, D = qf.shape
    Hkv, Lmax = kf.shape[1], kf.shape[2]
    G = Hq // Hkv
    kf = kf.repeat_interleave(G, dim=1)
    vf = vf.repeat_interleave(G, dim=1)
    mask = torch.zeros(B, 1, gamma, Lmax, dtype=torch.bool)
    for b in range(B):
        for g in range(gamma):
            mask[b, 0, g, : int(kv_len[b]) - gamma + g + 1] = True
    o = torch.nn.functional.scaled_dot_product_attention(
        qf.permute(0, 2, 1, 3), kf, vf, attn_mask=mask)
    return o.permute(0, 2, 1, 3).numpy()


def test_matches_torch_sdpa_fp64(oracle_mod):
    rng = np.random.default_rng(1)
    q, k, v, kv_len, span = _rand_case(rng, B=2, gamma=4, Hq=6, Hkv=2, D=32, Lmax=75,
                                       kv_len=[75, 41], span=[[5, 60], [0, 30]])
    out, mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    np.testing.assert_allclose(out, _sdpa(q, k, v, kv_len), rtol=1e-11, atol=1e-12)


def test_mass_equals_sdpa_on_indicator_values(oracle_mod):
    """With V[j, 0] = 1 inside the span and 0 outside, SDPA's output channel 0
    is the softmax mass on the span: an independent route to the mass."""
    rng = np.random.default_rng(2)
    q, k, v, kv_len, span = _rand_case(rng, B=2, gamma=3, Hq=4, Hkv=2, D=16, Lmax=50,
                                       kv_len=[50, 33], span=[[7, 29], [2, 30]])
    _, mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    ind = np.zeros(k.shape, dtype=np.float32)
    for b in range(2):
        ind[b, :, span[b, 0]:span[b, 1], 0] = 1.0
    ref = _sdpa(q, k, _bits(ind), kv_len)[..., 0]
    np.testing.assert_allclose(mass, ref, rtol=1e-11, atol=1e-13)


def test_numpy_brute_force_tiny(oracle_mod):
    rng = np.random.default_rng(3)
    q, k, v, kv_len, span = _rand_case(rng, B=1, gamma=2, Hq=2, Hkv=1, D=8, Lmax=9,
                                       kv_len=[9], span=[[2, 6]])
    out, mass, probs = oracle_mod.verify_attention(q, k, v, kv_len, span, return_probs=True)
    qf, kf, vf = (W.bf16_bits_to_f32(a).astype(np.float64) for a in (q, k, v))
    for g in range(2):
        n = 9 - 2 + g + 1
        for h in range(2):
            s = kf[0, 0, :n] @ qf[0, g, h] / np.sqrt(8.0)
            p = np.exp(s - s.max())
            p /= p.sum()
            np.testing.assert_allclose(probs[0, g, h, :n], p, rtol=1e-12)
            assert (probs[0, g, h, n:] == 0).all()
            np.testing.assert_allclose(out[0, g, h], p @ vf[0, 0, :n], rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(mass[0, g, h], p[2:6].sum(), rtol=1e-12)


def test_identical_keys_give_mean_value_and_visual_fraction(oracle_mod):
    rng = np.random.default_rng(4)
    B, gamma, Hq, Hkv, D, L = 1, 3, 4, 2, 16, 37
    q, k, v, kv_len, span = _rand_case(rng, B, gamma, Hq, Hkv, D, L, span=[[4, 20]])
    k[:] = k[:, :, :1, :]                      # every key of a head is the same vector
    out, mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    vf = W.bf16_bits_to_f32(v).astype(np.float64)
    for g in range(gamma):
        n = L - gamma + g + 1
        for h in range(Hq):
            np.testing.assert_allclose(out[0, g, h], vf[0, h // 2, :n].mean(0),
                                       rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(mass[0, g, h], 16.0 / n, rtol=1e-12)


def test_dominant_key_selects_its_value_row(oracle_mod):
    B, gamma, Hq, Hkv, D, L = 1, 2, 2, 1, 16, 30
    q = _bits(np.full((B, gamma, Hq, D), 4.0))
    kf = np.zeros((B, Hkv, L, D), dtype=np.float32)
    kf[0, 0, 11] = 8.0                         # score 4*8*16/4 = 128 above the rest
    rng = np.random.default_rng(5)
    v = _bits(rng.standard_normal((B, Hkv, L, D)))
    kv_len = np.asarray([L], dtype=np.int32)
    vf = W.bf16_bits_to_f32(v).astype(np.float64)
    for span, expect in (([[5, 20]], 1.0), ([[12, 20]], 0.0)):
        out, mass = oracle_mod.verify_attention(q, _bits(kf), v, kv_len,
                                                np.asarray(span, dtype=np.int32))
        np.testing.assert_allclose(out[0, :, :], np.broadcast_to(vf[0, 0, 11], (2, 2, D)),
                                   atol=1e-40 + 1e-12)
        np.testing.assert_allclose(mass, expect, atol=1e-12)


def test_key_translation_leaves_probabilities_unchanged(oracle_mod):
    """Adding one vector c to every key shifts all scores of a row by q.c."""
    rng = np.random.default_rng(6)
    B, gamma, Hq, Hkv, D, L = 1, 2, 2, 1, 8, 20
    q = _bits(rng.integers(-4, 5, (B, gamma, Hq, D)) * 0.5)
    kf = (rng.integers(-4, 5, (B, Hkv, L, D)) * 0.5).astype(np.float32)
    c = (rng.integers(-2, 3, (D,)) * 4.0).astype(np.float32)   # k + c stays exact in bf16
    v = _bits(rng.standard_normal((B, Hkv, L, D)))
    kv_len = np.asarray([L], dtype=np.int32)
    span = np.asarray([[3, 11]], dtype=np.int32)
    assert (W.bf16_bits_to_f32(_bits(kf + c)) == kf + c).all()
    o1, m1, p1 = oracle_mod.verify_attention(q, _bits(kf), v, kv_len, span, return_probs=True)
    o2, m2, p2 = oracle_mod.verify_attention(q, _bits(kf + c), v, kv_len, span, return_probs=True)
    np.testing.assert_allclose(p1, p2, rtol=1e-10, atol=1e-300)
    np.testing.assert_allclose(o1, o2, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(m1, m2, rtol=1e-10)


def test_probability_rows_and_mass_invariants(oracle_mod):
    rng = np.random.default_rng(7)
    B, gamma, Lmax = 2, 4, 64
    q, k, v, kv_len, _ = _rand_case(rng, B=B, gamma=gamma, Hq=4, Hkv=2, D=16, Lmax=Lmax,
                                    kv_len=[64, 50])
    def run(span):
        return oracle_mod.verify_attention(q, k, v, kv_len, np.asarray(span, dtype=np.int32),
                                           return_probs=True)
    _, m_a, probs = run([[5, 20], [5, 20]])
    np.testing.assert_allclose(probs.sum(-1), 1.0, atol=1e-12)
    assert (m_a >= 0).all() and (m_a <= 1).all()
    _, m_b, _ = run([[20, 41], [20, 41]])
    _, m_ab, _ = run([[5, 41], [5, 41]])
    np.testing.assert_allclose(m_a + m_b, m_ab, atol=1e-13)            # additivity
    _, m_empty, _ = run([[9, 9], [0, 0]])
    assert (m_empty == 0).all()
    # span = everything before the draft tail: 1 - mass is the tail's share
    full = [[0, int(kv_len[0]) - gamma], [0, int(kv_len[1]) - gamma]]
    _, m_full, _ = run(full)
    for b in range(B):
        tail = probs[b, :, :, int(kv_len[b]) - gamma:int(kv_len[b])].sum(-1)
        np.testing.assert_allclose(m_full[b], 1.0 - tail, atol=1e-13)


def test_causal_tail_and_slots_beyond_kv_len_are_invisible(oracle_mod):
    rng = np.random.default_rng(8)
    gamma, Lmax, L = 3, 48, 40
    q, k, v, kv_len, span = _rand_case(rng, B=1, gamma=gamma, Hq=2, Hkv=1, D=16, Lmax=Lmax,
                                       kv_len=[L], span=[[2, 30]])
    o1, m1 = oracle_mod.verify_attention(q, k, v, kv_len, span)
    for g in range(gamma):
        k2, v2 = k.copy(), v.copy()
        first_hidden = L - gamma + g + 1
        k2[:, :, first_hidden:] = _bits(rng.standard_normal(k2[:, :, first_hidden:].shape) * 9)
        v2[:, :, first_hidden:] = _bits(rng.standard_normal(v2[:, :, first_hidden:].shape) * 9)
        o2, m2 = oracle_mod.verify_attention(q, k2, v2, kv_len, span)
        assert (o2[0, g] == o1[0, g]).all() and (m2[0, g] == m1[0, g]).all()
        if g + 1 < gamma:
            assert not (o2[0, g + 1:] == o1[0, g + 1:]).all()
    # the last visible key does matter to its query
    k3 = k.copy()
    k3[0, 0, L - gamma] = _bits(rng.standard_normal(16) * 9)
    o3, _ = oracle_mod.verify_attention(q, k3, v, kv_len, span)
    assert not (o3[0, 0] == o1[0, 0]).all()


def test_gqa_head_mapping(oracle_mod):
    """Query head h reads KV head h // G: zeroing one KV head's values zeroes
    exactly its G query heads."""
    rng = np.random.default_rng(9)
    q, k, v, kv_len, span = _rand_case(rng, B=1, gamma=2, Hq=6, Hkv=3, D=8, Lmax=12)
    v[0, 1] = 0
    out, _ = oracle_mod.verify_attention(q, k, v, kv_len, span)
    zero_heads = [h for h in range(6) if (out[0, :, h] == 0).all()]
    assert zero_heads == [2, 3]


def test_config0_mass_reflects_the_planted_key_shift(oracle_mod):
    """Workload sanity: visual keys carry a mean shift, so the visual mass of
    config 0 must sit in (0, 1) and differ between heads."""
    cfg = W.CONFIGS[0]
    q, k, v, kv_len, span = W.attention_inputs(cfg)
    out, mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    assert out.shape == (1, 4, 8, 64) and mass.shape == (1, 4, 8)
    assert 0.3 < mass.min() and mass.max() < 0.99 and mass.std() > 1e-3
