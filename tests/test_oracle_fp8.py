"""Pins of the oracle's fp8-cache attention: the E4M3 decode against the format's
published definition (spot values written out, and an independent library decoder), the
attention against torch's scaled-dot-product attention in fp64 on the decoded cache, scale
identities, and agreement with the (separately pinned) bf16-cache oracle where the cache
values are exactly representable in both formats."""
import numpy as np
import pytest
import torch

from paper_2604_05650_b200 import workloads as W


def test_e4m3_decode_spot_values(oracle_mod):
    d = oracle_mod.e4m3_decode
    assert d(0x00) == 0.0 and d(0x80) == 0.0 and np.signbit(d(0x80))
    assert d(0x38) == 1.0 and d(0xB8) == -1.0            # exponent field 7 = bias
    assert d(0x01) == 2.0 ** -9                          # smallest subnormal
    assert d(0x07) == 7 * 2.0 ** -9                      # largest subnormal
    assert d(0x08) == 2.0 ** -6                          # smallest normal
    assert d(0x7E) == 448.0 and d(0xFE) == -448.0        # largest finite
    assert d(0x40) == 2.0 and d(0x3C) == 1.5 and d(0x39) == 1.125
    assert np.isnan(d(0x7F)) and np.isnan(d(0xFF))       # the two NaN codes
    pos = [d(c) for c in range(0x7F)]
    assert all(b > a for a, b in zip(pos, pos[1:]))      # codes order like their values
    assert all(d(c | 0x80) == -d(c) for c in range(0x7F))


def test_e4m3_decode_matches_torch_float8(oracle_mod):
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = np.asarray([oracle_mod.e4m3_decode(c) for c in range(256)])
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok]) and np.array_equal(np.signbit(ref[ok]), np.signbit(got[ok]))


def test_input_encoder_rounds_to_nearest_even(oracle_mod):
    """The generator's encoder (input preparation, not part of the oracle): every code
    encodes to itself, midpoints go to the even code, values beyond 448 saturate, and
    random values agree with torch's own conversion."""
    vals = np.asarray([oracle_mod.e4m3_decode(c) for c in range(0x7F)])
    assert np.array_equal(W.f32_to_e4m3_bits(vals.astype(np.float32)), np.arange(0x7F, dtype=np.uint8))
    mid = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)            # exact in fp32
    got = W.f32_to_e4m3_bits(mid)
    assert all(g % 2 == 0 and g in (i, i + 1) for i, g in enumerate(got))
    assert W.f32_to_e4m3_bits(np.asarray([1e6, -500.0], dtype=np.float32)).tolist() == [0x7E, 0xFE]
    x = (np.random.default_rng(5).standard_normal(20000) * 40).astype(np.float32)
    x = x[np.abs(x) <= 448]
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(W.f32_to_e4m3_bits(x), ref)


def _case(seed, B, gamma, Hq, Hkv, D, Lmax, kv_len, span):
    rng = np.random.default_rng(seed)
    bits = lambda shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    q, k, v = bits((B, gamma, Hq, D)), bits((B, Hkv, Lmax, D)), bits((B, Hkv, Lmax, D))
    k8, ks = W.quantize_cache_e4m3(k)
    v8, vs = W.quantize_cache_e4m3(v)
    return q, k8, v8, ks, vs, np.asarray(kv_len, np.int32), np.asarray(span, np.int32)


def _decode_torch(c8, scale):
    x = torch.from_numpy(c8).view(torch.float8_e4m3fn).to(torch.float64)
    return x * torch.from_numpy(scale.astype(np.float64))[:, :, None, None]


def test_fp8_attention_matches_torch_sdpa_fp64(oracle_mod):
    B, gamma, Hq, Hkv, D, Lmax = 2, 3, 6, 2, 64, 200
    q, k8, v8, ks, vs, kv_len, span = _case(1, B, gamma, Hq, Hkv, D, Lmax, [200, 131], [[10, 150], [0, 100]])
    out, mass = oracle_mod.verify_attention_fp8(q, k8, v8, ks, vs, kv_len, span)
    qd = torch.from_numpy(W.bf16_bits_to_f32(q)).double()
    kd, vd = _decode_torch(k8, ks), _decode_torch(v8, vs)
    G = Hq // Hkv
    for b in range(B):
        L = int(kv_len[b])
        kk = kd[b, :, :L].repeat_interleave(G, dim=0)
        vv = vd[b, :, :L].repeat_interleave(G, dim=0)
        qq = qd[b].permute(1, 0, 2)                                 # [Hq, gamma, D]
        j = torch.arange(L)[None, :]
        visible = j < (L - gamma + torch.arange(gamma)[:, None] + 1)
        ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, attn_mask=visible[None])
        assert np.abs(out[b] - ref.permute(1, 0, 2).numpy()).max() < 1e-12
        # mass = SDPA on indicator values: the share of probability inside the span
        ind = ((j[0] >= span[b, 0]) & (j[0] < span[b, 1])).double()[None, :, None].expand(Hq, L, 1)
        m_ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, ind.contiguous(), attn_mask=visible[None])
        assert np.abs(mass[b] - m_ref[..., 0].permute(1, 0).numpy()).max() < 1e-12


def test_scale_identities(oracle_mod):
    q, k8, v8, ks, vs, kv_len, span = _case(2, 1, 4, 4, 2, 64, 150, [150], [[20, 120]])
    out, mass = oracle_mod.verify_attention_fp8(q, k8, v8, ks, vs, kv_len, span)
    # V scale is linear in out and leaves the probabilities alone
    out3, mass3 = oracle_mod.verify_attention_fp8(q, k8, v8, ks, vs * np.float32(4.0), kv_len, span)
    assert np.array_equal(out3, out * 4.0) and np.array_equal(mass3, mass)
    # doubling the K scale is doubling q (both exact)
    q2 = W.f32_to_bf16_bits(W.bf16_bits_to_f32(q) * np.float32(2.0))
    a = oracle_mod.verify_attention_fp8(q, k8, v8, ks * np.float32(2.0), vs, kv_len, span)
    b = oracle_mod.verify_attention_fp8(q2, k8, v8, ks, vs, kv_len, span)
    assert np.abs(a[0] - b[0]).max() < 1e-12 and np.abs(a[1] - b[1]).max() < 1e-12
    # a zero K scale makes every score equal: out = mean of the visible values, mass = visible share
    z = oracle_mod.verify_attention_fp8(q, k8, v8, ks * 0, vs, kv_len, span)
    vd = _decode_torch(v8, vs).numpy()
    for g in range(4):
        n = 150 - 4 + g + 1
        assert np.abs(z[0][0, g, 0] - vd[0, 0, :n].mean(0)).max() < 1e-12
        assert abs(z[1][0, g, 3] - 100.0 / n) < 1e-12


def test_agrees_with_the_bf16_cache_oracle_on_values_both_formats_hold(oracle_mod):
    """Cache values drawn from the E4M3 grid are exact in bf16 too (3 mantissa bits, small
    exponents); with scale 1 both oracle functions must give the same numbers."""
    rng = np.random.default_rng(3)
    B, gamma, Hq, Hkv, D, Lmax = 1, 5, 4, 2, 64, 300
    k8 = rng.integers(0, 0x60, (B, Hkv, Lmax, D)).astype(np.uint8) | (rng.integers(0, 2, (B, Hkv, Lmax, D)) << 7).astype(np.uint8)
    v8 = rng.integers(0, 0x60, (B, Hkv, Lmax, D)).astype(np.uint8) | (rng.integers(0, 2, (B, Hkv, Lmax, D)) << 7).astype(np.uint8)
    dec = np.vectorize(oracle_mod.e4m3_decode)
    kf, vf = dec(k8).astype(np.float32) / 8, dec(v8).astype(np.float32)
    kb, vb = W.f32_to_bf16_bits(kf), W.f32_to_bf16_bits(vf)
    assert np.array_equal(W.bf16_bits_to_f32(kb), kf) and np.array_equal(W.bf16_bits_to_f32(vb), vf)
    q = W.f32_to_bf16_bits(rng.standard_normal((B, gamma, Hq, D)).astype(np.float32))
    kv_len, span = np.asarray([290], np.int32), np.asarray([[30, 200]], np.int32)
    one = np.ones((B, Hkv), np.float32)
    a = oracle_mod.verify_attention_fp8(q, k8, v8, one / 8, one, kv_len, span)
    b = oracle_mod.verify_attention(q, kb, vb, kv_len, span)
    assert np.abs(a[0] - b[0]).max() < 1e-12 and np.abs(a[1] - b[1]).max() < 1e-12
    assert ((a[1] >= 0) & (a[1] <= 1 + 1e-12)).all()
