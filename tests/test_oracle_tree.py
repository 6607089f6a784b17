"""Pins of the oracle's draft-tree variant (App. "Exploration on Draft Token
Trees": a static tree of branches with K draft tokens each, loose verification
along every branch, the branch with the longest accepted length is kept)."""
import numpy as np

from paper_2604_05650_b200 import workloads as W


def _case(seed, B, R, K, Hq, Hkv, D, ctx_len, span):
    rng = np.random.default_rng(seed)
    g = R * K
    L = ctx_len + g
    bits = lambda shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    return (bits((B, g, Hq, D)), bits((B, Hkv, L, D)), bits((B, Hkv, L, D)),
            np.full((B,), L, dtype=np.int32), np.tile(np.asarray([span], dtype=np.int32), (B, 1)))


def test_each_branch_equals_the_chain_on_its_own_cache(oracle_mod):
    """A branch must see exactly what it would see if the other branches were not
    in the cache at all."""
    B, R, K, ctx = 2, 3, 4, 37
    q, k, v, kv_len, span = _case(0, B, R, K, 4, 2, 16, ctx, (5, 30))
    out, mass = oracle_mod.verify_attention(q, k, v, kv_len, span, branch_len=K)
    for r in range(R):
        keep = list(range(ctx)) + list(range(ctx + r * K, ctx + (r + 1) * K))
        o1, m1 = oracle_mod.verify_attention(q[:, r * K:(r + 1) * K], k[:, :, keep], v[:, :, keep],
                                             np.full((B,), ctx + K, dtype=np.int32), span)
        assert np.abs(out[:, r * K:(r + 1) * K] - o1).max() < 1e-12
        assert np.abs(mass[:, r * K:(r + 1) * K] - m1).max() < 1e-12


def test_matches_torch_sdpa_with_the_tree_mask(oracle_mod):
    import torch
    B, R, K, ctx, Hq, Hkv, D = 1, 2, 5, 23, 6, 3, 8
    q, k, v, kv_len, span = _case(1, B, R, K, Hq, Hkv, D, ctx, (2, 20))
    out, _, probs = oracle_mod.verify_attention(q, k, v, kv_len, span, return_probs=True, branch_len=K)
    g, L = R * K, ctx + R * K
    tq = torch.from_numpy(W.bf16_bits_to_f32(q).astype(np.float64)).permute(0, 2, 1, 3)      # B,Hq,g,D
    rep = Hq // Hkv
    tk = torch.from_numpy(W.bf16_bits_to_f32(k).astype(np.float64)).repeat_interleave(rep, dim=1)
    tv = torch.from_numpy(W.bf16_bits_to_f32(v).astype(np.float64)).repeat_interleave(rep, dim=1)
    mask = torch.zeros(g, L, dtype=torch.bool)
    for i in range(g):
        mask[i, :ctx] = True
        r, j = divmod(i, K)
        mask[i, ctx + r * K: ctx + r * K + j + 1] = True
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)
    assert np.abs(out - ref.permute(0, 2, 1, 3).numpy()).max() < 1e-12
    assert (probs[0][:, :, :][~mask.numpy()[:, None, :].repeat(Hq, 1)] == 0).all()
    assert np.abs(probs.sum(-1) - 1.0).max() < 1e-12


def test_one_branch_is_the_plain_chain(oracle_mod):
    q, k, v, kv_len, span = _case(2, 1, 1, 6, 4, 2, 16, 40, (3, 33))
    a = oracle_mod.verify_attention(q, k, v, kv_len, span)
    b = oracle_mod.verify_attention(q, k, v, kv_len, span, branch_len=6)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()


def test_select_branch(oracle_mod):
    a = np.array([[3, 7], [5, 5], [0, 0], [10, 2]], dtype=np.int32)
    bb, bl = oracle_mod.select_branch(a)
    assert bb.tolist() == [1, 0, 0, 0] and bl.tolist() == [7, 5, 0, 10]      # ties keep the first branch
    rng = np.random.default_rng(3)
    a = rng.integers(0, 11, (500, 4)).astype(np.int32)
    bb, bl = oracle_mod.select_branch(a)
    assert (bb == np.argmax(a, axis=1)).all() and (bl == a.max(axis=1)).all()
