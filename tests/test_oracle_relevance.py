"""Pins of the oracle's visual-relevance score (Sec. 3.1, Eq. 4: mean of the
Top-N cosine similarities between a draft token's hidden state and the visual
tokens' hidden states) against things other than itself."""
import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W


def _bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _rand(seed, B, K, lv, d):
    rng = np.random.default_rng(seed)
    return (_bits(rng.standard_normal((B, K, d))), _bits(rng.standard_normal((B, lv, d))))


def test_matches_torch_cosine_similarity_and_topk(oracle_mod):
    """Library special case: torch's cosine_similarity and topk in fp64."""
    import torch
    hd, hv = _rand(0, 2, 5, 300, 96)
    rel, cos = oracle_mod.visual_relevance(hd, hv, 10, return_cosines=True)
    td = torch.from_numpy(W.bf16_bits_to_f32(hd).astype(np.float64))
    tv = torch.from_numpy(W.bf16_bits_to_f32(hv).astype(np.float64))
    tc = torch.nn.functional.cosine_similarity(td[:, :, None, :], tv[:, None, :, :], dim=-1)
    assert np.abs(cos - tc.numpy()).max() < 1e-12
    tr = torch.topk(tc, 10, dim=-1).values.mean(-1)
    assert np.abs(rel - tr.numpy()).max() < 1e-12


def test_numpy_brute_force(oracle_mod):
    hd, hv = _rand(1, 1, 3, 40, 16)
    rel = oracle_mod.visual_relevance(hd, hv, 4)
    fd = W.bf16_bits_to_f32(hd).astype(np.float64)[0]
    fv = W.bf16_bits_to_f32(hv).astype(np.float64)[0]
    for k in range(3):
        c = [float(fd[k] @ fv[j]) / (np.linalg.norm(fd[k]) * np.linalg.norm(fv[j])) for j in range(40)]
        assert abs(rel[0, k] - np.mean(sorted(c)[-4:])) < 1e-12


def test_special_values_of_n(oracle_mod):
    """N = 1 is the largest cosine, N = lv (or more) the plain mean."""
    hd, hv = _rand(2, 1, 4, 50, 32)
    _, cos = oracle_mod.visual_relevance(hd, hv, 1, return_cosines=True)
    assert np.abs(oracle_mod.visual_relevance(hd, hv, 1) - cos.max(-1)).max() < 1e-15
    assert np.abs(oracle_mod.visual_relevance(hd, hv, 50) - cos.mean(-1)).max() < 1e-14
    assert np.abs(oracle_mod.visual_relevance(hd, hv, 500) - cos.mean(-1)).max() < 1e-14
    # more of the top values can only lower the mean
    r = [oracle_mod.visual_relevance(hd, hv, n) for n in (1, 2, 5, 10, 50)]
    for a, b in zip(r, r[1:]):
        assert (a >= b - 1e-15).all()


def test_closed_forms(oracle_mod):
    d, lv = 64, 20
    rng = np.random.default_rng(3)
    v = rng.standard_normal((1, lv, d)).astype(np.float32)
    hv = _bits(v)
    fv = W.bf16_bits_to_f32(hv)
    # a draft row equal to visual row 7: its best cosine is exactly 1; the negated row: -1 is its worst
    hd = np.stack([hv[0, 7], _bits(-fv[0, 7]), _bits(3.5 * fv[0, 7])])[None]
    rel, cos = oracle_mod.visual_relevance(hd, hv, 1, return_cosines=True)
    assert abs(rel[0, 0] - 1.0) < 1e-12 and abs(cos[0, 1, 7] + 1.0) < 1e-12
    assert np.abs(cos[0, 0] + cos[0, 1]).max() < 1e-12            # odd in the draft vector
    assert np.abs(cos[0, 2] - cos[0, 0]).max() < 2e-3             # scale-free (up to bf16 rounding of 3.5 x)
    # orthogonal axes: cosine 0 everywhere but on the own axis
    e = np.eye(8, dtype=np.float32)
    rel, cos = oracle_mod.visual_relevance(_bits(e[None, :3]), _bits(2.0 * e[None]), 2, return_cosines=True)
    assert np.abs(cos[0] - e[:3]).max() == 0.0 and np.abs(rel - 0.5).max() == 0.0
    # every |cosine| <= 1
    hd, hv = _rand(4, 2, 6, 100, 48)
    _, cos = oracle_mod.visual_relevance(hd, hv, 3, return_cosines=True)
    assert np.abs(cos).max() <= 1.0 + 1e-12


def test_zero_vectors_score_zero(oracle_mod):
    hd, hv = _rand(5, 1, 2, 10, 16)
    hd[0, 1] = 0
    hv[0, 3] = 0
    rel, cos = oracle_mod.visual_relevance(hd, hv, 10, return_cosines=True)
    assert (cos[0, 1] == 0).all() and (cos[0, :, 3] == 0).all() and np.isfinite(rel).all()


def test_planted_rows_rank_as_visual_relevant(oracle_mod):
    """The synthetic recipe pulls even draft positions towards a few visual rows:
    with the paper's N = 10 they score higher than the unrelated odd positions."""
    import dataclasses
    cfg = dataclasses.replace(W.CONFIGS[0], gamma=8)
    hd, hv = W.relevance_inputs(cfg, n_visual=600, dim=256)
    rel = oracle_mod.visual_relevance(hd, hv, 10)
    assert rel[0, 0::2].min() > rel[0, 1::2].max()
