"""Pins of the oracle's emit step (the tokens a verify step hands back).  The
paper fixes the accepted length only (Eq. 2); the pins are hand-worked cases and
the textbook property of speculative decoding the step must reduce to: under
strict exact-match verification the emitted tokens are exactly the tokens the
target itself generates, one per position, up to and including the first
disagreement."""
import numpy as np


def test_hand_worked_cases(oracle_mod):
    draft = np.array([[5, 7, 7, 9], [1, 2, 3, 4], [1, 2, 3, 4], [9, 9, 9, 9]], dtype=np.int32)
    target = np.array([[5, 8, 7, 7], [1, 2, 3, 4], [6, 2, 3, 4], [9, 9, 9, 1]], dtype=np.int32)
    tau = np.array([3, 4, 0, 3], dtype=np.int32)
    kv = np.array([100, 50, 20, 8], dtype=np.int32)
    em, n, new_kv = oracle_mod.emit(draft, target, tau, kv)
    # row 0: position 1 was loosened (draft 7 kept although the target says 8); rejected at 3 -> target's 7
    assert em.tolist() == [[5, 7, 7, 7], [1, 2, 3, 4], [6, -1, -1, -1], [9, 9, 9, 1]]
    assert n.tolist() == [4, 4, 1, 4]
    assert new_kv.tolist() == [99, 50, 16, 7]


def test_strict_verification_emits_the_targets_own_tokens(oracle_mod):
    rng = np.random.default_rng(0)
    B, g, V = 200, 6, 50
    target = rng.integers(0, 4, (B, g)).astype(np.int32)
    draft = np.where(rng.random((B, g)) < 0.7, target, rng.integers(0, 4, (B, g))).astype(np.int32)
    logits = np.zeros((B, g, V), dtype=np.float32)
    logits[np.arange(B)[:, None], np.arange(g)[None, :], target] = 5.0
    mass = np.zeros((B, g, 1), dtype=np.float32)
    tau, tgt, _ = oracle_mod.loose_accept(logits, draft, mass, 0, 0)      # lambda = 0, PST off
    em, n, _ = oracle_mod.emit(draft, tgt, tau)
    for b in range(B):
        assert n[b] == min(tau[b] + 1, g)
        assert (em[b, :n[b]] == target[b, :n[b]]).all()                   # textbook speculative decoding
        assert (em[b, n[b]:] == -1).all()


def test_loose_verification_keeps_the_accepted_draft_tokens(oracle_mod):
    rng = np.random.default_rng(1)
    B, g, V = 100, 8, 30
    logits = rng.standard_normal((B, g, V)).astype(np.float32)
    draft = rng.integers(0, V, (B, g)).astype(np.int32)
    mass = rng.random((B, g, 2)).astype(np.float32)
    tau, tgt, acc = oracle_mod.loose_accept(logits, draft, mass, 5, 8)
    em, n, _ = oracle_mod.emit(draft, tgt, tau)
    for b in range(B):
        t = tau[b]
        assert (em[b, :t] == draft[b, :t]).all()
        if t < g:
            assert em[b, t] == tgt[b, t] and n[b] == t + 1 and acc[b, t] == 0
        else:
            assert n[b] == g
