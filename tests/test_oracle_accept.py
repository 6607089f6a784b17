"""Pins of the acceptance oracle: hand-worked cases, exhaustive enumeration
against an independent set/sort formulation, library special cases and the
closed forms the paper proves."""
import itertools
import json
import math
import os

import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _logits_from_targets(target, V=16):
    """Rows whose largest entry sits at the wanted token id."""
    target = np.asarray(target)
    lg = np.zeros(target.shape + (V,), dtype=np.float32)
    idx = np.indices(target.shape)
    lg[(*idx, target)] = 5.0
    return lg


def _cases():
    with open(os.path.join(GOLD, "rule_cases.txt")) as f:
        return [json.loads(l) for l in f if l.strip() and not l.startswith("#")]


@pytest.mark.parametrize("case", _cases())
def test_hand_worked_cases(oracle_mod, case):
    draft = np.asarray([case["draft"]], dtype=np.int32)
    mass = np.asarray([case["mass"]], dtype=np.float32)
    tau, target, acc = oracle_mod.loose_accept(_logits_from_targets([case["target"]]), draft, mass,
                                               case["n_loose"], case["W"])
    assert target[0].tolist() == case["target"]
    assert acc[0].tolist() == case["acc"]
    assert int(tau[0]) == case["tau"]


def test_n_loose_table(oracle_mod):
    with open(os.path.join(GOLD, "n_loose.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) >= 10
    for lam, K, n in rows:
        assert oracle_mod.n_loose(float(lam), int(K)) == int(n), (lam, K)


def _independent_rule(draft, target, score, n_loose, W):
    """The rule restated with Python sets and sorted(): a position is accepted
    iff it matches, or is among the n' positions of lowest (score, index), or
    its target token is in the set of draft tokens within W positions; the
    length is the count of leading accepted positions."""
    g = len(draft)
    loosened = set(sorted(range(g), key=lambda i: (score[i], i))[:n_loose])
    acc = []
    for i in range(g):
        near = {draft[k] for k in range(g) if abs(k - i) <= W}
        acc.append(draft[i] == target[i] or i in loosened or target[i] in near)
    tau = len(list(itertools.takewhile(bool, acc)))
    return acc, tau


def test_exhaustive_small_gamma(oracle_mod):
    """gamma = 4, tokens from a 3-letter alphabet for draft and target, all
    score orders with ties, every n' and W: batched through the oracle."""
    g = 4
    toks = list(itertools.product(range(3), repeat=g))
    rng = np.random.default_rng(0)
    score_sets = [list(p) for p in itertools.permutations([0.1, 0.2, 0.3, 0.4])][::5]
    score_sets += [[0.2, 0.2, 0.1, 0.1], [0.5, 0.5, 0.5, 0.5], [0.3, 0.1, 0.3, 0.1]]
    pairs = [(d, t) for d in toks for t in toks]
    pairs = [pairs[i] for i in rng.choice(len(pairs), size=900, replace=False)]
    draft = np.asarray([p[0] for p in pairs], dtype=np.int32)
    target = np.asarray([p[1] for p in pairs])
    logits = _logits_from_targets(target, V=8)
    checked = 0
    for sc in score_sets:
        mass = np.tile(np.asarray(sc, dtype=np.float32)[None, :, None], (len(pairs), 1, 1))
        for n_loose in range(g + 1):
            for Wn in range(g + 1):
                tau, tgt, acc = oracle_mod.loose_accept(logits, draft, mass, n_loose, Wn)
                assert (tgt == target).all()
                for r in range(0, len(pairs), 7):
                    a, t = _independent_rule(list(pairs[r][0]), list(pairs[r][1]), sc, n_loose, Wn)
                    assert acc[r].tolist() == [int(x) for x in a]
                    assert int(tau[r]) == t
                    checked += 1
    assert checked > 10000


def test_strict_mode_is_longest_common_prefix(oracle_mod):
    """lambda -> 0 with PST off recovers exact-match verification (Sec. 3.2)."""
    rng = np.random.default_rng(1)
    B, g = 500, 10
    target = rng.integers(0, 4, (B, g))
    draft = rng.integers(0, 4, (B, g)).astype(np.int32)
    mass = rng.random((B, g, 3), dtype=np.float32)
    tau, _, acc = oracle_mod.loose_accept(_logits_from_targets(target), draft, mass, 0, 0)
    eq = (draft == target)
    assert (acc.astype(bool) == eq).all()
    assert (tau == np.cumprod(eq, axis=1).sum(1)).all()


def test_everything_loosened_accepts_all(oracle_mod):
    rng = np.random.default_rng(2)
    B, g = 50, 8
    target = rng.integers(0, 9, (B, g))
    draft = rng.integers(0, 9, (B, g)).astype(np.int32)
    mass = rng.random((B, g, 2), dtype=np.float32)
    tau, _, _ = oracle_mod.loose_accept(_logits_from_targets(target), draft, mass, g, 0)
    assert (tau == g).all()


def test_paper_pst_is_membership_in_the_whole_draft(oracle_mod):
    """Eq. 7: with the shift range set to the draft length, clause 3 is plain
    membership of the target token in the set of draft tokens."""
    rng = np.random.default_rng(3)
    B, g = 400, 10
    target = rng.integers(0, 12, (B, g))
    draft = rng.integers(0, 12, (B, g)).astype(np.int32)
    mass = rng.random((B, g, 1), dtype=np.float32)
    for Wn in (g - 1, g, g + 5):
        _, _, acc = oracle_mod.loose_accept(_logits_from_targets(target), draft, mass, 0, Wn)
        for b in range(B):
            s = set(draft[b].tolist())
            assert acc[b].tolist() == [int(t in s) for t in target[b]]


def test_monotone_in_n_loose_and_window(oracle_mod):
    rng = np.random.default_rng(4)
    B, g = 300, 8
    target = rng.integers(0, 6, (B, g))
    draft = rng.integers(0, 6, (B, g)).astype(np.int32)
    mass = rng.random((B, g, 4), dtype=np.float32)
    lg = _logits_from_targets(target)
    grid = np.asarray([[oracle_mod.loose_accept(lg, draft, mass, n, w)[0] for w in range(g + 1)]
                       for n in range(g + 1)])
    assert (np.diff(grid, axis=0) >= 0).all() and (np.diff(grid, axis=1) >= 0).all()
    assert (grid[-1] == g).all()


def test_loosened_set_is_the_lowest_scores(oracle_mod):
    """With all drafts wrong and PST off, the accepted positions are exactly the
    loosened set, which numpy's stable argsort gives independently."""
    rng = np.random.default_rng(5)
    B, g, H = 200, 10, 5
    target = np.zeros((B, g), dtype=np.int64)
    draft = np.ones((B, g), dtype=np.int32)
    mass = (rng.integers(0, 4, (B, g, H)) * 0.25).astype(np.float32)   # many exact ties
    for n in (0, 3, 7, 10):
        _, _, acc = oracle_mod.loose_accept(_logits_from_targets(target), draft, mass, n, 0)
        order = np.argsort(mass.astype(np.float64).sum(-1), axis=1, kind="stable")
        want = np.zeros((B, g), dtype=np.uint8)
        np.put_along_axis(want, order[:, :n], 1, axis=1)
        assert (acc == want).all()


def test_argmax_matches_numpy_and_breaks_ties_low(oracle_mod):
    rng = np.random.default_rng(6)
    B, g, V = 3, 5, 1000
    lg = rng.integers(-3, 4, (B, g, V)).astype(np.float32)          # heavy ties
    draft = np.zeros((B, g), dtype=np.int32)
    mass = np.zeros((B, g, 1), dtype=np.float32)
    _, tgt, _ = oracle_mod.loose_accept(lg, draft, mass, 0, 0)
    assert (tgt == np.argmax(lg, axis=-1)).all()
    lg2 = rng.standard_normal((B, g, V)).astype(np.float32)
    lg2[0, 0, :] = -np.inf                                          # nothing above -inf -> 0
    lg2[0, 1, 7] = np.nan                                           # NaN never wins
    lg2[0, 1, 9] = 50.0
    lg2[0, 2, :] = np.nan
    lg2[1, 0, V - 1] = 60.0
    lg2[1, 1, 0] = 60.0
    lg2[1, 2, 3] = np.inf
    lg2[1, 2, 5] = np.inf
    _, tgt2, _ = oracle_mod.loose_accept(lg2, draft, mass, 0, 0)
    assert tgt2[0, 0] == 0 and tgt2[0, 1] == 9 and tgt2[0, 2] == 0
    assert tgt2[1, 0] == V - 1 and tgt2[1, 1] == 0 and tgt2[1, 2] == 3
    finite = np.where(np.isnan(lg2), -np.inf, lg2)
    assert (tgt2 == np.argmax(finite, axis=-1)).all()


def test_strict_expectation_matches_prop_2_2(oracle_mod):
    """i.i.d. matches with accuracy alpha: E[tau_strict] = sum_k alpha^k
    = alpha (1 - alpha^K) / (1 - alpha)  (Prop. 2.2 and its proof)."""
    rng = np.random.default_rng(7)
    B, K = 200000, 10
    for alpha in (0.341, 0.7):
        match = rng.random((B, K)) < alpha
        target = np.zeros((B, K), dtype=np.int64)
        draft = np.where(match, 0, 1).astype(np.int32)
        mass = np.zeros((B, K, 1), dtype=np.float32)
        tau, _, _ = oracle_mod.loose_accept(_logits_from_targets(target, V=4), draft, mass, 0, 0)
        closed = alpha * (1 - alpha ** K) / (1 - alpha)
        assert abs(closed - sum(alpha ** k for k in range(1, K + 1))) < 1e-12
        sigma = tau.std() / math.sqrt(B)
        assert abs(tau.mean() - closed) < 4 * sigma + 1e-9


def test_loose_expectation_matches_hypergeometric_form(oracle_mod):
    """Scores independent of matches, PST off: the first k positions hold m
    loosened ones with hypergeometric probability, the other k-m must match:
    P(tau >= k) = sum_m C(k,m) C(K-k,n'-m) / C(K,n') alpha^(k-m).  The loosened
    share turns the failure rate eps into about rho*eps (Thm. 2.3's dilution)."""
    rng = np.random.default_rng(8)
    B, K, n, alpha = 200000, 10, 7, 0.341
    match = rng.random((B, K)) < alpha
    target = np.zeros((B, K), dtype=np.int64)
    draft = np.where(match, 0, 1).astype(np.int32)
    mass = rng.random((B, K, 1), dtype=np.float32)
    tau, _, _ = oracle_mod.loose_accept(_logits_from_targets(target, V=4), draft, mass, n, 0)
    expect = 0.0
    for k in range(1, K + 1):
        expect += sum(math.comb(k, m) * math.comb(K - k, n - m) / math.comb(K, n) * alpha ** (k - m)
                      for m in range(0, min(k, n) + 1) if n - m <= K - k)
    sigma = tau.std() / math.sqrt(B)
    assert abs(tau.mean() - expect) < 4 * sigma
    strict = alpha * (1 - alpha ** K) / (1 - alpha)
    assert tau.mean() > 2 * strict          # loosening 7 of 10 more than doubles the length


def test_config0_workload_statistics(oracle_mod):
    cfg = W.CONFIGS[0]
    lg, draft = W.accept_inputs(cfg)
    mass = W.synthetic_mass(cfg)
    tau, tgt, acc = oracle_mod.loose_accept(lg, draft, mass, oracle_mod.n_loose(cfg.lam, cfg.gamma),
                                            cfg.shift_window)
    assert (tgt == np.argmax(lg, -1)).all() and 0 <= tau[0] <= cfg.gamma
