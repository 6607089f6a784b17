"""The tensor-core attention kernel has two organisations of its softmax stage: all
warp groups on every tile, each on a share of the columns, and the groups taking the
tiles in turn (chosen by the library from the stream length per CTA and the cache
format; LVSPEC_TC_TURNS=0/1, read at every launch, forces one).  Both must pass the same
parity bar, above all where the reference exponents move while other groups are at work
on later tiles: scores that climb along the cache, tile after tile."""
import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

import test_gpu_attention as A
import test_gpu_fp8 as F8
import test_gpu_paged as PG
import test_gpu_tree as TR

pytestmark = pytest.mark.gpu

if 2 not in A.KERNELS:  # pragma: no cover
    pytest.skip("needs the tcgen05 kernel", allow_module_level=True)


@pytest.fixture(scope="module")
def ctx():
    from paper_2604_05650_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


@pytest.fixture(params=["0", "1"], ids=["shared-columns", "tiles-in-turn"])
def organisation(request, monkeypatch):
    monkeypatch.setenv("LVSPEC_TC_TURNS", request.param)
    return request.param


@pytest.mark.parametrize("shape", [
    # B, gamma, Hq, Hkv, Lmax, kv_len, span, n_split
    (1, 8, 40, 8, 4096, [4096], [[256, 3000]], 0),
    (1, 8, 40, 8, 4096, [4000], [[256, 3000]], 1),          # 32 tiles in one CTA
    (2, 10, 16, 2, 3072, [3072, 1111], [[100, 2500], [0, 1000]], 2),
    (1, 16, 40, 8, 1536, [1500], [[64, 1400]], 3),          # 80 rows
    (1, 16, 16, 2, 900, [897], [[0, 881]], 1),              # 128 rows: two S^T buffers, one P^T buffer
    (3, 4, 8, 2, 640, [640, 130, 385], [[10, 600], [0, 126], [5, 381]], 4),   # splits without tiles
])
def test_shapes(ctx, oracle_mod, organisation, shape):
    B, gamma, Hq, Hkv, Lmax, kv_len, span, n_split = shape
    A._check(ctx, oracle_mod, A._case(31, B, gamma, Hq, Hkv, 128, Lmax, kv_len, span), n_split=n_split, kernel=2)


@pytest.mark.parametrize("shape", [
    (1, 4, 8, 2, 1024, [1024], [[64, 832]], 0),             # the tiny config's shape
    (2, 8, 16, 4, 2048, [2000, 300], [[100, 1500], [0, 290]], 1),
])
def test_head_dim_64(ctx, oracle_mod, organisation, shape):
    B, gamma, Hq, Hkv, Lmax, kv_len, span, n_split = shape
    A._check(ctx, oracle_mod, A._case(36, B, gamma, Hq, Hkv, 64, Lmax, kv_len, span), n_split=n_split, kernel=2)


@pytest.mark.parametrize("n_split", [1, 3])
def test_scores_climbing_tile_after_tile(ctx, oracle_mod, organisation, n_split):
    """The score of every row grows by about 80 binades per 128-position tile (more than
    the guard of 60), so every tile moves the reference exponents, while the groups that
    hold the next tiles have already read the old ones; twice the climb pauses for a few
    tiles and once a single late position spikes."""
    B, gamma, Hq, Hkv, D, L = 1, 4, 8, 2, 128, 4096
    q, k, v, kv_len, span = A._case(32, B, gamma, Hq, Hkv, D, L, [L - 5], [[100, 3500]])
    q[:] = W.f32_to_bf16_bits(np.full(q.shape, 1.0, dtype=np.float32))
    kf = W.bf16_bits_to_f32(k) * 0.25
    tile = np.arange(L) // 128
    climb = np.where(tile < 10, tile, np.where(tile < 14, 10, np.where(tile < 24, tile - 4, 20))).astype(np.float32)
    kf += (climb * 4.875)[None, None, :, None]     # q = 1: + 4.875 * sqrt(128) * log2(e) = 79.6 binades per tile
    kf[0, 1, 4000] += 8.0                          # one late spike
    A._check(ctx, oracle_mod, (q, W.f32_to_bf16_bits(kf), v, kv_len, span), n_split=n_split, kernel=2)


def test_junk_beyond_kv_len(ctx, oracle_mod, organisation):
    case = list(A._case(33, 2, 4, 8, 2, 128, 1024, [900, 385], [[10, 800], [0, 381]]))
    for t in (1, 2):
        case[t][0, :, 900:] = 0x7FC0            # NaN
        case[t][1, :, 385:] = 0x7F80            # +Inf
    A._check(ctx, oracle_mod, tuple(case), n_split=1, kernel=2)


def test_reproducible_and_split_invariant(ctx, oracle_mod, organisation):
    case = A._case(34, 1, 8, 16, 2, 128, 3000, [2990], [[40, 2500]])
    a = A._check(ctx, oracle_mod, case, n_split=1, kernel=2)
    b = A._check(ctx, oracle_mod, case, n_split=1, kernel=2)
    c = A._check(ctx, oracle_mod, case, n_split=5, kernel=2)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()
    assert np.abs(a[0] - c[0]).max() <= 1e-2 and np.abs(a[1] - c[1]).max() <= 2e-4


@pytest.mark.parametrize("shape", [
    (1, 2, 10, 10, 2, 128, [3000], [[300, 2500]], 1),        # two branches of ten, one CTA per head
    (2, 2, 4, 8, 2, 128, [700, 391], [[10, 500], [0, 380]], 3),
])
def test_tree(ctx, oracle_mod, organisation, shape):
    TR.test_tree_attention(ctx, oracle_mod, shape, 2)


@pytest.mark.parametrize("case", [PG.CASES[1], PG.CASES[3]], ids=["ragged", "one-cta-per-head"])
def test_paged(ctx, oracle_mod, organisation, case):
    PG.test_paged_matches_oracle_and_contiguous(ctx, oracle_mod, case)


@pytest.mark.parametrize("rows", [40, 80])
def test_fp8_cache(ctx, oracle_mod, organisation, rows):
    gamma = rows // 5
    F8._check(ctx, oracle_mod, F8._case(35, 1, gamma, 10, 2, 2304, [2300], [[128, 2000]]), n_split=2)


def test_fp8_scores_climbing(ctx, oracle_mod, organisation):
    F8.test_scores_climbing_far_above_the_first_tile(ctx, oracle_mod, 1)


def test_random_shapes_with_moving_references(ctx, oracle_mod, organisation):
    """Seeded random shapes, split counts and lengths; the keys are scaled up so that scores
    spread over a hundred binades and the reference exponents move at unpredictable tiles.
    A few positions then carry a row's whole mass, where nothing averages the rounding of
    the probabilities to bf16 (2^-9 relative each) away: the visual mass, a ratio of two sums
    of the same rounded probabilities, is held to that bound here, not to the 1e-3 of the
    workload configs."""
    from gpu_util import run_attention
    rng = np.random.default_rng(2604)
    for case_id in range(24):
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 5, 8]))
        gamma = int(rng.integers(1, min(16, 128 // G) + 1))
        D = int(rng.choice([64, 128, 128]))
        B = int(rng.choice([1, 1, 2, 3]))
        Lmax = int(rng.integers(3, 40)) * 128 + int(rng.integers(0, 128))
        kv_len = [int(rng.integers(max(gamma, 130), Lmax + 1)) for _ in range(B)]
        span = []
        for L in kv_len:
            a = int(rng.integers(0, L - gamma + 1))
            span.append([a, int(rng.integers(a, L - gamma + 1))])
        n_split = int(rng.choice([0, 1, 1, 2, 3, 7]))
        q, k, v, kl, sp = A._case(1000 + case_id, B, gamma, G * Hkv, Hkv, D, Lmax, kv_len, span)
        gain = float(rng.choice([1.0, 3.0, 8.0]))
        k = W.f32_to_bf16_bits(W.bf16_bits_to_f32(k) * gain)
        ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kl, sp)
        out, mass = run_attention(ctx, q, k, v, kl, sp, n_split=n_split, kernel=2)
        assert np.isfinite(out).all() and np.isfinite(mass).all(), case_id
        assert (np.abs(out - ref_out) <= 1e-2 + 1e-2 * np.abs(ref_out)).all(), case_id
        assert np.abs(mass - ref_mass).max() <= 2.0 ** -9, (case_id, np.abs(mass - ref_mass).max())


@pytest.mark.parametrize("ring", ["2,2,1,2", "2,2,2,2", "3,2,2,3", "1,1,1,2", "2,3,3,3"])
def test_turns_with_fewer_buffers(ctx, oracle_mod, monkeypatch, ring):
    """LVSPEC_TC_RING="K slots,V slots,P buffers,S buffers" (read at every launch) forces the
    buffer counts that large row counts make the library fall back to: groups that share
    P^T and S^T buffers wait for tiles other groups hold, and the hand-over barriers, indexed
    by tile, must still tell every phase apart.  One CTA streams 32 tiles, with moving
    reference exponents in the second case."""
    monkeypatch.setenv("LVSPEC_TC_TURNS", "1")
    monkeypatch.setenv("LVSPEC_TC_RING", ring)
    A._check(ctx, oracle_mod, A._case(37, 1, 8, 40, 8, 128, 4096, [4001], [[256, 3000]]), n_split=1, kernel=2)
    q, k, v, kv_len, span = A._case(38, 2, 4, 8, 2, 128, 2304, [2304, 700], [[100, 2000], [0, 650]])
    k = W.f32_to_bf16_bits(W.bf16_bits_to_f32(k) * 6.0)
    from gpu_util import run_attention
    ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    out, mass = run_attention(ctx, q, k, v, kv_len, span, n_split=2, kernel=2)
    assert (np.abs(out - ref_out) <= 1e-2 + 1e-2 * np.abs(ref_out)).all()
    assert np.abs(mass - ref_mass).max() <= 2.0 ** -9
