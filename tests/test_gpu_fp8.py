"""GPU parity of lvspec_verify_attention_fp8 (E4M3 cache with per-head scales) against
the fp64 oracle on the same codes and scales, through the C ABI, element by element, at
the tolerances of the bf16 call: |out - ref| <= 1e-2 + 1e-2 |ref|, visual mass 1e-3 abs."""
import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05650_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _quantize(q, k, v):
    k8, ks = W.quantize_cache_e4m3(k)
    v8, vs = W.quantize_cache_e4m3(v)
    return q, k8, v8, ks, vs


def _case(seed, B, gamma, Hq, Hkv, Lmax, kv_len, span, k_gain=1.0):
    rng = np.random.default_rng(seed)
    bits = lambda shape, s=1.0: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * s)
    q, k, v = bits((B, gamma, Hq, 128)), bits((B, Hkv, Lmax, 128), k_gain), bits((B, Hkv, Lmax, 128))
    return _quantize(q, k, v) + (np.asarray(kv_len, np.int32), np.asarray(span, np.int32))


def run_fp8(ctx, q, k8, v8, ks, vs, kv_len, span, n_split=0):
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import dev_bf16, bf16_to_f64
    B, gamma, Hq, D = q.shape
    Hkv, Lmax = k8.shape[1], k8.shape[2]
    dq = dev_bf16(q)
    dk, dv = torch.from_numpy(k8).cuda(), torch.from_numpy(v8).cuda()
    dks, dvs = torch.from_numpy(ks).cuda(), torch.from_numpy(vs).cuda()
    out = torch.full((B, gamma, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    mass = torch.full((B, gamma, Hq), float("nan"), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(B, gamma, Hq, Hkv, D, Lmax, n_split)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention_fp8(shape, dq, dk, dv, dks, dvs, kv_len, span, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return bf16_to_f64(out), mass.cpu().numpy().astype(np.float64)


def _check(ctx, oracle_mod, case, n_split=0):
    from gpu_util import assert_attention_close
    ref_out, ref_mass = oracle_mod.verify_attention_fp8(*case)
    out, mass = run_fp8(ctx, *case, n_split=n_split)
    assert_attention_close(out, mass, ref_out, ref_mass)
    return out, mass


@pytest.mark.parametrize("shape", [
    # B, gamma, Hq, Hkv, Lmax, kv_len, span, n_split
    (1, 8, 10, 2, 1500, [1500], [[100, 1200]], 3),
    (2, 8, 8, 2, 700, [700, 389], [[10, 500], [0, 381]], 0),          # ragged batch, ragged tiles
    (3, 3, 6, 3, 520, [33, 520, 3], [[5, 20], [100, 101], [0, 0]], 4),   # kv_len == gamma; splits without tiles
    (1, 10, 16, 2, 2100, [2077], [[512, 1900]], 5),                    # M = 80: the most rows of this call
    (1, 16, 5, 1, 777, [777], [[0, 761]], 7),                          # gamma 16, one KV head
    (2, 4, 28, 4, 600, [600, 599], [[256, 500], [1, 2]], 0),           # G = 7
    (2, 5, 10, 2, 640, [640, 517], [[7, 300], [0, 512]], 1),           # M = 25, one split: direct epilogue
    (1, 8, 40, 8, 4096, [4096], [[256, 3328]], 0),                     # the sweep's head shape
    (1, 4, 4, 4, 300, [257], [[31, 33]], 2),                           # span inside one 32-position block
])
def test_small_shapes(ctx, oracle_mod, shape):
    B, gamma, Hq, Hkv, Lmax, kv_len, span, n_split = shape
    _check(ctx, oracle_mod, _case(41, B, gamma, Hq, Hkv, Lmax, kv_len, span), n_split=n_split)


def test_full_size_layer_config2(ctx, oracle_mod):
    """One whole layer of the Qwen2.5-VL-32B shaped config with its cache quantised to
    E4M3, default launch configuration, every output element against the oracle."""
    cfg = W.CONFIGS[2]
    q, k, v, kv_len, span = W.attention_inputs(cfg, layer=cfg.layers - 1)
    _check(ctx, oracle_mod, _quantize(q, k, v) + (kv_len, span))


def test_full_size_layer_config3(ctx, oracle_mod):
    cfg = W.CONFIGS[3]
    q, k, v, kv_len, span = W.attention_inputs(cfg, layer=0)
    _check(ctx, oracle_mod, _quantize(q, k, v) + (kv_len, span))


def test_single_split_batch(ctx, oracle_mod):
    """Batch 16 x 8 KV heads: one split per head, the kernel normalises and writes itself."""
    cfg = W.sweep_config(gamma=4, kv_len=4096, batch=16, point=9)
    q, k, v, kv_len, span = W.attention_inputs(cfg)
    _check(ctx, oracle_mod, _quantize(q, k, v) + (kv_len, span))


@pytest.mark.parametrize("n_split", [1, 2])
def test_scores_climbing_far_above_the_first_tile(ctx, oracle_mod, n_split):
    """Scores grow by far more than E4M3's range along the cache (in steps, and once by a
    single spike): the reference exponent has to follow, and the accumulators with it."""
    B, gamma, Hq, Hkv, L = 1, 4, 4, 2, 2048
    rng = np.random.default_rng(15)
    q = W.f32_to_bf16_bits(np.full((B, gamma, Hq, 128), 1.0, dtype=np.float32))
    kf = rng.standard_normal((B, Hkv, L, 128)).astype(np.float32) * 0.25
    kf += ((np.arange(L) // 300).astype(np.float32) * 1.5)[None, None, :, None]      # +17 per step in score
    kf[0, 0, 1999] += 4.0                                                            # one late spike (+45)
    v = W.f32_to_bf16_bits(rng.standard_normal((B, Hkv, L, 128)).astype(np.float32))
    case = _quantize(q, W.f32_to_bf16_bits(kf), v) + (np.asarray([L], np.int32), np.asarray([[100, 1700]], np.int32))
    _check(ctx, oracle_mod, case, n_split=n_split)


def test_first_position_far_above_the_rest(ctx, oracle_mod):
    """An attention sink: the first position's score exceeds all others by about 2^30 in
    probability, and a second cluster sits 2^9 below the rest.  The reference exponent
    comes from the first tile's largest score, and what lies far below it is negligible
    in the exact result too."""
    B, gamma, Hq, Hkv, L = 1, 4, 4, 2, 1024
    rng = np.random.default_rng(16)
    q = W.f32_to_bf16_bits(np.full((B, gamma, Hq, 128), 0.5, dtype=np.float32))
    kf = rng.standard_normal((B, Hkv, L, 128)).astype(np.float32) * 0.1
    kf[:, :, 0, :] += 3.0                                     # score + 3 * 0.5 * 128 / sqrt(128) = +17
    kf[:, :, 512:, :] -= 1.0
    v = W.f32_to_bf16_bits(rng.standard_normal((B, Hkv, L, 128)).astype(np.float32))
    case = _quantize(q, W.f32_to_bf16_bits(kf), v) + (np.asarray([L], np.int32), np.asarray([[1, 900]], np.int32))
    _check(ctx, oracle_mod, case, n_split=1)
    _check(ctx, oracle_mod, case, n_split=3)


def test_large_and_small_q(ctx, oracle_mod):
    """q is rescaled by a power of two per CTA before it is split into E4M3 terms: rows of
    very different magnitude in one tile, and tiny / huge q overall."""
    for gain in (2.0 ** -20, 1.0, 300.0):
        q, k8, v8, ks, vs, kv_len, span = _case(43, 1, 8, 8, 2, 900, [900], [[64, 700]], k_gain=0.3)
        qf = W.bf16_bits_to_f32(q) * np.float32(gain)
        qf[0, 3] *= 0.01                                      # one query far smaller than the others
        case = (W.f32_to_bf16_bits(qf), k8, v8, (ks / np.float32(gain)).astype(np.float32), vs, kv_len, span)
        _check(ctx, oracle_mod, case, n_split=2)


def test_junk_beyond_kv_len_is_ignored(ctx, oracle_mod):
    """Cache slots past kv_len hold the NaN code and the largest values; nothing may leak."""
    case = list(_case(46, 2, 4, 8, 2, 640, [500, 385], [[10, 400], [0, 381]]))
    for t in (1, 2):
        case[t][0, :, 500:] = 0x7F            # NaN
        case[t][1, :, 385:] = 0xFE            # -448
    _check(ctx, oracle_mod, tuple(case), n_split=2)


def test_split_count_invariance_and_reproducibility(ctx, oracle_mod):
    case = _case(47, 1, 8, 10, 2, 3000, [2950], [[300, 2500]])
    outs = [run_fp8(ctx, *case, n_split=n) for n in (1, 2, 5, 23, 23)]
    for o, m in outs[1:]:
        assert np.abs(o - outs[0][0]).max() <= 1e-2 and np.abs(m - outs[0][1]).max() <= 2e-4
    assert (outs[3][0] == outs[4][0]).all() and (outs[3][1] == outs[4][1]).all()


def test_identical_keys_closed_form(ctx):
    """Independent of the oracle: identical keys give the mean of the visible values and
    the visible visual fraction."""
    q, k8, v8, ks, vs, kv_len, span = _case(48, 1, 4, 4, 2, 900, [900], [[64, 700]])
    k8[:] = k8[:, :, :1, :]
    out, mass = run_fp8(ctx, q, k8, v8, ks, vs, kv_len, span, n_split=4)
    import torch
    vf = torch.from_numpy(v8).view(torch.float8_e4m3fn).to(torch.float64).numpy() * vs[:, :, None, None].astype(np.float64)
    for g in range(4):
        n = 900 - 4 + g + 1
        for h in range(4):
            assert np.abs(out[0, g, h] - vf[0, h // 2, :n].mean(0)).max() <= 1e-2
            assert abs(mass[0, g, h] - 636.0 / n) <= 1e-3


def test_unsupported_shapes_are_refused(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    kv = torch.zeros(1, 2, 256, 128, dtype=torch.uint8, device="cuda")
    sc = torch.ones(1, 2, device="cuda")
    before = ctx.launch_count()

    def expect(status, gamma=4, Hq=8, D=128, kernel=0, k_scale=sc):
        q = torch.zeros(1, gamma, Hq, D, dtype=torch.bfloat16, device="cuda")
        out, mass = torch.zeros_like(q), torch.zeros(1, gamma, Hq, device="cuda")
        s = binding.attn_shape(1, gamma, Hq, 2, D, 256, 0, kernel)
        with pytest.raises(binding.LvspecError) as e:
            ctx.verify_attention_fp8(s, q, kv, kv, k_scale, sc, [256], [[0, 10]], out, mass)
        assert e.value.status == status

    expect(binding.ERR_UNSUPPORTED, gamma=11, Hq=16)          # 88 rows per KV head
    expect(binding.ERR_UNSUPPORTED, D=64)
    expect(binding.ERR_UNSUPPORTED, kernel=binding.KERNEL_SIMT)
    expect(binding.ERR_INVALID_ARG, k_scale=None)
    assert ctx.launch_count() == before
