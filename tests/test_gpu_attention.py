"""GPU parity of lvspec_verify_attention against the fp64 oracle, through the
C ABI, element by element on the same seeded bytes."""
import dataclasses

import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

pytestmark = pytest.mark.gpu

KERNELS = [1]   # LVSPEC_KERNEL_SIMT; the tensor-core kernel is added to this list below
try:
    from paper_2604_05650_b200 import binding as _b
    if getattr(_b, "HAVE_TCGEN05", False):
        KERNELS.append(2)
except Exception:  # pragma: no cover
    pass


@pytest.fixture(scope="module")
def ctx():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05650_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _case(seed, B, gamma, Hq, Hkv, D, Lmax, kv_len, span):
    rng = np.random.default_rng(seed)
    bits = lambda shape, s=1.0: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * s)
    return (bits((B, gamma, Hq, D)), bits((B, Hkv, Lmax, D)), bits((B, Hkv, Lmax, D)),
            np.asarray(kv_len, dtype=np.int32), np.asarray(span, dtype=np.int32))


def _skip_unless_covered(kernel, case):
    q, k = case[0], case[1]
    if kernel == 2 and k.shape[2] < 128:
        pytest.skip("the tcgen05 kernel needs kv_capacity >= 128")


def _check(ctx, oracle_mod, case, n_split=0, kernel=1):
    from gpu_util import run_attention, assert_attention_close
    _skip_unless_covered(kernel, case)
    q, k, v, kv_len, span = case
    ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    out, mass = run_attention(ctx, q, k, v, kv_len, span, n_split=n_split, kernel=kernel)
    assert_attention_close(out, mass, ref_out, ref_mass)
    return out, mass


@pytest.mark.parametrize("kernel", KERNELS)
def test_config0(ctx, oracle_mod, kernel):
    _check(ctx, oracle_mod, W.attention_inputs(W.CONFIGS[0]), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("shape", [
    # B, gamma, Hq, Hkv, D, Lmax, kv_len, span, n_split
    (1, 4, 8, 2, 64, 1000, [1000], [[64, 832]], 3),            # ragged last tile
    (2, 8, 8, 2, 128, 700, [700, 389], [[10, 500], [0, 381]], 0),   # ragged batch, full span
    (3, 3, 6, 3, 128, 520, [33, 520, 3], [[5, 20], [100, 101], [0, 0]], 4),  # kv_len == gamma
    (1, 10, 16, 2, 128, 2100, [2077], [[512, 1900]], 5),       # M = 80 rows
    (1, 16, 5, 1, 128, 777, [777], [[0, 761]], 7),             # M = 80, gamma 16
    (1, 1, 4, 4, 64, 300, [257], [[3, 200]], 2),               # gamma 1, G 1
    (2, 4, 28, 4, 128, 600, [600, 599], [[256, 500], [1, 2]], 0),   # G = 7 (M = 28)
    (1, 8, 16, 1, 64, 130, [130], [[20, 100]], 64),            # more splits than tiles
    (1, 16, 16, 2, 128, 1500, [1500], [[100, 1200]], 4),       # M = 128: the most rows a KV head takes
    (1, 64, 4, 2, 128, 900, [900], [[0, 700]], 1),             # gamma 64 (the most), one split
    (2, 5, 10, 2, 128, 640, [640, 517], [[7, 300], [0, 512]], 3),   # M = 25: last chunk of 8 columns not full
    (1, 13, 26, 2, 128, 1300, [1290], [[200, 1000]], 0),       # M = 169 > 128 rows: refused
])
def test_small_shapes(ctx, oracle_mod, shape, kernel):
    B, gamma, Hq, Hkv, D, Lmax, kv_len, span, n_split = shape
    if gamma * (Hq // Hkv) > 128:
        from paper_2604_05650_b200 import binding
        with pytest.raises(binding.LvspecError) as e:
            _check(ctx, oracle_mod, _case(11, B, gamma, Hq, Hkv, D, Lmax, kv_len, span), kernel=kernel)
        assert e.value.status == binding.ERR_UNSUPPORTED
        return
    _check(ctx, oracle_mod, _case(11, B, gamma, Hq, Hkv, D, Lmax, kv_len, span),
           n_split=n_split, kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_split_count_invariance_and_reproducibility(ctx, oracle_mod, kernel):
    from gpu_util import run_attention
    case = _case(12, 1, 8, 10, 2, 128, 3000, [2950], [[300, 2500]])
    _skip_unless_covered(kernel, case)
    outs = [run_attention(ctx, *case, n_split=n, kernel=kernel) for n in (1, 2, 5, 23, 23)]
    for o, m in outs[1:]:
        assert np.abs(o - outs[0][0]).max() <= 1e-2 and np.abs(m - outs[0][1]).max() <= 2e-4
    assert (outs[3][0] == outs[4][0]).all() and (outs[3][1] == outs[4][1]).all()


@pytest.mark.parametrize("kernel", KERNELS)
def test_more_splits_than_one_combine_batch(ctx, oracle_mod, kernel):
    """The combine merges 32 splits per round trip: 45 splits take two rounds, the second
    with a moved reference exponent (the scores rise along the cache)."""
    case = _case(14, 1, 6, 8, 2, 128, 6016, [6000], [[100, 5000]])
    q, k, v, kv_len, span = case
    ramp = np.linspace(0.0, 3.0, k.shape[2], dtype=np.float32)[None, None, :, None]
    k = W.f32_to_bf16_bits(W.bf16_bits_to_f32(k) + ramp * np.sign(W.bf16_bits_to_f32(q).mean()))
    _check(ctx, oracle_mod, (q, k, v, kv_len, span), n_split=45, kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_peaked_scores(ctx, oracle_mod, kernel):
    """Scores with a wide dynamic range that rise along the cache, so the
    running maximum moves repeatedly and late keys dominate."""
    B, gamma, Hq, Hkv, D, L = 1, 4, 4, 2, 128, 1500
    q, k, v, kv_len, span = _case(13, B, gamma, Hq, Hkv, D, L, [L], [[100, 1200]])
    kf = W.bf16_bits_to_f32(k)
    qf = W.bf16_bits_to_f32(q)
    ramp = np.linspace(0.0, 6.0, L, dtype=np.float32)[None, None, :, None]
    kf = kf * 0.3 + ramp * np.sign(qf[:, 0, ::2, None, :]) * 0.25     # aligns with the queries
    _check(ctx, oracle_mod, (q, W.f32_to_bf16_bits(kf), v, kv_len, span), n_split=3, kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("n_split", [1, 2])
def test_scores_climbing_far_above_the_first_tile(ctx, oracle_mod, kernel, n_split):
    """Scores grow by more than 2^100 along the cache (in steps, and once by a
    single spike), so a running maximum fixed at the first tile would
    overflow: the accumulators have to be rescaled several times."""
    B, gamma, Hq, Hkv, D, L = 1, 4, 4, 2, 128, 2048
    q, k, v, kv_len, span = _case(15, B, gamma, Hq, Hkv, D, L, [L], [[100, 1700]])
    q[:] = W.f32_to_bf16_bits(np.full(q.shape, 1.0, dtype=np.float32))
    kf = W.bf16_bits_to_f32(k) * 0.25
    steps = (np.arange(L) // 300).astype(np.float32) * 1.5            # +17 per step in score
    kf += steps[None, None, :, None]
    kf[0, 0, 1999] += 4.0                                             # one late spike (+45)
    _check(ctx, oracle_mod, (q, W.f32_to_bf16_bits(kf), v, kv_len, span), n_split=n_split,
           kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_junk_beyond_kv_len_is_ignored(ctx, oracle_mod, kernel):
    """Cache slots past kv_len hold NaN / Inf bit patterns; nothing may leak."""
    case = list(_case(16, 2, 4, 8, 2, 128, 640, [500, 385], [[10, 400], [0, 381]]))
    for t in (1, 2):
        case[t][0, :, 500:] = 0x7FC0            # NaN
        case[t][1, :, 385:] = 0x7F80            # +Inf
    _check(ctx, oracle_mod, tuple(case), n_split=2, kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_identical_keys_closed_form(ctx, kernel):
    """Independent of the oracle: identical keys give the mean of the visible
    values and the visible visual fraction."""
    from gpu_util import run_attention
    q, k, v, kv_len, span = _case(14, 1, 4, 4, 2, 128, 900, [900], [[64, 700]])
    _skip_unless_covered(kernel, (q, k))
    k[:] = k[:, :, :1, :]
    out, mass = run_attention(ctx, q, k, v, kv_len, span, n_split=4, kernel=kernel)
    vf = W.bf16_bits_to_f32(v).astype(np.float64)
    for g in range(4):
        n = 900 - 4 + g + 1
        for h in range(4):
            assert np.abs(out[0, g, h] - vf[0, h // 2, :n].mean(0)).max() <= 1e-2
            assert abs(mass[0, g, h] - 636.0 / n) <= 1e-3


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("cfg_id", [1, 2, 3])
def test_full_size_layer(ctx, oracle_mod, cfg_id, kernel):
    """One whole layer of the Qwen2.5-VL-7B / -32B / LLaVA-OneVision-72B shaped
    configs, default launch configuration (the one the benchmark times), every
    output element against the oracle."""
    cfg = W.CONFIGS[cfg_id]
    _check(ctx, oracle_mod, W.attention_inputs(cfg, layer=cfg.layers - 1), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_sweep_point_batched(ctx, oracle_mod, kernel):
    cfg = W.sweep_config(gamma=16, kv_len=4096, batch=4, point=3)
    _check(ctx, oracle_mod, W.attention_inputs(cfg), kernel=kernel)


def test_host_buffer_entry_point(ctx, oracle_mod):
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import assert_attention_close
    cfg = W.CONFIGS[0]
    q, k, v, kv_len, span = W.attention_inputs(cfg)
    out = np.zeros(q.shape, dtype=np.uint16)
    mass = np.zeros(q.shape[:3], dtype=np.float32)
    shape = binding.attn_shape(1, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention_host(shape, q, k, v, kv_len, span, out, mass)
    ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    assert_attention_close(W.bf16_bits_to_f32(out).astype(np.float64), mass.astype(np.float64),
                           ref_out, ref_mass)


def test_invalid_arguments_launch_nothing(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    q = torch.zeros(1, 4, 8, 64, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 2, 256, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    mass = torch.zeros(1, 4, 8, device="cuda")
    good = dict(batch=1, gamma=4, n_q_heads=8, n_kv_heads=2, head_dim=64, kv_capacity=256)
    before = ctx.launch_count()

    def expect(status, kv_len=(256,), span=((0, 10),), **over):
        s = binding.attn_shape(**{**good, **over})
        with pytest.raises(binding.LvspecError) as e:
            ctx.verify_attention(s, q, kv, kv, kv_len, span, out, mass)
        assert e.value.status == status

    expect(binding.ERR_INVALID_ARG, n_q_heads=7)
    expect(binding.ERR_UNSUPPORTED, head_dim=96)
    expect(binding.ERR_UNSUPPORTED, gamma=64, n_q_heads=32, n_kv_heads=2)
    expect(binding.ERR_INVALID_ARG, batch=0)
    expect(binding.ERR_INVALID_ARG, kv_len=(257,))
    expect(binding.ERR_INVALID_ARG, kv_len=(3,))
    expect(binding.ERR_INVALID_ARG, span=((0, 253),))       # reaches into the draft tail
    expect(binding.ERR_INVALID_ARG, span=((11, 10),))
    expect(binding.ERR_INVALID_ARG, span=((-1, 10),))
    s = binding.attn_shape(**good)
    with pytest.raises(binding.LvspecError):
        ctx.verify_attention(s, None, kv, kv, (256,), ((0, 10),), out, mass)
    with pytest.raises(binding.LvspecError):
        ctx.verify_attention(s, q.data_ptr() + 2, kv, kv, (256,), ((0, 10),), out, mass)
    assert ctx.launch_count() == before


@pytest.mark.parametrize("kernel", KERNELS)
def test_sweep_point_single_split(ctx, oracle_mod, kernel):
    """Batch 16 x 8 KV heads fills the device with one split per head: the
    tensor-core kernel then normalises and writes the results itself."""
    cfg = W.sweep_config(gamma=4, kv_len=4096, batch=16, point=9)
    _check(ctx, oracle_mod, W.attention_inputs(cfg), kernel=kernel)


def test_plain_launches_give_the_same_results(oracle_mod, monkeypatch):
    """LVSPEC_NO_PDL=1 (read when the context is created) launches the attention
    kernels without programmatic dependence; results must not depend on it."""
    from paper_2604_05650_b200 import binding
    from gpu_util import run_attention
    case = _case(21, 2, 8, 10, 2, 128, 1500, [1500, 777], [[100, 1200], [0, 700]])
    outs = []
    for flag in ("1", "0"):
        monkeypatch.setenv("LVSPEC_NO_PDL", flag)
        c = binding.Context(0)
        try:
            # several calls back to back, so that launches do follow one another
            for _ in range(3):
                res = run_attention(c, *case, kernel=2)
            outs.append(res)
        finally:
            c.close()
    assert (outs[0][0] == outs[1][0]).all() and (outs[0][1] == outs[1][1]).all()
    ref_out, ref_mass = oracle_mod.verify_attention(*case)
    from gpu_util import assert_attention_close
    assert_attention_close(outs[0][0], outs[0][1], ref_out, ref_mass)

