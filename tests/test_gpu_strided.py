"""lvspec_verify_attention_strided: the cache in the caller's own layout (position-major,
K and V interleaved in one buffer, padded rows), both kernels, against the oracle on the
equivalent dense cache; and bit for bit the dense call's results."""
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


def _case(seed, B, gamma, Hq, Hkv, D, L, kv_len, span):
    rng = np.random.default_rng(seed)
    bits = lambda shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    return (bits((B, gamma, Hq, D)), bits((B, Hkv, L, D)), bits((B, Hkv, L, D)),
            np.asarray(kv_len, np.int32), np.asarray(span, np.int32))


def _run(ctx, q, kbuf, vbuf, k_strides, v_strides, dims, kv_len, span, kernel, n_split=0, v_offset=0):
    """kbuf / vbuf: torch device tensors holding the caches in their layout."""
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import dev_bf16, bf16_to_f64
    B, gamma, Hq, Hkv, D, L = dims
    out = torch.full((B, gamma, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    mass = torch.full((B, gamma, Hq), float("nan"), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(B, gamma, Hq, Hkv, D, L, n_split, kernel)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention_strided(shape, k_strides, v_strides, dev_bf16(q), kbuf.data_ptr(),
                                 vbuf.data_ptr() + 2 * v_offset, kv_len, span, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return bf16_to_f64(out), mass.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("layout", ["position_major", "interleaved", "padded_rows", "dense"])
def test_layouts(ctx, oracle_mod, layout, kernel):
    import torch
    from gpu_util import dev_bf16, run_attention, assert_attention_close
    B, gamma, Hq, Hkv, D, L = 2, 8, 10, 2, 128, 1400
    q, k, v, kv_len, span = _case(61, B, gamma, Hq, Hkv, D, L, [1400, 777], [[100, 1200], [0, 700]])
    dk, dv = dev_bf16(k), dev_bf16(v)                      # dense [B, Hkv, L, D]
    v_offset = 0
    if layout == "position_major":                         # [B, L, Hkv, D]
        kbuf, vbuf = dk.permute(0, 2, 1, 3).contiguous(), dv.permute(0, 2, 1, 3).contiguous()
        ks = vs = (L * Hkv * D, D, Hkv * D)
    elif layout == "interleaved":                          # one buffer [B, Hkv, L, 2, D]: K then V per position
        kbuf = torch.stack([dk, dv], dim=3).contiguous()
        vbuf, v_offset = kbuf, D
        ks = vs = (2 * Hkv * L * D, 2 * L * D, 2 * D)
    elif layout == "padded_rows":                          # rows of 136 elements, junk in the padding
        kbuf = torch.full((B, Hkv, L, D + 8), float("nan"), dtype=torch.bfloat16, device="cuda")
        vbuf = torch.full((B, Hkv, L, D + 8), float("nan"), dtype=torch.bfloat16, device="cuda")
        kbuf[..., :D], vbuf[..., :D] = dk, dv
        ks = vs = (Hkv * L * (D + 8), L * (D + 8), D + 8)
    else:
        kbuf, vbuf = dk, dv
        ks = vs = (Hkv * L * D, L * D, D)
    out, mass = _run(ctx, q, kbuf, vbuf, ks, vs, (B, gamma, Hq, Hkv, D, L), kv_len, span, kernel, n_split=3,
                     v_offset=v_offset)
    ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    assert_attention_close(out, mass, ref_out, ref_mass)
    dense_out, dense_mass = run_attention(ctx, q, k, v, kv_len, span, n_split=3, kernel=kernel)
    assert (out == dense_out).all() and (mass == dense_mass).all()


def test_bad_strides_are_refused(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    q = torch.zeros(1, 4, 8, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 2, 256, 128, dtype=torch.bfloat16, device="cuda")
    out, mass = torch.zeros_like(q), torch.zeros(1, 4, 8, device="cuda")
    s = binding.attn_shape(1, 4, 8, 2, 128, 256)
    good = (2 * 256 * 128, 256 * 128, 128)
    before = ctx.launch_count()
    for bad in [(good[0], good[1], 64), (good[0], good[1], 132), (good[0], 0, 128), (-8, good[1], 128)]:
        with pytest.raises(binding.LvspecError) as e:
            ctx.verify_attention_strided(s, bad, good, q, kv, kv, [256], [[0, 10]], out, mass)
        assert e.value.status == binding.ERR_INVALID_ARG
    assert ctx.launch_count() == before
