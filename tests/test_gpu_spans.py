"""GPU parity of lvspec_verify_attention_spans: the visual mass over several spans.
The oracle's mass is additive over disjoint spans (one of its pins), so the reference
is the sum of its single-span masses; `out` does not depend on the spans at all."""
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


def _case(seed, B, gamma, Hq, Hkv, D, Lmax, kv_len):
    rng = np.random.default_rng(seed)
    bits = lambda shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    return bits((B, gamma, Hq, D)), bits((B, Hkv, Lmax, D)), bits((B, Hkv, Lmax, D)), np.asarray(kv_len, np.int32)


def frames(start, n_frames, frame_len, gap_len):
    """[start, end) of n_frames spans of frame_len positions with gap_len positions between."""
    out, pos = [], start
    for _ in range(n_frames):
        out.append([pos, pos + frame_len])
        pos += frame_len + gap_len
    return out


def oracle_union_mass(oracle_mod, q, k, v, kv_len, spans):
    """Sum over the span slots of the oracle's single-span mass (empty slots add nothing)."""
    spans = np.asarray(spans, dtype=np.int32)
    ref_out, total = None, 0.0
    for i in range(spans.shape[1]):
        o, m = oracle_mod.verify_attention(q, k, v, kv_len, spans[:, i, :])
        ref_out, total = o, total + m
    return ref_out, total


def run_spans(ctx, q, k, v, kv_len, spans, n_split=0, kernel=0):
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import dev_bf16, bf16_to_f64
    B, gamma, Hq, D = q.shape
    Hkv, Lmax = k.shape[1], k.shape[2]
    out = torch.full((B, gamma, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    mass = torch.full((B, gamma, Hq), float("nan"), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(B, gamma, Hq, Hkv, D, Lmax, n_split, kernel)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention_spans(shape, dev_bf16(q), dev_bf16(k), dev_bf16(v), kv_len, spans, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return bf16_to_f64(out), mass.cpu().numpy().astype(np.float64)


CASES = [
    # seed, B, gamma, Hq, Hkv, D, Lmax, kv_len, spans [B][S][2], n_split, kernel
    (51, 1, 4, 8, 2, 128, 2048, [2000], [frames(40, 9, 196, 3)], 0, 0),
    (52, 2, 8, 10, 2, 128, 3072, [3072, 1500],
     [frames(100, 10, 196, 5) + [[0, 0]], frames(0, 5, 100, 70) + [[1000, 1000]] * 6], 3, 0),
    (53, 1, 5, 12, 4, 128, 1024, [1000], [[[10, 300], [300, 500], [640, 900]]], 0, 1),      # adjacent spans, one long gap
    (54, 2, 4, 8, 2, 64, 1024, [1024, 600], [frames(5, 4, 150, 40), frames(0, 4, 100, 33)], 0, 0),   # head_dim 64
    (55, 1, 8, 40, 8, 128, 4096, [4096], [frames(256, 18, 196, 4)], 0, 0),
    # 80 (sequence, head) units: the automatic choice would be one split per unit
    (56, 40, 4, 8, 2, 128, 512, [512, 400, 300, 200] * 10, [frames(0, 2, 60, 10)] * 40, 0, 2),
]


@pytest.mark.parametrize("case", CASES, ids=[f"seed{c[0]}" for c in CASES])
def test_union_of_spans(ctx, oracle_mod, case):
    from gpu_util import assert_attention_close
    seed, B, gamma, Hq, Hkv, D, Lmax, kv_len, spans, n_split, kernel = case
    q, k, v, kv_len = _case(seed, B, gamma, Hq, Hkv, D, Lmax, kv_len)
    ref_out, ref_mass = oracle_union_mass(oracle_mod, q, k, v, kv_len, spans)
    out, mass = run_spans(ctx, q, k, v, kv_len, spans, n_split, kernel)
    assert_attention_close(out, mass, ref_out, ref_mass)


def test_one_span_is_the_base_call(ctx, oracle_mod):
    """A single span (padded with empty ones): the same bits as lvspec_verify_attention."""
    from gpu_util import run_attention
    q, k, v, kv_len = _case(57, 1, 8, 10, 2, 128, 3000, [2950])
    out, mass = run_spans(ctx, q, k, v, kv_len, [[[300, 2500], [2500, 2500], [0, 0]]], n_split=5)
    o2, m2 = run_attention(ctx, q, k, v, kv_len, np.asarray([[300, 2500]], np.int32), n_split=5)
    assert (out == o2).all() and (mass == m2).all()


def test_invalid_spans_launch_nothing(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    q = torch.zeros(1, 4, 8, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 2, 1024, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    mass = torch.zeros(1, 4, 8, device="cuda")
    shape = binding.attn_shape(1, 4, 8, 2, 128, 1024, 0, 0)
    before = ctx.launch_count()
    for spans in ([[[100, 200], [150, 300]]],          # overlap
                  [[[300, 400], [100, 200]]],          # not sorted
                  [[[0, 1021]]],                       # reaches into the draft slots
                  [[[-1, 5]]]):
        with pytest.raises(binding.LvspecError) as e:
            ctx.verify_attention_spans(shape, q, kv, kv, [1024], spans, out, mass)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.LvspecError) as e:       # one split forced on the tensor-core kernel
        ctx.verify_attention_spans(binding.attn_shape(1, 4, 8, 2, 128, 1024, 1, 2), q, kv, kv, [1024],
                                   [[[0, 10], [20, 30]]], out, mass)
    assert e.value.status == binding.ERR_UNSUPPORTED
    assert ctx.launch_count() == before
