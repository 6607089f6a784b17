"""GPU parity of lvspec_row_inv_norms / lvspec_visual_relevance (the paper's
relevance score, Sec. 3.1, Eq. 4) against the fp64 oracle, through the C ABI.

Tolerance: inputs are bf16, every product is exact in fp32, and the tensor
core adds d of them in fp32; with |cos| <= 1 the accumulated rounding stays
below d * 2^-24 (3e-4 at d = 5120) in the worst case and is far smaller in
practice.  The score is compared at 5e-4 absolute."""
import dataclasses

import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

pytestmark = pytest.mark.gpu
TOL = 5e-4


@pytest.fixture(scope="module")
def ctx():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05650_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _run(ctx, hd, hv, top_n):
    import torch
    from gpu_util import dev_bf16
    B, K, d = hd.shape
    lv = hv.shape[1]
    dd, dv = dev_bf16(hd), dev_bf16(hv)
    inv = torch.full((B, lv), float("nan"), dtype=torch.float32, device="cuda")
    rel = torch.full((B, K), float("nan"), dtype=torch.float32, device="cuda")
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.row_inv_norms(B * lv, d, dv, inv)
    ctx.visual_relevance(B, K, lv, d, dd, dv, inv, top_n, rel)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return rel.cpu().numpy().astype(np.float64), inv.cpu().numpy().astype(np.float64)


def _rand(seed, B, K, lv, d):
    rng = np.random.default_rng(seed)
    return (W.f32_to_bf16_bits(rng.standard_normal((B, K, d)).astype(np.float32)),
            W.f32_to_bf16_bits(rng.standard_normal((B, lv, d)).astype(np.float32)))


@pytest.mark.parametrize("shape", [
    # B, K, lv, d, top_n
    (1, 4, 300, 256, 10),
    (2, 10, 1000, 512, 10),        # ragged: 1000 = 62 groups of 16 + 8 rows
    (3, 8, 777, 128, 5),           # chunks cross batch elements
    (1, 16, 2100, 64, 1),          # N = 1: the maximum; one stage per chunk
    (1, 17, 500, 192, 100),        # K padded to 32; N = 100
    (2, 1, 5, 64, 10),             # fewer visual tokens than N: plain mean
    (1, 64, 130, 128, 3),          # the widest draft tile
    (1, 10, 20000, 320, 10),       # more chunks than SMs
])
def test_small_shapes(ctx, oracle_mod, shape):
    B, K, lv, d, n = shape
    hd, hv = _rand(31, B, K, lv, d)
    ref = oracle_mod.visual_relevance(hd, hv, n)
    got, inv = _run(ctx, hd, hv, n)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= TOL, np.abs(got - ref).max()
    norms = np.linalg.norm(W.bf16_bits_to_f32(hv).astype(np.float64), axis=-1)
    assert np.abs(inv * norms - 1.0).max() <= 1e-5


def test_planted_structure_and_reproducibility(ctx, oracle_mod):
    cfg = dataclasses.replace(W.CONFIGS[0], gamma=8)
    hd, hv = W.relevance_inputs(cfg, n_visual=3000, dim=512)
    ref = oracle_mod.visual_relevance(hd, hv, 10)
    a, _ = _run(ctx, hd, hv, 10)
    b, _ = _run(ctx, hd, hv, 10)
    assert np.abs(a - ref).max() <= TOL
    assert (a == b).all()                                   # bitwise reproducible
    assert a[0, 0::2].min() > a[0, 1::2].max()              # planted rows rank as visual-relevant


def test_zero_rows_and_duplicates(ctx, oracle_mod):
    hd, hv = _rand(33, 1, 6, 400, 128)
    hd[0, 2] = 0                      # a zero draft row: cosine 0 with everything
    hv[0, 17] = 0                     # a zero visual row
    hv[0, 100:140] = hv[0, 99]        # 41 identical rows: ties inside the Top-N
    hd[0, 4] = hv[0, 99]              # ... with cosine exactly 1 for this draft row
    ref = oracle_mod.visual_relevance(hd, hv, 10)
    got, inv = _run(ctx, hd, hv, 10)
    assert np.abs(got - ref).max() <= TOL
    assert got[0, 2] == 0.0 and inv[0, 17] == 0.0
    assert abs(got[0, 4] - 1.0) <= TOL


@pytest.mark.parametrize("cfg_id", [2, 3])
def test_full_size(ctx, oracle_mod, cfg_id):
    """The visual span and hidden size of the Qwen2.5-VL-32B / LLaVA-OneVision-72B
    shaped configs (25088 x 5120 and 23328 x 8192), the paper's N = 10."""
    cfg = W.CONFIGS[cfg_id]
    hd, hv = W.relevance_inputs(cfg)
    ref = oracle_mod.visual_relevance(hd, hv, 10)
    got, _ = _run(ctx, hd, hv, 10)
    assert np.abs(got - ref).max() <= TOL, np.abs(got - ref).max()


def test_score_feeds_the_acceptance_rule(ctx, oracle_mod):
    """A_s goes into lvspec_loose_accept as a ready per-position score; the rule
    is checked against the oracle evaluated on the GPU's own score bytes."""
    from gpu_util import run_accept
    cfg = dataclasses.replace(W.CONFIGS[0], gamma=10)
    hd, hv = W.relevance_inputs(cfg, n_visual=1200, dim=256)
    got, _ = _run(ctx, hd, hv, 10)
    score = got.astype(np.float32)[:, :, None]
    logits, draft = W.accept_inputs(cfg)
    n = oracle_mod.n_loose(0.7, cfg.gamma)
    ref = oracle_mod.loose_accept(logits, draft, score, n, cfg.gamma)
    res = run_accept(ctx, logits, draft, score, cfg.gamma, n_loose=n)
    assert (res[0] == ref[0]).all() and (res[2] == ref[2]).all()


def test_invalid_arguments_launch_nothing(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    hd = torch.zeros(1, 4, 128, dtype=torch.bfloat16, device="cuda")
    hv = torch.zeros(1, 50, 128, dtype=torch.bfloat16, device="cuda")
    inv = torch.zeros(1, 50, device="cuda")
    rel = torch.zeros(1, 4, device="cuda")
    before = ctx.launch_count()
    for args, status in [((0, 4, 50, 128), binding.ERR_INVALID_ARG), ((1, 0, 50, 128), binding.ERR_INVALID_ARG),
                         ((1, 65, 50, 128), binding.ERR_INVALID_ARG), ((1, 4, 0, 128), binding.ERR_INVALID_ARG),
                         ((1, 4, 50, 96), binding.ERR_UNSUPPORTED), ((1, 4, 50, 32), binding.ERR_INVALID_ARG)]:
        with pytest.raises(binding.LvspecError) as e:
            ctx.visual_relevance(*args, hd, hv, inv, 10, rel)
        assert e.value.status == status, args
    with pytest.raises(binding.LvspecError):
        ctx.visual_relevance(1, 4, 50, 128, hd, hv, inv, 0, rel)
    with pytest.raises(binding.LvspecError):
        ctx.visual_relevance(1, 4, 50, 128, None, hv, inv, 10, rel)
    with pytest.raises(binding.LvspecError):
        ctx.row_inv_norms(50, 100, hv, inv)
    assert ctx.launch_count() == before
