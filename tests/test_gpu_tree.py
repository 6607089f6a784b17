"""GPU parity of the draft-tree variant (App. "Exploration on Draft Token Trees"):
tree attention against the oracle, then loose acceptance per branch and the
choice of the longest branch, bit-exact on the same inputs."""
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


def _case(seed, B, R, K, Hq, Hkv, D, kv_len, span):
    rng = np.random.default_rng(seed)
    g = R * K
    Lmax = max(kv_len)
    bits = lambda shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    return (bits((B, g, Hq, D)), bits((B, Hkv, Lmax, D)), bits((B, Hkv, Lmax, D)),
            np.asarray(kv_len, dtype=np.int32), np.asarray(span, dtype=np.int32))


def _run_tree(ctx, case, R, kernel, n_split=0):
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import dev_bf16, bf16_to_f64
    q, k, v, kv_len, span = case
    B, g, Hq, D = q.shape
    dq, dk, dv = dev_bf16(q), dev_bf16(k), dev_bf16(v)
    out = torch.full((B, g, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    mass = torch.full((B, g, Hq), float("nan"), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(B, g, Hq, k.shape[1], D, k.shape[2], n_split, kernel)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention_tree(shape, R, dq, dk, dv, kv_len, span, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return bf16_to_f64(out), mass.cpu().numpy().astype(np.float64), mass


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("shape", [
    # B, R, K, Hq, Hkv, D, kv_len, span, n_split
    (1, 2, 10, 10, 2, 128, [3000], [[300, 2500]], 0),        # the paper's tree: two branches of ten
    (2, 2, 4, 8, 2, 128, [700, 391], [[10, 500], [0, 380]], 3),
    (1, 4, 3, 4, 1, 128, [520], [[5, 300]], 2),              # four branches, tail crosses a tile edge
    (1, 3, 5, 8, 2, 64, [1000], [[64, 832]], 4),
])
def test_tree_attention(ctx, oracle_mod, shape, kernel):
    from gpu_util import assert_attention_close
    B, R, K, Hq, Hkv, D, kv_len, span, n_split = shape
    case = _case(41, B, R, K, Hq, Hkv, D, kv_len, span)
    ref_out, ref_mass = oracle_mod.verify_attention(*case, branch_len=K)
    out, mass, _ = _run_tree(ctx, case, R, kernel, n_split)
    assert_attention_close(out, mass, ref_out, ref_mass)


def test_tree_step_end_to_end(ctx, oracle_mod):
    """Tree attention -> loose acceptance per branch (fed by the GPU's own mass)
    -> longest branch; decisions bit-exact against the oracle on the same bytes."""
    import torch
    B, R, K, Hq, Hkv, D, V = 3, 2, 10, 10, 2, 128, 5000
    case = _case(42, B, R, K, Hq, Hkv, D, [2048, 1500, 1999], [[100, 1500], [50, 1200], [0, 1900]])
    _, mass64, dmass = _run_tree(ctx, case, R, 2)
    rng = np.random.default_rng(43)
    logits = (rng.standard_normal((B * R, K, V)) * 3).astype(np.float32)
    top = logits.argmax(-1)
    draft = np.where(rng.random((B * R, K)) < 0.6, top, rng.integers(0, V, (B * R, K))).astype(np.int32)
    dl, dd = torch.from_numpy(logits).cuda(), torch.from_numpy(draft).cuda()
    alen = torch.full((B * R,), -3, dtype=torch.int32, device="cuda")
    bb = torch.full((B,), -3, dtype=torch.int32, device="cuda")
    bl = torch.full((B,), -3, dtype=torch.int32, device="cuda")
    n = oracle_mod.n_loose(0.7, K)
    # the attention's mass [B, R*K, Hq] is read as [B*R, K, Hq]
    ctx.loose_accept(B * R, K, V, Hq, dl, dd, dmass, alen, K, n_loose=n)
    ctx.select_branch(B, R, alen, bb, bl)
    torch.cuda.synchronize()
    ref_len, _, _ = oracle_mod.loose_accept(logits, draft, mass64.astype(np.float32).reshape(B * R, K, Hq), n, K)
    ref_bb, ref_bl = oracle_mod.select_branch(ref_len.reshape(B, R))
    assert (alen.cpu().numpy() == ref_len).all()
    assert (bb.cpu().numpy() == ref_bb).all() and (bl.cpu().numpy() == ref_bl).all()


def test_invalid_branch_counts(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    q = torch.zeros(1, 6, 4, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 2, 256, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    mass = torch.zeros(1, 6, 4, device="cuda")
    shape = binding.attn_shape(1, 6, 4, 2, 128, 256)
    before = ctx.launch_count()
    for r in (0, 4, -1):
        with pytest.raises(binding.LvspecError):
            ctx.verify_attention_tree(shape, r, q, kv, kv, (256,), ((0, 10),), out, mass)
    a = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.LvspecError):
        ctx.select_branch(0, 2, a, a, a)
    assert ctx.launch_count() == before
