"""GPU parity of lvspec_verify_attention_paged: the same attention on a cache whose
pages are scattered over a pool.  The oracle works on the contiguous cache (the paged
layout is an indirection, not another operation); the pages are scattered on the host,
with junk in the pages no sequence owns, and the paged call has to give the oracle's
values, and bit for bit what the contiguous call gives."""
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


def _contiguous_case(seed, B, gamma, Hq, Hkv, Lmax, kv_len, span):
    rng = np.random.default_rng(seed)
    bits = lambda shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    return (bits((B, gamma, Hq, 128)), bits((B, Hkv, Lmax, 128)), bits((B, Hkv, Lmax, 128)),
            np.asarray(kv_len, dtype=np.int32), np.asarray(span, dtype=np.int32))


def scatter_pages(seed, k, v, page_size, spare_pages=3):
    """Cuts [B, Hkv, Lmax, D] caches into pages and places them at random in pools
    [n_pages, Hkv, page_size, D]; pages nobody owns hold large junk."""
    rng = np.random.default_rng(seed)
    B, Hkv, Lmax, D = k.shape
    per_seq = Lmax // page_size
    n_pages = B * per_seq + spare_pages
    order = rng.permutation(n_pages)[:B * per_seq].reshape(B, per_seq).astype(np.int32)
    junk = W.f32_to_bf16_bits(np.full((n_pages, Hkv, page_size, D), 3.0e4, dtype=np.float32))
    k_pool, v_pool = junk.copy(), junk.copy()
    for b in range(B):
        for j in range(per_seq):
            sl = slice(j * page_size, (j + 1) * page_size)
            k_pool[order[b, j]] = k[b, :, sl, :]
            v_pool[order[b, j]] = v[b, :, sl, :]
    return k_pool, v_pool, order, n_pages


def run_paged(ctx, q, k_pool, v_pool, table, n_pages, page_size, Lmax, kv_len, span, n_split=0):
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import dev_bf16, bf16_to_f64
    B, gamma, Hq, D = q.shape
    Hkv = k_pool.shape[1]
    dq, dk, dv = dev_bf16(q), dev_bf16(k_pool), dev_bf16(v_pool)
    dt = torch.from_numpy(np.ascontiguousarray(table, dtype=np.int32)).cuda()
    out = torch.full((B, gamma, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    mass = torch.full((B, gamma, Hq), float("nan"), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(B, gamma, Hq, Hkv, D, Lmax, n_split, 0)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention_paged(shape, page_size, n_pages, dq, dk, dv, dt, kv_len, span, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return out, mass


CASES = [
    # seed, B, gamma, Hq, Hkv, Lmax, page_size, kv_len, span, n_split
    (31, 1, 4, 8, 2, 1024, 128, [1000], [[64, 832]], 0),
    (32, 2, 8, 10, 2, 2048, 256, [2048, 700], [[100, 1500], [0, 692]], 3),
    (33, 3, 5, 12, 4, 1536, 512, [1536, 133, 900], [[0, 0], [5, 100], [128, 640]], 0),
    (34, 1, 8, 40, 8, 4096, 128, [4001], [[512, 3000]], 1),
]


@pytest.mark.parametrize("case", CASES, ids=[f"seed{c[0]}" for c in CASES])
def test_paged_matches_oracle_and_contiguous(ctx, oracle_mod, case):
    from gpu_util import assert_attention_close, bf16_to_f64, dev_bf16
    from paper_2604_05650_b200 import binding
    import torch
    seed, B, gamma, Hq, Hkv, Lmax, page_size, kv_len, span, n_split = case
    q, k, v, kv_len, span = _contiguous_case(seed, B, gamma, Hq, Hkv, Lmax, kv_len, span)
    ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    k_pool, v_pool, table, n_pages = scatter_pages(seed + 100, k, v, page_size)
    out, mass = run_paged(ctx, q, k_pool, v_pool, table, n_pages, page_size, Lmax, kv_len, span, n_split)
    assert_attention_close(bf16_to_f64(out), mass.cpu().numpy().astype(np.float64), ref_out, ref_mass)

    # the contiguous call with the same splits: identical arithmetic, identical bits
    out_c = torch.full_like(out, float("nan"))
    mass_c = torch.full_like(mass, float("nan"))
    shape = binding.attn_shape(B, gamma, Hq, Hkv, 128, Lmax, n_split, 2)
    ctx.verify_attention(shape, dev_bf16(q), dev_bf16(k), dev_bf16(v), kv_len, span, out_c, mass_c)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out_c.view(torch.int16))
    assert torch.equal(mass.view(torch.int32), mass_c.view(torch.int32))


def test_pages_beyond_kv_len_are_never_needed(ctx, oracle_mod):
    """Entries of logical pages past kv_len may be anything, even outside the pool."""
    from gpu_util import assert_attention_close, bf16_to_f64
    q, k, v, kv_len, span = _contiguous_case(41, 2, 6, 8, 2, 2048, [300, 1025], [[10, 200], [0, 1000]])
    ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
    k_pool, v_pool, table, n_pages = scatter_pages(141, k, v, 128)
    table = table.copy()
    table[0, 3:] = -5            # 300 positions live in pages 0..2
    table[1, 9:] = n_pages + 7   # 1025 positions live in pages 0..8
    out, mass = run_paged(ctx, q, k_pool, v_pool, table, n_pages, 128, 2048, kv_len, span)
    assert_attention_close(bf16_to_f64(out), mass.cpu().numpy().astype(np.float64), ref_out, ref_mass)


def test_full_size_layer_paged(ctx, oracle_mod):
    """Config 2's shape with 512-position pages, checked on sampled outputs."""
    import torch
    from gpu_util import bf16_to_f64
    cfg = W.CONFIGS[2]
    q, k, v, kv_len, span = W.attention_inputs(cfg, layer=1)
    k_pool, v_pool, table, n_pages = scatter_pages(7, k, v, 512, spare_pages=2)
    out, mass = run_paged(ctx, q, k_pool, v_pool, table, n_pages, 512, cfg.kv_len, kv_len, span)
    out, mass = bf16_to_f64(out), mass.cpu().numpy().astype(np.float64)
    heads = [0, cfg.n_q_heads // 2, cfg.n_q_heads - 1]
    G = cfg.n_q_heads // cfg.n_kv_heads
    for h in heads:
        kvh = h // G
        ro, rm = oracle_mod.verify_attention(q[:, :, h:h + 1, :], k[:, kvh:kvh + 1], v[:, kvh:kvh + 1], kv_len, span)
        err = np.abs(out[:, :, h:h + 1, :] - ro) - (1e-2 + 1e-2 * np.abs(ro))
        assert err.max() <= 0
        assert np.abs(mass[:, :, h:h + 1] - rm).max() <= 1e-3


def test_invalid_paged_arguments_launch_nothing(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    q = torch.zeros(1, 4, 8, 128, dtype=torch.bfloat16, device="cuda")
    pool = torch.zeros(10, 2, 128, 128, dtype=torch.bfloat16, device="cuda")
    table = torch.zeros(1, 8, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(q)
    mass = torch.zeros(1, 4, 8, device="cuda")
    good = dict(page_size=128, n_pages=10, Lmax=1024, D=128, kernel=0)
    bad = [dict(page_size=100), dict(page_size=0), dict(n_pages=0), dict(Lmax=1000), dict(kernel=1)]
    before = ctx.launch_count()
    for change in bad:
        a = {**good, **change}
        shape = binding.attn_shape(1, 4, 8, 2, a["D"], a["Lmax"], 0, a["kernel"])
        with pytest.raises(binding.LvspecError) as e:
            ctx.verify_attention_paged(shape, a["page_size"], a["n_pages"], q, pool, pool, table,
                                       [512], [[0, 100]], out, mass)
        assert e.value.status in (binding.ERR_INVALID_ARG, binding.ERR_UNSUPPORTED)
    assert ctx.launch_count() == before
