"""GPU parity of lvspec_verify_attention against the fp64 oracle on the long streams of
the head-shape sweep (40 query heads, 8 KV heads, head_dim 128; 64K and 128K cache
positions; batch 1, 4 and 16), with the default kernel and the default split choice: the
launch configuration the benchmark's sweep times.

At batch 16 the library takes one split per (sequence, KV head), so one CTA streams
512 to 1024 tiles: its shared-memory rings and barrier phases wrap hundreds of times,
the reference exponent of a row stays fixed over the whole stream, and byte offsets into
the caches pass 2^32.

The caches of the largest case hold 8.6 GB, so K and V are drawn on the device (seeded)
and parity is SAMPLED: the units (sequence, KV head) listed in `_units` are copied to the
host, and for each of them every draft query of every query head that reads this KV
head is compared with the oracle, element by element, at the usual tolerances."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

HQ, HKV, D = 40, 8, 128
G = HQ // HKV


@pytest.fixture(scope="module")
def ctx():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05650_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _units(batch):
    """Sampled (sequence, KV head) units: first, middle and last sequence x first and
    last KV head."""
    seqs = sorted({0, batch // 2, batch - 1})
    return [(b, h) for b in seqs for h in (0, HKV - 1)]


def _draw(seed, batch, gamma, capacity, span):
    """Q, K, V ~ N(0,1) in bf16 on the device, the visual keys shifted by +0.5 on 8
    channels per KV head: the recipe of the workload configs, drawn by torch's seeded
    generator one sequence at a time (the fp32 draws of all sequences at once would take
    twice the memory of the caches)."""
    import torch
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    q = torch.randn((batch, gamma, HQ, D), generator=gen, device=dev).to(torch.bfloat16)
    k = torch.empty((batch, HKV, capacity, D), dtype=torch.bfloat16, device=dev)
    v = torch.empty((batch, HKV, capacity, D), dtype=torch.bfloat16, device=dev)
    dims = [torch.randperm(D, generator=gen, device=dev)[:8] for _ in range(HKV)]
    for b in range(batch):
        kb = torch.randn((HKV, capacity, D), generator=gen, device=dev)
        for h in range(HKV):
            kb[h, span[0]:span[1], dims[h]] += 0.5
        k[b] = kb.to(torch.bfloat16)
        del kb
        v[b] = torch.randn((HKV, capacity, D), generator=gen, device=dev).to(torch.bfloat16)
    return q, k, v


def _bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _check_units(oracle_mod, q, k, v, kv_len, span, out, mass, gamma):
    from gpu_util import assert_attention_close
    for b, h in _units(q.shape[0]):
        hq = slice(h * G, (h + 1) * G)
        ref_out, ref_mass = oracle_mod.verify_attention(
            _bits(q[b:b + 1, :, hq]), _bits(k[b:b + 1, h:h + 1]), _bits(v[b:b + 1, h:h + 1]),
            np.asarray([kv_len[b]], dtype=np.int32), np.asarray([span[b]], dtype=np.int32))
        got_out = out[b:b + 1, :, hq].float().cpu().numpy().astype(np.float64)
        got_mass = mass[b:b + 1, :, hq].cpu().numpy().astype(np.float64)
        assert_attention_close(got_out, got_mass, ref_out, ref_mass)


CASES = [
    # batch, capacity, gamma, kv_len per sequence (None = full), seed
    (1, 131072, 16, None, 4101),
    (4, 65536, 8, [65536, 65459, 40000, 65536], 4102),        # ragged lengths, ragged last tiles
    (16, 65536, 4, None, 4103),                               # one split per head: 512 tiles per CTA
    (16, 131072, 8, None, 4104),                              # 1024 tiles per CTA, 4.3 GB per cache
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"b{c[0]}-kv{c[1]}-g{c[2]}")
def test_sweep_long_stream(ctx, oracle_mod, case):
    import torch
    from paper_2604_05650_b200 import binding
    batch, capacity, gamma, lens, seed = case
    kv_len = np.asarray(lens if lens else [capacity] * batch, dtype=np.int32)
    # 75 % of the cache visual, after a 256-token prefix (the sweep's recipe); a shorter
    # sequence keeps its span inside its own length
    span = np.asarray([[256, min(256 + (capacity * 3) // 4, int(l) - gamma)] for l in kv_len], dtype=np.int32)
    q, k, v = _draw(seed, batch, gamma, capacity, (256, 256 + (capacity * 3) // 4))
    out = torch.full((batch, gamma, HQ, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    mass = torch.full((batch, gamma, HQ), float("nan"), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(batch, gamma, HQ, HKV, D, capacity)
    if batch == 16:
        assert ctx.attention_splits(shape, int(kv_len.max())) == 1
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention(shape, q, k, v, kv_len, span, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert torch.isfinite(out.float()).all() and torch.isfinite(mass).all()
    _check_units(oracle_mod, q, k, v, kv_len, span, out, mass, gamma)
    del q, k, v
    torch.cuda.empty_cache()


def test_sweep_long_stream_paged(ctx, oracle_mod):
    """The same kind of stream through the paged call: batch 4 x 64K positions in
    512-position pages scattered over the pool; bit-identical to the contiguous call and
    equal to the oracle on the sampled units."""
    import torch
    from paper_2604_05650_b200 import binding
    batch, capacity, gamma, page = 4, 65536, 16, 512
    kv_len = np.asarray([65536, 65536, 51234, 65536], dtype=np.int32)
    span = np.asarray([[256, 256 + 49152]] * batch, dtype=np.int32)
    q, k, v = _draw(4105, batch, gamma, capacity, (256, 256 + 49152))
    per_seq = capacity // page
    n_pages = batch * per_seq
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(4105))
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(n_pages)
    to_pool = lambda t: t.view(batch, HKV, per_seq, page, D).permute(0, 2, 1, 3, 4) \
        .reshape(n_pages, HKV, page, D)[perm.cuda()].contiguous()
    k_pool, v_pool = to_pool(k), to_pool(v)
    table = inv.view(batch, per_seq).to(torch.int32).cuda()
    shape = binding.attn_shape(batch, gamma, HQ, HKV, D, capacity)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    res = []
    for paged in (False, True):
        out = torch.full((batch, gamma, HQ, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        mass = torch.full((batch, gamma, HQ), float("nan"), dtype=torch.float32, device="cuda")
        if paged:
            ctx.verify_attention_paged(shape, page, n_pages, q, k_pool, v_pool, table, kv_len, span, out, mass)
        else:
            ctx.verify_attention(shape, q, k, v, kv_len, span, out, mass)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        res.append((out, mass))
    assert torch.equal(res[0][0].view(torch.int16), res[1][0].view(torch.int16))
    assert torch.equal(res[0][1], res[1][1])
    _check_units(oracle_mod, q, k, v, kv_len, span, res[1][0], res[1][1], gamma)
