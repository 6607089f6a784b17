"""Scratch memory of a context: sizing it up front (lvspec_*_workspace_bytes,
lvspec_reserve), what happens when it would have to grow during a stream capture, and
that stale scratch contents never reach a result."""
import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _fresh_ctx():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05650_b200 import binding
    return binding.Context(0)


def _big_shape():
    """64 splits x 32 (sequence, head) units x 40 rows x 128 channels of fp32 partials:
    42 MB, far beyond the few MiB a new context holds."""
    from paper_2604_05650_b200 import binding
    return binding.attn_shape(4, 8, 40, 8, 128, 8192, n_split=64)


def test_reserve_sizes_the_scratch_before_a_capture(oracle_mod):
    import torch
    from paper_2604_05650_b200 import binding
    ctx = _fresh_ctx()
    try:
        shape = _big_shape()
        need = ctx.attention_workspace_bytes(shape, 8192)
        assert need > ctx.workspace_capacity() > 0
        assert need >= 4 * 8 * 64 * 40 * (128 + 4) * 4
        ctx.reserve(need)
        cap = ctx.workspace_capacity()
        assert cap >= need
        ctx.reserve(1)                                 # never shrinks
        assert ctx.workspace_capacity() == cap

        cfg = W.sweep_config(gamma=8, kv_len=8192, batch=4, point=55)
        q, k, v, kv_len, span = W.attention_inputs(cfg)
        from gpu_util import dev_bf16, bf16_to_f64, assert_attention_close
        dq, dk, dv = dev_bf16(q), dev_bf16(k), dev_bf16(v)
        out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        mass = torch.full(q.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
        stream = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ctx.set_stream(torch.cuda.current_stream().cuda_stream)
            ctx.verify_attention(shape, dq, dk, dv, kv_len, span, out, mass)   # no growth: captured
        assert ctx.workspace_capacity() == cap
        ctx.set_stream(stream.cuda_stream)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
        assert_attention_close(bf16_to_f64(out), mass.cpu().numpy().astype(np.float64), ref_out, ref_mass)
    finally:
        ctx.close()


def test_growth_during_a_capture_is_refused_and_the_capture_survives():
    import torch
    from paper_2604_05650_b200 import binding
    ctx = _fresh_ctx()
    try:
        shape = _big_shape()
        cap = ctx.workspace_capacity()
        assert ctx.attention_workspace_bytes(shape, 8192) > cap
        q = torch.zeros(4, 8, 40, 128, dtype=torch.bfloat16, device="cuda")
        kv = torch.zeros(4, 8, 8192, 128, dtype=torch.bfloat16, device="cuda")
        out = torch.zeros_like(q)
        mass = torch.zeros(4, 8, 40, device="cuda")
        x = torch.zeros(1024, device="cuda")
        kv_len, span = [8192] * 4, [[0, 100]] * 4
        before = ctx.launch_count()
        stream = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ctx.set_stream(torch.cuda.current_stream().cuda_stream)
            x += 1.0
            with pytest.raises(binding.LvspecError) as e:
                ctx.verify_attention(shape, q, kv, kv, kv_len, span, out, mass)
            assert e.value.status == binding.ERR_WORKSPACE
            assert "lvspec_reserve" in str(e.value)
            with pytest.raises(binding.LvspecError) as e:
                ctx.reserve(64 << 20)
            assert e.value.status == binding.ERR_WORKSPACE
            x += 1.0
        assert ctx.launch_count() == before and ctx.workspace_capacity() == cap
        graph.replay()                                  # the capture stayed valid
        torch.cuda.synchronize()
        assert float(x[0]) == 2.0
        # outside the capture the same call grows the scratch by itself
        ctx.set_stream(torch.cuda.current_stream().cuda_stream)
        ctx.verify_attention(shape, q, kv, kv, kv_len, span, out, mass)
        torch.cuda.synchronize()
        assert ctx.workspace_capacity() > cap and ctx.device_status() == 0
    finally:
        ctx.close()


def test_workspace_queries_cover_what_the_calls_take():
    """Reserving exactly the figure each query returns is enough: the calls that follow
    leave the capacity alone."""
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import run_attention, run_accept
    ctx = _fresh_ctx()
    try:
        cfg = W.sweep_config(gamma=16, kv_len=6000, batch=3, point=56)
        shape = binding.attn_shape(cfg.batch, cfg.gamma, 40, 8, 128, cfg.kv_len)
        need = max(ctx.attention_workspace_bytes(shape, cfg.kv_len),
                   ctx.accept_workspace_bytes(cfg.batch, cfg.gamma, cfg.vocab),
                   ctx.relevance_workspace_bytes(cfg.batch, cfg.gamma, 60000, 512))
        assert need > ctx.workspace_capacity()
        ctx.reserve(need)
        cap = ctx.workspace_capacity()
        q, k, v, kv_len, span = W.attention_inputs(cfg)
        run_attention(ctx, q, k, v, kv_len, span)
        logits, draft = W.accept_inputs(cfg)
        run_accept(ctx, logits, draft, W.synthetic_mass(cfg), cfg.shift_window)
        hd, hv = W.relevance_inputs(cfg, n_visual=60000, dim=512, batch=1)
        hd, hv = np.repeat(hd, cfg.batch, 0), np.repeat(hv, cfg.batch, 0)
        from gpu_util import dev_bf16
        dhd, dhv = dev_bf16(hd), dev_bf16(hv)
        inv = torch.empty((cfg.batch, 60000), dtype=torch.float32, device="cuda")
        rel = torch.empty((cfg.batch, cfg.gamma), dtype=torch.float32, device="cuda")
        ctx.row_inv_norms(cfg.batch * 60000, 512, dhv, inv)
        ctx.visual_relevance(cfg.batch, cfg.gamma, 60000, 512, dhd, dhv, inv, 10, rel)
        torch.cuda.synchronize()
        assert ctx.workspace_capacity() == cap and ctx.device_status() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("kernel", [1, 2])
def test_splits_without_tiles_after_the_scratch_held_nan(oracle_mod, kernel):
    """A ragged batch leaves the shorter sequences with splits that own no tile; such a
    split writes no partial rows, so whatever an earlier call left in the scratch sits
    there when the splits are merged.  The earlier call here fills the partials with NaN
    (an all-NaN key cache); the ragged call after it must still match the oracle."""
    import torch
    from gpu_util import run_attention, assert_attention_close
    ctx = _fresh_ctx()
    try:
        rng = np.random.default_rng(77)
        bits = lambda shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
        B, gamma, Hq, Hkv, Dh, Lmax = 3, 3, 6, 3, 128, 520
        q, k, v = bits((B, gamma, Hq, Dh)), bits((B, Hkv, Lmax, Dh)), bits((B, Hkv, Lmax, Dh))
        k_nan = np.full_like(k, 0x7FC0)
        full = np.asarray([Lmax] * B, dtype=np.int32)
        span_full = np.asarray([[5, 20]] * B, dtype=np.int32)
        out_nan, _ = _run_unchecked(ctx, q, k_nan, v, full, span_full, 4, kernel)
        assert np.isnan(out_nan).all()
        kv_len = np.asarray([33, 520, 3], dtype=np.int32)
        span = np.asarray([[5, 20], [100, 101], [0, 0]], dtype=np.int32)
        out, mass = run_attention(ctx, q, k, v, kv_len, span, n_split=4, kernel=kernel)
        ref_out, ref_mass = oracle_mod.verify_attention(q, k, v, kv_len, span)
        assert_attention_close(out, mass, ref_out, ref_mass)
    finally:
        ctx.close()


def _run_unchecked(ctx, q, k, v, kv_len, span, n_split, kernel):
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import dev_bf16, bf16_to_f64
    B, gamma, Hq, Dh = q.shape
    out = torch.zeros((B, gamma, Hq, Dh), dtype=torch.bfloat16, device="cuda")
    mass = torch.zeros((B, gamma, Hq), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(B, gamma, Hq, k.shape[1], Dh, k.shape[2], n_split, kernel)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention(shape, dev_bf16(q), dev_bf16(k), dev_bf16(v), kv_len, span, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() & binding.DEV_WAIT_EXPIRED == 0
    return bf16_to_f64(out), mass.cpu().numpy()
