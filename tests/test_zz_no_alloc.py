"""lvspec_loose_accept_static: the acceptance pass for callers that cannot
allocate device memory (servers whose own pool owns the GPU, fixed memory
budgets, loops that must avoid the synchronisation of cudaMalloc).  It keeps
its scratch in a fixed array inside the library, shared by every call, so the
check is that two calls in a row, through the C ABI and without any context,
give exactly what the context-based lvspec_loose_accept gives on the same
inputs (all outputs are integers: the comparison is bit-exact).

This file sorts last on purpose: a run that stops at the first failure has
then already run every other test."""
import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _inputs(cfg, batch):
    logits, draft = W.accept_inputs(cfg, batch=batch)
    mass = W.synthetic_mass(cfg, batch=batch)
    return logits, draft, mass


def test_two_calls_in_a_row_match_the_context_entry_point():
    import torch
    from paper_2604_05650_b200 import binding
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream()

    # first call: many rows and slices; second call: fewer rows, other vocab, so
    # what the first call left in the shared array is stale for the second
    cases = [(W.sweep_config(gamma=8, kv_len=4096, batch=16, point=77), 16, 8),
             (W.CONFIGS[0], 3, 1)]
    got = []
    for cfg, batch, window in cases:
        logits, draft, mass = _inputs(cfg, batch)
        dl = torch.from_numpy(logits).cuda()
        dd = torch.from_numpy(draft).cuda()
        dm = torch.from_numpy(mass).cuda()
        alen = torch.full((batch,), -5, dtype=torch.int32, device="cuda")
        binding.loose_accept_static(stream, batch, cfg.gamma, cfg.vocab, mass.shape[2], dl, dd, dm,
                                    alen, window, lam=cfg.lam)
        torch.cuda.synchronize()
        got.append(alen.cpu().numpy())

    ctx = binding.Context(0)
    try:
        ctx.set_stream(stream.cuda_stream)
        for (cfg, batch, window), g in zip(cases, got):
            logits, draft, mass = _inputs(cfg, batch)
            dl = torch.from_numpy(logits).cuda()
            dd = torch.from_numpy(draft).cuda()
            dm = torch.from_numpy(mass).cuda()
            ref = torch.full((batch,), -9, dtype=torch.int32, device="cuda")
            ctx.loose_accept(batch, cfg.gamma, cfg.vocab, mass.shape[2], dl, dd, dm, ref, window,
                             lam=cfg.lam)
            torch.cuda.synchronize()
            assert (g == ref.cpu().numpy()).all()
            assert (g >= 0).all() and (g <= cfg.gamma).all()
    finally:
        ctx.close()


def test_sizes_beyond_the_fixed_array_are_refused():
    import torch
    from paper_2604_05650_b200 import binding
    torch.cuda.set_device(0)
    batch, gamma, vocab = 128, 16, 64                  # 2048 rows > LVSPEC_STATIC_MAX_ROWS
    assert batch * gamma > binding.STATIC_MAX_ROWS
    dl = torch.zeros(batch, gamma, vocab, device="cuda")
    dd = torch.zeros(batch, gamma, dtype=torch.int32, device="cuda")
    dm = torch.zeros(batch, gamma, 1, device="cuda")
    alen = torch.full((batch,), -5, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.LvspecError) as e:
        binding.loose_accept_static(None, batch, gamma, vocab, 1, dl, dd, dm, alen, 0)
    assert e.value.status == binding.ERR_UNSUPPORTED
    assert "LVSPEC_STATIC_MAX_ROWS" in str(e.value)
    torch.cuda.synchronize()
    assert (alen.cpu().numpy() == -5).all()            # nothing was launched
