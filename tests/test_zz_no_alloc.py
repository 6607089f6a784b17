"""lvspec_loose_accept_static: the acceptance pass for callers that cannot
allocate device memory (servers whose own pool owns the GPU, fixed memory
budgets, loops that must avoid the synchronisation of cudaMalloc).  It keeps
its scratch in a fixed array inside the library, shared by every call, so the
check is that two calls in a row, through the C ABI and without any context,
give exactly what the context-based lvspec_loose_accept gives on the same
inputs, and what the CPU oracle gives (all outputs are integers: the
comparisons are bit-exact).

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


def test_two_calls_in_a_row_match_the_context_entry_point(oracle_mod):
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
            want, _, _ = oracle_mod.loose_accept(logits, draft, mass, oracle_mod.n_loose(cfg.lam, cfg.gamma),
                                                 window)
            assert (g == want).all()
    finally:
        ctx.close()


def test_most_rows_the_array_takes_and_special_logits(oracle_mod):
    """batch * gamma = LVSPEC_STATIC_MAX_ROWS: the number of vocabulary slices is then
    bounded by the array (8 partials per row), not by the device; one row holds a NaN and
    a -inf logit (NaN ranks as -inf), another nothing above -inf (token 0).  Checked
    against the oracle directly."""
    import torch
    from paper_2604_05650_b200 import binding
    torch.cuda.set_device(0)
    batch, gamma, vocab, heads = 128, 8, 40000, 2
    assert batch * gamma == binding.STATIC_MAX_ROWS
    rng = np.random.default_rng(4242)
    logits = rng.standard_normal((batch, gamma, vocab), dtype=np.float32)
    top = logits.argmax(-1)
    draft = np.where(rng.random((batch, gamma)) < 0.6, top, rng.integers(0, vocab, (batch, gamma))).astype(np.int32)
    logits[3, 2, 17] = np.nan
    logits[3, 2, 31000] = -np.inf
    logits[5, 0, :] = -np.inf
    logits[5, 1, :] = np.nan
    mass = rng.random((batch, gamma, heads), dtype=np.float32)
    dl, dd, dm = torch.from_numpy(logits).cuda(), torch.from_numpy(draft).cuda(), torch.from_numpy(mass).cuda()
    for window in (0, 3):
        alen = torch.full((batch,), -5, dtype=torch.int32, device="cuda")
        binding.loose_accept_static(torch.cuda.current_stream(), batch, gamma, vocab, heads, dl, dd, dm, alen,
                                    window, n_loose=3)
        torch.cuda.synchronize()
        want, _, _ = oracle_mod.loose_accept(logits, draft, mass, 3, window)
        assert (alen.cpu().numpy() == want).all()


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
