"""GPU parity of lvspec_loose_accept against the oracle: bit-exact target
tokens, decisions and accepted lengths on byte-identical inputs."""
import itertools

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


def _same(ctx, oracle_mod, logits, draft, mass, window, n_loose):
    from gpu_util import run_accept
    ref = oracle_mod.loose_accept(logits, draft, mass, n_loose, window)
    got = run_accept(ctx, logits, draft, mass, window, n_loose=n_loose)
    assert (got[1] == ref[1]).all(), "target tokens differ"
    assert (got[2] == ref[2]).all(), "decisions differ"
    assert (got[0] == ref[0]).all(), "accepted lengths differ"
    return got


@pytest.mark.parametrize("cfg_id", [0, 1, 2, 3])
def test_configs(ctx, oracle_mod, cfg_id):
    from gpu_util import run_accept
    cfg = W.CONFIGS[cfg_id]
    logits, draft = W.accept_inputs(cfg)
    mass = W.synthetic_mass(cfg)
    n = oracle_mod.n_loose(cfg.lam, cfg.gamma)
    for window in (0, 1, cfg.shift_window):
        _same(ctx, oracle_mod, logits, draft, mass, window, n)
    # lambda given instead of n_loose resolves to the same count
    ref = oracle_mod.loose_accept(logits, draft, mass, n, cfg.shift_window)
    got = run_accept(ctx, logits, draft, mass, cfg.shift_window, lam=cfg.lam, n_loose=-1)
    assert (got[0] == ref[0]).all() and (got[2] == ref[2]).all()


@pytest.mark.parametrize("batch,gamma", [(4, 16), (16, 8), (16, 4), (128, 2)])
def test_sweep_batches(ctx, oracle_mod, batch, gamma):
    cfg = W.sweep_config(gamma=gamma, kv_len=4096, batch=batch, point=batch + gamma)
    if batch == 128:
        import dataclasses
        cfg = dataclasses.replace(cfg, vocab=20001)       # odd vocab: unaligned rows
    logits, draft = W.accept_inputs(cfg)
    mass = W.synthetic_mass(cfg)
    for n, w in ((oracle_mod.n_loose(0.7, gamma), gamma), (0, 0), (1, 1)):
        _same(ctx, oracle_mod, logits, draft, mass, w, n)


def test_ties_across_every_reduction_boundary(ctx, oracle_mod):
    """Equal maxima planted on both sides of vector, warp, CTA-pass and slice
    boundaries; the lowest index must win each time."""
    from paper_2604_05650_b200 import binding
    V = 152064
    probe = [0, 1, 3, 4, 5, 127, 128, 1023, 1024, 1027, 4095, 4096, 8191, 8192, 37999, 38000,
             38015, 38016, 38017, 76031, 76032, 152060, 152063]
    pairs = [(a, b) for a in probe for b in probe if a < b][:: 3]
    rng = np.random.default_rng(3)
    for chunk in range(0, len(pairs), 64):
        sel = pairs[chunk:chunk + 64]
        B, gamma = len(sel), 1
        logits = rng.standard_normal((B, gamma, V)).astype(np.float32)
        for r, (a, b) in enumerate(sel):
            logits[r, 0, a] = 40.0
            logits[r, 0, b] = 40.0
        draft = np.zeros((B, gamma), dtype=np.int32)
        mass = np.zeros((B, gamma, 1), dtype=np.float32)
        got = _same(ctx, oracle_mod, logits, draft, mass, 0, 0)
        assert got[1][:, 0].tolist() == [a for a, _ in sel]


def test_special_values(ctx, oracle_mod):
    from paper_2604_05650_b200 import binding
    rng = np.random.default_rng(4)
    B, gamma, V = 2, 6, 5003
    lg = rng.standard_normal((B, gamma, V)).astype(np.float32)
    lg[0, 0, :] = -np.inf
    lg[0, 1, 7] = np.nan
    lg[0, 1, 9] = 50.0
    lg[0, 2, :] = np.nan
    lg[0, 3, V - 1] = 60.0
    lg[0, 4, 0] = 60.0
    lg[0, 5, 3] = np.inf
    lg[0, 5, 4000] = np.inf
    lg[1, 0, :] = 0.0
    lg[1, 0, 4099] = 1e-42           # a denormal is still greater than zero
    lg[1, 1, :] = -0.0
    lg[1, 1, 17] = 0.0               # +0 and -0 compare equal: first index wins
    lg[1, 2, :] = -1e-41
    lg[1, 2, 4999] = -1e-42
    draft = rng.integers(0, V, (B, gamma)).astype(np.int32)
    mass = rng.random((B, gamma, 3), dtype=np.float32)
    ctx.device_status()
    got = _same(ctx, oracle_mod, lg, draft, mass, 1, 2)
    assert got[1][0].tolist() == [0, 9, 0, V - 1, 0, 3]
    assert got[1][1, :3].tolist() == [4099, 0, 4999]
    assert ctx.device_status() & binding.DEV_NAN_LOGIT
    assert ctx.device_status() == 0


def test_rule_exhaustive_through_the_gpu(ctx, oracle_mod):
    """Every (n', W) for gamma = 4 over random draft/target pairs from a small
    alphabet with tied and untied scores; 128 sequences per call."""
    g, V = 4, 8
    rng = np.random.default_rng(5)
    B = 128
    for trial in range(3):
        target = rng.integers(0, 3, (B, g))
        draft = rng.integers(0, 3, (B, g)).astype(np.int32)
        logits = np.zeros((B, g, V), dtype=np.float32)
        logits[np.arange(B)[:, None], np.arange(g)[None, :], target] = 3.0
        mass = (rng.integers(0, 3, (B, g, 2)) * 0.25).astype(np.float32)
        for n, w in itertools.product(range(g + 1), range(g + 1)):
            _same(ctx, oracle_mod, logits, draft, mass, w, n)


def test_chained_with_attention_mass(ctx, oracle_mod):
    """Attention mass from the GPU feeds the acceptance pass; the rule is then
    checked against the oracle evaluated on the GPU's own mass bytes."""
    from gpu_util import run_attention, run_accept
    cfg = W.CONFIGS[0]
    q, k, v, kv_len, span = W.attention_inputs(cfg)
    _, mass = run_attention(ctx, q, k, v, kv_len, span)
    mass32 = mass.astype(np.float32)
    logits, draft = W.accept_inputs(cfg)
    n = oracle_mod.n_loose(cfg.lam, cfg.gamma)
    _same(ctx, oracle_mod, logits, draft, mass32, cfg.shift_window, n)


def test_host_buffer_entry_point(ctx, oracle_mod):
    import torch
    cfg = W.CONFIGS[0]
    logits, draft = W.accept_inputs(cfg)
    mass = W.synthetic_mass(cfg)
    alen = np.full((1,), -1, dtype=np.int32)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.loose_accept_host(1, cfg.gamma, cfg.vocab, cfg.n_q_heads, logits, draft, mass, alen,
                          cfg.shift_window, lam=cfg.lam)
    ref = oracle_mod.loose_accept(logits, draft, mass, oracle_mod.n_loose(cfg.lam, cfg.gamma),
                                  cfg.shift_window)
    assert (alen == ref[0]).all()


def test_invalid_arguments_launch_nothing(ctx):
    import torch
    from paper_2604_05650_b200 import binding
    lg = torch.zeros(1, 4, 100, device="cuda")
    dr = torch.zeros(1, 4, dtype=torch.int32, device="cuda")
    ms = torch.zeros(1, 4, 2, device="cuda")
    al = torch.zeros(1, dtype=torch.int32, device="cuda")
    before = ctx.launch_count()
    bad = [dict(batch=0), dict(gamma=0), dict(gamma=65), dict(vocab=0), dict(n_mass_heads=0),
           dict(shift_window=-1), dict(lam=1.5), dict(n_loose=5), dict(lam=float("nan"))]
    for over in bad:
        a = dict(batch=1, gamma=4, vocab=100, n_mass_heads=2, shift_window=1, lam=0.7, n_loose=-1)
        a.update(over)
        with pytest.raises(binding.LvspecError) as e:
            ctx.loose_accept(a["batch"], a["gamma"], a["vocab"], a["n_mass_heads"], lg, dr, ms, al,
                             a["shift_window"], lam=a["lam"], n_loose=a["n_loose"])
        assert e.value.status == binding.ERR_INVALID_ARG, over
    with pytest.raises(binding.LvspecError):
        ctx.loose_accept(1, 4, 100, 2, None, dr, ms, al, 1)
    assert ctx.launch_count() == before


@pytest.mark.parametrize("cfg_id", [0, 2, 3])
def test_emit_step(ctx, oracle_mod, cfg_id):
    """Accepted draft tokens, correction token, token count and new cache length,
    bit-exact against the oracle's emit step on the same inputs."""
    import torch
    cfg = W.CONFIGS[cfg_id]
    B = 5
    logits, draft = W.accept_inputs(cfg, batch=B)
    mass = W.synthetic_mass(cfg, batch=B)
    kv_len = np.array([cfg.kv_len - 3 * b for b in range(B)], dtype=np.int32)
    n = oracle_mod.n_loose(cfg.lam, cfg.gamma)
    for window in (0, cfg.shift_window):
        tau, tgt, _ = oracle_mod.loose_accept(logits, draft, mass, n, window)
        ref_em, ref_n, ref_kv = oracle_mod.emit(draft, tgt, tau, kv_len)
        dl, dd, dm = (torch.from_numpy(x).cuda() for x in (logits, draft, mass))
        dkv = torch.from_numpy(kv_len).cuda()
        alen = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        em = torch.full((B, cfg.gamma), -7, dtype=torch.int32, device="cuda")
        ne = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        nkv = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        ctx.set_stream(torch.cuda.current_stream().cuda_stream)
        ctx.loose_accept_emit(B, cfg.gamma, cfg.vocab, mass.shape[2], dl, dd, dm, alen, em, ne, window,
                              n_loose=n, kv_len=dkv, new_kv_len=nkv)
        torch.cuda.synchronize()
        assert (alen.cpu().numpy() == tau).all()
        assert (em.cpu().numpy() == ref_em).all()
        assert (ne.cpu().numpy() == ref_n).all()
        assert (nkv.cpu().numpy() == ref_kv).all()
    # without cache lengths
    ctx.loose_accept_emit(B, cfg.gamma, cfg.vocab, mass.shape[2], dl, dd, dm, alen, em, ne, window, n_loose=n)
    torch.cuda.synchronize()
    assert (em.cpu().numpy() == ref_em).all()
    from paper_2604_05650_b200 import binding
    with pytest.raises(binding.LvspecError):
        ctx.loose_accept_emit(B, cfg.gamma, cfg.vocab, mass.shape[2], dl, dd, dm, alen, em, ne, window,
                              n_loose=n, kv_len=dkv)          # kv_len without new_kv_len
    with pytest.raises(binding.LvspecError):
        ctx.loose_accept_emit(B, cfg.gamma, cfg.vocab, mass.shape[2], dl, dd, dm, alen, None, ne, window, n_loose=n)
