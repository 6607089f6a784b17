"""Failure detection without a GPU fault: a bounded device-side wait that runs
out (a barrier nothing ever completes) must come back as an error status the
host can read, leave no hang behind, and leave the context usable."""
import time

import numpy as np
import pytest

from paper_2604_05650_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_context_stays_usable(oracle_mod):
    import torch
    from paper_2604_05650_b200 import binding
    from gpu_util import run_attention, assert_attention_close
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    ctx = binding.Context(0)
    try:
        ctx.set_stream(torch.cuda.current_stream().cuda_stream)
        assert ctx.device_status_code() == (binding.OK, 0)
        t0 = time.perf_counter()
        ctx.selftest_wait_expiry(20)                      # gives up after 20 ms
        code, flags = ctx.device_status_code()            # synchronises the stream
        waited = time.perf_counter() - t0
        assert code == binding.ERR_TIMEOUT and flags & binding.DEV_WAIT_EXPIRED
        assert 0.015 <= waited < 1.5, waited
        assert ctx.device_status_code() == (binding.OK, 0)   # reported once, then cleared
        # the context and the device still work
        cfg = W.sweep_config(gamma=4, kv_len=2048, batch=1)
        case = W.attention_inputs(cfg)
        out, mass = run_attention(ctx, *case)
        ref_out, ref_mass = oracle_mod.verify_attention(*case)
        assert_attention_close(out, mass, ref_out, ref_mass)
        with pytest.raises(binding.LvspecError):
            ctx.selftest_wait_expiry(0)
    finally:
        ctx.close()
