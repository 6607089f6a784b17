"""Helpers of the GPU parity tests: device buffers via torch (plumbing only)."""
import numpy as np
import torch

from paper_2604_05650_b200 import binding


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def run_attention(ctx, q, k, v, kv_len, span, n_split=0, kernel=0):
    """q/k/v: uint16 bf16 bit patterns (numpy).  Returns (out fp64, mass fp64)."""
    B, gamma, Hq, D = q.shape
    Hkv, Lmax = k.shape[1], k.shape[2]
    dq, dk, dv = dev_bf16(q), dev_bf16(k), dev_bf16(v)
    out = torch.full((B, gamma, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    mass = torch.full((B, gamma, Hq), float("nan"), dtype=torch.float32, device="cuda")
    shape = binding.attn_shape(B, gamma, Hq, Hkv, D, Lmax, n_split, kernel)
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.verify_attention(shape, dq, dk, dv, kv_len, span, out, mass)
    torch.cuda.synchronize()
    assert ctx.device_status() & binding.DEV_WAIT_EXPIRED == 0
    return bf16_to_f64(out), mass.cpu().numpy().astype(np.float64)


def assert_attention_close(out, mass, ref_out, ref_mass):
    """Tolerances of the parity bar: |out - ref| <= 1e-2 + 1e-2 |ref|; mass 1e-3 abs."""
    assert np.isfinite(out).all() and np.isfinite(mass).all()
    err = np.abs(out - ref_out) - (1e-2 + 1e-2 * np.abs(ref_out))
    assert err.max() <= 0, f"out: worst excess {err.max():.3e}, max abs err {np.abs(out - ref_out).max():.3e}"
    merr = np.abs(mass - ref_mass).max()
    assert merr <= 1e-3, f"visual mass: max abs err {merr:.3e}"


def run_accept(ctx, logits, draft, mass, shift_window, lam=0.7, n_loose=-1):
    B, gamma, V = logits.shape
    Hm = mass.shape[2]
    dl = torch.from_numpy(np.ascontiguousarray(logits)).cuda()
    dd = torch.from_numpy(np.ascontiguousarray(draft, dtype=np.int32)).cuda()
    dm = torch.from_numpy(np.ascontiguousarray(mass, dtype=np.float32)).cuda()
    alen = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    tgt = torch.full((B, gamma), -7, dtype=torch.int32, device="cuda")
    acc = torch.full((B, gamma), 9, dtype=torch.uint8, device="cuda")
    ctx.set_stream(torch.cuda.current_stream().cuda_stream)
    ctx.loose_accept(B, gamma, V, Hm, dl, dd, dm, alen, shift_window, lam=lam, n_loose=n_loose,
                     target_tokens=tgt, accepted=acc)
    torch.cuda.synchronize()
    return alen.cpu().numpy(), tgt.cpu().numpy(), acc.cpu().numpy()
