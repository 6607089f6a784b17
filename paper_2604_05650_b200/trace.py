"""Time-stamp traces of the attention and merge kernels, for performance work.

    python -m paper_2604_05650_b200.trace --config 2 [--fp8] [--layers 6]

builds a second copy of the library with -DLVSPEC_TRACE (liblvspec_trace.so next to the
shipped one; the shipped library carries no trace code), runs a few layers of the
config's attention from one CUDA graph and prints

  * per layer, when its attention and merge CTAs became resident, got past their
    prologue / dependency wait, issued their last K.Q^T and finished (%globaltimer,
    microseconds from the first stamp; first / median / last CTA), and
  * per tile of one attention CTA, clock64 stamps of the first softmax warp and of the
    two MMA-issuing warps.

The stamps lengthen a layer by a few tenths of a microsecond; they are for finding where
the time goes, not for quoting a layer time (bench.py does that on the shipped library).
"""
from __future__ import annotations

import argparse
import ctypes
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
TRACE_LIB = os.path.join(_HERE, "liblvspec_trace.so")
CTA_RECORDS = 4000          # kTraceCtaRecords of lvspec_internal.h


def build_trace_library() -> str:
    from . import build as _build
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = TRACE_LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc, *_build.NVCC_FLAGS, "-DLVSPEC_TRACE", "-I", os.path.join(_ROOT, "include"), "-I", _build.CSRC,
           "-o", tmp, *_build.sources()]
    subprocess.run(cmd, check=True)
    os.replace(tmp, TRACE_LIB)
    return TRACE_LIB


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--layers", type=int, default=6)
    ap.add_argument("--fp8", action="store_true", help="E4M3 cache (lvspec_verify_attention_fp8)")
    ap.add_argument("--n-split", type=int, default=0)
    args = ap.parse_args()
    import torch
    from . import binding, workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("the trace needs a CUDA device")
    lib = binding.load_library(build_trace_library())
    binding._lib = lib                       # contexts created below use the trace build
    lib.lvspec_trace_set_buffer.argtypes = [ctypes.c_void_p]

    cfg = W.CONFIGS[args.config]
    dev = torch.device("cuda", 0)
    B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len
    nl = args.layers
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed)
    rand = lambda *shape: torch.randn(shape, generator=gen, device=dev)

    def cache():
        t = rand(B, Hkv, L, D)
        if not args.fp8:
            return t.to(torch.bfloat16), None
        scale = (t.abs().amax(dim=(2, 3)) / 448.0).clamp_min(1e-30)
        return (t / scale[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8).contiguous(), scale.contiguous()

    qs = [rand(B, g, Hq, D).to(torch.bfloat16) for _ in range(nl)]
    ks, vs = [cache() for _ in range(nl)], [cache() for _ in range(nl)]
    out = torch.empty((B, g, Hq, D), dtype=torch.bfloat16, device=dev)
    mass = torch.empty((B, g, Hq), dtype=torch.float32, device=dev)
    ctx = binding.Context(0)
    shape = binding.attn_shape(B, g, Hq, Hkv, D, L, args.n_split, binding.KERNEL_TCGEN05)
    kv_len = np.full((B,), L, np.int32)
    span = np.tile(np.asarray([cfg.span], np.int32), (B, 1))
    words = torch.zeros(8 + 8 * CTA_RECORDS + 4 * 32 * 8, dtype=torch.int64, device=dev)
    stream = torch.cuda.Stream()

    def calls():
        for l in range(nl):
            if args.fp8:
                ctx.verify_attention_fp8(shape, qs[l], ks[l][0], vs[l][0], ks[l][1], vs[l][1], kv_len, span, out, mass)
            else:
                ctx.verify_attention(shape, qs[l], ks[l][0], vs[l][0], kv_len, span, out, mass)

    with torch.cuda.stream(stream):
        ctx.set_stream(stream.cuda_stream)
        calls()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ctx.set_stream(torch.cuda.current_stream().cuda_stream)
            calls()
        graph.replay()
        torch.cuda.synchronize()
        assert lib.lvspec_trace_set_buffer(words.data_ptr()) == 0
        graph.replay()
        torch.cuda.synchronize()
    ctx.set_stream(stream.cuda_stream)
    print("device status", ctx.device_status(), "| splits", ctx.attention_splits(shape, L),
          "| cache", "E4M3" if args.fp8 else "bf16")
    w = words.cpu().numpy()
    n = min(int(w[0]), CTA_RECORDS)
    R = w[8:8 + n * 8].reshape(n, 8)
    layer_of = {int(q.data_ptr()): i for i, q in enumerate(qs)}
    lay = np.array([layer_of.get(int(x), -1) for x in R[:, 1]])
    t0 = int(R[:, 3].min())
    us = lambda x: round((int(x) - t0) / 1000.0, 2)
    three = lambda col: f"{us(col.min())} / {us(np.median(col))} / {us(col.max())}"
    print("microseconds from the first stamp; first / median / last CTA")
    for l in range(nl):
        A, C = R[(R[:, 0] == 1) & (lay == l)], R[(R[:, 0] == 2) & (lay == l)]
        if len(A):
            print(f"layer {l} attention ({len(A)} CTAs): resident {three(A[:, 3])} | past the prologue {three(A[:, 4])}"
                  f" | last K.Q^T done {three(A[:, 5])} | end {three(A[:, 6])}")
            late = A[np.argsort(A[:, 6])[-4:]]
            print("        last to finish (split, KV head: end, tiles done at): " + "; ".join(
                f"{int(r[2]) % 1000}, {int(r[2]) // 1000 % 1000}: {us(r[6])}, {us(r[5])}" for r in late))
        if len(C):
            print(f"        merge ({len(C)} CTAs): resident {three(C[:, 3])} | attention grid complete {three(C[:, 4])}"
                  f" | end {three(C[:, 6])}")
    T = w[8 + 8 * CTA_RECORDS:].reshape(4, 32, 8)
    if T.any():
        c0 = int(T[T > 0].min())
        print("tiles of attention CTA (split 3, KV head 2) of the last traced layer; cycles from its first stamp")
        print("tile | K.Q^T issuer: waits for K, K there, S^T free, issued | first softmax warp: see below | P.V issuer: waits"
              " for P^T, there, V there, issued | softmax pass of that warp, per four chunks of columns (tiles in turn"
              " only): asks for S^T, has it, probabilities stored")
        print("first softmax warp, all groups on every tile (short streams per CTA, bf16 cache): waits for S^T, there,"
              " exponentials done, group agreed on the guard, P buffer free, P^T handed over")
        print("first softmax warp, groups take the tiles in turn (it has every third tile; long streams, fp8 cache): waits"
              " for S^T, there, P buffer free, exponentials done, its turn came and m stood, P^T handed over")
        rel = lambda a: " ".join(f"{int(x) - c0:6d}" if x else "     -" for x in a)
        for i in range(32):
            if not T[:, i].any():
                break
            print(f"{i:3d} | {rel(T[1, i, :4])} | {rel(T[0, i, :6])} | {rel(T[2, i, :4])} | {rel(T[3, i, :6])}")
    ctx.close()


if __name__ == "__main__":
    main()
