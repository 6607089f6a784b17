"""Seeded synthetic inputs for the LVSpec verify step.

This module only *draws inputs*: normal variates, bf16 rounding of the drawn
values, draft-token planting.  It holds none of the method's arithmetic (no
attention, no softmax, no acceptance rule) and is the one module that both the
CPU oracle's tests and the CUDA path's tests/bench read, so that both sides see
the same bytes.  The only library reduction used is ``numpy.argmax``, and only
to label which synthetic draft tokens are "exact" or "shifted" copies of the
target token; the drafts are then plain inputs to either side.

Shapes follow the video workloads the paper evaluates (Sec. 4, "Target and
Draft Models"; App. "Benchmark Details": 64 or 128 sampled frames): a short
text prefix, a long run of visual tokens, a text remainder, and gamma (= the
paper's K) draft positions in the last slots of the cache.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Tuple

import numpy as np


@dataclasses.dataclass(frozen=True)
class VerifyConfig:
    """One verify-step workload.  ``kv_len`` counts the gamma draft slots."""
    name: str
    layers: int
    batch: int
    gamma: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    kv_len: int
    span: Tuple[int, int]          # [start, end) visual positions
    vocab: int
    mix: Tuple[float, float, float]  # exact / one-position shift / random
    shift_window: int
    lam: float = 0.7               # Sec. 4 "Implementation Details": lambda = 0.7
    seed: int = 0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def kv_bytes_per_layer(self) -> int:
        return 2 * self.batch * self.n_kv_heads * self.kv_len * self.head_dim * 2


CONFIGS: Dict[int, VerifyConfig] = {
    0: VerifyConfig("tiny", 1, 1, 4, 8, 2, 64, 1024, (64, 832), 4096,
                    (0.5, 0.2, 0.3), 1, seed=0),
    1: VerifyConfig("qwen2.5-vl-7b", 28, 1, 8, 28, 4, 128, 16384,
                    (256, 256 + 64 * 196), 152064, (0.5, 0.2, 0.3), 8, seed=1),
    2: VerifyConfig("qwen2.5-vl-32b", 64, 1, 8, 40, 8, 128, 32768,
                    (512, 512 + 128 * 196), 152064, (0.4, 0.25, 0.35), 8, seed=2),
    3: VerifyConfig("llava-onevision-72b", 80, 1, 10, 64, 8, 128, 32768,
                    (512, 512 + 32 * 729), 152064, (0.4, 0.25, 0.35), 10, seed=3),
}


def sweep_config(gamma: int, kv_len: int, batch: int, point: int = 0) -> VerifyConfig:
    """One point of the head-shape sweep (40 query heads, 8 KV heads, D=128,
    75 % of the cache visual, single layer)."""
    vis = (kv_len * 3) // 4
    return VerifyConfig(f"sweep-g{gamma}-l{kv_len}-b{batch}", 1, batch, gamma, 40, 8,
                        128, kv_len, (256, 256 + vis), 152064, (0.4, 0.25, 0.35),
                        gamma, seed=1000 + point)


SWEEP_GAMMAS = (4, 8, 16)
SWEEP_KV_LENS = (4096, 16384, 65536, 131072)
SWEEP_BATCHES = (1, 4, 16)


# ----------------------------------------------------------------------------
# bf16 storage helpers (value <-> bit pattern; round to nearest even)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest even) and return uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    bits = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        bits = np.where(nan, np.uint16(0x7FC0), bits)
    return bits


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32)
            << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# 8-bit storage helper: float32 -> OCP FP8 E4M3 codes (round to nearest even)
# ----------------------------------------------------------------------------
def _e4m3_positive_values() -> np.ndarray:
    """The 127 finite non-negative E4M3 values in code order (0x00..0x7E): exponent
    field 0 is subnormal, (m/8) 2^-6; otherwise (1 + m/8) 2^(e-7); 0x7F is NaN."""
    codes = np.arange(127)
    e, m = codes >> 3, codes & 7
    return np.where(e == 0, (m / 8.0) * 2.0 ** -6, (1.0 + m / 8.0) * 2.0 ** (e.astype(np.float64) - 7.0))


def f32_to_e4m3_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest E4M3 value (ties to the even code, magnitudes
    beyond 448 saturate to 448) and return the uint8 codes.  NaN is not expected."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    vals = _e4m3_positive_values()
    a = np.minimum(np.abs(x).astype(np.float64), 448.0)
    hi = np.clip(np.searchsorted(vals, a, side="left"), 1, 126)     # vals[hi-1] <= a <= vals[hi] (a > 0)
    lo = hi - 1
    d_lo, d_hi = a - vals[lo], vals[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & ((hi & 1) == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return np.where(np.signbit(x), code | np.uint8(0x80), code).astype(np.uint8)


def quantize_cache_e4m3(bits: np.ndarray):
    """A bf16 cache [B, Hkv, L, D] (bit patterns) as an fp8 cache: E4M3 codes of the same
    shape and one fp32 scale per (sequence, KV head), chosen so that the largest magnitude
    of that head maps to 448.  Returns (codes uint8, scale float32 [B, Hkv])."""
    x = bf16_bits_to_f32(bits)
    amax = np.abs(x).max(axis=(2, 3))
    scale = (np.where(amax > 0, amax, 1.0) / np.float32(448.0)).astype(np.float32)
    codes = f32_to_e4m3_bits(x / scale[:, :, None, None])
    return codes, scale


# ----------------------------------------------------------------------------
# attention inputs
# ----------------------------------------------------------------------------
def attention_inputs(cfg: VerifyConfig, layer: int = 0, kv_capacity: int | None = None):
    """Q, K, V of one layer as bf16 bit patterns plus kv_len / span arrays.

    q        uint16 [B, gamma, Hq, D]
    k, v     uint16 [B, Hkv, Lmax, D]   (slots >= kv_len hold finite junk)
    kv_len   int32  [B]
    span     int32  [B, 2]

    Values ~ N(0, 1); keys at visual positions get +0.5 on 8 coordinates chosen
    per KV head by the seeded generator, before rounding to bf16.
    """
    B, g, Hq, Hkv, D, L = (cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads,
                           cfg.head_dim, cfg.kv_len)
    Lmax = L if kv_capacity is None else int(kv_capacity)
    assert Lmax >= L
    rng = np.random.default_rng([cfg.seed, layer, 0xA77])
    q = rng.standard_normal((B, g, Hq, D), dtype=np.float32)
    k = rng.standard_normal((B, Hkv, Lmax, D), dtype=np.float32)
    v = rng.standard_normal((B, Hkv, Lmax, D), dtype=np.float32)
    vs, ve = cfg.span
    for h in range(Hkv):
        dims = rng.choice(D, size=8, replace=False)
        k[:, h, vs:ve, dims] += np.float32(0.5)
    kv_len = np.full((B,), L, dtype=np.int32)
    span = np.tile(np.asarray([[vs, ve]], dtype=np.int32), (B, 1))
    return (f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v), kv_len, span)


# ----------------------------------------------------------------------------
# acceptance inputs
# ----------------------------------------------------------------------------
def accept_inputs(cfg: VerifyConfig, batch: int | None = None):
    """Target logits and draft tokens.

    logits  float32 [B, gamma, V]  ~ N(0, sigma=3) with +8 added at one random
            token id per row
    draft   int32   [B, gamma]     by ``cfg.mix``: equal to the row's largest
            logit id / equal to a neighbouring row's largest logit id (side
            uniform, reflected at the ends) / uniform random id
    """
    B = cfg.batch if batch is None else batch
    g, V = cfg.gamma, cfg.vocab
    rng = np.random.default_rng([cfg.seed, 0xACC])
    logits = rng.standard_normal((B, g, V), dtype=np.float32) * np.float32(3.0)
    planted = rng.integers(0, V, size=(B, g))
    bi, gi = np.meshgrid(np.arange(B), np.arange(g), indexing="ij")
    logits[bi, gi, planted] += np.float32(8.0)
    top = np.argmax(logits, axis=-1)            # labelling only, see module docstring
    kind = rng.choice(3, size=(B, g), p=np.asarray(cfg.mix, dtype=np.float64))
    side = rng.integers(0, 2, size=(B, g)) * 2 - 1
    rand_tok = rng.integers(0, V, size=(B, g))
    draft = np.empty((B, g), dtype=np.int32)
    for b in range(B):
        for i in range(g):
            if kind[b, i] == 0 or g == 1:
                draft[b, i] = top[b, i]
            elif kind[b, i] == 1:
                j = i + side[b, i]
                if j < 0 or j >= g:
                    j = i - side[b, i]
                draft[b, i] = top[b, j]
            else:
                draft[b, i] = rand_tok[b, i]
    return np.ascontiguousarray(logits), draft


def synthetic_mass(cfg: VerifyConfig, batch: int | None = None) -> np.ndarray:
    """A stand-in per-head visual mass in [0, 1], float32 [B, gamma, Hq], for
    exercising the acceptance pass on its own."""
    B = cfg.batch if batch is None else batch
    rng = np.random.default_rng([cfg.seed, 0x3A55])
    return rng.random((B, cfg.gamma, cfg.n_q_heads), dtype=np.float32)


# ----------------------------------------------------------------------------
# hidden states for the paper's own relevance score (Eq. 4)
# ----------------------------------------------------------------------------
def relevance_inputs(cfg: VerifyConfig, n_visual: int | None = None, dim: int | None = None,
                     batch: int | None = None):
    """Synthetic final-layer hidden states (the trained models are not available).

    h_draft   uint16 [B, gamma, d]   bf16 bits, H_D of Eq. 3
    h_visual  uint16 [B, lv, d]      bf16 bits, H_V of Eq. 3

    d defaults to n_q_heads * head_dim and lv to the config's visual span.  Rows
    ~ N(0, 1); every other draft row is pulled towards a small random set of
    "salient" visual rows (weight 0.6), so that its largest similarities stand
    out from the background the way Sec. 3.1 describes for visual-relevant
    tokens; the remaining draft rows stay unrelated to the video.
    """
    B = cfg.batch if batch is None else batch
    lv = cfg.span[1] - cfg.span[0] if n_visual is None else int(n_visual)
    d = cfg.n_q_heads * cfg.head_dim if dim is None else int(dim)
    g = cfg.gamma
    rng = np.random.default_rng([cfg.seed, 0x4E1])
    hv = rng.standard_normal((B, lv, d), dtype=np.float32)
    hd = rng.standard_normal((B, g, d), dtype=np.float32)
    for b in range(B):
        for k in range(0, g, 2):
            n_sal = int(rng.integers(1, 13))
            rows = rng.choice(lv, size=min(n_sal, lv), replace=False)
            hd[b, k] = np.float32(0.8) * hd[b, k] + np.float32(0.6) * hv[b, rows].mean(axis=0) * \
                np.float32(np.sqrt(len(rows)))
    return f32_to_bf16_bits(hd), f32_to_bf16_bits(hv)
