"""ctypes binding of the C oracle (``lvspec_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Tests, the smoke check and the benchmark's
CPU-baseline leg may import this; the product package never does.  The library
is compiled with gcc on first use (``build()``); arrays go in and out as numpy.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lvspec_oracle.c")
_LIB = os.path.join(_HERE, "liblvspec_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source."""
    with _lock:
        stale = (not os.path.exists(_LIB)
                 or os.path.getmtime(_LIB) < os.path.getmtime(_SRC))
        if force or stale:
            tmp = _LIB + f".{os.getpid()}.tmp"
            subprocess.run(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-std=c99",
                            "-o", tmp, _SRC, "-lm"], check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.c_void_p
        i = ctypes.c_int
        lib.lvspec_oracle_verify_attention.argtypes = [p, p, p, p, p, i, i, i, i, i, i, p, p, p]
        lib.lvspec_oracle_verify_attention.restype = None
        lib.lvspec_oracle_verify_attention_tree.argtypes = [p, p, p, p, p, i, i, i, i, i, i, i, p, p, p]
        lib.lvspec_oracle_verify_attention_tree.restype = None
        lib.lvspec_oracle_verify_attention_fp8.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, i, p, p]
        lib.lvspec_oracle_verify_attention_fp8.restype = None
        lib.lvspec_oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
        lib.lvspec_oracle_e4m3_decode.restype = ctypes.c_double
        lib.lvspec_oracle_select_branch.argtypes = [p, i, i, p, p]
        lib.lvspec_oracle_select_branch.restype = None
        lib.lvspec_oracle_loose_accept.argtypes = [p, p, p, i, i, i, i, i, i, p, p, p]
        lib.lvspec_oracle_loose_accept.restype = None
        lib.lvspec_oracle_visual_relevance.argtypes = [p, p, i, i, i, i, i, p, p]
        lib.lvspec_oracle_visual_relevance.restype = None
        lib.lvspec_oracle_emit.argtypes = [p, p, p, p, i, i, p, p, p]
        lib.lvspec_oracle_emit.restype = None
        lib.lvspec_oracle_n_loose.argtypes = [ctypes.c_double, i]
        lib.lvspec_oracle_n_loose.restype = i
        try:
            omp = ctypes.CDLL("libgomp.so.1")
            omp.omp_get_max_threads.restype = i
            omp.omp_set_num_threads.argtypes = [i]
            lib._omp = omp
        except OSError:  # pragma: no cover
            lib._omp = None
        _lib = lib
    return _lib


def max_threads() -> int:
    lib = _load()
    return int(lib._omp.omp_get_max_threads()) if lib._omp else 1


def set_threads(n: int) -> None:
    lib = _load()
    if lib._omp:
        lib._omp.omp_set_num_threads(int(n))


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def verify_attention(q, k, v, kv_len, span, return_probs: bool = False, branch_len: int = 0):
    """q [B,gamma,Hq,D], k/v [B,Hkv,Lmax,D] as uint16 bf16 bit patterns;
    kv_len int32 [B]; span int32 [B,2].  Returns (out, mass[, probs]) in fp64.
    ``branch_len`` > 0: the gamma draft slots are gamma / branch_len tree branches."""
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.uint16)
    k = np.ascontiguousarray(k, dtype=np.uint16)
    v = np.ascontiguousarray(v, dtype=np.uint16)
    kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
    span = np.ascontiguousarray(span, dtype=np.int32)
    B, gamma, Hq, D = q.shape
    Bk, Hkv, Lmax, Dk = k.shape
    assert (Bk, Dk) == (B, D) and v.shape == k.shape and Hq % Hkv == 0
    assert kv_len.shape == (B,) and span.shape == (B, 2)
    assert (kv_len >= gamma).all() and (kv_len <= Lmax).all()
    out = np.empty((B, gamma, Hq, D), dtype=np.float64)
    mass = np.empty((B, gamma, Hq), dtype=np.float64)
    probs = np.empty((B, gamma, Hq, Lmax), dtype=np.float64) if return_probs else None
    bl = gamma if branch_len <= 0 else int(branch_len)
    assert gamma % bl == 0
    lib.lvspec_oracle_verify_attention_tree(_ptr(q), _ptr(k), _ptr(v), _ptr(kv_len), _ptr(span),
                                            B, gamma, bl, Hq, Hkv, D, Lmax, _ptr(out), _ptr(mass),
                                            _ptr(probs))
    return (out, mass, probs) if return_probs else (out, mass)


def e4m3_decode(code: int) -> float:
    """Value of one E4M3 code (0..255)."""
    return float(_load().lvspec_oracle_e4m3_decode(int(code) & 0xFF))


def verify_attention_fp8(q, k8, v8, k_scale, v_scale, kv_len, span):
    """q [B,gamma,Hq,D] uint16 bf16 bits; k8/v8 [B,Hkv,Lmax,D] uint8 E4M3 codes;
    k_scale/v_scale fp32 [B,Hkv]; kv_len int32 [B]; span int32 [B,2].
    Returns (out, mass) in fp64."""
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.uint16)
    k8 = np.ascontiguousarray(k8, dtype=np.uint8)
    v8 = np.ascontiguousarray(v8, dtype=np.uint8)
    k_scale = np.ascontiguousarray(k_scale, dtype=np.float32)
    v_scale = np.ascontiguousarray(v_scale, dtype=np.float32)
    kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
    span = np.ascontiguousarray(span, dtype=np.int32)
    B, gamma, Hq, D = q.shape
    Bk, Hkv, Lmax, Dk = k8.shape
    assert (Bk, Dk) == (B, D) and v8.shape == k8.shape and Hq % Hkv == 0
    assert k_scale.shape == (B, Hkv) and v_scale.shape == (B, Hkv)
    assert kv_len.shape == (B,) and span.shape == (B, 2)
    assert (kv_len >= gamma).all() and (kv_len <= Lmax).all()
    out = np.empty((B, gamma, Hq, D), dtype=np.float64)
    mass = np.empty((B, gamma, Hq), dtype=np.float64)
    lib.lvspec_oracle_verify_attention_fp8(_ptr(q), _ptr(k8), _ptr(v8), _ptr(k_scale), _ptr(v_scale),
                                           _ptr(kv_len), _ptr(span), B, gamma, Hq, Hkv, D, Lmax,
                                           _ptr(out), _ptr(mass))
    return out, mass


def loose_accept(logits, draft, mass, n_loose: int, window: int):
    """logits fp32 [B,gamma,V]; draft int32 [B,gamma]; mass fp32 [B,gamma,Hm].
    Returns (accept_len int32 [B], target int32 [B,gamma], acc uint8 [B,gamma])."""
    lib = _load()
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    draft = np.ascontiguousarray(draft, dtype=np.int32)
    mass = np.ascontiguousarray(mass, dtype=np.float32)
    B, gamma, V = logits.shape
    assert draft.shape == (B, gamma) and mass.shape[:2] == (B, gamma) and mass.ndim == 3
    Hm = mass.shape[2]
    accept_len = np.empty((B,), dtype=np.int32)
    target = np.empty((B, gamma), dtype=np.int32)
    acc = np.empty((B, gamma), dtype=np.uint8)
    lib.lvspec_oracle_loose_accept(_ptr(logits), _ptr(draft), _ptr(mass), B, gamma, V, Hm,
                                   int(n_loose), int(window), _ptr(accept_len), _ptr(target),
                                   _ptr(acc))
    return accept_len, target, acc


def n_loose(lam: float, gamma: int) -> int:
    return int(_load().lvspec_oracle_n_loose(float(lam), int(gamma)))


def visual_relevance(h_draft, h_visual, top_n: int, return_cosines: bool = False):
    """h_draft [B,K,d], h_visual [B,lv,d] as uint16 bf16 bit patterns.  Returns the
    paper's relevance score A_s, fp64 [B,K] (and the cosines [B,K,lv])."""
    lib = _load()
    h_draft = np.ascontiguousarray(h_draft, dtype=np.uint16)
    h_visual = np.ascontiguousarray(h_visual, dtype=np.uint16)
    B, K, d = h_draft.shape
    Bv, lv, dv = h_visual.shape
    assert (Bv, dv) == (B, d)
    rel = np.empty((B, K), dtype=np.float64)
    cos = np.empty((B, K, lv), dtype=np.float64) if return_cosines else None
    lib.lvspec_oracle_visual_relevance(_ptr(h_draft), _ptr(h_visual), B, K, lv, d, int(top_n),
                                       _ptr(rel), _ptr(cos))
    return (rel, cos) if return_cosines else rel


def emit(draft, target, accept_len, kv_len=None):
    """Tokens a verify step hands back: (emitted int32 [B,gamma] with -1 padding,
    n_emitted int32 [B], new_kv_len int32 [B] or None)."""
    lib = _load()
    draft = np.ascontiguousarray(draft, dtype=np.int32)
    target = np.ascontiguousarray(target, dtype=np.int32)
    accept_len = np.ascontiguousarray(accept_len, dtype=np.int32)
    B, gamma = draft.shape
    emitted = np.empty((B, gamma), dtype=np.int32)
    n_emitted = np.empty((B,), dtype=np.int32)
    kv = None if kv_len is None else np.ascontiguousarray(kv_len, dtype=np.int32)
    new_kv = None if kv is None else np.empty((B,), dtype=np.int32)
    lib.lvspec_oracle_emit(_ptr(draft), _ptr(target), _ptr(accept_len), _ptr(kv), B, gamma,
                           _ptr(emitted), _ptr(n_emitted), _ptr(new_kv))
    return emitted, n_emitted, new_kv


def select_branch(accept_len):
    """accept_len int32 [B,R] -> (best_branch int32 [B], best_len int32 [B])."""
    lib = _load()
    a = np.ascontiguousarray(accept_len, dtype=np.int32)
    B, R = a.shape
    bb = np.empty((B,), dtype=np.int32)
    bl = np.empty((B,), dtype=np.int32)
    lib.lvspec_oracle_select_branch(_ptr(a), B, R, _ptr(bb), _ptr(bl))
    return bb, bl
