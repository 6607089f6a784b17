"""Thin ctypes binding of liblvspec.so: argument marshalling only.

Every step of the verify path runs in the library's CUDA kernels.  There is no
CPU fallback: if the shared library is missing or no CUDA device is present,
loading or ``Context()`` raises.

Device tensors are passed as objects with ``data_ptr()`` (torch tensors, used
for device memory and streams only) or as raw integer addresses.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblvspec.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
KERNEL_DEFAULT, KERNEL_SIMT, KERNEL_TCGEN05 = 0, 1, 2
DEV_WAIT_EXPIRED, DEV_NAN_LOGIT = 0x1, 0x2
MAX_BATCH, MAX_ROWS, MAX_GAMMA = 128, 128, 64

EXPORTS = (
    "lvspec_create", "lvspec_destroy", "lvspec_set_stream", "lvspec_device_status",
    "lvspec_last_error", "lvspec_status_string", "lvspec_launch_count",
    "lvspec_attention_splits", "lvspec_attention_splits_fp8", "lvspec_verify_attention", "lvspec_verify_attention_host",
    "lvspec_loose_accept", "lvspec_loose_accept_ex", "lvspec_loose_accept_host",
    "lvspec_loose_accept_static", "lvspec_row_inv_norms", "lvspec_visual_relevance",
    "lvspec_selftest_wait_expiry", "lvspec_loose_accept_emit",
    "lvspec_verify_attention_tree", "lvspec_select_branch", "lvspec_verify_attention_paged",
    "lvspec_verify_attention_spans", "lvspec_last_device_status",
    "lvspec_attention_workspace_bytes", "lvspec_accept_workspace_bytes",
    "lvspec_relevance_workspace_bytes", "lvspec_workspace_capacity", "lvspec_reserve",
    "lvspec_verify_attention_fp8", "lvspec_verify_attention_strided",
)


class AttnShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("batch", "gamma", "n_q_heads", "n_kv_heads", "head_dim", "kv_capacity",
                 "n_split", "kernel")]


class KvStrides(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int64), ("head", ctypes.c_int64), ("position", ctypes.c_int64)]


class Thresholds(ctypes.Structure):
    _fields_ = [("lam", ctypes.c_double), ("n_loose", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


class LvspecError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"lvspec status {status}: {text}")
        self.status = status


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads liblvspec.so; raises OSError when it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise OSError(f"{path} not found: build it with "
                      "`python -m paper_2604_05650_b200.build` (needs nvcc)")
    lib = ctypes.CDLL(path)
    vp, i32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64
    S = ctypes.POINTER(AttnShape)
    T = ctypes.POINTER(Thresholds)
    lib.lvspec_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
    lib.lvspec_destroy.argtypes = [vp]
    lib.lvspec_set_stream.argtypes = [vp, vp]
    lib.lvspec_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.lvspec_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    sz = ctypes.c_size_t
    lib.lvspec_attention_workspace_bytes.argtypes = [vp, S, i32]
    lib.lvspec_attention_workspace_bytes.restype = sz
    lib.lvspec_accept_workspace_bytes.argtypes = [vp, i32, i32, i32]
    lib.lvspec_accept_workspace_bytes.restype = sz
    lib.lvspec_relevance_workspace_bytes.argtypes = [vp, i32, i32, i32, i32]
    lib.lvspec_relevance_workspace_bytes.restype = sz
    lib.lvspec_workspace_capacity.argtypes = [vp]
    lib.lvspec_workspace_capacity.restype = sz
    lib.lvspec_reserve.argtypes = [vp, sz]
    lib.lvspec_last_error.argtypes = [vp]
    lib.lvspec_last_error.restype = ctypes.c_char_p
    lib.lvspec_status_string.argtypes = [ctypes.c_int]
    lib.lvspec_status_string.restype = ctypes.c_char_p
    lib.lvspec_launch_count.argtypes = [vp]
    lib.lvspec_launch_count.restype = u64
    lib.lvspec_attention_splits.argtypes = [vp, S, i32]
    lib.lvspec_attention_splits.restype = i32
    lib.lvspec_attention_splits_fp8.argtypes = [vp, S, i32]
    lib.lvspec_attention_splits_fp8.restype = i32
    lib.lvspec_verify_attention.argtypes = [vp, S, vp, vp, vp, vp, vp, vp, vp]
    lib.lvspec_verify_attention_host.argtypes = [vp, S, vp, vp, vp, vp, vp, vp, vp]
    lib.lvspec_verify_attention_fp8.argtypes = [vp, S, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    KS = ctypes.POINTER(KvStrides)
    lib.lvspec_verify_attention_strided.argtypes = [vp, S, KS, KS, vp, vp, vp, vp, vp, vp, vp]
    lib.lvspec_loose_accept.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, T, i32, vp]
    lib.lvspec_loose_accept_ex.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, T, i32, vp, vp, vp]
    lib.lvspec_loose_accept_host.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, T, i32, vp]
    lib.lvspec_selftest_wait_expiry.argtypes = [vp, i32]
    lib.lvspec_verify_attention_tree.argtypes = [vp, S, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.lvspec_select_branch.argtypes = [vp, i32, i32, vp, vp, vp]
    lib.lvspec_verify_attention_paged.argtypes = [vp, S, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.lvspec_verify_attention_spans.argtypes = [vp, S, vp, vp, vp, vp, i32, vp, vp, vp]
    lib.lvspec_loose_accept_emit.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, T, i32, vp, vp, vp, vp, vp]
    lib.lvspec_row_inv_norms.argtypes = [vp, ctypes.c_int64, i32, vp, vp]
    lib.lvspec_visual_relevance.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, i32, vp]
    lib.lvspec_loose_accept_static.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, T, i32, vp,
                                               ctypes.c_char_p, ctypes.c_size_t]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int and name not in ("lvspec_attention_splits", "lvspec_attention_splits_fp8"):
            fn.restype = ctypes.c_int
    if path == LIB_PATH:
        _lib = lib
    return lib


def _addr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return int(x.data_ptr())


def _i32(a: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


class Context:
    """One library context on one CUDA device (``lvspec_create``)."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        h = ctypes.c_void_p()
        st = self._lib.lvspec_create(ctypes.byref(h), int(device))
        if st != OK:
            raise LvspecError(st, self._lib.lvspec_last_error(None).decode())
        self._h = h

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.lvspec_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int) -> None:
        if st != OK:
            raise LvspecError(st, self._lib.lvspec_last_error(self._h).decode())

    def set_stream(self, stream) -> None:
        """``stream``: a raw cudaStream_t address, or an object with ``cuda_stream``."""
        s = getattr(stream, "cuda_stream", stream)
        self._check(self._lib.lvspec_set_stream(self._h, ctypes.c_void_p(int(s) if s else 0)))

    def device_status(self) -> int:
        flags = ctypes.c_uint32(0)
        st = self._lib.lvspec_device_status(self._h, ctypes.byref(flags))
        if st not in (OK, ERR_TIMEOUT):
            self._check(st)
        return int(flags.value)

    def device_status_code(self):
        """(status code, flags) of ``lvspec_device_status``: the code is ERR_TIMEOUT
        when a bounded device-side wait ran out since the last call."""
        flags = ctypes.c_uint32(0)
        st = self._lib.lvspec_device_status(self._h, ctypes.byref(flags))
        return int(st), int(flags.value)

    def selftest_wait_expiry(self, limit_ms: int = 5) -> None:
        self._check(self._lib.lvspec_selftest_wait_expiry(self._h, int(limit_ms)))

    # -- scratch memory --------------------------------------------------------------
    def attention_workspace_bytes(self, shape: AttnShape, max_kv_len: int) -> int:
        return int(self._lib.lvspec_attention_workspace_bytes(self._h, ctypes.byref(shape), int(max_kv_len)))

    def accept_workspace_bytes(self, batch, gamma, vocab) -> int:
        return int(self._lib.lvspec_accept_workspace_bytes(self._h, int(batch), int(gamma), int(vocab)))

    def relevance_workspace_bytes(self, batch, gamma, n_visual, dim) -> int:
        return int(self._lib.lvspec_relevance_workspace_bytes(self._h, int(batch), int(gamma), int(n_visual),
                                                              int(dim)))

    def workspace_capacity(self) -> int:
        return int(self._lib.lvspec_workspace_capacity(self._h))

    def reserve(self, workspace_bytes: int) -> None:
        self._check(self._lib.lvspec_reserve(self._h, int(workspace_bytes)))

    def launch_count(self) -> int:
        return int(self._lib.lvspec_launch_count(self._h))

    def attention_splits(self, shape: AttnShape, max_kv_len: int, fp8: bool = False) -> int:
        fn = self._lib.lvspec_attention_splits_fp8 if fp8 else self._lib.lvspec_attention_splits
        return int(fn(self._h, ctypes.byref(shape), int(max_kv_len)))

    # -- lvspec_verify_attention ------------------------------------------------
    def verify_attention(self, shape: AttnShape, q, k_cache, v_cache, kv_len, visual_span,
                         out, visual_mass) -> None:
        kv_len, span = _i32(kv_len), _i32(visual_span)
        if shape.batch >= 1 and (kv_len.size != shape.batch or span.size != 2 * shape.batch):
            raise ValueError("kv_len needs B entries and visual_span B pairs")
        self._check(self._lib.lvspec_verify_attention(
            self._h, ctypes.byref(shape), _addr(q), _addr(k_cache), _addr(v_cache),
            kv_len.ctypes.data, span.ctypes.data, _addr(out), _addr(visual_mass)))

    def verify_attention_strided(self, shape: AttnShape, k_strides, v_strides, q, k_cache, v_cache, kv_len,
                                 visual_span, out, visual_mass) -> None:
        """k_strides / v_strides: (batch, head, position) strides in elements."""
        kv_len, span = _i32(kv_len), _i32(visual_span)
        if shape.batch >= 1 and (kv_len.size != shape.batch or span.size != 2 * shape.batch):
            raise ValueError("kv_len needs B entries and visual_span B pairs")
        ks, vs = KvStrides(*[int(x) for x in k_strides]), KvStrides(*[int(x) for x in v_strides])
        self._check(self._lib.lvspec_verify_attention_strided(
            self._h, ctypes.byref(shape), ctypes.byref(ks), ctypes.byref(vs), _addr(q), _addr(k_cache),
            _addr(v_cache), kv_len.ctypes.data, span.ctypes.data, _addr(out), _addr(visual_mass)))

    def verify_attention_fp8(self, shape: AttnShape, q, k_cache, v_cache, k_scale, v_scale, kv_len,
                             visual_span, out, visual_mass) -> None:
        """k_cache / v_cache: device uint8 E4M3 codes [B, Hkv, Lmax, D]; k_scale / v_scale:
        device fp32 [B, Hkv]."""
        kv_len, span = _i32(kv_len), _i32(visual_span)
        if shape.batch >= 1 and (kv_len.size != shape.batch or span.size != 2 * shape.batch):
            raise ValueError("kv_len needs B entries and visual_span B pairs")
        self._check(self._lib.lvspec_verify_attention_fp8(
            self._h, ctypes.byref(shape), _addr(q), _addr(k_cache), _addr(v_cache), _addr(k_scale),
            _addr(v_scale), kv_len.ctypes.data, span.ctypes.data, _addr(out), _addr(visual_mass)))

    def verify_attention_tree(self, shape: AttnShape, n_branches, q, k_cache, v_cache, kv_len, visual_span,
                              out, visual_mass) -> None:
        kv_len, span = _i32(kv_len), _i32(visual_span)
        if shape.batch >= 1 and (kv_len.size != shape.batch or span.size != 2 * shape.batch):
            raise ValueError("kv_len needs B entries and visual_span B pairs")
        self._check(self._lib.lvspec_verify_attention_tree(
            self._h, ctypes.byref(shape), int(n_branches), _addr(q), _addr(k_cache), _addr(v_cache),
            kv_len.ctypes.data, span.ctypes.data, _addr(out), _addr(visual_mass)))

    def verify_attention_paged(self, shape: AttnShape, page_size, n_pages, q, k_pool, v_pool, block_table,
                               kv_len, visual_span, out, visual_mass) -> None:
        """k_pool / v_pool: device [n_pages, Hkv, page_size, D]; block_table: device int32
        [B, kv_capacity / page_size]; kv_len, visual_span: host."""
        kv_len, span = _i32(kv_len), _i32(visual_span)
        if shape.batch >= 1 and (kv_len.size != shape.batch or span.size != 2 * shape.batch):
            raise ValueError("kv_len needs B entries and visual_span B pairs")
        self._check(self._lib.lvspec_verify_attention_paged(
            self._h, ctypes.byref(shape), int(page_size), int(n_pages), _addr(q), _addr(k_pool),
            _addr(v_pool), _addr(block_table), kv_len.ctypes.data, span.ctypes.data, _addr(out),
            _addr(visual_mass)))

    def verify_attention_spans(self, shape: AttnShape, q, k_cache, v_cache, kv_len, visual_spans,
                               out, visual_mass) -> None:
        """visual_spans: host int32 [B, n_spans, 2], sorted and disjoint per sequence."""
        kv_len = _i32(kv_len)
        spans = np.ascontiguousarray(np.asarray(visual_spans, dtype=np.int32))
        if spans.ndim != 3 or spans.shape[0] != shape.batch or spans.shape[2] != 2 or kv_len.size != shape.batch:
            raise ValueError("visual_spans needs shape [B, n_spans, 2] and kv_len B entries")
        self._check(self._lib.lvspec_verify_attention_spans(
            self._h, ctypes.byref(shape), _addr(q), _addr(k_cache), _addr(v_cache), kv_len.ctypes.data,
            int(spans.shape[1]), spans.ctypes.data, _addr(out), _addr(visual_mass)))

    def select_branch(self, batch, n_branches, accept_len, best_branch, best_len) -> None:
        self._check(self._lib.lvspec_select_branch(self._h, int(batch), int(n_branches), _addr(accept_len),
                                                   _addr(best_branch), _addr(best_len)))

    def verify_attention_host(self, shape: AttnShape, q, k_cache, v_cache, kv_len, visual_span,
                              out, visual_mass) -> None:
        kv_len, span = _i32(kv_len), _i32(visual_span)
        if shape.batch >= 1 and (kv_len.size != shape.batch or span.size != 2 * shape.batch):
            raise ValueError("kv_len needs B entries and visual_span B pairs")
        self._check(self._lib.lvspec_verify_attention_host(
            self._h, ctypes.byref(shape), _addr(q), _addr(k_cache), _addr(v_cache),
            kv_len.ctypes.data, span.ctypes.data, _addr(out), _addr(visual_mass)))

    # -- lvspec_loose_accept ----------------------------------------------------
    def loose_accept(self, batch, gamma, vocab, n_mass_heads, target_logits, draft_tokens,
                     visual_mass, accept_len, shift_window, lam: float = 0.7,
                     n_loose: int = -1, target_tokens=None, accepted=None) -> None:
        th = Thresholds(float(lam), int(n_loose), 0)
        self._check(self._lib.lvspec_loose_accept_ex(
            self._h, batch, gamma, vocab, n_mass_heads, _addr(target_logits),
            _addr(draft_tokens), _addr(visual_mass), ctypes.byref(th), int(shift_window),
            _addr(accept_len), _addr(target_tokens), _addr(accepted)))

    # -- the paper's own relevance score (Eq. 4) ---------------------------------
    def row_inv_norms(self, rows, dim, x, inv_norm) -> None:
        self._check(self._lib.lvspec_row_inv_norms(self._h, int(rows), int(dim), _addr(x), _addr(inv_norm)))

    def visual_relevance(self, batch, gamma, n_visual, dim, h_draft, h_visual, visual_inv_norm,
                         top_n, relevance) -> None:
        self._check(self._lib.lvspec_visual_relevance(
            self._h, batch, gamma, n_visual, dim, _addr(h_draft), _addr(h_visual),
            _addr(visual_inv_norm), int(top_n), _addr(relevance)))

    def loose_accept_emit(self, batch, gamma, vocab, n_mass_heads, target_logits, draft_tokens,
                          visual_mass, accept_len, emitted, n_emitted, shift_window, lam: float = 0.7,
                          n_loose: int = -1, kv_len=None, new_kv_len=None) -> None:
        th = Thresholds(float(lam), int(n_loose), 0)
        self._check(self._lib.lvspec_loose_accept_emit(
            self._h, batch, gamma, vocab, n_mass_heads, _addr(target_logits), _addr(draft_tokens),
            _addr(visual_mass), ctypes.byref(th), int(shift_window), _addr(kv_len), _addr(accept_len),
            _addr(emitted), _addr(n_emitted), _addr(new_kv_len)))

    def loose_accept_host(self, batch, gamma, vocab, n_mass_heads, target_logits, draft_tokens,
                          visual_mass, accept_len, shift_window, lam: float = 0.7,
                          n_loose: int = -1) -> None:
        th = Thresholds(float(lam), int(n_loose), 0)
        self._check(self._lib.lvspec_loose_accept_host(
            self._h, batch, gamma, vocab, n_mass_heads, _addr(target_logits),
            _addr(draft_tokens), _addr(visual_mass), ctypes.byref(th), int(shift_window),
            _addr(accept_len)))


STATIC_MAX_ROWS = 1024


def loose_accept_static(stream, batch, gamma, vocab, n_mass_heads, target_logits, draft_tokens,
                        visual_mass, accept_len, shift_window, lam: float = 0.7,
                        n_loose: int = -1) -> None:
    """``lvspec_loose_accept_static``: the acceptance pass for callers that may
    not allocate device memory.  No context; runs on the current CUDA device,
    on ``stream`` (raw cudaStream_t address, an object with ``cuda_stream``, or
    None).  Raises ``LvspecError`` with the library's own text on failure."""
    lib = load_library()
    s = getattr(stream, "cuda_stream", stream)
    th = Thresholds(float(lam), int(n_loose), 0)
    text = ctypes.create_string_buffer(256)
    st = lib.lvspec_loose_accept_static(
        ctypes.c_void_p(int(s) if s else 0), batch, gamma, vocab, n_mass_heads,
        _addr(target_logits), _addr(draft_tokens), _addr(visual_mass), ctypes.byref(th),
        int(shift_window), _addr(accept_len), text, len(text))
    if st != OK:
        raise LvspecError(st, text.value.decode())


HAVE_TCGEN05 = True


def available_kernels():
    """Kernel selectors this build of the library accepts."""
    return [KERNEL_SIMT, KERNEL_TCGEN05] if HAVE_TCGEN05 else [KERNEL_SIMT]


def attn_shape(batch, gamma, n_q_heads, n_kv_heads, head_dim, kv_capacity, n_split=0,
               kernel=KERNEL_DEFAULT) -> AttnShape:
    return AttnShape(batch, gamma, n_q_heads, n_kv_heads, head_dim, kv_capacity, n_split, kernel)
