"""Thin ctypes binding of the C ABI declared in ``include/zigzag.h``.

Argument marshalling only: every step of the hot path runs in the library's CUDA
kernels.  PyTorch is used for device memory and streams (plumbing).  There is no CPU
fallback: if the shared library is missing or fails to load, importing symbols from it
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libzigzag_b200.so")

ZZ_OK = 0
ZZ_ERR_INVALID_ARG = -1
ZZ_ERR_UNSUPPORTED = -2
ZZ_ERR_CAPACITY = -3
ZZ_ERR_WORKSPACE = -4
ZZ_ERR_CUDA = -5
ZZ_ERR_TIMEOUT = -6
ZZ_MAX_BATCH = 64
KIND_STREAMING = 0
KIND_RETRIEVAL = 1


class ZZConfig(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32),
        ("batch", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("sink", ctypes.c_int32),
        ("recent", ctypes.c_int32),
        ("max_new_tokens", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("layer_is_retrieval", ctypes.c_void_p),
        ("kvhead_is_retrieval", ctypes.c_void_p),
        ("capacity", ctypes.c_void_p),
        ("retrieval_kv_fp8", ctypes.c_int32),
    ]


class ZigzagError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_str(status)} ({status})")


_lib: Optional[ctypes.CDLL] = None

# every symbol include/zigzag.h declares: name -> (restype, argtypes)
_vp, _i32, _i64, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
_cfgp = ctypes.POINTER(ZZConfig)
SYMBOLS = {
    "zz_version": (_i32, []),
    "zz_status_str": (ctypes.c_char_p, [_i32]),
    "zz_launch_count": (_i64, []),
    "zz_cache_query": (_i32, [_cfgp, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "zz_cache_create": (_i32, [_cfgp, _vp, _sz, _vp, _sz, ctypes.POINTER(_vp)]),
    "zz_cache_query_paged": (_i32, [_cfgp, _i32, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "zz_cache_create_paged": (_i32, [_cfgp, _i32, _vp, _sz, _vp, _sz, ctypes.POINTER(_vp)]),
    "zz_cache_pages": (_i32, [_vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]),
    "zz_cache_reserve": (_i32, [_vp, _i32, _vp]),
    "zz_cache_sync_len": (_i32, [_vp, _vp]),
    "zz_cache_destroy": (_i32, [_vp]),
    "zz_cache_reset": (_i32, [_vp, _i32, _vp]),
    "zz_cache_len": (_i32, [_vp, _i32, _i32, ctypes.POINTER(ctypes.c_int32)]),
    "zz_tune": (_i32, [_vp, ctypes.c_char_p, _i32]),
    "zz_kv_append": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp]),
    "zz_prefill_attn": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "zz_decode_attn": (_i32, [_vp, _i32, _vp, _vp, _vp]),
    "zz_decode_step": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp]),
    "zz_decode_step_all": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "zz_profile_enable": (_i32, [_i32]),
    "zz_profile_read": (_i32, [_i32, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double), _i32]),
    "zz_stage_bytes": (_sz, [_vp, _i64]),
    "zz_decode_step_host": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "zz_decode_step_all_host": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "zz_prefill_host": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "zz_cache_export_shape": (_i32, [_vp, _i32, _i32, _i32, ctypes.POINTER(ctypes.c_int32),
                                     ctypes.POINTER(ctypes.c_int32)]),
    "zz_cache_export": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, ctypes.POINTER(ctypes.c_int32), _vp]),
    "zz_cache_import": (_i32, [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _vp]),
    "zz_cache_export_fp8": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, ctypes.POINTER(ctypes.c_int32), _vp]),
    "zz_cache_import_fp8": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _i32, _vp]),
    "zz_get_last_status": (_i32, [_vp, _vp]),
    "zz_selftest_wait_timeout": (_i32, [_vp, _i32, _vp]),
    "zz_layer_mask_solve": (_i32, [_vp, _i32, _i32, _i32, ctypes.c_double, _vp, _vp, ctypes.POINTER(ctypes.c_double)]),
    "zz_decode_attn_static": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, ctypes.c_float, _vp]),
    "zz_decode_attn_static_limits": (_i32, [ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32),
                                            ctypes.POINTER(_sz)]),
}


def load() -> ctypes.CDLL:
    """Loads the CUDA library (raises if it has not been built: there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          f"`python -m paper_2508_12407_b200.build` (nvcc, sm_100a)")
    lib = ctypes.CDLL(LIB_PATH)
    for name, (res, args) in SYMBOLS.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def status_str(status: int) -> str:
    return load().zz_status_str(int(status)).decode()


def version() -> int:
    return int(load().zz_version())


def launch_count() -> int:
    return int(load().zz_launch_count())


PROF_KINDS = {"append": 0, "decode_retrieval": 1, "decode_streaming": 2, "prefill_retrieval": 3,
              "prefill_streaming": 4, "regroup": 5}


def profile_enable(period: int) -> None:
    """0 = off; n >= 1 = bracket every n-th launch of each kernel class with CUDA events."""
    load().zz_profile_enable(int(period))


def profile_read(reset: bool = True) -> dict:
    """{kernel class: (launches, total device ms)} recorded since the last reset."""
    lib = load()
    out = {}
    names = list(PROF_KINDS.items())
    for i, (name, kind) in enumerate(names):
        n, ms = ctypes.c_int64(0), ctypes.c_double(0.0)
        last = i == len(names) - 1
        rc = lib.zz_profile_read(kind, ctypes.byref(n), ctypes.byref(ms), 1 if (reset and last) else 0)
        if rc != ZZ_OK:
            raise ZigzagError(rc, "zz_profile_read")
        out[name] = (int(n.value), float(ms.value))
    return out


def _check(status: int, what: str) -> None:
    if status != ZZ_OK:
        raise ZigzagError(status, what)


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dptr(t) -> int:
    """Device (or pinned host) pointer of a contiguous torch tensor."""
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensors crossing the C ABI must be contiguous")
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


GUARD_BYTE = 0xA5


class ZigzagCache:
    """Owner of the device arena/workspace (torch allocations) and of the library handle.

    guard_bytes > 0 (a multiple of 256; `ZigzagCache.default_guard_bytes` when not given): the arena
    and the workspace are each allocated with that many extra bytes on either side, filled with a
    pattern; `guards_intact()` tells whether any kernel wrote outside the memory the library was
    given, and `close()` raises if one did."""

    default_guard_bytes = 0

    def __init__(self, n_layers: int, batch: int, n_q_heads: int, n_kv_heads: int, sink: int,
                 recent: int, layer_is_retrieval: Sequence[int], capacity: Sequence[int],
                 max_new_tokens: int, softmax_scale: Optional[float] = None,
                 kvhead_is_retrieval: Optional[np.ndarray] = None, head_dim: int = 128,
                 device: str = "cuda:0", pool_pages: int = 0, guard_bytes: Optional[int] = None,
                 kv_fp8: bool = False):
        import torch
        lib = load()
        self._lib = lib
        self.n_layers, self.batch = n_layers, batch
        self.n_q_heads, self.n_kv_heads, self.head_dim = n_q_heads, n_kv_heads, head_dim
        self.sink, self.recent = sink, recent
        self._kinds = np.ascontiguousarray(np.asarray(layer_is_retrieval, dtype=np.uint8))
        self._cap = np.ascontiguousarray(np.asarray(capacity, dtype=np.int32))
        self._kvk = None
        if kvhead_is_retrieval is not None:
            self._kvk = np.ascontiguousarray(np.asarray(kvhead_is_retrieval, dtype=np.uint8))
            assert self._kvk.size == n_layers * n_kv_heads
        assert self._kinds.shape == (n_layers,) and self._cap.shape == (batch,)
        scale = float(softmax_scale) if softmax_scale is not None else 1.0 / float(np.sqrt(head_dim))
        cfg = ZZConfig(n_layers, batch, n_q_heads, n_kv_heads, head_dim, sink, recent,
                       int(max_new_tokens), scale,
                       self._kinds.ctypes.data, None if self._kvk is None else self._kvk.ctypes.data,
                       self._cap.ctypes.data, 1 if kv_fp8 else 0)
        self.kv_fp8 = bool(kv_fp8)
        self._cfg = cfg
        a, w = ctypes.c_size_t(0), ctypes.c_size_t(0)
        self.pool_pages = int(pool_pages)
        if self.pool_pages:
            _check(lib.zz_cache_query_paged(ctypes.byref(cfg), self.pool_pages, ctypes.byref(a), ctypes.byref(w)),
                   "zz_cache_query_paged")
        else:
            _check(lib.zz_cache_query(ctypes.byref(cfg), ctypes.byref(a), ctypes.byref(w)), "zz_cache_query")
        self.arena_bytes, self.workspace_bytes = int(a.value), int(w.value)
        self.device = torch.device(device)
        g = int(self.default_guard_bytes if guard_bytes is None else guard_bytes)
        assert g >= 0 and g % 256 == 0
        self.guard_bytes = g
        with torch.cuda.device(self.device):
            self._arena_alloc = torch.empty(self.arena_bytes + 2 * g, dtype=torch.uint8, device=self.device)
            self._work_alloc = torch.empty(self.workspace_bytes + 2 * g, dtype=torch.uint8, device=self.device)
            if g:
                for t in (self._arena_alloc, self._work_alloc):
                    t[:g].fill_(GUARD_BYTE)
                    t[t.numel() - g:].fill_(GUARD_BYTE)
            self._arena = self._arena_alloc[g:g + self.arena_bytes]
            self._work = self._work_alloc[g:g + self.workspace_bytes]
            h = ctypes.c_void_p(None)
            if self.pool_pages:
                _check(lib.zz_cache_create_paged(ctypes.byref(cfg), self.pool_pages, self._arena.data_ptr(),
                                                 self.arena_bytes, self._work.data_ptr(), self.workspace_bytes,
                                                 ctypes.byref(h)), "zz_cache_create_paged")
            else:
                _check(lib.zz_cache_create(ctypes.byref(cfg), self._arena.data_ptr(), self.arena_bytes,
                                           self._work.data_ptr(), self.workspace_bytes, ctypes.byref(h)),
                       "zz_cache_create")
        self._h = h

    def guards_intact(self) -> bool:
        """True when no byte of the guard bands around arena and workspace has changed (synchronises)."""
        import torch
        g = self.guard_bytes
        if not g:
            return True
        torch.cuda.synchronize(self.device)
        for t in (self._arena_alloc, self._work_alloc):
            if not bool((t[:g] == GUARD_BYTE).all()) or not bool((t[t.numel() - g:] == GUARD_BYTE).all()):
                return False
        return True

    # -- lifetime ---------------------------------------------------------------------------
    def close(self) -> None:
        if getattr(self, "_h", None):
            intact = self.guards_intact() if self.guard_bytes else True
            self._lib.zz_cache_destroy(self._h)
            self._h = None
            if not intact:
                raise RuntimeError("a kernel wrote outside the arena or the workspace (guard band changed)")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers ------------------------------------------------------------------------------
    def _n_new(self, n_new) -> np.ndarray:
        a = np.ascontiguousarray(np.asarray(n_new, dtype=np.int32))
        assert a.shape == (self.batch,)
        return a

    def len(self, layer: int, seq: int = 0) -> int:
        v = ctypes.c_int32(0)
        _check(self._lib.zz_cache_len(self._h, layer, seq, ctypes.byref(v)), "zz_cache_len")
        return int(v.value)

    def pages(self):
        """(pages in the pool, pages free now); (0, 0) for a cache with contiguous retrieval stores."""
        t, f = ctypes.c_int32(0), ctypes.c_int32(0)
        _check(self._lib.zz_cache_pages(self._h, ctypes.byref(t), ctypes.byref(f)), "zz_cache_pages")
        return int(t.value), int(f.value)

    def reserve(self, extra_tokens: int, stream=None) -> None:
        """Room (and, for a paged cache, pages) for `extra_tokens` more tokens in every sequence."""
        _check(self._lib.zz_cache_reserve(self._h, int(extra_tokens), _stream_ptr(stream)), "zz_cache_reserve")

    def sync_len(self, stream=None) -> None:
        """Host mirror of the lengths := device lengths (after decode steps replayed from a CUDA graph)."""
        _check(self._lib.zz_cache_sync_len(self._h, _stream_ptr(stream)), "zz_cache_sync_len")

    def tune(self, key: str, value: int) -> None:
        _check(self._lib.zz_tune(self._h, key.encode(), int(value)), "zz_tune")

    def reset(self, seq: int = -1, stream=None) -> None:
        _check(self._lib.zz_cache_reset(self._h, seq, _stream_ptr(stream)), "zz_cache_reset")

    # -- the hot path -----------------------------------------------------------------------
    def kv_append(self, layer: int, k, v, n_new, stream=None) -> None:
        nn = self._n_new(n_new)
        _check(self._lib.zz_kv_append(self._h, layer, _dptr(k), _dptr(v), _np_ptr(nn),
                                      _stream_ptr(stream)), "zz_kv_append")

    def prefill_attn(self, layer: int, q, k, v, out, n_new, stream=None) -> None:
        nn = self._n_new(n_new)
        _check(self._lib.zz_prefill_attn(self._h, layer, _dptr(q), _dptr(k), _dptr(v), _dptr(out),
                                         _np_ptr(nn), _stream_ptr(stream)), "zz_prefill_attn")

    def decode_attn(self, layer: int, q, out, stream=None) -> None:
        _check(self._lib.zz_decode_attn(self._h, layer, _dptr(q), _dptr(out), _stream_ptr(stream)),
               "zz_decode_attn")

    def decode_step(self, layer: int, q, k, v, out, stream=None) -> None:
        _check(self._lib.zz_decode_step(self._h, layer, _dptr(q), _dptr(k), _dptr(v), _dptr(out),
                                        _stream_ptr(stream)), "zz_decode_step")

    def decode_step_all(self, q, k, v, out, stream=None) -> None:
        _check(self._lib.zz_decode_step_all(self._h, _dptr(q), _dptr(k), _dptr(v), _dptr(out),
                                            _stream_ptr(stream)), "zz_decode_step_all")

    def stage_bytes(self, n_tokens: int) -> int:
        return int(self._lib.zz_stage_bytes(self._h, int(n_tokens)))

    def decode_step_host(self, layer: int, h_q, h_k, h_v, h_out, d_stage, stream=None) -> None:
        _check(self._lib.zz_decode_step_host(self._h, layer, _dptr(h_q), _dptr(h_k), _dptr(h_v),
                                             _dptr(h_out), _dptr(d_stage), d_stage.numel(),
                                             _stream_ptr(stream)), "zz_decode_step_host")

    def decode_step_all_host(self, h_q, h_k, h_v, h_out, d_stage, stream=None) -> None:
        _check(self._lib.zz_decode_step_all_host(self._h, _dptr(h_q), _dptr(h_k), _dptr(h_v), _dptr(h_out),
                                                 _dptr(d_stage), d_stage.numel(), _stream_ptr(stream)),
               "zz_decode_step_all_host")

    def prefill_host(self, layer: int, h_q, h_k, h_v, h_out, n_new, d_stage, stream=None) -> None:
        nn = self._n_new(n_new)
        _check(self._lib.zz_prefill_host(self._h, layer, _dptr(h_q), _dptr(h_k), _dptr(h_v),
                                         _dptr(h_out), _np_ptr(nn), _dptr(d_stage), d_stage.numel(),
                                         _stream_ptr(stream)), "zz_prefill_host")

    # -- snapshots ------------------------------------------------------------------------------
    def export_shape(self, layer: int, seq: int, kind: int):
        nh, ns = ctypes.c_int32(0), ctypes.c_int32(0)
        _check(self._lib.zz_cache_export_shape(self._h, layer, seq, kind, ctypes.byref(nh),
                                               ctypes.byref(ns)), "zz_cache_export_shape")
        return int(nh.value), int(ns.value)

    def export(self, layer: int, seq: int, kind: int, stream=None):
        """Returns (k, v, pos, len): k, v uint16 [heads_of_kind, slots, 128], pos int32 [slots]."""
        nh, ns = self.export_shape(layer, seq, kind)
        k = np.zeros((nh, ns, self.head_dim), dtype=np.uint16)
        v = np.zeros((nh, ns, self.head_dim), dtype=np.uint16)
        pos = np.zeros(ns, dtype=np.int32)
        ln = ctypes.c_int32(0)
        _check(self._lib.zz_cache_export(self._h, layer, seq, kind, _np_ptr(k), _np_ptr(v), _np_ptr(pos),
                                         ctypes.byref(ln), _stream_ptr(stream)), "zz_cache_export")
        return k, v, pos, int(ln.value)

    def export_fp8(self, layer: int, seq: int, stream=None):
        """FP8 retrieval group: (k codes, v codes uint8 [heads, cap, 128], k scale, v scale uint8 [heads, cap], len)."""
        nh, ns = self.export_shape(layer, seq, KIND_RETRIEVAL)
        k = np.zeros((nh, ns, self.head_dim), dtype=np.uint8)
        v = np.zeros_like(k)
        ks = np.zeros((nh, ns), dtype=np.uint8)
        vs = np.zeros_like(ks)
        ln = ctypes.c_int32(0)
        _check(self._lib.zz_cache_export_fp8(self._h, layer, seq, _np_ptr(k), _np_ptr(v), _np_ptr(ks), _np_ptr(vs),
                                             ctypes.byref(ln), _stream_ptr(stream)), "zz_cache_export_fp8")
        return k, v, ks, vs, int(ln.value)

    def import_fp8(self, layer: int, seq: int, k, v, ks, vs, length: int, stream=None) -> None:
        nh, ns = self.export_shape(layer, seq, KIND_RETRIEVAL)
        k, v = np.ascontiguousarray(k, dtype=np.uint8), np.ascontiguousarray(v, dtype=np.uint8)
        ks, vs = np.ascontiguousarray(ks, dtype=np.uint8), np.ascontiguousarray(vs, dtype=np.uint8)
        assert k.shape == (nh, ns, self.head_dim) and v.shape == k.shape and ks.shape == (nh, ns) and vs.shape == ks.shape
        _check(self._lib.zz_cache_import_fp8(self._h, layer, seq, _np_ptr(k), _np_ptr(v), _np_ptr(ks), _np_ptr(vs),
                                             int(length), _stream_ptr(stream)), "zz_cache_import_fp8")

    def import_(self, layer: int, seq: int, kind: int, k: np.ndarray, v: np.ndarray, pos: np.ndarray,
                length: int, stream=None) -> None:
        nh, ns = self.export_shape(layer, seq, kind)
        k = np.ascontiguousarray(k, dtype=np.uint16)
        v = np.ascontiguousarray(v, dtype=np.uint16)
        pos = np.ascontiguousarray(pos, dtype=np.int32)
        assert k.shape == (nh, ns, self.head_dim) and v.shape == k.shape and pos.shape == (ns,)
        _check(self._lib.zz_cache_import(self._h, layer, seq, kind, _np_ptr(k), _np_ptr(v), _np_ptr(pos),
                                         int(length), _stream_ptr(stream)), "zz_cache_import")

    def last_status(self, stream=None) -> int:
        return int(self._lib.zz_get_last_status(self._h, _stream_ptr(stream)))

    def selftest_wait_timeout(self, max_polls: int = 1000, stream=None) -> None:
        """One warp waits, bounded, on a barrier nothing completes; afterwards last_status() is ZZ_ERR_TIMEOUT."""
        _check(self._lib.zz_selftest_wait_timeout(self._h, int(max_polls), _stream_ptr(stream)),
               "zz_selftest_wait_timeout")


def decode_attn_static(q, k, v, out, lens, softmax_scale: Optional[float] = None, stream=None) -> None:
    """Workspace-free decode attention for callers that cannot allocate device memory.

    q/out [batch, n_q_heads, 128], k/v [batch, n_kv_heads, capacity, 128] (device, bf16),
    lens: host integers.  The scratch is a fixed array inside the library, shared by all calls:
    keep calls that might overlap on the GPU on one stream."""
    B, Hq, D = q.shape
    _, Hkv, cap, _ = k.shape
    hl = np.ascontiguousarray(np.asarray(lens, dtype=np.int32))
    assert hl.shape == (B,) and v.shape == k.shape and out.shape == q.shape
    scale = float(softmax_scale) if softmax_scale is not None else 1.0 / float(np.sqrt(D))
    _check(load().zz_decode_attn_static(_dptr(q), _dptr(k), _dptr(v), _dptr(out), _np_ptr(hl), B, Hq, Hkv,
                                        cap, scale, _stream_ptr(stream)), "zz_decode_attn_static")


def decode_attn_static_limits():
    mb, mr, sb = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_size_t(0)
    _check(load().zz_decode_attn_static_limits(ctypes.byref(mb), ctypes.byref(mr), ctypes.byref(sb)),
           "zz_decode_attn_static_limits")
    return int(mb.value), int(mr.value), int(sb.value)


def layer_mask_solve(alpha: np.ndarray, n_streaming_layers: int, omega: float):
    """Layer-mask solver (Eq. 5): alpha [n_layers, n_heads] -> (layer_is_retrieval uint8 [n_layers],
    head_is_retrieval uint8 [n_layers, n_heads] of the quantile split, minimum cost)."""
    a = np.ascontiguousarray(alpha, dtype=np.float32)
    L, H = a.shape
    layers = np.zeros(L, dtype=np.uint8)
    heads = np.zeros((L, H), dtype=np.uint8)
    cost = ctypes.c_double(0.0)
    _check(load().zz_layer_mask_solve(_np_ptr(a), L, H, int(n_streaming_layers), float(omega), _np_ptr(layers),
                                      _np_ptr(heads), ctypes.byref(cost)), "zz_layer_mask_solve")
    return layers, heads, float(cost.value)


def bf16_bits_to_tensor(bits: np.ndarray, device="cuda:0"):
    """uint16 bit patterns -> torch bf16 tensor on `device` (a byte copy, no arithmetic)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device)


def tensor_to_bf16_bits(t) -> np.ndarray:
    """torch bf16 tensor -> uint16 bit patterns on the host."""
    import torch
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16).copy()
