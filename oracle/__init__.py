"""ctypes front end of the fp64 CPU oracle (``zz_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Used by ``tests/``, by the smoke check and by the timed
CPU-baseline leg of ``bench.py``; the CUDA library and its Python binding never
import this package, and this package imports nothing from them.  All arithmetic
lives in the C file; this module only marshals numpy arrays (bf16 values travel as
their 16-bit patterns in ``uint16`` arrays) and keeps per-sequence bookkeeping.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zz_oracle.c")
_LIB = os.path.join(_HERE, "libzz_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent (row, head) units)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    i64, i32, dbl, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
    lib.zzo_visible.argtypes = [i32, i64, i64, i64, i64]
    lib.zzo_visible.restype = i32
    lib.zzo_visible_count.argtypes = [i32, i64, i64, i64]
    lib.zzo_visible_count.restype = i64
    lib.zzo_slot.argtypes = [i64, i64, i64]
    lib.zzo_slot.restype = i64
    lib.zzo_attn_rows.argtypes = [vp, vp, i64, vp, vp, i64, i32, i32, i32, vp, i64, i64, dbl, vp, vp]
    lib.zzo_attn_rows.restype = i32
    lib.zzo_ring_append.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, i32, i64, i64]
    lib.zzo_ring_append.restype = i32
    lib.zzo_full_append.argtypes = [vp, vp, i64, vp, vp, vp, i64, i32, i32]
    lib.zzo_full_append.restype = i32
    lib.zzo_attn_from_slots.argtypes = [vp, i64, vp, vp, vp, i64, i32, i32, i32, vp, i64, i64, dbl, vp]
    lib.zzo_attn_from_slots.restype = i32
    lib.zzo_num_threads.restype = i32
    lib.zzo_layer_mask_enumerate.argtypes = [vp, vp, i32, i32, i32, dbl, vp, vp, vp]
    lib.zzo_layer_mask_enumerate.restype = i32
    lib.zzo_quantile_split.argtypes = [vp, i32, i32, vp]
    lib.zzo_quantile_split.restype = i32
    lib.zzo_e4m3_value.argtypes = [ctypes.c_uint8]
    lib.zzo_e4m3_value.restype = dbl
    lib.zzo_e4m3_encode.argtypes = [dbl]
    lib.zzo_e4m3_encode.restype = ctypes.c_uint8
    lib.zzo_fp8_quantize_rows.argtypes = [vp, i64, i32, vp, vp]
    lib.zzo_fp8_quantize_rows.restype = i32
    lib.zzo_fp8_dequantize_rows.argtypes = [vp, vp, i64, i32, vp]
    lib.zzo_fp8_dequantize_rows.restype = i32
    _lib = lib
    return lib


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 tensors travel as uint16 bit patterns")
    return a


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().zzo_num_threads())


def visible(kind: int, j: int, t: int, S: int, W: int) -> bool:
    return bool(_load().zzo_visible(int(kind), int(j), int(t), int(S), int(W)))


def visible_count(kind: int, t: int, S: int, W: int) -> int:
    return int(_load().zzo_visible_count(int(kind), int(t), int(S), int(W)))


def slot(t: int, S: int, W: int) -> int:
    return int(_load().zzo_slot(int(t), int(S), int(W)))


def attn_rows(q: np.ndarray, t_rows: Sequence[int], k: np.ndarray, v: np.ndarray,
              kv_kind: Sequence[int], S: int, W: int, scale: float,
              return_psum: bool = False):
    """Rows of attention from the full history.

    q [n_rows, Hq, D] (row i is the query at absolute position t_rows[i]),
    k, v [n_hist, Hkv, D], kv_kind [Hkv] (1 retrieval / 0 streaming).
    Returns out [n_rows, Hq, D] float64 (and the per-row softmax weight sums)."""
    q, k, v = _u16(q), _u16(k), _u16(v)
    n_rows, Hq, D = q.shape
    n_hist, Hkv, D2 = k.shape
    assert D == D2 and v.shape == k.shape
    t = np.ascontiguousarray(np.asarray(t_rows, dtype=np.int64))
    assert t.shape == (n_rows,)
    kinds = np.ascontiguousarray(np.asarray(kv_kind, dtype=np.uint8))
    assert kinds.shape == (Hkv,)
    out = np.empty((n_rows, Hq, D), dtype=np.float64)
    psum = np.empty((n_rows, Hq), dtype=np.float64) if return_psum else None
    rc = _load().zzo_attn_rows(_ptr(q), _ptr(t), n_rows, _ptr(k), _ptr(v), n_hist, Hq, Hkv, D,
                               _ptr(kinds), int(S), int(W), float(scale), _ptr(out), _ptr(psum))
    if rc != 0:
        raise ValueError(f"zzo_attn_rows failed: {rc}")
    return (out, psum) if return_psum else out


def attn_from_slots(q: np.ndarray, t: int, store_k: np.ndarray, store_v: np.ndarray,
                    pos: np.ndarray, kv_kind: Sequence[int], S: int, W: int,
                    scale: float) -> np.ndarray:
    """One row from a slot store: q [Hq, D], store_k/v [Hkv, n_slots, D], pos [n_slots]."""
    q, store_k, store_v = _u16(q), _u16(store_k), _u16(store_v)
    Hq, D = q.shape
    Hkv, n_slots, _ = store_k.shape
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    kinds = np.ascontiguousarray(np.asarray(kv_kind, dtype=np.uint8))
    out = np.empty((Hq, D), dtype=np.float64)
    rc = _load().zzo_attn_from_slots(_ptr(q), int(t), _ptr(store_k), _ptr(store_v), _ptr(pos),
                                     n_slots, Hq, Hkv, D, _ptr(kinds), int(S), int(W),
                                     float(scale), _ptr(out))
    if rc != 0:
        raise ValueError(f"zzo_attn_from_slots failed: {rc}")
    return out


def quantile_split(alpha: np.ndarray, n_streaming: int) -> np.ndarray:
    """uint8 mask over the flattened heads: 0 for the n_streaming heads of smallest alpha."""
    a = np.ascontiguousarray(alpha, dtype=np.float64).ravel()
    out = np.zeros(a.size, dtype=np.uint8)
    rc = _load().zzo_quantile_split(_ptr(a), a.size, int(n_streaming), _ptr(out))
    if rc != 0:
        raise ValueError(f"zzo_quantile_split failed: {rc}")
    return out.reshape(np.shape(alpha))


def layer_mask_enumerate(alpha: np.ndarray, head_is_retr: np.ndarray, p: int, omega: float):
    """Exhaustive minimisation of Eq. 5 over all subsets of p streaming layers.
    Returns (layer_is_retrieval uint8 [L], minimum cost, second smallest cost)."""
    a = np.ascontiguousarray(alpha, dtype=np.float64)
    L, H = a.shape
    hr = np.ascontiguousarray(head_is_retr, dtype=np.uint8)
    assert hr.shape == (L, H)
    out = np.zeros(L, dtype=np.uint8)
    best, second = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = _load().zzo_layer_mask_enumerate(_ptr(a), _ptr(hr), L, H, int(p), float(omega), _ptr(out),
                                          ctypes.byref(best), ctypes.byref(second))
    if rc != 0:
        raise ValueError(f"zzo_layer_mask_enumerate failed: {rc}")
    return out, float(best.value), float(second.value)


def e4m3_value(code: int) -> float:
    return float(_load().zzo_e4m3_value(int(code) & 0xFF))


def e4m3_encode(y: float) -> int:
    return int(_load().zzo_e4m3_encode(float(y)))


def fp8_quantize_rows(x: np.ndarray):
    """bf16 bit patterns [..., D] -> (E4M3 codes uint8 [..., D], scale bytes uint8 [...])."""
    x = _u16(x)
    D = x.shape[-1]
    n = x.size // D
    codes = np.empty(x.shape, dtype=np.uint8)
    scale = np.empty(x.shape[:-1], dtype=np.uint8)
    rc = _load().zzo_fp8_quantize_rows(_ptr(x), n, D, _ptr(codes), _ptr(scale))
    if rc != 0:
        raise ValueError(f"zzo_fp8_quantize_rows failed: {rc}")
    return codes, scale


def fp8_dequantize_rows(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """Stored values as float64: value(code) * 2^(scale - 127)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scale = np.ascontiguousarray(scale, dtype=np.uint8)
    D = codes.shape[-1]
    assert codes.shape[:-1] == scale.shape
    out = np.empty(codes.shape, dtype=np.float64)
    rc = _load().zzo_fp8_dequantize_rows(_ptr(codes), _ptr(scale), codes.size // D, D, _ptr(out))
    if rc != 0:
        raise ValueError(f"zzo_fp8_dequantize_rows failed: {rc}")
    return out


def fp8_stored_as_bf16_bits(x: np.ndarray) -> np.ndarray:
    """What rows read back as after FP8 storage, as bf16 bit patterns.  The stored values have four
    significant bits and a power-of-two scale, so they are bf16 numbers exactly (checked)."""
    codes, scale = fp8_quantize_rows(x)
    v = fp8_dequantize_rows(codes, scale)
    f = v.astype(np.float32)
    bits = (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    back = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if not np.array_equal(back, v):
        raise ValueError("a stored FP8 value is not a bf16 number (exponent out of range)")
    return bits


class Fp8Store:
    """Retrieval KV store in FP8: slot j holds the codes and the scale byte of token j."""

    def __init__(self, Hkv: int, D: int, cap: int):
        self.Hkv, self.D, self.cap = Hkv, D, cap
        self.k = np.zeros((Hkv, cap, D), dtype=np.uint8)
        self.v = np.zeros((Hkv, cap, D), dtype=np.uint8)
        self.k_scale = np.zeros((Hkv, cap), dtype=np.uint8)
        self.v_scale = np.zeros((Hkv, cap), dtype=np.uint8)
        self.len = 0

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        C = k_new.shape[0]
        if self.len + C > self.cap:
            raise ValueError("retrieval store overflow")
        for src, codes, scales in ((k_new, self.k, self.k_scale), (v_new, self.v, self.v_scale)):
            c, s = fp8_quantize_rows(np.ascontiguousarray(_u16(src).transpose(1, 0, 2)))
            codes[:, self.len:self.len + C] = c
            scales[:, self.len:self.len + C] = s
        self.len += C


class RingStore:
    """Streaming KV store of one (layer, sequence): S+W slots, simulated token by token."""

    def __init__(self, Hkv: int, D: int, S: int, W: int):
        self.Hkv, self.D, self.S, self.W = Hkv, D, S, W
        self.k = np.zeros((Hkv, S + W, D), dtype=np.uint16)
        self.v = np.zeros((Hkv, S + W, D), dtype=np.uint16)
        self.pos = np.full(S + W, -1, dtype=np.int32)
        self._len = ctypes.c_int64(0)

    @property
    def len(self) -> int:
        return int(self._len.value)

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        k_new, v_new = _u16(k_new), _u16(v_new)
        C = k_new.shape[0]
        assert k_new.shape == (C, self.Hkv, self.D) and v_new.shape == k_new.shape
        rc = _load().zzo_ring_append(_ptr(self.k), _ptr(self.v), _ptr(self.pos),
                                     ctypes.byref(self._len), _ptr(k_new), _ptr(v_new), C,
                                     self.Hkv, self.D, self.S, self.W)
        if rc != 0:
            raise ValueError(f"zzo_ring_append failed: {rc}")


class FullStore:
    """Retrieval KV store of one (layer, sequence): slot j holds token j."""

    def __init__(self, Hkv: int, D: int, cap: int):
        self.Hkv, self.D, self.cap = Hkv, D, cap
        self.k = np.zeros((Hkv, cap, D), dtype=np.uint16)
        self.v = np.zeros((Hkv, cap, D), dtype=np.uint16)
        self._len = ctypes.c_int64(0)

    @property
    def len(self) -> int:
        return int(self._len.value)

    @property
    def pos(self) -> np.ndarray:
        p = np.full(self.cap, -1, dtype=np.int32)
        p[: self.len] = np.arange(self.len, dtype=np.int32)
        return p

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        k_new, v_new = _u16(k_new), _u16(v_new)
        C = k_new.shape[0]
        rc = _load().zzo_full_append(_ptr(self.k), _ptr(self.v), self.cap,
                                     ctypes.byref(self._len), _ptr(k_new), _ptr(v_new), C,
                                     self.Hkv, self.D)
        if rc != 0:
            raise ValueError(f"zzo_full_append failed: {rc}")


class History:
    """Whole K/V history of one (layer, sequence), nothing waived: a growing array."""

    def __init__(self, Hkv: int, D: int):
        self.k = np.zeros((0, Hkv, D), dtype=np.uint16)
        self.v = np.zeros((0, Hkv, D), dtype=np.uint16)

    @property
    def len(self) -> int:
        return int(self.k.shape[0])

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        self.k = np.concatenate([self.k, _u16(k_new)], axis=0)
        self.v = np.concatenate([self.v, _u16(v_new)], axis=0)
