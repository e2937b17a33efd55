"""Shared helpers of the GPU parity tests: an oracle-side mirror of the cache state and
the error metrics.  Tolerances are the ones stated for the method's bf16 path: relative
L2 error <= 5e-3 and max absolute error <= 2e-2 against the fp64 oracle; cache contents,
positions and lengths bit-exact."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2508_12407_b200 import binding, inputs

REL_L2_TOL = 5e-3
MAX_ABS_TOL = 2e-2


def errors(got_bits: np.ndarray, want_f64: np.ndarray):
    got = inputs.bf16_bits_to_f64(got_bits)
    diff = got - want_f64
    rel = float(np.linalg.norm(diff.ravel()) / max(np.linalg.norm(want_f64.ravel()), 1e-30))
    return rel, float(np.max(np.abs(diff))) if diff.size else 0.0


def assert_close(got_bits, want_f64, what=""):
    assert np.all(np.isfinite(inputs.bf16_bits_to_f64(got_bits))), f"{what}: non-finite output"
    rel, mx = errors(got_bits, want_f64)
    assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL, f"{what}: rel_l2={rel:.3e} max_abs={mx:.3e}"
    return rel, mx


class OracleSeq:
    """Oracle state of one (layer, sequence): the whole history plus the simulated stores."""

    def __init__(self, Hkv, D, S, W, cap, kv_kind):
        self.kv_kind = np.asarray(kv_kind, dtype=np.uint8)
        self.S, self.W = S, W
        self.hist = oracle.History(Hkv, D)
        r_heads = [h for h in range(Hkv) if self.kv_kind[h]]
        s_heads = [h for h in range(Hkv) if not self.kv_kind[h]]
        self.r_heads, self.s_heads = r_heads, s_heads
        self.full = oracle.FullStore(len(r_heads), D, cap) if r_heads else None
        self.ring = oracle.RingStore(len(s_heads), D, S, W) if s_heads else None

    def append(self, k, v):
        self.hist.append(k, v)
        if self.full is not None:
            self.full.append(np.ascontiguousarray(k[:, self.r_heads]), np.ascontiguousarray(v[:, self.r_heads]))
        if self.ring is not None:
            self.ring.append(np.ascontiguousarray(k[:, self.s_heads]), np.ascontiguousarray(v[:, self.s_heads]))

    @property
    def len(self):
        return self.hist.len

    def rows(self, q, t_rows, k_all=None, v_all=None, scale=None):
        k = self.hist.k if k_all is None else k_all
        v = self.hist.v if v_all is None else v_all
        return oracle.attn_rows(q, t_rows, k, v, self.kv_kind, self.S, self.W, scale)


def check_export(cache: binding.ZigzagCache, layer: int, seq: int, o: OracleSeq):
    """GPU store contents == oracle stores, byte for byte (K, V, pos, len)."""
    if o.full is not None:
        k, v, pos, ln = cache.export(layer, seq, binding.KIND_RETRIEVAL)
        assert ln == o.full.len
        assert np.array_equal(pos, o.full.pos)
        n = o.full.len
        assert np.array_equal(k[:, :n], o.full.k[:, :n]) and np.array_equal(v[:, :n], o.full.v[:, :n])
    if o.ring is not None:
        k, v, pos, ln = cache.export(layer, seq, binding.KIND_STREAMING)
        assert ln == o.ring.len
        assert np.array_equal(pos, o.ring.pos)
        occ = o.ring.pos >= 0
        assert np.array_equal(k[:, occ], o.ring.k[:, occ]) and np.array_equal(v[:, occ], o.ring.v[:, occ])


def to_dev(bits):
    return binding.bf16_bits_to_tensor(bits, "cuda:0")


def to_bits(t):
    return binding.tensor_to_bf16_bits(t)
