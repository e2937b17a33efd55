"""Seeded synthetic inputs for the ZigzagAttention inference hot path.

This module only *draws numbers and shapes*; it contains none of the method's
arithmetic (no softmax, no visibility rule, no slot function), so both the CUDA
path and the CPU oracle can be fed from it without sharing any computation.

Every tensor is i.i.d. N(0,1) drawn in fp32 by a counter-based generator
(Philox) keyed by (seed, stream id), rounded to bf16 with round-to-nearest-even,
and handed out as the raw 16-bit patterns (numpy uint16).  The bit patterns are
the contract: the same bytes go to both sides of a parity test.

The workloads restate the five benchmark configurations (a LLaMA-3-8B shaped
attention stack: 32 layers, 32 query / 8 KV heads, head_dim 128; sink 128,
window 256, 50 % streaming layers -- Section 3.1 "Settings" and the paragraph
that fixes sink/window/sparsity in Section 3.3).
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

BASE_SEED = 20250812

# tensor tags used in stream ids
T_Q, T_K, T_V = 1, 2, 3


def _stream_id(*parts: int) -> int:
    """Pack small non-negative integers into one 64-bit stream id (mixed, not summed)."""
    h = 0xCBF29CE484222325
    for p in parts:
        h ^= (int(p) + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
        h = (h * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
        h ^= h >> 29
    return h & 0xFFFFFFFFFFFFFFFF


def _rng(seed: int, *parts: int) -> np.random.Generator:
    key = np.array([seed & 0xFFFFFFFFFFFFFFFF, _stream_id(*parts)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 -> bf16 (round-to-nearest-even), return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    u = b.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def normal_bf16(shape: Sequence[int], seed: int, *stream: int) -> np.ndarray:
    """N(0,1) values as bf16 bit patterns, shape `shape`, keyed by (seed, stream...)."""
    g = _rng(seed, *stream)
    x = g.standard_normal(size=tuple(int(s) for s in shape), dtype=np.float32)
    return f32_to_bf16_bits(x)


def checksum(*arrays: np.ndarray) -> int:
    c = 0
    for a in arrays:
        c = zlib.crc32(np.ascontiguousarray(a).view(np.uint8), c)
    return c & 0xFFFFFFFF


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    sink: int
    recent: int
    n_retrieval_layers: int
    prefill_len: int            # tokens per sequence (0 = caches pre-filled, lengths ragged)
    prefill_chunk: int          # chunk size of the prefill calls (== prefill_len: single shot)
    decode_steps: int
    ragged_lo: int = 0          # inclusive bounds of ragged context lengths
    ragged_hi: int = 0
    mixed_retrieval_kv_heads: int = 0   # >0: comparison arm with this many retrieval KV heads per layer
    seed: int = BASE_SEED

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(np.float64(self.head_dim)))

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


WORKLOADS: Dict[str, Workload] = {
    # tiny parity case: layer 0 retrieval, layer 1 streaming
    "cfg1": Workload("cfg1", 2, 1, 8, 2, 128, 64, 256, 1, 2048, 2048, 16),
    # LLaMA-3-8B shape, 32K single-shot prefill + 256 decode steps, 16 R / 16 S
    "cfg2": Workload("cfg2", 32, 1, 32, 8, 128, 128, 256, 16, 32768, 32768, 256),
    # 128K prefill in 8K chunks + 512 decode steps, 8 R / 24 S, window 1024
    "cfg3": Workload("cfg3", 32, 1, 32, 8, 128, 128, 1024, 8, 131072, 8192, 512),
    # ragged batch-16 decode, lengths U{4096..65536}, caches pre-filled
    "cfg4": Workload("cfg4", 32, 16, 32, 8, 128, 128, 256, 16, 0, 0, 128,
                     ragged_lo=4096, ragged_hi=65536),
    # exclusive vs mixed comparison at 64K, batch 4
    "cfg5": Workload("cfg5", 32, 4, 32, 8, 128, 128, 256, 16, 65536, 65536, 256,
                     mixed_retrieval_kv_heads=4),
}


def layer_kinds(w: Workload) -> np.ndarray:
    """uint8[n_layers], 1 = retrieval layer.  cfg1 is fixed (layer 0 retrieval,
    layer 1 streaming); otherwise a seeded choice of `n_retrieval_layers` layers."""
    kinds = np.zeros(w.n_layers, dtype=np.uint8)
    if w.name == "cfg1":
        kinds[0] = 1
        return kinds
    g = _rng(w.seed, 101, w.n_layers, w.n_retrieval_layers)
    perm = g.permutation(w.n_layers)
    kinds[np.sort(perm[: w.n_retrieval_layers])] = 1
    return kinds


def mixed_kvhead_kinds(w: Workload, n_retrieval_heads: Optional[int] = None) -> np.ndarray:
    """uint8[n_layers, n_kv_heads], 1 = retrieval KV head: a seeded choice of
    `n_retrieval_heads` heads per layer (generally non-contiguous)."""
    r = w.mixed_retrieval_kv_heads if n_retrieval_heads is None else n_retrieval_heads
    out = np.zeros((w.n_layers, w.n_kv_heads), dtype=np.uint8)
    for l in range(w.n_layers):
        g = _rng(w.seed, 102, l, r)
        perm = g.permutation(w.n_kv_heads)
        out[l, np.sort(perm[:r])] = 1
    return out


def ragged_lengths(w: Workload) -> np.ndarray:
    """int32[batch] context lengths: uniform in [ragged_lo, ragged_hi] when ragged,
    else the prefill length for every sequence."""
    if w.ragged_hi > 0:
        g = _rng(w.seed, 103, w.batch)
        return g.integers(w.ragged_lo, w.ragged_hi + 1, size=w.batch).astype(np.int32)
    return np.full(w.batch, w.prefill_len, dtype=np.int32)


def qkv_bf16(w: Workload, layer: int, seq: int, start: int, n_tokens: int,
             n_q_heads: Optional[int] = None, n_kv_heads: Optional[int] = None
             ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Q [n, Hq, D], K [n, Hkv, D], V [n, Hkv, D] bit patterns for tokens
    start..start+n-1 of one (layer, sequence).  Keyed per (layer, tensor, seq, start)
    so the same call always returns the same bytes."""
    hq = w.n_q_heads if n_q_heads is None else n_q_heads
    hkv = w.n_kv_heads if n_kv_heads is None else n_kv_heads
    q = normal_bf16((n_tokens, hq, w.head_dim), w.seed, 7, layer, T_Q, seq, start)
    k = normal_bf16((n_tokens, hkv, w.head_dim), w.seed, 7, layer, T_K, seq, start)
    v = normal_bf16((n_tokens, hkv, w.head_dim), w.seed, 7, layer, T_V, seq, start)
    return q, k, v


def random_chunking(total: int, seed: int, *stream: int, max_chunk: int = 0) -> List[int]:
    """A seeded split of `total` tokens into positive chunk sizes."""
    g = _rng(seed, 104, *stream)
    out: List[int] = []
    left = total
    cap = max_chunk if max_chunk > 0 else max(1, total)
    while left > 0:
        c = int(g.integers(1, min(cap, left) + 1))
        out.append(c)
        left -= c
    return out
