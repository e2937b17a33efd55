"""FP8 retrieval stores on the GPU against the oracle: the stored bytes (codes and scale bytes) bit
for bit, and attention over the stored values within the usual tolerances -- the oracle is given
the stored values (exactly, as bf16 numbers), so the tolerances measure the kernels, not the
quantisation.  The distance to attention over the original bf16 rows is printed, not asserted."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_12407_b200 import binding, build, inputs
from zz_testlib import assert_close, errors, to_bits, to_dev

pytestmark = pytest.mark.gpu
D = 128


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


class Fp8Seq:
    """Oracle state of one (layer, sequence) of an FP8 cache."""

    def __init__(self, Hkv, S, W, cap, kv_kind):
        self.kind = np.asarray(kv_kind, dtype=np.uint8)
        self.S, self.W, self.Hkv = S, W, Hkv
        self.r_heads = [h for h in range(Hkv) if self.kind[h]]
        self.s_heads = [h for h in range(Hkv) if not self.kind[h]]
        self.raw_k = np.zeros((0, Hkv, D), np.uint16); self.raw_v = np.zeros((0, Hkv, D), np.uint16)
        self.st_k = np.zeros((0, Hkv, D), np.uint16); self.st_v = np.zeros((0, Hkv, D), np.uint16)   # as stored
        self.fp8 = oracle.Fp8Store(len(self.r_heads), D, cap) if self.r_heads else None
        self.ring = oracle.RingStore(len(self.s_heads), D, S, W) if self.s_heads else None

    @property
    def len(self):
        return self.raw_k.shape[0]

    def stored_view(self, k, v):
        sk, sv = k.copy(), v.copy()
        for h in self.r_heads:
            sk[:, h] = oracle.fp8_stored_as_bf16_bits(np.ascontiguousarray(k[:, h]))
            sv[:, h] = oracle.fp8_stored_as_bf16_bits(np.ascontiguousarray(v[:, h]))
        return sk, sv

    def append(self, k, v):
        sk, sv = self.stored_view(k, v)
        self.raw_k, self.raw_v = np.concatenate([self.raw_k, k]), np.concatenate([self.raw_v, v])
        self.st_k, self.st_v = np.concatenate([self.st_k, sk]), np.concatenate([self.st_v, sv])
        if self.fp8 is not None:
            self.fp8.append(np.ascontiguousarray(k[:, self.r_heads]), np.ascontiguousarray(v[:, self.r_heads]))
        if self.ring is not None:
            self.ring.append(np.ascontiguousarray(k[:, self.s_heads]), np.ascontiguousarray(v[:, self.s_heads]))

    def decode_row(self, q, scale):
        """after append: the query of the last token over the stored values"""
        return oracle.attn_rows(q, [self.len - 1], self.st_k, self.st_v, self.kind, self.S, self.W, scale)

    def decode_row_unquantised(self, q, scale):
        return oracle.attn_rows(q, [self.len - 1], self.raw_k, self.raw_v, self.kind, self.S, self.W, scale)

    def prefill_rows(self, q, k, v, scale):
        """before append: the chunk's queries over (earlier rows as stored) + (the chunk as given)"""
        P, C = self.len, q.shape[0]
        return oracle.attn_rows(q, P + np.arange(C), np.concatenate([self.st_k, k]), np.concatenate([self.st_v, v]),
                                self.kind, self.S, self.W, scale)


def check_stores(cache, layer, seq, o):
    if o.fp8 is not None:
        k, v, ks, vs, ln = cache.export_fp8(layer, seq)
        n = o.fp8.len
        assert ln == n
        assert np.array_equal(ks[:, :n], o.fp8.k_scale[:, :n]) and np.array_equal(vs[:, :n], o.fp8.v_scale[:, :n])
        assert np.array_equal(k[:, :n], o.fp8.k[:, :n]) and np.array_equal(v[:, :n], o.fp8.v[:, :n])
    if o.ring is not None:
        k, v, pos, ln = cache.export(layer, seq, binding.KIND_STREAMING)
        assert ln == o.ring.len and np.array_equal(pos, o.ring.pos)
        occ = o.ring.pos >= 0
        assert np.array_equal(k[:, occ], o.ring.k[:, occ]) and np.array_equal(v[:, occ], o.ring.v[:, occ])


def spread_scales(k, v, seed):
    """Give some tokens much larger or smaller rows, so that the scale bytes differ widely inside a block."""
    rng = np.random.default_rng(seed)
    n = k.shape[0]
    sh = rng.integers(-6, 7, size=(n, 1, 1))
    big = rng.random((n, 1, 1)) < 0.1
    sh = np.where(big, sh, 0).astype(np.int32)
    out = []
    # keys grow or shrink; values only shrink, so that the outputs stay of order one and the absolute
    # tolerance keeps its meaning
    for x, shift in ((k, sh), (v, -np.abs(sh) * 2)):
        f = inputs.bf16_bits_to_f64(x) * np.exp2(shift.astype(np.float64))
        out.append(inputs.f32_to_bf16_bits(f.astype(np.float32)))
    return out


def run(L, B, Hq, Hkv, S, W, kinds, lens, n_decode, seed, kvk=None, chunk=1000, step_all=False, spread=False):
    scale = 1.0 / np.sqrt(D)
    cap = [int(n) + n_decode + 3 for n in lens]
    cache = binding.ZigzagCache(L, B, Hq, Hkv, S, W, kinds, cap, max(4096, chunk * B), kvhead_is_retrieval=kvk, kv_fp8=True)
    w = inputs.Workload("f8", L, B, Hq, Hkv, D, S, W, int(sum(kinds)), 0, 0, n_decode, seed=seed)
    kv_kinds = [list(np.asarray(kvk).reshape(L, Hkv)[l]) if kvk is not None else [int(kinds[l])] * Hkv for l in range(L)]
    orc = [[Fp8Seq(Hkv, S, W, cap[b], kv_kinds[l]) for b in range(B)] for l in range(L)]
    worst_q = 0.0
    # chunked prefill: attend, then append
    for l in range(L):
        done = [0] * B
        while any(done[b] < lens[b] for b in range(B)):
            n_new = [int(min(chunk, lens[b] - done[b])) for b in range(B)]
            qs, ks, vs = [], [], []
            for b in range(B):
                if not n_new[b]:
                    continue
                q, k, v = inputs.qkv_bf16(w, l, b, done[b], n_new[b])
                if spread:
                    k, v = spread_scales(k, v, seed + 7 * b + done[b])
                qs.append(q); ks.append(k); vs.append(v)
            dq, dk, dv = to_dev(np.concatenate(qs)), to_dev(np.concatenate(ks)), to_dev(np.concatenate(vs))
            out = torch.zeros_like(dq)
            cache.prefill_attn(l, dq, dk, dv, out, n_new)
            cache.kv_append(l, dk, dv, n_new)
            got = to_bits(out)
            off = i = 0
            for b in range(B):
                if not n_new[b]:
                    continue
                want = orc[l][b].prefill_rows(qs[i], ks[i], vs[i], scale)
                assert_close(got[off:off + n_new[b]], want, f"prefill layer {l} seq {b} at {done[b]}")
                orc[l][b].append(ks[i], vs[i])
                off += n_new[b]; done[b] += n_new[b]; i += 1
        for b in range(B):
            check_stores(cache, l, b, orc[l][b])
    # decode steps
    for step in range(n_decode):
        qa = np.zeros((L, B, Hq, D), np.uint16); ka = np.zeros((L, B, Hkv, D), np.uint16); va = np.zeros_like(ka)
        for l in range(L):
            for b in range(B):
                q, k, v = inputs.qkv_bf16(w, l, b, orc[l][b].len, 1)
                if spread:
                    k, v = spread_scales(k, v, seed + 13 * b + orc[l][b].len)
                qa[l, b], ka[l, b], va[l, b] = q[0], k[0], v[0]
                orc[l][b].append(k, v)
        dq, dk, dv = to_dev(qa), to_dev(ka), to_dev(va)
        out = torch.zeros_like(dq)
        if step_all:
            cache.decode_step_all(dq, dk, dv, out)
        else:
            for l in range(L):
                cache.decode_step(l, dq[l], dk[l], dv[l], out[l])
        got = to_bits(out)
        for l in range(L):
            for b in range(B):
                want = orc[l][b].decode_row(qa[l, b:b + 1], scale)
                assert_close(got[l, b:b + 1], want, f"decode step {step} layer {l} seq {b}")
                ref = orc[l][b].decode_row_unquantised(qa[l, b:b + 1], scale)
                worst_q = max(worst_q, errors(got[l, b:b + 1], ref)[0])
    for l in range(L):
        for b in range(B):
            check_stores(cache, l, b, orc[l][b])
            assert cache.len(l, b) == lens[b] + n_decode
    assert cache.last_status() == 0
    cache.close()
    print(f"\n  [reported only] worst rel-L2 of FP8-store decode against attention over the original bf16 rows: {worst_q:.3e}")


def test_tiny_stack_shape_with_fp8_retrieval_layer():
    run(2, 1, 8, 2, 64, 256, [1, 0], [2048], 8, seed=1)


@pytest.mark.parametrize("n", [1, 15, 16, 17, 31, 32, 33, 255, 256, 257, 700])
def test_lengths_around_block_and_split_edges(n):
    run(1, 1, 8, 2, 8, 24, [1], [n], 3, seed=50 + n, chunk=300)


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (8, 2), (16, 1), (12, 4), (32, 8)])
def test_group_sizes(Hq, Hkv):
    run(2, 1, Hq, Hkv, 8, 24, [1, 0], [900], 3, seed=Hq * 31 + Hkv)


def test_many_splits_and_ragged_batch():
    run(2, 3, 8, 2, 16, 48, [1, 0], [9000, 37, 2600], 3, seed=9, chunk=3000)


def test_rows_of_very_different_magnitude():
    run(1, 2, 8, 2, 8, 24, [1], [1500, 300], 4, seed=21, chunk=500, spread=True)


def test_whole_stack_step_and_mixed_heads():
    kvk = np.array([[1, 1], [0, 0], [1, 0], [0, 1]], dtype=np.uint8)
    run(4, 2, 8, 2, 16, 48, [1, 0, 0, 0], [1200, 2300], 5, seed=33, kvk=kvk, step_all=True)
    run(3, 1, 8, 2, 16, 48, [1, 0, 1], [5000], 4, seed=34, step_all=True, chunk=2500)


def test_export_import_round_trip_and_refusals():
    cache = binding.ZigzagCache(1, 1, 4, 2, 4, 8, [1], [40], 64, kv_fp8=True)
    w = inputs.Workload("t", 1, 1, 4, 2, D, 4, 8, 1, 0, 0, 1, seed=4)
    q, k, v = inputs.qkv_bf16(w, 0, 0, 0, 30)
    cache.kv_append(0, to_dev(k), to_dev(v), [30])
    snap = cache.export_fp8(0, 0)
    with pytest.raises(binding.ZigzagError) as e:
        cache.export(0, 0, binding.KIND_RETRIEVAL)
    assert e.value.status == binding.ZZ_ERR_UNSUPPORTED
    dq = to_dev(q[29:30]); out = torch.zeros_like(dq)
    cache.decode_attn(0, dq, out)
    first = to_bits(out)
    cache.reset()
    cache.import_fp8(0, 0, *snap)
    again = cache.export_fp8(0, 0)
    for a, b in zip(snap, again):
        assert np.array_equal(a, b)
    cache.decode_attn(0, dq, out)
    assert np.array_equal(first, to_bits(out))
    with pytest.raises(binding.ZigzagError) as e:          # 30 + 11 > capacity 40: nothing is stored
        cache.kv_append(0, to_dev(k[:11]), to_dev(v[:11]), [11])
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    assert cache.export_fp8(0, 0)[4] == 30
    with pytest.raises(binding.ZigzagError) as e:          # FP8 stores are contiguous
        binding.ZigzagCache(1, 1, 4, 2, 4, 8, [1], [40], 64, kv_fp8=True, pool_pages=4)
    assert e.value.status == binding.ZZ_ERR_UNSUPPORTED
    cache.close()


def test_replayed_steps_on_fp8_stores_and_refusal_when_full():
    """Decode steps of an FP8 cache replayed from a CUDA graph (quantising append + attention per step):
    outputs against the oracle, stores bit for bit, and one replay beyond the reserved room is refused
    on the device without touching a store."""
    L, B, Hq, Hkv, S, W = 2, 2, 8, 2, 16, 48
    kinds = [1, 0]
    lens = [1500, 300]
    n_replay = 20
    scale = 1.0 / np.sqrt(D)
    cap = [n + n_replay for n in lens]
    cache = binding.ZigzagCache(L, B, Hq, Hkv, S, W, kinds, cap, 4096, kv_fp8=True)
    w = inputs.Workload("f8g", L, B, Hq, Hkv, D, S, W, 1, 0, 0, n_replay, seed=808)
    orc = [[Fp8Seq(Hkv, S, W, cap[b], [kinds[l]] * Hkv) for b in range(B)] for l in range(L)]
    for l in range(L):
        ks, vs = [], []
        for b in range(B):
            _, k, v = inputs.qkv_bf16(w, l, b, 0, lens[b])
            orc[l][b].append(k, v)
            ks.append(k); vs.append(v)
        cache.kv_append(l, to_dev(np.concatenate(ks)), to_dev(np.concatenate(vs)), lens)
    cache.reserve(n_replay)
    sq = torch.zeros((L, B, Hq, D), dtype=torch.bfloat16, device="cuda:0")
    sk = torch.zeros((L, B, Hkv, D), dtype=torch.bfloat16, device="cuda:0")
    sv, so = torch.zeros_like(sk), torch.zeros_like(sq)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        cache.decode_step_all(sq, sk, sv, so)
    for i in range(n_replay):
        q = np.zeros((L, B, Hq, D), np.uint16); k = np.zeros((L, B, Hkv, D), np.uint16); v = np.zeros_like(k)
        for l in range(L):
            for b in range(B):
                qq, kk, vv = inputs.qkv_bf16(w, l, b, lens[b] + i, 1)
                q[l, b], k[l, b], v[l, b] = qq[0], kk[0], vv[0]
                orc[l][b].append(kk, vv)
        sq.copy_(to_dev(q)); sk.copy_(to_dev(k)); sv.copy_(to_dev(v))
        g.replay()
        got = to_bits(so)
        if i % 6 == 0 or i == n_replay - 1:
            for l in range(L):
                for b in range(B):
                    assert_close(got[l, b:b + 1], orc[l][b].decode_row(q[l, b:b + 1], scale), f"replay {i} layer {l} seq {b}")
    torch.cuda.synchronize()
    assert cache.last_status() == 0
    cache.sync_len()
    for l in range(L):
        for b in range(B):
            assert cache.len(l, b) == lens[b] + n_replay
            check_stores(cache, l, b, orc[l][b])
    before = [cache.export_fp8(0, b) for b in range(B)]
    g.replay()                                   # the retrieval stores are full
    torch.cuda.synchronize()
    assert cache.last_status() == binding.ZZ_ERR_CAPACITY
    after = [cache.export_fp8(0, b) for b in range(B)]
    for x, y in zip(before, after):
        assert x[4] == y[4] and all(np.array_equal(a, b_) for a, b_ in zip(x[:4], y[:4]))
    cache.close()
