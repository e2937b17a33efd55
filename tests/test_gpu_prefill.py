"""GPU parity of prefill attention (retrieval: causal over store + chunk; streaming: sink
tiles + local band, token-exact mask) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2508_12407_b200 import binding, build, inputs
from zz_testlib import OracleSeq, assert_close, check_export, to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def run_prefill(L, B, Hq, Hkv, S, W, kinds, chunk_plans, seed, kvk=None, n_decode=0, sample_rows=None,
                pool_pages=0, D=128):
    """chunk_plans[b] = list of chunk sizes of sequence b (a 0 skips the sequence in that call)."""
    scale = 1.0 / np.sqrt(D)
    total = [int(sum(pl)) for pl in chunk_plans]
    cap = [t + n_decode + 1 for t in total]
    max_new = max(sum(pl[r] if r < len(pl) else 0 for pl in chunk_plans)
                  for r in range(max(len(pl) for pl in chunk_plans)))
    cache = binding.ZigzagCache(L, B, Hq, Hkv, S, W, kinds, cap, max(max_new, B), kvhead_is_retrieval=kvk,
                                pool_pages=pool_pages, head_dim=D)
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, int(sum(kinds)), 0, 0, n_decode, seed=seed)

    def kv_kinds(l):
        if kvk is not None:
            return list(np.asarray(kvk).reshape(L, Hkv)[l])
        return [int(kinds[l])] * Hkv

    orc = [[OracleSeq(Hkv, D, S, W, cap[b], kv_kinds(l)) for b in range(B)] for l in range(L)]
    rounds = max(len(pl) for pl in chunk_plans)
    worst = [0.0, 0.0]
    for l in range(L):
        for r in range(rounds):
            n_new = [chunk_plans[b][r] if r < len(chunk_plans[b]) else 0 for b in range(B)]
            qs, ks, vs, wants = [], [], [], []
            for b in range(B):
                c = n_new[b]
                if c == 0:
                    continue
                P = orc[l][b].len
                q, k, v = inputs.qkv_bf16(w, l, b, P, c)
                k_all = np.concatenate([orc[l][b].hist.k, k])
                v_all = np.concatenate([orc[l][b].hist.v, v])
                rows = np.arange(c) if sample_rows is None else np.unique(
                    np.clip(np.asarray(sample_rows(P, c)), 0, c - 1))
                want = orc[l][b].rows(np.ascontiguousarray(q[rows]), P + rows, k_all, v_all, scale)
                qs.append(q); ks.append(k); vs.append(v); wants.append((b, rows, want))
            dq, dk, dv = (to_dev(np.concatenate(x)) for x in (qs, ks, vs))
            out = dq.new_zeros(dq.shape)
            before = [cache.export(l, b, int(kv_kinds(l)[0]))[3] for b in range(B)]
            cache.prefill_attn(l, dq, dk, dv, out, n_new)
            got = to_bits(out)
            assert [cache.export(l, b, int(kv_kinds(l)[0]))[3] for b in range(B)] == before  # store untouched
            off = 0
            for (b, rows, want) in wants:
                rel, mx = assert_close(got[off + rows], want, f"prefill layer {l} round {r} seq {b}")
                worst = [max(worst[0], rel), max(worst[1], mx)]
                off += n_new[b]
            cache.kv_append(l, dk, dv, n_new)
            i = 0
            for b in range(B):
                if n_new[b]:
                    orc[l][b].append(ks[i], vs[i])
                    i += 1
        for b in range(B):
            check_export(cache, l, b, orc[l][b])
    for step in range(n_decode):
        for l in range(L):
            qs, ks, vs = [], [], []
            for b in range(B):
                q, k, v = inputs.qkv_bf16(w, l, b, orc[l][b].len, 1)
                orc[l][b].append(k, v)
                qs.append(q); ks.append(k); vs.append(v)
            dq = to_dev(np.concatenate(qs))
            out = dq.new_zeros(dq.shape)
            cache.decode_step(l, dq, to_dev(np.concatenate(ks)), to_dev(np.concatenate(vs)), out)
            got = to_bits(out)
            for b in range(B):
                want = orc[l][b].rows(qs[b], [orc[l][b].len - 1], scale=scale)
                assert_close(got[b:b + 1], want, f"decode {step} layer {l} seq {b}")
    assert cache.last_status() == 0
    cache.close()
    return worst


def test_tiny_stack_config1():
    # 2 layers (retrieval, streaming), 8 q / 2 kv heads, prefill 2048 single shot, 16 decode steps,
    # sink 64, recent 256: every output element checked
    run_prefill(2, 1, 8, 2, 64, 256, [1, 0], [[2048]], seed=1, n_decode=16)


@pytest.mark.parametrize("C", [1, 2, 127, 128, 129, 257, 640])
def test_single_shot_lengths(C):
    run_prefill(2, 1, 8, 2, 64, 256, [1, 0], [[C]], seed=10 + C)


@pytest.mark.parametrize("plan", [[5, 1, 122, 1, 300], [128, 128, 128], [200, 57, 700], [1, 1, 1, 400],
                                  [63, 1, 1, 255, 1, 1, 64, 500]])
def test_chunked_prefill_straddling_sink_and_window(plan):
    run_prefill(2, 1, 8, 2, 64, 256, [1, 0], [plan], seed=20 + len(plan))


@pytest.mark.parametrize("S,W", [(0, 1), (3, 5), (0, 128), (128, 1), (130, 140), (100, 1000)])
def test_ring_shapes(S, W):
    run_prefill(2, 1, 4, 1, S, W, [0, 1], [[300, 77, 400]], seed=30 + S + W)


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (3, 1), (4, 1), (16, 2)])
def test_group_sizes(Hq, Hkv):
    run_prefill(2, 1, Hq, Hkv, 16, 100, [1, 0], [[333, 200]], seed=40 + Hq)


def test_ragged_batch_packed():
    plans = [[300, 40], [1, 500], [129, 0], [0, 77]]
    run_prefill(2, 4, 8, 2, 32, 96, [1, 0], plans, seed=50, n_decode=2)


def test_maximum_batch_packed_prefill():
    # ZZ_MAX_BATCH sequences in one packed call, some of them absent from a round
    rng = np.random.default_rng(65)
    plans = [[int(rng.integers(0, 200)), int(rng.integers(1, 150))] for _ in range(binding.ZZ_MAX_BATCH)]
    plans[0] = [0, 1]
    plans[1] = [129, 0]
    run_prefill(2, binding.ZZ_MAX_BATCH, 4, 2, 8, 24, [1, 0], plans, seed=65, n_decode=1)


def test_odd_group_many_items_persistent_path():
    # odd group size (the second tile of some head pairs is absent) with more work items than SMs,
    # so the streaming layer runs persistent CTAs that meet both kinds of item; two chunks, so the
    # second one also reads ring tiles
    def rows(P, c):
        return [0, 1, 127, 128, 129, 255, 256, 383, 384, c // 2, c - 130, c - 1]
    run_prefill(2, 1, 3, 1, 100, 200, [0, 1], [[128 * 90 + 5, 128 * 80 + 77]], seed=81, sample_rows=rows)


def test_decode_step_equals_prefill_row():
    # the last row of a prefill and a decode step at the same position agree within tolerance
    D, S, W, n = 128, 32, 64, 500
    w = inputs.Workload("t", 2, 1, 8, 2, D, S, W, 1, 0, 0, 0, seed=60)
    for l, kind in enumerate([1, 0]):
        q, k, v = inputs.qkv_bf16(w, l, 0, 0, n)
        a = binding.ZigzagCache(2, 1, 8, 2, S, W, [1, 0], [n], n)
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        out = dq.new_zeros(dq.shape)
        a.prefill_attn(l, dq, dk, dv, out, [n])
        pre = inputs.bf16_bits_to_f64(to_bits(out))
        a.kv_append(l, dk, dv, [n])
        dec = dq.new_zeros((1, 8, D))
        a.decode_attn(l, dq[n - 1:n].contiguous(), dec)
        d = inputs.bf16_bits_to_f64(to_bits(dec))
        assert np.max(np.abs(d[0] - pre[n - 1])) <= 2e-2
        assert np.linalg.norm(d[0] - pre[n - 1]) / np.linalg.norm(pre[n - 1]) <= 5e-3
        a.close()


def test_long_prefill_sampled_rows():
    # many KV tiles per query tile; only sampled rows go through the oracle
    def rows(P, c):
        return [0, 1, 63, 64, 127, 128, 319, 320, 321, c // 2, c - 129, c - 128, c - 2, c - 1]
    run_prefill(2, 1, 8, 2, 64, 256, [1, 0], [[6000, 2500]], seed=70, sample_rows=rows)


def test_scores_of_very_different_magnitude():
    """Keys (and values) of some tokens 64 times larger or smaller than the rest: scores hundreds of
    units apart, so most probabilities underflow.  Every exponential path must turn those into zeros
    (the polynomial one has no hardware underflow to lean on)."""
    import torch
    D, Hq, Hkv, S, W, C = 128, 8, 2, 16, 48, 700
    scale = 1.0 / np.sqrt(D)
    w = inputs.Workload("t", 2, 1, Hq, Hkv, D, S, W, 1, 0, 0, 0, seed=909)
    cache = binding.ZigzagCache(2, 1, Hq, Hkv, S, W, [1, 0], [2 * C + 4], C)
    rng = np.random.default_rng(909)
    for l, kind in enumerate([1, 0]):
        o = OracleSeq(Hkv, D, S, W, 2 * C + 4, [kind] * Hkv)
        for chunk in range(2):
            q, k, v = inputs.qkv_bf16(w, l, 0, chunk * C, C)
            sh = np.where(rng.random((C, 1, 1)) < 0.1, rng.integers(-6, 7, (C, 1, 1)), 0).astype(np.float64)
            k = inputs.f32_to_bf16_bits((inputs.bf16_bits_to_f64(k) * np.exp2(sh)).astype(np.float32))
            v = inputs.f32_to_bf16_bits((inputs.bf16_bits_to_f64(v) * np.exp2(-np.abs(sh))).astype(np.float32))   # outputs stay of order one
            want = o.rows(q, chunk * C + np.arange(C), np.concatenate([o.hist.k, k]), np.concatenate([o.hist.v, v]), scale)
            dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
            out = torch.zeros_like(dq)
            cache.prefill_attn(l, dq, dk, dv, out, [C])
            cache.kv_append(l, dk, dv, [C])
            o.append(k, v)
            assert_close(to_bits(out), want, f"layer {l} chunk {chunk}")
        q, k, v = inputs.qkv_bf16(w, l, 0, 2 * C, 1)
        o.append(k, v)
        dq = to_dev(q); out = torch.zeros_like(dq)
        cache.decode_step(l, dq, to_dev(k), to_dev(v), out)
        assert_close(to_bits(out), o.rows(q, [2 * C], scale=scale), f"layer {l} decode")
    assert cache.last_status() == 0
    cache.close()


# head_dim 64: tiles of one 64-column sub-tile, four MMA steps per Q K^T, N = 64 for P V
def test_head_dim_64_single_shot_and_chunked():
    run_prefill(2, 1, 8, 2, 64, 256, [1, 0], [[2048]], seed=6401, n_decode=2, D=64)
    run_prefill(2, 1, 8, 2, 16, 48, [1, 0], [[300, 77, 1, 500, 129]], seed=6402, n_decode=2, D=64)


def test_head_dim_64_ragged_batch_odd_heads_and_mixed_layer():
    run_prefill(2, 3, 6, 2, 16, 48, [1, 0], [[700, 50], [33, 0], [128, 300]], seed=6403, n_decode=1, D=64)
    kvk = np.array([[1, 0], [0, 1]], dtype=np.uint8)
    run_prefill(2, 2, 8, 2, 16, 48, [0, 0], [[400, 300], [129, 64]], seed=6404, kvk=kvk, n_decode=1, D=64)


def test_head_dim_64_many_items_persistent_launch():
    # more work items than SMs, so the persistent instantiation and the per-CTA item order run
    run_prefill(1, 1, 32, 8, 16, 48, [1], [[4096]], seed=6405, D=64,
                sample_rows=lambda P, c: [0, 1, 127, 128, 129, 1000, 2047, 2048, 4095])
    run_prefill(1, 1, 32, 8, 128, 256, [0], [[4096, 2048]], seed=6406, D=64,
                sample_rows=lambda P, c: [0, 1, 127, 128, 383, 384, 385, 1000, c - 1])
