"""GPU parity of the DuoAttention-style mixed-head layer (two passes plus head gather /
scatter) against the oracle with the kind chosen per KV head, and agreement with the
exclusive path head by head."""
import numpy as np
import pytest

from paper_2508_12407_b200 import binding, build, inputs
from test_gpu_append_decode import run_append_decode
from test_gpu_prefill import run_prefill
from zz_testlib import to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def test_mixed_decode_non_contiguous_heads():
    kvk = np.array([[1, 0, 0, 1], [0, 1, 1, 0], [1, 1, 1, 1]], dtype=np.uint8)
    run_append_decode(3, 2, 8, 4, 8, 24, [0, 0, 0], [300, 1200], 4, seed=11, kvk=kvk)


def test_mixed_prefill_and_decode():
    kvk = np.array([[0, 1, 0, 1], [1, 0, 0, 0]], dtype=np.uint8)
    run_prefill(2, 2, 16, 4, 16, 100, [0, 0], [[300, 150], [129, 40]], seed=12, kvk=kvk, n_decode=3)


def test_mixed_seeded_half_heads_cfg5_shape():
    w = inputs.Workload("m", 2, 1, 32, 8, 128, 128, 256, 1, 0, 0, 0, mixed_retrieval_kv_heads=4, seed=5)
    kvk = inputs.mixed_kvhead_kinds(w)
    assert kvk.sum(axis=1).tolist() == [4, 4]
    run_prefill(2, 1, 32, 8, 128, 256, [0, 0], [[700]], seed=13, kvk=kvk, n_decode=2)


def test_mixed_equals_exclusive_per_head():
    # same inputs through an all-retrieval layer, an all-streaming layer and a mixed layer:
    # every head of the mixed layer reproduces the bits of the exclusive layer of its kind
    D, S, W, n, Hq, Hkv = 128, 16, 64, 400, 8, 4
    w = inputs.Workload("t", 1, 1, Hq, Hkv, D, S, W, 1, 0, 0, 0, seed=14)
    q, k, v = inputs.qkv_bf16(w, 0, 0, 0, n)
    kinds = [1, 0, 0, 1]
    outs = {}
    for name, kvk in [("R", [1] * 4), ("S", [0] * 4), ("M", kinds)]:
        c = binding.ZigzagCache(1, 1, Hq, Hkv, S, W, [0], [n + 1], n,
                                kvhead_is_retrieval=np.array([kvk], dtype=np.uint8))
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        o = dq.new_zeros(dq.shape)
        c.prefill_attn(0, dq, dk, dv, o, [n])
        c.kv_append(0, dk, dv, [n])
        od = dq.new_zeros((1, Hq, D))
        c.decode_attn(0, dq[n - 1:n].contiguous(), od)
        outs[name] = (to_bits(o), to_bits(od))
        c.close()
    G = Hq // Hkv
    for h in range(Hq):
        src = "R" if kinds[h // G] else "S"
        assert np.array_equal(outs["M"][0][:, h], outs[src][0][:, h])
        assert np.array_equal(outs["M"][1][:, h], outs[src][1][:, h])


@pytest.mark.parametrize("same_nr", [True, False])
def test_whole_stack_step_with_mixed_layers(same_nr):
    """A decode step over a stack of mixed and exclusive layers: the launches batched over layers
    (mixed layers with equal retrieval-head counts) give the bits of the layer-by-layer path, the
    cache contents agree bit for bit, and the last step matches the oracle.  With unequal counts
    the batched path must decline and the layer-by-layer path runs."""
    import torch
    from test_gpu_append_decode import make
    from zz_testlib import OracleSeq, assert_close
    D, B, Hq, Hkv, S, W = 128, 2, 8, 4, 16, 48
    kvk = np.array([[1, 0, 0, 1], [1, 1, 1, 1], [0, 1, 1, 0], [0, 0, 0, 0],
                    [1, 1, 0, 0] if same_nr else [1, 1, 1, 0]], dtype=np.uint8)
    L = len(kvk)
    lens = [5000, 2300]
    steps = 6
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, 1, 0, 0, steps, seed=777)
    hist = [[inputs.qkv_bf16(w, l, b, 0, lens[b]) for b in range(B)] for l in range(L)]
    dec = [[[inputs.qkv_bf16(w, l, b, lens[b] + i, 1) for b in range(B)] for l in range(L)] for i in range(steps)]
    results, stores = {}, {}
    # the third run keeps the retrieval rows in 128-token pages (one page per retrieval head and block)
    pool = int(kvk.sum()) * sum((n + steps + 127) // 128 for n in lens)
    for mode in (0, 3, "paged"):
        cache = make(L, B, Hq, Hkv, S, W, [0] * L, [n + steps + 4 for n in lens], kvk=kvk, max_new=8192,
                     pool_pages=pool if mode == "paged" else 0)
        cache.tune("decode_overlap", 3 if mode == "paged" else mode)
        for l in range(L):
            k = np.concatenate([hist[l][b][1] for b in range(B)])
            v = np.concatenate([hist[l][b][2] for b in range(B)])
            cache.kv_append(l, to_dev(k), to_dev(v), lens)
        outs = []
        for i in range(steps):
            q = np.stack([np.concatenate([dec[i][l][b][0] for b in range(B)]) for l in range(L)])
            k = np.stack([np.concatenate([dec[i][l][b][1] for b in range(B)]) for l in range(L)])
            v = np.stack([np.concatenate([dec[i][l][b][2] for b in range(B)]) for l in range(L)])
            dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
            out = torch.zeros_like(dq)
            cache.decode_step_all(dq, dk, dv, out)
            outs.append(to_bits(out))
        torch.cuda.synchronize()
        assert cache.last_status() == 0
        results[mode] = np.stack(outs)
        for l in range(L):
            for b in range(B):
                assert cache.len(l, b) == lens[b] + steps
        stores[mode] = [cache.export(l, b, kind) for l in range(L) for b in range(B)
                        for kind in (binding.KIND_RETRIEVAL, binding.KIND_STREAMING)
                        if (kvk[l] == (kind == binding.KIND_RETRIEVAL)).any()]
        cache.close()
    assert np.array_equal(results[0], results[3])
    assert np.array_equal(results[0], results["paged"])
    for other in (3, "paged"):
        for a, b_ in zip(stores[0], stores[other]):
            for x, y in zip(a, b_):
                assert np.array_equal(np.asarray(x), np.asarray(y))
    scale = 1 / np.sqrt(D)
    for l in range(L):
        for b in range(B):
            o = OracleSeq(Hkv, D, S, W, lens[b] + steps + 4, list(kvk[l]))
            o.append(hist[l][b][1], hist[l][b][2])
            for i in range(steps):
                o.append(dec[i][l][b][1], dec[i][l][b][2])
            want = o.rows(dec[steps - 1][l][b][0], [lens[b] + steps - 1], scale=scale)
            assert_close(results[3][steps - 1, l, b:b + 1], want, f"layer {l} seq {b}")
