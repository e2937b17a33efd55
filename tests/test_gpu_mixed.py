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
