"""GPU parity of KV append / eviction (bit-exact) and of decode attention (within the
stated tolerances) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2508_12407_b200 import binding, build, inputs
from zz_testlib import OracleSeq, assert_close, check_export, to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def make(L, B, Hq, Hkv, S, W, kinds, cap, kvk=None, max_new=4096, pool_pages=0, D=128):
    return binding.ZigzagCache(L, B, Hq, Hkv, S, W, kinds, cap, max_new, kvhead_is_retrieval=kvk,
                               pool_pages=pool_pages, head_dim=D)


def layer_kv_kinds(kinds, Hkv, kvk, l):
    if kvk is not None:
        return list(np.asarray(kvk).reshape(len(kinds), Hkv)[l])
    return [int(kinds[l])] * Hkv


def run_append_decode(L, B, Hq, Hkv, S, W, kinds, lens, n_decode, seed, kvk=None, chunk_cap=300,
                      check_every=1, pool_pages=0, tune=None, D=128):
    scale = 1.0 / np.sqrt(D)
    cap = [int(n) + n_decode for n in lens]
    cache = make(L, B, Hq, Hkv, S, W, kinds, cap, kvk, max_new=max(4096, chunk_cap * B), pool_pages=pool_pages, D=D)
    for key, value in (tune or {}).items():
        cache.tune(key, value)
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, int(sum(kinds)), 0, 0, n_decode, seed=seed)
    orc = [[OracleSeq(Hkv, D, S, W, cap[b], layer_kv_kinds(kinds, Hkv, kvk, l)) for b in range(B)]
           for l in range(L)]
    # fill the stores with seeded chunks of ragged sizes (several appends per sequence)
    for l in range(L):
        plans = [inputs.random_chunking(int(lens[b]), seed, l, b, max_chunk=chunk_cap) for b in range(B)]
        rounds = max(len(p) for p in plans)
        for r in range(rounds):
            n_new = [plans[b][r] if r < len(plans[b]) else 0 for b in range(B)]
            ks, vs = [], []
            for b in range(B):
                if n_new[b] == 0:
                    continue
                _, k, v = inputs.qkv_bf16(w, l, b, orc[l][b].len, n_new[b])
                orc[l][b].append(k, v)
                ks.append(k)
                vs.append(v)
            cache.kv_append(l, to_dev(np.concatenate(ks)), to_dev(np.concatenate(vs)), n_new)
        for b in range(B):
            check_export(cache, l, b, orc[l][b])
            assert cache.len(l, b) == lens[b]
    # decode steps
    worst = (0.0, 0.0)
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
            if step % check_every and step != n_decode - 1:
                continue
            got = to_bits(out)
            for b in range(B):
                t = orc[l][b].len - 1
                want = orc[l][b].rows(qs[b], [t], scale=scale)
                rel, mx = assert_close(got[b:b + 1], want, f"decode step {step} layer {l} seq {b}")
                worst = (max(worst[0], rel), max(worst[1], mx))
    for l in range(L):
        for b in range(B):
            check_export(cache, l, b, orc[l][b])
    assert cache.last_status() == 0
    cache.close()
    return worst


def test_tiny_stack_config1_shape():
    # layer 0 retrieval, layer 1 streaming, 8 query / 2 KV heads, 2048 tokens then 16 steps
    run_append_decode(2, 1, 8, 2, 64, 256, [1, 0], [2048], 16, seed=1)


@pytest.mark.parametrize("n", [1, 2, 63, 64, 65, 127, 128, 129, 319, 320, 321, 2 * 256 + 64 + 3])
def test_adversarial_lengths(n):
    run_append_decode(2, 1, 8, 2, 64, 256, [1, 0], [n], 3, seed=100 + n)


@pytest.mark.parametrize("S,W", [(0, 1), (3, 5), (4, 8), (0, 16), (17, 1)])
def test_small_rings(S, W):
    run_append_decode(2, 1, 4, 1, S, W, [0, 1], [S + 2 * W + 3], 2 * W + 3, seed=7 + S + W)


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (8, 2), (16, 1), (12, 4), (16, 2)])
def test_group_sizes(Hq, Hkv):
    run_append_decode(2, 1, Hq, Hkv, 8, 24, [1, 0], [700], 4, seed=Hq * 31 + Hkv)


def test_many_splits_long_context():
    # long enough that the retrieval layer is split over many CTAs and merged
    run_append_decode(2, 1, 8, 2, 128, 256, [1, 0], [9000], 3, seed=5, chunk_cap=4000)


# One KV head in the group and a store of about 50K tokens: at 384 tokens per split the short plan
# would need more splits (129-148) than the kernel's merge rows hold, so the planner must switch to
# the long plan there, and the short plan with a split count just below the limit must be right too.
@pytest.mark.parametrize("n", [40000, 46000, 50000, 56832 - 2])
def test_one_kv_head_store_near_the_split_limit(n):
    run_append_decode(2, 1, 4, 1, 128, 256, [1, 0], [n], 2, seed=n, chunk_cap=8192)


def test_one_kv_head_ring_near_the_split_limit():
    # the same plan question on a streaming layer whose ring is that large
    run_append_decode(2, 1, 4, 1, 128, 52000, [0, 1], [53000], 2, seed=53, chunk_cap=8192)


@pytest.mark.parametrize("n", [50000, 56000])
def test_mixed_layer_with_one_retrieval_head_near_the_split_limit(n):
    kvk = np.array([[1, 0], [0, 1]], dtype=np.uint8)
    run_append_decode(2, 1, 8, 2, 128, 256, [0, 0], [n], 2, seed=n + 1, kvk=kvk, chunk_cap=8192)


def test_one_long_one_short_sequence_near_the_split_limit():
    run_append_decode(1, 2, 4, 1, 128, 256, [1], [52000, 300], 2, seed=523, chunk_cap=8192)


@pytest.mark.parametrize("short,n", [(512, 70000), (1024, 100000), (1024, 130000)])
def test_short_plan_threshold_tuned_up(short, n):
    # 137 splits of 512 tokens would overrun the merge rows (long plan instead); 98 splits of 1024
    # tokens is a legal short plan with many splits; 127 of 1024 is again past the limit
    run_append_decode(1, 1, 4, 1, 128, 256, [1], [n], 2, seed=n, chunk_cap=8192, tune={"decode_short_tokens": short})


# head_dim 64 (half the row bytes, twice the pipeline stages, half the MMA steps)
@pytest.mark.parametrize("n", [1, 17, 320, 321, 700])
def test_head_dim_64_lengths(n):
    run_append_decode(2, 1, 8, 2, 64, 256, [1, 0], [n], 3, seed=640 + n, D=64)


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (8, 2), (16, 1), (12, 4)])
def test_head_dim_64_group_sizes(Hq, Hkv):
    run_append_decode(2, 1, Hq, Hkv, 8, 24, [1, 0], [700], 4, seed=64 + Hq * 31 + Hkv, D=64)


def test_head_dim_64_many_splits_ragged_batch_and_mixed_heads():
    run_append_decode(2, 3, 8, 2, 16, 48, [1, 0], [9000, 37, 2600], 3, seed=641, chunk_cap=3000, D=64)
    kvk = np.array([[1, 0], [0, 1]], dtype=np.uint8)
    run_append_decode(2, 2, 8, 2, 16, 48, [0, 0], [5000, 300], 3, seed=642, kvk=kvk, chunk_cap=3000, D=64)


def test_ragged_batch():
    lens = [37, 1500, 300, 4100, 1]
    run_append_decode(2, 5, 8, 2, 16, 48, [1, 0], lens, 5, seed=9, chunk_cap=1500)


def test_maximum_batch():
    # ZZ_MAX_BATCH sequences, ragged from 1 token upwards, several of them shorter than the ring
    rng = np.random.default_rng(64)
    lens = [int(x) for x in rng.integers(1, 700, size=binding.ZZ_MAX_BATCH)]
    lens[0], lens[1], lens[-1] = 1, 2, 699
    run_append_decode(2, binding.ZZ_MAX_BATCH, 8, 2, 16, 48, [1, 0], lens, 2, seed=64, chunk_cap=700)


def test_store_filled_to_capacity_exactly():
    # the last decode step lands on the last slot of every retrieval store; one more is refused
    import torch
    D, B = 128, 2
    lens = [130, 257]
    cap = [n + 1 for n in lens]
    cache = make(1, B, 4, 1, 8, 8, [1], cap)
    w = inputs.Workload("t", 1, B, 4, 1, D, 8, 8, 1, 0, 0, 1, seed=5)
    for b in range(B):
        pass
    ks = np.concatenate([inputs.qkv_bf16(w, 0, b, 0, lens[b])[1] for b in range(B)])
    vs = np.concatenate([inputs.qkv_bf16(w, 0, b, 0, lens[b])[2] for b in range(B)])
    cache.kv_append(0, to_dev(ks), to_dev(vs), lens)
    q = to_dev(np.concatenate([inputs.qkv_bf16(w, 0, b, lens[b], 1)[0] for b in range(B)]))
    k = to_dev(np.concatenate([inputs.qkv_bf16(w, 0, b, lens[b], 1)[1] for b in range(B)]))
    v = to_dev(np.concatenate([inputs.qkv_bf16(w, 0, b, lens[b], 1)[2] for b in range(B)]))
    out = torch.zeros_like(q)
    cache.decode_step(0, q, k, v, out)                       # fills the last slot
    assert [cache.len(0, b) for b in range(B)] == cap
    with pytest.raises(binding.ZigzagError) as e:
        cache.decode_step(0, q, k, v, out)
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    with pytest.raises(binding.ZigzagError) as e:
        cache.decode_step_all(q.view(1, B, 4, D), k.view(1, B, 1, D), v.view(1, B, 1, D), out.view(1, B, 4, D))
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    assert [cache.export(0, b, binding.KIND_RETRIEVAL)[3] for b in range(B)] == cap
    assert cache.last_status() == 0
    cache.close()


def test_min_chunk_tuning_keeps_results():
    D = 128
    w = inputs.Workload("t", 1, 1, 8, 2, D, 8, 8, 1, 0, 0, 1, seed=77)
    q, k, v = inputs.qkv_bf16(w, 0, 0, 0, 3000)
    outs = []
    for mc in (64, 256, 1024):
        cache = make(1, 1, 8, 2, 8, 8, [1], [3000])
        cache.tune("decode_min_chunk", mc)
        cache.kv_append(0, to_dev(k), to_dev(v), [3000])
        dq = to_dev(q[2999:3000])
        out = dq.new_zeros(dq.shape)
        cache.decode_attn(0, dq, out)
        outs.append(to_bits(out))
        cache.close()
    o = OracleSeq(2, D, 8, 8, 3000, [1, 1])
    o.append(k, v)
    want = o.rows(q[2999:3000], [2999], scale=1 / np.sqrt(D))
    for got in outs:
        assert_close(got, want, "tuned split")


def test_whole_stack_step_overlap_modes_agree():
    """zz_decode_step_all with its layers overlapped (programmatic dependent launch, with and
    without the wait between layers) or batched into one launch per kind gives the same bits as
    plain stream order, and matches the oracle: the layers of a step share no scratch."""
    import torch
    D, L, B, Hq, Hkv, S, W = 128, 6, 2, 8, 2, 16, 48
    kinds = [1, 0, 1, 1, 0, 1]
    lens = [5000, 2300]
    steps = 12
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, 4, 0, 0, steps, seed=4242)
    hist = [[inputs.qkv_bf16(w, l, b, 0, lens[b]) for b in range(B)] for l in range(L)]
    dec = [[[inputs.qkv_bf16(w, l, b, lens[b] + i, 1) for b in range(B)] for l in range(L)] for i in range(steps)]
    results = {}
    for mode in (0, 1, 2, 3):
        cache = make(L, B, Hq, Hkv, S, W, kinds, [n + steps + 4 for n in lens], max_new=8192)
        cache.tune("decode_overlap", mode)
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
        cache.close()
    for mode in (1, 2, 3):
        assert np.array_equal(results[0], results[mode]), f"overlap mode {mode} differs from plain stream order"
    # last step of every layer and sequence against the oracle
    scale = 1 / np.sqrt(D)
    for l in range(L):
        for b in range(B):
            o = OracleSeq(Hkv, D, S, W, lens[b] + steps + 4, [kinds[l]] * Hkv)
            o.append(hist[l][b][1], hist[l][b][2])
            for i in range(steps):
                o.append(dec[i][l][b][1], dec[i][l][b][2])
            t = lens[b] + steps - 1
            want = o.rows(dec[steps - 1][l][b][0], [t], scale=scale)
            got = results[3][steps - 1, l, b:b + 1]
            assert_close(got, want, f"layer {l} seq {b}")


def test_error_paths_leave_cache_untouched():
    cache = make(2, 1, 8, 2, 4, 8, [1, 0], [10])
    w = inputs.Workload("t", 2, 1, 8, 2, 128, 4, 8, 1, 0, 0, 1, seed=3)
    q, k, v = inputs.qkv_bf16(w, 0, 0, 0, 12)
    dk, dv, dq = to_dev(k), to_dev(v), to_dev(q[:1])
    out = dq.new_zeros(dq.shape)
    with pytest.raises(binding.ZigzagError) as e:          # decode before any append
        cache.decode_attn(0, dq, out)
    assert e.value.status == binding.ZZ_ERR_INVALID_ARG
    cache.kv_append(0, dk[:8], dv[:8], [8])
    before = cache.export(0, 0, binding.KIND_RETRIEVAL)
    with pytest.raises(binding.ZigzagError) as e:          # 8 + 4 > capacity 10
        cache.kv_append(0, dk[8:], dv[8:], [4])
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    with pytest.raises(binding.ZigzagError) as e:
        cache.kv_append(5, dk, dv, [1])
    assert e.value.status == binding.ZZ_ERR_INVALID_ARG
    with pytest.raises(binding.ZigzagError) as e:
        cache.kv_append(0, dk, dv, [-1])
    assert e.value.status == binding.ZZ_ERR_INVALID_ARG
    after = cache.export(0, 0, binding.KIND_RETRIEVAL)
    assert all(np.array_equal(a, b) for a, b in zip(before[:3], after[:3])) and before[3] == after[3] == 8
    # streaming stores have no capacity limit
    cache.kv_append(1, dk, dv, [12])
    assert cache.len(1) == 12
    cache.reset()
    assert cache.len(0) == 0 and cache.export(1, 0, binding.KIND_STREAMING)[3] == 0
    assert np.all(cache.export(1, 0, binding.KIND_STREAMING)[2] == -1)
    cache.close()


def test_export_import_roundtrip():
    cache = make(2, 2, 8, 2, 4, 8, [1, 0], [40, 40])
    w = inputs.Workload("t", 2, 2, 8, 2, 128, 4, 8, 1, 0, 0, 1, seed=4)
    for l in range(2):
        ks, vs = [], []
        for b in range(2):
            _, k, v = inputs.qkv_bf16(w, l, b, 0, 30)
            ks.append(k); vs.append(v)
        cache.kv_append(l, to_dev(np.concatenate(ks)), to_dev(np.concatenate(vs)), [30, 30])
    snap_r = cache.export(0, 1, binding.KIND_RETRIEVAL)
    snap_s = cache.export(1, 1, binding.KIND_STREAMING)
    cache.reset(1)
    assert cache.len(0, 1) == 0 and cache.len(0, 0) == 30
    cache.import_(0, 1, binding.KIND_RETRIEVAL, *snap_r)
    cache.import_(1, 1, binding.KIND_STREAMING, *snap_s)
    again_r = cache.export(0, 1, binding.KIND_RETRIEVAL)
    again_s = cache.export(1, 1, binding.KIND_STREAMING)
    for a, b in zip(snap_r, again_r):
        assert np.array_equal(a, b)
    for a, b in zip(snap_s, again_s):
        assert np.array_equal(a, b)
    cache.close()
