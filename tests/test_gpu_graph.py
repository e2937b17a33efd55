"""Decode steps replayed from a CUDA graph: the captured launch plan is reused while the stores
grow, the kernels take the lengths from the device, and the last split absorbs the new tokens.
Every replayed step is checked against the fp64 oracle, the stores bit for bit, and a replay
past the reserved room is refused on the device without touching anything."""
import numpy as np
import pytest

from paper_2508_12407_b200 import binding, build, inputs
from test_gpu_append_decode import make
from zz_testlib import OracleSeq, assert_close, check_export, to_bits, to_dev

pytestmark = pytest.mark.gpu
D = 128


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def _fill(cache, w, L, B, lens, orc):
    for l in range(L):
        ks, vs = [], []
        for b in range(B):
            _, k, v = inputs.qkv_bf16(w, l, b, 0, lens[b])
            orc[l][b].append(k, v)
            ks.append(k); vs.append(v)
        cache.kv_append(l, to_dev(np.concatenate(ks)), to_dev(np.concatenate(vs)), lens)


@pytest.mark.parametrize("paged,kvk", [(False, None), (True, None),
                                       (True, np.array([[1, 0], [0, 1], [1, 0]], dtype=np.uint8))])
def test_replayed_steps_match_oracle(paged, kvk):
    import torch
    L, B, Hq, Hkv, S, W = 3, 2, 8, 2, 16, 48
    kinds = [1, 0, 1]
    lens = [3000, 700]            # 700 + replays crosses page boundaries; 3000 uses the split plan
    n_replay = 70
    kv_kinds = [list(kvk[l]) if kvk is not None else [kinds[l]] * Hkv for l in range(L)]
    cap = [n + n_replay for n in lens]
    pool = int(np.sum(kv_kinds)) * sum((c + 127) // 128 for c in cap) if paged else 0
    cache = make(L, B, Hq, Hkv, S, W, kinds, cap, kvk=kvk, max_new=4096, pool_pages=pool)
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, 2, 0, 0, n_replay, seed=515)
    orc = [[OracleSeq(Hkv, D, S, W, cap[b], kv_kinds[l]) for b in range(B)] for l in range(L)]
    _fill(cache, w, L, B, lens, orc)

    cache.reserve(n_replay)
    if paged:
        assert cache.pages()[1] == 0      # every page the replays will need is taken now
    sq = torch.zeros((L, B, Hq, D), dtype=torch.bfloat16, device="cuda:0")
    sk = torch.zeros((L, B, Hkv, D), dtype=torch.bfloat16, device="cuda:0")
    sv = torch.zeros_like(sk)
    so = torch.zeros_like(sq)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        cache.decode_step_all(sq, sk, sv, so)
    scale = 1 / np.sqrt(D)
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
        if i % 9 == 0 or i == n_replay - 1:
            for l in range(L):
                for b in range(B):
                    want = orc[l][b].rows(q[l, b:b + 1], [lens[b] + i], scale=scale)
                    assert_close(got[l, b:b + 1], want, f"replay {i} layer {l} seq {b}")
    torch.cuda.synchronize()
    assert cache.last_status() == 0
    cache.sync_len()
    for l in range(L):
        for b in range(B):
            assert cache.len(l, b) == lens[b] + n_replay
            check_export(cache, l, b, orc[l][b])

    # one replay too many: the retrieval stores are full, the device refuses and leaves them alone
    before = [cache.export(l, b, binding.KIND_RETRIEVAL) for l in range(L) for b in range(B)
              if any(kv_kinds[l])]
    g.replay()
    torch.cuda.synchronize()
    assert cache.last_status() == binding.ZZ_ERR_CAPACITY
    after = [cache.export(l, b, binding.KIND_RETRIEVAL) for l in range(L) for b in range(B)
             if any(kv_kinds[l])]
    for x, y in zip(before, after):
        assert x[3] == y[3] and np.array_equal(x[0], y[0]) and np.array_equal(x[1], y[1])
    cache.close()


def test_reserve_refuses_beyond_capacity_or_pool():
    cache = make(1, 1, 4, 2, 4, 8, [1], [1000], pool_pages=6)
    w = inputs.Workload("t", 1, 1, 4, 2, D, 4, 8, 1, 0, 0, 0, seed=5)
    _, k, v = inputs.qkv_bf16(w, 0, 0, 0, 200)
    cache.kv_append(0, to_dev(k), to_dev(v), [200])           # 2 blocks x 2 heads = 4 pages
    with pytest.raises(binding.ZigzagError) as e:
        cache.reserve(801)                                       # past the capacity
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    with pytest.raises(binding.ZigzagError) as e:
        cache.reserve(200)                                       # 4 blocks x 2 heads = 8 pages > 6
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    assert cache.pages() == (6, 2)
    cache.reserve(56)                                            # up to 256 tokens: no new page
    assert cache.pages() == (6, 2)
    cache.reserve(57)                                            # 257 tokens: a third block
    assert cache.pages() == (6, 0)
    cache.close()


def test_replayed_per_layer_steps_and_a_replay_after_reset():
    """One zz_decode_step per layer (what a model calls between its own kernels), captured once:
    consecutive retrieval layers let a launch fetch the first blocks of its store while the launch
    before it drains.  The graph is replayed while the stores grow, then once more after the cache
    was emptied: the captured launches then carry lengths the stores no longer have, and must fall
    back to what the device says."""
    import torch
    L, B, Hq, Hkv, S, W = 4, 2, 8, 2, 16, 48
    kinds = [1, 1, 0, 1]
    lens = [3000, 700]
    n_replay = 40
    cap = [n + n_replay for n in lens]
    cache = make(L, B, Hq, Hkv, S, W, kinds, cap, max_new=4096)
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, 3, 0, 0, n_replay, seed=616)
    new_orc = lambda: [[OracleSeq(Hkv, D, S, W, cap[b], [kinds[l]] * Hkv) for b in range(B)] for l in range(L)]
    orc = new_orc()
    _fill(cache, w, L, B, lens, orc)
    cache.reserve(n_replay)
    sq = torch.zeros((L, B, Hq, D), dtype=torch.bfloat16, device="cuda:0")
    sk = torch.zeros((L, B, Hkv, D), dtype=torch.bfloat16, device="cuda:0")
    sv = torch.zeros_like(sk)
    so = torch.zeros_like(sq)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for l in range(L):
            cache.decode_step(l, sq[l], sk[l], sv[l], so[l])
    scale = 1 / np.sqrt(D)

    def replay(base, i, check):
        q = np.zeros((L, B, Hq, D), np.uint16); k = np.zeros((L, B, Hkv, D), np.uint16); v = np.zeros_like(k)
        for l in range(L):
            for b in range(B):
                qq, kk, vv = inputs.qkv_bf16(w, l, b, base[b] + i, 1)
                q[l, b], k[l, b], v[l, b] = qq[0], kk[0], vv[0]
                orc[l][b].append(kk, vv)
        sq.copy_(to_dev(q)); sk.copy_(to_dev(k)); sv.copy_(to_dev(v))
        g.replay()
        got = to_bits(so)
        if check:
            for l in range(L):
                for b in range(B):
                    want = orc[l][b].rows(q[l, b:b + 1], [orc[l][b].len - 1], scale=scale)
                    assert_close(got[l, b:b + 1], want, f"replay {i} layer {l} seq {b}")

    for i in range(n_replay):
        replay(lens, i, i % 7 == 0 or i == n_replay - 1)
    torch.cuda.synchronize()
    assert cache.last_status() == 0
    cache.sync_len()
    for l in range(L):
        for b in range(B):
            assert cache.len(l, b) == lens[b] + n_replay
            check_export(cache, l, b, orc[l][b])

    # the cache is emptied; the captured launches still carry the old lengths and split plan
    cache.reset()
    orc = new_orc()
    for i in range(20):
        replay([0, 0], i, True)
    torch.cuda.synchronize()
    assert cache.last_status() == 0
    cache.sync_len()
    for l in range(L):
        for b in range(B):
            assert cache.len(l, b) == 20
            check_export(cache, l, b, orc[l][b])
    cache.close()
