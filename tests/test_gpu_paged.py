"""GPU parity of the paged retrieval stores (a pool of 128-token pages shared by all layers and
sequences) against the same oracle as the contiguous stores: the attention computed does not
depend on where the rows live.  Also the pool's bookkeeping: exhaustion is refused cleanly,
a reset returns pages, a pool smaller than the sum of the capacities serves what fits."""
import numpy as np
import pytest

from paper_2508_12407_b200 import binding, build, inputs
from test_gpu_append_decode import make, run_append_decode
from test_gpu_prefill import run_prefill
from zz_testlib import OracleSeq, assert_close, to_bits, to_dev

pytestmark = pytest.mark.gpu
D = 128


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def test_paged_append_decode_ragged_batch():
    # ragged chunks, page boundaries crossed inside chunks and by single decode steps (255 -> 257)
    run_append_decode(3, 3, 8, 2, 8, 24, [1, 0, 1], [255, 1000, 130], 6, seed=31, pool_pages=64)


def test_paged_long_context_many_splits():
    # long store: 4-warp split plan with 16-token aligned splits, several pages per warp
    run_append_decode(2, 1, 32, 8, 16, 48, [1, 0], [40000], 3, seed=32, chunk_cap=8192, pool_pages=8 * 314)


def test_paged_group_size_16_and_mixed_layer():
    kvk = np.array([[1, 0, 0, 1], [0, 1, 1, 0], [1, 1, 1, 1]], dtype=np.uint8)
    run_append_decode(3, 2, 8, 4, 8, 24, [0, 0, 0], [300, 1200], 4, seed=33, kvk=kvk, pool_pages=110)
    run_append_decode(1, 1, 16, 1, 4, 12, [1], [777], 3, seed=34, pool_pages=8)


def test_paged_chunked_prefill_reads_past_pages():
    # later chunks attend to earlier ones through the page table; chunk sizes off the page size
    run_prefill(2, 2, 8, 2, 16, 100, [1, 0], [[300, 150, 129], [129, 40, 500]], seed=35, n_decode=3,
                pool_pages=2 * (5 + 6))
    kvk = np.array([[0, 1, 0, 1], [1, 0, 0, 0]], dtype=np.uint8)
    run_prefill(2, 2, 16, 4, 16, 100, [0, 0], [[300, 150], [129, 40]], seed=36, kvk=kvk, n_decode=3, pool_pages=40)


def test_paged_whole_stack_step_matches_contiguous_bits():
    """decode_step_all over a paged cache gives the bits of the contiguous cache when both use the
    same split plan (short stores), and matches the oracle."""
    import torch
    D, L, B, Hq, Hkv, S, W = 128, 4, 2, 8, 2, 16, 48
    kinds = [1, 0, 1, 1]
    lens = [1000, 380]
    steps = 8
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, 3, 0, 0, steps, seed=909)
    hist = [[inputs.qkv_bf16(w, l, b, 0, lens[b]) for b in range(B)] for l in range(L)]
    dec = [[[inputs.qkv_bf16(w, l, b, lens[b] + i, 1) for b in range(B)] for l in range(L)] for i in range(steps)]
    results = {}
    for pool in (0, 80):
        cache = make(L, B, Hq, Hkv, S, W, kinds, [n + steps + 4 for n in lens], max_new=8192, pool_pages=pool)
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
        results[pool] = np.stack(outs)
        if pool:
            total, free = cache.pages()
            # 3 retrieval layers x 2 KV heads x (ceil(1008/128) + ceil(388/128)) token blocks
            assert total == 80 and total - free == 3 * 2 * (8 + 4)
        cache.close()
    assert np.array_equal(results[0], results[80])
    scale = 1 / np.sqrt(D)
    for l in range(L):
        for b in range(B):
            o = OracleSeq(Hkv, D, S, W, lens[b] + steps + 4, [kinds[l]] * Hkv)
            o.append(hist[l][b][1], hist[l][b][2])
            for i in range(steps):
                o.append(dec[i][l][b][1], dec[i][l][b][2])
            want = o.rows(dec[steps - 1][l][b][0], [lens[b] + steps - 1], scale=scale)
            assert_close(results[80][steps - 1, l, b:b + 1], want, f"layer {l} seq {b}")


def test_pool_exhaustion_is_refused_and_reset_returns_pages():
    D, Hq, Hkv = 128, 4, 2
    w = inputs.Workload("t", 1, 2, Hq, Hkv, D, 4, 8, 1, 0, 0, 0, seed=77)
    # capacities of 1024 tokens each (16 pages per sequence at 2 heads), but only 10 pages in the pool
    cache = make(1, 2, Hq, Hkv, 4, 8, [1], [1024, 1024], pool_pages=10)
    assert cache.pages() == (10, 10)
    q0, k0, v0 = inputs.qkv_bf16(w, 0, 0, 0, 300)
    q1, k1, v1 = inputs.qkv_bf16(w, 0, 1, 0, 300)
    cache.kv_append(0, to_dev(k0), to_dev(v0), [300, 0])         # 3 blocks x 2 heads = 6 pages
    assert cache.pages() == (10, 4)
    with pytest.raises(binding.ZigzagError) as e:                  # 6 more do not fit
        cache.kv_append(0, to_dev(k1), to_dev(v1), [0, 300])
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    assert cache.pages() == (10, 4) and cache.len(0, 1) == 0 and cache.len(0, 0) == 300
    cache.kv_append(0, to_dev(k1[:256]), to_dev(v1[:256]), [0, 256])   # 4 pages: exactly what is left
    assert cache.pages() == (10, 0)
    # sequence 0 still decodes correctly from its pages; its step needs no new page (300 -> 301)
    o = OracleSeq(Hkv, D, 4, 8, 1024, [1, 1])
    o.append(k0, v0)
    qd, kd, vd = inputs.qkv_bf16(w, 0, 0, 300, 1)
    qe, ke, ve = inputs.qkv_bf16(w, 0, 1, 256, 1)
    dq = to_dev(np.concatenate([qd, qe]))
    out = dq.new_zeros(dq.shape)
    with pytest.raises(binding.ZigzagError) as e:                  # sequence 1 would need a new block
        cache.decode_step(0, dq, to_dev(np.concatenate([kd, ke])), to_dev(np.concatenate([vd, ve])), out)
    assert e.value.status == binding.ZZ_ERR_CAPACITY
    assert cache.len(0, 0) == 300 and cache.len(0, 1) == 256
    cache.reset(1)                                                 # its 4 pages come back
    assert cache.pages() == (10, 4)
    cache.kv_append(0, to_dev(k1[:100]), to_dev(v1[:100]), [0, 100])
    cache.decode_step(0, dq, to_dev(np.concatenate([kd, ke])), to_dev(np.concatenate([vd, ve])), out)
    o.append(kd, vd)
    got = to_bits(out)
    assert_close(got[0:1], o.rows(qd, [300], scale=1 / np.sqrt(D)), "seq 0 after refusals")
    o1 = OracleSeq(Hkv, D, 4, 8, 1024, [1, 1])
    o1.append(k1[:100], v1[:100])
    o1.append(ke, ve)
    assert_close(got[1:2], o1.rows(qe, [100], scale=1 / np.sqrt(D)), "seq 1 on recycled pages")
    assert cache.last_status() == 0
    cache.close()


def test_paged_export_import_roundtrip():
    D, Hq, Hkv, n = 128, 4, 2, 333
    w = inputs.Workload("t", 1, 1, Hq, Hkv, D, 4, 8, 1, 0, 0, 0, seed=78)
    q, k, v = inputs.qkv_bf16(w, 0, 0, 0, n)
    a = make(1, 1, Hq, Hkv, 4, 8, [1], [400], pool_pages=9)
    a.kv_append(0, to_dev(k), to_dev(v), [n])
    ek, ev, pos, ln = a.export(0, 0, binding.KIND_RETRIEVAL)
    assert ln == n and np.array_equal(ek[:, :n], np.transpose(k, (1, 0, 2))) and np.array_equal(
        ev[:, :n], np.transpose(v, (1, 0, 2)))
    b = make(1, 1, Hq, Hkv, 4, 8, [1], [400], pool_pages=9)
    b.import_(0, 0, binding.KIND_RETRIEVAL, ek, ev, pos, ln)
    assert b.len(0, 0) == n and b.pages() == (9, 9 - 6)
    dq = to_dev(q[n - 1:n])
    oa, ob = dq.new_zeros(dq.shape), dq.new_zeros(dq.shape)
    a.decode_attn(0, dq, oa)
    b.decode_attn(0, dq, ob)
    assert np.array_equal(to_bits(oa), to_bits(ob))
    a.close()
    b.close()


@pytest.mark.parametrize("paged", [False, True])
def test_million_token_store_maximum_splits(paged):
    """One KV head with a million tokens: the split plan runs into its limit of 120 splits, every
    CTA's range spans more than 32 pages (the paged kernel reloads its window of page ids) and a
    warp walks ~2000 tokens.  Decode rows against the oracle over the full history."""
    import oracle
    Hq, Hkv, S, W = 4, 1, 4, 12
    n, steps = 1_000_000, 2
    cap = n + steps
    pool = (cap + 127) // 128 if paged else 0
    cache = make(1, 1, Hq, Hkv, S, W, [1], [cap], max_new=65536, pool_pages=pool)
    hk = np.empty((cap, Hkv, D), np.uint16)
    hv = np.empty((cap, Hkv, D), np.uint16)
    done = 0
    while done < n:
        c = min(65536, n - done)
        hk[done:done + c] = inputs.normal_bf16((c, Hkv, D), 4321, 1, done)
        hv[done:done + c] = inputs.normal_bf16((c, Hkv, D), 4321, 2, done)
        cache.kv_append(0, to_dev(hk[done:done + c]), to_dev(hv[done:done + c]), [c])
        done += c
    for i in range(steps):
        q = inputs.normal_bf16((1, Hq, D), 4321, 3, i)
        hk[n + i] = inputs.normal_bf16((1, Hkv, D), 4321, 4, i)[0]
        hv[n + i] = inputs.normal_bf16((1, Hkv, D), 4321, 5, i)[0]
        dq = to_dev(q)
        out = dq.new_zeros(dq.shape)
        cache.decode_step(0, dq, to_dev(hk[n + i:n + i + 1]), to_dev(hv[n + i:n + i + 1]), out)
        want = oracle.attn_rows(q, [n + i], hk[:n + i + 1], hv[:n + i + 1], [1], S, W, 1 / np.sqrt(D))
        assert_close(to_bits(out), want, f"step {i}")
    assert cache.last_status() == 0 and cache.len(0, 0) == n + steps
    cache.close()
