"""Parity at the full sizes of the benchmark workloads, in the launch configurations the
benchmark times (same batch, heads, context lengths, chunking and calls; fewer layers, since the
launch shape does not depend on the layer count).  Outputs are checked on sampled rows the fp64
oracle can compute one by one: prefill rows at the sink / window / tile / chunk boundaries, every
row of the decode steps, and the ring stores bit for bit."""
import numpy as np
import pytest

import oracle
from paper_2508_12407_b200 import binding, build, inputs
from zz_testlib import assert_close, to_bits, to_dev

pytestmark = pytest.mark.gpu
D = 128


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def _rows(P, c, S, W, n_extra, rng):
    fixed = [0, 1, 127, 128, S - 1 - P, S - P, S + W - 1 - P, S + W - P, W - 1, W, c // 2 - 1, c // 2, c - 129,
             c - 128, c - 1]
    extra = rng.integers(0, c, size=n_extra).tolist()
    r = np.unique(np.clip(np.asarray(fixed + extra), 0, c - 1))
    return r


def run_full(w: inputs.Workload, kinds, lens, chunk, n_decode, kvk=None, prefilled=False, rows_per_call=6,
             decode_seqs=None, same_prompt_all_layers=False, paged=False, fp8=False):
    L, B, Hq, Hkv, S, W = len(kinds), len(lens), w.n_q_heads, w.n_kv_heads, w.sink, w.recent
    import torch
    scale = w.scale
    rng = np.random.default_rng(w.seed)
    cap = [int(n) + n_decode + 8 for n in lens]
    max_new = B * chunk if chunk else B
    kk = np.asarray(kvk).reshape(L, Hkv) if kvk is not None else np.repeat(np.asarray(kinds)[:, None], Hkv, axis=1)
    # paged: a pool with exactly the pages the run needs (one per retrieval head per 128 tokens)
    pool = int(kk.sum()) * sum((int(n) + n_decode + 127) // 128 for n in lens) if paged else 0
    cache = binding.ZigzagCache(L, B, Hq, Hkv, S, W, kinds, cap, max_new, kvhead_is_retrieval=kvk, pool_pages=pool,
                                kv_fp8=fp8)
    kv_kinds = [list(np.asarray(kvk).reshape(L, Hkv)[l]) if kvk is not None else [int(kinds[l])] * Hkv
                for l in range(L)]
    hist_k = [[np.zeros((cap[b], Hkv, D), np.uint16) for b in range(B)] for l in range(L)]
    hist_v = [[np.zeros((cap[b], Hkv, D), np.uint16) for b in range(B)] for l in range(L)]
    pos = np.zeros((L, B), dtype=np.int64)
    shared = {}

    def as_stored(l, x):
        """Rows as they read back from the stores: FP8 retrieval heads hold quantised values (exactly bf16 numbers)."""
        if not fp8:
            return x
        y = x.copy()
        for h in range(Hkv):
            if kv_kinds[l][h]:
                y[:, h] = oracle.fp8_stored_as_bf16_bits(np.ascontiguousarray(x[:, h]))
        return y

    for l in range(L):
        step = chunk if chunk else 8192
        done = np.zeros(B, dtype=np.int64)
        while (done < np.asarray(lens)).any():
            n_new = [int(min(step, lens[b] - done[b])) for b in range(B)]
            qs, ks, vs = [], [], []
            for b in range(B):
                if not n_new[b]:
                    continue
                lk = 0 if same_prompt_all_layers else l      # the prompt tensors may be shared by the layers
                if prefilled:                                # stores filled without attention: no queries
                    q = None
                    k = inputs.normal_bf16((n_new[b], Hkv, D), w.seed, 7, lk, inputs.T_K, b, int(done[b]))
                    v = inputs.normal_bf16((n_new[b], Hkv, D), w.seed, 7, lk, inputs.T_V, b, int(done[b]))
                elif l > 0 and same_prompt_all_layers:
                    q, k, v = shared[(b, int(done[b]))]
                else:
                    q, k, v = inputs.qkv_bf16(w, lk, b, int(done[b]), n_new[b])
                    if same_prompt_all_layers:
                        shared[(b, int(done[b]))] = (q, k, v)
                # the chunk attends to itself as given; what it leaves in the history is what the stores hold
                hist_k[l][b][done[b]:done[b] + n_new[b]] = k
                hist_v[l][b][done[b]:done[b] + n_new[b]] = v
                qs.append(q); ks.append(k); vs.append(v)
            dk, dv = to_dev(np.concatenate(ks)), to_dev(np.concatenate(vs))
            if not prefilled:
                dq = to_dev(np.concatenate(qs))
                out = torch.zeros_like(dq)
                cache.prefill_attn(l, dq, dk, dv, out, n_new)
                off, i = 0, 0
                for b in range(B):
                    c = n_new[b]
                    if not c:
                        continue
                    P = int(done[b])
                    rows = _rows(P, c, S, W, rows_per_call, rng)
                    got = to_bits(out[off + torch.as_tensor(rows, device=out.device)])
                    want = oracle.attn_rows(np.ascontiguousarray(qs[i][rows]), P + rows, hist_k[l][b][:P + c],
                                            hist_v[l][b][:P + c], kv_kinds[l], S, W, scale)
                    assert_close(got, want, f"{w.name} prefill layer {l} seq {b} at {P}")
                    off += c; i += 1
                del dq, out
            cache.kv_append(l, dk, dv, n_new)
            if fp8:
                i = 0
                for b in range(B):
                    if n_new[b]:
                        sl = slice(int(done[b]), int(done[b]) + n_new[b])
                        hist_k[l][b][sl] = as_stored(l, ks[i]); hist_v[l][b][sl] = as_stored(l, vs[i])
                        i += 1
            done += np.asarray(n_new)
        pos[l] = done
    # decode steps through the whole-stack call the benchmark times
    check_b = range(B) if decode_seqs is None else decode_seqs
    for step in range(n_decode):
        q = np.zeros((L, B, Hq, D), np.uint16); k = np.zeros((L, B, Hkv, D), np.uint16); v = np.zeros_like(k)
        for l in range(L):
            for b in range(B):
                qq, kk, vv = inputs.qkv_bf16(w, l, b, int(pos[l, b]), 1)
                q[l, b], k[l, b], v[l, b] = qq[0], kk[0], vv[0]
                hist_k[l][b][pos[l, b]] = as_stored(l, kk)[0]; hist_v[l][b][pos[l, b]] = as_stored(l, vv)[0]
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        out = torch.zeros_like(dq)
        cache.decode_step_all(dq, dk, dv, out)
        got = to_bits(out)
        pos += 1
        if step in (0, n_decode - 1):
            for l in range(L):
                for b in check_b:
                    t = int(pos[l, b]) - 1
                    want = oracle.attn_rows(q[l, b:b + 1], [t], hist_k[l][b][:t + 1], hist_v[l][b][:t + 1],
                                            kv_kinds[l], S, W, scale)
                    assert_close(got[l, b:b + 1], want, f"{w.name} decode step {step} layer {l} seq {b}")
    # stores: rings bit for bit against the simulated ring, a slice of the retrieval stores, lengths
    for l in range(L):
        s_heads = [h for h in range(Hkv) if not kv_kinds[l][h]]
        r_heads = [h for h in range(Hkv) if kv_kinds[l][h]]
        for b in (check_b if decode_seqs is not None else range(min(B, 2))):
            n = int(pos[l, b])
            if s_heads:
                ring = oracle.RingStore(len(s_heads), D, S, W)
                ring.append(np.ascontiguousarray(hist_k[l][b][:n][:, s_heads]),
                            np.ascontiguousarray(hist_v[l][b][:n][:, s_heads]))
                gk, gv, gpos, glen = cache.export(l, b, binding.KIND_STREAMING)
                assert glen == n and np.array_equal(gpos, ring.pos)
                assert np.array_equal(gk, ring.k) and np.array_equal(gv, ring.v)
            if r_heads and fp8:
                # the history holds the values the oracle's quantiser leaves in a store: the GPU's codes and scale
                # bytes must decode to exactly those (the codes themselves are compared in tests/test_gpu_fp8.py)
                gk, gv, gks, gvs, glen = cache.export_fp8(l, b)
                assert glen == n
                sl = slice(max(0, n - 3000), n)
                for got_c, got_s, hist in ((gk, gks, hist_k), (gv, gvs, hist_v)):
                    want_vals = inputs.bf16_bits_to_f64(np.ascontiguousarray(hist[l][b][sl][:, r_heads].transpose(1, 0, 2)))
                    assert np.array_equal(oracle.fp8_dequantize_rows(got_c[:, sl], got_s[:, sl]), want_vals)
            elif r_heads:
                gk, gv, gpos, glen = cache.export(l, b, binding.KIND_RETRIEVAL)
                assert glen == n and np.array_equal(gpos[:n], np.arange(n)) and (gpos[n:] == -1).all()
                sl = slice(max(0, n - 3000), n)
                assert np.array_equal(gk[:, sl], np.ascontiguousarray(hist_k[l][b][sl][:, r_heads]).transpose(1, 0, 2))
                assert np.array_equal(gv[:, :2000], np.ascontiguousarray(hist_v[l][b][:2000][:, r_heads]).transpose(1, 0, 2))
    assert cache.last_status() == 0
    if paged:
        assert cache.pages()[1] == 0          # every page of the exactly sized pool is in use
    cache.close()


def test_cfg2_32k_prefill_and_decode():
    w = inputs.WORKLOADS["cfg2"]
    run_full(w, [1, 0, 0, 1], [w.prefill_len], w.prefill_chunk, 4)


def test_cfg3_128k_chunked_prefill_and_decode():
    w = inputs.WORKLOADS["cfg3"]
    run_full(w, [1, 0], [w.prefill_len], w.prefill_chunk, 3, rows_per_call=1)


def test_cfg4_ragged_batch16_decode():
    w = inputs.WORKLOADS["cfg4"]
    lens = [int(x) for x in inputs.ragged_lengths(w)]
    run_full(w, [1, 0], lens, 0, 3, prefilled=True, decode_seqs=[0, 5, 11, 15])


def test_cfg5_64k_batch4_exclusive_and_mixed():
    w = inputs.WORKLOADS["cfg5"]
    kvk = np.stack([np.ones(8, np.uint8), np.zeros(8, np.uint8), inputs.mixed_kvhead_kinds(w)[0]])
    run_full(w, [1, 0, 0], [w.prefill_len] * w.batch, w.prefill_chunk, 2, kvk=kvk, rows_per_call=2,
             decode_seqs=[0, 3], same_prompt_all_layers=True)


def test_cfg3_128k_paged_stores():
    # the same 8K-chunked 128K prefill and decode with the retrieval store in 128-token pages
    w = inputs.WORKLOADS["cfg3"]
    run_full(w, [1, 0], [w.prefill_len], w.prefill_chunk, 3, rows_per_call=1, paged=True)


def test_cfg4_ragged_batch16_paged_stores():
    w = inputs.WORKLOADS["cfg4"]
    lens = [int(x) for x in inputs.ragged_lengths(w)]
    run_full(w, [1, 0], lens, 0, 3, prefilled=True, decode_seqs=[0, 5, 11, 15], paged=True)


def test_cfg2_32k_fp8_retrieval_stores():
    w = inputs.WORKLOADS["cfg2"]
    run_full(w, [1, 0, 1], [w.prefill_len], w.prefill_chunk, 4, fp8=True)


def test_cfg4_ragged_batch16_fp8_retrieval_stores():
    w = inputs.WORKLOADS["cfg4"]
    lens = [int(x) for x in inputs.ragged_lengths(w)]
    run_full(w, [1, 0], lens, 0, 3, prefilled=True, decode_seqs=[0, 5, 11, 15], fp8=True)


def test_cfg3_chunked_prefill_over_fp8_stores():
    # 8K chunks attending to an FP8 store that grows to 64K: the bf16 scratch path of the prefill
    w = inputs.WORKLOADS["cfg3"]
    run_full(w, [1, 0], [65536], w.prefill_chunk, 2, rows_per_call=1, fp8=True)
