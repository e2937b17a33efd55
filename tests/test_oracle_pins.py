"""Pins of the CPU oracle against things fixed by the paper and by mathematics.

None of these tests retypes the oracle's loops: they use hand-enumerated visible
sets, closed forms, special cases, a differently written brute force (explicit
score matrix, explicit mask matrix, long double, no max subtraction) and
invariants.  Citations are to the paper: full / streaming attention are the two
terms of Eq. 1 (Section 2.1); sink + recent window with the rest of the KV waived
is the streaming head of the Introduction; sink 128 / window 256 are the values of
Section 3.3.
"""
import os

import numpy as np
import pytest

import oracle
from paper_2508_12407_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, *vals = line.split()
                out[key] = [float(x) for x in vals]
    return out


def rand_qkv(n, Hq, Hkv, D, seed):
    q = inputs.normal_bf16((n, Hq, D), seed, 1)
    k = inputs.normal_bf16((n, Hkv, D), seed, 2)
    v = inputs.normal_bf16((n, Hkv, D), seed, 3)
    return q, k, v


def f64(b):
    return inputs.bf16_bits_to_f64(b)


def brute_force(q, k, v, kv_kind, S, W, scale):
    """Whole [n, n] score matrix per head, mask matrix from broadcasting, plain
    exp without max subtraction, long double.  Tiny inputs only."""
    n, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    Q = f64(q).astype(np.longdouble)
    K = f64(k).astype(np.longdouble)
    V = f64(v).astype(np.longdouble)
    T = np.arange(n)[:, None]
    J = np.arange(n)[None, :]
    causal = J <= T
    local = (J < S) | ((T - J) < W)
    out = np.zeros((n, Hq, D), dtype=np.longdouble)
    for h in range(Hq):
        g = h // G
        mask = causal if kv_kind[g] else (causal & local)
        scores = np.longdouble(scale) * (Q[:, h, :] @ K[:, g, :].T)
        e = np.where(mask, np.exp(scores), np.longdouble(0))
        out[:, h, :] = (e / e.sum(axis=1, keepdims=True)) @ V[:, g, :]
    return out.astype(np.float64)


# ---------------------------------------------------------------- visible set

def test_visible_sets_enumerated_by_hand():
    # S=2, W=3: the query at t=7 sees the sinks {0,1} and the last three keys {5,6,7}
    S, W = 2, 3
    assert [j for j in range(-1, 10) if oracle.visible(0, j, 7, S, W)] == [0, 1, 5, 6, 7]
    # t=3: sinks {0,1} and window {1,2,3}: no key counted twice
    assert [j for j in range(-1, 10) if oracle.visible(0, j, 3, S, W)] == [0, 1, 2, 3]
    # t=4: window {2,3,4} still touches the sinks; t=5: key 2 has just left the window
    assert [j for j in range(-1, 10) if oracle.visible(0, j, 4, S, W)] == [0, 1, 2, 3, 4]
    assert [j for j in range(-1, 10) if oracle.visible(0, j, 5, S, W)] == [0, 1, 3, 4, 5]
    # a retrieval head sees the whole causal prefix
    assert [j for j in range(-1, 10) if oracle.visible(1, j, 4, S, W)] == [0, 1, 2, 3, 4]
    # no sinks, window of one: only the current token
    assert [j for j in range(-1, 10) if oracle.visible(0, j, 6, 0, 1)] == [6]


def test_visible_count_closed_form_at_paper_setting():
    g = golden()
    S, W = int(g["sink"][0]), int(g["window"][0])
    assert (S, W) == (128, 256)
    for t in [0, 1, S - 1, S, S + 1, S + W - 2, S + W - 1, S + W, S + W + 1, 5000]:
        assert oracle.visible_count(0, t, S, W) == min(t + 1, S + W)
        assert oracle.visible_count(1, t, S, W) == t + 1
    for (S, W) in [(0, 1), (3, 5), (64, 256), (1, 1)]:
        for t in range(0, 3 * (S + W) + 2):
            assert oracle.visible_count(0, t, S, W) == min(t + 1, S + W)


def test_slot_function_and_ring_positions():
    S, W = 3, 4
    # sinks keep their slot; recent tokens cycle through the W slots after them
    assert [oracle.slot(t, S, W) for t in range(12)] == [0, 1, 2, 3, 4, 5, 6, 3, 4, 5, 6, 3]
    Hkv, D = 2, 8
    ring = oracle.RingStore(Hkv, D, S, W)
    _, k, v = rand_qkv(40, 2, Hkv, D, 11)
    for n in range(1, 41):
        ring.append(k[n - 1:n], v[n - 1:n])
        assert ring.len == n
        held = sorted(int(p) for p in ring.pos if p >= 0)
        expect = sorted(set(range(min(S, n))) | set(range(max(S, n - W), n)))
        assert held == expect
        for sl, p in enumerate(ring.pos):
            if p >= 0:  # the slot holds exactly the bytes of token p
                assert np.array_equal(ring.k[:, sl, :], k[p])
                assert np.array_equal(ring.v[:, sl, :], v[p])


def test_ring_chunked_append_equals_token_by_token():
    S, W, Hkv, D = 4, 6, 2, 8
    _, k, v = rand_qkv(57, 2, Hkv, D, 12)
    a = oracle.RingStore(Hkv, D, S, W)
    for i in range(57):
        a.append(k[i:i + 1], v[i:i + 1])
    b = oracle.RingStore(Hkv, D, S, W)
    off = 0
    for c in inputs.random_chunking(57, 5, 1, max_chunk=23):
        b.append(k[off:off + c], v[off:off + c])
        off += c
    assert np.array_equal(a.k, b.k) and np.array_equal(a.v, b.v)
    assert np.array_equal(a.pos, b.pos) and a.len == b.len == 57


def test_full_store_append_and_overflow():
    Hkv, D = 2, 8
    _, k, v = rand_qkv(10, 2, Hkv, D, 13)
    st = oracle.FullStore(Hkv, D, 10)
    st.append(k[:4], v[:4])
    st.append(k[4:9], v[4:9])
    assert st.len == 9
    for j in range(9):
        assert np.array_equal(st.k[:, j, :], k[j]) and np.array_equal(st.v[:, j, :], v[j])
    assert list(st.pos) == list(range(9)) + [-1]
    before = st.k.copy()
    with pytest.raises(ValueError):
        st.append(k[:2], v[:2])
    assert st.len == 9 and np.array_equal(st.k, before)


# ---------------------------------------------------------------- attention rows

@pytest.mark.parametrize("S,W", [(0, 1), (2, 3), (4, 8), (5, 64)])
@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 1), (8, 2)])
def test_brute_force_tiny(S, W, Hq, Hkv):
    n, D = 48, 8
    q, k, v = rand_qkv(n, Hq, Hkv, D, 21 + S)
    scale = 0.37
    for kinds in ([1] * Hkv, [0] * Hkv, [i % 2 for i in range(Hkv)]):
        got = oracle.attn_rows(q, np.arange(n), k, v, kinds, S, W, scale)
        want = brute_force(q, k, v, kinds, S, W, scale)
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)


def test_softmax_rows_sum_to_one():
    n, Hq, Hkv, D = 300, 4, 2, 16
    q, k, v = rand_qkv(n, Hq, Hkv, D, 31)
    for kinds in ([1, 1], [0, 0], [1, 0]):
        _, psum = oracle.attn_rows(q, np.arange(n), k, v, kinds, 16, 32, 0.25, return_psum=True)
        assert np.max(np.abs(psum - 1.0)) < 1e-12


def test_zero_query_gives_mean_of_visible_values():
    # closed form: q = 0 -> all scores equal -> o_t = arithmetic mean of v_j over V(t);
    # V(t) written out literally: sinks {0..S-1} and the last W keys
    n, Hq, Hkv, D = 40, 2, 1, 8
    S, W = 3, 5
    _, k, v = rand_qkv(n, Hq, Hkv, D, 41)
    q = np.zeros((n, Hq, D), dtype=np.uint16)
    V = f64(v)[:, 0, :]
    got_s = oracle.attn_rows(q, np.arange(n), k, v, [0], S, W, 1.0)
    got_r = oracle.attn_rows(q, np.arange(n), k, v, [1], S, W, 1.0)
    for t in range(n):
        if t < S + W:
            vis = list(range(t + 1))
        else:
            vis = [0, 1, 2] + [t - 4, t - 3, t - 2, t - 1, t]
        np.testing.assert_allclose(got_s[t, 0], V[vis].mean(axis=0), rtol=0, atol=1e-13)
        np.testing.assert_allclose(got_r[t, 1], V[: t + 1].mean(axis=0), rtol=0, atol=1e-13)


def test_dominant_key_selects_its_value_iff_visible():
    # k_j = c*q for one j with c large: the softmax collapses onto j when j is in V(t)
    n, D, S, W = 30, 16, 2, 4
    q, k, v = rand_qkv(n, 1, 1, D, 51)
    t = n - 1
    qt = f64(q)[t, 0]
    for j, in_stream in [(0, True), (1, True), (2, False), (10, False), (25, False),
                         (26, True), (29, True)]:
        k2 = k.copy()
        k2[j, 0] = inputs.f32_to_bf16_bits((qt * 64.0).astype(np.float32))
        o_s = oracle.attn_rows(q[t:t + 1], [t], k2, v, [0], S, W, 1.0)[0, 0]
        o_r = oracle.attn_rows(q[t:t + 1], [t], k2, v, [1], S, W, 1.0)[0, 0]
        vj = f64(v)[j, 0]
        assert np.allclose(o_r, vj, atol=1e-9)           # full attention always finds it
        assert np.allclose(o_s, vj, atol=1e-9) == in_stream


def test_scale_and_sign_of_scores():
    # two keys, D=1: weights are exp(scale*q*k_j) normalised -- closed form with numbers
    # q = 2, k = (1, -1), v = (1, 0), scale = 0.5 -> p0 = e^1/(e^1+e^-1)
    one, mone, two, zero = 0x3F80, 0xBF80, 0x4000, 0x0000
    q = np.array([[[zero]], [[two]]], dtype=np.uint16)
    k = np.array([[[one]], [[mone]]], dtype=np.uint16)
    v = np.array([[[one]], [[zero]]], dtype=np.uint16)
    o = oracle.attn_rows(q, [0, 1], k, v, [1], 0, 1, 0.5)
    assert o[0, 0, 0] == 1.0
    assert abs(o[1, 0, 0] - np.e / (np.e + 1 / np.e)) < 1e-15


def test_window_covering_context_equals_full_attention_bitwise():
    n, Hq, Hkv, D = 200, 4, 2, 16
    q, k, v = rand_qkv(n, Hq, Hkv, D, 61)
    full = oracle.attn_rows(q, np.arange(n), k, v, [1, 1], 0, 1, 0.3)
    for S, W in [(0, n), (n, 1), (50, 150), (64, 256)]:
        stream = oracle.attn_rows(q, np.arange(n), k, v, [0, 0], S, W, 0.3)
        assert np.array_equal(full, stream)
    short = oracle.attn_rows(q, np.arange(n), k, v, [0, 0], 50, 149, 0.3)
    assert np.array_equal(full[:199], short[:199]) and not np.array_equal(full[199], short[199])


def test_no_sink_window_one_returns_current_value():
    n, Hq, Hkv, D = 20, 2, 1, 8
    q, k, v = rand_qkv(n, Hq, Hkv, D, 71)
    o = oracle.attn_rows(q, np.arange(n), k, v, [0], 0, 1, 0.5)
    assert np.array_equal(o[:, 0, :], f64(v)[:, 0, :]) and np.array_equal(o[:, 1, :], f64(v)[:, 0, :])


def test_decode_step_equals_prefill_row_and_chunking():
    # a decode step at position t is the row t of a (t+1)-token prefill; rows do not
    # depend on how the prompt was chunked (each row only names its own position)
    n, Hq, Hkv, D, S, W = 90, 4, 2, 16, 4, 16
    q, k, v = rand_qkv(n, Hq, Hkv, D, 81)
    for kinds in ([1, 1], [0, 0]):
        whole = oracle.attn_rows(q, np.arange(n), k, v, kinds, S, W, 0.2)
        for t in [0, 3, 4, 19, 20, 21, 89]:
            step = oracle.attn_rows(q[t:t + 1], [t], k[: t + 1], v[: t + 1], kinds, S, W, 0.2)
            assert np.array_equal(step[0], whole[t])
        off, parts = 0, []
        for c in inputs.random_chunking(n, 9, 2, max_chunk=40):
            parts.append(oracle.attn_rows(q[off:off + c], np.arange(off, off + c),
                                          k[: off + c], v[: off + c], kinds, S, W, 0.2))
            off += c
        assert np.array_equal(np.concatenate(parts, axis=0), whole)


def test_ring_route_equals_history_route():
    n, Hq, Hkv, D, S, W = 120, 4, 2, 16, 5, 12
    q, k, v = rand_qkv(n, Hq, Hkv, D, 91)
    ring = oracle.RingStore(Hkv, D, S, W)
    full = oracle.FullStore(Hkv, D, n)
    for t in range(n):
        ring.append(k[t:t + 1], v[t:t + 1])
        full.append(k[t:t + 1], v[t:t + 1])
        want_s = oracle.attn_rows(q[t:t + 1], [t], k[: t + 1], v[: t + 1], [0, 0], S, W, 0.2)[0]
        got_s = oracle.attn_from_slots(q[t], t, ring.k, ring.v, ring.pos, [0, 0], S, W, 0.2)
        # same keys, different visiting order -> equal up to summation order
        np.testing.assert_allclose(got_s, want_s, rtol=0, atol=1e-13)
        if t < S + W:   # ring not yet wrapped: same order, identical bits
            assert np.array_equal(got_s, want_s)
        want_r = oracle.attn_rows(q[t:t + 1], [t], k[: t + 1], v[: t + 1], [1, 1], S, W, 0.2)[0]
        got_r = oracle.attn_from_slots(q[t], t, full.k, full.v, full.pos, [1, 1], S, W, 0.2)
        assert np.array_equal(got_r, want_r)


def test_slot_permutation_invariance():
    n, Hq, Hkv, D, S, W = 60, 2, 1, 8, 3, 9
    q, k, v = rand_qkv(n, Hq, Hkv, D, 95)
    ring = oracle.RingStore(Hkv, D, S, W)
    ring.append(k, v)
    base = oracle.attn_from_slots(q[n - 1], n - 1, ring.k, ring.v, ring.pos, [0], S, W, 0.3)
    perm = np.random.default_rng(3).permutation(S + W)
    got = oracle.attn_from_slots(q[n - 1], n - 1, np.ascontiguousarray(ring.k[:, perm]),
                                 np.ascontiguousarray(ring.v[:, perm]), ring.pos[perm],
                                 [0], S, W, 0.3)
    np.testing.assert_allclose(got, base, rtol=0, atol=1e-12)


def test_gqa_replication():
    n, Hq, Hkv, D = 64, 8, 2, 16
    q, k, v = rand_qkv(n, Hq, Hkv, D, 97)
    G = Hq // Hkv
    k_rep = np.ascontiguousarray(np.repeat(k, G, axis=1))
    v_rep = np.ascontiguousarray(np.repeat(v, G, axis=1))
    for kinds in ([1, 1], [0, 1]):
        a = oracle.attn_rows(q, np.arange(n), k, v, kinds, 4, 8, 0.25)
        b = oracle.attn_rows(q, np.arange(n), k_rep, v_rep, np.repeat(kinds, G), 4, 8, 0.25)
        assert np.array_equal(a, b)
    # heads 0..3 use KV head 0, heads 4..7 KV head 1 (contiguous groups): swapping the
    # KV heads swaps which group sees what
    sw = oracle.attn_rows(q, np.arange(n), np.ascontiguousarray(k[:, ::-1]),
                          np.ascontiguousarray(v[:, ::-1]), [1, 1], 4, 8, 0.25)
    q_sw = np.ascontiguousarray(np.concatenate([q[:, 4:], q[:, :4]], axis=1))
    ref = oracle.attn_rows(q_sw, np.arange(n), k, v, [1, 1], 4, 8, 0.25)
    assert np.array_equal(sw[:, :4], ref[:, 4:]) and np.array_equal(sw[:, 4:], ref[:, :4])


def test_mixed_layer_equals_per_head_kinds():
    # Eq. 1 with alpha in {0, 1}: a mixed layer is full attention on its retrieval heads
    # and streaming attention on the others, head by head
    n, Hq, Hkv, D, S, W = 80, 8, 4, 16, 3, 10
    q, k, v = rand_qkv(n, Hq, Hkv, D, 99)
    kinds = [1, 0, 0, 1]
    mixed = oracle.attn_rows(q, np.arange(n), k, v, kinds, S, W, 0.2)
    all_r = oracle.attn_rows(q, np.arange(n), k, v, [1] * 4, S, W, 0.2)
    all_s = oracle.attn_rows(q, np.arange(n), k, v, [0] * 4, S, W, 0.2)
    for h in range(Hq):
        src = all_r if kinds[h // 2] else all_s
        assert np.array_equal(mixed[:, h], src[:, h])
    assert not np.array_equal(all_r[n - 1], all_s[n - 1])


def test_transposed_operands_would_fail():
    # value and key roles are distinguishable: swapping K and V changes the result
    n, Hq, Hkv, D = 24, 1, 1, 8
    q, k, v = rand_qkv(n, Hq, Hkv, D, 103)
    a = oracle.attn_rows(q, np.arange(n), k, v, [1], 0, 1, 0.5)
    b = brute_force(q, v, k, [1], 0, 1, 0.5)
    assert not np.allclose(a, b)
    # D-ordering: o lives in value space -- a one-hot value dimension shows up in that dimension
    v2 = np.zeros_like(v)
    v2[:, 0, 5] = 0x3F80
    o = oracle.attn_rows(q, np.arange(n), k, v2, [1], 0, 1, 0.5)
    assert np.allclose(o[:, 0, 5], 1.0) and np.allclose(np.delete(o[:, 0], 5, axis=1), 0.0)


def test_bad_arguments_rejected():
    q, k, v = rand_qkv(4, 2, 1, 8, 1)
    with pytest.raises(ValueError):
        oracle.attn_rows(q, [0, 1, 2, 4], k, v, [1], 0, 1, 1.0)      # row beyond the history
    with pytest.raises(ValueError):
        oracle.attn_rows(q, [0, 1, 2, 3], k, v, [1], 0, 0, 1.0)      # empty window


def test_input_generator_is_deterministic_and_bf16_exact():
    a = inputs.normal_bf16((1000,), 5, 1, 2)
    b = inputs.normal_bf16((1000,), 5, 1, 2)
    c = inputs.normal_bf16((1000,), 5, 1, 3)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    x = f64(a)
    assert abs(x.mean()) < 0.15 and 0.85 < x.std() < 1.15
    # RNE: 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0)
    t = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0], dtype=np.float32)
    assert list(inputs.f32_to_bf16_bits(t)) == [0x3F80, 0x3F82, 0xC020, 0x0000]
