"""The workspace-free decode entry point (for callers that cannot allocate device memory, e.g.
a server that owns the whole device through its own pool) against the regular entry point and
against the fp64 oracle.

Collected last on purpose: it exercises a fixed scratch array shared by every call in the
process, so it must also pass after all other tests have run, and a failure here cannot hide
another test's result in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_12407_b200 import binding, build, inputs
from zz_testlib import MAX_ABS_TOL, REL_L2_TOL, to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def regular_path(w, lens, q_bits, kv):
    """Output of zz_decode_attn on a retrieval layer filled with the same K/V."""
    B = len(lens)
    cache = binding.ZigzagCache(1, B, w.n_q_heads, w.n_kv_heads, 4, 4, [1], [max(lens)] * B, max(lens) * B)
    ks = np.concatenate([kv[b][0] for b in range(B)])
    vs = np.concatenate([kv[b][1] for b in range(B)])
    cache.kv_append(0, to_dev(ks), to_dev(vs), list(lens))
    dq = to_dev(q_bits)
    out = torch.zeros_like(dq)
    cache.decode_attn(0, dq, out)
    torch.cuda.synchronize()
    got = to_bits(out)
    cache.close()
    return got


def close(got, want, what):
    assert np.all(np.isfinite(got)), what
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    mx = np.max(np.abs(got - want))
    assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL, f"{what}: rel_l2={rel:.3e} max_abs={mx:.3e}"


def run_case(Hq, Hkv, lens, seed, v_below_k=False, side_stream=False):
    """Two calls in a row (they share the scratch; the second must not see stale state), each
    compared with zz_decode_attn on the same stores and, element by element, with the oracle."""
    D, B = 128, len(lens)
    w = inputs.Workload("na", 1, B, Hq, Hkv, D, 4, 4, 1, 0, 0, 0, seed=seed)
    cap = max(lens)
    kv = [inputs.qkv_bf16(w, 0, b, 0, lens[b])[1:] for b in range(B)]
    # the caller's own stores: [batch, kv heads, capacity, 128]; v may lie below k in memory
    both = torch.zeros(2, B, Hkv, cap, D, dtype=torch.bfloat16, device="cuda")
    dk, dv = (both[1], both[0]) if v_below_k else (both[0], both[1])
    for b in range(B):
        dk[b, :, :lens[b]] = to_dev(np.ascontiguousarray(kv[b][0].transpose(1, 0, 2)))
        dv[b, :, :lens[b]] = to_dev(np.ascontiguousarray(kv[b][1].transpose(1, 0, 2)))
    stream = torch.cuda.Stream() if side_stream else None
    torch.cuda.synchronize()
    for call in range(2):
        q_bits = inputs.normal_bf16((B, Hq, D), seed, 900 + call)
        dq = to_dev(q_bits)
        out = torch.zeros_like(dq)
        torch.cuda.synchronize()
        binding.decode_attn_static(dq, dk, dv, out, lens, stream=stream)
        torch.cuda.synchronize()
        got = inputs.bf16_bits_to_f64(to_bits(out))
        close(got, inputs.bf16_bits_to_f64(regular_path(w, lens, q_bits, kv)), f"call {call} vs zz_decode_attn")
        for b in range(B):
            want = oracle.attn_rows(q_bits[b:b + 1], [lens[b] - 1], kv[b][0], kv[b][1], [1] * Hkv, 4, 4, w.scale)
            close(got[b:b + 1], want, f"call {call} seq {b} vs oracle")


def test_static_scratch_decode_matches_regular_entry_point_twice():
    mb, mrows, nbytes = binding.decode_attn_static_limits()
    assert mb >= 2 and mrows >= 64 and nbytes < 4 << 20
    run_case(32, 8, [9000, 3111], seed=4242)


@pytest.mark.parametrize("Hq,Hkv,lens", [
    (32, 8, [1]),                                    # a single key: one split, output written directly
    (32, 8, [200, 256]),                             # no split anywhere
    (4, 1, [300000]),                                # long enough to run into the 64-split cap
    (4, 4, [1 + 997 * b for b in range(16)]),        # the batch limit, 16 x 4 rows, ragged from one token up
    (16, 1, [5000, 77, 2500, 1]),                    # 16 query heads per KV head, 64 rows
])
def test_static_scratch_decode_at_its_limits(Hq, Hkv, lens):
    run_case(Hq, Hkv, lens, seed=77 + Hq + len(lens))


def test_static_scratch_decode_with_v_below_k_and_on_a_side_stream():
    run_case(8, 2, [4100, 9], seed=31, v_below_k=True, side_stream=True)


def test_static_scratch_rejects_oversized_problems():
    Hq, Hkv, D = 32, 8, 128
    q = torch.zeros(3, Hq, D, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(3, Hkv, 16, D, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.ZigzagError) as e:        # 3 * 32 rows > 64
        binding.decode_attn_static(q, k, k, torch.zeros_like(q), [16, 16, 16])
    assert e.value.status == binding.ZZ_ERR_WORKSPACE
    with pytest.raises(binding.ZigzagError) as e:        # length beyond the stores
        binding.decode_attn_static(q[:1], k[:1], k[:1], torch.zeros_like(q[:1]), [17])
    assert e.value.status == binding.ZZ_ERR_INVALID_ARG
    q17 = torch.zeros(17, 2, D, dtype=torch.bfloat16, device="cuda")
    k17 = torch.zeros(17, 1, 16, D, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.ZigzagError) as e:        # 17 sequences > 16
        binding.decode_attn_static(q17, k17, k17, torch.zeros_like(q17), [16] * 17)
    assert e.value.status == binding.ZZ_ERR_WORKSPACE
