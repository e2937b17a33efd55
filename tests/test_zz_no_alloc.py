"""The workspace-free decode entry point (for callers that cannot allocate device memory, e.g.
a server that owns the whole device through its own pool) against the regular entry point.

Collected last on purpose: it exercises a fixed scratch array shared by every call in the
process, so it must also pass after all other tests have run, and a failure here cannot hide
another test's result in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

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


def test_static_scratch_decode_matches_regular_entry_point_twice():
    mb, mrows, nbytes = binding.decode_attn_static_limits()
    assert mb >= 2 and mrows >= 64 and nbytes < 4 << 20
    Hq, Hkv, D = 32, 8, 128
    w = inputs.Workload("na", 1, 2, Hq, Hkv, D, 4, 4, 1, 0, 0, 0, seed=4242)
    lens = [9000, 3111]
    cap = max(lens)
    kv = [inputs.qkv_bf16(w, 0, b, 0, lens[b])[1:] for b in range(2)]
    # the caller's own stores: [batch, kv heads, capacity, 128]
    k_store = np.zeros((2, Hkv, cap, D), dtype=np.uint16)
    v_store = np.zeros((2, Hkv, cap, D), dtype=np.uint16)
    for b in range(2):
        k_store[b, :, :lens[b]] = kv[b][0].transpose(1, 0, 2)
        v_store[b, :, :lens[b]] = kv[b][1].transpose(1, 0, 2)
    dk, dv = to_dev(k_store), to_dev(v_store)
    for call in range(2):   # two calls in a row share the scratch; the second must not see stale state
        q_bits = inputs.normal_bf16((2, Hq, D), 4242, 900 + call)
        want = inputs.bf16_bits_to_f64(regular_path(w, lens, q_bits, kv))
        dq = to_dev(q_bits)
        out = torch.zeros_like(dq)
        binding.decode_attn_static(dq, dk, dv, out, lens)
        torch.cuda.synchronize()
        got = inputs.bf16_bits_to_f64(to_bits(out))
        assert np.all(np.isfinite(got))
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert rel <= REL_L2_TOL and np.max(np.abs(got - want)) <= MAX_ABS_TOL, (call, rel)


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
