"""Host-buffer entry points: the same kernels fed from pinned host memory must give the same
bits as the device-pointer calls."""
import numpy as np
import pytest

from paper_2508_12407_b200 import binding, build, inputs
from zz_testlib import to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def _pinned(bits):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.pin_memory()


def test_host_entries_match_device_entries():
    import torch
    D, L, B, Hq, Hkv, S, W = 128, 3, 2, 8, 2, 16, 48
    kinds = [1, 0, 1]
    C = 300
    w = inputs.Workload("t", L, B, Hq, Hkv, D, S, W, 2, 0, 0, 4, seed=99)
    caches = [binding.ZigzagCache(L, B, Hq, Hkv, S, W, kinds, [C + 16] * B, B * C) for _ in range(2)]
    dev_c, host_c = caches
    stage = torch.empty(max(host_c.stage_bytes(B * C), host_c.stage_bytes(L * B)), dtype=torch.uint8, device="cuda:0")
    # prefill: device path vs zz_prefill_host
    for l in range(L):
        qs, ks, vs = zip(*[inputs.qkv_bf16(w, l, b, 0, C) for b in range(B)])
        q, k, v = np.concatenate(qs), np.concatenate(ks), np.concatenate(vs)
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        out = torch.zeros_like(dq)
        dev_c.prefill_attn(l, dq, dk, dv, out, [C] * B)
        dev_c.kv_append(l, dk, dv, [C] * B)
        ho = _pinned(np.zeros_like(q))
        host_c.prefill_host(l, _pinned(q), _pinned(k), _pinned(v), ho, [C] * B, stage)
        torch.cuda.synchronize()
        assert np.array_equal(to_bits(out), to_bits(ho))
    # one decode step through the whole-stack host entry, one through the per-layer host entry
    for step in range(3):
        qkv = [[inputs.qkv_bf16(w, l, b, C + step, 1) for b in range(B)] for l in range(L)]
        q = np.stack([np.concatenate([qkv[l][b][0] for b in range(B)]) for l in range(L)])
        k = np.stack([np.concatenate([qkv[l][b][1] for b in range(B)]) for l in range(L)])
        v = np.stack([np.concatenate([qkv[l][b][2] for b in range(B)]) for l in range(L)])
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        out = torch.zeros_like(dq)
        dev_c.decode_step_all(dq, dk, dv, out)
        ho = _pinned(np.zeros_like(q))
        hq, hk, hv = _pinned(q), _pinned(k), _pinned(v)
        if step == 0:
            host_c.decode_step_all_host(hq, hk, hv, ho, stage)
        elif step == 2:
            # q, k, v back to back in one pinned buffer: the library sends them in one copy
            buf = torch.empty(hq.numel() + hk.numel() + hv.numel(), dtype=hq.dtype).pin_memory()
            nq, nk = hq.numel(), hk.numel()
            bq, bk, bv = buf[:nq].view(hq.shape), buf[nq:nq + nk].view(hk.shape), buf[nq + nk:].view(hv.shape)
            bq.copy_(hq); bk.copy_(hk); bv.copy_(hv)
            assert bk.data_ptr() == bq.data_ptr() + nq * 2 and bv.data_ptr() == bk.data_ptr() + nk * 2
            host_c.decode_step_all_host(bq, bk, bv, ho, stage)
        else:
            for l in range(L):
                host_c.decode_step_host(l, hq[l], hk[l], hv[l], ho[l], stage)
        torch.cuda.synchronize()
        assert np.array_equal(to_bits(out), to_bits(ho))
    assert dev_c.last_status() == 0 and host_c.last_status() == 0
    for c in caches:
        c.close()
