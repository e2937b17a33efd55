"""Failure detection on the device, in the form that leaves the GPU usable: a bounded wait that
runs out returns a status, and memory outside what the library was given stays untouched."""
import numpy as np
import pytest
import torch

from paper_2508_12407_b200 import binding, build, inputs
from zz_testlib import to_bits, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.load()


def test_bounded_wait_runs_out_and_reports_timeout():
    cache = binding.ZigzagCache(1, 1, 4, 1, 4, 8, [1], [64], 64)
    assert cache.last_status() == binding.ZZ_OK
    cache.selftest_wait_timeout(1000)            # a barrier nothing completes: the wait gives up
    assert cache.last_status() == binding.ZZ_ERR_TIMEOUT
    assert cache.last_status() == binding.ZZ_OK  # reading clears the word
    assert binding.status_str(binding.ZZ_ERR_TIMEOUT) == "bounded device-side wait expired"
    # the context is still usable: a normal decode step runs and matches itself on a second cache
    w = inputs.Workload("t", 1, 1, 4, 1, 128, 4, 8, 1, 0, 0, 1, seed=11)
    q, k, v = inputs.qkv_bf16(w, 0, 0, 0, 40)
    cache.kv_append(0, to_dev(k), to_dev(v), [40])
    dq = to_dev(q[39:40])
    out = torch.zeros_like(dq)
    cache.decode_attn(0, dq, out)
    torch.cuda.synchronize()
    assert np.all(np.isfinite(inputs.bf16_bits_to_f64(to_bits(out))))
    assert cache.last_status() == binding.ZZ_OK
    with pytest.raises(binding.ZigzagError):
        cache.selftest_wait_timeout(0)
    cache.close()


def test_guard_bands_catch_a_write_outside_the_workspace():
    # the detector itself: a byte changed by the host side of the test (never by a kernel) is seen
    cache = binding.ZigzagCache(1, 1, 4, 1, 4, 8, [1], [64], 64)
    assert cache.guard_bytes > 0 and cache.guards_intact()
    cache._work_alloc[cache.guard_bytes - 1] = 0
    assert not cache.guards_intact()
    cache._work_alloc[cache.guard_bytes - 1] = binding.GUARD_BYTE
    assert cache.guards_intact()
    cache.close()
