"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, and validates configurations without touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2508_12407_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "zigzag.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zz_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_exported(lib):
    names = declared_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), f"{n} declared in zigzag.h but not exported"
        assert n in binding.SYMBOLS, f"{n} has no binding"


def test_version_and_status_strings(lib):
    assert binding.version() >= 100
    seen = set()
    for code in [0, -1, -2, -3, -4, -5, -6]:
        s = binding.status_str(code)
        assert s and s != "unknown status" and s not in seen
        seen.add(s)
    assert binding.status_str(-99) == "unknown status"


def make_cfg(**kw):
    L, B = kw.get("L", 2), kw.get("B", 1)
    kinds = np.array(kw.get("kinds", [1, 0]), dtype=np.uint8)
    cap = np.array(kw.get("cap", [1024] * B), dtype=np.int32)
    cfg = binding.ZZConfig(L, B, kw.get("Hq", 8), kw.get("Hkv", 2), kw.get("D", 128), kw.get("S", 64),
                           kw.get("W", 256), kw.get("max_new", 2048), kw.get("scale", 0.088),
                           kinds.ctypes.data, None, cap.ctypes.data, kw.get("fp8", 0))
    cfg._keep = (kinds, cap)
    return cfg


def query(lib, cfg):
    a, w = ctypes.c_size_t(0), ctypes.c_size_t(0)
    rc = lib.zz_cache_query(ctypes.byref(cfg), ctypes.byref(a), ctypes.byref(w))
    return rc, a.value, w.value


def test_query_sizes(lib):
    rc, a, w = query(lib, make_cfg())
    assert rc == 0
    # layer 0 retrieval: 2 heads * 1024 slots * 128 * 2 B for K and for V; layer 1: ring of 320 slots
    expect = 2 * (2 * 1024 * 256) + 2 * (2 * 320 * 256)
    assert expect <= a <= expect + 128 * 256 + 256
    assert w > 0 and a % 256 == 0 and w % 256 == 0


@pytest.mark.parametrize("kw,code", [
    (dict(D=96), binding.ZZ_ERR_UNSUPPORTED),
    (dict(D=256), binding.ZZ_ERR_UNSUPPORTED),
    (dict(D=64, fp8=1), binding.ZZ_ERR_UNSUPPORTED),
    (dict(fp8=2), binding.ZZ_ERR_INVALID_ARG),
    (dict(Hq=6, Hkv=4), binding.ZZ_ERR_UNSUPPORTED),
    (dict(Hq=34, Hkv=2), binding.ZZ_ERR_UNSUPPORTED),
    (dict(B=65, cap=[8] * 65, max_new=100), binding.ZZ_ERR_UNSUPPORTED),
    (dict(W=0), binding.ZZ_ERR_INVALID_ARG),
    (dict(S=-1), binding.ZZ_ERR_INVALID_ARG),
    (dict(cap=[0]), binding.ZZ_ERR_INVALID_ARG),
    (dict(scale=0.0), binding.ZZ_ERR_INVALID_ARG),
    (dict(max_new=0), binding.ZZ_ERR_INVALID_ARG),
])
def test_query_rejects_bad_configs(lib, kw, code):
    rc, _, _ = query(lib, make_cfg(**kw))
    assert rc == code


def test_query_sizes_head_dim_64_fp8_and_paged(lib):
    rc, a, w = query(lib, make_cfg(D=64))
    assert rc == 0
    expect = 2 * (2 * 1024 * 128) + 2 * (2 * 320 * 128)        # rows of 64 bf16
    assert expect <= a <= expect + 128 * 128 + 256
    # FP8 retrieval stores: 128 code bytes + 1 scale byte per row, then one layer's worth of bf16 scratch
    rc, a8, _ = query(lib, make_cfg(fp8=1))
    assert rc == 0
    codes = 2 * (2 * 1024 * 128) + 2 * (2 * 1024)
    ring = 2 * (2 * 320 * 256)
    scratch = 2 * (2 * 1024 * 256)
    assert codes + ring + scratch <= a8 <= codes + ring + scratch + 4 * 256 + 128 * 256 + 256
    a2, w2 = ctypes.c_size_t(0), ctypes.c_size_t(0)
    cfg = make_cfg(D=64)
    assert lib.zz_cache_query_paged(ctypes.byref(cfg), 8, ctypes.byref(a2), ctypes.byref(w2)) == binding.ZZ_ERR_UNSUPPORTED
    cfg = make_cfg(fp8=1)
    assert lib.zz_cache_query_paged(ctypes.byref(cfg), 8, ctypes.byref(a2), ctypes.byref(w2)) == binding.ZZ_ERR_UNSUPPORTED


def test_null_arguments(lib):
    assert lib.zz_cache_query(None, None, None) == binding.ZZ_ERR_INVALID_ARG
    cfg = make_cfg()
    assert lib.zz_cache_query(ctypes.byref(cfg), None, None) == binding.ZZ_ERR_INVALID_ARG
    assert lib.zz_cache_destroy(None) == binding.ZZ_ERR_INVALID_ARG
    assert lib.zz_decode_attn(None, 0, None, None, None) == binding.ZZ_ERR_INVALID_ARG
    assert lib.zz_kv_append(None, 0, None, None, None, None) == binding.ZZ_ERR_INVALID_ARG
    assert lib.zz_prefill_attn(None, 0, None, None, None, None, None, None) == binding.ZZ_ERR_INVALID_ARG
    assert lib.zz_get_last_status(None, None) == binding.ZZ_ERR_INVALID_ARG
    assert lib.zz_stage_bytes(None, 5) == 0


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    # no fallback of any kind: a missing extension is an ImportError that says how to build it
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libzigzag_b200.so"))
    with pytest.raises(ImportError) as e:
        binding.load()
    assert "build" in str(e.value)


def test_no_product_module_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2508_12407_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f), errors="ignore").read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, flags=re.M), f
                assert "zz_oracle" not in text, f


def test_paged_query_sizes_pool_and_table(lib):
    cfg = make_cfg(L=3, B=2, kinds=[1, 0, 1], cap=[1000, 300], Hq=8, Hkv=2, S=16, W=48)
    rc0, a0, w0 = query(lib, cfg)
    assert rc0 == 0
    a, w = ctypes.c_size_t(0), ctypes.c_size_t(0)
    assert lib.zz_cache_query_paged(ctypes.byref(cfg), 0, ctypes.byref(a), ctypes.byref(w)) == binding.ZZ_ERR_INVALID_ARG
    pool = 40
    assert lib.zz_cache_query_paged(ctypes.byref(cfg), pool, ctypes.byref(a), ctypes.byref(w)) == 0
    # arena: the contiguous retrieval stores (2 layers x 2 heads x (1000 + 300) slots x K and V) are
    # replaced by the pool of 64 KB pages; the rings stay
    contiguous = 2 * 2 * (1000 + 300) * 128 * 2 * 2
    assert abs((a0 - contiguous + pool * 65536) - a.value) <= 512
    # workspace: + the page table, 2 retrieval layers x 2 heads x (ceil(1000/128) + ceil(300/128)) entries
    entries = 2 * 2 * (8 + 3)
    assert 0 <= (w.value - w0) - entries * 4 <= 512
