"""The C-ABI library builds for sm_100a, loads, and exports every symbol the header declares
(no compute call is made here: that needs a GPU)."""
import ctypes
import os
import re

import numpy as np

import oracle
from oracle import VAL_DTYPE
import hostindex
from paper_2511_16138_b200 import build, lsmkv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    with open(os.path.join(ROOT, "include", "lsmkv.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lsmkv_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_batch_calls():
    syms = declared_symbols()
    for s in ("lsmkv_encode_batch", "lsmkv_probe_batch", "lsmkv_decode_batch", "lsmkv_create",
              "lsmkv_destroy", "lsmkv_last_status"):
        assert s in syms


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    for s in declared_symbols():
        assert hasattr(L, s), f"{s} declared in lsmkv.h but not exported"
    assert sorted(lsmkv.EXPORTS) == declared_symbols()


def test_binding_struct_layouts_match_the_header():
    assert ctypes.sizeof(lsmkv.GeomStruct) == 32
    assert ctypes.sizeof(lsmkv.RunStruct) == 56
    assert ctypes.sizeof(lsmkv.PoolStruct) == 16
    assert ctypes.sizeof(lsmkv.StatusStruct) == 56
    assert VAL_DTYPE.itemsize == lsmkv.VAL_BYTES == 16 and lsmkv.KEY_BYTES == 32
    assert lsmkv.lsmkv_format_version() == 1


def test_host_argument_validation_needs_no_gpu():
    L = lsmkv.lib()
    assert L.lsmkv_destroy(None) == 0
    assert L.lsmkv_create(None, None, 0) == lsmkv.EINVAL
    h = ctypes.c_void_p()
    bad = lsmkv.Geom(4, 8, 128, page_tokens=16, chunk_tokens=40).c()     # C not a multiple of P
    assert L.lsmkv_create(ctypes.byref(h), ctypes.byref(bad), 0) == lsmkv.EINVAL
    bad = lsmkv.Geom(4, 1, 3, elem_bytes=2, page_tokens=1, chunk_tokens=1).c()  # 6-byte pages
    assert L.lsmkv_create(ctypes.byref(h), ctypes.byref(bad), 0) == lsmkv.EINVAL
    assert lsmkv.strerror(lsmkv.ECAPACITY) == "output buffer too small"


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(lsmkv, "_lib", None)
    monkeypatch.setattr(lsmkv, "LIB_PATH", "/nonexistent/liblsmkv.so")
    try:
        lsmkv.lib()
    except ImportError as e:
        assert "missing" in str(e)
    else:
        raise AssertionError("expected ImportError")


def test_host_flush_and_merge_equal_the_oracle():
    rng = np.random.default_rng(0)
    keys = rng.integers(0, 2**64, (3000, 4), dtype=np.uint64)
    keys[:, 0] = rng.integers(0, 4, 3000)
    keys[:, 1] = rng.integers(0, 8, 3000)
    keys[1000:1500] = keys[:500]
    keys[0, 0] = 2**63 + 5
    vals = np.zeros(3000, dtype=VAL_DTYPE)
    vals["offset"] = np.arange(3000)
    k1, v1 = hostindex.flush(keys, vals)
    k2, v2 = oracle.flush(keys, vals)
    assert np.array_equal(k1, k2) and np.array_equal(v1, v2)
    runs = [hostindex.flush(keys[a:b], vals[a:b]) for a, b in ((0, 300), (200, 1800), (900, 3000))]
    m1 = hostindex.merge_runs(runs)
    m2 = oracle.merge_runs(runs)
    assert np.array_equal(m1[0], m2[0]) and np.array_equal(m1[1], m2[1])
