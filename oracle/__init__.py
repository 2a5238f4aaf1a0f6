"""CPU oracle for the batch codec and the longest-cached-prefix probe.

TEST INFRASTRUCTURE ONLY: a thin ctypes wrapper over ``lsmkv_oracle.c`` (plain C, compiled
with gcc). It shares no code with the CUDA library and never imports it. Only the tests, the
smoke check and the benchmark's CPU-baseline leg may use it; the product path must not.

Array conventions (numpy, little-endian host):
  keys   uint64 [n, 4]                       (w0, w1, w2, w3)
  vals   VAL_DTYPE [n]                       {file_id u32, reserved u32, offset u64}
  pool   uint8  [2L, num_pages, page_bytes]  K of layers 0..L-1, then V of layers 0..L-1
  runs   list of (keys, vals), newest first
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lsmkv_oracle.c")
_LIB = os.path.join(_HERE, "_build", "liblsmkv_oracle.so")

VAL_DTYPE = np.dtype([("file_id", "<u4"), ("reserved", "<u4"), ("offset", "<u8")])

OK, EINVAL, ECAPACITY, EBADPAGE, EBADREC = 0, -1, -2, -3, -4


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle returned {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle's C source into a shared object next to it (gcc -O2)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.run(["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-shared", "-fPIC",
                    "-o", tmp, _SRC], check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _Geom(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_layers", "n_kv_heads", "head_dim", "elem_bytes",
                                          "page_tokens", "chunk_tokens", "ns", "flags")]


class _Run(C.Structure):
    _fields_ = [("keys", C.c_void_p), ("vals", C.c_void_p), ("n", C.c_uint64)]


@dataclass(frozen=True)
class Geom:
    n_layers: int
    n_kv_heads: int
    head_dim: int
    elem_bytes: int = 2
    page_tokens: int = 16
    chunk_tokens: int = 16
    ns: int = 0
    flags: int = 0

    def c(self) -> _Geom:
        return _Geom(self.n_layers, self.n_kv_heads, self.head_dim, self.elem_bytes,
                     self.page_tokens, self.chunk_tokens, self.ns, self.flags)

    @property
    def page_bytes(self) -> int:
        return self.page_tokens * self.n_kv_heads * self.head_dim * self.elem_bytes

    @property
    def pages_per_chunk(self) -> int:
        return self.chunk_tokens // self.page_tokens

    @property
    def chunk_bytes(self) -> int:
        return self.pages_per_chunk * 2 * self.n_layers * self.page_bytes


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_digest.restype = C.c_uint64
        _lib.orc_digest.argtypes = [C.c_void_p, C.c_uint64, C.c_int]
        _lib.orc_digest_step.restype = C.c_uint64
        _lib.orc_digest_step.argtypes = [C.c_uint64, C.c_uint32, C.c_int]
        _lib.orc_chunk_keys.restype = C.c_uint64
        _lib.orc_chunk_keys.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64,
                                        C.c_void_p]
        _lib.orc_key_cmp.restype = C.c_int
        _lib.orc_key_cmp.argtypes = [C.c_void_p, C.c_void_p]
        _lib.orc_encode_batch.restype = C.c_int
        _lib.orc_encode_batch.argtypes = [
            C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_uint64, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint64,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64]
        _lib.orc_lookup.restype = C.c_int
        _lib.orc_lookup.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p,
                                    C.c_void_p]
        _lib.orc_flush.restype = C.c_int64
        _lib.orc_flush.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p,
                                   C.c_void_p]
        _lib.orc_merge_runs.restype = C.c_int64
        _lib.orc_merge_runs.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        _lib.orc_bloom_blocks.restype = C.c_uint64
        _lib.orc_bloom_blocks.argtypes = [C.c_uint64]
        _lib.orc_bloom_build.restype = None
        _lib.orc_bloom_build.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.orc_bloom_may_contain.restype = C.c_int
        _lib.orc_bloom_may_contain.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.orc_hindex_buckets.restype = C.c_uint64
        _lib.orc_hindex_buckets.argtypes = [C.c_uint64]
        _lib.orc_hindex_build.restype = C.c_int
        _lib.orc_hindex_build.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.orc_hindex_find.restype = C.c_uint64
        _lib.orc_hindex_find.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64,
                                         C.c_void_p]
        _lib.orc_xp12_slab_bound.restype = C.c_uint64
        _lib.orc_xp12_slab_bound.argtypes = [C.c_uint64]
        _lib.orc_xp12_dir_bytes.restype = C.c_uint64
        _lib.orc_xp12_dir_bytes.argtypes = [C.c_void_p]
        _lib.orc_xp12_chunk_bound.restype = C.c_uint64
        _lib.orc_xp12_chunk_bound.argtypes = [C.c_void_p]
        _lib.orc_xp12_slab_encode.restype = C.c_uint64
        _lib.orc_xp12_slab_encode.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.orc_xp12_slab_decode.restype = C.c_uint64
        _lib.orc_xp12_slab_decode.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p]
        _lib.orc_encode_batch_xp12.restype = C.c_int
        _lib.orc_encode_batch_xp12.argtypes = [
            C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_uint64, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint64,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.orc_decode_batch_xp12.restype = C.c_int
        _lib.orc_decode_batch_xp12.argtypes = [
            C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint64]
        _lib.orc_relocate_records.restype = C.c_uint64
        _lib.orc_relocate_records.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint32]
        _lib.orc_xprobe_batch.restype = C.c_int
        _lib.orc_xprobe_batch.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p,
                                          C.c_void_p]
        _lib.orc_probe_batch.restype = C.c_int
        _lib.orc_probe_batch.argtypes = [
            C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_decode_batch.restype = C.c_int
        _lib.orc_decode_batch.argtypes = [
            C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint64]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _pool_ptrs(pool: np.ndarray):
    """Pointer table for a [2L, num_pages, page_bytes] uint8 pool."""
    assert pool.dtype == np.uint8 and pool.ndim == 3 and pool.flags.c_contiguous
    n = pool.shape[0]
    stride = pool.shape[1] * pool.shape[2]
    base = pool.ctypes.data
    return (C.c_void_p * n)(*[base + i * stride for i in range(n)])


def _runs_struct(runs):
    keep = []
    arr = (_Run * max(1, len(runs)))()
    for i, (k, v) in enumerate(runs):
        k = _arr(k, np.uint64).reshape(-1, 4)
        v = np.ascontiguousarray(v, dtype=VAL_DTYPE)
        assert len(k) == len(v)
        keep.append((k, v))
        arr[i].keys = k.ctypes.data if len(k) else None
        arr[i].vals = v.ctypes.data if len(v) else None
        arr[i].n = len(k)
    return arr, keep


# ---- public wrappers -------------------------------------------------------------------

def digest(tokens, lane: int) -> int:
    t = _arr(tokens, np.uint32)
    return int(lib().orc_digest(_p(t), t.size, lane))


def digest_step(h: int, token: int, lane: int) -> int:
    return int(lib().orc_digest_step(h, token, lane))


def key_cmp(a, b) -> int:
    a = _arr(a, np.uint64)
    b = _arr(b, np.uint64)
    return int(lib().orc_key_cmp(_p(a), _p(b)))


def chunk_keys(g: Geom, tokens, j_begin: int = 0) -> np.ndarray:
    t = _arr(tokens, np.uint32)
    nch = t.size // g.chunk_tokens
    out = np.zeros((max(0, nch - j_begin), 4), dtype=np.uint64)
    gc = g.c()
    n = lib().orc_chunk_keys(C.byref(gc), _p(t), t.size, j_begin, _p(out))
    assert n == len(out)
    return out


def encode_batch(g: Geom, tokens, seq_off, start_chunk, chunk_off, page_table, pool,
                 file_id: int, base_offset: int, with_blob: bool = True):
    """Returns (keys [n,4] u64, vals VAL_DTYPE[n], blob uint8[n*chunk_bytes] or None)."""
    tokens = _arr(tokens, np.uint32)
    seq_off = _arr(seq_off, np.uint64)
    chunk_off = _arr(chunk_off, np.uint64)
    start_chunk = None if start_chunk is None else _arr(start_chunk, np.uint32)
    n_req = len(seq_off) - 1
    n_chunks = int(chunk_off[-1]) if n_req else 0
    keys = np.zeros((n_chunks, 4), dtype=np.uint64)
    vals = np.zeros(n_chunks, dtype=VAL_DTYPE)
    blob = ptrs = None
    num_pages = 0
    if with_blob:
        page_table = _arr(page_table, np.uint32)
        assert len(page_table) == n_chunks * g.pages_per_chunk
        blob = np.zeros(n_chunks * g.chunk_bytes, dtype=np.uint8)
        ptrs = _pool_ptrs(pool)
        num_pages = pool.shape[1]
        assert pool.shape[0] == 2 * g.n_layers and pool.shape[2] == g.page_bytes
    gc = g.c()
    rc = lib().orc_encode_batch(C.byref(gc), n_req, _p(tokens), _p(seq_off), _p(start_chunk),
                                _p(chunk_off), n_chunks,
                                _p(page_table) if with_blob else None,
                                ptrs, num_pages, file_id, base_offset, _p(keys), _p(vals),
                                _p(blob), 0 if blob is None else blob.size)
    if rc != OK:
        raise OracleError(rc)
    return keys, vals, blob


def lookup(runs, key):
    """Returns (record as VAL_DTYPE scalar, deciding run index) or None."""
    arr, keep = _runs_struct(runs)
    key = _arr(key, np.uint64)
    val = np.zeros(1, dtype=VAL_DTYPE)
    ridx = C.c_uint32(0)
    hit = lib().orc_lookup(arr, len(runs), _p(key), _p(val), C.byref(ridx))
    del keep
    return (val[0], ridx.value) if hit else None


def flush(keys, vals):
    keys = _arr(keys, np.uint64).reshape(-1, 4)
    vals = np.ascontiguousarray(vals, dtype=VAL_DTYPE)
    ko = np.zeros_like(keys)
    vo = np.zeros_like(vals)
    m = lib().orc_flush(_p(keys), _p(vals), len(keys), _p(ko), _p(vo))
    if m < 0:
        raise OracleError(int(m))
    return ko[:m].copy(), vo[:m].copy()


def merge_runs(runs):
    arr, keep = _runs_struct(runs)
    total = sum(len(k) for k, _ in keep)
    ko = np.zeros((total, 4), dtype=np.uint64)
    vo = np.zeros(total, dtype=VAL_DTYPE)
    m = lib().orc_merge_runs(arr, len(runs), _p(ko), _p(vo))
    if m < 0:
        raise OracleError(int(m))
    return ko[:m].copy(), vo[:m].copy()


def bloom_blocks(n: int) -> int:
    return int(lib().orc_bloom_blocks(n))


def bloom_build(keys) -> np.ndarray:
    """Bloom filter bytes (32 per block) of a set of keys."""
    keys = _arr(keys, np.uint64).reshape(-1, 4)
    out = np.zeros(32 * bloom_blocks(len(keys)), dtype=np.uint8)
    lib().orc_bloom_build(_p(keys), len(keys), _p(out))
    return out


def bloom_may_contain(bloom: np.ndarray, key) -> bool:
    key = _arr(key, np.uint64)
    return bool(lib().orc_bloom_may_contain(_p(bloom), bloom.size // 32, _p(key)))


def hindex_buckets(n: int) -> int:
    return int(lib().orc_hindex_buckets(n))


def hindex_build(keys) -> np.ndarray:
    """Hash index (u32 slots, 8 per bucket) of a run's keys, inserted by ascending position."""
    keys = _arr(keys, np.uint64).reshape(-1, 4)
    out = np.zeros(8 * hindex_buckets(len(keys)), dtype=np.uint32)
    rc = lib().orc_hindex_build(_p(keys), len(keys), _p(out))
    if rc != OK:
        raise OracleError(rc)
    return out


def hindex_find(table: np.ndarray, keys, key) -> int:
    """Position of `key` in the run `keys` by the table's lookup rule, or -1. Works on any valid
    table of the run, whatever the order its keys were inserted in."""
    keys = _arr(keys, np.uint64).reshape(-1, 4)
    key = _arr(key, np.uint64)
    table = _arr(table, np.uint32)
    at = int(lib().orc_hindex_find(_p(table), table.size // 8, _p(keys), len(keys), _p(key)))
    return -1 if at == 2**64 - 1 else at


def probe_batch(g: Geom, tokens, seq_off, qchunk_off, runs, want_keys: bool = False):
    """Returns (hit u32[Q], recs VAL_DTYPE[total chunks], keys or None, lookups done)."""
    tokens = _arr(tokens, np.uint32)
    seq_off = _arr(seq_off, np.uint64)
    qchunk_off = _arr(qchunk_off, np.uint64)
    nq = len(seq_off) - 1
    total = int(qchunk_off[-1]) if nq else 0
    hit = np.zeros(nq, dtype=np.uint32)
    recs = np.zeros(total, dtype=VAL_DTYPE)
    keys = np.zeros((total, 4), dtype=np.uint64) if want_keys else None
    arr, keep = _runs_struct(runs)
    lookups = C.c_uint64(0)
    gc = g.c()
    rc = lib().orc_probe_batch(C.byref(gc), nq, _p(tokens), _p(seq_off), _p(qchunk_off), arr,
                               len(runs), _p(hit), _p(recs), _p(keys), C.byref(lookups))
    del keep
    if rc != OK:
        raise OracleError(rc)
    return hit, recs, keys, lookups.value


def decode_batch(g: Geom, qchunk_off, hit, recs, arenas, dst_page_table, pool) -> None:
    """Scatter hit blobs into ``pool`` (modified in place). ``arenas``: list of uint8 arrays."""
    qchunk_off = _arr(qchunk_off, np.uint64)
    hit = _arr(hit, np.uint32)
    recs = np.ascontiguousarray(recs, dtype=VAL_DTYPE)
    dst_page_table = _arr(dst_page_table, np.uint32)
    arenas = [np.ascontiguousarray(a, dtype=np.uint8) for a in arenas]
    aptr = (C.c_void_p * max(1, len(arenas)))(*[a.ctypes.data for a in arenas])
    abytes = np.array([a.size for a in arenas], dtype=np.uint64)
    ptrs = _pool_ptrs(pool)
    gc = g.c()
    rc = lib().orc_decode_batch(C.byref(gc), len(hit), _p(qchunk_off), _p(hit), _p(recs), aptr,
                                _p(abytes), len(arenas), _p(dst_page_table), ptrs,
                                pool.shape[1])
    if rc != OK:
        raise OracleError(rc)


# ---- compressing codec "xp12" ----------------------------------------------------------------

def xp12_slab_encode(elems) -> np.ndarray:
    """Compressed bytes of one slab of 16-bit elements."""
    e = _arr(elems, np.uint16)
    out = np.zeros(int(lib().orc_xp12_slab_bound(e.size)), dtype=np.uint8)
    n = lib().orc_xp12_slab_encode(_p(e), e.size, _p(out))
    return out[:n].copy()


def xp12_slab_decode(blob, n_elems: int):
    """Decoded 16-bit elements of one slab, or None if the bytes are malformed."""
    b = _arr(blob, np.uint8)
    out = np.zeros(n_elems, dtype=np.uint16)
    used = lib().orc_xp12_slab_decode(_p(b), b.size, n_elems, _p(out))
    return out if used else None


def xp12_chunk_bound(g: Geom) -> int:
    gc = g.c()
    return int(lib().orc_xp12_chunk_bound(C.byref(gc)))


def xp12_dir_bytes(g: Geom) -> int:
    gc = g.c()
    return int(lib().orc_xp12_dir_bytes(C.byref(gc)))


def encode_batch_xp12(g: Geom, tokens, seq_off, start_chunk, chunk_off, page_table, pool,
                      file_id: int, base_offset: int):
    """Returns (keys, vals, blob bytes actually used)."""
    tokens = _arr(tokens, np.uint32)
    seq_off = _arr(seq_off, np.uint64)
    chunk_off = _arr(chunk_off, np.uint64)
    start_chunk = None if start_chunk is None else _arr(start_chunk, np.uint32)
    page_table = _arr(page_table, np.uint32)
    n_req = len(seq_off) - 1
    n_chunks = int(chunk_off[-1]) if n_req else 0
    keys = np.zeros((n_chunks, 4), dtype=np.uint64)
    vals = np.zeros(n_chunks, dtype=VAL_DTYPE)
    cap = n_chunks * xp12_chunk_bound(g)
    blob = np.zeros(max(16, cap), dtype=np.uint8)
    used = C.c_uint64(0)
    gc = g.c()
    rc = lib().orc_encode_batch_xp12(C.byref(gc), n_req, _p(tokens), _p(seq_off),
                                     _p(start_chunk), _p(chunk_off), n_chunks, _p(page_table),
                                     _pool_ptrs(pool), pool.shape[1], file_id, base_offset,
                                     _p(keys), _p(vals), _p(blob), cap, C.byref(used))
    if rc != OK:
        raise OracleError(rc)
    return keys, vals, blob[:used.value].copy()


def decode_batch_xp12(g: Geom, qchunk_off, hit, recs, arenas, dst_page_table, pool) -> None:
    qchunk_off = _arr(qchunk_off, np.uint64)
    hit = _arr(hit, np.uint32)
    recs = np.ascontiguousarray(recs, dtype=VAL_DTYPE)
    dst_page_table = _arr(dst_page_table, np.uint32)
    arenas = [np.ascontiguousarray(a, dtype=np.uint8) for a in arenas]
    aptr = (C.c_void_p * max(1, len(arenas)))(*[a.ctypes.data for a in arenas])
    abytes = np.array([a.size for a in arenas], dtype=np.uint64)
    gc = g.c()
    rc = lib().orc_decode_batch_xp12(C.byref(gc), len(hit), _p(qchunk_off), _p(hit), _p(recs),
                                     aptr, _p(abytes), len(arenas), _p(dst_page_table),
                                     _pool_ptrs(pool), pool.shape[1])
    if rc != OK:
        raise OracleError(rc)


RELOC_DTYPE = np.dtype([("old_file", "<u4"), ("new_file", "<u4"), ("delta", "<u8")])


def relocate_records(vals, table):
    """Copy of ``vals`` with the relocation table applied, and the number of records changed."""
    v = np.ascontiguousarray(vals, dtype=VAL_DTYPE).copy()
    t = np.ascontiguousarray(table, dtype=RELOC_DTYPE)
    changed = lib().orc_relocate_records(_p(v), len(v), _p(t), len(t))
    return v, int(changed)


# ---- exact prefix index ----------------------------------------------------------------------

class _XRun(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("seq_off", C.c_void_p), ("n_seq", C.c_uint32),
                ("vals", C.c_void_p), ("chunk_off", C.c_void_p)]


def xprobe_batch(g: Geom, tokens, seq_off, qchunk_off, xruns):
    """xruns: list (newest first) of (tokens u32, seq_off u64[n+1], vals VAL_DTYPE per chunk in
    sequence-major order). Returns (hit u32[Q], recs VAL_DTYPE[total query chunks])."""
    tokens = _arr(tokens, np.uint32)
    seq_off = _arr(seq_off, np.uint64)
    qchunk_off = _arr(qchunk_off, np.uint64)
    nq = len(seq_off) - 1
    total = int(qchunk_off[-1]) if nq else 0
    arr = (_XRun * max(1, len(xruns)))()
    keep = []
    for i, (t, so, v) in enumerate(xruns):
        t = _arr(t, np.uint32)
        so = _arr(so, np.uint64)
        v = np.ascontiguousarray(v, dtype=VAL_DTYPE)
        nch = (np.diff(so.astype(np.int64)) // g.chunk_tokens).astype(np.uint64)
        co = np.zeros(len(so), dtype=np.uint64)
        np.cumsum(nch, out=co[1:])
        assert len(v) == int(co[-1])
        keep.append((t, so, v, co))
        arr[i].tokens, arr[i].seq_off, arr[i].n_seq = t.ctypes.data, so.ctypes.data, len(so) - 1
        arr[i].vals, arr[i].chunk_off = v.ctypes.data, co.ctypes.data
    hit = np.zeros(nq, dtype=np.uint32)
    recs = np.zeros(total, dtype=VAL_DTYPE)
    gc = g.c()
    rc = lib().orc_xprobe_batch(C.byref(gc), nq, _p(tokens), _p(seq_off), _p(qchunk_off), arr,
                                len(xruns), _p(hit), _p(recs))
    del keep
    if rc != OK:
        raise OracleError(rc)
    return hit, recs


def xrun_order(tokens, seq_off) -> np.ndarray:
    """Sequence numbers in token-lexicographic order (prefix first, identical ones by number)."""
    tokens = _arr(tokens, np.uint32)
    seq_off = _arr(seq_off, np.uint64)
    n = len(seq_off) - 1
    out = np.zeros(n, dtype=np.uint32)
    L = lib()
    L.orc_xrun_order.restype = C.c_int
    L.orc_xrun_order.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
    rc = L.orc_xrun_order(_p(tokens), _p(seq_off), n, _p(out))
    if rc != OK:
        raise OracleError(rc)
    return out
