"""ctypes binding of liblsmkv.so -- the same entry points as include/lsmkv.h.

Argument marshalling only: tensors (anything with ``data_ptr()``), raw integer addresses or
``None`` become pointers; every step of the path runs inside the CUDA library. There is no CPU
fallback: if the shared library is missing or fails to load, importing a symbol raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblsmkv.so")

OK, EINVAL, ECAPACITY, ECUDA, ENOMEM = 0, -1, -2, -3, -4
ST_BAD_PAGE, ST_BAD_RECORD, ST_BAD_COUNT, ST_MISALIGNED, ST_WAIT_EXPIRED = 1, 2, 4, 8, 16
MAX_RUNS = 64
KEY_BYTES, VAL_BYTES = 32, 16

EXPORTS = (
    "lsmkv_create", "lsmkv_destroy", "lsmkv_reserve", "lsmkv_encode_batch",
    "lsmkv_probe_batch", "lsmkv_decode_batch", "lsmkv_last_status", "lsmkv_last_cuda_error",
    "lsmkv_launch_count", "lsmkv_set_tuning", "lsmkv_get_tuning", "lsmkv_strerror",
    "lsmkv_format_version", "lsmkv_profile_enable", "lsmkv_profile_read",
    "lsmkv_decode_batch_static", "lsmkv_flush_batch", "lsmkv_merge_runs",
    "lsmkv_put_batch_host", "lsmkv_probe_batch_host", "lsmkv_decode_batch_host",
    "lsmkv_bloom_blocks", "lsmkv_bloom_build", "lsmkv_encode_bound", "lsmkv_last_cuda_line",
    "lsmkv_hindex_buckets", "lsmkv_hindex_build", "lsmkv_xrun_merge", "lsmkv_plan_compaction",
    "lsmkv_relocate_records", "lsmkv_xrun_build", "lsmkv_xprobe_batch",
)
ST_OVERFLOW = 32
CODEC_IDENTITY, CODEC_XP12 = 0, 1
ETOOBIG = -5
STATIC_MAX_QUERIES, STATIC_MAX_CHUNKS = 4096, 262144
K_KEYS, K_PACK, K_PROBE, K_PLAN, K_UNPACK, K_CLASSES = 0, 1, 2, 3, 4, 8
K_NAMES = ("keys", "pack", "probe", "plan", "unpack", "flush", "merge")


class LsmkvError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0, line: int = 0):
        msg = f"{where}: {strerror(code)} ({code})"
        if cuda:
            msg += f", cudaError {cuda}" + (f" at library line {line}" if line else "")
        super().__init__(msg)
        self.code = code
        self.cuda = cuda


class XRunStruct(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("seq_off", C.c_void_p), ("vals", C.c_void_p),
                ("order", C.c_void_p), ("chunk_off", C.c_void_p), ("n_seq", C.c_uint32),
                ("reserved", C.c_uint32)]


class GeomStruct(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_layers", "n_kv_heads", "head_dim", "elem_bytes",
                                          "page_tokens", "chunk_tokens", "ns", "flags")]


class RunStruct(C.Structure):
    _fields_ = [("keys", C.c_void_p), ("vals", C.c_void_p), ("n", C.c_uint64),
                ("bloom", C.c_void_p), ("bloom_blocks", C.c_uint64),
                ("hindex", C.c_void_p), ("hindex_buckets", C.c_uint64)]


def _run_array(runs):
    """runs: sequence of (keys, vals, n), (keys, vals, n, bloom, bloom_blocks) or
    (keys, vals, n, bloom, bloom_blocks, hindex, hindex_buckets); bloom / hindex may be None."""
    arr = (RunStruct * max(1, len(runs)))()
    for i, r in enumerate(runs):
        arr[i].keys, arr[i].vals, arr[i].n = _ptr(r[0]), _ptr(r[1]), r[2]
        if len(r) > 3 and r[3] is not None:
            arr[i].bloom, arr[i].bloom_blocks = _ptr(r[3]), r[4]
        if len(r) > 5 and r[5] is not None:
            arr[i].hindex, arr[i].hindex_buckets = _ptr(r[5]), r[6]
    return arr


class CompactionStruct(C.Structure):
    _fields_ = [("first_run", C.c_uint32), ("n_runs", C.c_uint32), ("to_level", C.c_uint32),
                ("reserved", C.c_uint32)]


class PoolStruct(C.Structure):
    _fields_ = [("kv_ptrs", C.c_void_p), ("num_pages", C.c_uint64)]


class StatusStruct(C.Structure):
    _fields_ = [("flags", C.c_uint32), ("reserved", C.c_uint32), ("first_bad", C.c_uint64),
                ("chunks_encoded", C.c_uint64), ("lookups", C.c_uint64),
                ("chunks_hit", C.c_uint64), ("empty_probes", C.c_uint64),
                ("chunks_decoded", C.c_uint64)]


class RelocStruct(C.Structure):
    _fields_ = [("old_file", C.c_uint32), ("new_file", C.c_uint32), ("delta", C.c_uint64)]


class ProfileStruct(C.Structure):
    _fields_ = [("ms", C.c_double * 8), ("launches", C.c_uint64 * 8)]


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

    @property
    def page_bytes(self) -> int:
        return self.page_tokens * self.n_kv_heads * self.head_dim * self.elem_bytes

    @property
    def pages_per_chunk(self) -> int:
        return self.chunk_tokens // self.page_tokens

    @property
    def chunk_bytes(self) -> int:
        return self.pages_per_chunk * 2 * self.n_layers * self.page_bytes

    def c(self) -> GeomStruct:
        return GeomStruct(self.n_layers, self.n_kv_heads, self.head_dim, self.elem_bytes,
                          self.page_tokens, self.chunk_tokens, self.ns, self.flags)


_lib = None


def lib() -> C.CDLL:
    """Load liblsmkv.so (built in-tree by ``paper_2511_16138_b200.build``). Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          "`python -m paper_2511_16138_b200.build` (needs nvcc)")
    L = C.CDLL(LIB_PATH)
    vp, u32, u64, i64 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int64
    L.lsmkv_create.restype = C.c_int
    L.lsmkv_create.argtypes = [C.POINTER(vp), C.POINTER(GeomStruct), C.c_int]
    L.lsmkv_destroy.restype = C.c_int
    L.lsmkv_destroy.argtypes = [vp]
    L.lsmkv_reserve.restype = C.c_int
    L.lsmkv_reserve.argtypes = [vp, u64, u64]
    L.lsmkv_encode_batch.restype = C.c_int
    L.lsmkv_encode_batch.argtypes = [vp, vp, u32, vp, vp, vp, vp, u64, vp,
                                     C.POINTER(PoolStruct), u32, u64, vp, vp, vp, u64]
    L.lsmkv_probe_batch.restype = C.c_int
    L.lsmkv_probe_batch.argtypes = [vp, vp, u32, vp, vp, vp, u64, C.POINTER(RunStruct), u32,
                                    vp, vp, vp]
    L.lsmkv_decode_batch.restype = C.c_int
    L.lsmkv_decode_batch.argtypes = [vp, vp, u32, vp, u64, vp, vp, C.POINTER(vp),
                                     C.POINTER(u64), u32, vp, C.POINTER(PoolStruct)]
    L.lsmkv_decode_batch_static.restype = C.c_int
    L.lsmkv_decode_batch_static.argtypes = [C.POINTER(GeomStruct), C.c_int, vp, u32, vp, u64, vp,
                                            vp, C.POINTER(vp), C.POINTER(u64), u32, vp,
                                            C.POINTER(PoolStruct), vp]
    L.lsmkv_put_batch_host.restype = C.c_int
    L.lsmkv_put_batch_host.argtypes = [vp, vp, u32, vp, vp, vp, vp, C.POINTER(PoolStruct), u32,
                                       u64, vp, vp, vp, u64, C.POINTER(u64), C.POINTER(u64)]
    L.lsmkv_probe_batch_host.restype = C.c_int
    L.lsmkv_probe_batch_host.argtypes = [vp, vp, u32, vp, vp, C.POINTER(RunStruct), u32, vp, vp,
                                         vp, C.POINTER(u64)]
    L.lsmkv_decode_batch_host.restype = C.c_int
    L.lsmkv_decode_batch_host.argtypes = [vp, vp, u32, vp, vp, vp, C.POINTER(vp),
                                          C.POINTER(u64), u32, vp, C.POINTER(PoolStruct)]
    L.lsmkv_relocate_records.restype = C.c_int
    L.lsmkv_relocate_records.argtypes = [vp, vp, vp, u64, C.POINTER(RelocStruct), u32, vp]
    L.lsmkv_xrun_build.restype = C.c_int
    L.lsmkv_xrun_build.argtypes = [vp, vp, vp, vp, u32, vp, vp]
    L.lsmkv_plan_compaction.restype = C.c_int
    L.lsmkv_plan_compaction.argtypes = [vp, vp, u32, u64, u32, u32, vp]
    L.lsmkv_xrun_merge.restype = C.c_int
    L.lsmkv_xrun_merge.argtypes = [vp, vp, vp, vp, vp, u32, vp, u32, vp, vp]
    L.lsmkv_xprobe_batch.restype = C.c_int
    L.lsmkv_xprobe_batch.argtypes = [vp, vp, u32, vp, vp, vp, u64, C.POINTER(XRunStruct), u32,
                                     vp, vp]
    L.lsmkv_encode_bound.restype = u64
    L.lsmkv_encode_bound.argtypes = [vp, u64]
    L.lsmkv_bloom_blocks.restype = u64
    L.lsmkv_bloom_blocks.argtypes = [u64]
    L.lsmkv_bloom_build.restype = C.c_int
    L.lsmkv_bloom_build.argtypes = [vp, vp, vp, u64, vp]
    L.lsmkv_hindex_buckets.restype = u64
    L.lsmkv_hindex_buckets.argtypes = [u64]
    L.lsmkv_hindex_build.restype = C.c_int
    L.lsmkv_hindex_build.argtypes = [vp, vp, vp, u64, vp]
    L.lsmkv_flush_batch.restype = C.c_int
    L.lsmkv_flush_batch.argtypes = [vp, vp, vp, vp, u64, vp, vp, vp]
    L.lsmkv_merge_runs.restype = C.c_int
    L.lsmkv_merge_runs.argtypes = [vp, vp, C.POINTER(RunStruct), u32, vp, vp, vp]
    L.lsmkv_last_status.restype = C.c_int
    L.lsmkv_last_status.argtypes = [vp, vp, C.POINTER(StatusStruct)]
    L.lsmkv_last_cuda_error.restype = C.c_int
    L.lsmkv_last_cuda_error.argtypes = [vp]
    L.lsmkv_last_cuda_line.restype = C.c_int
    L.lsmkv_last_cuda_line.argtypes = [vp]
    L.lsmkv_launch_count.restype = u64
    L.lsmkv_launch_count.argtypes = [vp]
    L.lsmkv_set_tuning.restype = C.c_int
    L.lsmkv_set_tuning.argtypes = [vp, C.c_char_p, i64]
    L.lsmkv_get_tuning.restype = i64
    L.lsmkv_get_tuning.argtypes = [vp, C.c_char_p]
    L.lsmkv_strerror.restype = C.c_char_p
    L.lsmkv_strerror.argtypes = [C.c_int]
    L.lsmkv_format_version.restype = C.c_int
    L.lsmkv_format_version.argtypes = []
    L.lsmkv_profile_enable.restype = C.c_int
    L.lsmkv_profile_enable.argtypes = [vp, C.c_int]
    L.lsmkv_profile_read.restype = C.c_int
    L.lsmkv_profile_read.argtypes = [vp, C.POINTER(ProfileStruct)]
    _lib = L
    return L


def strerror(code: int) -> str:
    try:
        return lib().lsmkv_strerror(code).decode()
    except Exception:
        return "error"


def _ptr(x):
    """tensor / int / None -> address."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(ctx, rc: int, where: str):
    if rc != OK:
        raise LsmkvError(rc, where, lib().lsmkv_last_cuda_error(ctx) if ctx else 0,
                         lib().lsmkv_last_cuda_line(ctx) if ctx else 0)


# ---- the C entry points, one to one ------------------------------------------------------

def lsmkv_create(geom: Geom, device: int = 0) -> int:
    h = C.c_void_p()
    g = geom.c()
    _check(None, lib().lsmkv_create(C.byref(h), C.byref(g), device), "lsmkv_create")
    return h.value


def lsmkv_destroy(ctx) -> None:
    _check(None, lib().lsmkv_destroy(ctx), "lsmkv_destroy")


def lsmkv_reserve(ctx, n_seq: int, n_chunks: int) -> None:
    _check(ctx, lib().lsmkv_reserve(ctx, n_seq, n_chunks), "lsmkv_reserve")


def _pool(pool):
    if pool is None:
        return None
    kv_ptrs, num_pages = pool
    return PoolStruct(_ptr(kv_ptrs), num_pages)


def lsmkv_encode_batch(ctx, stream, n_req, tokens, seq_off, start_chunk, chunk_off, n_chunks,
                       page_table, pool, file_id, base_offset, keys_out, vals_out, blob_out,
                       blob_capacity) -> None:
    p = _pool(pool)
    rc = lib().lsmkv_encode_batch(ctx, _stream(stream), n_req, _ptr(tokens), _ptr(seq_off),
                                  _ptr(start_chunk), _ptr(chunk_off), n_chunks,
                                  _ptr(page_table), C.byref(p) if p is not None else None,
                                  file_id, base_offset, _ptr(keys_out), _ptr(vals_out),
                                  _ptr(blob_out), blob_capacity)
    _check(ctx, rc, "lsmkv_encode_batch")


def lsmkv_probe_batch(ctx, stream, n_query, tokens, seq_off, qchunk_off, n_qchunks, runs,
                      hit_chunks_out, recs_out, keys_out=None) -> None:
    """runs: sequence of (keys, vals, n), newest first."""
    n_runs = len(runs)
    arr = _run_array(runs)
    rc = lib().lsmkv_probe_batch(ctx, _stream(stream), n_query, _ptr(tokens), _ptr(seq_off),
                                 _ptr(qchunk_off), n_qchunks, arr, n_runs,
                                 _ptr(hit_chunks_out), _ptr(recs_out), _ptr(keys_out))
    _check(ctx, rc, "lsmkv_probe_batch")


def lsmkv_decode_batch(ctx, stream, n_query, qchunk_off, n_qchunks, hit_chunks, recs, arenas,
                       dst_page_table, pool) -> None:
    """arenas: sequence of (base, n_bytes) indexed by file_id."""
    n = len(arenas)
    bases = (C.c_void_p * max(1, n))(*[_ptr(a) for a, _ in arenas])
    sizes = (C.c_uint64 * max(1, n))(*[b for _, b in arenas])
    p = _pool(pool)
    rc = lib().lsmkv_decode_batch(ctx, _stream(stream), n_query, _ptr(qchunk_off), n_qchunks,
                                  _ptr(hit_chunks), _ptr(recs), bases, sizes, n,
                                  _ptr(dst_page_table), C.byref(p) if p is not None else None)
    _check(ctx, rc, "lsmkv_decode_batch")


def _hptr(x):
    """host array (numpy, pinned torch tensor) / int / None -> address."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    return x.data_ptr()


def lsmkv_put_batch_host(ctx, stream, n_req, tokens, seq_off, start_chunk, page_table, pool,
                         file_id, base_offset, keys_out, vals_out, blob_out, blob_capacity,
                         want_bytes: bool = False):
    """Host buffers in and out (numpy arrays or pinned tensors). Returns the chunk count, or
    (chunk count, blob bytes placed) with ``want_bytes``."""
    p = _pool(pool)
    n = C.c_uint64(0)
    nb = C.c_uint64(0)
    rc = lib().lsmkv_put_batch_host(ctx, _stream(stream), n_req, _hptr(tokens), _hptr(seq_off),
                                    _hptr(start_chunk), _hptr(page_table),
                                    C.byref(p) if p is not None else None, file_id, base_offset,
                                    _hptr(keys_out), _hptr(vals_out), _hptr(blob_out),
                                    blob_capacity, C.byref(n), C.byref(nb) if want_bytes else None)
    _check(ctx, rc, "lsmkv_put_batch_host")
    return (int(n.value), int(nb.value)) if want_bytes else int(n.value)


def lsmkv_probe_batch_host(ctx, stream, n_query, tokens, seq_off, runs, hit_chunks_out,
                           recs_out, keys_out=None) -> int:
    """runs: device runs (keys, vals, n), newest first; everything else host. Returns the
    number of query chunks."""
    n_runs = len(runs)
    arr = _run_array(runs)
    total = C.c_uint64(0)
    rc = lib().lsmkv_probe_batch_host(ctx, _stream(stream), n_query, _hptr(tokens),
                                      _hptr(seq_off), arr, n_runs, _hptr(hit_chunks_out),
                                      _hptr(recs_out), _hptr(keys_out), C.byref(total))
    _check(ctx, rc, "lsmkv_probe_batch_host")
    return int(total.value)


def lsmkv_decode_batch_host(ctx, stream, n_query, qchunk_off, hit_chunks, recs, arenas,
                            dst_page_table, pool) -> None:
    """arenas: sequence of (host base, n_bytes) indexed by file_id; all arrays host."""
    n = len(arenas)
    bases = (C.c_void_p * max(1, n))(*[_hptr(a) for a, _ in arenas])
    sizes = (C.c_uint64 * max(1, n))(*[b for _, b in arenas])
    p = _pool(pool)
    rc = lib().lsmkv_decode_batch_host(ctx, _stream(stream), n_query, _hptr(qchunk_off),
                                       _hptr(hit_chunks), _hptr(recs), bases, sizes, n,
                                       _hptr(dst_page_table),
                                       C.byref(p) if p is not None else None)
    _check(ctx, rc, "lsmkv_decode_batch_host")


def lsmkv_relocate_records(ctx, stream, vals, n, table, changed_out=None) -> None:
    """table: sequence of (old_file, new_file, delta)."""
    arr = (RelocStruct * max(1, len(table)))(*[RelocStruct(*t) for t in table])
    rc = lib().lsmkv_relocate_records(ctx, _stream(stream), _ptr(vals), n, arr, len(table),
                                      _ptr(changed_out))
    _check(ctx, rc, "lsmkv_relocate_records")


def lsmkv_xrun_build(ctx, stream, tokens, seq_off, n_seq, order_out, chunk_off_out) -> None:
    rc = lib().lsmkv_xrun_build(ctx, _stream(stream), _ptr(tokens), _ptr(seq_off), n_seq,
                                _ptr(order_out), _ptr(chunk_off_out))
    _check(ctx, rc, "lsmkv_xrun_build")


def lsmkv_xrun_merge(ctx, stream, tokens, seq_off, order_a, n_a, order_b, n_b, order_out,
                     chunk_off_out) -> None:
    rc = lib().lsmkv_xrun_merge(ctx, _stream(stream), _ptr(tokens), _ptr(seq_off), _ptr(order_a),
                                n_a, _ptr(order_b), n_b, _ptr(order_out), _ptr(chunk_off_out))
    _check(ctx, rc, "lsmkv_xrun_merge")


def lsmkv_xprobe_batch(ctx, stream, n_query, tokens, seq_off, qchunk_off, n_qchunks, xruns,
                       hit_chunks_out, recs_out) -> None:
    """xruns: sequence of (tokens, seq_off, vals, order, chunk_off, n_seq), newest first."""
    arr = (XRunStruct * max(1, len(xruns)))()
    for i, (t, so, v, o, co, n) in enumerate(xruns):
        arr[i] = XRunStruct(_ptr(t), _ptr(so), _ptr(v), _ptr(o), _ptr(co), n, 0)
    rc = lib().lsmkv_xprobe_batch(ctx, _stream(stream), n_query, _ptr(tokens), _ptr(seq_off),
                                  _ptr(qchunk_off), n_qchunks, arr, len(xruns),
                                  _ptr(hit_chunks_out), _ptr(recs_out))
    _check(ctx, rc, "lsmkv_xprobe_batch")


def lsmkv_encode_bound(ctx, n_chunks: int) -> int:
    return int(lib().lsmkv_encode_bound(ctx, n_chunks))


def lsmkv_bloom_blocks(n: int) -> int:
    return int(lib().lsmkv_bloom_blocks(n))


def lsmkv_plan_compaction(levels, entries, buffer_entries: int, size_ratio: int,
                          runs_per_level: int):
    """Next merge the (T, K) policy asks for: (first_run, n_runs, to_level), or None when the
    index is in shape. levels / entries describe the runs newest first (host sequences)."""
    n = len(levels)
    lv = (C.c_uint32 * max(1, n))(*[int(x) for x in levels])
    en = (C.c_uint64 * max(1, n))(*[int(x) for x in entries])
    out = CompactionStruct()
    rc = lib().lsmkv_plan_compaction(lv, en, n, buffer_entries, size_ratio, runs_per_level,
                                     C.byref(out))
    if rc < 0:
        raise LsmkvError(rc, "lsmkv_plan_compaction")
    return (out.first_run, out.n_runs, out.to_level) if rc == 1 else None


def lsmkv_hindex_buckets(n: int) -> int:
    return int(lib().lsmkv_hindex_buckets(n))


def lsmkv_hindex_build(ctx, stream, keys, n, hindex_out) -> None:
    _check(ctx, lib().lsmkv_hindex_build(ctx, _stream(stream), _ptr(keys), n, _ptr(hindex_out)),
           "lsmkv_hindex_build")


def lsmkv_bloom_build(ctx, stream, keys, n, bloom_out) -> None:
    _check(ctx, lib().lsmkv_bloom_build(ctx, _stream(stream), _ptr(keys), n, _ptr(bloom_out)),
           "lsmkv_bloom_build")


def lsmkv_flush_batch(ctx, stream, keys, vals, n, run_keys_out, run_vals_out, n_out) -> None:
    rc = lib().lsmkv_flush_batch(ctx, _stream(stream), _ptr(keys), _ptr(vals), n,
                                 _ptr(run_keys_out), _ptr(run_vals_out), _ptr(n_out))
    _check(ctx, rc, "lsmkv_flush_batch")


def lsmkv_merge_runs(ctx, stream, runs, keys_out, vals_out, n_out) -> None:
    """runs: sequence of (keys, vals, n), newest first."""
    n_runs = len(runs)
    arr = _run_array(runs)
    rc = lib().lsmkv_merge_runs(ctx, _stream(stream), arr, n_runs, _ptr(keys_out),
                                _ptr(vals_out), _ptr(n_out))
    _check(ctx, rc, "lsmkv_merge_runs")


def lsmkv_decode_batch_static(geom: Geom, device, stream, n_query, qchunk_off, n_qchunks,
                              hit_chunks, recs, arenas, dst_page_table, pool,
                              status_out=None) -> None:
    """Decode without a context and without any device allocation: the scratch it needs is a
    fixed array inside the library (see include/lsmkv.h for the limits and the sharing rules).
    ``status_out``: optional device buffer of 56 bytes that receives this call's status block."""
    n = len(arenas)
    bases = (C.c_void_p * max(1, n))(*[_ptr(a) for a, _ in arenas])
    sizes = (C.c_uint64 * max(1, n))(*[b for _, b in arenas])
    p = _pool(pool)
    g = geom.c()
    rc = lib().lsmkv_decode_batch_static(C.byref(g), device, _stream(stream), n_query,
                                         _ptr(qchunk_off), n_qchunks, _ptr(hit_chunks),
                                         _ptr(recs), bases, sizes, n, _ptr(dst_page_table),
                                         C.byref(p) if p is not None else None,
                                         _ptr(status_out))
    if rc != OK:
        raise LsmkvError(rc, "lsmkv_decode_batch_static")


def lsmkv_last_status(ctx, stream=None) -> dict:
    st = StatusStruct()
    _check(ctx, lib().lsmkv_last_status(ctx, _stream(stream), C.byref(st)), "lsmkv_last_status")
    return {n: getattr(st, n) for n, _ in StatusStruct._fields_ if n != "reserved"}


def lsmkv_launch_count(ctx) -> int:
    return int(lib().lsmkv_launch_count(ctx))


def lsmkv_set_tuning(ctx, name: str, value: int) -> None:
    _check(ctx, lib().lsmkv_set_tuning(ctx, name.encode(), value), f"lsmkv_set_tuning({name})")


def lsmkv_get_tuning(ctx, name: str) -> int:
    return int(lib().lsmkv_get_tuning(ctx, name.encode()))


def lsmkv_profile_enable(ctx, on: bool) -> None:
    _check(ctx, lib().lsmkv_profile_enable(ctx, int(on)), "lsmkv_profile_enable")


def lsmkv_profile_read(ctx) -> dict:
    """{kernel class name: (device ms, launches)} since the previous read."""
    p = ProfileStruct()
    _check(ctx, lib().lsmkv_profile_read(ctx, C.byref(p)), "lsmkv_profile_read")
    return {n: (p.ms[i], int(p.launches[i])) for i, n in enumerate(K_NAMES)}


def lsmkv_format_version() -> int:
    return int(lib().lsmkv_format_version())


# ---- convenience: a context object and a pool pointer table ------------------------------

class Context:
    """Owns one lsmkv_ctx. Methods forward to the functions above with ``self.handle``."""

    def __init__(self, geom: Geom, device: int = 0):
        self.geom = geom
        self.device = device
        self.handle = lsmkv_create(geom, device)

    def close(self):
        if self.handle:
            lsmkv_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reserve(self, n_seq, n_chunks):
        lsmkv_reserve(self.handle, n_seq, n_chunks)

    def encode_batch(self, n_req, tokens, seq_off, start_chunk, chunk_off, n_chunks, page_table,
                     pool, file_id, base_offset, keys_out, vals_out, blob_out, blob_capacity,
                     stream=None):
        lsmkv_encode_batch(self.handle, stream, n_req, tokens, seq_off, start_chunk, chunk_off,
                           n_chunks, page_table, pool, file_id, base_offset, keys_out, vals_out,
                           blob_out, blob_capacity)

    def probe_batch(self, n_query, tokens, seq_off, qchunk_off, n_qchunks, runs, hit_chunks_out,
                    recs_out, keys_out=None, stream=None):
        lsmkv_probe_batch(self.handle, stream, n_query, tokens, seq_off, qchunk_off, n_qchunks,
                          runs, hit_chunks_out, recs_out, keys_out)

    def decode_batch(self, n_query, qchunk_off, n_qchunks, hit_chunks, recs, arenas,
                     dst_page_table, pool, stream=None):
        lsmkv_decode_batch(self.handle, stream, n_query, qchunk_off, n_qchunks, hit_chunks, recs,
                           arenas, dst_page_table, pool)

    def put_batch_host(self, n_req, tokens, seq_off, start_chunk, page_table, pool, file_id,
                       base_offset, keys_out, vals_out, blob_out, blob_capacity, stream=None,
                       want_bytes=False):
        return lsmkv_put_batch_host(self.handle, stream, n_req, tokens, seq_off, start_chunk,
                                    page_table, pool, file_id, base_offset, keys_out, vals_out,
                                    blob_out, blob_capacity, want_bytes)

    def probe_batch_host(self, n_query, tokens, seq_off, runs, hit_chunks_out, recs_out,
                         keys_out=None, stream=None):
        return lsmkv_probe_batch_host(self.handle, stream, n_query, tokens, seq_off, runs,
                                      hit_chunks_out, recs_out, keys_out)

    def decode_batch_host(self, n_query, qchunk_off, hit_chunks, recs, arenas, dst_page_table,
                          pool, stream=None):
        lsmkv_decode_batch_host(self.handle, stream, n_query, qchunk_off, hit_chunks, recs,
                                arenas, dst_page_table, pool)

    def xrun_build(self, tokens, seq_off, n_seq, order_out, chunk_off_out, stream=None):
        lsmkv_xrun_build(self.handle, stream, tokens, seq_off, n_seq, order_out, chunk_off_out)

    def xrun_merge(self, tokens, seq_off, order_a, n_a, order_b, n_b, order_out, chunk_off_out,
                   stream=None):
        lsmkv_xrun_merge(self.handle, stream, tokens, seq_off, order_a, n_a, order_b, n_b,
                         order_out, chunk_off_out)

    def xprobe_batch(self, n_query, tokens, seq_off, qchunk_off, n_qchunks, xruns,
                     hit_chunks_out, recs_out, stream=None):
        lsmkv_xprobe_batch(self.handle, stream, n_query, tokens, seq_off, qchunk_off, n_qchunks,
                           xruns, hit_chunks_out, recs_out)

    def relocate_records(self, vals, n, table, changed_out=None, stream=None):
        lsmkv_relocate_records(self.handle, stream, vals, n, table, changed_out)

    def encode_bound(self, n_chunks: int) -> int:
        return lsmkv_encode_bound(self.handle, n_chunks)

    def bloom_build(self, keys, n, bloom_out, stream=None):
        lsmkv_bloom_build(self.handle, stream, keys, n, bloom_out)

    def hindex_build(self, keys, n, hindex_out, stream=None):
        lsmkv_hindex_build(self.handle, stream, keys, n, hindex_out)

    def flush_batch(self, keys, vals, n, run_keys_out, run_vals_out, n_out, stream=None):
        lsmkv_flush_batch(self.handle, stream, keys, vals, n, run_keys_out, run_vals_out, n_out)

    def merge_runs(self, runs, keys_out, vals_out, n_out, stream=None):
        lsmkv_merge_runs(self.handle, stream, runs, keys_out, vals_out, n_out)

    def last_status(self, stream=None) -> dict:
        return lsmkv_last_status(self.handle, stream)

    def profile_enable(self, on=True):
        lsmkv_profile_enable(self.handle, on)

    def profile_read(self) -> dict:
        return lsmkv_profile_read(self.handle)

    def launch_count(self) -> int:
        return lsmkv_launch_count(self.handle)

    def last_cuda_error(self) -> int:
        """The cudaError_t behind the context's last LSMKV_ECUDA (0 if there was none)."""
        return lib().lsmkv_last_cuda_error(self.handle)

    def set_tuning(self, name, value):
        lsmkv_set_tuning(self.handle, name, value)

    def get_tuning(self, name):
        return lsmkv_get_tuning(self.handle, name)


def pool_table(buffers):
    """Device pointer table for 2L pool buffers (K layers, then V layers). Returns
    ``(kv_ptrs tensor, num_pages)``; keep the tensor alive while kernels use it."""
    import torch
    ptrs = torch.tensor([b.data_ptr() for b in buffers], dtype=torch.int64,
                        device=buffers[0].device)
    return ptrs, int(buffers[0].shape[0])
