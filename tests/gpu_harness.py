"""Helpers for the GPU parity tests: move numpy inputs to the device, run the CUDA library
through its C ABI, run the oracle on the same inputs, and compare byte for byte."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import VAL_DTYPE
import hostindex
from paper_2511_16138_b200 import lsmkv, synth

DEV = "cuda:0"


def dev(a: np.ndarray) -> torch.Tensor:
    """numpy array -> device byte tensor holding the same bytes (at least 16 bytes long)."""
    b = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
    t = torch.zeros(max(16, b.size), dtype=torch.uint8, device=DEV)
    if b.size:
        t[:b.size] = torch.from_numpy(b.copy())
    return t


def host(t: torch.Tensor, dtype, n_bytes=None) -> np.ndarray:
    a = t.detach().cpu().numpy().reshape(-1)
    if n_bytes is not None:
        a = a[:n_bytes]
    return a.view(dtype)


def ogeom(g: lsmkv.Geom) -> oracle.Geom:
    return oracle.Geom(g.n_layers, g.n_kv_heads, g.head_dim, g.elem_bytes, g.page_tokens,
                       g.chunk_tokens, g.ns, g.flags)


class DevPool:
    def __init__(self, g: lsmkv.Geom, num_pages: int, init: np.ndarray | None = None):
        self.g, self.num_pages = g, num_pages
        self.t = torch.zeros((2 * g.n_layers, num_pages, g.page_bytes), dtype=torch.uint8,
                             device=DEV)
        if init is not None:
            self.t.copy_(torch.from_numpy(init))
        self.table = lsmkv.pool_table([self.t[i] for i in range(2 * g.n_layers)])

    def numpy(self) -> np.ndarray:
        return self.t.cpu().numpy()


def gpu_encode(ctx, g, batch, start_chunk, chunk_off, page_table, pool: DevPool | None,
               file_id=0, base_offset=0):
    n = int(chunk_off[-1])
    d_tok, d_off, d_coff = dev(batch.tokens), dev(batch.seq_off), dev(chunk_off)
    d_start = None if start_chunk is None else dev(np.asarray(start_chunk, np.uint32))
    d_keys = torch.zeros(max(1, n) * 32, dtype=torch.uint8, device=DEV)
    d_vals = torch.zeros(max(1, n) * 16, dtype=torch.uint8, device=DEV)
    d_blob = d_pt = None
    if pool is not None:
        d_pt = dev(np.asarray(page_table, np.uint32))
        d_blob = torch.zeros(max(16, n * g.chunk_bytes), dtype=torch.uint8, device=DEV)
    ctx.encode_batch(batch.n, d_tok, d_off, d_start, d_coff, n, d_pt,
                     pool.table if pool is not None else None, file_id, base_offset, d_keys,
                     d_vals, d_blob, 0 if d_blob is None else n * g.chunk_bytes)
    torch.cuda.synchronize()
    keys = host(d_keys, np.uint64, n * 32).reshape(-1, 4)
    vals = host(d_vals, VAL_DTYPE, n * 16)
    blob = None if d_blob is None else host(d_blob, np.uint8, n * g.chunk_bytes)
    return keys, vals, blob, d_blob


def dev_runs(runs):
    keep, out = [], []
    for k, v in runs:
        dk, dv = dev(k), dev(v)
        keep.append((dk, dv))
        out.append((dk, dv, len(k)))
    return out, keep


def with_hindex(ctx, druns):
    """The same device runs with their hash indexes attached (the form the benchmark probes)."""
    out, keep = [], []
    for r in druns:
        dk, dv, n = r[0], r[1], r[2]
        nb = lsmkv.lsmkv_hindex_buckets(n)
        t = torch.full((nb * 32,), 0xFF, dtype=torch.uint8, device=DEV)
        ctx.hindex_build(dk, n, t)
        keep.append(t)
        out.append((dk, dv, n, None, 0, t, nb))
    return out, keep


def gpu_probe(ctx, batch, qoff, runs, want_keys=True):
    """Probe twice -- searching the sorted runs, then through their hash indexes -- and insist
    on identical outputs; returns those of the second."""
    nq, total = batch.n, int(qoff[-1])
    d_tok, d_off, d_qoff = dev(batch.tokens), dev(batch.seq_off), dev(qoff)
    druns, keep = dev_runs(runs)
    hruns, hkeep = with_hindex(ctx, druns)
    outs = []
    for rr in (druns, hruns):
        d_hit = torch.full((max(4, nq),), 0x7FFFFFFF, dtype=torch.int32, device=DEV)
        d_recs = torch.full((max(1, total) * 16,), 0xAB, dtype=torch.uint8, device=DEV)
        d_keys = (torch.zeros(max(1, total) * 32, dtype=torch.uint8, device=DEV)
                  if want_keys else None)
        ctx.probe_batch(nq, d_tok, d_off, d_qoff, total, rr, d_hit, d_recs, d_keys)
        torch.cuda.synchronize()
        hit = d_hit.cpu().numpy().view(np.uint32)[:nq]
        recs = host(d_recs, VAL_DTYPE, total * 16)
        keys = host(d_keys, np.uint64, total * 32).reshape(-1, 4) if want_keys else None
        outs.append((hit, recs, keys, (d_qoff, d_hit, d_recs)))
    a, b = outs
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert (a[2] is None and b[2] is None) or np.array_equal(a[2], b[2])
    return b


def assert_status_clean(ctx):
    st = ctx.last_status()
    assert st["flags"] == 0, st
    return st


def roundtrip(g: lsmkv.Geom, store, query, start_chunk=None, n_runs=1, num_pages=None,
              tuning=None, seed=0, base_offset=0):
    """Encode `store`, flush into n_runs runs, probe `query`, decode the hits into a zeroed pool;
    every output is compared with the oracle's. Returns a dict of the interesting outputs."""
    og = ogeom(g)
    rng = np.random.default_rng(seed)
    C = g.chunk_tokens
    nch = synth.chunk_counts(store.seq_off, C)
    st = np.zeros(store.n, np.uint32) if start_chunk is None else np.asarray(start_chunk, np.uint32)
    coff = synth.offsets(np.maximum(nch - st.astype(np.int64), 0))
    n = int(coff[-1])
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, C))
    nq_chunks = int(qoff[-1])
    m = g.pages_per_chunk                          # page-table entries per chunk
    num_pages = num_pages or max(n, nq_chunks, 1) * m + 3
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    src_pages = synth.random_pages(rng, num_pages, n * m)
    dst_pages = synth.random_pages(rng, num_pages, nq_chunks * m)

    # ---- oracle
    o_keys, o_vals, o_blob = oracle.encode_batch(og, store.tokens, store.seq_off,
                                                 None if start_chunk is None else st, coff,
                                                 src_pages, pool_np, 0, base_offset)
    owner = rng.integers(0, n_runs, n)
    o_runs = [oracle.flush(o_keys[owner == r], o_vals[owner == r]) for r in range(n_runs)]
    o_hit, o_recs, o_qkeys, _ = oracle.probe_batch(og, query.tokens, query.seq_off, qoff, o_runs,
                                                   want_keys=True)
    o_dst = np.zeros_like(pool_np)
    arena_np = np.concatenate([np.zeros(base_offset, np.uint8), o_blob])
    oracle.decode_batch(og, qoff, o_hit, o_recs, [arena_np], dst_pages, o_dst)

    # ---- CUDA library
    with lsmkv.Context(g, 0) as ctx:
        for k, v in (tuning or {}).items():
            ctx.set_tuning(k, v)
        pool = DevPool(g, num_pages, pool_np)
        keys, vals, blob, d_blob = gpu_encode(ctx, g, store, None if start_chunk is None else st,
                                              coff, src_pages, pool, 0, base_offset)
        assert np.array_equal(keys, o_keys), "chunk keys differ"
        assert np.array_equal(vals, o_vals), "records differ"
        assert np.array_equal(blob, o_blob), "blobs differ"
        assert np.array_equal(pool.numpy(), pool_np), "encode modified the pool"
        runs = [hostindex.flush(keys[owner == r], vals[owner == r]) for r in range(n_runs)]
        for (k, v), (ok, ov) in zip(runs, o_runs):
            assert np.array_equal(k, ok) and np.array_equal(v, ov)
        hit, recs, qkeys, (d_qoff, d_hit, d_recs) = gpu_probe(ctx, query, qoff, runs)
        assert np.array_equal(hit, o_hit), "hit lengths differ"
        assert np.array_equal(qkeys, o_qkeys), "query keys differ"
        assert np.array_equal(recs, o_recs), "hit records differ"
        hit2, recs2, _, _ = gpu_probe(ctx, query, qoff, runs, want_keys=False)
        assert np.array_equal(hit2, o_hit) and np.array_equal(recs2, o_recs)
        dst = DevPool(g, num_pages)
        d_arena = torch.zeros(max(16, base_offset + blob.size), dtype=torch.uint8, device=DEV)
        d_arena[base_offset:base_offset + blob.size] = d_blob[:blob.size]
        ctx.decode_batch(query.n, d_qoff, nq_chunks, d_hit, d_recs,
                         [(d_arena, base_offset + blob.size)], dev(dst_pages), dst.table)
        torch.cuda.synchronize()
        assert np.array_equal(dst.numpy(), o_dst), "restored pool differs"
        status = assert_status_clean(ctx)
        assert status["chunks_encoded"] == n
        assert status["chunks_hit"] == int(o_hit.sum()) * 4       # two calls, each probing both ways
        assert status["chunks_decoded"] == int(o_hit.sum())
    return dict(hit=o_hit, n=n, status=status)


# ---- full-size helpers: pools as one tensor per buffer, checks on sampled pieces ---------------

class BigPool:
    """2L separate device buffers [num_pages, page_bytes], optionally filled with bf16 N(0,1)."""

    def __init__(self, g: lsmkv.Geom, num_pages: int, fill: bool, seed: int = 0):
        self.g, self.num_pages = g, num_pages
        gen = torch.Generator(device=DEV)
        gen.manual_seed(seed)
        self.bufs = []
        for _ in range(2 * g.n_layers):
            if fill:
                t = torch.randn(num_pages * g.page_bytes // 2, dtype=torch.bfloat16, device=DEV,
                                generator=gen)
                self.bufs.append(t.view(torch.uint8).view(num_pages, g.page_bytes))
            else:
                self.bufs.append(torch.zeros((num_pages, g.page_bytes), dtype=torch.uint8,
                                             device=DEV))
        self.table = lsmkv.pool_table(self.bufs)

    def gather(self, pages) -> np.ndarray:
        """Host copy [2L, n, page_bytes] of the given pages."""
        idx = torch.as_tensor(np.asarray(pages, dtype=np.int64), device=DEV)
        return torch.stack([b[idx] for b in self.bufs]).cpu().numpy()

    def zero_(self):
        for b in self.bufs:
            b.zero_()


def pages_equal_on_gpu(src: BigPool, src_pages, dst: BigPool, dst_pages, slice_pages=8192) -> bool:
    """dst page dst_pages[i] == src page src_pages[i] in every buffer (device-side compare)."""
    sp = torch.as_tensor(np.asarray(src_pages, dtype=np.int64), device=DEV)
    dp = torch.as_tensor(np.asarray(dst_pages, dtype=np.int64), device=DEV)
    for sb, db in zip(src.bufs, dst.bufs):
        for a in range(0, len(sp), slice_pages):
            if not torch.equal(sb[sp[a:a + slice_pages]], db[dp[a:a + slice_pages]]):
                return False
    return True


def untouched_pages_zero(dst: BigPool, touched_pages) -> bool:
    mask = torch.ones(dst.num_pages, dtype=torch.bool, device=DEV)
    if len(touched_pages):
        mask[torch.as_tensor(np.asarray(touched_pages, dtype=np.int64), device=DEV)] = False
    idx = torch.nonzero(mask).flatten()
    for b in dst.bufs:
        for a in range(0, len(idx), 8192):
            if b[idx[a:a + 8192]].any():
                return False
    return True


def oracle_blob_range(g, seq_tokens, a, b, pool: BigPool, pages_ab, file_id, rec_offset_of_a):
    """Oracle encode of chunks [a, b) of one sequence whose pool pages are pages_ab: returns
    (keys, vals, blob) computed on the CPU from a compact host copy of those pages."""
    og = ogeom(g)
    C = g.chunk_tokens
    host_pool = pool.gather(pages_ab)
    toks = np.ascontiguousarray(seq_tokens[:b * C])
    return oracle.encode_batch(og, toks, np.array([0, len(toks)], np.uint64),
                               np.array([a], np.uint32), np.array([0, b - a], np.uint64),
                               np.arange(b - a, dtype=np.uint32), host_pool, file_id,
                               rec_offset_of_a)


def oracle_decode_one(g, rec, blob_bytes):
    """Oracle decode of one record whose blob is ``blob_bytes``: compact pool [2L, 1, page_bytes]."""
    og = ogeom(g)
    r = np.zeros(1, dtype=VAL_DTYPE)
    r["file_id"] = 0
    r["offset"] = 0
    assert int(rec["reserved"]) == 0
    out = np.zeros((2 * g.n_layers, 1, g.page_bytes), dtype=np.uint8)
    oracle.decode_batch(og, np.array([0, 1], np.uint64), np.array([1], np.uint32), r,
                        [np.ascontiguousarray(blob_bytes)], np.array([0], np.uint32), out)
    return out


def gpu_flush_run(ctx, keys: np.ndarray, vals: np.ndarray):
    """Flush on the device; returns the trimmed run as host arrays (keys [m,4], vals [m])."""
    n = len(keys)
    if n == 0:
        return np.zeros((0, 4), np.uint64), np.zeros(0, VAL_DTYPE)
    ok = torch.empty(n * 32, dtype=torch.uint8, device=DEV)
    ov = torch.empty(n * 16, dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    ctx.flush_batch(dev(keys), dev(np.ascontiguousarray(vals)), n, ok, ov, cnt)
    torch.cuda.synchronize()
    m = int(cnt.item())
    return (host(ok, np.uint64, n * 32).reshape(-1, 4)[:m].copy(),
            host(ov, VAL_DTYPE, n * 16)[:m].copy())


def gpu_merge_runs(ctx, runs):
    total = sum(len(k) for k, _ in runs)
    druns, keep = dev_runs(runs)
    ok = torch.empty(max(1, total) * 32, dtype=torch.uint8, device=DEV)
    ov = torch.empty(max(1, total) * 16, dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    ctx.merge_runs(druns, ok, ov, cnt)
    torch.cuda.synchronize()
    m = int(cnt.item())
    return (host(ok, np.uint64, total * 32).reshape(-1, 4)[:m].copy(),
            host(ov, VAL_DTYPE, total * 16)[:m].copy())


def roundtrip_xp12(g: lsmkv.Geom, store, query, seed=0, tuning=None):
    """Whole path with the compressing codec: encode, flush on the device, probe, decode into a
    zeroed pool; every output against the oracle's."""
    og = ogeom(g)
    rng = np.random.default_rng(seed)
    C = g.chunk_tokens
    nch = synth.chunk_counts(store.seq_off, C)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, C))
    nq = int(qoff[-1])
    m = g.pages_per_chunk
    num_pages = max(n, nq) * m + 3
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    src_pages = synth.random_pages(rng, num_pages, n * m)
    dst_pages = synth.random_pages(rng, num_pages, nq * m)
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(og, store.tokens, store.seq_off, None, coff,
                                                      src_pages, pool_np, 0, 0)
    o_run = oracle.flush(o_keys, o_vals)
    o_hit, o_recs, _, _ = oracle.probe_batch(og, query.tokens, query.seq_off, qoff, [o_run])
    o_dst = np.zeros_like(pool_np)
    oracle.decode_batch_xp12(og, qoff, o_hit, o_recs, [o_blob], dst_pages, o_dst)
    with lsmkv.Context(g, 0) as ctx:
        for k, v in (tuning or {}).items():
            ctx.set_tuning(k, v)
        pool = DevPool(g, num_pages, pool_np)
        bound = ctx.encode_bound(n)
        d_keys = torch.zeros(n * 32, dtype=torch.uint8, device=DEV)
        d_vals = torch.zeros(n * 16, dtype=torch.uint8, device=DEV)
        d_blob = torch.zeros(bound, dtype=torch.uint8, device=DEV)
        ctx.encode_batch(store.n, dev(store.tokens), dev(store.seq_off), None, dev(coff), n,
                         dev(src_pages), pool.table, 0, 0, d_keys, d_vals, d_blob, bound)
        torch.cuda.synchronize()
        keys = host(d_keys, np.uint64, n * 32).reshape(-1, 4)
        vals = host(d_vals, VAL_DTYPE, n * 16)
        assert np.array_equal(keys, o_keys) and np.array_equal(vals, o_vals)
        used = int(vals["offset"][-1]) + int(vals["reserved"][-1])
        assert np.array_equal(d_blob[:used].cpu().numpy(), o_blob)
        run = gpu_flush_run(ctx, keys, vals)
        assert np.array_equal(run[0], o_run[0]) and np.array_equal(run[1], o_run[1])
        hit, recs, _, (d_qoff, d_hit, d_recs) = gpu_probe(ctx, query, qoff, [run], want_keys=False)
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        dst = DevPool(g, num_pages)
        ctx.decode_batch(query.n, d_qoff, nq, d_hit, d_recs, [(d_blob, used)], dev(dst_pages),
                         dst.table)
        torch.cuda.synchronize()
        assert np.array_equal(dst.numpy(), o_dst)
        assert_status_clean(ctx)
    return dict(hit=o_hit, ratio=used / (n * g.chunk_bytes))
