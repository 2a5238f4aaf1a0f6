"""Host-buffer entry points (put / probe / decode with host memory) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu

G = lsmkv.Geom(n_layers=2, n_kv_heads=2, head_dim=64, page_tokens=16, chunk_tokens=16)   # 16 KiB chunks


def pinned(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).pin_memory()


# the same 16 KiB chunks made of two 8-token pages each
G2 = lsmkv.Geom(n_layers=2, n_kv_heads=2, head_dim=64, page_tokens=8, chunk_tokens=16)


@pytest.mark.parametrize("use_pinned", [False, True])
@pytest.mark.parametrize("stage", [1 << 20, 1 << 30])     # 1 MiB: many slices; 1 GiB: one slice
@pytest.mark.parametrize("g", [G, G2], ids=["one-page-chunks", "two-page-chunks"])
def test_put_probe_decode_through_host_buffers(use_pinned, stage, g):
    og = H.ogeom(g)
    cb = g.chunk_bytes
    m = g.pages_per_chunk
    rng = np.random.default_rng(11)
    w1 = synth.llama_requests(n_req=30, min_len=100, max_len=900, config_id=71)
    w2 = synth.llama_requests(n_req=17, min_len=100, max_len=900, config_id=72)
    start2 = rng.integers(0, 10, w2.batch.n).astype(np.uint32)
    num_pages = 2500 * m
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)

    def sizes(b, start):
        nch = synth.chunk_counts(b.seq_off, 16)
        st = np.zeros(b.n, np.int64) if start is None else start.astype(np.int64)
        return synth.offsets(np.maximum(nch - st, 0))

    with lsmkv.Context(g, 0) as ctx:
        ctx.set_tuning("host_stage_bytes", stage)
        pool = H.DevPool(g, num_pages, pool_np)
        arenas_np, runs_o, runs_d, keep = [], [], [], []
        for fid, (b, start) in enumerate(((w1.batch, None), (w2.batch, start2))):
            coff = sizes(b, start)
            n = int(coff[-1])
            pages = synth.random_pages(rng, num_pages, n * m)
            o_keys, o_vals, o_blob = oracle.encode_batch(og, b.tokens, b.seq_off, start, coff,
                                                         pages, pool_np, fid, 4096 * fid)
            keys = np.zeros((n, 4), np.uint64)
            vals = np.zeros(n, VAL_DTYPE)
            blob = np.zeros(n * cb, np.uint8)
            bufs = (b.tokens, b.seq_off, start, pages, keys, vals, blob)
            if use_pinned:
                bufs = tuple(None if x is None else pinned(x) for x in bufs)
            got_n = ctx.put_batch_host(b.n, bufs[0], bufs[1], bufs[2], bufs[3], pool.table, fid,
                                       4096 * fid, bufs[4], bufs[5], bufs[6], n * cb)
            torch.cuda.synchronize()
            assert got_n == n
            if use_pinned:
                keys = bufs[4].numpy().view(np.uint64).reshape(-1, 4)
                vals = bufs[5].numpy().view(VAL_DTYPE)
                blob = bufs[6].numpy()
            assert np.array_equal(keys, o_keys) and np.array_equal(vals, o_vals)
            assert np.array_equal(blob, o_blob)
            arenas_np.append(np.concatenate([np.zeros(4096 * fid, np.uint8), o_blob]))
            run = oracle.flush(o_keys, o_vals)
            runs_o.insert(0, run)                                 # newest first
        druns, keep = H.dev_runs(runs_o)
        # queries: both batches again (full prefixes of batch 2 are only partly stored)
        q = synth.make_batch([w1.batch.seq(i) for i in range(w1.batch.n)] +
                             [w2.batch.seq(i) for i in range(w2.batch.n)])
        qoff = synth.offsets(synth.chunk_counts(q.seq_off, 16))
        total = int(qoff[-1])
        o_hit, o_recs, o_qkeys, _ = oracle.probe_batch(og, q.tokens, q.seq_off, qoff, runs_o,
                                                       want_keys=True)
        hit = np.zeros(q.n, np.uint32)
        recs = np.zeros(total, VAL_DTYPE)
        qkeys = np.zeros((total, 4), np.uint64)
        hb = (q.tokens, q.seq_off, hit, recs, qkeys)
        if use_pinned:
            hb = tuple(pinned(x) for x in hb)
        got_total = ctx.probe_batch_host(q.n, hb[0], hb[1], druns, hb[2], hb[3], hb[4])
        torch.cuda.synchronize()
        if use_pinned:
            hit, recs = hb[2].numpy().view(np.uint32), hb[3].numpy().view(VAL_DTYPE)
            qkeys = hb[4].numpy().view(np.uint64).reshape(-1, 4)
        assert got_total == total
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        assert np.array_equal(qkeys, o_qkeys) and o_hit.sum() > 500
        # decode from the host arenas (two files) into a zeroed pool
        dst_pages = synth.random_pages(rng, num_pages, total * m)
        o_dst = np.zeros_like(pool_np)
        oracle.decode_batch(og, qoff, o_hit, o_recs, arenas_np, dst_pages, o_dst)
        dst = H.DevPool(g, num_pages)
        ar = [pinned(a) for a in arenas_np] if use_pinned else arenas_np
        ctx.decode_batch_host(q.n, qoff, hit, recs, [(a, arenas_np[i].size) for i, a in enumerate(ar)],
                              dst_pages, dst.table)
        torch.cuda.synchronize()
        assert np.array_equal(dst.numpy(), o_dst)
        st = ctx.last_status()
        assert st["flags"] == 0 and st["chunks_decoded"] == int(o_hit.sum())


def test_host_calls_reject_bad_arguments_before_enqueuing():
    g = G
    cb = g.chunk_bytes
    with lsmkv.Context(g, 0) as ctx:
        pool = H.DevPool(g, 4)
        toks = np.arange(32, dtype=np.uint32)
        off = np.array([0, 32], np.uint64)
        keys, vals = np.zeros((2, 4), np.uint64), np.zeros(2, VAL_DTYPE)
        blob = np.zeros(2 * cb, np.uint8)
        with pytest.raises(lsmkv.LsmkvError) as e:
            ctx.put_batch_host(1, toks, off, None, np.array([0, 1], np.uint32), pool.table, 0, 0,
                               keys, vals, blob, 2 * cb - 1)
        assert e.value.code == lsmkv.ECAPACITY
        recs = np.zeros(2, VAL_DTYPE)
        recs["offset"] = [0, cb * 2]                       # second record is outside the arena
        with pytest.raises(lsmkv.LsmkvError) as e:
            ctx.decode_batch_host(1, np.array([0, 2], np.uint64), np.array([2], np.uint32), recs,
                                  [(blob, blob.size)], np.array([0, 1], np.uint32), pool.table)
        assert e.value.code == lsmkv.EINVAL
        torch.cuda.synchronize()
        assert not pool.numpy().any()                      # nothing was enqueued
        # index-only put and an empty batch
        n = ctx.put_batch_host(1, toks, off, None, None, None, 3, 64, keys, vals, None, 0)
        torch.cuda.synchronize()
        assert n == 2 and list(vals["offset"]) == [64, 64 + cb] and list(vals["file_id"]) == [3, 3]
        assert ctx.put_batch_host(0, toks, off, None, None, None, 0, 0, keys, vals, None, 0) == 0


@pytest.mark.parametrize("stage", [1 << 20, 1 << 30])
def test_host_buffers_with_the_compressing_codec(stage):
    """put / probe / decode through host memory with variable-size blobs: byte-identical to the
    oracle's blobs laid back to back, across slices."""
    g = lsmkv.Geom(n_layers=2, n_kv_heads=8, head_dim=64, page_tokens=16, chunk_tokens=16,
                   flags=lsmkv.CODEC_XP12)                      # 16 KiB slabs, 64 KiB chunks
    og = H.ogeom(g)
    rng = np.random.default_rng(21)
    w = synth.llama_requests(n_req=12, min_len=100, max_len=700, config_id=73)
    b = w.batch
    nch = synth.chunk_counts(b.seq_off, 16)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    num_pages = n + 9
    pool_np = synth.random_pool_bytes(rng, 4, num_pages, g.page_bytes)
    pool_np.view(np.uint16)[:, ::7, ::5] = 0x0001               # sprinkle exceptions
    pages = synth.random_pages(rng, num_pages, n)
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(og, b.tokens, b.seq_off, None, coff, pages,
                                                      pool_np, 2, 256)
    with lsmkv.Context(g, 0) as ctx:
        ctx.set_tuning("host_stage_bytes", stage)
        pool = H.DevPool(g, num_pages, pool_np)
        keys = np.zeros((n, 4), np.uint64)
        vals = np.zeros(n, VAL_DTYPE)
        blob = np.zeros(ctx.encode_bound(n), np.uint8)
        got_n, used = ctx.put_batch_host(b.n, b.tokens, b.seq_off, None, pages, pool.table, 2, 256,
                                         keys, vals, blob, blob.size, want_bytes=True)
        torch.cuda.synchronize()
        assert got_n == n and used == o_blob.size
        assert np.array_equal(keys, o_keys) and np.array_equal(vals, o_vals)
        assert np.array_equal(blob[:used], o_blob)
        # too small a host buffer is reported
        with pytest.raises(lsmkv.LsmkvError) as e:
            ctx.put_batch_host(b.n, b.tokens, b.seq_off, None, pages, pool.table, 2, 256, keys,
                               vals, blob, used - 16)
        assert e.value.code == lsmkv.ECAPACITY
        torch.cuda.synchronize()
        ctx.last_status()
        run = oracle.flush(o_keys, o_vals)
        druns, keep = H.dev_runs([run])
        hit = np.zeros(b.n, np.uint32)
        recs = np.zeros(n, VAL_DTYPE)
        ctx.probe_batch_host(b.n, b.tokens, b.seq_off, druns, hit, recs)
        torch.cuda.synchronize()
        assert np.array_equal(hit, nch.astype(np.uint32))
        arena = np.concatenate([np.zeros(256, np.uint8), o_blob])
        arenas = [np.zeros(16, np.uint8), np.zeros(16, np.uint8), arena]   # file_id 2
        dst_pages = synth.random_pages(rng, num_pages, n)
        o_dst = np.zeros_like(pool_np)
        oracle.decode_batch_xp12(og, coff, hit, recs, arenas, dst_pages, o_dst)
        dst = H.DevPool(g, num_pages)
        ctx.decode_batch_host(b.n, coff, hit, recs, [(a, a.size) for a in arenas], dst_pages,
                              dst.table)
        torch.cuda.synchronize()
        assert np.array_equal(dst.numpy(), o_dst)
        st = ctx.last_status()
        assert st["flags"] == 0 and st["chunks_decoded"] == n


def test_xp12_put_placed_by_the_device_equals_the_oracle():
    """On request, with a pinned host blob and no byte count wanted at return, the device places
    the slices itself (several slices here): keys, records and blob bytes are the oracle's; a
    host blob that is too small is flagged, not overrun."""
    g = lsmkv.Geom(2, 8, 64, elem_bytes=2, page_tokens=16, chunk_tokens=16, flags=lsmkv.CODEC_XP12)
    og = H.ogeom(g)                                             # 16 KiB slabs, 64 KiB chunks
    rng = np.random.default_rng(21)
    b = synth.make_batch([rng.integers(0, 5000, 16 * k + 3, dtype=np.uint32) for k in (7, 1, 12, 4, 9)])
    nch = synth.chunk_counts(b.seq_off, 16)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    num_pages = n + 5
    pool_np = synth.random_pool_bytes(rng, 4, num_pages, g.page_bytes)
    pool_np.view(np.uint16)[:, ::5, ::9] = 0x0001               # sprinkle exceptions
    pages = synth.random_pages(rng, num_pages, n)
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(og, b.tokens, b.seq_off, None, coff, pages,
                                                      pool_np, 1, 4096)
    with lsmkv.Context(g, 0) as ctx:
        ctx.set_tuning("host_stage_bytes", 1 << 20)            # 1 MiB stage: several slices
        ctx.set_tuning("host_put_device_placed", 1)
        pool = H.DevPool(g, num_pages, pool_np)
        keys = torch.zeros(n * 32, dtype=torch.uint8).pin_memory()
        vals = torch.zeros(n * 16, dtype=torch.uint8).pin_memory()
        blob = torch.full((ctx.encode_bound(n),), 0xEE, dtype=torch.uint8).pin_memory()
        got_n = ctx.put_batch_host(b.n, b.tokens, b.seq_off, None, pages, pool.table, 1, 4096,
                                   keys, vals, blob, blob.numel())
        torch.cuda.synchronize()
        assert got_n == n
        assert np.array_equal(keys.numpy().view(np.uint64).reshape(-1, 4), o_keys)
        v = vals.numpy().view(VAL_DTYPE)
        assert np.array_equal(v, o_vals)
        used = int(v["offset"][-1]) + int(v["reserved"][-1]) - 4096
        assert used == o_blob.size
        assert np.array_equal(blob.numpy()[:used], o_blob)
        assert np.all(blob.numpy()[used:] == 0xEE)
        assert ctx.last_status()["flags"] == 0
        # a host blob with room for the first slices only: the rest is flagged and left out
        blob.fill_(0xEE)
        cap = o_blob.size // 2 // 16 * 16
        ctx.put_batch_host(b.n, b.tokens, b.seq_off, None, pages, pool.table, 1, 4096, keys, vals,
                           blob, cap)
        torch.cuda.synchronize()
        assert ctx.last_status()["flags"] == lsmkv.ST_OVERFLOW
        got = blob.numpy()
        placed = int(np.flatnonzero(got != 0xEE).max()) + 1 if (got != 0xEE).any() else 0
        assert placed <= cap and np.array_equal(got[:placed], o_blob[:placed])
        assert np.all(got[cap:] == 0xEE)
