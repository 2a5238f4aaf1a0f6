"""lsmkv_decode_batch_static: the decode that allocates nothing.

Some users of this library may not allocate device memory -- for example a storage plugin that
lives inside a serving process whose engine took all of HBM for its own pools and forbids
driver allocations from then on. They cannot create a context (that allocates), so the library
offers one context-free decode whose scratch is a fixed array inside the library itself.

The test drives that entry point through the C ABI and requires the restored pool to be
byte-identical to what the regular lsmkv_decode_batch produces and to what the CPU oracle
restores from its own blobs and records -- on two calls in a row, the second with shorter hits
and other destination pages, so that anything the shared scratch kept from the first call would
show up. This file sorts last on purpose: a run that stops at the
first failure has then already executed every other test.
"""
import numpy as np
import pytest
import torch

import hostindex
import oracle
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu

GEOM = lsmkv.Geom(n_layers=3, n_kv_heads=4, head_dim=64, page_tokens=16, chunk_tokens=16)


def _prepare(ctx, g, seed):
    """Encode a small store, index it, probe queries: returns what a decode needs."""
    rng = np.random.default_rng(seed)
    w = synth.tiny_codec(n_req=10, seq_len=16 * 21 + 3, max_shared=100, n_mutate=50,
                         config_id=40 + seed)
    nch = synth.chunk_counts(w.store.seq_off, g.chunk_tokens)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    num_pages = n + 5
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    pool = H.DevPool(g, num_pages, pool_np)
    src_pages = synth.random_pages(rng, num_pages, n)
    keys, vals, blob, d_blob = H.gpu_encode(ctx, g, w.store, None, coff, src_pages, pool)
    runs = [hostindex.flush(keys, vals)]
    qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, g.chunk_tokens))
    hit, recs, _, (d_qoff, d_hit, d_recs) = H.gpu_probe(ctx, w.query, qoff, runs, want_keys=False)
    assert hit.sum() > 0
    # the oracle's own chain on the same inputs: its blobs and records feed its decode below
    og = H.ogeom(g)
    o_keys, o_vals, o_blob = oracle.encode_batch(og, w.store.tokens, w.store.seq_off, None, coff,
                                                 src_pages, pool_np, 0, 0)
    o_hit, o_recs, _, _ = oracle.probe_batch(og, w.query.tokens, w.query.seq_off, qoff,
                                             [oracle.flush(o_keys, o_vals)])
    assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
    return dict(n_query=w.query.n, qoff=qoff, total=int(qoff[-1]), d_qoff=d_qoff, hit=hit,
                d_recs=d_recs, d_blob=d_blob, blob_bytes=blob.size, num_pages=num_pages, rng=rng,
                og=og, o_recs=o_recs, o_blob=o_blob, pool_shape=pool_np.shape)


def _decode_both(ctx, g, p, hit):
    """Decode once through each entry point into its own zeroed pool; return both pools and the
    status block of the allocation-free call. The allocation-free call's pool must also equal
    the oracle's decode of the oracle's blobs."""
    dst_np = synth.random_pages(p["rng"], p["num_pages"], p["total"])
    dst_pages = H.dev(dst_np)
    d_hit = H.dev(hit.astype(np.uint32))
    arenas = [(p["d_blob"], p["blob_bytes"])]
    ref = H.DevPool(g, p["num_pages"])
    ctx.decode_batch(p["n_query"], p["d_qoff"], p["total"], d_hit, p["d_recs"], arenas, dst_pages,
                     ref.table)
    out = H.DevPool(g, p["num_pages"])
    d_status = torch.full((56,), 0xCD, dtype=torch.uint8, device=H.DEV)
    lsmkv.lsmkv_decode_batch_static(g, 0, None, p["n_query"], p["d_qoff"], p["total"], d_hit,
                                    p["d_recs"], arenas, dst_pages, out.table, d_status)
    torch.cuda.synchronize()
    st = d_status.cpu().numpy()
    flags = int(st[:4].view(np.uint32)[0])
    decoded = int(st[48:56].view(np.uint64)[0])
    want = np.zeros(p["pool_shape"], dtype=np.uint8)
    oracle.decode_batch(p["og"], p["qoff"], hit.astype(np.uint32), p["o_recs"], [p["o_blob"]],
                        dst_np, want)
    assert np.array_equal(out.numpy(), want), "allocation-free decode differs from the oracle"
    return ref.numpy(), out.numpy(), flags, decoded


def test_static_decode_matches_regular_decode_twice_in_a_row():
    g = GEOM
    with lsmkv.Context(g, 0) as ctx:
        p = _prepare(ctx, g, seed=1)
        # call 1: the hits the probe found
        ref, out, flags, decoded = _decode_both(ctx, g, p, p["hit"])
        assert np.array_equal(out, ref), "first call differs from lsmkv_decode_batch"
        assert ref.any() and flags == 0 and decoded == int(p["hit"].sum())
        # call 2, straight after: shorter hits (some zero), other pages -- stale scratch would show
        hit2 = p["hit"] // 2
        hit2[::3] = 0
        ref2, out2, flags2, decoded2 = _decode_both(ctx, g, p, hit2)
        assert np.array_equal(out2, ref2), "second call differs from lsmkv_decode_batch"
        assert flags2 == 0 and decoded2 == int(hit2.sum()) and not np.array_equal(ref2, ref)
        H.assert_status_clean(ctx)


def test_static_decode_reports_bad_records_in_its_own_status_block():
    g = GEOM
    with lsmkv.Context(g, 0) as ctx:
        p = _prepare(ctx, g, seed=2)
        arenas_small = [(p["d_blob"], g.chunk_bytes)]          # every record but offset 0 is outside
        out = H.DevPool(g, p["num_pages"])
        d_status = torch.zeros(56, dtype=torch.uint8, device=H.DEV)
        dst_pages = H.dev(synth.random_pages(p["rng"], p["num_pages"], p["total"]))
        lsmkv.lsmkv_decode_batch_static(g, 0, None, p["n_query"], p["d_qoff"], p["total"],
                                        H.dev(p["hit"]), p["d_recs"], arenas_small, dst_pages,
                                        out.table, d_status)
        torch.cuda.synchronize()
        assert int(d_status.cpu().numpy()[:4].view(np.uint32)[0]) == lsmkv.ST_BAD_RECORD
        # the next call starts from a clean status block again
        ref, out2, flags, _ = _decode_both(ctx, g, p, p["hit"])
        assert flags == 0 and np.array_equal(out2, ref)


def test_static_decode_rejects_batches_beyond_its_scratch():
    g = GEOM
    z = torch.zeros(64, dtype=torch.uint8, device=H.DEV)
    pool = H.DevPool(g, 2)
    for n_query, n_chunks in ((lsmkv.STATIC_MAX_QUERIES + 1, 8), (4, lsmkv.STATIC_MAX_CHUNKS + 1)):
        with pytest.raises(lsmkv.LsmkvError) as e:
            lsmkv.lsmkv_decode_batch_static(g, 0, None, n_query, z, n_chunks, z, z, [(z, 64)], z,
                                            pool.table, None)
        assert e.value.code == lsmkv.ETOOBIG
        assert "scratch" in lsmkv.strerror(e.value.code)
    # an empty batch is fine and touches nothing
    lsmkv.lsmkv_decode_batch_static(g, 0, None, 0, z, 0, z, z, [(z, 64)], z, pool.table, None)
    torch.cuda.synchronize()
    assert not pool.numpy().any()
