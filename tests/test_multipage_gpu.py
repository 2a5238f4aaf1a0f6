"""Chunks that span several pages (chunk_tokens = m * page_tokens) on the GPU: the whole path
against the oracle, byte for byte, with both copy kernels and with the compressing codec; the
allocation-free decode against the regular one; a bad page in the middle of a chunk."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


def ragged_store_and_queries(C, seed):
    rng = np.random.default_rng(seed)
    lens = [0, 1, C - 1, C, C + 1, 9 * C + 2, 33 * C, 5 * C, 32 * C + C // 2]
    base = rng.integers(0, 5, 40 * C, dtype=np.uint32)
    seqs = []
    for n in lens:
        s = base[:n].copy()
        cut = int(rng.integers(0, n + 1))
        s[cut:] = rng.integers(5, 10, n - cut)
        seqs.append(s)
    qs = [s.copy() for s in seqs] + [base[:30 * C].copy(), rng.integers(5, 10, 4 * C, dtype=np.uint32)]
    qs[5][3 * C + 1] ^= 1
    return synth.make_batch(seqs), synth.make_batch(qs)


@pytest.mark.parametrize("P,m", [(16, 2), (4, 3), (16, 4), (1, 5)])
@pytest.mark.parametrize("mode", [0, 1])
def test_whole_path_with_chunks_of_m_pages(P, m, mode):
    g = lsmkv.Geom(3, 2, 32, elem_bytes=2, page_tokens=P, chunk_tokens=m * P)
    store, query = ragged_store_and_queries(g.chunk_tokens, 10 * P + m)
    out = H.roundtrip(g, store, query, n_runs=2, seed=P + m,
                      tuning={"copy_mode": mode, "copy_stage_bytes": 64})
    assert out["hit"].sum() > 0


@pytest.mark.parametrize("generic", [0, 1])
def test_compressing_codec_with_chunks_of_two_pages(generic):
    # 2048-element slabs x 4 sweeps = 8192 elements per page: the fast kernels' smallest size
    g = lsmkv.Geom(2, 4, 128, elem_bytes=2, page_tokens=16, chunk_tokens=32, flags=lsmkv.CODEC_XP12)
    w = synth.tiny_codec(n_req=6, seq_len=32 * 9 + 5, max_shared=150, n_mutate=40, config_id=91)
    out = H.roundtrip_xp12(g, w.store, w.query, seed=3 + generic,
                           tuning={"xp_generic": generic})
    assert 0.74 < out["ratio"] < 0.77 and out["hit"].sum() > 0


def test_allocation_free_decode_equals_the_regular_one_with_two_page_chunks():
    g = lsmkv.Geom(2, 2, 64, elem_bytes=2, page_tokens=8, chunk_tokens=16)
    m = g.pages_per_chunk
    rng = np.random.default_rng(4)
    w = synth.tiny_codec(n_req=6, seq_len=16 * 12 + 3, max_shared=80, n_mutate=40, config_id=92)
    coff = synth.offsets(synth.chunk_counts(w.store.seq_off, 16))
    n = int(coff[-1])
    num_pages = n * m + 5
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    with lsmkv.Context(g, 0) as ctx:
        pool = H.DevPool(g, num_pages, pool_np)
        keys, vals, blob, d_blob = H.gpu_encode(ctx, g, w.store, None, coff,
                                                synth.random_pages(rng, num_pages, n * m), pool)
        run = H.gpu_flush_run(ctx, keys, vals)
        qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
        total = int(qoff[-1])
        hit, recs, _, (d_qoff, d_hit, d_recs) = H.gpu_probe(ctx, w.query, qoff, [run],
                                                           want_keys=False)
        assert hit.sum() > 0
        dst_pages = H.dev(synth.random_pages(rng, num_pages, total * m))
        arenas = [(d_blob, blob.size)]
        ref, out = H.DevPool(g, num_pages), H.DevPool(g, num_pages)
        ctx.decode_batch(w.query.n, d_qoff, total, d_hit, d_recs, arenas, dst_pages, ref.table)
        d_status = torch.zeros(56, dtype=torch.uint8, device=H.DEV)
        lsmkv.lsmkv_decode_batch_static(g, 0, None, w.query.n, d_qoff, total, d_hit, d_recs,
                                        arenas, dst_pages, out.table, d_status)
        torch.cuda.synchronize()
        assert ref.numpy().any() and np.array_equal(out.numpy(), ref.numpy())
        assert ctx.last_status()["flags"] == 0


def test_a_bad_page_inside_a_chunk_is_flagged_and_only_that_page_is_skipped():
    g = lsmkv.Geom(2, 1, 32, elem_bytes=2, page_tokens=4, chunk_tokens=12)     # three pages a chunk
    og = H.ogeom(g)
    rng = np.random.default_rng(2)
    b = synth.make_batch([rng.integers(0, 50, 12 * 4, dtype=np.uint32)])
    coff = synth.offsets([4])
    num_pages = 16
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    pages = synth.random_pages(rng, num_pages, 12)
    _, _, o_blob = oracle.encode_batch(og, b.tokens, b.seq_off, None, coff, pages, pool_np, 0, 0)
    bad = pages.copy()
    bad[2 * 3 + 1] = 999                                   # chunk 2, its middle page
    with lsmkv.Context(g, 0) as ctx:
        pool = H.DevPool(g, num_pages, pool_np)
        d_keys = torch.zeros(4 * 32, dtype=torch.uint8, device=H.DEV)
        d_vals = torch.zeros(4 * 16, dtype=torch.uint8, device=H.DEV)
        d_blob = torch.full((o_blob.size,), 0xEE, dtype=torch.uint8, device=H.DEV)
        ctx.encode_batch(1, H.dev(b.tokens), H.dev(b.seq_off), None, H.dev(coff), 4, H.dev(bad),
                         pool.table, 0, 0, d_keys, d_vals, d_blob, o_blob.size)
        torch.cuda.synchronize()
        st = ctx.last_status()
        assert st["flags"] == lsmkv.ST_BAD_PAGE and st["first_bad"] == 2
        blob = d_blob.cpu().numpy()
        per_page = 2 * g.n_layers * g.page_bytes
        lo = 2 * g.chunk_bytes + per_page
        assert np.array_equal(blob[:lo], o_blob[:lo]) and np.all(blob[lo:lo + per_page] == 0xEE)
        assert np.array_equal(blob[lo + per_page:], o_blob[lo + per_page:])
