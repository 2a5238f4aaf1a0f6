"""Scratch buffers of one context keep to themselves: growing the sort scratch (a flush or a
merge larger than any before) must leave the compressing codec's scratch alone. On one XP12
context: encode, flush more entries than ever before, encode, merge more entries than ever
before, encode -- with a foreign allocation of about the codec scratch's size made and filled in
between, which is what would be handed a wrongly freed block. Every encode is compared with the
oracle byte for byte, no CUDA error may be recorded, and the context must destroy cleanly."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


def _encode_and_compare(ctx, g, w, pool, pool_np, src_pages, coff, n, bufs):
    bound = ctx.encode_bound(n)
    bufs["keys"].zero_()
    bufs["vals"].zero_()
    bufs["blob"].zero_()
    ctx.encode_batch(w.store.n, bufs["tok"], bufs["off"], None, bufs["coff"], n, bufs["src"],
                     pool.table, 3, 4096, bufs["keys"], bufs["vals"], bufs["blob"], bound)
    torch.cuda.synchronize()
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(H.ogeom(g), w.store.tokens, w.store.seq_off,
                                                      None, coff, src_pages, pool_np, 3, 4096)
    keys = H.host(bufs["keys"], np.uint64, n * 32).reshape(-1, 4)
    vals = H.host(bufs["vals"], VAL_DTYPE, n * 16)
    assert np.array_equal(keys, o_keys), "chunk keys differ"
    assert np.array_equal(vals, o_vals), "records differ"
    assert np.array_equal(bufs["blob"][:o_blob.size].cpu().numpy(), o_blob), "blobs differ"
    assert ctx.last_cuda_error() == 0
    return keys, vals


def test_xp12_encode_survives_growth_of_the_sort_scratch():
    g = lsmkv.Geom(2, 2, 64, elem_bytes=2, page_tokens=16, chunk_tokens=16, flags=lsmkv.CODEC_XP12)
    w = synth.tiny_codec(n_req=10, seq_len=16 * 30 + 3, max_shared=160, n_mutate=32, config_id=91)
    coff = synth.offsets(synth.chunk_counts(w.store.seq_off, 16))
    n = int(coff[-1])
    assert 200 <= n <= 400
    rng = np.random.default_rng(5)
    num_pages = n + 4
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    src_pages = synth.random_pages(rng, num_pages, n)
    ctx = lsmkv.Context(g, 0)
    pool = H.DevPool(g, num_pages, pool_np)
    bound = ctx.encode_bound(n)
    bufs = dict(tok=H.dev(w.store.tokens), off=H.dev(w.store.seq_off), coff=H.dev(coff),
                src=H.dev(src_pages),
                keys=torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV),
                vals=torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV),
                blob=torch.zeros(bound, dtype=torch.uint8, device=H.DEV))
    # bytes of the codec's encoder scratch for n chunks (sizes, offsets, flags per slab and chunk)
    xp_scratch = n * 2 * g.n_layers * 12 + (n + 2) * 8 + 256

    keys, vals = _encode_and_compare(ctx, g, w, pool, pool_np, src_pages, coff, n, bufs)

    # a flush of more entries than this context has sorted before: the sort scratch grows
    big = 5 * n
    fk = np.tile(keys, (5, 1))
    fv = np.tile(vals, 5)
    run = H.gpu_flush_run(ctx, fk, fv)
    o_run = oracle.flush(fk, fv)
    assert np.array_equal(run[0], o_run[0]) and np.array_equal(run[1], o_run[1])
    foreign = [torch.full((xp_scratch,), 0x5A, dtype=torch.uint8, device=H.DEV) for _ in range(8)]
    _encode_and_compare(ctx, g, w, pool, pool_np, src_pages, coff, n, bufs)
    assert all(bool((t == 0x5A).all()) for t in foreign), "a foreign allocation was written"

    # a merge of more entries than any sort before: the sort scratch grows again
    older = (run[0].copy(), run[1].copy())
    older[1]["file_id"] = 9
    runs = [run] + [older] * 6
    assert sum(len(k) for k, _ in runs) > big
    mk, mv = H.gpu_merge_runs(ctx, runs)
    o_mk, o_mv = oracle.merge_runs(runs)
    assert np.array_equal(mk, o_mk) and np.array_equal(mv, o_mv)
    foreign += [torch.full((xp_scratch,), 0xA5, dtype=torch.uint8, device=H.DEV) for _ in range(8)]
    _encode_and_compare(ctx, g, w, pool, pool_np, src_pages, coff, n, bufs)
    assert all(bool((t == 0x5A).all()) for t in foreign[:8])
    assert all(bool((t == 0xA5).all()) for t in foreign[8:]), "a foreign allocation was written"

    assert ctx.last_status()["flags"] == 0
    assert ctx.last_cuda_error() == 0
    ctx.close()                                    # raises unless lsmkv_destroy returned LSMKV_OK
    assert ctx.handle is None
