"""Exact prefix index on the GPU (build + probe, then the ordinary decode) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


def geom(C):
    return lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=C, chunk_tokens=C)


def make_vals(g, batch, file_id, rng=None):
    n = int(synth.chunk_counts(batch.seq_off, g.chunk_tokens).sum())
    v = np.zeros(n, dtype=VAL_DTYPE)
    v["file_id"] = file_id
    v["offset"] = (np.arange(n) if rng is None else rng.permutation(n)) * g.chunk_bytes
    return v


def gpu_xrun(ctx, g, batch, vals):
    """-> (descriptor tuple for xprobe, order, chunk_off) with the device arrays kept alive in it."""
    d_tok, d_off, d_vals = H.dev(batch.tokens), H.dev(batch.seq_off), H.dev(vals)
    d_order = torch.full((max(4, batch.n),), -1, dtype=torch.int32, device=H.DEV)
    d_coff = torch.full((batch.n + 1,), -1, dtype=torch.int64, device=H.DEV)
    ctx.xrun_build(d_tok, d_off, batch.n, d_order, d_coff)
    torch.cuda.synchronize()
    order = d_order.cpu().numpy().view(np.uint32)[:batch.n]
    coff = d_coff.cpu().numpy().view(np.uint64)
    return (d_tok, d_off, d_vals, d_order, d_coff, batch.n), order, coff


def gpu_xprobe(ctx, query, qoff, xruns):
    nq, total = query.n, int(qoff[-1])
    d_tok, d_off, d_qoff = H.dev(query.tokens), H.dev(query.seq_off), H.dev(qoff)
    d_hit = torch.full((max(4, nq),), 0x7FFFFFFF, dtype=torch.int32, device=H.DEV)
    d_recs = torch.full((max(1, total) * 16,), 0xAB, dtype=torch.uint8, device=H.DEV)
    ctx.xprobe_batch(nq, d_tok, d_off, d_qoff, total, xruns, d_hit, d_recs)
    torch.cuda.synchronize()
    return (d_hit.cpu().numpy().view(np.uint32)[:nq], H.host(d_recs, VAL_DTYPE, total * 16),
            (d_qoff, d_hit, d_recs))


def check(g, stores, query):
    """stores: list (newest first) of (batch, vals)."""
    og = H.ogeom(g)
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, g.chunk_tokens))
    o_hit, o_recs = oracle.xprobe_batch(og, query.tokens, query.seq_off, qoff,
                                        [(b.tokens, b.seq_off, v) for b, v in stores])
    with lsmkv.Context(g, 0) as ctx:
        xruns = []
        for b, v in stores:
            x, order, coff = gpu_xrun(ctx, g, b, v)
            assert np.array_equal(order, oracle.xrun_order(b.tokens, b.seq_off)), "order differs"
            assert np.array_equal(coff, synth.offsets(synth.chunk_counts(b.seq_off, g.chunk_tokens)))
            xruns.append(x)
        hit, recs, _ = gpu_xprobe(ctx, query, qoff, xruns)
        assert np.array_equal(hit, o_hit), "hit lengths differ"
        assert np.array_equal(recs, o_recs), "records differ"
        st = H.assert_status_clean(ctx)
        assert st["chunks_hit"] == int(o_hit.sum())
    return o_hit


def test_binary_alphabet_many_ties_three_runs():
    g = geom(2)
    rng = np.random.default_rng(11)
    stores = []
    for r in range(3):
        seqs = [rng.integers(0, 2, rng.integers(0, 40), dtype=np.uint32) for _ in range(700)]
        seqs += [seqs[3].copy(), seqs[3].copy(), np.array([], np.uint32)]
        b = synth.make_batch(seqs)
        stores.append((b, make_vals(g, b, r, rng)))
    qs = [rng.integers(0, 2, rng.integers(0, 48), dtype=np.uint32) for _ in range(900)]
    qs += [stores[1][0].seq(3).copy(), stores[2][0].seq(5)[:7].copy(),
           np.concatenate([stores[0][0].seq(9), np.array([7, 7, 7, 7], np.uint32)])]
    hit = check(g, stores, synth.make_batch(qs))
    assert hit.max() >= 6 and (hit == 0).any()


def test_long_shared_prefixes_across_tiles():
    """Shared prefixes longer than one 32-token comparison step, differences at every offset."""
    g = geom(16)
    rng = np.random.default_rng(12)
    base = rng.integers(0, 50000, 700, dtype=np.uint32)
    seqs = []
    for k in range(400):
        cut = int(rng.integers(0, 700))
        tail = rng.integers(0, 50000, rng.integers(0, 80), dtype=np.uint32)
        seqs.append(np.concatenate([base[:cut], tail]))
    store = synth.make_batch(seqs)
    qs = []
    for k in range(300):
        cut = int(rng.integers(0, 700))
        qs.append(np.concatenate([base[:cut], rng.integers(0, 50000, rng.integers(0, 200),
                                                           dtype=np.uint32)]))
    qs.append(base.copy())
    qs.append(np.concatenate([base, base]))
    hit = check(g, [(store, make_vals(g, store, 4, rng))], synth.make_batch(qs))
    assert hit.max() >= 40


def test_probe_heavy_store_agrees_with_planted_hits():
    g = geom(16)
    w = synth.probe_heavy(n_keys=20000, run_sizes=(200, 1800, 18000), n_query=200, min_len=64,
                          max_len=2000, n_prefix=8)
    hit = check(g, [(w.store, make_vals(g, w.store, 1))], w.query)
    assert np.array_equal(hit, w.expected_hit.astype(np.uint32))


def test_empty_inputs():
    g = geom(16)
    empty = synth.make_batch([])
    some = synth.make_batch([np.arange(64, dtype=np.uint32), np.arange(5, dtype=np.uint32)])
    check(g, [], some)                                       # no runs
    check(g, [(empty, make_vals(g, empty, 0))], some)        # an empty run
    check(g, [(some, make_vals(g, some, 0))], empty)         # no queries
    check(g, [(some, make_vals(g, some, 0))], synth.make_batch([np.array([], np.uint32)]))


def test_exact_probe_then_decode_restores_the_pages():
    """put (encode) -> exact index -> exact probe -> decode, against the oracle end to end."""
    g = lsmkv.Geom(2, 2, 16, elem_bytes=2, page_tokens=16, chunk_tokens=16)
    og = H.ogeom(g)
    w = synth.tiny_codec(n_req=12, seq_len=400, max_shared=256, n_mutate=100)
    rng = np.random.default_rng(3)
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
    nq = int(qoff[-1])
    num_pages = max(n, nq) + 5
    pool_np = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    src_pages = synth.random_pages(rng, num_pages, n)
    dst_pages = synth.random_pages(rng, num_pages, nq)
    _, o_vals, o_blob = oracle.encode_batch(og, w.store.tokens, w.store.seq_off, None, coff,
                                            src_pages, pool_np, 0, 0)
    o_hit, o_recs = oracle.xprobe_batch(og, w.query.tokens, w.query.seq_off, qoff,
                                        [(w.store.tokens, w.store.seq_off, o_vals)])
    o_dst = np.zeros_like(pool_np)
    oracle.decode_batch(og, qoff, o_hit, o_recs, [o_blob], dst_pages, o_dst)
    assert o_hit.sum() > 0
    with lsmkv.Context(g, 0) as ctx:
        pool = H.DevPool(g, num_pages, pool_np)
        _, vals, blob, d_blob = H.gpu_encode(ctx, g, w.store, None, coff, src_pages, pool, 0, 0)
        assert np.array_equal(vals, o_vals) and np.array_equal(blob, o_blob)
        x, _, _ = gpu_xrun(ctx, g, w.store, vals)
        hit, recs, (d_qoff, d_hit, d_recs) = gpu_xprobe(ctx, w.query, qoff, [x])
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        dst = H.DevPool(g, num_pages)
        ctx.decode_batch(w.query.n, d_qoff, nq, d_hit, d_recs, [(d_blob, blob.size)],
                         H.dev(dst_pages), dst.table)
        torch.cuda.synchronize()
        assert np.array_equal(dst.numpy(), o_dst)
        H.assert_status_clean(ctx)


def test_bad_counts_are_flagged_not_read():
    g = geom(16)
    some = synth.make_batch([np.arange(64, dtype=np.uint32)])
    qoff = np.array([0, 3], np.uint64)                       # the query has 4 chunks
    with lsmkv.Context(g, 0) as ctx:
        x, _, _ = gpu_xrun(ctx, g, some, make_vals(g, some, 0))
        hit, _, _ = gpu_xprobe(ctx, some, qoff, [x])
        assert hit[0] == 0
        assert ctx.last_status()["flags"] & lsmkv.ST_BAD_COUNT


def random_store(rng, n_seq, alphabet, max_len, n_dup):
    """Sequences over a small alphabet (many shared prefixes), a few of them repeated verbatim."""
    seqs = [rng.integers(0, alphabet, int(rng.integers(0, max_len + 1)), dtype=np.uint32)
            for _ in range(n_seq)]
    for _ in range(n_dup):
        seqs[int(rng.integers(0, n_seq))] = seqs[int(rng.integers(0, n_seq))].copy()
    return seqs


@pytest.mark.parametrize("n_a,n_b", [(0, 0), (0, 5), (7, 0), (1, 1), (40, 3), (300, 900), (1500, 700)])
def test_merge_of_two_runs_equals_a_build_of_the_whole_arena(n_a, n_b):
    g = geom(4)
    rng = np.random.default_rng(1000 * n_a + n_b)
    seqs = random_store(rng, n_a + n_b, 3, 40, (n_a + n_b) // 5) if n_a + n_b else []
    whole = synth.make_batch(seqs)
    part_a, part_b = synth.make_batch(seqs[:n_a]), synth.make_batch(seqs[n_a:])
    want_order = oracle.xrun_order(whole.tokens, whole.seq_off)
    want_coff = synth.offsets(synth.chunk_counts(whole.seq_off, g.chunk_tokens))
    with lsmkv.Context(g, 0) as ctx:
        def build(b):
            d_order = torch.full((max(4, b.n),), -1, dtype=torch.int32, device=H.DEV)
            d_coff = torch.full((b.n + 1,), -1, dtype=torch.int64, device=H.DEV)
            ctx.xrun_build(H.dev(b.tokens), H.dev(b.seq_off), b.n, d_order, d_coff)
            return d_order
        order_a, order_b = build(part_a), build(part_b)       # B numbered within B
        n = n_a + n_b
        d_out = torch.full((max(4, n),), -1, dtype=torch.int32, device=H.DEV)
        d_coff = torch.full((n + 1,), -1, dtype=torch.int64, device=H.DEV)
        ctx.xrun_merge(H.dev(whole.tokens), H.dev(whole.seq_off), order_a, n_a, order_b, n_b,
                       d_out, d_coff)
        torch.cuda.synchronize()
        assert np.array_equal(d_out.cpu().numpy().view(np.uint32)[:n], want_order)
        assert np.array_equal(d_coff.cpu().numpy().view(np.uint64), want_coff)
        H.assert_status_clean(ctx)


def test_probe_through_a_merged_run_equals_the_oracle_on_the_whole_store():
    g = geom(4)
    og = H.ogeom(g)
    rng = np.random.default_rng(77)
    seqs = random_store(rng, 600, 3, 64, 100)
    whole = synth.make_batch(seqs)
    vals = make_vals(g, whole, 5, rng)
    n_a = 350
    query = synth.make_batch(random_store(rng, 200, 3, 80, 0) + [s.copy() for s in seqs[::7]])
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, g.chunk_tokens))
    o_hit, o_recs = oracle.xprobe_batch(og, query.tokens, query.seq_off, qoff,
                                        [(whole.tokens, whole.seq_off, vals)])
    with lsmkv.Context(g, 0) as ctx:
        part_a, part_b = synth.make_batch(seqs[:n_a]), synth.make_batch(seqs[n_a:])
        xa, _, _ = gpu_xrun(ctx, g, part_a, make_vals(g, part_a, 0))
        xb, _, _ = gpu_xrun(ctx, g, part_b, make_vals(g, part_b, 0))
        d_tok, d_off, d_vals = H.dev(whole.tokens), H.dev(whole.seq_off), H.dev(vals)
        d_order = torch.full((whole.n,), -1, dtype=torch.int32, device=H.DEV)
        d_coff = torch.full((whole.n + 1,), -1, dtype=torch.int64, device=H.DEV)
        ctx.xrun_merge(d_tok, d_off, xa[3], n_a, xb[3], whole.n - n_a, d_order, d_coff)
        hit, recs, _ = gpu_xprobe(ctx, query, qoff,
                                  [(d_tok, d_off, d_vals, d_order, d_coff, whole.n)])
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        H.assert_status_clean(ctx)
