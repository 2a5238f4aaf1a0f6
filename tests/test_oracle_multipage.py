"""Pins for chunks that span several pages (chunk_tokens = m * page_tokens): keys follow the
chunk size, records the larger blobs, and a chunk's blob is its m page blobs in token order --
checked against numpy indexing, against the one-page-per-chunk oracle on the same pool, and by
an encode/decode round trip."""
import numpy as np
import pytest

import oracle
from oracle import Geom
from paper_2511_16138_b200 import synth

from test_oracle_codec import position_pool, simple_batch


@pytest.mark.parametrize("m", [2, 3])
def test_blob_is_the_page_blobs_in_token_order(m):
    P, L = 4, 3
    g = Geom(n_layers=L, n_kv_heads=2, head_dim=8, page_tokens=P, chunk_tokens=m * P)
    b, st, coff = simple_batch(g, [m * P * 3 + 1, m * P - 1, m * P * 2])
    n = int(coff[-1])
    assert n == 3 + 0 + 2 and g.chunk_bytes == m * 2 * L * g.page_bytes
    pool = position_pool(g, 32)
    pt = synth.random_pages(np.random.default_rng(4), 32, n * m)
    keys, vals, blob = oracle.encode_batch(g, b.tokens, b.seq_off, None, coff, pt, pool, 7, 100)
    # blob[i, k, l, kv] = pool[kv*L + l, pt[i*m + k]]
    want = pool.reshape(2, L, 32, g.page_bytes)[:, :, pt, :].transpose(2, 1, 0, 3).reshape(-1)
    assert np.array_equal(blob, want)
    assert np.array_equal(vals["offset"], 100 + g.chunk_bytes * np.arange(n, dtype=np.uint64))
    # keys are those of chunks of m*P tokens
    want_keys = np.concatenate([oracle.chunk_keys(g, b.seq(r), 0) for r in range(b.n)])
    assert np.array_equal(keys, want_keys)
    # the same pages packed one page per chunk give the same bytes: a chunk is m page blobs
    g1 = Geom(n_layers=L, n_kv_heads=2, head_dim=8, page_tokens=P, chunk_tokens=P)
    b1, _, coff1 = simple_batch(g1, [P * n * m])
    _, _, blob1 = oracle.encode_batch(g1, b1.tokens, b1.seq_off, None, coff1, pt, pool, 0, 0)
    assert np.array_equal(blob, blob1)


@pytest.mark.parametrize("m", [2, 4])
def test_round_trip_restores_every_page_of_every_hit_chunk(m):
    P = 2
    g = Geom(n_layers=2, n_kv_heads=2, head_dim=8, page_tokens=P, chunk_tokens=m * P)
    b, st, coff = simple_batch(g, [m * P * 4, m * P * 2 + 1])
    n = int(coff[-1])
    rng = np.random.default_rng(6)
    pool = synth.random_pool_bytes(rng, 4, 40, g.page_bytes)
    src = synth.random_pages(rng, 40, n * m)
    keys, vals, blob = oracle.encode_batch(g, b.tokens, b.seq_off, None, coff, src, pool, 0, 0)
    hit = np.array([3, 2], dtype=np.uint32)                   # the first sequence's last chunk is left out
    dst_pages = synth.random_pages(rng, 40, n * m)
    out = np.zeros_like(pool)
    oracle.decode_batch(g, coff, hit, vals, [blob], dst_pages, out)
    touched = np.zeros(40, dtype=bool)
    for q in range(2):
        for j in range(int(hit[q])):
            for k in range(m):
                i = (int(coff[q]) + j) * m + k
                assert np.array_equal(out[:, dst_pages[i]], pool[:, src[i]])
                touched[dst_pages[i]] = True
    assert not out[:, ~touched].any()


def test_compressed_chunks_of_two_pages_round_trip_and_list_every_slab():
    P, L, m = 4, 3, 2
    g = Geom(n_layers=L, n_kv_heads=2, head_dim=16, page_tokens=P, chunk_tokens=m * P)
    b, st, coff = simple_batch(g, [m * P * 3])
    n = 3
    rng = np.random.default_rng(8)
    pool = synth.random_pool_bytes(rng, 2 * L, 16, g.page_bytes)
    src = synth.random_pages(rng, 16, n * m)
    keys, vals, blob = oracle.encode_batch_xp12(g, b.tokens, b.seq_off, None, coff, src, pool, 0, 0)
    dirb = oracle.xp12_dir_bytes(g)
    assert dirb == (4 * (m * 2 * L + 1) + 15) // 16 * 16
    for i in range(n):
        o = int(vals["offset"][i])
        d = blob[o:o + 4 * (m * 2 * L + 1)].view(np.uint32)
        assert d[0] == dirb and d[-1] == vals["reserved"][i] and np.all(np.diff(d.astype(np.int64)) >= 16)
    out = np.zeros_like(pool)
    dst = synth.random_pages(rng, 16, n * m)
    oracle.decode_batch_xp12(g, coff, np.array([3], np.uint32), vals, [blob], dst, out)
    for i in range(n * m):
        assert np.array_equal(out[:, dst[i]], pool[:, src[i]])


def test_chunk_size_must_be_a_multiple_of_the_page_size():
    g = Geom(n_layers=1, n_kv_heads=1, head_dim=8, page_tokens=4, chunk_tokens=6)
    b = synth.make_batch([np.arange(12, dtype=np.uint32)])
    with pytest.raises(oracle.OracleError):
        oracle.encode_batch(g, b.tokens, b.seq_off, None, synth.offsets([2]), None, None, 0, 0,
                            with_blob=False)
