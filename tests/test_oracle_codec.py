"""Pins for the oracle's records, pack (encode) and unpack (decode)."""
import numpy as np
import pytest

import oracle
from oracle import Geom, VAL_DTYPE
from paper_2511_16138_b200 import synth


def position_pool(g: Geom, num_pages: int) -> np.ndarray:
    """Every 16-bit element encodes where it sits: buffer (5 bits), page (5 bits), slot (6 bits)
    -- any misplaced slab or element shows."""
    n16 = g.page_bytes // 2
    buf = np.arange(2 * g.n_layers, dtype=np.uint32)[:, None, None]
    page = np.arange(num_pages, dtype=np.uint32)[None, :, None]
    slot = np.arange(n16, dtype=np.uint32)[None, None, :]
    v = ((buf & 31) << 11) | ((page & 31) << 6) | (slot & 63)
    v = v ^ ((slot >> 6) * 0x9E37 & 0xFFFF)
    return np.ascontiguousarray(v.astype(np.uint16)).view(np.uint8).reshape(
        2 * g.n_layers, num_pages, g.page_bytes)


def simple_batch(g, lens, start=None):
    rng = np.random.default_rng(1)
    b = synth.make_batch([rng.integers(0, 1000, n, dtype=np.uint32) for n in lens])
    nch = synth.chunk_counts(b.seq_off, g.chunk_tokens)
    st = np.zeros(b.n, dtype=np.uint32) if start is None else np.array(start, dtype=np.uint32)
    cnt = np.maximum(nch - st.astype(np.int64), 0)
    return b, st, synth.offsets(cnt)


def test_records_closed_form():
    g = Geom(n_layers=3, n_kv_heads=2, head_dim=8, page_tokens=4, chunk_tokens=4)
    b, st, coff = simple_batch(g, [9, 4, 3, 17])
    n = int(coff[-1])
    assert n == 2 + 1 + 0 + 4
    pool = position_pool(g, 16)
    pt = np.arange(n, dtype=np.uint32)
    keys, vals, blob = oracle.encode_batch(g, b.tokens, b.seq_off, None, coff, pt, pool,
                                           file_id=42, base_offset=1000)
    cb = 2 * 3 * (4 * 2 * 8 * 2)
    assert g.chunk_bytes == cb and blob.size == n * cb
    assert np.all(vals["file_id"] == 42) and np.all(vals["reserved"] == 0)
    assert np.array_equal(vals["offset"], 1000 + cb * np.arange(n, dtype=np.uint64))
    assert int(vals["offset"][-1]) + cb == 1000 + blob.size
    assert vals.dtype.itemsize == 16


def test_keys_in_batch_match_per_sequence_keys_and_start_chunk():
    g = Geom(n_layers=1, n_kv_heads=1, head_dim=8, page_tokens=4, chunk_tokens=4, ns=3)
    b, st, coff = simple_batch(g, [16, 7, 40, 4], start=[1, 0, 7, 5])
    keys, vals, _ = oracle.encode_batch(g, b.tokens, b.seq_off, st, coff, None, None, 0, 0,
                                        with_blob=False)
    assert int(coff[-1]) == 3 + 1 + 3 + 0
    want = np.concatenate([oracle.chunk_keys(g, b.seq(r), int(st[r])) for r in range(b.n)])
    assert np.array_equal(keys, want)


def test_pack_L1_identity_table_is_a_library_gather():
    """One layer, page table = identity: the blob is [K page, V page] per chunk, which numpy
    writes as a stack + reshape."""
    g = Geom(n_layers=1, n_kv_heads=2, head_dim=16, page_tokens=4, chunk_tokens=4)
    n = 6
    b, st, coff = simple_batch(g, [4 * n])
    rng = np.random.default_rng(2)
    pool = synth.random_pool_bytes(rng, 2, n, g.page_bytes)
    _, _, blob = oracle.encode_batch(g, b.tokens, b.seq_off, None, coff,
                                     np.arange(n, dtype=np.uint32), pool, 0, 0)
    want = np.stack([pool[0], pool[1]], axis=1).reshape(-1)
    assert np.array_equal(blob, want)


def test_pack_general_equals_fancy_indexing():
    g = Geom(n_layers=3, n_kv_heads=2, head_dim=8, page_tokens=4, chunk_tokens=4)
    b, st, coff = simple_batch(g, [12, 20, 8])
    n = int(coff[-1])
    pool = position_pool(g, 32)
    pt = synth.random_pages(np.random.default_rng(4), 32, n)
    _, _, blob = oracle.encode_batch(g, b.tokens, b.seq_off, None, coff, pt, pool, 0, 0)
    L = g.n_layers
    # blob[i, l, kv] = pool[kv*L + l, pt[i]]
    want = pool.reshape(2, L, 32, g.page_bytes)[:, :, pt, :].transpose(2, 1, 0, 3).reshape(-1)
    assert np.array_equal(blob, want)
    # and the position code says the same, slab by slab
    slabs = blob.view(np.uint16).reshape(n, L, 2, -1)
    for i in range(n):
        for l in range(L):
            for kv in range(2):
                code = int(slabs[i, l, kv, 0])
                assert code >> 11 == (kv * L + l) & 31 and (code >> 6) & 31 == int(pt[i]) & 31


def test_encode_decode_identity_and_untouched_pages():
    g = Geom(n_layers=2, n_kv_heads=2, head_dim=8, page_tokens=4, chunk_tokens=4)
    b, st, coff = simple_batch(g, [12, 9, 4])
    n = int(coff[-1])
    rng = np.random.default_rng(6)
    pool = synth.random_pool_bytes(rng, 4, 20, g.page_bytes)
    src = synth.random_pages(rng, 20, n)
    keys, vals, blob = oracle.encode_batch(g, b.tokens, b.seq_off, None, coff, src, pool, 0, 64)
    arena = np.concatenate([np.full(64, 0xEE, np.uint8), blob])     # records carry base 64
    dst_pool = np.zeros_like(pool)
    dst = synth.random_pages(rng, 20, n)
    hit = synth.chunk_counts(b.seq_off, 4).astype(np.uint32)
    hit[1] = 1                                                      # decode only 1 of 2 chunks
    oracle.decode_batch(g, coff, hit, vals, [arena], dst, dst_pool)
    touched = np.zeros(20, dtype=bool)
    for q in range(b.n):
        for j in range(int(coff[q + 1] - coff[q])):
            i = int(coff[q]) + j
            if j < hit[q]:
                assert np.array_equal(dst_pool[:, dst[i]], pool[:, src[i]])
                touched[dst[i]] = True
    assert not dst_pool[:, ~touched].any()
    assert touched.sum() == 3 + 1 + 1


def test_decode_routes_by_file_id_and_offset():
    g = Geom(n_layers=1, n_kv_heads=1, head_dim=8, page_tokens=2, chunk_tokens=2)
    cb = g.chunk_bytes
    a0 = np.arange(3 * cb, dtype=np.uint32).astype(np.uint8)
    a1 = (np.arange(2 * cb, dtype=np.uint32) * 7 + 1).astype(np.uint8)
    recs = np.zeros(3, dtype=VAL_DTYPE)
    recs["file_id"] = [1, 0, 0]
    recs["offset"] = [cb, 2 * cb, 0]
    pool = np.zeros((2, 5, g.page_bytes), dtype=np.uint8)
    oracle.decode_batch(g, np.array([0, 3], np.uint64), np.array([3], np.uint32), recs,
                        [a0, a1], np.array([4, 0, 2], np.uint32), pool)
    pb = g.page_bytes
    assert np.array_equal(pool[0, 4], a1[cb:cb + pb]) and np.array_equal(pool[1, 4], a1[cb + pb:])
    assert np.array_equal(pool[0, 0], a0[2 * cb:2 * cb + pb])
    assert np.array_equal(pool[1, 2], a0[pb:2 * pb])
    assert not pool[:, [1, 3]].any()


def test_errors_are_reported_not_raised_as_faults():
    g = Geom(n_layers=1, n_kv_heads=1, head_dim=8, page_tokens=2, chunk_tokens=2)
    b, st, coff = simple_batch(g, [4])
    pool = np.zeros((2, 2, g.page_bytes), dtype=np.uint8)
    with pytest.raises(oracle.OracleError) as e:
        oracle.encode_batch(g, b.tokens, b.seq_off, None, coff, np.array([0, 2], np.uint32),
                            pool, 0, 0)
    assert e.value.code == oracle.EBADPAGE
    recs = np.zeros(1, dtype=VAL_DTYPE)
    recs["offset"] = 8
    with pytest.raises(oracle.OracleError) as e:
        oracle.decode_batch(g, np.array([0, 1], np.uint64), np.array([1], np.uint32), recs,
                            [np.zeros(g.chunk_bytes, np.uint8)], np.array([0], np.uint32), pool)
    assert e.value.code == oracle.EBADREC
    with pytest.raises(oracle.OracleError):
        oracle.encode_batch(g, b.tokens, b.seq_off, None, np.array([0, 1], np.uint64),
                            np.array([0], np.uint32), pool, 0, 0)   # chunk_off disagrees
