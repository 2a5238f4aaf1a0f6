"""The compressing codec on the GPU against the oracle: blobs, records and restored pages are
byte-identical; malformed blobs and short buffers are flagged, never dereferenced."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


def geom(L, H_, D, P):
    return lsmkv.Geom(L, H_, D, elem_bytes=2, page_tokens=P, chunk_tokens=P, flags=lsmkv.CODEC_XP12)


def mixed_pool(rng, g, num_pages):
    """Pages of several kinds, so every branch of the codec is taken."""
    pool = synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages, g.page_bytes)
    v = pool.view(np.uint16)
    n = v.shape[2]
    for p in range(num_pages):
        kind = p % 6
        for b in range(2 * g.n_layers):
            if kind == 1:
                v[b, p] = 0
            elif kind == 2:
                v[b, p] = rng.integers(0, 65536, n, dtype=np.uint16)        # incompressible
            elif kind == 3:
                m = rng.random(n) < 0.3
                v[b, p][m] = 0x0001                                          # many exceptions
            elif kind == 4:
                v[b, p][: n // 2] = 0                                        # exactly half below
            elif kind == 5:                                                  # inf / nan: e_max = 255
                v[b, p] = rng.choice(np.array([0x7F80, 0xFF80, 0x7FC1, 0x8000, 0x3F80, 0x0001,
                                               0x8001, 0x7F00, 0xFF7F], np.uint16), n)
    return pool


@pytest.mark.parametrize("g,generic,one_pass", [
    (geom(3, 2, 16, 4), 0, 1), (geom(2, 8, 128, 16), 0, 1), (geom(2, 8, 128, 16), 0, 0),
    (geom(2, 8, 128, 16), 1, 1), (geom(2, 1, 24, 3), 0, 1), (geom(1, 4, 128, 64), 0, 1),
    (geom(1, 4, 128, 64), 1, 1), (geom(2, 8, 64, 16), 0, 1), (geom(2, 8, 64, 16), 0, 0)])
def test_encode_and_decode_equal_the_oracle(g, generic, one_pass):
    """Slabs of 128, 16384, 72, 32768 and 8192 elements: the one-pass encoder where it applies
    (16384 and 8192 elements), the three-step fast kernels on the same shapes and on 32768, and
    the generic ones forced on the same shapes."""
    og = H.ogeom(g)
    rng = np.random.default_rng(g.page_bytes)
    C = g.chunk_tokens
    b = synth.make_batch([rng.integers(0, 999, n * C + (n % 3), dtype=np.uint32)
                          for n in (5, 1, 0, 9, 14)])
    nch = synth.chunk_counts(b.seq_off, C)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    num_pages = n + 7
    pool_np = mixed_pool(rng, g, num_pages)
    pages = synth.random_pages(rng, num_pages, n)
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(og, b.tokens, b.seq_off, None, coff, pages,
                                                      pool_np, 5, 1024)
    with lsmkv.Context(g, 0) as ctx:
        ctx.set_tuning("xp_generic", generic)
        ctx.set_tuning("xp_one_pass", one_pass)
        bound = ctx.encode_bound(n)
        assert bound == n * oracle.xp12_chunk_bound(og)
        pool = H.DevPool(g, num_pages, pool_np)
        d_keys = torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV)
        d_vals = torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV)
        d_blob = torch.full((bound,), 0xEE, dtype=torch.uint8, device=H.DEV)
        ctx.encode_batch(b.n, H.dev(b.tokens), H.dev(b.seq_off), None, H.dev(coff), n,
                         H.dev(pages), pool.table, 5, 1024, d_keys, d_vals, d_blob, bound)
        torch.cuda.synchronize()
        keys = H.host(d_keys, np.uint64, n * 32).reshape(-1, 4)
        vals = H.host(d_vals, VAL_DTYPE, n * 16)
        assert np.array_equal(keys, o_keys) and np.array_equal(vals, o_vals)
        used = int(vals["offset"][-1]) + int(vals["reserved"][-1]) - 1024
        assert used == o_blob.size < n * g.chunk_bytes + n * 64
        blob = d_blob.cpu().numpy()
        assert np.array_equal(blob[:used], o_blob)
        assert np.all(blob[used:] == 0xEE)                         # nothing written past the end
        # decode: arena holds 1024 bytes of other data, then the blobs
        d_arena = torch.zeros(1024 + used, dtype=torch.uint8, device=H.DEV)
        d_arena[1024:] = d_blob[:used]
        recs = vals.copy()
        recs["file_id"] = 0
        hit = nch.astype(np.uint32)
        hit[0] = 3
        dst_pages = synth.random_pages(rng, num_pages, n)
        o_dst = np.zeros_like(pool_np)
        oracle.decode_batch_xp12(og, coff, hit, recs, [np.concatenate([np.zeros(1024, np.uint8), o_blob])],
                                 dst_pages, o_dst)
        dst = H.DevPool(g, num_pages)
        ctx.decode_batch(b.n, H.dev(coff), n, H.dev(hit), H.dev(recs), [(d_arena, 1024 + used)],
                         H.dev(dst_pages), dst.table)
        torch.cuda.synchronize()
        assert np.array_equal(dst.numpy(), o_dst)
        st = H.assert_status_clean(ctx)
        assert st["chunks_decoded"] == int(hit.sum())


def test_normal_payload_compresses_to_three_quarters_and_roundtrips_through_probe():
    g = geom(4, 8, 128, 16)
    w = synth.tiny_codec(n_req=8, seq_len=256, max_shared=128, n_mutate=64)
    out = H.roundtrip_xp12(g, w.store, w.query, seed=3)
    assert 0.750 < out["ratio"] < 0.753
    assert np.array_equal(out["hit"], w.expected_hit_tokens // 16)


def test_short_blob_buffer_is_flagged_and_malformed_blobs_are_refused():
    g = geom(2, 2, 64, 16)
    og = H.ogeom(g)
    rng = np.random.default_rng(9)
    b = synth.make_batch([rng.integers(0, 99, 16 * 6, dtype=np.uint32)])
    coff = synth.offsets([6])
    pool_np = synth.random_pool_bytes(rng, 4, 8, g.page_bytes)
    pages = np.arange(6, dtype=np.uint32)
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(og, b.tokens, b.seq_off, None, coff, pages,
                                                      pool_np, 0, 0)
    with lsmkv.Context(g, 0) as ctx:
        pool = H.DevPool(g, 8, pool_np)
        cap = int(o_vals["offset"][4])                       # room for 4 of the 6 blobs only
        d_keys = torch.zeros(6 * 32, dtype=torch.uint8, device=H.DEV)
        d_vals = torch.zeros(6 * 16, dtype=torch.uint8, device=H.DEV)
        d_blob = torch.full((o_blob.size,), 0xEE, dtype=torch.uint8, device=H.DEV)
        ctx.encode_batch(1, H.dev(b.tokens), H.dev(b.seq_off), None, H.dev(coff), 6, H.dev(pages),
                         pool.table, 0, 0, d_keys, d_vals, d_blob, cap)
        torch.cuda.synchronize()
        st = ctx.last_status()
        assert st["flags"] == lsmkv.ST_OVERFLOW and st["first_bad"] == 4
        vals = H.host(d_vals, VAL_DTYPE, 6 * 16)
        assert np.array_equal(vals[:4], o_vals[:4]) and not vals["reserved"][4:].any()
        blob = d_blob.cpu().numpy()
        assert np.array_equal(blob[:cap], o_blob[:cap]) and np.all(blob[cap:] == 0xEE)
        # decode with damaged blobs: every damaged chunk is flagged, the others are restored
        arena = o_blob.copy()
        dirb = oracle.xp12_dir_bytes(og)
        o1, o2, o3 = (int(o_vals["offset"][k]) for k in (1, 2, 3))
        arena[o1 + dirb] ^= 0xFF                               # chunk 1: slab 0 magic
        arena[o2 + 4] += 16                                    # chunk 2: directory entry 1 shifted
        arena[o3 + dirb + 4] += 1                              # chunk 3: n_exc disagrees with size
        recs = o_vals.copy()
        recs["reserved"][5] += 16                              # chunk 5: record size != directory
        dst = H.DevPool(g, 8)
        d_arena = torch.from_numpy(arena).to(H.DEV)
        ctx.decode_batch(1, H.dev(coff), 6, H.dev(np.array([6], np.uint32)), H.dev(recs),
                         [(d_arena, arena.size + 64)], H.dev(pages), dst.table)
        torch.cuda.synchronize()
        st = ctx.last_status()
        assert st["flags"] == lsmkv.ST_BAD_RECORD and st["first_bad"] == 1
        out = dst.numpy()
        for p in (0, 4):
            assert np.array_equal(out[:, p], pool_np[:, p])
        assert not out[:, 5].any() and not out[:, 6:].any()    # chunk 5 refused as a whole


def test_codec_needs_16_bit_elements():
    with pytest.raises(lsmkv.LsmkvError):
        lsmkv.Context(lsmkv.Geom(2, 2, 64, elem_bytes=1, flags=lsmkv.CODEC_XP12), 0)
    with pytest.raises(lsmkv.LsmkvError):
        lsmkv.Context(lsmkv.Geom(2, 2, 64, flags=2), 0)


@pytest.mark.parametrize("L,Hh,D", [(16, 8, 128), (12, 8, 64)])
def test_one_pass_encoder_over_many_slabs_equals_the_three_step_one_and_the_oracle(L, Hh, D):
    """Enough slabs that every CTA of the one-pass encoder takes many turns (a few thousand
    slabs of 16384 / 8192 elements, N(0,1) payload with planted special pages): blobs and records
    must equal the three-step encoder's byte for byte, and the oracle's."""
    g = geom(L, Hh, D, 16)
    og = H.ogeom(g)
    rng = np.random.default_rng(L)
    C = 16
    b = synth.make_batch([rng.integers(0, 32000, n * C + 1, dtype=np.uint32)
                          for n in (37, 1, 64, 5, 90)])
    nch = synth.chunk_counts(b.seq_off, C)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    assert n * 2 * L > 4000
    num_pages = n + 3
    pool_np = synth.random_pool_bytes(rng, 2 * L, num_pages, g.page_bytes)
    v = pool_np.view(np.uint16)
    v[3, 5] = 0                                                       # an all-zero slab
    v[0, 7] = rng.integers(0, 65536, v.shape[2], dtype=np.uint16)     # an incompressible one
    v[1, 9][::3] = 0x0001                                             # many exceptions
    pages = synth.random_pages(rng, num_pages, n)
    pages[11] = num_pages + 100                                       # an unusable page id
    outs = []
    with lsmkv.Context(g, 0) as ctx:
        bound = ctx.encode_bound(n)
        pool = H.DevPool(g, num_pages, pool_np)
        for one_pass in (1, 0):
            ctx.set_tuning("xp_one_pass", one_pass)
            d_keys = torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV)
            d_vals = torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV)
            d_blob = torch.full((bound,), 0xEE, dtype=torch.uint8, device=H.DEV)
            ctx.encode_batch(b.n, H.dev(b.tokens), H.dev(b.seq_off), None, H.dev(coff), n,
                             H.dev(pages), pool.table, 2, 0, d_keys, d_vals, d_blob, bound)
            torch.cuda.synchronize()
            st = ctx.last_status()
            assert st["flags"] == lsmkv.ST_BAD_PAGE and st["first_bad"] == 11
            outs.append((H.host(d_vals, VAL_DTYPE, n * 16).copy(), d_blob.cpu().numpy()))
    (v1, b1), (v0, b0) = outs
    assert np.array_equal(v1, v0), "records differ between the two encoders"
    assert np.array_equal(b1, b0), "blobs differ between the two encoders"
    # the oracle refuses an unusable page id, so it encodes the batch with that page readable and
    # the comparison leaves that one chunk out
    good = pages.copy()
    good[11] = 0
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(og, b.tokens, b.seq_off, None, coff, good,
                                                      pool_np, 2, 0)
    a, e = int(o_vals["offset"][11]), int(o_vals["offset"][12])
    assert np.array_equal(v1[:11], o_vals[:11]) and np.array_equal(b1[:a], o_blob[:a])
    shift = int(v1["offset"][12]) - e                                 # the raw-zero chunk's size differs
    assert np.array_equal(v1["reserved"][12:], o_vals["reserved"][12:])
    assert np.array_equal(v1["offset"][12:] - shift, o_vals["offset"][12:])
    used = int(v1["offset"][-1]) + int(v1["reserved"][-1])
    assert np.array_equal(b1[e + shift:used], o_blob[e:])
    assert np.all(b1[used:] == 0xEE)
