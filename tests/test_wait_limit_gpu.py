"""The bounded waits of the bulk copy kernel and of the one-pass encoder, made to run out
without anything in flight: one designated piece (slab) arms its completion barrier but starts
no copy (the library's test hook), with the limit set to about a millisecond. The kernel must
come back, report LSMKV_ST_WAIT_EXPIRED, leave what does not depend on the missing piece exactly
as the oracle has it, and the context must go on working."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    g = lsmkv.Geom(2, 2, 64, elem_bytes=2, page_tokens=16, chunk_tokens=16)   # 4 KiB slabs, 4 a chunk
    og = H.ogeom(g)
    rng = np.random.default_rng(3)
    b = synth.make_batch([rng.integers(0, 999, 16 * 4, dtype=np.uint32)])      # 4 chunks: 16 slabs
    coff = synth.offsets([4])
    pool_np = synth.random_pool_bytes(rng, 4, 6, g.page_bytes)
    pages = np.array([3, 0, 5, 1], np.uint32)
    o_keys, o_vals, o_blob = oracle.encode_batch(og, b.tokens, b.seq_off, None, coff, pages,
                                                 pool_np, 0, 0)
    dropped = 5                                               # piece = slab number here
    with lsmkv.Context(g, 0) as ctx:
        pool = H.DevPool(g, 6, pool_np)
        d_tok, d_off, d_coff, d_pt = (H.dev(a) for a in (b.tokens, b.seq_off, coff, pages))
        d_keys = torch.zeros(4 * 32, dtype=torch.uint8, device=H.DEV)
        d_vals = torch.zeros(4 * 16, dtype=torch.uint8, device=H.DEV)
        d_blob = torch.full((4 * g.chunk_bytes,), 0xEE, dtype=torch.uint8, device=H.DEV)

        def encode():
            ctx.encode_batch(1, d_tok, d_off, None, d_coff, 4, d_pt, pool.table, 0, 0, d_keys,
                             d_vals, d_blob, 4 * g.chunk_bytes)
            torch.cuda.synchronize()

        ctx.set_tuning("wait_cycles", 2_000_000)              # about a millisecond
        ctx.set_tuning("test_drop_piece", dropped)
        encode()                                              # returns: the wait is bounded
        st = ctx.last_status()
        assert st["flags"] == lsmkv.ST_WAIT_EXPIRED and st["first_bad"] == dropped
        blob = d_blob.cpu().numpy().reshape(16, g.page_bytes)
        want = o_blob.reshape(16, g.page_bytes)
        for slab in range(16):
            if slab == dropped:
                assert np.all(blob[slab] == 0xEE)             # never copied, never half-written
            else:
                assert np.array_equal(blob[slab], want[slab])
        assert np.array_equal(H.host(d_keys, np.uint64, 4 * 32).reshape(-1, 4), o_keys)
        # the same context, hook off: everything as the oracle has it
        ctx.set_tuning("test_drop_piece", -1)
        ctx.set_tuning("wait_cycles", 2_000_000_000)
        encode()
        assert np.array_equal(d_blob.cpu().numpy(), o_blob)
        assert ctx.last_status()["flags"] == 0
        assert ctx.last_cuda_error() == 0


def test_a_fetch_that_never_comes_ends_the_one_pass_encoder_and_the_context_stays_usable():
    """The one-pass encoder of the compressing codec, with the fetch of one slab armed but never
    started (the library's test hook) and the limit at about a millisecond: the wait for that
    slab runs out, every role of every CTA leaves through its bounded waits, the call reports
    LSMKV_ST_WAIT_EXPIRED, and the next call of the same context, hook off, equals the oracle."""
    g = lsmkv.Geom(3, 8, 64, elem_bytes=2, page_tokens=16, chunk_tokens=16,
                   flags=lsmkv.CODEC_XP12)                    # slabs of 8192 elements, 6 a chunk
    og = H.ogeom(g)
    rng = np.random.default_rng(8)
    n = 40                                                    # 240 slabs: every CTA gets a few
    b = synth.make_batch([rng.integers(0, 999, 16 * n, dtype=np.uint32)])
    coff = synth.offsets([n])
    pool_np = synth.random_pool_bytes(rng, 6, n + 2, g.page_bytes)
    pages = synth.random_pages(rng, n + 2, n)
    o_keys, o_vals, o_blob = oracle.encode_batch_xp12(og, b.tokens, b.seq_off, None, coff, pages,
                                                      pool_np, 0, 0)
    with lsmkv.Context(g, 0) as ctx:
        assert ctx.get_tuning("xp_one_pass") == 1
        bound = ctx.encode_bound(n)
        pool = H.DevPool(g, n + 2, pool_np)
        d_tok, d_off, d_coff, d_pt = (H.dev(a) for a in (b.tokens, b.seq_off, coff, pages))
        d_keys = torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV)
        d_vals = torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV)
        d_blob = torch.full((bound,), 0xEE, dtype=torch.uint8, device=H.DEV)

        def encode():
            ctx.encode_batch(1, d_tok, d_off, None, d_coff, n, d_pt, pool.table, 0, 0, d_keys,
                             d_vals, d_blob, bound)
            torch.cuda.synchronize()

        ctx.set_tuning("wait_cycles", 2_000_000)              # about a millisecond
        ctx.set_tuning("test_drop_piece", 77)                 # slab 77 = chunk 12, slab 5 of it
        encode()                                              # returns: every wait is bounded
        st = ctx.last_status()
        assert st["flags"] & lsmkv.ST_WAIT_EXPIRED
        vals = H.host(d_vals, VAL_DTYPE, n * 16)
        # what was finished before the missing slab is as the oracle has it; the chunk of the
        # missing slab and those behind it have no record
        assert np.array_equal(vals[:12], o_vals[:12])
        end = int(o_vals["offset"][12])
        assert np.array_equal(d_blob.cpu().numpy()[:end], o_blob[:end])
        assert not vals[12:]["offset"].any() and not vals[12:]["reserved"].any()
        ctx.set_tuning("test_drop_piece", -1)
        ctx.set_tuning("wait_cycles", 2_000_000_000)
        encode()
        used = len(o_blob)
        assert np.array_equal(H.host(d_vals, VAL_DTYPE, n * 16), o_vals)
        assert np.array_equal(d_blob.cpu().numpy()[:used], o_blob)
        assert ctx.last_status()["flags"] == 0
        assert ctx.last_cuda_error() == 0
