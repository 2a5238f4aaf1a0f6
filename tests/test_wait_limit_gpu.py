"""The bounded wait of the bulk copy kernel, made to run out without anything in flight: one
designated piece arms its completion barrier but starts no copy (the library's test hook), with
the limit set to about a millisecond. The kernel must come back, report LSMKV_ST_WAIT_EXPIRED
with the piece's number, leave every other slab exactly as the oracle has it, and the context
must go on working."""
import numpy as np
import pytest
import torch

import oracle
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
