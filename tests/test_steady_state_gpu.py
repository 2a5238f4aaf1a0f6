"""The hot path allocates nothing once it is warm: after lsmkv_reserve() and one call of every
kind at the batch's size, repeating the calls leaves the device's free memory where it was (the
library's header promises that only creation, reserve and a larger batch than any before
allocate)."""
import numpy as np
import pytest
import torch

from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("flags", [lsmkv.CODEC_IDENTITY, lsmkv.CODEC_XP12])
def test_repeated_calls_do_not_allocate(flags):
    g = lsmkv.Geom(2, 2, 64, elem_bytes=2, page_tokens=16, chunk_tokens=16, flags=flags)
    w = synth.tiny_codec(n_req=12, seq_len=16 * 40 + 5, max_shared=200, n_mutate=64, config_id=77)
    coff = synth.offsets(synth.chunk_counts(w.store.seq_off, 16))
    n = int(coff[-1])
    qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
    total = int(qoff[-1])
    rng = np.random.default_rng(1)
    num_pages = max(n, total) + 4
    with lsmkv.Context(g, 0) as ctx:
        ctx.reserve(max(w.store.n, w.query.n), max(n, total))
        pool = H.DevPool(g, num_pages, synth.random_pool_bytes(rng, 2 * g.n_layers, num_pages,
                                                               g.page_bytes))
        dst = H.DevPool(g, num_pages)
        bound = ctx.encode_bound(n)
        t = dict(tok=H.dev(w.store.tokens), off=H.dev(w.store.seq_off), coff=H.dev(coff),
                 src=H.dev(synth.random_pages(rng, num_pages, n)),
                 keys=torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV),
                 vals=torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV),
                 blob=torch.zeros(bound, dtype=torch.uint8, device=H.DEV),
                 rk=torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV),
                 rv=torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV),
                 rn=torch.zeros(1, dtype=torch.int64, device=H.DEV),
                 hx=torch.zeros(32 * lsmkv.lsmkv_hindex_buckets(n), dtype=torch.uint8, device=H.DEV),
                 qtok=H.dev(w.query.tokens), qseq=H.dev(w.query.seq_off), qoff=H.dev(qoff),
                 hit=torch.zeros(w.query.n, dtype=torch.int32, device=H.DEV),
                 recs=torch.zeros(max(1, total) * 16, dtype=torch.uint8, device=H.DEV),
                 dstp=H.dev(synth.random_pages(rng, num_pages, total)))

        def one_pass():
            ctx.encode_batch(w.store.n, t["tok"], t["off"], None, t["coff"], n, t["src"],
                             pool.table, 0, 0, t["keys"], t["vals"], t["blob"], bound)
            ctx.flush_batch(t["keys"], t["vals"], n, t["rk"], t["rv"], t["rn"])
            ctx.hindex_build(t["rk"], n, t["hx"])
            runs = [(t["rk"], t["rv"], n, None, 0, t["hx"], lsmkv.lsmkv_hindex_buckets(n))]
            ctx.probe_batch(w.query.n, t["qtok"], t["qseq"], t["qoff"], total, runs, t["hit"],
                            t["recs"], None)
            ctx.decode_batch(w.query.n, t["qoff"], total, t["hit"], t["recs"],
                             [(t["blob"], bound)], t["dstp"], dst.table)
            torch.cuda.synchronize()

        one_pass()                                           # warm: scratch reaches its size
        free_before, _ = torch.cuda.mem_get_info()
        for _ in range(3):
            one_pass()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        assert np.array_equal(t["hit"].cpu().numpy(), (w.expected_hit_tokens // 16).astype(np.int32))
        assert ctx.last_status()["flags"] == 0
        assert ctx.last_cuda_error() == 0
        ctx.close()                                # raises unless lsmkv_destroy returned LSMKV_OK
        assert ctx.handle is None
