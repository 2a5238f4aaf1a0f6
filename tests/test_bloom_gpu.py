"""Bloom filters of runs on the GPU: the filter bytes equal the oracle's, and probing with
filters gives exactly the answers of probing without them (and of the oracle)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu

G = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=16, chunk_tokens=16)


def digest_keys(rng, n):
    k = np.zeros((n, 4), dtype=np.uint64)
    k[:, 0] = rng.integers(0, 3000, n)
    k[:, 1] = rng.integers(0, 2**61 - 1, n, dtype=np.uint64)
    k[:, 2] = rng.integers(0, 2**61 - 1, n, dtype=np.uint64)
    k[:, 3] = rng.integers(0, 2**64, n, dtype=np.uint64)
    return k


def gpu_bloom(ctx, keys_dev, n):
    nb = lsmkv.lsmkv_bloom_blocks(n)
    out = torch.full((nb * 32,), 0xFF, dtype=torch.uint8, device=H.DEV)
    ctx.bloom_build(keys_dev, n, out)
    torch.cuda.synchronize()
    return out, nb


@pytest.mark.parametrize("n", [0, 1, 25, 26, 1000, 123457])
def test_bloom_bytes_equal_the_oracle(n):
    rng = np.random.default_rng(n)
    keys = digest_keys(rng, n)
    with lsmkv.Context(G, 0) as ctx:
        out, nb = gpu_bloom(ctx, H.dev(keys), n)
        assert nb == oracle.bloom_blocks(n)
        assert np.array_equal(out.cpu().numpy(), oracle.bloom_build(keys))


def test_probe_with_filters_equals_probe_without_and_the_oracle():
    w = synth.probe_heavy(n_keys=60000, run_sizes=(60, 540, 5400, 54000), n_query=300,
                          min_len=64, max_len=4096, n_prefix=16)
    g, og = G, H.ogeom(G)
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch - w.store_start_chunk)
    with lsmkv.Context(g, 0) as ctx:
        keys, _, _, _ = H.gpu_encode(ctx, g, w.store, w.store_start_chunk, coff, None, None)
        vals = np.zeros(w.n_stored, dtype=VAL_DTYPE)
        vals["offset"] = np.arange(w.n_stored) * 16 + 16
        runs = []
        for r in range(4):
            sel = w.run_of_key == r
            d = w.dup_idx[w.dup_run == r]
            dv = vals[d].copy()
            dv["file_id"] = 1
            runs.append(H.gpu_flush_run(ctx, np.concatenate([keys[sel], keys[d]]),
                                        np.concatenate([vals[sel], dv])))
        qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
        total = int(qoff[-1])
        o_hit, o_recs, _, _ = oracle.probe_batch(og, w.query.tokens, w.query.seq_off, qoff, runs)
        druns, keep = H.dev_runs(runs)
        with_bloom = []
        for (dk, dv, n), (k, _) in zip(druns, runs):
            b, nb = gpu_bloom(ctx, dk, n)
            assert np.array_equal(b.cpu().numpy(), oracle.bloom_build(k))
            with_bloom.append((dk, dv, n, b, nb))
        d_tok, d_off, d_qoff = H.dev(w.query.tokens), H.dev(w.query.seq_off), H.dev(qoff)
        outs = []
        ctx.last_status()
        for rr in (druns, with_bloom):
            d_hit = torch.full((w.query.n,), -1, dtype=torch.int32, device=H.DEV)
            d_recs = torch.full((total * 16,), 0xAB, dtype=torch.uint8, device=H.DEV)
            ctx.probe_batch(w.query.n, d_tok, d_off, d_qoff, total, rr, d_hit, d_recs, None)
            torch.cuda.synchronize()
            st = ctx.last_status()
            assert st["flags"] == 0
            outs.append((d_hit.cpu().numpy().view(np.uint32), H.host(d_recs, VAL_DTYPE, total * 16)))
        for hit, recs in outs:
            assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        assert np.array_equal(o_hit, w.expected_hit.astype(np.uint32))


def test_filter_over_a_padded_flush_output_ignores_the_padding():
    rng = np.random.default_rng(5)
    keys = digest_keys(rng, 4000)
    keys[2000:] = keys[:2000]                                   # half are duplicates
    vals = np.zeros(4000, dtype=VAL_DTYPE)
    vals["offset"] = np.arange(4000) * 16
    with lsmkv.Context(G, 0) as ctx:
        ok = torch.empty(4000 * 32, dtype=torch.uint8, device=H.DEV)
        ov = torch.empty(4000 * 16, dtype=torch.uint8, device=H.DEV)
        cnt = torch.zeros(1, dtype=torch.int64, device=H.DEV)
        ctx.flush_batch(H.dev(keys), H.dev(vals), 4000, ok, ov, cnt)
        b, nb = gpu_bloom(ctx, ok, 4000)                       # built over the padded length
        torch.cuda.synchronize()
        assert int(cnt.item()) == 2000
        run_keys = H.host(ok, np.uint64, 4000 * 32).reshape(-1, 4)[:2000]
        bloom = b.cpu().numpy()
        # same bits as the definition applied to the 2000 real keys with the padded block count
        want = np.zeros(32 * nb, dtype=np.uint8)
        for k in run_keys:
            blk = (int(k[1]) * nb) >> 61
            for i in range(6):
                p = (int(k[2]) >> (8 * i)) & 255
                want[32 * blk + (p >> 3)] |= 1 << (p & 7)
        assert np.array_equal(bloom, want)
