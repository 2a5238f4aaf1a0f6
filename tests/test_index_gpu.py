"""GPU flush (write batch -> sorted run) and compaction (runs -> one run) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu

G = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=16, chunk_tokens=16)


def rand_batch(rng, n, dup_frac=0.2):
    keys = rng.integers(0, 2**64, (n, 4), dtype=np.uint64)
    if n:
        keys[:, 0] = rng.integers(0, 5, n)                      # ties in the leading words
        keys[:, 1] = rng.integers(0, 7, n, dtype=np.uint64) << np.uint64(58)
        keys[rng.random(n) < 0.3, 2] = 0
        nd = int(n * dup_frac)
        if nd:
            keys[rng.integers(0, n, nd)] = keys[rng.integers(0, n, nd)]   # exact duplicates
        keys[0, 0] = 2**64 - 2                                   # top bit set compares high
    vals = np.zeros(n, dtype=VAL_DTYPE)
    vals["file_id"] = rng.integers(0, 9, n)
    vals["offset"] = np.arange(n) * 16 + 16
    return keys, vals


def gpu_flush(ctx, keys, vals):
    n = len(keys)
    dk, dv = H.dev(keys), H.dev(vals)
    ok = torch.full((max(1, n) * 32,), 0x11, dtype=torch.uint8, device=H.DEV)
    ov = torch.full((max(1, n) * 16,), 0x22, dtype=torch.uint8, device=H.DEV)
    cnt = torch.full((1,), -1, dtype=torch.int64, device=H.DEV)
    ctx.flush_batch(dk, dv, n, ok, ov, cnt)
    torch.cuda.synchronize()
    m = int(cnt.item())
    k = H.host(ok, np.uint64, n * 32).reshape(-1, 4)
    v = H.host(ov, VAL_DTYPE, n * 16)
    return m, k, v, (ok, ov)


def check_padding(k, v, m):
    assert np.all(k[m:] == np.uint64(2**64 - 1)) and not v[m:].view(np.uint8).any()


@pytest.mark.parametrize("n", [0, 1, 2, 3, 255, 256, 511, 512, 513, 1000, 1024, 1025, 4097, 70000])
def test_flush_equals_oracle(n):
    rng = np.random.default_rng(n + 1)
    keys, vals = rand_batch(rng, n)
    want_k, want_v = oracle.flush(keys, vals)
    with lsmkv.Context(G, 0) as ctx:
        m, k, v, _ = gpu_flush(ctx, keys, vals)
        assert m == len(want_k)
        assert np.array_equal(k[:m], want_k) and np.array_equal(v[:m], want_v)
        check_padding(k, v, m)
        # a second flush through the same scratch, smaller, must not see stale data
        keys2, vals2 = rand_batch(rng, n // 2)
        w2 = oracle.flush(keys2, vals2)
        m2, k2, v2, _ = gpu_flush(ctx, keys2, vals2)
        assert m2 == len(w2[0]) and np.array_equal(k2[:m2], w2[0]) and np.array_equal(v2[:m2], w2[1])


def test_flush_of_encoded_keys_and_probe_through_padded_run():
    """Keys straight from the encoder (shared prefixes give duplicates); the padded output is
    used as a run of the input length without reading the count back."""
    g = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=16, chunk_tokens=16)
    w = synth.llama_requests(n_req=40, min_len=256, max_len=2048)
    nch = synth.chunk_counts(w.batch.seq_off, 16)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    with lsmkv.Context(g, 0) as ctx:
        keys, vals, _, _ = H.gpu_encode(ctx, g, w.batch, None, coff, None, None)
        want = oracle.flush(keys, vals)
        m, k, v, (dk, dv) = gpu_flush(ctx, keys, vals)
        assert m == len(want[0]) < n                            # duplicates were dropped
        assert np.array_equal(k[:m], want[0]) and np.array_equal(v[:m], want[1])
        q = w.batch
        d_tok, d_off, d_coff = H.dev(q.tokens), H.dev(q.seq_off), H.dev(coff)
        d_hit = torch.zeros(q.n, dtype=torch.int32, device=H.DEV)
        d_recs = torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV)
        ctx.probe_batch(q.n, d_tok, d_off, d_coff, n, [(dk, dv, n)], d_hit, d_recs, None)
        torch.cuda.synchronize()
        o_hit, o_recs, _, _ = oracle.probe_batch(H.ogeom(g), q.tokens, q.seq_off, coff, [want])
        assert np.array_equal(d_hit.cpu().numpy().view(np.uint32), o_hit)
        assert np.array_equal(H.host(d_recs, VAL_DTYPE, n * 16), o_recs)
        assert ctx.last_status()["flags"] == 0


@pytest.mark.parametrize("sizes", [(5,), (0, 7), (300, 20), (20, 300, 4000), (1, 1, 1, 1, 1),
                                   (1000, 0, 900, 50000, 3), (64,) * 9])
def test_merge_runs_equals_oracle(sizes):
    rng = np.random.default_rng(len(sizes) * 1000 + sum(sizes))
    pool_k, _ = rand_batch(rng, max(8, sum(sizes) // 2 + 8), dup_frac=0.0)   # forces overlaps
    runs = []
    for r, sz in enumerate(sizes):
        idx = rng.integers(0, len(pool_k), sz)
        v = np.zeros(sz, dtype=VAL_DTYPE)
        v["file_id"] = r
        v["offset"] = rng.integers(0, 1 << 40, sz)
        runs.append(oracle.flush(pool_k[idx], v))
    want_k, want_v = oracle.merge_runs(runs)
    total = sum(len(k) for k, _ in runs)
    with lsmkv.Context(G, 0) as ctx:
        druns, keep = H.dev_runs(runs)
        ok = torch.zeros(max(1, total) * 32, dtype=torch.uint8, device=H.DEV)
        ov = torch.zeros(max(1, total) * 16, dtype=torch.uint8, device=H.DEV)
        cnt = torch.full((1,), -1, dtype=torch.int64, device=H.DEV)
        ctx.merge_runs(druns, ok, ov, cnt)
        torch.cuda.synchronize()
        m = int(cnt.item())
        k = H.host(ok, np.uint64, total * 32).reshape(-1, 4)
        v = H.host(ov, VAL_DTYPE, total * 16)
        assert m == len(want_k)
        assert np.array_equal(k[:m], want_k) and np.array_equal(v[:m], want_v)
        check_padding(k, v, m)


def test_flush_argument_checks():
    with lsmkv.Context(G, 0) as ctx:
        z = torch.zeros(64, dtype=torch.uint8, device=H.DEV)
        with pytest.raises(lsmkv.LsmkvError):
            ctx.flush_batch(z, z, 1, z, z, None)
        with pytest.raises(lsmkv.LsmkvError):
            ctx.flush_batch(None, z, 1, z, z, z)
        with pytest.raises(lsmkv.LsmkvError):
            ctx.merge_runs([(z, z, 1)] * 65, z, z, z)


def test_relocate_records_equals_oracle():
    rng = np.random.default_rng(31)
    n = 70001
    v = np.zeros(n, dtype=VAL_DTYPE)
    v["file_id"] = rng.integers(0, 7, n)
    v["reserved"] = rng.integers(0, 2**32, n, dtype=np.uint64).astype(np.uint32)
    v["offset"] = rng.integers(0, 1 << 44, n, dtype=np.uint64)
    table = [(1, 0, 1 << 35), (2, 0, 3 << 35), (5, 4, 4096), (0, 9, 16)]
    want, changed = oracle.relocate_records(v, np.array(table, dtype=oracle.RELOC_DTYPE))
    with lsmkv.Context(G, 0) as ctx:
        dv = H.dev(v)
        cnt = torch.full((1,), -1, dtype=torch.int64, device=H.DEV)
        ctx.relocate_records(dv, n, table, cnt)
        torch.cuda.synchronize()
        assert np.array_equal(H.host(dv, VAL_DTYPE, n * 16), want) and int(cnt.item()) == changed
        ctx.relocate_records(dv, n, [], cnt)                   # empty table: nothing changes
        torch.cuda.synchronize()
        assert np.array_equal(H.host(dv, VAL_DTYPE, n * 16), want) and int(cnt.item()) == 0
        with pytest.raises(lsmkv.LsmkvError):
            ctx.relocate_records(dv, n, [(0, 1, 0)] * 65, cnt)
