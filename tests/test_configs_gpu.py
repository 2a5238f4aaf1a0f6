"""Full-size parity on the named workloads, in the launch configuration the benchmark times
(default tuning, waves sized for HBM). Metadata (keys, records, hit lengths, hit records) is
compared with the oracle in full. Payload: every blob of every wave is checked on the device,
slab by slab, against the pool pages it must hold (a statement of the blob layout in tensor
indexing, independent of the library); one whole wave of the Llama-shaped workload and the whole
long-context workload are also streamed through the oracle's encoder in slices and compared byte
for byte; the other waves on sampled chunk ranges. Restored pages: sampled against the oracle's
decode, plus device-side identities that hold at any size (decode(encode(x)) == x on every
page, untouched pages stay zero)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
import hostindex
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


def up(a):
    return H.dev(a)


def down(t, dtype, n_bytes):
    return H.host(t, dtype, n_bytes)


def sample_ranges(rng, nch, n_samples, width):
    """(request, a, b) chunk ranges, always including the first chunks of the first request and
    the last chunks of the last one."""
    out = []
    reqs = [r for r in range(len(nch)) if nch[r] > 0]
    for r in rng.choice(reqs, size=min(n_samples, len(reqs)), replace=False):
        n = int(nch[r])
        a = int(rng.integers(0, max(1, n - width + 1)))
        out.append((int(r), a, min(n, a + width)))
    r0, rl = reqs[0], reqs[-1]
    out.append((r0, 0, min(int(nch[r0]), 2)))
    out.append((rl, max(0, int(nch[rl]) - 2), int(nch[rl])))
    return out


def blobs_hold_their_pages_on_gpu(g, arena, n, src, src_pages, slice_chunks=2048) -> bool:
    """The blob layout written out with tensor indexing: blob i is 2L slabs, slab 2l + kv is page
    src_pages[i] of buffer kv * L + l (K of layer l, then V of layer l). One page per chunk."""
    assert g.pages_per_chunk == 1
    L = g.n_layers
    blobs = arena[:n * g.chunk_bytes].view(n, 2 * L, g.page_bytes)
    sp = torch.as_tensor(np.asarray(src_pages, dtype=np.int64), device=H.DEV)
    for kv in range(2):
        for l in range(L):
            buf = src.bufs[kv * L + l]
            for a in range(0, n, slice_chunks):
                if not torch.equal(blobs[a:a + slice_chunks, 2 * l + kv], buf[sp[a:a + slice_chunks]]):
                    return False
    return True


class PinnedFetch:
    """Device -> host copies through one reusable pinned buffer."""

    def __init__(self, nbytes):
        self.t = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)

    def __call__(self, d):
        d = d.reshape(-1)
        out = self.t[:d.numel()]
        out.copy_(d)
        torch.cuda.synchronize()
        return out.numpy()


def whole_wave_against_oracle(g, batch, nch, coff, src, src_pages, arena, keys, vals,
                              slice_bytes=1 << 30):
    """Every blob of the wave from the oracle's encoder, in slices of whole chunk ranges of one
    request (host copies of that range's pages in, blob bytes out), against the arena."""
    og = H.ogeom(g)
    cb, C, L2 = g.chunk_bytes, g.chunk_tokens, 2 * g.n_layers
    per = max(1, slice_bytes // cb)
    fetch_pool, fetch_blob = PinnedFetch(per * cb), PinnedFetch(per * cb)
    checked = 0
    for r in range(batch.n):
        toks = batch.seq(r)
        for a in range(0, int(nch[r]), per):
            b = min(int(nch[r]), a + per)
            i0 = int(coff[r]) + a
            idx = torch.as_tensor(src_pages[i0:i0 + b - a].astype(np.int64), device=H.DEV)
            host_pool = fetch_pool(torch.stack([buf[idx] for buf in src.bufs])).reshape(
                L2, b - a, g.page_bytes)
            t = np.ascontiguousarray(toks[:b * C])
            k, v, blob = oracle.encode_batch(og, t, np.array([0, len(t)], np.uint64),
                                             np.array([a], np.uint32),
                                             np.array([0, b - a], np.uint64),
                                             np.arange(b - a, dtype=np.uint32), host_pool, 0,
                                             i0 * cb)
            assert np.array_equal(k, keys[i0:i0 + b - a]) and np.array_equal(v, vals[i0:i0 + b - a])
            got = fetch_blob(arena[i0 * cb:(i0 + b - a) * cb])
            assert np.array_equal(got, blob), f"blob of request {r} chunks [{a},{b}) differs"
            checked += b - a
    assert checked == int(coff[-1])


def check_restored_sample(g, rng, sel, recs, arena, dst, dst_pages, n_sample):
    """Sampled restored pages against the oracle's decode of the blob their record names."""
    cb = g.chunk_bytes
    for i in rng.choice(sel, size=min(n_sample, len(sel)), replace=False):
        i = int(i)
        off = int(recs[i]["offset"])
        want = H.oracle_decode_one(g, recs[i], arena[off:off + cb].cpu().numpy())
        assert np.array_equal(dst.gather(dst_pages[i:i + 1]), want)


def encode_probe_decode_wave(ctx, g, batch, nch, src, dst, arena, rng, n_sample=4, width=8,
                             whole_wave=False):
    """One wave of 'full encode, probe, decode' with every check. Returns (keys, vals)."""
    og = H.ogeom(g)
    cb = g.chunk_bytes
    coff = synth.offsets(nch)
    n = int(coff[-1])
    src_pages = synth.random_pages(rng, src.num_pages, n)
    dst_pages = synth.random_pages(rng, dst.num_pages, n)
    d_tok, d_off, d_coff = up(batch.tokens), up(batch.seq_off), up(coff)
    d_keys = torch.empty(n * 32, dtype=torch.uint8, device=H.DEV)
    d_vals = torch.empty(n * 16, dtype=torch.uint8, device=H.DEV)
    ctx.encode_batch(batch.n, d_tok, d_off, None, d_coff, n, up(src_pages), src.table, 0, 0,
                     d_keys, d_vals, arena, n * cb)
    torch.cuda.synchronize()
    keys = down(d_keys, np.uint64, n * 32).reshape(-1, 4)
    vals = down(d_vals, VAL_DTYPE, n * 16)
    # metadata: full compare
    o_keys, o_vals, _ = oracle.encode_batch(og, batch.tokens, batch.seq_off, None, coff, None,
                                            None, 0, 0, with_blob=False)
    assert np.array_equal(keys, o_keys) and np.array_equal(vals, o_vals)
    run = H.gpu_flush_run(ctx, keys, vals)
    o_run = oracle.flush(o_keys, o_vals)
    assert np.array_equal(run[0], o_run[0]) and np.array_equal(run[1], o_run[1])
    d_hit = torch.zeros(batch.n, dtype=torch.int32, device=H.DEV)
    d_recs = torch.empty(n * 16, dtype=torch.uint8, device=H.DEV)
    druns, keep = H.dev_runs([run])
    hruns, hkeep = H.with_hindex(ctx, druns)            # the form the benchmark probes
    ctx.probe_batch(batch.n, d_tok, d_off, d_coff, n, druns, d_hit, d_recs, None)
    torch.cuda.synchronize()
    hit_searched = d_hit.cpu().numpy().view(np.uint32).copy()
    recs_searched = down(d_recs, VAL_DTYPE, n * 16).copy()
    d_hit.zero_()
    d_recs.fill_(0xAB)
    ctx.probe_batch(batch.n, d_tok, d_off, d_coff, n, hruns, d_hit, d_recs, None)
    torch.cuda.synchronize()
    hit = d_hit.cpu().numpy().view(np.uint32)
    recs = down(d_recs, VAL_DTYPE, n * 16)
    assert np.array_equal(hit, hit_searched) and np.array_equal(recs, recs_searched)
    o_hit, o_recs, _, _ = oracle.probe_batch(og, batch.tokens, batch.seq_off, coff, [run])
    assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
    assert np.array_equal(hit, nch.astype(np.uint32))
    dst.zero_()
    ctx.decode_batch(batch.n, d_coff, n, d_hit, d_recs, [(arena, n * cb)], up(dst_pages), dst.table)
    torch.cuda.synchronize()
    # payload: every blob against the pages it must hold (device side), the whole wave or
    # sampled ranges against the oracle
    assert blobs_hold_their_pages_on_gpu(g, arena, n, src, src_pages), "a blob differs from its pages"
    if whole_wave:
        whole_wave_against_oracle(g, batch, nch, coff, src, src_pages, arena, keys, vals)
    for r, a, b in sample_ranges(rng, nch, n_sample, width):
        i0 = int(coff[r]) + a
        k, v, blob = H.oracle_blob_range(g, batch.seq(r), a, b, src, src_pages[i0:i0 + b - a], 0,
                                         i0 * cb)
        assert np.array_equal(k, keys[i0:i0 + b - a]) and np.array_equal(v, vals[i0:i0 + b - a])
        got = arena[i0 * cb:(i0 + b - a) * cb].cpu().numpy()
        assert np.array_equal(got, blob), f"blob of request {r} chunks [{a},{b}) differs"
    # restored pages: follow the record (a shared chunk's record names the last writer's blob)
    check_restored_sample(g, rng, np.arange(n), recs, arena, dst, dst_pages, 2 * n_sample)
    # identities at full size, on the device
    src_of_rec = src_pages[(recs["offset"] // cb).astype(np.int64)]
    assert H.pages_equal_on_gpu(src, src_of_rec, dst, dst_pages)
    assert H.untouched_pages_zero(dst, dst_pages)
    assert ctx.last_status()["flags"] == 0
    return keys, vals


def test_config2_llama8b_full_encode_probe_decode():
    """256 requests of 1k-8k tokens, 32x8x128 bf16, page 16 (~147 GiB per direction), in four
    waves as in the benchmark."""
    g = lsmkv.Geom(32, 8, 128, page_tokens=16, chunk_tokens=16)
    w = synth.llama_requests()
    nch = synth.chunk_counts(w.batch.seq_off, 16)
    assert nch.sum() > 70000
    n_waves = 4
    cum = np.cumsum(nch)
    cuts = [int(np.searchsorted(cum, nch.sum() * k / n_waves)) + 1 for k in range(1, n_waves)]
    bounds = [0] + cuts + [len(nch)]
    cap = max(int(nch[a:b].sum()) for a, b in zip(bounds[:-1], bounds[1:]))
    src = H.BigPool(g, cap, fill=True, seed=2)
    dst = H.BigPool(g, cap, fill=False)
    arena = torch.empty(cap * g.chunk_bytes, dtype=torch.uint8, device=H.DEV)
    rng = synth.rng_for(2, 5)
    with lsmkv.Context(g, 0) as ctx:
        for k, (a, b) in enumerate(zip(bounds[:-1], bounds[1:])):
            t0, t1 = int(w.batch.seq_off[a]), int(w.batch.seq_off[b])
            wb = synth.Batch(w.batch.tokens[t0:t1], w.batch.seq_off[a:b + 1] - w.batch.seq_off[a])
            encode_probe_decode_wave(ctx, g, wb, nch[a:b], src, dst, arena, rng, whole_wave=k == 1)


def test_config5_long_context_encode_probe_decode():
    """80x8x128 bf16, page 16; 4 x 32768 tokens, two sharing 16k tokens; encode, then probe and
    decode with the last 1k tokens changed (40 GiB per direction)."""
    g = lsmkv.Geom(80, 8, 128, page_tokens=16, chunk_tokens=16)
    og = H.ogeom(g)
    cb = g.chunk_bytes
    w = synth.long_context()
    nch = synth.chunk_counts(w.store.seq_off, 16)
    n = int(nch.sum())
    assert n == 8192
    src = H.BigPool(g, n, fill=True, seed=5)
    dst = H.BigPool(g, n, fill=False)
    arena = torch.empty(n * cb, dtype=torch.uint8, device=H.DEV)
    rng = synth.rng_for(5, 5)
    with lsmkv.Context(g, 0) as ctx:
        keys, vals = encode_probe_decode_wave(ctx, g, w.store, nch, src, dst, arena, rng, width=4,
                                              whole_wave=True)
        run = H.gpu_flush_run(ctx, keys, vals)
        qn = synth.chunk_counts(w.query.seq_off, 16)
        qoff = synth.offsets(qn)
        hit, recs, qkeys, (d_qoff, d_hit, d_recs) = H.gpu_probe(ctx, w.query, qoff, [run])
        o_hit, o_recs, o_qkeys, _ = oracle.probe_batch(og, w.query.tokens, w.query.seq_off, qoff,
                                                       [oracle.flush(keys, vals)], want_keys=True)
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        assert np.array_equal(qkeys, o_qkeys)
        assert list(hit) == [1984] * 4
        dst.zero_()
        dst_pages = synth.random_pages(rng, n, int(qoff[-1]))
        ctx.decode_batch(4, d_qoff, int(qoff[-1]), d_hit, d_recs, [(arena, n * cb)], up(dst_pages),
                         dst.table)
        torch.cuda.synchronize()
        sel = np.concatenate([np.arange(int(qoff[q]), int(qoff[q]) + int(hit[q])) for q in range(4)])
        assert H.untouched_pages_zero(dst, dst_pages[sel])
        check_restored_sample(g, rng, sel, recs, arena, dst, dst_pages, 6)
        assert ctx.last_status()["flags"] == 0


def test_config3_probe_heavy_full():
    """1M stored chunk keys in 4 runs (900 / 9000 / 90000 / 900100, 1% newer duplicates), 4096
    queries of 2k-32k tokens, 60% with a cached prefix; decode of the hits into an 8x8x128 pool
    from an arena of 32768 aliased blobs."""
    g = lsmkv.Geom(8, 8, 128, page_tokens=16, chunk_tokens=16)
    og = H.ogeom(g)
    cb = g.chunk_bytes
    w = synth.probe_heavy()
    n_blobs = 32768
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch - w.store_start_chunk)
    assert int(coff[-1]) == w.n_stored == 1_000_000
    with lsmkv.Context(g, 0) as ctx:
        keys, _, _, _ = H.gpu_encode(ctx, g, w.store, w.store_start_chunk, coff, None, None)
        o_keys, _, _ = oracle.encode_batch(og, w.store.tokens, w.store.seq_off,
                                           w.store_start_chunk, coff, None, None, 0, 0,
                                           with_blob=False)
        assert np.array_equal(keys, o_keys)
        vals = np.zeros(w.n_stored, dtype=VAL_DTYPE)
        vals["offset"] = (np.arange(w.n_stored) % n_blobs) * cb
        runs = []
        for r in range(4):
            sel = w.run_of_key == r
            d = w.dup_idx[w.dup_run == r]
            dv = vals[d].copy()
            dv["offset"] = ((d + 7919) % n_blobs) * cb            # newer copy, different record
            runs.append(H.gpu_flush_run(ctx, np.concatenate([keys[sel], keys[d]]),
                                        np.concatenate([vals[sel], dv])))
            o_run = oracle.flush(np.concatenate([keys[sel], keys[d]]),
                                 np.concatenate([vals[sel], dv]))
            assert np.array_equal(runs[r][0], o_run[0]) and np.array_equal(runs[r][1], o_run[1])
        assert len(runs[3][0]) == 900_100
        qn = synth.chunk_counts(w.query.seq_off, 16)
        qoff = synth.offsets(qn)
        total = int(qoff[-1])
        hit, recs, _, (d_qoff, d_hit, d_recs) = H.gpu_probe(ctx, w.query, qoff, runs,
                                                           want_keys=False)
        o_hit, o_recs, _, _ = oracle.probe_batch(og, w.query.tokens, w.query.seq_off, qoff, runs)
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        assert np.array_equal(hit, w.expected_hit.astype(np.uint32))
        st = ctx.last_status()
        assert st["flags"] == 0 and st["chunks_hit"] == 2 * int(hit.sum())   # probed both ways
        assert st["empty_probes"] == 2 * int((hit == 0).sum())

        # decode the hits in waves of queries into a 64 GiB pool
        num_pages = 131072
        gen = torch.Generator(device=H.DEV)
        gen.manual_seed(3)
        arena = torch.randn(n_blobs * cb // 2, dtype=torch.bfloat16, device=H.DEV,
                            generator=gen).view(torch.uint8)
        dst = H.BigPool(g, num_pages, fill=False)
        rng = synth.rng_for(3, 5)
        arena_blobs = arena.view(n_blobs, 2 * g.n_layers, g.page_bytes)
        L = g.n_layers
        q0 = n_waves = 0
        while q0 < w.query.n:
            q1, acc = q0, 0
            while q1 < w.query.n and acc + int(hit[q1]) <= num_pages:
                acc += int(hit[q1])
                q1 += 1
            sel = np.concatenate([np.arange(int(qoff[q]), int(qoff[q]) + int(hit[q]))
                                  for q in range(q0, q1)] + [np.zeros(0, np.int64)]).astype(np.int64)
            dst_pages = np.zeros(total, dtype=np.uint32)
            dst_pages[sel] = synth.random_pages(rng, num_pages, len(sel))
            hit_w = np.zeros_like(hit)
            hit_w[q0:q1] = hit[q0:q1]
            dst.zero_()
            ctx.decode_batch(w.query.n, d_qoff, total, up(hit_w), d_recs, [(arena, n_blobs * cb)],
                             up(dst_pages), dst.table)
            torch.cuda.synchronize()
            # every restored page equals the slab of the blob its record names (device side)
            blob_idx = torch.as_tensor((recs["offset"][sel] // cb).astype(np.int64), device=H.DEV)
            dp = torch.as_tensor(dst_pages[sel].astype(np.int64), device=H.DEV)
            for bi, buf in enumerate(dst.bufs):
                slab = 2 * (bi % L) + (bi // L)                 # buffers: K layers, then V layers
                for a in range(0, len(sel), 16384):
                    assert torch.equal(buf[dp[a:a + 16384]],
                                       arena_blobs[blob_idx[a:a + 16384], slab])
            assert H.untouched_pages_zero(dst, dst_pages[sel])
            if len(sel):
                check_restored_sample(g, rng, sel, recs, arena, dst, dst_pages, 6)
            q0 = q1
            n_waves += 1
        assert n_waves >= 2
        st = ctx.last_status()
        assert st["flags"] == 0 and st["chunks_decoded"] == int(hit.sum())


def test_config4_gqa_multi_turn():
    """28x4x128 bf16, page 64; 512 conversations x 8 turns of 256-1024 new tokens: per turn probe
    and decode the stored history, then encode the new chunks (start_chunk) and flush them as a
    new newest run; conversations in groups of 64, the two oldest runs merged when more than 4
    pile up."""
    g = lsmkv.Geom(28, 4, 128, page_tokens=64, chunk_tokens=64)
    og = H.ogeom(g)
    cb, C = g.chunk_bytes, 64
    w = synth.multi_turn()
    n_conv, n_turns, group = w.full.n, w.turn_end.shape[1], 64
    final_nch = synth.chunk_counts(w.full.seq_off, C)
    cap = int(max(final_nch[a:a + group].sum() for a in range(0, n_conv, group)))
    src = H.BigPool(g, cap, fill=True, seed=4)
    dst = H.BigPool(g, cap, fill=False)
    arena = torch.empty(cap * cb, dtype=torch.uint8, device=H.DEV)
    rng = synth.rng_for(4, 5)
    total_encoded = total_decoded = 0
    with lsmkv.Context(g, 0) as ctx:
        for g0 in range(0, n_conv, group):
            convs = list(range(g0, min(n_conv, g0 + group)))
            perm = synth.random_pages(rng, cap, int(final_nch[g0:g0 + group].sum()))
            page_of, at = {}, 0
            for c in convs:                        # every conversation owns its source pages
                page_of[c] = perm[at:at + int(final_nch[c])]
                at += int(final_nch[c])
            runs, o_runs = [], []
            stored = np.zeros(len(convs), dtype=np.int64)
            used = 0
            blob_page = np.zeros(cap, dtype=np.int64)   # arena blob index -> source page packed
            for t in range(n_turns):
                hist = synth.make_batch([w.full.seq(c)[:int(w.turn_end[c, t])] for c in convs])
                nch = synth.chunk_counts(hist.seq_off, C)
                qoff = synth.offsets(nch)
                total = int(qoff[-1])
                if runs:                           # probe + decode the history stored so far
                    hit, recs, _, (d_qoff, d_hit, d_recs) = H.gpu_probe(ctx, hist, qoff, runs,
                                                                       want_keys=False)
                    o_hit, o_recs, _, _ = oracle.probe_batch(og, hist.tokens, hist.seq_off, qoff,
                                                             o_runs)
                    assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
                    assert np.array_equal(hit, stored.astype(np.uint32))
                    dst_pages = synth.random_pages(rng, cap, total)
                    dst.zero_()
                    ctx.decode_batch(hist.n, d_qoff, total, d_hit, d_recs, [(arena, used * cb)],
                                     up(dst_pages), dst.table)
                    torch.cuda.synchronize()
                    sel = np.concatenate([np.arange(int(qoff[q]), int(qoff[q]) + int(hit[q]))
                                          for q in range(hist.n)]).astype(np.int64)
                    want_src = blob_page[(recs["offset"][sel] // cb).astype(np.int64)]
                    assert H.pages_equal_on_gpu(src, want_src, dst, dst_pages[sel])
                    assert H.untouched_pages_zero(dst, dst_pages[sel])
                    check_restored_sample(g, rng, sel, recs, arena, dst, dst_pages, 1)
                    total_decoded += len(sel)
                start = stored.astype(np.uint32)   # encode the new chunks of this turn
                coff = synth.offsets(nch - stored)
                n = int(coff[-1])
                src_pages = np.concatenate([page_of[c][int(stored[k]):int(nch[k])]
                                            for k, c in enumerate(convs)]).astype(np.uint32)
                d_keys = torch.empty(max(1, n) * 32, dtype=torch.uint8, device=H.DEV)
                d_vals = torch.empty(max(1, n) * 16, dtype=torch.uint8, device=H.DEV)
                ctx.encode_batch(hist.n, up(hist.tokens), up(hist.seq_off), up(start), up(coff), n,
                                 up(src_pages), src.table, 0, used * cb, d_keys, d_vals,
                                 arena[used * cb:], (cap - used) * cb)
                torch.cuda.synchronize()
                keys = down(d_keys, np.uint64, n * 32).reshape(-1, 4)
                vals = down(d_vals, VAL_DTYPE, n * 16)
                o_keys, o_vals, _ = oracle.encode_batch(og, hist.tokens, hist.seq_off, start, coff,
                                                        None, None, 0, used * cb, with_blob=False)
                assert np.array_equal(keys, o_keys) and np.array_equal(vals, o_vals)
                blob_page[used:used + n] = src_pages
                assert blobs_hold_their_pages_on_gpu(g, arena[used * cb:], n, src, src_pages)
                for _ in range(2):                 # sampled blob ranges against the oracle
                    k = int(rng.integers(0, hist.n))
                    if nch[k] == stored[k]:
                        continue
                    a = int(rng.integers(int(stored[k]), int(nch[k])))
                    b = min(int(nch[k]), a + 2)
                    i0 = int(coff[k]) + a - int(stored[k])
                    kk, vv, blob = H.oracle_blob_range(g, hist.seq(k), a, b, src,
                                                       src_pages[i0:i0 + b - a], 0,
                                                       (used + i0) * cb)
                    assert np.array_equal(kk, keys[i0:i0 + b - a])
                    assert np.array_equal(vv, vals[i0:i0 + b - a])
                    got = arena[(used + i0) * cb:(used + i0 + b - a) * cb].cpu().numpy()
                    assert np.array_equal(got, blob)
                used += n
                total_encoded += n
                stored = nch.copy()
                runs.insert(0, H.gpu_flush_run(ctx, keys, vals))
                o_runs.insert(0, oracle.flush(o_keys, o_vals))
                assert np.array_equal(runs[0][0], o_runs[0][0])
                assert np.array_equal(runs[0][1], o_runs[0][1])
                if len(runs) > 4:                  # compaction of the two oldest runs
                    runs[-2:] = [H.gpu_merge_runs(ctx, runs[-2:])]
                    o_runs[-2:] = [oracle.merge_runs(o_runs[-2:])]
                    assert np.array_equal(runs[-1][0], o_runs[-1][0])
                    assert np.array_equal(runs[-1][1], o_runs[-1][1])
            assert used == int(final_nch[g0:g0 + group].sum())
        assert ctx.last_status()["flags"] == 0
    assert total_encoded == int(final_nch.sum()) and total_decoded > 3 * total_encoded
