"""A put / probe / get round trip with torch tensors, through the library's public calls.

    python -m paper_2511_16138_b200.example

Eight requests put their KV pages into one blob (keys, records, blob: `encode_batch`), the batch
becomes a sorted run with its hash index (`flush_batch`, `hindex_build`), new requests that share
prefixes with the stored ones are probed for their longest cached prefix (`probe_batch`) and the
hit chunks are scattered into fresh pages of a second pool (`decode_batch`). The script checks
the hit lengths it planted and that every restored page equals its source page. Needs a CUDA
device and the built library (`python -m paper_2511_16138_b200.build`).
"""
from __future__ import annotations

import numpy as np
import torch

from . import lsmkv


def offsets(counts) -> np.ndarray:
    return np.concatenate([[0], np.cumsum(counts)]).astype(np.uint64)


def main() -> None:
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(0)
    g = lsmkv.Geom(n_layers=4, n_kv_heads=8, head_dim=128, page_tokens=16, chunk_tokens=16)
    C = g.chunk_tokens

    def up(a: np.ndarray) -> torch.Tensor:
        return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).to(dev)

    # ---- the stored requests: token sequences and the pages that hold their KV entries
    stored = [rng.integers(0, 32000, int(n), dtype=np.uint32) for n in rng.integers(64, 600, 8)]
    s_tok, s_off = np.concatenate(stored), offsets([len(s) for s in stored])
    s_nch = np.array([len(s) // C for s in stored])          # whole chunks only
    s_coff = offsets(s_nch)
    n = int(s_coff[-1])
    num_pages = n + 8
    src = [torch.randn(num_pages * g.page_bytes // 2, dtype=torch.bfloat16, device=dev)
           .view(torch.uint8).view(num_pages, g.page_bytes) for _ in range(2 * g.n_layers)]
    src_pages = rng.permutation(num_pages)[:n].astype(np.uint32)     # one page per chunk

    with lsmkv.Context(g, 0) as ctx:
        # ---- put: keys, records and the packed blob of the batch
        keys = torch.empty(n * 32, dtype=torch.uint8, device=dev)
        vals = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        blob = torch.empty(n * g.chunk_bytes, dtype=torch.uint8, device=dev)
        ctx.encode_batch(len(stored), up(s_tok), up(s_off), None, up(s_coff), n, up(src_pages),
                         lsmkv.pool_table(src), 0, 0, keys, vals, blob, n * g.chunk_bytes)
        # ---- the batch becomes a sorted run, with a hash index for point lookups
        run_keys, run_vals = torch.empty_like(keys), torch.empty_like(vals)
        run_n = torch.zeros(1, dtype=torch.int64, device=dev)
        ctx.flush_batch(keys, vals, n, run_keys, run_vals, run_n)
        m = int(run_n.item())
        n_buckets = lsmkv.lsmkv_hindex_buckets(m)
        hindex = torch.empty(n_buckets * 32, dtype=torch.uint8, device=dev)
        ctx.hindex_build(run_keys, m, hindex)
        runs = [(run_keys, run_vals, m, None, 0, hindex, n_buckets)]

        # ---- new requests: a stored prefix of known length, then other tokens
        want, queries = [], []
        for i, s in enumerate(stored):
            share = int(rng.integers(0, len(s) // C + 1))    # chunks shared with stored request i
            tail = rng.integers(32000, 64000, int(rng.integers(1, 200)), dtype=np.uint32)
            queries.append(np.concatenate([s[:share * C], tail]))
            want.append(share)
        q_tok, q_off = np.concatenate(queries), offsets([len(q) for q in queries])
        q_nch = np.array([len(q) // C for q in queries])
        q_coff = offsets(q_nch)
        total = int(q_coff[-1])
        hit = torch.zeros(len(queries), dtype=torch.int32, device=dev)
        recs = torch.empty(max(1, total) * 16, dtype=torch.uint8, device=dev)
        d_qcoff = up(q_coff)
        ctx.probe_batch(len(queries), up(q_tok), up(q_off), d_qcoff, total, runs, hit, recs, None)
        got = hit.cpu().numpy().tolist()
        assert got == want, (got, want)

        # ---- get: the hit chunks go into fresh pages of another pool
        dst_num_pages = total + 8                            # a page for every query chunk
        dst = [torch.zeros((dst_num_pages, g.page_bytes), dtype=torch.uint8, device=dev)
               for _ in range(2 * g.n_layers)]
        dst_pages = rng.permutation(dst_num_pages)[:total].astype(np.uint32)
        ctx.decode_batch(len(queries), d_qcoff, total, hit, recs, [(blob, n * g.chunk_bytes)],
                         up(dst_pages), lsmkv.pool_table(dst))
        torch.cuda.synchronize()
        status = ctx.last_status()
        assert status["flags"] == 0, status

    # every restored page equals the page its chunk was put from
    checked = 0
    for i, share in enumerate(want):
        for j in range(share):
            sp = int(src_pages[int(s_coff[i]) + j])
            dp = int(dst_pages[int(q_coff[i]) + j])
            for a, b in zip(src, dst):
                assert torch.equal(a[sp], b[dp])
            checked += 1
    print("put %d chunks (%.1f MiB), hit lengths %s, %d chunks restored and compared"
          % (n, n * g.chunk_bytes / 2**20, got, checked))


if __name__ == "__main__":
    main()
