"""Seeded synthetic workloads (numpy only).

This module only draws random inputs -- token ids, sequence lengths, sharing structure, page
tables, payload bits. It contains none of the method's arithmetic (no key, digest, record or
blob computation), so both the CUDA library's harness and the CPU checker can be fed from it.

The five workloads mirror the shapes the store is meant for: requests that share system/context
prefixes (the paper's evaluation drives the expected hit rate by the ratio of shared to total
prompt tokens, Sec. 4.1 "Workload"), prompt lengths of thousands of tokens, and per-token KV
sizes of tens to hundreds of KB (Sec. 4.1 "Models").
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SEED0 = 20251116


@dataclass
class Batch:
    """A flat batch of token sequences."""
    tokens: np.ndarray    # uint32 [sum len]
    seq_off: np.ndarray   # uint64 [n+1]

    @property
    def n(self) -> int:
        return len(self.seq_off) - 1

    def seq(self, i: int) -> np.ndarray:
        return self.tokens[int(self.seq_off[i]):int(self.seq_off[i + 1])]

    def lengths(self) -> np.ndarray:
        return np.diff(self.seq_off.astype(np.int64))


def make_batch(seqs) -> Batch:
    lens = np.array([len(s) for s in seqs], dtype=np.uint64)
    off = np.zeros(len(seqs) + 1, dtype=np.uint64)
    np.cumsum(lens, out=off[1:])
    tokens = (np.concatenate(seqs).astype(np.uint32) if len(seqs) and off[-1] > 0
              else np.zeros(0, dtype=np.uint32))
    return Batch(tokens, off)


def chunk_counts(seq_off: np.ndarray, chunk_tokens: int) -> np.ndarray:
    """Whole chunks per sequence (a trailing partial chunk is never stored)."""
    return (np.diff(seq_off.astype(np.int64)) // chunk_tokens).astype(np.int64)


def offsets(counts) -> np.ndarray:
    off = np.zeros(len(counts) + 1, dtype=np.uint64)
    np.cumsum(np.asarray(counts, dtype=np.uint64), out=off[1:])
    return off


def rng_for(config_id: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([SEED0 + config_id, stream]))


def random_pages(rng: np.random.Generator, num_pages: int, n: int) -> np.ndarray:
    """n distinct page ids out of num_pages, in random order (fragmented pool)."""
    assert n <= num_pages
    return rng.permutation(num_pages)[:n].astype(np.uint32)


def bf16_normal_bits(rng: np.random.Generator, n: int) -> np.ndarray:
    """n bf16 bit patterns of N(0,1) samples (round-to-nearest-even from float32)."""
    x = rng.standard_normal(n, dtype=np.float32).view(np.uint32)
    x = x + np.uint32(0x7FFF) + ((x >> np.uint32(16)) & np.uint32(1))
    return (x >> np.uint32(16)).astype(np.uint16)


def random_pool_bytes(rng: np.random.Generator, n_buffers: int, num_pages: int,
                      page_bytes: int) -> np.ndarray:
    """uint8 [n_buffers, num_pages, page_bytes] filled with bf16 N(0,1) bit patterns."""
    n16 = n_buffers * num_pages * page_bytes // 2
    return bf16_normal_bits(rng, n16).view(np.uint8).reshape(n_buffers, num_pages, page_bytes)


def zipf_choice(rng: np.random.Generator, n_items: int, a: float, size: int) -> np.ndarray:
    """Zipf(a) over ranks 1..n_items, ranks mapped through a seeded permutation."""
    p = 1.0 / np.arange(1, n_items + 1, dtype=np.float64) ** a
    p /= p.sum()
    perm = rng.permutation(n_items)
    return perm[rng.choice(n_items, size=size, p=p)]


def _redraw_tail(rng, seq: np.ndarray, n_tail: int, vocab: int) -> np.ndarray:
    """Copy of seq with its last n_tail tokens re-drawn; the first re-drawn token is forced to
    differ from the original so the divergence point is exact."""
    out = seq.copy()
    if n_tail <= 0 or len(seq) == 0:
        return out
    n_tail = min(n_tail, len(seq))
    a = len(seq) - n_tail
    out[a:] = rng.integers(0, vocab, n_tail, dtype=np.uint32)
    if out[a] == seq[a]:
        out[a] = (int(seq[a]) + 1) % vocab
    return out


# ---- config 1: tiny codec -----------------------------------------------------------------

@dataclass
class TinyCodec:
    store: Batch
    query: Batch
    expected_hit_tokens: np.ndarray  # tokens of each query that equal its stored sequence


def tiny_codec(n_req: int = 32, seq_len: int = 512, vocab: int = 32000, max_shared: int = 256,
               n_mutate: int = 64, config_id: int = 1) -> TinyCodec:
    rng = rng_for(config_id)
    base = rng.integers(0, vocab, seq_len, dtype=np.uint32)
    seqs = []
    for _ in range(n_req):
        s = rng.integers(0, vocab, seq_len, dtype=np.uint32)
        k = int(rng.integers(0, max_shared + 1))
        s[:k] = base[:k]
        seqs.append(s)
    queries = [_redraw_tail(rng, s, n_mutate, vocab) for s in seqs]
    exp = np.array([seq_len - min(n_mutate, seq_len)] * n_req, dtype=np.int64)
    return TinyCodec(make_batch(seqs), make_batch(queries), exp)


# ---- config 2: Llama-3-8B-shaped requests over a Zipf prefix tree ---------------------------

@dataclass
class PrefixTreeBatch:
    batch: Batch
    node_of_req: np.ndarray      # which of the shared prefixes each request starts with
    shared_tokens: np.ndarray    # how many leading tokens come from that shared prefix


def llama_requests(n_req: int = 256, vocab: int = 128000, min_len: int = 1024,
                   max_len: int = 8192, n_system: int = 8, n_ext: int = 8, zipf_a: float = 1.1,
                   align: int = 16, config_id: int = 2) -> PrefixTreeBatch:
    rng = rng_for(config_id)
    nodes = []
    for _ in range(n_system):
        slen = int(rng.integers(512 // align, 2048 // align + 1)) * align
        sysp = rng.integers(0, vocab, slen, dtype=np.uint32)
        for _ in range(n_ext):
            elen = int(rng.integers(0, 2048 // align + 1)) * align
            nodes.append(np.concatenate([sysp, rng.integers(0, vocab, elen, dtype=np.uint32)]))
    pick = zipf_choice(rng, len(nodes), zipf_a, n_req)
    seqs, shared = [], []
    for r in range(n_req):
        total = int(rng.integers(min_len, max_len + 1))
        pre = nodes[pick[r]][:total]
        suf = rng.integers(0, vocab, total - len(pre), dtype=np.uint32)
        seqs.append(np.concatenate([pre, suf]))
        shared.append(len(pre))
    return PrefixTreeBatch(make_batch(seqs), pick.astype(np.int64),
                           np.array(shared, dtype=np.int64))


# ---- config 3: probe-heavy ----------------------------------------------------------------

@dataclass
class ProbeHeavy:
    store: Batch                 # stored corpus
    store_start_chunk: np.ndarray  # uint32: leading chunks already stored by an earlier sequence
    n_stored: int                # number of stored chunk keys (sum of encoded chunks)
    run_of_key: np.ndarray       # int8 [n_stored]: which run (0 = newest) holds each key
    dup_idx: np.ndarray          # int64: stored keys also planted in a newer run ...
    dup_run: np.ndarray          # int8: ... namely this one, with a different record
    run_sizes: tuple
    query: Batch
    expected_hit: np.ndarray     # planted hit length in chunks per query
    src_of_query: np.ndarray     # stored sequence a query copies from, or -1


def probe_heavy(n_keys: int = 1_000_000, run_sizes=(900, 9_000, 90_000, 900_100),
                n_query: int = 4096, vocab: int = 128000, chunk: int = 16,
                min_len: int = 2048, max_len: int = 32768, n_prefix: int = 256,
                zipf_a: float = 1.2, cached_frac: float = 0.6, dup_frac: float = 0.01,
                config_id: int = 3) -> ProbeHeavy:
    assert sum(run_sizes) == n_keys
    rng = rng_for(config_id)
    pre_max = min(8192, max_len // 2)
    pre_min = min(512, pre_max)
    prefixes = [rng.integers(0, vocab,
                             int(rng.integers(pre_min // chunk, pre_max // chunk + 1)) * chunk,
                             dtype=np.uint32)
                for _ in range(n_prefix)]
    p = 1.0 / np.arange(1, n_prefix + 1, dtype=np.float64) ** zipf_a
    p /= p.sum()
    perm = rng.permutation(n_prefix)
    stored_pre = np.zeros(n_prefix, dtype=np.int64)   # leading prefix chunks already stored
    seqs, starts, total = [], [], 0
    while total < n_keys:
        pid = int(perm[rng.choice(n_prefix, p=p)])
        length = int(rng.integers(min_len, max_len + 1))
        pre = prefixes[pid][:length]
        s = np.concatenate([pre, rng.integers(0, vocab, length - len(pre), dtype=np.uint32)])
        # chunks fully inside a shared prefix that an earlier sequence stored are skipped
        start = int(min(len(pre) // chunk, stored_pre[pid]))
        nch = len(s) // chunk
        new = nch - start
        if new <= 0:
            continue
        if total + new > n_keys:           # truncate the last sequence: exact key count
            nch = start + (n_keys - total)
            s = s[:nch * chunk]
            new = nch - start
        stored_pre[pid] = max(stored_pre[pid], min(nch, len(prefixes[pid]) // chunk))
        seqs.append(s)
        starts.append(start)
        total += new
    store = make_batch(seqs)

    deal = rng.permutation(n_keys)
    run_of_key = np.zeros(n_keys, dtype=np.int8)
    at = 0
    for r, sz in enumerate(run_sizes):
        run_of_key[deal[at:at + sz]] = r
        at += sz
    cand = np.flatnonzero(run_of_key > 0)
    dup_idx = np.sort(rng.choice(cand, size=int(dup_frac * n_keys), replace=False))
    dup_run = (rng.random(len(dup_idx)) * run_of_key[dup_idx]).astype(np.int8)  # newer run

    nch_store = chunk_counts(store.seq_off, chunk)
    qs, exp, src = [], [], []
    for _ in range(n_query):
        length = int(rng.integers(min_len, max_len + 1))
        qn = length // chunk
        if rng.random() < cached_frac:
            sid = int(rng.integers(0, store.n))
            h = int(rng.integers(1, qn + 1))
            h = min(h, int(nch_store[sid]))
            s = store.seq(sid)
            q = rng.integers(0, vocab, length, dtype=np.uint32)
            q[:h * chunk] = s[:h * chunk]
            if h * chunk < min(length, len(s)) and q[h * chunk] == s[h * chunk]:
                q[h * chunk] = (int(s[h * chunk]) + 1) % vocab
            qs.append(q)
            exp.append(h)
            src.append(sid)
        else:
            qs.append(rng.integers(0, vocab, length, dtype=np.uint32))
            exp.append(0)
            src.append(-1)
    return ProbeHeavy(store, np.array(starts, dtype=np.uint32), n_keys, run_of_key, dup_idx,
                      dup_run, tuple(run_sizes), make_batch(qs),
                      np.array(exp, dtype=np.int64), np.array(src, dtype=np.int64))


# ---- config 4: multi-turn conversations ----------------------------------------------------

@dataclass
class MultiTurn:
    full: Batch                  # every conversation's final token history
    turn_end: np.ndarray         # int64 [n_conv, n_turns]: history length after each turn

    def history(self, turn: int) -> Batch:
        """Token histories as they stand after ``turn`` (0-based) has been appended."""
        return make_batch([self.full.seq(c)[:int(self.turn_end[c, turn])]
                           for c in range(self.full.n)])


def multi_turn(n_conv: int = 512, n_turns: int = 8, min_new: int = 256, max_new: int = 1024,
               vocab: int = 128000, config_id: int = 4) -> MultiTurn:
    rng = rng_for(config_id)
    new = rng.integers(min_new, max_new + 1, size=(n_conv, n_turns))
    turn_end = np.cumsum(new, axis=1).astype(np.int64)
    seqs = [rng.integers(0, vocab, int(turn_end[c, -1]), dtype=np.uint32)
            for c in range(n_conv)]
    return MultiTurn(make_batch(seqs), turn_end)


# ---- config 5: long context ----------------------------------------------------------------

@dataclass
class LongContext:
    store: Batch
    query: Batch
    expected_hit_tokens: np.ndarray


def long_context(n_req: int = 4, seq_len: int = 32768, shared: int = 16384, n_mutate: int = 1024,
                 vocab: int = 128000, config_id: int = 5) -> LongContext:
    rng = rng_for(config_id)
    seqs = [rng.integers(0, vocab, seq_len, dtype=np.uint32) for _ in range(n_req)]
    if n_req >= 4:
        seqs[3][:shared] = seqs[2][:shared]
    elif n_req >= 2:
        seqs[1][:shared] = seqs[0][:shared]
    queries = [_redraw_tail(rng, s, n_mutate, vocab) for s in seqs]
    exp = np.array([seq_len - min(n_mutate, seq_len)] * n_req, dtype=np.int64)
    return LongContext(make_batch(seqs), make_batch(queries), exp)
