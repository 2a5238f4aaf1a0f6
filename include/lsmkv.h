/*
 * lsmkv.h -- C ABI of the B200 batch codec and longest-cached-prefix probe for an LSM-backed
 * KV-cache store (device half of the put_batch / probe / get_batch operations of
 * "On 10X Better Scalability: KV Stores Scale Up KV Cache", Sec. 3.2 and App. B, with the
 * batch codec of Sec. 3.4).
 *
 * General rules
 *   - Pointers marked [dev] are device pointers on the context's GPU, [host] are host pointers.
 *     The caller owns every buffer; the library keeps no reference after a call returns,
 *     except that device work enqueued by the call reads/writes the [dev] buffers until the
 *     stream reaches the point following the call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Every
 *     batch call only enqueues work and returns; none of them synchronises (one documented
 *     exception: lsmkv_put_batch_host with the compressing codec, which waits briefly for the
 *     records of each slice unless asked to place the bytes from the device).
 *   - Return value: 0 = enqueued, negative = LSMKV_E* and nothing was enqueued.
 *   - Problems only the GPU can see (a page id beyond the pool, a record that points outside
 *     its arena, a misaligned buffer, a wait that ran out) never fault: the offending item is
 *     skipped and recorded in a device status block read back by lsmkv_last_status().
 *   - A context is not thread-safe and orders nothing by itself: calls that share internal
 *     scratch (two probes, two decodes, two flushes/merges, two host-buffer calls of the same
 *     kind) must be ordered by the caller -- same stream, or events. A put on one stream and a
 *     probe/decode on another are independent. Use one context per stream for more.
 *   - No call allocates device memory except lsmkv_create(), lsmkv_reserve() and a call whose
 *     batch is larger than any before it (the internal scratch of that kind of call grows;
 *     lsmkv_reserve() pre-sizes the scratch of probe and decode, a first full-size call that
 *     of flush, merge, the compressing codec and the host-buffer calls; the first host-buffer
 *     put with the compressing codec also creates a stream and three events of the context's).
 *
 * Formats (version 1). The paper states properties (key order follows token-prefix order;
 * index values are a file identifier plus a byte offset; a batch's tensors are stored
 * contiguously); the concrete layouts are this library's:
 *   key     4 x u64, ordered lexicographically as unsigned words:
 *             w0 = (namespace << 32) | chunk index j
 *             w1, w2 = two digests of the token prefix S[0 : (j+1)*C)
 *             w3 = (first token of chunk j << 32) | last token of chunk j
 *   digest  h <- 0; per token t: h <- (h*BASE + t + 1) mod (2^61 - 1), canonical in [0, 2^61-1)
 *             BASE_A = 0x0B4E0EF37BC32127, BASE_B = 0x16A09E667F3BCC90
 *   record  {u32 file_id, u32 reserved, u64 offset}; identity codec: reserved = 0 and the blob
 *             length is chunk_bytes; compressing codec: reserved = the blob's length
 *   pool    2L buffers: K of layers 0..L-1, then V of layers 0..L-1, each
 *             [num_pages][page_tokens][n_kv_heads][head_dim] elements (a page slab of
 *             page_bytes = page_tokens*n_kv_heads*head_dim*elem_bytes is contiguous)
 *   blob    for every page of the chunk, in token order: for l in 0..L-1: K slab of layer l,
 *             V slab of layer l  (chunk_bytes = m*2L*page_bytes)
 *   A chunk is C = chunk_tokens = m * page_tokens tokens (m >= 1 whole pages); a sequence of len
 *   tokens has floor(len / C) chunks and a trailing partial chunk is never encoded, probed or
 *   decoded. Page tables carry m entries per chunk: entry i*m + k names the pool page of the
 *   k-th page of chunk i.
 */
#ifndef LSMKV_H
#define LSMKV_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LSMKV_FORMAT_VERSION 1
#define LSMKV_MAX_RUNS 64

/* return codes */
#define LSMKV_OK 0
#define LSMKV_EINVAL (-1)     /* null / misaligned pointer, unsupported geometry, bad count */
#define LSMKV_ECAPACITY (-2)  /* an output buffer is too small */
#define LSMKV_ECUDA (-3)      /* a CUDA call failed; see lsmkv_last_cuda_error() */
#define LSMKV_ENOMEM (-4)     /* host or device allocation failed */
#define LSMKV_ETOOBIG (-5)    /* lsmkv_decode_batch_static(): batch larger than the built-in scratch */

/* bits of lsmkv_status_t.flags */
#define LSMKV_ST_BAD_PAGE 0x1u     /* a page id >= num_pages (item skipped) */
#define LSMKV_ST_BAD_RECORD 0x2u   /* file_id >= n_arenas, or offset outside / misaligned (skipped) */
#define LSMKV_ST_BAD_COUNT 0x4u    /* chunk_off / qchunk_off / hit disagree with the sequence lengths */
#define LSMKV_ST_MISALIGNED 0x8u   /* a pool buffer is not 16-byte aligned (skipped) */
#define LSMKV_ST_WAIT_EXPIRED 0x10u /* a bounded wait inside a kernel gave up */
#define LSMKV_ST_OVERFLOW 0x20u    /* compressing codec: a blob did not fit blob_capacity (chunk skipped, empty record) */

/* lsmkv_geom_t.flags */
#define LSMKV_CODEC_IDENTITY 0u    /* blobs are bit copies of the page slabs */
#define LSMKV_CODEC_XP12 1u        /* lossless exponent packing of 16-bit float slabs (see below) */

typedef struct lsmkv_ctx lsmkv_ctx;

typedef struct { uint64_t w[4]; } lsmkv_key_t;                               /* 32 bytes */
typedef struct { uint32_t file_id, reserved; uint64_t offset; } lsmkv_val_t; /* 16 bytes */

typedef struct {
    uint32_t n_layers, n_kv_heads, head_dim, elem_bytes;
    uint32_t page_tokens, chunk_tokens, ns, flags; /* chunk_tokens = m * page_tokens, m >= 1; flags = LSMKV_CODEC_* */
} lsmkv_geom_t;

/* One immutable sorted run of the index: keys ascending and unique, vals[i] belongs to keys[i].
 * bloom (optional, NULL = none): the run's Bloom filter as built by lsmkv_bloom_build, with
 * bloom_blocks 32-byte blocks; the probe then skips the run for keys the filter rules out.
 * hindex (optional, NULL = none): the run's hash index as built by lsmkv_hindex_build, with
 * hindex_buckets 32-byte buckets. When every non-empty run of a probe brings one, point lookups
 * go through the hash indexes instead of searching the sorted keys (and ignore the Bloom
 * filters, which the tables make redundant); otherwise the probe ignores the hash indexes.
 * Alignment: keys, vals, bloom and hindex on 16-byte boundaries (LSMKV_EINVAL otherwise); when
 * keys and hindex of every non-empty run also start on 32-byte boundaries the probe fetches a
 * bucket or a key with one 32-byte load instead of two 16-byte ones (same answers). */
typedef struct {
    const lsmkv_key_t *keys; /* [dev] */
    const lsmkv_val_t *vals; /* [dev] */
    uint64_t n;
    const void *bloom;       /* [dev] or NULL */
    uint64_t bloom_blocks;
    const void *hindex;      /* [dev] or NULL */
    uint64_t hindex_buckets;
} lsmkv_run_t;

/* The paged KV pool. */
typedef struct {
    void *const *kv_ptrs; /* [dev] array of 2L [dev] pointers, each 16-byte aligned */
    uint64_t num_pages;
} lsmkv_pool_t;

typedef struct {
    uint32_t flags;        /* OR of LSMKV_ST_* since the last lsmkv_last_status() */
    uint32_t reserved;
    uint64_t first_bad;    /* smallest item index that set a flag (chunk / query index), or ~0 */
    uint64_t chunks_encoded; /* counters since the last lsmkv_last_status() */
    uint64_t lookups;        /* point lookups performed by probes */
    uint64_t chunks_hit;     /* sum of hit lengths */
    uint64_t empty_probes;   /* queries with hit length 0 */
    uint64_t chunks_decoded;
} lsmkv_status_t;

/*
 * Create a context on `device` for one KV geometry. Allocates the context, a small device
 * status block and the workspace. Errors: LSMKV_EINVAL for a zero field, chunk_tokens not a
 * multiple of page_tokens (or more than 4096 pages per chunk), or page_bytes not a multiple of
 * 16; LSMKV_ECUDA / LSMKV_ENOMEM.
 */
int lsmkv_create(lsmkv_ctx **out, const lsmkv_geom_t *geom, int device);

/* Free everything the context owns. Synchronises the device. NULL is accepted. */
int lsmkv_destroy(lsmkv_ctx *ctx);

/* Make the workspace large enough for batches of up to n_seq sequences and n_chunks chunks
 * (n_chunks < 2^32 - 1), so that later batch calls of that size allocate nothing. May
 * synchronise (it frees the old workspace). */
int lsmkv_reserve(lsmkv_ctx *ctx, uint64_t n_seq, uint64_t n_chunks);

/*
 * put_batch, device half (App. B "Put Batch"; Sec. 3.4 "Batch Codec Operations").
 * For request r with tokens[seq_off[r] .. seq_off[r+1]) and n_r = floor(len_r / C) chunks,
 * chunks j = start_r .. n_r-1 are encoded (start_r = start_chunk[r], or 0 when start_chunk is
 * NULL; the digest always covers the whole prefix from token 0). Encoded chunk number c of
 * request r has output index i = chunk_off[r] + c and produces
 *   keys_out[i]  the chunk key,
 *   vals_out[i]  {file_id, 0, base_offset + i*chunk_bytes},
 *   blob_out[i*chunk_bytes ..)  the 2L page slabs of each of the pool pages
 *                page_table[i*m .. i*m+m), page after page.
 *   tokens      [dev] u32, all sequences back to back
 *   seq_off     [dev] u64[n_req+1], ascending
 *   start_chunk [dev] u32[n_req] or NULL
 *   chunk_off   [dev] u64[n_req+1], exclusive prefix sums of max(0, n_r - start_r);
 *               chunk_off[n_req] must equal n_chunks (a mismatch sets LSMKV_ST_BAD_COUNT and
 *               the request is skipped)
 *   page_table  [dev] u32[n_chunks * m]; may be NULL together with pool and blob_out for an
 *               index-only encode (keys and records, no payload)
 *   blob_out    [dev], 16-byte aligned, blob_capacity >= n_chunks*chunk_bytes else
 *               LSMKV_ECAPACITY
 * Ordering (the paper's two-phase write, Sec. 3.2): keys, records and blobs of one call are
 * complete at the same point of the stream; publish the records only after that point.
 */
int lsmkv_encode_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_req, const uint32_t *tokens,
                       const uint64_t *seq_off, const uint32_t *start_chunk,
                       const uint64_t *chunk_off, uint64_t n_chunks, const uint32_t *page_table,
                       const lsmkv_pool_t *pool, uint32_t file_id, uint64_t base_offset,
                       lsmkv_key_t *keys_out, lsmkv_val_t *vals_out, void *blob_out,
                       uint64_t blob_capacity);

/*
 * probe + the index half of get_batch (App. B "Probe", "Get Batch"; Sec. 2.2 "Point Lookups").
 * For query q with n_q = floor(len_q / C) chunks, each chunk key is looked up in runs[0]
 * (newest) .. runs[n_runs-1] (oldest) and the first run that holds it decides.
 *   hit_chunks_out[q] = largest h <= n_q such that chunks 0..h-1 were all found,
 *   recs_out[qchunk_off[q] + j] = the record found for j < h, all-zero bytes for j >= h.
 *   runs       [host] array of n_runs <= LSMKV_MAX_RUNS descriptors (copied by the call)
 *   qchunk_off [dev] u64[n_query+1], exclusive prefix sums of n_q; n_qchunks = qchunk_off[n_query]
 *   keys_out   [dev] optional [n_qchunks]: every chunk key of every query (NULL to skip; the
 *              probe then stops hashing a query at its first miss)
 */
int lsmkv_probe_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_query, const uint32_t *tokens,
                      const uint64_t *seq_off, const uint64_t *qchunk_off, uint64_t n_qchunks,
                      const lsmkv_run_t *runs, uint32_t n_runs, uint32_t *hit_chunks_out,
                      lsmkv_val_t *recs_out, lsmkv_key_t *keys_out);

/*
 * get_batch, tensor half (App. B "Get Batch"; Sec. 3.4). For every query q and j < hit_chunks[q]
 * the blob at arenas[rec.file_id] + rec.offset (rec = recs[qchunk_off[q] + j]) is split into
 * its m*2L page slabs, which are written to pages dst_page_table[idx*m .. idx*m+m) of the pool
 * (idx = qchunk_off[q] + j; dst_page_table has m entries per query chunk).
 * No other byte of the pool changes. Destination pages must be distinct within the call.
 *   arenas      [host] array of n_arenas [dev] base pointers (16-byte aligned), indexed by file_id
 *   arena_bytes [host] size of each arena; records must satisfy offset + chunk_bytes <= size
 *               and offset % 16 == 0 (else LSMKV_ST_BAD_RECORD, chunk skipped)
 *   n_arenas    <= 64
 */
int lsmkv_decode_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_query,
                       const uint64_t *qchunk_off, uint64_t n_qchunks,
                       const uint32_t *hit_chunks, const lsmkv_val_t *recs,
                       const void *const *arenas, const uint64_t *arena_bytes,
                       uint32_t n_arenas, const uint32_t *dst_page_table,
                       const lsmkv_pool_t *pool);

/*
 * Flush: one sorted run out of a write batch (Sec. 2.2 "Updates": out-of-place writes are
 * buffered and flushed as a sorted run). keys/vals [dev] hold n entries in arrival order,
 * duplicates allowed; of equal keys the LAST arrival survives. Output [dev]: run_keys_out and
 * run_vals_out need room for n entries; entries [0, *n_out) are the run (ascending, unique),
 * entries [*n_out, n) are padding -- all-ones keys, which compare above every real key, with
 * zero records -- so the buffers may be used as a run of length n without reading *n_out back.
 * n_out [dev] receives the run length. Outputs must not overlap the inputs. n < 2^32 - 1.
 * Uses (and may grow) the context's sort scratch: 88 bytes per entry.
 */
int lsmkv_flush_batch(lsmkv_ctx *ctx, void *stream, const lsmkv_key_t *keys,
                      const lsmkv_val_t *vals, uint64_t n, lsmkv_key_t *run_keys_out,
                      lsmkv_val_t *run_vals_out, uint64_t *n_out);

/*
 * Compaction: several runs ([host] array, newest first, as for lsmkv_probe_batch) merged into
 * one: the union of their keys, each key with the record of the newest run that holds it
 * (Sec. 2.2: compaction merges runs and removes obsolete entries). keys_out / vals_out [dev]
 * need room for the sum of the run lengths and are padded like a flush; n_out [dev] receives
 * the merged length. Sum of lengths < 2^32 - 1. Outputs must not overlap the input runs.
 */
int lsmkv_merge_runs(lsmkv_ctx *ctx, void *stream, const lsmkv_run_t *runs, uint32_t n_runs,
                     lsmkv_key_t *keys_out, lsmkv_val_t *vals_out, uint64_t *n_out);

/*
 * Compaction policy (Sec. 2.2 "LSM-Tree Structure": levels whose capacities grow by a size ratio
 * T, at most K sorted runs per level; K = 1 is leveling, K = T - 1 tiering; Sec. 3.3 and App. C:
 * T and K change while the store runs and take effect lazily, as data is merged anyway). A pure
 * host function: it looks at the shape of the index and names the next merge, which the caller
 * carries out with lsmkv_merge_runs (or lsmkv_xrun_merge) and reports back by calling again.
 *   level, entries [host, n_runs]: the runs newest first; level[r] >= 1, non-decreasing in r (a
 *           flushed batch enters level 1); entries[r] = keys in run r
 *   buffer_entries = M, keys in one flushed batch; level i holds M * T^i keys
 *   size_ratio = T >= 2, runs_per_level = K >= 1
 * Starting from the shallowest level, the first level that needs work decides:
 *   - it holds M * T^i keys or more: all its runs are merged and the result moves to level
 *     i + 1; if level i + 1 already holds K runs they join the same merge (with K = 1 this is
 *     leveling's merge into the resident run);
 *   - else it holds more than K runs: they are merged into one run that stays at level i.
 * Returns 1 and fills *out (runs [first_run, first_run + n_runs) become one run of level
 * to_level, at position first_run of the list; n_runs == 1 is a move without a merge), 0 when
 * nothing is due, LSMKV_EINVAL for bad arguments. Because T and K come with every call, new
 * values apply from the next merge on and never force a reorganisation by themselves. With
 * K = T - 1, distinct keys and batches of M keys the run counts of the levels are the digits of
 * the number of flushes written in base T.
 */
typedef struct { uint32_t first_run, n_runs, to_level, reserved; } lsmkv_compaction_t;
int lsmkv_plan_compaction(const uint32_t *level, const uint64_t *entries, uint32_t n_runs,
                          uint64_t buffer_entries, uint32_t size_ratio, uint32_t runs_per_level,
                          lsmkv_compaction_t *out);

/*
 * Exact prefix index (Sec. 3.1/3.2: keys that keep the structure of token prefixes, so that key
 * order is prefix order). An "xrun" indexes WHOLE stored sequences by their tokens themselves:
 * no digest takes part, so two different prefixes can never be confused. The caller keeps, on
 * the device and alive while the xrun is in use: the token arena and offsets of the stored
 * sequences, and one record per whole chunk of every sequence, sequence-major (the records of
 * chunks a sequence shares with an earlier one are copies of that one's records -- what a probe
 * returned for them before the put). lsmkv_xrun_build writes the two index arrays:
 *   order_out     [dev] u32[n_seq]: sequence numbers in token-lexicographic order (a sequence
 *                 that is a prefix of another comes first; identical sequences by number)
 *   chunk_off_out [dev] u64[n_seq + 1]: prefix sums of floor(len_s / C), the row of sequence s
 *                 in the record array
 * n_seq < 2^32 - 1. Uses (and may grow) the context's sort scratch. A sequence with
 * seq_off[s + 1] < seq_off[s] sets LSMKV_ST_BAD_COUNT and counts as empty.
 */
typedef struct {
    const uint32_t *tokens;      /* [dev] arena of the stored sequences */
    const uint64_t *seq_off;     /* [dev] u64[n_seq + 1] */
    const lsmkv_val_t *vals;     /* [dev] records, 16-byte aligned: vals[chunk_off[s] + j] */
    const uint32_t *order;       /* [dev] from lsmkv_xrun_build */
    const uint64_t *chunk_off;   /* [dev] from lsmkv_xrun_build */
    uint32_t n_seq;
    uint32_t reserved;           /* 0 */
} lsmkv_xrun_t;

int lsmkv_xrun_build(lsmkv_ctx *ctx, void *stream, const uint32_t *tokens,
                     const uint64_t *seq_off, uint32_t n_seq, uint32_t *order_out,
                     uint64_t *chunk_off_out);

/*
 * Compaction of two xruns (Sec. 2.2 "Updates": runs are merged as the index grows). The caller
 * has laid run B's sequences behind run A's in ONE arena: tokens / seq_off describe n_a + n_b
 * sequences, A's first (the record arrays are concatenated the same way, B's rows behind A's).
 *   order_a [dev] u32[n_a]: A's sequences (numbers 0..n_a-1) in token order, from a build or merge
 *   order_b [dev] u32[n_b]: B's sequences in token order, numbered 0..n_b-1 within B as
 *           lsmkv_xrun_build returned them for B alone; the call adds n_a to every number
 *   order_out [dev] u32[n_a + n_b] and chunk_off_out [dev] u64[n_a + n_b + 1]: the index arrays of
 *           the merged run, equal to what lsmkv_xrun_build gives for the whole arena at the price
 *           of one merge step instead of a sort. order_out must not overlap the inputs.
 * A number outside its part sets LSMKV_ST_BAD_COUNT (that entry is replaced, the result is then
 * not a valid order). n_a + n_b < 2^32 - 1. Uses (and may grow) the context's sort scratch.
 */
int lsmkv_xrun_merge(lsmkv_ctx *ctx, void *stream, const uint32_t *tokens,
                     const uint64_t *seq_off, const uint32_t *order_a, uint32_t n_a,
                     const uint32_t *order_b, uint32_t n_b, uint32_t *order_out,
                     uint64_t *chunk_off_out);

/*
 * Probe of xruns ([host] array, newest first, n_runs <= LSMKV_MAX_RUNS; queries laid out as for
 * lsmkv_probe_batch). Per run, the whole chunks of the longest token prefix the query shares
 * with any stored sequence are present; hit_chunks_out[q] is the largest such count over the
 * runs, and chunk j takes its record from the newest run that reaches beyond j. Within a run
 * the records come from the query's neighbour in token order among the sequences sharing that
 * longest prefix: the largest one not above the query, else the smallest one above it.
 * recs_out [dev, n_qchunks entries, 16-byte aligned]: records of the hit chunks, zeros after.
 * Errors as lsmkv_probe_batch (LSMKV_ST_BAD_COUNT for a query whose counts disagree).
 */
int lsmkv_xprobe_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_query, const uint32_t *tokens,
                       const uint64_t *seq_off, const uint64_t *qchunk_off, uint64_t n_qchunks,
                       const lsmkv_xrun_t *runs, uint32_t n_runs, uint32_t *hit_chunks_out,
                       lsmkv_val_t *recs_out);

/*
 * Record relocation (Sec. 3.4 "Automatic Tensor File Merging": when tensor files are merged,
 * the file_id + offset values in the index are updated). Every record of vals [dev, n entries,
 * rewritten in place -- typically the vals array of a run] whose file_id equals table[t].old_file
 * gets file_id = table[t].new_file and offset += table[t].delta; the first matching entry
 * applies, other records are untouched. table [host], n_table <= 64. changed_out [dev,
 * optional] receives the number of records rewritten.
 */
typedef struct { uint32_t old_file, new_file; uint64_t delta; } lsmkv_reloc_t;
int lsmkv_relocate_records(lsmkv_ctx *ctx, void *stream, lsmkv_val_t *vals, uint64_t n,
                           const lsmkv_reloc_t *table, uint32_t n_table, uint64_t *changed_out);

/*
 * Compressing codec LSMKV_CODEC_XP12 (Sec. 3.4 "Batch Codec Operations": combined tensors are
 * compressed before storage and decompressed together on load; the paper names no algorithm,
 * this one is lossless so restored pages stay bit-exact). Selected per context through
 * lsmkv_geom_t.flags; needs elem_bytes == 2. It changes only blobs and records:
 *   slab of N 16-bit elements v = s<<15 | e<<7 | m:  base = max(0, e_max - 14);
 *     16-byte header {u32 0x32315058, u32 n_exc, u8 base, u8 mode, u16 0, u32 size}
 *     mode 0: N bytes (s<<7 | m), N/2 bytes of 4-bit codes (e - base, 15 = below the window;
 *             element i in byte i/2, even i in the low nibble), n_exc raw exponent bytes of the
 *             code-15 elements in element order, zero padding to a multiple of 16
 *     mode 1 (n_exc >= N/2): the 2N raw bytes
 *   chunk blob: directory of m*2L+1 u32 (byte offset of every slab, then the blob size; padded
 *     to 16 bytes) followed by the slabs in blob order (page by page, K0 V0 K1 V1 ...)
 *   records: {file_id, reserved = blob size, offset}; blobs are placed back to back, so
 *     offset = base_offset + sum of the sizes of the chunks before it. Data-dependent: size
 *     blob_out with lsmkv_encode_bound(); the bytes used are the last record's offset + size
 *     - base_offset. A chunk that does not fit blob_capacity sets LSMKV_ST_OVERFLOW and gets
 *     an all-zero-size record.
 *   Encoding reads the pool once when blob_capacity >= lsmkv_encode_bound(n_chunks) and the slab
 *   has 8192 or 16384 elements (see "xp_one_pass" below), twice otherwise; the bytes are the same.
 *   The encoder's scratch (12 bytes per slab) belongs to the context and grows with the batch.
 * lsmkv_decode_batch validates every directory entry and slab header (LSMKV_ST_BAD_RECORD).
 * lsmkv_decode_batch_static supports the identity codec only.
 */
uint64_t lsmkv_encode_bound(const lsmkv_ctx *ctx, uint64_t n_chunks); /* worst-case blob bytes */

/*
 * Bloom filter of a run (Sec. 2.2 "Point Lookups", App. B "Probe": filters rule out runs that
 * cannot hold a key). Result-neutral: probes return the same answers with or without it.
 * Format: blocks of 256 bits; lsmkv_bloom_blocks(n) = max(1, ceil(10 n / 256)) blocks for n keys;
 * a key goes to block floor(w1 * n_blocks / 2^61) and sets the six bits at positions
 * (w2 >> 8i) & 255, i = 0..5 (position p = bit p&7 of byte p>>3 of the block). Entries whose
 * w1 is not a digest (the all-ones padding of a flushed run) are ignored.
 * lsmkv_bloom_build: keys [dev, n entries] -> bloom_out [dev, 32 * lsmkv_bloom_blocks(n) bytes,
 * 16-byte aligned], cleared and filled on `stream`.
 */
uint64_t lsmkv_bloom_blocks(uint64_t n);
int lsmkv_bloom_build(lsmkv_ctx *ctx, void *stream, const lsmkv_key_t *keys, uint64_t n,
                      void *bloom_out);

/*
 * Hash index of a run (Sec. 2.2 "Point Lookups": a run carries auxiliary structures -- fence
 * pointers, filters -- built once when the run is written, so that a point lookup touches as
 * little of the run as possible; this one plays both parts for runs that live in device memory).
 * Result-neutral: probes return the same answers with or without it.
 * Format: lsmkv_hindex_buckets(n) = max(1, ceil(n / 2)) buckets of eight u32 slots. A slot is 0
 * (empty) or (w2 & 0xFF) << 24 | (i + 1) for the key at position i of the run. A key's home
 * bucket is floor(w1 * n_buckets / 2^61); it occupies the first slot that was free at its
 * insertion, scanning from slot 0 of the home bucket through the following buckets (wrapping
 * around). Lookups scan in the same order and stop at the first empty slot. Which of several
 * keys of one bucket got which slot depends on the order of insertion and is not specified.
 * Entries whose w1 is not a digest (the all-ones padding of a flushed run) are left out.
 * n <= 2^24 - 2 (LSMKV_EINVAL beyond; such a run is probed without a hash index).
 * lsmkv_hindex_build: keys [dev, n entries] -> hindex_out [dev, 32 * lsmkv_hindex_buckets(n)
 * bytes, 16-byte aligned], cleared and filled on `stream`.
 */
uint64_t lsmkv_hindex_buckets(uint64_t n);
int lsmkv_hindex_build(lsmkv_ctx *ctx, void *stream, const lsmkv_key_t *keys, uint64_t n,
                       void *hindex_out);

/*
 * Host-buffer variants (the form the paper's service interface has: token sequences and
 * tensors handed over by the serving process, App. B). Same results as the device-buffer
 * calls; every pointer except `pool` and `runs[].keys/vals` is a HOST pointer (use pinned
 * memory for full transfer speed; pageable memory works). The calls stage through device
 * scratch owned by the context (grown on demand, bounded by twice the "host_stage_bytes" knob
 * plus the descriptors; default 1 GiB of blobs per slice), enqueue all copies and kernels on
 * `stream` -- the blobs of a put with the compressing codec and of a get with several slices on
 * a second stream of the context's own, from or into two stages in turn, so that one slice
 * travels while its neighbour is packed or scattered; that stream starts behind `stream` and
 * `stream` waits for it, the caller sees one stream -- and return; host outputs are valid, and host inputs may be reused, once the stream
 * has reached the end of the call's work. Offsets (chunk_off / qchunk_off) are computed by
 * the library from the sequence lengths.
 *
 * lsmkv_put_batch_host: put_batch. keys_out / vals_out / blob_out [host] receive what
 *   lsmkv_encode_batch produces; *n_chunks_out (optional) is set before returning. blob_out
 *   may be NULL together with page_table and pool (index-only). *blob_bytes_out (optional) =
 *   bytes placed in blob_out. With the compressing codec blob sizes depend on the data: the
 *   call then waits, once per slice, for that slice's records (a short wait: only the slice's
 *   encode is ahead of it; the slice before is meanwhile on its way to the host on a stream of
 *   the context's own, from the other of two stages), copies exactly the bytes produced behind
 *   those of the slices before, sets *blob_bytes_out and returns LSMKV_ECAPACITY if blob_out is
 *   too small; the caller's stream reaches the end of the call's work only when those copies
 *   have landed. With the knob "host_put_device_placed", pinned 16-byte aligned blob_out and
 *   blob_bytes_out == NULL the call never waits instead: kernels place every slice's bytes in
 *   blob_out themselves (at about four fifths of the copy engines' rate); the bytes used are
 *   then the last record's offset + size - base_offset, and a blob_out that is too small sets
 *   LSMKV_ST_OVERFLOW (the slice is left out) instead of an error code. With the identity codec
 *   the call never waits.
 * lsmkv_probe_batch_host: probe. hit_chunks_out [host n_query], recs_out [host, sum of
 *   floor(len/C)], optional keys_out; *n_qchunks_out (optional) is set before returning.
 * lsmkv_decode_batch_host: get_batch, tensor half. qchunk_off, hit_chunks, recs and
 *   dst_page_table are host arrays (typically what lsmkv_probe_batch_host returned, after a
 *   stream synchronisation); `arenas` are HOST base pointers of the tensor-log buffers indexed
 *   by file_id. The blobs of the hit chunks are copied to the device slice by slice (blobs
 *   adjacent in an arena travel as one copy) and scattered into the pool. Records are checked
 *   on the host first: LSMKV_EINVAL and nothing enqueued if one points outside its arena.
 */
int lsmkv_put_batch_host(lsmkv_ctx *ctx, void *stream, uint32_t n_req, const uint32_t *tokens,
                         const uint64_t *seq_off, const uint32_t *start_chunk,
                         const uint32_t *page_table, const lsmkv_pool_t *pool, uint32_t file_id,
                         uint64_t base_offset, lsmkv_key_t *keys_out, lsmkv_val_t *vals_out,
                         void *blob_out, uint64_t blob_capacity, uint64_t *n_chunks_out,
                         uint64_t *blob_bytes_out);
int lsmkv_probe_batch_host(lsmkv_ctx *ctx, void *stream, uint32_t n_query,
                           const uint32_t *tokens, const uint64_t *seq_off,
                           const lsmkv_run_t *runs, uint32_t n_runs, uint32_t *hit_chunks_out,
                           lsmkv_val_t *recs_out, lsmkv_key_t *keys_out,
                           uint64_t *n_qchunks_out);
int lsmkv_decode_batch_host(lsmkv_ctx *ctx, void *stream, uint32_t n_query,
                            const uint64_t *qchunk_off, const uint32_t *hit_chunks,
                            const lsmkv_val_t *recs, const void *const *arenas,
                            const uint64_t *arena_bytes, uint32_t n_arenas,
                            const uint32_t *dst_page_table, const lsmkv_pool_t *pool);

/*
 * Allocation-free decode (an addition of this library; the paper has no counterpart).
 *
 * Same result as lsmkv_decode_batch(), for callers that are not allowed to allocate device
 * memory at all -- typically a plugin inside a serving process whose engine has claimed the
 * whole of HBM for its own pools at start-up and forbids driver allocations afterwards, where
 * a cudaMalloc can fail outright or stall every stream of the process while it runs. Such a
 * caller cannot even create an lsmkv_ctx (lsmkv_create allocates), so this call takes the
 * geometry and the device instead of a context and makes no cudaMalloc, cudaFree or other
 * allocating call.
 *
 * The scratch the decode needs (prefix sums of the hit lengths, the list of chunks to copy, a
 * status block) lives in a fixed array inside the library image, about 1.03 MiB per GPU that
 * loads the library, held until the process exits. Consequences:
 *   - limits: n_query <= LSMKV_STATIC_MAX_QUERIES and n_qchunks <= LSMKV_STATIC_MAX_CHUNKS;
 *     anything larger returns LSMKV_ETOOBIG and enqueues nothing (split the batch);
 *   - every call on a device uses the same array. The call resets what has to start from zero
 *     (the status block); the rest is rewritten before it is read, so stale contents of an
 *     earlier call never show. Two calls that overlap on the GPU (different streams without an
 *     ordering between them) race on the array and give undefined results: serialise them;
 *   - the first call on each device looks up the device address of the array (one-time
 *     set-up, done with that device current). Make that first call before any stream capture
 *     is started.
 * Arguments as for lsmkv_decode_batch(), plus
 *   geom, device   what lsmkv_create() would have been given
 *   status_out     [dev] optional: receives the status block of this call (flags, first_bad,
 *                  chunks_decoded) at the end of the enqueued work
 * Launch shape is fixed (bulk-async copies, 32 KiB pieces); tuning knobs do not apply.
 */
#define LSMKV_STATIC_MAX_QUERIES 4096u
#define LSMKV_STATIC_MAX_CHUNKS 262144u
int lsmkv_decode_batch_static(const lsmkv_geom_t *geom, int device, void *stream,
                              uint32_t n_query, const uint64_t *qchunk_off, uint64_t n_qchunks,
                              const uint32_t *hit_chunks, const lsmkv_val_t *recs,
                              const void *const *arenas, const uint64_t *arena_bytes,
                              uint32_t n_arenas, const uint32_t *dst_page_table,
                              const lsmkv_pool_t *pool, lsmkv_status_t *status_out);

/* Synchronise `stream`, copy the device status block to *out [host] and clear it. */
int lsmkv_last_status(lsmkv_ctx *ctx, void *stream, lsmkv_status_t *out);

/*
 * Optional per-kernel timing. While enabled, every kernel launch of this context is bracketed
 * by CUDA events on the launching stream (no synchronisation). lsmkv_profile_read() waits for
 * the recorded events, returns the summed device time and launch count per kernel class since
 * the previous read, and clears them. Class LSMKV_K_PLAN covers the two small kernels that
 * turn hit lengths into the list of chunks to copy.
 * Independently of that switch the launches of every call of a context sit inside an NVTX
 * range named after their class ("lsmkv:keys", "lsmkv:pack", "lsmkv:probe", "lsmkv:plan",
 * "lsmkv:unpack", "lsmkv:flush", "lsmkv:merge"): a timeline tool that collects NVTX shows
 * them, without such a tool the ranges do nothing. lsmkv_decode_batch_static opens none.
 */
#define LSMKV_K_KEYS 0
#define LSMKV_K_PACK 1
#define LSMKV_K_PROBE 2
#define LSMKV_K_PLAN 3
#define LSMKV_K_UNPACK 4
#define LSMKV_K_FLUSH 5
#define LSMKV_K_MERGE 6
#define LSMKV_K_CLASSES 8
typedef struct {
    double ms[LSMKV_K_CLASSES];
    uint64_t launches[LSMKV_K_CLASSES];
} lsmkv_profile_t;
int lsmkv_profile_enable(lsmkv_ctx *ctx, int on);
int lsmkv_profile_read(lsmkv_ctx *ctx, lsmkv_profile_t *out /* [host] */);

/* The cudaError_t behind the last LSMKV_ECUDA of this context (0 if none). */
int lsmkv_last_cuda_error(const lsmkv_ctx *ctx);

/* Source line (in the library's own files) of the CUDA call behind that error, 0 if unknown. */
int lsmkv_last_cuda_line(const lsmkv_ctx *ctx);

/* Number of kernels this context has launched so far (for launch accounting). */
uint64_t lsmkv_launch_count(const lsmkv_ctx *ctx);

/*
 * Tuning knobs (launch shapes only; results never depend on them). Returns LSMKV_EINVAL for an
 * unknown name or a value outside its documented range.
 *   "copy_mode"         0 = bulk-async copy engine (cp.async.bulk), 1 = 16-byte vector loads/stores
 *   "copy_stage_bytes"  bytes per bulk copy, multiple of 16, 16..131072 (clamped to page_bytes)
 *   "copy_stages"       bulk copies in flight per CTA, 1..32 (reduced to fit shared memory)
 *   "copy_ctas_per_sm"  1..8        "copy_l2_hint"  0/1 = evict-first L2 policy on the copies
 *   "simt_ctas_per_sm"  1..32       "probe_warps_per_cta"  1..8
 *   "host_stage_bytes"  blob bytes staged per slice by the host-buffer calls, 1 MiB..64 GiB
 *   "xp_generic"        1 = compressing codec always uses its generic kernels (0 = fast kernels
 *                       for slabs of 8192 / 16384 / 32768 elements)
 *   "xp_one_pass"       1 (default) = the compressing codec encodes slabs of 8192 / 16384 elements
 *                       in one pass over the pool whenever blob_capacity >= lsmkv_encode_bound()
 *                       (a persistent pipeline per SM; same bytes out); 0 = always three steps
 *   "host_put_device_placed"  1 = lsmkv_put_batch_host with the compressing codec never waits
 *                       (see there); "host_copy_ctas" = CTAs of the kernel that then writes the
 *                       host blob, 1..4096 (default 32: posted writes need little parallelism)
 *   "host_copy_piece_bytes"  the host-buffer calls move blobs in copies of at most this many
 *                       bytes, 1 MiB..64 GiB (default 128 MiB). Copies of one direction are served
 *                       in issue order even across streams, so a smaller piece lets another
 *                       stream's small copies in sooner and a larger one loses less at the piece
 *                       boundaries (end to end, put and get side by side: 87 GB/s with 32 MiB,
 *                       89 GB/s with 128 MiB on the same box)
 *   "test_drop_piece"   test hook, -1 = off (default): the bulk copy kernel arms the completion
 *                       barrier of the piece with this number (pieces are numbered over the
 *                       whole launch) but starts no copy for it, so that wait runs out: the
 *                       kernel records LSMKV_ST_WAIT_EXPIRED with first_bad = the piece and
 *                       returns; the warp that owned the piece copies nothing further. The
 *                       one-pass encoder of the compressing codec does the same with the fetch of
 *                       the slab of this number (slabs numbered over the whole batch): the wait
 *                       for it runs out, every role of every CTA leaves through its bounded
 *                       waits, and the records of chunks that were not finished are zeroed
 *   "wait_cycles"       limit, in GPU clock cycles, of every bounded wait inside a kernel (the bulk
 *                       copies' completion, the one-pass encoder's hand-offs); default 2e9, about
 *                       a second; 1e5..1e11. A wait that runs out sets LSMKV_ST_WAIT_EXPIRED
 */
int lsmkv_set_tuning(lsmkv_ctx *ctx, const char *name, int64_t value);
int64_t lsmkv_get_tuning(const lsmkv_ctx *ctx, const char *name);

/* Static text for a return code. */
const char *lsmkv_strerror(int code);

/* LSMKV_FORMAT_VERSION the library was built with. */
int lsmkv_format_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LSMKV_H */
