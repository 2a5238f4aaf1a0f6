/*
 * lsmkv_oracle.c -- plain, slow, single-threaded CPU statement of the batch codec and the
 * batched longest-cached-prefix probe of an LSM-backed KV-cache store.
 *
 * THIS IS TEST INFRASTRUCTURE. It exists so that the CUDA library can be checked against
 * something obviously correct. It shares no code, header, table or constant generator with
 * the CUDA library, is never linked into it, and must not be used as a product path.
 *
 * What it follows (paper section names; the paper fixes properties, this build fixes formats):
 *   - Sec. 3.2 "Prefix-Preserving Storage Engine": the index maps a key that encodes a token
 *     prefix to a compact record holding a file identifier and a byte offset; tensors live in
 *     an append-only log (key-value separation).
 *   - Sec. 3.4 "Batch Codec Operations": a batch's tensors are combined into one contiguous
 *     payload on put and split again on get (identity codec here: a bit copy).
 *   - App. B "Basic Operations": put_batch (keys + file_id/offset records + contiguous
 *     tensors), probe (longest cached prefix by point lookups), get_batch (locations, then
 *     batch tensor loading).
 *   - Sec. 2.2 "Point Lookups": levels are checked in order and the first match is returned.
 *
 * Formats (this build's reading; the paper is silent on all of them):
 *   key     = 4 x u64 {w0,w1,w2,w3}, compared lexicographically as unsigned words
 *             w0 = (namespace << 32) | chunk index j
 *             w1 = digest A of the token prefix S[0 : (j+1)*C)
 *             w2 = digest B of the same prefix
 *             w3 = (first token of chunk j << 32) | last token of chunk j
 *   digest  = h <- 0; for every token t in order: h <- (h * BASE + (t + 1)) mod (2^61 - 1),
 *             always the canonical representative in [0, 2^61 - 1)
 *   record  = {u32 file_id, u32 reserved = 0, u64 offset}, offset = base + i * chunk_bytes
 *   blob    = for every page of the chunk, in token order: for l in 0..L-1: K page slab of
 *             layer l, then V page slab of layer l (chunk_tokens = m * page_tokens, m >= 1)
 *   pool    = 2L buffers (K of layers 0..L-1, then V of layers 0..L-1), each
 *             [num_pages][page_tokens][kv_heads][head_dim] elements, page slab contiguous
 *
 * Every function reports an error by return value; nothing here aborts.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_EINVAL (-1)
#define ORC_ECAPACITY (-2)
#define ORC_EBADPAGE (-3)
#define ORC_EBADREC (-4)

static const uint64_t ORC_P = 0x1FFFFFFFFFFFFFFFULL; /* 2^61 - 1 */
static const uint64_t ORC_BASE[2] = {0x0B4E0EF37BC32127ULL, 0x16A09E667F3BCC90ULL};

typedef struct { uint64_t w[4]; } orc_key;
typedef struct { uint32_t file_id, reserved; uint64_t offset; } orc_val;
typedef struct {
    uint32_t n_layers, n_kv_heads, head_dim, elem_bytes;
    uint32_t page_tokens, chunk_tokens, ns, flags;
} orc_geom;
typedef struct { const orc_key *keys; const orc_val *vals; uint64_t n; } orc_run;

/* ---- geometry ---------------------------------------------------------------------- */

uint64_t orc_page_bytes(const orc_geom *g)
{
    return (uint64_t)g->page_tokens * g->n_kv_heads * g->head_dim * g->elem_bytes;
}

/* A chunk covers m = chunk_tokens / page_tokens whole pages (m = 1: a chunk is a page). Its
 * blob is the m page blobs one after the other, each K0 V0 K1 V1 ...; page tables carry m
 * entries per chunk, entry i*m + k for the k-th page of chunk i. */
static uint64_t pages_per_chunk(const orc_geom *g)
{
    return g->chunk_tokens / g->page_tokens;
}

uint64_t orc_chunk_bytes(const orc_geom *g)
{
    return pages_per_chunk(g) * 2ull * g->n_layers * orc_page_bytes(g);
}

static int geom_ok(const orc_geom *g)
{
    return g && g->n_layers && g->n_kv_heads && g->head_dim && g->elem_bytes &&
           g->page_tokens && g->chunk_tokens && g->chunk_tokens % g->page_tokens == 0;
}

/* ---- digest: one Horner step of the polynomial hash over the Mersenne prime 2^61-1 -- */

uint64_t orc_digest_step(uint64_t h, uint32_t token, int lane)
{
    unsigned __int128 x = (unsigned __int128)h * ORC_BASE[lane] + ((uint64_t)token + 1ull);
    return (uint64_t)(x % ORC_P);
}

/* digest of a whole token string (used by the pins) */
uint64_t orc_digest(const uint32_t *tokens, uint64_t n, int lane)
{
    uint64_t h = 0;
    for (uint64_t i = 0; i < n; ++i) h = orc_digest_step(h, tokens[i], lane);
    return h;
}

/* ---- keys -------------------------------------------------------------------------- */

int orc_key_cmp(const orc_key *a, const orc_key *b)
{
    for (int i = 0; i < 4; ++i) {
        if (a->w[i] < b->w[i]) return -1;
        if (a->w[i] > b->w[i]) return 1;
    }
    return 0;
}

/*
 * Keys of chunks j = j_begin .. floor(len / C) - 1 of one sequence, written to keys_out in
 * ascending j. The digest always runs from token 0: a key names the whole prefix, also when
 * earlier chunks are not emitted. Returns the number of keys written.
 */
uint64_t orc_chunk_keys(const orc_geom *g, const uint32_t *tokens, uint64_t len,
                        uint64_t j_begin, orc_key *keys_out)
{
    const uint64_t C = g->chunk_tokens;
    const uint64_t nch = len / C;
    uint64_t hA = 0, hB = 0, written = 0;
    for (uint64_t j = 0; j < nch; ++j) {
        for (uint64_t i = 0; i < C; ++i) {
            const uint32_t t = tokens[j * C + i];
            hA = orc_digest_step(hA, t, 0);
            hB = orc_digest_step(hB, t, 1);
        }
        if (j >= j_begin) {
            orc_key *k = &keys_out[written++];
            k->w[0] = ((uint64_t)g->ns << 32) | (uint64_t)(uint32_t)j;
            k->w[1] = hA;
            k->w[2] = hB;
            k->w[3] = ((uint64_t)tokens[j * C] << 32) | (uint64_t)tokens[j * C + C - 1];
        }
    }
    return written;
}

/* ---- put_batch, device half: keys + records + packed blobs -------------------------- */

/*
 * kv_ptrs: 2L host pointers, K of layer 0..L-1 then V of layer 0..L-1.
 * blob_out may be NULL (index-only encode: keys and records, no payload).
 */
int orc_encode_batch(const orc_geom *g, uint32_t n_req, const uint32_t *tokens,
                     const uint64_t *seq_off, const uint32_t *start_chunk,
                     const uint64_t *chunk_off, uint64_t n_chunks, const uint32_t *page_table,
                     const uint8_t *const *kv_ptrs, uint64_t num_pages, uint32_t file_id,
                     uint64_t base_offset, orc_key *keys_out, orc_val *vals_out,
                     uint8_t *blob_out, uint64_t blob_capacity)
{
    if (!geom_ok(g)) return ORC_EINVAL;
    const uint64_t C = g->chunk_tokens, L = g->n_layers, m = pages_per_chunk(g);
    const uint64_t pb = orc_page_bytes(g), cb = orc_chunk_bytes(g);
    if (blob_out && blob_capacity < n_chunks * cb) return ORC_ECAPACITY;
    if (n_req && chunk_off[n_req] != n_chunks) return ORC_EINVAL;

    for (uint32_t r = 0; r < n_req; ++r) {
        const uint64_t len = seq_off[r + 1] - seq_off[r];
        const uint64_t nch = len / C;
        const uint64_t start = start_chunk ? start_chunk[r] : 0;
        const uint64_t cnt = nch > start ? nch - start : 0;
        if (chunk_off[r + 1] - chunk_off[r] != cnt) return ORC_EINVAL;
        if (cnt == 0) continue;
        const uint64_t i0 = chunk_off[r];
        if (orc_chunk_keys(g, tokens + seq_off[r], len, start, keys_out + i0) != cnt)
            return ORC_EINVAL;
        for (uint64_t c = 0; c < cnt; ++c) {
            const uint64_t i = i0 + c;
            vals_out[i].file_id = file_id;
            vals_out[i].reserved = 0;
            vals_out[i].offset = base_offset + i * cb;
            if (!blob_out) continue;
            for (uint64_t k = 0; k < m; ++k) {           /* the chunk's pages, in token order */
                const uint64_t page = page_table[i * m + k];
                if (page >= num_pages) return ORC_EBADPAGE;
                uint8_t *dst = blob_out + i * cb + k * 2 * L * pb;
                for (uint64_t l = 0; l < L; ++l) {
                    memcpy(dst + (2 * l) * pb, kv_ptrs[l] + page * pb, pb);         /* K, layer l */
                    memcpy(dst + (2 * l + 1) * pb, kv_ptrs[L + l] + page * pb, pb); /* V, layer l */
                }
            }
        }
    }
    return ORC_OK;
}

/* ---- the index: immutable sorted runs, newest first --------------------------------- */

/* first position in run whose key is >= key (plain binary search on a sorted array) */
static uint64_t run_lower_bound(const orc_run *run, const orc_key *key)
{
    uint64_t lo = 0, hi = run->n;
    while (lo < hi) {
        const uint64_t mid = lo + (hi - lo) / 2;
        if (orc_key_cmp(&run->keys[mid], key) < 0) lo = mid + 1; else hi = mid;
    }
    return lo;
}

/*
 * Point lookup: runs are checked from newest (index 0) to oldest and the first run that holds
 * the key decides. Returns 1 and fills *val on a hit, 0 on a miss. *run_idx (optional) gets
 * the deciding run.
 */
int orc_lookup(const orc_run *runs, uint32_t n_runs, const orc_key *key, orc_val *val,
               uint32_t *run_idx)
{
    for (uint32_t r = 0; r < n_runs; ++r) {
        const uint64_t pos = run_lower_bound(&runs[r], key);
        if (pos < runs[r].n && orc_key_cmp(&runs[r].keys[pos], key) == 0) {
            if (val) *val = runs[r].vals[pos];
            if (run_idx) *run_idx = r;
            return 1;
        }
    }
    return 0;
}

/*
 * Flush: turn a write batch (keys in arrival order, duplicates allowed) into one sorted run
 * with unique keys; of equal keys the LAST arrival survives (out-of-place update semantics).
 * Returns the run length. keys_out/vals_out need room for n entries.
 */
typedef struct { orc_key k; orc_val v; uint64_t seq; } flush_ent;

static int flush_cmp(const void *a, const void *b)
{
    const flush_ent *x = (const flush_ent *)a, *y = (const flush_ent *)b;
    const int c = orc_key_cmp(&x->k, &y->k);
    if (c) return c;
    return (x->seq < y->seq) ? -1 : (x->seq > y->seq);
}

int64_t orc_flush(const orc_key *keys, const orc_val *vals, uint64_t n, orc_key *keys_out,
                  orc_val *vals_out)
{
    if (n == 0) return 0;
    flush_ent *e = (flush_ent *)malloc(n * sizeof(flush_ent));
    if (!e) return ORC_ECAPACITY;
    for (uint64_t i = 0; i < n; ++i) { e[i].k = keys[i]; e[i].v = vals[i]; e[i].seq = i; }
    qsort(e, n, sizeof(flush_ent), flush_cmp);
    uint64_t m = 0;
    for (uint64_t i = 0; i < n; ++i) {
        /* equal keys are adjacent and ordered by arrival: keep the last of each group */
        if (i + 1 < n && orc_key_cmp(&e[i].k, &e[i + 1].k) == 0) continue;
        keys_out[m] = e[i].k;
        vals_out[m] = e[i].v;
        ++m;
    }
    free(e);
    return (int64_t)m;
}

/*
 * Compaction of several runs (newest first) into one: the union of their keys, each key with
 * the record of the newest run that holds it. Written as "concatenate oldest..newest, then
 * flush", which is the definition of newest-wins. Returns the merged length.
 */
int64_t orc_merge_runs(const orc_run *runs, uint32_t n_runs, orc_key *keys_out,
                       orc_val *vals_out)
{
    uint64_t total = 0;
    for (uint32_t r = 0; r < n_runs; ++r) total += runs[r].n;
    if (total == 0) return 0;
    orc_key *k = (orc_key *)malloc(total * sizeof(orc_key));
    orc_val *v = (orc_val *)malloc(total * sizeof(orc_val));
    if (!k || !v) { free(k); free(v); return ORC_ECAPACITY; }
    uint64_t at = 0;
    for (uint32_t r = n_runs; r-- > 0;) { /* oldest first, so the newest arrives last */
        memcpy(k + at, runs[r].keys, runs[r].n * sizeof(orc_key));
        memcpy(v + at, runs[r].vals, runs[r].n * sizeof(orc_val));
        at += runs[r].n;
    }
    const int64_t m = orc_flush(k, v, total, keys_out, vals_out);
    free(k);
    free(v);
    return m;
}

/* ---- Bloom filter of a run (Sec. 2.2 "Point Lookups", App. B "Probe": filters let a lookup skip
 * runs that cannot hold the key). Result-neutral: a filter may say "maybe" for an absent key but
 * never "no" for a present one.
 *
 * Format (this build's): blocked filter, blocks of 256 bits (32 bytes), 10 bits per key:
 *   n_blocks = max(1, ceil(10 * n / 256));   block(key) = floor(w1 * n_blocks / 2^61)
 *   six bits per key inside its block, at positions (w2 >> 8i) & 255 for i = 0..5;
 *   position p is bit (p & 7) of byte (p >> 3) of the block.
 */
uint64_t orc_bloom_blocks(uint64_t n)
{
    const uint64_t b = (10 * n + 255) / 256;
    return b ? b : 1;
}

static uint64_t bloom_block_of(const orc_key *k, uint64_t n_blocks)
{
    return (uint64_t)(((unsigned __int128)k->w[1] * n_blocks) >> 61);
}

void orc_bloom_build(const orc_key *keys, uint64_t n, uint8_t *bloom /* 32 * orc_bloom_blocks(n) */)
{
    const uint64_t nb = orc_bloom_blocks(n);
    memset(bloom, 0, nb * 32);
    for (uint64_t i = 0; i < n; ++i) {
        uint8_t *blk = bloom + 32 * bloom_block_of(&keys[i], nb);
        for (int t = 0; t < 6; ++t) {
            const unsigned p = (unsigned)((keys[i].w[2] >> (8 * t)) & 255u);
            blk[p >> 3] |= (uint8_t)(1u << (p & 7u));
        }
    }
}

int orc_bloom_may_contain(const uint8_t *bloom, uint64_t n_blocks, const orc_key *key)
{
    const uint8_t *blk = bloom + 32 * bloom_block_of(key, n_blocks);
    for (int t = 0; t < 6; ++t) {
        const unsigned p = (unsigned)((key->w[2] >> (8 * t)) & 255u);
        if (!(blk[p >> 3] & (1u << (p & 7u)))) return 0;
    }
    return 1;
}

/* ---- hash index of a run -------------------------------------------------------------- */

/*
 * Sec. 2.2 "Point Lookups": a run carries auxiliary structures, built when the run is written,
 * that let a point lookup touch as little of the run as possible. For runs held in memory a
 * hash table over the run's keys does that: it answers "where in the run is this key, if
 * anywhere" without a search. Results of lookups never depend on it.
 *
 * Format (this build's): n_buckets = max(1, ceil(n / 2)) buckets of eight u32 slots.
 *   slot = 0 (empty) or (w2 & 0xFF) << 24 | (i + 1) for the key at position i of the run;
 *   home bucket of a key = floor(w1 * n_buckets / 2^61);
 *   a key takes the first empty slot found scanning slot 0..7 of its home bucket, then of the
 *   following buckets, wrapping around; a lookup scans the same way, compares the full key
 *   wherever the 8-bit tag matches, and stops at the first empty slot.
 * Keys whose w1 is not a digest (>= 2^61: the padding of a flushed run) are left out.
 * Inserting in a different order gives a different, equally valid table; this builder inserts
 * by ascending position. n <= 2^24 - 2.
 */
uint64_t orc_hindex_buckets(uint64_t n)
{
    const uint64_t b = n / 2 + (n & 1);
    return b ? b : 1;
}

static uint64_t hindex_home(const orc_key *k, uint64_t n_buckets)
{
    return (uint64_t)(((unsigned __int128)k->w[1] * n_buckets) >> 61);
}

int orc_hindex_build(const orc_key *keys, uint64_t n, uint32_t *table /* 8 * orc_hindex_buckets(n) */)
{
    if (n > (1ull << 24) - 2) return ORC_EINVAL;
    const uint64_t nb = orc_hindex_buckets(n), slots = 8 * nb;
    memset(table, 0, slots * sizeof(uint32_t));
    for (uint64_t i = 0; i < n; ++i) {
        if (keys[i].w[1] >> 61) continue;
        uint64_t s = 8 * hindex_home(&keys[i], nb);
        while (table[s]) s = s + 1 == slots ? 0 : s + 1;      /* at most n of >= 4n slots are taken */
        table[s] = (uint32_t)((keys[i].w[2] & 0xFFu) << 24) | (uint32_t)(i + 1);
    }
    return ORC_OK;
}

/* position of `key` in the run according to the table, or UINT64_MAX */
uint64_t orc_hindex_find(const uint32_t *table, uint64_t n_buckets, const orc_key *keys,
                         uint64_t n, const orc_key *key)
{
    const uint64_t slots = 8 * n_buckets;
    const uint32_t tag = (uint32_t)(key->w[2] & 0xFFu);
    uint64_t s = 8 * hindex_home(key, n_buckets);
    for (uint64_t seen = 0; seen < slots; ++seen) {
        const uint32_t w = table[s];
        if (w == 0) return UINT64_MAX;
        const uint64_t at = (uint64_t)(w & 0xFFFFFFu) - 1;
        if ((w >> 24) == tag && at < n && memcmp(&keys[at], key, sizeof(orc_key)) == 0) return at;
        s = s + 1 == slots ? 0 : s + 1;
    }
    return UINT64_MAX;
}

/* ---- probe: longest cached prefix, first-miss rule ---------------------------------- */

/*
 * For query q with n_q = floor(len_q / C) chunks: hit_q = the largest h <= n_q such that the
 * key of every chunk j < h is found by orc_lookup. recs_out[qchunk_off[q] + j] = the record
 * found for j < hit_q and all-zero for j >= hit_q. keys_out (optional) receives every chunk
 * key of every query. lookups_out (optional) counts point lookups performed.
 */
int orc_probe_batch(const orc_geom *g, uint32_t n_query, const uint32_t *tokens,
                    const uint64_t *seq_off, const uint64_t *qchunk_off, const orc_run *runs,
                    uint32_t n_runs, uint32_t *hit_out, orc_val *recs_out, orc_key *keys_out,
                    uint64_t *lookups_out)
{
    if (!geom_ok(g)) return ORC_EINVAL;
    const uint64_t C = g->chunk_tokens;
    uint64_t lookups = 0;
    for (uint32_t q = 0; q < n_query; ++q) {
        const uint64_t len = seq_off[q + 1] - seq_off[q];
        const uint64_t nch = len / C;
        if (qchunk_off[q + 1] - qchunk_off[q] != nch) return ORC_EINVAL;
        orc_key *keys = keys_out ? keys_out + qchunk_off[q]
                                 : (orc_key *)malloc((nch ? nch : 1) * sizeof(orc_key));
        if (!keys) return ORC_ECAPACITY;
        orc_chunk_keys(g, tokens + seq_off[q], len, 0, keys);
        orc_val *recs = recs_out + qchunk_off[q];
        memset(recs, 0, nch * sizeof(orc_val));
        uint64_t h = 0;
        while (h < nch) {
            orc_val v;
            ++lookups;
            if (!orc_lookup(runs, n_runs, &keys[h], &v, NULL)) break;
            recs[h] = v;
            ++h;
        }
        hit_out[q] = (uint32_t)h;
        if (!keys_out) free(keys);
    }
    if (lookups_out) *lookups_out = lookups;
    return ORC_OK;
}

/* ---- get_batch, tensor half: split hit blobs back into pool pages ------------------- */

/*
 * For every query q and chunk j < hit[q]: the blob at arenas[rec.file_id] + rec.offset is cut
 * into 2L page slabs (K0,V0,K1,V1,...) which are written to page dst_page_table[idx] of the
 * matching pool buffer. Nothing else in the pool is touched.
 */
int orc_decode_batch(const orc_geom *g, uint32_t n_query, const uint64_t *qchunk_off,
                     const uint32_t *hit, const orc_val *recs, const uint8_t *const *arenas,
                     const uint64_t *arena_bytes, uint32_t n_arenas,
                     const uint32_t *dst_page_table, uint8_t *const *kv_ptrs,
                     uint64_t num_pages)
{
    if (!geom_ok(g)) return ORC_EINVAL;
    const uint64_t L = g->n_layers, m = pages_per_chunk(g);
    const uint64_t pb = orc_page_bytes(g), cb = orc_chunk_bytes(g);
    for (uint32_t q = 0; q < n_query; ++q) {
        const uint64_t nch = qchunk_off[q + 1] - qchunk_off[q];
        if (hit[q] > nch) return ORC_EINVAL;
        for (uint64_t j = 0; j < hit[q]; ++j) {
            const uint64_t idx = qchunk_off[q] + j;
            const orc_val rec = recs[idx];
            if (rec.file_id >= n_arenas) return ORC_EBADREC;
            if (rec.offset > arena_bytes[rec.file_id] ||
                arena_bytes[rec.file_id] - rec.offset < cb) return ORC_EBADREC;
            for (uint64_t k = 0; k < m; ++k) {
                const uint64_t page = dst_page_table[idx * m + k];
                if (page >= num_pages) return ORC_EBADPAGE;
                const uint8_t *src = arenas[rec.file_id] + rec.offset + k * 2 * L * pb;
                for (uint64_t l = 0; l < L; ++l) {
                    memcpy(kv_ptrs[l] + page * pb, src + (2 * l) * pb, pb);
                    memcpy(kv_ptrs[L + l] + page * pb, src + (2 * l + 1) * pb, pb);
                }
            }
        }
    }
    return ORC_OK;
}

/* ---- compressing batch codec "xp12" (Sec. 3.4 "Batch Codec Operations": the combined tensors
 * of a batch are compressed before storage and decompressed together on load). The paper names
 * no algorithm; this build's is lossless, so restored pages stay bit-exact: bf16 values are
 * split into a sign+mantissa byte and an exponent, and the exponents of a page slab, which
 * cluster in a narrow window below the slab's largest, are stored in 4 bits each.
 *
 * One slab of N 16-bit elements v = (s << 15) | (e << 7) | m  (N a multiple of 8):
 *   e_max = largest e in the slab; base = max(0, e_max - 14); code = e - base if
 *   base <= e <= base + 14, else 15 ("exception").  n_exc = number of exceptions.
 *   mode 0 (packed), used when n_exc < N / 2:
 *     [0..16)        header: u32 magic 0x32315058, u32 n_exc, u8 base, u8 mode, u16 0, u32 size
 *     [16..16+N)     byte i = (s_i << 7) | m_i
 *     [.. +N/2)      nibble codes, element i in byte i/2, even i in the low nibble
 *     [.. +n_exc)    the raw e of every exception, in element order
 *     zero padding to a multiple of 16; size = that total
 *   mode 1 (raw), otherwise: the same header with n_exc = 0, base = 0, then the 2N raw bytes.
 * One chunk: a directory of 2L+1 u32 (byte offset of every slab inside the chunk blob, last =
 * the blob's size; zero-padded to a multiple of 16), then the slabs in blob order (K0 V0 K1 ...).
 * Record of a chunk: {file_id, reserved = blob size, offset}; blobs are placed back to back.
 */
#define ORC_XP_MAGIC 0x32315058u

static uint64_t round16(uint64_t x) { return (x + 15) & ~(uint64_t)15; }

uint64_t orc_xp12_slab_bound(uint64_t n_elems) { return 16 + 2 * n_elems; }

uint64_t orc_xp12_dir_bytes(const orc_geom *g)
{
    return round16(4ull * (g->chunk_tokens / g->page_tokens * 2ull * g->n_layers + 1));
}

/* Returns the encoded size; out needs orc_xp12_slab_bound(n) bytes. */
uint64_t orc_xp12_slab_encode(const uint16_t *in, uint64_t n, uint8_t *out)
{
    unsigned e_max = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const unsigned e = (in[i] >> 7) & 0xFF;
        if (e > e_max) e_max = e;
    }
    const unsigned base = e_max > 14 ? e_max - 14 : 0;
    uint64_t n_exc = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const unsigned e = (in[i] >> 7) & 0xFF;
        if (e < base) ++n_exc;                 /* e > base + 14 cannot happen: base + 14 >= e_max */
    }
    uint32_t hdr[4] = {ORC_XP_MAGIC, 0, 0, 0};
    uint64_t size;
    if (n_exc < n / 2) {
        size = round16(16 + n + n / 2 + n_exc);
        memset(out, 0, size);
        uint8_t *sm = out + 16, *codes = sm + n, *exc = codes + n / 2;
        uint64_t k = 0;
        for (uint64_t i = 0; i < n; ++i) {
            const unsigned v = in[i], e = (v >> 7) & 0xFF;
            sm[i] = (uint8_t)(((v >> 15) << 7) | (v & 0x7F));
            unsigned code = 15;
            if (e >= base) code = e - base; else exc[k++] = (uint8_t)e;
            codes[i / 2] |= (uint8_t)(code << (4 * (i & 1)));
        }
        hdr[1] = (uint32_t)n_exc;
        hdr[2] = base;                         /* base in byte 8, mode 0 in byte 9 */
    } else {
        size = 16 + 2 * n;
        memcpy(out + 16, in, 2 * n);
        hdr[2] = 1u << 8;                      /* mode 1 */
    }
    hdr[3] = (uint32_t)size;
    memcpy(out, hdr, 16);
    return size;
}

/* Returns the number of bytes consumed, or 0 if the slab is malformed. */
uint64_t orc_xp12_slab_decode(const uint8_t *in, uint64_t avail, uint64_t n, uint16_t *out)
{
    uint32_t hdr[4];
    if (avail < 16) return 0;
    memcpy(hdr, in, 16);
    const unsigned base = hdr[2] & 0xFF, mode = (hdr[2] >> 8) & 0xFF;
    const uint64_t n_exc = hdr[1], size = hdr[3];
    if (hdr[0] != ORC_XP_MAGIC || size > avail) return 0;
    if (mode == 1) {
        if (size != 16 + 2 * n) return 0;
        memcpy(out, in + 16, 2 * n);
        return size;
    }
    if (mode != 0 || size != round16(16 + n + n / 2 + n_exc)) return 0;
    const uint8_t *sm = in + 16, *codes = sm + n, *exc = codes + n / 2;
    uint64_t k = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const unsigned code = (codes[i / 2] >> (4 * (i & 1))) & 15;
        unsigned e;
        if (code == 15) { if (k >= n_exc) return 0; e = exc[k++]; } else e = base + code;
        out[i] = (uint16_t)(((sm[i] >> 7) << 15) | (e << 7) | (sm[i] & 0x7F));
    }
    return k == n_exc ? size : 0;
}

/*
 * put_batch with the compressing codec: as orc_encode_batch, but every chunk's blob is the
 * directory + compressed slabs, blobs are placed back to back from blob_out (which needs
 * n_chunks * orc_xp12_chunk_bound bytes), and records carry the blob size in `reserved`.
 * *blob_bytes_out = total bytes written.
 */
uint64_t orc_xp12_chunk_bound(const orc_geom *g)
{
    return orc_xp12_dir_bytes(g) +
           pages_per_chunk(g) * 2ull * g->n_layers * orc_xp12_slab_bound(orc_page_bytes(g) / 2);
}

int orc_encode_batch_xp12(const orc_geom *g, uint32_t n_req, const uint32_t *tokens,
                          const uint64_t *seq_off, const uint32_t *start_chunk,
                          const uint64_t *chunk_off, uint64_t n_chunks,
                          const uint32_t *page_table, const uint8_t *const *kv_ptrs,
                          uint64_t num_pages, uint32_t file_id, uint64_t base_offset,
                          orc_key *keys_out, orc_val *vals_out, uint8_t *blob_out,
                          uint64_t blob_capacity, uint64_t *blob_bytes_out)
{
    if (!geom_ok(g) || g->elem_bytes != 2 || orc_page_bytes(g) % 16) return ORC_EINVAL;
    /* keys exactly as in the identity codec */
    int rc = orc_encode_batch(g, n_req, tokens, seq_off, start_chunk, chunk_off, n_chunks, NULL,
                              NULL, 0, file_id, base_offset, keys_out, vals_out, NULL, 0);
    if (rc != ORC_OK) return rc;
    const uint64_t L = g->n_layers, pb = orc_page_bytes(g), ne = pb / 2;
    const uint64_t m = pages_per_chunk(g), slabs = m * 2 * L;
    const uint64_t dirb = orc_xp12_dir_bytes(g);
    uint64_t at = 0;
    for (uint64_t i = 0; i < n_chunks; ++i) {
        if (blob_capacity - at < orc_xp12_chunk_bound(g)) return ORC_ECAPACITY;
        uint8_t *blob = blob_out + at;
        uint32_t *dir = (uint32_t *)blob;
        memset(blob, 0, dirb);
        uint64_t pos = dirb;
        for (uint64_t b = 0; b < slabs; ++b) {      /* blob order: page by page, K0 V0 K1 V1 ... */
            const uint64_t page = page_table[i * m + b / (2 * L)];
            if (page >= num_pages) return ORC_EBADPAGE;
            const uint64_t bb = b % (2 * L), buf = (bb & 1) * L + (bb >> 1);
            dir[b] = (uint32_t)pos;
            pos += orc_xp12_slab_encode((const uint16_t *)(kv_ptrs[buf] + page * pb), ne,
                                        blob + pos);
        }
        dir[slabs] = (uint32_t)pos;
        vals_out[i].file_id = file_id;
        vals_out[i].reserved = (uint32_t)pos;
        vals_out[i].offset = base_offset + at;
        at += pos;
    }
    if (blob_bytes_out) *blob_bytes_out = at;
    return ORC_OK;
}

int orc_decode_batch_xp12(const orc_geom *g, uint32_t n_query, const uint64_t *qchunk_off,
                          const uint32_t *hit, const orc_val *recs, const uint8_t *const *arenas,
                          const uint64_t *arena_bytes, uint32_t n_arenas,
                          const uint32_t *dst_page_table, uint8_t *const *kv_ptrs,
                          uint64_t num_pages)
{
    if (!geom_ok(g) || g->elem_bytes != 2) return ORC_EINVAL;
    const uint64_t L = g->n_layers, pb = orc_page_bytes(g), ne = pb / 2;
    const uint64_t m = pages_per_chunk(g), slabs = m * 2 * L;
    const uint64_t dirb = orc_xp12_dir_bytes(g);
    for (uint32_t q = 0; q < n_query; ++q) {
        if (hit[q] > qchunk_off[q + 1] - qchunk_off[q]) return ORC_EINVAL;
        for (uint64_t j = 0; j < hit[q]; ++j) {
            const uint64_t idx = qchunk_off[q] + j;
            const orc_val rec = recs[idx];
            if (rec.file_id >= n_arenas || rec.reserved < dirb) return ORC_EBADREC;
            if (rec.offset > arena_bytes[rec.file_id] ||
                arena_bytes[rec.file_id] - rec.offset < rec.reserved) return ORC_EBADREC;
            const uint8_t *blob = arenas[rec.file_id] + rec.offset;
            const uint32_t *dir = (const uint32_t *)blob;
            if (dir[slabs] != rec.reserved) return ORC_EBADREC;
            for (uint64_t b = 0; b < slabs; ++b) {
                const uint64_t page = dst_page_table[idx * m + b / (2 * L)];
                if (page >= num_pages) return ORC_EBADPAGE;
                const uint64_t bb = b % (2 * L), buf = (bb & 1) * L + (bb >> 1);
                if (dir[b] < dirb || dir[b] > dir[b + 1] || dir[b + 1] > rec.reserved)
                    return ORC_EBADREC;
                if (!orc_xp12_slab_decode(blob + dir[b], dir[b + 1] - dir[b], ne,
                                          (uint16_t *)(kv_ptrs[buf] + page * pb)))
                    return ORC_EBADREC;
            }
        }
    }
    return ORC_OK;
}

/* ---- tensor-file merging (Sec. 3.4 "Automatic Tensor File Merging"): when adjacent tensor files
 * are merged into one, the file identifier and offset stored in the index are updated. A
 * relocation entry says: records of file `old_file` now live in `new_file`, `delta` bytes
 * further in. Records of files not in the table stay as they are. Returns the number of
 * records changed.
 */
typedef struct { uint32_t old_file, new_file; uint64_t delta; } orc_reloc;

uint64_t orc_relocate_records(orc_val *vals, uint64_t n, const orc_reloc *table, uint32_t n_table)
{
    uint64_t changed = 0;
    for (uint64_t i = 0; i < n; ++i) {
        for (uint32_t t = 0; t < n_table; ++t) {
            if (vals[i].file_id == table[t].old_file) {      /* first matching entry applies */
                vals[i].file_id = table[t].new_file;
                vals[i].offset += table[t].delta;
                ++changed;
                break;
            }
        }
    }
    return changed;
}

/* ---- exact prefix index ("xrun"): the index keyed by the token prefixes themselves, so that key
 * order IS prefix order and nothing depends on a digest (Sec. 3.1/3.2: keys keep the structure
 * of token prefixes; lexicographic order coincides with prefix order).
 *
 * One xrun holds whole stored sequences, each with one record per whole chunk (the records of
 * chunks it shares with an earlier sequence are copies of that sequence's records). The chunk
 * prefixes of a query Q present in it form an interval [0, m), m = floor(L / C), L = the
 * longest token prefix Q shares with any stored sequence. All of Q's records from that run
 * come from ONE stored sequence, the NEIGHBOUR of Q: among the sequences that reach L, the
 * largest one not above Q in token-lexicographic order (a sequence that is a prefix of another
 * is smaller; identical sequences order by arrival), and if none is, the smallest one above Q.
 * Across runs (newest first): hit = max over runs of m_run; the record of chunk j comes from
 * the newest run with m_run > j.
 *
 * Everything below is the definition by brute force: no sorting, no tree.
 */
typedef struct {
    const uint32_t *tokens;     /* arena */
    const uint64_t *seq_off;    /* [n_seq + 1] */
    uint32_t n_seq;
    const orc_val *vals;        /* records per chunk, sequence-major: chunk_off[s] + j */
    const uint64_t *chunk_off;  /* [n_seq + 1] prefix sums of floor(len_s / C) */
} orc_xrun;

static uint64_t lcp_tokens(const uint32_t *a, uint64_t na, const uint32_t *b, uint64_t nb)
{
    const uint64_t n = na < nb ? na : nb;
    uint64_t i = 0;
    while (i < n && a[i] == b[i]) ++i;
    return i;
}

/* token-lexicographic three-way comparison; a proper prefix is smaller */
static int tok_cmp(const uint32_t *a, uint64_t na, const uint32_t *b, uint64_t nb)
{
    const uint64_t l = lcp_tokens(a, na, b, nb);
    if (l < na && l < nb) return a[l] < b[l] ? -1 : 1;
    return na < nb ? -1 : na > nb ? 1 : 0;
}

int orc_xprobe_batch(const orc_geom *g, uint32_t n_query, const uint32_t *tokens,
                     const uint64_t *seq_off, const uint64_t *qchunk_off, const orc_xrun *runs,
                     uint32_t n_runs, uint32_t *hit_out, orc_val *recs_out)
{
    if (!geom_ok(g)) return ORC_EINVAL;
    const uint64_t C = g->chunk_tokens;
    for (uint32_t q = 0; q < n_query; ++q) {
        const uint32_t *Q = tokens + seq_off[q];
        const uint64_t len = seq_off[q + 1] - seq_off[q], nch = len / C;
        if (qchunk_off[q + 1] - qchunk_off[q] != nch) return ORC_EINVAL;
        orc_val *recs = recs_out + qchunk_off[q];
        memset(recs, 0, nch * sizeof(orc_val));
        uint64_t hit = 0;
        for (uint32_t r = 0; r < n_runs; ++r) {              /* newest first */
            const orc_xrun *x = &runs[r];
            uint64_t L = 0;
            for (uint32_t s = 0; s < x->n_seq; ++s) {
                const uint64_t l = lcp_tokens(Q, len, x->tokens + x->seq_off[s],
                                              x->seq_off[s + 1] - x->seq_off[s]);
                if (l > L) L = l;
            }
            const uint64_t m = L / C;
            if (m <= hit) continue;      /* newer runs already decided everything this one has */
            int have_lo = 0, have_hi = 0;
            uint32_t lo = 0, hi = 0;     /* largest reaching-L sequence <= Q; smallest one > Q */
            for (uint32_t s = 0; s < x->n_seq; ++s) {
                const uint32_t *S = x->tokens + x->seq_off[s];
                const uint64_t ns = x->seq_off[s + 1] - x->seq_off[s];
                if (lcp_tokens(Q, len, S, ns) != L) continue;
                if (tok_cmp(S, ns, Q, len) <= 0) {
                    if (!have_lo || tok_cmp(S, ns, x->tokens + x->seq_off[lo],
                                            x->seq_off[lo + 1] - x->seq_off[lo]) >= 0) {
                        lo = s;          /* >= : among identical sequences the later arrival */
                        have_lo = 1;
                    }
                } else if (!have_hi || tok_cmp(S, ns, x->tokens + x->seq_off[hi],
                                               x->seq_off[hi + 1] - x->seq_off[hi]) < 0) {
                    hi = s;              /* <  : among identical sequences the earlier arrival */
                    have_hi = 1;
                }
            }
            const uint32_t owner = have_lo ? lo : hi;
            for (uint64_t j = hit; j < m; ++j) recs[j] = x->vals[x->chunk_off[owner] + j];
            hit = m;
        }
        hit_out[q] = (uint32_t)hit;
    }
    return ORC_OK;
}

/* The sorted order an xrun is searched in: sequence numbers by token-lexicographic order, a
 * proper prefix first, identical sequences by number. Library sort with the comparison above. */
static const orc_xrun *g_sort_run;
static int order_cmp(const void *pa, const void *pb)
{
    const uint32_t a = *(const uint32_t *)pa, b = *(const uint32_t *)pb;
    const orc_xrun *x = g_sort_run;
    const int c = tok_cmp(x->tokens + x->seq_off[a], x->seq_off[a + 1] - x->seq_off[a],
                          x->tokens + x->seq_off[b], x->seq_off[b + 1] - x->seq_off[b]);
    return c ? c : (a < b ? -1 : a > b ? 1 : 0);
}

int orc_xrun_order(const uint32_t *tokens, const uint64_t *seq_off, uint32_t n_seq,
                   uint32_t *order_out)
{
    orc_xrun x = { tokens, seq_off, n_seq, NULL, NULL };
    for (uint32_t s = 0; s < n_seq; ++s) order_out[s] = s;
    g_sort_run = &x;
    qsort(order_out, n_seq, sizeof(uint32_t), order_cmp);
    g_sort_run = NULL;
    return ORC_OK;
}
