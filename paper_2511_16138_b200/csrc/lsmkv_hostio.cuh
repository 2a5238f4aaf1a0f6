// Host-buffer variants of the batch calls: inputs and outputs live in host memory (pinned for
// full speed), the KV pool stays on the device. They stage through device scratch owned by the
// context, slice large batches so the scratch stays bounded, and call the device-buffer entry
// points for the actual work -- every copy and kernel is enqueued on the caller's stream.
// Included at the end of lsmkv.cu (needs the context's internals).
#pragma once

namespace {

struct IoLayout {
    unsigned char *base;
    size_t at;
    explicit IoLayout(void *p) : base(static_cast<unsigned char *>(p)), at(0) {}
    template <typename T> T *take(size_t n)
    {
        at = (at + 255) & ~size_t(255);
        T *p = reinterpret_cast<T *>(base + at);
        at += n * sizeof(T);
        return p;
    }
};

// One staging area per kind of call (0 = put, 1 = probe, 2 = decode), so that a put on one
// stream and a get on another do not share scratch.
int ensure_io(lsmkv_ctx *ctx, int kind, size_t bytes)
{
    if (bytes <= ctx->io_cap[kind] && ctx->d_io[kind]) return LSMKV_OK;
    void *p = nullptr;
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { cuda_fail(ctx, e); return LSMKV_ENOMEM; }
    if (ctx->d_io[kind]) cudaFree(ctx->d_io[kind]);   // waits for work that may still use it
    ctx->d_io[kind] = p;
    cudaGetLastError();   // drop any stale last-error left by the allocation calls
    ctx->io_cap[kind] = bytes;
    return LSMKV_OK;
}

size_t pad256(size_t b) { return (b + 255) & ~size_t(255); }

// Pinned host scratch for the small descriptor arrays a call uploads. Every kind of call
// (0 = put, 1 = probe, 2 = decode) alternates between two slots of its own; a slot is reused
// only after the stream work of the call that used it last has finished (its event), so the
// asynchronous uploads never read rewritten memory and a put never waits for a get.
struct ScratchLease {
    lsmkv_ctx *ctx;
    lsmkv_ctx::HostScratch *slot;
    cudaStream_t s;
    unsigned char *p;
    size_t at;
    ScratchLease(lsmkv_ctx *c, int kind, cudaStream_t st, size_t bytes)
        : ctx(c), slot(nullptr), s(st), p(nullptr), at(0)
    {
        lsmkv_ctx::HostScratch &h = c->hs[kind][c->hs_next[kind]];
        c->hs_next[kind] ^= 1;
        if (h.used && h.done) cudaEventSynchronize(h.done);
        if (!h.done && cudaEventCreateWithFlags(&h.done, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            return;
        }
        if (h.cap < bytes) {
            if (h.p) cudaFreeHost(h.p);
            h.p = nullptr;
            h.cap = 0;
            if (cudaHostAlloc(&h.p, bytes, cudaHostAllocDefault) != cudaSuccess) {
                cudaGetLastError();
                h.p = nullptr;
                return;
            }
            h.cap = bytes;
        }
        slot = &h;
        p = static_cast<unsigned char *>(h.p);
    }
    bool ok() const { return p != nullptr; }
    template <typename T> T *take(size_t n)
    {
        at = (at + 15) & ~size_t(15);
        T *r = reinterpret_cast<T *>(p + at);
        at += n * sizeof(T);
        return r;
    }
    ~ScratchLease()
    {
        if (!slot) return;
        cudaEventRecord(slot->done, s);
        slot->used = true;
    }
};

}  // namespace

extern "C" int lsmkv_put_batch_host(lsmkv_ctx *ctx, void *stream, uint32_t n_req,
                                    const uint32_t *tokens, const uint64_t *seq_off,
                                    const uint32_t *start_chunk, const uint32_t *page_table,
                                    const lsmkv_pool_t *pool, uint32_t file_id,
                                    uint64_t base_offset, lsmkv_key_t *keys_out,
                                    lsmkv_val_t *vals_out, void *blob_out,
                                    uint64_t blob_capacity, uint64_t *n_chunks_out,
                                    uint64_t *blob_bytes_out)
{
    if (!ctx) return LSMKV_EINVAL;
    if (n_chunks_out) *n_chunks_out = 0;
    if (blob_bytes_out) *blob_bytes_out = 0;
    if (n_req == 0) return LSMKV_OK;
    if (!tokens || !seq_off || !keys_out || !vals_out) return LSMKV_EINVAL;
    const bool with_blob = blob_out != nullptr;
    if (with_blob && (!page_table || !pool || !pool->kv_ptrs)) return LSMKV_EINVAL;
    const uint64_t C = ctx->geom.chunk_tokens, cb = ctx->chunk_bytes;
    // output index of every request's first encoded chunk
    std::vector<uint64_t> &coff = ctx->h_off_a;
    coff.assign((size_t)n_req + 1, 0);
    for (uint32_t r = 0; r < n_req; ++r) {
        if (seq_off[r + 1] < seq_off[r]) return LSMKV_EINVAL;
        const uint64_t nch = (seq_off[r + 1] - seq_off[r]) / C;
        const uint64_t st = start_chunk ? start_chunk[r] : 0;
        coff[r + 1] = coff[r] + (nch > st ? nch - st : 0);
    }
    const uint64_t n_chunks = coff[n_req];
    if (n_chunks_out) *n_chunks_out = n_chunks;
    if (n_chunks == 0) return LSMKV_OK;
    const bool coded = with_blob && ctx->codec != LSMKV_CODEC_IDENTITY;
    if (with_blob && !coded && blob_capacity / cb < n_chunks) return LSMKV_ECAPACITY;
    // bytes one chunk can take in the stage (worst case of the codec)
    const uint64_t slot = coded ? lsmkv_encode_bound(ctx, 1) : cb;
    if (with_blob && !coded && blob_bytes_out) *blob_bytes_out = n_chunks * cb;

    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint64_t stage_chunks_max = std::max<uint64_t>(1, (uint64_t)ctx->host_stage_bytes / slot);
    uint64_t host_used = 0;                          // compressing codec: bytes placed so far
    ScratchLease lease(ctx, 0, s, (4 * (size_t)n_req + 8) * 8 + 64 * (size_t)n_req + 4096);
    if (!lease.ok()) return LSMKV_ENOMEM;
    for (uint32_t a = 0; a < n_req;) {
        // slice [a, b): as many requests as fit the blob stage (always at least one)
        uint32_t b = a + 1;
        while (b < n_req && coff[b + 1] - coff[a] <= stage_chunks_max) ++b;
        const uint32_t nr = b - a;
        const uint64_t m = coff[b] - coff[a];
        const uint64_t t0 = seq_off[a], nt = seq_off[b] - t0;
        if (m == 0) { a = b; continue; }
        size_t need = pad256(nt * 4) + 2 * pad256(((size_t)nr + 1) * 8) + pad256((size_t)nr * 4) +
                      pad256(m * 4) + pad256(m * 32) + pad256(m * 16) +
                      (with_blob ? pad256(m * slot) : 0) + 4096;
        int rc = ensure_io(ctx, 0, need);
        if (rc != LSMKV_OK) return rc;
        IoLayout io(ctx->d_io[0]);
        uint32_t *d_tok = io.take<uint32_t>(nt);
        uint64_t *d_seq = io.take<uint64_t>((size_t)nr + 1);
        uint64_t *d_coff = io.take<uint64_t>((size_t)nr + 1);
        uint32_t *d_start = io.take<uint32_t>(nr);
        uint32_t *d_pages = io.take<uint32_t>(m);
        lsmkv_key_t *d_keys = io.take<lsmkv_key_t>(m);
        lsmkv_val_t *d_vals = io.take<lsmkv_val_t>(m);
        unsigned char *d_blob = with_blob ? io.take<unsigned char>(m * slot) : nullptr;
        // offsets relative to the slice, in pinned scratch that lives until the call's work ends
        uint64_t *rel = lease.take<uint64_t>(2 * ((size_t)nr + 1));
        for (uint32_t k = 0; k <= nr; ++k) {
            rel[k] = seq_off[a + k] - t0;
            rel[(size_t)nr + 1 + k] = coff[a + k] - coff[a];
        }
        CU(ctx, cudaMemcpyAsync(d_tok, tokens + t0, nt * 4, cudaMemcpyHostToDevice, s));
        CU(ctx, cudaMemcpyAsync(d_seq, rel, ((size_t)nr + 1) * 8, cudaMemcpyHostToDevice, s));
        CU(ctx, cudaMemcpyAsync(d_coff, rel + nr + 1, ((size_t)nr + 1) * 8,
                                cudaMemcpyHostToDevice, s));
        if (start_chunk)
            CU(ctx, cudaMemcpyAsync(d_start, start_chunk + a, (size_t)nr * 4, cudaMemcpyHostToDevice, s));
        if (with_blob)
            CU(ctx, cudaMemcpyAsync(d_pages, page_table + coff[a], m * 4, cudaMemcpyHostToDevice, s));
        rc = lsmkv_encode_batch(ctx, stream, nr, d_tok, d_seq, start_chunk ? d_start : nullptr,
                                d_coff, m, with_blob ? d_pages : nullptr, with_blob ? pool : nullptr,
                                file_id, base_offset + (coded ? host_used : coff[a] * cb), d_keys,
                                d_vals, d_blob, with_blob ? m * slot : 0);
        if (rc != LSMKV_OK) return rc;
        CU(ctx, cudaMemcpyAsync(keys_out + coff[a], d_keys, m * 32, cudaMemcpyDeviceToHost, s));
        CU(ctx, cudaMemcpyAsync(vals_out + coff[a], d_vals, m * 16, cudaMemcpyDeviceToHost, s));
        if (coded) {
            // blob sizes depend on the data: wait for this slice's records, then copy exactly
            // the bytes it produced behind the previous slice's
            CU(ctx, cudaStreamSynchronize(s));
            const lsmkv_val_t &last = vals_out[coff[b] - 1];
            if (last.reserved == 0) return LSMKV_ECAPACITY;   // stage overflow (flagged on device)
            const uint64_t used = last.offset + last.reserved - (base_offset + host_used);
            if (blob_capacity - host_used < used) return LSMKV_ECAPACITY;
            CU(ctx, cudaMemcpyAsync(static_cast<unsigned char *>(blob_out) + host_used, d_blob, used,
                                    cudaMemcpyDeviceToHost, s));
            host_used += used;
            if (blob_bytes_out) *blob_bytes_out = host_used;
        } else if (with_blob) {
            CU(ctx, cudaMemcpyAsync(static_cast<unsigned char *>(blob_out) + coff[a] * cb, d_blob,
                                    m * cb, cudaMemcpyDeviceToHost, s));
        }
        a = b;
    }
    return LSMKV_OK;
}

extern "C" int lsmkv_probe_batch_host(lsmkv_ctx *ctx, void *stream, uint32_t n_query,
                                      const uint32_t *tokens, const uint64_t *seq_off,
                                      const lsmkv_run_t *runs, uint32_t n_runs,
                                      uint32_t *hit_chunks_out, lsmkv_val_t *recs_out,
                                      lsmkv_key_t *keys_out, uint64_t *n_qchunks_out)
{
    if (!ctx) return LSMKV_EINVAL;
    if (n_qchunks_out) *n_qchunks_out = 0;
    if (n_query == 0) return LSMKV_OK;
    if (!seq_off || !hit_chunks_out) return LSMKV_EINVAL;
    const uint64_t C = ctx->geom.chunk_tokens;
    std::vector<uint64_t> &qoff = ctx->h_off_a;
    qoff.assign((size_t)n_query + 1, 0);
    for (uint32_t q = 0; q < n_query; ++q) {
        if (seq_off[q + 1] < seq_off[q]) return LSMKV_EINVAL;
        qoff[q + 1] = qoff[q] + (seq_off[q + 1] - seq_off[q]) / C;
    }
    const uint64_t total = qoff[n_query];
    if (n_qchunks_out) *n_qchunks_out = total;
    const uint64_t t0 = seq_off[0], nt = seq_off[n_query] - t0;
    if (total && (!tokens || !recs_out)) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    size_t need = pad256(nt * 4) + 2 * pad256(((size_t)n_query + 1) * 8) + pad256((size_t)n_query * 4) +
                  pad256(total * 16) + (keys_out ? pad256(total * 32) : 0) + 4096;
    int rc = ensure_io(ctx, 1, need);
    if (rc != LSMKV_OK) return rc;
    IoLayout io(ctx->d_io[1]);
    uint32_t *d_tok = io.take<uint32_t>(nt ? nt : 1);
    uint64_t *d_seq = io.take<uint64_t>((size_t)n_query + 1);
    uint64_t *d_qoff = io.take<uint64_t>((size_t)n_query + 1);
    uint32_t *d_hit = io.take<uint32_t>(n_query);
    lsmkv_val_t *d_recs = io.take<lsmkv_val_t>(total ? total : 1);
    lsmkv_key_t *d_keys = keys_out ? io.take<lsmkv_key_t>(total ? total : 1) : nullptr;
    ScratchLease lease(ctx, 1, s, (2 * (size_t)n_query + 4) * 8 + 256);
    if (!lease.ok()) return LSMKV_ENOMEM;
    uint64_t *rel = lease.take<uint64_t>((size_t)n_query + 1);
    uint64_t *qo = lease.take<uint64_t>((size_t)n_query + 1);
    for (uint32_t q = 0; q <= n_query; ++q) { rel[q] = seq_off[q] - t0; qo[q] = qoff[q]; }
    if (nt) CU(ctx, cudaMemcpyAsync(d_tok, tokens + t0, nt * 4, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(d_seq, rel, ((size_t)n_query + 1) * 8, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(d_qoff, qo, ((size_t)n_query + 1) * 8, cudaMemcpyHostToDevice, s));
    rc = lsmkv_probe_batch(ctx, stream, n_query, d_tok, d_seq, d_qoff, total, runs, n_runs, d_hit,
                           d_recs, d_keys);
    if (rc != LSMKV_OK) return rc;
    CU(ctx, cudaMemcpyAsync(hit_chunks_out, d_hit, (size_t)n_query * 4, cudaMemcpyDeviceToHost, s));
    if (total) {
        CU(ctx, cudaMemcpyAsync(recs_out, d_recs, total * 16, cudaMemcpyDeviceToHost, s));
        if (keys_out)
            CU(ctx, cudaMemcpyAsync(keys_out, d_keys, total * 32, cudaMemcpyDeviceToHost, s));
    }
    return LSMKV_OK;
}

extern "C" int lsmkv_decode_batch_host(lsmkv_ctx *ctx, void *stream, uint32_t n_query,
                                       const uint64_t *qchunk_off, const uint32_t *hit_chunks,
                                       const lsmkv_val_t *recs, const void *const *arenas,
                                       const uint64_t *arena_bytes, uint32_t n_arenas,
                                       const uint32_t *dst_page_table, const lsmkv_pool_t *pool)
{
    if (!ctx) return LSMKV_EINVAL;
    if (n_query == 0) return LSMKV_OK;
    if (!qchunk_off || !hit_chunks || !recs || !dst_page_table || !pool || !pool->kv_ptrs ||
        !arenas || !arena_bytes || n_arenas == 0)
        return LSMKV_EINVAL;
    const uint64_t cb = ctx->chunk_bytes;
    const bool coded = ctx->codec != LSMKV_CODEC_IDENTITY;
    // the hit chunks in order, validated on the host (nothing is enqueued if one is bad)
    uint64_t total_hits = 0, max_len = coded ? 0 : cb, min_len = coded ? ~0ull : cb, sum_len = 0;
    for (uint32_t q = 0; q < n_query; ++q) {
        if (qchunk_off[q + 1] < qchunk_off[q] || hit_chunks[q] > qchunk_off[q + 1] - qchunk_off[q])
            return LSMKV_EINVAL;
        for (uint64_t j = 0; j < hit_chunks[q]; ++j) {
            const lsmkv_val_t &r = recs[qchunk_off[q] + j];
            const uint64_t len = coded ? r.reserved : cb;
            if (r.file_id >= n_arenas || !arenas[r.file_id] || r.offset > arena_bytes[r.file_id] ||
                arena_bytes[r.file_id] - r.offset < len || (coded && (len < 32 || (len & 15))))
                return LSMKV_EINVAL;
            max_len = std::max(max_len, len);
            min_len = std::min(min_len, len);
            sum_len += len;
        }
        total_hits += hit_chunks[q];
    }
    if (total_hits == 0) return LSMKV_OK;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // a slice holds at most m_max chunks and stage_bytes bytes of blobs (at least one blob)
    const uint64_t stage_bytes_max = std::max<uint64_t>((uint64_t)ctx->host_stage_bytes, max_len);
    const uint64_t stage_chunks = std::max<uint64_t>(1, stage_bytes_max / min_len);
    const uint64_t m_max = std::min<uint64_t>(stage_chunks, total_hits);
    const uint64_t blob_stage = coded ? stage_bytes_max : m_max * cb;
    size_t need = pad256(blob_stage) + pad256(m_max * 16) + pad256(m_max * 4) + 3 * 256 + 4096;
    int rc = ensure_io(ctx, 2, need);
    if (rc != LSMKV_OK) return rc;
    IoLayout io(ctx->d_io[2]);
    unsigned char *d_blob = io.take<unsigned char>(blob_stage);
    lsmkv_val_t *d_recs = io.take<lsmkv_val_t>(m_max);
    uint32_t *d_pages = io.take<uint32_t>(m_max);
    uint64_t *d_qoff = io.take<uint64_t>(2);
    uint32_t *d_hit = io.take<uint32_t>(1);
    const void *stage_arena[1] = {d_blob};

    // descriptors of all hit chunks (each slice uploads its part), plus 32 bytes per slice
    // every slice stages at least one chunk, and at least half the stage unless blobs are huge
    uint64_t n_slices_max = total_hits;
    if (max_len <= blob_stage / 2)
        n_slices_max = std::min<uint64_t>(total_hits, 2 * (sum_len / blob_stage) + total_hits / m_max + 2);
    n_slices_max = std::min<uint64_t>(n_slices_max, 1u << 20);
    ScratchLease lease(ctx, 2, s, total_hits * 20 + n_slices_max * 48 + 4096);
    if (!lease.ok()) return LSMKV_ENOMEM;
    lsmkv_val_t *srecs_all = lease.take<lsmkv_val_t>(total_hits);
    uint32_t *spages_all = lease.take<uint32_t>(total_hits);
    uint32_t q = 0;
    uint64_t j = 0, left = total_hits, done = 0, slices = 0;
    while (q < n_query && left) {
        // one slice: up to m_max hit chunks and blob_stage bytes, blobs gathered into the stage
        // in hit order; blobs that sit back to back in a host arena travel as one copy
        const uint64_t cap = std::min<uint64_t>(m_max, left);
        lsmkv_val_t *srecs = srecs_all + done;
        uint32_t *spages = spages_all + done;
        uint64_t m = 0, at = 0;              // chunks and bytes staged in this slice
        uint64_t run_dst = 0;                // stage offset of the pending contiguous copy
        const unsigned char *run_src = nullptr;
        uint64_t run_bytes = 0;
        while (q < n_query && m < cap) {
            if (j >= hit_chunks[q]) { ++q; j = 0; continue; }
            const uint64_t idx = qchunk_off[q] + j;
            const lsmkv_val_t &r = recs[idx];
            const uint64_t len = coded ? r.reserved : cb;
            if (at + len > blob_stage) break;                    // slice is full (m >= 1 here)
            const unsigned char *src = static_cast<const unsigned char *>(arenas[r.file_id]) + r.offset;
            if (run_bytes && src == run_src + run_bytes) {
                run_bytes += len;
            } else {
                if (run_bytes)
                    CU(ctx, cudaMemcpyAsync(d_blob + run_dst, run_src, run_bytes,
                                            cudaMemcpyHostToDevice, s));
                run_dst = at;
                run_src = src;
                run_bytes = len;
            }
            srecs[m] = lsmkv_val_t{0, coded ? r.reserved : 0u, at};
            spages[m] = dst_page_table[idx];
            at += len;
            ++m;
            ++j;
        }
        if (run_bytes)
            CU(ctx, cudaMemcpyAsync(d_blob + run_dst, run_src, run_bytes, cudaMemcpyHostToDevice, s));
        if (m == 0) break;
        left -= m;
        done += m;
        if (++slices > n_slices_max) return LSMKV_EINVAL;     // cannot happen: see the bound above
        uint64_t *qoff2 = lease.take<uint64_t>(2);
        uint32_t *hit1 = lease.take<uint32_t>(1);
        qoff2[0] = 0;
        qoff2[1] = m;
        *hit1 = (uint32_t)m;
        CU(ctx, cudaMemcpyAsync(d_recs, srecs, m * 16, cudaMemcpyHostToDevice, s));
        CU(ctx, cudaMemcpyAsync(d_pages, spages, m * 4, cudaMemcpyHostToDevice, s));
        CU(ctx, cudaMemcpyAsync(d_qoff, qoff2, 16, cudaMemcpyHostToDevice, s));
        CU(ctx, cudaMemcpyAsync(d_hit, hit1, 4, cudaMemcpyHostToDevice, s));
        const uint64_t stage_bytes = at;
        rc = lsmkv_decode_batch(ctx, stream, 1, d_qoff, m, d_hit, d_recs, stage_arena, &stage_bytes,
                                1, d_pages, pool);
        if (rc != LSMKV_OK) return rc;
    }
    return LSMKV_OK;
}
