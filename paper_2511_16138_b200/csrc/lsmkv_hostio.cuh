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
    return grow_scratch(ctx, &ctx->d_io[kind], &ctx->io_cap[kind], bytes, bytes, __LINE__);
}

// Second stream and events of the host-buffer put with the compressing codec.
int ensure_io_stream(lsmkv_ctx *ctx)
{
    if (ctx->io_stream) return LSMKV_OK;
    CU(ctx, cudaStreamCreateWithFlags(&ctx->io_stream, cudaStreamNonBlocking));
    CU(ctx, cudaEventCreateWithFlags(&ctx->io_ev_enc, cudaEventDisableTiming));
    CU(ctx, cudaEventCreateWithFlags(&ctx->io_ev_free[0], cudaEventDisableTiming));
    CU(ctx, cudaEventCreateWithFlags(&ctx->io_ev_free[1], cudaEventDisableTiming));
    return LSMKV_OK;
}

size_t pad256(size_t b) { return (b + 255) & ~size_t(255); }

// Large transfers go out in pieces: copies of one direction are served in issue order even
// when they sit on different streams, so one multi-GiB copy would hold up every small copy
// another stream issues in the same direction (and with it that stream's kernels). With
// bounded pieces a put on one stream and a get on another keep both PCIe directions busy.
// The piece is the context's "host_copy_piece_bytes" (every piece boundary costs the link a
// little, every piece makes the other stream's small copies wait that much longer).
cudaError_t copy_pieces(const lsmkv_ctx *ctx, void *dst, const void *src, size_t bytes,
                        cudaMemcpyKind kind, cudaStream_t s)
{
    unsigned char *d = static_cast<unsigned char *>(dst);
    const unsigned char *p = static_cast<const unsigned char *>(src);
    const size_t piece = (size_t)ctx->host_copy_piece;
    for (size_t at = 0; at < bytes; at += piece) {
        const size_t n = std::min(piece, bytes - at);
        const cudaError_t e = cudaMemcpyAsync(d + at, p + at, n, kind, s);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

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

// put with the compressing codec, without a stop per slice: how many bytes a slice's encode
// produced is only known on the device, so the device itself moves them from the stage to the
// caller's host blob (pinned memory is visible to kernels), behind the bytes of the slices
// before, and keeps the running total. `last` is the slice's last record: its end, less the
// call's base offset and the total so far, is the slice's size.
__device__ __forceinline__ bool slice_extent(const uint64_t *total, const lsmkv_val_t *last,
                                             uint64_t base_offset, uint64_t capacity,
                                             uint64_t stage_bytes, uint64_t *start, uint64_t *used)
{
    const uint4 r = *reinterpret_cast<const uint4 *>(last);
    *start = *total;
    if (r.y == 0) return false;                          // the encode overflowed its stage (flagged)
    *used = (((uint64_t)r.z | ((uint64_t)r.w << 32)) + r.y) - base_offset - *start;
    return *used <= stage_bytes && (*used & 15u) == 0 && *start <= capacity && *used <= capacity - *start;
}

__global__ void __launch_bounds__(256)
k_blob_to_host(const unsigned char *__restrict__ stage, unsigned char *__restrict__ host_blob,
               const uint64_t *total, const lsmkv_val_t *last, uint64_t base_offset,
               uint64_t capacity, uint64_t stage_bytes, lsmkv::DevStatus *st)
{
    uint64_t start, used;
    if (!slice_extent(total, last, base_offset, capacity, stage_bytes, &start, &used)) {
        if (blockIdx.x == 0 && threadIdx.x == 0) lsmkv::st_flag(st, LSMKV_ST_OVERFLOW, 0);
        return;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(stage);
    uint4 *dst = reinterpret_cast<uint4 *>(host_blob + start);
    const uint64_t n = used >> 4, step = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += step)
        dst[i] = __ldcs(src + i);
}

__global__ void k_blob_advance(uint64_t *total, const lsmkv_val_t *last, uint64_t base_offset,
                               uint64_t capacity, uint64_t stage_bytes)
{
    uint64_t start, used;
    if (slice_extent(total, last, base_offset, capacity, stage_bytes, &start, &used))
        *total = start + used;
}

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
    // slices [a, b): as many requests as fit the blob stage (always at least one)
    std::vector<uint32_t> &cuts = ctx->h_cuts;
    cuts.clear();
    uint64_t m_max = 0;
    for (uint32_t a = 0; a < n_req;) {
        uint32_t b = a + 1;
        while (b < n_req && coff[b + 1] - coff[a] <= stage_chunks_max) ++b;
        cuts.push_back(a);
        m_max = std::max(m_max, coff[b] - coff[a]);
        a = b;
    }
    cuts.push_back(n_req);
    const size_t n_slices = cuts.size() - 1;
    const uint64_t t_first = seq_off[0], nt = seq_off[n_req] - t_first;
    // With the compressing codec, whose sizes the host has to wait for, blobs leave from two
    // stages in turn on a second stream, so that a slice is packed while the one before it is
    // on its way. (With the identity codec the same was measured slower end to end, 76 against
    // 87-90 GB/s with a get running beside the put: everything stays on the caller's stream.)
    const bool two_stages = with_blob && coded;

    // device scratch: every descriptor of the call (uploaded once, up front), the blob stages
    const size_t n_rel = (size_t)n_req + n_slices;        // sum over slices of (requests + 1)
    size_t need = pad256(nt * 4) + 2 * pad256(n_rel * 8) + pad256((size_t)n_req * 4) +
                  pad256(n_chunks * ctx->ppc * 4) + pad256(m_max * 32) + pad256(m_max * 16) +
                  (with_blob ? pad256(m_max * slot) : 0) + (two_stages ? pad256(m_max * slot) : 0) + 4096;
    int rc = ensure_io(ctx, 0, need);
    if (rc != LSMKV_OK) return rc;
    IoLayout io(ctx->d_io[0]);
    uint32_t *d_tok = io.take<uint32_t>(nt ? nt : 1);
    uint64_t *d_seq = io.take<uint64_t>(n_rel);
    uint64_t *d_coff = io.take<uint64_t>(n_rel);
    uint32_t *d_start = io.take<uint32_t>(n_req);
    uint32_t *d_pages = io.take<uint32_t>(n_chunks * ctx->ppc);      // ppc entries per chunk
    lsmkv_key_t *d_keys = io.take<lsmkv_key_t>(m_max);
    lsmkv_val_t *d_vals = io.take<lsmkv_val_t>(m_max);
    unsigned char *d_blob = with_blob ? io.take<unsigned char>(m_max * slot) : nullptr;
    unsigned char *d_blob2 = two_stages ? io.take<unsigned char>(m_max * slot) : nullptr;

    ScratchLease lease(ctx, 0, s, 2 * n_rel * 8 + 256);
    if (!lease.ok()) return LSMKV_ENOMEM;
    uint64_t *h_seq = lease.take<uint64_t>(n_rel), *h_coff = lease.take<uint64_t>(n_rel);
    size_t at = 0;
    for (size_t k = 0; k < n_slices; ++k) {              // offsets relative to each slice
        const uint32_t a = cuts[k], b = cuts[k + 1];
        for (uint32_t r = a; r <= b; ++r) {
            h_seq[at + (r - a)] = seq_off[r] - seq_off[a];
            h_coff[at + (r - a)] = coff[r] - coff[a];
        }
        at += (size_t)(b - a) + 1;
    }
    if (nt) CU(ctx, copy_pieces(ctx, d_tok, tokens + t_first, nt * 4, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(d_seq, h_seq, n_rel * 8, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(d_coff, h_coff, n_rel * 8, cudaMemcpyHostToDevice, s));
    if (start_chunk)
        CU(ctx, cudaMemcpyAsync(d_start, start_chunk, (size_t)n_req * 4, cudaMemcpyHostToDevice, s));
    if (with_blob)
        CU(ctx, copy_pieces(ctx, d_pages, page_table, n_chunks * ctx->ppc * 4, cudaMemcpyHostToDevice, s));

    // Compressing codec: how many bytes a slice produced is only known on the device. Either
    // the device places the slices in the host blob itself and nothing ever stops (on request:
    // "host_put_device_placed", needs pinned memory and no byte count at return), or -- the
    // default, which moves the bytes with the copy engines at the link's full rate -- the host
    // waits for each slice's records only (a short wait: the slice before it is still on its way
    // to the host on a second stream and from the other of two stages).
    unsigned char *host_blob_dev = nullptr;
    uint64_t *d_total = reinterpret_cast<uint64_t *>(reinterpret_cast<char *>(ctx->d_status) + 128);
    if (coded && !blob_bytes_out && ctx->host_put_device_placed) {
        void *dp = nullptr;
        if (cudaHostGetDevicePointer(&dp, blob_out, 0) == cudaSuccess && dp && aligned16(dp))
            host_blob_dev = static_cast<unsigned char *>(dp);
        else
            cudaGetLastError();                      // pageable memory: the waiting path below
    }
    if (host_blob_dev) CU(ctx, cudaMemsetAsync(d_total, 0, sizeof(uint64_t), s));
    uint64_t host_used = 0;                          // waiting path: bytes placed so far
    bool stage_used[2] = {false, false};
    const bool staged = two_stages && !host_blob_dev;   // the two-stage path
    if (staged) {
        rc = ensure_io_stream(ctx);
        if (rc != LSMKV_OK) return rc;
    }
    size_t staged_slices = 0;
    at = 0;
    for (size_t k = 0; k < n_slices; ++k) {
        const uint32_t a = cuts[k], b = cuts[k + 1], nr = b - a;
        const uint64_t m = coff[b] - coff[a];
        const size_t rel_at = at;
        at += (size_t)nr + 1;
        if (m == 0) continue;
        // slices alternate between two stages; a stage is free again once the copy of the slice
        // it held two slices ago has left on the second stream
        const int sg = staged ? (int)(staged_slices & 1) : 0;
        unsigned char *stage = sg ? d_blob2 : d_blob;
        if (staged && stage_used[sg])
            CU(ctx, cudaStreamWaitEvent(s, ctx->io_ev_free[sg], 0));
        ctx->xp_base_add = host_blob_dev ? d_total : nullptr;   // records count from the device's total
        rc = lsmkv_encode_batch(ctx, stream, nr, d_tok + (seq_off[a] - t_first), d_seq + rel_at,
                                start_chunk ? d_start + a : nullptr, d_coff + rel_at, m,
                                with_blob ? d_pages + coff[a] * ctx->ppc : nullptr,
                                with_blob ? pool : nullptr,
                                file_id, base_offset + (coded ? host_used : coff[a] * cb), d_keys,
                                d_vals, stage, with_blob ? m * slot : 0);
        ctx->xp_base_add = nullptr;
        if (rc != LSMKV_OK) return rc;
        CU(ctx, cudaMemcpyAsync(keys_out + coff[a], d_keys, m * 32, cudaMemcpyDeviceToHost, s));
        CU(ctx, cudaMemcpyAsync(vals_out + coff[a], d_vals, m * 16, cudaMemcpyDeviceToHost, s));
        if (host_blob_dev) {
            // posted writes over the host link need little parallelism: a few CTAs saturate it
            // and leave the other SMs to whatever runs beside the put
            k_blob_to_host<<<(unsigned)ctx->host_copy_ctas, 256, 0, s>>>(
                stage, host_blob_dev, d_total, d_vals + (m - 1), base_offset, blob_capacity,
                m * slot, ctx->d_status);
            k_blob_advance<<<1, 1, 0, s>>>(d_total, d_vals + (m - 1), base_offset, blob_capacity,
                                           m * slot);
            ctx->launches += 2;
            CU(ctx, cudaGetLastError());
        } else if (coded) {
            // wait for this slice's records (only the encode and two small copies are ahead of
            // the event), then send exactly the bytes it produced, behind the previous slice's
            CU(ctx, cudaEventRecord(ctx->io_ev_enc, s));
            CU(ctx, cudaEventSynchronize(ctx->io_ev_enc));
            const lsmkv_val_t &last = vals_out[coff[b] - 1];
            if (last.reserved == 0) return LSMKV_ECAPACITY;   // stage overflow (flagged on device)
            const uint64_t used = last.offset + last.reserved - (base_offset + host_used);
            if (blob_capacity - host_used < used) return LSMKV_ECAPACITY;
            CU(ctx, cudaStreamWaitEvent(ctx->io_stream, ctx->io_ev_enc, 0));
            CU(ctx, copy_pieces(ctx, static_cast<unsigned char *>(blob_out) + host_used, stage, used,
                                cudaMemcpyDeviceToHost, ctx->io_stream));
            CU(ctx, cudaEventRecord(ctx->io_ev_free[sg], ctx->io_stream));
            stage_used[sg] = true;
            ++staged_slices;
            host_used += used;
            if (blob_bytes_out) *blob_bytes_out = host_used;
        } else if (with_blob) {
            CU(ctx, copy_pieces(ctx, static_cast<unsigned char *>(blob_out) + coff[a] * cb, d_blob, m * cb,
                                cudaMemcpyDeviceToHost, s));
        }
    }
    for (int sg = 0; sg < 2; ++sg)                   // the call's work ends when its copies have
        if (stage_used[sg]) CU(ctx, cudaStreamWaitEvent(s, ctx->io_ev_free[sg], 0));
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
    if (total_hits >= 0xFFFFFFFFull) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // a slice holds at most blob_stage bytes of blobs (always at least one blob)
    const uint64_t blob_stage = std::max<uint64_t>((uint64_t)ctx->host_stage_bytes, max_len);

    // pass 1 (host): where each slice starts, then the stage-relative records and destination
    // pages of every hit chunk, in hit order
    std::vector<uint64_t> &first = ctx->h_off_a;                     // first hit of every slice
    first.clear();
    uint64_t k = 0, at = 0, m_max = 0;
    for (uint32_t q = 0; q < n_query; ++q) {
        for (uint64_t j = 0; j < hit_chunks[q]; ++j, ++k) {
            const uint64_t len = coded ? recs[qchunk_off[q] + j].reserved : cb;
            if (first.empty() || at + len > blob_stage) { first.push_back(k); at = 0; }
            at += len;
        }
    }
    first.push_back(total_hits);
    const size_t n_slices = first.size() - 1;
    const uint64_t ppc = ctx->ppc;                                   // page-table entries per chunk
    ScratchLease lease(ctx, 2, s, total_hits * (16 + 4 * ppc) + n_slices * 24 + 4096);
    if (!lease.ok()) return LSMKV_ENOMEM;
    lsmkv_val_t *h_recs = lease.take<lsmkv_val_t>(total_hits);
    uint32_t *h_pages = lease.take<uint32_t>(total_hits * ppc);
    uint64_t *h_qoff = lease.take<uint64_t>(2 * n_slices);           // {0, m} per slice
    uint32_t *h_hit = lease.take<uint32_t>(n_slices);                // m per slice
    k = 0;
    size_t sl_at = 0;
    for (uint32_t q = 0; q < n_query; ++q) {
        for (uint64_t j = 0; j < hit_chunks[q]; ++j, ++k) {
            const uint64_t idx = qchunk_off[q] + j;
            if (sl_at + 1 < first.size() && k == first[sl_at + 1]) ++sl_at;
            if (k == first[sl_at]) at = 0;
            h_recs[k] = lsmkv_val_t{0, coded ? recs[idx].reserved : 0u, at};
            for (uint64_t p = 0; p < ppc; ++p) h_pages[k * ppc + p] = dst_page_table[idx * ppc + p];
            at += coded ? recs[idx].reserved : cb;
        }
    }
    for (size_t sl = 0; sl < n_slices; ++sl) {
        m_max = std::max(m_max, first[sl + 1] - first[sl]);
        h_qoff[2 * sl] = 0;
        h_qoff[2 * sl + 1] = first[sl + 1] - first[sl];
        h_hit[sl] = (uint32_t)(first[sl + 1] - first[sl]);
    }
    (void)m_max;

    // several slices: their blobs come up on a second stream into two stages in turn, so that a
    // slice is on its way while the one before it is scattered
    const bool staged = n_slices > 1;
    size_t need = pad256(blob_stage) * (staged ? 2 : 1) + pad256(total_hits * 16) +
                  pad256(total_hits * ppc * 4) + pad256(n_slices * 16) + pad256(n_slices * 4) + 4096;
    int rc = ensure_io(ctx, 2, need);
    if (rc != LSMKV_OK) return rc;
    if (staged) {
        rc = ensure_io_stream(ctx);
        if (rc != LSMKV_OK) return rc;
    }
    IoLayout io(ctx->d_io[2]);
    unsigned char *d_blob = io.take<unsigned char>(blob_stage);
    unsigned char *d_blob2 = staged ? io.take<unsigned char>(blob_stage) : nullptr;
    lsmkv_val_t *d_recs = io.take<lsmkv_val_t>(total_hits);
    uint32_t *d_pages = io.take<uint32_t>(total_hits * ppc);
    uint64_t *d_qoff = io.take<uint64_t>(2 * n_slices);
    uint32_t *d_hit = io.take<uint32_t>(n_slices);
    // every descriptor goes up first, so that nothing small queues behind the blob copies
    CU(ctx, copy_pieces(ctx, d_recs, h_recs, total_hits * 16, cudaMemcpyHostToDevice, s));
    CU(ctx, copy_pieces(ctx, d_pages, h_pages, total_hits * ppc * 4, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(d_qoff, h_qoff, n_slices * 16, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(d_hit, h_hit, n_slices * 4, cudaMemcpyHostToDevice, s));
    cudaStream_t up = s;                             // the stream the blobs come up on
    bool stage_busy[2] = {false, false};
    if (staged) {                                    // it starts where the caller's stream is now
        up = ctx->io_stream;
        CU(ctx, cudaEventRecord(ctx->io_ev_enc, s));
        CU(ctx, cudaStreamWaitEvent(up, ctx->io_ev_enc, 0));
    }

    // pass 2: per slice, the blobs go to the stage in hit order (blobs that sit back to back in
    // a host arena travel as one run of copies) and are scattered into the pool
    k = 0;
    uint32_t q = 0;
    uint64_t j = 0;
    for (size_t sl = 0; sl < n_slices; ++sl) {
        const uint64_t m = first[sl + 1] - first[sl];
        uint64_t run_dst = 0, run_bytes = 0, stage_used = 0;
        const unsigned char *run_src = nullptr;
        const int sg = staged ? (int)(sl & 1) : 0;
        unsigned char *stage = sg ? d_blob2 : d_blob;
        const void *stage_arena[1] = {stage};
        if (staged && stage_busy[sg])                // the slice it held two slices ago is scattered
            CU(ctx, cudaStreamWaitEvent(up, ctx->io_ev_free[sg], 0));
        for (uint64_t c = 0; c < m; ++c, ++k) {
            while (j >= hit_chunks[q]) { ++q; j = 0; }
            const lsmkv_val_t &r = recs[qchunk_off[q] + j];
            ++j;
            const uint64_t len = coded ? r.reserved : cb;
            const unsigned char *src = static_cast<const unsigned char *>(arenas[r.file_id]) + r.offset;
            if (run_bytes && src == run_src + run_bytes) {
                run_bytes += len;
            } else {
                if (run_bytes)
                    CU(ctx, copy_pieces(ctx, stage + run_dst, run_src, run_bytes, cudaMemcpyHostToDevice, up));
                run_dst = h_recs[k].offset;
                run_src = src;
                run_bytes = len;
            }
            stage_used = h_recs[k].offset + len;
        }
        if (run_bytes)
            CU(ctx, copy_pieces(ctx, stage + run_dst, run_src, run_bytes, cudaMemcpyHostToDevice, up));
        if (staged) {
            CU(ctx, cudaEventRecord(ctx->io_ev_enc, up));
            CU(ctx, cudaStreamWaitEvent(s, ctx->io_ev_enc, 0));
        }
        rc = lsmkv_decode_batch(ctx, stream, 1, d_qoff + 2 * sl, m, d_hit + sl, d_recs + first[sl],
                                stage_arena, &stage_used, 1, d_pages + first[sl] * ppc, pool);
        if (rc != LSMKV_OK) return rc;
        if (staged) {
            CU(ctx, cudaEventRecord(ctx->io_ev_free[sg], s));
            stage_busy[sg] = true;
        }
    }
    return LSMKV_OK;
}
