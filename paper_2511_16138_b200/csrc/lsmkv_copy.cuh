// Pack (pool pages -> contiguous blobs) and unpack (blobs -> pool pages): pure slab copies.
//
// A unit of work is one page slab (page_bytes contiguous on both sides). Two kernels move them:
//   k_copy_slabs_bulk   each warp owns one shared-memory stage and lets the copy engine move
//                       data: cp.async.bulk global->shared (mbarrier-completed), then
//                       cp.async.bulk shared->global. One lane per warp issues; a CTA of S warps
//                       is S independent single-stage pipelines, so S * stage_bytes are in
//                       flight per CTA with almost no instruction traffic.
//   k_copy_slabs_simt   plain 16-byte vector loads and stores (streaming cache hints).
// Both read the same unit description, so pack and unpack share the movers.
#pragma once
#include "lsmkv_common.cuh"

namespace lsmkv {

constexpr int kMaxArenas = 64;

struct ArenaTable {
    const unsigned char *base[kMaxArenas];
    uint64_t bytes[kMaxArenas];
};

// What to copy. pack: item i = encoded chunk, pool pages page_table[i*m .. i*m+m) -> blob +
// i*chunk_bytes (m = pages_per_chunk; the blob is the m page blobs in token order).
// unpack: item t = t-th hit chunk, idx = plan[t]; blob at arena[rec.file_id] + rec.offset ->
// pool pages page_table[idx*m .. idx*m+m).
struct CopyJob {
    int unpack;                      // 0 = pack, 1 = unpack
    uint32_t n_layers;
    uint32_t pages_per_chunk;        // m = chunk_tokens / page_tokens
    uint32_t page_bytes;
    uint32_t piece_bytes;            // bytes moved per step (<= page_bytes, multiple of 16)
    uint32_t pieces_per_slab;
    uint64_t num_pages;
    void *const *kv_ptrs;            // [dev] 2L pool buffers
    const uint32_t *page_table;      // [dev]
    unsigned char *blob;             // pack: destination
    uint64_t n_items;                // pack: number of chunks
    const uint64_t *n_items_dev;     // unpack: [dev] number of hit chunks
    const uint32_t *plan;            // unpack: [dev] hit chunk -> query-chunk index, or kSkip
    const lsmkv_val_t *recs;         // unpack
    DevStatus *st;
    long long wait_cycles;           // limit of the wait for a bulk copy's completion
    uint64_t test_drop_piece;        // test hook: this piece arms its barrier but starts no copy,
                                     // so its wait runs out (~0 = none)
};

struct Piece { const unsigned char *src; unsigned char *dst; uint32_t bytes; };

// Resolve piece number p (global, over all units) to addresses. Returns false to skip it.
__device__ __forceinline__ bool resolve_piece(const CopyJob &job, const ArenaTable &ar,
                                              uint64_t p, Piece &out)
{
    const uint32_t per_page = 2u * job.n_layers, slabs = per_page * job.pages_per_chunk;
    const uint64_t unit = p / job.pieces_per_slab;
    const uint32_t piece = (uint32_t)(p - unit * job.pieces_per_slab);
    const uint64_t item = unit / slabs;
    const uint32_t b = (uint32_t)(unit - item * slabs);      // slab of the chunk's blob
    const uint32_t pg = b / per_page;                        // which of the chunk's pages
    const uint32_t bb = b - pg * per_page;                   // slab of that page: 2*layer + (0=K, 1=V)
    const uint32_t buf = (bb & 1u) * job.n_layers + (bb >> 1);   // pool buffer: K layers, then V layers
    const uint32_t off = piece * job.piece_bytes;
    const uint32_t bytes = min(job.piece_bytes, job.page_bytes - off);
    uint64_t idx = item;
    const unsigned char *blob_slab;
    if (job.unpack) {
        const uint32_t e = __ldg(job.plan + item);
        if (e == kSkip) return false;
        idx = e;
        const uint4 r = __ldg(reinterpret_cast<const uint4 *>(job.recs + idx));
        const uint64_t roff = (uint64_t)r.z | ((uint64_t)r.w << 32);
        blob_slab = ar.base[r.x] + roff + (uint64_t)b * job.page_bytes;   // validated by the plan
    } else {
        blob_slab = job.blob + (item * slabs + b) * (uint64_t)job.page_bytes;
    }
    const uint64_t page = __ldg(job.page_table + idx * job.pages_per_chunk + pg);
    unsigned char *pool_buf = static_cast<unsigned char *>(job.kv_ptrs[buf]);
    if (page >= job.num_pages) {
        if (piece == 0 && bb == 0) st_flag(job.st, LSMKV_ST_BAD_PAGE, idx);
        return false;
    }
    if ((reinterpret_cast<uintptr_t>(pool_buf) & 15u) != 0) {
        if (piece == 0) st_flag(job.st, LSMKV_ST_MISALIGNED, idx);
        return false;
    }
    unsigned char *pool_slab = pool_buf + page * (uint64_t)job.page_bytes;
    if (job.unpack) { out.src = blob_slab + off; out.dst = pool_slab + off; }
    else            { out.src = pool_slab + off; out.dst = const_cast<unsigned char *>(blob_slab) + off; }
    out.bytes = bytes;
    return true;
}

__device__ __forceinline__ uint64_t job_pieces(const CopyJob &job)
{
    const uint64_t items = job.unpack ? *job.n_items_dev : job.n_items;
    return items * (2ull * job.n_layers * job.pages_per_chunk) * job.pieces_per_slab;
}

// ---- bulk-async mover ----------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

// Wait for phase `parity` of an mbarrier for at most `limit` clock cycles; false = gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, long long limit)
{
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63u) == 63u && clock64() - t0 > limit) return false;
    }
}

template <bool kHint>
__global__ void __launch_bounds__(1024, 1)
k_copy_slabs_bulk(const __grid_constant__ CopyJob job, const __grid_constant__ ArenaTable ar)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t n_stage = blockDim.x >> 5;
    const uint32_t warp = threadIdx.x >> 5;
    // stage buffers first (128-byte aligned each), then one mbarrier per stage
    const uint32_t stage_stride = (job.piece_bytes + 127u) & ~127u;
    unsigned char *buf = smem + (size_t)warp * stage_stride;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)n_stage * stage_stride);
    if (lane_id() != 0) return;          // one issuing lane per warp; no CTA-wide barrier is used

    const uint32_t bar = smem_addr(&bars[warp]);
    const uint32_t sbuf = smem_addr(buf);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    uint64_t pol = 0;
    if (kHint) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));

    const uint64_t total = job_pieces(job);
    const uint64_t workers = (uint64_t)gridDim.x * n_stage;
    uint32_t parity = 0;
    for (uint64_t p = (uint64_t)blockIdx.x * n_stage + warp; p < total; p += workers) {
        Piece pc;
        if (!resolve_piece(job, ar, p, pc)) continue;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     :: "r"(bar), "r"(pc.bytes) : "memory");
        if (p == job.test_drop_piece) {
            // (test hook) nothing is started, so nothing is in flight when the wait gives up
        } else if (kHint)
            asm volatile(
                "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
                " [%0], [%1], %2, [%3], %4;"
                :: "r"(sbuf), "l"(pc.src), "r"(pc.bytes), "r"(bar), "l"(pol) : "memory");
        else
            asm volatile(
                "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes"
                " [%0], [%1], %2, [%3];"
                :: "r"(sbuf), "l"(pc.src), "r"(pc.bytes), "r"(bar) : "memory");
        if (!mbar_wait_bounded(bar, parity, job.wait_cycles)) {
            // The copy did not report completion in time: record it and stop using this stage.
            // A copy that was started gets one more bounded wait before the warp leaves, so
            // that it is not still writing this CTA's shared memory then.
            st_flag(job.st, LSMKV_ST_WAIT_EXPIRED, p);
            mbar_wait_bounded(bar, parity, job.wait_cycles);
            break;
        }
        parity ^= 1u;
        if (kHint)
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                         :: "l"(pc.dst), "r"(sbuf), "r"(pc.bytes), "l"(pol) : "memory");
        else
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         :: "l"(pc.dst), "r"(sbuf), "r"(pc.bytes) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // stage free again
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ---- plain vector mover --------------------------------------------------------------------

__global__ void __launch_bounds__(256)
k_copy_slabs_simt(const __grid_constant__ CopyJob job, const __grid_constant__ ArenaTable ar)
{
    const uint64_t total = job_pieces(job);
    for (uint64_t p = blockIdx.x; p < total; p += gridDim.x) {
        Piece pc;
        if (!resolve_piece(job, ar, p, pc)) continue;
        const uint4 *s = reinterpret_cast<const uint4 *>(pc.src);
        uint4 *d = reinterpret_cast<uint4 *>(pc.dst);
        const uint32_t n = pc.bytes >> 4;
        uint32_t i = threadIdx.x;
        for (; i + 3u * 256u < n; i += 4u * 256u) {
            const uint4 a = __ldcs(s + i), b = __ldcs(s + i + 256), c = __ldcs(s + i + 512),
                        e = __ldcs(s + i + 768);
            __stcs(d + i, a); __stcs(d + i + 256, b); __stcs(d + i + 512, c); __stcs(d + i + 768, e);
        }
        for (; i < n; i += 256u) __stcs(d + i, __ldcs(s + i));
    }
}

// ---- decode plan: hit lengths -> compact list of chunks to copy -----------------------------

// Exclusive prefix sums of the (validated) hit lengths; one CTA.
__global__ void __launch_bounds__(1024)
k_plan_scan(uint32_t n_query, const uint64_t *__restrict__ qchunk_off, uint64_t n_qchunks,
            const uint32_t *__restrict__ hit, uint64_t *__restrict__ hit_off, DevStatus *st)
{
    __shared__ uint64_t warp_sum[32];
    __shared__ uint64_t carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    for (uint64_t base = 0; base < n_query; base += blockDim.x) {
        const uint64_t q = base + threadIdx.x;
        uint64_t h = 0;
        if (q < n_query) {
            const uint64_t o0 = qchunk_off[q], o1 = qchunk_off[q + 1];
            h = hit[q];
            if (o1 < o0 || o1 > n_qchunks || h > o1 - o0) {
                st_flag(st, LSMKV_ST_BAD_COUNT, q);
                h = 0;
            }
        }
        uint64_t x = h;
#pragma unroll
        for (unsigned d = 1; d < 32; d <<= 1) {
            const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        if (lane == 31) warp_sum[warp] = x;
        __syncthreads();
        if (warp == 0) {
            uint64_t w = lane < (blockDim.x >> 5) ? warp_sum[lane] : 0;
#pragma unroll
            for (unsigned d = 1; d < 32; d <<= 1) {
                const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, w, d);
                if (lane >= d) w += y;
            }
            warp_sum[lane] = w;                   // inclusive sums of the warps
        }
        __syncthreads();
        const uint64_t before = carry_s + (warp ? warp_sum[warp - 1] : 0) + (x - h);
        if (q < n_query) hit_off[q] = before;
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry_s = before + h;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        hit_off[n_query] = carry_s;
        atomicAdd(&st->chunks_decoded, (unsigned long long)carry_s);
    }
}

// plan[hit_off[q] + j] = qchunk_off[q] + j for j < hit[q]; records are validated here once.
__global__ void __launch_bounds__(256)
k_plan_fill(uint32_t n_query, const uint64_t *__restrict__ qchunk_off,
            const uint64_t *__restrict__ hit_off, const lsmkv_val_t *__restrict__ recs,
            const __grid_constant__ ArenaTable ar, uint32_t n_arenas, uint64_t chunk_bytes,
            uint32_t min_coded_bytes, uint32_t *__restrict__ plan, DevStatus *st)
{
    const unsigned lane = lane_id();
    const uint64_t warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t q = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; q < n_query;
         q += warps) {
        const uint64_t t0 = hit_off[q], n = hit_off[q + 1] - t0, o0 = qchunk_off[q];
        for (uint64_t j = lane; j < n; j += 32) {
            const uint64_t idx = o0 + j;
            const uint4 r = __ldg(reinterpret_cast<const uint4 *>(recs + idx));
            const uint64_t off = (uint64_t)r.z | ((uint64_t)r.w << 32);
            // identity codec: blobs are chunk_bytes long; compressing codec (min_coded_bytes
            // != 0): the record carries its blob's size
            const uint64_t need = min_coded_bytes ? r.y : chunk_bytes;
            bool ok = r.x < n_arenas && (off & 15u) == 0;
            if (min_coded_bytes) ok = ok && r.y >= min_coded_bytes && (r.y & 15u) == 0;
            if (ok) ok = off <= ar.bytes[r.x] && ar.bytes[r.x] - off >= need;
            if (!ok) st_flag(st, LSMKV_ST_BAD_RECORD, idx);
            plan[t0 + j] = ok ? (uint32_t)idx : kSkip;
        }
    }
}

}  // namespace lsmkv
