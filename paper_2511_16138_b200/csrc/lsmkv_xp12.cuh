// Compressing batch codec "xp12": lossless exponent packing of bf16 page slabs.
//
// A slab of N 16-bit elements (s << 15 | e << 7 | m) becomes a 16-byte header, N bytes of
// sign+mantissa, N/2 bytes of 4-bit exponent codes relative to base = max(0, e_max - 14), and
// one raw exponent byte per element below the window (code 15), in element order; if half the
// elements or more fall below the window the slab is stored raw. A chunk blob is a directory
// of 2L+1 u32 slab offsets followed by the slabs; blobs are placed back to back and every
// record carries its blob's size. Encoding is three steps on the stream: measure every slab
// (k_xp_measure), turn sizes into offsets, records and directories (k_scan_blocks,
// k_xp_layout), then write the slabs (k_xp_pack). Decoding (k_xp_unpack) validates every
// directory entry and header before it trusts them.
#pragma once
#include "lsmkv_common.cuh"
#include "lsmkv_copy.cuh"

namespace lsmkv {

constexpr uint32_t kXpMagic = 0x32315058u;
constexpr int kXpThreads = 256;

struct XpJob {
    uint32_t n_layers;
    uint32_t pages_per_chunk;    // m = chunk_tokens / page_tokens; a chunk has 2L * m slabs
    uint32_t page_bytes;
    uint32_t n_elems;            // page_bytes / 2
    uint32_t dir_bytes;          // round16(4 * (2L * m + 1))
    uint64_t num_pages;
    void *const *kv_ptrs;
    const uint32_t *page_table;
    uint64_t n_chunks;
    uint32_t *slab_size;         // [n_chunks * 2L]
    uint32_t *slab_info;         // base | mode << 8
    uint32_t *slab_nexc;
    uint64_t *chunk_off;         // [n_chunks + 1] sizes, then exclusive offsets (+ total)
    unsigned char *blob;
    uint64_t blob_capacity;
    uint32_t file_id;
    uint64_t base_offset;
    const uint64_t *base_add;    // [dev] or NULL: added to base_offset in the records (a running
                                 // total kept on the device by the host-buffer put)
    lsmkv_val_t *vals_out;
    DevStatus *st;
};

__device__ __forceinline__ uint32_t round16u(uint32_t x) { return (x + 15u) & ~15u; }

// block-wide reductions / scan for 256 threads
__device__ __forceinline__ uint32_t block_max(uint32_t v, uint32_t *sh)
{
#pragma unroll
    for (int d = 16; d; d >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, d));
    if (lane_id() == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t r = sh[0];
#pragma unroll
    for (int w = 1; w < kXpThreads / 32; ++w) r = max(r, sh[w]);
    __syncthreads();
    return r;
}

__device__ __forceinline__ uint32_t block_sum(uint32_t v, uint32_t *sh)
{
#pragma unroll
    for (int d = 16; d; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    if (lane_id() == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t r = 0;
#pragma unroll
    for (int w = 0; w < kXpThreads / 32; ++w) r += sh[w];
    __syncthreads();
    return r;
}

// exclusive scan of v over the block's threads; *total = block sum
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t *sh, uint32_t *total)
{
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    uint32_t x = v;
#pragma unroll
    for (unsigned d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, d);
        if (lane >= d) x += y;
    }
    if (lane == 31) sh[warp] = x;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (unsigned w = 0; w < kXpThreads / 32; ++w) {
        const uint32_t s = sh[w];
        if (w < warp) before += s;
        all += s;
    }
    __syncthreads();
    *total = all;
    return before + x - v;
}

// exponents of the 8 elements in a uint4
__device__ __forceinline__ void exps8(const uint4 &q, uint32_t e[8])
{
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        e[2 * k] = (w[k] >> 7) & 0xFFu;
        e[2 * k + 1] = (w[k] >> 23) & 0xFFu;
    }
}

// source slab of (chunk i, blob slab b), or nullptr when the page id / buffer is unusable
__device__ __forceinline__ const unsigned char *xp_src(const XpJob &job, uint64_t i, uint32_t b,
                                                       bool report)
{
    const uint32_t per_page = 2u * job.n_layers, pg = b / per_page, bb = b - pg * per_page;
    const uint64_t page = __ldg(job.page_table + i * job.pages_per_chunk + pg);
    const uint32_t buf = (bb & 1u) * job.n_layers + (bb >> 1);
    const unsigned char *pool_buf = static_cast<const unsigned char *>(job.kv_ptrs[buf]);
    if (page >= job.num_pages) {
        if (report && bb == 0 && threadIdx.x == 0) st_flag(job.st, LSMKV_ST_BAD_PAGE, i);
        return nullptr;
    }
    if ((reinterpret_cast<uintptr_t>(pool_buf) & 15u) != 0) {
        if (report && threadIdx.x == 0) st_flag(job.st, LSMKV_ST_MISALIGNED, i);
        return nullptr;
    }
    return pool_buf + page * (uint64_t)job.page_bytes;
}

// step 1: per slab e_max, exceptions, encoded size
__global__ void __launch_bounds__(kXpThreads)
k_xp_measure(const __grid_constant__ XpJob job)
{
    __shared__ uint32_t sh[kXpThreads / 32];
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk, n8 = job.n_elems >> 3;
    const uint64_t total = job.n_chunks * slabs;
    for (uint64_t u = blockIdx.x; u < total; u += gridDim.x) {
        const uint64_t i = u / slabs;
        const uint32_t b = (uint32_t)(u - i * slabs);
        const unsigned char *src = xp_src(job, i, b, true);
        if (!src) {                                   // unusable page: an empty raw-size slot
            if (threadIdx.x == 0) {
                job.slab_size[u] = 16u + job.page_bytes;
                job.slab_info[u] = 0xFFFFu;           // marks "skip"
                job.slab_nexc[u] = 0;
            }
            continue;
        }
        const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
        uint32_t emax = 0;
        for (uint32_t k = threadIdx.x; k < n8; k += kXpThreads) {
            uint32_t e[8];
            exps8(__ldg(s4 + k), e);
#pragma unroll
            for (int t = 0; t < 8; ++t) emax = max(emax, e[t]);
        }
        emax = block_max(emax, sh);
        const uint32_t base = emax > 14u ? emax - 14u : 0u;
        uint32_t cnt = 0;
        for (uint32_t k = threadIdx.x; k < n8; k += kXpThreads) {
            uint32_t e[8];
            exps8(__ldg(s4 + k), e);
#pragma unroll
            for (int t = 0; t < 8; ++t) cnt += e[t] < base ? 1u : 0u;
        }
        cnt = block_sum(cnt, sh);
        if (threadIdx.x == 0) {
            const bool packed = cnt < job.n_elems / 2;
            job.slab_size[u] = packed ? round16u(16u + job.n_elems + job.n_elems / 2 + cnt)
                                      : 16u + 2u * job.n_elems;
            job.slab_info[u] = packed ? base : (1u << 8);
            job.slab_nexc[u] = packed ? cnt : 0u;
        }
    }
}

// step 2a: blob size of every chunk
__global__ void __launch_bounds__(256)
k_xp_chunk_sizes(const __grid_constant__ XpJob job)
{
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < job.n_chunks;
         i += (uint64_t)gridDim.x * blockDim.x) {
        uint64_t sz = job.dir_bytes;
        for (uint32_t b = 0; b < slabs; ++b) sz += job.slab_size[i * slabs + b];
        job.chunk_off[i] = sz;
    }
}

// step 2b (after the exclusive scan of chunk_off, total in chunk_off[n_chunks]): records and
// directories. A chunk that does not fit the blob buffer is flagged and gets an empty record.
__global__ void __launch_bounds__(256)
k_xp_layout(const __grid_constant__ XpJob job)
{
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < job.n_chunks;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t off = job.chunk_off[i], size = job.chunk_off[i + 1] - off;
        uint4 v;
        v.x = job.file_id;
        if (off + size > job.blob_capacity || size > 0xFFFFFFFFull) {
            st_flag(job.st, LSMKV_ST_OVERFLOW, i);
            v.y = 0; v.z = 0; v.w = 0;
            *reinterpret_cast<uint4 *>(job.vals_out + i) = v;
            continue;
        }
        const uint64_t o = job.base_offset + off + (job.base_add ? *job.base_add : 0ull);
        v.y = (uint32_t)size;
        v.z = (uint32_t)o;
        v.w = (uint32_t)(o >> 32);
        *reinterpret_cast<uint4 *>(job.vals_out + i) = v;
        uint32_t *dir = reinterpret_cast<uint32_t *>(job.blob + off);
        uint32_t pos = job.dir_bytes;
        for (uint32_t b = 0; b < slabs; ++b) {
            dir[b] = pos;
            pos += job.slab_size[i * slabs + b];
        }
        dir[slabs] = pos;
        for (uint32_t k = slabs + 1; k < job.dir_bytes / 4; ++k) dir[k] = 0;
    }
}

// step 3: write the slabs
__global__ void __launch_bounds__(kXpThreads)
k_xp_pack(const __grid_constant__ XpJob job)
{
    __shared__ uint32_t sh[kXpThreads / 32];
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk, n8 = job.n_elems >> 3, N = job.n_elems;
    const uint64_t total = job.n_chunks * slabs;
    for (uint64_t u = blockIdx.x; u < total; u += gridDim.x) {
        const uint64_t i = u / slabs;
        const uint32_t b = (uint32_t)(u - i * slabs);
        const uint64_t off = job.chunk_off[i], csize = job.chunk_off[i + 1] - off;
        if (off + csize > job.blob_capacity || csize > 0xFFFFFFFFull) continue;   // flagged above
        const uint32_t info = job.slab_info[u], size = job.slab_size[u];
        const uint32_t *dir = reinterpret_cast<const uint32_t *>(job.blob + off);
        unsigned char *out = job.blob + off + dir[b];
        const unsigned char *src = info == 0xFFFFu ? nullptr : xp_src(job, i, b, false);
        if (!src) {                                   // skipped page: a raw slab of zeros
            uint4 *o4 = reinterpret_cast<uint4 *>(out);
            for (uint32_t k = threadIdx.x; k < size / 16; k += kXpThreads)
                o4[k] = k == 0 ? make_uint4(kXpMagic, 0, 1u << 8, size) : make_uint4(0, 0, 0, 0);
            continue;
        }
        const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
        const uint32_t mode = (info >> 8) & 0xFFu, base = info & 0xFFu;
        if (threadIdx.x == 0)
            *reinterpret_cast<uint4 *>(out) =
                make_uint4(kXpMagic, job.slab_nexc[u], base | (mode << 8), size);
        if (mode == 1) {                              // raw
            uint4 *o4 = reinterpret_cast<uint4 *>(out + 16);
            for (uint32_t k = threadIdx.x; k < n8; k += kXpThreads) o4[k] = __ldg(s4 + k);
            continue;
        }
        unsigned char *sm = out + 16, *codes = sm + N, *exc = codes + N / 2;
        uint32_t exc_before = 0;                      // exceptions of earlier sweeps
        for (uint32_t k0 = 0; k0 < n8; k0 += kXpThreads) {
            const uint32_t k = k0 + threadIdx.x;
            uint32_t cnt = 0, c32 = 0;
            uint32_t ex[8];
            uint2 smv = make_uint2(0, 0);
            if (k < n8) {
                const uint4 q = __ldg(s4 + k);
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
                uint32_t smb[8];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const uint32_t lo = w[t] & 0xFFFFu, hi = w[t] >> 16;
                    smb[2 * t] = ((lo >> 15) << 7) | (lo & 0x7Fu);
                    smb[2 * t + 1] = ((hi >> 15) << 7) | (hi & 0x7Fu);
                    const uint32_t e0 = (lo >> 7) & 0xFFu, e1 = (hi >> 7) & 0xFFu;
                    uint32_t c0 = 15u, c1 = 15u;
                    if (e0 >= base) c0 = e0 - base; else ex[cnt++] = e0;
                    if (e1 >= base) c1 = e1 - base; else ex[cnt++] = e1;
                    c32 |= (c0 | (c1 << 4)) << (8 * t);
                }
                smv.x = smb[0] | (smb[1] << 8) | (smb[2] << 16) | (smb[3] << 24);
                smv.y = smb[4] | (smb[5] << 8) | (smb[6] << 16) | (smb[7] << 24);
                *reinterpret_cast<uint2 *>(sm + 8ull * k) = smv;
                *reinterpret_cast<uint32_t *>(codes + 4ull * k) = c32;
            }
            uint32_t sweep_total;
            const uint32_t at = exc_before + block_excl_scan(cnt, sh, &sweep_total);
            for (uint32_t t = 0; t < cnt; ++t) exc[at + t] = (unsigned char)ex[t];
            exc_before += sweep_total;
        }
        // zero padding up to the slab's size
        const uint32_t used = 16u + N + N / 2 + exc_before;
        if (threadIdx.x < size - used) out[used + threadIdx.x] = 0;
    }
}

// decode: one CTA per (hit chunk, slab); every offset and header is checked before use
struct XpUnpackJob {
    uint32_t n_layers;
    uint32_t pages_per_chunk;
    uint32_t page_bytes;
    uint32_t n_elems;
    uint32_t dir_bytes;
    uint64_t num_pages;
    void *const *kv_ptrs;
    const uint32_t *page_table;      // destination pages
    const uint64_t *n_items_dev;     // number of hit chunks
    const uint32_t *plan;            // hit chunk -> query-chunk index, or kSkip
    const lsmkv_val_t *recs;
    DevStatus *st;
};

__global__ void __launch_bounds__(kXpThreads)
k_xp_unpack(const __grid_constant__ XpUnpackJob job, const __grid_constant__ ArenaTable ar)
{
    __shared__ uint32_t sh[kXpThreads / 32];
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk, n8 = job.n_elems >> 3, N = job.n_elems;
    const uint64_t total = *job.n_items_dev * slabs;
    for (uint64_t u = blockIdx.x; u < total; u += gridDim.x) {
        const uint64_t item = u / slabs;
        const uint32_t b = (uint32_t)(u - item * slabs);
        const uint32_t idx = __ldg(job.plan + item);
        if (idx == kSkip) continue;
        const uint4 r = __ldg(reinterpret_cast<const uint4 *>(job.recs + idx));
        const uint64_t roff = (uint64_t)r.z | ((uint64_t)r.w << 32);
        const unsigned char *blob = ar.base[r.x] + roff;          // range validated by the plan
        const uint32_t csize = r.y;
        const uint32_t *dir = reinterpret_cast<const uint32_t *>(blob);
        const uint32_t d0 = __ldg(dir + b), d1 = __ldg(dir + b + 1);
        const uint32_t per_page = 2u * job.n_layers, pg = b / per_page, bb = b - pg * per_page;
        const uint64_t page = __ldg(job.page_table + (uint64_t)idx * job.pages_per_chunk + pg);
        const uint32_t buf = (bb & 1u) * job.n_layers + (bb >> 1);
        unsigned char *pool_buf = static_cast<unsigned char *>(job.kv_ptrs[buf]);
        bool ok = __ldg(dir + slabs) == csize && d0 >= job.dir_bytes && d0 <= d1 && d1 <= csize &&
                  (d0 & 15u) == 0 && d1 - d0 >= 16u;
        uint4 h = make_uint4(0, 0, 0, 0);
        if (ok) h = __ldg(reinterpret_cast<const uint4 *>(blob + d0));
        const uint32_t mode = (h.z >> 8) & 0xFFu, base = h.z & 0xFFu, n_exc = h.y;
        ok = ok && h.x == kXpMagic && h.w == d1 - d0 &&
             ((mode == 1 && h.w == 16u + 2u * N) ||
              (mode == 0 && n_exc < N && h.w == round16u(16u + N + N / 2 + n_exc)));
        if (!ok) {
            if (threadIdx.x == 0) st_flag(job.st, LSMKV_ST_BAD_RECORD, idx);
            continue;
        }
        if (page >= job.num_pages) {
            if (threadIdx.x == 0 && bb == 0) st_flag(job.st, LSMKV_ST_BAD_PAGE, idx);
            continue;
        }
        if ((reinterpret_cast<uintptr_t>(pool_buf) & 15u) != 0) {
            if (threadIdx.x == 0) st_flag(job.st, LSMKV_ST_MISALIGNED, idx);
            continue;
        }
        uint4 *dst = reinterpret_cast<uint4 *>(pool_buf + page * (uint64_t)job.page_bytes);
        const unsigned char *in = blob + d0 + 16;
        if (mode == 1) {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(in);
            for (uint32_t k = threadIdx.x; k < n8; k += kXpThreads) dst[k] = __ldg(s4 + k);
            continue;
        }
        const unsigned char *sm = in, *codes = in + N, *exc = codes + N / 2;
        uint32_t exc_before = 0;
        for (uint32_t k0 = 0; k0 < n8; k0 += kXpThreads) {
            const uint32_t k = k0 + threadIdx.x;
            uint2 smv = make_uint2(0, 0);
            uint32_t c32 = 0, cnt = 0;
            if (k < n8) {
                smv = __ldg(reinterpret_cast<const uint2 *>(sm + 8ull * k));
                c32 = __ldg(reinterpret_cast<const uint32_t *>(codes + 4ull * k));
#pragma unroll
                for (int t = 0; t < 8; ++t) cnt += ((c32 >> (4 * t)) & 15u) == 15u ? 1u : 0u;
            }
            uint32_t sweep_total;
            uint32_t at = exc_before + block_excl_scan(cnt, sh, &sweep_total);
            exc_before += sweep_total;
            if (k < n8) {
                uint32_t w[4];
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const uint32_t smb = ((t < 4 ? smv.x : smv.y) >> (8 * (t & 3))) & 0xFFu;
                    const uint32_t code = (c32 >> (4 * t)) & 15u;
                    uint32_t e = base + code;
                    if (code == 15u) { e = at < n_exc ? __ldg(exc + at) : 0u; ++at; }
                    const uint32_t v = ((smb >> 7) << 15) | ((e & 0xFFu) << 7) | (smb & 0x7Fu);
                    if (t & 1) w[t >> 1] |= v << 16; else w[t >> 1] = v;
                }
                dst[k] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        if (exc_before != n_exc && threadIdx.x == 0) st_flag(job.st, LSMKV_ST_BAD_RECORD, idx);
    }
}

// ---------------------------------------------------------------------------------------------
// Fast kernels for the common slab sizes (N = 2048 * SWEEPS elements, SWEEPS in {4, 8, 16}).
//
// The generic kernels above spend their time issuing instructions (ncu: 60-70 % issue active at
// under 40 % DRAM throughput): per-element bit fiddling and a block-wide scan with two barriers
// per sweep. The fast ones (a) treat the two 16-bit elements of a 32-bit word at once with plain
// integer SWAR arithmetic, (b) give every warp one contiguous eighth of the slab, so exception
// order is (warp, sweep, lane, element) and the only block-wide step is one exchange of eight
// warp totals, and (c) touch the exception path only in the rare sweeps that have one.
// Same bytes out as the generic kernels.
// ---------------------------------------------------------------------------------------------
namespace xpfast {

constexpr uint32_t kOnes2 = 0x00010001u;

// The exponent fields are tested and rebased where they sit (bits 7..14 of each half of a word):
// with lift = 0x8000 - (base << 7) per half, field + lift has bit 15 set exactly when e >= base,
// carries e - base in bits 7..10 then, and never spills into the other half (field <= 0x7F80).
__device__ __forceinline__ uint32_t window_lift(uint32_t base)
{
    return 0x80008000u - ((base | (base << 16)) << 7);
}

// sign+mantissa bytes of four words -> two packed words (only bytes 0 and 2 of a t survive)
__device__ __forceinline__ uint2 sm_bytes(const uint4 &q)
{
    const uint32_t t0 = (q.x & 0x007F007Fu) | ((q.x >> 8) & 0xFF80FF80u);
    const uint32_t t1 = (q.y & 0x007F007Fu) | ((q.y >> 8) & 0xFF80FF80u);
    const uint32_t t2 = (q.z & 0x007F007Fu) | ((q.z >> 8) & 0xFF80FF80u);
    const uint32_t t3 = (q.w & 0x007F007Fu) | ((q.w >> 8) & 0xFF80FF80u);
    return make_uint2(__byte_perm(t0, t1, 0x6420), __byte_perm(t2, t3, 0x6420));
}

// code byte (two nibbles) of one word; exc gets bit 0 / bit 16 for elements below the window
__device__ __forceinline__ uint32_t code_byte(uint32_t w, uint32_t lift, uint32_t &exc)
{
    const uint32_t t = (w & 0x7F807F80u) + lift;
    exc = ((t >> 15) & kOnes2) ^ kOnes2;
    const uint32_t c2 = ((t >> 7) & 0x000F000Fu) | (exc * 15u);   // e - base (< 15), or 15
    return (c2 | (c2 >> 12)) & 0xFFu;
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v)
{
    const unsigned lane = lane_id();
#pragma unroll
    for (unsigned d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += y;
    }
    return v;
}

// number of nibbles equal to 0xF in a word
__device__ __forceinline__ uint32_t count_f_nibbles(uint32_t x, uint32_t &mask)
{
    uint32_t t = x & (x >> 1);
    t &= t >> 2;
    mask = t & 0x11111111u;
    return __popc(mask);
}

}  // namespace xpfast

template <int SWEEPS>
__global__ void __launch_bounds__(kXpThreads)
k_xp_measure_fast(const __grid_constant__ XpJob job)
{
    __shared__ uint32_t sh[kXpThreads / 32];
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk;
    const uint64_t total = job.n_chunks * slabs;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    for (uint64_t u = blockIdx.x; u < total; u += gridDim.x) {
        const uint64_t i = u / slabs;
        const uint32_t b = (uint32_t)(u - i * slabs);
        const unsigned char *src = xp_src(job, i, b, true);
        if (!src) {
            if (threadIdx.x == 0) {
                job.slab_size[u] = 16u + job.page_bytes;
                job.slab_info[u] = 0xFFFFu;
                job.slab_nexc[u] = 0;
            }
            continue;
        }
        const uint4 *s4 = reinterpret_cast<const uint4 *>(src) + (size_t)warp * SWEEPS * 32 + lane;
        uint4 q[SWEEPS];
#pragma unroll
        for (int s = 0; s < SWEEPS; ++s) q[s] = __ldcs(s4 + s * 32);
        // exponent fields stay where they are (bits 7..14 of each half); the largest per half
        // comes from the two-halves maximum instruction
        uint32_t m = 0;
#pragma unroll
        for (int s = 0; s < SWEEPS; ++s) {
            m = __vimax3_u16x2(m, q[s].x & 0x7F807F80u, q[s].y & 0x7F807F80u);
            m = __vimax3_u16x2(m, q[s].z & 0x7F807F80u, q[s].w & 0x7F807F80u);
        }
        m = max(m & 0xFFFFu, m >> 16);
        const uint32_t emax = block_max(m, sh) >> 7;
        const uint32_t base = emax > 14u ? emax - 14u : 0u;
        // bit 15 of field + lift says "in the window"; the bits are summed per half
        const uint32_t lift = xpfast::window_lift(base);
        uint32_t acc = 0;
#pragma unroll
        for (int s = 0; s < SWEEPS; ++s) {
            acc += (((q[s].x & 0x7F807F80u) + lift) & 0x80008000u) >> 15;
            acc += (((q[s].y & 0x7F807F80u) + lift) & 0x80008000u) >> 15;
            acc += (((q[s].z & 0x7F807F80u) + lift) & 0x80008000u) >> 15;
            acc += (((q[s].w & 0x7F807F80u) + lift) & 0x80008000u) >> 15;
        }
        const uint32_t in_win = (acc & 0xFFFFu) + (acc >> 16);
        const uint32_t cnt = block_sum(8u * SWEEPS - in_win, sh);
        if (threadIdx.x == 0) {
            const bool packed = cnt < job.n_elems / 2;
            job.slab_size[u] = packed ? round16u(16u + job.n_elems + job.n_elems / 2 + cnt)
                                      : 16u + 2u * job.n_elems;
            job.slab_info[u] = packed ? base : (1u << 8);
            job.slab_nexc[u] = packed ? cnt : 0u;
        }
    }
}

// dynamic shared memory: n_elems bytes (per-warp exception lists) 
template <int SWEEPS>
__global__ void __launch_bounds__(kXpThreads, SWEEPS <= 8 ? 4 : 2)
k_xp_pack_fast(const __grid_constant__ XpJob job)
{
    extern __shared__ __align__(16) unsigned char xp_smem[];
    __shared__ uint32_t warp_total[kXpThreads / 32];
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk, N = job.n_elems;
    const uint64_t total = job.n_chunks * slabs;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned char *my_list = xp_smem + (size_t)warp * (N / 8);
    for (uint64_t u = blockIdx.x; u < total; u += gridDim.x) {
        const uint64_t i = u / slabs;
        const uint32_t b = (uint32_t)(u - i * slabs);
        // The slab's loads go out first: where it lands (offsets, directory) is a chain of small
        // dependent loads of its own, which then overlaps with the data on its way.
        const unsigned char *src = xp_src(job, i, b, false);
        const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
        const uint32_t k_first = warp * SWEEPS * 32 + lane;       // this lane's first uint4
        uint4 qs[SWEEPS];                                         // all loads in flight at once
        if (src) {
#pragma unroll
            for (int s = 0; s < SWEEPS; ++s) qs[s] = __ldcs(s4 + k_first + s * 32);
        }
        const uint64_t off = job.chunk_off[i], csize = job.chunk_off[i + 1] - off;
        const uint32_t info = job.slab_info[u], size = job.slab_size[u];
        if (off + csize > job.blob_capacity || csize > 0xFFFFFFFFull) continue;
        const uint32_t *dir = reinterpret_cast<const uint32_t *>(job.blob + off);
        unsigned char *out = job.blob + off + dir[b];
        if (!src || info == 0xFFFFu) {
            uint4 *o4 = reinterpret_cast<uint4 *>(out);
            for (uint32_t k = threadIdx.x; k < size / 16; k += kXpThreads)
                o4[k] = k == 0 ? make_uint4(kXpMagic, 0, 1u << 8, size) : make_uint4(0, 0, 0, 0);
            continue;
        }
        const uint32_t mode = (info >> 8) & 0xFFu, base = info & 0xFFu;
        if (threadIdx.x == 0)
            *reinterpret_cast<uint4 *>(out) =
                make_uint4(kXpMagic, job.slab_nexc[u], base | (mode << 8), size);
        if (mode == 1) {
            uint4 *o4 = reinterpret_cast<uint4 *>(out + 16) + k_first;
#pragma unroll
            for (int s = 0; s < SWEEPS; ++s) __stcs(o4 + s * 32, qs[s]);
            continue;
        }
        unsigned char *sm = out + 16, *codes = sm + N, *exc = codes + N / 2;
        const uint32_t lift = xpfast::window_lift(base);
        uint32_t warp_count = 0;
#pragma unroll
        for (int s = 0; s < SWEEPS; ++s) {
            const uint32_t k = k_first + s * 32;
            const uint4 q = qs[s];
            uint32_t x0, x1, x2, x3;
            const uint32_t c32 = xpfast::code_byte(q.x, lift, x0) |
                                 (xpfast::code_byte(q.y, lift, x1) << 8) |
                                 (xpfast::code_byte(q.z, lift, x2) << 16) |
                                 (xpfast::code_byte(q.w, lift, x3) << 24);
            __stcs(reinterpret_cast<uint2 *>(sm + 8ull * k), xpfast::sm_bytes(q));
            __stcs(reinterpret_cast<uint32_t *>(codes + 4ull * k), c32);
            const uint32_t any = x0 | x1 | x2 | x3;
            if (__any_sync(0xFFFFFFFFu, any != 0)) {              // rare: exceptions in this sweep
                const uint32_t cnt = __popc(x0) + __popc(x1) + __popc(x2) + __popc(x3);
                const uint32_t incl = xpfast::warp_incl_scan(cnt);
                uint32_t at = warp_count + incl - cnt;
                const uint32_t w[4] = {q.x, q.y, q.z, q.w}, x[4] = {x0, x1, x2, x3};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (x[t] & 1u) my_list[at++] = (unsigned char)((w[t] >> 7) & 0xFFu);
                    if (x[t] >> 16) my_list[at++] = (unsigned char)((w[t] >> 23) & 0xFFu);
                }
                warp_count += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
        }
        if (lane == 0) warp_total[warp] = warp_count;
        __syncthreads();
        uint32_t before = 0, all = 0;
#pragma unroll
        for (unsigned w = 0; w < kXpThreads / 32; ++w) {
            const uint32_t t = warp_total[w];
            if (w < warp) before += t;
            all += t;
        }
        __syncwarp();
        for (uint32_t t = lane; t < warp_count; t += 32) exc[before + t] = my_list[t];
        const uint32_t used = 16u + N + N / 2 + all;
        if (threadIdx.x < size - used) out[used + threadIdx.x] = 0;
        __syncthreads();                                          // lists and totals are reused
    }
}

template <int SWEEPS>
__global__ void __launch_bounds__(kXpThreads)
k_xp_unpack_fast(const __grid_constant__ XpUnpackJob job, const __grid_constant__ ArenaTable ar)
{
    __shared__ uint32_t warp_total[kXpThreads / 32];
    const uint32_t slabs = 2u * job.n_layers * job.pages_per_chunk, n8 = job.n_elems >> 3, N = job.n_elems;
    const uint64_t total = *job.n_items_dev * slabs;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    for (uint64_t u = blockIdx.x; u < total; u += gridDim.x) {
        const uint64_t item = u / slabs;
        const uint32_t b = (uint32_t)(u - item * slabs);
        const uint32_t idx = __ldg(job.plan + item);
        if (idx == kSkip) continue;
        const uint4 r = __ldg(reinterpret_cast<const uint4 *>(job.recs + idx));
        const uint64_t roff = (uint64_t)r.z | ((uint64_t)r.w << 32);
        const unsigned char *blob = ar.base[r.x] + roff;
        const uint32_t csize = r.y;
        const uint32_t *dir = reinterpret_cast<const uint32_t *>(blob);
        const uint32_t d0 = __ldg(dir + b), d1 = __ldg(dir + b + 1);
        const uint32_t per_page = 2u * job.n_layers, pg = b / per_page, bb = b - pg * per_page;
        const uint64_t page = __ldg(job.page_table + (uint64_t)idx * job.pages_per_chunk + pg);
        const uint32_t buf = (bb & 1u) * job.n_layers + (bb >> 1);
        unsigned char *pool_buf = static_cast<unsigned char *>(job.kv_ptrs[buf]);
        bool ok = __ldg(dir + slabs) == csize && d0 >= job.dir_bytes && d0 <= d1 && d1 <= csize &&
                  (d0 & 15u) == 0 && d1 - d0 >= 16u;
        uint4 h = make_uint4(0, 0, 0, 0);
        if (ok) h = __ldg(reinterpret_cast<const uint4 *>(blob + d0));
        // The packed planes are fetched together with the header rather than after it: every
        // well-formed slab is at least 16 + 1.5 N bytes long, so whenever the directory grants
        // that much the loads stay inside the slab, whatever the header turns out to say.
        const unsigned char *in = blob + d0 + 16;
        const uint32_t k_first = warp * SWEEPS * 32 + lane;
        uint2 sms[SWEEPS];                                       // all loads in flight at once
        uint32_t cds[SWEEPS];
        const bool early = ok && d1 - d0 >= 16u + N + N / 2;
        if (early) {
#pragma unroll
            for (int s = 0; s < SWEEPS; ++s) {
                sms[s] = __ldcs(reinterpret_cast<const uint2 *>(in + 8ull * (k_first + s * 32)));
                cds[s] = __ldcs(reinterpret_cast<const uint32_t *>(in + N + 4ull * (k_first + s * 32)));
            }
        }
        const uint32_t mode = (h.z >> 8) & 0xFFu, base = h.z & 0xFFu, n_exc = h.y;
        ok = ok && h.x == kXpMagic && h.w == d1 - d0 &&
             ((mode == 1 && h.w == 16u + 2u * N) ||
              (mode == 0 && n_exc < N && h.w == round16u(16u + N + N / 2 + n_exc)));
        if (!ok) {
            if (threadIdx.x == 0) st_flag(job.st, LSMKV_ST_BAD_RECORD, idx);
            continue;
        }
        if (page >= job.num_pages) {
            if (threadIdx.x == 0 && bb == 0) st_flag(job.st, LSMKV_ST_BAD_PAGE, idx);
            continue;
        }
        if ((reinterpret_cast<uintptr_t>(pool_buf) & 15u) != 0) {
            if (threadIdx.x == 0) st_flag(job.st, LSMKV_ST_MISALIGNED, idx);
            continue;
        }
        uint4 *dst = reinterpret_cast<uint4 *>(pool_buf + page * (uint64_t)job.page_bytes);
        if (mode == 0 && !early) continue;                       // cannot happen: see above
        if (mode == 1) {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(in);
            for (uint32_t k = threadIdx.x; k < n8; k += kXpThreads) __stcs(dst + k, __ldcs(s4 + k));
            continue;
        }
        const unsigned char *exc = in + N + N / 2;
        const uint32_t base2 = base | (base << 16);
        // exceptions before this warp's segment (only when the slab has any)
        uint32_t at_warp = 0;
        if (n_exc) {                                             // uniform over the CTA
            uint32_t mine = 0, mask;
#pragma unroll
            for (int s = 0; s < SWEEPS; ++s) mine += xpfast::count_f_nibbles(cds[s], mask);
#pragma unroll
            for (int d = 16; d; d >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, d);
            if (lane == 0) warp_total[warp] = mine;
            __syncthreads();
            uint32_t all = 0;
#pragma unroll
            for (unsigned w = 0; w < kXpThreads / 32; ++w) {
                const uint32_t t = warp_total[w];
                if (w < warp) at_warp += t;
                all += t;
            }
            __syncthreads();
            if (all != n_exc) {                                  // header and codes disagree
                if (threadIdx.x == 0) st_flag(job.st, LSMKV_ST_BAD_RECORD, idx);
                continue;
            }
        }
#pragma unroll
        for (int s = 0; s < SWEEPS; ++s) {
            const uint32_t k = k_first + s * 32;
            const uint2 smv = sms[s];
            const uint32_t c32 = cds[s];
            uint32_t w[4];
            // word t: elements 2t, 2t+1
            const uint32_t s2[4] = {__byte_perm(smv.x, 0, 0x4140), __byte_perm(smv.x, 0, 0x4342),
                                    __byte_perm(smv.y, 0, 0x4140), __byte_perm(smv.y, 0, 0x4342)};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const uint32_t cb = (c32 >> (8 * t)) & 0xFFu;
                // (masked: code 15 + base may pass 255; those halves are patched below)
                const uint32_t e2 = (((cb & 0xFu) | ((cb & 0xF0u) << 12)) + base2) & 0x00FF00FFu;
                w[t] = ((s2[t] & 0x00800080u) << 8) | (e2 << 7) | (s2[t] & 0x007F007Fu);
            }
            if (n_exc) {
                uint32_t mask;
                const uint32_t cnt = xpfast::count_f_nibbles(c32, mask);
                if (__any_sync(0xFFFFFFFFu, cnt != 0)) {
                    const uint32_t incl = xpfast::warp_incl_scan(cnt);
                    uint32_t at = at_warp + incl - cnt;
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        if ((mask >> (4 * t)) & 1u) {
                            const uint32_t e = at < n_exc ? __ldg(exc + at) : 0u;
                            ++at;
                            const int sh16 = (t & 1) * 16;
                            w[t >> 1] = (w[t >> 1] & ~(0x7F80u << sh16)) | ((e & 0xFFu) << (7 + sh16));
                        }
                    }
                    at_warp += __shfl_sync(0xFFFFFFFFu, incl, 31);
                }
            }
            __stcs(dst + k, make_uint4(w[0], w[1], w[2], w[3]));
        }
    }
}

}  // namespace lsmkv
