// Index maintenance on the device: flush (write batch -> one sorted run) and compaction
// (several sorted runs -> one), the LSM steps between put_batch and probe.
//
// Both are built on one primitive, a stable pairwise merge by ranks: every element finds, with
// one binary search in the sibling segment, how many sibling elements precede it, and that
// count plus its own offset is its output position. A flush sorts tiles of 512 entries in shared
// memory and then merges bottom-up with that primitive (segments of 512, 1024, ... elements); a
// compaction concatenates the runs newest
// first and merges neighbouring segments level by level. Ties keep left-before-right, so equal
// keys stay in arrival order (flush: the last one survives) or in age order (compaction: the
// first, i.e. newest, survives). A flag/scan/scatter pass then drops the losers, gathers the
// records and pads the tail with all-ones keys, which compare above every real key.
#pragma once
#include "lsmkv_common.cuh"

namespace lsmkv {

struct Key4 { uint64_t w0, w1, w2, w3; };

__device__ __forceinline__ Key4 load_key(const lsmkv_key_t *p)
{
    const ulonglong2 a = reinterpret_cast<const ulonglong2 *>(p)[0];
    const ulonglong2 b = reinterpret_cast<const ulonglong2 *>(p)[1];
    return Key4{a.x, a.y, b.x, b.y};
}

__device__ __forceinline__ void store_key4(lsmkv_key_t *p, const Key4 &k)
{
    reinterpret_cast<ulonglong2 *>(p)[0] = make_ulonglong2(k.w0, k.w1);
    reinterpret_cast<ulonglong2 *>(p)[1] = make_ulonglong2(k.w2, k.w3);
}

__device__ __forceinline__ bool key_less(const Key4 &a, const Key4 &b)
{
    if (a.w0 != b.w0) return a.w0 < b.w0;
    if (a.w1 != b.w1) return a.w1 < b.w1;
    if (a.w2 != b.w2) return a.w2 < b.w2;
    return a.w3 < b.w3;
}

__device__ __forceinline__ bool key_eq(const Key4 &a, const Key4 &b)
{
    return a.w0 == b.w0 && a.w1 == b.w1 && a.w2 == b.w2 && a.w3 == b.w3;
}

// Segment boundaries of one merge level when they are not uniform (compaction).
struct SegTable {
    uint64_t start[LSMKV_MAX_RUNS + 2];
    uint32_t n_seg;      // 0 = uniform segments of `width` elements
};

// One merge level: segments (2p, 2p+1) of src are merged into dst. idx carries where each
// element came from (src_idx == nullptr: identity).
__global__ void __launch_bounds__(256)
k_merge_level(const lsmkv_key_t *__restrict__ src, const uint32_t *__restrict__ src_idx,
              lsmkv_key_t *__restrict__ dst, uint32_t *__restrict__ dst_idx, uint64_t n,
              uint64_t width, const __grid_constant__ SegTable segs)
{
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (uint64_t)gridDim.x * blockDim.x) {
        uint64_t base, mid, end;
        if (segs.n_seg == 0) {
            base = i / (2 * width) * (2 * width);
            mid = min(n, base + width);
            end = min(n, base + 2 * width);
        } else {
            uint32_t s = 0;
            while (s + 1 < segs.n_seg && segs.start[s + 1] <= i) ++s;
            const uint32_t p = s & ~1u;
            base = segs.start[p];
            mid = segs.start[p + 1];
            end = p + 2 <= segs.n_seg ? segs.start[p + 2] : mid;
        }
        const Key4 x = load_key(src + i);
        uint64_t rank;
        if (i < mid) {                       // left element: sibling elements strictly below it
            uint64_t lo = mid, hi = end;
            while (lo < hi) {
                const uint64_t m = lo + ((hi - lo) >> 1);
                if (key_less(load_key(src + m), x)) lo = m + 1; else hi = m;
            }
            rank = (i - base) + (lo - mid);
        } else {                             // right element: sibling elements below or equal
            uint64_t lo = base, hi = mid;
            while (lo < hi) {
                const uint64_t m = lo + ((hi - lo) >> 1);
                if (key_less(x, load_key(src + m))) hi = m; else lo = m + 1;
            }
            rank = (i - mid) + (lo - base);
        }
        store_key4(dst + base + rank, x);
        dst_idx[base + rank] = src_idx ? src_idx[i] : (uint32_t)i;
    }
}

// First step of a flush: every CTA sorts one tile of kSortTile entries in shared memory with a
// bitonic network on (key, arrival index) -- the index makes the order total, so the result is
// the stable order -- and the merge levels start from segments of kSortTile instead of 1.
constexpr int kSortTile = 512;

__device__ __forceinline__ bool entry_less(const Key4 &a, uint32_t ia, const Key4 &b, uint32_t ib)
{
    if (a.w0 != b.w0) return a.w0 < b.w0;
    if (a.w1 != b.w1) return a.w1 < b.w1;
    if (a.w2 != b.w2) return a.w2 < b.w2;
    if (a.w3 != b.w3) return a.w3 < b.w3;
    return ia < ib;
}

__global__ void __launch_bounds__(kSortTile / 2)
k_tile_sort(const lsmkv_key_t *__restrict__ src, lsmkv_key_t *__restrict__ dst,
            uint32_t *__restrict__ dst_idx, uint64_t n)
{
    // one array per key word: neighbouring threads touch neighbouring words (no bank conflicts)
    __shared__ uint64_t s0[kSortTile], s1[kSortTile], s2[kSortTile], s3[kSortTile];
    __shared__ uint32_t si[kSortTile];
    const uint64_t tile0 = (uint64_t)blockIdx.x * kSortTile;
    for (unsigned t = threadIdx.x; t < kSortTile; t += blockDim.x) {
        const uint64_t i = tile0 + t;
        Key4 k{~0ull, ~0ull, ~0ull, ~0ull};                  // beyond the end: sorts last
        uint32_t id = 0xFFFFFFFFu;
        if (i < n) { k = load_key(src + i); id = (uint32_t)i; }
        s0[t] = k.w0; s1[t] = k.w1; s2[t] = k.w2; s3[t] = k.w3; si[t] = id;
    }
    __syncthreads();
    for (unsigned k = 2; k <= kSortTile; k <<= 1) {
        for (unsigned j = k >> 1; j > 0; j >>= 1) {
            const unsigned t = threadIdx.x;
            const unsigned i = 2 * t - (t & (j - 1)), l = i + j;
            const bool up = (i & k) == 0;
            const Key4 a{s0[i], s1[i], s2[i], s3[i]}, b{s0[l], s1[l], s2[l], s3[l]};
            const uint32_t ia = si[i], ib = si[l];
            const bool swap = up ? entry_less(b, ib, a, ia) : entry_less(a, ia, b, ib);
            if (swap) {
                s0[i] = b.w0; s1[i] = b.w1; s2[i] = b.w2; s3[i] = b.w3; si[i] = ib;
                s0[l] = a.w0; s1[l] = a.w1; s2[l] = a.w2; s3[l] = a.w3; si[l] = ia;
            }
            __syncthreads();
        }
    }
    for (unsigned t = threadIdx.x; t < kSortTile; t += blockDim.x) {
        const uint64_t i = tile0 + t;
        if (i < n) {
            store_key4(dst + i, Key4{s0[t], s1[t], s2[t], s3[t]});
            dst_idx[i] = si[t];
        }
    }
}

constexpr int kScanBlock = 1024;

__device__ __forceinline__ bool survives(const lsmkv_key_t *keys, uint64_t i, uint64_t n,
                                         int keep_last)
{
    const Key4 x = load_key(keys + i);
    if (keep_last) return i + 1 == n || !key_eq(x, load_key(keys + i + 1));
    return i == 0 || !key_eq(x, load_key(keys + i - 1));
}

// survivors per block of kScanBlock sorted elements
__global__ void __launch_bounds__(kScanBlock)
k_dedupe_count(const lsmkv_key_t *__restrict__ keys, uint64_t n, int keep_last,
               uint64_t *__restrict__ block_count)
{
    const uint64_t i = (uint64_t)blockIdx.x * kScanBlock + threadIdx.x;
    const int keep = i < n && survives(keys, i, n, keep_last);
    const int c = __syncthreads_count(keep);
    if (threadIdx.x == 0) block_count[blockIdx.x] = (uint64_t)c;
}

// in-place exclusive scan of the block counts (one CTA); total -> *n_out
__global__ void __launch_bounds__(1024)
k_scan_blocks(uint64_t *__restrict__ block_count, uint64_t n_blocks, uint64_t *__restrict__ n_out)
{
    __shared__ uint64_t warp_sum[32];
    __shared__ uint64_t carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    for (uint64_t base = 0; base < n_blocks; base += blockDim.x) {
        const uint64_t b = base + threadIdx.x;
        const uint64_t h = b < n_blocks ? block_count[b] : 0;
        uint64_t x = h;
#pragma unroll
        for (unsigned d = 1; d < 32; d <<= 1) {
            const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, x, d);
            if (lane >= d) x += y;
        }
        if (lane == 31) warp_sum[warp] = x;
        __syncthreads();
        if (warp == 0) {
            uint64_t w = warp_sum[lane];
#pragma unroll
            for (unsigned d = 1; d < 32; d <<= 1) {
                const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, w, d);
                if (lane >= d) w += y;
            }
            warp_sum[lane] = w;
        }
        __syncthreads();
        const uint64_t before = carry_s + (warp ? warp_sum[warp - 1] : 0) + (x - h);
        if (b < n_blocks) block_count[b] = before;
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry_s = before + h;
        __syncthreads();
    }
    if (threadIdx.x == 0) *n_out = carry_s;
}

// survivors move to their final position with their record; the tail [n_out, n) is padded
__global__ void __launch_bounds__(kScanBlock)
k_dedupe_scatter(const lsmkv_key_t *__restrict__ keys, const uint32_t *__restrict__ idx,
                 const lsmkv_val_t *__restrict__ vals_in, uint64_t n, int keep_last,
                 const uint64_t *__restrict__ block_offset, const uint64_t *__restrict__ n_out,
                 lsmkv_key_t *__restrict__ keys_out, lsmkv_val_t *__restrict__ vals_out)
{
    __shared__ uint32_t warp_cnt[32];
    const uint64_t i = (uint64_t)blockIdx.x * kScanBlock + threadIdx.x;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    const bool keep = i < n && survives(keys, i, n, keep_last);
    const unsigned m = __ballot_sync(0xFFFFFFFFu, keep);
    if (lane == 0) warp_cnt[warp] = __popc(m);
    __syncthreads();
    uint32_t before = 0;
    for (unsigned w = 0; w < warp; ++w) before += warp_cnt[w];
    if (keep) {
        const uint64_t o = block_offset[blockIdx.x] + before + __popc(m & ((1u << lane) - 1u));
        store_key4(keys_out + o, load_key(keys + i));
        reinterpret_cast<uint4 *>(vals_out)[o] =
            __ldg(reinterpret_cast<const uint4 *>(vals_in) + idx[i]);
    }
    if (i < n && i >= *n_out) {              // padding: above every real key, never matched
        store_key4(keys_out + i, Key4{~0ull, ~0ull, ~0ull, ~0ull});
        reinterpret_cast<uint4 *>(vals_out)[i] = make_uint4(0, 0, 0, 0);
    }
}

// Tensor-file merging: records of a merged file get their new file id and shifted offset.
constexpr int kMaxReloc = 64;
struct RelocTable {
    uint32_t old_file[kMaxReloc], new_file[kMaxReloc];
    uint64_t delta[kMaxReloc];
    uint32_t n;
};

__global__ void __launch_bounds__(256)
k_relocate_records(lsmkv_val_t *__restrict__ vals, uint64_t n, const __grid_constant__ RelocTable tab,
                   unsigned long long *__restrict__ changed_out)
{
    unsigned long long mine = 0;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (uint64_t)gridDim.x * blockDim.x) {
        uint4 r = reinterpret_cast<uint4 *>(vals)[i];
        for (uint32_t t = 0; t < tab.n; ++t) {
            if (r.x == tab.old_file[t]) {                    // first matching entry applies
                const uint64_t off = ((uint64_t)r.z | ((uint64_t)r.w << 32)) + tab.delta[t];
                r.x = tab.new_file[t];
                r.z = (uint32_t)off;
                r.w = (uint32_t)(off >> 32);
                reinterpret_cast<uint4 *>(vals)[i] = r;
                ++mine;
                break;
            }
        }
    }
#pragma unroll
    for (unsigned d = 16; d; d >>= 1) mine += __shfl_down_sync(0xFFFFFFFFu, mine, d);
    if (lane_id() == 0 && mine && changed_out) atomicAdd(changed_out, mine);
}

}  // namespace lsmkv
