// Batched longest-cached-prefix probe.
//
// A CTA takes one query at a time, longest queries first (a batch of no more queries than CTAs fit
// on the GPU, all runs with hash indexes: block b takes query b). Its W warps hash 32*W
// consecutive chunks per round (each warp one 32-chunk block; the block digests are chained
// through shared memory; the very first round is one warp's 32 chunks), every lane looks its key
// up in the runs newest -> oldest, a warp ballot finds each warp's first miss and a shared-memory
// minimum gives the query's. The hit length is the number of leading chunks that were all found
// (first-miss rule); hashing stops at the round of the first miss unless the caller asked for all
// keys.
//
// Lookups use fence pointers: the chunk index j is the most significant key field, so in every
// run the keys of one j form a contiguous bucket. k_run_dir finds all bucket boundaries of all
// runs up front (one binary search per boundary). Inside a bucket keys are ordered by the
// digest w1, which is uniform on [0, 2^61), so the position is interpolated and pinned by a
// branch-free binary search over a small window around the guess: ~6 dependent 8-byte loads
// per run instead of ~20 32-byte ones, with identical control flow across the lanes of a warp,
// the searches of four runs advancing together so that their loads overlap. When every run
// brings a hash index (k_hidx_build) no search happens at all: one 32-byte bucket per run says
// where the key is, if anywhere.
#pragma once
#include "lsmkv_keys.cuh"

namespace lsmkv {

struct RunTable {
    const lsmkv_key_t *keys[LSMKV_MAX_RUNS];
    const lsmkv_val_t *vals[LSMKV_MAX_RUNS];
    uint64_t n[LSMKV_MAX_RUNS];
    const uint32_t *bloom[LSMKV_MAX_RUNS];     // optional Bloom filter, 8 words per block
    uint64_t bloom_blocks[LSMKV_MAX_RUNS];
    const uint32_t *hidx[LSMKV_MAX_RUNS];      // optional hash index, 8 slots per bucket
    uint64_t hidx_buckets[LSMKV_MAX_RUNS];
};

constexpr uint64_t kDigestLimit = 1ull << 61;  // digests are < 2^61 - 1; padding keys are not

// Bloom filter of a run: block floor(w1 * n_blocks / 2^61), six bits at (w2 >> 8i) & 255.
__global__ void __launch_bounds__(256)
k_bloom_build(const lsmkv_key_t *__restrict__ keys, uint64_t n, uint32_t *__restrict__ bloom,
              uint64_t n_blocks)
{
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const ulonglong2 a = *reinterpret_cast<const ulonglong2 *>(
            reinterpret_cast<const unsigned long long *>(keys + i) + 1);   // w1, w2
        if (a.x >= kDigestLimit) continue;                                  // padding entry
        uint32_t *blk = bloom + 8ull * __umul64hi(a.x << 3, n_blocks);
#pragma unroll
        for (int t = 0; t < 6; ++t) {
            const uint32_t p = (uint32_t)(a.y >> (8 * t)) & 255u;
            atomicOr(blk + (p >> 5), 1u << (p & 31u));
        }
    }
}

__device__ __forceinline__ bool bloom_may_contain(const uint32_t *bloom, uint64_t n_blocks,
                                                  const ChunkKey &k)
{
    const uint32_t *blk = bloom + 8ull * __umul64hi(k.w1 << 3, n_blocks);
    bool ok = true;
#pragma unroll
    for (int t = 0; t < 6; ++t) {
        const uint32_t p = (uint32_t)(k.w2 >> (8 * t)) & 255u;
        ok = ok && ((__ldg(blk + (p >> 5)) >> (p & 31u)) & 1u);
    }
    return ok;
}

__device__ __forceinline__ uint64_t key_w(const lsmkv_key_t *e, int i)
{
    return __ldg(reinterpret_cast<const unsigned long long *>(e) + i);
}

// first index whose w0 >= w0_target
__device__ __forceinline__ uint64_t lower_bound_w0(const lsmkv_key_t *keys, uint64_t n,
                                                   uint64_t w0_target)
{
    uint64_t lo = 0, hi = n;
    while (lo < hi) {
        const uint64_t mid = lo + ((hi - lo) >> 1);
        if (key_w(keys + mid, 0) < w0_target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Length class of a query with nch chunks: 0..3 for itself, then four classes per power of two.
constexpr int kLenClasses = 128;
__device__ __forceinline__ uint32_t len_class(uint64_t nch)
{
    if (nch < 4) return (uint32_t)nch;
    if (nch > 0xFFFFFFFFull) return kLenClasses - 1;
    const uint32_t n = (uint32_t)nch, e = 31u - __clz(n);
    return 4u * e + ((n >> (e - 2u)) & 3u) - 4u;           // e >= 2: 4..123
}

// order[0..n_query) = the queries by descending length class (counting sort by one CTA; the
// order inside a class is whatever the atomics give, results do not depend on it). The probe
// hands queries out in this order, so the longest ones -- whose rounds run one after another in
// one CTA -- start first and the short ones fill the gaps at the end.
__device__ __forceinline__ void order_queries(uint32_t n_query, const uint64_t *__restrict__ seq_off,
                                              uint32_t C, uint32_t *__restrict__ order)
{
    __shared__ uint32_t s_cnt[kLenClasses];
    for (uint32_t t = threadIdx.x; t < kLenClasses; t += blockDim.x) s_cnt[t] = 0;
    __syncthreads();
    // four queries per thread at a time, their offsets asked for together: an atomic between
    // two loads would make every load wait for the one before it
    constexpr int kPer = 4;
    for (uint32_t q0 = 0; q0 < n_query; q0 += kPer * blockDim.x) {
        uint32_t cls[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const uint32_t q = q0 + (uint32_t)u * blockDim.x + threadIdx.x;
            cls[u] = ~0u;
            if (q < n_query) {
                const uint64_t s0 = seq_off[q], s1 = seq_off[q + 1];
                cls[u] = len_class(s1 >= s0 ? (s1 - s0) / C : 0);
            }
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u)
            if (cls[u] != ~0u) atomicAdd(&s_cnt[cls[u]], 1u);
    }
    __syncthreads();
    if (threadIdx.x < 32) {              // counts -> first slot of every class, longest class first
        static_assert(kLenClasses == 4 * 32, "four classes per lane");
        const unsigned lane = threadIdx.x;
        uint32_t n[4], tot = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            n[u] = s_cnt[kLenClasses - 1 - (4 * (int)lane + u)];
            tot += n[u];
        }
        uint32_t incl = tot;
#pragma unroll
        for (unsigned d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += v;
        }
        uint32_t at = incl - tot;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            s_cnt[kLenClasses - 1 - (4 * (int)lane + u)] = at;
            at += n[u];
        }
    }
    __syncthreads();
    for (uint32_t q0 = 0; q0 < n_query; q0 += kPer * blockDim.x) {
        uint32_t cls[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const uint32_t q = q0 + (uint32_t)u * blockDim.x + threadIdx.x;
            cls[u] = ~0u;
            if (q < n_query) {
                const uint64_t s0 = seq_off[q], s1 = seq_off[q + 1];
                cls[u] = len_class(s1 >= s0 ? (s1 - s0) / C : 0);
            }
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u)
            if (cls[u] != ~0u)
                order[atomicAdd(&s_cnt[cls[u]], 1u)] = q0 + (uint32_t)u * blockDim.x + threadIdx.x;
    }
}

// dir[r * stride + j] = first index of run r whose chunk index is >= j (same namespace),
// for j = 0..jcap (stride = jcap + 1).
// Also resets the probe's work counter (*next_query) for the launch that follows, and its last
// block writes the hand-out order of the queries when `order` is given.
__global__ void __launch_bounds__(1024)
k_run_dir(const __grid_constant__ RunTable rt, uint32_t n_runs, uint32_t ns, uint32_t jcap,
          uint64_t *__restrict__ dir, unsigned long long *next_query, uint32_t n_query,
          const uint64_t *__restrict__ seq_off, uint32_t C, uint32_t *__restrict__ order)
{
    if (blockIdx.x == 0 && threadIdx.x == 0) *next_query = 0;
    if (order && blockIdx.x == gridDim.x - 1) order_queries(n_query, seq_off, C, order);
    const uint64_t stride = (uint64_t)jcap + 1;
    const uint64_t total = (uint64_t)n_runs * stride;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const uint32_t r = (uint32_t)(i / stride);
        const uint64_t j = i - (uint64_t)r * stride;
        dir[i] = lower_bound_w0(rt.keys[r], rt.n[r], ((uint64_t)ns << 32) + j);
    }
}

// compare (w1,w2,w3) of entry e with the key; w0 is known to be equal inside a bucket
__device__ __forceinline__ int bucket_cmp(const lsmkv_key_t *e, const ChunkKey &k)
{
    const uint64_t w1 = key_w(e, 1);
    if (w1 != k.w1) return w1 < k.w1 ? -1 : 1;
    const uint64_t w2 = key_w(e, 2);
    if (w2 != k.w2) return w2 < k.w2 ? -1 : 1;
    const uint64_t w3 = key_w(e, 3);
    if (w3 != k.w3) return w3 < k.w3 ? -1 : 1;
    return 0;
}

// Plain exact binary search over [a, b) of a bucket with the full key (slow path).
__device__ __noinline__ uint64_t bucket_find_exact(const lsmkv_key_t *keys, uint64_t a, uint64_t b,
                                                   const ChunkKey k)   // by value: in registers
{
    while (a < b) {
        const uint64_t mid = a + ((b - a) >> 1);
        const int c = bucket_cmp(keys + mid, k);
        if (c == 0) return mid;
        if (c < 0) a = mid + 1; else b = mid;
    }
    return ~0ull;
}

// Point lookup, newest run first; the first run that holds the key decides.
//
// Inside a bucket the digest w1 is uniform, so the key's rank is close to w1 * cnt / 2^61
// (standard deviation <= sqrt(cnt) / 2). A branch-free binary search on w1 over a window of about
// +-2.5 standard deviations around that guess pins it with ~log2(window) loads. Whenever the
// window cannot prove presence or absence (the answer falls on a window edge, or digests tie) a
// plain search of the whole bucket with the full key decides, so the result is exact in every
// case.
//
// Each search is a chain of dependent loads that hit L2 at best, and a warp has nothing else to
// do while it waits. The runs are therefore searched kLookupGroup at a time in lock step: the
// bucket bounds of the whole group are fetched together, then every step of the window search
// issues one load per run before any of them is needed, so a group costs the latency of one
// chain. The answers are then taken in age order, which keeps the first-match rule.
constexpr int kLookupGroup = 4;

__device__ __forceinline__ bool lookup_runs(const RunTable &rt, uint32_t n_runs,
                                            const uint64_t *__restrict__ dir, uint32_t jcap,
                                            const ChunkKey &k, uint4 &val)
{
    const uint64_t j = k.w0 & 0xFFFFFFFFull;
    const uint64_t stride = (uint64_t)jcap + 1;
    for (uint32_t r0 = 0; r0 < n_runs; r0 += kLookupGroup) {
        uint64_t lo[kLookupGroup], hi[kLookupGroup];
#pragma unroll
        for (int g = 0; g < kLookupGroup; ++g) {
            const uint32_t r = r0 + g;
            lo[g] = 0;
            hi[g] = 0;
            if (r < n_runs) {                              // uniform over the grid
                if (j < jcap) {
                    lo[g] = __ldg(dir + r * stride + j);
                    hi[g] = __ldg(dir + r * stride + j + 1);
                } else {                                   // beyond the directory: find the bucket
                    lo[g] = lower_bound_w0(rt.keys[r], rt.n[r], k.w0);
                    hi[g] = lower_bound_w0(rt.keys[r], rt.n[r], k.w0 + 1);
                }
            }
        }
        // window of every run: [a0, e0) inside its bucket, n = entries still in play (0 = the
        // run cannot hold the key, or the bucket is too large for 32-bit positions)
        const unsigned long long *w1p[kLookupGroup];
        uint32_t pos[kLookupGroup], n[kLookupGroup], a0[kLookupGroup], e0[kLookupGroup];
        uint32_t n_max = 0;
#pragma unroll
        for (int g = 0; g < kLookupGroup; ++g) {
            const uint32_t r = r0 + g;
            uint64_t cnt64 = hi[g] - lo[g];
            if (r < n_runs && cnt64 && rt.bloom[r] &&
                !bloom_may_contain(rt.bloom[r], rt.bloom_blocks[r], k))
                cnt64 = 0;                                 // ruled out by the filter
            w1p[g] = r < n_runs
                         ? reinterpret_cast<const unsigned long long *>(rt.keys[r] + lo[g]) + 1
                         : nullptr;
            uint32_t a = 0, m = 0;
            if (cnt64 && cnt64 < 0x40000000ull) {
                const uint32_t cnt = (uint32_t)cnt64;
                m = cnt;
                if (cnt > 16) {
                    const uint32_t gs = (uint32_t)__umul64hi(k.w1 << 3, cnt64);   // w1 * cnt / 2^61
                    const uint32_t R = 4u + (uint32_t)(1.25f * sqrtf((float)cnt));
                    a = gs > R ? gs - R : 0u;
                    m = min(cnt, gs + R + 1u) - a;
                }
            }
            if (cnt64 == 0) hi[g] = lo[g];                 // remembered as "empty"
            a0[g] = a;
            e0[g] = a + m;
            pos[g] = a;
            n[g] = m;
            n_max = max(n_max, m);
        }
        // lock-step search: pos = last index in the window with w1 <= target
        while (n_max > 1) {
#pragma unroll
            for (int g = 0; g < kLookupGroup; ++g) {
                if (n[g] > 1) {
                    const uint32_t half = n[g] >> 1;
                    const uint64_t v = __ldg(w1p[g] + 4ull * (pos[g] + half));
                    pos[g] = v <= k.w1 ? pos[g] + half : pos[g];
                    n[g] -= half;
                }
            }
            n_max -= n_max >> 1;
        }
        uint64_t v[kLookupGroup];
#pragma unroll
        for (int g = 0; g < kLookupGroup; ++g)
            v[g] = n[g] ? __ldg(w1p[g] + 4ull * pos[g]) : 0;
        // answers in age order
#pragma unroll
        for (int g = 0; g < kLookupGroup; ++g) {
            const uint32_t r = r0 + g;
            if (r >= n_runs || hi[g] == lo[g]) continue;
            const lsmkv_key_t *keys = rt.keys[r];
            uint64_t at = ~0ull;
            if (n[g] == 0) {                               // huge bucket
                at = bucket_find_exact(keys, lo[g], hi[g], k);
            } else if (v[g] == k.w1) {
                const ulonglong2 w23 = __ldg(reinterpret_cast<const ulonglong2 *>(
                    reinterpret_cast<const unsigned long long *>(keys + lo[g] + pos[g]) + 2));
                if (w23.x == k.w2 && w23.y == k.w3) at = lo[g] + pos[g];
                else at = bucket_find_exact(keys, lo[g], hi[g], k);          // digest tie: be exact
            } else if (v[g] > k.w1) {                      // only possible at pos == a0
                if (a0[g] > 0) at = bucket_find_exact(keys, lo[g], lo[g] + a0[g], k);
            } else if (pos[g] + 1 == e0[g] && lo[g] + e0[g] < hi[g]) {
                // below the target at the window's last entry, and the bucket goes on
                at = bucket_find_exact(keys, lo[g] + e0[g], hi[g], k);
            }
            if (at != ~0ull) {
                val = __ldg(reinterpret_cast<const uint4 *>(rt.vals[r] + at));
                return true;
            }
        }
    }
    return false;
}

// ---------------------------------------------------------------------------------------------
// Hash index of a run: a table of 32-byte buckets of eight 4-byte slots that maps a key to its
// position in the sorted run. A slot is 0 (empty) or (w2 & 0xFF) << 24 | (position + 1). A key's
// home bucket is floor(w1 * n_buckets / 2^61); it sits in the first slot that was free when it
// was inserted, scanning the home bucket's slots 0..7 and then the following buckets (wrapping).
// Slots never empty again, so a lookup that scans in the same order may stop at the first empty
// slot: the key is not in the run. With n_buckets = ceil(n / 2) a bucket holds two keys on
// average and all eight slots of a bucket are taken for about one key in a thousand, so nearly
// every lookup is one 32-byte load, plus the key and record of the one slot whose tag matches.
// The sorted run stays what it is (merges and range scans use it); the table only replaces the
// binary search of a point lookup.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kHidxSlots = 8;
constexpr uint64_t kHidxMaxKeys = (1ull << 24) - 2;        // position + 1 must fit 24 bits

__device__ __forceinline__ uint64_t hidx_home(uint64_t w1, uint64_t n_buckets)
{
    return __umul64hi(w1 << 3, n_buckets);
}

__global__ void __launch_bounds__(256)
k_hidx_build(const lsmkv_key_t *__restrict__ keys, uint64_t n, uint32_t *__restrict__ hidx,
             uint64_t n_buckets)
{
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const ulonglong2 a = *reinterpret_cast<const ulonglong2 *>(
            reinterpret_cast<const unsigned long long *>(keys + i) + 1);   // w1, w2
        if (a.x >= kDigestLimit) continue;                                  // padding entry
        const uint32_t entry = (((uint32_t)a.y & 0xFFu) << 24) | (uint32_t)(i + 1);
        uint64_t b = hidx_home(a.x, n_buckets);
        bool placed = false;
        for (uint64_t it = 0; it < n_buckets && !placed; ++it) {            // slots >= 4 n: ends
            for (uint32_t t = 0; t < kHidxSlots && !placed; ++t)
                placed = atomicCAS(hidx + kHidxSlots * b + t, 0u, entry) == 0u;
            b = b + 1 == n_buckets ? 0 : b + 1;
        }
    }
}

__device__ __forceinline__ bool key_equals(const lsmkv_key_t *e, const ChunkKey &k)
{
    const ulonglong2 *p = reinterpret_cast<const ulonglong2 *>(e);
    const ulonglong2 a = __ldg(p), b = __ldg(p + 1);
    return a.x == k.w0 && a.y == k.w1 && b.x == k.w2 && b.y == k.w3;
}

// The lookup rule, slot by slot (any table, any fill). Returns the position or ~0.
__device__ __noinline__ uint64_t hidx_find(const uint32_t *hidx, uint64_t n_buckets,
                                           const lsmkv_key_t *keys, uint64_t n, const ChunkKey k)
{                                                          // (the key by value: in registers)
    const uint32_t tag = (uint32_t)k.w2 & 0xFFu;
    uint64_t b = hidx_home(k.w1, n_buckets);
    for (uint64_t it = 0; it < n_buckets; ++it) {
        for (uint32_t t = 0; t < kHidxSlots; ++t) {
            const uint32_t w = __ldg(hidx + kHidxSlots * b + t);
            if (w == 0) return ~0ull;
            const uint64_t at = (uint64_t)(w & 0xFFFFFFu) - 1;
            if ((w >> 24) == tag && at < n && key_equals(keys + at, k)) return at;
        }
        b = b + 1 == n_buckets ? 0 : b + 1;
    }
    return ~0ull;
}

// One 32-byte load (the address must be 32-byte aligned): a whole bucket, or a whole key.
__device__ __forceinline__ void ldg256(const void *p, uint4 &lo, uint4 &hi)
{
    asm("ld.global.nc.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z),
          "=r"(hi.w)
        : "l"(p));
}

// A bucket or a key: one load when the caller vouches for 32-byte alignment (WIDE), else two.
template <bool WIDE>
__device__ __forceinline__ void load32(const void *p, uint4 &lo, uint4 &hi)
{
    if (WIDE) {
        ldg256(p, lo, hi);
    } else {
        lo = __ldg(reinterpret_cast<const uint4 *>(p));
        hi = __ldg(reinterpret_cast<const uint4 *>(p) + 1);
    }
}

// What a bucket says about a key from slot `from` on: the first slot that is empty or carries the
// key's tag. Returns the position + 1 a tag match names (0: none) and sets `slot` to where the
// scan stopped (kHidxSlots: every slot from `from` on holds another tag).
__device__ __forceinline__ uint32_t bucket_stop(const uint4 &lo, const uint4 &hi, uint32_t tag,
                                                uint32_t from, uint32_t &slot)
{
    const uint32_t w[kHidxSlots] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    uint32_t cand = 0;
    slot = kHidxSlots;
#pragma unroll
    for (int t = (int)kHidxSlots - 1; t >= 0; --t) {       // the lowest slot wins
        if ((uint32_t)t >= from && (w[t] == 0 || (w[t] >> 24) == tag)) {
            cand = w[t] & 0xFFFFFFu;
            slot = (uint32_t)t;
        }
    }
    return cand;
}

// Point lookup through the hash indexes, newest run first. The home buckets of kLookupGroup
// runs are fetched together; then every lane fetches key and record of its newest candidate,
// whichever run that is in, so the lanes of a warp advance together: as a rule two dependent
// loads per group. A lane whose candidate is another key with the same tag (one lookup in a
// hundred) goes on behind it in the same bucket, read again from L1, and from there to its next
// run; a bucket without any answer (every slot taken by other tags) goes slot by slot.
// WIDE: every run's index and key array start on a 32-byte boundary.
template <bool WIDE>
__device__ __forceinline__ bool lookup_runs_hash(const RunTable &rt, uint32_t n_runs,
                                                 const ChunkKey &k, uint4 &val)
{
    const uint32_t tag = (uint32_t)k.w2 & 0xFFu;
    for (uint32_t r0 = 0; r0 < n_runs; r0 += kLookupGroup) {
        uint4 lo[kLookupGroup], hi[kLookupGroup];
#pragma unroll
        for (int g = 0; g < kLookupGroup; ++g) {
            const uint32_t r = r0 + g;
            lo[g] = make_uint4(0, 0, 0, 0);
            hi[g] = lo[g];
            if (r < n_runs && rt.n[r]) {
                const uint4 *bkt = reinterpret_cast<const uint4 *>(
                    rt.hidx[r] + kHidxSlots * hidx_home(k.w1, rt.hidx_buckets[r]));
                load32<WIDE>(bkt, lo[g], hi[g]);
            }
        }
        // per run: cand = position + 1 of the first tag match (0: none); todo bit g = the run may
        // still hold the key (a candidate, or a bucket that cannot say); slots = 4 bits per run,
        // where the scan stopped
        uint32_t cand[kLookupGroup], todo = 0, slots = 0;
#pragma unroll
        for (int g = 0; g < kLookupGroup; ++g) {
            uint32_t slot;
            cand[g] = bucket_stop(lo[g], hi[g], tag, 0, slot);
            const bool live = r0 + g < n_runs && rt.n[r0 + g] != 0;
            if (live && cand[g] > rt.n[r0 + g]) {           // not a position of this run
                cand[g] = 0;
                slot = kHidxSlots;
            }
            if (live && (cand[g] != 0 || slot == kHidxSlots)) todo |= 1u << g;
            slots |= slot << (4 * g);
        }
        while (todo) {                                       // newest run first
            const int g = __ffs((int)todo) - 1;
            const uint32_t r = r0 + (uint32_t)g;
            const uint32_t c = g == 0 ? cand[0] : g == 1 ? cand[1] : g == 2 ? cand[2] : cand[3];
            if (c) {
                uint4 k0, k1;
                load32<WIDE>(rt.keys[r] + (c - 1), k0, k1);
                const uint4 rec = __ldg(reinterpret_cast<const uint4 *>(rt.vals[r] + (c - 1)));
                if (k0.x == (uint32_t)k.w0 && k0.y == (uint32_t)(k.w0 >> 32) &&
                    k0.z == (uint32_t)k.w1 && k0.w == (uint32_t)(k.w1 >> 32) &&
                    k1.x == (uint32_t)k.w2 && k1.y == (uint32_t)(k.w2 >> 32) &&
                    k1.z == (uint32_t)k.w3 && k1.w == (uint32_t)(k.w3 >> 32)) {
                    val = rec;
                    return true;
                }
                // another key with the same tag: what does the rest of the bucket say
                const uint4 *bkt = reinterpret_cast<const uint4 *>(
                    rt.hidx[r] + kHidxSlots * hidx_home(k.w1, rt.hidx_buckets[r]));
                uint4 l2, h2;
                load32<WIDE>(bkt, l2, h2);
                uint32_t slot;
                uint32_t c2 = bucket_stop(l2, h2, tag, ((slots >> (4 * g)) & 15u) + 1u, slot);
                if (c2 > rt.n[r]) {
                    c2 = 0;
                    slot = kHidxSlots;
                }
                if (g == 0) cand[0] = c2; else if (g == 1) cand[1] = c2;
                else if (g == 2) cand[2] = c2; else cand[3] = c2;
                slots = (slots & ~(15u << (4 * g))) | (slot << (4 * g));
                if (c2 == 0 && slot != kHidxSlots) todo &= ~(1u << g);   // an empty slot: not here
            } else {
                const uint64_t at = hidx_find(rt.hidx[r], rt.hidx_buckets[r], rt.keys[r], rt.n[r], k);
                if (at != ~0ull) {
                    val = __ldg(reinterpret_cast<const uint4 *>(rt.vals[r] + at));
                    return true;
                }
                todo &= ~(1u << g);
            }
        }
    }
    return false;
}

template <bool HASHED, bool WIDE>
__global__ void __launch_bounds__(256, 3)
k_probe(const __grid_constant__ KeyConsts kc, const __grid_constant__ RunTable rt,
        uint32_t n_runs, const uint64_t *__restrict__ dir, uint32_t jcap, uint32_t C,
        uint32_t ns, uint32_t n_query, const uint32_t *__restrict__ tokens,
        const uint64_t *__restrict__ seq_off, const uint64_t *__restrict__ qchunk_off,
        uint64_t n_qchunks, uint32_t *__restrict__ hit_out, lsmkv_val_t *__restrict__ recs_out,
        lsmkv_key_t *__restrict__ keys_out, DevStatus *st, unsigned long long *next_query,
        const uint32_t *__restrict__ order)
{
    __shared__ KeyShared sh;
    // first miss of a round, by round mod 3: round r takes its minimum in slot r % 3 while
    // thread 0 resets slot (r + 1) % 3, whose last readers were two barriers ago
    __shared__ unsigned long long s_first_miss[3], s_q;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5, W = blockDim.x >> 5;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    unsigned long long n_lookups = 0;

    bool took = false;
    for (;;) {
        // queries are handed out one at a time: long and short ones balance across the CTAs
        // (without a counter there is a CTA per query: block b takes query b and leaves)
        __syncthreads();
        if (threadIdx.x == 0) {
            s_q = next_query ? atomicAdd(next_query, 1ull)
                             : (took ? (unsigned long long)n_query : (unsigned long long)blockIdx.x);
            s_first_miss[0] = ~0ull;
        }
        took = true;
        key_rounds_begin(sh);
        __syncthreads();
        if (s_q >= n_query) break;
        const uint64_t q = order ? order[s_q] : s_q;
        const uint64_t s0 = seq_off[q], s1 = seq_off[q + 1];
        const uint64_t nch = s1 >= s0 ? (s1 - s0) / C : 0;
        const uint64_t o0 = qchunk_off[q], o1 = qchunk_off[q + 1];
        if (s1 < s0 || o1 < o0 || o1 - o0 != nch || o1 > n_qchunks || nch > 0xFFFFFFFFull) {
            if (threadIdx.x == 0) { st_flag(st, LSMKV_ST_BAD_COUNT, q); hit_out[q] = 0; }
            continue;                                        // uniform over the CTA
        }
        const uint32_t *seq = tokens + s0;
        uint4 *recs = reinterpret_cast<uint4 *>(recs_out + o0);
        uint64_t hit = nch, base = 0;
        bool done = false;
        // Round 0 is one warp's 32 chunks -- a query without a cached prefix never gets past
        // it -- the later rounds take 32 chunks per warp of the CTA.
        for (unsigned rnd = 0; base < nch; ++rnd) {
            const unsigned wact = (rnd == 0 && !keys_out) ? 1u : W;
            const uint64_t span = 32ull * wact;
            const uint64_t j = base + 32ull * warp + lane;
            const bool valid = warp < wact && j < nch;
            if (!done) {                                     // next round's tokens on their way
                const uint64_t jn = base + span + 32ull * warp + lane;
                if (jn < nch) {
                    const char *nx = reinterpret_cast<const char *>(seq + jn * C);
                    for (uint32_t b = 0; b < 4u * C; b += 128u)
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(nx + b));
                }
            }
            const ChunkKey k = cta_chunk_keys(kc, seq, C, ns, base, nch, rnd, wact, sh, tokens,
                                              tokens + s1);
            if (threadIdx.x == 0) s_first_miss[(rnd + 1u) % 3u] = ~0ull;
            if (keys_out && valid) store_key(keys_out + o0 + j, k);
            if (done) {                                      // only the keys were wanted
                if (valid) recs[j] = zero;
                __syncthreads();                             // the exchange is rewritten next round
                base += span;
                continue;
            }
            uint4 val = zero;
            const bool found = valid && (HASHED ? lookup_runs_hash<WIDE>(rt, n_runs, k, val)
                                                : lookup_runs(rt, n_runs, dir, jcap, k, val));
            n_lookups += valid ? 1ull : 0ull;
            const unsigned miss = __ballot_sync(0xFFFFFFFFu, valid && !found);
            if (miss && lane == 0)
                atomicMin(&s_first_miss[rnd % 3u],
                          base + 32ull * warp + (unsigned)__ffs(miss) - 1ull);
            __syncthreads();
            const uint64_t fm = s_first_miss[rnd % 3u];
            if (valid) recs[j] = j < fm ? val : zero;
            base += span;
            if (fm != ~0ull) {
                hit = fm;
                done = true;
                if (!keys_out) {                             // nothing left but zeros
                    for (uint64_t z = base + threadIdx.x; z < nch; z += blockDim.x) recs[z] = zero;
                    break;
                }
            }
        }
        if (threadIdx.x == 0) {
            hit_out[q] = (uint32_t)hit;
            atomicAdd(&st->chunks_hit, (unsigned long long)hit);
            if (hit == 0) atomicAdd(&st->empty_probes, 1ull);
        }
    }
#pragma unroll
    for (unsigned d = 16; d; d >>= 1) n_lookups += __shfl_down_sync(0xFFFFFFFFu, n_lookups, d);
    if (lane == 0 && n_lookups) atomicAdd(&st->lookups, n_lookups);
}

}  // namespace lsmkv
