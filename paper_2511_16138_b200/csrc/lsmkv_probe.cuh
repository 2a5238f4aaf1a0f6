// Batched longest-cached-prefix probe: chunk keys of each query are looked up in the sorted
// runs from newest to oldest; the hit length is the number of leading chunks that were all
// found (first-miss rule), resolved per 32 chunks with one warp ballot.
#pragma once
#include "lsmkv_keys.cuh"

namespace lsmkv {

struct RunTable {
    const lsmkv_key_t *keys[LSMKV_MAX_RUNS];
    const lsmkv_val_t *vals[LSMKV_MAX_RUNS];
    uint64_t n[LSMKV_MAX_RUNS];
};

__device__ __forceinline__ int key_cmp_at(const lsmkv_key_t *e, const ChunkKey &k)
{
    const ulonglong2 *p = reinterpret_cast<const ulonglong2 *>(e);
    const ulonglong2 a = __ldg(p);
    if (a.x != k.w0) return a.x < k.w0 ? -1 : 1;
    if (a.y != k.w1) return a.y < k.w1 ? -1 : 1;
    const ulonglong2 b = __ldg(p + 1);
    if (b.x != k.w2) return b.x < k.w2 ? -1 : 1;
    if (b.y != k.w3) return b.y < k.w3 ? -1 : 1;
    return 0;
}

// Point lookup, newest run first; the first run that holds the key decides.
__device__ __forceinline__ bool lookup_runs(const RunTable &rt, uint32_t n_runs,
                                            const ChunkKey &k, uint4 &val)
{
    for (uint32_t r = 0; r < n_runs; ++r) {
        const lsmkv_key_t *keys = rt.keys[r];
        uint64_t lo = 0, hi = rt.n[r];
        while (lo < hi) {
            const uint64_t mid = lo + ((hi - lo) >> 1);
            const int c = key_cmp_at(keys + mid, k);
            if (c == 0) {
                val = __ldg(reinterpret_cast<const uint4 *>(rt.vals[r] + mid));
                return true;
            }
            if (c < 0) lo = mid + 1; else hi = mid;
        }
    }
    return false;
}

__global__ void __launch_bounds__(256)
k_probe(const __grid_constant__ KeyConsts kc, const __grid_constant__ RunTable rt,
        uint32_t n_runs, uint32_t C, uint32_t ns, uint32_t n_query,
        const uint32_t *__restrict__ tokens, const uint64_t *__restrict__ seq_off,
        const uint64_t *__restrict__ qchunk_off, uint64_t n_qchunks,
        uint32_t *__restrict__ hit_out, lsmkv_val_t *__restrict__ recs_out,
        lsmkv_key_t *__restrict__ keys_out, DevStatus *st)
{
    const unsigned lane = lane_id();
    const uint64_t warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    unsigned long long n_lookups = 0, n_hit = 0, n_empty = 0;
    for (uint64_t q = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; q < n_query;
         q += warps) {
        const uint64_t s0 = seq_off[q], s1 = seq_off[q + 1];
        const uint64_t nch = s1 >= s0 ? (s1 - s0) / C : 0;
        const uint64_t o0 = qchunk_off[q], o1 = qchunk_off[q + 1];
        if (s1 < s0 || o1 < o0 || o1 - o0 != nch || o1 > n_qchunks || nch > 0xFFFFFFFFull) {
            if (lane == 0) { st_flag(st, LSMKV_ST_BAD_COUNT, q); hit_out[q] = 0; }
            continue;
        }
        uint4 *recs = reinterpret_cast<uint4 *>(recs_out + o0);
        uint64_t hit = nch, cA = 0, cB = 0;
        bool done = false;
        for (uint64_t base = 0; base < nch; base += 32) {
            const uint64_t j = base + lane;
            const bool valid = j < nch;
            if (done && !keys_out) {                 // past the first miss: only zero-fill
                if (valid) recs[j] = zero;
                continue;
            }
            const ChunkKey k = warp_chunk_keys(kc, tokens + s0, C, ns, base, nch, cA, cB);
            if (keys_out && valid) store_key(keys_out + o0 + j, k);
            if (done) {
                if (valid) recs[j] = zero;
                continue;
            }
            uint4 val = zero;
            const bool found = valid && lookup_runs(rt, n_runs, k, val);
            const unsigned miss = __ballot_sync(0xFFFFFFFFu, valid && !found);
            const unsigned first_miss = miss ? (unsigned)__ffs(miss) - 1u : 32u;
            if (valid) recs[j] = lane < first_miss ? val : zero;
            n_lookups += valid ? 1ull : 0ull;
            if (miss) { hit = base + first_miss; done = true; }
        }
        if (lane == 0) {
            hit_out[q] = (uint32_t)hit;
            n_hit += hit;
            n_empty += hit == 0 ? 1ull : 0ull;
        }
    }
    // counters: lanes hold partial lookup counts, lane 0 holds hits / empties
#pragma unroll
    for (unsigned d = 16; d; d >>= 1) n_lookups += __shfl_down_sync(0xFFFFFFFFu, n_lookups, d);
    if (lane == 0) {
        if (n_lookups) atomicAdd(&st->lookups, n_lookups);
        if (n_hit) atomicAdd(&st->chunks_hit, n_hit);
        if (n_empty) atomicAdd(&st->empty_probes, n_empty);
    }
}

}  // namespace lsmkv
