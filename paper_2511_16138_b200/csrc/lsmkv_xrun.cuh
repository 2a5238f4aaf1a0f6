// Exact prefix index ("xrun"): stored sequences ordered by their tokens, so key order is prefix
// order and a lookup compares tokens, never digests (Sec. 3.1/3.2: keys that keep the prefix
// structure). Build = a rank-merge sort of sequence ids with a warp-cooperative token comparison;
// probe = one binary search per (query, run) that skips the tokens both bounds already share.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "lsmkv.h"
#include "lsmkv_common.cuh"

namespace lsmkv {

struct SeqView {
    const uint32_t *tok;
    uint64_t len;
};

__device__ __forceinline__ SeqView seq_view(const uint32_t *__restrict__ tokens,
                                            const uint64_t *__restrict__ seq_off, uint64_t s)
{
    const uint64_t a = __ldg(seq_off + s), b = __ldg(seq_off + s + 1);
    return SeqView{tokens + a, b >= a ? b - a : 0};
}

// One comparison step of warp_lcp: tokens [i, i + 32 * kUnroll) of a and b, all loads in flight at
// once. Returns the position of the first difference, or ~0 if there is none below n.
template <int kUnroll>
__device__ __forceinline__ uint64_t lcp_step(const SeqView &a, const SeqView &b, uint64_t i,
                                             uint64_t n)
{
    const unsigned lane = lane_id();
    bool differ[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const uint64_t k = i + 32u * u + lane;
        differ[u] = k < n && __ldg(a.tok + k) != __ldg(b.tok + k);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const unsigned m = __ballot_sync(0xFFFFFFFFu, differ[u]);
        if (m) return i + 32u * u + (unsigned)__ffs(m) - 1u;
    }
    return ~0ull;
}

// Warp-cooperative: length of the common token prefix of a and b, starting the comparison at
// `from` (the caller knows the first `from` tokens agree). Every lane returns the same value.
// Steps of 128 tokens; a comparison that is still running after two of them goes on in steps of
// 512 (a step costs one memory round trip whatever its width, most comparisons end in their
// first step, and the few long ones are what the sort and the probe wait for). The wide step
// needs registers: the kernels that call this allow themselves 128.
__device__ __forceinline__ uint64_t warp_lcp(const SeqView &a, const SeqView &b, uint64_t from)
{
    const uint64_t n = a.len < b.len ? a.len : b.len;
    uint64_t i = from;
    for (int step = 0; i < n; ++step) {
        if (step >= 2) {
            const uint64_t r = lcp_step<16>(a, b, i, n);
            if (r != ~0ull) return r;
            i += 512;
        } else {
            const uint64_t r = lcp_step<4>(a, b, i, n);
            if (r != ~0ull) return r;
            i += 128;
        }
    }
    return n;
}

// Where x belongs among the sorted sequences order[lo, hi): the first position whose sequence is
// above x. "Above" = larger in token order (a proper prefix is smaller); a sequence with the same
// tokens is above x when its number exceeds x_id. The two ends are compared before bisecting
// (in the sort an element usually falls wholly before or after the sibling segment); once both
// bounds are known every comparison starts at min(l_lo, l_hi): everything between the bounds
// shares at least that many tokens with x.
struct Located {
    uint64_t pos;            // order[pos - 1] is not above x, order[pos] is
    uint64_t l_lo, l_hi;     // tokens x shares with those two neighbours
    uint32_t s_lo, s_hi;     // their sequence numbers
    bool have_lo, have_hi;   // whether such a neighbour exists in [lo, hi)
};

__device__ __forceinline__ Located warp_locate(const SeqView &x, uint32_t x_id,
                                               const uint32_t *__restrict__ tokens,
                                               const uint64_t *__restrict__ seq_off,
                                               const uint32_t *__restrict__ order, uint64_t lo,
                                               uint64_t hi)
{
    Located r{lo, 0, 0, 0, 0, false, false};
    while (lo < hi) {
        const uint64_t m = !r.have_hi ? hi - 1 : !r.have_lo ? lo : lo + ((hi - lo) >> 1);
        const uint32_t y = __ldg(order + m);
        const SeqView vy = seq_view(tokens, seq_off, y);
        const uint64_t from = r.have_lo && r.have_hi ? (r.l_lo < r.l_hi ? r.l_lo : r.l_hi) : 0;
        const uint64_t l = warp_lcp(vy, x, from);
        // y ends at l: a prefix of x (below) or the same tokens (the numbers decide)
        const bool above = l < vy.len ? (l >= x.len || __ldg(vy.tok + l) > __ldg(x.tok + l))
                                      : (vy.len == x.len && y > x_id);
        if (above) { hi = m; r.l_hi = l; r.s_hi = y; r.have_hi = true; }
        else { lo = m + 1; r.l_lo = l; r.s_lo = y; r.have_lo = true; }
    }
    r.pos = lo;
    return r;
}

__global__ void __launch_bounds__(256)
k_xrun_init(const uint64_t *__restrict__ seq_off, uint32_t n_seq, uint32_t C,
            uint32_t *__restrict__ order, uint64_t *__restrict__ chunk_cnt, DevStatus *st)
{
    for (uint64_t s = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; s < n_seq;
         s += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t a = seq_off[s], b = seq_off[s + 1];
        if (b < a) st_flag(st, LSMKV_ST_BAD_COUNT, s);
        order[s] = (uint32_t)s;
        chunk_cnt[s] = b >= a ? (b - a) / C : 0;
    }
}

// One merge level over sequence ids, one warp per element: its rank among the sibling segment
// comes from a binary search with the token comparison. The order is total (ties by id), so the
// two halves never hold equal elements.
__global__ void __launch_bounds__(256, 2)
k_xrun_merge_level(const uint32_t *__restrict__ tokens, const uint64_t *__restrict__ seq_off,
                   const uint32_t *__restrict__ src, uint32_t *__restrict__ dst, uint64_t n,
                   uint64_t width)
{
    const uint64_t warp0 = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t i = warp0; i < n; i += n_warps) {
        const uint64_t base = i / (2 * width) * (2 * width);
        const uint64_t mid = min(n, base + width), end = min(n, base + 2 * width);
        const uint32_t x = __ldg(src + i);
        const SeqView vx = seq_view(tokens, seq_off, x);
        uint64_t lo, hi;
        if (i < mid) { lo = mid; hi = end; } else { lo = base; hi = mid; }
        const uint64_t below = warp_locate(vx, x, tokens, seq_off, src, lo, hi).pos - lo;
        const uint64_t own = i < mid ? i - base : i - mid;
        if (lane_id() == 0) dst[base + own + below] = x;
    }
}

// Merge of two sorted runs that share one arena: src[0, mid) and src[mid, n) are each in token
// order; one warp per element finds its rank in the other part, as in a merge level.
__global__ void __launch_bounds__(256, 2)
k_xrun_merge_two(const uint32_t *__restrict__ tokens, const uint64_t *__restrict__ seq_off,
                 const uint32_t *__restrict__ src, uint32_t *__restrict__ dst, uint64_t n,
                 uint64_t mid)
{
    const uint64_t warp0 = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t i = warp0; i < n; i += n_warps) {
        const uint32_t x = __ldg(src + i);
        const SeqView vx = seq_view(tokens, seq_off, x);
        uint64_t lo, hi;
        if (i < mid) { lo = mid; hi = n; } else { lo = 0; hi = mid; }
        const uint64_t below = warp_locate(vx, x, tokens, seq_off, src, lo, hi).pos - lo;
        const uint64_t own = i < mid ? i : i - mid;
        if (lane_id() == 0) dst[own + below] = x;
    }
}

// src = order_a, then order_b with n_a added to every number (run B's sequences follow run A's
// in the shared arena); chunk counts of all sequences as in k_xrun_init.
__global__ void __launch_bounds__(256)
k_xrun_concat(const uint32_t *__restrict__ order_a, uint32_t n_a,
              const uint32_t *__restrict__ order_b, uint32_t n_b,
              const uint64_t *__restrict__ seq_off, uint32_t C, uint32_t *__restrict__ src,
              uint64_t *__restrict__ chunk_cnt, DevStatus *st)
{
    const uint64_t n = (uint64_t)n_a + n_b;
    for (uint64_t s = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; s < n;
         s += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t a = seq_off[s], b = seq_off[s + 1];
        if (b < a) st_flag(st, LSMKV_ST_BAD_COUNT, s);
        chunk_cnt[s] = b >= a ? (b - a) / C : 0;
        uint32_t v = s < n_a ? order_a[s] : order_b[s - n_a] + n_a;
        // a number outside its part would send the comparisons out of the arena
        const bool ok = s < n_a ? v < n_a : (v >= n_a && v < n);
        if (!ok) { st_flag(st, LSMKV_ST_BAD_COUNT, s); v = (uint32_t)s; }
        src[s] = v;
    }
}

constexpr int kMaxXRuns = LSMKV_MAX_RUNS;

struct XRunTable {
    const uint32_t *tokens[kMaxXRuns];
    const uint64_t *seq_off[kMaxXRuns];
    const lsmkv_val_t *vals[kMaxXRuns];
    const uint32_t *order[kMaxXRuns];
    const uint64_t *chunk_off[kMaxXRuns];
    uint32_t n_seq[kMaxXRuns];
};

// One warp per query at a time, queries drawn from a counter in the order given (longest first
// when `order` is set, so that the long comparisons start early and the short queries fill in
// behind them). Per run, newest first: the position of the query among the sorted stored
// sequences; the longer of the prefixes shared with the two neighbours is the longest prefix
// shared with anything in the run, and that neighbour (the lower one on a tie) lends its records.
__global__ void __launch_bounds__(256, 2)
k_xprobe(const __grid_constant__ XRunTable rt, uint32_t n_runs, uint32_t C, uint32_t n_query,
         const uint32_t *__restrict__ tokens, const uint64_t *__restrict__ seq_off,
         const uint64_t *__restrict__ qchunk_off, uint64_t n_qchunks,
         uint32_t *__restrict__ hit_out, lsmkv_val_t *__restrict__ recs_out, DevStatus *st,
         unsigned long long *next_query, const uint32_t *__restrict__ order)
{
    const unsigned lane = lane_id();
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (;;) {
        unsigned long long t = 0;
        if (lane == 0) t = atomicAdd(next_query, 1ull);
        t = __shfl_sync(0xFFFFFFFFu, t, 0);
        if (t >= n_query) break;
        const uint64_t q = order ? order[t] : t;
        const uint64_t s0 = seq_off[q], s1 = seq_off[q + 1];
        const uint64_t nch = s1 >= s0 ? (s1 - s0) / C : 0;
        const uint64_t o0 = qchunk_off[q], o1 = qchunk_off[q + 1];
        if (s1 < s0 || o1 < o0 || o1 - o0 != nch || o1 > n_qchunks || nch > 0xFFFFFFFFull) {
            if (lane == 0) { st_flag(st, LSMKV_ST_BAD_COUNT, q); hit_out[q] = 0; }
            continue;
        }
        const SeqView Q{tokens + s0, s1 - s0};
        uint4 *recs = reinterpret_cast<uint4 *>(recs_out + o0);
        uint64_t hit = 0;
        for (uint32_t r = 0; r < n_runs; ++r) {
            const uint32_t n = rt.n_seq[r];
            if (n == 0 || hit >= nch) continue;
            // The search is written out here rather than shared with the sort's routine: the
            // shared form measured a third slower in this kernel.
            // invariant: order[lo - 1] <= Q < order[hi]; l_lo / l_hi = tokens Q shares with them
            uint64_t lo = 0, hi = n, l_lo = 0, l_hi = 0;
            uint32_t s_lo = 0, s_hi = 0;
            bool have_lo = false, have_hi = false;
            while (lo < hi) {
                const uint64_t m = lo + ((hi - lo) >> 1);
                const uint32_t y = __ldg(rt.order[r] + m);
                const SeqView vy = seq_view(rt.tokens[r], rt.seq_off[r], y);
                // everything between the bounds shares at least min(l_lo, l_hi) tokens with Q
                const uint64_t from = have_lo && have_hi ? (l_lo < l_hi ? l_lo : l_hi) : 0;
                const uint64_t l = warp_lcp(vy, Q, from);
                const bool above = l < vy.len && (l >= Q.len || __ldg(vy.tok + l) > __ldg(Q.tok + l));
                if (above) { hi = m; l_hi = l; s_hi = y; have_hi = true; }
                else { lo = m + 1; l_lo = l; s_lo = y; have_lo = true; }
            }
            const bool use_lo = have_lo && (!have_hi || l_lo >= l_hi);
            const uint64_t L = use_lo ? l_lo : l_hi;
            const uint64_t m_chunks = L / C;
            if (m_chunks <= hit) continue;
            const uint32_t owner = use_lo ? s_lo : s_hi;
            const uint4 *src = reinterpret_cast<const uint4 *>(rt.vals[r]) +
                               __ldg(rt.chunk_off[r] + owner);
            for (uint64_t j = hit + lane; j < m_chunks; j += 32) recs[j] = __ldg(src + j);
            hit = m_chunks;
        }
        for (uint64_t j = hit + lane; j < nch; j += 32) recs[j] = zero;
        if (lane == 0) {
            hit_out[q] = (uint32_t)hit;
            atomicAdd(&st->chunks_hit, (unsigned long long)hit);
            if (hit == 0) atomicAdd(&st->empty_probes, 1ull);
        }
    }
}

}  // namespace lsmkv
