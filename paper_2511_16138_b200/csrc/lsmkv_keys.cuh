// Chunk keys: two polynomial digests over the Mersenne prime 2^61-1 of every chunk-aligned
// token prefix, evaluated warp-cooperatively.
//
// The digest is defined sequentially (h <- h*B + t + 1 mod p per token). Because
// H(XY) = H(X) * B^|Y| + H(Y), a CTA hashes 32 chunks per warp at once: every lane digests its
// own chunk from h = 0 (16 tokens at a time as one dot product with the powers of B, see
// block16_dot). With M = B^C the digest of the prefix that ends with chunk j of a round is
//     P_j = c * M^(j+1) + sum_{i<=j} d_i * M^(j-i) = c * M^(j+1) + M^j * sum_{i<=j} d_i * M^(-i)
// (c = digest before the round, d_i = chunk digests; M is invertible because p is prime), so the
// chunk digests are scaled by M^(-i), summed with a plain additive scan, and scaled back: three
// independent modular multiplications per lane and digest instead of a chain of them through
// the scan. All arithmetic is exact in the field, so the canonical result is bit-identical to
// the sequential definition.
#pragma once
#include "lsmkv_common.cuh"

namespace lsmkv {

constexpr uint64_t kP = 0x1FFFFFFFFFFFFFFFull;  // 2^61 - 1
constexpr uint64_t kBaseA = 0x0B4E0EF37BC32127ull;
constexpr uint64_t kBaseB = 0x16A09E667F3BCC90ull;

// d[x][i] = BASE_x ^ (15 - i) mod p cut into limbs of 21, 21 and 19 bits: the weights of the 16
// tokens of a block (see block16_dot). sum[x] = BASE^0 + ... + BASE^15, b16[x] = BASE^16 (mod p).
// tab [dev]: four tables of kKeyTab entries, M = BASE ^ C:
//   tab[i] = M_A^(i+1), tab[kKeyTab + i] = M_B^(i+1), tab[2 kKeyTab + i] = M_A^(-i),
//   tab[3 kKeyTab + i] = M_B^(-i)   (i = position of a chunk inside a round, < 32 * warps)
constexpr int kKeyTab = 256;
struct KeyConsts {
    const uint64_t *tab;
    uint32_t dA[16][3];
    uint32_t dB[16][3];
    uint64_t sumA, sumB;
    uint64_t b16A, b16B;
};

// the canonical representative of s < 2^63
__host__ __device__ __forceinline__ uint64_t fold61(uint64_t s)
{
    s = (s & kP) + (s >> 61);
    return s >= kP ? s - kP : s;
}

__device__ __forceinline__ uint64_t mulmod61(uint64_t a, uint64_t b)
{
    const uint64_t lo = a * b;
    const uint64_t hi = __umul64hi(a, b);               // product < 2^122, hi < 2^58
    // 2^61 = 1 (mod p):  hi*2^64 + lo = (lo & p) + (lo >> 61) + hi*8
    return fold61((lo & kP) + ((lo >> 61) | (hi << 3)));
}

__device__ __forceinline__ uint64_t addmod61(uint64_t a, uint64_t b)  // a, b < p
{
    const uint64_t s = a + b;
    return s >= kP ? s - kP : s;
}

// The exchange below keeps its intermediate values only partly reduced -- any representative
// below 2^62 -- and takes the canonical one (fold61) once at the end; the value mod p is the same.
// a, b < 2^62  ->  a*b mod p, below 2^61 + 8
__device__ __forceinline__ uint64_t mulmod61_lazy(uint64_t a, uint64_t b)
{
    const uint64_t lo = a * b;
    const uint64_t hi = __umul64hi(a, b);               // product < 2^124, hi < 2^60
    const uint64_t s = (lo & kP) + ((lo >> 61) | (hi << 3));   // < 2^61 + 2^63
    return (s & kP) + (s >> 61);
}

// a + b mod p for a, b < 2^62, below 2^61 + 4
__device__ __forceinline__ uint64_t add61_lazy(uint64_t a, uint64_t b)
{
    const uint64_t s = a + b;                           // < 2^63
    return (s & kP) + (s >> 61);
}

__device__ __forceinline__ uint64_t horner61(uint64_t h, uint64_t base, uint32_t token)
{
    return fold61(mulmod61(h, base) + (uint64_t)token + 1ull);   // < p + 2^32 < 2^62
}

__device__ __forceinline__ uint64_t shfl_up64(uint64_t v, unsigned d)
{
    return __shfl_up_sync(0xFFFFFFFFu, v, d);
}

struct ChunkKey { uint64_t w0, w1, w2, w3; };

// a0 + a1 * 2^21 + a2 * 2^42 + sum (mod p), canonical; a0, a1 < 2^57, a2 < 2^55, sum < p.
// 2^61 = 1 (mod p), so the bits a shift pushes past bit 60 come back in at bit 0.
__device__ __forceinline__ uint64_t limbs_mod61(uint64_t a0, uint64_t a1, uint64_t a2, uint64_t sum)
{
    uint64_t s = a0 + ((a1 & ((1ull << 40) - 1)) << 21) + (a1 >> 40) +
                 ((a2 & ((1ull << 19) - 1)) << 42) + (a2 >> 19) + sum;      // < 2^63
    s = (s & kP) + (s >> 61);                                               // <= p + 3
    return s >= kP ? s - kP : s;
}

// Digest of the 16 tokens w[M .. M+15] from h = 0 (both lanes). Sixteen Horner steps from zero
// give sum_i (t_i + 1) * BASE^(15-i); with the weights cut into limbs of at most 21 bits every
// product t_i * limb is below 2^53, sixteen of them add up without overflow, and one reduction
// at the end replaces sixteen modular multiplications. Exact, hence the same value.
template <int M>
__device__ __forceinline__ void block16_dot(const KeyConsts &kc, const uint32_t (&w)[20],
                                            uint64_t &dA, uint64_t &dB, uint32_t &first,
                                            uint32_t &last)
{
    uint64_t a0 = 0, a1 = 0, a2 = 0, b0 = 0, b1 = 0, b2 = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        a0 += (uint64_t)w[i + M] * kc.dA[i][0];
        a1 += (uint64_t)w[i + M] * kc.dA[i][1];
        a2 += (uint64_t)w[i + M] * kc.dA[i][2];
        b0 += (uint64_t)w[i + M] * kc.dB[i][0];
        b1 += (uint64_t)w[i + M] * kc.dB[i][1];
        b2 += (uint64_t)w[i + M] * kc.dB[i][2];
    }
    dA = limbs_mod61(a0, a1, a2, kc.sumA);
    dB = limbs_mod61(b0, b1, b2, kc.sumB);
    first = w[M];
    last = w[M + 15];
}

// Hash of one chunk from h = 0 (both lanes), plus its first and last token: whole blocks of 16
// tokens by block16_dot, chained with BASE^16, the remaining tokens by the recurrence itself.
// A block is fetched with 16-byte loads: four when it starts on a 16-byte boundary, else the
// five aligned ones that cover it, as long as those stay inside [lim_lo, lim_hi) -- the token
// array up to the end of this sequence -- and token by token otherwise. Sequences are packed
// back to back, so three in four start off a boundary.
__device__ __forceinline__ void chunk_hash(const KeyConsts &kc, const uint32_t *t, uint32_t C,
                                           const uint32_t *lim_lo, const uint32_t *lim_hi,
                                           uint64_t &hA, uint64_t &hB, uint32_t &first,
                                           uint32_t &last)
{
    hA = 0;
    hB = 0;
    uint32_t i = 0;
    for (; i + 16 <= C; i += 16) {
        const uint32_t *blk = t + i;
        unsigned m = (unsigned)(reinterpret_cast<uintptr_t>(blk) >> 2) & 3u;   // words past a boundary
        const uint32_t *al = blk - m;
        uint32_t w[20];
        if (m == 0 || (al >= lim_lo && al + 20 <= lim_hi)) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(al) + q);
                w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
            }
            uint4 v = make_uint4(0, 0, 0, 0);
            if (m) v = __ldg(reinterpret_cast<const uint4 *>(al) + 4);
            w[16] = v.x; w[17] = v.y; w[18] = v.z; w[19] = v.w;
        } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) w[e] = __ldg(blk + e);
            w[16] = w[17] = w[18] = w[19] = 0;
            m = 0;
        }
        uint64_t dA, dB;
        uint32_t f, l;
        switch (m) {
        case 0: block16_dot<0>(kc, w, dA, dB, f, l); break;
        case 1: block16_dot<1>(kc, w, dA, dB, f, l); break;
        case 2: block16_dot<2>(kc, w, dA, dB, f, l); break;
        default: block16_dot<3>(kc, w, dA, dB, f, l); break;
        }
        if (i == 0) {
            first = f;
            hA = dA;
            hB = dB;
        } else {
            hA = addmod61(mulmod61(hA, kc.b16A), dA);
            hB = addmod61(mulmod61(hB, kc.b16B), dB);
        }
        last = l;
    }
    for (; i < C; ++i) {
        last = __ldg(t + i);
        if (i == 0) first = last;
        hA = horner61(hA, kBaseA, last);
        hB = horner61(hB, kBaseB, last);
    }
}

constexpr int kKeyMaxWarps = 8;   // one table entry per chunk of a round: 32 chunks per warp
static_assert(32 * kKeyMaxWarps <= kKeyTab, "a CTA's round must fit the power tables");

// Shared-memory exchange of a CTA that hashes one sequence round by round.
struct KeyShared {
    uint64_t aggA[kKeyMaxWarps], aggB[kKeyMaxWarps];   // scaled sum of each warp's 32-chunk block
    uint64_t carryA[2], carryB[2];                     // prefix before the round, by round parity
};

// Before the first round of a sequence (followed by a __syncthreads() before round 0).
__device__ __forceinline__ void key_rounds_begin(KeyShared &sh)
{
    if (threadIdx.x == 0) { sh.carryA[0] = 0; sh.carryB[0] = 0; }
}

// One round of a CTA: its first `wact` warps hash 32*wact consecutive chunks starting at `base`
// (warp w the 32-chunk block base + 32*w), as laid out at the top of this file: chunk digests
// scaled by M^(-i), an additive scan inside every warp, the warps' totals exchanged through
// shared memory, and the sum scaled back and joined with the prefix the previous round left.
// Every thread of an active warp ends up with the key of chunk base + 32*warp + lane; the last
// active warp leaves the prefix behind the round for round `rnd + 1`. Warps >= wact get an
// unspecified key. Contains one __syncthreads(); the caller must put another one between two
// calls (the exchange is rewritten). 32 * wact <= kKeyTab. [lim_lo, lim_hi) is the part of the
// token array that may be read: from its start to the end of this sequence.
__device__ __forceinline__ ChunkKey cta_chunk_keys(const KeyConsts &kc, const uint32_t *seq,
                                                   uint32_t C, uint32_t ns, uint64_t base,
                                                   uint64_t nch, unsigned rnd, unsigned wact,
                                                   KeyShared &sh, const uint32_t *lim_lo,
                                                   const uint32_t *lim_hi)
{
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    const unsigned idx = 32u * warp + lane;                // position inside the round
    const uint64_t j = base + idx;
    uint64_t zA = 0, zB = 0;
    uint64_t upA = 0, upB = 0, backA = 0, backB = 0;      // M^(idx+1) and M^idx, asked for early
    uint32_t first = 0, last = 0;
    if (warp < wact) {
        upA = __ldg(kc.tab + idx);
        upB = __ldg(kc.tab + kKeyTab + idx);
        if (idx) {
            backA = __ldg(kc.tab + idx - 1);
            backB = __ldg(kc.tab + kKeyTab + idx - 1);
        }
        uint64_t dA = 0, dB = 0;
        if (j < nch) {
            chunk_hash(kc, seq + j * C, C, lim_lo, lim_hi, dA, dB, first, last);
        }
        zA = mulmod61_lazy(dA, __ldg(kc.tab + 2 * kKeyTab + idx));
        zB = mulmod61_lazy(dB, __ldg(kc.tab + 3 * kKeyTab + idx));
#pragma unroll
        for (unsigned d = 1; d < 32; d <<= 1) {            // inclusive sums inside the warp
            const uint64_t uA = shfl_up64(zA, d), uB = shfl_up64(zB, d);
            if (lane >= d) {
                zA = add61_lazy(uA, zA);
                zB = add61_lazy(uB, zB);
            }
        }
        if (lane == 31) { sh.aggA[warp] = zA; sh.aggB[warp] = zB; }
    }
    __syncthreads();
    uint64_t hA = 0, hB = 0;
    if (warp < wact) {
        for (unsigned v = 0; v < warp; ++v) {              // the warps before this one
            zA = add61_lazy(zA, sh.aggA[v]);
            zB = add61_lazy(zB, sh.aggB[v]);
        }
        const uint64_t cA = mulmod61_lazy(sh.carryA[rnd & 1u], upA);
        const uint64_t cB = mulmod61_lazy(sh.carryB[rnd & 1u], upB);
        if (idx) {                                         // scale the sum back by M^idx
            zA = mulmod61_lazy(zA, backA);
            zB = mulmod61_lazy(zB, backB);
        }
        hA = fold61(cA + zA);
        hB = fold61(cB + zB);
        if (warp == wact - 1 && lane == 31) {              // meaningful when the round was full
            sh.carryA[(rnd + 1u) & 1u] = hA;
            sh.carryB[(rnd + 1u) & 1u] = hB;
        }
    }
    ChunkKey k;
    k.w0 = ((uint64_t)ns << 32) | (uint64_t)(uint32_t)j;
    k.w1 = hA;
    k.w2 = hB;
    k.w3 = ((uint64_t)first << 32) | (uint64_t)last;
    return k;
}

__device__ __forceinline__ void store_key(lsmkv_key_t *dst, const ChunkKey &k)
{
    ulonglong2 *p = reinterpret_cast<ulonglong2 *>(dst);
    p[0] = make_ulonglong2(k.w0, k.w1);
    p[1] = make_ulonglong2(k.w2, k.w3);
}

// put_batch keys + records: one CTA per request at a time (requests handed out round-robin),
// 32 * W chunks per round.
__global__ void __launch_bounds__(32 * kKeyMaxWarps)
k_encode_keys(const __grid_constant__ KeyConsts kc, uint32_t C, uint32_t ns, uint32_t n_req,
              const uint32_t *__restrict__ tokens, const uint64_t *__restrict__ seq_off,
              const uint32_t *__restrict__ start_chunk, const uint64_t *__restrict__ chunk_off,
              uint64_t n_chunks, uint32_t file_id, uint64_t base_offset, uint64_t chunk_bytes,
              lsmkv_key_t *__restrict__ keys_out, lsmkv_val_t *__restrict__ vals_out,
              DevStatus *st)
{
    __shared__ KeyShared sh;
    const unsigned W = blockDim.x >> 5;
    const uint64_t round_chunks = 32ull * W;
    for (uint64_t r = blockIdx.x; r < n_req; r += gridDim.x) {
        const uint64_t s0 = seq_off[r], s1 = seq_off[r + 1];
        const uint64_t nch = s1 >= s0 ? (s1 - s0) / C : 0;
        const uint64_t start = start_chunk ? start_chunk[r] : 0;
        const uint64_t cnt = nch > start ? nch - start : 0;
        const uint64_t o0 = chunk_off[r], o1 = chunk_off[r + 1];
        if (s1 < s0 || o1 < o0 || o1 - o0 != cnt || o1 > n_chunks || nch > 0xFFFFFFFFull) {
            if (threadIdx.x == 0) st_flag(st, LSMKV_ST_BAD_COUNT, r);
            continue;                                        // uniform over the CTA
        }
        if (cnt == 0) continue;
        key_rounds_begin(sh);
        __syncthreads();
        unsigned rnd = 0;
        for (uint64_t base = 0; base < nch; base += round_chunks, ++rnd) {
            const ChunkKey k = cta_chunk_keys(kc, tokens + s0, C, ns, base, nch, rnd, W, sh,
                                              tokens, tokens + s1);
            const uint64_t j = base + threadIdx.x;           // = base + 32 * warp + lane
            if (j >= start && j < nch) {
                const uint64_t i = o0 + (j - start);
                store_key(keys_out + i, k);
                uint4 v;
                const uint64_t off = base_offset + i * chunk_bytes;
                v.x = file_id;
                v.y = 0;
                v.z = (uint32_t)off;
                v.w = (uint32_t)(off >> 32);
                *reinterpret_cast<uint4 *>(vals_out + i) = v;
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) atomicAdd(&st->chunks_encoded, (unsigned long long)cnt);
    }
}

}  // namespace lsmkv
