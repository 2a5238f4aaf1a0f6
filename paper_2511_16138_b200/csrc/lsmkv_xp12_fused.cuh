// One-pass encoder of the compressing codec "xp12": every page slab is read from the pool once.
//
// The three-step encoder (lsmkv_xp12.cuh) reads the pool twice, because where a slab lands
// depends on the sizes of all slabs before it. Here a slab stays on the SM between being
// measured and being written: a persistent CTA per SM runs a pipeline of
//   producer warp   draws the next slab number from a counter, fetches the slab into a ring of
//                   shared-memory stages with one bulk copy (cp.async.bulk, mbarrier-completed);
//   compute groups  (8 or 16 warps) take the slab into registers, find its exponent window and
//                   exception count, publish its encoded size, and build the encoded slab in a
//                   ring of shared-memory output buffers;
//   commit warps    one per output buffer: sum the sizes of all earlier slabs (decoupled
//                   look-back over a per-slab state word: empty / size known / prefix known),
//                   publish the prefix, and send the buffer to its place with one bulk copy.
// Slab numbers are handed out in order by the counter, so every slab a look-back waits for is
// held by a CTA that is already running. A small kernel afterwards (k_xpf_layout) turns the
// prefixes into chunk directories and records. Bytes out are those of the three-step encoder.
//
// Every wait is bounded (the mbarrier waits and the look-back polls give up after `wait_cycles`
// clock cycles, set LSMKV_ST_WAIT_EXPIRED and an abort word that makes every other wait of the
// launch return at its next poll); a CTA leaves only after the bulk copies it issued have
// finished with its shared memory.
#pragma once
#include "lsmkv_common.cuh"
#include "lsmkv_copy.cuh"
#include "lsmkv_xp12.cuh"

namespace lsmkv {
namespace xpf {

constexpr uint64_t kFlagAgg = 1ull << 62;      // low 62 bits: bytes this slab adds to the blob
constexpr uint64_t kFlagIncl = 2ull << 62;     // low 62 bits: bytes of all slabs up to this one
constexpr uint64_t kValueMask = (1ull << 62) - 1;
constexpr uint64_t kEnd = ~0ull;               // slab number that tells a role to stop

// Shape of the pipeline for a slab of kWpg * kSweeps * 256 elements.
template <int SWEEPS, int WPG, int GROUPS, int RAW, int OUT>
struct Shape {
    static constexpr int kSweeps = SWEEPS, kWpg = WPG, kGroups = GROUPS, kRaw = RAW, kOut = OUT;
    static constexpr int kElems = WPG * SWEEPS * 256;
    static constexpr int kPageBytes = 2 * kElems;
    static constexpr int kOutStride = kPageBytes + 128;              // header + raw slab, padded
    static constexpr int kComputeWarps = WPG * GROUPS;
    static constexpr int kProducerWarp = kComputeWarps;
    static constexpr int kFirstCommitWarp = kComputeWarps + 1;
    static constexpr int kWarps = kComputeWarps + 1 + OUT;
    static constexpr int kThreads = kWarps * 32;
    static constexpr size_t kSmem = (size_t)RAW * kPageBytes + (size_t)OUT * kOutStride + 1024;
    // A ring position must always come back to the same group: a waiter tells phases apart by
    // their parity only, which is safe as long as it cannot be two phases ahead of the barrier --
    // true when the group that waits for use n of a stage is the one that finished use n - 1
    // of it, false when another group, running behind, still owes that use.
    static_assert(RAW % GROUPS == 0 && OUT % GROUPS == 0, "rings must divide among the groups");
};

struct Job {
    XpJob x;                       // geometry, pool, page table, blob, status (slab_* unused)
    unsigned long long *ticket;    // [dev] next slab number; zero before the launch
    unsigned long long *state;     // [dev] one word per slab; zero before the launch
    unsigned int *abort;           // [dev] zero before the launch
    long long wait_cycles;         // limit of every wait
};

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                 :: "r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned int ld_abort(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint64_t ld_state(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_state(unsigned long long *p, uint64_t v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// Wait for a phase of an mbarrier; false when the launch was aborted or the limit ran out (the
// caller then raises the abort itself).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const Job &job)
{
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (ld_abort(job.abort)) return false;
            if (clock64() - t0 > job.wait_cycles) return false;
        }
    }
}

// a * b + c as one multiply-add: the integer multiplier runs beside the logic/shift unit, which
// is what bounds this kernel, so shifts-and-adds are phrased as products where that is exact.
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// Sign+mantissa bytes of four words (eight elements). With u = w & 0x807F807F, byte 0 of a half
// holds the mantissa and byte 1 only the sign in its top bit, so u * 257 = u + (u << 8) adds the
// two into bytes 1 and 3 without a carry; the byte permutes collect those.
__device__ __forceinline__ uint2 sm_bytes_mul(const uint4 &q)
{
    const uint32_t p0 = mad_u32(q.x & 0x807F807Fu, 257u, 0u), p1 = mad_u32(q.y & 0x807F807Fu, 257u, 0u),
                   p2 = mad_u32(q.z & 0x807F807Fu, 257u, 0u), p3 = mad_u32(q.w & 0x807F807Fu, 257u, 0u);
    return make_uint2(__byte_perm(p0, p1, 0x7531), __byte_perm(p2, p3, 0x7531));
}

__device__ __forceinline__ void raise_abort(const Job &job, uint64_t slab)
{
    if (atomicExch(job.abort, 1u) == 0u) st_flag(job.x.st, LSMKV_ST_WAIT_EXPIRED, slab);
}

// Sum of the bytes of slabs 0 .. u-1, by the whole warp: walk back over the state words, adding
// sizes until a slab whose prefix is known. Returns false if the launch was aborted.
__device__ __forceinline__ bool look_back(const Job &job, uint64_t u, uint64_t *prefix)
{
    const unsigned lane = lane_id();
    uint64_t sum = 0;
    long long pos = (long long)u - 1;                     // nearest slab not yet accounted for
    const long long t0 = clock64();
    uint32_t polls = 0;
    while (pos >= 0) {
        uint64_t v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long long idx = pos - (j * 32 + (int)lane);
            v[j] = idx >= 0 ? ld_state(job.state + idx) : kFlagIncl;   // before slab 0: prefix 0
        }
        bool done = false, stalled = false;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (done || stalled) continue;
            const uint32_t flag = (uint32_t)(v[j] >> 62);
            const uint32_t incl = __ballot_sync(0xFFFFFFFFu, flag == 2u);
            const uint32_t empty = __ballot_sync(0xFFFFFFFFu, flag == 0u);
            const uint32_t first = incl ? (uint32_t)__ffs((int)incl) - 1u : 32u;
            const uint32_t need = first >= 31u ? 0xFFFFFFFFu : ((2u << first) - 1u);
            if (empty & need) { stalled = true; continue; }            // a size is still missing
            uint64_t c = lane <= first ? (v[j] & kValueMask) : 0ull;
#pragma unroll
            for (int d = 16; d; d >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, d);
            sum += c;
            if (first < 32u) done = true; else pos -= 32;
        }
        if (done) break;
        if (stalled && (++polls & 15u) == 0) {
            const bool give_up = ld_abort(job.abort) != 0u || clock64() - t0 > job.wait_cycles;
            if (__any_sync(0xFFFFFFFFu, give_up)) return false;
        }
    }
    *prefix = sum;
    return true;
}

}  // namespace xpf

// Dynamic shared memory: kRaw stages of page_bytes, kOut output buffers, barriers and mailboxes.
template <class S>
__global__ void __launch_bounds__(S::kThreads, 1)
k_xpf_encode(const __grid_constant__ xpf::Job job)
{
    using namespace xpf;
    extern __shared__ __align__(128) unsigned char xpf_smem[];
    constexpr int N = S::kElems;
    unsigned char *raw = xpf_smem;
    unsigned char *outb = xpf_smem + (size_t)S::kRaw * S::kPageBytes;
    unsigned char *tail = outb + (size_t)S::kOut * S::kOutStride;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail);             // 2 * kRaw + 4 * kOut
    uint64_t *raw_slab = bars + 2 * S::kRaw + 4 * S::kOut;           // [kRaw] slab number or kEnd
    uint32_t *raw_ok = reinterpret_cast<uint32_t *>(raw_slab + S::kRaw);   // [kRaw] page usable
    // per output buffer, by parity of its use: the slab it will hold (or kEnd) and its size
    uint64_t *out_slab = reinterpret_cast<uint64_t *>(raw_ok + S::kRaw + (S::kRaw & 1));
    uint32_t *out_size = reinterpret_cast<uint32_t *>(out_slab + 2 * S::kOut);  // [kOut][2]
    uint32_t *red = out_size + 2 * S::kOut;                          // [kGroups][2][kWpg]
    uint32_t *n_real = red + S::kGroups * 2 * S::kWpg;               // slabs this CTA was handed

    const uint32_t bar0 = smem_addr(bars);
    auto raw_full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto raw_empty = [&](int s) { return bar0 + 8u * (uint32_t)(S::kRaw + s); };
    auto out_full = [&](int s) { return bar0 + 8u * (uint32_t)(2 * S::kRaw + s); };
    auto out_empty = [&](int s) { return bar0 + 8u * (uint32_t)(2 * S::kRaw + S::kOut + s); };
    // "the size of the slab that buffer s will hold in its use n is known", one barrier per
    // parity of n: the commit warp starts its look-back there, while the slab is still being
    // packed. Two barriers, because the group announces use n + 1 before the commit warp is
    // known to have seen the announcement of use n; use n + 2 it cannot reach before that.
    auto size_known = [&](int s, uint32_t n) {
        return bar0 + 8u * (uint32_t)(2 * S::kRaw + 2 * S::kOut + 2 * s + (int)(n & 1u));
    };

    const unsigned warp = threadIdx.x >> 5, lane = lane_id();
    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kRaw; ++s) {
            mbar_init(raw_full(s), 1);                    // the producer's arrive (+ copy bytes)
            mbar_init(raw_empty(s), S::kWpg);             // one arrive per warp of the group
        }
        for (int s = 0; s < S::kOut; ++s) {
            mbar_init(out_full(s), S::kWpg * 32);         // every thread of the group
            mbar_init(out_empty(s), 1);                   // the commit warp
            mbar_init(size_known(s, 0), 1);               // one thread of the group
            mbar_init(size_known(s, 1), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();                                      // the only CTA-wide barrier

    const uint32_t slabs = 2u * job.x.n_layers * job.x.pages_per_chunk;
    const uint64_t total = job.x.n_chunks * slabs;

    if (warp == (unsigned)S::kProducerWarp) {
        // ---- producer: one lane hands out slab numbers and starts the fetches. Drawing a number
        // and looking up its page are two dependent round trips to L2; they run three and one
        // slab ahead of the fetch, so the loop turns at the pace of one round trip, not three.
        if (lane != 0) return;
        struct Where { const unsigned char *src; uint64_t chunk; uint32_t ok, first_of_page; };
        auto draw = [&](bool ended) -> uint64_t {
            return ended ? total : (uint64_t)atomicAdd(job.ticket, 1ull);
        };
        auto locate = [&](uint64_t u) -> Where {
            Where w{nullptr, 0, 0u, 0u};
            if (u >= total) return w;
            const uint64_t i = u / slabs;
            const uint32_t b = (uint32_t)(u - i * slabs);
            const uint32_t per_page = 2u * job.x.n_layers, pg = b / per_page, bb = b - pg * per_page;
            const uint64_t page = __ldg(job.x.page_table + i * job.x.pages_per_chunk + pg);
            const unsigned char *pool_buf = static_cast<const unsigned char *>(
                job.x.kv_ptrs[(bb & 1u) * job.x.n_layers + (bb >> 1)]);
            w.chunk = i;
            w.first_of_page = bb == 0 ? 1u : 0u;
            if (page >= job.x.num_pages) w.ok = 2u;                       // unusable page id
            else if ((reinterpret_cast<uintptr_t>(pool_buf) & 15u) != 0) w.ok = 3u;   // misaligned
            else { w.ok = 1u; w.src = pool_buf + page * (uint64_t)S::kPageBytes; }
            return w;
        };
        bool ended = false;
        uint64_t u_a = draw(false), u_b = draw(false), u_c = draw(false);
        Where w_a = locate(u_a);
        int ends = 0;
        uint32_t fetch_mask = 0, fetch_parity = 0;        // per stage: last arm was a fetch / its phase
        for (uint32_t k = 0;; ++k) {
            const uint64_t u_d = draw(ended);             // three slabs ahead
            const Where w_b = locate(u_b);                // one slab ahead
            ended = ended || u_b >= total;
            const int s = (int)(k % S::kRaw);
            const uint32_t ph = (k / S::kRaw) & 1u;
            if (!mbar_wait(raw_empty(s), ph ^ 1u, job)) { raise_abort(job, 0); break; }
            if (u_a >= total) {                           // every group gets its own stop mark
                if (ends == 0) *n_real = k;
                raw_slab[s] = kEnd;
                fetch_mask &= ~(1u << s);
                mbar_arrive(raw_full(s));
                if (++ends == S::kGroups) break;
            } else {
                if (w_a.ok == 2u && w_a.first_of_page) st_flag(job.x.st, LSMKV_ST_BAD_PAGE, w_a.chunk);
                if (w_a.ok == 3u) st_flag(job.x.st, LSMKV_ST_MISALIGNED, w_a.chunk);
                raw_slab[s] = u_a;
                raw_ok[s] = w_a.ok == 1u ? 1u : 0u;
                if (w_a.ok == 1u) {
                    mbar_arrive_expect(raw_full(s), (uint32_t)S::kPageBytes);
                    asm volatile(
                        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes"
                        " [%0], [%1], %2, [%3];"
                        :: "r"(smem_addr(raw + (size_t)s * S::kPageBytes)), "l"(w_a.src),
                           "r"((uint32_t)S::kPageBytes), "r"(raw_full(s)) : "memory");
                    fetch_mask |= 1u << s;
                    fetch_parity = (fetch_parity & ~(1u << s)) | (ph << s);
                } else {
                    fetch_mask &= ~(1u << s);
                    mbar_arrive(raw_full(s));
                }
            }
            u_a = u_b; w_a = w_b;
            u_b = u_c;
            u_c = u_d;
        }
        // Do not leave while a fetch may still be writing this CTA's shared memory. A stage
        // whose last arm was a fetch is waited for here (its group normally did so long ago); a
        // stage armed again since (stop mark, unusable page) had its earlier fetch consumed
        // before the producer was let back in.
        for (int s = 0; s < S::kRaw; ++s) {
            if (!(fetch_mask >> s & 1u)) continue;
            const long long t0 = clock64();
            while (!mbar_try(raw_full(s), (fetch_parity >> s) & 1u))
                if (clock64() - t0 > job.wait_cycles) break;
        }
        return;
    }

    if (warp >= (unsigned)S::kFirstCommitWarp) {
        // ---- commit warp c: slabs k = c, c + kOut, ... of this CTA, buffer c
        const int c = (int)warp - S::kFirstCommitWarp;
        const uint32_t obuf = smem_addr(outb + (size_t)c * S::kOutStride);
        for (uint32_t n = 0;; ++n) {
            bool ok = true;
            if (lane == 0) ok = mbar_wait(size_known(c, n), (n >> 1) & 1u, job);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) { if (lane == 0) raise_abort(job, 0); break; }
            uint64_t u = lane == 0 ? out_slab[2 * c + (n & 1u)] : 0;   // read by the lane that waited
            uint32_t size = lane == 0 ? out_size[2 * c + (n & 1u)] : 0;
            u = __shfl_sync(0xFFFFFFFFu, u, 0);
            size = __shfl_sync(0xFFFFFFFFu, size, 0);
            if (u == kEnd) break;
            const bool first = u % slabs == 0;            // the chunk's directory goes before it
            const uint64_t add = (uint64_t)size + (first ? job.x.dir_bytes : 0u);
            uint64_t before = 0;
            if (!look_back(job, u, &before)) { if (lane == 0) raise_abort(job, u); break; }
            if (lane == 0) {
                st_state(job.state + u, kFlagIncl | (before + add));
                ok = mbar_wait(out_full(c), n & 1u, job);             // the packed slab is there
                if (ok) {
                    if (before + add <= job.x.blob_capacity) {
                        unsigned char *dst = job.x.blob + before + (first ? job.x.dir_bytes : 0u);
                        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                     :: "l"(dst), "r"(obuf), "r"(size) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    } else {
                        st_flag(job.x.st, LSMKV_ST_OVERFLOW, u / slabs);
                    }
                    mbar_arrive(out_empty(c));
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) { if (lane == 0) raise_abort(job, u); break; }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        return;
    }

    // ---- compute group g: slabs k = g, g + kGroups, ... of this CTA
    const int g = (int)warp / S::kWpg;
    const unsigned gw = warp - (unsigned)g * S::kWpg;     // warp within the group
    const unsigned gt = threadIdx.x - (unsigned)g * S::kWpg * 32u;
    uint32_t *red_max = red + (size_t)g * 2 * S::kWpg, *red_cnt = red_max + S::kWpg;
    const uint32_t k_first = gw * S::kSweeps * 32 + lane; // this lane's first 16 bytes of the slab
    bool dead = false;                                    // a wait gave up: skip the rest
    for (uint32_t k = (uint32_t)g;; k += S::kGroups) {
        const int rs = (int)(k % S::kRaw), os = (int)(k % S::kOut);
        if (!dead && !mbar_wait(raw_full(rs), (k / S::kRaw) & 1u, job)) dead = true;
        uint64_t u = kEnd;
        bool page_ok = false;
        uint4 q[S::kSweeps];
        if (!dead) {
            u = raw_slab[rs];
            page_ok = u != kEnd && raw_ok[rs] != 0u;
        }
        if (page_ok) {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(raw + (size_t)rs * S::kPageBytes);
#pragma unroll
            for (int s = 0; s < S::kSweeps; ++s) q[s] = s4[k_first + s * 32];
        } else {
#pragma unroll
            for (int s = 0; s < S::kSweeps; ++s) q[s] = make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
        if (!dead && lane == 0) mbar_arrive(raw_empty(rs));   // the stage may be refilled
        // exponent fields of the slab's words (kept: the window test and the codes start from
        // them) and the largest of them
        uint32_t t[4 * S::kSweeps], least[S::kSweeps];    // least: smallest fields of a sweep
        uint32_t m = 0;
#pragma unroll
        for (int s = 0; s < S::kSweeps; ++s) {
            t[4 * s] = q[s].x & 0x7F807F80u; t[4 * s + 1] = q[s].y & 0x7F807F80u;
            t[4 * s + 2] = q[s].z & 0x7F807F80u; t[4 * s + 3] = q[s].w & 0x7F807F80u;
            m = __vimax3_u16x2(m, t[4 * s], t[4 * s + 1]);
            m = __vimax3_u16x2(m, t[4 * s + 2], t[4 * s + 3]);
            least[s] = __vimin3_u16x2(__vimin3_u16x2(t[4 * s], t[4 * s + 1], t[4 * s + 2]),
                                      t[4 * s + 3], t[4 * s + 3]);
        }
        m = max(m & 0xFFFFu, m >> 16);
#pragma unroll
        for (int d = 16; d; d >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
        if (lane == 0) red_max[gw] = m;
        // group barrier; it also tells every thread whether any of them gave up on a wait
        int any_dead;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 q, %1, 0;\n\t"
            "barrier.cta.red.or.pred p, %2, %3, q;\n\t"
            "selp.s32 %0, 1, 0, p;\n\t}"
            : "=r"(any_dead) : "r"(dead ? 1u : 0u), "r"(1 + g), "r"(S::kWpg * 32) : "memory");
        if (any_dead) {
            if (gt == 0) raise_abort(job, u == kEnd ? 0 : u);
            break;
        }
        if (u == kEnd) {
            // Stop marks for the commit warps: the buffers of the kOut slab positions that follow
            // the CTA's last real slab each get one, from the group whose turn that position is.
            const uint32_t K = *n_real;
            if (gt == 0) {
                for (uint32_t k2 = K; k2 < K + (uint32_t)S::kOut; ++k2) {
                    if (k2 % S::kGroups != (uint32_t)g) continue;
                    const int o2 = (int)(k2 % S::kOut);
                    const uint32_t n2 = k2 / S::kOut;
                    // (the mailbox of this parity was last used two uses ago, and this group
                    // packed the use between them only after the commit warp was done with that)
                    out_slab[2 * o2 + (n2 & 1u)] = kEnd;
                    mbar_arrive(size_known(o2, n2));
                }
            }
            break;
        }
        uint32_t emax = 0;
#pragma unroll
        for (int w = 0; w < S::kWpg; ++w) emax = max(emax, red_max[w]);
        emax >>= 7;
        const uint32_t base = emax > 14u ? emax - 14u : 0u;
        const uint32_t lift = xpfast::window_lift(base);
        // A field plus `lift` has bit 15 of its half set exactly when the element is in the
        // window, and then bits 7..10 of the half hold e - base with zeros up to bit 14. Elements
        // below the window are rare: a sweep is only looked at closely (and its count taken) when
        // its smallest fields say the warp has one.
        uint32_t my_exc = 0, exc_sweeps = 0;              // this lane's count; sweeps that had any
#pragma unroll
        for (int s = 0; s < S::kSweeps; ++s) {
            const uint32_t below = ~(least[s] + lift) & 0x80008000u;
            if (__any_sync(0xFFFFFFFFu, below != 0)) {
                my_exc += 8u - (__popc((t[4 * s] + lift) & 0x80008000u) +
                                __popc((t[4 * s + 1] + lift) & 0x80008000u) +
                                __popc((t[4 * s + 2] + lift) & 0x80008000u) +
                                __popc((t[4 * s + 3] + lift) & 0x80008000u));
                exc_sweeps |= 1u << s;
            }
        }
        // The fields are kept as f * 4097 = f + (f << 12) with f = field + lift: for a word whose
        // two elements are in the window that sets the low element's code right below the high
        // one's (bits 19..22 and 23..26: one byte's worth), and nothing overlaps or carries.
        const uint32_t lift4097 = lift * 4097u;
#pragma unroll
        for (int e = 0; e < 4 * S::kSweeps; ++e) t[e] = mad_u32(t[e], 4097u, lift4097);
        uint32_t warp_exc = 0;
        if (exc_sweeps) {                                 // the same in every lane of the warp
            warp_exc = my_exc;
#pragma unroll
            for (int d = 16; d; d >>= 1) warp_exc += __shfl_xor_sync(0xFFFFFFFFu, warp_exc, d);
        }
        if (lane == 0) red_cnt[gw] = warp_exc;
        asm volatile("barrier.cta.sync %0, %1;" :: "r"(1 + g), "r"(S::kWpg * 32) : "memory");
        uint32_t before = 0, n_exc = 0;
#pragma unroll
        for (int w = 0; w < S::kWpg; ++w) {
            const uint32_t c = red_cnt[w];
            if ((unsigned)w < gw) before += c;
            n_exc += c;
        }
        const bool packed = page_ok && n_exc < (uint32_t)N / 2;
        const uint32_t size = packed ? round16u(16u + N + N / 2 + n_exc) : 16u + 2u * N;
        const bool first = u % slabs == 0;
        // the size goes out before anything that may wait: later slabs' look-backs need it
        if (gt == 0) {
            const uint32_t n = k / S::kOut;               // which use of the buffer this is
            out_slab[2 * os + (n & 1u)] = u;
            out_size[2 * os + (n & 1u)] = size;
            mbar_arrive(size_known(os, n));               // the commit warp may start looking back
            // (after the arrive: an arrive orders the stores before it, and would sit out this
            // one's trip to L2)
            st_state(job.state + u, kFlagAgg | ((uint64_t)size + (first ? job.x.dir_bytes : 0u)));
        }
        if (!mbar_wait(out_empty(os), ((k / S::kOut) & 1u) ^ 1u, job)) {
            dead = true;                                  // reported at the next group barrier
            continue;
        }
        unsigned char *out = outb + (size_t)os * S::kOutStride;
        if (gt == 0)
            *reinterpret_cast<uint4 *>(out) =
                packed ? make_uint4(kXpMagic, n_exc, base, size) : make_uint4(kXpMagic, 0, 1u << 8, size);
        if (!packed) {                                    // raw slab (zeros for an unusable page)
            uint4 *o4 = reinterpret_cast<uint4 *>(out + 16) + k_first;
#pragma unroll
            for (int s = 0; s < S::kSweeps; ++s) o4[s * 32] = q[s];
        } else {
            unsigned char *sm = out + 16, *codes = sm + N, *exc = codes + N / 2;
            uint32_t at_warp = before;                    // exceptions before this warp's next one
#pragma unroll
            for (int s = 0; s < S::kSweeps; ++s) {
                const uint32_t kk = k_first + s * 32;
                const uint4 v = q[s];
                uint32_t c32;
                if (exc_sweeps >> s & 1u) {               // rare: a sweep with elements below
                    uint32_t x0, x1, x2, x3;
                    c32 = xpfast::code_byte(v.x, lift, x0) | (xpfast::code_byte(v.y, lift, x1) << 8) |
                          (xpfast::code_byte(v.z, lift, x2) << 16) | (xpfast::code_byte(v.w, lift, x3) << 24);
                    const uint32_t cnt = __popc(x0) + __popc(x1) + __popc(x2) + __popc(x3);
                    const uint32_t incl = xpfast::warp_incl_scan(cnt);
                    uint32_t at = at_warp + incl - cnt;
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w}, x[4] = {x0, x1, x2, x3};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (x[e] & 1u) exc[at++] = (unsigned char)((w[e] >> 7) & 0xFFu);
                        if (x[e] >> 16) exc[at++] = (unsigned char)((w[e] >> 23) & 0xFFu);
                    }
                    at_warp += __shfl_sync(0xFFFFFFFFu, incl, 31);
                } else {
                    // both codes of a word are the byte at bits 19..26 of its kept product
                    c32 = __byte_perm(__byte_perm(t[4 * s] >> 19, t[4 * s + 1] >> 19, 0x0040),
                                      __byte_perm(t[4 * s + 2] >> 19, t[4 * s + 3] >> 19, 0x0040), 0x5410);
                }
                *reinterpret_cast<uint2 *>(sm + 8ull * kk) = sm_bytes_mul(v);
                *reinterpret_cast<uint32_t *>(codes + 4ull * kk) = c32;
            }
            const uint32_t used = 16u + N + N / 2 + n_exc;
            if (gt < size - used) out[used + gt] = 0;     // padding up to the slab's size
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads it
        mbar_arrive(out_full(os));
    }
}

// After the encode: chunk directories and records from the slabs' prefixes.
__global__ void __launch_bounds__(256)
k_xpf_layout(const __grid_constant__ xpf::Job job)
{
    using namespace xpf;
    const uint32_t slabs = 2u * job.x.n_layers * job.x.pages_per_chunk;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < job.x.n_chunks;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t u0 = i * slabs;
        const uint64_t s_prev = u0 ? job.state[u0 - 1] : kFlagIncl;
        const uint64_t s_last = job.state[u0 + slabs - 1];
        const uint64_t off = s_prev & kValueMask, end = s_last & kValueMask;
        uint4 v;
        v.x = job.x.file_id;
        bool ok = (s_prev >> 62) == 2u && (s_last >> 62) == 2u;
        if (!ok) st_flag(job.x.st, LSMKV_ST_WAIT_EXPIRED, i);          // the encode was cut short
        if (ok && (end > job.x.blob_capacity || end - off > 0xFFFFFFFFull)) {
            st_flag(job.x.st, LSMKV_ST_OVERFLOW, i);
            ok = false;
        }
        if (!ok) {
            v.y = 0; v.z = 0; v.w = 0;
            *reinterpret_cast<uint4 *>(job.x.vals_out + i) = v;
            continue;
        }
        const uint64_t o = job.x.base_offset + off;
        v.y = (uint32_t)(end - off);
        v.z = (uint32_t)o;
        v.w = (uint32_t)(o >> 32);
        *reinterpret_cast<uint4 *>(job.x.vals_out + i) = v;
        uint32_t *dir = reinterpret_cast<uint32_t *>(job.x.blob + off);
        dir[0] = job.x.dir_bytes;
        for (uint32_t b = 1; b < slabs; ++b)
            dir[b] = (uint32_t)((job.state[u0 + b - 1] & kValueMask) - off);
        dir[slabs] = (uint32_t)(end - off);
        for (uint32_t k = slabs + 1; k < job.x.dir_bytes / 4; ++k) dir[k] = 0;
    }
}

}  // namespace lsmkv
