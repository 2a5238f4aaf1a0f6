// One-pass encoder of the compressing codec "xp12": every page slab is read from the pool once.
//
// The three-step encoder (lsmkv_xp12.cuh) reads the pool twice, because where a slab lands
// depends on the sizes of all slabs before it. Here a slab stays on the SM, in a ring of
// shared-memory stages, between being measured and being written. A persistent CTA per SM runs
//   producer warp    draws the next slab number from a counter and fetches the slab into the
//                    ring with one bulk copy (cp.async.bulk, mbarrier-completed);
//   measuring warps  take each slab as it lands: exponent window and exception count give its
//                    encoded size, which is published at once;
//   look-back warps  sum the sizes of all earlier slabs (decoupled look-back over a per-slab
//                    state word: empty / size known / prefix known), publish the prefix and
//                    hand the slab's place on;
//   packing warps    take a measured slab into registers, which frees its stage, wait for the
//                    slab's place, and encode it straight into the blob.
// The three run side by side on different slabs, so each one's chain of short dependent steps
// (waits, shuffles, barriers) hides behind the others' arithmetic; a slab's size is known well
// before its place is, and the stages plus the packing warps' registers are what absorbs the
// differences in pace between the SMs while a look-back waits for its slowest predecessor.
// Slab numbers are handed out in order by the counter, so every slab a look-back waits for is
// held by a CTA that is already running. A small kernel afterwards (k_xpf_layout) turns the
// prefixes into chunk directories and records. Bytes out are those of the three-step encoder.
//
// Every wait is bounded (the mbarrier waits and the look-back polls give up after `wait_cycles`
// clock cycles, set LSMKV_ST_WAIT_EXPIRED and an abort word that makes every other wait of the
// launch return at its next poll); the producer leaves only after its fetches have landed.
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

// Shape of the pipeline for a slab of WARPS * SWEEPS * 256 elements. Packing: GROUPS groups of
// WARPS warps, each warp owning a contiguous part of SWEEPS * 256 elements, a group per slab
// (group g takes slabs g, g + GROUPS, ...). Measuring: WARPS / SPLIT warps, each covering SPLIT
// such parts. RING stages; LB look-back warps that share the slabs round-robin. What one role
// tells the next about a slab travels in kQ mailboxes (with their barriers), more than there
// are stages: a packing group takes its slab into registers as soon as it is measured, frees
// the stage, and only then waits for the slab's place.
template <int SWEEPS, int WARPS, int SPLIT, int GROUPS, int RING, int LB>
struct Shape {
    static constexpr int kSweeps = SWEEPS, kWarps = WARPS, kSplit = SPLIT, kGroups = GROUPS,
                         kRing = RING, kLb = LB, kQ = RING + GROUPS <= 8 ? 8 : 16;
    static constexpr int kMeasureWarps = WARPS / SPLIT, kMeasureSweeps = SWEEPS * SPLIT;
    static constexpr int kElems = WARPS * SWEEPS * 256;
    static constexpr int kPageBytes = 2 * kElems;
    static constexpr int kFirstPackWarp = kMeasureWarps;
    static constexpr int kProducerWarp = kMeasureWarps + GROUPS * WARPS;
    static constexpr int kFirstLbWarp = kProducerWarp + 1;
    static constexpr int kThreads = (kMeasureWarps + GROUPS * WARPS + 1 + LB) * 32;
    static constexpr size_t kTail = 1536 + (size_t)kQ * WARPS * 8;   // barriers and mailboxes
    static constexpr size_t kSmem = (size_t)RING * kPageBytes + kTail;
    static_assert(RING >= 3 && LB >= 1 && WARPS <= 16 && WARPS % SPLIT == 0 && kMeasureSweeps <= 32 &&
                  kThreads <= 1024, "shape out of range");
    // a mailbox is used again kQ slabs later; by then the slab it served must be packed: a stage
    // is only refilled once its slab is in a group's registers, and a group takes one slab at a
    // time, so when slab k + kQ is fetched the slabs up to k + kQ - RING - GROUPS are packed
    static_assert(kQ >= RING + GROUPS && kQ >= LB + GROUPS, "too few mailboxes");
};

struct Job {
    XpJob x;                       // geometry, pool, page table, blob, status (slab_* unused)
    unsigned long long *ticket;    // [dev] next slab number; zero before the launch
    unsigned long long *state;     // [dev] one word per slab; zero before the launch
    unsigned int *abort;           // [dev] zero before the launch
    long long wait_cycles;         // limit of every wait
    uint64_t test_drop_slab;       // test hook: the fetch of this slab is armed but never started,
                                   // so the wait for it runs out (~0 = none)
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

// Windows of 32 state words fetched per trip to L2. The state words near the front are read by
// every SM at once while they are being written: the fewer a look-back fetches, the faster all
// of them go (measured on 8 GiB: 8 windows per trip 3.76 ms, 4: 3.22, 2: 3.01, 1: 2.90).
constexpr int kLookBackWindows = 1;
constexpr unsigned kLookBackNap = 256;   // ns to wait before asking again for a missing size

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
        uint64_t v[kLookBackWindows];
#pragma unroll
        for (int j = 0; j < kLookBackWindows; ++j) {
            const long long idx = pos - (j * 32 + (int)lane);
            v[j] = idx >= 0 ? ld_state(job.state + idx) : kFlagIncl;   // before slab 0: prefix 0
        }
        bool done = false, stalled = false;
#pragma unroll
        for (int j = 0; j < kLookBackWindows; ++j) {
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
        if (stalled) __nanosleep(kLookBackNap);           // a size is on its way: do not hammer L2
        if (stalled && (++polls & 15u) == 0) {
            const bool give_up = ld_abort(job.abort) != 0u || clock64() - t0 > job.wait_cycles;
            if (__any_sync(0xFFFFFFFFu, give_up)) return false;
        }
    }
    *prefix = sum;
    return true;
}

}  // namespace xpf

// Dynamic shared memory: kRing stages of page_bytes, then barriers and per-stage mailboxes.
template <class S>
__global__ void __launch_bounds__(S::kThreads, 1)
k_xpf_encode(const __grid_constant__ xpf::Job job)
{
    using namespace xpf;
    extern __shared__ __align__(128) unsigned char xpf_smem[];
    constexpr int N = S::kElems, R = S::kRing, W = S::kWarps, WM = S::kMeasureWarps,
                  SM = S::kMeasureSweeps, Q = S::kQ;
    unsigned char *ring = xpf_smem;
    unsigned char *tail = xpf_smem + (size_t)R * S::kPageBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail);             // 2 per stage, 2 per mailbox
    uint64_t *slot_u = bars + 2 * R + 2 * Q;                         // producer: slab number / kEnd
    uint64_t *m_u = slot_u + R;                                      // measure: the same, per mailbox
    uint64_t *m_prefix = m_u + Q;                                    // look-back: bytes before the slab
    uint32_t *slot_ok = reinterpret_cast<uint32_t *>(m_prefix + Q);  // producer: page usable
    uint32_t *m_ok = slot_ok + R + (R & 1);                          // measure: the same, per mailbox
    uint32_t *m_size = m_ok + Q;                                     // measure: encoded size
    uint32_t *m_info = m_size + Q;                                   // measure: base | packed << 8 | first << 9
    uint32_t *m_nexc = m_info + Q;                                   // measure: exceptions of the slab
    uint32_t *m_wcnt = m_nexc + Q;                                   // measure: [Q][W] exceptions before a part
    uint32_t *m_wsweeps = m_wcnt + Q * W;                            // measure: [Q][W] sweeps that have any
    uint32_t *red_max = m_wsweeps + Q * W;                           // [WM]
    static_assert((2 * R + 2 * Q + R + 2 * Q) * 8 + (R + 1 + 4 * Q + 2 * Q * W + WM) * 4 <= S::kTail,
                  "mailboxes do not fit");

    const uint32_t bar0 = smem_addr(bars);
    auto raw_full = [&](int s) { return bar0 + 8u * (uint32_t)s; };              // fetch landed
    auto raw_empty = [&](int s) { return bar0 + 8u * (uint32_t)(R + s); };       // slab taken into registers
    auto measured = [&](int q) { return bar0 + 8u * (uint32_t)(2 * R + q); };    // size known
    auto placed = [&](int q) { return bar0 + 8u * (uint32_t)(2 * R + Q + q); };  // prefix known

    const unsigned warp = threadIdx.x >> 5, lane = lane_id();
    if (threadIdx.x == 0) {
        for (int s = 0; s < R; ++s) {
            mbar_init(raw_full(s), 1);                    // the producer's arrive (+ copy bytes)
            mbar_init(raw_empty(s), W);                   // one arrive per warp of a packing group
        }
        for (int q = 0; q < Q; ++q) {
            mbar_init(measured(q), 1);                    // one measuring thread
            mbar_init(placed(q), 1);                      // one look-back lane
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();                                      // the only CTA-wide barrier

    const uint32_t slabs = 2u * job.x.n_layers * job.x.pages_per_chunk;
    const uint64_t total = job.x.n_chunks * slabs;

    if (warp == (unsigned)S::kProducerWarp) {
        // ---- producer: one lane hands out slab numbers and starts the fetches. Drawing a number,
        // reading its page id and its layer's pool pointer are dependent round trips to L2; the
        // number is drawn three slabs ahead, the two loads are started one slab ahead and their
        // values first looked at after the wait for the stage, so none of them holds the loop.
        if (lane != 0) return;
        struct Where { const unsigned char *src; uint64_t chunk; uint32_t ok, first_of_page, first_of_chunk; };
        // loads on their way, and where the slab sits: chunk, slab of the chunk, slab of the page
        struct Asked { uint64_t page; const unsigned char *pool_buf; uint64_t chunk; uint32_t b, bb; };
        // One lane divides on its own here, and a 64-bit division is a chain of some eighty
        // dependent instructions: slab number / slabs per chunk is taken from the reciprocal
        // (at most one too small for any 63-bit number, put right by one comparison), slab of
        // the chunk / slabs per page likewise in 32 bits.
        const uint32_t per_page = 2u * job.x.n_layers;
        const uint64_t inv_slabs = ~0ull / slabs;
        const uint32_t inv_per_page = 0xFFFFFFFFu / per_page;
        auto draw = [&](bool ended) -> uint64_t {
            return ended ? total : (uint64_t)atomicAdd(job.ticket, 1ull);
        };
        auto ask = [&](uint64_t u) -> Asked {
            Asked a{0, nullptr, 0, 0u, 0u};
            if (u >= total) return a;
            uint64_t i = __umul64hi(u, inv_slabs);
            uint64_t b64 = u - i * slabs;
            if (b64 >= slabs) { ++i; b64 -= slabs; }
            const uint32_t b = (uint32_t)b64;
            uint32_t pg = __umulhi(b, inv_per_page), bb = b - pg * per_page;
            if (bb >= per_page) { ++pg; bb -= per_page; }
            a.chunk = i;
            a.b = b;
            a.bb = bb;
            a.page = __ldg(job.x.page_table + i * job.x.pages_per_chunk + pg);
            a.pool_buf = static_cast<const unsigned char *>(
                job.x.kv_ptrs[(bb & 1u) * job.x.n_layers + (bb >> 1)]);
            return a;
        };
        auto locate = [&](uint64_t u, const Asked &a) -> Where {
            Where w{nullptr, 0, 0u, 0u, 0u};
            if (u >= total) return w;
            w.chunk = a.chunk;
            w.first_of_page = a.bb == 0 ? 1u : 0u;
            w.first_of_chunk = a.b == 0 ? 2u : 0u;
            if (a.page >= job.x.num_pages) w.ok = 2u;                     // unusable page id
            else if ((reinterpret_cast<uintptr_t>(a.pool_buf) & 15u) != 0) w.ok = 3u;   // misaligned
            else { w.ok = 1u; w.src = a.pool_buf + a.page * (uint64_t)S::kPageBytes; }
            return w;
        };
        bool ended = false;
        uint32_t fetch_mask = 0, fetch_parity = 0;        // per stage: last arm was a fetch / its phase
        uint32_t k = 0;                                   // slabs of this CTA so far
        // One slab: draws the number three slabs ahead into `u_d`, asks for the loads of the
        // next slab `u_b` into `q_b`, and fetches slab `u_a` whose loads `q_a` were asked for a
        // slab ago. False when the loop is over. The caller rotates the variables by name: a
        // copy of a value still on its way would wait for it.
        auto step = [&](uint64_t &u_a, const uint64_t &u_b, uint64_t &u_d, const Asked &q_a,
                        Asked &q_b) -> bool {
            u_d = draw(ended);
            q_b = ask(u_b);
            ended = ended || u_b >= total;
            const int s = (int)(k % R);
            const uint32_t ph = (k / R) & 1u;
            ++k;
            if (!mbar_wait(raw_empty(s), ph ^ 1u, job)) { raise_abort(job, 0); return false; }
            const Where w_a = locate(u_a, q_a);
            if (u_a >= total) {                           // the stop mark
                slot_u[s] = kEnd;
                fetch_mask &= ~(1u << s);
                mbar_arrive(raw_full(s));
                return false;
            }
            if (w_a.ok == 2u && w_a.first_of_page) st_flag(job.x.st, LSMKV_ST_BAD_PAGE, w_a.chunk);
            if (w_a.ok == 3u) st_flag(job.x.st, LSMKV_ST_MISALIGNED, w_a.chunk);
            slot_u[s] = u_a;
            slot_ok[s] = (w_a.ok == 1u ? 1u : 0u) | w_a.first_of_chunk;   // bit 1: the chunk's first slab
            if (w_a.ok == 1u && u_a == job.test_drop_slab) {
                mbar_arrive_expect(raw_full(s), (uint32_t)S::kPageBytes);   // and nothing comes
                fetch_mask &= ~(1u << s);
            } else if (w_a.ok == 1u) {
                mbar_arrive_expect(raw_full(s), (uint32_t)S::kPageBytes);
                asm volatile(
                    "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes"
                    " [%0], [%1], %2, [%3];"
                    :: "r"(smem_addr(ring + (size_t)s * S::kPageBytes)), "l"(w_a.src),
                       "r"((uint32_t)S::kPageBytes), "r"(raw_full(s)) : "memory");
                fetch_mask |= 1u << s;
                fetch_parity = (fetch_parity & ~(1u << s)) | (ph << s);
            } else {
                fetch_mask &= ~(1u << s);
                mbar_arrive(raw_full(s));
            }
            return true;
        };
        uint64_t u0 = draw(false), u1 = draw(false), u2 = draw(false), u3 = 0;
        Asked q0 = ask(u0), q1{0, nullptr, 0, 0u, 0u};
        for (;;) {
            if (!step(u0, u1, u3, q0, q1)) break;
            if (!step(u1, u2, u0, q1, q0)) break;
            if (!step(u2, u3, u1, q0, q1)) break;
            if (!step(u3, u0, u2, q1, q0)) break;
        }
        // Do not leave while a fetch may still be writing this CTA's shared memory. A stage
        // whose last arm was a fetch is waited for here (the compute warps normally did so long
        // ago); a stage armed again since (stop mark, unusable page) had its earlier fetch read
        // before the producer was let back in.
        for (int s = 0; s < R; ++s) {
            if (!(fetch_mask >> s & 1u)) continue;
            const long long t0 = clock64();
            while (!mbar_try(raw_full(s), (fetch_parity >> s) & 1u))
                if (clock64() - t0 > job.wait_cycles) break;
        }
        return;
    }

    if (warp >= (unsigned)S::kFirstLbWarp) {
        // ---- look-back warp c: slabs k = c, c + kLb, ... of this CTA, as soon as they are measured
        const uint32_t c = warp - (unsigned)S::kFirstLbWarp;
        for (uint32_t k = c;; k += S::kLb) {
            const int s = (int)(k % Q);                   // the slab's mailbox
            bool ok = true;
            if (lane == 0) ok = mbar_wait(measured(s), (k / Q) & 1u, job);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) { if (lane == 0) raise_abort(job, 0); break; }
            uint64_t u = lane == 0 ? m_u[s] : 0;          // read by the lane that waited
            uint32_t size = 0;
            if (lane == 0 && u != kEnd) size = m_size[s] + ((m_info[s] & 0x200u) ? job.x.dir_bytes : 0u);
            u = __shfl_sync(0xFFFFFFFFu, u, 0);
            size = __shfl_sync(0xFFFFFFFFu, size, 0);
            if (u == kEnd) break;
            const uint64_t add = size;                    // bytes the slab adds to the blob
            uint64_t before = 0;
            if (!look_back(job, u, &before)) { if (lane == 0) raise_abort(job, u); break; }
            if (lane == 0) {
                m_prefix[s] = before;
                mbar_arrive(placed(s));                   // the compute warps may pack it
                st_state(job.state + u, kFlagIncl | (before + add));
            }
            __syncwarp();
        }
        return;
    }

    if (warp < (unsigned)S::kFirstPackWarp) {
        // ---- measuring warps: slab j of this CTA as soon as it has landed
        const unsigned gt = threadIdx.x;                  // thread within the measuring group
        const uint32_t k_first = warp * SM * 32 + lane;   // this lane's first 16 bytes of a slab
        bool dead = false;                                // a wait gave up: do nothing but leave
        for (uint32_t j = 0;; ++j) {
            const int s = (int)(j % R), qs = (int)(j % Q);    // the slab's stage and mailbox
            if (!dead && !mbar_wait(raw_full(s), (j / R) & 1u, job)) dead = true;
            uint64_t u = kEnd;
            bool page_ok = false;
            if (!dead) {
                u = slot_u[s];
                page_ok = u != kEnd && (slot_ok[s] & 1u) != 0u;
            }
            // the largest exponent field of the slab, and the smallest of every sweep (an
            // unusable page measures as zeros)
            uint32_t least[SM];
            uint32_t m = 0;
            const uint4 *s4 = reinterpret_cast<const uint4 *>(ring + (size_t)s * S::kPageBytes);
#pragma unroll
            for (int e = 0; e < SM; ++e) {
                const uint4 v = page_ok ? s4[k_first + e * 32] : make_uint4(0, 0, 0, 0);
                const uint32_t f0 = v.x & 0x7F807F80u, f1 = v.y & 0x7F807F80u,
                               f2 = v.z & 0x7F807F80u, f3 = v.w & 0x7F807F80u;
                m = __vimax3_u16x2(m, f0, f1);
                m = __vimax3_u16x2(m, f2, f3);
                least[e] = __vimin3_u16x2(__vimin3_u16x2(f0, f1, f2), f3, f3);
            }
            m = max(m & 0xFFFFu, m >> 16);
#pragma unroll
            for (int d = 16; d; d >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
            if (lane == 0) red_max[warp] = m;
            // group barrier; it also tells every thread whether any of them gave up on a wait
            int any_dead;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 q, %1, 0;\n\t"
                "barrier.cta.red.or.pred p, 1, %2, q;\n\t"
                "selp.s32 %0, 1, 0, p;\n\t}"
                : "=r"(any_dead) : "r"(dead ? 1u : 0u), "r"(WM * 32) : "memory");
            if (any_dead) {
                if (gt == 0) raise_abort(job, u == kEnd ? 0 : u);
                break;
            }
            if (u == kEnd) {
                // No more slabs. Every look-back warp and every packing group finds a stop mark
                // at its next position (mailboxes are free that far ahead: see the shape).
                if (gt == 0) {
                    constexpr uint32_t kMarks = S::kLb > S::kGroups ? S::kLb : S::kGroups;
                    for (uint32_t k2 = j; k2 < j + kMarks; ++k2) {
                        m_u[k2 % Q] = kEnd;
                        mbar_arrive(measured((int)(k2 % Q)));
                    }
                }
                break;
            }
            uint32_t emax = 0;
#pragma unroll
            for (int w = 0; w < WM; ++w) emax = max(emax, red_max[w]);
            emax >>= 7;
            const uint32_t base = emax > 14u ? emax - 14u : 0u;
            const uint32_t lift = xpfast::window_lift(base);
            // A field plus `lift` has bit 15 of its half set exactly when the element is in the
            // window. Elements below it are rare: a sweep is only looked at closely (and its
            // count taken) when its smallest fields say the warp has one.
            // (the sweep is then read again from the stage, which stays as it is until packed).
            // Counts and sweep masks are kept per part of the slab, one part per packing warp.
            uint32_t my_exc[S::kSplit], exc_sweeps[S::kSplit];
#pragma unroll
            for (int p = 0; p < S::kSplit; ++p) my_exc[p] = exc_sweeps[p] = 0;
#pragma unroll
            for (int e = 0; e < SM; ++e) {
                const uint32_t below = ~(least[e] + lift) & 0x80008000u;
                if (__any_sync(0xFFFFFFFFu, below != 0)) {
                    const uint4 v = page_ok ? s4[k_first + e * 32] : make_uint4(0, 0, 0, 0);
                    my_exc[e / S::kSweeps] +=
                        8u - (__popc(((v.x & 0x7F807F80u) + lift) & 0x80008000u) +
                              __popc(((v.y & 0x7F807F80u) + lift) & 0x80008000u) +
                              __popc(((v.z & 0x7F807F80u) + lift) & 0x80008000u) +
                              __popc(((v.w & 0x7F807F80u) + lift) & 0x80008000u));
                    exc_sweeps[e / S::kSweeps] |= 1u << (e % S::kSweeps);
                }
            }
#pragma unroll
            for (int p = 0; p < S::kSplit; ++p) {
                uint32_t part_exc = 0;
                if (exc_sweeps[p]) {                      // the same in every lane of the warp
                    part_exc = my_exc[p];
#pragma unroll
                    for (int d = 16; d; d >>= 1) part_exc += __shfl_xor_sync(0xFFFFFFFFu, part_exc, d);
                }
                if (lane == 0) {
                    m_wcnt[qs * W + warp * S::kSplit + p] = part_exc;
                    m_wsweeps[qs * W + warp * S::kSplit + p] = exc_sweeps[p];
                }
            }
            asm volatile("barrier.cta.sync 1, %0;" :: "r"(WM * 32) : "memory");
            if (warp == 0) {
                // counts become "exceptions before the part": a scan over the W parts by lanes
                static_assert(W <= 32, "one lane per part");
                const uint32_t c = lane < (unsigned)W ? m_wcnt[qs * W + lane] : 0u;
                const uint32_t incl = xpfast::warp_incl_scan(c);
                if (lane < (unsigned)W) m_wcnt[qs * W + lane] = incl - c;
                const uint32_t n_exc = __shfl_sync(0xFFFFFFFFu, incl, 31);
                __syncwarp();
                if (lane == 0) {
                    const bool packed = page_ok && n_exc < (uint32_t)N / 2;
                    const uint32_t size = packed ? round16u(16u + N + N / 2 + n_exc) : 16u + 2u * N;
                    const bool first = (slot_ok[s] & 2u) != 0u;   // the chunk's directory goes before it
                    m_u[qs] = u;
                    m_ok[qs] = page_ok ? 1u : 0u;
                    m_size[qs] = size;
                    m_info[qs] = base | (packed ? 0x100u : 0u) | (first ? 0x200u : 0u);
                    m_nexc[qs] = n_exc;
                    mbar_arrive(measured(qs));            // look-back and packing take it from here
                    // (after the arrive: an arrive orders the stores before it, and would sit
                    // out this one's trip to L2)
                    st_state(job.state + u,
                             kFlagAgg | ((uint64_t)size + (first ? job.x.dir_bytes : 0u)));
                }
            }
        }
        return;
    }

    // ---- packing groups: group g takes slabs g, g + kGroups, ... of this CTA. A slab goes into
    // the group's registers as soon as it is measured, which frees its stage; the group then
    // waits for the slab's place and encodes it straight into the blob. Each warp runs on its
    // own: no barrier, only the mbarriers of the stage and of the mailbox.
    const unsigned pg = (warp - (unsigned)S::kFirstPackWarp) / W;      // this warp's group
    const unsigned pw = (warp - (unsigned)S::kFirstPackWarp) % W;      // its part of a slab
    const unsigned pt = pw * 32u + lane;                                // thread within the group
    const uint32_t k_first = pw * S::kSweeps * 32 + lane;     // this lane's first 16 bytes of a slab
    for (uint32_t k = pg;; k += S::kGroups) {
        const int s = (int)(k % R), qs = (int)(k % Q);
        if (!mbar_wait(measured(qs), (k / Q) & 1u, job)) { raise_abort(job, 0); break; }
        const uint64_t u = m_u[qs];
        if (u == kEnd) break;
        const bool page_ok = m_ok[qs] != 0u;
        uint4 q[S::kSweeps];
        {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(ring + (size_t)s * S::kPageBytes);
#pragma unroll
            for (int e = 0; e < S::kSweeps; ++e)
                q[e] = page_ok ? s4[k_first + e * 32] : make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(raw_empty(s));         // this warp is done with the stage
        if (!mbar_wait(placed(qs), (k / Q) & 1u, job)) { raise_abort(job, u); break; }
        const uint64_t before_bytes = m_prefix[qs];
        const uint32_t size = m_size[qs], info = m_info[qs], n_exc = m_nexc[qs];
        const bool packed = (info & 0x100u) != 0u;
        const uint32_t my_sweeps = m_wsweeps[qs * W + pw];
        const uint32_t exc_before = m_wcnt[qs * W + pw];  // exceptions of the parts before this one
        const bool first = (info & 0x200u) != 0u;         // the chunk's directory goes before it
        const uint64_t add = (uint64_t)size + (first ? job.x.dir_bytes : 0u);
        if (before_bytes + add > job.x.blob_capacity) {   // cannot happen with a worst-case buffer
            if (pt == 0) st_flag(job.x.st, LSMKV_ST_OVERFLOW, u / slabs);
            continue;
        }
        unsigned char *out = job.x.blob + before_bytes + (first ? job.x.dir_bytes : 0u);
        if (pt == 0)
            __stcs(reinterpret_cast<uint4 *>(out),
                   packed ? make_uint4(kXpMagic, n_exc, info & 0xFFu, size)
                          : make_uint4(kXpMagic, 0, 1u << 8, size));
        if (!packed) {                                    // raw slab (zeros for an unusable page)
            uint4 *o4 = reinterpret_cast<uint4 *>(out + 16) + k_first;
#pragma unroll
            for (int e = 0; e < S::kSweeps; ++e) __stcs(o4 + e * 32, q[e]);
            continue;
        }
        unsigned char *sm = out + 16, *codes = sm + N, *exc = codes + N / 2;
        const uint32_t lift = xpfast::window_lift(info & 0xFFu), lift4097 = lift * 4097u;
        uint32_t at_warp = exc_before;                    // exceptions before this warp's next one
#pragma unroll
        for (int e = 0; e < S::kSweeps; ++e) {
            const uint32_t kk = k_first + e * 32;
            const uint4 v = q[e];
            uint32_t c32;
            if (my_sweeps >> e & 1u) {                    // rare: a sweep with elements below
                uint32_t x0, x1, x2, x3;
                c32 = xpfast::code_byte(v.x, lift, x0) | (xpfast::code_byte(v.y, lift, x1) << 8) |
                      (xpfast::code_byte(v.z, lift, x2) << 16) | (xpfast::code_byte(v.w, lift, x3) << 24);
                const uint32_t cnt = __popc(x0) + __popc(x1) + __popc(x2) + __popc(x3);
                const uint32_t incl = xpfast::warp_incl_scan(cnt);
                uint32_t at = at_warp + incl - cnt;
                const uint32_t w[4] = {v.x, v.y, v.z, v.w}, x[4] = {x0, x1, x2, x3};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (x[i] & 1u) exc[at++] = (unsigned char)((w[i] >> 7) & 0xFFu);
                    if (x[i] >> 16) exc[at++] = (unsigned char)((w[i] >> 23) & 0xFFu);
                }
                at_warp += __shfl_sync(0xFFFFFFFFu, incl, 31);
            } else {
                // With f = field + lift, f * 4097 = f + (f << 12) sets the low element's code
                // right below the high one's (bits 19..22 and 23..26); for a word whose elements
                // are both in the window nothing overlaps or carries, and the byte at bits
                // 19..26 is the word's code byte.
                const uint32_t y0 = mad_u32(v.x & 0x7F807F80u, 4097u, lift4097) >> 19,
                               y1 = mad_u32(v.y & 0x7F807F80u, 4097u, lift4097) >> 19,
                               y2 = mad_u32(v.z & 0x7F807F80u, 4097u, lift4097) >> 19,
                               y3 = mad_u32(v.w & 0x7F807F80u, 4097u, lift4097) >> 19;
                c32 = __byte_perm(__byte_perm(y0, y1, 0x0040), __byte_perm(y2, y3, 0x0040), 0x5410);
            }
            __stcs(reinterpret_cast<uint2 *>(sm + 8ull * kk), sm_bytes_mul(v));
            __stcs(reinterpret_cast<uint32_t *>(codes + 4ull * kk), c32);
        }
        const uint32_t used = 16u + N + N / 2 + n_exc;
        if (pt < size - used) out[used + pt] = 0;         // padding up to the slab's size
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
        const uint64_t o = job.x.base_offset + off + (job.x.base_add ? *job.x.base_add : 0ull);
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
