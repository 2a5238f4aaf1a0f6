// liblsmkv: host side of the C ABI declared in include/lsmkv.h. Validates arguments, keeps the
// per-context workspace, and enqueues the kernels on the caller's stream. Nothing here touches
// payload bytes on the host.
#include <cstdio>
#include <cstdlib>
#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "lsmkv.h"
#include "lsmkv_common.cuh"
#include "lsmkv_copy.cuh"
#include "lsmkv_keys.cuh"
#include "lsmkv_probe.cuh"
#include "lsmkv_sort.cuh"
#include "lsmkv_xp12.cuh"
#include "lsmkv_xp12_fused.cuh"
#include "lsmkv_xrun.cuh"

using namespace lsmkv;

struct lsmkv_ctx {
    lsmkv_geom_t geom;
    int device;
    int sm_count;
    int max_smem_optin;
    uint64_t page_bytes, chunk_bytes;
    KeyConsts kc;
    DevStatus *d_status;
    // workspace: hit_off u64[ws_seq + 1] followed by plan u32[ws_chunks]
    void *d_ws;
    uint64_t ws_seq, ws_chunks;
    // scratch of flush / compaction (key and index ping-pong buffers, records, block counts)
    void *d_sort;
    uint64_t sort_cap;
    // compressing codec: 0 = identity, 1 = xp12; scratch of its encoder
    uint32_t codec;
    uint32_t xp_dir_bytes;
    void *d_xp;
    uint64_t xp_cap;     // chunks
    const uint64_t *xp_base_add;   // set by the host-buffer put for its next encode, else NULL
    // fence-pointer directory of the probe: u64[n_runs * (jcap + 1)]
    uint64_t *d_dir;
    uint64_t dir_cap;
    int last_cuda;
    int last_cuda_line;   // source line of the failing CUDA call (diagnostics)
    uint64_t launches;
    // tuning
    int64_t copy_mode, copy_stage_bytes, copy_stages, copy_ctas_per_sm, copy_l2_hint;
    int64_t probe_warps_per_cta, simt_ctas_per_sm, host_stage_bytes, xp_generic;
    int64_t xp_one_pass, wait_cycles, host_copy_ctas, host_put_device_placed, test_drop_piece;
    int64_t host_copy_piece;
    uint32_t ppc;        // pages per chunk: chunk_tokens / page_tokens
    // host-buffer calls: device staging and host scratch
    void *d_io[3];
    uint64_t io_cap[3];
    cudaStream_t io_stream;          // second stream + events of the compressing host-buffer put
    cudaEvent_t io_ev_enc, io_ev_free[2];
    std::vector<uint64_t> h_off_a;
    std::vector<uint32_t> h_cuts;
    struct HostScratch { void *p; size_t cap; cudaEvent_t done; bool used; };
    HostScratch hs[3][2];
    int hs_next[3];
    // optional per-kernel timing with CUDA events on the launching stream
    bool profiling;
    struct Timed { cudaEvent_t a, b; int cls; };
    std::vector<Timed> pending;
    std::vector<cudaEvent_t> free_events;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int cuda_fail(lsmkv_ctx *ctx, cudaError_t e, int line = 0)
{
    if (ctx) { ctx->last_cuda = (int)e; ctx->last_cuda_line = line; }
    cudaGetLastError();   // clear the sticky-less error state
    return LSMKV_ECUDA;
}

#define CU(ctx, call)                                            \
    do {                                                         \
        cudaError_t e__ = (call);                                \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__, __LINE__); \
    } while (0)

// (a * b) mod (2^61 - 1) on the host, for the power tables only
uint64_t host_mulmod(uint64_t a, uint64_t b)
{
    const unsigned __int128 x = (unsigned __int128)a * b;
    uint64_t s = (uint64_t)(x & kP) + (uint64_t)(x >> 61);
    s = (s & kP) + (s >> 61);
    return s >= kP ? s - kP : s;
}

uint64_t host_powmod(uint64_t b, uint64_t e)
{
    uint64_t r = 1;
    while (e) {
        if (e & 1) r = host_mulmod(r, b);
        b = host_mulmod(b, b);
        e >>= 1;
    }
    return r;
}

// tab [host, 4 * kKeyTab]: powers and inverse powers of M = BASE ^ C (layout: see KeyConsts)
void fill_key_consts(KeyConsts &kc, uint32_t C, uint64_t *tab)
{
    const uint64_t mA = host_powmod(kBaseA, C), mB = host_powmod(kBaseB, C);
    const uint64_t iA = host_powmod(mA, kP - 2), iB = host_powmod(mB, kP - 2);   // p is prime
    uint64_t a = mA, b = mB, ia = 1, ib = 1;
    for (int i = 0; i < kKeyTab; ++i) {
        tab[i] = a;
        tab[kKeyTab + i] = b;
        tab[2 * kKeyTab + i] = ia;
        tab[3 * kKeyTab + i] = ib;
        a = host_mulmod(a, mA);
        b = host_mulmod(b, mB);
        ia = host_mulmod(ia, iA);
        ib = host_mulmod(ib, iB);
    }
    // weights of the 16 tokens of a block, BASE^(15-i), in limbs of 21 + 21 + 19 bits
    a = 1;
    b = 1;
    kc.sumA = 0;
    kc.sumB = 0;
    for (int i = 15; i >= 0; --i) {
        const uint64_t w[2] = {a, b};
        for (int x = 0; x < 2; ++x) {
            uint32_t *d = x == 0 ? kc.dA[i] : kc.dB[i];
            d[0] = (uint32_t)(w[x] & 0x1FFFFFu);
            d[1] = (uint32_t)((w[x] >> 21) & 0x1FFFFFu);
            d[2] = (uint32_t)(w[x] >> 42);
        }
        kc.sumA = (kc.sumA + a) % kP;
        kc.sumB = (kc.sumB + b) % kP;
        a = host_mulmod(a, kBaseA);
        b = host_mulmod(b, kBaseB);
    }
    kc.b16A = a;
    kc.b16B = b;
}

// Brackets one kernel launch with events when profiling is on.
// Around the launches of one ABI call: an NVTX range named after the kernel class (a no-op
// unless a tool that collects NVTX is attached) and, when profiling is on, a pair of events.
struct LaunchTimer {
    lsmkv_ctx *ctx;
    cudaStream_t s;
    lsmkv_ctx::Timed t{};
    bool on;
    static const char *range_name(int cls)
    {
        static const char *const names[LSMKV_K_CLASSES] = {
            "lsmkv:keys", "lsmkv:pack", "lsmkv:probe", "lsmkv:plan",
            "lsmkv:unpack", "lsmkv:flush", "lsmkv:merge", "lsmkv:other"};
        return names[cls >= 0 && cls < LSMKV_K_CLASSES ? cls : LSMKV_K_CLASSES - 1];
    }
    static cudaEvent_t get(lsmkv_ctx *c)
    {
        cudaEvent_t e = nullptr;
        if (!c->free_events.empty()) { e = c->free_events.back(); c->free_events.pop_back(); }
        else if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); e = nullptr; }
        return e;
    }
    LaunchTimer(lsmkv_ctx *c, cudaStream_t st, int cls) : ctx(c), s(st), on(c->profiling)
    {
        nvtxRangePushA(range_name(cls));
        if (!on) return;
        t.a = get(c);
        t.b = get(c);
        t.cls = cls;
        if (!t.a || !t.b) { on = false; return; }
        cudaEventRecord(t.a, s);
    }
    ~LaunchTimer()
    {
        nvtxRangePop();
        if (!on) return;
        cudaEventRecord(t.b, s);
        ctx->pending.push_back(t);
    }
};

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The bulk copy kernels and the one-pass encoder take their stages as dynamic shared memory
// beyond the default limit.
// The limit is a per-device attribute of the function: it is raised once per device, to the
// device's maximum, with that device current -- never per call with a call-specific size, so
// that callers on different host threads (regular and allocation-free decodes alike) cannot
// lower it under one another between setting it and launching.
// one-pass encoder of the compressing codec: slabs of 8192 and 16384 elements
using XpfShape8k = xpf::Shape<2, 16, 2, 1, 12, 1>;
using XpfShape16k = xpf::Shape<4, 16, 2, 1, 7, 1>;

constexpr int kMaxDevices = 64;
std::mutex g_smem_limit_mu;
bool g_smem_limit_set[kMaxDevices];

cudaError_t set_copy_smem_limit(int max_smem_optin)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_smem_limit_mu);
    if (g_smem_limit_set[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(k_copy_slabs_bulk<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             max_smem_optin);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_copy_slabs_bulk<false>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem_optin);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_xpf_encode<XpfShape8k>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)XpfShape8k::kSmem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_xpf_encode<XpfShape16k>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)XpfShape16k::kSmem);
    if (e == cudaSuccess) g_smem_limit_set[dev] = true;
    return e;
}

// Every scratch buffer of a context has exactly one owner (a pointer field and its capacity
// field) and goes through the two helpers below: nothing else frees or replaces one.
// release_scratch: free, null the pointer and zero the capacity in one step, so that a stale
// pointer can never be used or freed again; the result of cudaFree is reported.
template <typename T>
int release_scratch(lsmkv_ctx *ctx, T **slot, uint64_t *cap, int line)
{
    if (!*slot) { *cap = 0; return LSMKV_OK; }
    void *old = *slot;
    *slot = nullptr;
    *cap = 0;
    const cudaError_t e = cudaFree(old);   // waits for work that may still use the buffer
    return e == cudaSuccess ? LSMKV_OK : cuda_fail(ctx, e, line);
}

// grow_scratch: a fresh allocation of `bytes` replaces the slot's buffer; `cap` receives
// `new_cap` (in whatever unit the owner counts). On failure the old buffer stays in place.
template <typename T>
int grow_scratch(lsmkv_ctx *ctx, T **slot, uint64_t *cap, size_t bytes, uint64_t new_cap, int line)
{
    void *p = nullptr;
    const cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { cuda_fail(ctx, e, line); return LSMKV_ENOMEM; }
    const int rc = release_scratch(ctx, slot, cap, line);
    if (rc != LSMKV_OK) { cudaFree(p); return rc; }
    *slot = static_cast<T *>(p);
    *cap = new_cap;
    return LSMKV_OK;
}

int ensure_workspace(lsmkv_ctx *ctx, uint64_t n_seq, uint64_t n_chunks)
{
    if (n_seq <= ctx->ws_seq && n_chunks <= ctx->ws_chunks && ctx->d_ws) return LSMKV_OK;
    const uint64_t ns = n_seq > ctx->ws_seq ? n_seq : ctx->ws_seq;
    const uint64_t nc = n_chunks > ctx->ws_chunks ? n_chunks : ctx->ws_chunks;
    const size_t bytes = (size_t)(ns + 2) * 8 + (size_t)(nc + 4) * 4;
    const int rc = grow_scratch(ctx, &ctx->d_ws, &ctx->ws_seq, bytes, ns, __LINE__);
    ctx->ws_chunks = rc == LSMKV_OK ? nc : (ctx->d_ws ? ctx->ws_chunks : 0);
    return rc;
}

int ensure_dir(lsmkv_ctx *ctx, uint64_t entries)
{
    if (entries <= ctx->dir_cap && ctx->d_dir) return LSMKV_OK;
    return grow_scratch(ctx, &ctx->d_dir, &ctx->dir_cap, (size_t)entries * sizeof(uint64_t),
                        entries, __LINE__);
}

struct SortWs {
    lsmkv_key_t *keys[2];
    uint32_t *idx[2];
    lsmkv_val_t *vals;
    uint64_t *block_count;
};

size_t sort_ws_bytes(uint64_t n)
{
    return (size_t)n * (2 * 32 + 2 * 4 + 16) + ((size_t)n / kScanBlock + 4) * 8 + 256;
}

int ensure_sort(lsmkv_ctx *ctx, uint64_t n, SortWs *ws)
{
    if (n > ctx->sort_cap || !ctx->d_sort) {
        const int rc = grow_scratch(ctx, &ctx->d_sort, &ctx->sort_cap, sort_ws_bytes(n), n, __LINE__);
        if (rc != LSMKV_OK) return rc;
    }
    const uint64_t cap = ctx->sort_cap;
    unsigned char *b = static_cast<unsigned char *>(ctx->d_sort);
    ws->keys[0] = reinterpret_cast<lsmkv_key_t *>(b);
    ws->keys[1] = reinterpret_cast<lsmkv_key_t *>(b + cap * 32);
    ws->vals = reinterpret_cast<lsmkv_val_t *>(b + cap * 64);
    ws->block_count = reinterpret_cast<uint64_t *>(b + cap * 80);
    const size_t bc = ((size_t)cap / kScanBlock + 4) * 8;
    ws->idx[0] = reinterpret_cast<uint32_t *>(b + cap * 80 + bc);
    ws->idx[1] = ws->idx[0] + cap;
    return LSMKV_OK;
}

// flag / scan / scatter: sorted keys + origin indices -> final run (+ padding) and its length
int launch_dedupe(lsmkv_ctx *ctx, cudaStream_t s, const SortWs &ws, int buf, uint64_t n,
                  const lsmkv_val_t *vals_in, int keep_last, lsmkv_key_t *keys_out,
                  lsmkv_val_t *vals_out, uint64_t *n_out)
{
    const uint64_t blocks = (n + kScanBlock - 1) / kScanBlock;
    k_dedupe_count<<<(unsigned)blocks, kScanBlock, 0, s>>>(ws.keys[buf], n, keep_last,
                                                            ws.block_count);
    k_scan_blocks<<<1, 1024, 0, s>>>(ws.block_count, blocks, n_out);
    k_dedupe_scatter<<<(unsigned)blocks, kScanBlock, 0, s>>>(ws.keys[buf], ws.idx[buf], vals_in,
                                                              n, keep_last, ws.block_count, n_out,
                                                              keys_out, vals_out);
    ctx->launches += 3;
    CU(ctx, cudaGetLastError());
    return LSMKV_OK;
}

unsigned merge_grid(const lsmkv_ctx *ctx, uint64_t n)
{
    uint64_t g = (n + 255) / 256;
    const uint64_t cap = (uint64_t)ctx->sm_count * 8;
    if (g > cap) g = cap;
    return g ? (unsigned)g : 1u;
}

// Grid of a kernel that strides over its work: no more CTAs than the GPU holds at once (those
// beyond would only start when others have finished their whole share, and run under-occupied).
template <typename Kernel>
unsigned resident_grid(const lsmkv_ctx *ctx, Kernel kern, int threads, size_t smem, uint64_t want)
{
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem) != cudaSuccess ||
        per_sm < 1) {
        cudaGetLastError();
        per_sm = 1;
    }
    const uint64_t cap = (uint64_t)ctx->sm_count * (uint64_t)per_sm;
    const uint64_t g = want < cap ? want : cap;
    return g ? (unsigned)g : 1u;
}

constexpr uint64_t kDirMaxJ = 65536;   // chunk indices covered by the probe's directory
constexpr uint64_t kOrderMaxQueries = 65536;   // batches up to this size are handed out longest first

uint64_t *ws_hit_off(lsmkv_ctx *ctx) { return static_cast<uint64_t *>(ctx->d_ws); }
uint32_t *ws_plan(lsmkv_ctx *ctx)
{
    return reinterpret_cast<uint32_t *>(static_cast<uint64_t *>(ctx->d_ws) + ctx->ws_seq + 2);
}

int launch_copy(lsmkv_ctx *ctx, cudaStream_t s, CopyJob &job, const ArenaTable &ar,
                uint64_t max_items)
{
    LaunchTimer timer(ctx, s, job.unpack ? LSMKV_K_UNPACK : LSMKV_K_PACK);
    const uint64_t slabs = 2ull * ctx->geom.n_layers * ctx->ppc;
    job.pages_per_chunk = ctx->ppc;
    job.wait_cycles = ctx->wait_cycles;
    job.test_drop_piece = ctx->test_drop_piece < 0 ? ~0ull : (uint64_t)ctx->test_drop_piece;
    if (ctx->copy_mode == 1) {
        job.piece_bytes = (uint32_t)ctx->page_bytes;
        job.pieces_per_slab = 1;
        uint64_t grid = (uint64_t)ctx->sm_count * (uint64_t)ctx->simt_ctas_per_sm;
        const uint64_t units = max_items * slabs;
        if (grid > units) grid = units;
        if (grid == 0) return LSMKV_OK;
        k_copy_slabs_simt<<<(unsigned)grid, 256, 0, s>>>(job, ar);
    } else {
        uint64_t piece = (uint64_t)ctx->copy_stage_bytes;
        if (piece > ctx->page_bytes) piece = ctx->page_bytes;
        job.piece_bytes = (uint32_t)piece;
        job.pieces_per_slab = (uint32_t)((ctx->page_bytes + piece - 1) / piece);
        const uint64_t stride = (piece + 127) & ~127ull;
        int stages = (int)ctx->copy_stages;
        const size_t per_cta_budget = (size_t)ctx->max_smem_optin / (size_t)ctx->copy_ctas_per_sm;
        while (stages > 1 && (size_t)stages * stride + (size_t)stages * 8 + 1024 > per_cta_budget)
            --stages;
        const size_t smem = (size_t)stages * stride + (size_t)stages * 8;
        if (smem > (size_t)ctx->max_smem_optin) return LSMKV_EINVAL;
        uint64_t grid = (uint64_t)ctx->sm_count * (uint64_t)ctx->copy_ctas_per_sm;
        const uint64_t pieces = max_items * slabs * job.pieces_per_slab;
        const uint64_t need = (pieces + stages - 1) / stages;
        if (grid > need) grid = need;
        if (grid == 0) return LSMKV_OK;
        // (the shared-memory limit of both instantiations was raised at lsmkv_create)
        if (ctx->copy_l2_hint)
            k_copy_slabs_bulk<true><<<(unsigned)grid, stages * 32, smem, s>>>(job, ar);
        else
            k_copy_slabs_bulk<false><<<(unsigned)grid, stages * 32, smem, s>>>(job, ar);
    }
    ++ctx->launches;
    CU(ctx, cudaGetLastError());
    return LSMKV_OK;
}

// put_batch with the compressing codec: measure slabs, lay blobs out, write them.
int encode_xp12(lsmkv_ctx *ctx, cudaStream_t s, uint64_t n_chunks, const uint32_t *page_table,
                const lsmkv_pool_t *pool, uint32_t file_id, uint64_t base_offset,
                lsmkv_val_t *vals_out, void *blob_out, uint64_t blob_capacity)
{
    const uint64_t slabs = 2ull * ctx->geom.n_layers * ctx->ppc;
    if (n_chunks > ctx->xp_cap || !ctx->d_xp) {
        const int rc = grow_scratch(ctx, &ctx->d_xp, &ctx->xp_cap,
                                    (size_t)n_chunks * slabs * 12 + ((size_t)n_chunks + 2) * 8 + 256,
                                    n_chunks, __LINE__);
        if (rc != LSMKV_OK) return rc;
    }
    XpJob job;
    std::memset(&job, 0, sizeof(job));
    job.n_layers = ctx->geom.n_layers;
    job.pages_per_chunk = ctx->ppc;
    job.page_bytes = (uint32_t)ctx->page_bytes;
    job.n_elems = (uint32_t)(ctx->page_bytes / 2);
    job.dir_bytes = ctx->xp_dir_bytes;
    job.num_pages = pool->num_pages;
    job.kv_ptrs = pool->kv_ptrs;
    job.page_table = page_table;
    job.n_chunks = n_chunks;
    job.chunk_off = static_cast<uint64_t *>(ctx->d_xp);
    job.slab_size = reinterpret_cast<uint32_t *>(job.chunk_off + ctx->xp_cap + 2);
    job.slab_info = job.slab_size + ctx->xp_cap * slabs;
    job.slab_nexc = job.slab_info + ctx->xp_cap * slabs;
    job.blob = static_cast<unsigned char *>(blob_out);
    job.blob_capacity = blob_capacity;
    job.file_id = file_id;
    job.base_offset = base_offset;
    job.base_add = ctx->xp_base_add;
    ctx->xp_base_add = nullptr;
    job.vals_out = vals_out;
    job.st = ctx->d_status;
    LaunchTimer timer(ctx, s, LSMKV_K_PACK);
    const uint64_t units = n_chunks * slabs;
    // One pass over the pool when the slab size has a pipeline shape, the blob buffer takes the
    // worst case (so no chunk can overflow half-written) and the pipeline fits the device.
    if (ctx->xp_one_pass && !ctx->xp_generic && (job.n_elems == 8192u || job.n_elems == 16384u) &&
        blob_capacity >= lsmkv_encode_bound(ctx, n_chunks) &&
        (size_t)ctx->max_smem_optin >= (job.n_elems == 8192u ? XpfShape8k::kSmem : XpfShape16k::kSmem)) {
        unsigned char *scratch = static_cast<unsigned char *>(ctx->d_xp);
        xpf::Job fj;
        fj.x = job;
        fj.ticket = reinterpret_cast<unsigned long long *>(scratch);
        fj.abort = reinterpret_cast<unsigned int *>(scratch + 8);
        fj.state = reinterpret_cast<unsigned long long *>(scratch + 256);
        fj.wait_cycles = ctx->wait_cycles;
        fj.test_drop_slab = ctx->test_drop_piece < 0 ? ~0ull : (uint64_t)ctx->test_drop_piece;
        CU(ctx, cudaMemsetAsync(scratch, 0, 256 + (size_t)units * 8, s));
        const unsigned grid = (unsigned)std::min<uint64_t>((uint64_t)ctx->sm_count, units);
        if (job.n_elems == 8192u)
            k_xpf_encode<XpfShape8k><<<grid, XpfShape8k::kThreads, XpfShape8k::kSmem, s>>>(fj);
        else
            k_xpf_encode<XpfShape16k><<<grid, XpfShape16k::kThreads, XpfShape16k::kSmem, s>>>(fj);
        k_xpf_layout<<<merge_grid(ctx, n_chunks), 256, 0, s>>>(fj);
        ctx->launches += 2;
        CU(ctx, cudaGetLastError());
        return LSMKV_OK;
    }
    // common slab sizes take the fast kernels (2048 * {4, 8, 16} elements), the rest the generic
    const uint32_t sweeps = job.n_elems % 2048u == 0 && !ctx->xp_generic ? job.n_elems / 2048u : 0;
    const size_t list_bytes = job.n_elems;
    void (*measure)(XpJob) = sweeps == 4 ? k_xp_measure_fast<4>
                           : sweeps == 8 ? k_xp_measure_fast<8>
                           : sweeps == 16 ? k_xp_measure_fast<16> : k_xp_measure;
    void (*pack)(XpJob) = sweeps == 4 ? k_xp_pack_fast<4>
                        : sweeps == 8 ? k_xp_pack_fast<8>
                        : sweeps == 16 ? k_xp_pack_fast<16> : k_xp_pack;
    const bool fast = sweeps == 4 || sweeps == 8 || sweeps == 16;
    const size_t pack_smem = fast ? list_bytes : 0;
    measure<<<resident_grid(ctx, measure, kXpThreads, 0, units), kXpThreads, 0, s>>>(job);
    k_xp_chunk_sizes<<<merge_grid(ctx, n_chunks), 256, 0, s>>>(job);
    k_scan_blocks<<<1, 1024, 0, s>>>(job.chunk_off, n_chunks, job.chunk_off + n_chunks);
    k_xp_layout<<<merge_grid(ctx, n_chunks), 256, 0, s>>>(job);
    pack<<<resident_grid(ctx, pack, kXpThreads, pack_smem, units), kXpThreads, pack_smem, s>>>(job);
    ctx->launches += 5;
    CU(ctx, cudaGetLastError());
    return LSMKV_OK;
}

unsigned warp_grid(const lsmkv_ctx *ctx, uint64_t n_warps_wanted, unsigned threads,
                   unsigned ctas_per_sm)
{
    const uint64_t wpc = threads / 32;
    uint64_t grid = (n_warps_wanted + wpc - 1) / wpc;
    const uint64_t cap = (uint64_t)ctx->sm_count * ctas_per_sm;
    if (grid > cap) grid = cap;
    return grid ? (unsigned)grid : 1u;
}

}  // namespace

extern "C" {

int lsmkv_create(lsmkv_ctx **out, const lsmkv_geom_t *g, int device)
{
    if (!out || !g) return LSMKV_EINVAL;
    *out = nullptr;
    if (!g->n_layers || !g->n_kv_heads || !g->head_dim || !g->elem_bytes || !g->page_tokens ||
        !g->chunk_tokens || g->chunk_tokens % g->page_tokens != 0 || g->flags > LSMKV_CODEC_XP12)
        return LSMKV_EINVAL;
    const uint64_t pb = (uint64_t)g->page_tokens * g->n_kv_heads * g->head_dim * g->elem_bytes;
    const uint64_t ppc = g->chunk_tokens / g->page_tokens;
    if (pb % 16 != 0 || pb > 0x40000000ull || g->n_layers > 4096 || ppc > 4096 ||
        2ull * g->n_layers * ppc > 0x100000ull)
        return LSMKV_EINVAL;
    if (g->flags == LSMKV_CODEC_XP12 &&
        (g->elem_bytes != 2 ||
         ppc * (2ull * g->n_layers * (pb + 16) + 8ull * g->n_layers) + 16 > 0xFFFFFFF0ull))
        return LSMKV_EINVAL;
    lsmkv_ctx *ctx = new (std::nothrow) lsmkv_ctx();   // value-initialised: all fields zero
    if (!ctx) return LSMKV_ENOMEM;
    ctx->geom = *g;
    ctx->device = device;
    ctx->page_bytes = pb;
    ctx->ppc = (uint32_t)ppc;
    ctx->chunk_bytes = ppc * 2ull * g->n_layers * pb;
    uint64_t key_tab[4 * kKeyTab];
    fill_key_consts(ctx->kc, g->chunk_tokens, key_tab);
    ctx->codec = g->flags;
    ctx->xp_dir_bytes = (uint32_t)((4ull * (ppc * 2ull * g->n_layers + 1) + 15) & ~15ull);
    ctx->copy_mode = 0;
    ctx->copy_stage_bytes = 16384;
    ctx->copy_stages = 12;
    ctx->copy_ctas_per_sm = 1;
    ctx->copy_l2_hint = 0;
    ctx->probe_warps_per_cta = 4;
    ctx->simt_ctas_per_sm = 8;
    ctx->host_stage_bytes = 1ll << 30;
    ctx->xp_one_pass = 1;
    ctx->host_copy_ctas = 32;
    ctx->test_drop_piece = -1;
    ctx->host_copy_piece = 128ll << 20;
    ctx->wait_cycles = 2000000000ll;

    DeviceGuard guard(device);
    cudaError_t e = guard.ok ? cudaSuccess : cudaErrorInvalidDevice;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    // one small block: the status words, then (256 bytes in) the key tables
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, 256 + sizeof(key_tab));
    if (e == cudaSuccess) {
        DevStatus z;
        std::memset(&z, 0, sizeof(z));
        z.first_bad = ~0ull;
        e = cudaMemcpy(ctx->d_status, &z, sizeof(z), cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) {
        uint64_t *d_tab = reinterpret_cast<uint64_t *>(reinterpret_cast<char *>(ctx->d_status) + 256);
        e = cudaMemcpy(d_tab, key_tab, sizeof(key_tab), cudaMemcpyHostToDevice);
        ctx->kc.tab = d_tab;
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        lsmkv_destroy(ctx);
        return LSMKV_ECUDA;
    }
    int rc = ensure_workspace(ctx, 1024, 65536);
    if (rc == LSMKV_OK) rc = ensure_dir(ctx, 2 + 8 * (kDirMaxJ + 1) + kOrderMaxQueries / 2);
    if (rc == LSMKV_OK) rc = set_copy_smem_limit(ctx->max_smem_optin) == cudaSuccess ? LSMKV_OK : LSMKV_ECUDA;
    if (rc != LSMKV_OK) {
        cudaGetLastError();
        lsmkv_destroy(ctx);
        return rc;
    }
    *out = ctx;
    return LSMKV_OK;
}

int lsmkv_destroy(lsmkv_ctx *ctx)
{
    if (!ctx) return LSMKV_OK;
    DeviceGuard guard(ctx->device);
    // Everything is released even when one step fails; the first failure is what is reported.
    cudaError_t first = guard.ok ? cudaSuccess : cudaErrorInvalidDevice;
    auto note = [&first](cudaError_t e) { if (first == cudaSuccess && e != cudaSuccess) first = e; };
    note(cudaDeviceSynchronize());
    uint64_t cap = 0;
    if (release_scratch(ctx, &ctx->d_ws, &ctx->ws_seq, __LINE__) != LSMKV_OK) note((cudaError_t)ctx->last_cuda);
    ctx->ws_chunks = 0;
    if (release_scratch(ctx, &ctx->d_dir, &ctx->dir_cap, __LINE__) != LSMKV_OK) note((cudaError_t)ctx->last_cuda);
    if (release_scratch(ctx, &ctx->d_sort, &ctx->sort_cap, __LINE__) != LSMKV_OK) note((cudaError_t)ctx->last_cuda);
    if (release_scratch(ctx, &ctx->d_xp, &ctx->xp_cap, __LINE__) != LSMKV_OK) note((cudaError_t)ctx->last_cuda);
    for (int k = 0; k < 3; ++k)
        if (release_scratch(ctx, &ctx->d_io[k], &ctx->io_cap[k], __LINE__) != LSMKV_OK)
            note((cudaError_t)ctx->last_cuda);
    for (auto &kind : ctx->hs)
        for (auto &h : kind) {
            if (h.p) note(cudaFreeHost(h.p));
            if (h.done) note(cudaEventDestroy(h.done));
        }
    if (ctx->io_stream) {
        note(cudaStreamDestroy(ctx->io_stream));
        note(cudaEventDestroy(ctx->io_ev_enc));
        note(cudaEventDestroy(ctx->io_ev_free[0]));
        note(cudaEventDestroy(ctx->io_ev_free[1]));
    }
    if (release_scratch(ctx, &ctx->d_status, &cap, __LINE__) != LSMKV_OK) note((cudaError_t)ctx->last_cuda);
    for (auto &t : ctx->pending) { note(cudaEventDestroy(t.a)); note(cudaEventDestroy(t.b)); }
    for (auto e : ctx->free_events) note(cudaEventDestroy(e));
    if (first != cudaSuccess) cudaGetLastError();
    delete ctx;
    return first == cudaSuccess ? LSMKV_OK : LSMKV_ECUDA;
}

int lsmkv_reserve(lsmkv_ctx *ctx, uint64_t n_seq, uint64_t n_chunks)
{
    if (!ctx || n_chunks >= 0xFFFFFFFFull) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    int rc = ensure_workspace(ctx, n_seq, n_chunks);
    if (rc != LSMKV_OK) return rc;
    return ensure_dir(ctx, 2 + 8 * ((n_chunks < kDirMaxJ ? n_chunks : kDirMaxJ) + 1) +
                               kOrderMaxQueries / 2);
}

int lsmkv_encode_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_req, const uint32_t *tokens,
                       const uint64_t *seq_off, const uint32_t *start_chunk,
                       const uint64_t *chunk_off, uint64_t n_chunks, const uint32_t *page_table,
                       const lsmkv_pool_t *pool, uint32_t file_id, uint64_t base_offset,
                       lsmkv_key_t *keys_out, lsmkv_val_t *vals_out, void *blob_out,
                       uint64_t blob_capacity)
{
    if (!ctx) return LSMKV_EINVAL;
    if (n_req == 0 || n_chunks == 0) return n_chunks == 0 ? LSMKV_OK : LSMKV_EINVAL;
    if (!seq_off || !chunk_off || !tokens || !keys_out || !vals_out) return LSMKV_EINVAL;
    if (!aligned16(keys_out) || !aligned16(vals_out)) return LSMKV_EINVAL;
    const bool with_blob = blob_out != nullptr;
    if (with_blob) {
        if (!page_table || !pool || !pool->kv_ptrs || !aligned16(blob_out)) return LSMKV_EINVAL;
        if (n_chunks > UINT64_MAX / (ctx->chunk_bytes + 65536)) return LSMKV_EINVAL;
        if (ctx->codec == LSMKV_CODEC_IDENTITY && blob_capacity < n_chunks * ctx->chunk_bytes)
            return LSMKV_ECAPACITY;
        if (ctx->codec == LSMKV_CODEC_XP12 &&
            (blob_capacity < n_chunks * ctx->xp_dir_bytes || (base_offset & 15u)))
            return LSMKV_ECAPACITY;
    } else if (page_table || pool) {
        return LSMKV_EINVAL;
    }
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    {
        LaunchTimer timer(ctx, s, LSMKV_K_KEYS);
        // few long requests: wide CTAs; many requests: narrower ones, more of them resident
        const unsigned warps = n_req < (unsigned)ctx->sm_count ? 8u : 4u;
        uint64_t grid = n_req;
        const uint64_t cap = (uint64_t)ctx->sm_count * (2048u / (warps * 32u));
        if (grid > cap) grid = cap;
        k_encode_keys<<<(unsigned)grid, warps * 32u, 0, s>>>(ctx->kc, ctx->geom.chunk_tokens,
                                           ctx->geom.ns, n_req,
                                           tokens, seq_off, start_chunk, chunk_off, n_chunks,
                                           file_id, base_offset, ctx->chunk_bytes, keys_out,
                                           vals_out, ctx->d_status);
    }
    ++ctx->launches;
    CU(ctx, cudaGetLastError());
    if (!with_blob) return LSMKV_OK;
    if (ctx->codec == LSMKV_CODEC_XP12)
        return encode_xp12(ctx, s, n_chunks, page_table, pool, file_id, base_offset, vals_out,
                           blob_out, blob_capacity);

    CopyJob job;
    std::memset(&job, 0, sizeof(job));
    job.unpack = 0;
    job.n_layers = ctx->geom.n_layers;
    job.page_bytes = (uint32_t)ctx->page_bytes;
    job.num_pages = pool->num_pages;
    job.kv_ptrs = pool->kv_ptrs;
    job.page_table = page_table;
    job.blob = static_cast<unsigned char *>(blob_out);
    job.n_items = n_chunks;
    job.st = ctx->d_status;
    ArenaTable ar;
    std::memset(&ar, 0, sizeof(ar));
    return launch_copy(ctx, s, job, ar, n_chunks);
}

int lsmkv_probe_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_query, const uint32_t *tokens,
                      const uint64_t *seq_off, const uint64_t *qchunk_off, uint64_t n_qchunks,
                      const lsmkv_run_t *runs, uint32_t n_runs, uint32_t *hit_chunks_out,
                      lsmkv_val_t *recs_out, lsmkv_key_t *keys_out)
{
    if (!ctx) return LSMKV_EINVAL;
    if (n_query == 0) return LSMKV_OK;
    if (!seq_off || !qchunk_off || !hit_chunks_out) return LSMKV_EINVAL;
    if (n_qchunks && (!tokens || !recs_out || !aligned16(recs_out))) return LSMKV_EINVAL;
    if (keys_out && !aligned16(keys_out)) return LSMKV_EINVAL;
    if (n_runs > LSMKV_MAX_RUNS || (n_runs && !runs)) return LSMKV_EINVAL;
    RunTable rt;
    std::memset(&rt, 0, sizeof(rt));
    bool hashed = true;   // every non-empty run brings its hash index: no directory, no searches
    bool wide = true;     // ... and index and keys start on 32-byte boundaries: 32-byte loads
    for (uint32_t r = 0; r < n_runs; ++r) {
        if (runs[r].n && (!runs[r].keys || !runs[r].vals || !aligned16(runs[r].keys) ||
                          !aligned16(runs[r].vals)))
            return LSMKV_EINVAL;
        if (runs[r].bloom && (runs[r].bloom_blocks == 0 || !aligned16(runs[r].bloom)))
            return LSMKV_EINVAL;
        rt.keys[r] = runs[r].keys;
        rt.vals[r] = runs[r].vals;
        rt.n[r] = runs[r].n;
        rt.bloom[r] = runs[r].n ? static_cast<const uint32_t *>(runs[r].bloom) : nullptr;
        rt.bloom_blocks[r] = runs[r].bloom_blocks;
        if (runs[r].hindex && (runs[r].hindex_buckets == 0 || !aligned16(runs[r].hindex) ||
                               runs[r].n > kHidxMaxKeys))
            return LSMKV_EINVAL;
        rt.hidx[r] = static_cast<const uint32_t *>(runs[r].hindex);
        rt.hidx_buckets[r] = runs[r].hindex_buckets;
        if (runs[r].n && !runs[r].hindex) hashed = false;
        if (runs[r].n && ((reinterpret_cast<uintptr_t>(runs[r].hindex) & 31u) ||
                          (reinterpret_cast<uintptr_t>(runs[r].keys) & 31u)))
            wide = false;
    }
    if (n_runs == 0) hashed = false;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t jcap = (uint32_t)(n_qchunks < kDirMaxJ ? n_qchunks : kDirMaxJ);
    // d_dir: [0] = the probe's work counter, [2..] = the directory, then the hand-out order
    const uint32_t dir_runs = hashed ? 0 : n_runs;
    const uint64_t dir_entries = (uint64_t)dir_runs * ((uint64_t)jcap + 1);
    const bool ordered = n_query > 1 && n_query <= kOrderMaxQueries;
    {
        int rc = ensure_dir(ctx, 2 + dir_entries + (ordered ? (n_query + 1) / 2 : 0));
        if (rc != LSMKV_OK) return rc;
    }
    unsigned long long *next_query = reinterpret_cast<unsigned long long *>(ctx->d_dir);
    uint64_t *dir = ctx->d_dir + 2;
    uint32_t *order = ordered ? reinterpret_cast<uint32_t *>(dir + dir_entries) : nullptr;
    const unsigned warps = (unsigned)ctx->probe_warps_per_cta;
    const unsigned threads = warps * 32u;
    // six CTAs of four warps per SM: with more of them every round takes longer, and the
    // rounds of the longest query, one after another, are what the launch waits for
    const uint64_t cap = (uint64_t)ctx->sm_count * (threads <= 768u ? 768u / threads : 1u);
    // Few queries and no directory to fill: a CTA per query, no hand-out order, no counter,
    // and so no launch before the probe's own.
    const bool cta_per_query = hashed && n_query <= cap;
    if (cta_per_query) {
        next_query = nullptr;
        order = nullptr;
    }
    {
        LaunchTimer timer(ctx, s, LSMKV_K_PROBE);
        if (!cta_per_query) {
            // blocks of 1024: the last one also orders the queries, a few per thread (without a
            // directory to fill it is the only block)
            uint64_t dgrid = (dir_entries + 1023) / 1024;
            const uint64_t dcap = (uint64_t)ctx->sm_count * 2;
            if (dgrid > dcap) dgrid = dcap;
            if (dgrid == 0) dgrid = 1;
            k_run_dir<<<(unsigned)dgrid, 1024, 0, s>>>(rt, dir_runs, ctx->geom.ns, jcap, dir,
                                                       next_query, n_query, seq_off,
                                                       ctx->geom.chunk_tokens, order);
            ++ctx->launches;
        }
        uint64_t grid = n_query;
        if (grid > cap) grid = cap;
        auto kern = !hashed ? k_probe<false, false>
                            : (wide ? k_probe<true, true> : k_probe<true, false>);
        kern<<<(unsigned)grid, threads, 0, s>>>(ctx->kc, rt, n_runs, dir, jcap,
                                                ctx->geom.chunk_tokens, ctx->geom.ns, n_query,
                                                tokens, seq_off, qchunk_off, n_qchunks,
                                                hit_chunks_out, recs_out, keys_out,
                                                ctx->d_status, next_query, order);
        ++ctx->launches;
    }
    CU(ctx, cudaGetLastError());
    return LSMKV_OK;
}

int lsmkv_decode_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_query,
                       const uint64_t *qchunk_off, uint64_t n_qchunks,
                       const uint32_t *hit_chunks, const lsmkv_val_t *recs,
                       const void *const *arenas, const uint64_t *arena_bytes,
                       uint32_t n_arenas, const uint32_t *dst_page_table,
                       const lsmkv_pool_t *pool)
{
    if (!ctx) return LSMKV_EINVAL;
    if (n_query == 0 || n_qchunks == 0) return LSMKV_OK;
    if (!qchunk_off || !hit_chunks || !recs || !dst_page_table || !pool || !pool->kv_ptrs)
        return LSMKV_EINVAL;
    if (n_arenas == 0 || n_arenas > (uint32_t)kMaxArenas || !arenas || !arena_bytes)
        return LSMKV_EINVAL;
    if (n_qchunks >= 0xFFFFFFFFull || !aligned16(recs)) return LSMKV_EINVAL;
    ArenaTable ar;
    std::memset(&ar, 0, sizeof(ar));
    for (uint32_t a = 0; a < n_arenas; ++a) {
        if (arena_bytes[a] && (!arenas[a] || !aligned16(arenas[a]))) return LSMKV_EINVAL;
        ar.base[a] = static_cast<const unsigned char *>(arenas[a]);
        ar.bytes[a] = arena_bytes[a];
    }
    DeviceGuard guard(ctx->device);
    int rc = ensure_workspace(ctx, n_query, n_qchunks);
    if (rc != LSMKV_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    uint64_t *hit_off = ws_hit_off(ctx);
    uint32_t *plan = ws_plan(ctx);
    {
        LaunchTimer timer(ctx, s, LSMKV_K_PLAN);
        k_plan_scan<<<1, 1024, 0, s>>>(n_query, qchunk_off, n_qchunks, hit_chunks, hit_off,
                                       ctx->d_status);
        ++ctx->launches;
        CU(ctx, cudaGetLastError());
        k_plan_fill<<<warp_grid(ctx, n_query, 256, 8), 256, 0, s>>>(
            n_query, qchunk_off, hit_off, recs, ar, n_arenas, ctx->chunk_bytes,
            ctx->codec == LSMKV_CODEC_XP12 ? ctx->xp_dir_bytes + 16u : 0u, plan, ctx->d_status);
        ++ctx->launches;
        CU(ctx, cudaGetLastError());
    }

    if (ctx->codec == LSMKV_CODEC_XP12) {
        XpUnpackJob uj;
        std::memset(&uj, 0, sizeof(uj));
        uj.n_layers = ctx->geom.n_layers;
        uj.pages_per_chunk = ctx->ppc;
        uj.page_bytes = (uint32_t)ctx->page_bytes;
        uj.n_elems = (uint32_t)(ctx->page_bytes / 2);
        uj.dir_bytes = ctx->xp_dir_bytes;
        uj.num_pages = pool->num_pages;
        uj.kv_ptrs = pool->kv_ptrs;
        uj.page_table = dst_page_table;
        uj.n_items_dev = hit_off + n_query;
        uj.plan = plan;
        uj.recs = recs;
        uj.st = ctx->d_status;
        LaunchTimer timer(ctx, s, LSMKV_K_UNPACK);
        const uint64_t units = n_qchunks * 2ull * ctx->geom.n_layers * ctx->ppc;
        const uint32_t sweeps = uj.n_elems % 2048u == 0 && !ctx->xp_generic ? uj.n_elems / 2048u : 0;
        void (*unpack)(XpUnpackJob, ArenaTable) = sweeps == 4 ? k_xp_unpack_fast<4>
                                                : sweeps == 8 ? k_xp_unpack_fast<8>
                                                : sweeps == 16 ? k_xp_unpack_fast<16> : k_xp_unpack;
        unpack<<<resident_grid(ctx, unpack, kXpThreads, 0, units), kXpThreads, 0, s>>>(uj, ar);
        ++ctx->launches;
        CU(ctx, cudaGetLastError());
        return LSMKV_OK;
    }
    CopyJob job;
    std::memset(&job, 0, sizeof(job));
    job.unpack = 1;
    job.n_layers = ctx->geom.n_layers;
    job.page_bytes = (uint32_t)ctx->page_bytes;
    job.num_pages = pool->num_pages;
    job.kv_ptrs = pool->kv_ptrs;
    job.page_table = dst_page_table;
    job.n_items_dev = hit_off + n_query;
    job.plan = plan;
    job.recs = recs;
    job.st = ctx->d_status;
    return launch_copy(ctx, s, job, ar, n_qchunks);
}

int lsmkv_flush_batch(lsmkv_ctx *ctx, void *stream, const lsmkv_key_t *keys,
                      const lsmkv_val_t *vals, uint64_t n, lsmkv_key_t *run_keys_out,
                      lsmkv_val_t *run_vals_out, uint64_t *n_out)
{
    if (!ctx || !n_out) return LSMKV_EINVAL;
    if (n >= 0xFFFFFFFFull) return LSMKV_EINVAL;
    if (n && (!keys || !vals || !run_keys_out || !run_vals_out || !aligned16(keys) ||
              !aligned16(vals) || !aligned16(run_keys_out) || !aligned16(run_vals_out)))
        return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        CU(ctx, cudaMemsetAsync(n_out, 0, sizeof(uint64_t), s));
        return LSMKV_OK;
    }
    SortWs ws;
    int rc = ensure_sort(ctx, n, &ws);
    if (rc != LSMKV_OK) return rc;
    LaunchTimer timer(ctx, s, LSMKV_K_FLUSH);
    SegTable segs;
    std::memset(&segs, 0, sizeof(segs));
    // tiles of kSortTile entries are sorted in shared memory, then merged level by level
    int buf = 0;
    k_tile_sort<<<(unsigned)((n + kSortTile - 1) / kSortTile), kSortTile / 2, 0, s>>>(
        keys, ws.keys[0], ws.idx[0], n);
    ++ctx->launches;
    const unsigned grid = merge_grid(ctx, n);
    for (uint64_t width = kSortTile; width < n; width *= 2) {
        k_merge_level<<<grid, 256, 0, s>>>(ws.keys[buf], ws.idx[buf], ws.keys[buf ^ 1],
                                           ws.idx[buf ^ 1], n, width, segs);
        ++ctx->launches;
        buf ^= 1;
    }
    CU(ctx, cudaGetLastError());
    return launch_dedupe(ctx, s, ws, buf, n, vals, /*keep_last=*/1, run_keys_out, run_vals_out,
                         n_out);
}

int lsmkv_merge_runs(lsmkv_ctx *ctx, void *stream, const lsmkv_run_t *runs, uint32_t n_runs,
                     lsmkv_key_t *keys_out, lsmkv_val_t *vals_out, uint64_t *n_out)
{
    if (!ctx || !n_out || n_runs > LSMKV_MAX_RUNS || (n_runs && !runs)) return LSMKV_EINVAL;
    uint64_t total = 0;
    for (uint32_t r = 0; r < n_runs; ++r) {
        if (runs[r].n && (!runs[r].keys || !runs[r].vals)) return LSMKV_EINVAL;
        total += runs[r].n;
    }
    if (total >= 0xFFFFFFFFull) return LSMKV_EINVAL;
    if (total && (!keys_out || !vals_out || !aligned16(keys_out) || !aligned16(vals_out)))
        return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (total == 0) {
        CU(ctx, cudaMemsetAsync(n_out, 0, sizeof(uint64_t), s));
        return LSMKV_OK;
    }
    SortWs ws;
    int rc = ensure_sort(ctx, total, &ws);
    if (rc != LSMKV_OK) return rc;
    LaunchTimer timer(ctx, s, LSMKV_K_MERGE);
    // concatenate newest first; ties then resolve to the newer run
    SegTable segs;
    std::memset(&segs, 0, sizeof(segs));
    uint64_t at = 0;
    uint32_t n_seg = 0;
    for (uint32_t r = 0; r < n_runs; ++r) {
        if (runs[r].n == 0) continue;
        CU(ctx, cudaMemcpyAsync(ws.keys[0] + at, runs[r].keys, runs[r].n * sizeof(lsmkv_key_t),
                                cudaMemcpyDeviceToDevice, s));
        CU(ctx, cudaMemcpyAsync(ws.vals + at, runs[r].vals, runs[r].n * sizeof(lsmkv_val_t),
                                cudaMemcpyDeviceToDevice, s));
        segs.start[n_seg++] = at;
        at += runs[r].n;
    }
    segs.start[n_seg] = total;
    segs.n_seg = n_seg;
    int buf = 0;
    const uint32_t *src_idx = nullptr;
    const unsigned grid = merge_grid(ctx, total);
    for (;;) {
        k_merge_level<<<grid, 256, 0, s>>>(ws.keys[buf], src_idx, ws.keys[buf ^ 1], ws.idx[buf ^ 1],
                                           total, 0, segs);
        ++ctx->launches;
        buf ^= 1;
        src_idx = ws.idx[buf];
        const uint32_t next = (segs.n_seg + 1) / 2;
        for (uint32_t k = 0; k < next; ++k) segs.start[k] = segs.start[2 * k];
        segs.start[next] = total;
        segs.n_seg = next;
        if (next <= 1) break;
    }
    CU(ctx, cudaGetLastError());
    return launch_dedupe(ctx, s, ws, buf, total, ws.vals, /*keep_last=*/0, keys_out, vals_out,
                         n_out);
}

int lsmkv_xrun_build(lsmkv_ctx *ctx, void *stream, const uint32_t *tokens,
                     const uint64_t *seq_off, uint32_t n_seq, uint32_t *order_out,
                     uint64_t *chunk_off_out)
{
    if (!ctx || !chunk_off_out || n_seq == 0xFFFFFFFFu) return LSMKV_EINVAL;
    if (n_seq && (!seq_off || !order_out)) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n_seq == 0) {
        CU(ctx, cudaMemsetAsync(chunk_off_out, 0, sizeof(uint64_t), s));
        return LSMKV_OK;
    }
    SortWs ws;
    int rc = ensure_sort(ctx, n_seq, &ws);
    if (rc != LSMKV_OK) return rc;
    LaunchTimer timer(ctx, s, LSMKV_K_FLUSH);
    k_xrun_init<<<merge_grid(ctx, n_seq), 256, 0, s>>>(seq_off, n_seq, ctx->geom.chunk_tokens,
                                                       ws.idx[0], chunk_off_out, ctx->d_status);
    k_scan_blocks<<<1, 1024, 0, s>>>(chunk_off_out, n_seq, chunk_off_out + n_seq);
    ctx->launches += 2;
    int buf = 0;
    // one warp per element; the grid covers the elements once or caps at 8 CTAs per SM
    const unsigned grid = warp_grid(ctx, n_seq, 256, 8);
    for (uint64_t width = 1; width < n_seq; width *= 2) {
        k_xrun_merge_level<<<grid, 256, 0, s>>>(tokens, seq_off, ws.idx[buf], ws.idx[buf ^ 1],
                                                n_seq, width);
        ++ctx->launches;
        buf ^= 1;
    }
    CU(ctx, cudaGetLastError());
    CU(ctx, cudaMemcpyAsync(order_out, ws.idx[buf], (size_t)n_seq * sizeof(uint32_t),
                            cudaMemcpyDeviceToDevice, s));
    return LSMKV_OK;
}

int lsmkv_xrun_merge(lsmkv_ctx *ctx, void *stream, const uint32_t *tokens,
                     const uint64_t *seq_off, const uint32_t *order_a, uint32_t n_a,
                     const uint32_t *order_b, uint32_t n_b, uint32_t *order_out,
                     uint64_t *chunk_off_out)
{
    const uint64_t n = (uint64_t)n_a + n_b;
    if (!ctx || !chunk_off_out || n >= 0xFFFFFFFFull) return LSMKV_EINVAL;
    if (n && (!seq_off || !order_out)) return LSMKV_EINVAL;
    if ((n_a && !order_a) || (n_b && !order_b)) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        CU(ctx, cudaMemsetAsync(chunk_off_out, 0, sizeof(uint64_t), s));
        return LSMKV_OK;
    }
    SortWs ws;
    int rc = ensure_sort(ctx, n, &ws);
    if (rc != LSMKV_OK) return rc;
    LaunchTimer timer(ctx, s, LSMKV_K_MERGE);
    k_xrun_concat<<<merge_grid(ctx, n), 256, 0, s>>>(order_a, n_a, order_b, n_b, seq_off,
                                                     ctx->geom.chunk_tokens, ws.idx[0],
                                                     chunk_off_out, ctx->d_status);
    k_scan_blocks<<<1, 1024, 0, s>>>(chunk_off_out, n, chunk_off_out + n);
    k_xrun_merge_two<<<warp_grid(ctx, n, 256, 8), 256, 0, s>>>(tokens, seq_off, ws.idx[0],
                                                               order_out, n, n_a);
    ctx->launches += 3;
    CU(ctx, cudaGetLastError());
    return LSMKV_OK;
}

int lsmkv_xprobe_batch(lsmkv_ctx *ctx, void *stream, uint32_t n_query, const uint32_t *tokens,
                       const uint64_t *seq_off, const uint64_t *qchunk_off, uint64_t n_qchunks,
                       const lsmkv_xrun_t *runs, uint32_t n_runs, uint32_t *hit_chunks_out,
                       lsmkv_val_t *recs_out)
{
    if (!ctx) return LSMKV_EINVAL;
    if (n_query == 0) return LSMKV_OK;
    if (!seq_off || !qchunk_off || !hit_chunks_out) return LSMKV_EINVAL;
    if (n_qchunks && (!tokens || !recs_out || !aligned16(recs_out))) return LSMKV_EINVAL;
    if (n_runs > LSMKV_MAX_RUNS || (n_runs && !runs)) return LSMKV_EINVAL;
    XRunTable rt;
    std::memset(&rt, 0, sizeof(rt));
    for (uint32_t r = 0; r < n_runs; ++r) {
        if (runs[r].n_seq && (!runs[r].seq_off || !runs[r].order || !runs[r].chunk_off ||
                              !runs[r].vals || !aligned16(runs[r].vals)))
            return LSMKV_EINVAL;
        rt.tokens[r] = runs[r].tokens;
        rt.seq_off[r] = runs[r].seq_off;
        rt.vals[r] = runs[r].vals;
        rt.order[r] = runs[r].order;
        rt.chunk_off[r] = runs[r].chunk_off;
        rt.n_seq[r] = runs[r].n_seq;
    }
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the probe's scratch: [0] = work counter, then the hand-out order (longest query first)
    const bool ordered = n_query > 1 && n_query <= kOrderMaxQueries;
    {
        int rc = ensure_dir(ctx, 2 + (ordered ? ((uint64_t)n_query + 1) / 2 : 0));
        if (rc != LSMKV_OK) return rc;
    }
    unsigned long long *next_query = reinterpret_cast<unsigned long long *>(ctx->d_dir);
    uint32_t *order = ordered ? reinterpret_cast<uint32_t *>(ctx->d_dir + 2) : nullptr;
    LaunchTimer timer(ctx, s, LSMKV_K_PROBE);
    {
        RunTable none;
        std::memset(&none, 0, sizeof(none));
        k_run_dir<<<1, 256, 0, s>>>(none, 0, ctx->geom.ns, 0, ctx->d_dir + 2, next_query, n_query,
                                    seq_off, ctx->geom.chunk_tokens, order);
    }
    k_xprobe<<<warp_grid(ctx, n_query, 256, 2), 256, 0, s>>>(
        rt, n_runs, ctx->geom.chunk_tokens, n_query, tokens, seq_off, qchunk_off, n_qchunks,
        hit_chunks_out, recs_out, ctx->d_status, next_query, order);
    ctx->launches += 2;
    CU(ctx, cudaGetLastError());
    return LSMKV_OK;
}

int lsmkv_relocate_records(lsmkv_ctx *ctx, void *stream, lsmkv_val_t *vals, uint64_t n,
                           const lsmkv_reloc_t *table, uint32_t n_table, uint64_t *changed_out)
{
    if (!ctx || (n && (!vals || !aligned16(vals))) || n_table > (uint32_t)kMaxReloc ||
        (n_table && !table))
        return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (changed_out) CU(ctx, cudaMemsetAsync(changed_out, 0, sizeof(uint64_t), s));
    if (n == 0 || n_table == 0) return LSMKV_OK;
    RelocTable tab;
    std::memset(&tab, 0, sizeof(tab));
    tab.n = n_table;
    for (uint32_t t = 0; t < n_table; ++t) {
        tab.old_file[t] = table[t].old_file;
        tab.new_file[t] = table[t].new_file;
        tab.delta[t] = table[t].delta;
    }
    k_relocate_records<<<merge_grid(ctx, n), 256, 0, s>>>(
        vals, n, tab, reinterpret_cast<unsigned long long *>(changed_out));
    ++ctx->launches;
    CU(ctx, cudaGetLastError());
    return LSMKV_OK;
}

uint64_t lsmkv_encode_bound(const lsmkv_ctx *ctx, uint64_t n_chunks)
{
    if (!ctx) return 0;
    if (ctx->codec == LSMKV_CODEC_XP12)
        return n_chunks * (ctx->xp_dir_bytes +
                           2ull * ctx->geom.n_layers * ctx->ppc * (16 + ctx->page_bytes));
    return n_chunks * ctx->chunk_bytes;
}

uint64_t lsmkv_bloom_blocks(uint64_t n)
{
    const uint64_t b = (10 * n + 255) / 256;
    return b ? b : 1;
}

int lsmkv_bloom_build(lsmkv_ctx *ctx, void *stream, const lsmkv_key_t *keys, uint64_t n,
                      void *bloom_out)
{
    if (!ctx || !bloom_out || !aligned16(bloom_out) || (n && (!keys || !aligned16(keys))))
        return LSMKV_EINVAL;
    if (n > (UINT64_MAX - 255) / 10) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint64_t nb = lsmkv_bloom_blocks(n);
    CU(ctx, cudaMemsetAsync(bloom_out, 0, nb * 32, s));
    if (n) {
        k_bloom_build<<<merge_grid(ctx, n), 256, 0, s>>>(keys, n, static_cast<uint32_t *>(bloom_out), nb);
        ++ctx->launches;
        CU(ctx, cudaGetLastError());
    }
    return LSMKV_OK;
}

uint64_t lsmkv_hindex_buckets(uint64_t n)
{
    const uint64_t b = n / 2 + (n & 1);
    return b ? b : 1;
}

int lsmkv_hindex_build(lsmkv_ctx *ctx, void *stream, const lsmkv_key_t *keys, uint64_t n,
                       void *hindex_out)
{
    if (!ctx || !hindex_out || !aligned16(hindex_out) || (n && (!keys || !aligned16(keys))))
        return LSMKV_EINVAL;
    if (n > kHidxMaxKeys) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint64_t nb = lsmkv_hindex_buckets(n);
    LaunchTimer timer(ctx, s, LSMKV_K_FLUSH);   // part of writing a run
    CU(ctx, cudaMemsetAsync(hindex_out, 0, nb * 32, s));
    if (n) {
        k_hidx_build<<<merge_grid(ctx, n), 256, 0, s>>>(keys, n, static_cast<uint32_t *>(hindex_out), nb);
        ++ctx->launches;
        CU(ctx, cudaGetLastError());
    }
    return LSMKV_OK;
}

int lsmkv_last_status(lsmkv_ctx *ctx, void *stream, lsmkv_status_t *out)
{
    if (!ctx || !out) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(ctx, cudaMemcpyAsync(out, ctx->d_status, sizeof(DevStatus), cudaMemcpyDeviceToHost, s));
    CU(ctx, cudaStreamSynchronize(s));
    DevStatus z;
    std::memset(&z, 0, sizeof(z));
    z.first_bad = ~0ull;
    CU(ctx, cudaMemcpyAsync(ctx->d_status, &z, sizeof(z), cudaMemcpyHostToDevice, s));
    CU(ctx, cudaStreamSynchronize(s));
    return LSMKV_OK;
}

int lsmkv_profile_enable(lsmkv_ctx *ctx, int on)
{
    if (!ctx) return LSMKV_EINVAL;
    ctx->profiling = on != 0;
    return LSMKV_OK;
}

int lsmkv_profile_read(lsmkv_ctx *ctx, lsmkv_profile_t *out)
{
    if (!ctx || !out) return LSMKV_EINVAL;
    DeviceGuard guard(ctx->device);
    std::memset(out, 0, sizeof(*out));
    int rc = LSMKV_OK;
    for (auto &t : ctx->pending) {
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(t.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t.a, t.b);
        if (e == cudaSuccess) {
            out->ms[t.cls] += ms;
            out->launches[t.cls] += 1;
        } else {
            rc = cuda_fail(ctx, e);
        }
        ctx->free_events.push_back(t.a);
        ctx->free_events.push_back(t.b);
    }
    ctx->pending.clear();
    return rc;
}

int lsmkv_last_cuda_error(const lsmkv_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }

int lsmkv_last_cuda_line(const lsmkv_ctx *ctx) { return ctx ? ctx->last_cuda_line : 0; }

uint64_t lsmkv_launch_count(const lsmkv_ctx *ctx) { return ctx ? ctx->launches : 0; }

static int64_t *tuning_slot(lsmkv_ctx *ctx, const char *name, int64_t *lo, int64_t *hi)
{
    struct { const char *n; int64_t *p; int64_t lo, hi; } tab[] = {
        {"copy_mode", &ctx->copy_mode, 0, 1},
        {"copy_stage_bytes", &ctx->copy_stage_bytes, 16, 1 << 17},
        {"copy_stages", &ctx->copy_stages, 1, 32},
        {"copy_ctas_per_sm", &ctx->copy_ctas_per_sm, 1, 8},
        {"copy_l2_hint", &ctx->copy_l2_hint, 0, 1},
        {"probe_warps_per_cta", &ctx->probe_warps_per_cta, 1, 8},
        {"simt_ctas_per_sm", &ctx->simt_ctas_per_sm, 1, 32},
        {"host_stage_bytes", &ctx->host_stage_bytes, 1 << 20, 1ll << 36},
        {"xp_generic", &ctx->xp_generic, 0, 1},
        {"xp_one_pass", &ctx->xp_one_pass, 0, 1},
        {"host_copy_ctas", &ctx->host_copy_ctas, 1, 4096},
        {"host_put_device_placed", &ctx->host_put_device_placed, 0, 1},
        {"test_drop_piece", &ctx->test_drop_piece, -1, 1ll << 40},
        {"host_copy_piece_bytes", &ctx->host_copy_piece, 1 << 20, 1ll << 36},
        {"wait_cycles", &ctx->wait_cycles, 100000, 100000000000ll},
    };
    for (auto &t : tab)
        if (std::strcmp(t.n, name) == 0) { *lo = t.lo; *hi = t.hi; return t.p; }
    return nullptr;
}

int lsmkv_set_tuning(lsmkv_ctx *ctx, const char *name, int64_t value)
{
    if (!ctx || !name) return LSMKV_EINVAL;
    int64_t lo, hi;
    int64_t *p = tuning_slot(ctx, name, &lo, &hi);
    if (!p || value < lo || value > hi) return LSMKV_EINVAL;
    if (std::strcmp(name, "copy_stage_bytes") == 0 && value % 16 != 0) return LSMKV_EINVAL;
    *p = value;
    return LSMKV_OK;
}

int64_t lsmkv_get_tuning(const lsmkv_ctx *ctx, const char *name)
{
    if (!ctx || !name) return LSMKV_EINVAL;
    int64_t lo, hi;
    int64_t *p = tuning_slot(const_cast<lsmkv_ctx *>(ctx), name, &lo, &hi);
    return p ? *p : LSMKV_EINVAL;
}

const char *lsmkv_strerror(int code)
{
    switch (code) {
    case LSMKV_OK: return "ok";
    case LSMKV_EINVAL: return "invalid argument";
    case LSMKV_ECAPACITY: return "output buffer too small";
    case LSMKV_ECUDA: return "CUDA error";
    case LSMKV_ENOMEM: return "out of memory";
    case LSMKV_ETOOBIG: return "batch exceeds the built-in scratch of the allocation-free entry point";
    default: return "unknown error";
    }
}

int lsmkv_plan_compaction(const uint32_t *level, const uint64_t *entries, uint32_t n_runs,
                          uint64_t buffer_entries, uint32_t size_ratio, uint32_t runs_per_level,
                          lsmkv_compaction_t *out)
{
    if (!out || buffer_entries == 0 || size_ratio < 2 || runs_per_level == 0) return LSMKV_EINVAL;
    if (n_runs && (!level || !entries)) return LSMKV_EINVAL;
    for (uint32_t r = 0; r < n_runs; ++r)
        if (level[r] == 0 || (r && level[r] < level[r - 1])) return LSMKV_EINVAL;
    uint64_t cap = buffer_entries;                      // capacity of level i = M * T^i, saturating
    uint32_t cap_level = 0;
    for (uint32_t a = 0; a < n_runs;) {
        const uint32_t i = level[a];
        uint32_t b = a;
        uint64_t sum = 0;
        while (b < n_runs && level[b] == i) {
            sum = sum + entries[b] < sum ? UINT64_MAX : sum + entries[b];
            ++b;
        }
        while (cap_level < i) {
            cap = cap > UINT64_MAX / size_ratio ? UINT64_MAX : cap * size_ratio;
            ++cap_level;
        }
        const uint32_t count = b - a;
        if (sum >= cap && cap != UINT64_MAX) {          // full: its runs leave for the next level
            uint32_t c = b;                              // runs of level i + 1
            while (c < n_runs && level[c] == i + 1) ++c;
            const bool join = c - b >= runs_per_level;  // one more run would be too many there
            out->first_run = a;
            out->n_runs = (join ? c : b) - a;
            out->to_level = i + 1;
            return 1;
        }
        if (count > runs_per_level) {                   // too many runs: they become one, in place
            out->first_run = a;
            out->n_runs = count;
            out->to_level = i;
            return 1;
        }
        a = b;
    }
    out->first_run = 0;
    out->n_runs = 0;
    out->to_level = 0;
    return 0;
}

int lsmkv_format_version(void) { return LSMKV_FORMAT_VERSION; }

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Allocation-free decode.
//
// lsmkv_decode_batch() needs a little global memory of its own: the exclusive prefix sums of the
// hit lengths, the compact list of chunks to copy, and a status block. The regular entry point
// keeps them in a cudaMalloc'ed per-context workspace. The variant below keeps them in a
// fixed-size array that is part of the library image, so it runs without a context and without
// any allocation. Layout of the array: [status block | hit_off u64[kStaticMaxQueries + 2] |
// plan u32[kStaticMaxChunks]].
// ---------------------------------------------------------------------------------------------
namespace {

constexpr uint64_t kStaticMaxQueries = LSMKV_STATIC_MAX_QUERIES;
constexpr uint64_t kStaticMaxChunks = LSMKV_STATIC_MAX_CHUNKS;
constexpr size_t kStaticStatusBytes = 256;
constexpr size_t kStaticHitOffBytes = (kStaticMaxQueries + 2) * sizeof(uint64_t);
constexpr size_t kStaticBytes =
    kStaticStatusBytes + kStaticHitOffBytes + kStaticMaxChunks * sizeof(uint32_t);

// Lives in every GPU context that loads this library, until the process exits (~1.03 MiB).
// NOTE: in host code `g_static_scratch` is only a handle for cudaGetSymbolAddress(); it is not
// a device address and must never be handed to a kernel directly.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// Device code may name the array directly: reset the status block at the start of a call
// (everything else in the array is fully rewritten by the plan kernels before it is read).
__global__ void k_static_reset()
{
    DevStatus *st = reinterpret_cast<DevStatus *>(g_static_scratch);
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        st->flags = 0;
        st->reserved = 0;
        st->first_bad = ~0ull;
        st->chunks_encoded = st->lookups = st->chunks_hit = st->empty_probes = 0;
        st->chunks_decoded = 0;
    }
}

constexpr int kStaticMaxDevices = kMaxDevices;
struct StaticDev {
    bool ready;
    unsigned char *scratch;   // device address of g_static_scratch on this device
    int sm_count;
    int max_smem_optin;
};
StaticDev g_static_dev[kStaticMaxDevices];
std::mutex g_static_mu;

// Once per device, with that device current: resolve the device address of the scratch array.
int static_setup(int device, StaticDev **out)
{
    if (device < 0 || device >= kStaticMaxDevices) return LSMKV_EINVAL;
    std::lock_guard<std::mutex> lock(g_static_mu);
    StaticDev &d = g_static_dev[device];
    if (!d.ready) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
        if (e == cudaSuccess) e = set_copy_smem_limit(d.max_smem_optin);
        if (e != cudaSuccess || !ptr) {
            cudaGetLastError();
            return LSMKV_ECUDA;
        }
        d.scratch = static_cast<unsigned char *>(ptr);
        d.ready = true;
    }
    *out = &d;
    return LSMKV_OK;
}

}  // namespace

extern "C" int lsmkv_decode_batch_static(const lsmkv_geom_t *g, int device, void *stream,
                                         uint32_t n_query, const uint64_t *qchunk_off,
                                         uint64_t n_qchunks, const uint32_t *hit_chunks,
                                         const lsmkv_val_t *recs, const void *const *arenas,
                                         const uint64_t *arena_bytes, uint32_t n_arenas,
                                         const uint32_t *dst_page_table,
                                         const lsmkv_pool_t *pool, lsmkv_status_t *status_out)
{
    if (!g || !g->n_layers || !g->n_kv_heads || !g->head_dim || !g->elem_bytes ||
        !g->page_tokens || !g->chunk_tokens || g->chunk_tokens % g->page_tokens != 0 ||
        g->flags != 0)
        return LSMKV_EINVAL;
    const uint64_t pb = (uint64_t)g->page_tokens * g->n_kv_heads * g->head_dim * g->elem_bytes;
    const uint64_t ppc = g->chunk_tokens / g->page_tokens;
    if (pb % 16 != 0 || pb > 0x40000000ull || g->n_layers > 4096 || ppc > 4096 ||
        2ull * g->n_layers * ppc > 0x100000ull)
        return LSMKV_EINVAL;
    const uint64_t cb = ppc * 2ull * g->n_layers * pb;
    if (n_query > kStaticMaxQueries || n_qchunks > kStaticMaxChunks) return LSMKV_ETOOBIG;
    if (!qchunk_off || !hit_chunks || !recs || !dst_page_table || !pool || !pool->kv_ptrs)
        return LSMKV_EINVAL;
    if (n_arenas == 0 || n_arenas > (uint32_t)kMaxArenas || !arenas || !arena_bytes ||
        !aligned16(recs))
        return LSMKV_EINVAL;
    ArenaTable ar;
    std::memset(&ar, 0, sizeof(ar));
    for (uint32_t a = 0; a < n_arenas; ++a) {
        if (arena_bytes[a] && (!arenas[a] || !aligned16(arenas[a]))) return LSMKV_EINVAL;
        ar.base[a] = static_cast<const unsigned char *>(arenas[a]);
        ar.bytes[a] = arena_bytes[a];
    }
    DeviceGuard guard(device);
    if (!guard.ok) return LSMKV_ECUDA;
    StaticDev *sd = nullptr;
    int rc = static_setup(device, &sd);
    if (rc != LSMKV_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    DevStatus *st = reinterpret_cast<DevStatus *>(sd->scratch);
    uint64_t *hit_off = reinterpret_cast<uint64_t *>(sd->scratch + kStaticStatusBytes);
    uint32_t *plan = reinterpret_cast<uint32_t *>(sd->scratch + kStaticStatusBytes + kStaticHitOffBytes);

    k_static_reset<<<1, 32, 0, s>>>();
    if (n_query && n_qchunks) {
        k_plan_scan<<<1, 1024, 0, s>>>(n_query, qchunk_off, n_qchunks, hit_chunks, hit_off, st);
        uint64_t fill_grid = ((uint64_t)n_query + 7) / 8;
        const uint64_t fill_cap = (uint64_t)sd->sm_count * 8;
        if (fill_grid > fill_cap) fill_grid = fill_cap;
        k_plan_fill<<<(unsigned)fill_grid, 256, 0, s>>>(n_query, qchunk_off, hit_off, recs, ar,
                                                        n_arenas, cb, 0u, plan, st);
        CopyJob job;
        std::memset(&job, 0, sizeof(job));
        job.unpack = 1;
        job.n_layers = g->n_layers;
        job.pages_per_chunk = (uint32_t)ppc;
        job.page_bytes = (uint32_t)pb;
        job.num_pages = pool->num_pages;
        job.kv_ptrs = pool->kv_ptrs;
        job.page_table = dst_page_table;
        job.n_items_dev = hit_off + n_query;
        job.plan = plan;
        job.recs = recs;
        job.st = st;
        job.wait_cycles = 2000000000ll;
        job.test_drop_piece = ~0ull;
        const uint64_t piece = pb < 32768 ? pb : 32768;
        job.piece_bytes = (uint32_t)piece;
        job.pieces_per_slab = (uint32_t)((pb + piece - 1) / piece);
        const uint64_t stride = (piece + 127) & ~127ull;
        int stages = 6;
        while (stages > 1 && (size_t)stages * stride + (size_t)stages * 8 + 1024 > (size_t)sd->max_smem_optin)
            --stages;
        const size_t smem = (size_t)stages * stride + (size_t)stages * 8;
        const uint64_t pieces = n_qchunks * ppc * 2ull * g->n_layers * job.pieces_per_slab;
        uint64_t grid = (uint64_t)sd->sm_count;
        const uint64_t need = (pieces + stages - 1) / stages;
        if (grid > need) grid = need;
        // (the kernel's shared-memory limit was raised to the device maximum by the set-up)
        k_copy_slabs_bulk<false><<<(unsigned)grid, stages * 32, smem, s>>>(job, ar);
    }
    if (status_out) {
        cudaError_t e = cudaMemcpyAsync(status_out, st, sizeof(DevStatus), cudaMemcpyDeviceToDevice, s);
        if (e != cudaSuccess) { cudaGetLastError(); return LSMKV_ECUDA; }
    }
    if (cudaGetLastError() != cudaSuccess) return LSMKV_ECUDA;
    return LSMKV_OK;
}

#include "lsmkv_hostio.cuh"
