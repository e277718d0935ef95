// Host side of libkdn: the C ABI declared in include/kdn.h.  Validates arguments, turns ops into
// 96-byte device records, and launches the tile pipeline of kdn_kernels.cuh on the caller's stream.
// Paper anchors: Sec. 3.2 "Interface with LLM serving engines" (store / retrieve), Sec. 3.1 (storage,
// delivery and blending modules).
#include "kdn.h"
#include "kdn_kernels.cuh"
#include "kdn_td.cuh"

#include <cerrno>
#include <cstdio>
#include <cstring>
#include <functional>
#include <mutex>
#include <new>
#include <atomic>
#include <thread>
#include <utility>
#include <vector>

#include <sys/mman.h>
#include <sys/stat.h>
#include <unistd.h>

using namespace kdn;

#define KDN_CUDA(call)                                                                  \
    do {                                                                                \
        cudaError_t e_ = (call);                                                        \
        if (e_ != cudaSuccess) return e_ == cudaErrorMemoryAllocation ? KDN_E_NOMEM : KDN_E_CUDA; \
    } while (0)

namespace {

constexpr int kRing = 8;                   // launches that may be queued before the host has to wait
constexpr int kMaxOpsPerLaunch = 4096;
constexpr unsigned kMaxTilesPerLaunch = 0x7fff0000u;
constexpr size_t kDefaultSlabBytes = (size_t)256 << 20;
constexpr unsigned kTdCols = 128;           // channels per CTA of the token-delta kernels
constexpr unsigned kKcCols = 256;           // channels per CTA of the key-plane store of the per-channel key codecs

struct Pool {
    int L, H, D, bs;
    long long nb;
    void **d_k = nullptr;                   // device copies of the per-layer pointer arrays
    void **d_v = nullptr;
};

struct RingSlot {
    DevOp *h_ops = nullptr;                 // pinned
    DevOp *d_ops = nullptr;
    RopeParam *h_rope = nullptr;            // pinned
    RopeParam *d_rope = nullptr;
    float2 *d_table = nullptr;
    size_t table_rows_cap = 0;
    int table_half = 0;
    cudaEvent_t done = nullptr;
    bool used = false;
};

struct HostOp {                             // one op (or one layer range of one) before tiling
    DevOp op;
    bool rotate = false;
    RopeParam rp{};
    int fd = -1;                            // >= 0: the chunk's bytes live in this file, from file_off on
    long long file_off = 0;
};

struct Piece {                              // host <-> slab copies belonging to a staged op
    unsigned char *host;                    // page-locked host memory, or nullptr: the piece lives in a file
    size_t slab_off;
    size_t bytes;
    int fd;
    long long file_off;
};

// What a launch needs to know about its device, and what it has already asked the runtime about each kernel:
// one per context (and one per device for kdn_compose_static), so a launch takes no lock and no device query.
// Every kernel's dynamic shared-memory limit is raised to the device's opt-in maximum the first time it is seen,
// whatever the launch at hand needs: the value is the same for every context of the process, so contexts cannot
// lower each other's grants.
struct LaunchEnv {
    int sm_count = 0;
    int smem_optin = 0;
    struct Entry { const void *fn; size_t smem; int threads; int per_sm; };
    static constexpr int kEntries = 64;
    Entry cache[kEntries];
    int n = 0, next = 0;

    // CTAs of `kernel` resident per SM at this shape (0 = does not fit); sets the kernel's attribute on first sight.
    template <typename K>
    kdn_status resident(K kernel, int threads, size_t smem, int *per_sm)
    {
        const void *fn = (const void *)kernel;
        bool seen = false;
        for (int i = 0; i < n; ++i) {
            if (cache[i].fn != fn) continue;
            seen = true;
            if (cache[i].smem == smem && cache[i].threads == threads) { *per_sm = cache[i].per_sm; return KDN_OK; }
        }
        if (!seen) KDN_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin));
        int r = 0;
        KDN_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, kernel, threads, smem));
        Entry &e = n < kEntries ? cache[n++] : cache[next++ % kEntries];
        e.fn = fn; e.smem = smem; e.threads = threads; e.per_sm = r;
        *per_sm = r;
        return KDN_OK;
    }
};

}  // namespace

struct kdn_ctx {
    int device = 0;
    LaunchEnv env;                          // SM count, shared-memory limit, per-kernel occupancy cache
    std::vector<Pool> pools;
    RingSlot ring[kRing];
    unsigned ring_next = 0;
    int *d_status = nullptr;
    int *h_status = nullptr;                // pinned
    cudaStream_t own_side = nullptr;
    unsigned char *slab[2] = { nullptr, nullptr };
    size_t slab_bytes = kDefaultSlabBytes;
    cudaEvent_t slab_free[2] = { nullptr, nullptr };   // last consumer of the slab has finished
    cudaEvent_t slab_ready[2] = { nullptr, nullptr };  // the slab's producer has finished
    unsigned slab_next = 0;
    unsigned char *bounce[2] = { nullptr, nullptr };   // page-locked mirrors of the slabs for file-backed chunks
    cudaEvent_t bounce_done[2] = { nullptr, nullptr }; // the copies between bounce[i] and slab[i] have finished
    bool bounce_busy[2] = { false, false };
    std::vector<Piece> pending_writes[2];              // file pieces whose bytes are on their way into bounce[i]
    uint64_t launches = 0;
    kdn_tuning tuning{};
    unsigned long long wait_limit_ns = kWaitLimitNs;
    kdn_launch_info last{};                 // shape of the most recent tile-pipeline launch
    cudaEvent_t fork = nullptr;             // orders the side stream after the caller's stream at the start of a staged call
};

namespace {

bool shape_ok(const kdn_pool_desc *p)
{
    return p && p->n_layers > 0 && p->n_kv_heads > 0 && p->head_dim > 0 && p->block_size > 0 && p->n_blocks > 0;
}

kdn_status check_shape(const kdn_pool_desc *p)
{
    if (!shape_ok(p)) return KDN_E_INVAL;
    if (((long long)p->n_kv_heads * p->head_dim * 2) % 16) return KDN_E_ALIGN;
    if ((long long)p->n_kv_heads * p->head_dim > (1 << 24) || p->block_size > (1 << 20)) return KDN_E_UNSUPPORTED;
    return KDN_OK;
}

bool is_kc(int codec) { return codec == KDN_CODEC_INT8_KC64 || codec == KDN_CODEC_INT4_KC64; }
bool is_int4(int codec) { return codec == KDN_CODEC_INT4_G64 || codec == KDN_CODEC_INT4_KC64; }
bool is_td(int codec) { return codec == KDN_CODEC_INT8_TD64 || codec == KDN_CODEC_INT4_TD64; }

// fp32 scales one layer of a chunk holds (0 for raw bf16).
size_t scales_per_layer(size_t row, size_t T, int codec)
{
    if (codec == KDN_CODEC_RAW_BF16) return 0;
    if (is_kc(codec)) return (T + 63) / 64 * row + T * row / 64;         // key scales per channel, then value scales
    return 2 * T * row / 64;
}

// The per-channel key codecs group 64 consecutive chunk tokens; a pool block must lie inside one group.
kdn_status check_kc(const kdn_pool_desc *p, const kdn_chunk *c, int64_t pos)
{
    if ((!is_kc(c->codec) && !is_td(c->codec)) || c->n_tokens == 0) return KDN_OK;
    if (64 % p->block_size || pos % p->block_size) return KDN_E_UNSUPPORTED;
    return KDN_OK;
}

kdn_status check_chunk(const kdn_pool_desc *p, const kdn_chunk *c)
{
    if (c->n_tokens < 0) return KDN_E_INVAL;
    if (c->codec < KDN_CODEC_RAW_BF16 || c->codec > KDN_CODEC_INT4_TD64) return KDN_E_INVAL;
    if (c->mem != KDN_MEM_DEVICE && c->mem != KDN_MEM_PINNED_HOST) return KDN_E_INVAL;
    if (c->codec != KDN_CODEC_RAW_BF16 && p->head_dim % 64) return KDN_E_UNSUPPORTED;
    if (c->bytes != kdn_chunk_bytes(p, c->n_tokens, c->codec)) return KDN_E_SHAPE;
    if (c->n_tokens > 0) {
        if (!c->data) return KDN_E_INVAL;
        if ((uintptr_t)c->data % 16) return KDN_E_ALIGN;
    }
    return KDN_OK;
}

kdn_status check_range(const kdn_pool_desc *p, const int32_t *table, int32_t n_table, int64_t off, int32_t T)
{
    if (n_table < 0 || off < 0) return KDN_E_INVAL;
    if (T > 0 && !table) return KDN_E_INVAL;
    if (off + (int64_t)T > (int64_t)n_table * p->block_size) return KDN_E_RANGE;
    return KDN_OK;
}

unsigned gcd_u(unsigned a, unsigned b) { while (b) { unsigned t = a % b; a = b; b = t; } return a; }
unsigned lcm_u(unsigned a, unsigned b) { return a / gcd_u(a, b) * b; }

// Make `device` current; the runtime's own switch costs a fraction of a microsecond even when nothing changes.
kdn_status use_device(int device)
{
    int cur = -1;
    if (cudaGetDevice(&cur) == cudaSuccess && cur == device) return KDN_OK;
    return cudaSetDevice(device) == cudaSuccess ? KDN_OK : KDN_E_CUDA;
}

kdn_status ensure_side(kdn_ctx *ctx)
{
    if (!ctx->own_side) KDN_CUDA(cudaStreamCreateWithFlags(&ctx->own_side, cudaStreamNonBlocking));
    return KDN_OK;
}

kdn_status ensure_slabs(kdn_ctx *ctx)
{
    for (int i = 0; i < 2; ++i) {
        if (!ctx->slab[i]) KDN_CUDA(cudaMalloc((void **)&ctx->slab[i], ctx->slab_bytes));
        if (!ctx->slab_free[i]) KDN_CUDA(cudaEventCreateWithFlags(&ctx->slab_free[i], cudaEventDisableTiming));
        if (!ctx->slab_ready[i]) KDN_CUDA(cudaEventCreateWithFlags(&ctx->slab_ready[i], cudaEventDisableTiming));
    }
    return KDN_OK;
}

kdn_status ensure_bounce(kdn_ctx *ctx)
{
    for (int i = 0; i < 2; ++i) {
        if (!ctx->bounce[i]) KDN_CUDA(cudaMallocHost((void **)&ctx->bounce[i], ctx->slab_bytes));
        if (!ctx->bounce_done[i]) KDN_CUDA(cudaEventCreateWithFlags(&ctx->bounce_done[i], cudaEventDisableTiming));
    }
    return KDN_OK;
}

// Whole-range pread / pwrite (short transfers are continued, EINTR retried).
bool read_fully(int fd, unsigned char *dst, size_t bytes, long long off)
{
    while (bytes) {
        const ssize_t n = pread(fd, dst, bytes, (off_t)off);
        if (n < 0 && errno == EINTR) continue;
        if (n <= 0) return false;                            // error, or the file ends before the chunk does
        dst += n; off += n; bytes -= (size_t)n;
    }
    return true;
}
bool write_fully(int fd, const unsigned char *src, size_t bytes, long long off)
{
    while (bytes) {
        const ssize_t n = pwrite(fd, src, bytes, (off_t)off);
        if (n < 0 && errno == EINTR) continue;
        if (n <= 0) return false;
        src += n; off += n; bytes -= (size_t)n;
    }
    return true;
}

// Move the file pieces among `pieces` between their files and `bounce` (write = bounce -> file).  One thread copies
// out of the page cache at 5-6 GB/s, a tenth of the host link, so the pieces are cut into slices of kIoSlice bytes
// and up to kIoThreads threads work through them.
// Writes go through a shared mapping of the file where that is possible: buffered writes to ONE file take its inode
// lock exclusively, so parallel pwrite()s queue up behind each other (measured: 5 GB/s however many threads), while
// stores through a mapping only meet at the page level.  Each piece is mapped once by the calling thread and unmapped
// once after the workers are done (an unmap per slice made every worker interrupt all the others to flush their
// address translations).  A regular file is grown to its final length first: a mapping cannot reach past the end.
constexpr size_t kIoSlice = (size_t)4 << 20;
constexpr unsigned kIoThreads = 16;
bool file_io(const std::vector<Piece> &pieces, unsigned char *bounce, bool write)
{
    static const long long page = sysconf(_SC_PAGESIZE) > 0 ? sysconf(_SC_PAGESIZE) : 4096;
    struct Slice { int fd; unsigned char *mem; size_t bytes; long long off; unsigned char *mapped; };
    struct Mapping { void *base; size_t bytes; };
    std::vector<Slice> slices;
    std::vector<Mapping> mappings;
    for (const Piece &p : pieces) {
        if (p.host) continue;
        unsigned char *mapped = nullptr;                     // where the piece's first byte sits in the mapping, if any
        if (write) {
            struct stat sb;
            if (fstat(p.fd, &sb) == 0 && S_ISREG(sb.st_mode)) {
                const long long end = p.file_off + (long long)p.bytes;
                if (sb.st_size >= end || ftruncate(p.fd, (off_t)end) == 0) {
                    const long long a = p.file_off / page * page;
                    const size_t d = (size_t)(p.file_off - a);
                    void *m = mmap(nullptr, p.bytes + d, PROT_READ | PROT_WRITE, MAP_SHARED, p.fd, (off_t)a);
                    if (m != MAP_FAILED) {
                        mappings.push_back(Mapping{ m, p.bytes + d });
                        mapped = (unsigned char *)m + d;
                    }
                }
            }
        }
        for (size_t o = 0; o < p.bytes; o += kIoSlice)
            slices.push_back(Slice{ p.fd, bounce + p.slab_off + o, p.bytes - o < kIoSlice ? p.bytes - o : kIoSlice,
                                    p.file_off + (long long)o, mapped ? mapped + o : nullptr });
    }
    std::atomic<size_t> next{ 0 };
    std::atomic<bool> ok{ true };
    auto work = [&]() {
        for (size_t i = next.fetch_add(1); i < slices.size(); i = next.fetch_add(1)) {
            const Slice &c = slices[i];
            if (write) {
                if (c.mapped) std::memcpy(c.mapped, c.mem, c.bytes);
                else if (!write_fully(c.fd, c.mem, c.bytes, c.off)) ok = false;
            } else if (!read_fully(c.fd, c.mem, c.bytes, c.off)) {
                ok = false;
            }
        }
    };
    const unsigned n_threads = slices.size() < kIoThreads ? (unsigned)slices.size() : kIoThreads;
    std::vector<std::thread> helpers;
    for (unsigned t = 1; t < n_threads; ++t) {
        try { helpers.emplace_back(work); } catch (...) { break; }   // no thread to be had: the caller does the rest
    }
    work();
    for (std::thread &t : helpers) t.join();
    for (const Mapping &m : mappings) munmap(m.base, m.bytes);
    return ok;
}

// Store path: once the slab -> bounce copies of slab `s` have finished, write their pieces to the files.
kdn_status drain_writes(kdn_ctx *ctx, unsigned s)
{
    if (ctx->pending_writes[s].empty()) return KDN_OK;
    KDN_CUDA(cudaEventSynchronize(ctx->bounce_done[s]));
    ctx->bounce_busy[s] = false;
    const bool ok = file_io(ctx->pending_writes[s], ctx->bounce[s], true);
    ctx->pending_writes[s].clear();
    return ok ? KDN_OK : KDN_E_IO;
}

// `overlap`: the launch may start while the kernel before it in the stream (the rotation-table kernel) still runs;
// the warps that read that kernel's output wait for it on the device.
template <typename K>
kdn_status launch_kernel(LaunchEnv &env, K kernel, int threads, unsigned grid, size_t smem, cudaStream_t stream,
                         const Launch &lp, bool overlap = false)
{
    // the pipeline is written for CTAs that are all resident at once: never launch more than fit
    int per_sm = 0;
    kdn_status st = env.resident(kernel, threads, smem, &per_sm);
    if (st != KDN_OK) return st;
    if (per_sm < 1) return KDN_E_UNSUPPORTED;
    const unsigned long long cap = (unsigned long long)per_sm * (unsigned long long)env.sm_count;
    if (grid > cap) grid = (unsigned)cap;
    if (overlap) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3((unsigned)threads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr{};
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        KDN_CUDA(cudaLaunchKernelEx(&cfg, kernel, lp));
    } else {
        kernel<<<grid, threads, smem, stream>>>(lp);
    }
    KDN_CUDA(cudaGetLastError());
    return KDN_OK;
}

// Built-in launch shapes, from sweeps on 8B-shaped KV with fully fragmented tables on B200.  The copy
// form runs best with about two tiles of loads and two of stores in flight per SM; deeper queues lose
// 3-4 % of bandwidth.  The coding forms want more compute warps per SM than the copy form needs.
struct Shape { int tile_bytes, stages, ctas_per_sm, groups, lag; int gw = 4; };
Shape default_shape(int OP, bool any_coded, bool any_rot)
{
    if (!any_coded && !any_rot) return Shape{ 32768, 4, 1, 0, 2 };
    if (OP != OP_COMPOSE || !any_rot) return Shape{ 8192, 6, 3, 2, 2 };
    if (!any_coded) return Shape{ 16384, 4, 2, 1, 2 };
    return Shape{ 8192, 4, 4, 1, 1 };
}

// Pipeline slots: at least lag + 2, a multiple of the compute groups (a slot must always belong to the
// same group), and, unless the caller fixed the count, few enough for ctas_per_sm CTAs to share an SM.
kdn_status fit_stages(int &stages, int groups, int lag, bool shrink, unsigned stage_bytes, int ctas_per_sm, size_t smem_limit,
                      int rows_per_tile = 1, bool wide = false)
{
    const int g = groups > 0 ? groups : 1;
    if (stages > kMaxStages) stages = kMaxStages;
    int min_stages = (lag + 2 + g - 1) / g * g;
    if (stages < min_stages) stages = min_stages;
    stages = stages / g * g;
    if (shrink)
        while (stages - g >= min_stages &&
               smem_bytes(stages, stage_bytes, rows_per_tile, wide) * (size_t)ctas_per_sm > smem_limit - 1024u * (size_t)ctas_per_sm)
            stages -= g;
    return smem_bytes(stages, stage_bytes, rows_per_tile, wide) > smem_limit ? KDN_E_UNSUPPORTED : KDN_OK;
}

// Launch the instantiation for (OP, compute groups, warps per group); groups = 0 is the pure-copy form.
kdn_status launch_tiles(LaunchEnv &env, int OP, int groups, int gw, unsigned grid, size_t smem, cudaStream_t stream,
                        const Launch &lp, bool overlap = false, bool wide = false)
{
#define KDN_CASE(G, W)                                                                                             \
    if (groups == G && (G == 0 || gw == W)) {                                                                      \
        if (OP == OP_STORE) return launch_kernel(env, kdn_store_kernel<G, W>, threads_for(G, W), grid, smem, stream, lp, overlap);      \
        if (OP == OP_RETRIEVE) return launch_kernel(env, kdn_retrieve_kernel<G, W>, threads_for(G, W), grid, smem, stream, lp, overlap); \
        return launch_kernel(env, kdn_compose_kernel<G, W>, threads_for(G, W), grid, smem, stream, lp, overlap);               \
    }
    if (wide) {
        // tiles of up to 16 token rows: the kernels that keep the row indices in shared memory (store and retrieve, copy
        // form and two single-warp groups)
#define KDN_ROWS_CASE(G, W)                                                                                        \
        if (groups == G && (G == 0 || gw == W)) {                                                                  \
            if (OP == OP_STORE) return launch_kernel(env, kdn_store_rows_kernel<G, W>, threads_for(G, W), grid, smem, stream, lp, overlap);       \
            if (OP == OP_RETRIEVE) return launch_kernel(env, kdn_retrieve_rows_kernel<G, W>, threads_for(G, W), grid, smem, stream, lp, overlap); \
        }
        KDN_ROWS_CASE(0, 4) KDN_ROWS_CASE(2, 1)
#undef KDN_ROWS_CASE
        return KDN_E_UNSUPPORTED;
    }
    KDN_CASE(0, 4) KDN_CASE(1, 4) KDN_CASE(2, 4) KDN_CASE(3, 4) KDN_CASE(4, 4) KDN_CASE(6, 4)
    KDN_CASE(2, 1) KDN_CASE(4, 1) KDN_CASE(8, 1)
#undef KDN_CASE
    return KDN_E_UNSUPPORTED;
}

// The rotation table of a launch lives in a ring slot; make it large enough.
kdn_status ensure_table(RingSlot *slot, int n_rope, int half)
{
    if (slot->table_rows_cap >= (size_t)n_rope && slot->table_half == half) return KDN_OK;
    KDN_CUDA(cudaEventSynchronize(slot->done));
    if (slot->d_table) KDN_CUDA(cudaFree(slot->d_table));
    slot->d_table = nullptr;
    const size_t rows = (size_t)n_rope < 64 ? 64 : (size_t)n_rope;
    KDN_CUDA(cudaMalloc((void **)&slot->d_table, rows * (size_t)half * sizeof(float2)));
    slot->table_rows_cap = rows;
    slot->table_half = half;
    return KDN_OK;
}

// Tile one batch of host ops (at most kMaxOpsPerLaunch, all on the device side) and launch it.
kdn_status launch_batch(kdn_ctx *ctx, const Pool &pool, int OP, const HostOp *hops, int n, cudaStream_t stream)
{
    if (n <= 0) return KDN_OK;
    bool any_coded = false, any_rot = false, any_list = false, all_list = true, any_kc = false, all_int4 = true;
    for (int i = 0; i < n; ++i) {
        any_coded |= hops[i].op.codec != KDN_CODEC_RAW_BF16;
        all_int4 &= is_int4(hops[i].op.codec);
        any_kc |= is_kc(hops[i].op.codec);
        any_rot |= hops[i].rotate;
        any_list |= hops[i].op.list_mode != 0;
        all_list &= hops[i].op.list_mode != 0;
    }
    const bool compute = any_coded || any_rot;
    const unsigned row_elems = (unsigned)pool.H * (unsigned)pool.D;
    // Pool blocks of 2 KiB or less (block_size 1 or 2 with whole rows, a few tokens of one KV head): a coding tile that stops
    // at the end of its block is far too small.  Such launches run as keep-list launches over the implied list 0, 1, 2, ...
    // (list_mode 3): a tile then takes several token rows, wherever their blocks are, and rows that are neighbours in the
    // pool still share a copy (8B shape, block_size 1: int8 store / retrieve 3.5 / 3.7 -> 5.2 / 5.3 TB/s).
    std::vector<HostOp> as_rows;
    // (the kernels for tiles of many rows exist for the built-in shapes only: a caller-set shape keeps the ordinary kernels)
    const bool own_shape = ctx->tuning.compute_groups > 0 || ctx->tuning.group_warps > 0;
    if (any_coded && !any_rot && !any_list && !any_kc && (OP == OP_STORE || OP == OP_RETRIEVE) && ctx->tuning.tile_bytes <= 0 && !own_shape &&
        (unsigned long long)pool.bs * row_elems * 2ull <= 2048ull && (unsigned long long)pool.nb * (unsigned)pool.bs < 0xffffffffull) {
        as_rows.assign(hops, hops + n);
        for (HostOp &h : as_rows) {
            h.op.list_mode = 3;
            h.op.n_list = h.op.T;
            h.op.list = nullptr;
        }
        hops = as_rows.data();
        any_list = all_list = true;
    }

    // tile size: whole 16-byte units; whole 64-element groups with int8 / int4; whole head rows with rotation
    unsigned unit = 8;
    if (any_coded) unit = lcm_u(unit, 64);
    if (any_rot) unit = lcm_u(unit, (unsigned)pool.D);
    // decoding a key tile of a per-channel key codec takes one scale per channel: such tiles are whole token rows
    const bool kc_decode = any_kc && OP != OP_STORE;
    if (kc_decode) unit = lcm_u(unit, row_elems);
    Shape def = default_shape(OP, any_coded, any_rot);
    if (kc_decode) def = Shape{ 16384, 4, 2, 1, 1 };      // larger tiles: a key tile also loads a whole row of scales
    // a launch of 4-bit codes only writes (store) or reads (retrieve) a quarter of what crosses the other way: one store
    // group in flight instead of two recycles the slots sooner (8B shape: store 5.96 -> 6.22 TB/s, retrieve 5.98 -> 6.03;
    // with 8-bit codes the same setting loses 5 %)
    else if (all_int4 && !any_rot && !any_list) def.lag = 1;
    else if (all_int4 && any_rot && !any_list) def = Shape{ 8192, 6, 3, 1, 1 };   // compose of 4-bit parts: six slots in three CTAs, 5.66 -> 5.81 TB/s
    if (!compute && !any_list) {
        // a small copy launch (one chunk per call) is mostly pipeline fill and drain: half-size tiles in six slots start
        // storing sooner and end on a shorter tail (one 512-token 8B chunk: 24.8 -> 24.2 us); batched launches keep the
        // larger tiles, which are worth 1 % there
        unsigned long long bytes = 0;
        for (int i = 0; i < n; ++i) bytes += (unsigned long long)hops[i].op.nl * 4ull * (unsigned long long)hops[i].op.T * row_elems;
        if (bytes / 32768ull < 48ull * (unsigned long long)ctx->env.sm_count) def = Shape{ 16384, 6, 1, 0, 2 };
    }
    int tile_bytes = ctx->tuning.tile_bytes > 0 ? ctx->tuning.tile_bytes : def.tile_bytes;
    unsigned tile_elems = (unsigned)tile_bytes / 2u / unit * unit;
    if (tile_elems < unit) tile_elems = unit;
    const unsigned long long block_elems = (unsigned long long)pool.bs * row_elems;
    if (tile_elems > block_elems) tile_elems = (unsigned)((block_elems + unit - 1) / unit * unit);
    // a token-list op moves one token row per tile: the tile must hold a row; a launch of only such ops uses
    // row-sized slots and as many of them as fit, to keep enough bytes in flight
    if (any_list && tile_elems < row_elems) tile_elems = row_elems;
    int rows_per_tile = 1;
    if (all_list) {
        // row-sized tiles are bound by the per-CTA loader and storer, not by bytes in flight per CTA: measured on
        // the 8B shape (2 KiB rows), throughput grows with CTAs per SM up to 8 (copy form 3.0 -> 6.4 TB/s)
        tile_elems = row_elems;
        bool all_keep = true;
        for (int i = 0; i < n; ++i) all_keep &= hops[i].op.list_mode == 1 || hops[i].op.list_mode == 3;
        int want_rows = ctx->tuning.tile_bytes > 0 ? ctx->tuning.tile_bytes / 2 / (int)row_elems : 2048 / (int)row_elems;
        if (kc_decode)                                     // a key tile must lie inside one 64-token group: a power of two
            while (want_rows & (want_rows - 1)) want_rows &= want_rows - 1;
        if (own_shape && want_rows > kMaxRowsPerTile) want_rows = kMaxRowsPerTile;
        if (!any_coded && !any_rot && all_keep && want_rows >= 2 && row_elems < 1024u && (unsigned long long)pool.nb * (unsigned)pool.bs < 0xffffffffull) {
            // copy form on rows shorter than 2 KiB (few KV heads per GPU): several rows per tile as well
            rows_per_tile = want_rows > kWideRowsPerTile ? kWideRowsPerTile : want_rows;
            tile_elems = (unsigned)rows_per_tile * row_elems;
            def = Shape{ 0, 4, 8, 0, 1 };
        } else if (any_coded && !any_rot && all_keep && want_rows >= 2 && (unsigned long long)pool.nb * (unsigned)pool.bs < 0xffffffffull) {
            // coded keep-list launches: a tile takes several listed rows -- neighbours in the chunk, so its codes and
            // scales move with one copy each, and rows that are neighbours in the pool share a copy too.  From a sweep on
            // the 8B shape with half of the tokens kept: two 1024-element rows per tile, five CTAs per SM with two
            // single-warp groups each, one store in flight (int8 5.1 -> 5.9 TB/s, int4 4.0 -> 4.9)
            rows_per_tile = want_rows > kWideRowsPerTile ? kWideRowsPerTile : want_rows;
            tile_elems = (unsigned)rows_per_tile * row_elems;
            def = Shape{ 0, 6, 5, 2, 1, 1 };
        } else if (!any_coded && !any_rot) def = Shape{ 0, 4, 8, 0, 1 };
        else if (OP == OP_STORE) def = Shape{ 0, 8, 8, 2, 2, 1 };      // two single-warp groups: a row is one warp's work
        else def = Shape{ 0, 8, 6, 2, 1, 1 };
    }
    const unsigned tpb = (unsigned)((block_elems + tile_elems - 1) / tile_elems);
    if (!any_list && kc_decode && ctx->tuning.tile_bytes <= 0 && tile_elems * 2u < (unsigned)def.tile_bytes) {
        // per-channel key chunks on small pool blocks (2 / 1 KV heads of the 8B shape: retrieve 4.7 / 2.9 -> 6.3 / 5.8 TB/s)
        def = tile_elems * 2u <= 4096u ? Shape{ 0, 8, 8, 2, 1, 1 } : Shape{ 0, 4, 4, 1, 1 };
    }
    if (!any_list && !kc_decode && ctx->tuning.tile_bytes <= 0) {
        // A pool block smaller than the tile the shape was tuned for (few KV heads per GPU under tensor parallelism, or
        // a small block_size) caps the tile at the block.  From sweeps on the 8B shape with 4, 2 and 1 KV heads:
        // the copy form keeps the same bytes in flight per SM with more CTAs, then more slots (one head, 4 KiB blocks:
        // 1.9 -> 6.3 TB/s); the coding forms give a tile of 4 KiB or less to one warp instead of four (int8 store /
        // retrieve 4.2 / 4.6 -> 5.8 / 5.7, compose 3.8 -> 5.4, eight slots in four CTAs); a rotation-only compose takes six slots in as many CTAs
        // as fit (2.7 -> 6.2); a coded compose whose every tile needs its own table entry takes six slots (5.6 -> 6.2).
        const unsigned tb = tile_elems * 2u;
        const bool capped = tb < (unsigned)def.tile_bytes;
        if (!compute) {
            if (capped) {
                const unsigned in_flight = (unsigned)def.tile_bytes * (unsigned)def.stages * (unsigned)def.ctas_per_sm;
                unsigned ctas = (unsigned)def.tile_bytes / tb * (unsigned)def.ctas_per_sm;
                if (ctas > 8u) ctas = 8u;
                unsigned st = in_flight / (ctas * tb);
                if (st < (unsigned)def.stages) st = (unsigned)def.stages;
                if (st > 16u) st = 16u;
                def.ctas_per_sm = (int)ctas;
                def.stages = (int)st;
            }
        } else if (!any_rot) {
            if (tb <= 4096u) def = Shape{ 0, 8, 4, 2, def.lag, 1 };
        } else if (!any_coded) {
            if (capped) {
                unsigned ctas = (unsigned)ctx->env.smem_optin / (6u * tb + 1024u);
                if (ctas > 6u) ctas = 6u;
                if (ctas < 1u) ctas = 1u;
                def = Shape{ 0, 6, (int)ctas, 1, 1 };
            }
        } else if (tb <= 4096u) {
            def = Shape{ 0, 8, 4, 2, 1, 1 };
        } else if (tpb == 1u) {
            def = Shape{ 0, 6, 3, 1, 1 };
        }
    }
    const unsigned a_bytes = (tile_elems * 2u + 127u) & ~127u;
    const unsigned b_bytes = compute ? ((tile_elems + 127u) & ~127u) : 0u;
    unsigned s_bytes = compute ? ((tile_elems / 16u + 127u) & ~127u) : 0u;
    if (kc_decode && s_bytes < row_elems * 4u) s_bytes = (row_elems * 4u + 127u) & ~127u;   // one scale per channel
    const unsigned stage_bytes = a_bytes + b_bytes + s_bytes;
    int groups = 0;
    if (compute) groups = ctx->tuning.compute_groups > 0 ? ctx->tuning.compute_groups : def.groups;
    const int lag = ctx->tuning.store_lag > 0 ? ctx->tuning.store_lag : def.lag;
    int ctas_per_sm = ctx->tuning.ctas_per_sm > 0 ? ctx->tuning.ctas_per_sm : def.ctas_per_sm;
    int stages = ctx->tuning.stages > 0 ? ctx->tuning.stages : def.stages;
    const size_t smem_limit = (size_t)ctx->env.smem_optin;
    // more than four rows per tile, and dense ops run as rows, go to the kernels built for that
    const bool wide = rows_per_tile > kMaxRowsPerTile || !as_rows.empty();
    kdn_status fit = fit_stages(stages, groups, lag, ctx->tuning.stages <= 0, stage_bytes, ctas_per_sm, smem_limit, rows_per_tile, wide);
    if (fit != KDN_OK) return fit;
    const size_t smem = smem_bytes(stages, stage_bytes, rows_per_tile, wide);

    // Few ops travel as kernel parameters; otherwise through a ring slot (pinned staging + device copy).  A ring
    // slot is also what owns the rotation table.
    const bool inl = n <= kInlineOps;
    RingSlot *slot = nullptr;
    if (!inl || any_rot) {
        slot = &ctx->ring[ctx->ring_next++ % kRing];
        if (slot->used) KDN_CUDA(cudaEventSynchronize(slot->done));
    }
    Launch lp{};
    RopeInline rope_inl{};
    DevOp *h_ops = inl ? lp.inline_ops : slot->h_ops;
    RopeParam *h_rope = inl ? rope_inl.p : (slot ? slot->h_rope : nullptr);

    unsigned long long tiles = 0;
    int n_rope = 0;
    int kc_layers = 0, kc_groups = 0;                      // grid of the key-plane store kernel (0: not needed)
    for (int i = 0; i < n; ++i) {
        DevOp op = hops[i].op;
        op.tile_begin = (unsigned)tiles;
        op.rope = -1;
        if (hops[i].rotate) {
            h_rope[n_rope] = hops[i].rp;
            op.rope = n_rope++;
        }
        if (OP == OP_STORE && is_kc(op.codec)) {
            // the tile pipeline codes the value planes; the key planes go through kdn_store_kc_kernel below
            op.kv_sel = 2;
            if (op.nl > kc_layers) kc_layers = op.nl;
            const int g = (op.T + 63) / 64;
            if (g > kc_groups) kc_groups = g;
        }
        h_ops[i] = op;
        tiles += (unsigned long long)op.nl * (op.kv_sel ? 1ull : 2ull) *
                 (op.list_mode ? ((unsigned long long)op.n_list + (unsigned)rows_per_tile - 1ull) / (unsigned)rows_per_tile
                               : (unsigned long long)op.nblk * tpb);
        if (tiles > kMaxTilesPerLaunch) return KDN_E_UNSUPPORTED;
    }
    if (tiles == 0) return KDN_OK;

    if (!inl) KDN_CUDA(cudaMemcpyAsync(slot->d_ops, slot->h_ops, sizeof(DevOp) * (size_t)n, cudaMemcpyHostToDevice, stream));
    const int half = pool.D / 2;
    if (n_rope) {
        {
            kdn_status r = ensure_table(slot, n_rope, half);
            if (r != KDN_OK) return r;
        }
        if (!inl) KDN_CUDA(cudaMemcpyAsync(slot->d_rope, slot->h_rope, sizeof(RopeParam) * (size_t)n_rope, cudaMemcpyHostToDevice, stream));
        const long long total = (long long)n_rope * half;
        kdn_rope_table_kernel<<<(unsigned)((total + 127) / 128), 128, 0, stream>>>(inl ? nullptr : slot->d_rope, rope_inl, n_rope,
                                                                              pool.D, slot->d_table);
        KDN_CUDA(cudaGetLastError());
        ctx->launches++;
    }

    lp.ops = inl ? nullptr : slot->d_ops;
    lp.n_ops = n;
    lp.n_tiles = (unsigned)tiles;
    lp.k_layers = pool.d_k;
    lp.v_layers = pool.d_v;
    lp.n_blocks = pool.nb;
    lp.bs = pool.bs;
    lp.D = pool.D;
    lp.row_elems = row_elems;
    lp.tile_elems = tile_elems;
    lp.tpb = tpb;
    lp.rope = slot ? slot->d_table : nullptr;
    lp.status = ctx->d_status;
    lp.stages = stages;
    lp.stage_bytes = stage_bytes;
    lp.off_b = a_bytes;
    lp.off_s = a_bytes + b_bytes;
    lp.store_lag = lag;
    lp.reload_first = (!compute && tile_elems * 2u >= 8192u) ? 1 : 0;
    lp.wait_limit_ns = ctx->wait_limit_ns;
    lp.one = 1.0f;
    lp.rows_per_tile = rows_per_tile;

    if (kc_groups > 0) {
        // key planes of the per-channel key codecs: one CTA per (64-token group, layer, op)
        // channels per CTA: at most 256 (36 KiB of shared memory, six CTAs per SM), a multiple of eight that divides the row
        unsigned n_split = 1;
        while (row_elems / n_split > kKcCols && row_elems % (n_split * 2u * 8u) == 0u) n_split *= 2u;
        const unsigned cols = row_elems / n_split;
        const size_t kc_smem = kc_smem_bytes(cols);
        if (kc_smem > smem_limit) return KDN_E_UNSUPPORTED;
        unsigned kc_threads = (cols / 8u + 7u) / 8u * 32u;       // a warp per 64 channels
        if (kc_threads > 512u) kc_threads = 512u;
        if (kc_threads < 64u) kc_threads = 64u;
        KcLaunch kp{};
        kp.one = 1.0f;
        kp.wait_limit_ns = ctx->wait_limit_ns;
        kp.cols = cols;
        kp.n_split = n_split;
        kp.ops = inl ? nullptr : slot->d_ops;
        kp.n_ops = n;
        kp.k_layers = pool.d_k;
        kp.n_blocks = pool.nb;
        kp.bs = pool.bs;
        kp.row_elems = row_elems;
        kp.status = ctx->d_status;
        if (inl) std::memcpy(kp.inline_ops, lp.inline_ops, sizeof(DevOp) * (size_t)n);
        {
            int per_sm = 0;                                  // first sight of the kernel raises its shared-memory limit
            kdn_status r = ctx->env.resident(kdn_store_kc_kernel, (int)kc_threads, kc_smem, &per_sm);
            if (r != KDN_OK) return r;
            if (per_sm < 1) return KDN_E_UNSUPPORTED;
        }
        kdn_store_kc_kernel<<<dim3((unsigned)kc_groups * n_split, (unsigned)kc_layers, (unsigned)n), kc_threads, kc_smem, stream>>>(kp);
        KDN_CUDA(cudaGetLastError());
        ctx->launches++;
    }

    unsigned long long want = (unsigned long long)ctx->env.sm_count * (unsigned)ctas_per_sm;
    const unsigned grid = (unsigned)(tiles < want ? tiles : want);
    const int gw = ctx->tuning.group_warps > 0 ? ctx->tuning.group_warps : def.gw;
    // Every launch of the pipeline is a programmatic dependent launch.  After the rotation-table kernel only the warps
    // that read the table wait for it; otherwise every thread waits for the kernel before it, whatever that was.
    lp.wait_all = (OP == OP_COMPOSE && n_rope > 0) ? 0 : 1;
    kdn_status st = launch_tiles(ctx->env, OP, groups, gw, grid, smem, stream, lp, true, wide);
    if (st != KDN_OK) return st;
    ctx->launches++;
    ctx->last.op = OP;
    ctx->last.compute_groups = groups;
    ctx->last.group_warps = groups ? gw : 4;
    ctx->last.tile_bytes = (int32_t)(tile_elems * 2u);
    ctx->last.stages = stages;
    ctx->last.ctas_per_sm = ctas_per_sm;
    ctx->last.store_lag = lag;
    ctx->last.grid = (int32_t)grid;
    ctx->last.smem_bytes = (int32_t)smem;
    ctx->last.n_tiles = (uint32_t)tiles;
    ctx->last.rows_per_tile = rows_per_tile;
    ctx->last.rows_kernel = wide ? 1 : 0;
    if (slot) {
        KDN_CUDA(cudaEventRecord(slot->done, stream));
        slot->used = true;
    }
    return KDN_OK;
}

// Ops whose chunk is in a token-delta Rice codec: at most kInlineOps per launch, their records travel as kernel
// parameters.  Store is three launches (plan, scan, encode), retrieve and compose one (plus the rotation table).
kdn_status launch_td(kdn_ctx *ctx, const Pool &pool, int OP, const HostOp *hops, int n, cudaStream_t stream)
{
    const unsigned row_elems = (unsigned)pool.H * (unsigned)pool.D;
    // channels per CTA: a multiple of 16 that divides the row, whole heads when keys are re-rotated, kTdCols if possible
    // (small slices: many CTAs share an SM, and each one's loads, decoding and stores overlap the others')
    bool any_rot = false;
    for (int i = 0; i < n; ++i) any_rot |= hops[i].rotate;
    const unsigned unit = any_rot ? lcm_u(16u, (unsigned)pool.D) : 16u;
    unsigned n_split = 1;
    while (row_elems / n_split > kTdCols && row_elems % (n_split * 2u) == 0u && (row_elems / (n_split * 2u)) % unit == 0u) n_split *= 2u;
    const unsigned cols = row_elems / n_split;
    if (cols % 16u || cols > 1024u) return KDN_E_UNSUPPORTED;
    unsigned threads = (cols + 31u) & ~31u;                  // one thread per channel in the coding loops
    if (threads < 64u) threads = 64u;
    if (threads > 512u) return KDN_E_UNSUPPORTED;
    const size_t smem_limit = (size_t)ctx->env.smem_optin;

    for (int first = 0; first < n; first += kInlineOps) {
        const int m = n - first < kInlineOps ? n - first : kInlineOps;
        TdLaunch tp{};
        tp.wait_limit_ns = ctx->wait_limit_ns;
        RopeInline rope_inl{};
        int n_rope = 0, max_groups = 0, max_layers = 0;
        for (int i = 0; i < m; ++i) {
            DevOp op = hops[first + i].op;
            op.rope = -1;
            if (hops[first + i].rotate) {
                rope_inl.p[n_rope] = hops[first + i].rp;
                op.rope = n_rope++;
            }
            tp.inline_ops[i] = op;
            const int g = (op.T + 63) / 64;
            if (g > max_groups) max_groups = g;
            if (op.nl > max_layers) max_layers = op.nl;
        }
        if (max_groups == 0 || max_layers == 0) continue;
        tp.ops = nullptr;
        tp.n_ops = m;
        tp.k_layers = pool.d_k;
        tp.v_layers = pool.d_v;
        tp.n_blocks = pool.nb;
        tp.bs = pool.bs;
        tp.D = pool.D;
        tp.L = pool.L;
        tp.row_elems = row_elems;
        tp.cols = cols;
        tp.n_split = n_split;
        tp.status = ctx->d_status;
        const dim3 grid((unsigned)max_groups * n_split, (unsigned)max_layers * 2u, (unsigned)m);
        int per_sm = 0;
        if (OP == OP_STORE) {
            const size_t smem_plan = td_store_smem_bytes(cols, false), smem_enc = td_store_smem_bytes(cols, true);
            if (smem_enc > smem_limit) return KDN_E_UNSUPPORTED;
            kdn_status r = ctx->env.resident(kdn_td_plan_kernel, (int)threads, smem_plan, &per_sm);
            if (r == KDN_OK && per_sm >= 1) r = ctx->env.resident(kdn_td_encode_kernel, (int)threads, smem_enc, &per_sm);
            if (r != KDN_OK) return r;
            if (per_sm < 1) return KDN_E_UNSUPPORTED;
            kdn_td_plan_kernel<<<grid, threads, smem_plan, stream>>>(tp);
            KDN_CUDA(cudaGetLastError());
            kdn_td_scan_kernel<<<(unsigned)m, 256, 0, stream>>>(tp);
            KDN_CUDA(cudaGetLastError());
            kdn_td_encode_kernel<<<grid, threads, smem_enc, stream>>>(tp);
            KDN_CUDA(cudaGetLastError());
            ctx->launches += 3;
        } else {
            const size_t smem = td_decode_smem_bytes(cols);
            if (smem > smem_limit) return KDN_E_UNSUPPORTED;
            RingSlot *slot = nullptr;
            if (n_rope) {
                slot = &ctx->ring[ctx->ring_next++ % kRing];
                if (slot->used) KDN_CUDA(cudaEventSynchronize(slot->done));
                kdn_status r = ensure_table(slot, n_rope, pool.D / 2);
                if (r != KDN_OK) return r;
                const long long total = (long long)n_rope * (pool.D / 2);
                kdn_rope_table_kernel<<<(unsigned)((total + 127) / 128), 128, 0, stream>>>(nullptr, rope_inl, n_rope, pool.D, slot->d_table);
                KDN_CUDA(cudaGetLastError());
                ctx->launches++;
                tp.rope = slot->d_table;
            }
            kdn_status r = KDN_OK;
#define KDN_TD_DECODE(COMPOSE, COLS)                                                                        \
            {                                                                                               \
                r = ctx->env.resident(kdn_td_decode_kernel<COMPOSE, COLS>, (int)threads, smem, &per_sm);    \
                if (r != KDN_OK) return r;                                                                  \
                if (per_sm < 1) return KDN_E_UNSUPPORTED;                                                   \
                kdn_td_decode_kernel<COMPOSE, COLS><<<grid, threads, smem, stream>>>(tp);                   \
            }
            if (cols == kTdCols && threads == kTdCols) {
                if (OP == OP_COMPOSE) KDN_TD_DECODE(true, kTdCols) else KDN_TD_DECODE(false, kTdCols)
            } else {
                if (OP == OP_COMPOSE) KDN_TD_DECODE(true, 0) else KDN_TD_DECODE(false, 0)
            }
#undef KDN_TD_DECODE
            KDN_CUDA(cudaGetLastError());
            ctx->launches++;
            if (slot) {
                KDN_CUDA(cudaEventRecord(slot->done, stream));
                slot->used = true;
            }
        }
    }
    return KDN_OK;
}

kdn_status launch_all(kdn_ctx *ctx, const Pool &pool, int OP, const std::vector<HostOp> &hops, cudaStream_t stream,
                      size_t max_ops = kMaxOpsPerLaunch)
{
    bool any_td = false;
    for (const HostOp &h : hops) any_td |= is_td(h.op.codec);
    if (any_td) {
        // token-delta chunks go through their own kernels; everything else through the tile pipeline
        std::vector<HostOp> td, rest;
        for (const HostOp &h : hops) (is_td(h.op.codec) ? td : rest).push_back(h);
        kdn_status st = launch_td(ctx, pool, OP, td.data(), (int)td.size(), stream);
        if (st != KDN_OK) return st;
        for (size_t i = 0; i < rest.size(); i += max_ops) {
            size_t n = rest.size() - i < max_ops ? rest.size() - i : max_ops;
            st = launch_batch(ctx, pool, OP, rest.data() + i, (int)n, stream);
            if (st != KDN_OK) return st;
        }
        return KDN_OK;
    }
    for (size_t i = 0; i < hops.size(); i += max_ops) {
        size_t n = hops.size() - i < max_ops ? hops.size() - i : max_ops;
        kdn_status st = launch_batch(ctx, pool, OP, hops.data() + i, (int)n, stream);
        if (st != KDN_OK) return st;
    }
    return KDN_OK;
}

// The device record of an op that covers all layers of a device-resident chunk.
HostOp make_host_op(const Pool &pool, const int32_t *table, int32_t n_table, int64_t off, const kdn_chunk &c)
{
    HostOp h;
    std::memset(&h.op, 0, sizeof h.op);
    h.op.table = table;
    h.op.data = (unsigned char *)c.data;
    h.op.off = off;
    h.op.T = c.n_tokens;
    h.op.codec = c.codec;
    h.op.j0 = (int)(off / pool.bs);
    h.op.nblk = c.n_tokens > 0 ? (int)((off + c.n_tokens - 1) / pool.bs - off / pool.bs + 1) : 0;
    h.op.rope = -1;
    h.op.l0 = 0;
    h.op.nl = pool.L;
    h.op.pos_end = (long long)n_table * pool.bs;
    const size_t elems = (size_t)pool.L * 2u * (size_t)c.n_tokens * (size_t)pool.H * (size_t)pool.D;
    if (is_td(c.codec))       // these codecs keep their scales inside the chunk: the field points behind the bytes that exist
        h.op.scales = (unsigned char *)c.data + td_layout(pool.L, (unsigned)pool.H * (unsigned)pool.D, c.n_tokens, c.codec).capacity;
    if (c.codec != KDN_CODEC_RAW_BF16 && !is_td(c.codec)) h.op.scales = (unsigned char *)c.data + (is_int4(c.codec) ? elems / 2u : elems);
    return h;
}

// Ops whose chunk lives in pinned host memory go through the two staging slabs in layer ranges:
//   retrieve / compose: side stream copies host -> slab, main stream runs the kernel on the slab;
//   store:              main stream runs the kernel into the slab, side stream copies slab -> host.
// While one slab is being copied the kernel works on the other.
// `between` is called once per slab hand-over, at the point where the main stream would otherwise only wait for the
// host link: the caller uses it to enqueue a share of its device-resident work there.
kdn_status run_staged(kdn_ctx *ctx, const Pool &pool, int OP, const std::vector<HostOp> &hops,
                      cudaStream_t stream, cudaStream_t side, const std::function<kdn_status()> &between)
{
    kdn_status st = ensure_slabs(ctx);
    if (st != KDN_OK) return st;
    const size_t row = (size_t)pool.H * pool.D;
    std::vector<HostOp> batch;
    std::vector<Piece> pieces;
    size_t used = 0;

    auto flush = [&]() -> kdn_status {
        if (batch.empty()) return KDN_OK;
        const unsigned s = ctx->slab_next++ & 1u;
        bool any_file = false;
        for (const Piece &p : pieces) any_file |= p.host == nullptr;
        if (any_file) {
            kdn_status r = ensure_bounce(ctx);
            if (r != KDN_OK) return r;
        }
        if (OP == OP_STORE) {
            // bounce[s] still holds file pieces of the store before last: put them into their files first
            kdn_status r = drain_writes(ctx, s);
            if (r != KDN_OK) return r;
            KDN_CUDA(cudaStreamWaitEvent(stream, ctx->slab_free[s], 0));
            r = launch_all(ctx, pool, OP, batch, stream);
            if (r != KDN_OK) return r;
            KDN_CUDA(cudaEventRecord(ctx->slab_ready[s], stream));
            KDN_CUDA(cudaStreamWaitEvent(side, ctx->slab_ready[s], 0));
            for (const Piece &p : pieces)
                KDN_CUDA(cudaMemcpyAsync(p.host ? p.host : ctx->bounce[s] + p.slab_off, ctx->slab[s] + p.slab_off, p.bytes,
                                         cudaMemcpyDeviceToHost, side));
            KDN_CUDA(cudaEventRecord(ctx->slab_free[s], side));
            if (any_file) {
                KDN_CUDA(cudaEventRecord(ctx->bounce_done[s], side));
                ctx->bounce_busy[s] = true;
                for (const Piece &p : pieces)
                    if (!p.host) ctx->pending_writes[s].push_back(p);
            }
            r = between();                                       // device-resident work runs while the slab drains
            if (r != KDN_OK) return r;
        } else {
            if (any_file) {
                // the host reads the file pieces into bounce[s] while the GPU works on the other slab
                if (ctx->bounce_busy[s]) KDN_CUDA(cudaEventSynchronize(ctx->bounce_done[s]));
                ctx->bounce_busy[s] = false;
                if (!file_io(pieces, ctx->bounce[s], false)) return KDN_E_IO;
            }
            KDN_CUDA(cudaStreamWaitEvent(side, ctx->slab_free[s], 0));
            for (const Piece &p : pieces)
                KDN_CUDA(cudaMemcpyAsync(ctx->slab[s] + p.slab_off, p.host ? p.host : ctx->bounce[s] + p.slab_off, p.bytes,
                                         cudaMemcpyHostToDevice, side));
            if (any_file) {
                KDN_CUDA(cudaEventRecord(ctx->bounce_done[s], side));
                ctx->bounce_busy[s] = true;
            }
            KDN_CUDA(cudaEventRecord(ctx->slab_ready[s], side));
            kdn_status r = between();                            // device-resident work runs while the slab fills
            if (r != KDN_OK) return r;
            KDN_CUDA(cudaStreamWaitEvent(stream, ctx->slab_ready[s], 0));
            r = launch_all(ctx, pool, OP, batch, stream);
            if (r != KDN_OK) return r;
            KDN_CUDA(cudaEventRecord(ctx->slab_free[s], stream));
        }
        batch.clear();
        pieces.clear();
        used = 0;
        return KDN_OK;
    };

    for (const HostOp &h : hops) {
        const size_t T = (size_t)h.op.T;
        if (T == 0) continue;
        const bool coded = h.op.codec != KDN_CODEC_RAW_BF16;
        const size_t codes_per_layer = is_int4(h.op.codec) ? T * row : 2 * T * row * (coded ? 1 : 2);
        const size_t scale_bytes_per_layer = scales_per_layer(row, T, h.op.codec) * 4;
        const size_t per_layer = ((codes_per_layer + 255) & ~(size_t)255) + ((scale_bytes_per_layer + 255) & ~(size_t)255);
        if (per_layer > ctx->slab_bytes) return KDN_E_UNSUPPORTED;
        unsigned char *host = h.op.data;
        const size_t host_codes_total = (size_t)pool.L * codes_per_layer;
        int l = h.op.l0;                                    // the op's own layer range (the whole chunk unless layer-wise)
        const int l_end = h.op.l0 + h.op.nl;
        while (l < l_end) {
            size_t room = ctx->slab_bytes - used;
            if (room < per_layer) {
                st = flush();
                if (st != KDN_OK) return st;
                room = ctx->slab_bytes;
            }
            int nl = (int)(room / per_layer);
            if (nl > l_end - l) nl = l_end - l;
            // a piece is laid out exactly like a chunk of nl layers: codes, then scales
            const size_t base = used;
            const size_t cbytes = (size_t)nl * codes_per_layer;
            const size_t sbytes = (size_t)nl * scale_bytes_per_layer;
            HostOp sub = h;
            sub.op.l0 = l;
            sub.op.nl = nl;
            const unsigned s = ctx->slab_next & 1u;
            sub.op.data = ctx->slab[s] + base;
            sub.op.scales = sbytes ? ctx->slab[s] + base + cbytes : nullptr;
            if (h.fd >= 0) {
                pieces.push_back(Piece{ nullptr, base, cbytes, h.fd, h.file_off + (long long)((size_t)l * codes_per_layer) });
                if (sbytes)
                    pieces.push_back(Piece{ nullptr, base + cbytes, sbytes, h.fd,
                                            h.file_off + (long long)(host_codes_total + (size_t)l * scale_bytes_per_layer) });
            } else {
                pieces.push_back(Piece{ host + (size_t)l * codes_per_layer, base, cbytes, -1, 0 });
                if (sbytes)
                    pieces.push_back(Piece{ host + host_codes_total + (size_t)l * scale_bytes_per_layer, base + cbytes, sbytes, -1, 0 });
            }
            batch.push_back(sub);
            used = (base + cbytes + sbytes + 255) & ~(size_t)255;
            l += nl;
        }
    }
    st = flush();
    if (OP == OP_STORE) {
        // a store into files returns once the files hold the chunks
        for (unsigned s = 0; s < 2; ++s) {
            const kdn_status w = drain_writes(ctx, s);
            if (st == KDN_OK) st = w;
        }
    }
    return st;
}

// Bytes of the chunk side of one op (what crosses the host link when the chunk is host resident).
size_t chunk_side_bytes(const Pool &pool, const HostOp &h)
{
    const size_t elems = (size_t)h.op.nl * 2u * (size_t)h.op.T * (size_t)pool.H * (size_t)pool.D;
    if (h.op.codec == KDN_CODEC_RAW_BF16) return elems * 2u;
    return (is_int4(h.op.codec) ? elems / 2u : elems) +
           (size_t)h.op.nl * scales_per_layer((size_t)pool.H * (size_t)pool.D, (size_t)h.op.T, h.op.codec) * 4u;
}

// Retrieve / compose from token-delta chunks in page-locked host memory: the bytes each chunk uses (its own offset
// table says how many) are copied into a staging slab on the side stream, as many chunks as fit, and decoded from there
// while the next slab fills.
kdn_status run_td_host(kdn_ctx *ctx, const Pool &pool, int OP, const std::vector<HostOp> &hops, cudaStream_t stream, cudaStream_t side)
{
    kdn_status st = ensure_slabs(ctx);
    if (st != KDN_OK) return st;
    const unsigned row_elems = (unsigned)pool.H * (unsigned)pool.D;
    std::vector<HostOp> batch;
    std::vector<Piece> pieces;
    size_t fill = 0;
    auto flush = [&]() -> kdn_status {
        if (batch.empty()) return KDN_OK;
        const unsigned s = ctx->slab_next++ & 1u;
        bool any_file = false;
        for (const Piece &p : pieces) any_file |= p.host == nullptr;
        if (any_file) {
            // chunks in files: the host reads their bytes in use into the page-locked mirror of the slab first
            kdn_status r = ensure_bounce(ctx);
            if (r != KDN_OK) return r;
            if (ctx->bounce_busy[s]) KDN_CUDA(cudaEventSynchronize(ctx->bounce_done[s]));
            ctx->bounce_busy[s] = false;
            if (!file_io(pieces, ctx->bounce[s], false)) return KDN_E_IO;
        }
        KDN_CUDA(cudaStreamWaitEvent(side, ctx->slab_free[s], 0));
        for (const Piece &p : pieces)
            KDN_CUDA(cudaMemcpyAsync(ctx->slab[s] + p.slab_off, p.host ? p.host : ctx->bounce[s] + p.slab_off, p.bytes,
                                     cudaMemcpyHostToDevice, side));
        if (any_file) {
            KDN_CUDA(cudaEventRecord(ctx->bounce_done[s], side));
            ctx->bounce_busy[s] = true;
        }
        KDN_CUDA(cudaEventRecord(ctx->slab_ready[s], side));
        KDN_CUDA(cudaStreamWaitEvent(stream, ctx->slab_ready[s], 0));
        for (HostOp &h : batch) {                                                             // offsets become addresses
            h.op.data = ctx->slab[s] + (size_t)(uintptr_t)h.op.data;
            h.op.scales = ctx->slab[s] + (size_t)(uintptr_t)h.op.scales;
        }
        kdn_status r = launch_td(ctx, pool, OP, batch.data(), (int)batch.size(), stream);
        if (r != KDN_OK) return r;
        KDN_CUDA(cudaEventRecord(ctx->slab_free[s], stream));
        batch.clear();
        pieces.clear();
        fill = 0;
        return KDN_OK;
    };
    for (const HostOp &h : hops) {
        const TdLayout lay = td_layout(pool.L, row_elems, h.op.T, h.op.codec);
        // the chunk's own offset table says how many bytes it uses: in host memory it is read in place, from a file it
        // is read first (a short blocking read of 8 (S + 1) bytes)
        std::vector<unsigned long long> from_file;
        const unsigned long long *seg_off = reinterpret_cast<const unsigned long long *>(h.op.data);
        if (h.fd >= 0) {
            from_file.resize((size_t)lay.S + 1u);
            if (!read_fully(h.fd, reinterpret_cast<unsigned char *>(from_file.data()), from_file.size() * 8u, h.file_off)) return KDN_E_IO;
            seg_off = from_file.data();
        }
        const unsigned long long used = seg_off[lay.S];
        bool stored = used >= lay.streams && used <= lay.capacity && !(used & 15ull) && seg_off[0] == lay.streams;
        for (unsigned long long i = 0; stored && i < lay.S; ++i) stored = seg_off[i] <= seg_off[i + 1];
        if (!stored) return KDN_E_SHAPE;                     // not a chunk a store has written
        if (used > ctx->slab_bytes) return KDN_E_UNSUPPORTED;
        if (fill + used > ctx->slab_bytes) {
            st = flush();
            if (st != KDN_OK) return st;
        }
        pieces.push_back(h.fd >= 0 ? Piece{ nullptr, fill, (size_t)used, h.fd, h.file_off } : Piece{ h.op.data, fill, (size_t)used, -1, 0 });
        HostOp sub = h;
        sub.op.data = (unsigned char *)(uintptr_t)fill;      // offset inside the slab until the slab is known
        sub.op.scales = (unsigned char *)(uintptr_t)(fill + (size_t)used);   // the slab holds no more of the chunk than this
        batch.push_back(sub);
        fill = (fill + (size_t)used + 255) & ~(size_t)255;
    }
    return flush();
}

kdn_status run_ops(kdn_ctx *ctx, int pool_id, int OP, std::vector<HostOp> &dev_ops, std::vector<HostOp> &host_ops,
                   void *cuda_stream, void *side_stream)
{
    const Pool &pool = ctx->pools[(size_t)pool_id];
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (host_ops.empty()) return launch_all(ctx, pool, OP, dev_ops, stream);
    cudaStream_t side = (cudaStream_t)side_stream;
    if (!side) {
        kdn_status st = ensure_side(ctx);
        if (st != KDN_OK) return st;
        side = ctx->own_side;
    }
    // Host-resident token-delta chunks travel whole (only the bytes they use), apart from the layer-range staging
    std::vector<HostOp> td_host;
    for (size_t i = 0; i < host_ops.size();) {
        if (is_td(host_ops[i].op.codec)) { td_host.push_back(host_ops[i]); host_ops.erase(host_ops.begin() + (long)i); }
        else ++i;
    }
    if (!td_host.empty()) {
        if (OP == OP_STORE) return KDN_E_UNSUPPORTED;        // the size of the result is not known before the kernels ran
        if (!ctx->fork) KDN_CUDA(cudaEventCreateWithFlags(&ctx->fork, cudaEventDisableTiming));
        KDN_CUDA(cudaEventRecord(ctx->fork, stream));
        KDN_CUDA(cudaStreamWaitEvent(side, ctx->fork, 0));
        kdn_status st = run_td_host(ctx, pool, OP, td_host, stream, side);
        if (st != KDN_OK) return st;
        if (host_ops.empty()) return launch_all(ctx, pool, OP, dev_ops, stream);
    }
    // Host-resident chunks cross the link slab by slab.  The device-resident ops of the same call are cut into about
    // as many launches as there are slab hand-overs and enqueued between them, so the GPU works on them while the
    // link is busy instead of before it (one stream: a single big launch up front would leave the link idle behind it).
    size_t staged = 0;
    for (const HostOp &h : host_ops) staged += chunk_side_bytes(pool, h);
    size_t n_parts = staged / ctx->slab_bytes + 1;
    if (n_parts > dev_ops.size()) n_parts = dev_ops.size();
    size_t dev_total = 0;
    for (const HostOp &h : dev_ops) dev_total += chunk_side_bytes(pool, h);
    size_t next = 0, done_bytes = 0, part = 0;
    auto between = [&]() -> kdn_status {
        if (next >= dev_ops.size()) return KDN_OK;
        ++part;
        const size_t target = part >= n_parts ? dev_total : dev_total / n_parts * part;
        std::vector<HostOp> share;
        while (next < dev_ops.size() && (share.empty() || done_bytes < target)) {
            done_bytes += chunk_side_bytes(pool, dev_ops[next]);
            share.push_back(dev_ops[next++]);
        }
        // at most kInlineOps ops per launch: their records then travel as kernel parameters.  A descriptor copy
        // would queue on the copy engine behind the slab transfer in flight and hold the launch back by a whole slab.
        return launch_all(ctx, pool, OP, share, stream, (size_t)kInlineOps);
    };
    // Fork: the side stream's copies come after everything already queued on the caller's stream (a copy that filled
    // the pinned chunk, an earlier store into it through another side stream).
    if (!ctx->fork) KDN_CUDA(cudaEventCreateWithFlags(&ctx->fork, cudaEventDisableTiming));
    KDN_CUDA(cudaEventRecord(ctx->fork, stream));
    KDN_CUDA(cudaStreamWaitEvent(side, ctx->fork, 0));
    kdn_status st = run_staged(ctx, pool, OP, host_ops, stream, side, between);
    while (st == KDN_OK && next < dev_ops.size()) st = between();
    // Join: a store's device-to-host copies run on the side stream; the caller's stream waits for them, so that an
    // event or a synchronisation on cuda_stream covers the whole call.  (Retrieve and compose end with kernels on
    // cuda_stream that already waited for their copies.)
    if (OP == OP_STORE)
        for (int i = 0; i < 2; ++i)
            if (ctx->slab_free[i]) {
                const cudaError_t e = cudaStreamWaitEvent(stream, ctx->slab_free[i], 0);
                if (e != cudaSuccess && st == KDN_OK) st = KDN_E_CUDA;
            }
    return st;
}

// The record of `h` restricted to layers [l0, l0 + nl) of a device-resident chunk.
HostOp layer_range(const Pool &pool, const HostOp &h, int l0, int nl)
{
    HostOp sub = h;
    const size_t plane = 2u * (size_t)h.op.T * (size_t)pool.H * (size_t)pool.D;     // elements of one layer
    sub.op.l0 = l0;
    sub.op.nl = nl;
    if (is_td(h.op.codec)) return sub;                      // segments are found through the chunk's own offset table
    if (h.op.codec != KDN_CODEC_RAW_BF16) {
        sub.op.data = h.op.data + (size_t)l0 * (is_int4(h.op.codec) ? plane / 2u : plane);
        sub.op.scales = h.op.scales + (size_t)l0 * scales_per_layer((size_t)pool.H * (size_t)pool.D, (size_t)h.op.T, h.op.codec) * 4u;
    } else {
        sub.op.data = h.op.data + (size_t)l0 * plane * 2u;
    }
    return sub;
}

kdn_pool_desc shape_of(const Pool &p)
{
    kdn_pool_desc d{};
    d.n_layers = p.L; d.n_kv_heads = p.H; d.head_dim = p.D; d.block_size = p.bs; d.n_blocks = p.nb;
    return d;
}

kdn_status xfer(kdn_ctx *ctx, int pool_id, int OP, const kdn_xfer_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    if (!ctx || pool_id < 0 || (size_t)pool_id >= ctx->pools.size()) return KDN_E_INVAL;
    const Pool &pool = ctx->pools[(size_t)pool_id];
    const kdn_pool_desc shape = shape_of(pool);
    kdn_status st = kdn_validate_xfer(&shape, ops, n_ops);
    if (st != KDN_OK) return st;
    if (use_device(ctx->device) != KDN_OK) return KDN_E_CUDA;
    if (n_ops == 1 && ops[0].chunk.mem == KDN_MEM_DEVICE && ops[0].chunk.n_tokens > 0 && !is_td(ops[0].chunk.codec)) {
        // one device-resident chunk, the call a serving engine makes per request: no lists to build
        const HostOp h = make_host_op(pool, ops[0].block_table, ops[0].n_table_blocks, ops[0].token_offset, ops[0].chunk);
        return launch_batch(ctx, pool, OP, &h, 1, (cudaStream_t)cuda_stream);
    }
    std::vector<HostOp> dev_ops, host_ops;
    for (int i = 0; i < n_ops; ++i) {
        if (ops[i].chunk.n_tokens == 0) continue;
        HostOp h = make_host_op(pool, ops[i].block_table, ops[i].n_table_blocks, ops[i].token_offset, ops[i].chunk);
        (ops[i].chunk.mem == KDN_MEM_PINNED_HOST ? host_ops : dev_ops).push_back(h);
    }
    return run_ops(ctx, pool_id, OP, dev_ops, host_ops, cuda_stream, side_stream);
}

// Keep-list transfers: the chunk holds only the listed tokens (chunk token i <-> token_offset + keep[i]).
kdn_status xfer_sparse(kdn_ctx *ctx, int pool_id, int OP, const kdn_sparse_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    if (!ctx || pool_id < 0 || (size_t)pool_id >= ctx->pools.size()) return KDN_E_INVAL;
    if (n_ops < 0 || (n_ops > 0 && !ops)) return KDN_E_INVAL;
    const Pool &pool = ctx->pools[(size_t)pool_id];
    const kdn_pool_desc shape = shape_of(pool);
    kdn_status st = check_shape(&shape);
    if (st != KDN_OK) return st;
    for (int i = 0; i < n_ops; ++i) {
        const kdn_xfer_op &o = ops[i].op;
        st = check_chunk(&shape, &o.chunk);
        if (st != KDN_OK) return st;
        // (the per-channel key and the token-delta codecs group the chunk's own tokens, listed or not; every row is found
        // through its own table entry, so there is no rule on token_offset or block_size here)
        if (o.n_table_blocks < 0 || o.token_offset < 0) return KDN_E_INVAL;
        if (o.chunk.n_tokens > 0 && (!o.block_table || !ops[i].keep)) return KDN_E_INVAL;
        // the listed tokens are distinct positions below the end of the table, so there cannot be more of them
        if ((int64_t)o.chunk.n_tokens > (int64_t)o.n_table_blocks * pool.bs - o.token_offset) return KDN_E_RANGE;
    }
    if (cudaSetDevice(ctx->device) != cudaSuccess) return KDN_E_CUDA;
    std::vector<HostOp> dev_ops, host_ops;
    for (int i = 0; i < n_ops; ++i) {
        const kdn_xfer_op &o = ops[i].op;
        if (o.chunk.n_tokens == 0) continue;
        HostOp h = make_host_op(pool, o.block_table, o.n_table_blocks, o.token_offset, o.chunk);
        h.op.list = ops[i].keep;
        h.op.n_list = o.chunk.n_tokens;
        h.op.list_mode = 1;
        (o.chunk.mem == KDN_MEM_PINNED_HOST ? host_ops : dev_ops).push_back(h);
    }
    return run_ops(ctx, pool_id, OP, dev_ops, host_ops, cuda_stream, side_stream);
}

}  // namespace

extern "C" {

size_t kdn_chunk_bytes(const kdn_pool_desc *pool, int32_t n_tokens, int32_t codec)
{
    if (!shape_ok(pool) || n_tokens < 0) return 0;
    const size_t elems = (size_t)pool->n_layers * 2u * (size_t)n_tokens * (size_t)pool->n_kv_heads * (size_t)pool->head_dim;
    if (codec == KDN_CODEC_RAW_BF16) return elems * 2u;
    if (codec == KDN_CODEC_INT8_G64) return pool->head_dim % 64 ? 0 : elems + elems / 64u * 4u;
    if (codec == KDN_CODEC_INT4_G64) return pool->head_dim % 64 ? 0 : elems / 2u + elems / 64u * 4u;
    if (is_td(codec)) {
        if (pool->head_dim % 64) return 0;
        return (size_t)td_layout(pool->n_layers, (unsigned)(pool->n_kv_heads * pool->head_dim), n_tokens, codec).capacity;
    }
    if (is_kc(codec)) {
        if (pool->head_dim % 64) return 0;
        const size_t row = (size_t)pool->n_kv_heads * (size_t)pool->head_dim;
        return (codec == KDN_CODEC_INT4_KC64 ? elems / 2u : elems) +
               4u * (size_t)pool->n_layers * scales_per_layer(row, (size_t)n_tokens, codec);
    }
    return 0;
}

kdn_status kdn_td_layout(const kdn_pool_desc *pool, int32_t n_tokens, int32_t codec, kdn_td_layout_info *out)
{
    if (!shape_ok(pool) || n_tokens < 0 || !out) return KDN_E_INVAL;
    if (!is_td(codec) || pool->head_dim % 64) return KDN_E_UNSUPPORTED;
    const TdLayout t = td_layout(pool->n_layers, (unsigned)(pool->n_kv_heads * pool->head_dim), n_tokens, codec);
    out->segments = t.S; out->scales_offset = t.scales; out->lens_offset = t.lens; out->params_offset = t.params;
    out->streams_offset = t.streams; out->capacity = t.capacity;
    return KDN_OK;
}

kdn_status kdn_validate_xfer(const kdn_pool_desc *pool, const kdn_xfer_op *ops, int n_ops)
{
    kdn_status st = check_shape(pool);
    if (st != KDN_OK) return st;
    if (n_ops < 0 || (n_ops > 0 && !ops)) return KDN_E_INVAL;
    for (int i = 0; i < n_ops; ++i) {
        st = check_chunk(pool, &ops[i].chunk);
        if (st != KDN_OK) return st;
        st = check_range(pool, ops[i].block_table, ops[i].n_table_blocks, ops[i].token_offset, ops[i].chunk.n_tokens);
        if (st != KDN_OK) return st;
        st = check_kc(pool, &ops[i].chunk, ops[i].token_offset);
        if (st != KDN_OK) return st;
    }
    return KDN_OK;
}

kdn_status kdn_validate_compose(const kdn_pool_desc *pool, const kdn_compose_req *reqs, int n_reqs)
{
    kdn_status st = check_shape(pool);
    if (st != KDN_OK) return st;
    if (n_reqs < 0 || (n_reqs > 0 && !reqs)) return KDN_E_INVAL;
    for (int r = 0; r < n_reqs; ++r) {
        const kdn_compose_req &q = reqs[r];
        if (q.n_parts < 0 || (q.n_parts > 0 && (!q.parts || !q.part_dst_pos))) return KDN_E_INVAL;
        if (q.rope_style != 0) return KDN_E_UNSUPPORTED;
        bool rotates = false;
        for (int j = 0; j < q.n_parts; ++j) {
            st = check_chunk(pool, &q.parts[j]);
            if (st != KDN_OK) return st;
            st = check_range(pool, q.block_table, q.n_table_blocks, q.part_dst_pos[j], q.parts[j].n_tokens);
            if (st != KDN_OK) return st;
            st = check_kc(pool, &q.parts[j], q.part_dst_pos[j]);
            if (st != KDN_OK) return st;
            rotates |= q.parts[j].n_tokens > 0 && q.part_dst_pos[j] != q.parts[j].base_pos;
        }
        if (rotates) {
            if (!(q.rope_theta > 0.0) || q.rope_theta != q.rope_theta || q.rope_theta > 1e300) return KDN_E_INVAL;
            if (pool->head_dim % 16) return KDN_E_UNSUPPORTED;
        }
        // parts of one request must not overlap
        for (int a = 0; a < q.n_parts; ++a)
            for (int b = a + 1; b < q.n_parts; ++b) {
                const int64_t a0 = q.part_dst_pos[a], a1 = a0 + q.parts[a].n_tokens;
                const int64_t b0 = q.part_dst_pos[b], b1 = b0 + q.parts[b].n_tokens;
                if (a0 < b1 && b0 < a1) return KDN_E_RANGE;
            }
    }
    return KDN_OK;
}

kdn_status kdn_create(kdn_ctx **out, int device)
{
    if (!out) return KDN_E_INVAL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return KDN_E_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return KDN_E_CUDA;
    kdn_ctx *ctx = new (std::nothrow) kdn_ctx();
    if (!ctx) return KDN_E_NOMEM;
    ctx->device = device;
    kdn_status st = KDN_OK;
    auto fail = [&](kdn_status s) { kdn_destroy(ctx); return s; };
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return fail(KDN_E_CUDA);
    if (major < 10) return fail(KDN_E_UNSUPPORTED);       // the kernels are built for sm_100a only
    if (cudaDeviceGetAttribute(&ctx->env.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return fail(KDN_E_CUDA);
    if (cudaDeviceGetAttribute(&ctx->env.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) return fail(KDN_E_CUDA);
    if (cudaMalloc((void **)&ctx->d_status, sizeof(int)) != cudaSuccess) return fail(KDN_E_NOMEM);
    if (cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess) return fail(KDN_E_CUDA);
    if (cudaMallocHost((void **)&ctx->h_status, sizeof(int)) != cudaSuccess) return fail(KDN_E_NOMEM);
    for (int i = 0; i < kRing; ++i) {
        RingSlot &s = ctx->ring[i];
        if (cudaMallocHost((void **)&s.h_ops, sizeof(DevOp) * kMaxOpsPerLaunch) != cudaSuccess) return fail(KDN_E_NOMEM);
        if (cudaMalloc((void **)&s.d_ops, sizeof(DevOp) * kMaxOpsPerLaunch) != cudaSuccess) return fail(KDN_E_NOMEM);
        if (cudaMallocHost((void **)&s.h_rope, sizeof(RopeParam) * kMaxOpsPerLaunch) != cudaSuccess) return fail(KDN_E_NOMEM);
        if (cudaMalloc((void **)&s.d_rope, sizeof(RopeParam) * kMaxOpsPerLaunch) != cudaSuccess) return fail(KDN_E_NOMEM);
        if (cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming) != cudaSuccess) return fail(KDN_E_CUDA);
    }
    *out = ctx;
    return st;
}

void kdn_destroy(kdn_ctx *ctx)
{
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    for (int i = 0; i < kRing; ++i) {
        RingSlot &s = ctx->ring[i];
        if (s.h_ops) cudaFreeHost(s.h_ops);
        if (s.d_ops) cudaFree(s.d_ops);
        if (s.h_rope) cudaFreeHost(s.h_rope);
        if (s.d_rope) cudaFree(s.d_rope);
        if (s.d_table) cudaFree(s.d_table);
        if (s.done) cudaEventDestroy(s.done);
    }
    for (Pool &p : ctx->pools) {
        if (p.d_k) cudaFree(p.d_k);
        if (p.d_v) cudaFree(p.d_v);
    }
    for (int i = 0; i < 2; ++i) {
        if (ctx->slab[i]) cudaFree(ctx->slab[i]);
        if (ctx->slab_free[i]) cudaEventDestroy(ctx->slab_free[i]);
        if (ctx->slab_ready[i]) cudaEventDestroy(ctx->slab_ready[i]);
    }
    for (int i = 0; i < 2; ++i) {
        if (ctx->bounce[i]) cudaFreeHost(ctx->bounce[i]);
        if (ctx->bounce_done[i]) cudaEventDestroy(ctx->bounce_done[i]);
    }
    if (ctx->fork) cudaEventDestroy(ctx->fork);
    if (ctx->own_side) cudaStreamDestroy(ctx->own_side);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    delete ctx;
}

kdn_status kdn_pool_register(kdn_ctx *ctx, const kdn_pool_desc *pool, int *pool_id)
{
    if (!ctx || !pool_id) return KDN_E_INVAL;
    kdn_status st = check_shape(pool);
    if (st != KDN_OK) return st;
    if (!pool->k_layers || !pool->v_layers) return KDN_E_INVAL;
    for (int l = 0; l < pool->n_layers; ++l) {
        if (!pool->k_layers[l] || !pool->v_layers[l]) return KDN_E_INVAL;
        if ((uintptr_t)pool->k_layers[l] % 16 || (uintptr_t)pool->v_layers[l] % 16) return KDN_E_ALIGN;
    }
    if (cudaSetDevice(ctx->device) != cudaSuccess) return KDN_E_CUDA;
    Pool p;
    p.L = pool->n_layers; p.H = pool->n_kv_heads; p.D = pool->head_dim; p.bs = pool->block_size; p.nb = pool->n_blocks;
    const size_t bytes = sizeof(void *) * (size_t)p.L;
    KDN_CUDA(cudaMalloc((void **)&p.d_k, bytes));
    if (cudaMalloc((void **)&p.d_v, bytes) != cudaSuccess) { cudaFree(p.d_k); return KDN_E_NOMEM; }
    if (cudaMemcpy(p.d_k, pool->k_layers, bytes, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(p.d_v, pool->v_layers, bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaFree(p.d_k); cudaFree(p.d_v);
        return KDN_E_CUDA;
    }
    ctx->pools.push_back(p);
    *pool_id = (int)ctx->pools.size() - 1;
    return KDN_OK;
}

kdn_status kdn_store(kdn_ctx *ctx, int pool_id, const kdn_xfer_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    return xfer(ctx, pool_id, OP_STORE, ops, n_ops, cuda_stream, side_stream);
}

kdn_status kdn_retrieve(kdn_ctx *ctx, int pool_id, const kdn_xfer_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    return xfer(ctx, pool_id, OP_RETRIEVE, ops, n_ops, cuda_stream, side_stream);
}

static kdn_status xfer_file(kdn_ctx *ctx, int pool_id, int OP, const kdn_file_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    if (!ctx || pool_id < 0 || (size_t)pool_id >= ctx->pools.size()) return KDN_E_INVAL;
    if (n_ops < 0 || (n_ops > 0 && !ops)) return KDN_E_INVAL;
    const Pool &pool = ctx->pools[(size_t)pool_id];
    const kdn_pool_desc shape = shape_of(pool);
    kdn_status st = check_shape(&shape);
    if (st != KDN_OK) return st;
    for (int i = 0; i < n_ops; ++i) {
        const kdn_xfer_op &o = ops[i].op;
        kdn_chunk c = o.chunk;
        c.data = (void *)(uintptr_t)16;                      // a file-backed chunk has no address to check
        c.mem = KDN_MEM_PINNED_HOST;
        st = check_chunk(&shape, &c);
        if (st != KDN_OK) return st;
        st = check_range(&shape, o.block_table, o.n_table_blocks, o.token_offset, o.chunk.n_tokens);
        if (st != KDN_OK) return st;
        st = check_kc(&shape, &o.chunk, o.token_offset);
        if (st != KDN_OK) return st;
        // (a token-delta chunk in a file: its offset table first, then the bytes it uses; storing one is refused below,
        // as for host memory: the size of the result is not known before the kernels have run)
        if (ops[i].fd < 0 || ops[i].file_offset < 0) return KDN_E_INVAL;
    }
    if (cudaSetDevice(ctx->device) != cudaSuccess) return KDN_E_CUDA;
    std::vector<HostOp> dev_ops, host_ops;
    for (int i = 0; i < n_ops; ++i) {
        const kdn_xfer_op &o = ops[i].op;
        if (o.chunk.n_tokens == 0) continue;
        kdn_chunk c = o.chunk;
        c.data = nullptr;
        HostOp h = make_host_op(pool, o.block_table, o.n_table_blocks, o.token_offset, c);
        h.fd = ops[i].fd;
        h.file_off = ops[i].file_offset;
        host_ops.push_back(h);
    }
    return run_ops(ctx, pool_id, OP, dev_ops, host_ops, cuda_stream, side_stream);
}

kdn_status kdn_store_file(kdn_ctx *ctx, int pool_id, const kdn_file_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    return xfer_file(ctx, pool_id, OP_STORE, ops, n_ops, cuda_stream, side_stream);
}

kdn_status kdn_retrieve_file(kdn_ctx *ctx, int pool_id, const kdn_file_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    return xfer_file(ctx, pool_id, OP_RETRIEVE, ops, n_ops, cuda_stream, side_stream);
}

kdn_status kdn_retrieve_layerwise(kdn_ctx *ctx, int pool_id, const kdn_xfer_op *ops, int n_ops, int layers_per_step,
                                  void *cuda_stream, void *side_stream, void *const *layer_ready)
{
    if (!ctx || pool_id < 0 || (size_t)pool_id >= ctx->pools.size() || layers_per_step < 1) return KDN_E_INVAL;
    const Pool &pool = ctx->pools[(size_t)pool_id];
    const kdn_pool_desc shape = shape_of(pool);
    kdn_status st = kdn_validate_xfer(&shape, ops, n_ops);
    if (st != KDN_OK) return st;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return KDN_E_CUDA;
    std::vector<HostOp> dev_all, host_all;
    for (int i = 0; i < n_ops; ++i) {
        if (ops[i].chunk.n_tokens == 0) continue;
        HostOp h = make_host_op(pool, ops[i].block_table, ops[i].n_table_blocks, ops[i].token_offset, ops[i].chunk);
        (ops[i].chunk.mem == KDN_MEM_PINNED_HOST ? host_all : dev_all).push_back(h);
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    for (int l0 = 0; l0 < pool.L; l0 += layers_per_step) {
        const int nl = pool.L - l0 < layers_per_step ? pool.L - l0 : layers_per_step;
        std::vector<HostOp> dev_ops, host_ops;
        for (const HostOp &h : dev_all) dev_ops.push_back(layer_range(pool, h, l0, nl));
        // a host-resident chunk keeps its full-chunk addresses; run_staged cuts out the layer range itself
        for (const HostOp &h : host_all) { HostOp sub = h; sub.op.l0 = l0; sub.op.nl = nl; host_ops.push_back(sub); }
        st = run_ops(ctx, pool_id, OP_RETRIEVE, dev_ops, host_ops, cuda_stream, side_stream);
        if (st != KDN_OK) return st;
        if (layer_ready)
            for (int l = l0; l < l0 + nl; ++l)
                if (layer_ready[l]) KDN_CUDA(cudaEventRecord((cudaEvent_t)layer_ready[l], stream));
    }
    return KDN_OK;
}

static kdn_status compose_impl(kdn_ctx *ctx, int pool_id, const kdn_compose_req *reqs, const kdn_select *selects, int n_reqs,
                               void *cuda_stream, void *side_stream);

kdn_status kdn_compose(kdn_ctx *ctx, int pool_id, const kdn_compose_req *reqs, int n_reqs, void *cuda_stream, void *side_stream)
{
    return compose_impl(ctx, pool_id, reqs, nullptr, n_reqs, cuda_stream, side_stream);
}

kdn_status kdn_compose_select(kdn_ctx *ctx, int pool_id, const kdn_compose_req *reqs, const kdn_select *selects, int n_reqs,
                              void *cuda_stream, void *side_stream)
{
    if (n_reqs > 0 && !selects) return KDN_E_INVAL;
    return compose_impl(ctx, pool_id, reqs, selects, n_reqs, cuda_stream, side_stream);
}

kdn_status kdn_store_sparse(kdn_ctx *ctx, int pool_id, const kdn_sparse_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    return xfer_sparse(ctx, pool_id, OP_STORE, ops, n_ops, cuda_stream, side_stream);
}

kdn_status kdn_retrieve_sparse(kdn_ctx *ctx, int pool_id, const kdn_sparse_op *ops, int n_ops, void *cuda_stream, void *side_stream)
{
    return xfer_sparse(ctx, pool_id, OP_RETRIEVE, ops, n_ops, cuda_stream, side_stream);
}

static kdn_status compose_impl(kdn_ctx *ctx, int pool_id, const kdn_compose_req *reqs, const kdn_select *selects, int n_reqs,
                               void *cuda_stream, void *side_stream)
{
    if (!ctx || pool_id < 0 || (size_t)pool_id >= ctx->pools.size()) return KDN_E_INVAL;
    const Pool &pool = ctx->pools[(size_t)pool_id];
    const kdn_pool_desc shape = shape_of(pool);
    kdn_status st = kdn_validate_compose(&shape, reqs, n_reqs);
    if (st != KDN_OK) return st;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return KDN_E_CUDA;
    std::vector<HostOp> dev_ops, host_ops;
    for (int r = 0; r < n_reqs; ++r) {
        const kdn_compose_req &q = reqs[r];
        for (int j = 0; j < q.n_parts; ++j) {
            const kdn_chunk &c = q.parts[j];
            if (c.n_tokens == 0) continue;
            HostOp h = make_host_op(pool, q.block_table, q.n_table_blocks, q.part_dst_pos[j], c);
            const long long delta = (long long)(q.part_dst_pos[j] - c.base_pos);
            if (delta != 0) {
                h.rotate = true;
                h.rp.delta = delta;
                h.rp.theta = q.rope_theta;
            }
            if (selects && selects[r].part_select && selects[r].part_select[j]) {
                if (!selects[r].part_n_select || selects[r].part_n_select[j] < 0 || selects[r].part_n_select[j] > c.n_tokens)
                    return KDN_E_INVAL;
                if (selects[r].part_n_select[j] == 0) continue;          // nothing of this part is delivered
                h.op.list = selects[r].part_select[j];
                h.op.n_list = selects[r].part_n_select[j];
                h.op.list_mode = 2;
            }
            (c.mem == KDN_MEM_PINNED_HOST ? host_ops : dev_ops).push_back(h);
        }
    }
    return run_ops(ctx, pool_id, OP_COMPOSE, dev_ops, host_ops, cuda_stream, side_stream);
}

kdn_status kdn_status_sync(kdn_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return KDN_E_INVAL;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return KDN_E_CUDA;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    KDN_CUDA(cudaStreamSynchronize(stream));
    if (ctx->own_side) KDN_CUDA(cudaStreamSynchronize(ctx->own_side));
    KDN_CUDA(cudaStreamSynchronize(stream));              // work the side stream released onto `stream`
    KDN_CUDA(cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream));
    KDN_CUDA(cudaMemsetAsync(ctx->d_status, 0, sizeof(int), stream));
    KDN_CUDA(cudaStreamSynchronize(stream));
    const int s = *ctx->h_status;
    return (s >= KDN_OK && s <= KDN_E_TIMEOUT) ? (kdn_status)s : KDN_E_CUDA;
}

kdn_status kdn_set_tuning(kdn_ctx *ctx, const kdn_tuning *tuning)
{
    if (!ctx) return KDN_E_INVAL;
    if (!tuning) { ctx->tuning = kdn_tuning{}; return KDN_OK; }
    if (tuning->tile_bytes < 0 || tuning->stages < 0 || tuning->ctas_per_sm < 0) return KDN_E_INVAL;
    if (tuning->tile_bytes % 128) return KDN_E_INVAL;
    if (tuning->stages > kMaxStages) return KDN_E_UNSUPPORTED;
    if (tuning->store_lag < 0) return KDN_E_INVAL;
    if (tuning->store_lag > kMaxStoreLag) return KDN_E_UNSUPPORTED;
    if (tuning->ctas_per_sm > 32) return KDN_E_UNSUPPORTED;
    if (tuning->compute_groups < 0) return KDN_E_INVAL;
    if (tuning->compute_groups > kMaxGroups) return KDN_E_UNSUPPORTED;
    if (tuning->group_warps != 0 && tuning->group_warps != 1 && tuning->group_warps != 4) return KDN_E_UNSUPPORTED;
    if (tuning->tile_bytes > ctx->env.smem_optin) return KDN_E_UNSUPPORTED;
    ctx->tuning = *tuning;
    return KDN_OK;
}

kdn_status kdn_set_staging_bytes(kdn_ctx *ctx, size_t bytes_per_slab)
{
    if (!ctx || bytes_per_slab < 4096) return KDN_E_INVAL;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return KDN_E_CUDA;
    KDN_CUDA(cudaDeviceSynchronize());
    for (int i = 0; i < 2; ++i) {
        if (ctx->slab[i]) KDN_CUDA(cudaFree(ctx->slab[i]));
        ctx->slab[i] = nullptr;
        if (ctx->bounce[i]) KDN_CUDA(cudaFreeHost(ctx->bounce[i]));
        ctx->bounce[i] = nullptr;
        ctx->bounce_busy[i] = false;
    }
    ctx->slab_bytes = bytes_per_slab & ~(size_t)255;
    return KDN_OK;
}

kdn_status kdn_set_wait_limit_ns(kdn_ctx *ctx, uint64_t ns)
{
    if (!ctx) return KDN_E_INVAL;
    ctx->wait_limit_ns = ns ? (unsigned long long)ns : kWaitLimitNs;
    return KDN_OK;
}

uint64_t kdn_launch_count(const kdn_ctx *ctx) { return ctx ? ctx->launches : 0; }

kdn_status kdn_last_launch(const kdn_ctx *ctx, kdn_launch_info *out)
{
    if (!ctx || !out) return KDN_E_INVAL;
    *out = ctx->last;
    return KDN_OK;
}

const char *kdn_strerror(kdn_status status)
{
    switch (status) {
    case KDN_OK: return "ok";
    case KDN_E_INVAL: return "invalid argument";
    case KDN_E_SHAPE: return "chunk size does not match the pool shape";
    case KDN_E_ALIGN: return "pointer or row size not 16-byte aligned";
    case KDN_E_RANGE: return "token range or block id out of range";
    case KDN_E_UNSUPPORTED: return "unsupported shape, codec or setting";
    case KDN_E_CUDA: return "CUDA runtime error";
    case KDN_E_NOMEM: return "out of memory";
    case KDN_E_TIMEOUT: return "a bounded wait inside a kernel expired";
    case KDN_E_NOTFOUND: return "no chunk under this key";
    case KDN_E_CHECKSUM: return "payload does not match the header's checksum";
    case KDN_E_IO: return "reading or writing a chunk file failed";
    }
    return "unknown status";
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// kdn_compose_static: compose without any device allocation (no paper counterpart; see kdn.h).
// Its scratch is this fixed array in the library's device image.  Layout (byte offsets):
//   0      int status                      (256 bytes reserved)
//   256    void *k_layers[128]
//   1280   void *v_layers[128]
//   2304   DevOp ops[128]
//   14592  RopeParam rope[128]
//   16640  float2 table[128 * 256]         (rows x head_dim/2, packed by the call's head_dim)
// In host code `g_static_scratch` is only a handle for cudaGetSymbolAddress, never an address to
// hand to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[KDN_STATIC_SCRATCH_BYTES];

namespace {

constexpr size_t kStOffK = 256, kStOffV = 1280, kStOffOps = 2304, kStOffRope = 14592, kStOffTable = 16640;
constexpr size_t kStHeadBytes = kStOffTable;                 // everything the host uploads per call
constexpr int kStMaxDevices = 64;
static_assert(kStOffTable + sizeof(float2) * KDN_STATIC_MAX_PARTS * (KDN_STATIC_MAX_HEAD_DIM / 2) == KDN_STATIC_SCRATCH_BYTES,
              "scratch layout and KDN_STATIC_SCRATCH_BYTES disagree");
static_assert(kStOffRope - kStOffOps == sizeof(DevOp) * KDN_STATIC_MAX_PARTS, "ops area");
static_assert(kStOffTable - kStOffRope == sizeof(RopeParam) * KDN_STATIC_MAX_PARTS, "rope area");

struct StaticDev {
    unsigned char *base = nullptr;          // device address of g_static_scratch on this device
    LaunchEnv env;
};
StaticDev g_static_dev[kStMaxDevices];
std::mutex g_static_mutex;

// One-time set-up per device, with that device current: resolve the array's device address.
kdn_status static_setup(int device, StaticDev **out)
{
    if (device < 0 || device >= kStMaxDevices) return KDN_E_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDev &d = g_static_dev[device];
    if (!d.base) {
        int major = 0;
        KDN_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
        if (major < 10) return KDN_E_UNSUPPORTED;
        KDN_CUDA(cudaDeviceGetAttribute(&d.env.sm_count, cudaDevAttrMultiProcessorCount, device));
        KDN_CUDA(cudaDeviceGetAttribute(&d.env.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device));
        void *ptr = nullptr;
        KDN_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return KDN_E_CUDA;
        // Load every kernel a later call can launch and raise its shared-memory limit now, so that no later call
        // meets a first-use step of the runtime: the three compose forms the built-in shapes use (pure copy, decoding
        // without rotation, rotation) and the rotation-table kernel.
        int per_sm = 0;
        kdn_status st = d.env.resident(kdn_compose_kernel<0, 4>, threads_for(0, 4), 1024, &per_sm);
        if (st == KDN_OK) st = d.env.resident(kdn_compose_kernel<1, 4>, threads_for(1, 4), 1024, &per_sm);
        if (st == KDN_OK) st = d.env.resident(kdn_compose_kernel<2, 4>, threads_for(2, 4), 1024, &per_sm);
        if (st != KDN_OK) return st;
        cudaFuncAttributes fa{};
        KDN_CUDA(cudaFuncGetAttributes(&fa, kdn_rope_table_kernel));
        d.base = (unsigned char *)ptr;
    }
    *out = &d;
    return KDN_OK;
}

}  // namespace

extern "C" kdn_status kdn_compose_static(int device, const kdn_pool_desc *pool, const kdn_compose_req *reqs, int n_reqs,
                                         void *cuda_stream, int wait)
{
    kdn_status st = kdn_validate_compose(pool, reqs, n_reqs);
    if (st != KDN_OK) return st;
    if (!pool->k_layers || !pool->v_layers) return KDN_E_INVAL;
    if (pool->n_layers > KDN_STATIC_MAX_LAYERS || pool->head_dim > KDN_STATIC_MAX_HEAD_DIM) return KDN_E_UNSUPPORTED;
    long long n_parts = 0;
    for (int r = 0; r < n_reqs; ++r) {
        for (int j = 0; j < reqs[r].n_parts; ++j) {
            if (reqs[r].parts[j].n_tokens == 0) continue;
            if (reqs[r].parts[j].mem != KDN_MEM_DEVICE) return KDN_E_UNSUPPORTED;
            if (is_kc(reqs[r].parts[j].codec) || is_td(reqs[r].parts[j].codec)) return KDN_E_UNSUPPORTED;
            ++n_parts;
        }
        if (n_parts > KDN_STATIC_MAX_PARTS) return KDN_E_UNSUPPORTED;
    }
    for (int l = 0; l < pool->n_layers; ++l) {
        if (!pool->k_layers[l] || !pool->v_layers[l]) return KDN_E_INVAL;
        if ((uintptr_t)pool->k_layers[l] % 16 || (uintptr_t)pool->v_layers[l] % 16) return KDN_E_ALIGN;
    }
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return KDN_E_CUDA;
    KDN_CUDA(cudaSetDevice(device));
    StaticDev *sd = nullptr;
    st = static_setup(device, &sd);
    if (st != KDN_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    Pool p;
    p.L = pool->n_layers; p.H = pool->n_kv_heads; p.D = pool->head_dim; p.bs = pool->block_size; p.nb = pool->n_blocks;
    const unsigned row_elems = (unsigned)p.H * (unsigned)p.D;

    // host image of the scratch head: status word (zero), layer pointers, part records, rotation rows
    alignas(16) unsigned char head[kStHeadBytes];
    std::memset(head, 0, sizeof head);
    std::memcpy(head + kStOffK, pool->k_layers, sizeof(void *) * (size_t)p.L);
    std::memcpy(head + kStOffV, pool->v_layers, sizeof(void *) * (size_t)p.L);
    DevOp *ops = reinterpret_cast<DevOp *>(head + kStOffOps);
    RopeParam *rope = reinterpret_cast<RopeParam *>(head + kStOffRope);

    // launch shape: the library defaults for a compose launch
    bool any_coded = false, any_rot = false;
    for (int r = 0; r < n_reqs; ++r)
        for (int j = 0; j < reqs[r].n_parts; ++j) {
            if (reqs[r].parts[j].n_tokens == 0) continue;
            any_coded |= reqs[r].parts[j].codec != KDN_CODEC_RAW_BF16;
            any_rot |= reqs[r].part_dst_pos[j] != reqs[r].parts[j].base_pos;
        }
    const bool compute = any_coded || any_rot;
    unsigned unit = 8;
    if (any_coded) unit = lcm_u(unit, 64);
    if (any_rot) unit = lcm_u(unit, (unsigned)p.D);
    const Shape def = default_shape(OP_COMPOSE, any_coded, any_rot);
    unsigned tile_elems = (unsigned)def.tile_bytes / 2u / unit * unit;
    if (tile_elems < unit) tile_elems = unit;
    const unsigned long long block_elems = (unsigned long long)p.bs * row_elems;
    if (tile_elems > block_elems) tile_elems = (unsigned)((block_elems + unit - 1) / unit * unit);
    const unsigned tpb = (unsigned)((block_elems + tile_elems - 1) / tile_elems);
    const unsigned a_bytes = (tile_elems * 2u + 127u) & ~127u;
    const unsigned b_bytes = compute ? ((tile_elems + 127u) & ~127u) : 0u;
    const unsigned s_bytes = compute ? ((tile_elems / 16u + 127u) & ~127u) : 0u;
    const unsigned stage_bytes = a_bytes + b_bytes + s_bytes;
    const int ctas_per_sm = def.ctas_per_sm;
    int stages = def.stages;
    const size_t smem_limit = (size_t)sd->env.smem_optin;
    st = fit_stages(stages, def.groups, def.lag, true, stage_bytes, ctas_per_sm, smem_limit);
    if (st != KDN_OK) return st;
    const size_t smem = smem_bytes(stages, stage_bytes);

    unsigned long long tiles = 0;
    int n = 0, n_rope = 0;
    for (int r = 0; r < n_reqs; ++r) {
        const kdn_compose_req &q = reqs[r];
        for (int j = 0; j < q.n_parts; ++j) {
            const kdn_chunk &c = q.parts[j];
            if (c.n_tokens == 0) continue;
            HostOp h = make_host_op(p, q.block_table, q.n_table_blocks, q.part_dst_pos[j], c);
            DevOp op = h.op;
            op.tile_begin = (unsigned)tiles;
            const long long delta = (long long)(q.part_dst_pos[j] - c.base_pos);
            if (delta != 0) {
                rope[n_rope].delta = delta;
                rope[n_rope].theta = q.rope_theta;
                op.rope = n_rope++;
            }
            ops[n++] = op;
            tiles += (unsigned long long)op.nl * 2ull * (unsigned long long)op.nblk * tpb;
            if (tiles > kMaxTilesPerLaunch) return KDN_E_UNSUPPORTED;
        }
    }
    const int half = p.D / 2;
    if ((size_t)n_rope * (size_t)half > (size_t)KDN_STATIC_MAX_PARTS * (KDN_STATIC_MAX_HEAD_DIM / 2)) return KDN_E_UNSUPPORTED;

    // upload the head (this also clears the status word); the source is ordinary host memory, so the
    // runtime has taken its copy of `head` by the time the call returns
    KDN_CUDA(cudaMemcpyAsync(sd->base, head, kStHeadBytes, cudaMemcpyHostToDevice, stream));
    if (tiles != 0) {
        float2 *d_table = reinterpret_cast<float2 *>(sd->base + kStOffTable);
        if (n_rope) {
            const long long total = (long long)n_rope * half;
            kdn_rope_table_kernel<<<(unsigned)((total + 127) / 128), 128, 0, stream>>>(
                reinterpret_cast<const RopeParam *>(sd->base + kStOffRope), RopeInline{}, n_rope, p.D, d_table);
            KDN_CUDA(cudaGetLastError());
        }
        Launch lp{};
        lp.ops = reinterpret_cast<const DevOp *>(sd->base + kStOffOps);
        lp.n_ops = n;
        lp.n_tiles = (unsigned)tiles;
        lp.k_layers = reinterpret_cast<void *const *>(sd->base + kStOffK);
        lp.v_layers = reinterpret_cast<void *const *>(sd->base + kStOffV);
        lp.n_blocks = p.nb;
        lp.bs = p.bs;
        lp.D = p.D;
        lp.row_elems = row_elems;
        lp.tile_elems = tile_elems;
        lp.tpb = tpb;
        lp.rope = d_table;
        lp.status = reinterpret_cast<int *>(sd->base);
        lp.stages = stages;
        lp.stage_bytes = stage_bytes;
        lp.off_b = a_bytes;
        lp.off_s = a_bytes + b_bytes;
        lp.store_lag = def.lag;
        const unsigned long long want = (unsigned long long)sd->env.sm_count * (unsigned)ctas_per_sm;
        const unsigned grid = (unsigned)(tiles < want ? tiles : want);
        lp.wait_limit_ns = kWaitLimitNs;
        lp.one = 1.0f;
        lp.rows_per_tile = 1;
        lp.wait_all = 0;
        {
            std::lock_guard<std::mutex> lock(g_static_mutex);     // the per-device occupancy cache is shared by all callers
            st = launch_tiles(sd->env, OP_COMPOSE, def.groups, def.gw, grid, smem, stream, lp);
        }
        if (st != KDN_OK) return st;
    }
    if (!wait) return KDN_OK;
    // the status word comes back on the caller's stream: no other stream of the process is involved
    int dev_status = 0;
    KDN_CUDA(cudaMemcpyAsync(&dev_status, sd->base, sizeof(int), cudaMemcpyDeviceToHost, stream));
    KDN_CUDA(cudaStreamSynchronize(stream));
    return (dev_status >= KDN_OK && dev_status <= KDN_E_TIMEOUT) ? (kdn_status)dev_status : KDN_E_CUDA;
}
