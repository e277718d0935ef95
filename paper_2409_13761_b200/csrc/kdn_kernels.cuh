// Device side of libkdn: one persistent, warp-specialised tile pipeline for sm_100a, instantiated
// as the three kernels of the path (paper Sec. 3.1: storage -> kdn_store_kernel, delivery with
// decompression on the GPU -> kdn_retrieve_kernel, blending -> kdn_compose_kernel).
//
// Work decomposition.  A chunk of T tokens and a paged pool meet in runs: for one (layer, K|V)
// plane and one logical block of the request, the tokens of that block that belong to the chunk
// are contiguous both in the pool block and in the chunk plane.  A run is cut into tiles of at most
// tile_elems elements; tile g of the launch is handled by CTA g % gridDim.x.  Nothing in a tile
// depends on another tile, so there is no inter-CTA synchronisation.  Ops with a token list (keep-list,
// select-list) are cut into one tile per listed token row instead.
//
// Pipeline inside a CTA (S slots of shared memory, all hand-offs through mbarriers):
//   loader warp   decodes tiles 32 at a time (one per lane: op lookup, block-table entry, addresses),
//                 then issues each tile's bulk async copies global -> shared
//   compute warps (G groups of 4 warps, or of 1 warp for row-sized tiles; group g owns slots g, g+G, ...) int8 coding / decoding and key
//                 rotation, shared -> shared
//   storer thread issues the bulk async copy shared -> global and recycles the slot
// Tiles that are a pure copy (raw bf16 without rotation) never touch the compute warps' ALUs.
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA records KDN_E_TIMEOUT,
// drains its own copies with bounded waits and returns.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace kdn {

constexpr int kLoaderWarp = 0;
constexpr int kMaxGroups = 8;                 // compute groups per CTA; group g owns slots g, g + G, ...
// A compute group is kGW warps (4 for ordinary tiles, 1 for row-sized tiles) that work together on one tile.
__host__ __device__ constexpr int threads_for(int groups, int group_warps) { return 32 + groups * group_warps * 32 + 32; }  // loader + compute + storer
// The launch shapes count on several CTAs per SM (eight of the two-single-warp-group form, three of the two-group
// form, ...): every instantiation is held to about 64 registers a thread.
__host__ __device__ constexpr int min_ctas_for(int groups, int group_warps)
{
    return 1024 / threads_for(groups, group_warps) > 0 ? 1024 / threads_for(groups, group_warps) : 1;
}
// The rotation needs more registers (eight frequencies of coefficients per thread) and its shapes fewer CTAs: four of
// the one-group form, two of the two-group form.
__host__ __device__ constexpr int min_ctas_for_compose(int groups, int group_warps)
{
    return group_warps != 4 ? min_ctas_for(groups, group_warps) : groups == 0 ? 8 : groups == 1 ? 4 : groups == 2 ? 2 : 1;
}
constexpr int kThreadsCopy = 64;                             // loader + storer
constexpr int kMaxStages = 32;
constexpr int kMaxStoreLag = 16;          // most bulk-store groups allowed to be still reading shared memory
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // default limit of a pipeline wait, and the limit of every drain wait

enum : uint32_t { TF_CODED = 1u, TF_ROTATE = 2u, TF_SCALES_PLAIN = 4u, TF_INT4 = 8u,   // TF_CODED: int8 or int4
                  TF_KCHAN = 16u,     // key tile of a per-channel key codec: one scale per channel, row_elems of them
                  TF_ROWS = 32u };    // several listed token rows: contiguous in the chunk, rows[] says where each sits in the pool
constexpr int kMaxRowsPerTile = 4;         // several-row tiles of the ordinary kernels
constexpr int kWideRowsPerTile = 16;       // ... of the kernels built for short rows (kWide)
constexpr unsigned kRowsAheadStride = 20;  // kWide: words per lane in the decoded-ahead row area (128-bit stores by 32 lanes at
                                           // this stride spread over all banks)
enum : int { OP_STORE = 0, OP_RETRIEVE = 1, OP_COMPOSE = 2 };

// Status values mirrored from kdn.h (kept numeric here so device code has no host header).
constexpr int kStatusRange = 4;
constexpr int kStatusTimeout = 8;

struct __align__(16) DevOp {
    const int32_t *table;     // device block table of the request
    unsigned char *data;      // layers [l0, l0 + nl) of the chunk: raw bf16, or int8 codes
    long long off;            // request position of chunk token 0
    int T;                    // tokens
    int codec;                // 0 raw bf16, 1 int8 group-64, 2 int4 group-64, 3 / 4 int8 / int4 with per-channel key groups
    int j0;                   // first logical block touched: off / block_size
    int nblk;                 // logical blocks touched
    unsigned tile_begin;      // index of this op's first tile in the launch
    int rope;                 // row of the rotation table, -1: keys are copied
    int l0;                   // first pool layer
    int nl;                   // layers held in data
    unsigned char *scales;    // int8 / int4: fp32 scales of the same layers; raw: unused
    const int32_t *list;      // device token list (list_mode != 0): relative request positions, increasing
    int n_list;               // listed tokens
    int list_mode;            // 0: every token; 1 keep-list: chunk token i <-> off + list[i];
                              // 2 select-list: chunk token list[i] <-> off + list[i]; 3 (kWide kernels only): keep-list
                              // 0, 1, 2, ... with no list in memory: a dense op whose tiles take whole token rows
    long long pos_end;        // request positions >= pos_end are outside the block table
    int kv_sel;               // 0: key and value planes; 2: value planes only (the keys of a per-channel key codec are
                              // stored by kdn_store_kc_kernel)
    int reserved;
};
static_assert(sizeof(DevOp) == 96, "DevOp is copied as 96-byte records");

struct RopeParam {            // one row of the rotation table to fill
    long long delta;          // dst_pos - base_pos
    double theta;
};

constexpr int kInlineOps = 32;            // launches of up to this many ops carry them as kernel parameters (3 KiB)

struct Launch {
    const DevOp *ops;         // device array of n_ops records, or nullptr: the records are in inline_ops
    int n_ops;
    unsigned n_tiles;
    void *const *k_layers;    // device arrays of per-layer pool pointers
    void *const *v_layers;
    long long n_blocks;
    int bs;
    int D;
    unsigned row_elems;       // H * D
    unsigned tile_elems;
    unsigned tpb;             // tiles per logical block
    const float2 *rope;       // [rows][D/2] (cos, sin)
    int *status;
    int stages;
    unsigned stage_bytes;
    unsigned off_b;           // offset of the code buffer inside a stage (compute launches)
    unsigned off_s;           // offset of the scale buffer inside a stage
    int store_lag;            // bulk-store groups that may still be reading shared memory (1..kMaxStoreLag)
    int reload_first;         // copy form: after recycling a slot the storer lets the loader queue the reload
                              // before it queues the next store (see the storer loop)
    unsigned long long wait_limit_ns;   // a pipeline wait gives up after this long (the drain waits keep kWaitLimitNs)
    int rows_per_tile;        // keep-list ops: listed token rows per tile (1: one row per tile)
    int wait_all;             // the launch may start while the kernel before it in the stream still runs (programmatic
                              // dependent launch): every thread waits for that kernel before it touches global memory.
                              // 0: only the warps that read the rotation table wait (the kernel before is the table kernel)
    float one;                // 1.0f, as a launch parameter: the coding loops form "product + constant" as
                              // fma(product, one, constant), and with a multiplier the assembler cannot see there
                              // is nothing it could contract with the multiply before it (the codecs round twice)
    DevOp inline_ops[kInlineOps];
};

struct __align__(16) TileDesc {
    unsigned long long g_pool;    // bf16 address in the pool
    unsigned long long g_chunk;   // chunk side: bf16 (raw) or codes (int8)
    unsigned long long g_scales;  // chunk side: scales (int8)
    unsigned n;                   // elements; 0: nothing to do
    unsigned flags;
    int rope;
    unsigned sbytes;              // bytes of scales that belong to the tile (coded tiles)
    unsigned runs;                // TF_ROWS: nibble r = how many rows the copy that starts at row r covers (0: row r rides
                                  // along with an earlier one); rows that are neighbours in the pool share one copy.  The
                                  // rows' places in the pool plane travel beside the descriptor in shared memory.
                                  // kWide kernels: bit r (r < 16) = a copy starts at row r and runs up to the next set bit;
                                  // bits 16..20 = rows in the tile.
};
static_assert(sizeof(TileDesc) == 48, "TileDesc is copied with 128-bit accesses");

// ------------------------------------------------------------------ PTX --

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// The same test, but the hardware may park the thread for up to `hint_ns` before answering "not yet" (it answers
// at once when the phase completes), so a waiting warp does not eat issue slots that working warps need.
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t bar, uint32_t parity, uint32_t hint_ns)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
// Bounded wait: true when the phase completed; false when the CTA is aborting or the limit passed.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                            unsigned long long limit_ns = kWaitLimitNs)
{
    const unsigned long long t0 = global_timer_ns();
    const uint32_t hint = limit_ns < 20000ull ? (uint32_t)limit_ns : 20000u;   // never park for longer than the limit
    for (;;) {
        if (mbar_try_wait_parked(bar, parity, hint)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, limit_ns);
}
// Bulk async copy global -> this CTA's shared memory, completion counted on an mbarrier.
// (No cluster is launched: the CTA's own shared window is the cluster window.)
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void *dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_read_n(int n)      // the instruction takes an immediate
{
    switch (n) {
    case 1: bulk_wait_read<1>(); break;
    case 2: bulk_wait_read<2>(); break;
    case 3: bulk_wait_read<3>(); break;
    case 4: bulk_wait_read<4>(); break;
    case 5: bulk_wait_read<5>(); break;
    case 6: bulk_wait_read<6>(); break;
    case 7: bulk_wait_read<7>(); break;
    case 8: bulk_wait_read<8>(); break;
    case 9: bulk_wait_read<9>(); break;
    case 10: bulk_wait_read<10>(); break;
    case 11: bulk_wait_read<11>(); break;
    case 12: bulk_wait_read<12>(); break;
    case 13: bulk_wait_read<13>(); break;
    case 14: bulk_wait_read<14>(); break;
    case 15: bulk_wait_read<15>(); break;
    default: bulk_wait_read<16>(); break;
    }
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void group_bar_sync(int group, unsigned gthreads)
{
    switch (group) {                                       // immediate ids: only kMaxGroups barriers are reserved
    case 0: asm volatile("bar.sync 1, %0;" ::"r"(gthreads) : "memory"); break;
    case 1: asm volatile("bar.sync 2, %0;" ::"r"(gthreads) : "memory"); break;
    case 2: asm volatile("bar.sync 3, %0;" ::"r"(gthreads) : "memory"); break;
    case 3: asm volatile("bar.sync 4, %0;" ::"r"(gthreads) : "memory"); break;
    case 4: asm volatile("bar.sync 5, %0;" ::"r"(gthreads) : "memory"); break;
    case 5: asm volatile("bar.sync 6, %0;" ::"r"(gthreads) : "memory"); break;
    case 6: asm volatile("bar.sync 7, %0;" ::"r"(gthreads) : "memory"); break;
    default: asm volatile("bar.sync 8, %0;" ::"r"(gthreads) : "memory"); break;
    }
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute may start while
// the kernel before it in the stream still runs; dependency_wait() returns once that kernel has finished and its
// writes are visible (at once when the launch carried no such attribute).  release_dependents() lets the next
// kernel start early.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint4 lds128(const void *p) { return *reinterpret_cast<const uint4 *>(p); }
__device__ __forceinline__ uint2 lds64(const void *p) { return *reinterpret_cast<const uint2 *>(p); }
__device__ __forceinline__ void sts128(void *p, uint4 v) { *reinterpret_cast<uint4 *>(p) = v; }
__device__ __forceinline__ void sts64(void *p, uint2 v) { *reinterpret_cast<uint2 *>(p) = v; }

// ----------------------------------------------------------- arithmetic --

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);     // round to nearest even, lo in the low half
    return *reinterpret_cast<uint32_t *>(&v);
}

// Two fp32 values in one 64-bit register for the packed fp32 instructions of sm_100 (each half is an
// ordinary IEEE round-to-nearest operation; nothing is fused unless fma2 is asked for).
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 pack2_bits(uint32_t lo, uint32_t hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void unpack2_bits(f32x2 v, uint32_t &lo, uint32_t &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b)
{
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b)
{
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// p + c with its own rounding when p is a product.  The assembler contracts a packed multiply whose only
// use is a packed add into one fused multiply-add (measured: it does so even though both carry .rn, unlike
// the scalar forms), which would round x * inv + c once instead of twice.  Written as fma(p, one, c) with
// one = 1.0f arriving as a launch parameter the sum is the same correctly rounded p + c, and a multiplier
// whose value the assembler does not know leaves it nothing to contract (with a literal 1.0f it folded the
// multiply away again in one of the kernels: codes at exact ties came out one step off).
__device__ __forceinline__ f32x2 add2_unfused(f32x2 p, f32x2 c, f32x2 one) { return fma2(p, one, c); }
// The two bf16 halves of w as a packed fp32 pair (exact).
__device__ __forceinline__ f32x2 bf16x2_to_f32x2(uint32_t w) { return pack2_bits(w << 16, w & 0xffff0000u); }
// The same through the mixed-precision add of sm_100 (bf16 + fp32 -> fp32; x + (-0) = x for every x, signed zeros and
// subnormals included): the widening leaves the integer pipe, which the coding loops load most.
__device__ __forceinline__ f32x2 bf16x2_widen(uint32_t w)
{
    f32x2 d;
    asm("{ .reg .b16 l, h; .reg .f32 fl, fh; mov.b32 {l, h}, %1; add.rn.f32.bf16 fl, l, %2; add.rn.f32.bf16 fh, h, %2;"
        " mov.b64 %0, {fl, fh}; }" : "=l"(d) : "r"(w), "f"(-0.0f));
    return d;
}
// max(|a|, |b|) on both bf16 halves; the sign of the result is meaningless.
__device__ __forceinline__ uint32_t maxabs_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Rounding trick used by quantise_tile: round_half_even(x * inv) sits in the low mantissa bits of the fp32 sum of the
// (already rounded) product with 1.5 * 2^23 + bias.  For |x * inv| < 2^22 the adder itself rounds the sum to an
// integer, ties to even (the bias is even, so ties fall the same way), and the mantissa holds code + bias.  The
// product and the sum are two separately rounded fp32 operations, as the codec's definition requires.
// Codes are then gathered in the floating-point pipe, exactly: with r = M + bias + code (M = 1.5 * 2^23) of two
// element pairs, (r_b - M) * 256 + r_a = M + (code_a + bias) + 256 (code_b + bias) in each half, no carries since
// 0 < code + bias < 256.  For int8 (bias 128) one byte permute interleaves the two halves' 16-bit fields and one XOR
// takes the bias off; for int4 (bias 8) the odd half is added in shifted by one nibble first.
__device__ __forceinline__ f32x2 gather2(f32x2 ra, f32x2 rb, f32x2 minus_m, f32x2 k256)
{
    return fma2(add2(rb, minus_m), k256, ra);
}
__device__ __forceinline__ uint32_t codes4_from(f32x2 t)        // int8: t = gather2 of pairs (0,1) and (2,3)
{
    uint32_t lo, hi;
    unpack2_bits(t, lo, hi);
    return __byte_perm(lo, hi, 0x5140) ^ 0x80808080u;
}
__device__ __forceinline__ uint32_t nibbles4_from(f32x2 t)      // int4: four nibbles in the low 16 bits, biased
{
    uint32_t lo, hi;
    unpack2_bits(t, lo, hi);
    return hi * 16u + lo;
}
// Encode n elements (a multiple of 64) of bf16 at A into int8 codes at B and one fp32 scale per 64
// elements (to shared S, or straight to global when the destination is not 16-byte aligned).
// Two lanes share a group, 32 elements each, read as four 128-bit shared loads in a lane-rotated
// order (bank-conflict free); the absmax is reduced with one shuffle; each lane issues one of the
// group's two IEEE divides.  ct is the thread's index inside its compute group.
// kInt4: codes in [-7, 7], two per byte (element 2k in the low nibble), 16 bytes per lane instead of 32.
template <bool kInt4>
__device__ __forceinline__ void quantise_tile(const unsigned char *A, unsigned char *B, float *S, float *g_scales,
                                              unsigned n, int ct, unsigned gthreads, float one)
{
    const float qmax = kInt4 ? 7.0f : 127.0f;
    const unsigned nhalf = n >> 5;                         // 32-element half groups
    const unsigned lane = (unsigned)ct & 31u;
    const unsigned rot = (lane >> 1) & 3u;
    for (unsigned hb = (unsigned)ct & ~31u; hb < nhalf; hb += gthreads) {
        const unsigned h = hb + lane;
        const bool act = h < nhalf;
        const unsigned char *src = A + (size_t)h * 64u;
        uint4 x[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            x[j] = act ? lds128(src + (((unsigned)j + rot) & 3u) * 16u) : make_uint4(0u, 0u, 0u, 0u);
        // absmax on the packed bf16 pairs, two chains
        uint32_t m0 = maxabs_bf16x2(x[0].x, x[0].y), m1 = maxabs_bf16x2(x[0].z, x[0].w);
#pragma unroll
        for (int j = 1; j < 4; ++j) {
            m0 = maxabs_bf16x2(m0, x[j].x); m1 = maxabs_bf16x2(m1, x[j].y);
            m0 = maxabs_bf16x2(m0, x[j].z); m1 = maxabs_bf16x2(m1, x[j].w);
        }
        m0 = maxabs_bf16x2(m0, m1);
        float a = fmaxf(__uint_as_float((m0 << 16) & 0x7fffffffu), __uint_as_float(m0 & 0x7fff0000u));
        a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
        // the two IEEE divides of the group are shared by its two lanes: the even lane forms a / qmax, the odd
        // lane qmax / a, and one shuffle swaps them
        const bool odd = (lane & 1u) != 0u;
        const float mine = __fdiv_rn(odd ? qmax : a, odd ? a : qmax);      // one divide per lane, operands selected first
        const float other = __shfl_xor_sync(0xffffffffu, mine, 1);
        float scale = odd ? other : mine;
        const bool ok = scale >= 1.17549435e-38f;         // smallest normal fp32; false for NaN too
        const float inv = ok ? (odd ? mine : other) : 0.0f;
        scale = ok ? scale : 0.0f;
        if (act) {
            const f32x2 inv2 = pack2(inv, inv);
            const float magic = 12582912.0f + (kInt4 ? 8.0f : 128.0f);
            const f32x2 magic2 = pack2(magic, magic);
            const f32x2 minus_m2 = pack2(-12582912.0f, -12582912.0f);
            const f32x2 k256 = pack2(256.0f, 256.0f);
            const f32x2 one2 = pack2(one, one);
            unsigned char *dst = B + (size_t)h * (kInt4 ? 16u : 32u);
            uint32_t nib[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // per pair: one rounded product, one rounded sum with 1.5 * 2^23 + bias (see above)
                const f32x2 r01 = add2_unfused(mul2(bf16x2_widen(x[j].x), inv2), magic2, one2);
                const f32x2 r23 = add2_unfused(mul2(bf16x2_widen(x[j].y), inv2), magic2, one2);
                const f32x2 r45 = add2_unfused(mul2(bf16x2_widen(x[j].z), inv2), magic2, one2);
                const f32x2 r67 = add2_unfused(mul2(bf16x2_widen(x[j].w), inv2), magic2, one2);
                const f32x2 ta = gather2(r01, r23, minus_m2, k256), tb = gather2(r45, r67, minus_m2, k256);
                if (kInt4) {
                    // byte k = code 2k | code 2k+1 << 4
                    nib[j] = __byte_perm(nibbles4_from(ta), nibbles4_from(tb), 0x5410) ^ 0x88888888u;
                } else {
                    sts64(dst + (((unsigned)j + rot) & 3u) * 8u, make_uint2(codes4_from(ta), codes4_from(tb)));
                }
            }
            if (kInt4) {
                // nib[j] belongs at word (j + rot) & 3: rotate the registers, then one 128-bit store
                uint32_t o0 = nib[0], o1 = nib[1], o2 = nib[2], o3 = nib[3];
                if (rot & 1u) { const uint32_t t = o3; o3 = o2; o2 = o1; o1 = o0; o0 = t; }
                if (rot & 2u) { uint32_t t = o0; o0 = o2; o2 = t; t = o1; o1 = o3; o3 = t; }
                sts128(dst, make_uint4(o0, o1, o2, o3));
            }
            if ((lane & 1u) == 0u) {
                if (g_scales) g_scales[h >> 1] = scale; else S[h >> 1] = scale;
            }
        }
    }
}

// (float)code for bytes K and K+1 of w (four codes already XORed with 0x80) as a packed pair: each
// byte is placed in the mantissa of 2^23 (giving 2^23 + code + 128) and 2^23 + 128 is subtracted. Exact.
template <int K> __device__ __forceinline__ f32x2 codes_to_f32x2(uint32_t w_biased, f32x2 minus_bias)
{
    return add2(pack2_bits(__byte_perm(w_biased, 0x4B000000u, 0x7650 + K),
                           __byte_perm(w_biased, 0x4B000000u, 0x7650 + K + 1)), minus_bias);
}
__device__ __forceinline__ uint32_t pack_bf16x2(f32x2 v)
{
    float lo, hi;
    unpack2(v, lo, hi);
    return pack_bf16x2(lo, hi);
}

// Decode n int8 codes at B with scales S into bf16 at A: one fp32 product per element, rounded to bf16.
__device__ __forceinline__ void dequantise_tile(const unsigned char *B, const float *S, unsigned char *A,
                                                unsigned n, int ct, unsigned gthreads)
{
    const unsigned nvec = n >> 4;
    const f32x2 minus_bias = pack2(-8388736.0f, -8388736.0f);
    for (unsigned v = (unsigned)ct; v < nvec; v += gthreads) {
        const uint4 c = lds128(B + (size_t)v * 16u);
        const float sc = S[v >> 2];
        const f32x2 sc2 = pack2(sc, sc);
        const uint32_t w[4] = { c.x ^ 0x80808080u, c.y ^ 0x80808080u, c.z ^ 0x80808080u, c.w ^ 0x80808080u };
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            o[2 * j] = pack_bf16x2(mul2(codes_to_f32x2<0>(w[j], minus_bias), sc2));
            o[2 * j + 1] = pack_bf16x2(mul2(codes_to_f32x2<2>(w[j], minus_bias), sc2));
        }
        sts128(A + (size_t)v * 32u, make_uint4(o[0], o[1], o[2], o[3]));
        sts128(A + (size_t)v * 32u + 16u, make_uint4(o[4], o[5], o[6], o[7]));
    }
}

// Eight int4 codes of one word as four packed fp32 pairs (elements 0-1, 2-3, 4-5, 6-7), exact: the nibbles are
// biased by 8, split into even and odd bytes, and each byte goes through the same 2^23 mantissa trick.
__device__ __forceinline__ void nibbles_to_f32x2(uint32_t w, f32x2 minus_bias4, f32x2 *out)
{
    const uint32_t b = w ^ 0x88888888u;
    const uint32_t e = b & 0x0f0f0f0fu, o = (b >> 4) & 0x0f0f0f0fu;
    out[0] = add2(pack2_bits(__byte_perm(e, 0x4B000000u, 0x7650), __byte_perm(o, 0x4B000000u, 0x7650)), minus_bias4);
    out[1] = add2(pack2_bits(__byte_perm(e, 0x4B000000u, 0x7651), __byte_perm(o, 0x4B000000u, 0x7651)), minus_bias4);
    out[2] = add2(pack2_bits(__byte_perm(e, 0x4B000000u, 0x7652), __byte_perm(o, 0x4B000000u, 0x7652)), minus_bias4);
    out[3] = add2(pack2_bits(__byte_perm(e, 0x4B000000u, 0x7653), __byte_perm(o, 0x4B000000u, 0x7653)), minus_bias4);
}

// Decode n int4 codes (n/2 bytes at B) with scales S into bf16 at A.
__device__ __forceinline__ void dequantise4_tile(const unsigned char *B, const float *S, unsigned char *A,
                                                 unsigned n, int ct, unsigned gthreads)
{
    const unsigned nvec = n >> 4;                          // 16 codes = 8 bytes per step
    const f32x2 minus_bias4 = pack2(-8388616.0f, -8388616.0f);   // -(2^23 + 8)
    for (unsigned v = (unsigned)ct; v < nvec; v += gthreads) {
        const uint2 c = lds64(B + (size_t)v * 8u);
        const float sc = S[v >> 2];
        const f32x2 sc2 = pack2(sc, sc);
        f32x2 f[8];
        nibbles_to_f32x2(c.x, minus_bias4, f);
        nibbles_to_f32x2(c.y, minus_bias4, f + 4);
        uint32_t o[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) o[k] = pack_bf16x2(mul2(f[k], sc2));
        sts128(A + (size_t)v * 32u, make_uint4(o[0], o[1], o[2], o[3]));
        sts128(A + (size_t)v * 32u + 16u, make_uint4(o[4], o[5], o[6], o[7]));
    }
}

// Two consecutive fp32 values of shared memory as a packed pair.
__device__ __forceinline__ f32x2 lds_f32x2(const float *p)
{
    const uint2 v = lds64(p);
    return pack2_bits(v.x, v.y);
}

// Decode a key tile of a per-channel key codec: n codes at B (whole token rows of row_elems channels), one scale per
// channel at S, bf16 to A.  One item is 8 consecutive channels of one token.
// kKeep: keep a thread's eight scales in registers from item to item (not in the compose kernels, whose rotation
// path already fills their register budget).
template <bool kInt4, bool kKeep = true>
__device__ __forceinline__ void dequantise_kc_tile(const unsigned char *B, const float *S, unsigned char *A,
                                                   unsigned n, unsigned row_elems, int ct, unsigned gthreads)
{
    const unsigned nitems = n >> 3;
    const f32x2 minus_bias = pack2(-8388736.0f, -8388736.0f);
    const f32x2 minus_bias4 = pack2(-8388616.0f, -8388616.0f);
    // A thread's items are gthreads * 8 elements apart; where that is a whole number of rows (1024-element rows, four
    // warps) every item of the thread has the same eight channels, and their scales are loaded once, not once per item.
    unsigned have_ch = 0xffffffffu;
    f32x2 sc[4];
    for (unsigned v = (unsigned)ct; v < nitems; v += gthreads) {
        const unsigned e = v << 3;
        const unsigned ch = e - (e / row_elems) * row_elems;
        if (!kKeep || ch != have_ch) {
            const uint4 s0 = lds128(S + ch), s1 = lds128(S + ch + 4);
            sc[0] = pack2_bits(s0.x, s0.y); sc[1] = pack2_bits(s0.z, s0.w);
            sc[2] = pack2_bits(s1.x, s1.y); sc[3] = pack2_bits(s1.z, s1.w);
            have_ch = ch;
        }
        f32x2 f[4];
        if (kInt4) {
            nibbles_to_f32x2(*reinterpret_cast<const uint32_t *>(B + (e >> 1)), minus_bias4, f);
        } else {
            const uint2 c = lds64(B + e);
            const uint32_t w0 = c.x ^ 0x80808080u, w1 = c.y ^ 0x80808080u;
            f[0] = codes_to_f32x2<0>(w0, minus_bias); f[1] = codes_to_f32x2<2>(w0, minus_bias);
            f[2] = codes_to_f32x2<0>(w1, minus_bias); f[3] = codes_to_f32x2<2>(w1, minus_bias);
        }
        uint4 o;
        o.x = pack_bf16x2(mul2(f[0], sc[0]));
        o.y = pack_bf16x2(mul2(f[1], sc[1]));
        o.z = pack_bf16x2(mul2(f[2], sc[2]));
        o.w = pack_bf16x2(mul2(f[3], sc[3]));
        sts128(A + (size_t)e * 2u, o);
    }
}

// Rotation coefficients a thread keeps in registers: (cos, sin, -sin) for 8 consecutive frequencies,
// as four packed pairs each.
struct RotCoef {
    f32x2 c[4], s[4], ns[4];
    int rope;      // table row they belong to
    unsigned col;  // first frequency index
};

__device__ __forceinline__ void load_coef(RotCoef &rc, const float2 *table, int rope, unsigned col, unsigned half)
{
    if (rc.rope == rope && rc.col == col) return;
    const float4 *p = reinterpret_cast<const float4 *>(table + (size_t)rope * half + col);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float4 v = __ldg(p + k);                     // (cos, sin) of frequencies 2k and 2k + 1
        rc.c[k] = pack2(v.x, v.z);
        rc.s[k] = pack2(v.y, v.w);
        rc.ns[k] = pack2(-v.y, -v.w);
    }
    rc.rope = rope; rc.col = col;
}

// u' = u cos - w sin, w' = w cos + u sin for four packed pairs of (u, w); each result is one rounded
// product folded into one fused multiply-add.
__device__ __forceinline__ void rotate8(const f32x2 *u, const f32x2 *w, const RotCoef &rc, uint4 &lo, uint4 &hi)
{
    uint32_t ou[4], ow[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        ou[k] = pack_bf16x2(fma2(u[k], rc.c[k], mul2(w[k], rc.ns[k])));
        ow[k] = pack_bf16x2(fma2(w[k], rc.c[k], mul2(u[k], rc.s[k])));
    }
    lo = make_uint4(ou[0], ou[1], ou[2], ou[3]);
    hi = make_uint4(ow[0], ow[1], ow[2], ow[3]);
}

// Rotate a tile of whole head rows (n a multiple of D, D a multiple of 16).  One work item is 8
// frequencies of one head row: elements [col, col+8) and [D/2 + col, D/2 + col + 8).
// kCodec = 0: bf16 at A, in place.  kCodec = 1 / 2: int8 / int4 codes at B and scales at S -> bf16 at A.
// kChan: the codes carry one scale per channel (S[channel], row_elems of them) instead of one per 64 elements.
template <int kCodec, bool kChan = false>
__device__ __forceinline__ void rotate_tile(unsigned char *A, const unsigned char *B, const float *S, unsigned n,
                                            unsigned D, const float2 *table, int rope, RotCoef &rc, int ct, unsigned gthreads,
                                            unsigned row_elems = 0)
{
    const unsigned half = D >> 1;
    const unsigned per_row = D >> 4;                      // work items per head row
    const bool pow2 = (per_row & (per_row - 1u)) == 0u;
    const unsigned shift = 31u - (unsigned)__clz(per_row);
    const unsigned items = n >> 4;
    const f32x2 minus_bias = pack2(-8388736.0f, -8388736.0f);
    for (unsigned it = (unsigned)ct; it < items; it += gthreads) {
        const unsigned r = pow2 ? it >> shift : it / per_row;
        const unsigned col = (it - r * per_row) << 3;
        load_coef(rc, table, rope, col, half);
        const unsigned e_lo = r * D + col, e_hi = e_lo + half;
        f32x2 u[4], w[4];
        if (kCodec != 0) {
            if (kCodec == 2) {
                const f32x2 minus_bias4 = pack2(-8388616.0f, -8388616.0f);
                nibbles_to_f32x2(*reinterpret_cast<const uint32_t *>(B + (e_lo >> 1)), minus_bias4, u);
                nibbles_to_f32x2(*reinterpret_cast<const uint32_t *>(B + (e_hi >> 1)), minus_bias4, w);
            } else {
                const uint2 cl = lds64(B + e_lo), ch = lds64(B + e_hi);
                const uint32_t l0 = cl.x ^ 0x80808080u, l1 = cl.y ^ 0x80808080u;
                const uint32_t h0 = ch.x ^ 0x80808080u, h1 = ch.y ^ 0x80808080u;
                u[0] = codes_to_f32x2<0>(l0, minus_bias); u[1] = codes_to_f32x2<2>(l0, minus_bias);
                u[2] = codes_to_f32x2<0>(l1, minus_bias); u[3] = codes_to_f32x2<2>(l1, minus_bias);
                w[0] = codes_to_f32x2<0>(h0, minus_bias); w[1] = codes_to_f32x2<2>(h0, minus_bias);
                w[2] = codes_to_f32x2<0>(h1, minus_bias); w[3] = codes_to_f32x2<2>(h1, minus_bias);
            }
            if (kChan) {
                const unsigned c_lo = e_lo - (e_lo / row_elems) * row_elems, c_hi = c_lo + half;
                const uint4 a0 = lds128(S + c_lo), a1 = lds128(S + c_lo + 4);     // 128-bit loads: two lanes to a bank at worst
                const uint4 b0 = lds128(S + c_hi), b1 = lds128(S + c_hi + 4);     // (kept per item: caching sixteen scales spills)
                u[0] = mul2(u[0], pack2_bits(a0.x, a0.y)); u[1] = mul2(u[1], pack2_bits(a0.z, a0.w));
                u[2] = mul2(u[2], pack2_bits(a1.x, a1.y)); u[3] = mul2(u[3], pack2_bits(a1.z, a1.w));
                w[0] = mul2(w[0], pack2_bits(b0.x, b0.y)); w[1] = mul2(w[1], pack2_bits(b0.z, b0.w));
                w[2] = mul2(w[2], pack2_bits(b1.x, b1.y)); w[3] = mul2(w[3], pack2_bits(b1.z, b1.w));
            } else {
                const float sl = S[e_lo >> 6], sh = S[e_hi >> 6];
                const f32x2 sl2 = pack2(sl, sl), sh2 = pack2(sh, sh);
#pragma unroll
                for (int k = 0; k < 4; ++k) { u[k] = mul2(u[k], sl2); w[k] = mul2(w[k], sh2); }
            }
        } else {
            const uint4 xl = lds128(A + (size_t)e_lo * 2u), xh = lds128(A + (size_t)e_hi * 2u);
            u[0] = bf16x2_to_f32x2(xl.x); u[1] = bf16x2_to_f32x2(xl.y); u[2] = bf16x2_to_f32x2(xl.z); u[3] = bf16x2_to_f32x2(xl.w);
            w[0] = bf16x2_to_f32x2(xh.x); w[1] = bf16x2_to_f32x2(xh.y); w[2] = bf16x2_to_f32x2(xh.z); w[3] = bf16x2_to_f32x2(xh.w);
        }
        uint4 lo, hi;
        rotate8(u, w, rc, lo, hi);
        sts128(A + (size_t)e_lo * 2u, lo);
        sts128(A + (size_t)e_hi * 2u, hi);
    }
}

// ---------------------------------------------------------- tile decode --

// Address resolution (request position -> block-table entry -> pool address) and chunk addressing
// for tile g.  Records KDN_E_RANGE and yields an empty tile for a block id outside the pool.
// rows_out: shared memory for the token-row indices of a several-row tile (TF_ROWS); untouched otherwise.
template <int OP, bool kWide = false>
__device__ __forceinline__ void decode_tile(const Launch &P, unsigned g, TileDesc &d, unsigned *rows_out)
{
    d.n = 0; d.flags = 0; d.rope = -1; d.sbytes = 0;
    d.g_pool = 0; d.g_chunk = 0; d.g_scales = 0; d.runs = 0;
    if (g >= P.n_tiles) return;                             // lanes past this CTA's last tile
    const DevOp *ops = P.ops ? P.ops : P.inline_ops;       // global memory, or the kernel's parameter space
    int lo = 0, hi = P.n_ops - 1;
    while (lo < hi) {                                       // last op with tile_begin <= g
        int mid = (lo + hi + 1) >> 1;
        if (ops[mid].tile_begin <= g) lo = mid; else hi = mid - 1;
    }
    const DevOp op = ops[lo];
    const unsigned gl = g - op.tile_begin;
    unsigned plane, n;
    long long id_index;                                     // block-table entry of the tile
    unsigned long long pool_elem;                           // element offset of the tile inside its pool block
    unsigned long long ce;                                  // element offset of the tile inside the chunk
    bool many_rows = false;
    if (kWide && (op.list_mode == 1 || op.list_mode == 3)) {
        // kWide: every keep-list tile goes this way, whatever its row count
        const unsigned rpt = (unsigned)P.rows_per_tile;
        const unsigned tpp = ((unsigned)op.n_list + rpt - 1u) / rpt;
        plane = gl / tpp;
        const unsigned i0 = (gl - plane * tpp) * rpt;
        const unsigned nr = (unsigned)op.n_list - i0 < rpt ? (unsigned)op.n_list - i0 : rpt;
        bool bad = false;
        unsigned starts = 0u, prev = 0u;
        // four rows at a time, so that their look-ups are in flight together; the indices go to shared memory
        auto resolve4 = [&](unsigned r0) {
            unsigned rows4[4] = { 0u, 0u, 0u, 0u };
#pragma unroll
            for (unsigned k = 0; k < 4u; ++k) {
                const unsigned r = r0 + k;
                if (r < nr) {
                    const long long rel = op.list_mode == 3 ? (long long)(i0 + r) : (long long)__ldg(op.list + i0 + r);
                    const long long p = op.off + rel;
                    unsigned row = 0u;
                    if (rel < 0 || p >= op.pos_end || (long long)(i0 + r) >= op.T) {
                        bad = true;
                    } else {
                        const long long bi = p / P.bs;
                        const long long id = __ldg(op.table + bi);
                        if (id < 0 || id >= P.n_blocks) bad = true;
                        else row = (unsigned)(id * P.bs + (p - bi * P.bs));
                    }
                    if (r == 0u || row != prev + 1u) starts |= 1u << r;
                    prev = row;
                    rows4[k] = row;
                }
            }
            *reinterpret_cast<uint4 *>(rows_out + r0) = make_uint4(rows4[0], rows4[1], rows4[2], rows4[3]);
        };
        resolve4(0u);                                       // tiles of up to four rows end here
        for (unsigned r0 = 4u; r0 < nr; r0 += 4u) resolve4(r0);
        if (bad) { atomicCAS(P.status, 0, kStatusRange); return; }          // the whole tile is skipped
        d.runs = starts | (nr << 16);
        d.flags |= TF_ROWS;
        many_rows = true;
        id_index = 0;
        pool_elem = 0;
        ce = (unsigned long long)i0 * P.row_elems;
        n = nr * P.row_elems;
    } else if (op.list_mode == 1 && P.rows_per_tile > 1) {
        // keep-list: up to rows_per_tile consecutive listed tokens per tile; they are consecutive chunk tokens, and
        // each sits wherever its own block-table entry says
        const unsigned rpt = (unsigned)P.rows_per_tile;
        const unsigned tpp = ((unsigned)op.n_list + rpt - 1u) / rpt;
        plane = gl / tpp;
        const unsigned i0 = (gl - plane * tpp) * rpt;
        const unsigned nr = (unsigned)op.n_list - i0 < rpt ? (unsigned)op.n_list - i0 : rpt;
        bool bad = false;
        unsigned rows[kMaxRowsPerTile];
#pragma unroll
        for (int r = 0; r < kMaxRowsPerTile; ++r) {
            rows[r] = 0u;
            if ((unsigned)r < nr) {
                const long long rel = __ldg(op.list + i0 + (unsigned)r);
                const long long p = op.off + rel;
                if (rel < 0 || p >= op.pos_end || (long long)(i0 + (unsigned)r) >= op.T) { bad = true; continue; }
                const long long bi = p / P.bs;
                const long long id = __ldg(op.table + bi);
                if (id < 0 || id >= P.n_blocks) { bad = true; continue; }
                rows[r] = (unsigned)(id * P.bs + (p - bi * P.bs));
            }
        }
        if (bad) { atomicCAS(P.status, 0, kStatusRange); return; }          // the whole tile is skipped
        // runs of rows that are neighbours in the pool, worked out back to front (all indices are compile-time: the
        // arrays stay in registers)
        unsigned len[kMaxRowsPerTile + 1];
        len[kMaxRowsPerTile] = 0u;
        unsigned runs = 0u;
#pragma unroll
        for (int r = kMaxRowsPerTile - 1; r >= 0; --r) {
            const bool next_joins = r + 1 < kMaxRowsPerTile && (unsigned)(r + 1) < nr && rows[r + 1 < kMaxRowsPerTile ? r + 1 : r] == rows[r] + 1u;
            len[r] = (unsigned)r < nr ? 1u + (next_joins ? len[r + 1] : 0u) : 0u;
        }
#pragma unroll
        for (int r = 0; r < kMaxRowsPerTile; ++r) {
            const bool joins_prev = r > 0 && rows[r] == rows[r > 0 ? r - 1 : 0] + 1u;
            if (!joins_prev) runs |= len[r] << (4 * r);
        }
        *reinterpret_cast<uint4 *>(rows_out) = make_uint4(rows[0], rows[1], rows[2], rows[3]);
        d.runs = runs;
        d.flags |= TF_ROWS;
        many_rows = true;
        id_index = 0;
        pool_elem = 0;
        ce = (unsigned long long)i0 * P.row_elems;
        n = nr * P.row_elems;
    } else if (op.list_mode != 0) {
        // one listed token (one row of H * D elements) per tile
        plane = gl / (unsigned)op.n_list;
        const unsigned i = gl - plane * (unsigned)op.n_list;
        const long long rel = __ldg(op.list + i);                        // (list_mode 3 never comes here: kWide kernels only)
        const long long c = op.list_mode == 2 ? rel : (long long)i;      // chunk token
        const long long p = op.off + rel;
        if (rel < 0 || p >= op.pos_end || c >= op.T) { atomicCAS(P.status, 0, kStatusRange); return; }
        id_index = p / P.bs;
        pool_elem = (unsigned long long)(p - id_index * P.bs) * P.row_elems;
        ce = (unsigned long long)c * P.row_elems;          // inside the plane; the plane is added below
        n = P.row_elems;
    } else {
        const unsigned per_plane = (unsigned)op.nblk * P.tpb;
        plane = gl / per_plane;
        const unsigned rem = gl - plane * per_plane;
        const unsigned j = rem / P.tpb;
        const unsigned k = rem - j * P.tpb;
        const long long blk_start = ((long long)op.j0 + j) * P.bs;
        const long long p_lo = op.off > blk_start ? op.off : blk_start;
        const long long p_end = op.off + op.T;
        const long long p_hi = p_end < blk_start + P.bs ? p_end : blk_start + P.bs;
        if (p_hi <= p_lo) return;
        const unsigned long long run = (unsigned long long)(p_hi - p_lo) * P.row_elems;
        const unsigned long long e0 = (unsigned long long)k * P.tile_elems;
        if (e0 >= run) return;
        n = (unsigned)((run - e0) < (unsigned long long)P.tile_elems ? (run - e0) : P.tile_elems);
        id_index = (long long)op.j0 + j;
        pool_elem = (unsigned long long)(p_lo - blk_start) * P.row_elems + e0;
        ce = (unsigned long long)(p_lo - op.off) * P.row_elems + e0;     // inside the plane
    }
    const int kv = op.kv_sel ? op.kv_sel - 1 : (int)(plane & 1u);
    const unsigned li = op.kv_sel ? plane : plane >> 1;     // layer index inside the op's layer range
    const int l = op.l0 + (int)li;
    const unsigned char *base = reinterpret_cast<const unsigned char *>(kv ? P.v_layers[l] : P.k_layers[l]);
    if (many_rows) {
        d.g_pool = (unsigned long long)base;
    } else {
        const long long id = __ldg(op.table + id_index);
        if (id < 0 || id >= P.n_blocks) { atomicCAS(P.status, 0, kStatusRange); d.flags = 0; return; }
        d.g_pool = (unsigned long long)(base + ((unsigned long long)id * P.bs * P.row_elems + pool_elem) * 2ull);
    }
    const unsigned long long ce_plane = ce;                                   // element offset inside the plane
    ce += ((unsigned long long)li * 2ull + (unsigned long long)kv) * (unsigned long long)op.T * P.row_elems;
    if (op.codec == 0) {
        d.g_chunk = (unsigned long long)(op.data + ce * 2ull);
    } else {
        d.flags |= TF_CODED;
        if (op.codec == 2 || op.codec == 4) { d.flags |= TF_INT4; d.g_chunk = (unsigned long long)(op.data + (ce >> 1)); }
        else d.g_chunk = (unsigned long long)(op.data + ce);
        if (op.codec >= 3) {
            // per layer: key scales [ceil(T / 64)][row_elems], then value scales [T][row_elems / 64]
            const unsigned long long n_groups = ((unsigned long long)op.T + 63ull) >> 6;
            const unsigned long long per_layer = n_groups * P.row_elems + (((unsigned long long)op.T * P.row_elems) >> 6);
            if (kv == 0) {
                // the tile is whole token rows of one 64-token group (the host sees to both)
                d.flags |= TF_KCHAN;
                d.g_scales = (unsigned long long)(op.scales + ((unsigned long long)li * per_layer +
                                                               ((ce_plane / P.row_elems) >> 6) * P.row_elems) * 4ull);
                d.sbytes = P.row_elems * 4u;
            } else {
                d.g_scales = (unsigned long long)(op.scales + ((unsigned long long)li * per_layer + n_groups * P.row_elems +
                                                               (ce_plane >> 6)) * 4ull);
                d.sbytes = n >> 4;
            }
        } else {
            d.g_scales = (unsigned long long)(op.scales + (ce >> 6) * 4ull);
            d.sbytes = n >> 4;
        }
        if ((d.g_scales & 15ull) || (d.sbytes & 15u)) d.flags |= TF_SCALES_PLAIN;
    }
    if (OP == OP_COMPOSE && kv == 0 && op.rope >= 0) { d.flags |= TF_ROTATE; d.rope = op.rope; }
    d.n = n;
}

// ------------------------------------------------------------- pipeline --

struct Smem {
    unsigned char *stage0;
    uint32_t full, empty, ready;      // shared addresses of the barrier arrays (8 bytes per stage)
    TileDesc *desc;
    unsigned *rows_stage;             // [stages][4]: token-row indices of the several-row tile in each slot
    unsigned *rows_ahead;             // [2][32][4]: the same for the tiles the loader has decoded but not yet queued
    volatile int *abort_flag;
    volatile unsigned *issued;        // tiles whose loads the loader has queued so far
};

template <bool kWide>
__device__ __forceinline__ Smem carve(const Launch &P, unsigned char *smem)
{
    Smem s;
    s.stage0 = smem;
    unsigned char *p = smem + (size_t)P.stages * P.stage_bytes;
    s.full = smem_u32(p);
    s.empty = s.full + 8u * (uint32_t)P.stages;
    s.ready = s.empty + 8u * (uint32_t)P.stages;
    p += 24u * (size_t)P.stages;
    p = (unsigned char *)(((uintptr_t)p + 15u) & ~(uintptr_t)15u);
    s.desc = reinterpret_cast<TileDesc *>(p);
    p += sizeof(TileDesc) * (size_t)P.stages;
    s.rows_stage = reinterpret_cast<unsigned *>(p);          // both areas exist only in launches with several-row tiles
    if constexpr (kWide) {
        s.rows_ahead = s.rows_stage + (size_t)kWideRowsPerTile * (size_t)P.stages;
        p += 4u * ((size_t)kWideRowsPerTile * (size_t)P.stages + 64u * kRowsAheadStride);
    } else {
        s.rows_ahead = s.rows_stage + 4u * (size_t)P.stages;
        if (P.rows_per_tile > 1) p += 16u * (size_t)P.stages + 16u * 64u;
    }
    s.abort_flag = reinterpret_cast<volatile int *>(p);
    s.issued = reinterpret_cast<volatile unsigned *>(s.abort_flag + 1);
    return s;
}

// Bytes of shared memory a launch needs (host mirrors this).
__host__ __device__ inline size_t smem_bytes(int stages, unsigned stage_bytes, int rows_per_tile = 1, bool wide = false)
{
    return (size_t)stages * stage_bytes + 24u * (size_t)stages + 16u + sizeof(TileDesc) * (size_t)stages + 16u +
           (wide ? 4u * ((size_t)kWideRowsPerTile * (size_t)stages + 64u * kRowsAheadStride)
                 : rows_per_tile > 1 ? 16u * (size_t)stages + 16u * 64u : 0u);
}

template <int OP, int kGroups, int kGW, bool kWide = false>
__device__ __forceinline__ void tile_pipeline(const Launch &P)
{
    constexpr bool kCompute = kGroups > 0;
    constexpr unsigned kGT = (unsigned)kGW * 32u;           // threads of one compute group
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // The next launch of this library in the stream may be scheduled as this kernel's CTAs leave, set up its barriers
    // and then wait (below) for this kernel to finish: back-to-back calls lose no time between kernels.
    release_dependents();
    const Smem sm = carve<kWide>(P, smem_raw);
    const int S = P.stages;
    const int tid = (int)threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(sm.full + 8u * s, 1u);
            mbar_init(sm.empty + 8u * s, 1u);
            mbar_init(sm.ready + 8u * s, (uint32_t)kGW);
        }
        *sm.abort_flag = 0;
        *sm.issued = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncthreads();
    if (P.wait_all) dependency_wait();                      // returns at once when the launch was an ordinary one

    const unsigned grid = gridDim.x, bid = blockIdx.x;
    const unsigned n_my = P.n_tiles > bid ? (P.n_tiles - bid + grid - 1u) / grid : 0u;
    const int storer_warp = 1 + kGroups * kGW;

    if (warp == kLoaderWarp) {
        // ------------------------------------------------------------ loader
        unsigned issued = 0;
        unsigned st = 0;                                      // pipeline slot of the next tile, and the phase of its
        uint32_t ph = 0;                                      // barriers (flips every time the slots wrap around)
        bool aborted = false;
        TileDesc cur;
        unsigned ahead = 0;                                   // which half of rows_ahead holds the rows of `cur`
        constexpr unsigned kAheadStride = kWide ? kRowsAheadStride : 4u;
        decode_tile<OP, kWide>(P, (unsigned)lane < n_my ? bid + (unsigned)lane * grid : 0xffffffffu, cur, sm.rows_ahead + (size_t)lane * kAheadStride);
        for (unsigned base = 0; base < n_my && !aborted; base += 32u) {
            TileDesc nxt;
            decode_tile<OP, kWide>(P, base + 32u + lane < n_my ? bid + (base + 32u + lane) * grid : 0xffffffffu, nxt,
                                   sm.rows_ahead + ((size_t)(ahead ^ 1u) * 32u + (size_t)lane) * kAheadStride);
            const unsigned cnt = n_my - base < 32u ? n_my - base : 32u;
            for (unsigned t = 0; t < cnt; ++t) {
                bool ok = true;                               // lane t: the slot was free and the tile's copies are queued
                if ((unsigned)lane == t) {
                    ok = mbar_wait(sm.empty + 8u * st, ph ^ 1u, sm.abort_flag, P.wait_limit_ns);
                    if (ok) {
                        sm.desc[st] = cur;
                        if constexpr (kWide) {
                            if (OP != OP_STORE && (cur.flags & TF_ROWS)) {                 // the storer scatters the rows
                                const unsigned *my_rows = sm.rows_ahead + ((size_t)ahead * 32u + (size_t)lane) * kRowsAheadStride;
                                const unsigned nr = cur.runs >> 16;
                                for (unsigned b = 0; b < nr; b += 4u)
                                    sts128(sm.rows_stage + (size_t)st * kWideRowsPerTile + b, lds128(my_rows + b));
                            }
                        } else
                        if (OP != OP_STORE && (cur.flags & TF_ROWS))       // the storer scatters the rows
                            *reinterpret_cast<uint4 *>(sm.rows_stage + (size_t)st * 4u) =
                                *reinterpret_cast<const uint4 *>(sm.rows_ahead + ((size_t)ahead * 32u + (size_t)lane) * 4u);
                        const uint32_t bar = sm.full + 8u * st;
                        unsigned char *A = sm.stage0 + (size_t)st * P.stage_bytes;
                        if (cur.n == 0u) {
                            mbar_arrive(bar);
                        } else if (OP == OP_STORE) {
                            mbar_arrive_expect_tx(bar, cur.n * 2u);
                            if (kWide && (cur.flags & TF_ROWS)) {
                                const unsigned rb = P.row_elems * 2u;
                                const unsigned *my_rows = sm.rows_ahead + ((size_t)ahead * 32u + (size_t)lane) * kRowsAheadStride;
                                const unsigned nr = cur.runs >> 16;
                                const unsigned starts = (cur.runs & 0xffffu) | (1u << nr);      // a stop bit behind the last row
                                for (unsigned b = 0; b < nr; b += 4u) {
                                    const uint4 rv = lds128(my_rows + b);
                                    const unsigned rows4[4] = { rv.x, rv.y, rv.z, rv.w };
#pragma unroll
                                    for (unsigned k = 0; k < 4u; ++k) {
                                        const unsigned r = b + k;
                                        if (r < nr && ((starts >> r) & 1u)) {
                                            const unsigned len = (unsigned)__ffs((int)(starts >> (r + 1u)));     // rows up to the next start
                                            bulk_g2s(smem_u32(A + (size_t)r * rb), (const void *)(cur.g_pool + (unsigned long long)rows4[k] * rb), len * rb, bar);
                                        }
                                    }
                                }
                            } else if (cur.flags & TF_ROWS) {
                                // one copy per run of rows that are neighbours in the pool
                                const unsigned rb = P.row_elems * 2u;
                                const uint4 rv = *reinterpret_cast<const uint4 *>(sm.rows_ahead + ((size_t)ahead * 32u + (size_t)lane) * 4u);
                                const unsigned rows[kMaxRowsPerTile] = { rv.x, rv.y, rv.z, rv.w };
#pragma unroll
                                for (int r = 0; r < kMaxRowsPerTile; ++r) {
                                    const unsigned len = (cur.runs >> (4 * r)) & 15u;
                                    if (len) bulk_g2s(smem_u32(A + (size_t)r * rb), (const void *)(cur.g_pool + (unsigned long long)rows[r] * rb),
                                                      len * rb, bar);
                                }
                            } else {
                                bulk_g2s(smem_u32(A), (const void *)cur.g_pool, cur.n * 2u, bar);
                            }
                        } else if (!(cur.flags & TF_CODED)) {
                            mbar_arrive_expect_tx(bar, cur.n * 2u);
                            bulk_g2s(smem_u32(A), (const void *)cur.g_chunk, cur.n * 2u, bar);
                        } else {
                            const uint32_t code_bytes = (cur.flags & TF_INT4) ? cur.n >> 1 : cur.n;
                            if (cur.flags & TF_SCALES_PLAIN) {
                                mbar_arrive_expect_tx(bar, code_bytes);
                                bulk_g2s(smem_u32(A + P.off_b), (const void *)cur.g_chunk, code_bytes, bar);
                            } else {
                                mbar_arrive_expect_tx(bar, code_bytes + cur.sbytes);
                                bulk_g2s(smem_u32(A + P.off_b), (const void *)cur.g_chunk, code_bytes, bar);
                                bulk_g2s(smem_u32(A + P.off_s), (const void *)cur.g_scales, cur.sbytes, bar);
                            }
                        }
                    }
                }
                if (__any_sync(0xffffffffu, !ok || *sm.abort_flag != 0)) {
                    // a tile queued just before the CTA gave up still counts: the drain below has to wait for it
                    if (__shfl_sync(0xffffffffu, ok ? 1 : 0, (int)t)) ++issued;
                    aborted = true;
                    break;
                }
                ++issued;
                if (lane == 0) *sm.issued = issued;
                if (++st == (unsigned)S) { st = 0; ph ^= 1u; }
            }
            cur = nxt;
            ahead ^= 1u;
        }
        if (aborted && lane == 0) {
            atomicCAS(P.status, 0, kStatusTimeout);
            // bounded drain of the copies this warp issued into the last S slots
            const unsigned first = issued > (unsigned)S ? issued - (unsigned)S : 0u;
            for (unsigned slot = first; slot < issued; ++slot) {
                unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(sm.full + 8u * (slot % (unsigned)S), (slot / (unsigned)S) & 1u))
                    if (global_timer_ns() - t0 > kWaitLimitNs) break;
            }
        }
    } else if (warp == storer_warp) {
        // ------------------------------------------------------------ storer
        if (lane == 0) {
            unsigned done = 0;                                // slots whose store group was committed
            unsigned st = 0, st2 = 0;                         // slot being stored / slot being recycled, with the
            uint32_t ph = 0, ph2 = 0;                         // phases of their barriers
            for (unsigned slot = 0; slot < n_my; ++slot) {
                if (!mbar_wait(sm.full + 8u * st, ph, sm.abort_flag, P.wait_limit_ns)) break;
                const TileDesc d = sm.desc[st];
                unsigned char *A = sm.stage0 + (size_t)st * P.stage_bytes;
                if (d.n != 0u) {
                    const bool computed = kCompute && (OP == OP_STORE ? (d.flags & TF_CODED) != 0u
                                                                       : (d.flags & (TF_CODED | TF_ROTATE)) != 0u);
                    if (computed && !mbar_wait(sm.ready + 8u * st, ph, sm.abort_flag, P.wait_limit_ns)) break;
                    if (OP == OP_STORE) {
                        if (d.flags & TF_CODED) {
                            bulk_s2g((void *)d.g_chunk, smem_u32(A + P.off_b), (d.flags & TF_INT4) ? d.n >> 1 : d.n);
                            if (!(d.flags & TF_SCALES_PLAIN))
                                bulk_s2g((void *)d.g_scales, smem_u32(A + P.off_s), d.sbytes);
                        } else {
                            bulk_s2g((void *)d.g_chunk, smem_u32(A), d.n * 2u);
                        }
                    } else if (kWide && (d.flags & TF_ROWS)) {
                        const unsigned rb = P.row_elems * 2u;
                        const unsigned *rows = sm.rows_stage + (size_t)st * kWideRowsPerTile;
                        const unsigned nr = d.runs >> 16;
                        const unsigned starts = (d.runs & 0xffffu) | (1u << nr);
                        for (unsigned b = 0; b < nr; b += 4u) {
                            const uint4 rv = lds128(rows + b);
                            const unsigned rows4[4] = { rv.x, rv.y, rv.z, rv.w };
#pragma unroll
                            for (unsigned k = 0; k < 4u; ++k) {
                                const unsigned r = b + k;
                                if (r < nr && ((starts >> r) & 1u)) {
                                    const unsigned len = (unsigned)__ffs((int)(starts >> (r + 1u)));
                                    bulk_s2g((void *)(d.g_pool + (unsigned long long)rows4[k] * rb), smem_u32(A + (size_t)r * rb), len * rb);
                                }
                            }
                        }
                    } else if (d.flags & TF_ROWS) {
                        const unsigned rb = P.row_elems * 2u;
                        const uint4 rv = *reinterpret_cast<const uint4 *>(sm.rows_stage + (size_t)st * 4u);
                        const unsigned rows[kMaxRowsPerTile] = { rv.x, rv.y, rv.z, rv.w };
#pragma unroll
                        for (int r = 0; r < kMaxRowsPerTile; ++r) {
                            const unsigned len = (d.runs >> (4 * r)) & 15u;
                            if (len) bulk_s2g((void *)(d.g_pool + (unsigned long long)rows[r] * rb), smem_u32(A + (size_t)r * rb), len * rb);
                        }
                    } else {
                        bulk_s2g((void *)d.g_pool, smem_u32(A), d.n * 2u);
                    }
                }
                bulk_commit();
                ++done;
                // recycle the slot committed store_lag slots ago: its store has read shared memory,
                // and every compute warp has moved past it
                bulk_wait_read_n(P.store_lag);
                if (slot >= (unsigned)P.store_lag) {
                    if (kCompute && !mbar_wait(sm.ready + 8u * st2, ph2, sm.abort_flag, P.wait_limit_ns)) break;
                    mbar_arrive(sm.empty + 8u * st2);
                    if (++st2 == (unsigned)S) { st2 = 0; ph2 ^= 1u; }
                    // The SM works through its bulk copies in the order they were queued, and a store holds the
                    // queue while it reads its tile out of shared memory.  With large tiles it pays to let the
                    // loader queue the reload of the slot just recycled first, so that its requests are on their
                    // way to HBM while the store drains (measured: 6.54 -> 6.64 TB/s on 32 KiB tiles; with row-sized
                    // tiles the wait costs more than it gains, so the host leaves it off there).  A short, bounded
                    // poll: the loader may be busy decoding its next batch of tiles.
                    if (!kCompute && P.reload_first) {
                        const unsigned want = slot - (unsigned)P.store_lag + (unsigned)S;   // the tile this recycle lets in
                        if (want < n_my)
                            for (int i = 0; i < 64 && *sm.issued <= want; ++i) { }
                    }
                }
                if (++st == (unsigned)S) { st = 0; ph ^= 1u; }
            }
            bulk_wait_read<0>();
            for (unsigned slot = done > (unsigned)P.store_lag ? done - (unsigned)P.store_lag : 0u; slot < done; ++slot)
                mbar_arrive(sm.empty + 8u * (slot % (unsigned)S));
            bulk_wait_all();
            if (done != n_my) atomicCAS(P.status, 0, kStatusTimeout);
        }
    } else if (kCompute) {
        // ----------------------------------------------------------- compute
        const int group = (tid - 32) / (int)kGT;            // this group owns slots group, group + kGroups, ...
        const int ct = (tid - 32) % (int)kGT;
        RotCoef rc;
        rc.rope = -1; rc.col = 0xffffffffu;
        // the rotation table is written by the kernel launched just before this one; only these warps read it
        if (OP == OP_COMPOSE) dependency_wait();
        unsigned st = (unsigned)group;                        // S is a multiple of kGroups: st wraps exactly at S
        uint32_t ph = 0;
        for (unsigned slot = (unsigned)group; slot < n_my; slot += (unsigned)kGroups) {
            if (!mbar_wait(sm.full + 8u * st, ph, sm.abort_flag, P.wait_limit_ns)) break;
            const unsigned n = sm.desc[st].n;
            const unsigned flags = sm.desc[st].flags;
            unsigned char *A = sm.stage0 + (size_t)st * P.stage_bytes;
            unsigned char *B = A + P.off_b;
            float *Sc = reinterpret_cast<float *>(A + P.off_s);
            bool computed = false;
            if (n != 0u) {
                if (OP == OP_STORE) {
                    if (flags & TF_CODED) {
                        float *gs = (flags & TF_SCALES_PLAIN) ? reinterpret_cast<float *>(sm.desc[st].g_scales) : nullptr;
                        // a full tile of exactly one pass per thread gets a copy of the routine specialised for
                        // that size (no loop, no tail predicates): about a quarter fewer instructions
                        constexpr unsigned kOnePass = kGT * 32u;
                        if (flags & TF_INT4) {
                            if (n == kOnePass) quantise_tile<true>(A, B, Sc, gs, kOnePass, ct, kGT, P.one);
                            else quantise_tile<true>(A, B, Sc, gs, n, ct, kGT, P.one);
                        } else {
                            if (n == kOnePass) quantise_tile<false>(A, B, Sc, gs, kOnePass, ct, kGT, P.one);
                            else quantise_tile<false>(A, B, Sc, gs, n, ct, kGT, P.one);
                        }
                        computed = true;
                    }
                } else if (flags & TF_CODED) {
                    if (flags & TF_SCALES_PLAIN) {
                        const float *gs = reinterpret_cast<const float *>(sm.desc[st].g_scales);
                        for (unsigned i = (unsigned)ct; i < (sm.desc[st].sbytes >> 2); i += kGT) Sc[i] = __ldg(gs + i);
                        group_bar_sync(group, kGT);
                    }
                    if (flags & TF_KCHAN) {
                        if (OP == OP_COMPOSE && (flags & TF_ROTATE)) {
                            if (flags & TF_INT4) rotate_tile<2, true>(A, B, Sc, n, (unsigned)P.D, P.rope, sm.desc[st].rope, rc, ct, kGT, P.row_elems);
                            else rotate_tile<1, true>(A, B, Sc, n, (unsigned)P.D, P.rope, sm.desc[st].rope, rc, ct, kGT, P.row_elems);
                        } else if (flags & TF_INT4) {
                            dequantise_kc_tile<true, OP != OP_COMPOSE>(B, Sc, A, n, P.row_elems, ct, kGT);
                        } else {
                            dequantise_kc_tile<false, OP != OP_COMPOSE>(B, Sc, A, n, P.row_elems, ct, kGT);
                        }
                    } else if (OP == OP_COMPOSE && (flags & TF_ROTATE)) {
                        if (flags & TF_INT4) rotate_tile<2>(A, B, Sc, n, (unsigned)P.D, P.rope, sm.desc[st].rope, rc, ct, kGT);
                        else rotate_tile<1>(A, B, Sc, n, (unsigned)P.D, P.rope, sm.desc[st].rope, rc, ct, kGT);
                    } else if (flags & TF_INT4) {
                        if (n == kGT * 32u) dequantise4_tile(B, Sc, A, kGT * 32u, ct, kGT);
                        else dequantise4_tile(B, Sc, A, n, ct, kGT);
                    } else {
                        if (n == kGT * 32u) dequantise_tile(B, Sc, A, kGT * 32u, ct, kGT);
                        else dequantise_tile(B, Sc, A, n, ct, kGT);
                    }
                    computed = true;
                } else if (OP == OP_COMPOSE && (flags & TF_ROTATE)) {
                    rotate_tile<0>(A, nullptr, nullptr, n, (unsigned)P.D, P.rope, sm.desc[st].rope, rc, ct, kGT);
                    computed = true;
                }
            }
            // one arrival per warp and slot: "this warp's shared-memory writes are visible to the
            // bulk store, and it no longer reads the slot"
            if (computed) fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.ready + 8u * st);
            st += (unsigned)kGroups;
            if (st >= (unsigned)S) { st -= (unsigned)S; ph ^= 1u; }
        }
    }
    __syncthreads();
}

// kGroups = 0 is the pure-copy form (loader + storer only); kGroups > 0 adds that many compute groups.
// The host keeps stages a multiple of kGroups, so a pipeline slot always belongs to the same group and
// every waiter visits a barrier once per phase (a parity wait cannot tell phases two apart).
// Sec. 3.2 call (i) store, Sec. 3.1 storage module: paged pool -> chunk, optional int8 coding.
template <int kGroups, int kGW>
__global__ void __launch_bounds__(threads_for(kGroups, kGW), min_ctas_for(kGroups, kGW))
kdn_store_kernel(const __grid_constant__ Launch P) { tile_pipeline<OP_STORE, kGroups, kGW>(P); }

// Store and retrieve for launches whose tiles take up to 16 token rows (keep-lists over short rows, dense ops on very
// small pool blocks): the row indices stay in shared memory.  Built apart so that the ordinary kernels keep their registers.
template <int kGroups, int kGW>
__global__ void __launch_bounds__(threads_for(kGroups, kGW), min_ctas_for(kGroups, kGW))
kdn_store_rows_kernel(const __grid_constant__ Launch P) { tile_pipeline<OP_STORE, kGroups, kGW, true>(P); }
template <int kGroups, int kGW>
__global__ void __launch_bounds__(threads_for(kGroups, kGW), min_ctas_for(kGroups, kGW))
kdn_retrieve_rows_kernel(const __grid_constant__ Launch P) { tile_pipeline<OP_RETRIEVE, kGroups, kGW, true>(P); }

// Sec. 3.2 call (ii) retrieve, Sec. 3.1 delivery module (decompression on the GPU): chunk -> pool.
template <int kGroups, int kGW>
__global__ void __launch_bounds__(threads_for(kGroups, kGW), min_ctas_for(kGroups, kGW))
kdn_retrieve_kernel(const __grid_constant__ Launch P) { tile_pipeline<OP_RETRIEVE, kGroups, kGW>(P); }

// Sec. 3.1 blending module: parts -> request blocks at new positions, keys re-rotated.
template <int kGroups, int kGW>
__global__ void __launch_bounds__(threads_for(kGroups, kGW), min_ctas_for_compose(kGroups, kGW))
kdn_compose_kernel(const __grid_constant__ Launch P) { tile_pipeline<OP_COMPOSE, kGroups, kGW>(P); }

// ------------------------------------------------ keys of the per-channel key codecs --

// Request position of row t of group g of an op: off + 64 g + t, or, for a keep-list op, off + list[64 g + t].
// Returns -1 for a list entry that is negative or points past the block table.
__device__ __forceinline__ long long group_row_pos(const DevOp &op, unsigned g, unsigned t)
{
    const unsigned i = (g << 6) + t;
    if (op.list_mode != 1) return op.off + (long long)i;      // (a select-list chooses among the chunk's tokens, it does not move them)
    const long long rel = __ldg(op.list + i);
    const long long p = op.off + rel;
    return (rel < 0 || p >= op.pos_end) ? -1ll : p;
}


// Storing the key planes of a per-channel key codec needs, for every channel, the largest magnitude over 64 tokens
// before the first code can be formed, so it does not fit the streaming tile pipeline.  One CTA takes one
// (op, layer, 64-token group, slice of `cols` channels): the slice of the group's token rows is brought into shared
// memory with bulk copies (one per token row; one per pool block when the slice is the whole row); pass 1 reduces
// |x| per channel over four token slices; one thread per channel combines them, forms scale and reciprocal
// (two IEEE divides) and writes the scale; pass 2 codes each element with its channel's reciprocal
// and writes the codes straight to the chunk.  Several CTAs share an SM (the host picks `cols` so that they fit), so
// one CTA's loads overlap the arithmetic of the others.
// The host guarantees: block_size divides 64, the op's token offset is a multiple of block_size, row_elems % 64 == 0,
// cols % 8 == 0 and cols divides row_elems.
// Shared memory: 64 * cols * 2 (rows) + 4 * cols * 2 (slice maxima) + cols * 4 (reciprocals) + 16.
struct KcLaunch {
    const DevOp *ops;         // device array, or nullptr: inline_ops
    int n_ops;
    void *const *k_layers;
    long long n_blocks;
    int bs;
    unsigned row_elems;
    unsigned cols;            // channels per CTA
    unsigned n_split;         // row_elems / cols
    int *status;
    float one;                // 1.0f (see Launch::one)
    unsigned long long wait_limit_ns;   // the wait for the tile gives up after this long
    DevOp inline_ops[kInlineOps];
};

constexpr unsigned kKcSlices = 4;                          // token slices in pass 1 and pass 2
constexpr unsigned kKcTok = 64u / kKcSlices;              // tokens per slice
__host__ __device__ inline size_t kc_smem_bytes(unsigned cols)
{
    return (size_t)64 * cols * 2u + 16u;                   // the tile, the barrier and the abort word
}

__global__ void __launch_bounds__(512) kdn_store_kc_kernel(const __grid_constant__ KcLaunch P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const DevOp *ops = P.ops ? P.ops : P.inline_ops;
    const DevOp op = ops[blockIdx.z];
    if (op.codec < 3) return;
    const unsigned g = blockIdx.x / P.n_split, part = blockIdx.x - g * P.n_split, li = blockIdx.y;
    const unsigned n_groups = ((unsigned)op.T + 63u) >> 6;
    if (g >= n_groups || li >= (unsigned)op.nl) return;
    const bool int4 = op.codec == 4;
    const float qmax = int4 ? 7.0f : 127.0f;
    const unsigned RE = P.row_elems, C = P.cols, c0 = part * C;
    const unsigned t0 = g << 6;
    const unsigned n_tok = (unsigned)op.T - t0 < 64u ? (unsigned)op.T - t0 : 64u;

    unsigned char *X = smem_raw;                                             // [n_tok][C] bf16
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(X + (size_t)64 * C * 2u);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bar_mem + 1);
    const uint32_t bar = smem_u32(bar_mem);
    const int tid = (int)threadIdx.x;

    if (tid == 0) {
        mbar_init(bar, 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncthreads();
    if (tid < 32) {
        // warp 0 brings the rows in: lane r takes token rows r and r + 32, each found through its own table entry
        const unsigned char *base = reinterpret_cast<const unsigned char *>(P.k_layers[op.l0 + (int)li]);
        long long id[2] = { 0, 0 }, pos[2] = { 0, 0 };
        bool bad = false;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const unsigned t = (unsigned)tid + 32u * (unsigned)k;
            if (t < n_tok) {
                pos[k] = group_row_pos(op, g, t);
                if (pos[k] < 0) { bad = true; continue; }
                id[k] = __ldg(op.table + pos[k] / P.bs);
                if (id[k] < 0 || id[k] >= P.n_blocks) bad = true;
            }
        }
        if (__any_sync(0xffffffffu, bad)) {
            if (tid == 0) {
                atomicCAS(P.status, 0, kStatusRange);
                *abort_flag = 1;                                              // nothing is loaded, nothing is written
            }
        } else {
            if (tid == 0) mbar_arrive_expect_tx(bar, n_tok * C * 2u);
            __syncwarp();
            if (P.n_split == 1u && op.list_mode == 0) {
                // the whole row: a block's tokens are contiguous in the pool, one copy per block (pieces <= 32 KiB)
                if (tid == 0) {
                    const long long first_block = (op.off + (long long)t0) / P.bs;
                    for (unsigned t = 0; t < n_tok; t += (unsigned)P.bs) {
                        const unsigned k = n_tok - t < (unsigned)P.bs ? n_tok - t : (unsigned)P.bs;
                        const long long b = __ldg(op.table + first_block + t / (unsigned)P.bs);
                        const unsigned char *src = base + (unsigned long long)b * P.bs * RE * 2ull;
                        const unsigned bytes = k * RE * 2u;
                        for (unsigned o = 0; o < bytes; o += 32768u)
                            bulk_g2s(smem_u32(X + (size_t)t * RE * 2u + o), src + o, bytes - o < 32768u ? bytes - o : 32768u, bar);
                    }
                }
            } else {
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const unsigned t = (unsigned)tid + 32u * (unsigned)k;
                    if (t < n_tok) {
                        const unsigned slot = (unsigned)(pos[k] % P.bs);
                        const unsigned char *src = base + (((unsigned long long)id[k] * P.bs + slot) * RE + c0) * 2ull;
                        bulk_g2s(smem_u32(X + (size_t)t * C * 2u), src, C * 2u, bar);
                    }
                }
            }
        }
    }
    __syncthreads();
    if (*abort_flag) return;
    const bool landed = mbar_wait(bar, 0u, abort_flag, P.wait_limit_ns);
    if (!__syncthreads_and(landed)) {                                         // all threads leave together
        if (tid == 0) {
            atomicCAS(P.status, 0, kStatusTimeout);
            // one more bounded wait, so that the CTA does not leave while a copy into its shared memory is in flight
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(bar, 0u))
                if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
        return;
    }

    // From here on the warps do not meet again: a warp owns 64 channels (eight octets) for all 64 tokens, lane (j, q)
    // takes octet j of them in token quarter q.  The group's largest magnitudes meet through two shuffles, each lane
    // forms the scale and the reciprocal of two of its octet's channels, and four more shuffles hand every lane the
    // reciprocals of all eight.
    const unsigned octets = C >> 3;
    const unsigned lane = (unsigned)tid & 31u, j = lane & 7u, q = lane >> 3;
    const unsigned o = ((unsigned)tid >> 5) * 8u + j;
    const bool act = o < octets;
    const unsigned ta = q * kKcTok, tb = ta + kKcTok < n_tok ? ta + kKcTok : n_tok;
    const unsigned char *Xo = X + (size_t)o * 16u;
    // pass 1: the largest magnitudes of the lane's octet over its tokens, as packed bf16 pairs
    uint32_t m0 = 0u, m1 = 0u, m2 = 0u, m3 = 0u;
    if (act) {
        if (n_tok == 64u) {                                                   // a full group: a fixed trip count, loads batched
#pragma unroll
            for (unsigned i = 0; i < kKcTok; ++i) {
                const uint4 x = lds128(Xo + (size_t)(ta + i) * C * 2u);
                m0 = maxabs_bf16x2(m0, x.x); m1 = maxabs_bf16x2(m1, x.y);
                m2 = maxabs_bf16x2(m2, x.z); m3 = maxabs_bf16x2(m3, x.w);
            }
        } else {
            for (unsigned t = ta; t < tb; ++t) {
                const uint4 x = lds128(Xo + (size_t)t * C * 2u);
                m0 = maxabs_bf16x2(m0, x.x); m1 = maxabs_bf16x2(m1, x.y);
                m2 = maxabs_bf16x2(m2, x.z); m3 = maxabs_bf16x2(m3, x.w);
            }
        }
    }
#pragma unroll
    for (int d = 8; d <= 16; d <<= 1) {
        m0 = maxabs_bf16x2(m0, __shfl_xor_sync(0xffffffffu, m0, d)); m1 = maxabs_bf16x2(m1, __shfl_xor_sync(0xffffffffu, m1, d));
        m2 = maxabs_bf16x2(m2, __shfl_xor_sync(0xffffffffu, m2, d)); m3 = maxabs_bf16x2(m3, __shfl_xor_sync(0xffffffffu, m3, d));
    }
    // scales of channels 2q and 2q + 1 of the octet (a layer's scales start wherever the previous layer's end, so only
    // 4-byte alignment is certain: plain fp32 stores)
    const uint32_t mq = q == 0u ? m0 : q == 1u ? m1 : q == 2u ? m2 : m3;
    const float a_lo = __uint_as_float((mq & 0x7fffu) << 16), a_hi = __uint_as_float(mq & 0x7fff0000u);
    const float sc_lo = __fdiv_rn(a_lo, qmax), sc_hi = __fdiv_rn(a_hi, qmax);
    const bool ok_lo = sc_lo >= 1.17549435e-38f, ok_hi = sc_hi >= 1.17549435e-38f;   // smallest normal fp32; false for NaN too
    const float inv_lo = ok_lo ? __fdiv_rn(qmax, a_lo) : 0.0f, inv_hi = ok_hi ? __fdiv_rn(qmax, a_hi) : 0.0f;
    if (act) {
        const unsigned long long per_layer = (unsigned long long)n_groups * RE + (((unsigned long long)op.T * RE) >> 6);
        float *g_scales = reinterpret_cast<float *>(op.scales) + (unsigned long long)li * per_layer + (unsigned long long)g * RE + c0 + o * 8u + q * 2u;
        g_scales[0] = ok_lo ? sc_lo : 0.0f;
        g_scales[1] = ok_hi ? sc_hi : 0.0f;
    }
    const f32x2 i0 = pack2(__shfl_sync(0xffffffffu, inv_lo, (int)j), __shfl_sync(0xffffffffu, inv_hi, (int)j));
    const f32x2 i1 = pack2(__shfl_sync(0xffffffffu, inv_lo, (int)j + 8), __shfl_sync(0xffffffffu, inv_hi, (int)j + 8));
    const f32x2 i2 = pack2(__shfl_sync(0xffffffffu, inv_lo, (int)j + 16), __shfl_sync(0xffffffffu, inv_hi, (int)j + 16));
    const f32x2 i3 = pack2(__shfl_sync(0xffffffffu, inv_lo, (int)j + 24), __shfl_sync(0xffffffffu, inv_hi, (int)j + 24));
    if (!act) return;
    // pass 2: codes
    const float magic = 12582912.0f + (int4 ? 8.0f : 128.0f);
    const f32x2 magic2 = pack2(magic, magic);
    const f32x2 minus_m2 = pack2(-12582912.0f, -12582912.0f);
    const f32x2 k256 = pack2(256.0f, 256.0f);
    const f32x2 one2 = pack2(P.one, P.one);
    const unsigned long long plane_elem = ((unsigned long long)li * 2ull * (unsigned long long)op.T + t0) * RE + c0 + o * 8u;   // K plane, token t0
    auto code_row = [&](unsigned t) {
        const uint4 x = lds128(Xo + (size_t)t * C * 2u);
        const f32x2 r01 = add2_unfused(mul2(bf16x2_widen(x.x), i0), magic2, one2);
        const f32x2 r23 = add2_unfused(mul2(bf16x2_widen(x.y), i1), magic2, one2);
        const f32x2 r45 = add2_unfused(mul2(bf16x2_widen(x.z), i2), magic2, one2);
        const f32x2 r67 = add2_unfused(mul2(bf16x2_widen(x.w), i3), magic2, one2);
        const f32x2 ga = gather2(r01, r23, minus_m2, k256), gb = gather2(r45, r67, minus_m2, k256);
        const unsigned long long e = plane_elem + (unsigned long long)t * RE;
        if (int4)
            *reinterpret_cast<uint32_t *>(op.data + (e >> 1)) = __byte_perm(nibbles4_from(ga), nibbles4_from(gb), 0x5410) ^ 0x88888888u;
        else
            *reinterpret_cast<uint2 *>(op.data + e) = make_uint2(codes4_from(ga), codes4_from(gb));
    };
    if (n_tok == 64u) {
#pragma unroll 4
        for (unsigned i = 0; i < kKcTok; ++i) code_row(ta + i);
    } else {
        for (unsigned t = ta; t < tb; ++t) code_row(t);
    }
}

// Rotation table: row r, frequency i -> (cos, sin) of delta_r * theta_r^(-2i/D), evaluated in fp64 and
// rounded once to fp32 (an fp32 angle would lose more than half a bf16 ulp at large position shifts).
struct RopeInline { RopeParam p[kInlineOps]; };

__global__ void kdn_rope_table_kernel(const RopeParam *params, const __grid_constant__ RopeInline inl, int n_rows, int D,
                                      float2 *table)
{
    release_dependents();                                  // the compose kernel may set up and start its loads now
    if (!params) params = inl.p;                           // few rows: passed as kernel parameters
    const int half = D >> 1;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)n_rows * half) return;
    const int r = (int)(idx / half), i = (int)(idx - (long long)r * half);
    const double inv_freq = pow(params[r].theta, -2.0 * (double)i / (double)D);
    const double phi = (double)params[r].delta * inv_freq;
    double s, c;
    sincos(phi, &s, &c);
    table[idx] = make_float2((float)c, (float)s);
}

}  // namespace kdn
