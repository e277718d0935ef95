// Token-delta Rice codecs (codec ids 5 and 6): quantise-then-encode for the delivery module (paper Sec. 3.2
// "KV-cache delivery" cites a scheme that quantises a KV cache and encodes it into binary strings, and Sec. 3.1 has
// the delivery module decompress on the GPU; the bitstream itself is this library's own, see kdn.h).
//
// Every (layer, K|V, 64-token group) is a SEGMENT of row_elems channels; a channel's n <= 64 codes are one
// SUB-STREAM: zigzag of the codes (mode 0) or of their token-to-token differences (mode 1), Rice-coded with a
// parameter k, bits filling bytes from the top.  A CTA works on one slice of `cols` channels of one segment:
//   store    plan   (kdn_td_plan_kernel):   quantise, pick (mode, k) per channel, write scales / lens / params
//            scan   (kdn_td_scan_kernel):   segment sizes -> seg_off (one CTA per op)
//            encode (kdn_td_encode_kernel): quantise again, write every sub-stream at its final place
//   retrieve / compose (kdn_td_decode_kernel): bulk-copy the slice's bytes into shared memory, one thread per
//            channel undoes Rice, zigzag and the delta into a code tile, which the ordinary per-channel decoder or
//            key rotation turns into bf16 rows that bulk copies scatter to the pool blocks.
// The store reads the pool twice instead of keeping codes in scratch memory: no kernel here uses memory beyond the
// pool and the chunk.  Every wait is bounded as in the tile pipeline.
#pragma once

#include "kdn_kernels.cuh"

namespace kdn {

struct TdLaunch {
    const DevOp *ops;         // device array, or nullptr: inline_ops
    int n_ops;
    void *const *k_layers;
    void *const *v_layers;
    long long n_blocks;
    int bs;
    int D;
    int L;                    // layers of the pool = layers of every chunk
    unsigned row_elems;
    unsigned cols;            // channels per CTA
    unsigned n_split;         // row_elems / cols
    const float2 *rope;
    int *status;
    unsigned long long wait_limit_ns;   // a wait for a slice's bytes gives up after this long
    DevOp inline_ops[kInlineOps];
};

__host__ __device__ inline int td_qmax(int codec) { return codec == 5 ? 127 : 7; }
__host__ __device__ inline int td_raw_bits(int codec) { return codec == 5 ? 9 : 5; }
__host__ __device__ inline unsigned td_max_len(int codec) { return codec == 5 ? 72u : 40u; }

// Byte offsets of the regions of a chunk of T tokens (see kdn.h).
struct TdLayout {
    unsigned long long S, scales, lens, params, streams, capacity;
};
__host__ __device__ inline TdLayout td_layout(int L, unsigned row_elems, int T, int codec)
{
    TdLayout t;
    const unsigned long long G = ((unsigned long long)T + 63ull) >> 6;
    t.S = 2ull * (unsigned long long)L * G;
    t.scales = (8ull * (t.S + 1ull) + 15ull) & ~15ull;
    t.lens = t.scales + 4ull * t.S * row_elems;
    t.params = t.lens + t.S * row_elems;
    t.streams = t.params + t.S * row_elems;
    t.capacity = t.streams + t.S * (((unsigned long long)row_elems * td_max_len(codec) + 15ull) & ~15ull);
    return t;
}

// Shared memory of the store kernels: token rows, slice maxima, reciprocals, the stream staging area (encode only),
// small per-warp scratch, barrier.
// (the plan kernel keeps two tables of code-word lengths in place of the staging area, each replicated so that the
// lanes of a warp never meet in a bank: 64 entries x 32 copies x 4 bytes and 64 entries x 16 copies x 8 bytes)
// Behind the encoder's staging area: room for the longest thing a channel could write from the last planned byte on (64
// symbols of 24 bits), so that a sub-stream that came out longer than planned -- the pool changed under the store --
// garbles the chunk's bytes, which the caller has then forfeited, but never leaves the area.
constexpr unsigned kTdStageSlack = 256u;
constexpr unsigned kTdCostBytes = 64u * 32u * 4u + 64u * 16u * 8u + 64u * 4u + 64u * 8u;   // the copies, and one set of entries to copy from
__host__ __device__ inline size_t td_store_smem_bytes(unsigned cols, bool encode)
{
    return (size_t)64 * cols * 2u + (size_t)kKcSlices * cols * 2u + (size_t)cols * 4u +
           (encode ? (size_t)cols * 72u + 32u + kTdStageSlack : (size_t)kTdCostBytes) + 256u + 16u;
}
// Shared memory of the decode kernel: the slice's stream bytes as they lie in the chunk, the same sub-streams
// interleaved word by word (so that the 32 lanes of a warp read 32 different banks), codes, scales, offsets, barrier.
// The bf16 rows reuse the two stream areas once the codes are complete.
constexpr unsigned kTdWords = 19;                           // 32-bit words per interleaved sub-stream: 72 bytes, and the word after
__host__ __device__ inline size_t td_decode_packed_bytes(unsigned cols) { return ((size_t)cols * 72u + 128u + 127u) & ~(size_t)127u; }
__host__ __device__ inline size_t td_decode_front_bytes(unsigned cols)
{
    const size_t a = (size_t)64 * cols * 2u, s = td_decode_packed_bytes(cols) + (size_t)kTdWords * cols * 4u;
    return a > s ? a : s;
}
__host__ __device__ inline size_t td_decode_smem_bytes(unsigned cols)
{
    return td_decode_front_bytes(cols) + (size_t)64 * cols + (size_t)cols * 4u + 256u + 16u;
}

// Bits of one Rice code word.
__device__ __forceinline__ unsigned td_cost(unsigned u, unsigned k, unsigned esc_bits)
{
    const unsigned quo = u >> k;
    return quo < 15u ? quo + 1u + k : esc_bits;
}
__device__ __forceinline__ unsigned td_zigzag(int e) { return ((unsigned)e << 1) ^ (unsigned)(e >> 31); }   // 2e, or -2e - 1 for e < 0

// Big-endian view of a little-endian word: the stream's first byte in the top bits.
__device__ __forceinline__ uint32_t td_be(uint32_t w) { return __byte_perm(w, 0u, 0x0123); }

// round_half_even(x * inv) as the low byte of the sum with 1.5 * 2^23: two separately rounded fp32 operations.
__device__ __forceinline__ int td_code(unsigned short x_bf16, float inv)
{
    const float p = __fmul_rn(__uint_as_float((uint32_t)x_bf16 << 16), inv);
    return (int)(signed char)(__float_as_uint(__fadd_rn(p, 12582912.0f)) & 0xffu);
}

// Exclusive prefix sum of one value per thread over the block (blockDim.x a multiple of 32, at most 1024);
// *total receives the sum.  `scratch` is 33 words of shared memory.
__device__ __forceinline__ unsigned td_block_scan(unsigned v, unsigned *scratch, unsigned *total)
{
    const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    unsigned inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned o = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= (unsigned)d) inc += o;
    }
    if (lane == 31u) scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned w = lane < nwarps ? scratch[lane] : 0u, winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned o = __shfl_up_sync(0xffffffffu, winc, d);
            if (lane >= (unsigned)d) winc += o;
        }
        scratch[lane] = winc - w;
        if (lane == 31u) scratch[32] = winc;
    }
    __syncthreads();
    const unsigned r = scratch[warp] + inc - v;
    *total = scratch[32];
    __syncthreads();
    return r;
}

// First index of the increasing list whose entry is >= key (n when there is none).  At most 32 steps.
__device__ __forceinline__ unsigned td_lower_bound(const int32_t *list, unsigned n, long long key)
{
    unsigned lo = 0, hi = n;
    while (lo < hi) {
        const unsigned mid = (lo + hi) >> 1;
        if ((long long)__ldg(list + mid) < key) lo = mid + 1u; else hi = mid;
    }
    return lo;
}

// Bring the slice [c0, c0 + C) of the n_tok token rows of one group (request positions pos0 ..) of a pool plane
// into X[n_tok][C] with bulk copies counted on `bar`.  Warp 0 calls this; returns false (and records KDN_E_RANGE)
// when a block id lies outside the pool, in which case nothing was issued.
__device__ __forceinline__ bool td_load_slice(unsigned char *X, uint32_t bar, const unsigned char *base, const DevOp &op, unsigned g,
                                              unsigned n_tok, int bs, long long n_blocks, unsigned RE,
                                              unsigned C, unsigned c0, bool whole_row, int *status)
{
    const unsigned lane = threadIdx.x & 31u;
    const int32_t *table = op.table;
    long long id[2] = { 0, 0 }, pos[2] = { 0, 0 };
    bool bad = false;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const unsigned t = lane + 32u * (unsigned)k;
        if (t < n_tok) {
            pos[k] = group_row_pos(op, g, t);
            if (pos[k] < 0) { bad = true; continue; }
            id[k] = __ldg(table + pos[k] / bs);
            if (id[k] < 0 || id[k] >= n_blocks) bad = true;
        }
    }
    if (__any_sync(0xffffffffu, bad)) {
        if (lane == 0) atomicCAS(status, 0, kStatusRange);
        return false;
    }
    if (lane == 0) mbar_arrive_expect_tx(bar, n_tok * C * 2u);
    __syncwarp();
    if (whole_row && op.list_mode == 0) {
        // a block's tokens are contiguous in the pool: one copy per block (pieces <= 32 KiB); the host sees to it that
        // the group starts at a block start
        if (lane == 0) {
            const long long first_block = (op.off + (long long)(g << 6)) / bs;
            for (unsigned t = 0; t < n_tok; t += (unsigned)bs) {
                const unsigned k = n_tok - t < (unsigned)bs ? n_tok - t : (unsigned)bs;
                const long long b = __ldg(table + first_block + t / (unsigned)bs);
                const unsigned char *src = base + (unsigned long long)b * bs * RE * 2ull;
                const unsigned bytes = k * RE * 2u;
                for (unsigned o = 0; o < bytes; o += 32768u)
                    bulk_g2s(smem_u32(X + (size_t)t * RE * 2u + o), src + o, bytes - o < 32768u ? bytes - o : 32768u, bar);
            }
        }
    } else {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const unsigned t = lane + 32u * (unsigned)k;
            if (t < n_tok) {
                const unsigned slot = (unsigned)(pos[k] % bs);
                const unsigned char *src = base + (((unsigned long long)id[k] * bs + slot) * RE + c0) * 2ull;
                for (unsigned o = 0; o < C * 2u; o += 32768u)              // (a slice is at most 1024 channels: one piece)
                    bulk_g2s(smem_u32(X + (size_t)t * C * 2u + o), src + o, C * 2u - o < 32768u ? C * 2u - o : 32768u, bar);
            }
        }
    }
    return true;
}

// Per-channel reciprocal (and scale) of the slice in X: largest magnitude over the group's tokens, then the two IEEE
// divides of the codec.  All threads of the block call this; X must have landed.  g_scales may be nullptr.
__device__ __forceinline__ void td_channel_scales(const unsigned char *X, unsigned char *pmax, float *inv, float *g_scales,
                                                  unsigned n_tok, unsigned C, float qmax)
{
    const unsigned tid = threadIdx.x, nthreads = blockDim.x;
    const unsigned octets = C >> 3, items = octets * kKcSlices;
    for (unsigned it = tid; it < items; it += nthreads) {
        const unsigned q = it / octets, o = it - q * octets;
        const unsigned ta = q * kKcTok, tb = ta + kKcTok < n_tok ? ta + kKcTok : n_tok;
        uint32_t m0 = 0u, m1 = 0u, m2 = 0u, m3 = 0u;
        for (unsigned t = ta; t < tb; ++t) {
            const uint4 x = lds128(X + ((size_t)t * C + (size_t)o * 8u) * 2u);
            m0 = maxabs_bf16x2(m0, x.x); m1 = maxabs_bf16x2(m1, x.y);
            m2 = maxabs_bf16x2(m2, x.z); m3 = maxabs_bf16x2(m3, x.w);
        }
        sts128(pmax + ((size_t)q * C + (size_t)o * 8u) * 2u, make_uint4(m0, m1, m2, m3));
    }
    __syncthreads();
    for (unsigned ch = tid; ch < C; ch += nthreads) {
        unsigned short mx = 0;
        for (unsigned q = 0; q < kKcSlices; ++q) {
            const unsigned short v = *reinterpret_cast<const unsigned short *>(pmax + ((size_t)q * C + ch) * 2u) & 0x7fffu;
            mx = v > mx ? v : mx;                              // magnitudes of bf16 order like their bit patterns
        }
        const float a = __uint_as_float((uint32_t)mx << 16);
        const float sc = __fdiv_rn(a, qmax);
        const bool ok = sc >= 1.17549435e-38f;                 // smallest normal fp32; false for NaN too
        if (g_scales) g_scales[ch] = ok ? sc : 0.0f;
        inv[ch] = ok ? __fdiv_rn(qmax, a) : 0.0f;
    }
    __syncthreads();
}

struct TdSlice {              // what a CTA of the store and decode kernels works on
    DevOp op;
    unsigned g, part, plane, li, kv, n_tok, c0, seg;
    unsigned long long G;
    bool valid;
};
__device__ __forceinline__ TdSlice td_slice(const TdLaunch &P)
{
    TdSlice s;
    const DevOp *ops = P.ops ? P.ops : P.inline_ops;
    s.op = ops[blockIdx.z];
    s.g = blockIdx.x / P.n_split;
    s.part = blockIdx.x - s.g * P.n_split;
    s.plane = blockIdx.y;                                      // index into the op's layer range: li * 2 + kv
    s.li = s.plane >> 1;
    s.kv = s.plane & 1u;
    s.G = ((unsigned long long)s.op.T + 63ull) >> 6;
    s.valid = s.op.codec >= 5 && s.g < s.G && s.li < (unsigned)s.op.nl;
    const unsigned t0 = s.g << 6;
    s.n_tok = s.valid ? ((unsigned)s.op.T - t0 < 64u ? (unsigned)s.op.T - t0 : 64u) : 0u;
    s.c0 = s.part * P.cols;
    s.seg = (unsigned)(((unsigned long long)(s.op.l0 + (int)s.li) * 2ull + s.kv) * s.G + s.g);
    return s;
}

// ------------------------------------------------------------------------------------------ store: plan --

__global__ void __launch_bounds__(512) kdn_td_plan_kernel(const __grid_constant__ TdLaunch P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const TdSlice s = td_slice(P);
    if (!s.valid) return;
    const unsigned C = P.cols, RE = P.row_elems;
    const int codec = s.op.codec;
    const float qmax = (float)td_qmax(codec);
    const unsigned esc_bits = 15u + (unsigned)td_raw_bits(codec);

    unsigned char *X = smem_raw;
    unsigned char *pmax = X + (size_t)64 * C * 2u;
    float *inv = reinterpret_cast<float *>(pmax + (size_t)kKcSlices * C * 2u);
    // code-word lengths as 8-bit fields.  lo[min(u, 60)][lane]: k = 0, 1, 2 (from u = 60 on all three are the escape);
    // hi[u >> 3][lane / 2]: k = 3 .. 7 (their quotients are functions of u >> 3).  One copy per lane / pair of lanes.
    uint32_t *lo_tab = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(inv) + (size_t)C * 4u);
    uint2 *hi_tab = reinterpret_cast<uint2 *>(lo_tab + 64u * 32u);
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(reinterpret_cast<unsigned char *>(lo_tab) + (size_t)kTdCostBytes + 256u);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bar_mem + 1);
    const uint32_t bar = smem_u32(bar_mem);
    const unsigned tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(bar, 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncthreads();
    if (tid < 32) {
        const unsigned char *base = reinterpret_cast<const unsigned char *>((s.kv ? P.v_layers : P.k_layers)[s.op.l0 + (int)s.li]);
        if (!td_load_slice(X, bar, base, s.op, s.g, s.n_tok, P.bs, P.n_blocks, RE, C, s.c0,
                           P.n_split == 1u, P.status) && tid == 0)
            *abort_flag = 1;
    }
    // while the rows are on their way: fill the tables -- every entry is worked out once, then copied
    {
        uint32_t *lo_one = reinterpret_cast<uint32_t *>(hi_tab + 64u * 16u);
        uint2 *hi_one = reinterpret_cast<uint2 *>(lo_one + 64u);
        for (unsigned i = tid; i < 128u; i += blockDim.x) {
            if (i < 64u) {
                lo_one[i] = td_cost(i, 0u, esc_bits) | (td_cost(i, 1u, esc_bits) << 8) | (td_cost(i, 2u, esc_bits) << 16);
            } else {
                const unsigned u = (i - 64u) << 3;
                hi_one[i - 64u] = make_uint2(td_cost(u, 3u, esc_bits) | (td_cost(u, 4u, esc_bits) << 8) | (td_cost(u, 5u, esc_bits) << 16) |
                                             (td_cost(u, 6u, esc_bits) << 24), td_cost(u, 7u, esc_bits));
            }
        }
        __syncthreads();
        for (unsigned i = tid; i < 64u * 32u; i += blockDim.x) lo_tab[i] = lo_one[i >> 5];
        for (unsigned i = tid; i < 64u * 16u; i += blockDim.x) hi_tab[i] = hi_one[i >> 4];
    }
    __syncthreads();
    const TdLayout lay = td_layout(P.L, RE, s.op.T, codec);
    const unsigned long long row = (unsigned long long)s.seg * RE + s.c0;
    // a slice that is given up (a block id outside the pool, a wait that ran out) leaves lengths of zero behind: the scan
    // and the encoder then see a consistent, if incomplete, chunk instead of whatever the buffer held before
    auto give_up = [&]() {
        for (unsigned ch = tid; ch < C; ch += blockDim.x) {
            s.op.data[lay.lens + row + ch] = 0;
            s.op.data[lay.params + row + ch] = 0;
        }
    };
    if (*abort_flag) { give_up(); return; }
    const bool landed = mbar_wait(bar, 0u, abort_flag, P.wait_limit_ns);
    if (!__syncthreads_and(landed)) {
        if (tid == 0) {
            atomicCAS(P.status, 0, kStatusTimeout);
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(bar, 0u))
                if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
        give_up();
        return;
    }
    td_channel_scales(X, pmax, inv, reinterpret_cast<float *>(s.op.data + lay.scales) + row, s.n_tok, C, qmax);
    // one thread per channel: the cost in bits of every (mode, k), then the first minimum.  Lengths are at most 24, so
    // the 8-bit fields hold eight symbols' worth; after every eight symbols they are spread into 16-bit fields.
    for (unsigned ch = tid; ch < C; ch += blockDim.x) {
        const float iv = inv[ch];
        const uint32_t *lo_l = lo_tab + (tid & 31u);
        const uint2 *hi_l = hi_tab + ((tid & 31u) >> 1);
        unsigned w02[2] = { 0u, 0u }, w1[2] = { 0u, 0u }, w35[2] = { 0u, 0u }, w46[2] = { 0u, 0u }, w7[2] = { 0u, 0u };
        int prev = 0;
        unsigned al[2], ah[2];
        auto symbol = [&](unsigned t) {
            const int q = td_code(*reinterpret_cast<const unsigned short *>(X + ((size_t)t * C + ch) * 2u), iv);
            const unsigned u[2] = { td_zigzag(q), td_zigzag(q - prev) };        // at most 4 * 127 < 512
            prev = q;
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                al[m] += lo_l[(u[m] < 60u ? u[m] : 60u) << 5];
                const uint2 h = hi_l[(u[m] >> 3) << 4];
                ah[m] += h.x;
                w7[m] += h.y;
            }
        };
        auto widen = [&]() {
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                w02[m] += al[m] & 0x00ff00ffu; w1[m] += (al[m] >> 8) & 0x00ff00ffu;
                w35[m] += ah[m] & 0x00ff00ffu; w46[m] += (ah[m] >> 8) & 0x00ff00ffu;
            }
        };
        if (s.n_tok == 64u) {                                   // a full group: fixed trip counts, eight symbols unrolled
#pragma unroll 1
            for (unsigned t0 = 0; t0 < 64u; t0 += 8u) {
                al[0] = al[1] = ah[0] = ah[1] = 0u;
#pragma unroll
                for (unsigned k = 0; k < 8u; ++k) symbol(t0 + k);
                widen();
            }
        } else {
            for (unsigned t0 = 0; t0 < s.n_tok; t0 += 8u) {
                al[0] = al[1] = ah[0] = ah[1] = 0u;
                const unsigned t1 = t0 + 8u < s.n_tok ? t0 + 8u : s.n_tok;
                for (unsigned t = t0; t < t1; ++t) symbol(t);
                widen();
            }
        }
        const unsigned b0[8] = { w02[0] & 0xffffu, w1[0] & 0xffffu, w02[0] >> 16, w35[0] & 0xffffu, w46[0] & 0xffffu, w35[0] >> 16, w46[0] >> 16, w7[0] };
        const unsigned b1[8] = { w02[1] & 0xffffu, w1[1] & 0xffffu, w02[1] >> 16, w35[1] & 0xffffu, w46[1] & 0xffffu, w35[1] >> 16, w46[1] >> 16, w7[1] };
        unsigned best = b0[0], param = 0u;
#pragma unroll
        for (int k = 1; k < 8; ++k) if (b0[k] < best) { best = b0[k]; param = (unsigned)k; }
#pragma unroll
        for (int k = 0; k < 8; ++k) if (b1[k] < best) { best = b1[k]; param = 8u + (unsigned)k; }
        s.op.data[lay.lens + row + ch] = (unsigned char)((best + 7u) >> 3);
        s.op.data[lay.params + row + ch] = (unsigned char)param;
    }
}

// ------------------------------------------------------------------------------------------ store: scan --

// One CTA per op: seg_off[s + 1] = seg_off[s] + the segment's sub-stream bytes rounded up to 16.
__global__ void __launch_bounds__(256) kdn_td_scan_kernel(const __grid_constant__ TdLaunch P)
{
    __shared__ unsigned long long part[256];
    const DevOp *ops = P.ops ? P.ops : P.inline_ops;
    const DevOp op = ops[blockIdx.x];
    if (op.codec < 5 || op.T <= 0) return;
    const unsigned RE = P.row_elems;
    const TdLayout lay = td_layout(P.L, RE, op.T, op.codec);
    unsigned long long *seg_off = reinterpret_cast<unsigned long long *>(op.data);
    const unsigned char *lens = op.data + lay.lens;
    const unsigned tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    // phase 1: one warp per segment sums its row of lengths
    for (unsigned long long sidx = warp; sidx < lay.S; sidx += 8u) {
        const uint32_t *rowp = reinterpret_cast<const uint32_t *>(lens + sidx * RE);     // RE is a multiple of 64
        unsigned sum = 0;
        for (unsigned w = lane; w < (RE >> 2); w += 32u) {
            const uint32_t v = rowp[w];
            sum += (v & 0xffu) + ((v >> 8) & 0xffu) + ((v >> 16) & 0xffu) + (v >> 24);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
        if (lane == 0) seg_off[sidx + 1ull] = ((unsigned long long)sum + 15ull) & ~15ull;
    }
    __syncthreads();
    // phase 2: running sum over the S sizes, each thread a contiguous range
    const unsigned long long per = (lay.S + 255ull) / 256ull;
    const unsigned long long a = (unsigned long long)tid * per, b = a + per < lay.S ? a + per : lay.S;
    unsigned long long local = 0;
    for (unsigned long long i = a; i < b; ++i) local += seg_off[i + 1ull];
    part[tid] = local;
    __syncthreads();
    if (tid == 0) {
        unsigned long long run = lay.streams;
        for (int i = 0; i < 256; ++i) { const unsigned long long v = part[i]; part[i] = run; run += v; }
        seg_off[0] = lay.streams;
        if ((lay.S + 1ull) & 1ull) seg_off[lay.S + 1ull] = 0ull;             // the table is padded to 16 bytes with zeros
    }
    __syncthreads();
    unsigned long long run = part[tid];
    for (unsigned long long i = a; i < b; ++i) { run += seg_off[i + 1ull]; seg_off[i + 1ull] = run; }
}

// ---------------------------------------------------------------------------------------- store: encode --

__global__ void __launch_bounds__(512) kdn_td_encode_kernel(const __grid_constant__ TdLaunch P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const TdSlice s = td_slice(P);
    if (!s.valid) return;
    const unsigned C = P.cols, RE = P.row_elems;
    const int codec = s.op.codec;
    const float qmax = (float)td_qmax(codec);
    const unsigned raw_bits = (unsigned)td_raw_bits(codec);

    unsigned char *X = smem_raw;
    unsigned char *pmax = X + (size_t)64 * C * 2u;
    float *inv = reinterpret_cast<float *>(pmax + (size_t)kKcSlices * C * 2u);
    unsigned char *stage = reinterpret_cast<unsigned char *>(inv) + (size_t)C * 4u;          // C * 72 + 32 bytes
    unsigned *scratch = reinterpret_cast<unsigned *>(stage + (size_t)C * 72u + 32u + kTdStageSlack);   // 64 words
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(reinterpret_cast<unsigned char *>(scratch) + 256u);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bar_mem + 1);
    const uint32_t bar = smem_u32(bar_mem);
    const unsigned tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(bar, 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncthreads();
    if (tid < 32) {
        const unsigned char *base = reinterpret_cast<const unsigned char *>((s.kv ? P.v_layers : P.k_layers)[s.op.l0 + (int)s.li]);
        if (!td_load_slice(X, bar, base, s.op, s.g, s.n_tok, P.bs, P.n_blocks, RE, C, s.c0,
                           P.n_split == 1u, P.status) && tid == 0)
            *abort_flag = 1;
    }
    // meanwhile: where the slice's bytes go.  Lengths of the channels before the slice, then of the slice itself.
    const TdLayout lay = td_layout(P.L, RE, s.op.T, codec);
    const unsigned long long row = (unsigned long long)s.seg * RE;
    const unsigned char *lens = s.op.data + lay.lens + row;
    unsigned before = 0;
    for (unsigned c = tid; c < s.c0; c += blockDim.x) before += lens[c];
    unsigned total_before, total_slice;
    td_block_scan(before, scratch, &total_before);
    const unsigned my_len = tid < C ? lens[s.c0 + tid] : 0u;                                 // blockDim.x >= C
    const unsigned my_off = td_block_scan(my_len, scratch, &total_slice);
    const unsigned long long seg_begin = reinterpret_cast<const unsigned long long *>(s.op.data)[s.seg];
    unsigned char *dst = s.op.data + seg_begin + total_before;
    const unsigned shift = (unsigned)((unsigned long long)dst & 15ull);                      // staging mirrors the destination's alignment
    // the lengths are the planner's, but a planner CTA may have given up: nothing may leave the staging area or the chunk
    // (the capacity ends on a 16-byte boundary, so the padding of a segment's last slice fits whenever its bytes do)
    const bool sane = total_slice <= C * td_max_len(codec) && seg_begin >= lay.streams &&
                      seg_begin + total_before + total_slice <= lay.capacity;
    if (tid == 0 && !sane) {
        atomicCAS(P.status, 0, kStatusRange);
        *abort_flag = 1;
    }
    __syncthreads();
    if (*abort_flag) return;
    const bool landed = mbar_wait(bar, 0u, abort_flag, P.wait_limit_ns);
    if (!__syncthreads_and(landed)) {
        if (tid == 0) {
            atomicCAS(P.status, 0, kStatusTimeout);
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(bar, 0u))
                if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
        return;
    }
    // the staging area starts out as zeros: sub-streams are OR-ed into it a 32-bit word at a time, since the first and
    // the last word of a sub-stream also hold bits of its neighbours
    for (unsigned i = tid; i < (C * 72u + 32u) / 16u; i += blockDim.x) sts128(stage + (size_t)i * 16u, make_uint4(0u, 0u, 0u, 0u));
    td_channel_scales(X, pmax, inv, nullptr, s.n_tok, C, qmax);                 // (its barriers also publish the zeros)
    if (tid < C && my_len != 0u && my_len <= td_max_len(codec)) {       // (a length of zero: the planner gave this slice up)
        const unsigned param = s.op.data[lay.params + row + s.c0 + tid];
        const bool delta = (param & 8u) != 0u;
        const unsigned k = param & 7u, kmask = (1u << k) - 1u, k1 = k + 1u;
        const float iv = inv[tid];
        const uint32_t addr = smem_u32(stage) + shift + my_off;          // first byte of the sub-stream
        uint32_t wp = addr & ~3u;                                         // the word it starts in ...
        unsigned nb = (addr & 3u) * 8u;                                   // ... after this many bits that are not its own
        unsigned long long acc = 0;
        int prev = 0;
#pragma unroll 4
        for (unsigned t = 0; t < s.n_tok; ++t) {
            const int q = td_code(*reinterpret_cast<const unsigned short *>(X + ((size_t)t * C + tid) * 2u), iv);
            const unsigned u = td_zigzag(delta ? q - prev : q);
            prev = q;
            const unsigned quo = u >> k;
            unsigned w = (((1u << quo) - 1u) << k1) | (u & kmask), len = quo + k1;
            if (__builtin_expect(quo >= 15u, 0)) { w = (0x7fffu << raw_bits) | u; len = 15u + raw_bits; }
            acc = (acc << len) | w;
            nb += len;
            if (nb >= 32u) {                                              // a full word: bytes in stream order, first byte lowest
                nb -= 32u;
                const uint32_t word = td_be((uint32_t)(acc >> nb));
                asm volatile("red.shared.or.b32 [%0], %1;" :: "r"(wp), "r"(word) : "memory");
                wp += 4u;
            }
        }
        if (nb > 0u) {
            const uint32_t word = td_be((uint32_t)(acc << (32u - nb)));
            asm volatile("red.shared.or.b32 [%0], %1;" :: "r"(wp), "r"(word) : "memory");
        }
    }
    // the last slice of a segment also writes the zero bytes that pad the segment to 16
    unsigned pad = 0;
    if (s.part == P.n_split - 1u) {
        pad = (16u - ((shift + total_slice) & 15u)) & 15u;
        if (tid < pad) stage[shift + total_slice + tid] = 0;
    }
    __syncthreads();
    const unsigned n_out = total_slice + pad;
    // staging -> chunk: bytes up to the first 16-byte boundary, 16-byte words, bytes after the last boundary
    const unsigned head = shift ? (16u - shift < n_out ? 16u - shift : n_out) : 0u;
    const unsigned vecs = (n_out - head) >> 4, tail = (n_out - head) & 15u;
    if (tid < head) dst[tid] = stage[shift + tid];
    for (unsigned v = tid; v < vecs; v += blockDim.x)
        *reinterpret_cast<uint4 *>(dst + head + (size_t)v * 16u) = lds128(stage + shift + head + (size_t)v * 16u);
    if (tid < tail) dst[head + vecs * 16u + tid] = stage[shift + head + vecs * 16u + tid];
}

// ----------------------------------------------------------------------------------- retrieve / compose --


// kCols: channels per CTA when known at compile time (the usual slice; every stride in the decoding loop is then an
// immediate), 0: taken from the launch record.
template <bool kCompose, unsigned kCols>
__global__ void __launch_bounds__(kCols ? kCols : 512) kdn_td_decode_kernel(const __grid_constant__ TdLaunch P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const TdSlice s = td_slice(P);
    if (!s.valid) return;
    const unsigned C = kCols ? kCols : P.cols, RE = P.row_elems;
    const int codec = s.op.codec;
    const unsigned raw_bits = (unsigned)td_raw_bits(codec);

    unsigned char *A = smem_raw;                                         // bf16 rows; first the slice's stream bytes ...
    uint32_t *I = reinterpret_cast<uint32_t *>(A + td_decode_packed_bytes(C));   // ... and the interleaved sub-streams [word][C]
    unsigned char *B = A + td_decode_front_bytes(C);                     // codes [n_tok][C]
    float *Sc = reinterpret_cast<float *>(B + (size_t)64 * C);           // scales [C]
    unsigned *scratch = reinterpret_cast<unsigned *>(Sc + C);            // 64 words
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(reinterpret_cast<unsigned char *>(scratch) + 256u);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bar_mem + 1);
    const uint32_t bar = smem_u32(bar_mem);
    const unsigned tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(bar, 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    // a select-list (compose): which of its entries fall into this group?  Two threads look; none: nothing to do here
    const bool selecting = kCompose && s.op.list_mode == 2;
    if (selecting && tid < 2u) scratch[40u + tid] = td_lower_bound(s.op.list, (unsigned)s.op.n_list, ((long long)s.g + tid) << 6);
    const TdLayout lay = td_layout(P.L, RE, s.op.T, codec);
    const unsigned long long row = (unsigned long long)s.seg * RE;
    const unsigned char *lens = s.op.data + lay.lens + row;
    unsigned before = 0;
    for (unsigned c = tid; c < s.c0; c += blockDim.x) before += lens[c];
    unsigned total_before, total_slice;
    td_block_scan(before, scratch, &total_before);                        // (its barriers also publish the mbarrier and the two indices)
    if (selecting && scratch[40] >= scratch[41]) return;                  // every thread alike, and no copy has been started
    const unsigned my_len = tid < C ? lens[s.c0 + tid] : 0u;               // blockDim.x >= C
    const unsigned my_off = td_block_scan(my_len, scratch, &total_slice);
    unsigned param = 0;
    if (tid < C) {
        param = s.op.data[lay.params + row + s.c0 + tid];
        Sc[tid] = reinterpret_cast<const float *>(s.op.data + lay.scales)[row + s.c0 + tid];
    }
    const unsigned long long seg_begin = reinterpret_cast<const unsigned long long *>(s.op.data)[s.seg];
    const unsigned long long src = seg_begin + total_before;
    const unsigned shift = (unsigned)(((unsigned long long)s.op.data + src) & 15ull);
    const unsigned bytes_al = (shift + total_slice + 15u) & ~15u;
    // a damaged chunk must not send a copy outside the chunk or outside the staging area
    // (op.scales, which these codecs have no other use for, points behind the bytes of the chunk that exist at op.data:
    // its capacity, or what a staging slab holds of it)
    const unsigned long long exist = (unsigned long long)(s.op.scales - s.op.data);
    const unsigned long long have = exist < lay.capacity ? exist : lay.capacity;
    const bool sane = total_slice <= C * td_max_len(codec) && src >= lay.streams && src - shift + bytes_al <= have;
    if (tid == 0) {
        if (!sane) {
            atomicCAS(P.status, 0, kStatusRange);
            *abort_flag = 1;
        } else if (bytes_al != 0u) {
            mbar_arrive_expect_tx(bar, bytes_al);
            const unsigned char *g = s.op.data + src - shift;
            for (unsigned o = 0; o < bytes_al; o += 32768u)
                bulk_g2s(smem_u32(A + o), g + o, bytes_al - o < 32768u ? bytes_al - o : 32768u, bar);
        } else {
            mbar_arrive(bar);
        }
    }
    __syncthreads();
    if (*abort_flag) return;
    const bool landed = mbar_wait(bar, 0u, abort_flag, P.wait_limit_ns);
    if (!__syncthreads_and(landed)) {
        if (tid == 0) {
            atomicCAS(P.status, 0, kStatusTimeout);
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(bar, 0u))
                if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
        return;
    }
    // one thread per channel: Rice, zigzag, delta -> codes
    if (tid < C) {
        const unsigned k = param & 7u;
        // the sub-stream, as big-endian words, into column tid of the interleaved area: word j of every channel sits in
        // one row, so a warp's loads below never meet in a bank wherever each lane is in its stream
        {
            const uint32_t addr = smem_u32(A) + shift + my_off;
            const uint32_t al = addr & ~3u;
            const unsigned sh8 = (addr & 3u) * 8u;
            // (a length no sub-stream can have means a damaged chunk: reported, and clamped so that nothing leaves the area)
            if (my_len > td_max_len(codec)) atomicCAS(P.status, 0, kStatusRange);
            const unsigned len_c = my_len < td_max_len(codec) ? my_len : td_max_len(codec);
            const unsigned nw = ((len_c + 3u) >> 2) + 1u;                 // the window below looks one word past the last bit
            uint32_t x0, x1;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x0) : "r"(al));
            for (unsigned j = 0; j < nw; ++j) {
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x1) : "r"(al + 4u * (j + 1u)));
                I[(size_t)j * C + tid] = td_be(__funnelshift_r(x0, x1, sh8));
                x0 = x1;
            }
        }
        // 32-bit shared addresses throughout: column tid of the interleaved words, column tid of the code tile
        const uint32_t col = smem_u32(I) + tid * 4u, row_b = C * 4u;
        uint32_t out = smem_u32(B) + tid;
        const unsigned k1 = k + 1u, kpow = 1u << k, krem = 32u - k;
        const bool delta = (param & 8u) != 0u;
        unsigned bp = 0;                                                  // bits consumed so far
        int prev = 0;
#pragma unroll 4
        for (unsigned t = 0; t < s.n_tok; ++t) {
            const unsigned wi = (bp >> 5) < kTdWords - 2u ? (bp >> 5) : kTdWords - 2u;   // a damaged stream cannot run off the area
            const uint32_t a = col + wi * row_b;
            uint32_t w0, w1;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w0) : "r"(a));
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w1) : "r"(a + row_b));
            const uint32_t hi = __funnelshift_l(w1, w0, bp);             // the next 32 bits of the stream
            const unsigned ones = (unsigned)__clz((int)~hi);
            // quo ones, a zero, k bits: the k bits are the top of hi << (ones + 1); a shift by 32 (k = 0) gives 0 in PTX
            unsigned rem;
            asm("shr.b32 %0, %1, %2;" : "=r"(rem) : "r"(hi << (ones + 1u)), "r"(krem));
            unsigned u = ones * kpow + rem;
            unsigned len = ones + k1;
            if (__builtin_expect(ones >= 15u, 0)) { u = (hi << 15) >> (32u - raw_bits); len = 15u + raw_bits; }   // the escape: rare
            bp += len;
            int sgn;
            asm("bfe.s32 %0, %1, 0, 1;" : "=r"(sgn) : "r"(u));           // -(u & 1)
            int q = (int)(u >> 1) ^ sgn;
            if (delta) q += prev;
            prev = q;
            asm volatile("st.shared.u8 [%0], %1;" :: "r"(out), "r"(q) : "memory");
            out += C;
        }
    }
    __syncthreads();                                                      // codes complete, stream bytes no longer read
    const unsigned n = s.n_tok * C;
    if (kCompose && s.kv == 0u && s.op.rope >= 0) {
        RotCoef rc;
        rc.rope = -1; rc.col = 0xffffffffu;
        rotate_tile<1, true>(A, B, Sc, n, (unsigned)P.D, P.rope, s.op.rope, rc, (int)tid, blockDim.x, C);
    } else {
        dequantise_kc_tile<false, !kCompose>(B, Sc, A, n, C, (int)tid, blockDim.x);
    }
    fence_async_smem();
    __syncthreads();
    // rows -> pool blocks
    if (tid < 32) {
        unsigned char *base = reinterpret_cast<unsigned char *>((s.kv ? P.v_layers : P.k_layers)[s.op.l0 + (int)s.li]);
        long long id[2] = { 0, 0 }, pos[2] = { 0, 0 };
        unsigned row_t[2] = { tid, tid + 32u };                       // which row of the group lane k writes (64: none)
        bool bad = false;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            if (selecting) {
                // the group's listed tokens, at most 64 of them: lane k takes entry first + tid + 32 k (the two indices
                // still sit where the search left them: the scans use the words below)
                const unsigned idx = scratch[40] + tid + 32u * (unsigned)k;
                row_t[k] = 64u;
                if (idx < scratch[41]) {
                    const long long c = (long long)__ldg(s.op.list + idx) - ((long long)s.g << 6);
                    if (c < 0 || c >= (long long)s.n_tok) bad = true;      // (a list that is not increasing)
                    else row_t[k] = (unsigned)c;
                }
            } else if (row_t[k] >= s.n_tok) {
                row_t[k] = 64u;
            }
            if (row_t[k] < 64u) {
                pos[k] = group_row_pos(s.op, s.g, row_t[k]);
                if (pos[k] < 0) { bad = true; continue; }
                id[k] = __ldg(s.op.table + pos[k] / P.bs);
                if (id[k] < 0 || id[k] >= P.n_blocks) bad = true;
            }
        }
        if (__any_sync(0xffffffffu, bad)) {
            if (tid == 0) atomicCAS(P.status, 0, kStatusRange);        // nothing of this slice is written
        } else {
            if (P.n_split == 1u && s.op.list_mode == 0) {
                if (tid == 0) {
                    const long long first_block = (s.op.off + (long long)(s.g << 6)) / P.bs;
                    for (unsigned t = 0; t < s.n_tok; t += (unsigned)P.bs) {
                        const unsigned k = s.n_tok - t < (unsigned)P.bs ? s.n_tok - t : (unsigned)P.bs;
                        const long long b = __ldg(s.op.table + first_block + t / (unsigned)P.bs);
                        unsigned char *d = base + (unsigned long long)b * P.bs * RE * 2ull;
                        const unsigned bytes = k * RE * 2u;
                        for (unsigned o = 0; o < bytes; o += 32768u)
                            bulk_s2g(d + o, smem_u32(A + (size_t)t * RE * 2u + o), bytes - o < 32768u ? bytes - o : 32768u);
                    }
                }
            } else {
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const unsigned t = row_t[k];
                    if (t < 64u) {
                        const unsigned slot = (unsigned)(pos[k] % P.bs);
                        unsigned char *d = base + (((unsigned long long)id[k] * P.bs + slot) * RE + s.c0) * 2ull;
                        bulk_s2g(d, smem_u32(A + (size_t)t * C * 2u), C * 2u);
                    }
                }
            }
            bulk_commit();
            bulk_wait_all();
        }
    }
}

}  // namespace kdn
