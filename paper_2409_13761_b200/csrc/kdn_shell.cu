// Storage-module shell of libkdn (paper Sec. 3.1: the storage module keeps KV caches under keys derived from
// their texts; Sec. 3.2: the engine hands over a KV cache together with its text and later asks for it by text).
// Host side: key hash, self-describing chunk header, and an index from key to chunk with least-recently-used
// eviction under a byte budget.  Device side: one kernel, the payload checksum.
#include "kdn.h"

#include <cuda_runtime.h>

#include <cstring>
#include <list>
#include <new>
#include <unordered_map>

namespace {

constexpr unsigned kChecksumXor = 0x9E3779B9u;
constexpr int kChecksumThreads = 256;

// checksum = sum_i ((w_i ^ 0x9E3779B9) * ((2 i + 1) mod 2^32)) mod 2^64 over 32-bit little-endian words.  The sum is
// commutative, so every thread accumulates its own words (one XOR and one 32x32+64 multiply-add each), a warp is
// reduced with shuffles and one 64-bit atomic per warp lands in *out.
__global__ void __launch_bounds__(kChecksumThreads)
kdn_checksum_kernel(const unsigned *__restrict__ words, unsigned long long n_words, unsigned first_index,
                    unsigned long long *out)
{
    unsigned long long acc = 0;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long n_vec = n_words >> 2;
    const bool aligned = ((unsigned long long)(size_t)words & 15ull) == 0ull;
    if (aligned) {
        const uint4 *v4 = reinterpret_cast<const uint4 *>(words);
        unsigned long long v = tid;
        // four independent 128-bit loads in flight per thread
        for (; v + 3ull * stride < n_vec; v += 4ull * stride) {
            uint4 x[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) x[k] = __ldcs(v4 + v + (unsigned long long)k * stride);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned i0 = first_index + (unsigned)((v + (unsigned long long)k * stride) << 2);      // word index mod 2^32
                acc += (unsigned long long)(x[k].x ^ kChecksumXor) * (unsigned long long)(2u * i0 + 1u);
                acc += (unsigned long long)(x[k].y ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 1u) + 1u);
                acc += (unsigned long long)(x[k].z ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 2u) + 1u);
                acc += (unsigned long long)(x[k].w ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 3u) + 1u);
            }
        }
        for (; v < n_vec; v += stride) {
            const uint4 x = __ldcs(v4 + v);
            const unsigned i0 = first_index + (unsigned)(v << 2);
            acc += (unsigned long long)(x.x ^ kChecksumXor) * (unsigned long long)(2u * i0 + 1u);
            acc += (unsigned long long)(x.y ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 1u) + 1u);
            acc += (unsigned long long)(x.z ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 2u) + 1u);
            acc += (unsigned long long)(x.w ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 3u) + 1u);
        }
        for (unsigned long long i = (n_vec << 2) + tid; i < n_words; i += stride)                  // up to 3 tail words
            acc += (unsigned long long)(words[i] ^ kChecksumXor) * (unsigned long long)(2u * (first_index + (unsigned)i) + 1u);
    } else {
        for (unsigned long long i = tid; i < n_words; i += stride)
            acc += (unsigned long long)(words[i] ^ kChecksumXor) * (unsigned long long)(2u * (first_index + (unsigned)i) + 1u);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if ((threadIdx.x & 31) == 0 && acc != 0ull) atomicAdd(out, acc);
}

// Minimal mbarrier / bulk-copy wrappers for the kernel below (this file is its own translation unit).
__device__ __forceinline__ uint32_t cs_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cs_mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void cs_mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cs_mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded, parked wait (2 s): false when it gave up or another thread of the CTA did.
__device__ __forceinline__ bool cs_mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    unsigned long long t0 = 0;
    for (uint32_t n = 0;; ++n) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
        if (ok) return true;
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        if (n == 0) t0 = t;
        if (*abort_flag) return false;
        if (t - t0 > 2000000000ull) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ void cs_bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// The same sum for 16-byte aligned payloads, fed by bulk async copies: one thread per CTA streams 16 KiB pieces into
// a ring of shared-memory slots (a read-only stream through the copy engine path reaches ~7 TB/s on B200, the plain
// 128-bit loads above ~6.3), eight warps add them up.  Piece g belongs to CTA g % gridDim.x.
constexpr int kCsTile = 16384;
constexpr int kCsStages = 6;
constexpr int kCsWarps = 8;
constexpr int kCsThreads = 32 + kCsWarps * 32;

__global__ void __launch_bounds__(kCsThreads)
kdn_checksum_bulk_kernel(const unsigned char *__restrict__ payload, unsigned long long n_pieces, unsigned tail_bytes,
                         unsigned long long *out)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[2 * kCsStages];
    __shared__ volatile int abort_flag;
    const int tid = (int)threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t full = cs_smem_u32(bars), empty = full + 8u * kCsStages;
    if (tid == 0) {
        for (int s = 0; s < kCsStages; ++s) { cs_mbar_init(full + 8u * s, 1u); cs_mbar_init(empty + 8u * s, (uint32_t)kCsWarps); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const unsigned long long bid = blockIdx.x, grid = gridDim.x;
    const unsigned long long n_my = n_pieces > bid ? (n_pieces - bid + grid - 1ull) / grid : 0ull;
    if (warp == 0) {
        if (lane == 0) {
            for (unsigned long long i = 0; i < n_my; ++i) {
                const unsigned st = (unsigned)(i % kCsStages);
                if (!cs_mbar_wait(empty + 8u * st, (uint32_t)((i / kCsStages) & 1ull) ^ 1u, &abort_flag)) break;
                const unsigned long long g = bid + i * grid;
                const unsigned bytes = (g == n_pieces - 1ull && tail_bytes) ? tail_bytes : (unsigned)kCsTile;
                cs_mbar_arrive_expect_tx(full + 8u * st, bytes);
                cs_bulk_g2s(cs_smem_u32(smem + (size_t)st * kCsTile), payload + g * (unsigned long long)kCsTile, bytes, full + 8u * st);
            }
        }
    } else {
        const unsigned ct = (unsigned)tid - 32u;
        unsigned long long acc = 0;
        for (unsigned long long i = 0; i < n_my; ++i) {
            const unsigned st = (unsigned)(i % kCsStages);
            if (!cs_mbar_wait(full + 8u * st, (uint32_t)((i / kCsStages) & 1ull), &abort_flag)) break;
            const unsigned long long g = bid + i * grid;
            const unsigned bytes = (g == n_pieces - 1ull && tail_bytes) ? tail_bytes : (unsigned)kCsTile;
            const uint4 *v4 = reinterpret_cast<const uint4 *>(smem + (size_t)st * kCsTile);
            const unsigned w0 = (unsigned)(g * (unsigned long long)(kCsTile / 4));             // word index mod 2^32
            for (unsigned v = ct; v < (bytes >> 4); v += (unsigned)kCsWarps * 32u) {
                const uint4 x = v4[v];
                const unsigned i0 = w0 + (v << 2);
                acc += (unsigned long long)(x.x ^ kChecksumXor) * (unsigned long long)(2u * i0 + 1u);
                acc += (unsigned long long)(x.y ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 1u) + 1u);
                acc += (unsigned long long)(x.z ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 2u) + 1u);
                acc += (unsigned long long)(x.w ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 3u) + 1u);
            }
            __syncwarp();
            if (lane == 0) cs_mbar_arrive(empty + 8u * st);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0 && acc != 0ull) atomicAdd(out, acc);
    }
    __syncthreads();
}

const char kMagic[8] = { 'K', 'D', 'N', 'C', 'H', 'N', 'K', '1' };

struct Entry {
    kdn_chunk chunk;
    std::list<uint64_t>::iterator lru;      // position in the recency list (front = most recent)
};

}  // namespace

struct kdn_index {
    size_t capacity = 0;
    size_t bytes = 0;
    uint64_t hits = 0, misses = 0, evictions = 0;
    std::unordered_map<uint64_t, Entry> map;
    std::list<uint64_t> order;
};

extern "C" {

uint64_t kdn_key_hash(const int32_t *token_ids, size_t n)
{
    uint64_t h = 0xcbf29ce484222325ull;                           // FNV-1a, 64 bit, over little-endian token ids
    for (size_t i = 0; i < n; ++i) {
        const uint32_t t = (uint32_t)token_ids[i];
        for (int b = 0; b < 4; ++b) {
            h ^= (t >> (8 * b)) & 0xffu;
            h *= 0x100000001b3ull;
        }
    }
    return h;
}

kdn_status kdn_checksum(int device, const void *payload, size_t bytes, uint64_t *device_out, void *cuda_stream)
{
    if (!device_out || (bytes > 0 && !payload)) return KDN_E_INVAL;
    if (bytes % 4 || (uintptr_t)payload % 4 || (uintptr_t)device_out % 8) return KDN_E_ALIGN;
    if (cudaSetDevice(device) != cudaSuccess) return KDN_E_CUDA;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(device_out, 0, sizeof(uint64_t), stream) != cudaSuccess) return KDN_E_CUDA;
    if (bytes == 0) return KDN_OK;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return KDN_E_CUDA;
    unsigned first_index = 0;
    if ((uintptr_t)payload % 16 == 0 && bytes >= (size_t)kCsTile * 64u) {
        // bulk-copy form over the whole 16-byte units; the 4..12 bytes that may remain go to the plain kernel
        const size_t body = bytes & ~(size_t)15;
        const unsigned long long n_pieces = (body + kCsTile - 1) / kCsTile;
        const unsigned tail = (unsigned)(body % kCsTile);
        const unsigned long long cap2 = (unsigned long long)sms * 2ull;
        const unsigned grid2 = (unsigned)(n_pieces < cap2 ? n_pieces : cap2);
        const size_t smem = (size_t)kCsStages * kCsTile;
        if (cudaFuncSetAttribute(kdn_checksum_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return KDN_E_CUDA;
        kdn_checksum_bulk_kernel<<<grid2, kCsThreads, smem, stream>>>((const unsigned char *)payload, n_pieces, tail,
                                                                      (unsigned long long *)device_out);
        if (cudaGetLastError() != cudaSuccess) return KDN_E_CUDA;
        if (body == bytes) return KDN_OK;
        payload = (const unsigned char *)payload + body;
        bytes -= body;
        first_index = (unsigned)(body / 4);
    }
    const unsigned long long n_words = bytes / 4;
    unsigned long long want = (n_words / 4 + kChecksumThreads - 1) / kChecksumThreads;
    if (want < 1) want = 1;
    const unsigned long long cap = (unsigned long long)sms * 8ull;     // 8 resident CTAs of 256 threads per SM
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    kdn_checksum_kernel<<<grid, kChecksumThreads, 0, stream>>>((const unsigned *)payload, n_words, first_index,
                                                               (unsigned long long *)device_out);
    return cudaGetLastError() == cudaSuccess ? KDN_OK : KDN_E_CUDA;
}

kdn_status kdn_header_fill(const kdn_pool_desc *pool, const kdn_chunk *chunk, uint64_t key, uint64_t checksum,
                           kdn_chunk_header *out)
{
    if (!pool || !chunk || !out) return KDN_E_INVAL;
    if (chunk->n_tokens < 0) return KDN_E_INVAL;
    const size_t want = kdn_chunk_bytes(pool, chunk->n_tokens, chunk->codec);
    if ((want == 0 && chunk->n_tokens > 0) || want != chunk->bytes) return KDN_E_SHAPE;
    std::memset(out, 0, sizeof *out);
    std::memcpy(out->magic, kMagic, 8);
    out->header_bytes = (uint32_t)sizeof *out;
    out->codec = (uint32_t)chunk->codec;
    out->n_layers = pool->n_layers;
    out->n_kv_heads = pool->n_kv_heads;
    out->head_dim = pool->head_dim;
    out->n_tokens = chunk->n_tokens;
    out->base_pos = chunk->base_pos;
    out->payload_bytes = chunk->bytes;
    out->key = key;
    out->checksum = checksum;
    return KDN_OK;
}

kdn_status kdn_header_check(const kdn_pool_desc *pool, const kdn_chunk_header *h, uint64_t checksum_of_payload,
                            kdn_chunk *out)
{
    if (!pool || !h) return KDN_E_INVAL;
    if (std::memcmp(h->magic, kMagic, 8) != 0 || h->header_bytes != sizeof *h) return KDN_E_INVAL;
    if (h->n_layers != pool->n_layers || h->n_kv_heads != pool->n_kv_heads || h->head_dim != pool->head_dim) return KDN_E_SHAPE;
    if (h->n_tokens < 0) return KDN_E_SHAPE;
    const size_t want = kdn_chunk_bytes(pool, h->n_tokens, (int32_t)h->codec);
    if ((want == 0 && h->n_tokens > 0) || want != h->payload_bytes) return KDN_E_SHAPE;
    if (h->checksum != checksum_of_payload) return KDN_E_CHECKSUM;
    if (out) {
        out->bytes = (size_t)h->payload_bytes;
        out->n_tokens = h->n_tokens;
        out->codec = (int32_t)h->codec;
        out->base_pos = h->base_pos;
    }
    return KDN_OK;
}

kdn_status kdn_index_create(kdn_index **out, size_t capacity_bytes)
{
    if (!out) return KDN_E_INVAL;
    *out = new (std::nothrow) kdn_index();
    if (!*out) return KDN_E_NOMEM;
    (*out)->capacity = capacity_bytes;
    return KDN_OK;
}

void kdn_index_destroy(kdn_index *idx) { delete idx; }

kdn_status kdn_index_put(kdn_index *idx, uint64_t key, const kdn_chunk *chunk, kdn_chunk *evicted, int max_evicted,
                         int *n_evicted)
{
    if (!idx || !chunk || max_evicted < 0 || (max_evicted > 0 && !evicted)) return KDN_E_INVAL;
    if (n_evicted) *n_evicted = 0;
    if (chunk->bytes > idx->capacity) return KDN_E_NOMEM;
    auto found = idx->map.find(key);
    const size_t replaced = found != idx->map.end() ? found->second.chunk.bytes : 0;
    // how many least-recently-used entries (other than `key`) must go?
    size_t bytes = idx->bytes - replaced + chunk->bytes;
    int need = 0;
    for (auto it = idx->order.rbegin(); bytes > idx->capacity && it != idx->order.rend(); ++it) {
        if (*it == key) continue;
        bytes -= idx->map[*it].chunk.bytes;
        ++need;
    }
    if (bytes > idx->capacity || need + (replaced ? 1 : 0) > max_evicted) return KDN_E_NOMEM;   // nothing was changed
    int n = 0;
    if (found != idx->map.end()) {                               // the replaced chunk is handed back first
        evicted[n++] = found->second.chunk;
        idx->order.erase(found->second.lru);
        idx->bytes -= replaced;
        idx->map.erase(found);
    }
    while (idx->bytes + chunk->bytes > idx->capacity) {
        const uint64_t victim = idx->order.back();
        auto v = idx->map.find(victim);
        evicted[n++] = v->second.chunk;
        idx->bytes -= v->second.chunk.bytes;
        idx->order.pop_back();
        idx->map.erase(v);
        idx->evictions++;
    }
    idx->order.push_front(key);
    idx->map[key] = Entry{ *chunk, idx->order.begin() };
    idx->bytes += chunk->bytes;
    if (n_evicted) *n_evicted = n;
    return KDN_OK;
}

kdn_status kdn_index_get(kdn_index *idx, uint64_t key, kdn_chunk *out)
{
    if (!idx) return KDN_E_INVAL;
    auto it = idx->map.find(key);
    if (it == idx->map.end()) { idx->misses++; return KDN_E_NOTFOUND; }
    idx->hits++;
    idx->order.splice(idx->order.begin(), idx->order, it->second.lru);     // most recently used
    if (out) *out = it->second.chunk;
    return KDN_OK;
}

kdn_status kdn_index_remove(kdn_index *idx, uint64_t key, kdn_chunk *out)
{
    if (!idx) return KDN_E_INVAL;
    auto it = idx->map.find(key);
    if (it == idx->map.end()) return KDN_E_NOTFOUND;
    if (out) *out = it->second.chunk;
    idx->bytes -= it->second.chunk.bytes;
    idx->order.erase(it->second.lru);
    idx->map.erase(it);
    return KDN_OK;
}

void kdn_index_stats(const kdn_index *idx, kdn_index_info *out)
{
    if (!out) return;
    std::memset(out, 0, sizeof *out);
    if (!idx) return;
    out->capacity_bytes = idx->capacity;
    out->bytes = idx->bytes;
    out->entries = idx->map.size();
    out->hits = idx->hits;
    out->misses = idx->misses;
    out->evictions = idx->evictions;
}

}  // extern "C"
