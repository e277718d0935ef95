// Storage-module shell of libkdn (paper Sec. 3.1: the storage module keeps KV caches "keyed by various texts";
// Sec. 3.2: the engine stores a KV cache "with the associated text" and retrieves it "using some text").
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
kdn_checksum_kernel(const unsigned *__restrict__ words, unsigned long long n_words, unsigned long long *out)
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
                const unsigned i0 = (unsigned)((v + (unsigned long long)k * stride) << 2);      // word index mod 2^32
                acc += (unsigned long long)(x[k].x ^ kChecksumXor) * (unsigned long long)(2u * i0 + 1u);
                acc += (unsigned long long)(x[k].y ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 1u) + 1u);
                acc += (unsigned long long)(x[k].z ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 2u) + 1u);
                acc += (unsigned long long)(x[k].w ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 3u) + 1u);
            }
        }
        for (; v < n_vec; v += stride) {
            const uint4 x = __ldcs(v4 + v);
            const unsigned i0 = (unsigned)(v << 2);
            acc += (unsigned long long)(x.x ^ kChecksumXor) * (unsigned long long)(2u * i0 + 1u);
            acc += (unsigned long long)(x.y ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 1u) + 1u);
            acc += (unsigned long long)(x.z ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 2u) + 1u);
            acc += (unsigned long long)(x.w ^ kChecksumXor) * (unsigned long long)(2u * (i0 + 3u) + 1u);
        }
        for (unsigned long long i = (n_vec << 2) + tid; i < n_words; i += stride)                  // up to 3 tail words
            acc += (unsigned long long)(words[i] ^ kChecksumXor) * (unsigned long long)(2u * (unsigned)i + 1u);
    } else {
        for (unsigned long long i = tid; i < n_words; i += stride)
            acc += (unsigned long long)(words[i] ^ kChecksumXor) * (unsigned long long)(2u * (unsigned)i + 1u);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if ((threadIdx.x & 31) == 0 && acc != 0ull) atomicAdd(out, acc);
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
    const unsigned long long n_words = bytes / 4;
    unsigned long long want = (n_words / 4 + kChecksumThreads - 1) / kChecksumThreads;
    if (want < 1) want = 1;
    const unsigned long long cap = (unsigned long long)sms * 8ull;     // 8 resident CTAs of 256 threads per SM
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    kdn_checksum_kernel<<<grid, kChecksumThreads, 0, stream>>>((const unsigned *)payload, n_words,
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
