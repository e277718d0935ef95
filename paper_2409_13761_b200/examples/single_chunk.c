/*
 * single_chunk.c -- libkdn from plain C: retrieve one stored chunk into a request's blocks, the call a serving
 * engine makes once per request (paper Sec. 3.2, the retrieve call of the interface with serving engines), and what
 * that call costs on the host and on the device.
 *
 *   gcc -std=c99 -O2 -I include -I $CUDA/include single_chunk.c -L <dir of libkdn.so> -lkdn -L $CUDA/lib64 -lcudart
 *
 * Llama-3-8B-shaped KV (32 layers, 8 KV heads, head_dim 128, block_size 16), one raw bf16 chunk of 512 tokens
 * (64 MiB), a pool of 256 blocks.  Checks the scattered bytes against the chunk by the layout's definition, then
 * times 200 back-to-back calls: host time per call (how long kdn_retrieve takes to return) and device time per call
 * (CUDA events around the batch).  Prints one line: ok host_us=... device_us=... gbs=...
 */
#define _POSIX_C_SOURCE 199309L
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

#include <cuda_runtime_api.h>

#include "kdn.h"

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 2; } } while (0)
#define CHECK_KDN(x) do { kdn_status s_ = (x); if (s_ != KDN_OK) { fprintf(stderr, "%s: %s\n", #x, kdn_strerror(s_)); return 3; } } while (0)

enum { L = 32, H = 8, D = 128, BS = 16, NB = 256, T = 512, CALLS = 200 };

static double now_us(void)
{
    struct timespec ts;
    clock_gettime(CLOCK_MONOTONIC, &ts);
    return ts.tv_sec * 1e6 + ts.tv_nsec * 1e-3;
}

int main(void)
{
    const size_t row = (size_t)H * D * 2;                     /* bytes of one token row of one plane */
    const size_t plane_bytes = (size_t)NB * BS * row;
    void *k_layers[L], *v_layers[L];
    int l, i;
    CHECK_CUDA(cudaSetDevice(0));
    for (l = 0; l < L; ++l) {
        CHECK_CUDA(cudaMalloc(&k_layers[l], plane_bytes));
        CHECK_CUDA(cudaMalloc(&v_layers[l], plane_bytes));
        CHECK_CUDA(cudaMemset(k_layers[l], 0, plane_bytes));
        CHECK_CUDA(cudaMemset(v_layers[l], 0, plane_bytes));
    }
    kdn_pool_desc pool;
    memset(&pool, 0, sizeof pool);
    pool.n_layers = L; pool.n_kv_heads = H; pool.head_dim = D; pool.block_size = BS; pool.n_blocks = NB;
    pool.k_layers = k_layers; pool.v_layers = v_layers;

    kdn_ctx *ctx = NULL;
    int pool_id = -1;
    CHECK_KDN(kdn_create(&ctx, 0));
    CHECK_KDN(kdn_pool_register(ctx, &pool, &pool_id));

    /* the chunk: bytes with a position-dependent pattern */
    const size_t chunk_bytes = kdn_chunk_bytes(&pool, T, KDN_CODEC_RAW_BF16);
    unsigned char *h_chunk = (unsigned char *)malloc(chunk_bytes);
    if (!h_chunk || chunk_bytes != (size_t)L * 2 * T * row) { fprintf(stderr, "chunk size\n"); return 4; }
    for (size_t b = 0; b < chunk_bytes; ++b) h_chunk[b] = (unsigned char)((b * 2654435761u) >> 24);
    void *d_chunk = NULL;
    CHECK_CUDA(cudaMalloc(&d_chunk, chunk_bytes));
    CHECK_CUDA(cudaMemcpy(d_chunk, h_chunk, chunk_bytes, cudaMemcpyHostToDevice));

    /* the request's block table: 32 scattered blocks */
    int32_t h_table[T / BS];
    for (i = 0; i < T / BS; ++i) h_table[i] = (i * 37 + 11) % NB;
    int32_t *d_table = NULL;
    CHECK_CUDA(cudaMalloc((void **)&d_table, sizeof h_table));
    CHECK_CUDA(cudaMemcpy(d_table, h_table, sizeof h_table, cudaMemcpyHostToDevice));

    cudaStream_t stream;
    CHECK_CUDA(cudaStreamCreateWithFlags(&stream, cudaStreamNonBlocking));

    kdn_xfer_op op;
    memset(&op, 0, sizeof op);
    op.block_table = d_table;
    op.n_table_blocks = T / BS;
    op.token_offset = 0;
    op.chunk.data = d_chunk;
    op.chunk.bytes = chunk_bytes;
    op.chunk.n_tokens = T;
    op.chunk.codec = KDN_CODEC_RAW_BF16;
    op.chunk.mem = KDN_MEM_DEVICE;

    CHECK_KDN(kdn_retrieve(ctx, pool_id, &op, 1, stream, NULL));
    CHECK_KDN(kdn_status_sync(ctx, stream));

    /* check: block j of plane (l, kv) holds chunk tokens 16 j .. 16 j + 15, which are contiguous in the chunk */
    unsigned char *h_block = (unsigned char *)malloc((size_t)BS * row);
    if (!h_block) return 4;
    for (l = 0; l < L; l += 7) {
        int kv, j;
        for (kv = 0; kv < 2; ++kv)
            for (j = 0; j < T / BS; j += 5) {
                const unsigned char *plane = (const unsigned char *)(kv ? v_layers[l] : k_layers[l]);
                CHECK_CUDA(cudaMemcpy(h_block, plane + (size_t)h_table[j] * BS * row, (size_t)BS * row, cudaMemcpyDeviceToHost));
                if (memcmp(h_block, h_chunk + (((size_t)l * 2 + kv) * T + (size_t)j * BS) * row, (size_t)BS * row)) {
                    fprintf(stderr, "mismatch at layer %d kv %d block %d\n", l, kv, j);
                    return 5;
                }
            }
    }

    /* timing */
    for (i = 0; i < 10; ++i) CHECK_KDN(kdn_retrieve(ctx, pool_id, &op, 1, stream, NULL));
    CHECK_CUDA(cudaStreamSynchronize(stream));
    cudaEvent_t a, b;
    CHECK_CUDA(cudaEventCreate(&a));
    CHECK_CUDA(cudaEventCreate(&b));
    CHECK_CUDA(cudaEventRecord(a, stream));
    const double t0 = now_us();
    for (i = 0; i < CALLS; ++i) CHECK_KDN(kdn_retrieve(ctx, pool_id, &op, 1, stream, NULL));
    const double host_us = (now_us() - t0) / CALLS;
    CHECK_CUDA(cudaEventRecord(b, stream));
    CHECK_CUDA(cudaStreamSynchronize(stream));
    float ms = 0.0f;
    CHECK_CUDA(cudaEventElapsedTime(&ms, a, b));
    CHECK_KDN(kdn_status_sync(ctx, stream));
    const double device_us = ms * 1e3 / CALLS;
    printf("ok host_us=%.2f device_us=%.2f gbs=%.1f\n", host_us, device_us, 2.0 * (double)chunk_bytes / device_us / 1e3);

    kdn_destroy(ctx);
    return 0;
}
