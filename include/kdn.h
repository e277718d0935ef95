/*
 * kdn.h -- C ABI of libkdn: the data-movement hot path of a Knowledge Delivery
 * Network (KDN) on one NVIDIA B200 (sm_100a).
 *
 * A KDN keeps precomputed KV caches apart from the serving engine and hands
 * them back on demand (paper Sec. 3.1: storage, delivery and blending
 * modules).  The engine talks to it through two calls, one that stores a
 * KV cache and one that retrieves it (Sec. 3.2, the paragraph on the interface
 * with serving engines), and a retrieved context may be put together from several stored
 * pieces (Sec. 3.1 blending module; Sec. 3.2 "KV-cache blending").  This
 * library is that path between an engine's paged GPU KV pool and compact
 * per-chunk buffers:
 *
 *   kdn_store     paged pool  -> chunk buffers   (gather, optional int8 coding)
 *   kdn_retrieve  chunk buffers -> paged pool    (optional decoding, scatter)
 *   kdn_compose   several chunks -> one request's blocks at new positions,
 *                 keys re-rotated by the rotary-embedding position shift
 *
 * Every step runs in CUDA kernels on the caller's stream.  There is no CPU
 * fallback: without a usable CUDA device kdn_create fails.
 *
 * ---------------------------------------------------------------- layouts --
 * Pool (engine-owned device memory), for every layer l and for K and V
 * separately:            bf16 pool[n_blocks][block_size][n_kv_heads][head_dim]
 * Block table (device):  int32 table[n_table_blocks]; request position p lives
 *                        in block table[p / block_size], slot p % block_size.
 * Chunk, T tokens, L layers, H heads, D head_dim, kv 0 = K, 1 = V:
 *   KDN_CODEC_RAW_BF16   bf16 data[L][2][T][H][D]               4*L*T*H*D bytes
 *   KDN_CODEC_INT8_G64   int8 codes[L][2][T][H][D] followed by
 *                        fp32 scales[L][2][T][H*D/64]           2*L*T*H*D*(1+4/64) bytes
 *   KDN_CODEC_INT4_G64   nibbles[L][2][T][H][D/2] bytes (element 2k in the low, 2k+1 in the high nibble,
 *                        two's complement) followed by the same fp32 scales       L*T*H*D*(1+1/8) bytes
 *   No header, no padding, little endian.  A chunk does not record where it
 *   sat in the pool; it can be retrieved into any blocks of any request.
 * int8 coding: group = 64 consecutive head_dim elements of one token-head row;
 *   a = max|x|, scale = a/127 in fp32; scale < FLT_MIN -> scale 0, codes 0;
 *   else code = round_half_even(x * (127/a)) in fp32, in [-127, 127];
 *   decode = bf16_round_nearest_even((float)code * scale).
 * int4 coding: the same with 7 in place of 127 (scale = a/7, code in [-7, 7]); a stronger codec towards the
 *   more-than-tenfold footprint reduction Sec. 3.2 ("KV-cache delivery") reports for combined techniques.
 * Per-channel key codecs (KDN_CODEC_INT8_KC64, KDN_CODEC_INT4_KC64; the paper prescribes no codec): keys carry a few
 *   channels of large magnitude in every token; a group along head_dim makes its ordinary channels share the step of
 *   such a channel.  These codecs group the KEYS along tokens instead -- the chunk tokens 64g .. 64g+63 of one
 *   (layer, head, channel) form a group -- and code the values as the G64 codecs do.  Codes lie as in
 *   INT8_G64 / INT4_G64; the scales that follow them are, per layer, fp32 k_scales[ceil(T/64)][H*D] and then
 *   fp32 v_scales[T][H*D/64].  Same bytes per element as the G64 codecs when T is a multiple of 64.
 *   They need block_size to divide 64 and the chunk's first token to sit at the start of a block (token_offset, or
 *   part_dst_pos in kdn_compose and kdn_compose_select, a multiple of block_size), else KDN_E_UNSUPPORTED;
 *   kdn_compose_static is not supported with them (KDN_E_UNSUPPORTED).  Keep-lists are (kdn_store_sparse, kdn_retrieve_sparse): the chunk
 *   then holds the listed tokens, a key group is 64 consecutive chunk tokens, and neither rule above applies, since
 *   every listed row is found through its own table entry.
 * Token-delta Rice codecs (KDN_CODEC_INT8_TD64, KDN_CODEC_INT4_TD64; Sec. 3.2 "KV-cache delivery" cites a scheme that
 *   quantises a KV cache and then encodes it into binary strings, and reports more than tenfold smaller caches when
 *   such techniques are combined; the paper prescribes no bitstream, this one is this library's).  Keys AND values
 *   are grouped along tokens as the keys of the per-channel key codecs are (chunk tokens 64g .. 64g+63 of one
 *   (layer, K|V, head, channel); codes in [-127, 127] or [-7, 7]).  The n <= 64 codes q_t of a group become one
 *   sub-stream of n symbols: e_t = q_t (mode 0) or e_t = q_t - q_{t-1} with q_{-1} = 0 (mode 1); u_t = 2 e_t for
 *   e_t >= 0, else -2 e_t - 1; Rice code with parameter k in 0..7: quo = u >> k; quo < 15: quo one-bits, a zero-bit, the
 *   k low bits of u from the highest down; else 15 one-bits and u in 9 (int8) or 5 (int4) bits.  Bits fill bytes from
 *   the most significant bit down; a sub-stream ends on a byte boundary (zero padded).  The store picks, per
 *   sub-stream, the (mode, k) with the fewest bits, the first such in the order (0,0) .. (0,7), (1,0) .. (1,7).
 *   Chunk of T tokens: S = 2 L ceil(T/64) segments, segment (l, kv, g) has index (2l + kv) ceil(T/64) + g and
 *   R = H*D channels:  uint64 seg_off[S+1] (padded to 16 bytes) | fp32 scales[S][R] | uint8 lens[S][R] (bytes of each
 *   sub-stream) | uint8 params[S][R] (mode*8 + k) | segment streams.  Segment s starts at byte seg_off[s] (a multiple of
 *   16), holds its R sub-streams back to back in channel order and is zero padded to 16 bytes; seg_off[S] = the bytes
 *   the chunk uses, which is what has to be kept or sent.  kdn_chunk_bytes gives the worst-case CAPACITY (a sub-stream
 *   never exceeds 72 or 40 bytes) and chunk.bytes must equal it; bytes past seg_off[S] are not written and not read
 *   (up to 15 beyond it may be read, never past the capacity).  kdn_td_layout gives the offsets.
 *   Same restrictions as the per-channel key codecs (kdn_compose_select included: whole groups are decoded, the listed
 *   rows delivered, a group without a listed token skipped), and the same freedom for keep-lists: kdn_store_sparse and kdn_retrieve_sparse
 *   take these codecs (the chunk then codes the LISTED tokens: groups are 64 consecutive chunk tokens, mode 1 differences
 *   a code from that of the listed token before it; no rule on token_offset or block_size, every row is found through
 *   its own table entry).  Dropping half of the tokens and coding the rest is what brings a chunk below a tenth of its
 *   span's bf16 bytes on token-correlated input.  kdn_store writes KDN_MEM_DEVICE chunks only (the size of the
 *   result is not known before the kernels have run); kdn_retrieve and kdn_compose also take KDN_MEM_PINNED_HOST
 *   chunks: the library reads seg_off[S] from host memory and copies just the bytes in use over the host link (a
 *   chunk whose bytes in use exceed a staging slab, or whose offset table no store can have written, is refused).
 *   kdn_retrieve_file takes them the same way (the offset table is read from the file first, then the bytes in use,
 *   so only those need be in the file); kdn_store_file does not, for the reason kdn_store does not write host chunks.
 * Key re-rotation in kdn_compose: the stored keys of a part carry rotary
 *   position embedding for positions base_pos + t; placing the part at
 *   dst_pos rotates each pair (k[i], k[i + D/2]) of every head by
 *   (dst_pos - base_pos) * theta^(-2i/D).  Angles are evaluated in fp64 on the
 *   device, the rotation itself in fp32.  Values are copied unchanged.
 *
 * -------------------------------------------------------------- ownership --
 * The caller owns pools, block tables, chunk buffers and streams.  The
 * library owns only the context: a status word, a small ring of launch
 * descriptors, a rotation table, and (on first use of pinned-host chunks) two
 * staging slabs.  It never frees or reallocates caller memory.
 *
 * ---------------------------------------------------------- stream order --
 * A call's work is ordered after everything enqueued on cuda_stream before it,
 * and everything enqueued on cuda_stream after the call returns is ordered
 * after the call's work -- including the copies between page-locked host
 * chunks and the device that run on side_stream: a call that uses the side
 * stream first makes it wait for cuda_stream, and a store ends by making
 * cuda_stream wait for its device-to-host copies.  An event recorded on
 * cuda_stream after kdn_store therefore covers the bytes in host memory, and a
 * host chunk filled by a copy on cuda_stream can be retrieved without a host
 * synchronisation in between.  (The library's kernels let a kernel that is launched behind them with CUDA's
 * programmatic stream serialisation start early; such a kernel has to call cudaGridDependencySynchronize before it
 * reads what the call wrote.  Ordinary launches, copies, events and synchronisations are ordered as usual.)
 *
 * ----------------------------------------------------------------- errors --
 * Argument errors are returned at once and nothing is enqueued.  Otherwise a
 * call returns after enqueueing its work; it does not wait for the GPU.
 * Errors found on the device (a block id outside the pool, a copy that never
 * completed) skip the affected tile, never fault, and are reported by
 * kdn_status_sync.  A context is not thread safe; use one per thread.
 */
#ifndef KDN_H
#define KDN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kdn_ctx kdn_ctx;   /* opaque */

typedef enum {
    KDN_OK = 0,
    KDN_E_INVAL = 1,        /* null pointer, negative count, unknown enum value */
    KDN_E_SHAPE = 2,        /* chunk.bytes or n_tokens does not match the pool's shape */
    KDN_E_ALIGN = 3,        /* a pointer is not 16-byte aligned, or H*D*2 is not a multiple of 16 */
    KDN_E_RANGE = 4,        /* token range beyond the block table; block id outside the pool (device) */
    KDN_E_UNSUPPORTED = 5,  /* int8 / int4 with head_dim % 64 != 0; rotation with head_dim % 16 != 0; ... */
    KDN_E_CUDA = 6,         /* a CUDA runtime call failed */
    KDN_E_NOMEM = 7,        /* context scratch could not be allocated */
    KDN_E_TIMEOUT = 8,      /* a bounded wait inside a kernel gave up (device) */
    KDN_E_NOTFOUND = 9,     /* kdn_index_get / kdn_index_remove: no chunk under this key */
    KDN_E_CHECKSUM = 10,    /* kdn_header_check: the payload does not match the header's checksum */
    KDN_E_IO = 11           /* kdn_store_file / kdn_retrieve_file: a read or write of the chunk file failed or came up short */
} kdn_status;

typedef enum { KDN_CODEC_RAW_BF16 = 0, KDN_CODEC_INT8_G64 = 1, KDN_CODEC_INT4_G64 = 2,
               KDN_CODEC_INT8_KC64 = 3, KDN_CODEC_INT4_KC64 = 4,
               KDN_CODEC_INT8_TD64 = 5, KDN_CODEC_INT4_TD64 = 6 } kdn_codec;
typedef enum { KDN_MEM_DEVICE = 0, KDN_MEM_PINNED_HOST = 1 } kdn_mem;

/* An engine's paged KV pool (Sec. 3.2 names vLLM's paged memory).  k_layers and v_layers are HOST
 * arrays of n_layers DEVICE pointers, each to bf16 [n_blocks][block_size][n_kv_heads][head_dim],
 * 16-byte aligned.  The arrays are copied at registration; the pool memory stays the caller's. */
typedef struct {
    int32_t n_layers, n_kv_heads, head_dim, block_size;
    int64_t n_blocks;
    void *const *k_layers;
    void *const *v_layers;
} kdn_pool_desc;

/* One stored chunk: the KV cache of n_tokens consecutive tokens (Sec. 3.1 storage module).
 * data: 16-byte aligned; device memory (mem = KDN_MEM_DEVICE) or page-locked host memory
 * (KDN_MEM_PINNED_HOST).  bytes must equal kdn_chunk_bytes(pool, n_tokens, codec).
 * base_pos: the absolute position of token 0 when its keys were computed; only kdn_compose reads it. */
typedef struct {
    void   *data;
    size_t  bytes;
    int32_t n_tokens;
    int32_t codec;      /* kdn_codec */
    int32_t mem;        /* kdn_mem */
    int32_t reserved;   /* 0 */
    int64_t base_pos;
} kdn_chunk;

/* One transfer between a request's blocks and one chunk.  Chunk token t <-> request position
 * token_offset + t.  block_table: DEVICE int32 [n_table_blocks] in the request's logical order.
 * Needs token_offset >= 0 and token_offset + n_tokens <= n_table_blocks * block_size.  Neither
 * token_offset nor n_tokens need be a multiple of block_size. */
typedef struct {
    const int32_t *block_table;
    int32_t  n_table_blocks;
    int32_t  reserved;  /* 0 */
    int64_t  token_offset;
    kdn_chunk chunk;
} kdn_xfer_op;

/* One composed request (Sec. 3.1 blending module): part j is written at request positions
 * part_dst_pos[j] + t.  parts and part_dst_pos are HOST arrays of n_parts entries.  Parts must not
 * overlap each other; positions no part covers keep their contents.
 * rope_style 0 = pairs (i, i + head_dim/2); no other style is implemented. */
typedef struct {
    const int32_t  *block_table;     /* device */
    int32_t         n_table_blocks;
    int32_t         n_parts;
    const kdn_chunk *parts;
    const int64_t  *part_dst_pos;
    double          rope_theta;
    int32_t         rope_style;
    int32_t         reserved;        /* 0 */
} kdn_compose_req;

/* Token lists.  Sec. 3.2 "KV-cache delivery" cites dropping tokens or KV elements by importance (LLMLingua, H2O)
 * and "KV-cache blending" cites recomputing a fraction of the tokens after composing (CacheBlend); deciding
 * which tokens is the engine's business, moving only those is this library's.
 *
 * Keep-list: the chunk of a kdn_sparse_op holds exactly op.chunk.n_tokens tokens, and chunk token i is request
 * position op.token_offset + keep[i].  keep: DEVICE int32 [op.chunk.n_tokens], non-negative, strictly
 * increasing.  The chunk's layout is the ordinary one for n_tokens tokens, so a sparse chunk can later be
 * retrieved or composed densely, and a dense chunk retrieved sparsely is not supported (store it sparsely). */
typedef struct {
    kdn_xfer_op    op;
    const int32_t *keep;
} kdn_sparse_op;

/* Select-lists for kdn_compose_select: part j of the request delivers only its chunk tokens
 * part_select[j][0 .. part_n_select[j]) (DEVICE int32 lists, strictly increasing, each < the part's n_tokens);
 * token c still lands at part_dst_pos[j] + c and the positions of unlisted tokens keep their contents, e.g.
 * for the engine to recompute.  part_select: HOST array [n_parts] (NULL, or NULL entries, = deliver every
 * token); part_n_select: HOST array [n_parts]. */
typedef struct {
    const int32_t *const *part_select;
    const int32_t        *part_n_select;
} kdn_select;

/* Launch shape of the tile pipeline.  0 in a field keeps the built-in default.  tile_bytes: bf16
 * bytes moved per pipeline slot (multiple of 128); stages: slots per CTA; ctas_per_sm: persistent
 * CTAs per SM; compute_groups: groups of four compute warps per CTA in launches that code, decode or
 * rotate; group_warps: warps per group, 4 (groups 1, 2, 3, 4 or 6) or 1 (groups 2, 4 or 8); store_lag: how many shared-to-global copies may still be draining before
 * the storer waits (1..16).  stages is raised to store_lag + 2 and rounded down to a multiple of
 * compute_groups.  Settings that do not fit in shared memory are rejected with KDN_E_UNSUPPORTED. */
typedef struct {
    int32_t tile_bytes;
    int32_t stages;
    int32_t ctas_per_sm;
    int32_t compute_groups;
    int32_t store_lag;
    int32_t group_warps;
} kdn_tuning;

/* Create a context on CUDA device `device` (makes it current for the call).  KDN_E_CUDA when no
 * such device can be used. */
kdn_status kdn_create(kdn_ctx **out, int device);
/* Wait for the context's own streams and free its scratch.  NULL is allowed. */
void kdn_destroy(kdn_ctx *ctx);

/* Register a pool (Sec. 3.2: the engine's paged memory); *pool_id is the handle for later calls. */
kdn_status kdn_pool_register(kdn_ctx *ctx, const kdn_pool_desc *pool, int *pool_id);

/* Bytes of one chunk of n_tokens tokens for this pool's shape; 0 if the codec cannot hold the
 * shape.  Pure host arithmetic; reads only the shape fields of *pool. */
size_t kdn_chunk_bytes(const kdn_pool_desc *pool, int32_t n_tokens, int32_t codec);

/* Byte offsets of the regions of a token-delta Rice chunk of n_tokens tokens (see the top of this file): the
 * number of segments S, where scales, lens, params and the first segment's streams begin, and the capacity
 * (= kdn_chunk_bytes).  After a store, the uint64 at byte 8*S of the chunk is the number of bytes in use.
 * Pure host arithmetic.  KDN_E_UNSUPPORTED for other codecs or head_dim % 64 != 0. */
typedef struct {
    uint64_t segments, scales_offset, lens_offset, params_offset, streams_offset, capacity;
} kdn_td_layout_info;
kdn_status kdn_td_layout(const kdn_pool_desc *pool, int32_t n_tokens, int32_t codec, kdn_td_layout_info *out);

/* Host-side argument check shared by kdn_store / kdn_retrieve (same status they would return);
 * touches no device.  Pointers are only compared and tested for alignment, never dereferenced,
 * except the host arrays ops[]. */
kdn_status kdn_validate_xfer(const kdn_pool_desc *pool, const kdn_xfer_op *ops, int n_ops);
/* Same for kdn_compose; reads reqs[], parts[] and part_dst_pos[]. */
kdn_status kdn_validate_compose(const kdn_pool_desc *pool, const kdn_compose_req *reqs, int n_reqs);

/* Sec. 3.2 call (i), store: for each op gather the chunk's tokens out of the pool blocks its table
 * names and write the chunk (int8-coded if chunk.codec says so).  One kernel launch covers the
 * whole batch.  Source blocks may repeat; chunk buffers of one call must not overlap.
 * A KDN_MEM_PINNED_HOST chunk is written to a staging slab and copied out on side_stream. */
kdn_status kdn_store(kdn_ctx *ctx, int pool_id, const kdn_xfer_op *ops, int n_ops,
                     void *cuda_stream, void *side_stream);

/* Sec. 3.2 call (ii), retrieve, with Sec. 3.1's decompression on the GPU: the inverse of
 * kdn_store.  Writes exactly the n_tokens addressed token slots of each op; every other byte of
 * the pool keeps its value.  Destination slots of one call must be pairwise distinct (otherwise
 * the overlapped slots hold one of the written values, unspecified which).  KDN_MEM_PINNED_HOST
 * chunks are copied to the device on side_stream (NULL = a stream the context owns), layer range by
 * layer range through two staging slabs, while the kernel of the previous range runs on
 * cuda_stream. */
kdn_status kdn_retrieve(kdn_ctx *ctx, int pool_id, const kdn_xfer_op *ops, int n_ops,
                        void *cuda_stream, void *side_stream);

/* Layer-wise delivery (Sec. 3.1 delivery module; Sec. 3 names the bandwidth of loading KV caches into GPU memory
 * as the constraint once they live outside it): kdn_retrieve issued in steps of layers_per_step layers, first
 * layers first, so that the engine can run layer l while later layers are still crossing the host link.
 * layer_ready: NULL, or a HOST array of n_layers CUDA events (cudaEvent_t, entries may be NULL) owned by the
 * caller; layer_ready[l] is recorded on cuda_stream once layers 0..l of every op of the call have been written.
 * Results are exactly those of kdn_retrieve.  Each step is one launch (plus staged copies for pinned-host
 * chunks), so small steps on small chunks cost launch overhead. */
kdn_status kdn_retrieve_layerwise(kdn_ctx *ctx, int pool_id, const kdn_xfer_op *ops, int n_ops, int layers_per_step,
                                  void *cuda_stream, void *side_stream, void *const *layer_ready);

/* A chunk kept in a file (Sec. 3: once KV caches move out of GPU and CPU memory to disks or remote servers, the
 * bandwidth of loading them back becomes the constraint; Sec. 3.1 delivery module).  The chunk's bytes, in the
 * ordinary chunk layout, occupy [file_offset, file_offset + op.chunk.bytes) of the open file descriptor fd (a
 * regular file, or anything pread / pwrite work on).  op.chunk.data and op.chunk.mem are ignored; every other
 * field means what it means in kdn_xfer_op. */
typedef struct {
    kdn_xfer_op op;
    int32_t     fd;
    int32_t     reserved;   /* 0 */
    int64_t     file_offset;
} kdn_file_op;

/* kdn_retrieve / kdn_store for file-backed chunks.  The bytes travel layer range by layer range through two
 * page-locked bounce buffers (as large as the staging slabs, allocated on first use) and the staging slabs: while
 * the calling thread reads the next range from the file, the previous one crosses the host link on side_stream and
 * the one before that is decoded and scattered on cuda_stream.  The calling thread does the file I/O, so these
 * calls take as long as the I/O does: kdn_retrieve_file returns when the last range has been read and enqueued (the
 * GPU may still be working; order later work after it on cuda_stream), kdn_store_file returns when the files hold
 * the chunks.  A failed or short read or write returns KDN_E_IO; ranges already enqueued still run.  Results are
 * exactly those of kdn_retrieve / kdn_store on a memory-resident copy of the same bytes. */
kdn_status kdn_retrieve_file(kdn_ctx *ctx, int pool_id, const kdn_file_op *ops, int n_ops,
                             void *cuda_stream, void *side_stream);
kdn_status kdn_store_file(kdn_ctx *ctx, int pool_id, const kdn_file_op *ops, int n_ops,
                          void *cuda_stream, void *side_stream);

/* Sec. 3.1 blending module: compose every request's parts into its blocks; keys of parts whose
 * part_dst_pos differs from base_pos are re-rotated (see the top of this file).  A part with equal
 * positions, and every value plane, is written exactly as kdn_retrieve writes it. */
kdn_status kdn_compose(kdn_ctx *ctx, int pool_id, const kdn_compose_req *reqs, int n_reqs,
                       void *cuda_stream, void *side_stream);

/* Limits of kdn_compose_static: one call may carry at most KDN_STATIC_MAX_PARTS parts (summed over
 * its requests), on a pool of at most KDN_STATIC_MAX_LAYERS layers and head_dim <= KDN_STATIC_MAX_HEAD_DIM.
 * The fixed device array behind it is KDN_STATIC_SCRATCH_BYTES bytes. */
#define KDN_STATIC_MAX_PARTS     128
#define KDN_STATIC_MAX_LAYERS    128
#define KDN_STATIC_MAX_HEAD_DIM  512
#define KDN_STATIC_SCRATCH_BYTES 278784

/* kdn_compose for callers that must not allocate device memory.  (The paper has no counterpart to
 * this call; it exists for integration reasons only.)
 *
 * Who needs it: an engine that handed all of the GPU's memory to its own allocator at start-up, so a
 * cudaMalloc from a library would fail; a thread that runs while another thread captures a CUDA graph
 * in global capture mode, where cudaMalloc is an error; a latency-critical loop that cannot take the
 * device-wide synchronisation cudaMalloc and cudaFree may imply.  kdn_create and kdn_pool_register
 * allocate (descriptor ring, pointer arrays, rotation table), so such callers cannot use a context.
 *
 * This call needs no context and calls no cudaMalloc, cudaFree or other allocating routine.  Its
 * scratch -- the device copies of the pool's layer pointers, the part records, the rotation table and
 * a status word -- lives in one fixed array inside the library's device image.  Every GPU that loads
 * the library holds those KDN_STATIC_SCRATCH_BYTES bytes until the process exits.
 *
 * Arguments are those of kdn_pool_register (pool) and kdn_compose (reqs, n_reqs, cuda_stream), with
 * the same layouts, preconditions and results: a part whose position is unchanged is written exactly
 * as kdn_retrieve writes it, so the call also serves as a retrieve.  device is the CUDA device that
 * owns the pool; it is made current.  Only KDN_MEM_DEVICE parts are accepted (staging slabs would
 * have to be allocated).  Sizes beyond the limits above return KDN_E_UNSUPPORTED and enqueue nothing.
 * The built-in launch shape is used; kdn_set_tuning does not apply.
 *
 * wait != 0: the call waits for cuda_stream and returns the first error the kernels recorded
 * (KDN_E_RANGE for a block id outside the pool, ...), or KDN_OK.  wait == 0: the call returns after
 * enqueueing; errors found on the device by that call are then not reported.
 *
 * The first call on each device does the one-time set-up: it looks up the array's device address, loads
 * every kernel a later call can launch and raises their shared-memory limits, so no later call meets a
 * first-use step of the CUDA runtime.  Make that first call before any stream capture begins.  All calls on a device share the one array,
 * and it still holds the previous call's records when the next call starts: each call rewrites the
 * records it uses and clears the status word, on cuda_stream, before its kernels run.  Two calls
 * whose work can overlap on the GPU (different streams without an ordering between them) therefore
 * race on the array and corrupt each other; issue them on one stream or order them yourself. */
kdn_status kdn_compose_static(int device, const kdn_pool_desc *pool, const kdn_compose_req *reqs, int n_reqs,
                              void *cuda_stream, int wait);

/* kdn_store / kdn_retrieve for chunks that hold only the tokens of a keep-list (see kdn_sparse_op).  A tile takes
 * one listed token row or several that follow one another in the list (up to 16); a list entry that points outside
 * the block table is reported as KDN_E_RANGE by kdn_status_sync and nothing is moved for it, nor, possibly, for the
 * rows that share its tile: after that error neither the chunk (store) nor the listed positions (retrieve) are to be
 * used.  kdn_retrieve_sparse writes the listed positions and nothing else. */
kdn_status kdn_store_sparse(kdn_ctx *ctx, int pool_id, const kdn_sparse_op *ops, int n_ops,
                            void *cuda_stream, void *side_stream);
kdn_status kdn_retrieve_sparse(kdn_ctx *ctx, int pool_id, const kdn_sparse_op *ops, int n_ops,
                               void *cuda_stream, void *side_stream);

/* kdn_compose that delivers only selected tokens of each part (see kdn_select); selects[r] belongs to reqs[r].
 * Rotation, codecs and everything else are as in kdn_compose. */
kdn_status kdn_compose_select(kdn_ctx *ctx, int pool_id, const kdn_compose_req *reqs, const kdn_select *selects,
                              int n_reqs, void *cuda_stream, void *side_stream);

/* Wait for cuda_stream (and the context's side stream) and return the first error a kernel of this
 * context recorded since the last call of this function, or KDN_OK. */
kdn_status kdn_status_sync(kdn_ctx *ctx, void *cuda_stream);

/* Change the launch shape for later calls.  NULL restores the defaults. */
kdn_status kdn_set_tuning(kdn_ctx *ctx, const kdn_tuning *tuning);
/* Bytes of each of the two staging slabs used for pinned-host chunks (default 256 MiB, allocated
 * on first use).  Takes effect at the next pinned-host call; frees slabs already allocated. */
kdn_status kdn_set_staging_bytes(kdn_ctx *ctx, size_t bytes_per_slab);

/* Limit, in nanoseconds, after which a wait inside the tile pipeline (and the wait of a key-plane or token-delta CTA for
 * its rows or bytes) gives up and the launch reports KDN_E_TIMEOUT
 * (default, and ns = 0: two seconds).  The waits that let a CTA's own copies finish before it leaves always keep the
 * default.  Meant for exercising the error path: with a limit shorter than a memory access the next launches give up
 * almost at once, write little or nothing, and kdn_status_sync returns KDN_E_TIMEOUT; nothing faults or hangs, and
 * after the default is restored the context works as before. */
kdn_status kdn_set_wait_limit_ns(kdn_ctx *ctx, uint64_t ns);

/* Kernels this context has launched so far (for accounting; never reset). */
uint64_t kdn_launch_count(const kdn_ctx *ctx);

/* Shape of the context's most recent launch of the tile pipeline, for reports: op 0 store / 1 retrieve / 2 compose
 * (the kernel is kdn_store_kernel / kdn_retrieve_kernel / kdn_compose_kernel<compute_groups, group_warps>, or, with
 * rows_kernel = 1, kdn_store_rows_kernel / kdn_retrieve_rows_kernel: tiles of up to 16 token rows, which keep-lists over
 * short rows and dense coded ops on pool blocks of 2 KiB or less are given); rows_per_tile: token rows per tile of a
 * keep-list launch (1 otherwise); grid is what was asked for (the launch itself never exceeds the CTAs resident at once). */
typedef struct {
    int32_t  op, compute_groups, group_warps, tile_bytes, stages, ctas_per_sm, store_lag, grid, smem_bytes;
    uint32_t n_tiles;
    int32_t  rows_per_tile, rows_kernel;
} kdn_launch_info;
kdn_status kdn_last_launch(const kdn_ctx *ctx, kdn_launch_info *out);

/* ------------------------------------------------------------------------------------------------
 * Storage-module shell (Sec. 3.1: the storage module keeps KV caches under keys derived from their texts; Sec. 3.2:
 * the engine hands over a KV cache together with its text and later asks for it by text).  The paper fixes
 * neither a key, a header nor an eviction rule; these are this library's choices.  The shell owns no chunk
 * memory: it maps keys to the caller's chunk descriptors and says which ones to drop. */

/* Key of a text: FNV-1a (64 bit) over its token ids, each taken as four little-endian bytes.  Host arithmetic. */
uint64_t kdn_key_hash(const int32_t *token_ids, size_t n);

/* Payload checksum, computed on the GPU: sum over the payload's little-endian 32-bit words w_i of
 * (w_i XOR 0x9E3779B9) * ((2 i + 1) mod 2^32), modulo 2^64.  payload: DEVICE memory, 4-byte aligned (16 for full
 * speed), bytes a multiple of 4 (every chunk layout is).  The result is written to *device_out (DEVICE uint64,
 * 8-byte aligned) by work enqueued on cuda_stream; read it after synchronising.  Needs no context. */
kdn_status kdn_checksum(int device, const void *payload, size_t bytes, uint64_t *device_out, void *cuda_stream);

/* Self-describing header a caller can keep in front of (or beside) a stored chunk: 128 bytes, little endian. */
typedef struct {
    char     magic[8];        /* "KDNCHNK1" */
    uint32_t header_bytes;    /* 128 */
    uint32_t codec;           /* kdn_codec */
    int32_t  n_layers, n_kv_heads, head_dim, n_tokens;
    int64_t  base_pos;
    uint64_t payload_bytes;
    uint64_t key;
    uint64_t checksum;
    uint8_t  reserved[64];    /* 0 */
} kdn_chunk_header;

/* Fill *out for `chunk` of a pool of this shape.  KDN_E_SHAPE if chunk.bytes does not fit shape, tokens and codec. */
kdn_status kdn_header_fill(const kdn_pool_desc *pool, const kdn_chunk *chunk, uint64_t key, uint64_t checksum,
                           kdn_chunk_header *out);
/* Check a header read back from storage against the pool's shape and against the checksum the caller computed over
 * the payload it read (kdn_checksum).  KDN_E_INVAL: not a header; KDN_E_SHAPE: another model shape or inconsistent
 * sizes; KDN_E_CHECKSUM: payload damaged.  On KDN_OK and out != NULL, fills out->bytes, n_tokens, codec, base_pos
 * (data and mem stay the caller's to set). */
kdn_status kdn_header_check(const kdn_pool_desc *pool, const kdn_chunk_header *header, uint64_t checksum_of_payload,
                            kdn_chunk *out);

/* Index from key to chunk descriptor with least-recently-used eviction under a byte budget.  Not thread safe. */
typedef struct kdn_index kdn_index;
typedef struct { size_t capacity_bytes, bytes, entries; uint64_t hits, misses, evictions; } kdn_index_info;

kdn_status kdn_index_create(kdn_index **out, size_t capacity_bytes);
void kdn_index_destroy(kdn_index *index);
/* Insert `chunk` under `key` as the most recently used entry.  A chunk already stored under the key is replaced and
 * handed back first in evicted[]; then least-recently-used entries are dropped until the budget holds, each handed
 * back in evicted[] (the caller frees or reuses their memory).  If more than max_evicted descriptors would have to be
 * handed back, or the chunk alone exceeds the budget, nothing changes and KDN_E_NOMEM is returned. */
kdn_status kdn_index_put(kdn_index *index, uint64_t key, const kdn_chunk *chunk, kdn_chunk *evicted, int max_evicted,
                         int *n_evicted);
/* Look a key up (KDN_E_NOTFOUND if absent) and mark it most recently used. */
kdn_status kdn_index_get(kdn_index *index, uint64_t key, kdn_chunk *out);
/* Drop a key; its descriptor is returned in *out (may be NULL). */
kdn_status kdn_index_remove(kdn_index *index, uint64_t key, kdn_chunk *out);
void kdn_index_stats(const kdn_index *index, kdn_index_info *out);

/* Static string for a status code. */
const char *kdn_strerror(kdn_status status);

#ifdef __cplusplus
}
#endif
#endif /* KDN_H */
