/*
 * CPU oracle for the KV-cache store / retrieve / compose path of a Knowledge
 * Delivery Network (paper Sec. 3.1: storage, delivery and blending modules;
 * Sec. 3.2 "Interface with LLM serving engines": the two calls (i) store and
 * (ii) retrieve).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, scalar statement of
 * what the path computes.  It shares no code, header, table or constant with
 * the CUDA library, and the CUDA library never calls it.  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * The paper states the problem (store KV caches apart from the engine's paged
 * memory, deliver them compressed and decompress on the GPU, compose several
 * of them in one query's context, reuse a chunk at another position) but
 * prints no layout, codec, formula or number for it.  The concrete readings
 * taken here, each one stated where it is used:
 *
 *   R1  paged pool   per layer l and kv in {0 = K, 1 = V}:
 *                    pool[l][kv][block][slot][head][d], bf16
 *                    (Sec. 3.2 names "paged memory" only).
 *   R2  chunk        raw : bf16  chunk[l][kv][t][head][d]
 *                    int8: int8  codes[l][kv][t][head][d] followed by
 *                          fp32  scales[l][kv][t][head*D/64 + g]
 *                    no header, no padding, little endian.
 *   R3  mapping      request position p sits in block table[p / bs], slot
 *                    p % bs; chunk token t of an op with token_offset s is
 *                    position p = s + t.
 *   R4  int8 codec   group = 64 consecutive d of one (l, kv, t, head);
 *                    a = max|x|; scale = a / 127 (fp32 divide);
 *                    scale below FLT_MIN (zero or subnormal) -> scale 0, codes 0;
 *                    else inv = 127 / a (fp32 divide),
 *                    q = clamp(round_half_even(x * inv), -127, 127), the
 *                    product being one fp32 multiply.
 *   R5  decode       x^ = bf16_rne((float)q * scale), one fp32 multiply.
 *   R4' int4 codec   (a stronger codec on the way to the "over 10x" footprint reduction Sec. 3.2 cites; not
 *                    prescribed by the paper) same as R4 with 7 in place of 127: scale = a / 7, inv = 7 / a,
 *                    q = clamp(round_half_even(x * inv), -7, 7); two codes per byte as two's-complement
 *                    nibbles, element 2k in the low nibble and 2k+1 in the high nibble of byte k;
 *                    chunk = nibbles[l][kv][t][head][D/2] bytes followed by the fp32 scales as in R2.
 *   R4" per-channel key codecs (codecs 3 = int8, 4 = int4; not prescribed by the paper: Sec. 3.2 "KV-cache delivery"
 *                    only cites quantisation among the techniques that shrink KV caches).  Keys have a few
 *                    channels of large magnitude in every token, which a group along head_dim shares with its
 *                    ordinary channels; grouping keys along TOKENS keeps such a channel to itself.
 *                    K planes: group = the chunk tokens 64 g .. min(64 g + 63, T - 1) of one (l, head, d) channel;
 *                    a = max over those tokens of |x|, then scale, inv and codes exactly as in R4 / R4' (127 or 7).
 *                    V planes: exactly R4 / R4'.  Codes lie where R2 / R4' put them.  Scales, per layer:
 *                    fp32 k_scales[ceil(T/64)][head*D] followed by fp32 v_scales[t][head*D/64]; layers follow
 *                    each other; the scales follow the codes.  Decode is R5 with the element's own scale.
 *                    With a keep-list (R7) the chunk's tokens are the listed ones and a key group is 64 consecutive
 *                    CHUNK tokens, as for R9; a select-list delivers the listed chunk tokens, each decoded with its
 *                    own scales, as for every fixed-rate codec.
 *   R9  token-delta Rice codecs (codecs 5 = int8, 6 = int4; not prescribed by the paper: Sec. 3.2 "KV-cache delivery"
 *                    cites a scheme that quantises a KV cache and then encodes it into binary strings, and reports
 *                    more than tenfold reductions for combined techniques.  This is this library's own bitstream.)
 *                    Quantisation: K AND V planes are grouped along tokens as the keys of R4" are: group = the chunk
 *                    tokens 64 g .. min(64 g + 63, T - 1) of one (l, kv, head, d) channel; scale, inv and codes as in
 *                    R4 / R4' (127 or 7).  A group's codes q_0 .. q_{n-1} become one SUB-STREAM of n symbols:
 *                      mode 0 (direct):       e_t = q_t
 *                      mode 1 (token delta):  e_t = q_t - q_{t-1}, with q_{-1} = 0
 *                      zigzag:                u_t = 2 e_t if e_t >= 0, else -2 e_t - 1
 *                      Rice code, parameter k in 0..7: quo = u >> k; if quo < 15: quo one-bits, a zero-bit, then
 *                      the k low bits of u, high bit first; else (escape): 15 one-bits, then u in `raw` bits, high
 *                      bit first, raw = 9 (int8: u <= 508) or 5 (int4: u <= 28).
 *                    Bits fill bytes from the most significant bit down; the sub-stream ends on a byte boundary,
 *                    padded with zero bits.  The encoder takes the (mode, k) with the fewest total bits, the first
 *                    such in the order (0,0), (0,1), .., (0,7), (1,0), .., (1,7); param = mode * 8 + k.  A sub-stream
 *                    is never longer than 72 bytes (int8: mode 0, k = 7 costs at most 9 bits a symbol) or 40 bytes
 *                    (int4: mode 0, k = 3 costs at most 5).
 *                    Chunk: S = 2 L ceil(T/64) segments, segment (l, kv, g) has index (2 l + kv) ceil(T/64) + g and
 *                    R = head * D channels.  uint64 seg_off[S + 1] (padded to 16 bytes), fp32 scales[S][R],
 *                    uint8 lens[S][R] (bytes of each sub-stream), uint8 params[S][R], then the segments' streams:
 *                    segment s starts at byte seg_off[s] (a multiple of 16; seg_off[0] = the end of params), holds
 *                    its R sub-streams back to back in channel order, and is padded with zero bytes to 16;
 *                    seg_off[S] = the bytes the chunk uses.  A chunk buffer has the worst-case capacity
 *                    fixed part + S * R * (72 or 40); bytes past seg_off[S] are not defined.
 *                    Decode: undo Rice, zigzag and the delta, then R5 with the channel's scale.  With a keep-list
 *                    (R7) the chunk's tokens are the listed ones: groups are 64 consecutive CHUNK tokens and mode 1
 *                    differences a code from that of the listed token before it (the combination the paper's Sec. 3.2
 *                    "KV-cache delivery" points to: drop tokens, then code what is left).  A select-list delivers
 *                    the listed chunk tokens of the decoded chunk, as for every codec.
 *   R6  re-rotation  stored keys carry rotary position embedding at absolute
 *                    positions base_pos + t (what an engine's pool holds), so
 *                    reuse at dst_pos (Sec. 3.2 "KV-cache blending": a
 *                    segment's cache reused at different positions) rotates
 *                    every pair (k[i], k[i + D/2]) of every head by
 *                    phi_i = delta * theta^(-2 i / D), delta = dst_pos - base_pos,
 *                    evaluated in fp64.  Values are copied.  delta == 0 keys
 *                    take the decode path unchanged.
 *
 *   R7  token lists  (Sec. 3.2 "KV-cache delivery" cites dropping tokens and KV elements by importance; Sec. 3.2
 *                    "KV-cache blending" cites recomputing a fraction of the tokens after blending.  The scoring
 *                    is not part of this path; moving only the listed tokens is.)
 *                    keep-list: a chunk may hold only some tokens of a span: chunk token t is the request position
 *                    off + keep[t], keep strictly increasing; store gathers those, retrieve writes only those.
 *                    select-list: compose may deliver only some tokens of a part: for each listed chunk token c
 *                    (strictly increasing) it writes position dst_pos + c and leaves the other positions alone.
 *
 *   R8  storage shell (Sec. 3.1 storage module: KV caches kept under keys derived from their texts; Sec. 3.2
 *                    interface: a cache is stored together with its text and asked for by text.)  key = FNV-1a 64-bit hash of the
 *                    text's token ids taken as little-endian 32-bit integers; payload checksum =
 *                    sum_i ((w_i XOR 0x9E3779B9) * ((2 i + 1) mod 2^32)) mod 2^64 over the payload's little-endian
 *                    32-bit words w_i.  Neither is prescribed by the paper.
 *
 * Parity pins (tests/test_oracle_*.py, all CPU): brute force against an
 * independent index-by-index formulation on tiny shapes; contiguous table
 * reduces store to a slice copy; store-then-retrieve identity on raw bf16 for
 * all bit-pattern classes; placement invariance; hand-worked codec groups
 * (tests/golden/); |x - q*scale| <= scale/2 bound; a second round-half-even
 * formulation; exhaustive-class bf16 rounding against torch; rotation
 * composition R(a)R(b) = R(a+b), norm preservation, quarter/half turns, and
 * rotary-from-scratch at p then re-rotation by delta equals rotary at p+delta.
 * End-to-end values: parity unpinned by the paper (it prints no value on this
 * path); every pin above comes from the definitions and from mathematics.
 */
#include <float.h>
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define KDN_ORACLE_RAW_BF16 0
#define KDN_ORACLE_INT8_G64 1
#define KDN_ORACLE_INT4_G64 2
#define KDN_ORACLE_INT8_KC64 3
#define KDN_ORACLE_INT4_KC64 4
#define KDN_ORACLE_INT8_TD64 5
#define KDN_ORACLE_INT4_TD64 6
#define KDN_ORACLE_GROUP 64

/* ---------------------------------------------------------------- bf16 -- */

float kdn_oracle_bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* fp32 -> bf16, round to nearest, ties to even.  NaN stays NaN (quiet). */
uint16_t kdn_oracle_f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u)          /* NaN */
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t keep = u >> 16;
    uint32_t rest = u & 0xffffu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u)))
        keep += 1u;                                /* may carry into inf: correct */
    return (uint16_t)keep;
}

/* The same conversion for n values (so a test can sweep every fp32 bit pattern). */
void kdn_oracle_f32_to_bf16_many(const float *f, uint16_t *out, size_t n)
{
    for (size_t i = 0; i < n; ++i) out[i] = kdn_oracle_f32_to_bf16(f[i]);
}

/* fp64 -> bf16, round to nearest even in ONE rounding (no trip through fp32):
 * take the bf16 at or below |x| and its upper neighbour, keep the nearer one,
 * the even one on a tie. */
uint16_t kdn_oracle_f64_to_bf16(double x)
{
    if (x != x) return 0x7fc0u;
    uint16_t sign = (uint16_t)(signbit(x) ? 0x8000u : 0u);
    double a = fabs(x);
    if (isinf(a)) return (uint16_t)(sign | 0x7f80u);
    /* largest bf16 magnitude <= a, by bisection over the 0..0x7f80 codes
     * (bf16 magnitudes are monotone in their bit pattern) */
    uint32_t lo = 0, hi = 0x7f80u;                 /* value(lo) <= a < value(hi)=inf */
    while (hi - lo > 1u) {
        uint32_t mid = (lo + hi) / 2u;
        if ((double)kdn_oracle_bf16_to_f32((uint16_t)mid) <= a) lo = mid; else hi = mid;
    }
    double vlo = (double)kdn_oracle_bf16_to_f32((uint16_t)lo);
    if (hi == 0x7f80u) {
        /* above the largest finite bf16: round to inf only past the half-way
         * point to the next (unrepresentable) step 2^128 */
        double step = ldexp(1.0, 127 - 7);
        double half = vlo + step / 2.0;
        uint32_t r = (a > half || (a == half && (lo & 1u))) ? hi : lo;
        return (uint16_t)(sign | r);
    }
    double vhi = (double)kdn_oracle_bf16_to_f32((uint16_t)hi);
    double dlo = a - vlo, dhi = vhi - a;           /* exact: all three are close doubles */
    uint32_t r;
    if (dlo < dhi) r = lo; else if (dhi < dlo) r = hi; else r = (lo & 1u) ? hi : lo;
    return (uint16_t)(sign | r);
}

/* --------------------------------------------------------------- sizes -- */

int kdn_oracle_td_layout(int L, int H, int D, int T, int codec, size_t *out);

/* R2: bytes of one chunk of T tokens.  0 when the codec cannot hold the shape. */
size_t kdn_oracle_chunk_bytes(int L, int H, int D, int T, int codec)
{
    if (L <= 0 || H <= 0 || D <= 0 || T < 0) return 0;
    size_t elems = (size_t)L * 2u * (size_t)T * (size_t)H * (size_t)D;
    if (codec == KDN_ORACLE_RAW_BF16) return 2u * elems;
    if (codec == KDN_ORACLE_INT8_G64) {
        if (D % KDN_ORACLE_GROUP) return 0;
        return elems + 4u * (elems / KDN_ORACLE_GROUP);
    }
    if (codec == KDN_ORACLE_INT4_G64) {
        if (D % KDN_ORACLE_GROUP) return 0;
        return elems / 2u + 4u * (elems / KDN_ORACLE_GROUP);
    }
    if (codec == KDN_ORACLE_INT8_KC64 || codec == KDN_ORACLE_INT4_KC64) {
        if (D % KDN_ORACLE_GROUP) return 0;
        size_t hd = (size_t)H * (size_t)D;
        size_t n_groups = ((size_t)T + KDN_ORACLE_GROUP - 1u) / KDN_ORACLE_GROUP;
        size_t scales_per_layer = n_groups * hd + (size_t)T * hd / KDN_ORACLE_GROUP;     /* R4": K then V */
        return (codec == KDN_ORACLE_INT4_KC64 ? elems / 2u : elems) + 4u * (size_t)L * scales_per_layer;
    }
    if (codec == KDN_ORACLE_INT8_TD64 || codec == KDN_ORACLE_INT4_TD64) {
        size_t lay[6];
        if (kdn_oracle_td_layout(L, H, D, T, codec, lay)) return 0;
        return lay[5];                                       /* R9: worst-case capacity */
    }
    return 0;
}

/* ------------------------------------------------------------ int8 codec -- */

/* R4 / R4': encode one group of 64 bf16 values with codes in [-qmax, qmax] (127 or 7). */
static void quant_values_q(const uint16_t *x_bf16, int n, int8_t *q, float *scale_out, float qmax)
{
    float a = 0.0f;
    for (int i = 0; i < n; ++i) {
        float v = fabsf(kdn_oracle_bf16_to_f32(x_bf16[i]));
        if (v > a) a = v;
    }
    volatile float scale = a / qmax;               /* volatile: one fp32 divide, stored as fp32 */
    if (!(scale >= FLT_MIN)) {
        *scale_out = 0.0f;
        for (int i = 0; i < n; ++i) q[i] = 0;
        return;
    }
    volatile float inv = qmax / a;
    for (int i = 0; i < n; ++i) {
        volatile float prod = kdn_oracle_bf16_to_f32(x_bf16[i]) * inv;   /* one fp32 multiply */
        float r = rintf(prod);                     /* default rounding mode: ties to even */
        if (r > qmax) r = qmax;
        if (r < -qmax) r = -qmax;
        q[i] = (int8_t)(int)r;
    }
    *scale_out = scale;
}

static void quant_group_q(const uint16_t *x_bf16, int8_t *q, float *scale_out, float qmax)
{
    quant_values_q(x_bf16, KDN_ORACLE_GROUP, q, scale_out, qmax);
}

/* R4": encode n <= 64 values of one key channel (consecutive chunk tokens) with codes in [-qmax, qmax]. */
void kdn_oracle_quant_channel(const uint16_t *x_bf16, int n, int qmax, int8_t *q, float *scale_out)
{
    quant_values_q(x_bf16, n, q, scale_out, (float)qmax);
}

void kdn_oracle_quant_group(const uint16_t *x_bf16, int8_t *q, float *scale_out)
{
    quant_group_q(x_bf16, q, scale_out, 127.0f);
}

/* R4': 64 values -> 32 bytes of nibbles + one scale. */
void kdn_oracle_quant4_group(const uint16_t *x_bf16, uint8_t *packed, float *scale_out)
{
    int8_t q[KDN_ORACLE_GROUP];
    quant_group_q(x_bf16, q, scale_out, 7.0f);
    for (int k = 0; k < KDN_ORACLE_GROUP / 2; ++k)
        packed[k] = (uint8_t)(((uint8_t)q[2 * k] & 0x0fu) | (((uint8_t)q[2 * k + 1] & 0x0fu) << 4));
}

/* R4': the code of element i (0 <= i < 64) of a packed group, sign-extended. */
int kdn_oracle_nibble(const uint8_t *packed, size_t i)
{
    int v = (i & 1u) ? (packed[i >> 1] >> 4) : (packed[i >> 1] & 0x0f);
    return v >= 8 ? v - 16 : v;
}

/* R5: decode one code. */
uint16_t kdn_oracle_dequant(int8_t q, float scale)
{
    volatile float prod = (float)q * scale;
    return kdn_oracle_f32_to_bf16(prod);
}

/* ------------------------------------------- token-delta Rice codecs (R9) -- */

static int td_is(int codec) { return codec == KDN_ORACLE_INT8_TD64 || codec == KDN_ORACLE_INT4_TD64; }
static int td_qmax(int codec) { return codec == KDN_ORACLE_INT8_TD64 ? 127 : 7; }
static int td_raw_bits(int qmax) { return qmax == 127 ? 9 : 5; }           /* bits that hold the largest symbol, 4 qmax */

/* R9: longest sub-stream in bytes. */
int kdn_oracle_td_max_len(int qmax) { return qmax == 127 ? 72 : 40; }

/* R9: byte offsets of a chunk's regions: out[0] = S (segments), out[1] = scales, out[2] = lens, out[3] = params,
 * out[4] = first segment's streams (the end of the fixed part), out[5] = capacity.  Non-zero: shape not codable. */
int kdn_oracle_td_layout(int L, int H, int D, int T, int codec, size_t *out)
{
    if (!td_is(codec) || L <= 0 || H <= 0 || D <= 0 || T < 0 || D % KDN_ORACLE_GROUP) return 3;
    size_t G = ((size_t)T + KDN_ORACLE_GROUP - 1u) / KDN_ORACLE_GROUP;
    size_t S = 2u * (size_t)L * G, R = (size_t)H * (size_t)D;
    out[0] = S;
    out[1] = (8u * (S + 1u) + 15u) / 16u * 16u;
    out[2] = out[1] + 4u * S * R;
    out[3] = out[2] + S * R;
    out[4] = out[3] + S * R;
    out[5] = out[4] + S * ((R * (size_t)kdn_oracle_td_max_len(td_qmax(codec)) + 15u) / 16u * 16u);
    return 0;
}

unsigned kdn_oracle_zigzag(int e) { return e >= 0 ? 2u * (unsigned)e : 2u * (unsigned)(-e) - 1u; }
int kdn_oracle_unzigzag(unsigned u) { return (u & 1u) ? -(int)((u + 1u) / 2u) : (int)(u / 2u); }

/* R9: bits one symbol costs. */
int kdn_oracle_rice_bits(unsigned u, int k, int raw_bits)
{
    unsigned quo = u >> k;
    return quo < 15u ? (int)quo + 1 + k : 15 + raw_bits;
}

/* Bit `pos` of a byte string, counted from the most significant bit of byte 0. */
static void put_bit(uint8_t *buf, size_t *pos, unsigned bit)
{
    if (bit) buf[*pos / 8u] |= (uint8_t)(0x80u >> (*pos % 8u));
    ++*pos;
}
static unsigned get_bit(const uint8_t *buf, size_t *pos)
{
    unsigned bit = (buf[*pos / 8u] >> (7u - *pos % 8u)) & 1u;
    ++*pos;
    return bit;
}

static void rice_put(uint8_t *buf, size_t *pos, unsigned u, int k, int raw_bits)
{
    unsigned quo = u >> k;
    if (quo < 15u) {
        for (unsigned i = 0; i < quo; ++i) put_bit(buf, pos, 1u);
        put_bit(buf, pos, 0u);
        for (int b = k - 1; b >= 0; --b) put_bit(buf, pos, (u >> b) & 1u);
    } else {
        for (int i = 0; i < 15; ++i) put_bit(buf, pos, 1u);
        for (int b = raw_bits - 1; b >= 0; --b) put_bit(buf, pos, (u >> b) & 1u);
    }
}

static unsigned rice_get(const uint8_t *buf, size_t *pos, int k, int raw_bits)
{
    unsigned quo = 0;
    while (quo < 15u && get_bit(buf, pos)) ++quo;             /* stops after the zero-bit, or after 15 one-bits */
    unsigned u = 0;
    if (quo < 15u) {
        for (int b = 0; b < k; ++b) u = (u << 1) | get_bit(buf, pos);
        return (quo << k) | u;
    }
    for (int b = 0; b < raw_bits; ++b) u = (u << 1) | get_bit(buf, pos);
    return u;
}

/* R9: the symbol of code t of a group under `mode`. */
static unsigned td_symbol(const int8_t *q, int t, int mode)
{
    int prev = (mode == 1 && t > 0) ? q[t - 1] : 0;
    return kdn_oracle_zigzag((int)q[t] - prev);
}

/* R9: encode the n <= 64 codes of one group into out (at least kdn_oracle_td_max_len(qmax) bytes, zeroed here).
 * *len_out = bytes used, *param_out = mode * 8 + k. */
void kdn_oracle_td_encode_channel(const int8_t *q, int n, int qmax, uint8_t *out, int *len_out, int *param_out)
{
    int raw_bits = td_raw_bits(qmax);
    long best_bits = -1;
    int best_mode = 0, best_k = 0;
    for (int mode = 0; mode < 2; ++mode)
        for (int k = 0; k < 8; ++k) {
            long bits = 0;
            for (int t = 0; t < n; ++t) bits += kdn_oracle_rice_bits(td_symbol(q, t, mode), k, raw_bits);
            if (best_bits < 0 || bits < best_bits) { best_bits = bits; best_mode = mode; best_k = k; }
        }
    memset(out, 0, (size_t)kdn_oracle_td_max_len(qmax));
    size_t pos = 0;
    for (int t = 0; t < n; ++t) rice_put(out, &pos, td_symbol(q, t, best_mode), best_k, raw_bits);
    *len_out = (int)((pos + 7u) / 8u);
    *param_out = best_mode * 8 + best_k;
}

/* R9: decode n codes of one group. */
void kdn_oracle_td_decode_channel(const uint8_t *in, int param, int n, int qmax, int8_t *q)
{
    int mode = param >> 3, k = param & 7, raw_bits = td_raw_bits(qmax);
    size_t pos = 0;
    int prev = 0;
    for (int t = 0; t < n; ++t) {
        int e = kdn_oracle_unzigzag(rice_get(in, &pos, k, raw_bits));
        int v = mode == 1 ? prev + e : e;
        q[t] = (int8_t)v;
        prev = v;
    }
}

/* ------------------------------------------------------------- rotation -- */

/* R6: angle of frequency index i (0 <= i < D/2) for a position shift delta. */
double kdn_oracle_rope_angle(int64_t delta, double theta, int i, int D)
{
    double inv_freq = pow(theta, -2.0 * (double)i / (double)D);
    return (double)delta * inv_freq;
}

/* R6: rotate the pair (u, w) = (k[i], k[i + D/2]) by phi. */
void kdn_oracle_rotate_pair(double u, double w, double phi, double *u_out, double *w_out)
{
    double c = cos(phi), s = sin(phi);
    *u_out = u * c - w * s;
    *w_out = w * c + u * s;
}

/* ------------------------------------------------------- index helpers -- */

typedef struct {
    int L, H, D, bs;
    int64_t nb;
} shape_t;

/* R1: element offset of pool[l][kv][block][slot][h][d]. */
static size_t pool_index(const shape_t *s, int l, int kv, int64_t block, int slot, int h, int d)
{
    size_t i = (size_t)l;
    i = i * 2u + (size_t)kv;
    i = i * (size_t)s->nb + (size_t)block;
    i = i * (size_t)s->bs + (size_t)slot;
    i = i * (size_t)s->H + (size_t)h;
    i = i * (size_t)s->D + (size_t)d;
    return i;
}

/* R2: element offset of chunk[l][kv][t][h][d] for a chunk of T tokens. */
static size_t chunk_index(const shape_t *s, int T, int l, int kv, int t, int h, int d)
{
    size_t i = (size_t)l;
    i = i * 2u + (size_t)kv;
    i = i * (size_t)T + (size_t)t;
    i = i * (size_t)s->H + (size_t)h;
    i = i * (size_t)s->D + (size_t)d;
    return i;
}

/* Validate one transfer of n listed tokens: token i sits at position off + (list ? list[i] : i). */
static int check_args_list(const shape_t *s, const int32_t *table, int n_table, int64_t off, int n, int codec,
                           const int32_t *list, int list_bound)
{
    if (s->L <= 0 || s->H <= 0 || s->D <= 0 || s->bs <= 0 || s->nb <= 0) return 1;
    if (n < 0 || off < 0 || n_table < 0) return 1;
    if (codec < KDN_ORACLE_RAW_BF16 || codec > KDN_ORACLE_INT4_TD64) return 3;
    if (codec != KDN_ORACLE_RAW_BF16 && s->D % KDN_ORACLE_GROUP) return 3;
    for (int i = 0; i < n; ++i) {
        int64_t rel = list ? list[i] : i;
        if (rel < 0 || (list && i > 0 && list[i] <= list[i - 1])) return 5;       /* strictly increasing */
        if (list_bound >= 0 && rel >= list_bound) return 5;
        int64_t p = off + rel;
        if (p >= (int64_t)n_table * (int64_t)s->bs) return 2;
        int32_t b = table[p / s->bs];
        if (b < 0 || (int64_t)b >= s->nb) return 4;
    }
    return 0;
}

/* R4": float index of the scale of chunk element (l, kv, t, head*D + d) in the scales area of a per-channel-key chunk. */
static size_t kc_scale_index(const shape_t *s, int T, int l, int kv, int t, size_t ch)
{
    size_t hd = (size_t)s->H * (size_t)s->D;
    size_t n_groups = ((size_t)T + KDN_ORACLE_GROUP - 1u) / KDN_ORACLE_GROUP;
    size_t per_layer = n_groups * hd + (size_t)T * hd / KDN_ORACLE_GROUP;
    if (kv == 0) return (size_t)l * per_layer + (size_t)(t / KDN_ORACLE_GROUP) * hd + ch;
    return (size_t)l * per_layer + n_groups * hd + ((size_t)t * hd + ch) / KDN_ORACLE_GROUP;
}

static void put_code(uint8_t *chunk, int int4, size_t c, int8_t q)
{
    if (!int4) { ((int8_t *)chunk)[c] = q; return; }
    uint8_t *b = chunk + c / 2u;
    if (c & 1u) *b = (uint8_t)((*b & 0x0fu) | (((uint8_t)q & 0x0fu) << 4));
    else *b = (uint8_t)((*b & 0xf0u) | ((uint8_t)q & 0x0fu));
}

/* R4": store with keys grouped along tokens and values grouped along head_dim. */
static int store_kc(const shape_t *s, const uint16_t *pool, const int32_t *table, int64_t off, int T, int codec,
                    const int32_t *keep, uint8_t *chunk)
{
    int int4 = codec == KDN_ORACLE_INT4_KC64;
    int qmax = int4 ? 7 : 127;
    size_t hd = (size_t)s->H * (size_t)s->D;
    size_t elems = (size_t)s->L * 2u * (size_t)T * hd;
    float *scales = (float *)(chunk + (int4 ? elems / 2u : elems));
    if (int4) memset(chunk, 0, elems / 2u);
    for (int l = 0; l < s->L; ++l) {
        /* keys: one group per (64-token span, channel) */
        for (int t0 = 0; t0 < T; t0 += KDN_ORACLE_GROUP) {
            int n = T - t0 < KDN_ORACLE_GROUP ? T - t0 : KDN_ORACLE_GROUP;
            for (int h = 0; h < s->H; ++h)
                for (int d = 0; d < s->D; ++d) {
                    uint16_t x[KDN_ORACLE_GROUP];
                    int8_t q[KDN_ORACLE_GROUP];
                    for (int i = 0; i < n; ++i) {
                        int64_t p = off + (keep ? keep[t0 + i] : t0 + i);                 /* R7: the listed tokens */
                        x[i] = pool[pool_index(s, l, 0, table[p / s->bs], (int)(p % s->bs), h, d)];
                    }
                    size_t ch = (size_t)h * (size_t)s->D + (size_t)d;
                    kdn_oracle_quant_channel(x, n, qmax, q, scales + kc_scale_index(s, T, l, 0, t0, ch));
                    for (int i = 0; i < n; ++i) put_code(chunk, int4, chunk_index(s, T, l, 0, t0 + i, h, d), q[i]);
                }
        }
        /* values: R4 / R4' */
        for (int t = 0; t < T; ++t) {
            int64_t p = off + (keep ? keep[t] : t);
            int64_t block = table[p / s->bs];
            int slot = (int)(p % s->bs);
            for (int h = 0; h < s->H; ++h)
                for (int g = 0; g < s->D / KDN_ORACLE_GROUP; ++g) {
                    int8_t q[KDN_ORACLE_GROUP];
                    size_t src = pool_index(s, l, 1, block, slot, h, g * KDN_ORACLE_GROUP);
                    size_t ch = (size_t)h * (size_t)s->D + (size_t)g * KDN_ORACLE_GROUP;
                    quant_group_q(pool + src, q, scales + kc_scale_index(s, T, l, 1, t, ch), (float)qmax);
                    for (int i = 0; i < KDN_ORACLE_GROUP; ++i)
                        put_code(chunk, int4, chunk_index(s, T, l, 1, t, h, g * KDN_ORACLE_GROUP + i), q[i]);
                }
        }
    }
    return 0;
}

/* R9: store with K and V grouped along tokens, every group's codes written as a Rice-coded sub-stream. */
static int store_td(const shape_t *s, const uint16_t *pool, const int32_t *table, int64_t off, int T, int codec,
                    const int32_t *keep, uint8_t *chunk)
{
    int qmax = td_qmax(codec);
    size_t lay[6];
    if (kdn_oracle_td_layout(s->L, s->H, s->D, T, codec, lay)) return 3;
    size_t R = (size_t)s->H * (size_t)s->D;
    int G = (T + KDN_ORACLE_GROUP - 1) / KDN_ORACLE_GROUP;
    uint64_t *seg_off = (uint64_t *)chunk;
    float *scales = (float *)(chunk + lay[1]);
    uint8_t *lens = chunk + lay[2], *params = chunk + lay[3];
    size_t cursor = lay[4];                                  /* where the next sub-stream goes */
    memset(chunk, 0, lay[4]);
    for (int l = 0; l < s->L; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int g = 0; g < G; ++g) {
                size_t seg = ((size_t)l * 2u + (size_t)kv) * (size_t)G + (size_t)g;
                int t0 = g * KDN_ORACLE_GROUP;
                int n = T - t0 < KDN_ORACLE_GROUP ? T - t0 : KDN_ORACLE_GROUP;
                seg_off[seg] = (uint64_t)cursor;
                for (int h = 0; h < s->H; ++h)
                    for (int d = 0; d < s->D; ++d) {
                        uint16_t x[KDN_ORACLE_GROUP];
                        int8_t q[KDN_ORACLE_GROUP];
                        uint8_t bytes[72];
                        int len, param;
                        for (int i = 0; i < n; ++i) {
                            int64_t p = off + (keep ? keep[t0 + i] : t0 + i);             /* R7: the listed tokens */
                            x[i] = pool[pool_index(s, l, kv, table[p / s->bs], (int)(p % s->bs), h, d)];
                        }
                        size_t ch = (size_t)h * (size_t)s->D + (size_t)d;
                        kdn_oracle_quant_channel(x, n, qmax, q, scales + seg * R + ch);
                        kdn_oracle_td_encode_channel(q, n, qmax, bytes, &len, &param);
                        lens[seg * R + ch] = (uint8_t)len;
                        params[seg * R + ch] = (uint8_t)param;
                        memcpy(chunk + cursor, bytes, (size_t)len);
                        cursor += (size_t)len;
                    }
                while (cursor % 16u) chunk[cursor++] = 0;    /* a segment ends on a 16-byte boundary */
            }
    seg_off[(size_t)s->L * 2u * (size_t)G] = (uint64_t)cursor;
    return 0;
}

/* R9: all codes of a token-delta chunk as plain int8 codes[l][kv][t][head][d] (malloc'ed; NULL when out of memory). */
static int8_t *td_unpack(const shape_t *s, int T, int codec, const uint8_t *chunk)
{
    size_t lay[6];
    if (kdn_oracle_td_layout(s->L, s->H, s->D, T, codec, lay)) return NULL;
    size_t R = (size_t)s->H * (size_t)s->D;
    int G = (T + KDN_ORACLE_GROUP - 1) / KDN_ORACLE_GROUP;
    const uint64_t *seg_off = (const uint64_t *)chunk;
    const uint8_t *lens = chunk + lay[2], *params = chunk + lay[3];
    int8_t *codes = (int8_t *)malloc((size_t)s->L * 2u * (size_t)T * R + 1u);
    if (!codes) return NULL;
    for (int l = 0; l < s->L; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int g = 0; g < G; ++g) {
                size_t seg = ((size_t)l * 2u + (size_t)kv) * (size_t)G + (size_t)g;
                int t0 = g * KDN_ORACLE_GROUP;
                int n = T - t0 < KDN_ORACLE_GROUP ? T - t0 : KDN_ORACLE_GROUP;
                size_t cursor = (size_t)seg_off[seg];
                for (size_t ch = 0; ch < R; ++ch) {
                    int8_t q[KDN_ORACLE_GROUP];
                    kdn_oracle_td_decode_channel(chunk + cursor, params[seg * R + ch], n, td_qmax(codec), q);
                    for (int i = 0; i < n; ++i)
                        codes[(((size_t)l * 2u + (size_t)kv) * (size_t)T + (size_t)(t0 + i)) * R + ch] = q[i];
                    cursor += lens[seg * R + ch];
                }
            }
    return codes;
}

/* ---------------------------------------------------------------- store -- */

/* Sec. 3.2 call (i): gather T tokens starting at request position `off` out
 * of the paged pool (R1, R3) into one chunk (R2), optionally int8-coded (R4).
 * Returns 0, or a small positive code for bad arguments (nothing written). */
int kdn_oracle_store_sparse(const uint16_t *pool, int L, int H, int D, int bs, int64_t nb,
                            const int32_t *table, int n_table, int64_t off, int T, int codec,
                            const int32_t *keep, uint8_t *chunk)
{
    shape_t s = { L, H, D, bs, nb };
    int rc = check_args_list(&s, table, n_table, off, T, codec, keep, -1);
    if (rc) return rc;
    size_t elems = (size_t)L * 2u * (size_t)T * (size_t)H * (size_t)D;
    if (codec == KDN_ORACLE_INT8_KC64 || codec == KDN_ORACLE_INT4_KC64)
        return store_kc(&s, pool, table, off, T, codec, keep, chunk);
    if (td_is(codec)) return store_td(&s, pool, table, off, T, codec, keep, chunk);
    uint16_t *raw = (uint16_t *)chunk;
    int8_t *codes = (int8_t *)chunk;
    float *scales = (float *)(chunk + (codec == KDN_ORACLE_INT4_G64 ? elems / 2u : elems));
    for (int l = 0; l < L; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int t = 0; t < T; ++t) {
                int64_t p = off + (keep ? keep[t] : t);             /* R3, R7 */
                int64_t block = table[p / bs];
                int slot = (int)(p % bs);
                for (int h = 0; h < H; ++h) {
                    if (codec == KDN_ORACLE_INT4_G64) {
                        for (int g = 0; g < D / KDN_ORACLE_GROUP; ++g) {
                            size_t src = pool_index(&s, l, kv, block, slot, h, g * KDN_ORACLE_GROUP);
                            size_t dst = chunk_index(&s, T, l, kv, t, h, g * KDN_ORACLE_GROUP);
                            kdn_oracle_quant4_group(pool + src, chunk + dst / 2u, scales + dst / KDN_ORACLE_GROUP);
                        }
                    } else if (codec == KDN_ORACLE_RAW_BF16) {
                        for (int d = 0; d < D; ++d)
                            raw[chunk_index(&s, T, l, kv, t, h, d)] =
                                pool[pool_index(&s, l, kv, block, slot, h, d)];
                    } else {
                        for (int g = 0; g < D / KDN_ORACLE_GROUP; ++g) {
                            size_t src = pool_index(&s, l, kv, block, slot, h, g * KDN_ORACLE_GROUP);
                            size_t dst = chunk_index(&s, T, l, kv, t, h, g * KDN_ORACLE_GROUP);
                            kdn_oracle_quant_group(pool + src, codes + dst, scales + dst / KDN_ORACLE_GROUP);
                        }
                    }
                }
            }
    return 0;
}

/* Sec. 3.2 call (i) for a whole span: every token, in order. */
int kdn_oracle_store(const uint16_t *pool, int L, int H, int D, int bs, int64_t nb,
                     const int32_t *table, int n_table, int64_t off, int T, int codec,
                     uint8_t *chunk)
{
    return kdn_oracle_store_sparse(pool, L, H, D, bs, nb, table, n_table, off, T, codec, NULL, chunk);
}

/* The stored value of chunk element c before any bf16 rounding: code and scale (raw: the bf16 itself). */
static void stored_code(const uint8_t *chunk, size_t elems, int codec, size_t c, int *q, float *scale,
                        const shape_t *s, int T, const int8_t *unpacked)
{
    if (td_is(codec)) {                                    /* R9: codes from td_unpack, one scale per (segment, channel) */
        size_t lay[6];
        kdn_oracle_td_layout(s->L, s->H, s->D, T, codec, lay);
        size_t hd = (size_t)s->H * (size_t)s->D;
        size_t ch = c % hd, row = c / hd;                  /* row = (l * 2 + kv) * T + t */
        size_t t = row % (size_t)T, plane = row / (size_t)T;
        size_t G = ((size_t)T + KDN_ORACLE_GROUP - 1u) / KDN_ORACLE_GROUP;
        *q = unpacked[c];
        *scale = ((const float *)(chunk + lay[1]))[(plane * G + t / KDN_ORACLE_GROUP) * hd + ch];
        return;
    }
    if (codec == KDN_ORACLE_INT8_KC64 || codec == KDN_ORACLE_INT4_KC64) {           /* R4" */
        int int4 = codec == KDN_ORACLE_INT4_KC64;
        size_t hd = (size_t)s->H * (size_t)s->D;
        size_t ch = c % hd, row = c / hd;                  /* row = (l * 2 + kv) * T + t */
        int t = (int)(row % (size_t)T), kv = (int)((row / (size_t)T) & 1u), l = (int)(row / (size_t)T / 2u);
        *q = int4 ? kdn_oracle_nibble(chunk, c) : ((const int8_t *)chunk)[c];
        *scale = ((const float *)(chunk + (int4 ? elems / 2u : elems)))[kc_scale_index(s, T, l, kv, t, ch)];
        return;
    }
    if (codec == KDN_ORACLE_INT8_G64) {
        *q = ((const int8_t *)chunk)[c];
        *scale = ((const float *)(chunk + elems))[c / KDN_ORACLE_GROUP];
    } else {                                       /* int4 */
        *q = kdn_oracle_nibble(chunk, c);
        *scale = ((const float *)(chunk + elems / 2u))[c / KDN_ORACLE_GROUP];
    }
}

/* R5: the bf16 a retrieve writes for chunk element c. */
static uint16_t decoded(const uint8_t *chunk, size_t elems, int codec, size_t c, const shape_t *s, int T,
                        const int8_t *unpacked)
{
    if (codec == KDN_ORACLE_RAW_BF16) return ((const uint16_t *)chunk)[c];
    int q;
    float scale;
    stored_code(chunk, elems, codec, c, &q, &scale, s, T, unpacked);
    return kdn_oracle_dequant((int8_t)q, scale);
}

/* ------------------------------------------------------------- retrieve -- */

/* Sec. 3.2 call (ii) with Sec. 3.1's decompression on the GPU: scatter a
 * chunk back into the pool blocks the table names, decoding int8 (R5).  Only
 * the T addressed token slots are written. */
int kdn_oracle_retrieve_sparse(uint16_t *pool, int L, int H, int D, int bs, int64_t nb,
                               const int32_t *table, int n_table, int64_t off, int T, int codec,
                               const int32_t *keep, const uint8_t *chunk)
{
    shape_t s = { L, H, D, bs, nb };
    int rc = check_args_list(&s, table, n_table, off, T, codec, keep, -1);
    if (rc) return rc;
    size_t elems = (size_t)L * 2u * (size_t)T * (size_t)H * (size_t)D;
    int8_t *unpacked = NULL;
    if (td_is(codec) && T > 0) {
        unpacked = td_unpack(&s, T, codec, chunk);
        if (!unpacked) return 6;
    }
    for (int l = 0; l < L; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int t = 0; t < T; ++t) {
                int64_t p = off + (keep ? keep[t] : t);
                int64_t block = table[p / bs];
                int slot = (int)(p % bs);
                for (int h = 0; h < H; ++h)
                    for (int d = 0; d < D; ++d) {
                        size_t c = chunk_index(&s, T, l, kv, t, h, d);
                        size_t o = pool_index(&s, l, kv, block, slot, h, d);
                        pool[o] = decoded(chunk, elems, codec, c, &s, T, unpacked);
                    }
            }
    free(unpacked);
    return 0;
}

int kdn_oracle_retrieve(uint16_t *pool, int L, int H, int D, int bs, int64_t nb,
                        const int32_t *table, int n_table, int64_t off, int T, int codec,
                        const uint8_t *chunk)
{
    return kdn_oracle_retrieve_sparse(pool, L, H, D, bs, nb, table, n_table, off, T, codec, NULL, chunk);
}

/* -------------------------------------------------------------- compose -- */

/* Sec. 3.1 blending module / Sec. 3.2 "KV-cache blending": place n_parts
 * chunks into one request's blocks, part j at positions dst_pos[j] + t, and
 * re-rotate the keys of every part whose delta = dst_pos - base_pos is not
 * zero (R6).  Values, and keys with delta == 0, are exactly a retrieve.
 *
 * For rotated keys the result is computed in fp64 from the stored value (raw
 * bf16, or the UNROUNDED product q * scale for int8) and written to the pool
 * rounded once to bf16.  When kref / kmag are not NULL they receive, for every
 * key element of every part (rotated or not), the fp64 result and |u| + |w| of
 * its pair, laid out [l][position][h][d] over the n_table * bs request
 * positions; entries no part covers are left as the caller set them.
 */
int kdn_oracle_compose_select(uint16_t *pool, int L, int H, int D, int bs, int64_t nb,
                              const int32_t *table, int n_table, int n_parts,
                              const uint8_t *const *chunks, const int32_t *part_T, const int32_t *part_codec,
                              const int64_t *base_pos, const int64_t *dst_pos, double theta,
                              const int32_t *const *part_sel, const int32_t *part_nsel,
                              double *kref, double *kmag)
{
    shape_t s = { L, H, D, bs, nb };
    if (n_parts < 0) return 1;
    if (D % 2) return 3;
    for (int j = 0; j < n_parts; ++j) {
        const int32_t *sel = part_sel ? part_sel[j] : NULL;
        int rc = check_args_list(&s, table, n_table, dst_pos[j], sel ? part_nsel[j] : part_T[j], part_codec[j], sel, part_T[j]);
        if (rc) return rc;
    }
    int64_t P = (int64_t)n_table * bs;
    int half = D / 2;
    for (int j = 0; j < n_parts; ++j) {
        int T = part_T[j];
        int codec = part_codec[j];
        int64_t delta = dst_pos[j] - base_pos[j];
        size_t elems = (size_t)L * 2u * (size_t)T * (size_t)H * (size_t)D;
        const uint16_t *raw = (const uint16_t *)chunks[j];
        const int32_t *sel = part_sel ? part_sel[j] : NULL;
        int n_deliver = sel ? part_nsel[j] : T;
        int8_t *unpacked = NULL;
        if (td_is(codec) && T > 0) {
            unpacked = td_unpack(&s, T, codec, chunks[j]);
            if (!unpacked) return 6;
        }
        for (int l = 0; l < L; ++l)
            for (int kv = 0; kv < 2; ++kv)
                for (int i_sel = 0; i_sel < n_deliver; ++i_sel) {
                    int t = sel ? sel[i_sel] : i_sel;                 /* R7: only the listed chunk tokens */
                    int64_t p = dst_pos[j] + t;
                    int64_t block = table[p / bs];
                    int slot = (int)(p % bs);
                    for (int h = 0; h < H; ++h) {
                        int rotate = (kv == 0 && delta != 0);
                        if (!rotate) {
                            for (int d = 0; d < D; ++d) {
                                size_t c = chunk_index(&s, T, l, kv, t, h, d);
                                size_t o = pool_index(&s, l, kv, block, slot, h, d);
                                pool[o] = decoded(chunks[j], elems, codec, c, &s, T, unpacked);
                                if (kv == 0 && kref) {
                                    size_t r = (((size_t)l * (size_t)P + (size_t)p) * (size_t)H + (size_t)h) * (size_t)D + (size_t)d;
                                    kref[r] = (double)kdn_oracle_bf16_to_f32(pool[o]);
                                    if (kmag) kmag[r] = 0.0;
                                }
                            }
                            continue;
                        }
                        for (int i = 0; i < half; ++i) {
                            size_t cu = chunk_index(&s, T, l, 0, t, h, i);
                            size_t cw = chunk_index(&s, T, l, 0, t, h, i + half);
                            double u, w;
                            if (codec == KDN_ORACLE_RAW_BF16) {
                                u = (double)kdn_oracle_bf16_to_f32(raw[cu]);
                                w = (double)kdn_oracle_bf16_to_f32(raw[cw]);
                            } else {
                                int qu, qw;
                                float su, sw;
                                stored_code(chunks[j], elems, codec, cu, &qu, &su, &s, T, unpacked);
                                stored_code(chunks[j], elems, codec, cw, &qw, &sw, &s, T, unpacked);
                                u = (double)qu * (double)su;
                                w = (double)qw * (double)sw;
                            }
                            double phi = kdn_oracle_rope_angle(delta, theta, i, D);
                            double u2, w2;
                            kdn_oracle_rotate_pair(u, w, phi, &u2, &w2);
                            size_t ou = pool_index(&s, l, 0, block, slot, h, i);
                            size_t ow = pool_index(&s, l, 0, block, slot, h, i + half);
                            pool[ou] = kdn_oracle_f64_to_bf16(u2);
                            pool[ow] = kdn_oracle_f64_to_bf16(w2);
                            if (kref) {
                                size_t r = (((size_t)l * (size_t)P + (size_t)p) * (size_t)H + (size_t)h) * (size_t)D;
                                kref[r + (size_t)i] = u2;
                                kref[r + (size_t)i + (size_t)half] = w2;
                                if (kmag) {
                                    kmag[r + (size_t)i] = fabs(u) + fabs(w);
                                    kmag[r + (size_t)i + (size_t)half] = fabs(u) + fabs(w);
                                }
                            }
                        }
                    }
                }
        free(unpacked);
    }
    return 0;
}

int kdn_oracle_compose(uint16_t *pool, int L, int H, int D, int bs, int64_t nb,
                       const int32_t *table, int n_table, int n_parts,
                       const uint8_t *const *chunks, const int32_t *part_T, const int32_t *part_codec,
                       const int64_t *base_pos, const int64_t *dst_pos, double theta,
                       double *kref, double *kmag)
{
    return kdn_oracle_compose_select(pool, L, H, D, bs, nb, table, n_table, n_parts, chunks, part_T, part_codec,
                                     base_pos, dst_pos, theta, NULL, NULL, kref, kmag);
}

/* ------------------------------------------------------- storage shell -- */

/* R8: FNV-1a, 64 bit, over n bytes. */
uint64_t kdn_oracle_fnv1a(const uint8_t *bytes, size_t n)
{
    uint64_t h = 0xcbf29ce484222325ull;
    for (size_t i = 0; i < n; ++i) {
        h ^= bytes[i];
        h *= 0x100000001b3ull;
    }
    return h;
}

/* R8: key of a text given as token ids (each id hashed as its four little-endian bytes). */
uint64_t kdn_oracle_key_hash(const int32_t *tokens, size_t n)
{
    uint64_t h = 0xcbf29ce484222325ull;
    for (size_t i = 0; i < n; ++i) {
        uint32_t t = (uint32_t)tokens[i];
        for (int b = 0; b < 4; ++b) {
            h ^= (t >> (8 * b)) & 0xffu;
            h *= 0x100000001b3ull;
        }
    }
    return h;
}

/* R8: payload checksum; bytes must be a multiple of 4 (every chunk layout is). */
uint64_t kdn_oracle_checksum(const uint8_t *payload, size_t bytes)
{
    uint64_t c = 0;
    for (size_t i = 0; i < bytes / 4; ++i) {
        uint32_t w = (uint32_t)payload[4 * i] | ((uint32_t)payload[4 * i + 1] << 8) |
                     ((uint32_t)payload[4 * i + 2] << 16) | ((uint32_t)payload[4 * i + 3] << 24);
        uint32_t a = w ^ 0x9E3779B9u;
        uint32_t m = (uint32_t)(2u * (uint32_t)i + 1u);
        c += (uint64_t)a * (uint64_t)m;
    }
    return c;
}
