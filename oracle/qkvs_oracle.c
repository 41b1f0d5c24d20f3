/*
 * CPU oracle for the CacheCard create / inject path.       *** TEST INFRASTRUCTURE ***
 *
 * This file is a plain, slow, scalar restatement of what the path computes, written to be
 * checked against the method's definition by eye.  It is not part of the product: only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.  It shares no
 * code, header, table or constant generator with the CUDA library; every constant below is
 * typed out here on its own.
 *
 * What the paper fixes (Sections 3.1, 3.3, 4.2.1, 4.2.2): a card holds the keys and values
 * as quantised groups, the per-token bit-width vector b(t) in {2,4,8,16} (16 = FP16 kept
 * as is), the sequence length, model and sender identifiers, a position-offset placeholder
 * and the achieved average bit-width; injection rebuilds FP16 keys and values in the
 * [heads, tokens, head_dim] layout of a HuggingFace cache.  The paper gives no formula,
 * group size, rounding rule or byte layout; the readings taken here are:
 *   - groups of 32 consecutive channels along head_dim, for K and V alike;
 *   - asymmetric min/max: zero = group minimum (fp32), scale = (max-min)/(2^b-1) (fp32);
 *   - codes q = clamp(rint((x-zero) * inv), 0, 2^b-1), inv = (2^b-1)/(max-min), one IEEE
 *     binary32 operation per step, round-to-nearest-even everywhere, nothing fused;
 *   - a constant group has scale = inv = 0 and all-zero codes; a zero minimum is stored +0;
 *   - reconstruction x^ = fp16_rne( fl32(fl32(q) * scale) + zero );
 *   - the byte layout described at write_prefix() / encode_record() below;
 *   - a compact variant that stores {scale, zero} as two FP16 values (zero exactly, scale rounded
 *     up), defined at orc_quantize_group_compact(); the paper's "about 0.5 bytes per element at
 *     4 bits" (Section 3.1) leaves no room for 8 bytes of metadata per 32 elements.
 * NaN or infinity inside a quantised (b < 16) token is outside the definition (codes are
 * then unspecified); inside an FP16 token the bit patterns are preserved.
 *
 * Pins (see tests): closed-form size, uniform offsets, brute-force scan, FP16 round trip,
 * |x - x^| <= scale/2 (+ rounding slack), min -> code 0 / max -> code 2^b-1, monotone codes,
 * hand-worked 2-bit and 4-bit groups with exact ties, exact-rational recomputation of codes,
 * the 8-bit case against the textbook affine uint8 quantiser, all-FP16 card == memcpy;
 * attention from the card: one token -> its value row, equal value rows -> that row, zero query
 * -> the mean of the value rows, a card of FP16 tokens -> the library softmax attention on the
 * original cache, one dominant key -> its value row.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* status values (same numbering as the library's public header, typed here separately) */
enum { ORC_OK = 0, ORC_INVALID_ARG = 1, ORC_UNSUPPORTED_SHAPE = 2, ORC_BAD_BITS = 3,
       ORC_BUFFER_TOO_SMALL = 4, ORC_BAD_CARD = 5 };

typedef struct {
    int32_t n_layers, n_kv_heads, head_dim, n_tokens;
    int32_t group_size; /* 32, or 64 / 128 (wider-group variant) */
    int32_t bits_mode;  /* 0: one bits[T] for the whole model; 1: bits[L*H][T] */
    int64_t head_stride;  /* elements between heads  */
    int64_t token_stride; /* elements between tokens */
    int32_t meta_bytes;   /* bytes of {scale, zero} per group: 8 (fp32 pair; 0 means 8) or 4 (FP16 pair) */
    int32_t reserved_;
} orc_layout;

static int meta_of(const orc_layout *L) { return L->meta_bytes == 0 ? 8 : L->meta_bytes; }
static int group_of(const orc_layout *L) { return L->group_size; }

/* ------------------------------------------------------------------ FP16 <-> FP32 */

/* Exact: every FP16 value is an FP32 value. */
float orc_half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    uint32_t e = (uint32_t)(h >> 10) & 31u;
    uint32_t m = (uint32_t)h & 1023u;
    float v;
    if (e == 31u) { /* infinity / NaN: keep the payload */
        uint32_t b = (sign << 31) | 0x7f800000u | (m << 13);
        memcpy(&v, &b, 4);
        return v;
    }
    if (e == 0u)
        v = (float)ldexp((double)m, -24);            /* subnormal: m * 2^-24 */
    else
        v = (float)ldexp((double)(1024u + m), (int)e - 25); /* 1.m * 2^(e-15) */
    return sign ? -v : v;
}

/* Round-to-nearest-even conversion of a binary32 value to FP16. */
uint16_t orc_float_to_half(float f)
{
    uint32_t b;
    memcpy(&b, &f, 4);
    uint16_t sign = (uint16_t)((b >> 31) << 15);
    uint32_t mag = b & 0x7fffffffu;
    if (mag > 0x7f800000u) return (uint16_t)(sign | 0x7e00u | ((mag >> 13) & 0x3ffu)); /* NaN */
    double v = fabs((double)f);
    if (v >= 65520.0) return (uint16_t)(sign | 0x7c00u); /* halfway to 65536 rounds to inf */
    if (v < 6.103515625e-05) {                           /* below 2^-14: multiples of 2^-24 */
        double r = nearbyint(v * 16777216.0);            /* ties to even; 1024 -> smallest normal */
        return (uint16_t)(sign | (uint16_t)r);
    }
    int e2;
    (void)frexp(v, &e2);      /* v = frac * 2^e2, frac in [0.5, 1) -> v = 1.x * 2^(e2-1) */
    int E = e2 - 1;
    double r = nearbyint(ldexp(v, 10 - E)); /* in [1024, 2048], ties to even */
    if (r == 2048.0) { r = 1024.0; E += 1; }
    return (uint16_t)(sign | (uint16_t)((E + 15) << 10) | (uint16_t)((int)r - 1024));
}

/* ------------------------------------------------------------------ sizes and offsets */

static uint64_t round_up_256(uint64_t x) { return (x + 255u) / 256u * 256u; }

/* Bytes of one token row inside one stream: d/group (scale, zero) pairs of `meta` bytes each (8: two
 * fp32; 4: two FP16), then the packed codes; an FP16 token is the row itself.  Code bytes alone
 * are d*b/8 (Section 3.1's bytes-per-element law).  With groups of 32 channels the pairs take
 * meta*d/32 bytes, which the supported shapes keep a multiple of 16; with the wider groups of 64
 * or 128 channels (fewer pairs: Section 3.1's 0.5 bytes per element is approached as the metadata
 * shrinks) the pairs are followed by zero bytes up to the next multiple of 16, so that the codes
 * start, and every record ends, on a 16-byte boundary as before. */
int64_t orc_record_bytes_g(int head_dim, int b, int meta, int group)
{
    if (meta != 8 && meta != 4) return -1;
    if (group != 32 && group != 64 && group != 128) return -1;
    if (head_dim % group != 0) return -1;
    if (b == 16) return 2 * (int64_t)head_dim;
    if (b == 2 || b == 4 || b == 8) {
        int64_t pairs = (int64_t)meta * (head_dim / group);
        if (group != 32) pairs = (pairs + 15) / 16 * 16;
        return (int64_t)head_dim * b / 8 + pairs;
    }
    return -1;
}

int64_t orc_record_bytes(int head_dim, int b, int meta) { return orc_record_bytes_g(head_dim, b, meta, 32); }

/* where the code bytes begin inside a record */
static int64_t codes_at(int head_dim, int meta, int group) { return orc_record_bytes_g(head_dim, 4, meta, group) - head_dim / 2; }

static int layout_ok(const orc_layout *L)
{
    if (!L) return ORC_INVALID_ARG;
    if (L->n_layers < 1 || L->n_kv_heads < 1 || L->n_tokens < 0) return ORC_INVALID_ARG;
    if (L->bits_mode != 0 && L->bits_mode != 1) return ORC_INVALID_ARG;
    if (L->group_size != 32 && L->group_size != 64 && L->group_size != 128) return ORC_UNSUPPORTED_SHAPE;
    if (L->head_dim % L->group_size != 0) return ORC_UNSUPPORTED_SHAPE;
    if (L->head_dim < 64 || L->head_dim % 64 != 0) return ORC_UNSUPPORTED_SHAPE;
    if (meta_of(L) != 8 && meta_of(L) != 4) return ORC_INVALID_ARG;
    /* records stay multiples of 16 bytes: FP16 pairs need head_dim to be a multiple of 128 */
    if (meta_of(L) == 4 && L->group_size == 32 && L->head_dim % 128 != 0) return ORC_UNSUPPORTED_SHAPE;
    return ORC_OK;
}

static int64_t n_segments(const orc_layout *L)
{
    return L->bits_mode == 0 ? 1 : (int64_t)L->n_layers * L->n_kv_heads;
}

/* stream index of (layer, kv, head); kv 0 = K, 1 = V */
static int64_t stream_index(const orc_layout *L, int l, int kv, int h)
{
    return ((int64_t)l * 2 + kv) * L->n_kv_heads + h;
}

static int64_t segment_of(const orc_layout *L, int l, int h)
{
    return L->bits_mode == 0 ? 0 : (int64_t)l * L->n_kv_heads + h;
}

/* Exclusive prefix sum of record sizes over one segment: off[0] = 0,
 * off[t+1] = off[t] + rec(b_t).  Returns ORC_BAD_BITS on a value outside {2,4,8,16}. */
int orc_scan_offsets_g(int head_dim, int meta, int group, const uint8_t *bits, int64_t n_tokens, uint32_t *off,
                       uint64_t *sum_bits)
{
    if (orc_record_bytes_g(head_dim, 16, meta, group) < 0) return ORC_INVALID_ARG;
    uint64_t run = 0, sb = 0;
    off[0] = 0;
    for (int64_t t = 0; t < n_tokens; ++t) {
        int64_t r = orc_record_bytes_g(head_dim, bits[t], meta, group);
        if (r < 0) return ORC_BAD_BITS;
        run += (uint64_t)r;
        sb += bits[t];
        off[t + 1] = (uint32_t)run;
    }
    if (sum_bits) *sum_bits = sb;
    return ORC_OK;
}

int orc_scan_offsets(int head_dim, int meta, const uint8_t *bits, int64_t n_tokens, uint32_t *off, uint64_t *sum_bits)
{
    return orc_scan_offsets_g(head_dim, meta, 32, bits, n_tokens, off, sum_bits);
}

/* Section sizes.  Card = header (256) | bits | offsets | [stream bases, mode 1] | payload. */
static void section_offsets(const orc_layout *L, uint64_t *bits_off, uint64_t *offs_off,
                            uint64_t *sbase_off, uint64_t *payload_off)
{
    uint64_t nseg = (uint64_t)n_segments(L), T = (uint64_t)L->n_tokens;
    uint64_t S = 2u * (uint64_t)L->n_layers * (uint64_t)L->n_kv_heads;
    *bits_off = 256;
    *offs_off = *bits_off + round_up_256(nseg * T);
    uint64_t after = *offs_off + round_up_256(4u * nseg * (T + 1u));
    if (L->bits_mode == 1) {
        *sbase_off = after;
        after += round_up_256(8u * (S + 1u));
    } else {
        *sbase_off = 0;
    }
    *payload_off = after;
}

/* Exact card size for a bit-width vector (host memory); bits == NULL gives the worst case
 * (every token FP16). */
int orc_card_size(const orc_layout *L, const uint8_t *bits, uint64_t *out_bytes)
{
    int st = layout_ok(L);
    if (st) return st;
    uint64_t bo, oo, so, po;
    section_offsets(L, &bo, &oo, &so, &po);
    uint64_t payload = 0;
    int64_t nseg = n_segments(L);
    for (int64_t seg = 0; seg < nseg; ++seg) {
        uint64_t seg_bytes = 0;
        for (int64_t t = 0; t < L->n_tokens; ++t) {
            int64_t r = orc_record_bytes_g(L->head_dim, bits ? bits[seg * L->n_tokens + t] : 16, meta_of(L), group_of(L));
            if (r < 0) return ORC_BAD_BITS;
            seg_bytes += (uint64_t)r;
        }
        /* mode 0: the one segment serves all 2*L*H streams; mode 1: K and V of (l,h) */
        payload += seg_bytes * (L->bits_mode == 0 ? 2u * (uint64_t)L->n_layers * L->n_kv_heads : 2u);
    }
    *out_bytes = po + payload;
    return ORC_OK;
}

/* ------------------------------------------------------------------ little-endian stores */

static void put_u32(uint8_t *p, uint32_t v)
{
    for (int i = 0; i < 4; ++i) p[i] = (uint8_t)(v >> (8 * i));
}
static void put_u64(uint8_t *p, uint64_t v)
{
    for (int i = 0; i < 8; ++i) p[i] = (uint8_t)(v >> (8 * i));
}
static void put_f32(uint8_t *p, float f)
{
    uint32_t b;
    memcpy(&b, &f, 4);
    put_u32(p, b);
}
static uint32_t get_u32(const uint8_t *p)
{
    uint32_t v = 0;
    for (int i = 0; i < 4; ++i) v |= (uint32_t)p[i] << (8 * i);
    return v;
}
static uint64_t get_u64(const uint8_t *p)
{
    uint64_t v = 0;
    for (int i = 0; i < 8; ++i) v |= (uint64_t)p[i] << (8 * i);
    return v;
}
static float get_f32(const uint8_t *p)
{
    uint32_t b = get_u32(p);
    float f;
    memcpy(&f, &b, 4);
    return f;
}
static void put_u16(uint8_t *p, uint16_t v)
{
    p[0] = (uint8_t)(v & 0xff);
    p[1] = (uint8_t)(v >> 8);
}
static uint16_t get_u16(const uint8_t *p) { return (uint16_t)(p[0] | (p[1] << 8)); }

/* ------------------------------------------------------------------ one group of 32 */

/* Quantise one group of n FP16 values (n = 32, 64 or 128) at b in {2,4,8} bits. */
void orc_quantize_span(const uint16_t *x, int n, int b, float *scale_out, float *zero_out, uint8_t *q)
{
    float xf[128] = {0};
    for (int i = 0; i < n; ++i) xf[i] = orc_half_to_float(x[i]);
    float mn = xf[0], mx = xf[0];
    for (int i = 1; i < n; ++i) {
        if (xf[i] < mn) mn = xf[i];
        if (xf[i] > mx) mx = xf[i];
    }
    if (mn == 0.0f) { /* a zero minimum is stored as +0 whatever sign it carried */
        uint32_t z = 0;
        memcpy(&mn, &z, 4);
    }
    int qmax = (1 << b) - 1;
    float qmaxf = (float)qmax;
    float range = mx - mn;
    float scale = 0.0f, inv = 0.0f;
    if (range > 0.0f) {
        scale = range / qmaxf;
        inv = qmaxf / range;
    }
    for (int i = 0; i < n; ++i) {
        float t = xf[i] - mn;
        float u = t * inv;
        float r = nearbyintf(u); /* ties to even (default rounding mode) */
        int qi;
        if (!(r >= 0.0f)) qi = 0;
        else if (r > qmaxf) qi = qmax;
        else qi = (int)r;
        q[i] = (uint8_t)qi;
    }
    *scale_out = scale;
    *zero_out = mn;
}

void orc_quantize_group(const uint16_t *x, int b, float *scale_out, float *zero_out, uint8_t *q)
{
    orc_quantize_span(x, 32, b, scale_out, zero_out, q);
}

/* Smallest FP16 value that is >= f, for finite f >= 0 not above the largest FP16 value:
 * round to nearest, then step one FP16 value up if that landed below f. */
uint16_t orc_float_to_half_up(float f)
{
    uint16_t h = orc_float_to_half(f);
    if (orc_half_to_float(h) < f) h = (uint16_t)(h + 1); /* positive FP16 values order like their bit patterns */
    return h;
}

/* Compact-metadata variant: the group stores {scale, zero} as two FP16 values.
 *   zero  = the group minimum, which is an FP16 value already (kept exactly; -0 stored as +0);
 *   scale = (max-min)/(2^b-1) computed in binary32 as above, then rounded UP to FP16, so that
 *           (x-zero)/scale never exceeds 2^b-1 by more than rounding;
 *   inv   = fl32(1 / scale) with the stored scale, so that the codes are the ones the receiver's
 *           scale implies: q = clamp(rint(fl32((x-zero) * inv)), 0, 2^b-1);
 *   a constant group has scale = inv = 0 and all-zero codes.
 * The largest possible scale, (65504+65504)/3, is below the largest FP16 value, so the rounding
 * up never overflows; the smallest, 2^-24/255, rounds up to the smallest FP16 subnormal 2^-24.
 * Reconstruction is orc_dequantize_group() with the two FP16 values widened to binary32. */
void orc_quantize_span_compact(const uint16_t *x, int n, int b, uint16_t *scale_out, uint16_t *zero_out,
                               uint8_t *q)
{
    float xf[128] = {0};
    for (int i = 0; i < n; ++i) xf[i] = orc_half_to_float(x[i]);
    float mn = xf[0], mx = xf[0];
    uint16_t mn_bits = x[0];
    for (int i = 1; i < n; ++i) {
        if (xf[i] < mn) { mn = xf[i]; mn_bits = x[i]; }
        if (xf[i] > mx) mx = xf[i];
    }
    if (mn == 0.0f) { /* a zero minimum is stored as +0 whatever sign it carried */
        mn = 0.0f;
        mn_bits = 0;
    }
    int qmax = (1 << b) - 1;
    float qmaxf = (float)qmax;
    float range = mx - mn;
    uint16_t scale16 = 0;
    float inv = 0.0f;
    if (range > 0.0f) {
        scale16 = orc_float_to_half_up(range / qmaxf);
        inv = 1.0f / orc_half_to_float(scale16);
    }
    for (int i = 0; i < n; ++i) {
        float t = xf[i] - mn;
        float u = t * inv;
        float r = nearbyintf(u); /* ties to even (default rounding mode) */
        int qi;
        if (!(r >= 0.0f)) qi = 0;
        else if (r > qmaxf) qi = qmax;
        else qi = (int)r;
        q[i] = (uint8_t)qi;
    }
    *scale_out = scale16;
    *zero_out = mn_bits;
}

void orc_quantize_group_compact(const uint16_t *x, int b, uint16_t *scale_out, uint16_t *zero_out, uint8_t *q)
{
    orc_quantize_span_compact(x, 32, b, scale_out, zero_out, q);
}

/* Reconstruct 32 FP16 values: multiply, then add, each rounded to binary32, then to FP16. */
void orc_dequantize_span(const uint8_t *q, int n, float scale, float zero, uint16_t *out)
{
    for (int i = 0; i < n; ++i) {
        float p = (float)q[i] * scale;
        float r = p + zero;
        out[i] = orc_float_to_half(r);
    }
}

void orc_dequantize_group(const uint8_t *q, float scale, float zero, uint16_t *out) { orc_dequantize_span(q, 32, scale, zero, out); }

/* Codes as a little-endian bit string: code i occupies bits [i*b, i*b+b). */
void orc_pack_codes(const uint8_t *q, int n, int b, uint8_t *out)
{
    memset(out, 0, (size_t)n * b / 8);
    for (int i = 0; i < n; ++i) {
        int bit = i * b;
        out[bit / 8] |= (uint8_t)(q[i] << (bit % 8));
    }
}

void orc_unpack_codes(const uint8_t *in, int n, int b, uint8_t *q)
{
    for (int i = 0; i < n; ++i) {
        int bit = i * b;
        q[i] = (uint8_t)((in[bit / 8] >> (bit % 8)) & ((1 << b) - 1));
    }
}

/* ------------------------------------------------------------------ one token row */

/* Record of a b<16 token: G pairs {scale_g, zero_g} (little-endian; two fp32 when meta == 8,
 * two FP16 when meta == 4), group g covering channels 32g..32g+31, then the d*b/8 code bytes of
 * the whole row.  b == 16: the row's FP16 bit patterns verbatim. */
static void encode_record(const uint16_t *row, int d, int b, int meta, int group, uint8_t *rec)
{
    if (b == 16) {
        for (int i = 0; i < d; ++i) {
            rec[2 * i] = (uint8_t)(row[i] & 0xff);
            rec[2 * i + 1] = (uint8_t)(row[i] >> 8);
        }
        return;
    }
    int G = d / group;
    int64_t codes = codes_at(d, meta, group);
    uint8_t q[128];
    memset(rec, 0, (size_t)codes); /* the pairs, and the zero bytes that follow them with wide groups */
    for (int g = 0; g < G; ++g) {
        if (meta == 8) {
            float scale, zero;
            orc_quantize_span(row + group * g, group, b, &scale, &zero, q);
            put_f32(rec + 8 * g, scale);
            put_f32(rec + 8 * g + 4, zero);
        } else {
            uint16_t scale16, zero16;
            orc_quantize_span_compact(row + group * g, group, b, &scale16, &zero16, q);
            put_u16(rec + 4 * g, scale16);
            put_u16(rec + 4 * g + 2, zero16);
        }
        orc_pack_codes(q, group, b, rec + codes + (size_t)g * group * b / 8);
    }
}

/* {scale, zero} of group g as binary32 (widening an FP16 pair is exact) */
static void group_meta(const uint8_t *rec, int g, int meta, float *scale, float *zero)
{
    if (meta == 8) {
        *scale = get_f32(rec + 8 * g);
        *zero = get_f32(rec + 8 * g + 4);
    } else {
        *scale = orc_half_to_float(get_u16(rec + 4 * g));
        *zero = orc_half_to_float(get_u16(rec + 4 * g + 2));
    }
}

static void decode_record(const uint8_t *rec, int d, int b, int meta, int group, uint16_t *row)
{
    if (b == 16) {
        for (int i = 0; i < d; ++i) row[i] = (uint16_t)(rec[2 * i] | (rec[2 * i + 1] << 8));
        return;
    }
    int G = d / group;
    int64_t codes = codes_at(d, meta, group);
    uint8_t q[128];
    for (int g = 0; g < G; ++g) {
        float scale, zero;
        group_meta(rec, g, meta, &scale, &zero);
        orc_unpack_codes(rec + codes + (size_t)g * group * b / 8, group, b, q);
        orc_dequantize_span(q, group, scale, zero, row + group * g);
    }
}

/* One stream (a [T, d] matrix with a row stride) -> its payload bytes. */
void orc_encode_stream_g(const uint16_t *x, int64_t token_stride, int64_t n_tokens, int d, int meta, int group,
                         const uint8_t *bits, const uint32_t *off, uint8_t *out)
{
    for (int64_t t = 0; t < n_tokens; ++t)
        encode_record(x + t * token_stride, d, bits[t], meta, group, out + off[t]);
}

void orc_decode_stream_g(const uint8_t *in, const uint8_t *bits, const uint32_t *off,
                         int64_t n_tokens, int d, int meta, int group, uint16_t *x, int64_t token_stride)
{
    for (int64_t t = 0; t < n_tokens; ++t)
        decode_record(in + off[t], d, bits[t], meta, group, x + t * token_stride);
}

void orc_encode_stream(const uint16_t *x, int64_t token_stride, int64_t n_tokens, int d, int meta,
                       const uint8_t *bits, const uint32_t *off, uint8_t *out)
{
    orc_encode_stream_g(x, token_stride, n_tokens, d, meta, 32, bits, off, out);
}

void orc_decode_stream(const uint8_t *in, const uint8_t *bits, const uint32_t *off,
                       int64_t n_tokens, int d, int meta, uint16_t *x, int64_t token_stride)
{
    orc_decode_stream_g(in, bits, off, n_tokens, d, meta, 32, x, token_stride);
}

/* ------------------------------------------------------------------ whole card */

/* Header (256 bytes, little-endian, fields at these byte offsets, everything else zero):
 *   0 magic "QKVS" = 0x53564B51   4 version = 1     8 status        12 bits_mode
 *  16 n_layers  20 n_kv_heads  24 head_dim  28 n_tokens  32 group_size
 *  36 meta_bytes_per_group (8|4)  40 model_id u64   48 sender_id u64
 *  56 position_offset i64 (placeholder)  64 sum_bits u64   72 avg_code_bits f32
 *  80 bits_off u64   88 offs_off u64   96 payload_off u64
 * 104 stream_bytes u64 (mode 0: bytes of one stream; mode 1: 0)   112 total_bytes u64
 * 120 sbase_off u64 (mode 1: offset of the u64 stream-base table; mode 0: 0)
 * Then bits[seg][t] u8, then off[seg][0..T] u32, then (mode 1) sbase[0..S] u64, each
 * section zero-padded to a multiple of 256, then the payload, stream after stream with
 * stream (l, kv, h) at index (l*2 + kv)*H + h. */
int orc_write_prefix(const orc_layout *L, const uint8_t *bits, uint64_t model_id,
                     uint64_t sender_id, int64_t position_offset, uint8_t *card,
                     uint64_t capacity)
{
    int st = layout_ok(L);
    if (st) return st;
    uint64_t bo, oo, so, po;
    section_offsets(L, &bo, &oo, &so, &po);
    if (capacity < po) return ORC_BUFFER_TOO_SMALL;
    memset(card, 0, (size_t)po);

    int64_t nseg = n_segments(L), T = L->n_tokens;
    uint64_t S = 2u * (uint64_t)L->n_layers * (uint64_t)L->n_kv_heads;
    uint64_t sum_bits = 0;
    int status = ORC_OK;
    for (int64_t seg = 0; seg < nseg && status == ORC_OK; ++seg) {
        uint32_t *off_tmp = (uint32_t *)(void *)(card + oo + 4u * (uint64_t)seg * (uint64_t)(T + 1));
        /* the host is little-endian, so writing uint32_t in place equals put_u32 */
        uint64_t sb = 0;
        status = orc_scan_offsets_g(L->head_dim, meta_of(L), group_of(L), bits + seg * T, T, off_tmp, &sb);
        sum_bits += sb;
        memcpy(card + bo + (uint64_t)seg * (uint64_t)T, bits + seg * T, (size_t)T);
    }
    uint64_t payload = 0, stream_bytes = 0;
    if (status == ORC_OK) {
        if (L->bits_mode == 0) {
            stream_bytes = get_u32(card + oo + 4u * (uint64_t)T);
            payload = S * stream_bytes;
        } else {
            for (int l = 0; l < L->n_layers; ++l)
                for (int kv = 0; kv < 2; ++kv)
                    for (int h = 0; h < L->n_kv_heads; ++h) {
                        int64_t s = stream_index(L, l, kv, h), seg = segment_of(L, l, h);
                        put_u64(card + so + 8u * (uint64_t)s, payload);
                        payload += get_u32(card + oo + 4u * ((uint64_t)seg * (uint64_t)(T + 1) + (uint64_t)T));
                    }
            put_u64(card + so + 8u * S, payload);
        }
        if (po + payload > capacity) status = ORC_BUFFER_TOO_SMALL;
    }
    put_u32(card + 0, 0x53564B51u);
    put_u32(card + 4, 1u);
    put_u32(card + 8, (uint32_t)status);
    put_u32(card + 12, (uint32_t)L->bits_mode);
    put_u32(card + 16, (uint32_t)L->n_layers);
    put_u32(card + 20, (uint32_t)L->n_kv_heads);
    put_u32(card + 24, (uint32_t)L->head_dim);
    put_u32(card + 28, (uint32_t)L->n_tokens);
    put_u32(card + 32, (uint32_t)L->group_size);
    put_u32(card + 36, (uint32_t)meta_of(L));
    put_u64(card + 40, model_id);
    put_u64(card + 48, sender_id);
    put_u64(card + 56, (uint64_t)position_offset);
    if (status == ORC_OK) {
        put_u64(card + 64, sum_bits);
        float avg = (nseg * T) > 0 ? (float)sum_bits / (float)((uint64_t)nseg * (uint64_t)T) : 0.0f;
        put_f32(card + 72, avg);
    }
    put_u64(card + 80, bo);
    put_u64(card + 88, oo);
    put_u64(card + 96, po);
    if (status == ORC_OK) {
        put_u64(card + 104, stream_bytes);
        put_u64(card + 112, po + payload);
    }
    put_u64(card + 120, so);
    return status;
}

/* Location of stream s inside a card whose prefix is already written. */
static uint64_t stream_base(const uint8_t *card, const orc_layout *L, int64_t s)
{
    uint64_t po = get_u64(card + 96);
    if (L->bits_mode == 0) return po + (uint64_t)s * get_u64(card + 104);
    return po + get_u64(card + get_u64(card + 120) + 8u * (uint64_t)s);
}

/* A card that is read back is untrusted: stream s must start on a 16-byte boundary inside the
 * payload and its last record must end inside the card.  Compared without forming base + length,
 * which a damaged stream-base entry close to 2^64 would wrap around. */
static int stream_in_bounds(const uint8_t *card, const orc_layout *L, int64_t s, uint64_t stream_len)
{
    uint64_t po = get_u64(card + 96), total = get_u64(card + 112);
    if (po > total) return 0;
    uint64_t rel;
    if (L->bits_mode == 0) {
        uint64_t sb = get_u64(card + 104);
        if (sb != 0 && (uint64_t)s > (total - po) / sb) return 0;
        rel = (uint64_t)s * sb;
    } else {
        rel = get_u64(card + get_u64(card + 120) + 8u * (uint64_t)s);
    }
    if (rel % 16u != 0 || rel > total - po) return 0;
    return stream_len <= total - po - rel;
}

/* FP16 cache + bit-widths -> card.  K_layers[l], V_layers[l] point at [H, *, d] FP16 blocks
 * addressed with the layout's strides.  Streams in [s_begin, s_end) are encoded (use 0 and
 * 2*L*H for the whole card); the prefix is always written. */
int orc_card_create_range(const orc_layout *L, const uint16_t *const *K_layers,
                          const uint16_t *const *V_layers, const uint8_t *bits,
                          uint64_t model_id, uint64_t sender_id, int64_t position_offset,
                          uint8_t *card, uint64_t capacity, int64_t s_begin, int64_t s_end)
{
    int st = orc_write_prefix(L, bits, model_id, sender_id, position_offset, card, capacity);
    if (st) return st;
    uint64_t bo = get_u64(card + 80), oo = get_u64(card + 88);
    int64_t T = L->n_tokens, S = 2 * (int64_t)L->n_layers * L->n_kv_heads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t s = s_begin; s < (s_end < S ? s_end : S); ++s) {
        int h = (int)(s % L->n_kv_heads);
        int kv = (int)((s / L->n_kv_heads) % 2);
        int l = (int)(s / (2 * L->n_kv_heads));
        int64_t seg = segment_of(L, l, h);
        const uint16_t *x = (kv == 0 ? K_layers[l] : V_layers[l]) + (int64_t)h * L->head_stride;
        orc_encode_stream_g(x, L->token_stride, T, L->head_dim, meta_of(L), group_of(L), card + bo + (uint64_t)seg * (uint64_t)T,
                          (const uint32_t *)(const void *)(card + oo + 4u * (uint64_t)seg * (uint64_t)(T + 1)),
                          card + stream_base(card, L, s));
    }
    return ORC_OK;
}

int orc_card_create(const orc_layout *L, const uint16_t *const *K_layers,
                    const uint16_t *const *V_layers, const uint8_t *bits, uint64_t model_id,
                    uint64_t sender_id, int64_t position_offset, uint8_t *card, uint64_t capacity)
{
    return orc_card_create_range(L, K_layers, V_layers, bits, model_id, sender_id,
                                 position_offset, card, capacity, 0,
                                 L ? 2 * (int64_t)L->n_layers * L->n_kv_heads : 0);
}

/* Card -> FP16 keys and values.  `dst` gives the destination's shape (which must be the
 * card's, n_tokens included) and strides; token t of the card lands on row
 * dst_token_offset + t, and those rows must fit inside one head's slab. */
int orc_card_inject(const uint8_t *card, uint64_t card_bytes, const orc_layout *dst,
                    uint16_t *const *K_out, uint16_t *const *V_out, int64_t dst_token_offset)
{
    int st = layout_ok(dst);
    if (st) return st;
    if (card_bytes < 256) return ORC_BAD_CARD;
    if (get_u32(card + 0) != 0x53564B51u || get_u32(card + 4) != 1u) return ORC_BAD_CARD;
    if (get_u32(card + 8) != 0u) return ORC_BAD_CARD;
    orc_layout C = *dst;
    C.bits_mode = (int32_t)get_u32(card + 12);
    C.n_tokens = (int32_t)get_u32(card + 28);
    if ((int32_t)get_u32(card + 16) != dst->n_layers || (int32_t)get_u32(card + 20) != dst->n_kv_heads ||
        (int32_t)get_u32(card + 24) != dst->head_dim || get_u32(card + 32) != (uint32_t)group_of(dst) ||
        get_u32(card + 36) != (uint32_t)meta_of(dst) || (C.bits_mode != 0 && C.bits_mode != 1) ||
        C.n_tokens != dst->n_tokens)
        return ORC_BAD_CARD;
    if (get_u64(card + 112) > card_bytes) return ORC_BAD_CARD;
    if (dst_token_offset < 0 || dst->token_stride < dst->head_dim) return ORC_INVALID_ARG;
    if (C.n_tokens > 0 &&
        (dst_token_offset + C.n_tokens - 1) * dst->token_stride + dst->head_dim > dst->head_stride)
        return ORC_INVALID_ARG;
    uint64_t bo = get_u64(card + 80), oo = get_u64(card + 88);
    int64_t T = C.n_tokens, S = 2 * (int64_t)C.n_layers * C.n_kv_heads;
    for (int64_t s = 0; s < S; ++s) {
        int64_t seg = segment_of(&C, (int)(s / (2 * C.n_kv_heads)), (int)(s % C.n_kv_heads));
        if (!stream_in_bounds(card, &C, s, get_u32(card + oo + 4u * ((uint64_t)seg * (uint64_t)(T + 1) + (uint64_t)T))))
            return ORC_BAD_CARD;
    }
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t s = 0; s < S; ++s) {
        int h = (int)(s % C.n_kv_heads);
        int kv = (int)((s / C.n_kv_heads) % 2);
        int l = (int)(s / (2 * C.n_kv_heads));
        int64_t seg = segment_of(&C, l, h);
        uint16_t *x = (kv == 0 ? K_out[l] : V_out[l]) + (int64_t)h * dst->head_stride +
                      dst_token_offset * dst->token_stride;
        orc_decode_stream_g(card + stream_base(card, &C, s), card + bo + (uint64_t)seg * (uint64_t)T,
                          (const uint32_t *)(const void *)(card + oo + 4u * (uint64_t)seg * (uint64_t)(T + 1)),
                          T, C.head_dim, meta_of(&C), group_of(&C), x, dst->token_stride);
    }
    return ORC_OK;
}

/* The values a record stands for, as real numbers: code * scale + zero for a quantised row,
 * the FP16 values themselves for a 16-bit row.  No rounding to FP16: that rounding belongs to
 * injection, which has to hand an FP16 cache to the receiving framework (Section 4.2.2); attention
 * that reads the card itself (Section 4.3) has no FP16 copy to round into. */
static void reconstruct_record(const uint8_t *rec, int d, int b, int meta, int group, double *row)
{
    if (b == 16) {
        for (int i = 0; i < d; ++i) row[i] = (double)orc_half_to_float((uint16_t)(rec[2 * i] | (rec[2 * i + 1] << 8)));
        return;
    }
    int G = d / group;
    int64_t codes = codes_at(d, meta, group);
    uint8_t q[128];
    for (int g = 0; g < G; ++g) {
        float scale, zero;
        group_meta(rec, g, meta, &scale, &zero);
        orc_unpack_codes(rec + codes + (size_t)g * group * b / 8, group, b, q);
        for (int i = 0; i < group; ++i) row[group * g + i] = (double)q[i] * (double)scale + (double)zero;
    }
}

/* The values injection hands to the receiving framework: the record decoded exactly as
 * orc_card_inject does (fp16_rne(fl32(fl32(q) * scale) + zero), Section 4.2.2), widened. */
static void injected_record(const uint8_t *rec, int d, int b, int meta, int group, double *row)
{
    uint16_t h[256];
    decode_record(rec, d, b, meta, group, h);
    for (int i = 0; i < d; ++i) row[i] = (double)orc_half_to_float(h[i]);
}

/* Decode-step attention over the tokens of a card (Section 4.3: consuming a foreign quantised
 * cache directly inside attention is the paper's stated goal; Section 3.1 for K, V per layer and
 * head).  One new token per layer attends to all n_tokens of the card.  Query head j of a layer
 * reads KV head j / (n_q_heads / n_kv_heads) (grouped-query attention; the paper's model,
 * Llama-3.1-8B, has 32 query and 8 KV heads):
 *     s_t  = softmax_scale * sum_c q[j][c] * K~[t][c]
 *     p_t  = exp(s_t - max_t s_t) / sum_t exp(s_t - max_t s_t)
 *     o[c] = sum_t p_t * V~[t][c]
 * The paper gives no formula for this step; this is the textbook definition, evaluated in double
 * precision.  Two readings of K~, V~ are provided:
 *   fp16_rounded = 0   the values the records stand for, code * scale + zero unrounded
 *                      (reconstruct_record): attention that reads the card itself forms no FP16
 *                      copy.  This is what orc_card_attend computes and what the CUDA path is
 *                      held to.
 *   fp16_rounded = 1   the FP16 cache that injection would have produced (injected_record):
 *                      "inject, then attend".  orc_card_attend_injected; reported beside the
 *                      other so that the distance between the two readings is a number.
 *   q    [n_layers][n_q_heads][head_dim] FP16 bit patterns
 *   out  [n_layers][n_q_heads][head_dim] double */
static int attend_over_card(const uint8_t *card, uint64_t card_bytes, const orc_layout *L, int n_q_heads,
                            const uint16_t *q, double softmax_scale, double *out, int fp16_rounded)
{
    int st = layout_ok(L);
    if (st) return st;
    if (fp16_rounded && L->head_dim > 256) return ORC_UNSUPPORTED_SHAPE; /* injected_record's row buffer */
    if (n_q_heads < L->n_kv_heads || n_q_heads % L->n_kv_heads != 0) return ORC_INVALID_ARG;
    if (card_bytes < 256) return ORC_BAD_CARD;
    if (get_u32(card + 0) != 0x53564B51u || get_u32(card + 4) != 1u || get_u32(card + 8) != 0u) return ORC_BAD_CARD;
    orc_layout C = *L;
    C.bits_mode = (int32_t)get_u32(card + 12);
    if ((int32_t)get_u32(card + 16) != L->n_layers || (int32_t)get_u32(card + 20) != L->n_kv_heads ||
        (int32_t)get_u32(card + 24) != L->head_dim || (int32_t)get_u32(card + 28) != L->n_tokens ||
        get_u32(card + 36) != (uint32_t)meta_of(L) || get_u32(card + 32) != (uint32_t)group_of(L) ||
        (C.bits_mode != 0 && C.bits_mode != 1) || get_u64(card + 112) > card_bytes)
        return ORC_BAD_CARD;
    const int d = C.head_dim, H = C.n_kv_heads, per_kv = n_q_heads / H;
    const int64_t T = C.n_tokens;
    const uint64_t bo = get_u64(card + 80), oo = get_u64(card + 88);
    if (T == 0) {
        memset(out, 0, sizeof(double) * (size_t)C.n_layers * (size_t)n_q_heads * (size_t)d);
        return ORC_OK;
    }
    for (int64_t s = 0; s < 2 * (int64_t)C.n_layers * H; ++s) {
        int64_t seg = segment_of(&C, (int)(s / (2 * H)), (int)(s % H));
        if (!stream_in_bounds(card, &C, s, get_u32(card + oo + 4u * ((uint64_t)seg * (uint64_t)(T + 1) + (uint64_t)T))))
            return ORC_BAD_CARD;
    }
    int failed = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t lh = 0; lh < (int64_t)C.n_layers * H; ++lh) {
        const int l = (int)(lh / H), h = (int)(lh % H);
        const int64_t seg = segment_of(&C, l, h);
        const uint8_t *bits = card + bo + (uint64_t)seg * (uint64_t)T;
        const uint32_t *off = (const uint32_t *)(const void *)(card + oo + 4u * (uint64_t)seg * (uint64_t)(T + 1));
        double *kx = (double *)malloc(sizeof(double) * (size_t)T * (size_t)d);
        double *vx = (double *)malloc(sizeof(double) * (size_t)T * (size_t)d);
        double *s = (double *)malloc(sizeof(double) * (size_t)T);
        if (!kx || !vx || !s) {
            failed = 1;
            free(kx);
            free(vx);
            free(s);
            continue;
        }
        const uint8_t *ks = card + stream_base(card, &C, stream_index(&C, l, 0, h));
        const uint8_t *vs = card + stream_base(card, &C, stream_index(&C, l, 1, h));
        for (int64_t t = 0; t < T; ++t) {
            if (fp16_rounded) {
                injected_record(ks + off[t], d, bits[t], meta_of(&C), group_of(&C), kx + t * d);
                injected_record(vs + off[t], d, bits[t], meta_of(&C), group_of(&C), vx + t * d);
            } else {
                reconstruct_record(ks + off[t], d, bits[t], meta_of(&C), group_of(&C), kx + t * d);
                reconstruct_record(vs + off[t], d, bits[t], meta_of(&C), group_of(&C), vx + t * d);
            }
        }
        for (int jj = 0; jj < per_kv; ++jj) {
            const int j = h * per_kv + jj;
            const uint16_t *qv = q + ((int64_t)l * n_q_heads + j) * d;
            double *o = out + ((int64_t)l * n_q_heads + j) * d;
            double mx = -INFINITY;
            for (int64_t t = 0; t < T; ++t) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c)
                    acc += (double)orc_half_to_float(qv[c]) * kx[t * d + c];
                s[t] = softmax_scale * acc;
                if (s[t] > mx) mx = s[t];
            }
            double denom = 0.0;
            for (int64_t t = 0; t < T; ++t) {
                s[t] = exp(s[t] - mx);
                denom += s[t];
            }
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int64_t t = 0; t < T; ++t) acc += s[t] * vx[t * d + c];
                o[c] = acc / denom;
            }
        }
        free(kx);
        free(vx);
        free(s);
    }
    return failed ? ORC_INVALID_ARG : ORC_OK;
}

/* Attention straight from the card: the records' own values, no FP16 rounding. */
int orc_card_attend(const uint8_t *card, uint64_t card_bytes, const orc_layout *L, int n_q_heads,
                    const uint16_t *q, double softmax_scale, double *out)
{
    return attend_over_card(card, card_bytes, L, n_q_heads, q, softmax_scale, out, 0);
}

/* Inject, then attend: the same attention over the FP16 cache orc_card_inject rebuilds. */
int orc_card_attend_injected(const uint8_t *card, uint64_t card_bytes, const orc_layout *L, int n_q_heads,
                             const uint16_t *q, double softmax_scale, double *out)
{
    return attend_over_card(card, card_bytes, L, n_q_heads, q, softmax_scale, out, 1);
}

/* Bit-width assignment from per-token importance scores, the step in front of card creation
 * (Section 3.3: tokens that matter more get more bits, under a budget; Section 4.1.2: the
 * controller outputs b(t) in {2, 4, 8, 16}).  The paper's controller is a trained network that is
 * not available; what is restated here is the rank rule of the benchmark's adaptive
 * configuration: order the tokens by score, highest first, equal scores by lower token index
 * first; the first n_fp16 tokens keep FP16, the next n_8bit get 8 bits, the next n_4bit get
 * 4 bits, all others 2 bits.  Plain sort on (score descending, index ascending). */
typedef struct { float score; int64_t index; } orc_ranked;

static int ranked_before(const void *a, const void *b)
{
    const orc_ranked *x = (const orc_ranked *)a, *y = (const orc_ranked *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return x->index < y->index ? -1 : (x->index > y->index ? 1 : 0);
}

int orc_bits_from_scores(const float *scores, int64_t n_tokens, int64_t n_fp16, int64_t n_8bit,
                         int64_t n_4bit, uint8_t *bits)
{
    if (n_tokens < 0 || n_fp16 < 0 || n_8bit < 0 || n_4bit < 0 || n_fp16 + n_8bit + n_4bit > n_tokens)
        return ORC_INVALID_ARG;
    orc_ranked *r = (orc_ranked *)malloc(sizeof(orc_ranked) * (size_t)(n_tokens > 0 ? n_tokens : 1));
    if (!r) return ORC_INVALID_ARG;
    for (int64_t t = 0; t < n_tokens; ++t) {
        r[t].score = scores[t];
        r[t].index = t;
    }
    qsort(r, (size_t)n_tokens, sizeof(orc_ranked), ranked_before);
    for (int64_t k = 0; k < n_tokens; ++k) {
        uint8_t b = 2;
        if (k < n_fp16) b = 16;
        else if (k < n_fp16 + n_8bit) b = 8;
        else if (k < n_fp16 + n_8bit + n_4bit) b = 4;
        bits[r[k].index] = b;
    }
    free(r);
    return ORC_OK;
}

/* Bit-widths under a byte budget (Section 3.3: minimise sum_t eps(t, b(t)) * S(t) subject to
 * sum_t b(t) * d <= M; the paper prints the objective and no solver).  The reading taken here is
 * the greedy solution of that knapsack by worth per byte, stated so that the result is unique:
 *   - every token starts at 2 bits; raising a token one rung up the ladder 2 -> 4 -> 8 -> 16 is an
 *     *upgrade* i = 0, 1, 2 with a cost in bytes, cost_i = rec(next rung) - rec(rung) (record sizes,
 *     metadata included), and a worth per byte  key = fl32(S(t) * weight_i), where weight_i > 0 says
 *     how much error an upgrade of that rung removes per byte (weight_0 >= weight_1 >= weight_2:
 *     the first bits buy the most);
 *   - all 3 T upgrades are put in one order: larger key first, equal keys by lower rung, then by
 *     lower token index; with non-negative scores a token's own upgrades appear in rung order;
 *   - upgrades are granted in that order while their cost still fits into what the budget leaves
 *     after 2 bits for everybody; the first one that does not fit ends the procedure.
 * budget_bytes bounds the bytes of one stream: sum_t rec(b(t)) <= budget_bytes.  Scores must be
 * finite and non-negative (a zero of either sign counts as zero).  Returns ORC_BUFFER_TOO_SMALL if
 * the budget does not even hold 2 bits per token. */
typedef struct { float key; int32_t rung; int64_t index; } orc_upgrade;

static int upgrade_before(const void *a, const void *b)
{
    const orc_upgrade *x = (const orc_upgrade *)a, *y = (const orc_upgrade *)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    if (x->rung != y->rung) return x->rung < y->rung ? -1 : 1;
    return x->index < y->index ? -1 : (x->index > y->index ? 1 : 0);
}

int orc_bits_from_scores_budget(const float *scores, int64_t n_tokens, int head_dim, int meta,
                                uint64_t budget_bytes, const float *weight, uint8_t *bits)
{
    static const int ladder[4] = {2, 4, 8, 16};
    if (n_tokens < 0 || !weight) return ORC_INVALID_ARG;
    if (!(weight[0] > 0.0f && weight[1] > 0.0f && weight[2] > 0.0f && weight[0] >= weight[1] && weight[1] >= weight[2]))
        return ORC_INVALID_ARG;
    int64_t rec[4];
    for (int i = 0; i < 4; ++i) {
        rec[i] = orc_record_bytes(head_dim, ladder[i], meta);
        if (rec[i] < 0) return ORC_INVALID_ARG;
    }
    for (int64_t t = 0; t < n_tokens; ++t)
        if (!(scores[t] >= 0.0f) || isinf(scores[t])) return ORC_INVALID_ARG;
    if ((uint64_t)n_tokens * (uint64_t)rec[0] > budget_bytes) return ORC_BUFFER_TOO_SMALL;
    uint64_t left = budget_bytes - (uint64_t)n_tokens * (uint64_t)rec[0];
    orc_upgrade *u = (orc_upgrade *)malloc(sizeof(orc_upgrade) * (size_t)(3 * n_tokens > 0 ? 3 * n_tokens : 1));
    if (!u) return ORC_INVALID_ARG;
    for (int64_t t = 0; t < n_tokens; ++t)
        for (int i = 0; i < 3; ++i) {
            float s = scores[t] == 0.0f ? 0.0f : scores[t];
            u[3 * t + i].key = s * weight[i];
            u[3 * t + i].rung = i;
            u[3 * t + i].index = t;
        }
    qsort(u, (size_t)(3 * n_tokens), sizeof(orc_upgrade), upgrade_before);
    for (int64_t t = 0; t < n_tokens; ++t) bits[t] = 2;
    for (int64_t j = 0; j < 3 * n_tokens; ++j) {
        uint64_t cost = (uint64_t)(rec[u[j].rung + 1] - rec[u[j].rung]);
        if (cost > left) break;
        left -= cost;
        bits[u[j].index] = (uint8_t)ladder[u[j].rung + 1];
    }
    free(u);
    return ORC_OK;
}

/* Combined importance score (Section 3.3): S(t) = alpha * I(t) + (1 - alpha) * T(t), in binary32,
 * every operation rounded on its own (the file is compiled without contraction). */
int orc_combine_scores(const float *importance, const float *transfer, float alpha, int64_t n, float *scores)
{
    if (n < 0 || !(alpha >= 0.0f && alpha <= 1.0f)) return ORC_INVALID_ARG;
    const float beta = 1.0f - alpha;
    for (int64_t i = 0; i < n; ++i) {
        const float a = alpha * importance[i];
        const float b = beta * transfer[i];
        scores[i] = a + b;
    }
    return ORC_OK;
}

/* Bit-widths from the controller of Section 4.1.2: a two-layer perceptron over six features per
 * token (frequency, quality, attention variance, entropy, downstream demand, segment type) whose
 * four outputs stand for the bit-widths 2, 4, 8, 16; the token gets the one with the largest
 * output.  The paper gives the shape (6 -> hidden -> 4, 512 parameters in all) and no formula; the
 * reading taken here: hidden_j = max(0, b1[j] + sum_i W1[j][i] x[i]), out_k = b2[k] + sum_j
 * W2[k][j] hidden_j, sums taken in index order starting from the bias, every product and every
 * sum rounded to binary32 on its own; the largest output wins, equal outputs go to the fewer bits.
 *   features  [n][6]; params: W1 [hidden][6], b1 [hidden], W2 [4][hidden], b2 [4], one after another
 *   bits      [n]; outputs (optional) [n][4] */
int orc_bits_from_features(const float *features, int64_t n, int hidden, const float *params, uint8_t *bits, float *outputs)
{
    static const int ladder[4] = {2, 4, 8, 16};
    if (n < 0 || hidden < 1 || hidden > 128) return ORC_INVALID_ARG;
    const float *w1 = params, *b1 = w1 + 6 * hidden, *w2 = b1 + hidden, *b2 = w2 + 4 * hidden;
    for (int64_t t = 0; t < n; ++t) {
        const float *x = features + 6 * t;
        float hid[128];
        for (int j = 0; j < hidden; ++j) {
            float acc = b1[j];
            for (int i = 0; i < 6; ++i) {
                const float prod = w1[6 * j + i] * x[i];
                acc = acc + prod;
            }
            hid[j] = acc > 0.0f ? acc : 0.0f;
        }
        int best = 0;
        float best_out = 0.0f;
        for (int k = 0; k < 4; ++k) {
            float acc = b2[k];
            for (int j = 0; j < hidden; ++j) {
                const float prod = w2[hidden * k + j] * hid[j];
                acc = acc + prod;
            }
            if (outputs) outputs[4 * t + k] = acc;
            if (k == 0 || acc > best_out) {
                best = k;
                best_out = acc;
            }
        }
        bits[t] = (uint8_t)ladder[best];
    }
    return ORC_OK;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
