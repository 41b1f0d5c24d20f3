// Decode-step attention straight from a card: one query token per layer attends to every token
// of the card, reading the records themselves -- no FP16 cache is written or even formed.
//
//     s_t = softmax_scale * q . K~_t,   p = softmax(s),   o = sum_t p_t V~_t
//
// with K~, V~ the values the records stand for (code * scale + zero per group of 32 channels, or
// the FP16 value of a 16-bit row), grouped queries (query head j reads KV head j / per_kv),
// head_dim 128.  Scale and zero never touch the elements: with D = sum_c q_c code_c per group,
//     q . K~_t   = sum_g scale_tg * D_tg + zero_tg * (sum_{c in g} q_c)
//     sum_t p_t V~_tc = sum_t (p_t scale_tg) code_tc + sum_t p_t zero_tg        (c in group g)
// so both contractions run on the tensor cores over the integer codes themselves (exact in FP16;
// mma.sync m16n8k16, FP32 accumulation) and the group parameters enter once per token and group.
//
// Work item: 256 consecutive tokens of one (layer, KV head), taken by one warp from a counter.
// The warp walks them in steps of 16 tokens; the spans of K and V records of a step are staged by
// two bulk copies (TMA) on one mbarrier, NS steps ahead.  Operand layouts are chosen -- the order
// of channels inside a group and of tokens inside a step is free in a contraction -- so that every
// lane builds its fragments from a few bytes of its own with shifts and masks:
//   scores   rows = the 16 tokens of a step, columns = the query heads of the group (up to 8);
//            lane (g, t) supplies 8 codes per group of the tokens g and g + 8 and holds the matching
//            channels of head g's query; it receives the scores of its two tokens for heads 2t, 2t+1;
//   outputs  rows = channels, columns = query heads; lane (g, t) supplies 4 channels per group of
//            the four tokens 2t, 2t+1, 2t+8, 2t+9; the weights (probabilities times the tokens'
//            scales, FP16) are moved from the score layout into the B fragment by an 8 x 8
//            transpose inside the warp (movmatrix); the accumulators are again heads 2t, 2t+1.
// Softmax is the usual running maximum / running sum; every item leaves (o, max, sum) per query
// head in the scratch buffer and a second small kernel merges the items of a head.
#pragma once

#include "qkvs_pipeline.cuh"

namespace qkvs {

constexpr int kAttendD = 128;
constexpr int kAttendRows = 16;          // tokens per step
constexpr int kAttendRecMax = 160;       // largest record of which a step takes 16 (8 bits, fp32 pairs)
constexpr int kAttendStageBytes = kAttendRows * kAttendRecMax;  // per stream; 16-bit rows go 8 per step
static_assert(kAttendStageBytes >= 8 * 2 * kAttendD && kAttendStageBytes % 128 == 0, "stage size");
constexpr int kAttendSteps = 16;         // steps of 16 tokens per work item
constexpr int kAttendPerLane = kAttendRows * kAttendSteps / 32;  // tokens of an item per lane when they are sorted
constexpr int kAttendMaxSteps = kAttendRows * kAttendSteps / 8 + 3;  // all 16-bit but three tokens, one per other class
constexpr int kAttendStepSlots = (kAttendMaxSteps + 31) / 32 * 32;   // whole rounds of one descriptor per lane
constexpr int kAttendMaxPerKv = 8;       // query heads per KV head
constexpr int kPartialFloats = kAttendD + 4;  // o[128], running maximum (base-2 exponent), running sum, padding

struct AttendParams {
    const uint8_t *card;
    uint64_t card_bytes;
    int32_t n_layers, n_kv_heads, n_tokens, n_q_heads;
    int32_t meta_bytes;      // 8 or 4: bytes of {scale, zero} per group in the card's records
    const __half *q;         // [n_layers][n_q_heads][128]
    float scale_log2;        // softmax_scale * log2(e)
    float *partials;         // [n_items][per_kv][kPartialFloats]
    float *out;              // [n_layers][n_q_heads][128]
    uint32_t subs_per_head;  // steps per (layer, KV head)
    uint32_t items_per_head;
    uint32_t n_items;
    uint32_t last_rows;      // tokens in the last step of a head
    int32_t *status_dev;
    uint32_t *work_counter;
};

template <int NS>
struct AttendWarpSmem {
    alignas(128) uint8_t k[NS][kAttendStageBytes];  // the step's records, packed one after another
    alignas(128) uint8_t v[NS][kAttendStageBytes];
    uint32_t list[kAttendRows * kAttendSteps];  // record offsets of the item's tokens, grouped by bit-width
    uint32_t steps[kAttendStepSlots];           // the item's step descriptors
    alignas(16) float qsum[4][8];               // per tig: sums over group g of the queries of heads 2tig + h, at [2g + h]
    alignas(8) uint64_t full[NS];
};

__device__ __forceinline__ void mma_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The same product with a zero accumulator coming in.
__device__ __forceinline__ void mma_m16n8k16_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                                   uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}

// Transposes an 8 x 8 matrix of 16-bit elements held one row per group of four lanes, two
// neighbouring columns per lane: afterwards lane (gid, tig) holds what was in rows 2tig, 2tig + 1
// of column gid.
__device__ __forceinline__ uint32_t transpose_8x8(uint32_t v)
{
    uint32_t r;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}

__device__ __forceinline__ float exp2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The order of tokens does not matter to attention, so a warp regroups the (up to) 256 tokens of
// its item by bit-width (classes 0..3 = 2, 4, 8, 16 bits) and walks them one width at a time:
// every step then deals with a single width and runs the body compiled for it, however the widths
// are mixed in the card.

// The item's steps are laid out once per item, one descriptor per step, by the lanes in parallel:
// the tokens of class c occupy [begin_c, end_c) of the list and are walked 16 at a time (16-bit
// rows, 256 bytes each, 8 at a time: a stage holds eight of them).
//   bits 0..9  first list position   10..14  tokens in the step   15..16  class
//   bit 17     the step's records are neighbours in the card (one copy per stream will do)
static_assert(kAttendRows * kAttendSteps <= 512 && kAttendMaxSteps <= kAttendStepSlots, "descriptor fields");

__device__ __forceinline__ uint32_t step_first(uint32_t d) { return d & 1023u; }
__device__ __forceinline__ int step_rows(uint32_t d) { return (int)((d >> 10) & 31u); }
__device__ __forceinline__ int step_class(uint32_t d) { return (int)((d >> 15) & 3u); }

// The record format is a template parameter of everything below, as one number: the bytes of a
// {scale, zero} pair (8 or 4) plus 16 times log2(channels per group / 32).  Formats with groups of
// 32 are therefore named by their pair size alone.
__host__ __device__ constexpr int format_code(int meta, int group_size) { return meta + 16 * (group_size == 128 ? 2 : (group_size == 64 ? 1 : 0)); }
__host__ __device__ constexpr int format_meta(int fmt) { return fmt & 15; }
__host__ __device__ constexpr int format_gs(int fmt) { return fmt >> 4; }
__host__ __device__ constexpr int format_group(int fmt) { return kGroup << format_gs(fmt); }
// bytes of a record's pairs, i.e. where its code bytes start
__host__ __device__ constexpr int format_pairs(int fmt) { return (int)pairs_bytes(kAttendD, format_meta(fmt), format_group(fmt)); }

template <int META>
__device__ __forceinline__ uint32_t class_record_bytes(int c)
{
    constexpr int P = format_pairs(META);
    return c == 0 ? (uint32_t)(kAttendD / 4 + P) : (c == 1 ? (uint32_t)(kAttendD / 2 + P) : (c == 2 ? (uint32_t)(kAttendD + P) : 2u * kAttendD));
}

// Descriptor of step `idx` given where the classes end in the list (e[c], with e[-1] = 0); 0 past the last step.
template <int META>
__device__ __forceinline__ uint32_t make_step(uint32_t idx, const uint32_t (&e)[4], const uint32_t *list)
{
    uint32_t begin = 0, first_step = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t per = c == 3 ? kAttendRows / 2 : kAttendRows;
        const uint32_t n_steps = (e[c] - begin + per - 1) / per;
        if (idx < first_step + n_steps) {
            const uint32_t s0 = begin + (idx - first_step) * per;
            const uint32_t rows = min(per, e[c] - s0);
            const bool neighbours = list[s0 + rows - 1] - list[s0] == (rows - 1) * class_record_bytes<META>(c);
            return s0 | (rows << 10) | ((uint32_t)c << 15) | (neighbours ? 1u << 17 : 0u);
        }
        first_step += n_steps;
        begin = e[c];
    }
    return 0u;
}

// Starts the copies of one step's K and V records into `stage`, packed in list order: one copy
// per stream when the tokens are neighbours in the card (the offsets grow with the token index,
// so first and last record a step's length apart leave no room for others in between), else
// gathered in 16-byte pieces.  Either way the stage's barrier completes when the bytes are there.
// All lanes call it.
template <int NS, int META>
__device__ __forceinline__ void attend_issue(AttendWarpSmem<NS> &sm, int stage, uint32_t d, uint64_t base_k, uint64_t base_v,
                                             const AttendParams &p, int lane)
{
    const int n = step_rows(d);
    const uint32_t rec = class_record_bytes<META>(step_class(d));
    if (d & (1u << 17)) {
        if (lane == 0) {
            const uint32_t first = sm.list[step_first(d)];
            mbar_arrive_expect_tx(&sm.full[stage], 2u * (uint32_t)n * rec);
            bulk_load(sm.k[stage], p.card + base_k + first, (uint32_t)n * rec, &sm.full[stage]);
            bulk_load(sm.v[stage], p.card + base_v + first, (uint32_t)n * rec, &sm.full[stage]);
        }
    } else {
        // scattered records of 48 to 256 bytes: 16-byte pieces, one per lane and round, which the
        // load unit merges into whole sectors; a bulk copy per record costs far more than it moves
        const uint32_t pieces = rec >> 4, total = (uint32_t)n * pieces;  // at most 160
        const uint32_t inv = 65536u / pieces + 1u;                      // i / pieces == (i * inv) >> 16 for i < 4096
        for (uint32_t i = (uint32_t)lane; i < total; i += 32u) {
            const uint32_t r = (i * inv) >> 16;
            const uint32_t src = sm.list[step_first(d) + r] + ((i - r * pieces) << 4);
            async_copy_16(sm.k[stage] + (i << 4), p.card + base_k + src);
            async_copy_16(sm.v[stage] + (i << 4), p.card + base_v + src);
        }
        async_copies_arrive_on(&sm.full[stage]);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.full[stage]);
    }
}

constexpr uint32_t kHalfMagic = 0x64006400u;  // two FP16 1024.0: 1024 + n has n in its low mantissa bits

// Two small integers, found in `word` under `mask` (one in each 16-bit half), as an FP16 pair:
// (word & mask) | 1024.0 puts them into the low mantissa bits of 1024 + n; minus 1024 is exact.
__device__ __forceinline__ uint32_t int_pair(uint32_t word, uint32_t mask)
{
    uint32_t f;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(f) : "r"(word), "r"(mask), "r"(kHalfMagic));  // (a & b) | c
    return as_u32(__hsub2(as_half2(f), as_half2(kHalfMagic)));
}

// The eight nibbles n0..n7 of a word as four FP16 pairs e[k] = (n_k, n_{k+4}).  The odd nibbles
// are picked up where they sit, four bits up, as 1024 + 16 n, and (1024 + 16 n) / 16 - 64 = n is
// exact in one fused multiply-add; so one shift serves the whole word.
__device__ __forceinline__ void nibble_pairs(uint32_t w, uint32_t (&e)[4])
{
    const __half2 sixteenth = __floats2half2_rn(0.0625f, 0.0625f), minus64 = __floats2half2_rn(-64.0f, -64.0f);
    const uint32_t hi = w >> 8;
    uint32_t f1, f3;
    e[0] = int_pair(w, 0x000f000fu);
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(f1) : "r"(w), "r"(0x00f000f0u), "r"(kHalfMagic));
    e[1] = as_u32(__hfma2(as_half2(f1), sixteenth, minus64));
    e[2] = int_pair(hi, 0x000f000fu);
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(f3) : "r"(hi), "r"(0x00f000f0u), "r"(kHalfMagic));
    e[3] = as_u32(__hfma2(as_half2(f3), sixteenth, minus64));
}

// The four 2-bit codes in the low byte of each half of a word as four FP16 pairs e[k] = (code k
// of the low half, code k of the high half), without shifts: code k is picked up where it sits,
// as 1024 + 4^k n, and brought down by an exact fused multiply-add.
__device__ __forceinline__ void crumb_pairs(uint32_t y, uint32_t (&e)[4])
{
    uint32_t f1, f2, f3;
    e[0] = int_pair(y, 0x00030003u);
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(f1) : "r"(y), "r"(0x000c000cu), "r"(kHalfMagic));
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(f2) : "r"(y), "r"(0x00300030u), "r"(kHalfMagic));
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(f3) : "r"(y), "r"(0x00c000c0u), "r"(kHalfMagic));
    e[1] = as_u32(__hfma2(as_half2(f1), __floats2half2_rn(0.25f, 0.25f), __floats2half2_rn(-256.0f, -256.0f)));
    e[2] = as_u32(__hfma2(as_half2(f2), __floats2half2_rn(0.0625f, 0.0625f), __floats2half2_rn(-64.0f, -64.0f)));
    e[3] = as_u32(__hfma2(as_half2(f3), __floats2half2_rn(0.015625f, 0.015625f), __floats2half2_rn(-16.0f, -16.0f)));
}

// Four 8 x 8 matrices of 16-bit elements from shared memory, rows of 16 bytes: lane l gives the
// address of row l % 8 of matrix l / 8; lane (gid, tig) receives from each matrix the word tig of
// row gid -- or, transposed, the element gid of the rows 2tig (low half) and 2tig + 1 (high half).
__device__ __forceinline__ void load_matrices(const void *row, uint32_t (&d)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(smem_addr(row))
                 : "memory");
}
__device__ __forceinline__ void load_matrices_transposed(const void *row, uint32_t (&d)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(smem_addr(row))
                 : "memory");
}

// Key side.  The lane's 8 channels of group g of one token (channels 32g + 8t + 0..7) as four
// FP16 pairs e[k] = (value k, value k + 4) -- codes for a quantised row, the FP16 values for a
// 16-bit row.  The query fragments pair channels the same way.
template <int B, int META>
__device__ __forceinline__ void key_pairs(const uint8_t *rec, int g, int tig, uint32_t (&e)[4])
{
    constexpr int bb = B;
    if (B == 16) {
        const uint4 h = *reinterpret_cast<const uint4 *>(rec + 64 * g + 16 * tig);
        e[0] = __byte_perm(h.x, h.z, 0x5410);
        e[1] = __byte_perm(h.x, h.z, 0x7632);
        e[2] = __byte_perm(h.y, h.w, 0x5410);
        e[3] = __byte_perm(h.y, h.w, 0x7632);
        return;
    }
    const uint8_t *codes = rec + format_pairs(META) + (4 * g + tig) * bb;  // the lane's 8 codes: b bytes
    if constexpr (B == 4) {
        nibble_pairs(*reinterpret_cast<const uint32_t *>(codes), e);  // nibble k and k + 4 are 16 bits apart
    } else if constexpr (B == 8) {
        const uint2 w = *reinterpret_cast<const uint2 *>(codes);
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(__byte_perm(w.x, w.y, 0x0011u * k + 0x1100u * (4 + k)), 0x00ff00ffu);
    } else if constexpr (B == 2) {
        const uint32_t w = *reinterpret_cast<const uint16_t *>(codes);
        crumb_pairs(__byte_perm(w, 0u, 0x4140), e);  // codes 0..3 in byte 0, codes 4..7 in byte 2
    }
}

// Value side, two tokens at once: the lane's 4 channels of group g (channels 32g + 4gid + 0..3)
// as four FP16 pairs e[k] = (token a's value k, token b's value k).
template <int B, int META>
__device__ __forceinline__ void value_pairs(const uint8_t *rec_a, const uint8_t *rec_b, int g, int gid, uint32_t (&e)[4])
{
    constexpr int CODES = format_pairs(META);  // the code bytes follow the {scale, zero} pairs
    if (B == 16) {
        const uint2 ha = *reinterpret_cast<const uint2 *>(rec_a + 64 * g + 8 * gid);
        const uint2 hb = *reinterpret_cast<const uint2 *>(rec_b + 64 * g + 8 * gid);
        e[0] = __byte_perm(ha.x, hb.x, 0x5410);
        e[1] = __byte_perm(ha.x, hb.x, 0x7632);
        e[2] = __byte_perm(ha.y, hb.y, 0x5410);
        e[3] = __byte_perm(ha.y, hb.y, 0x7632);
    } else if (B == 4) {
        const uint32_t wa = *reinterpret_cast<const uint16_t *>(rec_a + CODES + 16 * g + 2 * gid);
        const uint32_t wb = *reinterpret_cast<const uint16_t *>(rec_b + CODES + 16 * g + 2 * gid);
        nibble_pairs(wa | (wb << 16), e);
    } else if (B == 8) {
        const uint32_t wa = *reinterpret_cast<const uint32_t *>(rec_a + CODES + 32 * g + 4 * gid);
        const uint32_t wb = *reinterpret_cast<const uint32_t *>(rec_b + CODES + 32 * g + 4 * gid);
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(__byte_perm(wa, wb, 0x0011u * k + 0x1100u * (4 + k)), 0x00ff00ffu);
    } else {
        const uint32_t x = (uint32_t)*(rec_a + CODES + 8 * g + gid) | ((uint32_t)*(rec_b + CODES + 8 * g + gid) << 16);
        crumb_pairs(x, e);
    }
}

// Scale / zero pairs of a token's four spans of 32 channels; (1, 0) for a 16-bit row, (0, 0) for no
// token.  With groups of 64 or 128 channels neighbouring spans share a pair.
template <int B, int META>
__device__ __forceinline__ void group_params_of(const uint8_t *rec, bool valid, float (&sc)[4], float (&ze)[4])
{
    if (B != 16 && valid && format_gs(META) > 0) {
        constexpr int GS = format_gs(META);
        const uint4 m = *reinterpret_cast<const uint4 *>(rec);  // the whole (padded) pairs area
        const uint32_t w[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int pair = g >> GS;
            if (format_meta(META) == kMetaFp16) {
                const float2 f = __half22float2(as_half2(w[pair]));
                sc[g] = f.x;
                ze[g] = f.y;
            } else {
                sc[g] = __uint_as_float(w[2 * pair]);
                ze[g] = __uint_as_float(w[2 * pair + 1]);
            }
        }
    } else if (B != 16 && valid && META == kMetaFp16) {
        const uint4 m = *reinterpret_cast<const uint4 *>(rec);  // four FP16 pairs
        const uint32_t w[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const float2 f = __half22float2(as_half2(w[g]));
            sc[g] = f.x;
            ze[g] = f.y;
        }
    } else if (B != 16 && valid) {
        const uint4 m0 = *reinterpret_cast<const uint4 *>(rec), m1 = *reinterpret_cast<const uint4 *>(rec + 16);
        sc[0] = __uint_as_float(m0.x), ze[0] = __uint_as_float(m0.y), sc[1] = __uint_as_float(m0.z), ze[1] = __uint_as_float(m0.w);
        sc[2] = __uint_as_float(m1.x), ze[2] = __uint_as_float(m1.y), sc[3] = __uint_as_float(m1.z), ze[3] = __uint_as_float(m1.w);
    } else {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            sc[g] = valid ? 1.0f : 0.0f;
            ze[g] = 0.0f;
        }
    }
}

// One step: up to 16 tokens of one bit-width B, their K and V records packed one after another in
// `stage`, against the group's queries.  Lane (gid, tig) owns the tokens gid and gid + 8 of the
// step on the score side and the query heads 2tig and 2tig + 1 throughout, so that the running
// maximum and sum of a head, the factors that rescale its accumulators and the accumulators
// themselves sit in the same lane.  FULL: all 16 tokens are there.
//   qb[g][k]     query fragments (B operand): head gid, channels 32g + 8tig + k and + k + 4
//   sm.qsum      sums over a group of the queries of the lane's two heads (read here, once per step)
//   m_run[h], l_run[h]   running maximum of head 2tig + h (the same in all lanes of a tig) and this
//                lane's share of its running sum (tokens gid, gid + 8 of every step)
//   zacc[g][h]   this lane's share of sum_t p_t zero_tg for head 2tig + h
//   acc[g][j][.] channels 32g + 4gid + 2j (+1) x heads 2tig, 2tig + 1, without the zero-point part
template <int NS, int B, bool FULL, int META>
__device__ __forceinline__ void attend_step(const AttendWarpSmem<NS> &sm, int stage, int rows, int gid, int tig, float scale_log2,
                                            const uint32_t (&qb)[4][4], float (&m_run)[2],
                                            float (&l_run)[2], float (&zacc)[4][2], float (&acc)[4][2][4])
{
    constexpr int REC = B == 16 ? 2 * kAttendD : kAttendD * B / 8 + format_pairs(META);
    const bool have[2] = {FULL || gid < rows, FULL || gid + 8 < rows};
    const uint8_t *krec[2] = {sm.k[stage] + gid * REC, sm.k[stage] + (gid + 8) * REC};
    const uint8_t *vrec[2] = {sm.v[stage] + gid * REC, sm.v[stage] + (gid + 8) * REC};
    // ---- scores: rows = the 16 tokens, columns = the group's heads; per group of 32 channels
    // sum_c code_c q_c, two products of 16 channels each
    float x[2][2];  // logits (base 2): [token gid + 8k][head 2tig + h]
    {
        float sacc[4][4];
        const float4 qs_lo = *reinterpret_cast<const float4 *>(&sm.qsum[tig][0]), qs_hi = *reinterpret_cast<const float4 *>(&sm.qsum[tig][4]);
        const float qsum[4][2] = {{qs_lo.x, qs_lo.y}, {qs_lo.z, qs_lo.w}, {qs_hi.x, qs_hi.y}, {qs_hi.z, qs_hi.w}};
        // 4-bit rows: a (token, group) is 16 bytes of codes, a matrix row; two loads hand every
        // lane its words of all four groups of its two tokens
        uint32_t ka[4], kb[4];
        if (B == 4) {
            const int l = gid * 4 + tig;
            const uint8_t *row = sm.k[stage] + (l & 7) * REC + format_pairs(META) + 16 * (l >> 3);
            load_matrices(row, ka);
            load_matrices(row + 8 * REC, kb);
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            uint32_t ea[4] = {0u, 0u, 0u, 0u}, eb[4] = {0u, 0u, 0u, 0u};  // lanes without a token feed zeros
            if (B == 4) {
                if (have[0]) nibble_pairs(ka[g], ea);
                if (have[1]) nibble_pairs(kb[g], eb);
            } else {
                if (have[0]) key_pairs<B, META>(krec[0], g, tig, ea);
                if (have[1]) key_pairs<B, META>(krec[1], g, tig, eb);
            }
            mma_m16n8k16_first(sacc[g], ea[0], eb[0], ea[1], eb[1], qb[g][0], qb[g][1]);  // the whole warp, together
            mma_m16n8k16(sacc[g], ea[2], eb[2], ea[3], eb[3], qb[g][2], qb[g][3]);
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            float sc[4], ze[4];
            group_params_of<B, META>(krec[k], have[k], sc, ze);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float dot = 0.0f;
#pragma unroll
                for (int g = 0; g < 4; ++g) dot = fmaf(sc[g], sacc[g][2 * k + h], fmaf(ze[g], qsum[g][h], dot));
                x[k][h] = have[k] ? dot * scale_log2 : -INFINITY;
            }
        }
    }
    // ---- running softmax of heads 2tig and 2tig + 1.  The running maximum only moves when some
    // token of the step exceeds it, which after the first steps of an item is rare: one vote
    // decides whether the step goes through the reduction over its 16 tokens (the eight lanes of
    // a tig), the factor for what has been summed so far and the rescaling of the accumulators.
    float pr[2][2];
    const bool above = x[0][0] > m_run[0] || x[1][0] > m_run[0] || x[0][1] > m_run[1] || x[1][1] > m_run[1];
    if (__any_sync(0xffffffffu, above)) {
        float alpha[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float m_loc = fmaxf(x[0][h], x[1][h]);
            m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 4));
            m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 8));
            m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 16));
            const float m_new = fmaxf(m_run[h], m_loc);
            const float m_ref = m_new == -INFINITY ? 0.0f : m_new;
            alpha[h] = exp2_approx(m_run[h] - m_ref);  // 0 on the first tokens of the item
            l_run[h] *= alpha[h];
            m_run[h] = m_new;
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            zacc[g][0] *= alpha[0];
            zacc[g][1] *= alpha[1];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                acc[g][j][0] *= alpha[0];
                acc[g][j][1] *= alpha[1];
                acc[g][j][2] *= alpha[0];
                acc[g][j][3] *= alpha[1];
            }
        }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const float m_ref = m_run[h] == -INFINITY ? 0.0f : m_run[h];
        pr[0][h] = exp2_approx(x[0][h] - m_ref);
        pr[1][h] = exp2_approx(x[1][h] - m_ref);
        l_run[h] += pr[0][h] + pr[1][h];
    }
    // ---- values.  The weights p_t * scale_tg are formed where the probabilities are (tokens gid,
    // gid + 8 x heads 2tig, 2tig + 1), rounded to FP16 and transposed inside the warp into the B
    // operand (tokens 2tig, 2tig + 1, 2tig + 8, 2tig + 9 x head gid); the zero points go aside.
    uint32_t wb0[4], wb1[4];
    {
        float vs[2][4];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            float ze[4];
            group_params_of<B, META>(vrec[k], have[k], vs[k], ze);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                zacc[g][0] = fmaf(pr[k][0], ze[g], zacc[g][0]);
                zacc[g][1] = fmaf(pr[k][1], ze[g], zacc[g][1]);
            }
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            wb0[g] = transpose_8x8(as_u32(__floats2half2_rn(pr[0][0] * vs[0][g], pr[0][1] * vs[0][g])));
            wb1[g] = transpose_8x8(as_u32(__floats2half2_rn(pr[1][0] * vs[1][g], pr[1][1] * vs[1][g])));
        }
    }
    // records of tokens that are not there hold stale bytes: their weights are zero, and so that
    // nothing non-finite can come out of stale FP16 patterns their rows are read from token 0
    const uint8_t *rv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int t = 2 * tig + (i & 1) + 8 * (i >> 1);
        rv[i] = sm.v[stage] + ((FULL || t < rows) ? t : 0) * REC;
    }
    // 4-bit rows: transposed matrix loads deliver (token 2tig, token 2tig + 1) x channels 4gid..4gid+3
    // of a group in one word, tokens 0..7 and 8..15 of two groups per load.  Stale rows of tokens
    // that are not there are integers like any others, and their weights are zero.
    uint32_t va[4], vb[4];
    if (B == 4) {
        const int l = gid * 4 + tig;
        const uint8_t *row = sm.v[stage] + ((l & 7) + 8 * ((l >> 3) & 1)) * REC + format_pairs(META) + 16 * (l >> 4);
        load_matrices_transposed(row, va);       // groups 0, 1
        load_matrices_transposed(row + 32, vb);  // groups 2, 3
    }
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t eab[4], ecd[4];
        if (B == 4) {
            nibble_pairs(g < 2 ? va[2 * g] : vb[2 * g - 4], eab);
            nibble_pairs(g < 2 ? va[2 * g + 1] : vb[2 * g - 3], ecd);
        } else {
            value_pairs<B, META>(rv[0], rv[1], g, gid, eab);
            value_pairs<B, META>(rv[2], rv[3], g, gid, ecd);
        }
        mma_m16n8k16(acc[g][0], eab[0], eab[1], ecd[0], ecd[1], wb0[g], wb1[g]);
        mma_m16n8k16(acc[g][1], eab[2], eab[3], ecd[2], ecd[3], wb0[g], wb1[g]);
    }
}

#ifndef QKVS_ATTEND_CTAS
#define QKVS_ATTEND_CTAS 2
#endif

template <int NS, int WARPS, int META>
__global__ void __launch_bounds__(WARPS * 32, QKVS_ATTEND_CTAS) attend_kernel(AttendParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ int s_header_ok;
    __shared__ uint32_t s_bits_mode;
    __shared__ uint64_t s_stream_bytes, s_total_bytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    AttendWarpSmem<NS> &sm = reinterpret_cast<AttendWarpSmem<NS> *>(smem_raw)[warp];
    const qkvs_card_header_t *hdr = reinterpret_cast<const qkvs_card_header_t *>(p.card);

    if (threadIdx.x == 0) {
        PathParams hp;  // the fields header_matches looks at
        hp.card_bytes = p.card_bytes;
        hp.n_layers = p.n_layers;
        hp.n_kv_heads = p.n_kv_heads;
        hp.head_dim = kAttendD;
        hp.n_tokens = p.n_tokens;
        hp.meta_bytes = format_meta(META);
        hp.group_size = format_group(META);
        const uint32_t mode = hdr->bits_mode;
        int ok = 0;
        if (mode <= 1u) {
            const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, (int)mode);
            ok = sec.payload_off <= p.card_bytes && header_matches(hdr, hp, (int)mode, sec);
        }
        s_header_ok = ok;
        s_bits_mode = mode;
        s_stream_bytes = hdr->stream_bytes;
        s_total_bytes = hdr->total_bytes;
    }
    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(&sm.full[s], 1);
        fence_mbar_init();
    }
    __syncthreads();
    // the merge kernel may be brought onto the device now: it waits for this grid to complete
    // before it reads anything
    allow_dependents();
    if (!s_header_ok) {
        if (threadIdx.x == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
        return;
    }
    const int mode = (int)s_bits_mode;
    const uint64_t stream_bytes = s_stream_bytes, total_bytes = s_total_bytes;
    const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, mode);
    const uint32_t H = (uint32_t)p.n_kv_heads;
    const int per_kv = p.n_q_heads / p.n_kv_heads;
    const uint64_t T = (uint64_t)p.n_tokens;
    const uint32_t n_warps = gridDim.x * WARPS;

    int stage = 0;
    uint32_t parity = 0;
    bool ok = true;
    bool try_one_width = true;
    uint32_t item = blockIdx.x * WARPS + (uint32_t)warp;
    while (item < p.n_items && ok) {
        const uint32_t lh = item / p.items_per_head, ck = item - lh * p.items_per_head;
        const uint32_t layer = lh / H, head = lh - layer * H;
        const uint32_t sub0 = ck * kAttendSteps;

        const uint64_t seg = mode == 0 ? 0u : lh;
        const uint8_t *bits_tab = p.card + sec.bits_off + seg * T + (uint64_t)sub0 * kAttendRows;
        const uint32_t *offs_tab = reinterpret_cast<const uint32_t *>(p.card + sec.offs_off) + seg * (T + 1u) + (uint64_t)sub0 * kAttendRows;
        const uint64_t stream_k = ((uint64_t)layer * 2u) * H + head, stream_v = stream_k + H;
        uint64_t base_k, base_v;
        if (mode == 0) {
            base_k = sec.payload_off + stream_k * stream_bytes;
            base_v = sec.payload_off + stream_v * stream_bytes;
        } else {
            const uint64_t *sbase = reinterpret_cast<const uint64_t *>(p.card + sec.sbase_off);
            // entries beyond the card (a damaged table) must not wrap the sums around
            const uint64_t sk = __ldg(sbase + stream_k), sv = __ldg(sbase + stream_v);
            base_k = sk > total_bytes ? ~uint64_t(0) : sec.payload_off + sk;
            base_v = sv > total_bytes ? ~uint64_t(0) : sec.payload_off + sv;
        }
        // ---- the item's tokens, a run of kAttendPerLane per lane: check the table entries, sort by width into the list
        const uint32_t tok0 = sub0 * kAttendRows;
        const int n_tok = (int)min((uint64_t)(kAttendRows * kAttendSteps), T - tok0);
        uint32_t ends[4];  // where each class ends in the list
        const bool base_ok = base_k >= sec.payload_off && base_v >= sec.payload_off && ((base_k | base_v) & 15u) == 0u &&
                             base_k <= total_bytes && base_v <= total_bytes;
        const uint64_t room_k = base_ok ? total_bytes - base_k : 0u, room_v = base_ok ? total_bytes - base_v : 0u;
        // A whole item of one width (every item of a uniform card): eight bit-widths per lane in one
        // word, all equal, and the two offsets at the item's ends a whole item's records apart.  The
        // records are then neighbours from the first to the last -- the offsets cannot but grow by
        // the record size in between -- and the list is an arithmetic sequence.  Tried as long as
        // the warp's previous item was of that kind, so that a mixed card pays for the attempt once.
        static_assert(kAttendPerLane == 8, "one word of bit-widths per lane");
        bool one_width = false;
        if (try_one_width && n_tok == kAttendRows * kAttendSteps && (reinterpret_cast<uintptr_t>(bits_tab) & 7u) == 0u) {
            const uint2 w8 = __ldg(reinterpret_cast<const uint2 *>(bits_tab) + lane);
            const uint32_t o_first = __ldg(offs_tab), o_last = __ldg(offs_tab + n_tok);
            const uint32_t b0 = __shfl_sync(0xffffffffu, w8.x, 0) & 0xffu;
            const bool same = w8.x == b0 * 0x01010101u && w8.y == w8.x;
            const uint32_t rec = record_bytes(kAttendD, (int)b0, format_meta(META), format_group(META));
            one_width = __all_sync(0xffffffffu, same) && base_ok && rec != 0u && (o_first & 15u) == 0u && o_last >= o_first &&
                        o_last - o_first == (uint32_t)n_tok * rec && (uint64_t)o_last <= room_k && (uint64_t)o_last <= room_v;
            try_one_width = one_width;
            if (one_width) {
                const int cls = b0 == 2u ? 0 : (b0 == 4u ? 1 : (b0 == 8u ? 2 : 3));
#pragma unroll
                for (int c = 0; c < 4; ++c) ends[c] = c < cls ? 0u : (uint32_t)n_tok;
                __syncwarp();  // the previous item's list is no longer read
#pragma unroll
                for (int r = 0; r < kAttendPerLane; ++r) sm.list[kAttendPerLane * lane + r] = o_first + (uint32_t)(kAttendPerLane * lane + r) * rec;
                __syncwarp();
            }
        }
        uint32_t n_steps;
        if (!one_width) {
            uint32_t my_off[kAttendPerLane];
            int my_cls[kAttendPerLane];
            uint32_t counts = 0, counts_hi = 0;  // tokens of this lane per class: 16-bit fields (2 | 4 bits), (8 | 16 bits)
            {
                bool bad = false;
                uint32_t o_next = kAttendPerLane * lane <= n_tok ? __ldg(offs_tab + kAttendPerLane * lane) : 0u;
#pragma unroll
                for (int r = 0; r < kAttendPerLane; ++r) {
                    const int j = kAttendPerLane * lane + r;
                    const uint32_t o = o_next;
                    o_next = j + 1 <= n_tok ? __ldg(offs_tab + j + 1) : 0u;
                    my_off[r] = o;
                    my_cls[r] = 4;
                    if (j < n_tok) {
                        const uint32_t b = __ldg(bits_tab + j);
                        const uint32_t rec = record_bytes(kAttendD, (int)b, format_meta(META), format_group(META));
                        const bool fine = base_ok && rec != 0u && o_next >= o && o_next - o == rec && (o & 15u) == 0u &&
                                          (uint64_t)o_next <= room_k && (uint64_t)o_next <= room_v;
                        bad |= !fine;
                        if (fine) {
                            my_cls[r] = b == 2u ? 0 : (b == 4u ? 1 : (b == 8u ? 2 : 3));
                            if (my_cls[r] < 2) counts += 1u << (16 * my_cls[r]);
                            else counts_hi += 1u << (16 * (my_cls[r] - 2));
                        }
                    }
                }
                if (__any_sync(0xffffffffu, bad) && lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
            }
            // positions: class-major, then lane, then the lane's own order
            uint32_t inc = counts, inc_hi = counts_hi;
#pragma unroll
            for (int sft = 1; sft < 32; sft <<= 1) {
                const uint32_t a = __shfl_up_sync(0xffffffffu, inc, sft), bq = __shfl_up_sync(0xffffffffu, inc_hi, sft);
                if (lane >= sft) {
                    inc += a;
                    inc_hi += bq;
                }
            }
            const uint32_t tot = __shfl_sync(0xffffffffu, inc, 31), tot_hi = __shfl_sync(0xffffffffu, inc_hi, 31);
            ends[0] = tot & 0xffffu;
            ends[1] = ends[0] + (tot >> 16);
            ends[2] = ends[1] + (tot_hi & 0xffffu);
            ends[3] = ends[2] + (tot_hi >> 16);
            const uint32_t before = inc - counts, before_hi = inc_hi - counts_hi;  // in lower lanes
            uint32_t pos[4] = {before & 0xffffu, ends[0] + (before >> 16), ends[1] + (before_hi & 0xffffu), ends[2] + (before_hi >> 16)};
            __syncwarp();  // the previous item's list is no longer read
#pragma unroll
            for (int r = 0; r < kAttendPerLane; ++r) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (my_cls[r] == c) sm.list[pos[c]++] = my_off[r];
            }
            __syncwarp();
        }
        {
            // the steps, one descriptor per lane and round
            n_steps = 0;
#pragma unroll
            for (int r = 0; r < kAttendStepSlots / 32; ++r) {
                const uint32_t d = make_step<META>((uint32_t)(lane + 32 * r), ends, sm.list);
                sm.steps[lane + 32 * r] = d;
                n_steps += __popc(__ballot_sync(0xffffffffu, d != 0u));
            }
            __syncwarp();
        }

        // the group's queries as B fragments: lane (gid, tig) holds head gid, per group the channels
        // 32g + 8tig + k paired with + k + 4 (the pairing of key_pairs); and the sums over a group of
        // the queries of the lane's own two heads
        uint32_t qa[4][4];
        __syncwarp();  // the previous item's steps no longer read the query sums
        {
            const __half *qrow = p.q + ((uint64_t)layer * p.n_q_heads + (uint64_t)head * per_kv + gid) * kAttendD + 8 * tig;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint4 h = make_uint4(0u, 0u, 0u, 0u);
                if (gid < per_kv) h = __ldg(reinterpret_cast<const uint4 *>(qrow + 32 * g));
                qa[g][0] = __byte_perm(h.x, h.z, 0x5410);
                qa[g][1] = __byte_perm(h.x, h.z, 0x7632);
                qa[g][2] = __byte_perm(h.y, h.w, 0x5410);
                qa[g][3] = __byte_perm(h.y, h.w, 0x7632);
                const float2 f0 = __half22float2(as_half2(h.x)), f1 = __half22float2(as_half2(h.y));
                const float2 f2 = __half22float2(as_half2(h.z)), f3 = __half22float2(as_half2(h.w));
                float sum = ((f0.x + f0.y) + (f1.x + f1.y)) + ((f2.x + f2.y) + (f3.x + f3.y));
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);  // head gid's, in all four lanes of the gid
                const float s0 = __shfl_sync(0xffffffffu, sum, 8 * tig), s1 = __shfl_sync(0xffffffffu, sum, 8 * tig + 4);
                if (gid == 0) {
                    sm.qsum[tig][2 * g] = s0;
                    sm.qsum[tig][2 * g + 1] = s1;
                }
            }
        }
        __syncwarp();  // the query sums are in place
        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};
        float zacc[4][2] = {{0.0f, 0.0f}, {0.0f, 0.0f}, {0.0f, 0.0f}, {0.0f, 0.0f}};
        float acc[4][2][4];
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[g][h][i] = 0.0f;

        for (uint32_t i = 0; i < (uint32_t)NS && i < n_steps; ++i) {
            int st = stage + (int)i;
            if (st >= NS) st -= NS;
            attend_issue<NS, META>(sm, st, sm.steps[i], base_k, base_v, p, lane);
        }
        for (uint32_t i = 0; i < n_steps; ++i) {
            const uint32_t d = sm.steps[i];
            ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[stage], parity));
            if (!ok) break;
            const int rows = step_rows(d), cls = step_class(d);
            if (rows == kAttendRows) {  // 16-bit rows come at most eight per step
                switch (cls) {
                    case 0: attend_step<NS, 2, true, META>(sm, stage, rows, gid, tig, p.scale_log2, qa, m_run, l_run, zacc, acc); break;
                    case 1: attend_step<NS, 4, true, META>(sm, stage, rows, gid, tig, p.scale_log2, qa, m_run, l_run, zacc, acc); break;
                    default: attend_step<NS, 8, true, META>(sm, stage, rows, gid, tig, p.scale_log2, qa, m_run, l_run, zacc, acc); break;
                }
            } else {
                switch (cls) {
                    case 0: attend_step<NS, 2, false, META>(sm, stage, rows, gid, tig, p.scale_log2, qa, m_run, l_run, zacc, acc); break;
                    case 1: attend_step<NS, 4, false, META>(sm, stage, rows, gid, tig, p.scale_log2, qa, m_run, l_run, zacc, acc); break;
                    case 2: attend_step<NS, 8, false, META>(sm, stage, rows, gid, tig, p.scale_log2, qa, m_run, l_run, zacc, acc); break;
                    default: attend_step<NS, 16, false, META>(sm, stage, rows, gid, tig, p.scale_log2, qa, m_run, l_run, zacc, acc); break;
                }
            }
            __syncwarp();  // every lane has read the stage: it can be re-armed
            if (i + (uint32_t)NS < n_steps) attend_issue<NS, META>(sm, stage, sm.steps[i + NS], base_k, base_v, p, lane);
            if (++stage == NS) {
                stage = 0;
                parity ^= 1u;
            }
        }
        if (!ok) break;

        // ---- what the item found, per query head: unnormalised o (zero-point part added), maximum, sum
        // the lanes of a tig each hold a share (their tokens) of the sums of heads 2tig, 2tig + 1
        float z_lo[4], z_hi[4];
#pragma unroll
        for (int sft = 4; sft < 32; sft <<= 1) {
            l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sft);
            l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sft);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                zacc[g][0] += __shfl_xor_sync(0xffffffffu, zacc[g][0], sft);
                zacc[g][1] += __shfl_xor_sync(0xffffffffu, zacc[g][1], sft);
            }
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            z_lo[g] = zacc[g][0];
            z_hi[g] = zacc[g][1];
        }
        float *part = p.partials + (uint64_t)item * per_kv * kPartialFloats;
        if (gid == 0) {
#pragma unroll
            for (int h = 0; h < 2; ++h)
                if (2 * tig + h < per_kv) {
                    part[(2 * tig + h) * kPartialFloats + kAttendD] = m_run[h];
                    part[(2 * tig + h) * kPartialFloats + kAttendD + 1] = l_run[h];
                }
        }
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int ch = 32 * g + 4 * gid + 2 * h;
                if (2 * tig < per_kv)
                    *reinterpret_cast<float2 *>(part + (2 * tig) * kPartialFloats + ch) = make_float2(acc[g][h][0] + z_lo[g], acc[g][h][2] + z_lo[g]);
                if (2 * tig + 1 < per_kv)
                    *reinterpret_cast<float2 *>(part + (2 * tig + 1) * kPartialFloats + ch) = make_float2(acc[g][h][1] + z_hi[g], acc[g][h][3] + z_hi[g]);
            }

        uint32_t v = 0;
        if (lane == 0) v = atomicAdd(p.work_counter, 1u);
        v = __shfl_sync(0xffffffffu, v, 0);
        item = v < p.n_items ? n_warps + v : p.n_items;
    }
    if (!ok) {
        // an abandoned wait: nothing more is issued; the copies in flight (at most NS) get the
        // same bounded time to land before the shared memory is given back
        if (lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_TIMEOUT);
        for (int j = 0; j < NS; ++j) {
            mbar_wait(&sm.full[stage], parity);
            if (++stage == NS) {
                stage = 0;
                parity ^= 1u;
            }
        }
    }
}

// Merges the items of every query head: o = sum_i o_i 2^(m_i - M) / sum_i l_i 2^(m_i - M).
// One CTA of four warps per (layer, query head), a quarter of the items per warp, so that the
// whole merge is two rounds of loads and one exchange through shared memory; writes zeros when
// the first kernel reported a problem.  Inside a warp the items' maxima and sums are read one
// item per lane, so that the loads of an item's accumulators, which need its factor only for the
// multiplication, all go out at once.
__global__ void __launch_bounds__(128) attend_merge_kernel(AttendParams p)
{
    __shared__ float s_big[4], s_den[4];
    __shared__ float4 s_o[4][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t w = blockIdx.x;
    grid_dependency_wait();   // launched while the first kernel may still run: its results are complete from here on
    const int per_kv = p.n_q_heads / p.n_kv_heads;
    const uint32_t layer = w / (uint32_t)p.n_q_heads, j = w - layer * (uint32_t)p.n_q_heads;
    const uint32_t lh = layer * (uint32_t)p.n_kv_heads + j / (uint32_t)per_kv, jj = j % (uint32_t)per_kv;
    // the status word is only needed at the end: its load travels with the others
    const int32_t status = p.status_dev ? *reinterpret_cast<volatile const int32_t *>(p.status_dev) : 0;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    float big = -INFINITY, denom = 0.0f;
    if (p.items_per_head > 0) {
        const float *base = p.partials + ((uint64_t)lh * p.items_per_head * per_kv + jj) * kPartialFloats;
        const uint64_t stride = (uint64_t)per_kv * kPartialFloats;
        // this warp's items: [first, last), eight at a time: their maxima, sums and accumulators are
        // requested together, and the running maximum is brought up to date block by block
        const uint32_t share = (p.items_per_head + 3u) / 4u;
        const uint32_t first = min((uint32_t)warp * share, p.items_per_head), last = min(first + share, p.items_per_head);
        constexpr int kBlock = 8;
        for (uint32_t i0 = first; i0 < last; i0 += kBlock) {
            float2 ml[kBlock];   // maximum, sum
            float4 v[kBlock];
#pragma unroll
            for (int i = 0; i < kBlock; ++i) {
                const bool there = i0 + (uint32_t)i < last;
                const float *row = base + (there ? i0 + (uint32_t)i : i0) * stride;
                ml[i] = *reinterpret_cast<const float2 *>(row + kAttendD);
                v[i] = *reinterpret_cast<const float4 *>(row + 4 * lane);
                if (!there) ml[i] = make_float2(-INFINITY, 0.0f);
            }
            float top = big;
#pragma unroll
            for (int i = 0; i < kBlock; ++i) top = fmaxf(top, ml[i].x);
            const float keep = top == -INFINITY ? 0.0f : exp2f(big - top);   // 0 the first time round
            denom *= keep;
            o.x *= keep, o.y *= keep, o.z *= keep, o.w *= keep;
#pragma unroll
            for (int i = 0; i < kBlock; ++i) {
                const float f = ml[i].x == -INFINITY ? 0.0f : exp2f(ml[i].x - top);
                denom = fmaf(ml[i].y, f, denom);
                o.x = fmaf(v[i].x, f, o.x);
                o.y = fmaf(v[i].y, f, o.y);
                o.z = fmaf(v[i].z, f, o.z);
                o.w = fmaf(v[i].w, f, o.w);
            }
            big = top;
        }
    }
    const bool usable = p.items_per_head > 0 && status == 0;
    s_o[warp][lane] = o;
    if (lane == 0) {
        s_big[warp] = big;
        s_den[warp] = denom;
    }
    __syncthreads();
    if (warp == 0) {
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        if (usable) {
            const float top = fmaxf(fmaxf(s_big[0], s_big[1]), fmaxf(s_big[2], s_big[3]));
            float den = 0.0f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float f = s_big[k] == -INFINITY ? 0.0f : exp2f(s_big[k] - top);   // a warp without items
                const float4 v = s_o[k][lane];
                den = fmaf(s_den[k], f, den);
                sum.x = fmaf(v.x, f, sum.x);
                sum.y = fmaf(v.y, f, sum.y);
                sum.z = fmaf(v.z, f, sum.z);
                sum.w = fmaf(v.w, f, sum.w);
            }
            const float r = 1.0f / den;
            sum.x *= r, sum.y *= r, sum.z *= r, sum.w *= r;
        }
        *reinterpret_cast<float4 *>(p.out + (uint64_t)w * kAttendD + 4 * lane) = sum;
    }
}

}  // namespace qkvs
