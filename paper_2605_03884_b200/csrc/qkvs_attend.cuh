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
//   scores   rows = query heads of the group (up to 8 of 16 used), columns = 8 tokens; lane (g, t)
//            supplies 8 codes of token g from each group and holds the matching channels of Q;
//   outputs  rows = channels, columns = query heads; lane (g, t) supplies 4 channels per group of
//            the four tokens 2t, 2t+1, 2t+8, 2t+9, and the probabilities it computed itself, times
//            the tokens' scales, are already the B fragment.
// Softmax is the usual running maximum / running sum; every item leaves (o, max, sum) per query
// head in the scratch buffer and a second small kernel merges the items of a head.
#pragma once

#include "qkvs_pipeline.cuh"

namespace qkvs {

constexpr int kAttendD = 128;
constexpr int kAttendRows = 16;          // tokens per step
constexpr int kAttendSteps = 16;         // steps per work item
constexpr int kAttendMaxPerKv = 8;       // query heads per KV head
constexpr int kPartialFloats = kAttendD + 4;  // o[128], running maximum (base-2 exponent), running sum, padding

struct AttendParams {
    const uint8_t *card;
    uint64_t card_bytes;
    int32_t n_layers, n_kv_heads, n_tokens, n_q_heads;
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
    alignas(128) uint8_t k[NS][kAttendRows * 2 * kAttendD];
    alignas(128) uint8_t v[NS][kAttendRows * 2 * kAttendD];
    uint32_t info[NS][kAttendRows];  // per token: record offset inside the span << 8 | bit-width
    alignas(8) uint64_t full[NS];
    int32_t rows[NS];                // 0 when the step's table entries did not check out
    uint32_t uniform_bits[NS];       // bit-width shared by all 16 rows, else 0
};

__device__ __forceinline__ void mma_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float exp2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t word_of(const uint4 &v, int i)
{
    return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

// Checks a step's table entries, publishes the per-token record positions and starts the copies
// of its K and V spans (same offsets, two streams).  All lanes call it.
template <int NS>
__device__ __forceinline__ void attend_issue(AttendWarpSmem<NS> &sm, int stage, const Tables &t, uint64_t base_k, uint64_t base_v,
                                             const AttendParams &p, const Sections &sec, uint64_t total_bytes, int lane)
{
    const int rows = t.rows;
    const uint32_t off0 = __shfl_sync(0xffffffffu, t.off, 0);
    const uint32_t off_next = __shfl_down_sync(0xffffffffu, t.off, 1);
    const uint32_t off_end = __shfl_sync(0xffffffffu, t.off, rows);
    int bad = 0;
    if (lane < rows) {
        const uint32_t rec = record_bytes(kAttendD, (int)t.bits);
        bad = (rec == 0u) || (off_next < t.off) || (off_next - t.off != rec);
        sm.info[stage][lane] = ((t.off - off0) << 8) | (t.bits & 0xffu);
    }
    bad = __any_sync(0xffffffffu, bad);
    const uint32_t b0 = __shfl_sync(0xffffffffu, t.bits, 0);
    const bool uniform = rows == kAttendRows && __all_sync(0xffffffffu, lane >= rows || t.bits == b0);
    const uint32_t span = off_end - off0;  // consistent records: at most rows * 256 bytes, fits the stage
    bad |= (off0 & 15u) != 0u || base_k < sec.payload_off || base_v < sec.payload_off || ((base_k | base_v) & 15u) != 0u ||
           base_k + (uint64_t)off_end > total_bytes || base_v + (uint64_t)off_end > total_bytes;
    if (lane == 0) {
        sm.rows[stage] = bad ? 0 : rows;
        sm.uniform_bits[stage] = uniform ? b0 : 0u;
        if (bad && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
        if (!bad && span) {
            mbar_arrive_expect_tx(&sm.full[stage], 2u * span);
            bulk_load(sm.k[stage], p.card + base_k + off0, span, &sm.full[stage]);
            bulk_load(sm.v[stage], p.card + base_v + off0, span, &sm.full[stage]);
        } else {
            mbar_arrive(&sm.full[stage]);
        }
    }
    __syncwarp();
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

// Key side.  The lane's 8 channels of group g of one token (channels 32g + 8t + 0..7) as four
// FP16 pairs e[k] = (value k, value k + 4) -- codes for a quantised row, the FP16 values for a
// 16-bit row.  The query fragments pair channels the same way.
template <int B>
__device__ __forceinline__ void key_pairs(const uint8_t *rec, int b, int g, int tig, uint32_t (&e)[4])
{
    const int bb = B ? B : b;
    if (B == 16 || (B == 0 && bb == 16)) {
        const uint4 h = *reinterpret_cast<const uint4 *>(rec + 64 * g + 16 * tig);
        e[0] = __byte_perm(h.x, h.z, 0x5410);
        e[1] = __byte_perm(h.x, h.z, 0x7632);
        e[2] = __byte_perm(h.y, h.w, 0x5410);
        e[3] = __byte_perm(h.y, h.w, 0x7632);
        return;
    }
    const uint8_t *codes = rec + 4 * kMetaBytesPerGroup + (4 * g + tig) * bb;  // the lane's 8 codes: b bytes
    if constexpr (B == 4) {
        const uint32_t w = *reinterpret_cast<const uint32_t *>(codes);  // nibble k and k + 4 are 16 bits apart
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(w >> (4 * k), 0x000f000fu);
    } else if constexpr (B == 8) {
        const uint2 w = *reinterpret_cast<const uint2 *>(codes);
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(__byte_perm(w.x, w.y, 0x0011u * k + 0x1100u * (4 + k)), 0x00ff00ffu);
    } else if constexpr (B == 2) {
        const uint32_t w = *reinterpret_cast<const uint16_t *>(codes);
        const uint32_t y = __byte_perm(w, 0u, 0x4140);  // codes 0..3 in byte 0, codes 4..7 in byte 2
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(y >> (2 * k), 0x00030003u);
    } else if constexpr (B == 0) {
        // width known per lane only: one instruction stream for 2, 4 and 8 bits.  The b bytes sit
        // inside one aligned 8-byte window; codes 0..3 end up in `lo`, codes 4..7 in `hi`, each
        // at k * b bits, and a pair is (lo >> k*b) & mask | ((hi >> k*b) & mask) << 16.
        const uint32_t a = smem_addr(codes);
        const uint2 win = *reinterpret_cast<const uint2 *>(codes - (a & 7u));
        const uint32_t sh = (a & 7u) * 8u;
        const uint32_t lo = sh >= 32u ? win.y >> (sh - 32u) : __funnelshift_r(win.x, win.y, sh);  // first 32 bits of the codes
        const uint32_t hi = bb == 8 ? win.y : lo >> (4 * bb);                                         // from code 4 on
        const uint32_t mask = (1u << bb) - 1u;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t pair = ((lo >> (k * bb)) & mask) | (((hi >> (k * bb)) & mask) << 16);
            e[k] = int_pair(pair, 0x00ff00ffu);
        }
    }
}

// Value side, one token: the lane's 4 channels of group g (channels 32g + 4gid + 0..3) as two FP16
// pairs (value 0, value 1), (value 2, value 3).
__device__ __forceinline__ void value_quad(const uint8_t *rec, int b, int g, int gid, uint32_t &p01, uint32_t &p23)
{
    if (b == 16) {
        const uint2 h = *reinterpret_cast<const uint2 *>(rec + 64 * g + 8 * gid);
        p01 = h.x;
        p23 = h.y;
    } else {
        // one instruction stream for 2, 4 and 8 bits: the lane's 4 codes are b/2 bytes inside one
        // aligned 4-byte word
        const uint8_t *codes = rec + 4 * kMetaBytesPerGroup + (8 * g) * (b / 2) + gid * (b / 2);
        const uint32_t a = smem_addr(codes);
        const uint32_t x = *reinterpret_cast<const uint32_t *>(codes - (a & 3u)) >> ((a & 3u) * 8u);
        const uint32_t mask = (1u << b) - 1u;
        p01 = int_pair((x & mask) | (((x >> b) & mask) << 16), 0x00ff00ffu);
        p23 = int_pair(((x >> (2 * b)) & mask) | (((x >> (3 * b)) & mask) << 16), 0x00ff00ffu);
    }
}

// Value side, two tokens of one known width B at once: the lane's 4 channels of group g as four
// FP16 pairs e[k] = (token a's value k, token b's value k).
template <int B>
__device__ __forceinline__ void value_pairs(const uint8_t *rec_a, const uint8_t *rec_b, int g, int gid, uint32_t (&e)[4])
{
    if (B == 16) {
        const uint2 ha = *reinterpret_cast<const uint2 *>(rec_a + 64 * g + 8 * gid);
        const uint2 hb = *reinterpret_cast<const uint2 *>(rec_b + 64 * g + 8 * gid);
        e[0] = __byte_perm(ha.x, hb.x, 0x5410);
        e[1] = __byte_perm(ha.x, hb.x, 0x7632);
        e[2] = __byte_perm(ha.y, hb.y, 0x5410);
        e[3] = __byte_perm(ha.y, hb.y, 0x7632);
    } else if (B == 4) {
        const uint32_t wa = *reinterpret_cast<const uint16_t *>(rec_a + 32 + 16 * g + 2 * gid);
        const uint32_t wb = *reinterpret_cast<const uint16_t *>(rec_b + 32 + 16 * g + 2 * gid);
        const uint32_t x = wa | (wb << 16);
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(x >> (4 * k), 0x000f000fu);
    } else if (B == 8) {
        const uint32_t wa = *reinterpret_cast<const uint32_t *>(rec_a + 32 + 32 * g + 4 * gid);
        const uint32_t wb = *reinterpret_cast<const uint32_t *>(rec_b + 32 + 32 * g + 4 * gid);
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(__byte_perm(wa, wb, 0x0011u * k + 0x1100u * (4 + k)), 0x00ff00ffu);
    } else {
        const uint32_t x = (uint32_t)*(rec_a + 32 + 8 * g + gid) | ((uint32_t)*(rec_b + 32 + 8 * g + gid) << 16);
#pragma unroll
        for (int k = 0; k < 4; ++k) e[k] = int_pair(x >> (2 * k), 0x00030003u);
    }
}

// Scale / zero pairs of a token's four groups; (1, 0) for a 16-bit row, (0, 0) for no token.
// B != 0: the width is B and the token exists.
template <int B>
__device__ __forceinline__ void group_params_of(const uint8_t *rec, int b, bool valid, float (&sc)[4], float (&ze)[4])
{
    if (B ? B != 16 : (valid && b != 16)) {
        const uint4 m0 = *reinterpret_cast<const uint4 *>(rec), m1 = *reinterpret_cast<const uint4 *>(rec + 16);
        sc[0] = __uint_as_float(m0.x), ze[0] = __uint_as_float(m0.y), sc[1] = __uint_as_float(m0.z), ze[1] = __uint_as_float(m0.w);
        sc[2] = __uint_as_float(m1.x), ze[2] = __uint_as_float(m1.y), sc[3] = __uint_as_float(m1.z), ze[3] = __uint_as_float(m1.w);
    } else {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            sc[g] = (B || valid) ? 1.0f : 0.0f;
            ze[g] = 0.0f;
        }
    }
}

// One step: 16 tokens of K and V staged in `stage` against the group's queries.  Updates the
// running maximum / sum of head g, the zero-point sums and the output accumulators.  B is the
// bit-width shared by all 16 rows, or 0 when they differ or the step is short.
//   qa[g][k]    query fragments: head gid, channels 32g + 8tig + k and + k + 4
//   qsum[g]     sum of head gid's query over group g
//   zacc[g]     sum_t p_t zero_tg for head gid, over the tokens this lane has seen
//   acc[g][h]   channels 32g + 4gid + 2h (+1) x heads 2tig, 2tig + 1, without the zero-point part
template <int NS, int B>
__device__ __forceinline__ void attend_step(const AttendWarpSmem<NS> &sm, int stage, int rows, int gid, int tig, float scale_log2,
                                            const uint32_t (&qa)[4][4], const float (&qsum)[4], float &m_run, float &l_run,
                                            float (&zacc)[4], float (&acc)[4][2][4])
{
    // the lane's four tokens (the same ones on the score side and on the value side)
    int tok[4], bw[4];
    uint32_t off[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        tok[i] = 2 * tig + (i & 1) + 8 * (i >> 1);
        const uint32_t inf = (B || tok[i] < rows) ? sm.info[stage][tok[i]] : 0u;
        off[i] = inf >> 8;
        bw[i] = B ? B : (int)(inf & 0xffu);
    }
    // ---- scores: per group, sum_c q_c code_c for the heads of the group x 2 blocks of 8 tokens
    float x[4];  // logits (base 2) of head gid for the lane's four tokens
    {
        float sacc[2][4][4];
#pragma unroll
        for (int bi = 0; bi < 2; ++bi) {
            const int t = 8 * bi + gid;
            const uint32_t inf = (B || t < rows) ? sm.info[stage][t] : 0u;
            const uint8_t *rec = sm.k[stage] + (inf >> 8);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint32_t e[4] = {0u, 0u, 0u, 0u};  // lanes without a token feed zeros
                if (B || t < rows) key_pairs<B>(rec, (int)(inf & 0xffu), g, tig, e);
#pragma unroll
                for (int i = 0; i < 4; ++i) sacc[bi][g][i] = 0.0f;
                mma_m16n8k16(sacc[bi][g], qa[g][0], 0u, qa[g][1], 0u, e[0], e[1]);  // the whole warp, together
                mma_m16n8k16(sacc[bi][g], qa[g][2], 0u, qa[g][3], 0u, e[2], e[3]);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float sc[4], ze[4];
            group_params_of<B>(sm.k[stage] + off[i], bw[i], tok[i] < rows, sc, ze);
            float dot = 0.0f;
#pragma unroll
            for (int g = 0; g < 4; ++g) dot = fmaf(sc[g], sacc[i >> 1][g][i & 1], fmaf(ze[g], qsum[g], dot));
            x[i] = (B || tok[i] < rows) ? dot * scale_log2 : -INFINITY;
        }
    }
    // ---- running softmax for head gid
    float m_loc = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 1));
    m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 2));
    const float m_new = fmaxf(m_run, m_loc);
    const float m_ref = m_new == -INFINITY ? 0.0f : m_new;
    const float alpha = exp2_approx(m_run - m_ref);  // 0 on the first tokens of the item
    float pr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) pr[i] = exp2_approx(x[i] - m_ref);
    l_run = fmaf(l_run, alpha, (pr[0] + pr[1]) + (pr[2] + pr[3]));
    m_run = m_new;
    // the accumulators of this lane belong to heads 2t and 2t + 1, whose factors other lanes hold
    const float a_lo = __shfl_sync(0xffffffffu, alpha, 8 * tig);
    const float a_hi = __shfl_sync(0xffffffffu, alpha, 8 * tig + 4);
    if (__any_sync(0xffffffffu, a_lo != 1.0f || a_hi != 1.0f || alpha != 1.0f)) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            zacc[g] *= alpha;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                acc[g][h][0] *= a_lo;
                acc[g][h][1] *= a_hi;
                acc[g][h][2] *= a_lo;
                acc[g][h][3] *= a_hi;
            }
        }
    }
    // ---- values: probabilities times the tokens' scales against the codes; zero points aside
    float vs[4][4];  // [token][group]
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float ze[4];
        group_params_of<B>(sm.v[stage] + off[i], bw[i], tok[i] < rows, vs[i], ze);
#pragma unroll
        for (int g = 0; g < 4; ++g) zacc[g] = fmaf(pr[i], ze[g], zacc[g]);
    }
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t pb0 = as_u32(__floats2half2_rn(pr[0] * vs[0][g], pr[1] * vs[1][g]));
        const uint32_t pb1 = as_u32(__floats2half2_rn(pr[2] * vs[2][g], pr[3] * vs[3][g]));
        uint32_t eab[4], ecd[4];
        if (B) {
            value_pairs<B>(sm.v[stage] + off[0], sm.v[stage] + off[1], g, gid, eab);
            value_pairs<B>(sm.v[stage] + off[2], sm.v[stage] + off[3], g, gid, ecd);
        } else {
            uint32_t q01[4], q23[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                q01[i] = 0u;
                q23[i] = 0u;
                if (tok[i] < rows) value_quad(sm.v[stage] + off[i], bw[i], g, gid, q01[i], q23[i]);
            }
            eab[0] = __byte_perm(q01[0], q01[1], 0x5410), eab[1] = __byte_perm(q01[0], q01[1], 0x7632);
            eab[2] = __byte_perm(q23[0], q23[1], 0x5410), eab[3] = __byte_perm(q23[0], q23[1], 0x7632);
            ecd[0] = __byte_perm(q01[2], q01[3], 0x5410), ecd[1] = __byte_perm(q01[2], q01[3], 0x7632);
            ecd[2] = __byte_perm(q23[2], q23[3], 0x5410), ecd[3] = __byte_perm(q23[2], q23[3], 0x7632);
        }
        mma_m16n8k16(acc[g][0], eab[0], eab[1], ecd[0], ecd[1], pb0, pb1);
        mma_m16n8k16(acc[g][1], eab[2], eab[3], ecd[2], ecd[3], pb0, pb1);
    }
}

template <int NS, int WARPS>
__global__ void __launch_bounds__(WARPS * 32, 3) attend_kernel(AttendParams p)
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
    uint32_t item = blockIdx.x * WARPS + (uint32_t)warp;
    while (item < p.n_items && ok) {
        const uint32_t lh = item / p.items_per_head, ck = item - lh * p.items_per_head;
        const uint32_t layer = lh / H, head = lh - layer * H;
        const uint32_t sub0 = ck * kAttendSteps;
        const int n_steps = (int)min((uint32_t)kAttendSteps, p.subs_per_head - sub0);

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
            base_k = sec.payload_off + __ldg(sbase + stream_k);
            base_v = sec.payload_off + __ldg(sbase + stream_v);
        }
        auto fetch = [&](Tables &t, int step) {
            t.rows = (sub0 + (uint32_t)step + 1u == p.subs_per_head) ? (int)p.last_rows : kAttendRows;
            t.base = 0;
            t.off = lane <= t.rows ? __ldg(offs_tab + step * kAttendRows + lane) : 0u;
            t.bits = lane < t.rows ? (uint32_t)__ldg(bits_tab + step * kAttendRows + lane) : 0u;
        };

        // the group's queries as A fragments: lane (gid, tig) holds head gid, per group the channels
        // 32g + 8tig + k paired with + k + 4 (the pairing of key_pairs), and the query's sum over the group
        uint32_t qa[4][4];
        float qsum[4];
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
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                qsum[g] = sum;
            }
        }
        float m_run = -INFINITY, l_run = 0.0f;  // of head gid (same in the four lanes of a gid; l_run summed at the end)
        float zacc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        float acc[4][2][4];
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[g][h][i] = 0.0f;

        Tables nxt;
        fetch(nxt, 0);
        int issued = 0;
        for (; issued < NS && issued < n_steps; ++issued) {
            const Tables cur = nxt;
            if (issued + 1 < n_steps) fetch(nxt, issued + 1);
            int st = stage + issued;
            if (st >= NS) st -= NS;
            attend_issue<NS>(sm, st, cur, base_k, base_v, p, sec, total_bytes, lane);
        }

        for (int step = 0; step < n_steps; ++step) {
            ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[stage], parity));
            if (!ok) break;
            const int rows = sm.rows[stage];

            switch (sm.uniform_bits[stage]) {  // all 16 rows of one width: the specialised body
                case 4: attend_step<NS, 4>(sm, stage, rows, gid, tig, p.scale_log2, qa, qsum, m_run, l_run, zacc, acc); break;
                case 2: attend_step<NS, 2>(sm, stage, rows, gid, tig, p.scale_log2, qa, qsum, m_run, l_run, zacc, acc); break;
                case 8: attend_step<NS, 8>(sm, stage, rows, gid, tig, p.scale_log2, qa, qsum, m_run, l_run, zacc, acc); break;
                case 16: attend_step<NS, 16>(sm, stage, rows, gid, tig, p.scale_log2, qa, qsum, m_run, l_run, zacc, acc); break;
                default: attend_step<NS, 0>(sm, stage, rows, gid, tig, p.scale_log2, qa, qsum, m_run, l_run, zacc, acc); break;
            }
            __syncwarp();  // every lane has read the stage: it can be re-armed
            if (issued < n_steps) {
                const Tables cur = nxt;
                if (issued + 1 < n_steps) fetch(nxt, issued + 1);
                attend_issue<NS>(sm, stage, cur, base_k, base_v, p, sec, total_bytes, lane);
                ++issued;
            }
            if (++stage == NS) {
                stage = 0;
                parity ^= 1u;
            }
        }
        if (!ok) break;

        // ---- what the item found, per query head: unnormalised o (zero-point part added), maximum, sum
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        float z_lo[4], z_hi[4];  // of heads 2tig and 2tig + 1
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            float z = zacc[g];
            z += __shfl_xor_sync(0xffffffffu, z, 1);
            z += __shfl_xor_sync(0xffffffffu, z, 2);
            z_lo[g] = __shfl_sync(0xffffffffu, z, 8 * tig);
            z_hi[g] = __shfl_sync(0xffffffffu, z, 8 * tig + 4);
        }
        float *part = p.partials + (uint64_t)item * per_kv * kPartialFloats;
        if (tig == 0 && gid < per_kv) {
            part[gid * kPartialFloats + kAttendD] = m_run;
            part[gid * kPartialFloats + kAttendD + 1] = l_run;
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
// One warp per (layer, query head); writes zeros when the first kernel reported a problem.
__global__ void __launch_bounds__(128) attend_merge_kernel(AttendParams p)
{
    const int lane = threadIdx.x & 31;
    const uint32_t w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const uint32_t n_rows = (uint32_t)p.n_layers * (uint32_t)p.n_q_heads;
    if (w >= n_rows) return;
    const int per_kv = p.n_q_heads / p.n_kv_heads;
    const uint32_t layer = w / (uint32_t)p.n_q_heads, j = w - layer * (uint32_t)p.n_q_heads;
    const uint32_t lh = layer * (uint32_t)p.n_kv_heads + j / (uint32_t)per_kv, jj = j % (uint32_t)per_kv;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    const bool usable = p.items_per_head > 0 && (!p.status_dev || *p.status_dev == 0);
    if (usable) {
        const float *base = p.partials + ((uint64_t)lh * p.items_per_head * per_kv + jj) * kPartialFloats;
        const uint64_t stride = (uint64_t)per_kv * kPartialFloats;
        float big = -INFINITY;
        for (uint32_t i = 0; i < p.items_per_head; ++i) big = fmaxf(big, base[i * stride + kAttendD]);
        float denom = 0.0f;
        for (uint32_t i = 0; i < p.items_per_head; ++i) {
            const float *part = base + i * stride;
            const float f = exp2f(part[kAttendD] - big);
            denom += part[kAttendD + 1] * f;
            const float4 v = *reinterpret_cast<const float4 *>(part + 4 * lane);
            o.x += v.x * f;
            o.y += v.y * f;
            o.z += v.z * f;
            o.w += v.w * f;
        }
        const float r = 1.0f / denom;
        o.x *= r;
        o.y *= r;
        o.z *= r;
        o.w *= r;
    }
    *reinterpret_cast<float4 *>(p.out + (uint64_t)w * kAttendD + 4 * lane) = o;
}

}  // namespace qkvs
