// Decode-step attention straight from a card: one query token per layer attends to every token
// of the card, reading the records themselves -- the FP16 cache is never written out.
//
//     s_t = softmax_scale * q . K^_t,   p = softmax(s),   o = sum_t p_t V^_t
//
// with K^, V^ exactly the FP16 values injection reconstructs (the same decode_chunk), grouped
// queries (query head j reads KV head j / per_kv), head_dim 128.
//
// Work item: 256 consecutive tokens of one (layer, KV head), taken by one warp from a counter.
// The warp walks them in steps of 16 tokens; the spans of K and V records of a step are staged by
// two bulk copies (TMA) on one mbarrier, NS steps ahead.  Both products run on the tensor cores
// (mma.sync m16n8k16, FP16 inputs, FP32 accumulation) with operands laid out so that every lane
// decodes exactly the values its own fragments need -- nothing passes through shared memory
// after decoding:
//   scores   S = Q K^T : rows = query heads of the group (up to 8 of 16 used), columns = 8 tokens
//            per instruction; lane (g, t) supplies token g's group t (channels 32t .. 32t+31,
//            four per k-step), and holds the matching channels of Q;
//   outputs  O^T = V^T P^T : rows = channels, columns = query heads; lane (g, t) supplies channels
//            16g .. 16g+15 of the four tokens 2t, 2t+1, 2t+8, 2t+9, and the probabilities it
//            computed itself from S are already the B fragment.
// Softmax is the usual running maximum / running sum; every item leaves (max, sum, o) per query
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

// N consecutive chunks (pos0 .. pos0 + N - 1, all inside one group of a row whose record is `rec`)
// -> N x 8 FP16 values, bit for bit what injection reconstructs.  With the bit-width B known at
// compile time the group's scale / zero pair and its codes are fetched once for the whole run;
// B = 0 decodes chunk by chunk with the row's own width `b`.
template <int B, int N>
__device__ __forceinline__ void decode_run(const uint8_t *rec, int b, int pos0, uint4 (&out)[N])
{
    constexpr int G = kAttendD / kGroup;
    if (B == 0) {
#pragma unroll
        for (int i = 0; i < N; ++i) out[i] = decode_chunk<kAttendD, 0>(rec, b, pos0 + i);
        return;
    }
    if (B == 16) {
#pragma unroll
        for (int i = 0; i < N; ++i) out[i] = *reinterpret_cast<const uint4 *>(rec + (pos0 + i) * 16);
        return;
    }
    const float2 m = *reinterpret_cast<const float2 *>(rec + (pos0 >> 2) * kMetaBytesPerGroup);
    const Dequant dq = make_dequant(m.x, m.y);
    const uint8_t *codes = rec + G * kMetaBytesPerGroup + pos0 * B;  // N * B bytes, aligned to their size
    uint32_t w[N * B / 4 > 0 ? N * B / 4 : 1];
    if (N * B == 32) {
        const uint4 a = *reinterpret_cast<const uint4 *>(codes), c = *reinterpret_cast<const uint4 *>(codes + 16);
        w[0] = a.x, w[1] = a.y, w[2] = a.z, w[3] = a.w, w[4] = c.x, w[5] = c.y, w[6] = c.z, w[7] = c.w;
    } else if (N * B == 16) {
        const uint4 a = *reinterpret_cast<const uint4 *>(codes);
        w[0] = a.x, w[1] = a.y, w[2] = a.z, w[3] = a.w;
    } else if (N * B == 8) {
        const uint2 a = *reinterpret_cast<const uint2 *>(codes);
        w[0] = a.x, w[1] = a.y;
    } else {
        w[0] = *reinterpret_cast<const uint32_t *>(codes);
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
        uint32_t lo, hi;
        if (B == 8) {
            lo = w[2 * i];
            hi = w[2 * i + 1];
        } else if (B == 4) {
            unpack_nibbles(w[i], lo, hi);
        } else {
            unpack_nibbles(unpack_crumbs((w[i >> 1] >> (16 * (i & 1))) & 0xffffu), lo, hi);
        }
        out[i] = dequantize_chunk(lo, hi, dq);
    }
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

// One step: 16 tokens of K and V staged in `stage` against the group's queries.  Updates the
// running maximum / sum of head g and the output accumulators.  B is the bit-width shared by all
// 16 rows, or 0 when they differ or the step is short.
template <int NS, int B>
__device__ __forceinline__ void attend_step(const AttendWarpSmem<NS> &sm, int stage, int rows, int gid, int tig, float scale_log2,
                                            const uint32_t (&qa0)[8], const uint32_t (&qa2)[8], float &m_run, float &l_run,
                                            float (&acc)[8][4])
{
    // ---- scores of 2 x 8 tokens for the heads of the group
    float sacc[2][4];
#pragma unroll
    for (int bi = 0; bi < 2; ++bi) {
#pragma unroll
        for (int i = 0; i < 4; ++i) sacc[bi][i] = 0.0f;
        const int tok = 8 * bi + gid;
        uint4 kq[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) kq[c] = make_uint4(0, 0, 0, 0);  // lanes without a token feed zeros
        if (tok < rows) {
            const uint32_t inf = sm.info[stage][tok];
            const uint8_t *rec = sm.k[stage] + (inf >> 8);
            decode_run<B, 4>(rec, (int)(inf & 0xffu), 4 * tig, kq);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {  // the whole warp executes every mma together
            mma_m16n8k16(sacc[bi], qa0[2 * c], 0u, qa2[2 * c], 0u, kq[c].x, kq[c].y);
            mma_m16n8k16(sacc[bi], qa0[2 * c + 1], 0u, qa2[2 * c + 1], 0u, kq[c].z, kq[c].w);
        }
    }
    // ---- running softmax for head g over tokens 8bi + 2t + e
    float x[2][2];
    float m_loc = -INFINITY;
#pragma unroll
    for (int bi = 0; bi < 2; ++bi)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            x[bi][e] = (8 * bi + 2 * tig + e) < rows ? sacc[bi][e] * scale_log2 : -INFINITY;
            m_loc = fmaxf(m_loc, x[bi][e]);
        }
    m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 1));
    m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 2));
    const float m_new = fmaxf(m_run, m_loc);
    const float m_ref = m_new == -INFINITY ? 0.0f : m_new;
    const float alpha = exp2_approx(m_run - m_ref);  // 0 on the first tokens of the item
    float pr[2][2];
#pragma unroll
    for (int bi = 0; bi < 2; ++bi)
#pragma unroll
        for (int e = 0; e < 2; ++e) pr[bi][e] = exp2_approx(x[bi][e] - m_ref);
    l_run = l_run * alpha + (pr[0][0] + pr[0][1]) + (pr[1][0] + pr[1][1]);
    m_run = m_new;
    const uint32_t pb0 = as_u32(__floats2half2_rn(pr[0][0], pr[0][1]));
    const uint32_t pb1 = as_u32(__floats2half2_rn(pr[1][0], pr[1][1]));
    // the accumulators of this lane belong to heads 2t and 2t + 1, whose factors other lanes hold
    const float a_lo = __shfl_sync(0xffffffffu, alpha, 8 * tig);
    const float a_hi = __shfl_sync(0xffffffffu, alpha, 8 * tig + 4);
    if (__any_sync(0xffffffffu, a_lo != 1.0f || a_hi != 1.0f)) {
#pragma unroll
        for (int mb = 0; mb < 8; ++mb) {
            acc[mb][0] *= a_lo;
            acc[mb][1] *= a_hi;
            acc[mb][2] *= a_lo;
            acc[mb][3] *= a_hi;
        }
    }
    // ---- values: channels 16g .. 16g+15 of tokens 2t, 2t+1, 2t+8, 2t+9
    uint4 vq[4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int tok = 2 * tig + (i & 1) + 8 * (i >> 1);
        vq[i][0] = make_uint4(0, 0, 0, 0);
        vq[i][1] = make_uint4(0, 0, 0, 0);
        if (tok < rows) {
            const uint32_t inf = sm.info[stage][tok];
            const uint8_t *rec = sm.v[stage] + (inf >> 8);
            decode_run<B, 2>(rec, (int)(inf & 0xffu), 2 * gid, vq[i]);
        }
    }
#pragma unroll
    for (int mb = 0; mb < 8; ++mb) {
        const uint32_t wa = word_of(vq[0][mb >> 2], mb & 3), wb = word_of(vq[1][mb >> 2], mb & 3);
        const uint32_t wc = word_of(vq[2][mb >> 2], mb & 3), wd = word_of(vq[3][mb >> 2], mb & 3);
        mma_m16n8k16(acc[mb], __byte_perm(wa, wb, 0x5410), __byte_perm(wa, wb, 0x7632), __byte_perm(wc, wd, 0x5410),
                     __byte_perm(wc, wd, 0x7632), pb0, pb1);
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

        // the group's queries as A fragments: lane (g, t) holds head g, channels 32t + 4kk + {0,1 | 2,3}
        uint32_t qa0[8], qa2[8];
        {
            const __half *qrow = p.q + ((uint64_t)layer * p.n_q_heads + (uint64_t)head * per_kv + gid) * kAttendD + 32 * tig;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                qa0[kk] = gid < per_kv ? __ldg(reinterpret_cast<const uint32_t *>(qrow + 4 * kk)) : 0u;
                qa2[kk] = gid < per_kv ? __ldg(reinterpret_cast<const uint32_t *>(qrow + 4 * kk + 2)) : 0u;
            }
        }
        float m_run = -INFINITY, l_run = 0.0f;  // of head g (same in the four lanes of a g, l_run summed at the end)
        float acc[8][4];                        // O^T: channels 16g + 2mb (+1) x heads 2t, 2t + 1
#pragma unroll
        for (int mb = 0; mb < 8; ++mb)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mb][i] = 0.0f;

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
                case 4: attend_step<NS, 4>(sm, stage, rows, gid, tig, p.scale_log2, qa0, qa2, m_run, l_run, acc); break;
                case 2: attend_step<NS, 2>(sm, stage, rows, gid, tig, p.scale_log2, qa0, qa2, m_run, l_run, acc); break;
                case 8: attend_step<NS, 8>(sm, stage, rows, gid, tig, p.scale_log2, qa0, qa2, m_run, l_run, acc); break;
                case 16: attend_step<NS, 16>(sm, stage, rows, gid, tig, p.scale_log2, qa0, qa2, m_run, l_run, acc); break;
                default: attend_step<NS, 0>(sm, stage, rows, gid, tig, p.scale_log2, qa0, qa2, m_run, l_run, acc); break;
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

        // ---- what the item found, per query head: running maximum, running sum, unnormalised o
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        float *part = p.partials + (uint64_t)item * per_kv * kPartialFloats;
        if (tig == 0 && gid < per_kv) {
            part[gid * kPartialFloats + kAttendD] = m_run;
            part[gid * kPartialFloats + kAttendD + 1] = l_run;
        }
#pragma unroll
        for (int mb = 0; mb < 8; ++mb) {
            const int ch = 16 * gid + 2 * mb;
            if (2 * tig < per_kv) *reinterpret_cast<float2 *>(part + (2 * tig) * kPartialFloats + ch) = make_float2(acc[mb][0], acc[mb][2]);
            if (2 * tig + 1 < per_kv) *reinterpret_cast<float2 *>(part + (2 * tig + 1) * kPartialFloats + ch) = make_float2(acc[mb][1], acc[mb][3]);
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
