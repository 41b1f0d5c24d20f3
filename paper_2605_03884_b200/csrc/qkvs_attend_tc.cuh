// Decode-step attention straight from a card on the fifth-generation tensor cores (tcgen05):
// the tokens are the 128 rows of the tile, accumulators live in tensor memory, one thread per
// pipeline issues the matrix multiplies, and every other thread owns one token of the tile.
//
// Same mathematics as qkvs_attend.cuh (scale and zero folded out of both contractions):
//     q . K~_t        = sum_g  scale_tg * (sum_{c in g} q_c code_tc)  +  zero_tg * (sum_{c in g} q_c)
//     sum_t p_t V~_tc = sum_t (p_t scale_tg) code_tc  +  sum_t p_t zero_tg              (c in group g)
// so both products run over the integer codes themselves, exact in FP16.
//
// A CTA holds two independent *pipelines*.  A pipeline is four *token warps* (128 threads) and
// one *driver warp*; it works on one *item* at a time -- 512 consecutive tokens of one (layer,
// KV head), drawn from a counter -- and walks it in *tiles* of up to 128 tokens.  The order of
// tokens does not matter to attention, so the item's tokens are first grouped by bit-width, and
// every token warp of a tile takes a *slot* of up to 32 tokens of one width (16 for FP16 rows):
// the four warps of a tile may meet different widths, a warp never does, and lane i of token
// warp w owns row 32 w + i of the tile.  Per tile the token threads
//   1. turn their token's K codes into FP16 integers and store them as their row of the A
//      operand in tensor memory (64 columns: 128 channels, two per column);
//   3. expand their token's V codes into a [token][channel] FP16 matrix in shared memory (the
//      MN-major A operand of the second product);
//   4. read their row of the scores, apply the K scales and zeros, take exp2 against the head's
//      reference maximum and write their row of W[token][(group, head)] = p * V scale (FP16);
// and the driver warp, which never touches a token,
//   2. issues  S_g[128 tokens x 16] = A[:, group g] x Qg^T, one accumulator per group of 32
//      channels (four groups), eight instructions of K = 16; Q sits in shared memory, K-major;
//   5. issues  O[128 channels x (group, head)] += Vcodes^T[channels x tokens] x W, eight
//      instructions of K = 16 tokens; only the columns of a channel's own group are used;
//   -  starts the copies of the next tile's records (bulk copies for neighbouring records, 16-byte
//      asynchronous pieces for scattered ones) into the token warps' private rings of three
//      buffers, and reads, checks and sorts the tables of the next item while the token warps
//      work on the current one.
// The two sides meet only on mbarriers: "A is stored" and "W is stored" (token warps arrive, the
// driver waits; they also tell the driver which ring buffers are free again), "scores are there"
// and "outputs are accumulated" (tensor-core completion, the token threads wait), "item is
// prepared" / "item is done with".
// The reference maximum of a head is the largest logit seen when it was last refreshed; it is
// refreshed (exact maximum over the tile, accumulators and sums rescaled) whenever a logit exceeds
// it by more than 8 in the base-2 exponent -- or at all for a token whose V scales are huge --
// which bounds every weight by 2^8 * 128 in FP16 and, after the first tile, almost never happens.
// Every item leaves (o, reference maximum, sum) per query head in the scratch buffer; the merge
// kernel of qkvs_attend.cuh combines the items of a head.
// All waits are bounded; a wait that gives up raises a flag that every role checks at its next
// synchronisation point, and tensor memory is freed on every path.
#pragma once

#include "qkvs_attend.cuh"
#include "qkvs_tc.cuh"

namespace qkvs {

constexpr int kTcItemTokens = 512;
constexpr int kTcSlotTokens = 32;                   // tokens per slot; FP16 rows take half a slot
constexpr int kTcMaxSlots = 36;                     // 509 FP16 rows and one of each other width: 32 + 3, rounded up to tiles
constexpr int kTcMaxTiles = kTcMaxSlots / 4;
constexpr int kTcRawBytes = kTcSlotTokens * kAttendRecMax;  // 5120: 32 eight-bit records, or 16 FP16 rows
constexpr int kTcRing = 3;
constexpr int kTcPipes = 2;
constexpr int kTcTokenThreads = 128;                // per pipeline
constexpr int kTcThreads = kTcPipes * (kTcTokenThreads + 64);  // token warps, a driver warp and a planner warp per pipeline
constexpr uint32_t kTcTmemCols = 512, kTcPipeCols = 256;
constexpr uint32_t kTcColA = 0, kTcColS = 64, kTcColO = 128;  // inside a pipeline's 256 columns
constexpr float kTcRefreshAbove = 8.0f;             // base-2 exponent by which a logit may exceed the reference
constexpr float kTcLargeScale = 128.0f;             // V scales above this refresh the reference at any excess
static_assert(kAttendRecMax * kTcSlotTokens >= 16 * 2 * kAttendD, "a slot of FP16 rows fits the buffer");

struct TcItem {
    uint32_t item;       // index of the item, or n_items when there is none
    uint32_t n_slots;
    uint64_t base_k, base_v;          // byte offsets inside the card of the item's first record in the two streams
    uint32_t slots[kTcMaxSlots];      // per slot: first list position | tokens << 10 | class << 16 | neighbours << 18 |
                                      // (where the slot's records start in the tile's buffer, in 16-byte units) << 20
    uint32_t tiles[kTcMaxTiles];      // per tile: the whole tile is one run of neighbours | (bytes of its records >> 4) << 1 |
                                      // (list value of its first record) << 12
    uint16_t list[kTcItemTokens];     // the item's tokens grouped by bit-width: record offsets from the item's first, in 16-byte units
    float qsum[4][8];                 // sums of the item's queries over a group of channels, per head
    alignas(128) uint8_t qb[16 * kAttendD * 2];  // the item's queries, [head][channel], K-major core matrices
};

struct TcPipeSmem {
    alignas(128) uint8_t raw[kTcRing][4 * kTcRawBytes]; // records of a tile: its slots one after another, each packed in list order
    alignas(128) uint8_t a2[128 * kAttendD * 2];        // V codes as FP16, [token][channel], MN-major core matrices
    alignas(128) uint8_t w[128 * 32 * 2];               // weights, [token][(group, head)], MN-major core matrices
    TcItem items[2];
    alignas(8) uint64_t full[kTcRing];                  // a ring buffer's bytes have landed
    uint64_t a_ready, w_ready;                          // the token warps have stored A / W (and a2) of a tile
    uint64_t s_full, o_done;                            // the tensor cores have finished the scores / the outputs of a tile
    uint64_t item_ready[2], item_done[2];
    float red[4][8];                                    // per-warp maxima of a refresh
    float sums[4][8 + 4 * 8];                           // per-warp sums at the end of an item: l[h], then zero-point sums [group][head]
    int abort;                                          // read by the token threads after their barrier
    int driver_abort;                                   // raised by the driver; token thread 0 carries it over
};
static_assert(kTcPipes * sizeof(TcPipeSmem) <= 232448 - 1024, "two pipelines fit the shared memory of an SM");

__device__ __forceinline__ void tokens_sync(int pipe)
{
    asm volatile("bar.sync %0, %1;" ::"r"(pipe + 1), "n"(kTcTokenThreads) : "memory");
}
__device__ __forceinline__ bool tokens_any(int pipe, bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %2, 0;\n\t"
        "bar.red.or.pred p, %1, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(pipe + 1), "r"((uint32_t)pred), "n"(kTcTokenThreads)
        : "memory");
    return r != 0;
}

__device__ __forceinline__ uint32_t tc_slot_first(uint32_t d) { return d & 1023u; }
__device__ __forceinline__ int tc_slot_count(uint32_t d) { return (int)((d >> 10) & 63u); }
__device__ __forceinline__ int tc_slot_class(uint32_t d) { return (int)((d >> 16) & 3u); }
__device__ __forceinline__ uint32_t tc_slot_raw(uint32_t d) { return (d >> 20) << 4; }

// The 32 channels of group g of one token as 16 FP16 pairs: e[4 j + k] = (channel 8 j + k,
// channel 8 j + k + 4) inside the group -- codes for a quantised row, the values themselves for a
// 16-bit row.  The same order serves the K side (pair = one tensor-memory column of the A
// operand; the queries are laid out to match) and the V side (four pairs = one 16-byte piece of
// the shared-memory operand; the output channels come out in this order and are put back at the
// end).
template <int B, int META>
__device__ __forceinline__ void expand_group(const uint8_t *rec, int g, uint32_t (&e)[16])
{
    if constexpr (B == 16) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint4 h = *reinterpret_cast<const uint4 *>(rec + 64 * g + 16 * j);
            e[4 * j + 0] = __byte_perm(h.x, h.z, 0x5410);
            e[4 * j + 1] = __byte_perm(h.x, h.z, 0x7632);
            e[4 * j + 2] = __byte_perm(h.y, h.w, 0x5410);
            e[4 * j + 3] = __byte_perm(h.y, h.w, 0x7632);
        }
    } else if constexpr (B == 4) {
        const uint4 c = *reinterpret_cast<const uint4 *>(rec + 4 * META + 16 * g);
        const uint32_t wd[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t t[4];
            nibble_pairs(wd[k], t);
#pragma unroll
            for (int m = 0; m < 4; ++m) e[4 * k + m] = t[m];
        }
    } else if constexpr (B == 8) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint4 c = *reinterpret_cast<const uint4 *>(rec + 4 * META + 32 * g + 16 * i);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                e[8 * i + k] = int_pair(__byte_perm(c.x, c.y, 0x0011u * k + 0x1100u * (4 + k)), 0x00ff00ffu);
                e[8 * i + 4 + k] = int_pair(__byte_perm(c.z, c.w, 0x0011u * k + 0x1100u * (4 + k)), 0x00ff00ffu);
            }
        }
    } else {
        const uint2 c = *reinterpret_cast<const uint2 *>(rec + 4 * META + 8 * g);
        const uint32_t wd[2] = {c.x, c.y};
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            uint32_t lo[4], hi[4];
            crumb_pairs(__byte_perm(wd[k], 0u, 0x4140), lo);  // codes 0..3 in byte 0, 4..7 in byte 2
            crumb_pairs(__byte_perm(wd[k], 0u, 0x4342), hi);  // codes 8..11 and 12..15
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                e[8 * k + m] = lo[m];
                e[8 * k + 4 + m] = hi[m];
            }
        }
    }
}

// One token's K side: scale / zero pairs into registers, codes into its row of the A operand.
template <int B, int META>
__device__ __forceinline__ void store_key_row(const uint8_t *rec, uint32_t tmem_row, float (&sc)[4], float (&ze)[4])
{
    group_params_of<B, META>(rec, true, sc, ze);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t e[16];
        expand_group<B, META>(rec, g, e);
        tmem_st16(tmem_row + 16u * g, e);
    }
}

// One token's V side: scale / zero pairs into registers, codes into its row of the shared-memory
// operand (piece j of eight channels sits 128 bytes after piece j - 1).
template <int B, int META>
__device__ __forceinline__ void store_value_row(const uint8_t *rec, uint8_t *row, float (&sc)[4], float (&ze)[4])
{
    group_params_of<B, META>(rec, true, sc, ze);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t e[16];
        expand_group<B, META>(rec, g, e);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            *reinterpret_cast<uint4 *>(row + (4 * g + j) * 128) = make_uint4(e[4 * j], e[4 * j + 1], e[4 * j + 2], e[4 * j + 3]);
    }
}

// Starts the copy of one tile's K or V records into a ring buffer: its slots one after another,
// each packed in list order.  One bulk copy when the whole tile is a run of neighbours in the
// card, else one per slot of neighbours and 16-byte asynchronous pieces for the scattered ones;
// `bar` completes when all bytes are there.  Called by all lanes of the driver warp.
template <int META>
__device__ __forceinline__ void tc_issue_tile(uint8_t *dst, uint64_t *bar, const TcItem &it, uint32_t tile, uint64_t base,
                                              const AttendParams &p, int lane)
{
    const uint32_t info = it.tiles[tile];
    if (info & 1u) {
        if (lane == 0) {
            const uint32_t bytes = ((info >> 1) & 2047u) << 4;
            mbar_arrive_expect_tx(bar, bytes);
            bulk_load(dst, p.card + base + ((uint64_t)(info >> 12) << 4), bytes, bar);
        }
        return;
    }
    uint32_t bulk_bytes = 0;
    for (uint32_t w = 0; w < 4; ++w) {
        const uint32_t slot = 4u * tile + w;
        const uint32_t d = slot < it.n_slots ? it.slots[slot] : 0u;
        const int n = tc_slot_count(d);
        if (n == 0) continue;
        const uint32_t rec = class_record_bytes<META>(tc_slot_class(d));
        uint8_t *to = dst + tc_slot_raw(d);
        if (d & (1u << 18)) {
            if (lane == 0) bulk_load(to, p.card + base + ((uint32_t)it.list[tc_slot_first(d)] << 4), (uint32_t)n * rec, bar);
            bulk_bytes += (uint32_t)n * rec;
        } else {
            const uint32_t pieces = rec >> 4, total = (uint32_t)n * pieces;  // at most 320
            const uint32_t inv = 65536u / pieces + 1u;                       // i / pieces == (i * inv) >> 16 for i < 4096
            for (uint32_t i = (uint32_t)lane; i < total; i += 32u) {
                const uint32_t r = (i * inv) >> 16;
                async_copy_16(to + (i << 4), p.card + base + (((uint32_t)it.list[tc_slot_first(d) + r] + (i - r * pieces)) << 4));
            }
        }
    }
    // the barrier's one arrival comes last: bytes that land before it cannot complete the phase
    async_copies_arrive_on(bar);
    __syncwarp();
    if (lane == 0) {
        if (bulk_bytes) mbar_arrive_expect_tx(bar, bulk_bytes);
        else mbar_arrive(bar);
    }
}

// What the kernel knows about the card after checking its header.
struct TcCard {
    Sections sec;
    int mode;
    uint64_t stream_bytes, total_bytes;
};

// Planner warp, preparing an item in two steps.  tc_fetch reads the item's table entries (16
// consecutive tokens per lane) and its queries into registers; tc_finish checks and sorts the
// entries into buffer `it`, lays out its slots and tiles, and writes the queries as the B operand
// of the score product, and their sums.  A single warp runs this dependent code at a small
// fraction of an instruction per cycle (about 9000 cycles per item as measured), which is why it
// has a warp of its own, one item ahead of the others, instead of sitting in the driver's loop.
struct TcFetch {
    static constexpr int PER = kTcItemTokens / 32;
    uint32_t item;           // n_items when there is none
    uint32_t layer, head;
    int n_tok;
    uint64_t base_k, base_v;
    uint32_t o_first;
    uint32_t offs[PER + 1];
    uint32_t bits[PER];
    uint4 q[4];
};

__device__ __forceinline__ void tc_fetch(TcFetch &f, uint32_t item, const AttendParams &p, const TcCard &cd, int lane)
{
    f.item = min(item, p.n_items);
    if (item >= p.n_items) return;
    const uint32_t H = (uint32_t)p.n_kv_heads;
    const int per_kv = p.n_q_heads / p.n_kv_heads;
    const uint64_t T = (uint64_t)p.n_tokens;
    const uint32_t lh = item / p.items_per_head, ck = item - lh * p.items_per_head;
    f.layer = lh / H;
    f.head = lh - f.layer * H;
    const uint64_t tok0 = (uint64_t)ck * kTcItemTokens;
    f.n_tok = (int)min((uint64_t)kTcItemTokens, T - tok0);
    const uint64_t seg = cd.mode == 0 ? 0u : lh;
    const uint8_t *bits_tab = p.card + cd.sec.bits_off + seg * T + tok0;
    const uint32_t *offs_tab = reinterpret_cast<const uint32_t *>(p.card + cd.sec.offs_off) + seg * (T + 1u) + tok0;
    const uint64_t stream_k = ((uint64_t)f.layer * 2u) * H + f.head, stream_v = stream_k + H;
    if (cd.mode == 0) {
        f.base_k = cd.sec.payload_off + stream_k * cd.stream_bytes;
        f.base_v = cd.sec.payload_off + stream_v * cd.stream_bytes;
    } else {
        // entries beyond the card (a damaged table) must not wrap the sums around
        const uint64_t *sbase = reinterpret_cast<const uint64_t *>(p.card + cd.sec.sbase_off);
        const uint64_t sk = __ldg(sbase + stream_k), sv = __ldg(sbase + stream_v);
        f.base_k = sk > cd.total_bytes ? ~uint64_t(0) : cd.sec.payload_off + sk;
        f.base_v = sv > cd.total_bytes ? ~uint64_t(0) : cd.sec.payload_off + sv;
    }
    f.o_first = __ldg(offs_tab);
#pragma unroll
    for (int r = 0; r <= TcFetch::PER; ++r) {
        const int j = TcFetch::PER * lane + r;
        f.offs[r] = j <= f.n_tok ? __ldg(offs_tab + j) : 0u;
    }
#pragma unroll
    for (int r = 0; r < TcFetch::PER; ++r) {
        const int j = TcFetch::PER * lane + r;
        f.bits[r] = j < f.n_tok ? (uint32_t)__ldg(bits_tab + j) : 0u;
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int h = lane / 16 + 2 * r;
        f.q[r] = make_uint4(0u, 0u, 0u, 0u);
        if (h < per_kv)
            f.q[r] = __ldg(reinterpret_cast<const uint4 *>(p.q + ((uint64_t)f.layer * p.n_q_heads + (uint64_t)f.head * per_kv + h) * kAttendD) + lane % 16);
    }
}

template <int META>
__device__ __forceinline__ void tc_finish(TcItem &it, const TcFetch &f, const AttendParams &p, const TcCard &cd, int lane)
{
    if (f.item >= p.n_items) {
        if (lane == 0) {
            it.item = p.n_items;
            it.n_slots = 0;
        }
        __syncwarp();
        return;
    }
    const uint32_t item = f.item;
    const int n_tok = f.n_tok;
    const uint64_t base_k = f.base_k, base_v = f.base_v;
    const bool base_ok = base_k >= cd.sec.payload_off && base_v >= cd.sec.payload_off && ((base_k | base_v) & 15u) == 0u &&
                         base_k <= cd.total_bytes && base_v <= cd.total_bytes;
    const uint64_t room_k = base_ok ? cd.total_bytes - base_k : 0u, room_v = base_ok ? cd.total_bytes - base_v : 0u;

    // ---- the queries: lane l writes the pieces (head l / 16 + 2 r, channels 8 (l % 16) ..), r = 0..3, in
    // the pairing of expand_group (0, 4, 1, 5, 2, 6, 3, 7 inside a piece); rows of heads not in use stay zero
    {
        const int ch = lane % 16;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int h = lane / 16 + 2 * r;
            const uint4 qv = f.q[r];
            *reinterpret_cast<uint4 *>(it.qb + ch * 256 + (h % 8) * 16) =
                make_uint4(__byte_perm(qv.x, qv.z, 0x5410), __byte_perm(qv.x, qv.z, 0x7632), __byte_perm(qv.y, qv.w, 0x5410),
                           __byte_perm(qv.y, qv.w, 0x7632));
            const float2 f0 = __half22float2(as_half2(qv.x)), f1 = __half22float2(as_half2(qv.y));
            const float2 f2 = __half22float2(as_half2(qv.z)), f3 = __half22float2(as_half2(qv.w));
            float sum = ((f0.x + f0.y) + (f1.x + f1.y)) + ((f2.x + f2.y) + (f3.x + f3.y));
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);   // the four pieces of a group sit in neighbouring lanes
            if ((ch & 3) == 0) it.qsum[ch >> 2][h] = sum;
        }
    }

    // ---- the tables: 16 consecutive tokens per lane
    constexpr int PER = TcFetch::PER;
    uint32_t my_off[PER];
    uint8_t my_cls[PER];
    uint32_t counts = 0, counts_hi = 0;  // 16-bit fields: (2 | 4 bits), (8 | 16 bits)
    bool bad = false;
    const uint32_t o_first = f.o_first;
#pragma unroll
    for (int r = 0; r < PER; ++r) {
        const int j = PER * lane + r;
        const uint32_t o = f.offs[r], o_next = f.offs[r + 1];
        my_off[r] = o;
        my_cls[r] = 4;
        if (j < n_tok) {
            const uint32_t bw = f.bits[r];
            const uint32_t rec = record_bytes(kAttendD, (int)bw, META);
            // also: inside the span an item's records can take from its first one, which is what a list entry can express
            const bool fine = base_ok && rec != 0u && o_next >= o && o_next - o == rec && (o & 15u) == 0u && o >= o_first &&
                              o_next - o_first <= (uint32_t)n_tok * 2u * kAttendD && (uint64_t)o_next <= room_k && (uint64_t)o_next <= room_v;
            bad |= !fine;
            if (fine) {
                my_cls[r] = (uint8_t)(bw == 2u ? 0 : (bw == 4u ? 1 : (bw == 8u ? 2 : 3)));
                if (my_cls[r] < 2) counts += 1u << (16 * my_cls[r]);
                else counts_hi += 1u << (16 * (my_cls[r] - 2));
            }
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
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
    uint32_t ends[4];
    ends[0] = tot & 0xffffu;
    ends[1] = ends[0] + (tot >> 16);
    ends[2] = ends[1] + (tot_hi & 0xffffu);
    ends[3] = ends[2] + (tot_hi >> 16);
    const uint32_t before = inc - counts, before_hi = inc_hi - counts_hi;
    uint32_t pos[4] = {before & 0xffffu, ends[0] + (before >> 16), ends[1] + (before_hi & 0xffffu), ends[2] + (before_hi >> 16)};
#pragma unroll
    for (int r = 0; r < PER; ++r) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (my_cls[r] == c) it.list[pos[c]++] = (uint16_t)((my_off[r] - o_first) >> 4);
    }
    __syncwarp();
    // ---- slots: the tokens of class c occupy [begin_c, ends[c]) of the list, 32 per slot (16 for FP16 rows)
    uint32_t n_slots = 0, begin = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t cap = c == 3 ? kTcSlotTokens / 2 : kTcSlotTokens;
        const uint32_t ns = (ends[c] - begin + cap - 1) / cap;
        for (uint32_t s = (uint32_t)lane; s < ns; s += 32u) {
            const uint32_t s0 = begin + s * cap;
            const uint32_t cnt = min(cap, ends[c] - s0);
            const bool neighbours = ((uint32_t)(it.list[s0 + cnt - 1] - it.list[s0]) << 4) == (cnt - 1) * class_record_bytes<META>(c);
            it.slots[n_slots + s] = s0 | (cnt << 10) | ((uint32_t)c << 16) | (neighbours ? 1u << 18 : 0u);
        }
        n_slots += ns;
        begin = ends[c];
    }
    for (uint32_t s = n_slots + (uint32_t)lane; s < (uint32_t)kTcMaxSlots; s += 32u) it.slots[s] = 0u;
    __syncwarp();
    // ---- tiles: where each slot's records go in the tile's buffer, and whether the tile is one run
    if (lane < kTcMaxTiles) {
        uint32_t at = 0;          // bytes of the tile so far
        bool run = true;
        uint32_t follow = 0;      // list value the next slot's first record must have to continue the run
        uint32_t origin = 0;      // list value of the tile's first record
        for (uint32_t w = 0; w < 4; ++w) {
            const uint32_t slot = 4u * (uint32_t)lane + w;
            if (slot >= n_slots) break;
            const uint32_t d = it.slots[slot];
            const uint32_t bytes = (uint32_t)tc_slot_count(d) * class_record_bytes<META>(tc_slot_class(d));
            const uint32_t first = it.list[tc_slot_first(d)];
            run = run && (d & (1u << 18)) != 0u && (w == 0 || first == follow);
            if (w == 0) origin = first;
            follow = first + (bytes >> 4);
            it.slots[slot] = d | ((at >> 4) << 20);
            at += bytes;
        }
        it.tiles[lane] = (origin << 12) | ((at >> 4) << 1) | (run && at > 0u ? 1u : 0u);
    }
    if (lane == 0) {
        it.item = item;
        it.n_slots = n_slots;
        it.base_k = base_k + o_first;
        it.base_v = base_v + o_first;
    }
    fence_proxy_async();   // the queries are read by the tensor cores
    __syncwarp();
}

template <int PK, int META>
__global__ void __launch_bounds__(kTcThreads, 1) attend_tc_kernel(AttendParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ int s_header_ok;
    __shared__ uint32_t s_bits_mode, s_tmem_base;
    __shared__ uint64_t s_stream_bytes, s_total_bytes;
    const int tid = threadIdx.x;
    const int cta_warp = tid >> 5, lane = tid & 31;
    // warps 0..3, 4..7: token warps of the two pipelines; 8, 9: their drivers; 10, 11: their planners
    const bool is_driver = cta_warp >= 4 * kTcPipes && cta_warp < 5 * kTcPipes;
    const bool is_planner = cta_warp >= 5 * kTcPipes;
    const int pipe = is_planner ? cta_warp - 5 * kTcPipes : (is_driver ? cta_warp - 4 * kTcPipes : cta_warp / 4);
    const int warp = cta_warp % 4;                              // token warp inside the pipeline = its quarter of the tensor-memory lanes
    const int ptid = 32 * warp + lane;                          // token threads: row of the tile
    TcPipeSmem &sm = reinterpret_cast<TcPipeSmem *>(smem_raw)[pipe];
    const qkvs_card_header_t *hdr = reinterpret_cast<const qkvs_card_header_t *>(p.card);

    if (tid == 0) {
        PathParams hp;  // the fields header_matches looks at
        hp.card_bytes = p.card_bytes;
        hp.n_layers = p.n_layers;
        hp.n_kv_heads = p.n_kv_heads;
        hp.head_dim = kAttendD;
        hp.n_tokens = p.n_tokens;
        hp.meta_bytes = META;
        hp.group_size = kGroup;
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
    if (is_driver && lane == 0) {
        for (int s = 0; s < kTcRing; ++s) mbar_init(&sm.full[s], 1);
        mbar_init(&sm.a_ready, 4);
        mbar_init(&sm.w_ready, 4);
        mbar_init(&sm.s_full, 1);
        mbar_init(&sm.o_done, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.item_ready[b], 1);
            mbar_init(&sm.item_done[b], 5);   // four token warps and the driver
        }
        sm.abort = 0;
        sm.driver_abort = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (!s_header_ok) {
        if (tid == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
        return;
    }
    if (cta_warp == 4 * kTcPipes) {
        tmem_alloc(&s_tmem_base, kTcTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    TcCard cd;
    cd.mode = (int)s_bits_mode;
    cd.stream_bytes = s_stream_bytes;
    cd.total_bytes = s_total_bytes;
    cd.sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, cd.mode);
    const int per_kv = p.n_q_heads / p.n_kv_heads;
    constexpr int N2 = 4 * PK;                                  // columns of the output accumulator and of W
    constexpr uint32_t kWLbo = 16u * N2;                        // bytes between blocks of 8 tokens in W
    const uint32_t tm_pipe = s_tmem_base + (uint32_t)pipe * kTcPipeCols;

    if (is_planner) {
        // =====================================================================================
        // Planner warp: draws the pipeline's items and prepares each one item ahead of its use.
        const uint32_t n_pipes = gridDim.x * kTcPipes;
        uint32_t idx = (uint32_t)(blockIdx.x * kTcPipes + pipe);   // the first item is the pipeline's own index
        bool ok = true;
        TcFetch fetch;
        for (uint32_t k = 0;; ++k) {
            const uint32_t b = k & 1u;
            tc_fetch(fetch, idx, p, cd, lane);
            uint32_t drawn = 0;
            if (idx < p.n_items && lane == 0) drawn = atomicAdd(p.work_counter, 1u);
            // buffer b held item k - 2: the token warps and the driver must be done with it
            if (k >= 2) ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.item_done[b], ((k - 2u) >> 1) & 1u));
            if (!ok) break;
            tc_finish<META>(sm.items[b], fetch, p, cd, lane);
            if (lane == 0) mbar_arrive(&sm.item_ready[b]);
            if (idx >= p.n_items) break;
            drawn = __shfl_sync(0xffffffffu, drawn, 0);
            idx = drawn < p.n_items ? min(n_pipes + drawn, p.n_items) : p.n_items;
        }
        if (!ok) {
            sm.driver_abort = 1;
            if (lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_TIMEOUT);
        }
    } else if (is_driver) {
        // =====================================================================================
        // Driver warp: copies and matrix multiplies.  Lane 0 issues; all lanes share the gathers.
        const uint32_t idesc1 = mma_idesc_f16(128, 16, false, false);
        const uint32_t idesc2 = mma_idesc_f16(128, N2, true, true);
        uint32_t n = 0;                           // tiles of this pipeline so far (phase of the per-tile barriers)
        uint32_t k_issued = 0, v_issued = 0;      // tiles whose K / V loads are on their way
        bool ok = true;

        auto issue = [&](const TcItem &it, uint32_t tile, uint32_t kv, uint32_t flat) {
            const uint32_t ring = (2u * flat + kv) % kTcRing;   // loads are numbered K, V, K, V, ... over the pipeline's tiles
            tc_issue_tile<META>(sm.raw[ring], &sm.full[ring], it, tile, kv ? it.base_v : it.base_k, p, lane);
        };

        for (uint32_t k = 0; ok; ++k) {
            const uint32_t b = k & 1u;
            TcItem &it = sm.items[b];
            ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.item_ready[b], (k >> 1) & 1u));
            if (!ok || it.item >= p.n_items) break;
            const uint32_t nt = (it.n_slots + 3u) / 4u;
            bool next_seen = false;               // the planner has finished item k + 1
            for (uint32_t t = 0; t < nt && ok; ++t) {
                if (k_issued == n) {
                    issue(it, t, 0u, n);
                    ++k_issued;
                }
                if (v_issued == n) {
                    issue(it, t, 1u, n);
                    ++v_issued;
                }
                // the K records of the following tile go where the V records of the previous tile were
                const TcItem *nx = nullptr;
                uint32_t nx_tile = 0;
                if (t + 1 < nt) {
                    nx = &it;
                    nx_tile = t + 1;
                } else {
                    if (!next_seen) next_seen = __all_sync(0xffffffffu, mbar_try_wait_short(&sm.item_ready[b ^ 1u], ((k + 1u) >> 1) & 1u));
                    if (next_seen && sm.items[b ^ 1u].item < p.n_items && sm.items[b ^ 1u].n_slots > 0) nx = &sm.items[b ^ 1u];
                }
                if (nx && k_issued == n + 1) {
                    issue(*nx, nx_tile, 0u, n + 1);
                    ++k_issued;
                }
                // ---- scores, once the four token warps have stored their rows of A
                ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.a_ready, n & 1u));
                if (!ok) break;
                if (lane == 0) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int g = 0; g < 4; ++g)
#pragma unroll
                        for (int j = 0; j < 2; ++j)
                            mma_f16_ts(tm_pipe + kTcColS + 16u * g, tm_pipe + kTcColA + 16u * g + 8u * j,
                                       smem_matrix_desc(smem_addr(it.qb) + (uint32_t)(2 * g + j) * 512u, 256u, 128u), idesc1, j > 0);
                    tc_commit(&sm.s_full);
                }
                __syncwarp();
                // the K buffer of this tile is free: the V records of the following tile go there
                if (nx && v_issued == n + 1 && k_issued == n + 2) {
                    issue(*nx, nx_tile, 1u, n + 1);
                    ++v_issued;
                }
                // ---- outputs, once W and the V operand are stored
                ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.w_ready, n & 1u));
                if (!ok) break;
                if (lane == 0) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        mma_f16_ss(tm_pipe + kTcColO, smem_matrix_desc(smem_addr(sm.a2) + (uint32_t)j * 4096u, 2048u, 128u),
                                   smem_matrix_desc(smem_addr(sm.w) + (uint32_t)j * 2u * kWLbo, kWLbo, 128u), idesc2, t > 0 || j > 0);
                    tc_commit(&sm.o_done);
                }
                __syncwarp();
                ++n;
            }
            // the planner may put the item after the next into this buffer
            if (lane == 0) mbar_arrive(&sm.item_done[b]);
        }
        if (!ok) {
            sm.driver_abort = 1;
            if (lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_TIMEOUT);
        }
        // copies still in flight (only after a give-up) get the same bounded time to land: the last
        // three loads of every ring are the ones whose barriers still show their own phase
        {
            const int last = max(2 * (int)k_issued - 2, 2 * (int)v_issued - 1);
            for (int j = last; j > last - kTcRing && j >= 0; --j)
                mbar_wait(&sm.full[(uint32_t)j % kTcRing], ((uint32_t)j / kTcRing) & 1u);
        }
    } else {
        // =====================================================================================
        // Token warps: thread = token.
        const uint32_t tm_row = tm_pipe + ((uint32_t)(32 * warp) << 16);   // this thread's lane of tensor memory
        uint32_t n = 0;          // tiles so far
        bool ok = true;
        for (uint32_t k = 0;; ++k) {
            const uint32_t b = k & 1u;
            TcItem &it = sm.items[b];
            ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.item_ready[b], (k >> 1) & 1u));
            if (!ok || (ptid == 0 && sm.driver_abort)) sm.abort = 1;
            if (tokens_any(pipe, !ok) || sm.abort) break;
            if (it.item >= p.n_items) break;
            float mref[PK], l_run[PK], zacc[4][PK], qs[4][PK];
#pragma unroll
            for (int h = 0; h < PK; ++h) {
                mref[h] = -INFINITY;
                l_run[h] = 0.0f;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    qs[g][h] = it.qsum[g][h];
                    zacc[g][h] = 0.0f;
                }
            }
            const uint32_t nt = (it.n_slots + 3u) / 4u;
            bool left = false;
            for (uint32_t tile = 0; tile < nt; ++tile) {
                const uint32_t slot = 4u * tile + (uint32_t)warp;
                const uint32_t d = slot < it.n_slots ? it.slots[slot] : 0u;
                const int cnt = tc_slot_count(d), cls = tc_slot_class(d);
                const bool present = lane < cnt;
                float ksc[4], kze[4], vsc[4], vze[4];
                // ---- K: codes -> this token's row of the A operand in tensor memory
                {
                    const uint32_t j = 2u * n, ring = j % kTcRing;
                    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[ring], (j / kTcRing) & 1u));
                    const uint8_t *rec = sm.raw[ring] + tc_slot_raw(d) + (present ? lane : 0) * class_record_bytes<META>(cls);
                    if (ok && cnt > 0) {
                        switch (cls) {
                            case 0: store_key_row<2, META>(rec, tm_row + kTcColA, ksc, kze); break;
                            case 1: store_key_row<4, META>(rec, tm_row + kTcColA, ksc, kze); break;
                            case 2: store_key_row<8, META>(rec, tm_row + kTcColA, ksc, kze); break;
                            default: store_key_row<16, META>(rec, tm_row + kTcColA, ksc, kze); break;
                        }
                    } else {
#pragma unroll
                        for (int g = 0; g < 4; ++g) ksc[g] = kze[g] = 0.0f;
                    }
                    tmem_wait_st();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.a_ready);
                }
                // ---- V: codes -> this token's row of the [token][channel] operand in shared memory
                {
                    if (ok && n > 0) ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.o_done, (n - 1u) & 1u));  // the last product has read a2 and w
                    const uint32_t j = 2u * n + 1u, ring = j % kTcRing;
                    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[ring], (j / kTcRing) & 1u));
                    const uint8_t *rec = sm.raw[ring] + tc_slot_raw(d) + (present ? lane : 0) * class_record_bytes<META>(cls);
                    uint8_t *row = sm.a2 + (ptid >> 3) * 2048 + (ptid & 7) * 16;
                    if (ok && present) {
                        switch (cls) {
                            case 0: store_value_row<2, META>(rec, row, vsc, vze); break;
                            case 1: store_value_row<4, META>(rec, row, vsc, vze); break;
                            case 2: store_value_row<8, META>(rec, row, vsc, vze); break;
                            default: store_value_row<16, META>(rec, row, vsc, vze); break;
                        }
                    } else {
                        // no token in this row: zeros, so that whatever the row held before cannot reach the sums
#pragma unroll
                        for (int j2 = 0; j2 < 16; ++j2) *reinterpret_cast<uint4 *>(row + j2 * 128) = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                        for (int g = 0; g < 4; ++g) vsc[g] = vze[g] = 0.0f;
                    }
                }
                // ---- scores of this token: scales and zeros of its K groups
                float x[PK];
                {
                    if (ok) ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.s_full, n & 1u));
                    tc_fence_after_sync();
                    uint32_t s[4][PK];
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if constexpr (PK == 4) tmem_ld4(tm_row + kTcColS + 16u * g, s[g]);
                        else tmem_ld8(tm_row + kTcColS + 16u * g, s[g]);
                    }
                    tmem_wait_ld();
#pragma unroll
                    for (int h = 0; h < PK; ++h) {
                        float dot = 0.0f;
#pragma unroll
                        for (int g = 0; g < 4; ++g) dot = fmaf(ksc[g], __uint_as_float(s[g][h]), fmaf(kze[g], qs[g][h], dot));
                        x[h] = (present && ok) ? dot * p.scale_log2 : -INFINITY;
                    }
                }
                bool refresh = false;
                {
                    const float vs_max = fmaxf(fmaxf(vsc[0], vsc[1]), fmaxf(vsc[2], vsc[3]));
                    const float above = vs_max > kTcLargeScale ? 0.0f : kTcRefreshAbove;
#pragma unroll
                    for (int h = 0; h < PK; ++h) refresh |= x[h] > mref[h] + above;
                }
                if (!ok || (ptid == 0 && sm.driver_abort)) sm.abort = 1;
                refresh = tokens_any(pipe, refresh);
                if (sm.abort) {
                    left = true;
                    break;
                }
                if (refresh) {
                    float f[PK];
#pragma unroll
                    for (int h = 0; h < PK; ++h) {
                        float m = x[h];
#pragma unroll
                        for (int sft = 16; sft > 0; sft >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, sft));
                        if (lane == 0) sm.red[warp][h] = m;
                    }
                    tokens_sync(pipe);
#pragma unroll
                    for (int h = 0; h < PK; ++h) {
                        const float m_new = fmaxf(fmaxf(mref[h], fmaxf(sm.red[0][h], sm.red[1][h])), fmaxf(sm.red[2][h], sm.red[3][h]));
                        f[h] = m_new == -INFINITY ? 1.0f : exp2_approx(mref[h] - m_new);   // 0 at the first refresh of an item
                        mref[h] = m_new;
                        l_run[h] *= f[h];
#pragma unroll
                        for (int g = 0; g < 4; ++g) zacc[g][h] *= f[h];
                    }
                    if (tile > 0) {
                        // the output accumulators of this lane (channel), all (group, head) columns
#pragma unroll
                        for (int part = 0; part < N2 / 16; ++part) {
                            uint32_t o[16];
                            tmem_ld16(tm_row + kTcColO + 16u * part, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f[(16 * part + i) % PK]);
                            tmem_st16(tm_row + kTcColO + 16u * part, o);
                        }
                        tmem_wait_st();
                    }
                }
                // ---- weights of this token: p * V scale per (group, head), FP16, its row of W
                {
                    float pr[PK];
#pragma unroll
                    for (int h = 0; h < PK; ++h) {
                        const float m_use = mref[h] == -INFINITY ? 0.0f : mref[h];
                        pr[h] = exp2_approx(x[h] - m_use);   // 0 for a row without a token
                        l_run[h] += pr[h];
#pragma unroll
                        for (int g = 0; g < 4; ++g) zacc[g][h] = fmaf(pr[h], vze[g], zacc[g][h]);
                    }
                    uint8_t *row = sm.w + (ptid >> 3) * kWLbo + (ptid & 7) * 16;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint32_t hw[PK / 2];
#pragma unroll
                        for (int h = 0; h < PK / 2; ++h) hw[h] = as_u32(__floats2half2_rn(pr[2 * h] * vsc[g], pr[2 * h + 1] * vsc[g]));
                        // column g * PK + h: pieces of eight columns
                        if constexpr (PK == 8) {
                            *reinterpret_cast<uint4 *>(row + g * 128) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        } else {
                            *reinterpret_cast<uint2 *>(row + (g >> 1) * 128 + (g & 1) * 8) = make_uint2(hw[0], hw[1]);
                        }
                    }
                    fence_proxy_async();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.w_ready);
                }
                ++n;
            }
            if (left) break;

            // ---- what the item found, per query head: unnormalised o (zero-point part added), reference, sum
            if (nt > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait_short(&sm.o_done, (n - 1u) & 1u));
                tc_fence_after_sync();
            }
            if (!ok || (ptid == 0 && sm.driver_abort)) sm.abort = 1;
#pragma unroll
            for (int h = 0; h < PK; ++h) {
                float v = l_run[h];
#pragma unroll
                for (int sft = 16; sft > 0; sft >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sft);
                if (lane == 0) sm.sums[warp][h] = v;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float z = zacc[g][h];
#pragma unroll
                    for (int sft = 16; sft > 0; sft >>= 1) z += __shfl_xor_sync(0xffffffffu, z, sft);
                    if (lane == 0) sm.sums[warp][8 + 8 * g + h] = z;
                }
            }
            tokens_sync(pipe);
            if (sm.abort) break;
            uint32_t o[PK];
            if (nt > 0) {
                if constexpr (PK == 4) tmem_ld4(tm_row + kTcColO + (uint32_t)(warp * PK), o);
                else tmem_ld8(tm_row + kTcColO + (uint32_t)(warp * PK), o);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int h = 0; h < PK; ++h) o[h] = 0u;
            }
            // lane 32 w + i of the accumulator is position i of group w in the order of expand_group
            const int ch = 32 * warp + (lane & ~7) + ((lane & 7) >> 1) + 4 * (lane & 1);
            float *part = p.partials + (uint64_t)it.item * per_kv * kPartialFloats;
#pragma unroll
            for (int h = 0; h < PK; ++h)
                if (h < per_kv) {
                    const int i = 8 + 8 * warp + h;   // the zero-point sum of this thread's group of channels
                    part[h * kPartialFloats + ch] = __uint_as_float(o[h]) + ((sm.sums[0][i] + sm.sums[1][i]) + (sm.sums[2][i] + sm.sums[3][i]));
                }
            if (ptid < per_kv) {
                float m = -INFINITY;
#pragma unroll
                for (int h = 0; h < PK; ++h)
                    if (h == ptid) m = mref[h];
                part[ptid * kPartialFloats + kAttendD] = m;
                part[ptid * kPartialFloats + kAttendD + 1] = (sm.sums[0][ptid] + sm.sums[1][ptid]) + (sm.sums[2][ptid] + sm.sums[3][ptid]);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.item_done[b]);
        }
    }

    // ---- leaving: tensor memory goes back
    if (!is_driver && !is_planner && ptid == 0 && sm.abort && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_TIMEOUT);
    tc_fence_before_sync();
    __syncthreads();
    if (cta_warp == 4 * kTcPipes) tmem_dealloc(s_tmem_base, kTcTmemCols);
}

}  // namespace qkvs
