// The two streaming kernels of the path, written as persistent grids of self-contained warps.
//
// A *sub-tile* is R consecutive tokens of one stream (one (layer, K|V, head) matrix), with R
// chosen so that the sub-tile has one group of 32 channels per lane (R = 8 for head_dim 128).  On
// the FP16 side a sub-tile is R rows of 2*D bytes; on the card side it is one contiguous, 16-byte
// aligned span of records whose position and length follow from the offset table.  Every warp
// runs its own pipeline over sub-tiles -- a CTA owns a contiguous range of them and its warps
// take them in turn, so a warp stays inside one stream for many steps and its pointers advance
// by constant increments:
//   - a private ring of NS shared-memory stages, each filled by one bulk asynchronous copy (TMA)
//     that signals a private mbarrier; lane 0 re-arms a stage as soon as the warp has consumed it,
//     so NS - 1 copies per warp are in flight while it computes;
//   - the slice of the bits / offset tables a sub-tile needs is read one step ahead, one entry
//     per lane, and spread with shuffles.
// Warps never wait for one another, so many of them per SM hide the latency of each other's
// arithmetic and waits.
// create: one group of 32 channels per lane; records are written to a private shared-memory
//         buffer and lane 0 sends the contiguous span to the card with a bulk store.
// inject: records are read from the staged span, 16 output bytes per lane and pass, and FP16
//         rows are stored straight to the destination, 512 contiguous bytes per warp and pass.
// No wait is unbounded: see mbar_wait.
#pragma once

#include "qkvs_common.cuh"

namespace qkvs {

template <int D>
struct WarpCfg {
    static constexpr int WARPS = 8;                     // warps per CTA
    static constexpr int THREADS = WARPS * 32;
    static constexpr int G = D / kGroup;                // groups per token row
    static constexpr int R = 32 / G;                    // rows per sub-tile: 16, 8, 5, 4 for D = 64, 128, 192, 256
    static constexpr int GROUPS = R * G;                // lanes that own a group in create (30 for D = 192)
    static constexpr int ROW_BYTES = 2 * D;
    static constexpr int STAGE_BYTES = R * ROW_BYTES;   // 2048 (1920 for D = 192); a record never exceeds a row
    static constexpr int CPR = D / 8;                   // 16-byte chunks per row
    static constexpr int CHUNKS = R * CPR;              // chunks per sub-tile
    static constexpr int PASSES = (CHUNKS + 31) / 32;   // inject: passes of one chunk per lane
    static_assert(R >= 1 && GROUPS <= 32 && STAGE_BYTES % 16 == 0, "sub-tile shape");
};

// Position of a sub-tile: index inside its stream, kv * H + head, and layer inside the launch's
// pointer block.
struct Pos {
    uint32_t tt, r, layer;
};

__device__ __forceinline__ Pos first_pos(const PathParams &p, uint64_t sub)
{
    Pos c;
    const uint64_t s = sub / p.subs_per_stream;
    const uint32_t twoH = 2u * (uint32_t)p.n_kv_heads;
    c.tt = (uint32_t)(sub % p.subs_per_stream);
    c.r = (uint32_t)(s % twoH);
    c.layer = (uint32_t)(s / twoH);
    return c;
}

// Moves on by one warp step (WARPS sub-tiles).  Returns true when that left the stream, which
// is rare: the caller then recomputes its stream-level pointers instead of incrementing them.
template <int WARPS>
__device__ __forceinline__ bool step(Pos &c, const PathParams &p)
{
    c.tt += WARPS;
    if (c.tt < p.subs_per_stream) return false;
    const uint32_t twoH = 2u * (uint32_t)p.n_kv_heads;
    do {
        c.tt -= p.subs_per_stream;
        if (++c.r == twoH) {
            c.r = 0;
            ++c.layer;
        }
    } while (c.tt >= p.subs_per_stream);
    return true;
}

template <int R>
__device__ __forceinline__ int rows_at(const Pos &c, const PathParams &p)
{
    return c.tt + 1u == p.subs_per_stream ? (int)p.last_rows : R;
}

// Walks the caller's cache block (source of create, destination of inject): `row` points at the
// first row of the current sub-tile.
template <int R, int WARPS>
struct CacheWalk {
    Pos c;
    __half *row;

    __device__ __forceinline__ void locate(const PathParams &p, const LayerPtrs &ptrs, int64_t first_row)
    {
        const uint32_t H = (uint32_t)p.n_kv_heads;
        const bool is_v = c.r >= H;
        const uint32_t head = is_v ? c.r - H : c.r;
        row = reinterpret_cast<__half *>(is_v ? ptrs.v[c.layer] : ptrs.k[c.layer]) + (int64_t)head * p.head_stride +
              (first_row + (int64_t)c.tt * R) * p.token_stride;
    }
    __device__ __forceinline__ void next(const PathParams &p, const LayerPtrs &ptrs, int64_t first_row)
    {
        if (step<WARPS>(c, p)) locate(p, ptrs, first_row);
        else row += (int64_t)(WARPS * R) * p.token_stride;
    }
};

// Walks the card's tables: `offs` / `bits` point at the entries of the current sub-tile's first
// token, `base` is the byte offset of its stream inside the card.
template <int R, int WARPS>
struct TableWalk {
    Pos c;
    const uint32_t *offs;
    const uint8_t *bits;
    uint64_t base;

    __device__ __forceinline__ void locate(const PathParams &p, const Sections &sec, int bits_mode, uint64_t stream_bytes)
    {
        const uint64_t T = (uint64_t)p.n_tokens;
        const uint32_t H = (uint32_t)p.n_kv_heads;
        const uint32_t head = c.r >= H ? c.r - H : c.r;
        const uint64_t layer = (uint64_t)p.layer_begin + c.layer;
        const uint64_t stream = layer * 2u * H + c.r;                 // (layer * 2 + kv) * H + head
        const uint64_t seg = bits_mode == 0 ? 0u : layer * H + head;  // whose bits / offsets apply
        const uint64_t t0 = (uint64_t)c.tt * R;
        bits = p.card + sec.bits_off + seg * T + t0;
        offs = reinterpret_cast<const uint32_t *>(p.card + sec.offs_off) + seg * (T + 1u) + t0;
        if (bits_mode == 0) base = sec.payload_off + stream * stream_bytes;
        else base = sec.payload_off + __ldg(reinterpret_cast<const uint64_t *>(p.card + sec.sbase_off) + stream);
    }
    __device__ __forceinline__ void next(const PathParams &p, const Sections &sec, int bits_mode, uint64_t stream_bytes)
    {
        if (step<WARPS>(c, p)) {
            locate(p, sec, bits_mode, stream_bytes);
        } else {
            offs += WARPS * R;
            bits += WARPS * R;
        }
    }
};

// The table entries of one sub-tile, one per lane: lane i holds off[t0 + i] (i <= rows) and
// bits[t0 + i] (i < rows); `base` is the stream's byte offset inside the card.
struct Tables {
    uint32_t off, bits;
    uint64_t base;
    int rows;
};

template <int R, int WARPS>
__device__ __forceinline__ void fetch_tables(Tables &t, const TableWalk<R, WARPS> &w, const PathParams &p, int lane)
{
    t.rows = rows_at<R>(w.c, p);
    t.base = w.base;
    t.off = lane <= t.rows ? __ldg(w.offs + lane) : 0u;
    t.bits = lane < t.rows ? (uint32_t)__ldg(w.bits + lane) : 0u;
}

// Sub-tiles of this warp: CTA b owns the contiguous range of sub-tiles
// [b * q + min(b, rem), ...) of length q + (b < rem); inside it warp w takes the sub-tiles
// w, w + WARPS, ...  Returns how many that is and the first one's global index.
template <int WARPS>
__device__ __forceinline__ uint32_t my_share(const PathParams &p, int warp, uint64_t &first)
{
    const uint32_t b = blockIdx.x;
    const uint32_t len = p.subs_per_cta + (b < p.subs_rem ? 1u : 0u);
    first = (uint64_t)b * p.subs_per_cta + min(b, p.subs_rem) + (uint32_t)warp;
    return (uint32_t)warp < len ? (len - (uint32_t)warp + WARPS - 1) / WARPS : 0u;
}

// ---------------------------------------------------------------------------------------------
// create: FP16 rows -> records

template <int D, int NS>
struct CreateWarpSmem {
    using C = WarpCfg<D>;
    alignas(128) uint8_t in[NS][C::STAGE_BYTES];
    alignas(128) uint8_t out[C::STAGE_BYTES];
    alignas(8) uint64_t full[NS];
};

// One group per lane: lane l owns group l % G of row l / G, i.e. the 64 input bytes at offset
// l * 64 of the stage.  The four chunks are read in an order rotated by the lane so that the
// eight lanes served together by a 128-bit shared-memory access fall into eight different
// 16-byte bank columns.  B is the warp-uniform bit-width, or 0 when rows differ (then `b`).
template <int D, int B>
__device__ __forceinline__ void encode_group(const uint8_t *stage, uint8_t *rec, int lane, int g, int b)
{
    constexpr int G = D / kGroup;
    const uint8_t *src = stage + lane * 64;
    const int rot = lane >> 1;
    uint4 v[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = *reinterpret_cast<const uint4 *>(src + (((c + rot) & 3) << 4));
    const int bb = B ? B : b;
    if (bb == 16) {
#pragma unroll
        for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4 *>(rec + g * 64 + (((c + rot) & 3) << 4)) = v[c];
        return;
    }
    float mn, mx;
    group_min_max(v, mn, mx);
    const GroupParams gp = group_params(mn, mx, bb);
    *reinterpret_cast<float2 *>(rec + g * kMetaBytesPerGroup) = make_float2(gp.scale, gp.zero);
    const uint64_t inv2 = pack_f32x2(gp.inv, gp.inv);
    uint8_t *codes = rec + G * kMetaBytesPerGroup + g * (4 * bb);  // 32 codes of b bits = 4b bytes
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t f[8];
        quantize_chunk(v[c], gp.zero, inv2, f);
        pack_store_chunk<B>(f, bb, codes + ((c + rot) & 3) * bb);
    }
}

// Arms a stage and starts the copy of a sub-tile's FP16 rows into it.
template <int D, int NS>
__device__ __forceinline__ void create_issue(CreateWarpSmem<D, NS> &sm, int stage, const __half *src, int rows,
                                             const PathParams &p, int lane)
{
    using C = WarpCfg<D>;
    if (p.token_stride == D) {
        if (lane == 0) {
            mbar_arrive_expect_tx(&sm.full[stage], (uint32_t)rows * C::ROW_BYTES);
            bulk_load(sm.in[stage], src, (uint32_t)rows * C::ROW_BYTES, &sm.full[stage]);
        }
    } else {
        if (lane == 0) mbar_arrive_expect_tx(&sm.full[stage], (uint32_t)rows * C::ROW_BYTES);
        __syncwarp();
        if (lane < rows)
            bulk_load(sm.in[stage] + lane * C::ROW_BYTES, src + (int64_t)lane * p.token_stride, C::ROW_BYTES, &sm.full[stage]);
    }
}

template <int D, int NS>
__global__ void __launch_bounds__(WarpCfg<D>::THREADS, 3) create_kernel(PathParams p, LayerPtrs ptrs)
{
    using C = WarpCfg<D>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    CreateWarpSmem<D, NS> &sm = reinterpret_cast<CreateWarpSmem<D, NS> *>(smem_raw)[warp];

    qkvs_card_header_t *hdr = reinterpret_cast<qkvs_card_header_t *>(p.card);
    if (hdr->status != QKVS_OK) return;  // bad bits or short buffer: no payload is written
    const uint64_t stream_bytes = hdr->stream_bytes;
    const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, p.bits_mode);

    uint64_t first;
    const uint32_t n_mine = my_share<C::WARPS>(p, warp, first);
    if (n_mine == 0) return;

    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(&sm.full[s], 1);
        fence_mbar_init();
    }
    __syncwarp();

    CacheWalk<C::R, C::WARPS> ahead;  // runs NS sub-tiles ahead and starts the copies
    ahead.c = first_pos(p, first);
    ahead.locate(p, ptrs, 0);
    TableWalk<C::R, C::WARPS> tw;
    tw.c = ahead.c;
    tw.locate(p, sec, p.bits_mode, stream_bytes);

    uint32_t issued = 0;
    for (; issued < (uint32_t)NS && issued < n_mine; ++issued) {
        create_issue<D, NS>(sm, (int)issued, ahead.row, rows_at<C::R>(ahead.c, p), p, lane);
        if (issued + 1 < n_mine) ahead.next(p, ptrs, 0);
    }
    Tables nxt;
    fetch_tables(nxt, tw, p, lane);

    const int lrow = lane / C::G, g = lane % C::G;
    int stage = 0;
    uint32_t parity = 0, k = 0;
    bool ok = true;
    for (; k < n_mine; ++k) {
        const Tables cur = nxt;
        if (k + 1 < n_mine) {
            tw.next(p, sec, p.bits_mode, stream_bytes);
            fetch_tables(nxt, tw, p, lane);
        }

        // what this lane's row needs, spread from the lanes that hold the table entries
        const uint32_t off0 = __shfl_sync(0xffffffffu, cur.off, 0);
        const uint32_t off_end = __shfl_sync(0xffffffffu, cur.off, cur.rows);
        const uint32_t off_row = __shfl_sync(0xffffffffu, cur.off, lrow);
        const int b = (int)__shfl_sync(0xffffffffu, cur.bits, lrow);
        const int b0 = (int)__shfl_sync(0xffffffffu, cur.bits, 0);
        const bool mine = lane < C::GROUPS && lrow < cur.rows;
        const bool uniform = __all_sync(0xffffffffu, !mine || b == b0);

        ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[stage], parity));
        if (!ok) break;
        if (lane == 0) bulk_wait_read<0>();  // the previous bulk store has read the output buffer
        __syncwarp();
        if (mine) {
            uint8_t *rec = sm.out + (off_row - off0);
            const uint8_t *in = sm.in[stage];
            if (uniform) {
                switch (b0) {
                    case 4: encode_group<D, 4>(in, rec, lane, g, 4); break;
                    case 2: encode_group<D, 2>(in, rec, lane, g, 2); break;
                    case 8: encode_group<D, 8>(in, rec, lane, g, 8); break;
                    default: encode_group<D, 16>(in, rec, lane, g, 16); break;
                }
            } else {
                encode_group<D, 0>(in, rec, lane, g, b);
            }
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
            const uint32_t bytes = off_end - off0;
            if (bytes) bulk_store(p.card + cur.base + off0, sm.out, bytes);
            bulk_commit();
        }
        if (issued < n_mine) {  // the stage is consumed: re-arm it with the sub-tile NS steps ahead
            create_issue<D, NS>(sm, stage, ahead.row, rows_at<C::R>(ahead.c, p), p, lane);
            if (++issued < n_mine) ahead.next(p, ptrs, 0);
        }
        if (++stage == NS) {
            stage = 0;
            parity ^= 1u;
        }
    }
    if (!ok) {
        // A wait was abandoned: record it, and let the copies still in flight land (bounded)
        // before the shared memory is given back.
        if (lane == 0) atomicMax(&hdr->status, (uint32_t)QKVS_ERR_TIMEOUT);
        for (uint32_t j = k + 1; j < issued; ++j) {
            if (++stage == NS) {
                stage = 0;
                parity ^= 1u;
            }
            mbar_wait(&sm.full[stage], parity);
        }
    }
    if (lane == 0) bulk_wait<0>();
}

// ---------------------------------------------------------------------------------------------
// inject: records -> FP16 rows

template <int D, int NS>
struct InjectWarpSmem {
    using C = WarpCfg<D>;
    alignas(128) uint8_t in[NS][C::STAGE_BYTES];
    alignas(8) uint2 info[NS][C::R];   // per row: {record offset inside the span, bit-width}
    alignas(8) uint64_t full[NS];
    uint32_t uniform_bits[NS];         // bit-width shared by all R rows, else 0
    int32_t rows[NS];                  // 0 when the sub-tile's table entries did not check out
};

template <int D, int B>
__device__ __forceinline__ uint4 decode_chunk(const uint8_t *rec, int b, int pos)
{
    constexpr int G = D / kGroup;
    const int bb = B ? B : b;
    if (bb == 16) return *reinterpret_cast<const uint4 *>(rec + pos * 16);
    const float2 m = *reinterpret_cast<const float2 *>(rec + (pos >> 2) * kMetaBytesPerGroup);
    const uint8_t *codes = rec + G * kMetaBytesPerGroup + pos * bb;
    uint32_t lo, hi;
    if (bb == 8) {
        const uint2 w = *reinterpret_cast<const uint2 *>(codes);
        lo = w.x;
        hi = w.y;
    } else {
        uint32_t w;
        if (bb == 4) w = *reinterpret_cast<const uint32_t *>(codes);
        else w = unpack_crumbs(*reinterpret_cast<const uint16_t *>(codes));
        unpack_nibbles(w, lo, hi);
    }
    return dequantize_chunk(lo, hi, m.x, m.y);
}

// FULL: the sub-tile has all R rows and every lane has a chunk in every pass.
template <int D, int NS, int B, bool FULL>
__device__ __forceinline__ void inject_rows(const InjectWarpSmem<D, NS> &sm, int stage, int lane, int rows, __half *dst0,
                                            int64_t token_stride)
{
    using C = WarpCfg<D>;
    const uint8_t *in = sm.in[stage];
#pragma unroll
    for (int j = 0; j < C::PASSES; ++j) {
        const int ci = j * 32 + lane;
        const int row = ci / C::CPR, pos = ci % C::CPR;
        if (FULL || (ci < C::CHUNKS && row < rows)) {
            const uint2 inf = sm.info[stage][row];
            const uint4 out = decode_chunk<D, B>(in + inf.x, (int)inf.y, pos);
            __stcs(reinterpret_cast<uint4 *>(dst0 + (int64_t)row * token_stride + pos * 8), out);
        }
    }
}

// The card is untrusted input: nothing is read beyond card_bytes and no row is written unless the
// header and the sub-tile's table entries are consistent with the destination shape.
__device__ __forceinline__ bool header_matches(const qkvs_card_header_t *h, const PathParams &p, int bits_mode,
                                               const Sections &sec)
{
    bool ok = h->magic == kMagic && h->version == kVersion && h->status == QKVS_OK;
    ok = ok && h->n_layers == p.n_layers && h->n_kv_heads == p.n_kv_heads && h->head_dim == p.head_dim;
    ok = ok && h->n_tokens == p.n_tokens && h->group_size == kGroup && h->meta_bytes_per_group == kMetaBytesPerGroup;
    ok = ok && h->bits_off == sec.bits_off && h->offs_off == sec.offs_off && h->payload_off == sec.payload_off;
    ok = ok && h->sbase_off == sec.sbase_off;
    ok = ok && h->total_bytes <= p.card_bytes && h->total_bytes >= sec.payload_off;
    if (ok && bits_mode == 0) {
        const uint64_t S = 2u * (uint64_t)p.n_layers * (uint64_t)p.n_kv_heads;
        ok = h->stream_bytes <= (uint64_t)p.n_tokens * 2u * (uint64_t)p.head_dim &&
             sec.payload_off + S * h->stream_bytes == h->total_bytes;
    }
    return ok;
}

// Checks the table entries of a sub-tile, publishes the per-row record positions for the stage
// and starts the copy of its span -- or completes the stage's barrier by hand when the entries
// are inconsistent, so that the consuming side sees a sub-tile without rows.  All lanes call it.
template <int D, int NS>
__device__ __forceinline__ void inject_issue(InjectWarpSmem<D, NS> &sm, int stage, const Tables &t, const PathParams &p,
                                             const Sections &sec, uint64_t total_bytes, int lane)
{
    using C = WarpCfg<D>;
    const int rows = t.rows;
    const uint32_t off0 = __shfl_sync(0xffffffffu, t.off, 0);
    const uint32_t off_next = __shfl_down_sync(0xffffffffu, t.off, 1);
    const uint32_t off_end = __shfl_sync(0xffffffffu, t.off, rows);
    const uint32_t b0 = __shfl_sync(0xffffffffu, t.bits, 0);
    int bad = 0;
    if (lane < rows) {
        const uint32_t rec = record_bytes(D, (int)t.bits);
        bad = (rec == 0u) || (off_next < t.off) || (off_next - t.off != rec);
        sm.info[stage][lane] = make_uint2(t.off - off0, t.bits);
    }
    const bool uniform = rows == C::R && __all_sync(0xffffffffu, lane >= rows || t.bits == b0);
    bad = __any_sync(0xffffffffu, bad);
    // with consistent records the span is rows * (at most 2*D) bytes, so it fits the stage
    const uint32_t span = off_end - off0;
    bad |= (off0 & 15u) != 0u || t.base < sec.payload_off || (t.base & 15u) != 0u || t.base + (uint64_t)off_end > total_bytes;
    if (lane == 0) {
        sm.rows[stage] = bad ? 0 : rows;
        sm.uniform_bits[stage] = uniform ? b0 : 0u;
        if (bad && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
        if (!bad && span) {
            mbar_arrive_expect_tx(&sm.full[stage], span);
            bulk_load(sm.in[stage], p.card + t.base + off0, span, &sm.full[stage]);
        } else {
            mbar_arrive(&sm.full[stage]);
        }
    }
    __syncwarp();
}

template <int D, int NS>
__global__ void __launch_bounds__(WarpCfg<D>::THREADS, 3) inject_kernel(PathParams p, LayerPtrs ptrs)
{
    using C = WarpCfg<D>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ int s_header_ok;
    __shared__ uint32_t s_bits_mode;
    __shared__ uint64_t s_stream_bytes, s_total_bytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    InjectWarpSmem<D, NS> &sm = reinterpret_cast<InjectWarpSmem<D, NS> *>(smem_raw)[warp];
    const qkvs_card_header_t *hdr = reinterpret_cast<const qkvs_card_header_t *>(p.card);

    if (threadIdx.x == 0) {
        const uint32_t mode = hdr->bits_mode;
        int ok = 0;
        if (mode <= 1u) {
            const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, (int)mode);
            ok = sec.payload_off <= p.card_bytes && header_matches(hdr, p, (int)mode, sec);
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

    uint64_t first;
    const uint32_t n_mine = my_share<C::WARPS>(p, warp, first);
    if (n_mine == 0) return;

    // The copy of a span can only start once its table entries are known, so the table reads run
    // one step ahead of the copies, which run NS steps ahead of the arithmetic.
    TableWalk<C::R, C::WARPS> tw;
    tw.c = first_pos(p, first);
    tw.locate(p, sec, mode, stream_bytes);
    CacheWalk<C::R, C::WARPS> cons;
    cons.c = tw.c;
    cons.locate(p, ptrs, p.dst_token_offset);

    Tables nxt;
    fetch_tables(nxt, tw, p, lane);
    uint32_t issued = 0;
    for (; issued < (uint32_t)NS && issued < n_mine; ++issued) {
        const Tables cur = nxt;
        if (issued + 1 < n_mine) {
            tw.next(p, sec, mode, stream_bytes);
            fetch_tables(nxt, tw, p, lane);
        }
        inject_issue<D, NS>(sm, (int)issued, cur, p, sec, total_bytes, lane);
    }

    int stage = 0;
    uint32_t parity = 0, k = 0;
    bool ok = true;
    for (; k < n_mine; ++k) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[stage], parity));
        if (!ok) break;
        const int rows = sm.rows[stage];
        const uint32_t ub = sm.uniform_bits[stage];
        __half *dst0 = cons.row;
        if (C::CHUNKS % 32 == 0 && rows == C::R) {
            switch (ub) {
                case 4: inject_rows<D, NS, 4, true>(sm, stage, lane, rows, dst0, p.token_stride); break;
                case 2: inject_rows<D, NS, 2, true>(sm, stage, lane, rows, dst0, p.token_stride); break;
                case 8: inject_rows<D, NS, 8, true>(sm, stage, lane, rows, dst0, p.token_stride); break;
                case 16: inject_rows<D, NS, 16, true>(sm, stage, lane, rows, dst0, p.token_stride); break;
                default: inject_rows<D, NS, 0, true>(sm, stage, lane, rows, dst0, p.token_stride); break;
            }
        } else {
            inject_rows<D, NS, 0, false>(sm, stage, lane, rows, dst0, p.token_stride);
        }
        __syncwarp();  // every lane has read the stage: it can be re-armed
        if (k + 1 < n_mine) cons.next(p, ptrs, p.dst_token_offset);
        if (issued < n_mine) {
            const Tables cur = nxt;
            if (issued + 1 < n_mine) {
                tw.next(p, sec, mode, stream_bytes);
                fetch_tables(nxt, tw, p, lane);
            }
            inject_issue<D, NS>(sm, stage, cur, p, sec, total_bytes, lane);
            ++issued;
        }
        if (++stage == NS) {
            stage = 0;
            parity ^= 1u;
        }
    }
    if (!ok) {
        if (lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_TIMEOUT);
        for (uint32_t j = k + 1; j < issued; ++j) {
            if (++stage == NS) {
                stage = 0;
                parity ^= 1u;
            }
            mbar_wait(&sm.full[stage], parity);
        }
    }
}

}  // namespace qkvs
