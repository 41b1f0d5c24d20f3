// The two streaming kernels of the path, written as persistent grids of self-contained warps.
//
// A *sub-tile* is ROWS consecutive tokens of one stream (one (layer, K|V, head) matrix); ROWS is
// chosen so that a sub-tile holds U groups of 32 channels per lane (16 tokens for head_dim 128).
// On the FP16 side a sub-tile is ROWS rows of 2*D bytes; on the card side it is one contiguous,
// 16-byte aligned span of records whose position and length follow from the offset table.  Every
// warp runs its own pipeline over sub-tiles, which it takes in chunks of eight consecutive ones
// from a shared counter (see WorkSource):
//   - a private ring of NS shared-memory stages, each filled by one bulk asynchronous copy (TMA)
//     that signals a private mbarrier; lane 0 re-arms a stage as soon as the warp has consumed it,
//     so NS - 1 copies per warp are in flight while it computes;
//   - the slice of the bits / offset tables a sub-tile needs is read one step ahead, one entry
//     per lane, and spread with shuffles.
// Warps never wait for one another, so many of them per SM hide the latency of each other's
// arithmetic and waits.
// create: one group of 32 channels per lane and pass; every lane stores its group's scale / zero
//         pair and packed codes straight into the card (neighbouring lanes complete 32-byte
//         sectors, since a record is written by consecutive lanes).
// inject: records are read from the staged span, 16 output bytes per lane and pass, and FP16
//         rows are stored straight to the destination, 512 contiguous bytes per warp and pass.
// No wait is unbounded: see mbar_wait.
#pragma once

#include "qkvs_common.cuh"

namespace qkvs {

// Launch shape, per kernel: warps per CTA and pipeline stages per warp (CTAs per SM is what the
// shared memory then allows: three).  Injection has the longer dependent chains per warp and gains
// from more warps with a shallower ring; creation is the other way round.
#ifndef QKVS_WARPS_CREATE
#define QKVS_WARPS_CREATE 6
#endif
#ifndef QKVS_WARPS_INJECT
#define QKVS_WARPS_INJECT 8
#endif
#ifndef QKVS_CTAS_PER_SM
#define QKVS_CTAS_PER_SM 3
#endif

template <int D>
struct WarpCfg {
    static constexpr int G = D / kGroup;                // groups per token row
    static constexpr int R = 32 / G;                    // rows covered by one group per lane: 16, 8, 5, 4
    static constexpr int GROUPS = R * G;                // lanes that own a group in create (30 for D = 192)
    static constexpr int U = D == 64 ? 1 : 2;           // groups per lane and sub-tile
    static constexpr int ROWS = U * R;                  // rows per sub-tile: 16, 16, 10, 8 for D = 64, 128, 192, 256
    static constexpr int ROW_BYTES = 2 * D;
    static constexpr int STAGE_BYTES = ROWS * ROW_BYTES;  // 2048 / 4096 / 3840 / 4096; a record never exceeds a row
    static constexpr int CPR = D / 8;                   // 16-byte chunks per row
    static constexpr int CHUNKS = ROWS * CPR;           // chunks per sub-tile
    static constexpr int PASSES = (CHUNKS + 31) / 32;   // inject: passes of one chunk per lane
    static_assert(R >= 1 && GROUPS <= 32 && ROWS + 1 <= 32 && STAGE_BYTES % 16 == 0, "sub-tile shape");
};

// Position of a sub-tile: index inside its stream, kv * H + head, and layer inside the launch's
// pointer block.
struct Pos {
    uint32_t tt, r, layer;
};

__device__ __forceinline__ Pos position_of(const PathParams &p, uint32_t sub)
{
    Pos c;
    const uint32_t s = sub / p.subs_per_stream;
    const uint32_t twoH = 2u * (uint32_t)p.n_kv_heads;
    c.tt = sub - s * p.subs_per_stream;
    c.r = s % twoH;
    c.layer = s / twoH;
    return c;
}

// Moves on to the next sub-tile.  Returns true when that left the stream.
__device__ __forceinline__ bool next_sub_tile(Pos &c, const PathParams &p)
{
    if (++c.tt < p.subs_per_stream) return false;
    c.tt = 0;
    if (++c.r == 2u * (uint32_t)p.n_kv_heads) {
        c.r = 0;
        ++c.layer;
    }
    return true;
}

template <int R>
__device__ __forceinline__ int rows_at(const Pos &c, const PathParams &p)
{
    return c.tt + 1u == p.subs_per_stream ? (int)p.last_rows : R;
}

// Work distribution.  The sub-tiles of a launch are handed out in chunks of p.chunk consecutive
// ones (eight; four when the launch is so small that chunks of eight would leave most warps with
// one chunk and a few with two).  Every warp of the grid starts with the chunk of its own index; further chunks come from
// a counter in device memory -- first come, first served, which evens out SMs that run at
// different speeds -- or, when the caller gave no scratch block, at a fixed stride.
// A warp walks its sequence of sub-tiles with two cursors, one ahead of the other: the leading
// one takes the chunks and leaves their indices in a small ring in shared memory, the trailing
// one reads them there.  The index n_chunks marks the end of the sequence.
constexpr uint32_t kChunk = 8;       // sub-tiles per chunk
constexpr uint32_t kChunkSmall = 4;  // ... of a launch with fewer than two chunks of eight per warp

struct WorkSource {
    uint32_t *ring;       // shared memory, 4 entries: chunk indices in the order the warp took them
    uint32_t *counter;    // device memory, zero at launch; or null
    uint32_t n_chunks, n_warps;
    uint32_t last;        // last chunk taken
};

struct Cursor {
    Pos c;
    uint32_t left;   // sub-tiles of the current chunk after the current one
    uint32_t nth;    // index of the current chunk in the warp's sequence
    bool done;       // the sequence has ended; c is meaningless
};

__device__ __forceinline__ void enter_chunk(Cursor &cu, uint32_t chunk, const PathParams &p)
{
    const uint32_t first = chunk * p.chunk;
    cu.c = position_of(p, first);
    cu.left = min(p.chunk, (uint32_t)p.n_subs - first) - 1u;
}

// Moves a cursor to the warp's next sub-tile.  Returns false when that is simply the following
// sub-tile of the same stream (pointers advance by a constant), true otherwise (new stream or new
// chunk: recompute pointers, or the end: cu.done).  All lanes call it together.
template <bool LEAD>
__device__ __forceinline__ bool advance(Cursor &cu, WorkSource &ws, const PathParams &p, int lane)
{
    if (cu.left) {
        --cu.left;
        return next_sub_tile(cu.c, p);
    }
    ++cu.nth;
    uint32_t chunk;
    if (LEAD) {
        if (ws.last >= ws.n_chunks) {
            chunk = ws.n_chunks;
        } else if (ws.counter) {
            uint32_t v = 0;
            if (lane == 0) v = atomicAdd(ws.counter, 1u);
            v = __shfl_sync(0xffffffffu, v, 0);
            chunk = v < ws.n_chunks ? min(ws.n_warps + v, ws.n_chunks) : ws.n_chunks;
        } else {
            chunk = ws.n_chunks - ws.last > ws.n_warps ? ws.last + ws.n_warps : ws.n_chunks;
        }
        ws.last = chunk;
        if (lane == 0) ws.ring[cu.nth & 3u] = chunk;
        __syncwarp();
    } else {
        chunk = ws.ring[cu.nth & 3u];
    }
    if (chunk >= ws.n_chunks) cu.done = true;
    else enter_chunk(cu, chunk, p);
    return true;
}

// Walks the caller's cache block (source of create, destination of inject): `row` points at the
// first row of the current sub-tile.
template <int R, bool LEAD>
struct CacheWalk {
    Cursor cu;
    __half *row;

    __device__ __forceinline__ void locate(const PathParams &p, const LayerPtrs &ptrs, int64_t first_row)
    {
        const Pos &c = cu.c;
        const uint32_t H = (uint32_t)p.n_kv_heads;
        const bool is_v = c.r >= H;
        const uint32_t head = is_v ? c.r - H : c.r;
        row = reinterpret_cast<__half *>(is_v ? ptrs.v[c.layer] : ptrs.k[c.layer]) + (int64_t)head * p.head_stride +
              (first_row + (int64_t)c.tt * R) * p.token_stride;
    }
    __device__ __forceinline__ void next(WorkSource &ws, const PathParams &p, const LayerPtrs &ptrs, int64_t first_row, int lane)
    {
        if (advance<LEAD>(cu, ws, p, lane)) {
            if (!cu.done) locate(p, ptrs, first_row);
        } else {
            row += (int64_t)R * p.token_stride;
        }
    }
};

// Walks the card's tables: `offs` / `bits` point at the entries of the current sub-tile's first
// token, `base` is the byte offset of its stream inside the card.
template <int R, bool LEAD>
struct TableWalk {
    Cursor cu;
    const uint32_t *offs;
    const uint8_t *bits;
    uint64_t base;

    __device__ __forceinline__ void locate(const PathParams &p, const Sections &sec, int bits_mode, uint64_t stream_bytes)
    {
        const Pos &c = cu.c;
        const uint64_t T = (uint64_t)p.n_tokens;
        const uint32_t H = (uint32_t)p.n_kv_heads;
        const uint32_t head = c.r >= H ? c.r - H : c.r;
        const uint64_t layer = (uint64_t)p.layer_begin + c.layer;
        const uint64_t stream = layer * 2u * H + c.r;                 // (layer * 2 + kv) * H + head
        const uint64_t seg = bits_mode == 0 ? 0u : layer * H + head;  // whose bits / offsets apply
        const uint64_t t0 = (uint64_t)c.tt * R;
        bits = p.card + sec.bits_off + seg * T + t0;
        offs = reinterpret_cast<const uint32_t *>(p.card + sec.offs_off) + seg * (T + 1u) + t0;
        if (bits_mode == 0) {
            base = sec.payload_off + stream * stream_bytes;
        } else {
            // a table entry beyond the buffer (a damaged card) must not wrap the sum around
            const uint64_t sb = __ldg(reinterpret_cast<const uint64_t *>(p.card + sec.sbase_off) + stream);
            base = sb > p.card_bytes ? ~uint64_t(0) : sec.payload_off + sb;
        }
    }
    __device__ __forceinline__ void next(WorkSource &ws, const PathParams &p, const Sections &sec, int bits_mode,
                                         uint64_t stream_bytes, int lane)
    {
        if (advance<LEAD>(cu, ws, p, lane)) {
            if (!cu.done) locate(p, sec, bits_mode, stream_bytes);
        } else {
            offs += R;
            bits += R;
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

template <int R, bool LEAD>
__device__ __forceinline__ void fetch_tables(Tables &t, const TableWalk<R, LEAD> &w, const PathParams &p, int lane)
{
    t.rows = rows_at<R>(w.cu.c, p);
    t.base = w.base;
    t.off = lane <= t.rows ? __ldg(w.offs + lane) : 0u;
    t.bits = lane < t.rows ? (uint32_t)__ldg(w.bits + lane) : 0u;
}

// Sets up the warp's work source and the starting state of its two cursors.  Returns false when
// there is no chunk for this warp.
template <int WARPS>
__device__ __forceinline__ bool start_work(WorkSource &ws, Cursor &cu, uint32_t *ring, const PathParams &p, int warp, int lane)
{
    const uint32_t me = blockIdx.x * WARPS + (uint32_t)warp;
    ws.ring = ring;
    ws.counter = p.work_counter;
    ws.n_chunks = p.n_chunks;
    ws.n_warps = gridDim.x * WARPS;
    ws.last = me;
    if (me >= p.n_chunks) return false;
    if (lane == 0) ring[0] = me;
    __syncwarp();
    cu.nth = 0;
    cu.done = false;
    enter_chunk(cu, me, p);
    return true;
}

// ---------------------------------------------------------------------------------------------
// create: FP16 rows -> records

template <int D, int NS>
struct CreateWarpSmem {
    using C = WarpCfg<D>;
    alignas(128) uint8_t in[NS][C::STAGE_BYTES];
    alignas(8) uint64_t full[NS];
    uint32_t ring[4];
    static_assert(NS >= 2 && NS <= (int)kChunkSmall, "pipeline depth");
};

// One group: lane l owns group l % G of row l / G of the R rows at `rows_in`, i.e. the 64 input
// bytes at offset l * 64.  The four chunks are read in an order rotated by the lane so that the
// eight lanes served together by a 128-bit shared-memory access fall into eight different
// 16-byte bank columns; the packed codes are put back in channel order before they are stored.
// `rec` is the row's record in the card.  B is the warp-uniform bit-width, or 0 when rows
// differ (then `b`); META the bytes of {scale, zero} per group.
// GS: log2 of (channels per quantisation group / 32).  With wider groups the lanes that share a group
// (2 or 4 neighbours of one row) combine their minima and maxima and all arrive at the same scale
// and zero; `peers` names the lanes that run the quantiser (the shuffle's mask).
template <int D, int B, int META, int GS>
__device__ __forceinline__ void encode_group(const uint8_t *rows_in, uint8_t *rec, int lane, int g, int b, unsigned peers)
{
    constexpr int PAIRS = (int)pairs_bytes(D, META, kGroup << GS);
    const uint8_t *src = rows_in + lane * 64;
    const int rot = (lane >> 1) & 3;
    uint4 v[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = *reinterpret_cast<const uint4 *>(src + (((c + rot) & 3) << 4));
    const int bb = B ? B : b;
    if (bb == 16) {
#pragma unroll
        for (int c = 0; c < 4; ++c) __stcs(reinterpret_cast<uint4 *>(rec + g * 64 + (((c + rot) & 3) << 4)), v[c]);
        return;
    }
    float mn, mx;
    group_min_max(v, mn, mx);
#pragma unroll
    for (int s = 1; s < (1 << GS); s <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(peers, mn, s));
        mx = fmaxf(mx, __shfl_xor_sync(peers, mx, s));
    }
    const GroupParams gp = group_params<META>(mn, mx, bb);
    if ((g & ((1 << GS) - 1)) == 0) {  // one lane per group stores the pair
        if (META == kMetaFp16)  // both are FP16 values: the conversion is exact
            __stcs(reinterpret_cast<uint32_t *>(rec + (g >> GS) * META), as_u32(__floats2half2_rn(gp.scale, gp.zero)));
        else
            __stcs(reinterpret_cast<float2 *>(rec + (g >> GS) * META), make_float2(gp.scale, gp.zero));
    }
    if (GS > 0 && g == 0) {  // the zero bytes between the pairs and the codes
        constexpr int USED = (D >> (5 + GS)) * META;
#pragma unroll
        for (int o = USED; o < PAIRS; o += 4) __stcs(reinterpret_cast<uint32_t *>(rec + o), 0u);
    }
    const uint64_t inv2 = pack_f32x2(gp.inv, gp.inv);
    uint32_t lo[4], hi[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t f[8];
        quantize_chunk(v[c], gp.zero, inv2, f);
        pack_chunk<B>(f, bb, lo[c], hi[c]);
    }
    unrotate4(lo, rot);
    uint8_t *codes = rec + PAIRS + g * (4 * bb);  // 32 codes of b bits = 4b bytes
    if (bb == 8) {
        unrotate4(hi, rot);
        __stcs(reinterpret_cast<uint4 *>(codes), make_uint4(lo[0], hi[0], lo[1], hi[1]));
        __stcs(reinterpret_cast<uint4 *>(codes + 16), make_uint4(lo[2], hi[2], lo[3], hi[3]));
    } else if (bb == 4) {
        __stcs(reinterpret_cast<uint4 *>(codes), make_uint4(lo[0], lo[1], lo[2], lo[3]));
    } else {
        __stcs(reinterpret_cast<uint2 *>(codes), make_uint2(__byte_perm(lo[0], lo[1], 0x5410), __byte_perm(lo[2], lo[3], 0x5410)));
    }
}

// All U passes of a sub-tile.  Every lane of the warp calls this (it shuffles).
template <int D, int B, int META, int GS>
__device__ __forceinline__ void encode_rows(const uint8_t *in, uint8_t *stream, const Tables &t, int lane)
{
    using C = WarpCfg<D>;
    const int lrow = lane / C::G, g = lane % C::G;
#pragma unroll
    for (int u = 0; u < C::U; ++u) {
        const int row = u * C::R + lrow;
        const uint32_t off_row = __shfl_sync(0xffffffffu, t.off, row);
        const int b = B ? B : (int)__shfl_sync(0xffffffffu, t.bits, row);
        const bool mine = lane < C::GROUPS && row < t.rows;
        const unsigned peers = GS > 0 ? __ballot_sync(0xffffffffu, mine && b != 16) : 0u;
        if (mine) encode_group<D, B, META, GS>(in + u * (C::R * C::ROW_BYTES), stream + off_row, lane, g, b, peers);
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

template <int D, int NS, int WARPS, int META, int GS>
__global__ void __launch_bounds__(WARPS * 32, QKVS_CTAS_PER_SM) create_kernel(PathParams p, LayerPtrs ptrs)
{
    using C = WarpCfg<D>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    CreateWarpSmem<D, NS> &sm = reinterpret_cast<CreateWarpSmem<D, NS> *>(smem_raw)[warp];

    qkvs_card_header_t *hdr = reinterpret_cast<qkvs_card_header_t *>(p.card);
    const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, p.bits_mode);
    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(&sm.full[s], 1);
        fence_mbar_init();
    }
    __syncwarp();
    WorkSource ws;
    CacheWalk<C::ROWS, true> ahead;  // runs NS sub-tiles ahead and starts the copies
    if (!start_work<WARPS>(ws, ahead.cu, sm.ring, p, warp, lane)) return;
    ahead.locate(p, ptrs, 0);
    const Cursor first = ahead.cu;

    // The first copies need nothing but kernel parameters and the caller's cache, so they start
    // before this kernel waits for the scan kernel (which may still be running: see
    // grid_dependency_wait).  They stay inside the warp's first chunk, because taking another
    // chunk needs the work counter, which the scan kernel clears.
    uint32_t issued = 0, consumed = 0;
    const uint32_t early = min((uint32_t)NS, first.left + 1u);
    for (; issued < early; ++issued) {
        if (issued) ahead.next(ws, p, ptrs, 0, lane);
        create_issue<D, NS>(sm, (int)issued, ahead.row, rows_at<C::ROWS>(ahead.cu.c, p), p, lane);
    }
    grid_dependency_wait();
    if (hdr->status != QKVS_OK) {
        // bad bits or short buffer: no payload is written; let the copies land before leaving
        for (uint32_t j = 0; j < issued; ++j) mbar_wait(&sm.full[j], 0);
        return;
    }
    const uint64_t stream_bytes = hdr->stream_bytes;
    TableWalk<C::ROWS, false> tw;    // runs one sub-tile ahead and reads the tables
    tw.cu = first;
    tw.locate(p, sec, p.bits_mode, stream_bytes);
    ahead.next(ws, p, ptrs, 0, lane);
    while (issued < (uint32_t)NS && !ahead.cu.done) {
        create_issue<D, NS>(sm, (int)issued, ahead.row, rows_at<C::ROWS>(ahead.cu.c, p), p, lane);
        ++issued;
        ahead.next(ws, p, ptrs, 0, lane);
    }
    Tables nxt;
    fetch_tables(nxt, tw, p, lane);

    int stage = 0;
    uint32_t parity = 0;
    bool ok = true;
    for (; consumed < issued; ++consumed) {
        const Tables cur = nxt;
        if (consumed + 1 < issued) {  // the next sub-tile, if there is one, is on its way already (NS >= 2)
            tw.next(ws, p, sec, p.bits_mode, stream_bytes, lane);
            fetch_tables(nxt, tw, p, lane);
        }
        const int b0 = (int)__shfl_sync(0xffffffffu, cur.bits, 0);
        const bool uniform = __all_sync(0xffffffffu, lane >= cur.rows || (int)cur.bits == b0);

        ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[stage], parity));
        if (!ok) break;
        const uint8_t *in = sm.in[stage];
        uint8_t *stream = p.card + cur.base;
        if (uniform) {
            switch (b0) {
                case 4: encode_rows<D, 4, META, GS>(in, stream, cur, lane); break;
                case 2: encode_rows<D, 2, META, GS>(in, stream, cur, lane); break;
                case 8: encode_rows<D, 8, META, GS>(in, stream, cur, lane); break;
                default: encode_rows<D, 16, META, GS>(in, stream, cur, lane); break;
            }
        } else {
            encode_rows<D, 0, META, GS>(in, stream, cur, lane);
        }
        __syncwarp();  // every lane has read the stage: it can be re-armed
        if (!ahead.cu.done) {
            create_issue<D, NS>(sm, stage, ahead.row, rows_at<C::ROWS>(ahead.cu.c, p), p, lane);
            ++issued;
            ahead.next(ws, p, ptrs, 0, lane);
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
        for (uint32_t j = consumed + 1; j < issued; ++j) {
            if (++stage == NS) {
                stage = 0;
                parity ^= 1u;
            }
            mbar_wait(&sm.full[stage], parity);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// inject: records -> FP16 rows

template <int D, int NS>
struct InjectWarpSmem {
    using C = WarpCfg<D>;
    alignas(128) uint8_t in[NS][C::STAGE_BYTES];
    uint32_t info[NS][C::ROWS];        // per row: record offset inside the span << 8 | bit-width
    alignas(8) uint64_t full[NS];
    uint32_t uniform_bits[NS];         // bit-width shared by all ROWS rows, else 0
    int32_t rows[NS];                  // 0 when the sub-tile's table entries did not check out
    uint32_t ring[4];
    static_assert(NS >= 2 && NS < (int)kChunkSmall, "pipeline depth");
};

// One chunk (8 values) of a record.  B is the bit-width known at compile time, or 0 when it is
// only known per lane (`b`): then the widths 2, 4 and 8 share one instruction stream -- the codes
// are fetched as the aligned 8 bytes around them and shifted into place, and the unpacking steps
// are applied by selection -- so that lanes of different widths do not serialise; only FP16 rows
// branch off.  META: bytes of {scale, zero} per group (the code bytes start 16-byte aligned either
// way, see qkvs_card_create).
template <int D, int B, int META, int GS>
__device__ __forceinline__ uint4 decode_chunk(const uint8_t *rec, int b, int pos)
{
    constexpr int PAIRS = (int)pairs_bytes(D, META, kGroup << GS);
    const int bb = B ? B : b;
    if (bb == 16) return *reinterpret_cast<const uint4 *>(rec + pos * 16);
    float2 m;
    if (META == kMetaFp16) m = __half22float2(*reinterpret_cast<const __half2 *>(rec + (pos >> (2 + GS)) * META));
    else m = *reinterpret_cast<const float2 *>(rec + (pos >> (2 + GS)) * META);
    const uint8_t *codes = rec + PAIRS + pos * bb;
    uint32_t lo, hi;
    if (B == 8) {
        const uint2 w = *reinterpret_cast<const uint2 *>(codes);
        lo = w.x;
        hi = w.y;
    } else if (B == 4) {
        unpack_nibbles(*reinterpret_cast<const uint32_t *>(codes), lo, hi);
    } else if (B == 2) {
        unpack_nibbles(unpack_crumbs(*reinterpret_cast<const uint16_t *>(codes)), lo, hi);
    } else {
        // the codes start at a multiple of b bytes: inside one aligned 8-byte window
        const uint32_t a = smem_addr(codes);
        const uint2 w = *reinterpret_cast<const uint2 *>(codes - (a & 7u));
        const uint32_t sh = (a & 7u) * 8u;
        const uint32_t x = sh >= 32u ? w.y >> (sh - 32u) : __funnelshift_r(w.x, w.y, sh);  // first 32 bits of the codes
        const uint32_t nib = bb == 2 ? unpack_crumbs(x & 0xffffu) : x;
        uint32_t l4, h4;
        unpack_nibbles(nib, l4, h4);
        lo = bb == 8 ? w.x : l4;  // 8-bit codes are 8-byte aligned: the window is the codes
        hi = bb == 8 ? w.y : h4;
    }
    return dequantize_chunk(lo, hi, m.x, m.y);
}

// FULL: the sub-tile has all ROWS rows and every lane has a chunk in every pass.
template <int D, int NS, int B, bool FULL, int META, int GS>
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
            const uint32_t inf = sm.info[stage][row];
            const uint4 out = decode_chunk<D, B, META, GS>(in + (inf >> 8), (int)(inf & 0xffu), pos);
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
    ok = ok && h->n_tokens == p.n_tokens && h->group_size == p.group_size && h->meta_bytes_per_group == (uint32_t)p.meta_bytes;
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
        const uint32_t rec = record_bytes(D, (int)t.bits, p.meta_bytes, p.group_size);
        bad = (rec == 0u) || (off_next < t.off) || (off_next - t.off != rec);
        sm.info[stage][lane] = ((t.off - off0) << 8) | (t.bits & 0xffu);
    }
    const bool uniform = rows == C::ROWS && __all_sync(0xffffffffu, lane >= rows || t.bits == b0);
    bad = __any_sync(0xffffffffu, bad);
    // with consistent records the span is rows * (at most 2*D) bytes, so it fits the stage
    const uint32_t span = off_end - off0;
    // compared without forming base + off_end, which a crafted stream base could wrap around
    bad |= (off0 & 15u) != 0u || t.base < sec.payload_off || (t.base & 15u) != 0u || t.base > total_bytes ||
           (uint64_t)off_end > total_bytes - t.base;
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

template <int D, int NS, int WARPS, int META, int GS>
__global__ void __launch_bounds__(WARPS * 32, QKVS_CTAS_PER_SM) inject_kernel(PathParams p, LayerPtrs ptrs)
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

    // The copy of a span can only start once its table entries are known, so the table reads run
    // one step ahead of the copies, which run NS steps ahead of the arithmetic.
    WorkSource ws;
    TableWalk<C::ROWS, true> tw;
    if (!start_work<WARPS>(ws, tw.cu, sm.ring, p, warp, lane)) return;
    tw.locate(p, sec, mode, stream_bytes);
    CacheWalk<C::ROWS, false> cons;
    cons.cu = tw.cu;
    cons.locate(p, ptrs, p.dst_token_offset);

    Tables nxt;
    fetch_tables(nxt, tw, p, lane);
    bool more = true;  // nxt holds a sub-tile that has not been issued yet
    uint32_t issued = 0, consumed = 0;
    while (issued < (uint32_t)NS && more) {
        const Tables cur = nxt;
        tw.next(ws, p, sec, mode, stream_bytes, lane);
        more = !tw.cu.done;
        if (more) fetch_tables(nxt, tw, p, lane);
        inject_issue<D, NS>(sm, (int)issued, cur, p, sec, total_bytes, lane);
        ++issued;
    }

    int stage = 0;
    uint32_t parity = 0;
    bool ok = true;
    for (; consumed < issued; ++consumed) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.full[stage], parity));
        if (!ok) break;
        const int rows = sm.rows[stage];
        const uint32_t ub = sm.uniform_bits[stage];
        __half *dst0 = cons.row;
        if (C::CHUNKS % 32 == 0 && rows == C::ROWS) {
            switch (ub) {
                case 4: inject_rows<D, NS, 4, true, META, GS>(sm, stage, lane, rows, dst0, p.token_stride); break;
                case 2: inject_rows<D, NS, 2, true, META, GS>(sm, stage, lane, rows, dst0, p.token_stride); break;
                case 8: inject_rows<D, NS, 8, true, META, GS>(sm, stage, lane, rows, dst0, p.token_stride); break;
                case 16: inject_rows<D, NS, 16, true, META, GS>(sm, stage, lane, rows, dst0, p.token_stride); break;
                default: inject_rows<D, NS, 0, true, META, GS>(sm, stage, lane, rows, dst0, p.token_stride); break;
            }
        } else {
            inject_rows<D, NS, 0, false, META, GS>(sm, stage, lane, rows, dst0, p.token_stride);
        }
        __syncwarp();  // every lane has read the stage: it can be re-armed
        if (more) {
            const Tables cur = nxt;
            tw.next(ws, p, sec, mode, stream_bytes, lane);
            more = !tw.cu.done;
            if (more) fetch_tables(nxt, tw, p, lane);
            inject_issue<D, NS>(sm, stage, cur, p, sec, total_bytes, lane);
            ++issued;
        }
        if (consumed + 1 < issued) cons.next(ws, p, ptrs, p.dst_token_offset, lane);
        if (++stage == NS) {
            stage = 0;
            parity ^= 1u;
        }
    }
    if (!ok) {
        if (lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_TIMEOUT);
        for (uint32_t j = consumed + 1; j < issued; ++j) {
            if (++stage == NS) {
                stage = 0;
                parity ^= 1u;
            }
            mbar_wait(&sm.full[stage], parity);
        }
    }
}

}  // namespace qkvs
