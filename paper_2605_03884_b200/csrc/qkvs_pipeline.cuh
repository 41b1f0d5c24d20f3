// The two streaming kernels of the path, written as persistent, warp-specialised pipelines.
//
// A *tile* is TB consecutive tokens of one stream (one (layer, K|V, head) matrix).  On the FP16
// side a tile is TB rows of 2*D bytes; on the card side it is one contiguous, 16-byte aligned
// span of records whose length follows from the offset table.  Each CTA loops over tiles
// (tile = blockIdx.x, blockIdx.x + gridDim.x, ...) with
//   one producer warp   reads the tile's slice of the bits / offset tables, publishes per-row
//                       record positions in shared memory and issues the bulk asynchronous
//                       copy (TMA) of the tile's input into a ring of NS shared-memory stages;
//   NW consumer warps   wait on the stage's mbarrier, transform 16 bytes per lane per pass and
//                       hand the stage back through a second mbarrier.
// create: consumer warp w owns RPW consecutive rows of the tile, one group of 32 channels per
//         lane; it writes the rows' records into its own shared-memory buffer and one lane sends
//         that contiguous span to the card with a bulk store (double buffered per warp, so no
//         CTA-wide barrier is needed).
// inject: consumers read records from the staged span, 16 output bytes per lane and pass, and
//         store FP16 rows straight to the destination, 512 contiguous bytes per warp and pass.
// No wait is unbounded: see mbar_wait.
#pragma once

#include "qkvs_common.cuh"

namespace qkvs {

template <int D>
struct PipeCfg {
    static constexpr int NW = 8;                        // consumer warps
    static constexpr int THREADS = (NW + 1) * 32;       // + one producer warp
    static constexpr int CPR = D / 8;                   // 16-byte chunks (lanes) per token row
    static constexpr int RPP = 32 / CPR;                // rows a warp covers per pass
    static constexpr int LANES = RPP * CPR;             // lanes that carry data (24 for D = 192)
    static constexpr int TB = D == 192 ? 32 : 8192 / D; // tokens per tile
    static constexpr int RPW = TB / NW;                 // rows per consumer warp
    static constexpr int PASSES = RPW / RPP;
    static constexpr int ROW_BYTES = 2 * D;
    static constexpr int TILE_BYTES = TB * ROW_BYTES;
    static constexpr int G = D / kGroup;                // groups per token row
    static constexpr int GPW = RPW * G;                 // groups per consumer warp (24 for D = 192)
    static_assert(GPW <= 32, "one group per lane");
    static_assert(RPP >= 1 && RPW % RPP == 0 && TB % NW == 0, "tile shape");
};

struct StreamInfo {
    int layer_local;   // layer index inside this launch's pointer block
    int kv, head;
    int64_t seg;       // segment whose bits / offsets the stream uses
    uint64_t base;     // byte offset of the stream inside the card
};

__device__ __forceinline__ StreamInfo locate_stream(const PathParams &p, const Sections &sec, int bits_mode,
                                                    int64_t s_local, uint64_t stream_bytes)
{
    StreamInfo si;
    const int H = p.n_kv_heads;
    si.head = (int)(s_local % H);
    si.kv = (int)((s_local / H) & 1);
    si.layer_local = (int)(s_local / (2 * H));
    const int64_t layer = p.layer_begin + si.layer_local;
    const int64_t s = (layer * 2 + si.kv) * H + si.head;
    if (bits_mode == 0) {
        si.seg = 0;
        si.base = sec.payload_off + (uint64_t)s * stream_bytes;
    } else {
        si.seg = layer * H + si.head;
        si.base = sec.payload_off + reinterpret_cast<const uint64_t *>(p.card + sec.sbase_off)[s];
    }
    return si;
}

// What the producer needs to know about one tile, gathered one loop iteration ahead so that the
// global-memory latency of the table reads overlaps the previous tile.  Lane l holds table entries
// l, l + 32, ...
template <int TB>
struct TileFetch {
    static constexpr int NOFF = TB / 32 + 1;
    static constexpr int NBITS = (TB + 31) / 32;
    int64_t t0;
    int rows;
    int layer_local, kv, head;
    uint64_t base;
    uint32_t off[NOFF];
    uint32_t bits[NBITS];
};

template <int TB>
__device__ __forceinline__ void fetch_tile(TileFetch<TB> &f, const PathParams &p, const Sections &sec, int bits_mode,
                                           uint64_t stream_bytes, int64_t tile, int lane)
{
    const int64_t T = p.n_tokens;
    const int64_t s_local = tile / p.tiles_per_stream;
    f.t0 = (tile % p.tiles_per_stream) * TB;
    f.rows = (int)min((int64_t)TB, T - f.t0);
    const StreamInfo si = locate_stream(p, sec, bits_mode, s_local, stream_bytes);
    f.layer_local = si.layer_local;
    f.kv = si.kv;
    f.head = si.head;
    f.base = si.base;
    const uint8_t *bits = p.card + sec.bits_off + (uint64_t)si.seg * (uint64_t)T + f.t0;
    const uint32_t *offs = reinterpret_cast<const uint32_t *>(p.card + sec.offs_off) +
                           (uint64_t)si.seg * (uint64_t)(T + 1) + f.t0;
#pragma unroll
    for (int i = 0; i < TileFetch<TB>::NOFF; ++i) {
        const int r = lane + 32 * i;
        f.off[i] = r <= f.rows ? offs[r] : 0u;
    }
#pragma unroll
    for (int i = 0; i < TileFetch<TB>::NBITS; ++i) {
        const int r = lane + 32 * i;
        f.bits[i] = r < f.rows ? (uint32_t)bits[r] : 0u;
    }
}

// Publishes the fetched table slice in the producer's scratch arrays (all lanes call this).
template <int TB>
__device__ __forceinline__ void spill_tables(const TileFetch<TB> &f, uint32_t *off_tmp, uint8_t *bits_tmp, int lane)
{
#pragma unroll
    for (int i = 0; i < TileFetch<TB>::NOFF; ++i) {
        const int r = lane + 32 * i;
        if (r <= f.rows) off_tmp[r] = f.off[i];
    }
#pragma unroll
    for (int i = 0; i < TileFetch<TB>::NBITS; ++i) {
        const int r = lane + 32 * i;
        if (r < f.rows) bits_tmp[r] = (uint8_t)f.bits[i];
    }
    __syncwarp();
}

// Bit-width shared by rows [r0, r1) if they are a full warp share of RPW rows, else 0.
__device__ __forceinline__ uint32_t uniform_bits_of(const uint8_t *bits_tmp, int r0, int r1, int rpw)
{
    if (r1 - r0 != rpw) return 0u;
    uint32_t ub = bits_tmp[r0];
    for (int r = r0 + 1; r < r1; ++r) ub = bits_tmp[r] == ub ? ub : 0u;
    return ub;
}

// ---------------------------------------------------------------------------------------------
// create: FP16 rows -> records

template <int D, int NS>
struct CreateSmem {
    using C = PipeCfg<D>;
    alignas(128) uint8_t in[NS][C::TILE_BYTES];
    alignas(128) uint8_t out[C::NW][2][C::RPW * C::ROW_BYTES];
    uint2 info[NS][C::TB];          // per row: {record offset inside its warp's span, bit-width}
    uint64_t span_dst[NS][C::NW];   // per consumer warp: global address of its span
    uint32_t span_bytes[NS][C::NW];
    uint32_t uniform_bits[NS][C::NW];  // bit-width shared by all rows of the warp, else 0
    int32_t rows[NS];
    uint32_t off_tmp[C::TB + 1];    // producer scratch
    uint8_t bits_tmp[C::TB];
    uint64_t full[NS];
    uint64_t empty[NS];
    int abort_flag;
};

// One group per thread: lane l of consumer warp w owns group l % G of row w * RPW + l / G, i.e.
// the 64 input bytes at offset l * 64 of the warp's share of the tile.  The four chunks are read
// in an order rotated by the lane so that the eight lanes served together by a 128-bit
// shared-memory access fall into eight different 16-byte bank columns.
// B is the warp-uniform bit-width, or 0 when rows of the warp differ (then the row's own
// bit-width is used).  FULL: the tile has all TB rows and every lane has a group.
template <int D, int NS, int B, bool FULL>
__device__ __forceinline__ void create_tile_body(const CreateSmem<D, NS> &sm, int stage, int warp, int lane,
                                                 int rows_t, uint8_t *obuf)
{
    using C = PipeCfg<D>;
    const int lrow = lane / C::G, g = lane % C::G;
    const int row = warp * C::RPW + lrow;
    if (!FULL && (lane >= C::GPW || row >= rows_t)) return;
    const uint8_t *src = sm.in[stage] + (warp * C::RPW * C::ROW_BYTES + lane * 64);
    const int rot = lane >> 1;
    uint4 v[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = *reinterpret_cast<const uint4 *>(src + (((c + rot) & 3) << 4));
    const uint2 inf = sm.info[stage][row];
    const int b = B ? B : (int)inf.y;
    uint8_t *rec = obuf + inf.x;
    if (b == 16) {
#pragma unroll
        for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4 *>(rec + g * 64 + (((c + rot) & 3) << 4)) = v[c];
        return;
    }
    float mn, mx;
    group_min_max(v, mn, mx);
    const GroupParams gp = group_params(mn, mx, b);
    *reinterpret_cast<float2 *>(rec + g * kMetaBytesPerGroup) = make_float2(gp.scale, gp.zero);
    const uint64_t inv2 = pack_f32x2(gp.inv, gp.inv);
    uint8_t *codes = rec + C::G * kMetaBytesPerGroup + g * (4 * b);  // 32 codes of b bits = 4b bytes
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t f[8];
        quantize_chunk(v[c], gp.zero, inv2, f);
        pack_store_chunk<B>(f, b, codes + ((c + rot) & 3) * b);
    }
}

template <int D, int NS, bool FULL>
__device__ __forceinline__ void create_tile_dispatch(const CreateSmem<D, NS> &sm, int stage, int warp, int lane,
                                                     int rows_t, uint8_t *obuf)
{
    switch (sm.uniform_bits[stage][warp]) {
        case 4: create_tile_body<D, NS, 4, FULL>(sm, stage, warp, lane, rows_t, obuf); break;
        case 2: create_tile_body<D, NS, 2, FULL>(sm, stage, warp, lane, rows_t, obuf); break;
        case 8: create_tile_body<D, NS, 8, FULL>(sm, stage, warp, lane, rows_t, obuf); break;
        case 16: create_tile_body<D, NS, 16, FULL>(sm, stage, warp, lane, rows_t, obuf); break;
        default: create_tile_body<D, NS, 0, FULL>(sm, stage, warp, lane, rows_t, obuf); break;
    }
}

template <int D, int NS>
__global__ void __launch_bounds__(PipeCfg<D>::THREADS) create_kernel(PathParams p, LayerPtrs ptrs, int64_t n_tiles)
{
    using C = PipeCfg<D>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    CreateSmem<D, NS> &sm = *reinterpret_cast<CreateSmem<D, NS> *>(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    qkvs_card_header_t *hdr = reinterpret_cast<qkvs_card_header_t *>(p.card);
    if (hdr->status != QKVS_OK) return;  // bad bits or short buffer: no payload is written
    const uint64_t stream_bytes = hdr->stream_bytes;
    const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, p.bits_mode);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], C::NW);
        }
        sm.abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    volatile int *abort_flag = &sm.abort_flag;

    if (warp == C::NW) {
        uint32_t k = 0;
        // ---------------- producer
        const bool contiguous = p.token_stride == D;
        TileFetch<C::TB> cur, nxt;
        if ((int64_t)blockIdx.x < n_tiles) fetch_tile(nxt, p, sec, p.bits_mode, stream_bytes, blockIdx.x, lane);
        for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++k) {
            cur = nxt;
            if (tile + gridDim.x < n_tiles) fetch_tile(nxt, p, sec, p.bits_mode, stream_bytes, tile + gridDim.x, lane);
            const int stage = k % NS;
            if (!mbar_wait(&sm.empty[stage], ((k / NS) & 1) ^ 1, abort_flag)) break;
            const int rows = cur.rows;
            spill_tables(cur, sm.off_tmp, sm.bits_tmp, lane);
            for (int r = lane; r < rows; r += 32)
                sm.info[stage][r] = make_uint2(sm.off_tmp[r] - sm.off_tmp[(r / C::RPW) * C::RPW], sm.bits_tmp[r]);
            if (lane < C::NW) {
                const int r0 = min(lane * C::RPW, rows), r1 = min(r0 + C::RPW, rows);
                sm.span_dst[stage][lane] = reinterpret_cast<uint64_t>(p.card + cur.base + sm.off_tmp[r0]);
                sm.span_bytes[stage][lane] = sm.off_tmp[r1] - sm.off_tmp[r0];
                sm.uniform_bits[stage][lane] = uniform_bits_of(sm.bits_tmp, r0, r1, C::RPW);
            }
            if (lane == 0) sm.rows[stage] = rows;
            __syncwarp();
            const __half *src = reinterpret_cast<const __half *>(cur.kv == 0 ? ptrs.k[cur.layer_local] : ptrs.v[cur.layer_local]) +
                                (int64_t)cur.head * p.head_stride + cur.t0 * p.token_stride;
            if (lane == 0) mbar_arrive_expect_tx(&sm.full[stage], (uint32_t)rows * C::ROW_BYTES);
            __syncwarp();
            if (contiguous) {
                if (lane == 0) bulk_load(sm.in[stage], src, (uint32_t)rows * C::ROW_BYTES, &sm.full[stage]);
            } else {
                for (int r = lane; r < rows; r += 32)
                    bulk_load(sm.in[stage] + r * C::ROW_BYTES, src + (int64_t)r * p.token_stride, C::ROW_BYTES, &sm.full[stage]);
            }
        }
        // After an abandoned wait, stages may still have copies in flight: let them land
        // (bounded) before the CTA gives its shared memory back.
        if (*abort_flag) {
            for (uint32_t j = 0; j < (uint32_t)NS && j < k; ++j) {
                const uint32_t kk = k - 1 - j;
                mbar_wait(&sm.full[kk % NS], (kk / NS) & 1, abort_flag);
            }
            if (lane == 0) atomicMax(&hdr->status, (uint32_t)QKVS_ERR_TIMEOUT);
        }
    } else {
        // ---------------- consumers
        uint32_t k = 0;
        for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++k) {
            const int stage = k % NS;
            if (!mbar_wait(&sm.full[stage], (k / NS) & 1, abort_flag)) break;
            const int rows_t = sm.rows[stage];
            uint8_t *obuf = sm.out[warp][k & 1];
            if (lane == 0) bulk_wait_read<1>();  // the store that last used this buffer has read it
            __syncwarp();
            if (C::GPW == 32 && rows_t == C::TB) create_tile_dispatch<D, NS, true>(sm, stage, warp, lane, rows_t, obuf);
            else create_tile_dispatch<D, NS, false>(sm, stage, warp, lane, rows_t, obuf);
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                const uint64_t dst = sm.span_dst[stage][warp];
                const uint32_t bytes = sm.span_bytes[stage][warp];
                mbar_arrive(&sm.empty[stage]);
                if (bytes) bulk_store(reinterpret_cast<void *>(dst), obuf, bytes);
                bulk_commit();
            }
        }
        if (lane == 0) bulk_wait<0>();
    }
}

// ---------------------------------------------------------------------------------------------
// inject: records -> FP16 rows

template <int D, int NS>
struct InjectSmem {
    using C = PipeCfg<D>;
    alignas(128) uint8_t in[NS][C::TILE_BYTES];
    uint2 info[NS][C::TB];          // per row: {record offset inside the tile's span, bit-width}
    uint64_t dst_row0[NS];          // global address of the tile's first destination row
    uint32_t uniform_bits[NS][C::NW];
    int32_t rows[NS];               // 0 when the tile's table entries did not check out
    uint32_t off_tmp[C::TB + 1];    // producer scratch
    uint8_t bits_tmp[C::TB];
    uint64_t full[NS];
    uint64_t empty[NS];
    int abort_flag;
    int header_ok;
    uint32_t bits_mode;
    uint64_t stream_bytes, total_bytes;
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

template <int D, int NS, int B, bool FULL>
__device__ __forceinline__ void inject_tile_body(const InjectSmem<D, NS> &sm, int stage, int warp, int lane,
                                                 int rows_t, int64_t token_stride)
{
    using C = PipeCfg<D>;
    const uint8_t *tin = sm.in[stage];
    const int sub = lane / C::CPR, pos = lane % C::CPR;
    __half *dst0 = reinterpret_cast<__half *>(sm.dst_row0[stage]);
#pragma unroll
    for (int j = 0; j < C::PASSES; ++j) {
        const int row = warp * C::RPW + j * C::RPP + sub;
        if (FULL || (lane < C::LANES && row < rows_t)) {
            const uint2 inf = sm.info[stage][row];
            const uint4 out = decode_chunk<D, B>(tin + inf.x, (int)inf.y, pos);
            __stcs(reinterpret_cast<uint4 *>(dst0 + (int64_t)row * token_stride + pos * 8), out);
        }
    }
}

template <int D, int NS, bool FULL>
__device__ __forceinline__ void inject_tile_dispatch(const InjectSmem<D, NS> &sm, int stage, int warp, int lane,
                                                     int rows_t, int64_t token_stride)
{
    switch (sm.uniform_bits[stage][warp]) {
        case 4: inject_tile_body<D, NS, 4, FULL>(sm, stage, warp, lane, rows_t, token_stride); break;
        case 2: inject_tile_body<D, NS, 2, FULL>(sm, stage, warp, lane, rows_t, token_stride); break;
        case 8: inject_tile_body<D, NS, 8, FULL>(sm, stage, warp, lane, rows_t, token_stride); break;
        case 16: inject_tile_body<D, NS, 16, FULL>(sm, stage, warp, lane, rows_t, token_stride); break;
        default: inject_tile_body<D, NS, 0, FULL>(sm, stage, warp, lane, rows_t, token_stride); break;
    }
}

// The card is untrusted input: nothing is read beyond card_bytes and no row is written unless the
// header and the tile's table entries are consistent with the destination shape.
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

template <int D, int NS>
__global__ void __launch_bounds__(PipeCfg<D>::THREADS) inject_kernel(PathParams p, LayerPtrs ptrs, int64_t n_tiles)
{
    using C = PipeCfg<D>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    InjectSmem<D, NS> &sm = *reinterpret_cast<InjectSmem<D, NS> *>(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const qkvs_card_header_t *hdr = reinterpret_cast<const qkvs_card_header_t *>(p.card);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], C::NW);
        }
        sm.abort_flag = 0;
        fence_mbar_init();
        const uint32_t mode = hdr->bits_mode;
        int ok = 0;
        if (mode <= 1u) {
            const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, (int)mode);
            ok = sec.payload_off <= p.card_bytes && header_matches(hdr, p, (int)mode, sec);
        }
        sm.header_ok = ok;
        sm.bits_mode = mode;
        sm.stream_bytes = hdr->stream_bytes;
        sm.total_bytes = hdr->total_bytes;
    }
    __syncthreads();
    if (!sm.header_ok) {
        if (threadIdx.x == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
        return;
    }
    volatile int *abort_flag = &sm.abort_flag;
    const int mode = (int)sm.bits_mode;
    const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, mode);

    if (warp == C::NW) {
        uint32_t k = 0;
        // ---------------- producer
        const uint64_t total = sm.total_bytes;
        const uint64_t stream_bytes = sm.stream_bytes;
        TileFetch<C::TB> cur, nxt;
        if ((int64_t)blockIdx.x < n_tiles) fetch_tile(nxt, p, sec, mode, stream_bytes, blockIdx.x, lane);
        for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++k) {
            cur = nxt;
            if (tile + gridDim.x < n_tiles) fetch_tile(nxt, p, sec, mode, stream_bytes, tile + gridDim.x, lane);
            const int stage = k % NS;
            if (!mbar_wait(&sm.empty[stage], ((k / NS) & 1) ^ 1, abort_flag)) break;
            const int rows = cur.rows;
            spill_tables(cur, sm.off_tmp, sm.bits_tmp, lane);
            const uint32_t off0 = sm.off_tmp[0];
            int bad = 0;
            for (int r = lane; r < rows; r += 32) {
                const uint32_t b = sm.bits_tmp[r];
                const uint32_t rec = record_bytes(D, (int)b);
                bad |= (rec == 0u) || (sm.off_tmp[r + 1] < sm.off_tmp[r]) || (sm.off_tmp[r + 1] - sm.off_tmp[r] != rec);
                sm.info[stage][r] = make_uint2(sm.off_tmp[r] - off0, b);
            }
            bad = __any_sync(0xffffffffu, bad);
            // with consistent records the span is rows * (at most 2*D) bytes, so it fits the stage
            const uint32_t span = sm.off_tmp[rows] - off0;
            bad |= (off0 & 15u) != 0u || cur.base < sec.payload_off || (cur.base & 15u) != 0u ||
                   cur.base + (uint64_t)sm.off_tmp[rows] > total;
            if (lane < C::NW) {
                const int r0 = min(lane * C::RPW, rows), r1 = min(r0 + C::RPW, rows);
                sm.uniform_bits[stage][lane] = uniform_bits_of(sm.bits_tmp, r0, r1, C::RPW);
            }
            if (lane == 0) {
                sm.rows[stage] = bad ? 0 : rows;
                __half *dst = reinterpret_cast<__half *>(cur.kv == 0 ? ptrs.k[cur.layer_local] : ptrs.v[cur.layer_local]) +
                              (int64_t)cur.head * p.head_stride + (p.dst_token_offset + cur.t0) * p.token_stride;
                sm.dst_row0[stage] = reinterpret_cast<uint64_t>(dst);
                if (bad && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_BAD_CARD);
            }
            __syncwarp();
            if (lane == 0) {
                if (!bad && span) {
                    mbar_arrive_expect_tx(&sm.full[stage], span);
                    bulk_load(sm.in[stage], p.card + cur.base + off0, span, &sm.full[stage]);
                } else {
                    mbar_arrive(&sm.full[stage]);
                }
            }
        }
        if (*abort_flag) {
            for (uint32_t j = 0; j < (uint32_t)NS && j < k; ++j) {
                const uint32_t kk = k - 1 - j;
                mbar_wait(&sm.full[kk % NS], (kk / NS) & 1, abort_flag);
            }
            if (lane == 0 && p.status_dev) atomicMax(p.status_dev, (int)QKVS_ERR_TIMEOUT);
        }
    } else {
        // ---------------- consumers
        uint32_t k = 0;
        for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++k) {
            const int stage = k % NS;
            if (!mbar_wait(&sm.full[stage], (k / NS) & 1, abort_flag)) break;
            const int rows_t = sm.rows[stage];
            if (C::LANES == 32 && rows_t == C::TB) inject_tile_dispatch<D, NS, true>(sm, stage, warp, lane, rows_t, p.token_stride);
            else inject_tile_dispatch<D, NS, false>(sm, stage, warp, lane, rows_t, p.token_stride);
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[stage]);
        }
    }
}

}  // namespace qkvs
