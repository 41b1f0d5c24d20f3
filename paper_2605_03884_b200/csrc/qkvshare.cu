// CacheCard create / inject: kernels and the C entry points declared in qkvshare.h.
//
// Three kernels make up the path:
//   scan_offsets_kernel   per-segment exclusive prefix sum of record sizes over the bit-width
//                         vector; writes the card's header, bits and offset tables (this file)
//   create_kernel         fused group min/max -> scale/zero -> quantise -> bit-pack
//   inject_kernel         unpack -> dequantise -> scatter into the destination cache layout
// The last two are the persistent per-warp TMA pipelines of qkvs_pipeline.cuh.
// A stream is one (layer, K|V, head) matrix [tokens, head_dim].
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "qkvs_common.cuh"
#include "qkvs_pipeline.cuh"
#include "qkvs_attend.cuh"
#include "qkvs_attend_tc.cuh"
#include "qkvs_select.cuh"

namespace qkvs {

// ---------------------------------------------------------------------------------------------
// Offset scan

constexpr int kScanThreads = 1024;
constexpr int kScanItems = 8;

struct ScanParams {
    const uint8_t *bits;  // device, [nseg][T]
    uint8_t *card;
    uint64_t capacity;
    int32_t n_layers, n_kv_heads, head_dim, n_tokens, bits_mode;
    int32_t meta_bytes;   // 8 or 4
    int32_t group_size;   // 32, 64 or 128
    uint64_t model_id, sender_id;
    int64_t position_offset;
    uint32_t *workspace;  // the call's scratch block, cleared here for the kernels that follow; or null
};

// Exclusive scan of one value per thread over the block; returns the block total through
// `total`.  `warp_sums` is shared scratch of 32 entries.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t *warp_sums, uint32_t &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, inc, s);
        if (lane >= s) inc += n;
    }
    __syncthreads();  // warp_sums may still be read from the previous call
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < (int)(blockDim.x >> 5) ? warp_sums[lane] : 0u;
        uint32_t winc = w;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const uint32_t n = __shfl_up_sync(0xffffffffu, winc, s);
            if (lane >= s) winc += n;
        }
        warp_sums[lane] = winc - w;  // exclusive warp prefix
        if (lane == 31) warp_sums[32] = winc;
    }
    __syncthreads();
    total = warp_sums[32];
    return warp_sums[warp] + inc - v;
}

__device__ __forceinline__ void write_header_static(qkvs_card_header_t *h, const ScanParams &p, const Sections &sec)
{
    h->magic = kMagic;
    h->version = kVersion;
    h->bits_mode = (uint32_t)p.bits_mode;
    h->n_layers = p.n_layers;
    h->n_kv_heads = p.n_kv_heads;
    h->head_dim = p.head_dim;
    h->n_tokens = p.n_tokens;
    h->group_size = p.group_size;
    h->meta_bytes_per_group = (uint32_t)p.meta_bytes;
    h->model_id = p.model_id;
    h->sender_id = p.sender_id;
    h->position_offset = p.position_offset;
    h->pad0_ = 0;
    h->bits_off = sec.bits_off;
    h->offs_off = sec.offs_off;
    h->payload_off = sec.payload_off;
    h->sbase_off = sec.sbase_off;
}

__device__ __forceinline__ void zero_fill(uint8_t *p, uint64_t begin, uint64_t end)
{
    for (uint64_t i = begin + threadIdx.x; i < end; i += blockDim.x) p[i] = 0;
}

// bits_mode 1 only: the CTA that finishes last turns the per-segment totals into the stream-base
// table, pads the tables with zeros and completes the header.  The other CTAs' results are read
// past the first-level cache.  Works for any block size that is a multiple of 32.
__device__ void finalize_card(const ScanParams &p, uint64_t *s_carry_ptr, uint64_t *s_warp)
{
    uint64_t &s_carry = *s_carry_ptr;
    const int64_t T = p.n_tokens;
    const int H = p.n_kv_heads;
    const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, p.bits_mode);
    const int64_t nseg = (int64_t)p.n_layers * H;
    const int64_t S = 2 * nseg;
    qkvs_card_header_t *h = reinterpret_cast<qkvs_card_header_t *>(p.card);
    const uint32_t *offs = reinterpret_cast<const uint32_t *>(p.card + sec.offs_off);
    uint64_t *sbase = reinterpret_cast<uint64_t *>(p.card + sec.sbase_off);
    const bool bad = __ldcg(&h->status) != QKVS_OK;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < S; base += blockDim.x) {
        const int64_t s = base + threadIdx.x;
        uint64_t v = 0;
        if (s < S && !bad) {
            const int64_t l = s / (2 * H), hh = s % H;
            v = __ldcg(offs + (l * H + hh) * (T + 1) + T);
        }
        uint64_t inc = v;
#pragma unroll
        for (int k = 1; k < 32; k <<= 1) {
            const uint64_t n = __shfl_up_sync(0xffffffffu, inc, k);
            if (lane >= k) inc += n;
        }
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const uint64_t w = lane < (int)(blockDim.x >> 5) ? s_warp[lane] : 0u;
            uint64_t winc = w;
#pragma unroll
            for (int k = 1; k < 32; k <<= 1) {
                const uint64_t n = __shfl_up_sync(0xffffffffu, winc, k);
                if (lane >= k) winc += n;
            }
            s_warp[lane] = winc - w;
            if (lane == 31) s_warp[32] = winc;
        }
        __syncthreads();
        if (s < S) sbase[s] = bad ? 0 : s_carry + s_warp[warp] + inc - v;
        __syncthreads();
        if (threadIdx.x == 0) s_carry += s_warp[32];
        __syncthreads();
    }
    zero_fill(p.card, sec.bits_off + (uint64_t)nseg * (uint64_t)T, sec.offs_off);
    zero_fill(p.card, sec.offs_off + 4u * (uint64_t)nseg * (uint64_t)(T + 1), sec.sbase_off);
    zero_fill(p.card, sec.sbase_off + 8u * (uint64_t)(S + 1), sec.payload_off);
    if (threadIdx.x == 0) {
        const uint64_t payload = s_carry;
        sbase[S] = bad ? 0 : payload;
        uint32_t status = __ldcg(&h->status);
        const uint64_t total = sec.payload_off + payload;
        if (status == QKVS_OK && total > p.capacity) status = QKVS_ERR_BUFFER_TOO_SMALL;
        const uint64_t sb = __ldcg(&h->sum_bits);
        write_header_static(h, p, sec);
        h->status = status;
        const bool ok = status == QKVS_OK;
        h->sum_bits = ok ? sb : 0;
        h->avg_code_bits = (ok && nseg * T > 0) ? __fdiv_rn((float)sb, (float)(uint64_t)(nseg * T)) : 0.0f;
        h->stream_bytes = 0;
        h->total_bytes = ok ? total : 0;
        *reinterpret_cast<uint32_t *>(h->reserved_) = 0u;   // the count of finished CTAs
    }
}

// One CTA per segment.  bits_mode 0 has a single segment, and its CTA also finishes the
// header; in bits_mode 1 the CTA that finishes last combines the per-segment results (the header,
// cleared before the launch, counts the finished CTAs in its reserved bytes meanwhile).
__global__ void __launch_bounds__(kScanThreads) scan_offsets_kernel(ScanParams p)
{
    __shared__ uint32_t warp_sums[33];
    __shared__ int s_bad;
    allow_dependents();  // the create kernel may set itself up while this one runs
    const int seg = blockIdx.x;
    const int64_t T = p.n_tokens;
    const Sections sec = card_sections(p.n_layers, p.n_kv_heads, p.n_tokens, p.bits_mode);
    const uint8_t *bits = p.bits + (int64_t)seg * T;
    uint8_t *bits_out = p.card + sec.bits_off + (uint64_t)seg * (uint64_t)T;
    uint32_t *off_out = reinterpret_cast<uint32_t *>(p.card + sec.offs_off) + (uint64_t)seg * (uint64_t)(T + 1);
    const int d = p.head_dim;

    if (threadIdx.x == 0) s_bad = 0;
    if (p.workspace && seg == 0)
        for (int i = threadIdx.x; i < QKVS_WORKSPACE_BYTES / 4; i += blockDim.x) p.workspace[i] = 0u;
    uint32_t carry = 0;
    uint64_t sum_bits = 0;
    bool bad = false;
    // A thread's eight tokens are eight bytes in, eight bytes and 32 bytes out: moved as whole words
    // where the pointers allow (a warp then writes 1 KB of offsets contiguously instead of 32
    // four-byte pieces 32 bytes apart), one by one at a ragged end or on unaligned tables.
    static_assert(kScanItems == 8, "word-wise path");
    const bool words_in = (reinterpret_cast<uintptr_t>(bits) & 7u) == 0u;
    const bool words_bits = (reinterpret_cast<uintptr_t>(bits_out) & 7u) == 0u;
    const bool words_off = (reinterpret_cast<uintptr_t>(off_out) & 15u) == 0u;
    for (int64_t tile = 0; tile < T; tile += (int64_t)blockDim.x * kScanItems) {
        const int64_t t0 = tile + (int64_t)threadIdx.x * kScanItems;
        const bool whole = t0 + kScanItems <= T;
        uint32_t rec[kScanItems];
        uint8_t bv[kScanItems];
        uint32_t mine = 0;
        uint2 packed = make_uint2(0u, 0u);
        if (whole && words_in) {
            packed = *reinterpret_cast<const uint2 *>(bits + t0);
#pragma unroll
            for (int i = 0; i < kScanItems; ++i) bv[i] = (uint8_t)((i < 4 ? packed.x : packed.y) >> (8 * (i & 3)));
        } else {
#pragma unroll
            for (int i = 0; i < kScanItems; ++i) bv[i] = t0 + i < T ? bits[t0 + i] : (uint8_t)0;
        }
#pragma unroll
        for (int i = 0; i < kScanItems; ++i) {
            rec[i] = 0;
            if (t0 + i < T) {
                rec[i] = record_bytes(d, bv[i], p.meta_bytes, p.group_size);
                bad |= rec[i] == 0u;
                sum_bits += bv[i];
                mine += rec[i];
            }
        }
        uint32_t total;
        uint32_t run = carry + block_exclusive_scan(mine, warp_sums, total);
        uint32_t off[kScanItems];
#pragma unroll
        for (int i = 0; i < kScanItems; ++i) {
            off[i] = run;
            run += rec[i];
        }
        if (whole && words_off) {
            *reinterpret_cast<uint4 *>(off_out + t0) = make_uint4(off[0], off[1], off[2], off[3]);
            *reinterpret_cast<uint4 *>(off_out + t0 + 4) = make_uint4(off[4], off[5], off[6], off[7]);
        } else {
#pragma unroll
            for (int i = 0; i < kScanItems; ++i)
                if (t0 + i < T) off_out[t0 + i] = off[i];
        }
        if (whole && words_in && words_bits) {
            *reinterpret_cast<uint2 *>(bits_out + t0) = packed;
        } else {
#pragma unroll
            for (int i = 0; i < kScanItems; ++i)
                if (t0 + i < T) bits_out[t0 + i] = bv[i];
        }
        carry += total;
    }
    if (threadIdx.x == 0) off_out[T] = carry;
    if (bad) s_bad = 1;

    // total of sum_bits over the block
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) sum_bits += __shfl_xor_sync(0xffffffffu, sum_bits, s);
    __shared__ unsigned long long s_sum;
    __syncthreads();
    if (threadIdx.x == 0) s_sum = 0;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) atomicAdd(&s_sum, (unsigned long long)sum_bits);
    __syncthreads();

    qkvs_card_header_t *h = reinterpret_cast<qkvs_card_header_t *>(p.card);
    if (p.bits_mode == 0) {
        // zero padding of the tables and the header's reserved tail
        zero_fill(p.card, sec.bits_off + (uint64_t)T, sec.offs_off);
        zero_fill(p.card, sec.offs_off + 4u * (uint64_t)(T + 1), sec.payload_off);
        zero_fill(p.card, offsetof(qkvs_card_header_t, reserved_), kHeaderBytes);
        if (threadIdx.x == 0) {
            const uint64_t S = 2u * (uint64_t)p.n_layers * (uint64_t)p.n_kv_heads;
            const uint64_t total = sec.payload_off + S * (uint64_t)carry;
            uint32_t status = QKVS_OK;
            if (s_bad) status = QKVS_ERR_BAD_BITS;
            else if (total > p.capacity) status = QKVS_ERR_BUFFER_TOO_SMALL;
            write_header_static(h, p, sec);
            h->status = status;
            const bool ok = status == QKVS_OK;
            h->sum_bits = ok ? s_sum : 0;
            h->avg_code_bits = (ok && T > 0) ? __fdiv_rn((float)s_sum, (float)(uint64_t)T) : 0.0f;
            h->stream_bytes = ok ? carry : 0;
            h->total_bytes = ok ? total : 0;
        }
    } else {
        __shared__ int s_last;
        __shared__ uint64_t s_carry;
        __shared__ uint64_t s_warp64[33];
        if (threadIdx.x == 0) {
            // header was cleared before this launch; combine across segments
            atomicAdd(reinterpret_cast<unsigned long long *>(&h->sum_bits), s_sum);
            if (s_bad) atomicMax(&h->status, (uint32_t)QKVS_ERR_BAD_BITS);
        }
        __threadfence();   // this CTA's table entries, before it counts as finished
        __syncthreads();
        if (threadIdx.x == 0) s_last = atomicAdd(reinterpret_cast<uint32_t *>(h->reserved_), 1u) + 1u == gridDim.x;
        __syncthreads();
        if (s_last) {
            __threadfence();
            finalize_card(p, &s_carry, s_warp64);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// S = alpha * I + (1 - alpha) * T, elementwise; every step one rounded binary32 operation.
__global__ void __launch_bounds__(256) combine_scores_kernel(const float *__restrict__ imp, const float *__restrict__ tra,
                                                             float alpha, float beta, int64_t n, float *out)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        out[i] = __fadd_rn(__fmul_rn(alpha, imp[i]), __fmul_rn(beta, tra[i]));
}

// ---------------------------------------------------------------------------------------------
// The controller of Section 4.1.2 as a two-layer perceptron: six features per token -> hidden
// units (rectified) -> four outputs, one per bit-width; the largest output wins, equal outputs go
// to the fewer bits.  One thread per token, the parameters in shared memory; sums start from the
// bias and take the terms in index order, every product and every sum one rounded binary32
// operation (nothing fused), so that the outputs are the same bits wherever they are computed.
constexpr int kControllerMaxHidden = 128;

__global__ void __launch_bounds__(256) controller_kernel(const float *__restrict__ features, int64_t n, int hidden,
                                                         const float *__restrict__ params, uint8_t *bits, float *outputs)
{
    __shared__ float s_params[11 * kControllerMaxHidden + 4];
    for (int i = threadIdx.x; i < 11 * hidden + 4; i += blockDim.x) s_params[i] = params[i];
    __syncthreads();
    const float *w1 = s_params, *b1 = w1 + 6 * hidden, *w2 = b1 + hidden, *b2 = w2 + 4 * hidden;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += stride) {
        float x[6];
#pragma unroll
        for (int i = 0; i < 6; ++i) x[i] = features[6 * t + i];
        float out[4] = {b2[0], b2[1], b2[2], b2[3]};
        for (int j = 0; j < hidden; ++j) {
            float acc = b1[j];
#pragma unroll
            for (int i = 0; i < 6; ++i) acc = __fadd_rn(acc, __fmul_rn(w1[6 * j + i], x[i]));
            const float h = acc > 0.0f ? acc : 0.0f;
            // the four output sums advance together: each still takes its terms in the order of j
#pragma unroll
            for (int k = 0; k < 4; ++k) out[k] = __fadd_rn(out[k], __fmul_rn(w2[hidden * k + j], h));
        }
        int best = 0;
        float best_out = out[0];
#pragma unroll
        for (int k = 1; k < 4; ++k)
            if (out[k] > best_out) {
                best = k;
                best_out = out[k];
            }
        bits[t] = (uint8_t)(2 << best);   // 2, 4, 8, 16
        if (outputs) {
#pragma unroll
            for (int k = 0; k < 4; ++k) outputs[4 * t + k] = out[k];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Self-test of the two division shortcuts against the IEEE division, over every range value the
// path can produce (binary32 values from 2^-24 to 131008) and the three qmax values.

__global__ void selftest_division_kernel(unsigned long long *mismatches)
{
    const uint32_t first = 0x33800000u;  // 2^-24
    const uint32_t last = 0x47ffe000u;   // 131008 = 2 * 65504
    unsigned long long bad_inv = 0, bad_scale = 0;
    for (uint64_t u = (uint64_t)first + blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; u <= last;
         u += (uint64_t)gridDim.x * blockDim.x) {
        const float range = __uint_as_float((uint32_t)u);
        const float qm[3] = {3.0f, 15.0f, 255.0f};
        const float rc[3] = {0x1.555556p-2f, 0x1.111112p-4f, 0x1.010102p-8f};
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            bad_inv += __float_as_uint(qmax_over_range(qm[i], range)) != __float_as_uint(__fdiv_rn(qm[i], range));
            bad_scale += __float_as_uint(divide_by_qmax(range, qm[i], rc[i])) != __float_as_uint(__fdiv_rn(range, qm[i]));
        }
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        bad_inv += __shfl_xor_sync(0xffffffffu, bad_inv, s);
        bad_scale += __shfl_xor_sync(0xffffffffu, bad_scale, s);
    }
    if ((threadIdx.x & 31) == 0) {
        if (bad_inv) atomicAdd(&mismatches[0], bad_inv);
        if (bad_scale) atomicAdd(&mismatches[1], bad_scale);
    }
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait: a warp arms a barrier with a transaction count that no copy will
// ever deliver, waits on it with the given limit, and reports the give-up exactly as the
// pipelines do.  Nothing is in flight, so the kernel simply returns afterwards.
__global__ void selftest_wait_kernel(unsigned long long limit_ns, int32_t *status, unsigned long long *waited_ns)
{
    __shared__ alignas(8) uint64_t bar;
    const int lane = threadIdx.x & 31;
    if (lane == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (lane == 0) mbar_arrive_expect_tx(&bar, 16u);  // the phase now needs 16 bytes that never come
    __syncwarp();
    const unsigned long long t0 = global_timer_ns();
    const bool ok = __all_sync(0xffffffffu, mbar_wait(&bar, 0, limit_ns));
    const unsigned long long t1 = global_timer_ns();
    if (lane == 0) {
        if (!ok) atomicMax(status, (int)QKVS_ERR_TIMEOUT);
        if (waited_ns) *waited_ns = t1 - t0;
    }
}

// ---------------------------------------------------------------------------------------------
// Host side

static qkvs_status_t check_shape(const qkvs_layout_t *l)
{
    if (!l) return QKVS_ERR_INVALID_ARG;
    if (l->n_layers < 1 || l->n_kv_heads < 1 || l->n_tokens < 0) return QKVS_ERR_INVALID_ARG;
    if (l->bits_mode != 0 && l->bits_mode != 1) return QKVS_ERR_INVALID_ARG;
    if (l->group_size != kGroup && l->group_size != 64 && l->group_size != 128) return QKVS_ERR_UNSUPPORTED_SHAPE;
    if (l->head_dim != 64 && l->head_dim != 128 && l->head_dim != 192 && l->head_dim != 256)
        return QKVS_ERR_UNSUPPORTED_SHAPE;
    // the wider groups are built for the head dimensions of 128 and 256 channels
    if (l->group_size != kGroup && l->head_dim != 128 && l->head_dim != 256) return QKVS_ERR_UNSUPPORTED_SHAPE;
    // offsets inside a stream are 32-bit
    if ((uint64_t)l->n_tokens * 2u * (uint64_t)l->head_dim > 0xffffffffull) return QKVS_ERR_UNSUPPORTED_SHAPE;
    if ((uint64_t)l->n_layers * (uint64_t)l->n_kv_heads > (1u << 24)) return QKVS_ERR_UNSUPPORTED_SHAPE;
    const int meta = meta_bytes_of(l->meta_bytes);
    if (meta == 0) return QKVS_ERR_INVALID_ARG;
    // records must stay multiples of 16 bytes: four bytes per group need groups in fours
    if (meta == kMetaFp16 && l->head_dim % 128 != 0) return QKVS_ERR_UNSUPPORTED_SHAPE;
    return QKVS_OK;
}

static qkvs_status_t check_strides(const qkvs_layout_t *l, int64_t first_row)
{
    if (l->token_stride < l->head_dim || (l->token_stride & 7) || (l->head_stride & 7) || l->head_stride < 0)
        return QKVS_ERR_INVALID_ARG;
    if (first_row < 0) return QKVS_ERR_INVALID_ARG;
    // the element offsets the kernels form (head * head_stride + row * token_stride + channel) must
    // stay far inside 64 bits whatever the caller passes
    constexpr int64_t kMaxElements = int64_t(1) << 48;
    if (first_row > kMaxElements || l->token_stride > kMaxElements || l->head_stride > kMaxElements) return QKVS_ERR_INVALID_ARG;
    long long last = 0, span = 0;
    if (__builtin_mul_overflow((long long)(first_row + l->n_tokens), (long long)l->token_stride, &last) || last > kMaxElements ||
        __builtin_mul_overflow((long long)l->n_kv_heads, (long long)l->head_stride, &span) || span > kMaxElements)
        return QKVS_ERR_INVALID_ARG;
    if (l->n_tokens > 0 && (first_row + l->n_tokens - 1) * l->token_stride + l->head_dim > l->head_stride &&
        l->n_kv_heads > 1)
        return QKVS_ERR_INVALID_ARG;
    return QKVS_OK;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Work counter of the launch with the given index inside a call's scratch block (word 0 is the
// status word); null when there is no block or the call makes more launches than it has counters.
static uint32_t *work_counter(void *workspace_dev, int launch)
{
    if (!workspace_dev || launch + 1 >= QKVS_WORKSPACE_BYTES / 4) return nullptr;
    return static_cast<uint32_t *>(workspace_dev) + 1 + launch;
}

#ifndef QKVS_STAGES_CREATE
#define QKVS_STAGES_CREATE 3
#endif
#ifndef QKVS_STAGES_INJECT
#define QKVS_STAGES_INJECT 2
#endif
constexpr int kStagesCreate = QKVS_STAGES_CREATE;
constexpr int kStagesInject = QKVS_STAGES_INJECT;

// Persistent grid: as many CTAs as fit on the device at once, never more than there is work for.
// The occupancy of a kernel on a device does not change, so it is looked up once per device;
// TAG tells the kernels apart (they all have the same function type).
template <int TAG, typename Kernel>
static cudaError_t persistent_grid(Kernel kernel, int threads, size_t smem, int64_t max_ctas, unsigned *grid)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mutex;
    static int resident[kMaxDevices] = {};  // CTAs of this kernel the whole device holds; 0 = not known yet
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    int64_t fit = 0;
    {
        std::lock_guard<std::mutex> lock(mutex);
        if (dev >= 0 && dev < kMaxDevices) fit = resident[dev];
    }
    if (fit == 0) {
        int sms = 0, per_sm = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorInvalidConfiguration;
        fit = (int64_t)sms * per_sm;
        std::lock_guard<std::mutex> lock(mutex);
        if (dev >= 0 && dev < kMaxDevices) resident[dev] = (int)fit;
    }
    *grid = (unsigned)std::min<int64_t>(max_ctas, fit);
    return cudaSuccess;
}

// Splits `streams` streams into sub-tiles and chunks and launches `kernel` on a persistent grid.
template <int D, int WARPS, int TAG, typename Kernel>
static cudaError_t launch_path(Kernel kernel, size_t smem, const PathParams &pp, const LayerPtrs &ptrs, int64_t streams,
                               cudaStream_t st, bool overlap_previous)
{
    using C = WarpCfg<D>;
    PathParams p = pp;
    p.subs_per_stream = (uint32_t)(((int64_t)p.n_tokens + C::ROWS - 1) / C::ROWS);
    const uint64_t n_subs = (uint64_t)streams * p.subs_per_stream;
    if (n_subs == 0) return cudaSuccess;
    if (n_subs > 0x7fffffffull) return cudaErrorInvalidValue;
    p.n_subs = (uint32_t)n_subs;
    p.last_rows = (uint32_t)(p.n_tokens - (int64_t)(p.subs_per_stream - 1) * C::ROWS);
    unsigned grid = 0;
    cudaError_t e = persistent_grid<TAG>(kernel, WARPS * 32, smem, (int64_t)((n_subs + kChunkSmall * WARPS - 1) / (kChunkSmall * WARPS)), &grid);
    if (e != cudaSuccess) return e;
    // with fewer than two chunks of eight per warp the second round of chunks would keep only part
    // of the grid busy for as long as the first: halve the chunks then
    p.chunk = (p.n_subs + kChunk - 1) / kChunk < 2u * grid * WARPS ? kChunkSmall : kChunk;
    p.n_chunks = (p.n_subs + p.chunk - 1) / p.chunk;
    grid = std::min<unsigned>(grid, (p.n_chunks + WARPS - 1) / WARPS);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(WARPS * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    memset(&attr, 0, sizeof(attr));
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = overlap_previous ? 1 : 0;  // the kernel calls grid_dependency_wait() before it reads the card
    return cudaLaunchKernelEx(&cfg, kernel, p, ptrs);
}

template <int D, int META, int GS = 0>
static cudaError_t launch_create(const PathParams &p, const LayerPtrs &ptrs, int64_t streams, cudaStream_t st)
{
    return launch_path<D, QKVS_WARPS_CREATE, (D * 4 + META) * 8 + 2 * GS>(create_kernel<D, kStagesCreate, QKVS_WARPS_CREATE, META, GS>,
                                                                         QKVS_WARPS_CREATE * sizeof(CreateWarpSmem<D, kStagesCreate>), p, ptrs, streams, st, true);
}

template <int D, int META, int GS = 0>
static cudaError_t launch_inject(const PathParams &p, const LayerPtrs &ptrs, int64_t streams, cudaStream_t st)
{
    return launch_path<D, QKVS_WARPS_INJECT, (D * 4 + META) * 8 + 2 * GS + 1>(inject_kernel<D, kStagesInject, QKVS_WARPS_INJECT, META, GS>,
                                                                             QKVS_WARPS_INJECT * sizeof(InjectWarpSmem<D, kStagesInject>), p, ptrs, streams, st, false);
}

// The wider-group instances: head_dim 128 or 256, either kind of pair, groups of 64 or 128.
template <int GS>
static cudaError_t launch_create_wide(const PathParams &p, const LayerPtrs &ptrs, int64_t streams, cudaStream_t st)
{
    if (p.meta_bytes == kMetaFp16)
        return p.head_dim == 128 ? launch_create<128, kMetaFp16, GS>(p, ptrs, streams, st) : launch_create<256, kMetaFp16, GS>(p, ptrs, streams, st);
    return p.head_dim == 128 ? launch_create<128, kMetaFp32, GS>(p, ptrs, streams, st) : launch_create<256, kMetaFp32, GS>(p, ptrs, streams, st);
}

template <int GS>
static cudaError_t launch_inject_wide(const PathParams &p, const LayerPtrs &ptrs, int64_t streams, cudaStream_t st)
{
    if (p.meta_bytes == kMetaFp16)
        return p.head_dim == 128 ? launch_inject<128, kMetaFp16, GS>(p, ptrs, streams, st) : launch_inject<256, kMetaFp16, GS>(p, ptrs, streams, st);
    return p.head_dim == 128 ? launch_inject<128, kMetaFp32, GS>(p, ptrs, streams, st) : launch_inject<256, kMetaFp32, GS>(p, ptrs, streams, st);
}

// The kernel instance for a checked shape: every head_dim with fp32 pairs, 128 and 256 with FP16
// pairs.
static cudaError_t launch_create_for(const PathParams &p, const LayerPtrs &ptrs, int64_t streams, cudaStream_t st)
{
    if (p.group_size == 64) return launch_create_wide<1>(p, ptrs, streams, st);
    if (p.group_size == 128) return launch_create_wide<2>(p, ptrs, streams, st);
    if (p.meta_bytes == kMetaFp16)
        return p.head_dim == 128 ? launch_create<128, kMetaFp16>(p, ptrs, streams, st)
                                 : launch_create<256, kMetaFp16>(p, ptrs, streams, st);
    switch (p.head_dim) {
        case 64: return launch_create<64, kMetaFp32>(p, ptrs, streams, st);
        case 128: return launch_create<128, kMetaFp32>(p, ptrs, streams, st);
        case 192: return launch_create<192, kMetaFp32>(p, ptrs, streams, st);
        default: return launch_create<256, kMetaFp32>(p, ptrs, streams, st);
    }
}

static cudaError_t launch_inject_for(const PathParams &p, const LayerPtrs &ptrs, int64_t streams, cudaStream_t st)
{
    if (p.group_size == 64) return launch_inject_wide<1>(p, ptrs, streams, st);
    if (p.group_size == 128) return launch_inject_wide<2>(p, ptrs, streams, st);
    if (p.meta_bytes == kMetaFp16)
        return p.head_dim == 128 ? launch_inject<128, kMetaFp16>(p, ptrs, streams, st)
                                 : launch_inject<256, kMetaFp16>(p, ptrs, streams, st);
    switch (p.head_dim) {
        case 64: return launch_inject<64, kMetaFp32>(p, ptrs, streams, st);
        case 128: return launch_inject<128, kMetaFp32>(p, ptrs, streams, st);
        case 192: return launch_inject<192, kMetaFp32>(p, ptrs, streams, st);
        default: return launch_inject<256, kMetaFp32>(p, ptrs, streams, st);
    }
}

// ---------------------------------------------------------------------------------------------
// Scratch of qkvs_card_inject_noalloc: the work counters live in the library's own device
// memory instead of a block from the caller.  One word per kernel launch of a call (a launch
// covers kMaxLayersPerLaunch layers).  Every GPU that loads the library holds these bytes until
// the process exits.

constexpr int kNoAllocCounters = 64;
static_assert(kNoAllocCounters * kMaxLayersPerLaunch == QKVS_NOALLOC_MAX_LAYERS, "limit stated in the header");
static __device__ __align__(256) uint32_t g_noalloc_counters[kNoAllocCounters];

// Device address of g_noalloc_counters on the current device.  In host code the array's name only
// stands for the symbol, it is not a device pointer; the runtime has to be asked for the address,
// once per device, with that device current.
static cudaError_t noalloc_counters(uint32_t **out)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mutex;
    static uint32_t *address[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mutex);
    if (dev >= 0 && dev < kMaxDevices && address[dev]) {
        *out = address[dev];
        return cudaSuccess;
    }
    void *ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_counters);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices) address[dev] = static_cast<uint32_t *>(ptr);
    *out = static_cast<uint32_t *>(ptr);
    return cudaSuccess;
}

}  // namespace qkvs

using namespace qkvs;

extern "C" {

size_t qkvs_record_bytes(int32_t head_dim, int32_t b, int32_t meta_bytes)
{
    const int meta = meta_bytes_of(meta_bytes);
    if (head_dim <= 0 || head_dim % 64 != 0 || meta == 0) return 0;
    if (meta == kMetaFp16 && head_dim % 128 != 0) return 0;
    return record_bytes(head_dim, b, meta);
}

qkvs_status_t qkvs_card_prefix_size(const qkvs_layout_t *layout, size_t *out_bytes)
{
    const qkvs_status_t st = check_shape(layout);
    if (st != QKVS_OK) return st;
    if (!out_bytes) return QKVS_ERR_INVALID_ARG;
    *out_bytes = (size_t)card_sections(layout->n_layers, layout->n_kv_heads, layout->n_tokens, layout->bits_mode).payload_off;
    return QKVS_OK;
}

qkvs_status_t qkvs_card_size(const qkvs_layout_t *layout, const uint8_t *bits_host, size_t *out_bytes)
{
    const qkvs_status_t st = check_shape(layout);
    if (st != QKVS_OK) return st;
    if (!out_bytes) return QKVS_ERR_INVALID_ARG;
    const Sections sec = card_sections(layout->n_layers, layout->n_kv_heads, layout->n_tokens, layout->bits_mode);
    const int64_t nseg = layout->bits_mode == 0 ? 1 : (int64_t)layout->n_layers * layout->n_kv_heads;
    const uint64_t streams_per_seg = layout->bits_mode == 0 ? 2u * (uint64_t)layout->n_layers * (uint64_t)layout->n_kv_heads : 2u;
    const int64_t T = layout->n_tokens;
    uint64_t payload = 0;
    for (int64_t seg = 0; seg < nseg; ++seg) {
        uint64_t seg_bytes = 0;
        for (int64_t t = 0; t < T; ++t) {
            const uint32_t r = record_bytes(layout->head_dim, bits_host ? bits_host[seg * T + t] : 16, meta_bytes_of(layout->meta_bytes), layout->group_size);
            if (r == 0) return QKVS_ERR_BAD_BITS;
            seg_bytes += r;
        }
        payload += seg_bytes * streams_per_seg;
    }
    *out_bytes = (size_t)(sec.payload_off + payload);
    return QKVS_OK;
}

qkvs_status_t qkvs_card_create(const qkvs_layout_t *layout, const void *const *K_layers, const void *const *V_layers,
                               const uint8_t *bits_dev, const qkvs_card_meta_t *meta, void *card_dev,
                               size_t card_capacity, void *workspace_dev, void *stream)
{
    qkvs_status_t st = check_shape(layout);
    if (st != QKVS_OK) return st;
    if (!K_layers || !V_layers || !card_dev || (!bits_dev && layout->n_tokens > 0)) return QKVS_ERR_INVALID_ARG;
    st = check_strides(layout, 0);
    if (st != QKVS_OK) return st;
    if (!aligned16(card_dev) || !aligned16(workspace_dev)) return QKVS_ERR_INVALID_ARG;
    for (int l = 0; l < layout->n_layers; ++l)
        if (!K_layers[l] || !V_layers[l] || !aligned16(K_layers[l]) || !aligned16(V_layers[l])) return QKVS_ERR_INVALID_ARG;
    const Sections sec = card_sections(layout->n_layers, layout->n_kv_heads, layout->n_tokens, layout->bits_mode);
    if (card_capacity < sec.payload_off) return QKVS_ERR_BUFFER_TOO_SMALL;

    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    ScanParams sp;
    sp.bits = bits_dev;
    sp.card = static_cast<uint8_t *>(card_dev);
    sp.capacity = card_capacity;
    sp.n_layers = layout->n_layers;
    sp.n_kv_heads = layout->n_kv_heads;
    sp.head_dim = layout->head_dim;
    sp.n_tokens = layout->n_tokens;
    sp.bits_mode = layout->bits_mode;
    sp.meta_bytes = meta_bytes_of(layout->meta_bytes);
    sp.group_size = layout->group_size;
    sp.model_id = meta ? meta->model_id : 0;
    sp.sender_id = meta ? meta->sender_id : 0;
    sp.position_offset = meta ? meta->position_offset : 0;
    sp.workspace = static_cast<uint32_t *>(workspace_dev);
    const int nseg = layout->bits_mode == 0 ? 1 : layout->n_layers * layout->n_kv_heads;
    if (layout->bits_mode == 1 && cudaMemsetAsync(card_dev, 0, kHeaderBytes, cs) != cudaSuccess) return QKVS_ERR_CUDA;
    // no more threads than there are groups of eight tokens: a short context then pays for the
    // block-wide steps of four warps, not of thirty-two
    // ... and with a segment per (layer, head) CTAs of 256 threads, of which every SM holds several:
    // a thousand threads at the kernel's register count leave one CTA per SM and a second round
    const int64_t most_threads = nseg > 1 ? 256 : kScanThreads;
    const int scan_threads = (int)std::min<int64_t>(most_threads, std::max<int64_t>(32, (((int64_t)layout->n_tokens + kScanItems - 1) / kScanItems + 31) / 32 * 32));
    scan_offsets_kernel<<<nseg, scan_threads, 0, cs>>>(sp);
    if (cudaGetLastError() != cudaSuccess) return QKVS_ERR_CUDA;

    PathParams p;
    memset(&p, 0, sizeof(p));
    p.card = static_cast<uint8_t *>(card_dev);
    p.card_bytes = card_capacity;
    p.n_layers = layout->n_layers;
    p.n_kv_heads = layout->n_kv_heads;
    p.head_dim = layout->head_dim;
    p.n_tokens = layout->n_tokens;
    p.bits_mode = layout->bits_mode;
    p.meta_bytes = meta_bytes_of(layout->meta_bytes);
    p.group_size = layout->group_size;
    p.head_stride = layout->head_stride;
    p.token_stride = layout->token_stride;
    for (int l0 = 0; l0 < layout->n_layers; l0 += kMaxLayersPerLaunch) {
        const int n = std::min(kMaxLayersPerLaunch, layout->n_layers - l0);
        LayerPtrs ptrs;
        memset(&ptrs, 0, sizeof(ptrs));
        for (int i = 0; i < n; ++i) {
            ptrs.k[i] = const_cast<void *>(K_layers[l0 + i]);
            ptrs.v[i] = const_cast<void *>(V_layers[l0 + i]);
        }
        p.layer_begin = l0;
        p.layer_count = n;
        p.work_counter = work_counter(workspace_dev, l0 / kMaxLayersPerLaunch);
        const int64_t streams = 2ll * n * layout->n_kv_heads;
        if (launch_create_for(p, ptrs, streams, cs) != cudaSuccess) return QKVS_ERR_CUDA;
    }
    return QKVS_OK;
}

qkvs_status_t qkvs_card_inject(const void *card_dev, size_t card_bytes, const qkvs_layout_t *dst,
                               void *const *K_layers_out, void *const *V_layers_out, int64_t dst_token_offset,
                               void *workspace_dev, void *stream)
{
    qkvs_status_t st = check_shape(dst);
    if (st != QKVS_OK) return st;
    if (!card_dev || !K_layers_out || !V_layers_out) return QKVS_ERR_INVALID_ARG;
    st = check_strides(dst, dst_token_offset);
    if (st != QKVS_OK) return st;
    if (!aligned16(card_dev) || !aligned16(workspace_dev)) return QKVS_ERR_INVALID_ARG;
    if (card_bytes < (size_t)kHeaderBytes) return QKVS_ERR_BAD_CARD;
    for (int l = 0; l < dst->n_layers; ++l)
        if (!K_layers_out[l] || !V_layers_out[l] || !aligned16(K_layers_out[l]) || !aligned16(V_layers_out[l]))
            return QKVS_ERR_INVALID_ARG;
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    if (workspace_dev && cudaMemsetAsync(workspace_dev, 0, QKVS_WORKSPACE_BYTES, cs) != cudaSuccess) return QKVS_ERR_CUDA;

    PathParams p;
    memset(&p, 0, sizeof(p));
    p.card = const_cast<uint8_t *>(static_cast<const uint8_t *>(card_dev));
    p.card_bytes = card_bytes;
    p.n_layers = dst->n_layers;
    p.n_kv_heads = dst->n_kv_heads;
    p.head_dim = dst->head_dim;
    p.n_tokens = dst->n_tokens;
    p.bits_mode = 0;  // taken from the card on the device
    p.meta_bytes = meta_bytes_of(dst->meta_bytes);  // the card's header must say the same
    p.group_size = dst->group_size;                 // ... and this
    p.head_stride = dst->head_stride;
    p.token_stride = dst->token_stride;
    p.dst_token_offset = dst_token_offset;
    p.status_dev = static_cast<int32_t *>(workspace_dev);  // word 0 of the scratch block
    for (int l0 = 0; l0 < dst->n_layers; l0 += kMaxLayersPerLaunch) {
        const int n = std::min(kMaxLayersPerLaunch, dst->n_layers - l0);
        LayerPtrs ptrs;
        memset(&ptrs, 0, sizeof(ptrs));
        for (int i = 0; i < n; ++i) {
            ptrs.k[i] = K_layers_out[l0 + i];
            ptrs.v[i] = V_layers_out[l0 + i];
        }
        p.layer_begin = l0;
        p.layer_count = n;
        p.work_counter = work_counter(workspace_dev, l0 / kMaxLayersPerLaunch);
        const int64_t streams = 2ll * n * dst->n_kv_heads;
        if (launch_inject_for(p, ptrs, streams, cs) != cudaSuccess) return QKVS_ERR_CUDA;
    }
    return QKVS_OK;
}

qkvs_status_t qkvs_card_inject_noalloc(const void *card_dev, size_t card_bytes, const qkvs_layout_t *dst,
                                       void *const *K_layers_out, void *const *V_layers_out, int64_t dst_token_offset,
                                       int32_t *status_dev, void *stream)
{
    qkvs_status_t st = check_shape(dst);
    if (st != QKVS_OK) return st;
    if (dst->n_layers > QKVS_NOALLOC_MAX_LAYERS) return QKVS_ERR_UNSUPPORTED_SHAPE;
    if (!card_dev || !K_layers_out || !V_layers_out) return QKVS_ERR_INVALID_ARG;
    st = check_strides(dst, dst_token_offset);
    if (st != QKVS_OK) return st;
    if (!aligned16(card_dev) || (reinterpret_cast<uintptr_t>(status_dev) & 3u)) return QKVS_ERR_INVALID_ARG;
    if (card_bytes < (size_t)kHeaderBytes) return QKVS_ERR_BAD_CARD;
    for (int l = 0; l < dst->n_layers; ++l)
        if (!K_layers_out[l] || !V_layers_out[l] || !aligned16(K_layers_out[l]) || !aligned16(V_layers_out[l]))
            return QKVS_ERR_INVALID_ARG;
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    uint32_t *counters = nullptr;
    if (noalloc_counters(&counters) != cudaSuccess) return QKVS_ERR_CUDA;
    // the array keeps what the previous call left in it: the counters have to start at zero
    if (cudaMemsetAsync(counters, 0, sizeof(uint32_t) * kNoAllocCounters, cs) != cudaSuccess) return QKVS_ERR_CUDA;
    if (status_dev && cudaMemsetAsync(status_dev, 0, sizeof(int32_t), cs) != cudaSuccess) return QKVS_ERR_CUDA;

    PathParams p;
    memset(&p, 0, sizeof(p));
    p.card = const_cast<uint8_t *>(static_cast<const uint8_t *>(card_dev));
    p.card_bytes = card_bytes;
    p.n_layers = dst->n_layers;
    p.n_kv_heads = dst->n_kv_heads;
    p.head_dim = dst->head_dim;
    p.n_tokens = dst->n_tokens;
    p.bits_mode = 0;  // taken from the card on the device
    p.meta_bytes = meta_bytes_of(dst->meta_bytes);  // the card's header must say the same
    p.group_size = dst->group_size;                 // ... and this
    p.head_stride = dst->head_stride;
    p.token_stride = dst->token_stride;
    p.dst_token_offset = dst_token_offset;
    p.status_dev = status_dev;
    for (int l0 = 0; l0 < dst->n_layers; l0 += kMaxLayersPerLaunch) {
        const int n = std::min(kMaxLayersPerLaunch, dst->n_layers - l0);
        LayerPtrs ptrs;
        memset(&ptrs, 0, sizeof(ptrs));
        for (int i = 0; i < n; ++i) {
            ptrs.k[i] = K_layers_out[l0 + i];
            ptrs.v[i] = V_layers_out[l0 + i];
        }
        p.layer_begin = l0;
        p.layer_count = n;
        p.work_counter = counters + l0 / kMaxLayersPerLaunch;
        const int64_t streams = 2ll * n * dst->n_kv_heads;
        if (launch_inject_for(p, ptrs, streams, cs) != cudaSuccess) return QKVS_ERR_CUDA;
    }
    return QKVS_OK;
}

qkvs_status_t qkvs_card_send(const void *card_dev, size_t card_bytes, int32_t src_device, void *dst_dev,
                             size_t dst_capacity, int32_t dst_device, void *stream)
{
    if (!card_dev || !dst_dev || !aligned16(card_dev) || !aligned16(dst_dev)) return QKVS_ERR_INVALID_ARG;
    if (src_device < 0 || dst_device < 0) return QKVS_ERR_INVALID_ARG;
    if (card_bytes < (size_t)kHeaderBytes) return QKVS_ERR_BAD_CARD;
    if (dst_capacity < card_bytes) return QKVS_ERR_BUFFER_TOO_SMALL;
    int n_devices = 0, current = -1;
    if (cudaGetDeviceCount(&n_devices) != cudaSuccess || cudaGetDevice(&current) != cudaSuccess) return QKVS_ERR_CUDA;
    if (src_device >= n_devices || dst_device >= n_devices) return QKVS_ERR_INVALID_ARG;
    if (current != src_device && current != dst_device) return QKVS_ERR_INVALID_ARG;
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    if (src_device == dst_device)
        return cudaMemcpyAsync(dst_dev, card_dev, card_bytes, cudaMemcpyDeviceToDevice, cs) == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
    // a direct copy over NVLink needs peer access from the device that runs the copy to the other
    const int other = current == src_device ? dst_device : src_device;
    int can = 0;
    if (cudaDeviceCanAccessPeer(&can, current, other) != cudaSuccess) return QKVS_ERR_CUDA;
    if (can) {
        const cudaError_t e = cudaDeviceEnablePeerAccess(other, 0);
        if (e == cudaErrorPeerAccessAlreadyEnabled) (void)cudaGetLastError();  // on already: not an error
        else if (e != cudaSuccess) return QKVS_ERR_CUDA;
    }
    return cudaMemcpyPeerAsync(dst_dev, dst_device, card_dev, src_device, card_bytes, cs) == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

// Which attention kernel runs: the mma.sync one unless the environment asks for the tcgen05 one
// (QKVS_ATTEND_KERNEL=tcgen05), which is correct but, as measured, not yet the faster of the two.
static bool attend_on_tcgen05()
{
    static const bool v = [] {
        const char *e = getenv("QKVS_ATTEND_KERNEL");
        return e && strcmp(e, "tcgen05") == 0;
    }();
    return v;
}

// Shape of the attention work per (layer, KV head): items of 512 tokens for the tcgen05 kernel;
// steps of 16 tokens and items of 16 steps for the mma.sync kernel.
static qkvs_status_t attend_shape(const qkvs_layout_t *layout, int32_t n_q_heads, AttendParams *p)
{
    const qkvs_status_t st = check_shape(layout);
    if (st != QKVS_OK) return st;
    if (layout->head_dim != kAttendD) return QKVS_ERR_UNSUPPORTED_SHAPE;
    if (layout->group_size != kGroup && attend_on_tcgen05()) return QKVS_ERR_UNSUPPORTED_SHAPE;  // that variant reads groups of 32 only
    if (n_q_heads < layout->n_kv_heads || n_q_heads % layout->n_kv_heads != 0) return QKVS_ERR_INVALID_ARG;
    if (n_q_heads / layout->n_kv_heads > kAttendMaxPerKv) return QKVS_ERR_UNSUPPORTED_SHAPE;
    memset(p, 0, sizeof(*p));
    p->n_layers = layout->n_layers;
    p->n_kv_heads = layout->n_kv_heads;
    p->n_tokens = layout->n_tokens;
    p->n_q_heads = n_q_heads;
    p->meta_bytes = meta_bytes_of(layout->meta_bytes);
    p->subs_per_head = (uint32_t)(((int64_t)layout->n_tokens + kAttendRows - 1) / kAttendRows);
    p->items_per_head = attend_on_tcgen05() ? (uint32_t)(((int64_t)layout->n_tokens + kTcItemTokens - 1) / kTcItemTokens)
                                            : (p->subs_per_head + kAttendSteps - 1) / kAttendSteps;
    const uint64_t n_items = (uint64_t)layout->n_layers * (uint64_t)layout->n_kv_heads * p->items_per_head;
    if (n_items > 0x7fffffffull) return QKVS_ERR_UNSUPPORTED_SHAPE;
    p->n_items = (uint32_t)n_items;
    p->last_rows = p->subs_per_head ? (uint32_t)(layout->n_tokens - (int64_t)(p->subs_per_head - 1) * kAttendRows) : 0u;
    return QKVS_OK;
}

static size_t attend_scratch_bytes(const AttendParams &p)
{
    const size_t per_kv = (size_t)(p.n_q_heads / p.n_kv_heads);
    return (size_t)QKVS_WORKSPACE_BYTES + (size_t)p.n_items * per_kv * kPartialFloats * sizeof(float);
}

extern "C++" {
#ifndef QKVS_ATTEND_STAGES
#define QKVS_ATTEND_STAGES 2
#endif
#ifndef QKVS_ATTEND_WARPS
#define QKVS_ATTEND_WARPS 8  // two CTAs of eight warps per SM: neighbouring items, i.e. neighbouring spans of a stream, start together
#endif
constexpr int kAttendStages = QKVS_ATTEND_STAGES, kAttendWarps = QKVS_ATTEND_WARPS;

// One instance of the mma.sync kernel per record format (pair size x group size).
template <int FMT>
static qkvs_status_t launch_attend_format(const AttendParams &p, cudaStream_t cs)
{
    auto kernel = attend_kernel<kAttendStages, kAttendWarps, FMT>;
    const size_t smem = kAttendWarps * sizeof(AttendWarpSmem<kAttendStages>);
    unsigned grid = 0;
    if (persistent_grid<1000 + FMT>(kernel, kAttendWarps * 32, smem, (int64_t)((p.n_items + kAttendWarps - 1) / kAttendWarps), &grid) != cudaSuccess)
        return QKVS_ERR_CUDA;
    kernel<<<grid, kAttendWarps * 32, smem, cs>>>(p);
    return cudaGetLastError() == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

static qkvs_status_t launch_attend(const AttendParams &p, int group_size, cudaStream_t cs)
{
    switch (format_code(p.meta_bytes, group_size)) {
        case format_code(kMetaFp32, 32): return launch_attend_format<format_code(kMetaFp32, 32)>(p, cs);
        case format_code(kMetaFp16, 32): return launch_attend_format<format_code(kMetaFp16, 32)>(p, cs);
        case format_code(kMetaFp32, 64): return launch_attend_format<format_code(kMetaFp32, 64)>(p, cs);
        case format_code(kMetaFp16, 64): return launch_attend_format<format_code(kMetaFp16, 64)>(p, cs);
        case format_code(kMetaFp32, 128): return launch_attend_format<format_code(kMetaFp32, 128)>(p, cs);
        case format_code(kMetaFp16, 128): return launch_attend_format<format_code(kMetaFp16, 128)>(p, cs);
        default: return QKVS_ERR_UNSUPPORTED_SHAPE;
    }
}
}  // extern "C++"

qkvs_status_t qkvs_attend_scratch_size(const qkvs_layout_t *layout, int32_t n_q_heads, size_t *out_bytes)
{
    AttendParams p;
    const qkvs_status_t st = attend_shape(layout, n_q_heads, &p);
    if (st != QKVS_OK) return st;
    if (!out_bytes) return QKVS_ERR_INVALID_ARG;
    *out_bytes = attend_scratch_bytes(p);
    return QKVS_OK;
}

qkvs_status_t qkvs_card_attend(const void *card_dev, size_t card_bytes, const qkvs_layout_t *layout, int32_t n_q_heads,
                               const void *q_dev, float softmax_scale, float *out_dev, void *scratch_dev,
                               size_t scratch_bytes, void *stream)
{
    AttendParams p;
    const qkvs_status_t st = attend_shape(layout, n_q_heads, &p);
    if (st != QKVS_OK) return st;
    if (!card_dev || !q_dev || !out_dev || !scratch_dev) return QKVS_ERR_INVALID_ARG;
    if (!aligned16(card_dev) || !aligned16(q_dev) || !aligned16(out_dev) || !aligned16(scratch_dev)) return QKVS_ERR_INVALID_ARG;
    if (card_bytes < (size_t)kHeaderBytes) return QKVS_ERR_BAD_CARD;
    if (scratch_bytes < attend_scratch_bytes(p)) return QKVS_ERR_BUFFER_TOO_SMALL;
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(scratch_dev, 0, QKVS_WORKSPACE_BYTES, cs) != cudaSuccess) return QKVS_ERR_CUDA;
    p.card = static_cast<const uint8_t *>(card_dev);
    p.card_bytes = card_bytes;
    p.q = static_cast<const __half *>(q_dev);
    p.scale_log2 = softmax_scale * 1.4426950408889634f;
    p.out = out_dev;
    p.status_dev = static_cast<int32_t *>(scratch_dev);
    p.work_counter = static_cast<uint32_t *>(scratch_dev) + 1;
    p.partials = reinterpret_cast<float *>(static_cast<uint8_t *>(scratch_dev) + QKVS_WORKSPACE_BYTES);
    if (p.n_items > 0 && attend_on_tcgen05()) {
        const bool compact = p.meta_bytes == kMetaFp16, wide = n_q_heads / layout->n_kv_heads > 4;
        auto kernel = compact ? (wide ? attend_tc_kernel<8, kMetaFp16> : attend_tc_kernel<4, kMetaFp16>)
                              : (wide ? attend_tc_kernel<8, kMetaFp32> : attend_tc_kernel<4, kMetaFp32>);
        const size_t smem = kTcPipes * sizeof(TcPipeSmem);
        const int64_t want = (int64_t)((p.n_items + kTcPipes - 1) / kTcPipes);
        unsigned grid = 0;
        cudaError_t e = compact ? (wide ? persistent_grid<1013>(kernel, kTcThreads, smem, want, &grid) : persistent_grid<1012>(kernel, kTcThreads, smem, want, &grid))
                                : (wide ? persistent_grid<1011>(kernel, kTcThreads, smem, want, &grid) : persistent_grid<1010>(kernel, kTcThreads, smem, want, &grid));
        if (e != cudaSuccess) return QKVS_ERR_CUDA;
        kernel<<<grid, kTcThreads, smem, cs>>>(p);
        if (cudaGetLastError() != cudaSuccess) return QKVS_ERR_CUDA;
    } else if (p.n_items > 0) {
        const qkvs_status_t ls = launch_attend(p, layout->group_size, cs);
        if (ls != QKVS_OK) return ls;
    }
    // the merge is launched so that it can come onto the device while the first kernel drains
    // (it waits for that kernel's completion before its first read)
    const unsigned rows = (unsigned)p.n_layers * (unsigned)p.n_q_heads;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(rows);
    cfg.blockDim = dim3(128);
    cfg.stream = cs;
    cudaLaunchAttribute attr;
    memset(&attr, 0, sizeof(attr));
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, attend_merge_kernel, p) == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

qkvs_status_t qkvs_bits_from_scores(const float *scores_dev, int32_t n_segments, int32_t n_tokens, int32_t n_fp16,
                                    int32_t n_8bit, int32_t n_4bit, uint8_t *bits_dev, void *stream)
{
    if (n_segments < 1 || n_tokens < 0 || n_fp16 < 0 || n_8bit < 0 || n_4bit < 0) return QKVS_ERR_INVALID_ARG;
    if ((int64_t)n_fp16 + n_8bit + n_4bit > n_tokens) return QKVS_ERR_INVALID_ARG;
    if (n_tokens > (1 << 20) || n_segments > (1 << 24)) return QKVS_ERR_UNSUPPORTED_SHAPE;
    if (n_tokens == 0) return QKVS_OK;
    if (!scores_dev || !bits_dev || (reinterpret_cast<uintptr_t>(scores_dev) & 3u)) return QKVS_ERR_INVALID_ARG;
    bits_by_rank_kernel<<<(unsigned)n_segments, kSelThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        scores_dev, n_tokens, (uint32_t)n_fp16, (uint32_t)n_8bit, (uint32_t)n_4bit, bits_dev, nullptr, 128, kMetaFp32);
    return cudaGetLastError() == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

qkvs_status_t qkvs_bits_from_scores_budget(const float *scores_dev, int32_t n_segments, int32_t n_tokens, int32_t head_dim,
                                           int32_t meta_bytes, uint64_t budget_bytes, const float *upgrade_weight,
                                           uint8_t *bits_dev, uint32_t *offsets_dev, int32_t *status_dev, void *stream)
{
    static const float kDefaultWeight[3] = {0x1p-9f, 0x1p-14f, 0x1p-23f};
    if (n_segments < 1 || n_tokens < 0) return QKVS_ERR_INVALID_ARG;
    if (n_tokens > (1 << 20) || n_segments > (1 << 24)) return QKVS_ERR_UNSUPPORTED_SHAPE;
    const int meta = meta_bytes_of(meta_bytes);
    if (meta == 0) return QKVS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128 && head_dim != 192 && head_dim != 256) return QKVS_ERR_UNSUPPORTED_SHAPE;
    if (meta == kMetaFp16 && head_dim % 128 != 0) return QKVS_ERR_UNSUPPORTED_SHAPE;
    const float *w = upgrade_weight ? upgrade_weight : kDefaultWeight;
    if (!(w[0] > 0.0f && w[1] > 0.0f && w[2] > 0.0f && w[0] >= w[1] && w[1] >= w[2])) return QKVS_ERR_INVALID_ARG;
    BudgetParams bp;
    memset(&bp, 0, sizeof(bp));
    bp.rec2 = record_bytes(head_dim, 2, meta);
    const uint32_t ladder[4] = {bp.rec2, record_bytes(head_dim, 4, meta), record_bytes(head_dim, 8, meta), record_bytes(head_dim, 16, meta)};
    if ((uint64_t)n_tokens * bp.rec2 > budget_bytes) return QKVS_ERR_BUFFER_TOO_SMALL;
    if (n_tokens == 0) return QKVS_OK;
    if (!scores_dev || !bits_dev || (reinterpret_cast<uintptr_t>(scores_dev) & 3u) || (reinterpret_cast<uintptr_t>(offsets_dev) & 3u) ||
        (reinterpret_cast<uintptr_t>(status_dev) & 3u))
        return QKVS_ERR_INVALID_ARG;
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    if (status_dev && cudaMemsetAsync(status_dev, 0, sizeof(int32_t), cs) != cudaSuccess) return QKVS_ERR_CUDA;
    bp.scores = scores_dev;
    bp.T = n_tokens;
    bp.budget = budget_bytes;
    for (int i = 0; i < 3; ++i) {
        bp.weight[i] = w[i];
        bp.cost[i] = ladder[i + 1] - ladder[i];
    }
    bp.bits = bits_dev;
    bp.offsets = offsets_dev;
    bp.status = status_dev;
    bp.head_dim = head_dim;
    bp.meta = meta;
    bits_by_budget_kernel<<<(unsigned)n_segments, kSelThreads, 0, cs>>>(bp);
    return cudaGetLastError() == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

qkvs_status_t qkvs_combine_scores(const float *importance_dev, const float *transfer_dev, float alpha, int64_t n,
                                  float *scores_dev, void *stream)
{
    if (n < 0 || !(alpha >= 0.0f && alpha <= 1.0f)) return QKVS_ERR_INVALID_ARG;
    if (n == 0) return QKVS_OK;
    if (!importance_dev || !transfer_dev || !scores_dev) return QKVS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(importance_dev) | reinterpret_cast<uintptr_t>(transfer_dev) | reinterpret_cast<uintptr_t>(scores_dev)) & 3u)
        return QKVS_ERR_INVALID_ARG;
    const float beta = 1.0f - alpha;  // one rounded subtraction on the host, as in the definition
    const unsigned grid = (unsigned)std::min<int64_t>((n + 255) / 256, 148 * 8);
    combine_scores_kernel<<<grid, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(importance_dev, transfer_dev, alpha, beta, n, scores_dev);
    return cudaGetLastError() == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

qkvs_status_t qkvs_bits_from_features(const float *features_dev, int64_t n_tokens, int32_t hidden, const float *params_dev,
                                      uint8_t *bits_dev, float *outputs_dev, void *stream)
{
    if (n_tokens < 0 || hidden < 1) return QKVS_ERR_INVALID_ARG;
    if (hidden > kControllerMaxHidden) return QKVS_ERR_UNSUPPORTED_SHAPE;
    if (n_tokens == 0) return QKVS_OK;
    if (!features_dev || !params_dev || !bits_dev) return QKVS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(features_dev) | reinterpret_cast<uintptr_t>(params_dev) | reinterpret_cast<uintptr_t>(outputs_dev)) & 3u)
        return QKVS_ERR_INVALID_ARG;
    const unsigned grid = (unsigned)std::min<int64_t>((n_tokens + 255) / 256, 148 * 8);
    controller_kernel<<<grid, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(features_dev, n_tokens, hidden, params_dev, bits_dev, outputs_dev);
    return cudaGetLastError() == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

qkvs_status_t qkvs_card_info(const void *card_dev, void *stream, qkvs_card_header_t *out_host)
{
    if (!card_dev || !out_host) return QKVS_ERR_INVALID_ARG;
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(out_host, card_dev, kHeaderBytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return QKVS_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return QKVS_ERR_CUDA;
    if (out_host->magic != kMagic || out_host->version != kVersion) return QKVS_ERR_BAD_CARD;
    if (out_host->status > (uint32_t)QKVS_ERR_TIMEOUT) return QKVS_ERR_BAD_CARD;
    return (qkvs_status_t)out_host->status;
}

qkvs_status_t qkvs_selftest_division(uint64_t *mismatches_dev, void *stream)
{
    if (!mismatches_dev || (reinterpret_cast<uintptr_t>(mismatches_dev) & 7u)) return QKVS_ERR_INVALID_ARG;
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(mismatches_dev, 0, 2 * sizeof(uint64_t), cs) != cudaSuccess) return QKVS_ERR_CUDA;
    selftest_division_kernel<<<148 * 8, 256, 0, cs>>>(reinterpret_cast<unsigned long long *>(mismatches_dev));
    return cudaGetLastError() == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

qkvs_status_t qkvs_selftest_bounded_wait(uint32_t limit_us, int32_t *status_dev, uint64_t *waited_ns_dev, void *stream)
{
    if (!status_dev || (reinterpret_cast<uintptr_t>(status_dev) & 3u) || (reinterpret_cast<uintptr_t>(waited_ns_dev) & 7u))
        return QKVS_ERR_INVALID_ARG;
    if (limit_us == 0 || limit_us > 1000000u) return QKVS_ERR_INVALID_ARG;  // at most a second
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(status_dev, 0, sizeof(int32_t), cs) != cudaSuccess) return QKVS_ERR_CUDA;
    selftest_wait_kernel<<<1, 32, 0, cs>>>((unsigned long long)limit_us * 1000ull, status_dev,
                                           reinterpret_cast<unsigned long long *>(waited_ns_dev));
    return cudaGetLastError() == cudaSuccess ? QKVS_OK : QKVS_ERR_CUDA;
}

const char *qkvs_status_string(qkvs_status_t status)
{
    switch (status) {
        case QKVS_OK: return "ok";
        case QKVS_ERR_INVALID_ARG: return "invalid argument";
        case QKVS_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case QKVS_ERR_BAD_BITS: return "bit-width outside {2,4,8,16}";
        case QKVS_ERR_BUFFER_TOO_SMALL: return "card buffer too small";
        case QKVS_ERR_BAD_CARD: return "card header or tables do not check out";
        case QKVS_ERR_CUDA: return "CUDA runtime error";
        case QKVS_ERR_TIMEOUT: return "bounded wait inside a kernel gave up";
    }
    return "unknown status";
}

int32_t qkvs_version(void) { return 100; }

}  // extern "C"
