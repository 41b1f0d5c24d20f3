// Bit-widths from importance scores, the step in front of card creation, by selection instead of
// sorting: one CTA per segment finds, byte by byte from the top, the key at which a rank (or a byte
// budget) is reached, and then every token decides for itself on which side of that key it lies.
// Equal keys are told apart by token index through one block-wide prefix count.  Optionally the
// same launch also writes the offset table the bit-widths imply (exclusive prefix sum of record
// sizes), so that bit-widths and offsets come out of one kernel.
//
//   rank rule    tokens ordered by score, highest first, equal scores by lower index; the first
//                n16 keep FP16, the next n8 get 8 bits, the next n4 get 4 bits, the rest 2 bits.
//   budget rule  every token starts at 2 bits; the 3 T possible upgrades (token t one rung up the
//                ladder 2 -> 4 -> 8 -> 16, rung i = 0, 1, 2) are ordered by worth per byte
//                key = fl32(score_t * weight_i), larger first, equal keys by lower rung, then by
//                lower index, and granted in that order while their cost (difference of record
//                sizes) still fits into the byte budget of a stream; the first one that does not
//                fit ends the procedure.
// A thread owns a run of consecutive tokens, so a prefix count over threads is a count in index order.
#pragma once

#include "qkvs_common.cuh"

namespace qkvs {

constexpr int kSelThreads = 1024;
constexpr int kSelStaged = 8192;   // segments up to this many tokens are read once and kept in shared memory

// Larger score -> larger key; +0 and -0 get the same key.
__device__ __forceinline__ uint32_t order_key(float s)
{
    const float c = s == 0.0f ? 0.0f : s;
    const uint32_t u = __float_as_uint(c);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One warp looks for the byte value d with  above(d) < need <= above(d) + h[d],  above(d) being
// the sum of h over all larger byte values.  Returns d (or -1 when even the total is below need)
// and above(d) through `above`.  All 32 lanes call it; the result is the same in all.
__device__ __forceinline__ int pick_byte(const uint32_t *h, unsigned long long need, unsigned long long &above, int lane)
{
    unsigned long long mine = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) mine += h[8 * lane + i];
    unsigned long long incl = mine;  // sum over this lane and all higher lanes
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const unsigned long long o = __shfl_down_sync(0xffffffffu, incl, s);
        if (lane + s < 32) incl += o;
    }
    unsigned long long run = incl - mine;  // everything in higher lanes
    int found = -1;
    unsigned long long found_above = 0;
#pragma unroll
    for (int i = 7; i >= 0; --i) {
        const unsigned long long c = h[8 * lane + i];
        if (found < 0 && run < need && need <= run + c) {
            found = 8 * lane + i;
            found_above = run;
        }
        run += c;
    }
    const unsigned ballot = __ballot_sync(0xffffffffu, found >= 0);
    if (ballot == 0u) {
        above = 0;
        return -1;
    }
    const int src = 31 - __clz(ballot);  // exactly one lane can match; take the highest to be safe
    above = __shfl_sync(0xffffffffu, found_above, src);
    return __shfl_sync(0xffffffffu, found, src);
}

// Exclusive prefix sum of one 64-bit value per thread over the block; `scratch` holds 33 entries.
__device__ __forceinline__ unsigned long long block_exclusive_scan64(unsigned long long v, unsigned long long *scratch, unsigned long long &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const unsigned long long o = __shfl_up_sync(0xffffffffu, inc, s);
        if (lane >= s) inc += o;
    }
    __syncthreads();  // scratch may still be read from an earlier call
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const unsigned long long w = lane < (int)(blockDim.x >> 5) ? scratch[lane] : 0ull;
        unsigned long long winc = w;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const unsigned long long o = __shfl_up_sync(0xffffffffu, winc, s);
            if (lane >= s) winc += o;
        }
        scratch[lane] = winc - w;
        if (lane == 31) scratch[32] = winc;
    }
    __syncthreads();
    total = scratch[32];
    return scratch[warp] + inc - v;
}

// Adds `weight` to hist[digit] for every lane with `active` set.  When all active lanes of the
// warp hold the same digit (few distinct scores, or the leading bits of a narrow range) one lane
// adds for all; otherwise every lane adds for itself, and the digits being spread out keeps the
// counters from colliding.  All 32 lanes call it together.
__device__ __forceinline__ void hist_add(uint32_t *hist, uint32_t digit, uint32_t weight, bool active, int lane)
{
    const uint32_t who = __ballot_sync(0xffffffffu, active);
    if (who == 0u) return;
    const int leader = __ffs(who) - 1;
    const uint32_t d0 = __shfl_sync(0xffffffffu, digit, leader);
    if (__all_sync(0xffffffffu, !active || digit == d0)) {
        if (lane == leader) atomicAdd(&hist[d0], weight * (uint32_t)__popc(who));
    } else if (active) {
        atomicAdd(&hist[digit], weight);
    }
}

// Smallest and largest of one key per thread over the block (threads without a key pass
// 0xffffffff / 0); `scratch` holds 64 entries of 32 bits.
__device__ __forceinline__ void block_min_max(uint32_t &lo, uint32_t &hi, uint32_t *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    lo = __reduce_min_sync(0xffffffffu, lo);
    hi = __reduce_max_sync(0xffffffffu, hi);
    __syncthreads();
    if (lane == 0) {
        scratch[warp] = lo;
        scratch[32 + warp] = hi;
    }
    __syncthreads();
    const int n = (int)(blockDim.x >> 5);
    uint32_t a = lane < n ? scratch[lane] : 0xffffffffu, b = lane < n ? scratch[32 + lane] : 0u;
    lo = __reduce_min_sync(0xffffffffu, a);
    hi = __reduce_max_sync(0xffffffffu, b);
}

struct SelectShared {
    uint32_t hist[3][256];
    unsigned long long scratch[33];
    uint32_t minmax[64];
    uint32_t prefix[3];
    unsigned long long need[3];
    uint32_t ties[3];
    int take_all;
};

// The offset table of a segment from its bit-widths (already in `bits`), written by the block.
__device__ __forceinline__ void write_offsets(const uint8_t *bits, int64_t T, int64_t first, int64_t last, int d, int meta,
                                              uint32_t *off, SelectShared &sh)
{
    unsigned long long mine = 0;
    for (int64_t t = first; t < last; ++t) mine += record_bytes(d, bits[t], meta);
    unsigned long long total;
    unsigned long long run = block_exclusive_scan64(mine, sh.scratch, total);
    for (int64_t t = first; t < last; ++t) {
        off[t] = (uint32_t)run;
        run += record_bytes(d, bits[t], meta);
    }
    if (threadIdx.x == 0) off[T] = (uint32_t)total;
}

// ---------------------------------------------------------------------------------------------
// rank rule
__global__ void __launch_bounds__(kSelThreads) bits_by_rank_kernel(const float *scores, int64_t T, uint32_t n16, uint32_t n8, uint32_t n4,
                                                                    uint8_t *bits, uint32_t *offsets, int head_dim, int meta)
{
    __shared__ SelectShared sh;
    __shared__ float stage[kSelStaged];
    scores += (int64_t)blockIdx.x * T;
    bits += (int64_t)blockIdx.x * T;
    if (offsets) offsets += (int64_t)blockIdx.x * (T + 1);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool staged = T <= kSelStaged;
    if (staged)
        for (int64_t t = tid; t < T; t += kSelThreads) stage[t] = scores[t];
    auto score_at = [&](int64_t t) { return staged ? stage[t] : scores[t]; };
    const int64_t per = (T + kSelThreads - 1) / kSelThreads;
    const int64_t first = min(T, (int64_t)tid * per), last = min(T, first + per);
    // the three cuts: a token is in the top `cut` when fewer than `cut` tokens come before it
    const unsigned long long cut[3] = {n16, (unsigned long long)n16 + n8, (unsigned long long)n16 + n8 + n4};
    bool active[3];
#pragma unroll
    for (int j = 0; j < 3; ++j) active[j] = cut[j] > 0 && cut[j] < (unsigned long long)T;
    if (tid < 3) {
        sh.prefix[tid] = 0u;
        sh.need[tid] = cut[tid];
    }
    // ---- keys are taken relative to the smallest one, and only the bits in which they differ are
    // walked: scores crowd into a few values of a float's leading byte, but spread evenly over the
    // leading bits of their own range, so the counters of a pass are not all the same one
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    for (int64_t t = tid; t < T; t += kSelThreads) {
        const uint32_t key = order_key(score_at(t));
        kmin = min(kmin, key);
        kmax = max(kmax, key);
    }
    block_min_max(kmin, kmax, sh.minmax);
    const int nbits = 32 - __clz(kmax - kmin);   // 0 when all keys are equal
    auto rel_key = [&](int64_t t) { return order_key(score_at(t)) - kmin; };
    // ---- the key of the token of rank cut - 1, up to eight bits per pass from the top
    for (int hi = nbits; hi > 0; hi -= 8) {
        const int lo = max(hi - 8, 0);
        const uint32_t digit_mask = (1u << (hi - lo)) - 1u;
        for (int i = tid; i < 3 * 256; i += kSelThreads) (&sh.hist[0][0])[i] = 0u;
        __syncthreads();
        uint32_t pf[3];
#pragma unroll
        for (int j = 0; j < 3; ++j) pf[j] = sh.prefix[j];
        // counting does not care about the order: neighbouring threads read neighbouring scores
        for (int64_t t0 = (int64_t)(tid - lane); t0 < T; t0 += kSelThreads) {
            const int64_t t = t0 + lane;
            const uint32_t key = t < T ? rel_key(t) : 0u;
#pragma unroll
            for (int j = 0; j < 3; ++j)
                if (active[j]) hist_add(sh.hist[j], (key >> lo) & digit_mask, 1u, t < T && (hi >= 32 || (key >> hi) == (pf[j] >> hi)), lane);
        }
        __syncthreads();
        if (warp < 3 && active[warp]) {
            unsigned long long above;
            const int dsel = pick_byte(sh.hist[warp], sh.need[warp], above, lane);
            if (lane == 0) {
                sh.prefix[warp] |= (uint32_t)max(dsel, 0) << lo;
                sh.need[warp] -= above;
            }
        }
        __syncthreads();
    }
    // sh.prefix[j]: the key at the cut; sh.need[j]: how many of the tokens with exactly that key are inside
    uint32_t tau[3];
    unsigned long long inside[3];
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        tau[j] = sh.prefix[j];
        inside[j] = sh.need[j];
    }
    // ---- equal keys by index: how many tokens with the cut's key lie in front of this thread's run
    unsigned long long packed = 0;  // three counts of 21 bits (T <= 2^20)
    for (int64_t t = first; t < last; ++t) {
        const uint32_t key = rel_key(t);
#pragma unroll
        for (int j = 0; j < 3; ++j) packed += (unsigned long long)(active[j] && key == tau[j]) << (21 * j);
    }
    unsigned long long total;
    unsigned long long before = block_exclusive_scan64(packed, sh.scratch, total);
    for (int64_t t = first; t < last; ++t) {
        const uint32_t key = rel_key(t);
        bool top[3];
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            const unsigned long long rank_in_ties = (before >> (21 * j)) & 0x1fffffull;
            if (!active[j]) top[j] = cut[j] >= (unsigned long long)T && cut[j] > 0;
            else top[j] = key > tau[j] || (key == tau[j] && rank_in_ties < inside[j]);
            before += (unsigned long long)(active[j] && key == tau[j]) << (21 * j);
        }
        bits[t] = top[0] ? 16 : (top[1] ? 8 : (top[2] ? 4 : 2));
    }
    if (offsets) {
        __syncthreads();  // a thread's run of bits was written by itself; the scratch is reused
        write_offsets(bits, T, first, last, head_dim, meta, offsets, sh);
    }
}

// ---------------------------------------------------------------------------------------------
// budget rule
struct BudgetParams {
    const float *scores;
    int64_t T;
    unsigned long long budget;   // bytes of one stream
    float weight[3];
    uint32_t cost[3];            // bytes an upgrade of rung i adds to a record
    uint32_t rec2;               // bytes of a 2-bit record
    uint8_t *bits;
    uint32_t *offsets;           // or null
    int32_t *status;             // or null: raised to INVALID_ARG by a negative or non-finite score
    int head_dim, meta;
};

__global__ void __launch_bounds__(kSelThreads) bits_by_budget_kernel(BudgetParams p)
{
    __shared__ SelectShared sh;
    __shared__ float stage[kSelStaged];
    __shared__ unsigned long long s_left;
    __shared__ int s_bad;
    const float *scores = p.scores + (int64_t)blockIdx.x * p.T;
    uint8_t *bits = p.bits + (int64_t)blockIdx.x * p.T;
    uint32_t *offsets = p.offsets ? p.offsets + (int64_t)blockIdx.x * (p.T + 1) : nullptr;
    const int64_t T = p.T;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t per = (T + kSelThreads - 1) / kSelThreads;
    const int64_t first = min(T, (int64_t)tid * per), last = min(T, first + per);
    if (tid == 0) {
        sh.prefix[0] = 0u;
        sh.take_all = 0;
        s_left = p.budget - (unsigned long long)T * p.rec2;   // the host has checked that this is not negative
        s_bad = 0;
        sh.ties[0] = sh.ties[1] = sh.ties[2] = 0u;
    }
    const bool staged = T <= kSelStaged;
    if (staged)
        for (int64_t t = tid; t < T; t += kSelThreads) stage[t] = scores[t];
    auto score_at = [&](int64_t t) { return staged ? stage[t] : scores[t]; };
    __syncthreads();   // the flags above are set before anybody raises one
    auto abs_key = [&](float s, int i) { return order_key(__fmul_rn(s == 0.0f ? 0.0f : s, p.weight[i])); };
    // keys relative to the smallest one, walked over the bits in which they differ (see the rank rule)
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    bool bad = false;
    for (int64_t t = tid; t < T; t += kSelThreads) {
        const float s = score_at(t);
        bad |= !(s >= 0.0f) || s > 3.0e38f;
        kmin = min(kmin, abs_key(s, 2));    // weights do not increase with the rung
        kmax = max(kmax, abs_key(s, 0));
    }
    if (bad) s_bad = 1;
    block_min_max(kmin, kmax, sh.minmax);
    const int nbits = 32 - __clz(kmax - kmin);
    auto key_of = [&](float s, int i) { return abs_key(s, i) - kmin; };
    if (tid == 0 && (unsigned long long)T * (p.cost[0] + p.cost[1] + p.cost[2]) <= s_left) sh.take_all = 1;  // everything fits: all tokens keep FP16
    __syncthreads();
    // ---- the key at which the budget runs out, up to eight bits per pass from the top (sums of costs)
    for (int hi = sh.take_all ? 0 : nbits; hi > 0; hi -= 8) {
        const int lo = max(hi - 8, 0);
        const uint32_t digit_mask = (1u << (hi - lo)) - 1u;
        for (int i = tid; i < 256; i += kSelThreads) sh.hist[0][i] = 0u;
        __syncthreads();
        const uint32_t pf = sh.prefix[0];
        // sums of costs per digit (at most 2^20 tokens * 512 bytes: 32 bits hold them); the order
        // does not matter here, so neighbouring threads read neighbouring scores
        for (int64_t t0 = (int64_t)(tid - lane); t0 < T; t0 += kSelThreads) {
            const int64_t t = t0 + lane;
            const float s = t < T ? score_at(t) : 0.0f;
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const uint32_t key = key_of(s, i);
                hist_add(sh.hist[0], (key >> lo) & digit_mask, p.cost[i], t < T && (hi >= 32 || (key >> hi) == (pf >> hi)), lane);
            }
        }
        __syncthreads();
        if (warp == 0) {
            unsigned long long above;
            const int dsel = pick_byte(sh.hist[0], s_left + 1ull, above, lane);  // the digit with which the budget is first exceeded
            if (lane == 0) {
                sh.prefix[0] |= (uint32_t)max(dsel, 0) << lo;
                s_left -= above;
            }
        }
        __syncthreads();
    }
    const bool take_all = sh.take_all != 0;
    const uint32_t tau = sh.prefix[0];
    // ---- upgrades with exactly that key: by rung, then by index, as far as what is left reaches
    if (!take_all) {
        uint32_t c[3] = {0u, 0u, 0u};
        for (int64_t t = first; t < last; ++t)
#pragma unroll
            for (int i = 0; i < 3; ++i) c[i] += key_of(score_at(t), i) == tau;
#pragma unroll
        for (int i = 0; i < 3; ++i) {
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) c[i] += __shfl_xor_sync(0xffffffffu, c[i], s);
            if (lane == 0 && c[i]) atomicAdd(&sh.ties[i], c[i]);
        }
    }
    __syncthreads();
    int partial = 3;                 // rung whose equal-key upgrades are granted only in part (none: 3)
    unsigned long long granted = 0;  // ... and how many of them are
    if (!take_all) {
        unsigned long long left = s_left;
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            if (partial == 3) {
                const unsigned long long fit = left / p.cost[i];
                if (fit < sh.ties[i]) {
                    partial = i;
                    granted = fit;
                } else {
                    left -= (unsigned long long)sh.ties[i] * p.cost[i];
                }
            }
        }
    }
    unsigned long long mine = 0;
    if (partial < 3)
        for (int64_t t = first; t < last; ++t) mine += key_of(score_at(t), partial) == tau;
    unsigned long long total;
    unsigned long long before = block_exclusive_scan64(mine, sh.scratch, total);
    const bool invalid = s_bad != 0;
    for (int64_t t = first; t < last; ++t) {
        int up = 0;
        if (take_all) {
            up = 3;
        } else {
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const uint32_t key = key_of(score_at(t), i);
                bool take = key > tau;
                if (key == tau) {
                    take = i < partial || (i == partial && before < granted);
                    if (i == partial) ++before;
                }
                up += take;
            }
        }
        bits[t] = invalid ? 2 : (up == 0 ? 2 : (up == 1 ? 4 : (up == 2 ? 8 : 16)));
    }
    if (invalid && tid == 0 && p.status) atomicMax(p.status, (int)QKVS_ERR_INVALID_ARG);
    if (offsets) {
        __syncthreads();
        write_offsets(bits, T, first, last, p.head_dim, p.meta, offsets, sh);
    }
}

}  // namespace qkvs
