// Thin wrappers over the sm_100a PTX used by the pipelines: mbarriers, 1-D bulk asynchronous
// copies (TMA) between global and shared memory, the cross-proxy fence, the mixed-precision
// subtract and packed binary32 arithmetic.  Every wait is bounded: a wait that does not complete
// within kWaitLimitNs gives up and reports failure so that the kernel can record an error status
// and return.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace qkvs {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s
constexpr uint32_t kWaitHintNs = 1000000u;                    // suspend hint of one poll: 1 ms

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

// Makes barrier initialisation visible to the asynchronous proxy (follow with __syncthreads).
__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// 16 bytes global -> shared, asynchronously, by the calling thread (both addresses 16-byte aligned).
__device__ __forceinline__ void async_copy_16(void *dst_smem, const void *src_gmem)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst_smem)), "l"(src_gmem) : "memory");
}

// Ties the calling thread's async_copy_16 copies issued so far to `bar`: the barrier's count of
// pending arrivals goes up by one now and comes down again once those copies have landed (at once
// if there are none), so the current phase cannot complete before they have.  The thread that
// makes the phase's own arrival must do so after every thread has executed this.
__device__ __forceinline__ void async_copies_arrive_on(uint64_t *bar)
{
    asm volatile("cp.async.mbarrier.arrive.shared::cta.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}

// One poll of the phase with the given parity.  The hardware may suspend the warp inside the
// instruction until the phase completes or a time limit (the hint, in nanoseconds, or a shorter
// system limit) runs out, so a waiting warp spends almost no issue slots.
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity), "r"(kWaitHintNs)
        : "memory");
    return done != 0;
}

// A poll that never suspends the warp: it only tests whether the phase has completed.  For
// barriers completed a few hundred cycles after the wait begins (by other warps of the CTA or by
// the tensor cores), where the waiter wants to go on the moment that happens.
__device__ __forceinline__ bool mbar_try_wait_short(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Waits for the phase with the given parity.  Returns false if the phase did not complete within
// limit_ns; the caller then records an error status and winds down.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long start = global_timer_ns();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - start > limit_ns) return false;
    }
}

// The same wait built on the short poll.  The limit is counted in SM clock cycles (reading the
// cycle counter costs a few cycles, reading the nanosecond timer stalls the warp for far longer,
// which would put that delay between the arrival and the moment the waiter notices it):
// 4 * 10^9 cycles are at least two seconds at any clock this part runs at.
constexpr long long kWaitLimitCycles = 4000000000ll;

__device__ __forceinline__ bool mbar_wait_short(uint64_t *bar, uint32_t parity, long long limit_cycles = kWaitLimitCycles)
{
    if (mbar_try_wait_short(bar, parity)) return true;
    const long long start = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 8; ++i)
            if (mbar_try_wait_short(bar, parity)) return true;
        if (clock64() - start > limit_cycles) return false;
    }
}

// global -> shared bulk copy; completion is signalled on `bar` as `bytes` of transaction count.
// Addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// shared -> global bulk copy, tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_store(void *dst_gmem, const void *src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst_gmem), "r"(smem_addr(src_smem)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// Waits until at most N of this thread's bulk groups still have to *read* their source.
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

// Waits until at most N of this thread's bulk groups are still in flight at all.
template <int N>
__device__ __forceinline__ void bulk_wait()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

// Orders this thread's shared-memory writes (generic proxy) before later asynchronous-proxy
// reads of the same locations (a bulk store issued after a barrier).
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// (fl32(float(lo) - c), fl32(float(hi) - c)) for the two FP16 halves of `w`: each FP16 operand is
// widened exactly and the difference is rounded once to binary32.
__device__ __forceinline__ float2 sub_f32_f16x2(uint32_t w, float c)
{
    float2 d;
    asm("{\n\t.reg .b16 l, h;\n\t"
        "mov.b32 {l, h}, %2;\n\t"
        "sub.rn.f32.f16 %0, l, %3;\n\t"
        "sub.rn.f32.f16 %1, h, %3;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "r"(w), "f"(c));
    return d;
}

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute
// may start while the kernel before it in the stream still runs; grid_dependency_wait() then
// blocks until that kernel has completed and its writes are visible (without the attribute it
// returns at once).  allow_dependents() in the earlier kernel lets the next one start right away.
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void allow_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Packed binary32 arithmetic: one instruction performs the operation on both halves of a 64-bit
// register pair, each half rounded on its own exactly like the scalar instruction.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}

__device__ __forceinline__ void unpack_b32x2(uint64_t v, uint32_t &lo, uint32_t &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}

__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

}  // namespace qkvs
