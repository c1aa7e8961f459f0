// Shared device helpers for the GRAFT kernels (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#ifndef GRAFT_SPIN_LIMIT
#define GRAFT_SPIN_LIMIT (1u << 22)  // upper bound on mbarrier polls before a wait gives up
#endif

namespace graft {

constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.6931471805599453;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

// ---- total order on fp32 bit patterns -------------------------------------------------------
// ord(x) is monotone in x for all non-NaN x; -0 is mapped onto +0 so that equal values compare equal.
__device__ __forceinline__ uint32_t ord_from_bits(uint32_t u) {
    if ((u << 1) == 0u) u = 0u;
    return u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ uint32_t bits_from_ord(uint32_t o) {
    return o ^ ((o >> 31) ? 0x80000000u : 0xFFFFFFFFu);
}
__device__ __forceinline__ uint32_t ord_from_float(float x) { return ord_from_bits(__float_as_uint(x)); }
// 64-bit selection key: larger key = better candidate (value descending, then id ascending). 0 = empty.
__device__ __forceinline__ uint64_t make_key(uint32_t value_bits, uint32_t id) {
    return ((uint64_t)ord_from_bits(value_bits) << 32) | (uint64_t)(0xFFFFFFFFu - id);
}
__device__ __forceinline__ uint32_t key_id(uint64_t k) { return 0xFFFFFFFFu - (uint32_t)k; }
__device__ __forceinline__ float key_value(uint64_t k) { return __uint_as_float(bits_from_ord((uint32_t)(k >> 32))); }

// ---- math ------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t hmax2_bf16(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// ---- programmatic dependent launch ----------------------------------------------------------------
// A kernel launched with launch_pdl() may start before the kernel ahead of it in the stream has finished (once
// every CTA of that kernel has called pdl_launch_dependents() or exited); it must call pdl_wait() before it touches
// anything the earlier kernel writes.  pdl_wait() returns when the earlier grid has completed and its writes are
// visible; in a kernel launched the ordinary way both calls do nothing.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- mbarrier + TMA bulk copy -------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// The same with a suspend-time hint (ns): the thread may sleep that long in hardware before it polls again, which
// keeps the polls of a warp that has nothing else to do out of the issue slots of the warps beside it.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded_hint(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t ns) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;  // somebody gave up already: nobody waits any more
    for (uint32_t it = 0; it < GRAFT_SPIN_LIMIT; ++it) {
        if (mbar_try_wait_hint(bar, parity, ns)) return true;
        if ((it & 15u) == 15u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// Bounded wait.  Returns false (and raises *abort_flag) when the limit is hit or another thread already
// gave up; callers then carry on without waiting so that every thread still reaches the kernel's end.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;  // somebody gave up already: nobody waits any more
    for (uint32_t it = 0; it < GRAFT_SPIN_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// global -> shared bulk copy through the TMA unit; completion is signalled on `bar` (complete_tx bytes).
// src and dst 16-byte aligned, bytes a multiple of 16.  No multicast.
__device__ __forceinline__ void tma_load_1d(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tma_load_1d_hint(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            dst_smem),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// 16-byte read-only load that asks L2 to keep the line (table rows of frequent tokens are read round after round)
__device__ __forceinline__ float4 ldg_f4_keep(const float4* p, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p), "l"(policy));
    return v;
}
// named barrier among a subset of the CTA's warps
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

}  // namespace graft
