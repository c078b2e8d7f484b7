// Inline-PTX building blocks shared by the tensor-core kernels: mbarriers with bounded
// waits, TMA copies, ldmatrix / movmatrix / mma.sync, and small numeric helpers.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace concur {

constexpr uint64_t kWaitLimitNs = 2000000000ull;          // every in-kernel wait gives up after 2 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(count) : "memory");
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
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false if the limit ran out or another warp raised the abort flag.  A poll may
// itself block for a hardware-defined while, so time is measured, not counted -- but lazily, because
// most waits end within a few polls and reading the timer costs as much as several of them: the clock
// is first read at poll 256 (for limits below a millisecond: at the second poll) and the limit counts
// from that reading.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int32_t* abort_flag,
                                          uint64_t limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint32_t every = limit_ns < 1000000ull ? 0u : 255u;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & every) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}
// Records a wait that ran out: sticky flag, first failing site, CTA-wide abort.
__device__ __forceinline__ void wait_failed(const DecodeParams& p, volatile int32_t* abort_flag, int site) {
    *abort_flag = 1;
    atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagWaitLimit);
    atomicCAS(p.hdr + kHdrWaitSite, 0, site);
}
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, int32_t row, uint32_t bar,
                                              int32_t plane = 0) {
    // box {64 elements, P rows, 2 halves} at coordinates {0, row, plane}
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(row), "r"(plane), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}
// 16 bytes global -> shared, asynchronously, past L1 (one per lane: 512 B per warp instruction).
__device__ __forceinline__ void lane_copy16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// One arrival on the mbarrier once every lane_copy16 this thread issued before has landed.  The
// arrival is not added to the barrier's expected count: the count it was initialised with
// must include one per thread that executes this.
__device__ __forceinline__ void lane_copy_arrive(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^x on the FMA and integer pipes, for x <= 127 (anything below -126, -inf included, gives ~2^-126):
// x = n + f with n the nearest integer (the 1.5 * 2^23 trick leaves n in the low mantissa bits) and
// |f| <= 1/2; 2^f by a degree-4 polynomial (relative error 4e-5, far inside what a bf16 probability
// keeps); n goes into the exponent field by an integer add.  Used for a share of a softmax tile's
// exponentials so that they do not all queue on the special-function unit (4 lanes per clock and SM
// sub-partition against 32 for an FMA).
__device__ __forceinline__ float exp2_fma(float x) {
    x = fmaxf(x, -126.f);
    const float t = x + 12582912.f;                       // 1.5 * 2^23: rounds x to an integer
    const float f = x - (t - 12582912.f);
    float r = fmaf(f, 0.0096181291f, 0.0555041087f);
    r = fmaf(r, f, 0.2402265070f);
    r = fmaf(r, f, 0.6931471806f);
    r = fmaf(r, f, 1.0f);
    return __uint_as_float(__float_as_uint(r) + (__float_as_uint(t) << 23));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}


}  // namespace concur
