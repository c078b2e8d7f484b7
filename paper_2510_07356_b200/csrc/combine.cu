// Log-sum-exp combine kernel: merges the partial results of every (sequence, KV head)
// unit that the plan split over several ranges, and writes the result of empty
// sequences.  Units computed by a single segment were written by the partial kernel.
//
//   L = log2 sum_s 2^{lse_s};   out = sum_s 2^{lse_s - L} * out_s;   lse = L * ln 2
#include "common.cuh"

namespace concur {

constexpr int kCombineThreads = kD;

__global__ void __launch_bounds__(kCombineThreads) combine_kernel(DecodeParams p) {
    const int b = blockIdx.x / kHkv, g = blockIdx.x % kHkv;
    const int d = threadIdx.x;
    const int32_t tiles_b = p.tiles_prefix[b + 1] - p.tiles_prefix[b];
    const int64_t row0 = (int64_t)b * kHq + g * kGroup;
    if (tiles_b == 0) {                       // no cached token: out = 0, lse = -inf
        for (int h = 0; h < kGroup; ++h) {
            p.out[(row0 + h) * kD + d] = __float2bfloat16_rn(0.f);
            if (d == 0) p.lse[row0 + h] = -INFINITY;
        }
        return;
    }
    const int32_t R = p.hdr[kHdrNumRanges];
    const int32_t unit_start = kHkv * p.tiles_prefix[b] + g * tiles_b;
    const int32_t unit_end = unit_start + tiles_b;
    const int32_t r_lo = find_range(p.range_start, R, unit_start);
    const int32_t r_hi = find_range(p.range_start, R, unit_end - 1);
    if (r_lo == r_hi) return;                 // one segment covered the unit
    // the unit's segment in range r is the range's first segment unless the range began
    // before the unit did (possible for r_lo only)
    const int32_t slot_lo = 2 * r_lo + (p.range_start[r_lo] < unit_start ? 1 : 0);
    for (int h = 0; h < kGroup; ++h) {
        float M = p.part_lse[(int64_t)slot_lo * kGroup + h];
        for (int32_t r = r_lo + 1; r <= r_hi; ++r)
            M = fmaxf(M, p.part_lse[(int64_t)(2 * r) * kGroup + h]);
        float Z = 0.f, acc = 0.f;
        for (int32_t r = r_lo; r <= r_hi; ++r) {
            const int64_t slot = (r == r_lo) ? slot_lo : 2 * r;
            const float w = exp2f(p.part_lse[slot * kGroup + h] - M);
            Z += w;
            acc = fmaf(w, p.part_o[(slot * kGroup + h) * kD + d], acc);
        }
        p.out[(row0 + h) * kD + d] = __float2bfloat16_rn(acc / Z);
        if (d == 0) p.lse[row0 + h] = (M + log2f(Z)) * 0.6931471805599453f;
    }
}

cudaError_t launch_combine(const DecodeParams& p, cudaStream_t stream) {
    combine_kernel<<<p.batch * kHkv, kCombineThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace concur
