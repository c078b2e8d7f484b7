// Log-sum-exp combine kernel: merges the partial results of every (sequence, KV head)
// unit that the plan split over several ranges, and writes the result of empty
// sequences.  Units computed by a single segment were written by the partial kernel.
//
//   L = log2 sum_s 2^{lse_s};   out = sum_s 2^{lse_s - L} * out_s;   lse = L * ln 2
#include "common.cuh"

namespace concur {

constexpr int kCombineThreads = kD;

__global__ void __launch_bounds__(kCombineThreads) combine_kernel(DecodeParams p) {
    const int b = blockIdx.x / p.hkv, g = blockIdx.x % p.hkv;
    const int d = threadIdx.x;
    const int32_t tiles_b = p.tiles_prefix[b + 1] - p.tiles_prefix[b];
    const int64_t row0 = (int64_t)b * p.hq + g * p.group;
    if (tiles_b == 0) {                       // no cached token: out = 0, lse = -inf
        for (int h = 0; h < p.group; ++h) {
            p.out[(row0 + h) * kD + d] = __float2bfloat16_rn(0.f);
            if (d == 0) p.lse[row0 + h] = -INFINITY;
        }
        return;
    }
    const int32_t R = p.hdr[kHdrNumRanges];
    const int32_t unit_start = p.hkv * p.tiles_prefix[b] + g * tiles_b;
    const int32_t unit_end = unit_start + tiles_b;
    const int32_t r_lo = find_range(p.range_start, R, unit_start);
    const int32_t r_hi = find_range(p.range_start, R, unit_end - 1);
    if (r_lo == r_hi) return;                 // one segment covered the unit
    // the unit's segment in range r is the range's first segment unless the range began
    // before the unit did (possible for r_lo only)
    const int32_t slot_lo = 2 * r_lo + (p.range_start[r_lo] < unit_start ? 1 : 0);
    if (!in_bounds(p.hdr, slot_lo, p.slot_cap, 501) || !in_bounds(p.hdr, 2 * r_hi, p.slot_cap, 502) ||
        !in_bounds(p.hdr, row0 + p.group - 1, p.out_rows, 503))
        return;
    for (int h = 0; h < p.group; ++h) {
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
    combine_kernel<<<p.batch * p.hkv, kCombineThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace concur

// ---------------------------------------------------------------------------------------
// Cascade combine: merges, for every (sequence, KV head) unit, the partials of its suffix
// pass (slot r + u for every range r that covers the unit) with the partials of its group's
// prefix pass (one row per split of the prefix unit and sharing sibling).  One pass with a
// running maximum; all 8 heads of the group are in flight at once.
namespace concur {

__global__ void __launch_bounds__(kCombineThreads) combine_cascade_kernel(DecodeParams p, CascadeParams c) {
    const int b = blockIdx.x / p.hkv, g = blockIdx.x % p.hkv;
    const int d = threadIdx.x;
    float mx[kGroup], z[kGroup], acc[kGroup];
    #pragma unroll
    for (int h = 0; h < kGroup; ++h) { mx[h] = -INFINITY; z[h] = 0.f; acc[h] = 0.f; }
    auto add = [&](const float* lse_row, const float* o_row) {
        float l8[kGroup], v[kGroup];
        #pragma unroll
        for (int h = 0; h < kGroup; ++h) { l8[h] = __ldcg(lse_row + h); v[h] = __ldcg(o_row + h * kD + d); }
        #pragma unroll
        for (int h = 0; h < kGroup; ++h) {
            const float mn = fmaxf(mx[h], l8[h]);
            const float a = exp2f(mx[h] - mn), w = exp2f(l8[h] - mn);
            mx[h] = mn;
            z[h] = fmaf(z[h], a, w);
            acc[h] = fmaf(acc[h], a, w * v[h]);
        }
    };
    // suffix pass
    const int32_t tiles_b = p.tiles_prefix[b + 1] - p.tiles_prefix[b];
    if (tiles_b > 0) {
        const int32_t W = p.hdr[kHdrTotalTiles], R = p.hdr[kHdrNumRanges];
        const int32_t unit_start = p.hkv * p.tiles_prefix[b] + g * tiles_b;
        const int32_t r_lo = range_of(W, R, unit_start), r_hi = range_of(W, R, unit_start + tiles_b - 1);
        for (int32_t r = r_lo; r <= r_hi; ++r) {
            const int64_t slot = (int64_t)r + b * p.hkv + g;
            if (!in_bounds(p.hdr, slot, p.slot_cap, 504)) continue;
            add(p.part_lse + slot * kGroup, p.part_o + slot * kGroup * kD);
        }
    }
    // prefix pass
    const int32_t i = c.seq_group[b];
    if (i >= 0 && c.tok_offset[b] > 0) {
        const int32_t t_i = c.ptiles_prefix[i + 1] - c.ptiles_prefix[i];
        const int32_t b0 = c.group_start[i];
        const int32_t n = min(c.group_start[i + 1] - b0, kMaxShare);
        const int32_t W = c.chdr[kHdrTotalTiles], R = c.chdr[kHdrNumRanges];
        const int32_t start = p.hkv * c.ptiles_prefix[i] + g * t_i;
        const int32_t splits = range_of(W, R, start + t_i - 1) - range_of(W, R, start) + 1;
        const int64_t row0 = c.unit_rowbase[i * p.hkv + g] + (b - b0);
        for (int32_t s = 0; s < splits; ++s) {
            const int64_t row = row0 + (int64_t)s * n;
            if (!in_bounds(p.hdr, row, c.max_rows, 505)) continue;
            add(c.pre_lse + row * kGroup, c.pre_o + row * kGroup * kD);
        }
    }
    const int64_t row0 = (int64_t)b * p.hq + g * p.group;
    #pragma unroll
    for (int h = 0; h < kGroup; ++h) {
        if (h >= p.group) break;
        const bool any = z[h] > 0.f;
        p.out[(row0 + h) * kD + d] = __float2bfloat16_rn(any ? acc[h] / z[h] : 0.f);
        if (d == 0) p.lse[row0 + h] = any ? (mx[h] + log2f(z[h])) * 0.6931471805599453f : -INFINITY;
    }
}

cudaError_t launch_combine_cascade(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream) {
    combine_cascade_kernel<<<p.batch * p.hkv, kCombineThreads, 0, stream>>>(p, c);
    return cudaGetLastError();
}

}  // namespace concur
