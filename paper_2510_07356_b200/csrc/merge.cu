// Log-sum-exp merge of finished attention results: `parts` pairs (out bf16, lse fp32 natural log), each
// the result of the same query rows over a DIFFERENT part of the keys, into the result over all keys
//
//     L = ln sum_s exp(lse_s);   out = sum_s exp(lse_s - L) out_s;   a part with lse = -inf (no keys) weighs 0.
//
// This is the exchange step of context sharding: when one very long sequence's cache is spread over
// several GPUs, each GPU runs the decode step on its token range, the (out, lse) pairs -- 260 bytes per
// query row and GPU -- are gathered, and every GPU merges them with this kernel.  One warp per row, four
// dims per lane, one pass with a running maximum.
#include "../../include/concur_attn.h"

#include "common.cuh"
#include "ptx.cuh"

namespace concur {

constexpr int kMergeRowsPerBlock = 8;       // warps per block

__global__ void __launch_bounds__(kMergeRowsPerBlock * 32)
lse_merge_kernel(const __nv_bfloat16* __restrict__ outs, const float* __restrict__ lses, int32_t parts, int64_t rows,
                 __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const int64_t row = (int64_t)blockIdx.x * kMergeRowsPerBlock + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    float m = -INFINITY, z = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int32_t s = 0; s < parts; ++s) {
        const float l = lses[(int64_t)s * rows + row];
        if (l == -INFINITY) continue;                            // a part without keys (uniform over the warp)
        const uint2 raw = *reinterpret_cast<const uint2*>(outs + ((int64_t)s * rows + row) * kD + lane * 4);
        const float v0 = __uint_as_float(raw.x << 16), v1 = __uint_as_float(raw.x & 0xffff0000u);
        const float v2 = __uint_as_float(raw.y << 16), v3 = __uint_as_float(raw.y & 0xffff0000u);
        const float mn = fmaxf(m, l);
        const float a = __expf(m - mn), w = __expf(l - mn);      // exp(-inf) = 0 on the first part
        m = mn;
        z = fmaf(z, a, w);
        acc.x = fmaf(acc.x, a, w * v0); acc.y = fmaf(acc.y, a, w * v1);
        acc.z = fmaf(acc.z, a, w * v2); acc.w = fmaf(acc.w, a, w * v3);
    }
    const bool any = z > 0.f;
    const float inv = any ? 1.f / z : 0.f;
    *reinterpret_cast<uint2*>(out + row * kD + lane * 4) =
        make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
    if (lane == 0) lse[row] = any ? m + __logf(z) : -INFINITY;
}

}  // namespace concur

extern "C" int concur_lse_merge(const void* outs, const float* lses, int32_t parts, int64_t rows, void* out, float* lse,
                                void* cuda_stream) {
    if (parts < 1 || rows < 0) return CONCUR_ERR_INVALID_ARG;
    if (rows == 0) return CONCUR_OK;
    if (rows > ((int64_t)1 << 31) * concur::kMergeRowsPerBlock - 1) return CONCUR_ERR_TOO_LARGE;
    if (!outs || !lses || !out || !lse) return CONCUR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(outs) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u) ||
        (reinterpret_cast<uintptr_t>(lses) & 3u) || (reinterpret_cast<uintptr_t>(lse) & 3u))
        return CONCUR_ERR_INVALID_ARG;
    const unsigned blocks = (unsigned)((rows + concur::kMergeRowsPerBlock - 1) / concur::kMergeRowsPerBlock);
    concur::lse_merge_kernel<<<blocks, concur::kMergeRowsPerBlock * 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const __nv_bfloat16*>(outs), lses, parts, rows, static_cast<__nv_bfloat16*>(out), lse);
    if (cudaGetLastError() != cudaSuccess) return CONCUR_ERR_CUDA;
    return CONCUR_OK;
}
