// Plan kernel: per-sequence tile counts, their prefix sums, and the split-KV ranges.
//
// The KV cache of the batch is seen as one flat list of W = Hkv * sum_b ceil(len_b / 64)
// tiles (sequence-major, then KV head, then position).  The plan cuts [0, W) into R
// ranges of equal size (to within one tile).  CTAs of the partial kernel claim ranges
// one after another, so ragged context lengths balance over the SMs no matter how the
// lengths are distributed; a sequence is split exactly where a range boundary falls
// inside one of its (sequence, KV head) units.
#include "common.cuh"

namespace concur {

constexpr int kPlanThreads = 1024;

__global__ void __launch_bounds__(kPlanThreads) plan_kernel(DecodeParams p) {
    __shared__ int32_t warp_sums[kPlanThreads / 32];
    __shared__ int32_t carry_s;
    __shared__ int32_t max_s;
    __shared__ int32_t ranges_s;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    // lets a dependent launch (programmatic stream serialisation) start its prologue now; it
    // still waits for this grid to finish before it reads the plan
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) { carry_s = 0; max_s = 0; p.tiles_prefix[0] = 0; }
    __syncthreads();

    const int64_t max_len = (int64_t)p.bt_stride * p.page_size;
    uint32_t flags = 0;
    for (int base = 0; base < p.batch; base += kPlanThreads) {
        int b = base + tid;
        int32_t tiles = 0;
        if (b < p.batch) {
            int64_t len = p.seq_lens[b];
            if (len < 0) { len = 0; flags |= kFlagBadLen; }
            if (len > max_len) { len = max_len; flags |= kFlagBadLen; }
            tiles = (int32_t)((len + kTile - 1) / kTile);
        }
        // sequences without cached tokens get their result here (out = 0, lse = -inf): the
        // warp that found one writes it
        unsigned empties = __ballot_sync(0xffffffffu, p.out != nullptr && b < p.batch && tiles == 0);
        while (empties) {
            const int e = base + warp * 32 + (__ffs(empties) - 1);
            empties &= empties - 1;
            uint4* o = reinterpret_cast<uint4*>(p.out + (int64_t)e * p.hq * kD);
            for (int i = lane; i < p.hq * kD / 8; i += 32) o[i] = make_uint4(0, 0, 0, 0);
            for (int i = lane; i < p.hq; i += 32) p.lse[(int64_t)e * p.hq + i] = -INFINITY;
        }
        // the longest sequence (for the range-count heuristic)
        int32_t mx = tiles;
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0 && mx > 0) atomicMax(&max_s, mx);
        // inclusive scan over the block
        int32_t v = tiles;
        #pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int32_t n = __shfl_up_sync(0xffffffffu, v, o);
            if (lane >= o) v += n;
        }
        if (lane == 31) warp_sums[warp] = v;
        __syncthreads();
        if (warp == 0) {
            int32_t w = warp_sums[lane];
            #pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int32_t n = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += n;
            }
            warp_sums[lane] = w;
        }
        __syncthreads();
        int32_t incl = v + (warp ? warp_sums[warp - 1] : 0) + carry_s;
        if (b < p.batch) p.tiles_prefix[b + 1] = incl;
        __syncthreads();
        if (tid == kPlanThreads - 1) carry_s = incl;
        __syncthreads();
    }
    if (flags) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), flags);
    for (int i = tid; i < p.batch * p.hkv; i += kPlanThreads) p.unit_done[i] = 0;

    if (tid == 0) {
        const int32_t W = p.hkv * carry_s;
        const int32_t R = plan_num_ranges(p, W, max_s);
        p.hdr[kHdrTotalTiles] = W;
        p.hdr[kHdrNumRanges] = R;
        p.hdr[kHdrClaim] = p.grid_ctas;       // CTA i starts on range i; further ranges are claimed from here
        ranges_s = R;
    }
    __syncthreads();
    const int32_t R = ranges_s;
    const int64_t W = (int64_t)p.hkv * carry_s;
    for (int r = tid; r <= R; r += kPlanThreads)
        p.range_start[r] = (R > 0) ? (int32_t)((W * r) / R) : 0;
}

cudaError_t launch_plan(const DecodeParams& p, cudaStream_t stream) {
    plan_kernel<<<1, kPlanThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace concur
