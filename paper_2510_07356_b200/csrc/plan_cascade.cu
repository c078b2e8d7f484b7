// Plan of the shared-prefix (cascade) step.
//
// Sequences come in groups of consecutive siblings (the samples drawn for one prompt) whose
// first `prefix_lens[i]` tokens are the same cached pages.  The step is cut in two passes:
//   prefix pass  one unit per (group, KV head): the shared tiles are streamed once and
//                multiplied with the query rows of up to kMaxShare siblings;
//   suffix pass  one unit per (sequence, KV head) over the tokens after the shared part.
// Both passes write log-sum-exp partials that the cascade combine kernel merges.  Only whole
// 64-token tiles are shared: the shared part is rounded down to a multiple of 64 (and to the
// shortest sibling), the remainder is read by every sibling in its suffix pass, so the result
// is exactly that of the plain step on the same tables.
#include "common.cuh"

namespace concur {

constexpr int kPlanThreads = 1024;

// Block-wide exclusive scan of one value per thread; returns the exclusive prefix and leaves
// the running total (including all earlier calls' carry) in *carry.
__device__ __forceinline__ int32_t block_exclusive_scan(int32_t v, int32_t* warp_sums, int32_t* carry) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t incl = v;
    #pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) warp_sums[warp] = incl;
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
    const int32_t base = *carry + (warp ? warp_sums[warp - 1] : 0);
    const int32_t excl = base + incl - v;
    __syncthreads();
    if (threadIdx.x == kPlanThreads - 1) *carry = base + incl;
    __syncthreads();
    return excl;
}

__global__ void __launch_bounds__(kPlanThreads) plan_cascade_kernel(DecodeParams p, CascadeParams c) {
    __shared__ int32_t warp_sums[32];
    __shared__ int32_t carry;
    __shared__ int32_t Rs, Ws;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int64_t max_len = (int64_t)p.bt_stride * p.page_size;
    uint32_t flags = 0;
    // the prefix-pass kernel is launched as this grid's programmatic dependent: its prologue may start now,
    // it waits for this grid to finish before it reads the plan
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- per group: shared tiles, and each member's offset / group id
    if (tid == 0) { carry = 0; c.ptiles_prefix[0] = 0; }
    for (int b = tid; b < p.batch; b += kPlanThreads) { c.tok_offset[b] = 0; c.seq_group[b] = -1; }
    // The group table is device data and may hold anything.  It is usable only if it is a partition
    // of [0, batch) into consecutive runs: 0 <= group_start[0], group_start[i] <= group_start[i+1],
    // group_start[num_groups] <= batch.  Then the groups are disjoint, a group's sharing siblings are
    // real sequences, and the prefix pass writes at most 8 * batch + 10 * (ranges - 1) partial rows,
    // which is what the workspace holds.  Any violation turns sharing off for the whole call (every
    // sequence reads all of its tokens itself: the plain step's result) and is flagged; the later
    // kernels read group_start only for groups that share tiles, i.e. never in that case.
    int bad = 0;
    for (int i = tid; i < c.num_groups; i += kPlanThreads) {
        const int32_t b0 = c.group_start[i], b1 = c.group_start[i + 1];
        bad |= (b0 < 0) | (b0 > b1) | (b1 > p.batch);
    }
    const bool groups_ok = __syncthreads_or(bad) == 0;
    if (!groups_ok) flags |= kFlagBadGroup;
    for (int base = 0; base < c.num_groups; base += kPlanThreads) {
        const int i = base + tid;
        int32_t tiles = 0;
        if (groups_ok && i < c.num_groups) {
            const int32_t b0 = c.group_start[i], b1 = c.group_start[i + 1];
            const int32_t n_share = min(b1 - b0, kMaxShare);
            int64_t shared = c.prefix_lens[i];
            if (shared < 0) { shared = 0; flags |= kFlagBadLen; }
            for (int b = b0; b < b0 + n_share; ++b) {           // never beyond the shortest sharing sibling
                int64_t len = p.seq_lens[b];
                len = len < 0 ? 0 : (len > max_len ? max_len : len);
                if (shared > len) { shared = len; flags |= kFlagBadLen; }
            }
            tiles = n_share >= 2 ? (int32_t)(shared / kTile) : 0;
            for (int b = b0; b < b1; ++b) {
                c.tok_offset[b] = (b - b0 < n_share) ? tiles * kTile : 0;
                c.seq_group[b] = i;
            }
        }
        const int32_t excl = block_exclusive_scan(tiles, warp_sums, &carry);
        if (i < c.num_groups) c.ptiles_prefix[i + 1] = excl + tiles;
    }
    __syncthreads();
    if (tid == 0) {
        const int32_t W = p.hkv * carry;                 // prefix pass: flat tile space
        int32_t R = W / 2;
        if (R > c.grid_ctas) R = c.grid_ctas;
        if (R < 1 && W > 0) R = 1;
        c.chdr[kHdrTotalTiles] = W;
        c.chdr[kHdrNumRanges] = R;
        c.chdr[kHdrClaim] = c.grid_ctas;
        Ws = W; Rs = R;
        carry = 0;
    }
    __syncthreads();

    // ---- per prefix unit (group, KV head): rows of partials = splits x sharing siblings
    const int32_t Wp = Ws, Rp = Rs;
    const int32_t units = c.num_groups * p.hkv;
    if (tid == 0) c.unit_rowbase[0] = 0;
    for (int base = 0; base < units; base += kPlanThreads) {
        const int u = base + tid;
        int32_t rows = 0;
        if (u < units) {
            const int i = u / p.hkv, g = u % p.hkv;
            const int32_t t = c.ptiles_prefix[i + 1] - c.ptiles_prefix[i];
            if (t > 0) {
                const int32_t start = p.hkv * c.ptiles_prefix[i] + g * t;
                const int32_t splits = range_of(Wp, Rp, start + t - 1) - range_of(Wp, Rp, start) + 1;
                const int32_t n_share = min(c.group_start[i + 1] - c.group_start[i], kMaxShare);
                rows = splits * n_share;
            }
        }
        const int32_t excl = block_exclusive_scan(rows, warp_sums, &carry);
        if (u < units) c.unit_rowbase[u + 1] = excl + rows;
    }
    __syncthreads();
    if (tid == 0) { carry = 0; p.tiles_prefix[0] = 0; }
    __syncthreads();

    // ---- per sequence: tiles of the suffix pass
    for (int base = 0; base < p.batch; base += kPlanThreads) {
        const int b = base + tid;
        int32_t tiles = 0;
        if (b < p.batch) {
            int64_t len = p.seq_lens[b];
            if (len < 0) { len = 0; flags |= kFlagBadLen; }
            if (len > max_len) { len = max_len; flags |= kFlagBadLen; }
            len -= c.tok_offset[b];
            if (len < 0) { len = 0; flags |= kFlagBadLen; }       // only with overlapping groups
            tiles = (int32_t)((len + kTile - 1) / kTile);
        }
        const int32_t excl = block_exclusive_scan(tiles, warp_sums, &carry);
        if (b < p.batch) p.tiles_prefix[b + 1] = excl + tiles;
    }
    if (flags) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), flags);
    __syncthreads();
    if (tid == 0) {
        const int32_t W = p.hkv * carry;
        int32_t R = p.forced_ranges > 0 ? p.forced_ranges : min(W / p.min_range_tiles, p.grid_ctas * (p.ranges_per_cta > 0 ? p.ranges_per_cta : 1));
        if (R > p.max_ranges) R = p.max_ranges;
        if (R > W) R = W;
        if (R < 1 && W > 0) R = 1;
        p.hdr[kHdrTotalTiles] = W;
        p.hdr[kHdrNumRanges] = R;
        p.hdr[kHdrClaim] = p.grid_ctas;
        Ws = W; Rs = R;
    }
    __syncthreads();
    const int64_t W = Ws;
    const int32_t R = Rs;
    for (int r = tid; r <= R; r += kPlanThreads)
        p.range_start[r] = (R > 0) ? (int32_t)((W * r) / R) : 0;
    (void)lane; (void)warp;
}

cudaError_t launch_plan_cascade(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream) {
    plan_cascade_kernel<<<1, kPlanThreads, 0, stream>>>(p, c);
    return cudaGetLastError();
}

}  // namespace concur
