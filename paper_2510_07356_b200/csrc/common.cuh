// Shared declarations of the decode-attention kernels: the per-call parameter block,
// the workspace layout and the range -> segment arithmetic of the split-KV plan.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace concur {

constexpr int kHq = 64;          // most query heads
constexpr int kHkv = 8;          // most KV heads (workspace capacities); a call's count is DecodeParams::hkv
constexpr int kGroup = 8;        // most query heads per KV head; width of every partial slot
constexpr int kD = 128;          // head dimension
constexpr int kTile = 64;        // tokens per KV tile: the unit the plan counts in
constexpr int kRowBytes = kD * 2;

constexpr uint32_t kFlagBadPage = 1u;
constexpr uint32_t kFlagBadLen = 2u;
constexpr uint32_t kFlagWaitLimit = 4u;
constexpr uint32_t kFlagBadGroup = 8u;
constexpr uint32_t kFlagBounds = 16u;       // checked build only: an index the kernels computed fell outside its buffer

// Workspace header (int32 words).
enum HeaderWord : int {
    kHdrTotalTiles = 0,   // W: sum over (sequence, KV head) of ceil(len / 64)
    kHdrNumRanges = 1,    // R: ranges the flat tile index space [0, W) is cut into
    kHdrClaim = 2,        // next range to hand out (atomic)
    kHdrStatus = 3,       // sticky CONCUR_FLAG_* bits
    kHdrWaitSite = 4,     // which wait gave up first (diagnostic; 0 = none)
    kHdrClaimSelf = 5,    // launches without a plan kernel: ranges claimed so far beyond one per CTA; the
                          // launch's last claim puts it back to 0
    kHdrBoundsSite = 7,   // checked build: which check failed first (diagnostic; 0 = none)
    kHdrWords = 64
};

// Everything a launch needs.  Pointers are device pointers.
struct DecodeParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_pages;
    const __nv_bfloat16* v_pages;
    const int32_t* block_table;
    const int32_t* seq_lens;
    __nv_bfloat16* out;
    float* lse;
    float scale_log2e;        // scale * log2(e): scores are kept in the base-2 domain
    int32_t batch;
    int32_t num_pages;
    int32_t bt_stride;
    int32_t page_size;
    int32_t page_shift;       // log2(page_size)
    int32_t box_rows;         // rows of one TMA box = min(page_size, 64): a 64-token tile is 64 / box_rows boxes
    int32_t box_shift;        // log2(box_rows)
    int32_t lane_copy;        // tensor-core partial kernel, box_rows < 64: 1 = tiles are brought in by per-lane
                              // 16-byte asynchronous copies instead of one TMA box per (page, head) chunk
    int32_t token_major;      // 0: pools are [page][KV head][slot][D]; 1: [page][slot][KV head][D]
    int32_t group;            // query heads per KV head (1..kGroup); heads g*group .. g*group+group-1 share KV head g
    int32_t hkv;              // KV heads of the pools and of k_new / v_new: 1, 2, 4 or 8
    int32_t hq;               // query heads = hkv * group
    // plan controls
    int32_t grid_ctas;        // CTAs the partial kernel is launched with
    int32_t forced_ranges;    // > 0: use exactly this many ranges (clamped to [1, min(W, max_ranges)])
    int32_t ranges_per_cta;
    int32_t min_range_tiles;
    int32_t max_ranges;       // capacity of range_start / partial slots
    // capacities, for the checked build (-DCONCUR_BOUNDS) to hold computed indices against
    int32_t slot_cap;         // partial slots that part_o / part_lse hold
    int64_t out_rows;         // rows ([Hq-indexed]) of out / lse
    int32_t fuse_combine;     // tensor-core kernel: 1 = the last partial of a unit merges it in-kernel
    int32_t claim_ahead;      // tiles before a range's end at which the next range is claimed
    int32_t no_plan_launch;   // tensor-core partial kernel: 1 = no plan kernel ran before this launch.  Ranges are
                              // claimed from kHdrClaimSelf, which the launch's last claim resets; the CTA that merges
                              // a unit puts the unit's ticket counter back to 0; CTA 0 writes the results of empty
                              // sequences, the bad-length flag, W, R and the range table
    int32_t overlap_next;     // 1 = let the next launch on the stream (if it allows programmatic launch) start
                              // while this one drains
    int64_t wait_limit_ns;    // tensor-core partial kernel: after this long a role's wait gives up (flag, abort, return)
    // workspace
    int32_t* hdr;             // [kHdrWords]
    int32_t* tiles_prefix;    // [batch + 1] exclusive prefix of per-sequence tile counts
    int32_t* range_start;     // [R + 1] boundaries in flat tile space
    float* part_o;            // [2 * max_ranges][kGroup][kD] normalised partial outputs
    float* part_lse;          // [2 * max_ranges][kGroup]     base-2 log-sum-exp of each partial
    int32_t* unit_done;       // [batch * hkv] partial segments finished per (sequence, KV head) unit
    // shared-prefix (cascade) mode; both unset in the plain path
    // fused append (tensor-core partial kernel): the K / V rows [batch][hkv][D] of each sequence's LAST token
    // (position seq_lens[b] - 1) are taken from here instead of the pools, and stored into the pools by the
    // CTA that streams the tile they belong to; both null in every other call
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    const int32_t* tok_offset; // [batch] first token of each sequence that this pass covers (multiple of 64), or null
    int32_t all_partial;      // 1: every segment writes a partial into slot r + u (u = b * hkv + g)
};

constexpr int kMaxShare = 10;     // siblings of a group that share one read of their common prefix

// Shared-prefix (cascade) decode: groups of consecutive sequences whose first tokens are the
// same cached pages.  Device pointers.
struct CascadeParams {
    const int32_t* group_start;   // [num_groups + 1] first sequence of each group; last entry = batch
    const int32_t* prefix_lens;   // [num_groups] tokens the group's sequences have in common
    int32_t num_groups;
    int32_t grid_ctas;
    int32_t* chdr;                // [kHdrWords] W', R', claim counter of the prefix pass
    int32_t* tok_offset;          // [batch] shared tokens handled by the prefix pass (0 if none)
    int32_t* seq_group;           // [batch] group of each sequence
    int32_t* ptiles_prefix;       // [num_groups + 1] exclusive prefix of shared tiles per group
    int32_t* unit_rowbase;        // [num_groups * hkv + 1] first partial row of each prefix unit
    int32_t max_rows;             // rows that pre_o / pre_lse hold (checked build)
    float* pre_o;                 // [rows][kGroup][kD] normalised partials of the prefix pass; rows = 8 x max batch
                                  // + 10 x CTAs: every unit's siblings once, plus once more per range cut
    float* pre_lse;               // [rows][kGroup]     their base-2 log-sum-exp
};

// Prefill (several query tokens per sequence, causal).  Device pointer.
struct PrefillParams {
    const int32_t* q_start;       // [batch + 1] first query token of each sequence in q / out; last entry = total_q
    int32_t total_q;
    int32_t block;                // query tokens per unit of the kernel that runs: 16 (one tile of rows) or 32 (two)
};

// The checked build (-DCONCUR_BOUNDS) in place of a memory checker: every index a kernel computes for the
// workspace, the partial buffers or the outputs is held against its buffer's capacity first; a violation is
// recorded (CONCUR_FLAG_BOUNDS and the site of the first one) and the access is skipped instead of made.  In
// the normal build the check is the constant `true` and costs nothing.
#ifdef CONCUR_BOUNDS
__device__ __forceinline__ bool in_bounds(int32_t* hdr, int64_t idx, int64_t cap, int site) {
    if (idx >= 0 && idx < cap) return true;
    atomicOr(reinterpret_cast<unsigned int*>(hdr + kHdrStatus), kFlagBounds);
    atomicCAS(hdr + kHdrBoundsSite, 0, site);
    return false;
}
#else
__device__ __forceinline__ bool in_bounds(int32_t*, int64_t, int64_t, int) { return true; }
#endif

// Where token `slot` of KV head g of page `page` sits, as the (row, half-plane) coordinates of the
// tensor maps over a pool (a row is 64 elements of one half of one 128-wide K or V row; `half` is
// added to the plane by the caller) and as an element offset for plain loads and stores.
__device__ __forceinline__ int32_t pool_row(const DecodeParams& p, int32_t page, int32_t g, int32_t slot) {
    return p.token_major ? page * p.page_size + slot : (page * p.hkv + g) * p.page_size + slot;
}
__device__ __forceinline__ int32_t pool_plane(const DecodeParams& p, int32_t g) { return p.token_major ? 2 * g : 0; }
__device__ __forceinline__ int64_t pool_elem(const DecodeParams& p, int32_t page, int32_t g, int32_t slot) {
    return p.token_major ? (((int64_t)page * p.page_size + slot) * p.hkv + g) * kD
                         : (((int64_t)page * p.hkv + g) * p.page_size + slot) * kD;
}

// Number of split-KV ranges for W flat tiles: as many as keeps every CTA supplied `ranges_per_cta`
// times over, but none shorter than `min_range_tiles`; or the forced count.  One definition, because
// the plan kernel and a partial kernel that plans for itself must arrive at the same number.
// `max_tiles` is the tile count of the longest sequence.
__device__ __forceinline__ int32_t plan_num_ranges(const DecodeParams& p, int32_t W, int32_t max_tiles) {
    int32_t R;
    if (p.forced_ranges > 0) {
        R = p.forced_ranges;
    } else {
        R = W / p.min_range_tiles;
        // Ranges per CTA: the caller's, or (0) one -- but two for a skewed batch (the longest sequence
        // four times the mean or more) with 64 tiles or more left per range.  Ranges hold equal
        // numbers of tiles, but every (sequence, KV head) unit that ends inside one also costs a merge
        // worth about three tiles; when unit lengths differ much, so do these sums, and a CTA that
        // finishes early then takes a second range off one that does not.  On even batches the
        // second range only costs its start-up.
        const bool skewed = (int64_t)max_tiles * p.hkv * p.batch >= 4 * (int64_t)W;
        const int32_t per_cta = p.ranges_per_cta > 0 ? p.ranges_per_cta
                                                     : (skewed && W >= p.grid_ctas * 2 * 64 ? 2 : 1);
        const int32_t cap = p.grid_ctas * per_cta;
        if (R > cap) R = cap;
    }
    if (R > p.max_ranges) R = p.max_ranges;
    if (R > W) R = W;
    if (R < 1 && W > 0) R = 1;
    return R;
}

// First flat tile of range r when [0, W) is cut into R ranges of equal size.
__device__ __forceinline__ int32_t range_begin(int32_t W, int32_t R, int32_t r) {
    return (int32_t)(((int64_t)W * r) / R);
}

// The range that contains flat tile x (0 <= x < W), by arithmetic alone.
__device__ __forceinline__ int32_t range_of(int32_t W, int32_t R, int32_t x) {
    int32_t r = (int32_t)(((int64_t)x * R) / W);
    while (r + 1 < R && range_begin(W, R, r + 1) <= x) ++r;
    while (r > 0 && range_begin(W, R, r) > x) --r;
    return r;
}

// The flat tile space lists, for sequence b = 0.., KV head g = 0..hkv-1, that unit's tiles:
// unit (b, g) occupies [hkv * prefix[b] + g * tiles_b, ... + tiles_b).
struct Segment {
    int32_t b, g;
    int32_t tile0, tile1;     // tiles of the unit covered by this segment, [tile0, tile1)
    int32_t tiles_b;          // tiles of the whole unit
    int32_t slot;             // partial slot, or -1 when the segment covers the whole unit
};

// Largest b in [0, batch) with hkv * prefix[b] <= x  (x < W).
__device__ __forceinline__ int32_t find_sequence(const int32_t* __restrict__ prefix, int32_t batch, int32_t x,
                                                 int32_t hkv) {
    int32_t lo = 0, hi = batch;            // invariant: hkv*prefix[lo] <= x < hkv*prefix[hi]
    while (hi - lo > 1) {
        int32_t mid = (lo + hi) >> 1;
        if (hkv * prefix[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// Largest r in [0, R) with range_start[r] <= x  (x < W).
__device__ __forceinline__ int32_t find_range(const int32_t* __restrict__ range_start, int32_t R, int32_t x) {
    int32_t lo = 0, hi = R;
    while (hi - lo > 1) {
        int32_t mid = (lo + hi) >> 1;
        if (range_start[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// Segment of range r that starts at flat tile x (range_start[r] <= x < range_start[r+1]).
__device__ __forceinline__ Segment segment_at(const int32_t* __restrict__ prefix, int32_t batch, int32_t hkv,
                                              int32_t r, int32_t x0, int32_t x1, int32_t x,
                                              int32_t all_partial = 0) {
    Segment s;
    s.b = find_sequence(prefix, batch, x, hkv);
    int32_t base = hkv * prefix[s.b];
    s.tiles_b = prefix[s.b + 1] - prefix[s.b];
    s.g = (x - base) / s.tiles_b;
    int32_t unit_start = base + s.g * s.tiles_b;
    int32_t unit_end = unit_start + s.tiles_b;
    int32_t end = x1 < unit_end ? x1 : unit_end;
    s.tile0 = x - unit_start;
    s.tile1 = end - unit_start;
    bool whole = (s.tile0 == 0) && (s.tile1 == s.tiles_b);
    s.slot = whole ? -1 : 2 * r + (x > x0 ? 1 : 0);
    // cascade mode: every segment is a partial; (range, unit) pairs grow strictly along the flat
    // tile space, so r + u is a unique slot below R + batch * hkv
    if (all_partial) s.slot = r + s.b * hkv + s.g;
    return s;
}

// Host-side launchers (each enqueues on `stream` and returns the launch status).
cudaError_t launch_plan(const DecodeParams& p, cudaStream_t stream);
cudaError_t launch_partial_scalar(const DecodeParams& p, cudaStream_t stream);
struct RowsMapCache;
cudaError_t launch_partial_mma(const DecodeParams& p, cudaStream_t stream, RowsMapCache* maps = nullptr);
cudaError_t launch_combine(const DecodeParams& p, cudaStream_t stream);
cudaError_t launch_plan_cascade(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream);
cudaError_t launch_prefix_mma(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream);
cudaError_t launch_prefix_tc(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream);
cudaError_t launch_prefill_tc(const DecodeParams& p, const PrefillParams& f, int pair, cudaStream_t stream);
cudaError_t launch_prefill_pair(const DecodeParams& p, const PrefillParams& f, cudaStream_t stream);
int prefill_pair_block();
cudaError_t launch_combine_cascade(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream);
int partial_scalar_ctas_per_sm();
cudaError_t launch_append(const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                          const int32_t* block_table, int32_t* seq_lens, int32_t* hdr, int32_t batch,
                          int32_t num_pages, int32_t bt_stride, int32_t page_size, int32_t page_shift,
                          int32_t token_major, int32_t hkv, int32_t advance, cudaStream_t stream);

}  // namespace concur
