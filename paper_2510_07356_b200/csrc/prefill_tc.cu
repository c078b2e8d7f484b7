// Causal prefill attention on the 5th-generation tensor cores, two query tiles per CTA.
//
// A unit is (sequence, block of 32 query tokens, KV head): 32 tokens x the 8 query heads of the KV
// head = two tiles of 128 accumulator rows (tile A = tokens 0..15 of the block, tile B = tokens
// 16..31; row = 8 x token + head).  Both tiles stream the same K/V of that KV head, in STEPS of 128
// tokens, so every byte that reaches shared memory feeds two products and every tcgen05.mma has
// N = 128 (one instruction takes as long with N = 64 as with N = 128, so 64-token products leave half
// of the pipe idle):
//
//   S_t[128 x 128] = Q_t[128 x 128] . K_step^T          8 MMAs of K = 16, operands in shared memory
//   online softmax, one thread per row and 64-column half: P = 2^(S - m) as packed bf16, written over
//                 the first 32 of the thread's own 64 score columns
//   O_t[128 x 128] += P_t[128 x 128] . V_step            8 MMAs of K = 16, P from TMEM
//
// TMEM (512 columns): S_A [0,128), S_B [128,256), O_A [256,384), O_B [384,512).  There is no room for
// a second score buffer per tile, so a tile's chain is Q.K^T -> softmax -> P.V -> next Q.K^T; what keeps
// the tensor pipe and the special-function unit busy is the OTHER tile, which must be in the opposite
// phase.  One thread issues the products of both tiles in the order Q.K^T_A(j), P.V_B(j-1), Q.K^T_B(j),
// P.V_A(j), which holds the tiles half a step apart.  (With one issuing warp per tile the tiles fell into
// lockstep within a dozen steps, even when started apart: 7,200 clocks per step, both units idle two
// thirds of the time.)
//
// The softmax of one row is a serial chain (TMEM load, maximum, exponentials at 4 per clock and SM
// sub-partition, pack, store), and with one score buffer per tile that chain sits between two products
// of the tile.  So a row has TWO threads, one per 64-column half of the step, in warps w and w + 4 (a warp
// may touch the TMEM lanes 32 (w % 4) .. + 31 only): they exchange the maxima of their halves through
// shared memory, take the same decision about the row's reference, each sums its own half (the two sums
// are added at the end of the unit) and each looks after 64 of the 128 columns of the row's O.
//
// Warp roles: warps 0-7 softmax of tile A (0-3 columns 0..63, 4-7 columns 64..127), warps 8-15 of tile B,
// warp 16 producer (page table, step records, TMA copies issued by up to 8 lanes at once), warp 17 issues
// the MMAs (one lane; owns the TMEM allocation).
//
// A row's O is rescaled in TMEM only when a step raises its maximum by more than a fixed slack over the
// reference its probabilities are scaled with.
//
// Causality: token i of the unit sees columns c <= diag + i of a step.  A tile that sees at most 64
// columns of a step skips the second half (exponentials and P.V); one that sees none (tile A on the last
// step when the block straddles a step boundary, tile B of a block with at most 16 live tokens) skips
// the step.  Both sides take that decision from the step's record by the same function.
//
// Every wait is bounded (see mbar_wait); a wait that runs out raises the CTA-wide abort flag, all roles
// fall through to the common exit and the TMEM allocation is released there.  Every tcgen05.ld / st
// sits under warp-uniform conditions only.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"
#include "tensor_map.cuh"

namespace concur {

namespace {

constexpr int kPStep = 128;                               // tokens per step
constexpr int kPTileTok = 16;                             // query tokens per tile
constexpr int kPRows = 128;                               // MMA M
constexpr int kPKStages = 2, kPVStages = 3;
constexpr int kPSlab = kPStep * 128;                      // 16 KB: 128 rows of one 64-dim half, or one 64-token V tile
constexpr int kPStageBytes = 2 * kPSlab;                  // 32 KB: K or V of one step
constexpr int kPQTileBytes = 2 * kPRows * 128;            // 32 KB: one query tile, [half][128 rows][128 B]
constexpr int kPMetaRing = 8;                             // step records; readers trail the producer by < 4
constexpr int kPProducerWarp = 16;
constexpr int kPMmaWarp = 17;                             // issues every MMA; owns the TMEM allocation
constexpr int kPThreads = 18 * 32;                        // 96 registers per thread; the softmax loop is written to fit (see there)
constexpr uint32_t kPTmemCols = 512;
constexpr uint32_t kPTmemO = 256;                         // S_t at 128 t, O_t at 256 + 128 t

struct PMeta {
    int32_t n;            // live query tokens of the unit (1..32); 0 = no more work
    int32_t idx, cnt;     // index of the step in its unit, steps of the unit
    int32_t row;          // first query token of the unit (row of q / out divided by the number of query heads)
    int32_t g;            // KV head
    int32_t diag;         // token i of the unit sees columns c <= diag + i of the step
    int32_t nvalid;       // tokens of the step that exist and that some row may see (1..128)
    int32_t pad;
};
static_assert(sizeof(PMeta) == 32, "one record per 32 bytes");

// Shared memory, from a 1024-byte aligned base.
struct PSmem {
    static constexpr int kVOff = kPKStages * kPStageBytes;
    static constexpr int kQOff = kVOff + kPVStages * kPStageBytes;        // two query tiles
    static constexpr int kXchOff = kQOff + 2 * kPQTileBytes;              // [tile][half][128 rows] floats
    static constexpr int kMetaOff = kXchOff + 2 * 2 * kPRows * 4;
    static constexpr int kBarOff = kMetaOff + kPMetaRing * (int)sizeof(PMeta);
    // full_k, empty_k per K stage; full_v, empty_v per V stage; meta_full per record; q_full, q_empty;
    // per tile: s_full, p_full, pv_done, o_free; per tile and warp pair: xch
    static constexpr int kNumBars = 2 * kPKStages + 2 * kPVStages + kPMetaRing + 2 + 8 + 8;
    static constexpr int kTmemPtrOff = kBarOff + kNumBars * 8;
    static constexpr int kAbortOff = kTmemPtrOff + 8;
    static constexpr int kTotal = kAbortOff + 8;
    // The rings, the query tiles and the exchange buffer leave no room for alignment slack: the kernel
    // declares its dynamic shared memory 1024-byte aligned, checks the address it gets and gives up with a
    // flag (nothing else touched) should it ever not be.
    static constexpr int kBytes = kTotal;
};
static_assert(PSmem::kVOff % 1024 == 0 && PSmem::kQOff % 1024 == 0 && kPSlab % 1024 == 0,
              "operand slabs must be 1024-byte aligned");
static_assert(PSmem::kBytes <= 232448, "exceeds the 227 KB a CTA may use");
// Extents of what the tensor-core descriptors read, against the rings:
//   Q.K^T: A = 128 rows x 128 B from the start of each half of a query tile, B = 128 token rows x 128 B from
//   the start of each half of a K stage, the K = 16 steps up to 96 B further in; P.V: per K = 16 step 16
//   token rows (2,048 B) of both 8 KB halves of one of the stage's two 64-token tiles.
static_assert(2 * kPSlab == kPStageBytes && kPQTileBytes == 2 * kPSlab && 4 * 2048 == kPSlab / 2,
              "a stage is two slabs; a V tile is two 64-row halves of four 16-token steps");
static_assert(4 * 128 == (int)kPTmemCols, "two score buffers and two accumulators fill the 512 columns");

__device__ __forceinline__ void tma_load_box(uint32_t dst, const CUtensorMap* map, int32_t row, int32_t plane,
                                             uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(row), "r"(plane), "r"(bar) : "memory");
}

// A bounded wait whose outcome is the same for every lane: the warp-wide tcgen05 instructions that follow a
// wait must never be reached by a part of a warp.  Twenty warps share four schedulers here and most of them
// are waiting at any moment, so a poll carries a suspend-time hint: the hardware may park the thread until
// the phase completes (or for that long) instead of returning at once to a loop that takes issue slots from
// the warps that compute.
constexpr uint32_t kPollHintNs = 20000;
__device__ __forceinline__ bool try_wait_parked(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kPollHintNs) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool test_wait_now(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int32_t* abort_flag) {
    // (most waits of the issuing warp find their phase complete: ask without parking first)
    bool done = test_wait_now(bar, parity);
    if (!done) done = try_wait_parked(bar, parity);
    if (!done) {
        uint64_t t0 = 0;
        for (uint32_t it = 1;; ++it) {
            if (try_wait_parked(bar, parity)) { done = true; break; }
            if ((it & 15u) == 0) {
                if (*abort_flag) break;
                const uint64_t now = global_timer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > kWaitLimitNs) break;
            }
        }
    }
    return __all_sync(0xffffffffu, done);
}

// Live query tokens of tile t, and how many columns of a step at least one of its rows sees.
__device__ __forceinline__ int32_t tile_tokens(int32_t n, int t) {
    return min(max(n - t * kPTileTok, 0), kPTileTok);
}
__device__ __forceinline__ int32_t tile_cols(int32_t n, int t, int32_t diag, int32_t nvalid) {
    const int32_t nt = tile_tokens(n, t);
    return nt > 0 ? min(max(diag + t * kPTileTok + nt, 0), nvalid) : 0;
}
// Whether a step that tile t takes is the last one it takes in its unit: the unit's last step, or the next
// step (whose diag is 128 lower) shows the tile nothing.
__device__ __forceinline__ bool tile_last(int32_t n, int t, int32_t diag, int32_t idx, int32_t cnt) {
    return idx == cnt - 1 || diag - kPStep + t * kPTileTok + tile_tokens(n, t) <= 0;
}

}  // namespace

__global__ void __launch_bounds__(kPThreads, 1)
prefill_pair_kernel(DecodeParams p, PrefillParams f, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q) {
    using SM = PSmem;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    const uint32_t smem_base = smem_u32(smem);
    if (smem_base & 1023u) {                                     // (uniform over the CTA: nobody goes on)
        if (threadIdx.x == 0) {
            atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagWaitLimit);
            atomicCAS(p.hdr + kHdrWaitSite, 0, 50);
        }
        return;
    }
    float* xch = reinterpret_cast<float*>(smem + SM::kXchOff);
    PMeta* meta = reinterpret_cast<PMeta*>(smem + SM::kMetaOff);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(smem + SM::kAbortOff);
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(smem + SM::kTmemPtrOff);
    const uint32_t bar_base = smem_base + SM::kBarOff;
    constexpr int kB0 = 2 * kPKStages + 2 * kPVStages + kPMetaRing;
    auto full_k = [&](int s) { return bar_base + 8u * s; };
    auto empty_k = [&](int s) { return bar_base + 8u * (kPKStages + s); };
    auto full_v = [&](int s) { return bar_base + 8u * (2 * kPKStages + s); };
    auto empty_v = [&](int s) { return bar_base + 8u * (2 * kPKStages + kPVStages + s); };
    auto meta_full = [&](int s) { return bar_base + 8u * (2 * kPKStages + 2 * kPVStages + s); };
    const uint32_t q_full = bar_base + 8u * kB0, q_empty = q_full + 8u;
    auto s_full = [&](int t) { return bar_base + 8u * (kB0 + 2 + t); };
    auto p_full = [&](int t) { return bar_base + 8u * (kB0 + 4 + t); };
    auto pv_done = [&](int t) { return bar_base + 8u * (kB0 + 6 + t); };
    auto o_free = [&](int t) { return bar_base + 8u * (kB0 + 8 + t); };
    auto xch_bar = [&](int pair) { return bar_base + 8u * (kB0 + 10 + pair); };   // pair = 4 tile + warp % 4

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;

    // query rows of tokens that do not exist must at least be defined once
    for (int i = tid; i < 2 * kPQTileBytes / 16; i += kPThreads)
        reinterpret_cast<uint4*>(smem + SM::kQOff)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        // a stage is released once, by whoever is last to read it (tile B if it takes the step, else tile A)
        for (int s = 0; s < kPKStages; ++s) { mbar_init(full_k(s), 1); mbar_init(empty_k(s), 1); }
        for (int s = 0; s < kPVStages; ++s) { mbar_init(full_v(s), 1); mbar_init(empty_v(s), 1); }
        for (int s = 0; s < kPMetaRing; ++s) mbar_init(meta_full(s), 1);
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);                                   // one commit after the unit's last Q.K^T
        for (int t = 0; t < 2; ++t) {
            mbar_init(s_full(t), 1);
            // (arrivals of a softmax warp are made by one lane after a warp-wide sync: 256 arrivals on one
            // barrier are 256 shared-memory atomics in a row, behind which everything else the SM's
            // load/store path has to do queues up)
            mbar_init(p_full(t), 8);
            mbar_init(pv_done(t), 1);
            mbar_init(o_free(t), 8);
        }
        for (int i = 0; i < 8; ++i) mbar_init(xch_bar(i), 2);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == kPMmaWarp) tmem_alloc(smem_base + SM::kTmemPtrOff, kPTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr;
    // everything above overlaps the plan kernel when launched as its programmatic dependent; the plan's
    // outputs are read only below this wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int32_t W = p.hdr[kHdrTotalTiles];                     // units

    if (warp == kPProducerWarp) {
        // =========================================================== producer warp
        const int32_t R = p.box_rows;                            // token rows per TMA box (<= 64)
        const int32_t page_mask = p.page_size - 1;
        const uint32_t box_bytes = (uint32_t)R * 128u;           // one half of one box
        uint32_t it = 0, segs = 0;                               // steps, units issued
        int ks = 0, vs = 0;                                      // it % kPKStages, (it - 1) % kPVStages
        uint32_t kpar = 0, vpar = 0;
        bool ok = true, q_inflight = false;
        // lane q < 8 keeps the coordinates of box q of the latest step: its V is requested one step later
        int32_t v_row = 0, v_plane = 0, v_nbox = 0;
        bool v_pending = false;
        auto issue_v = [&]() {
            ok = warp_wait(empty_v(vs), vpar ^ 1u, abort_flag);
            if (!ok) return;
            if (lane == 0) mbar_arrive_expect_tx(full_v(vs), (uint32_t)v_nbox * 2u * box_bytes);
            __syncwarp();
            if (lane < v_nbox) {
                const int32_t t0 = lane * R;                     // first token of the box inside the step
                const uint32_t dst = smem_base + SM::kVOff + vs * kPStageBytes + (uint32_t)(t0 >> 6) * kPSlab +
                                     (uint32_t)(t0 & 63) * 128u;
                tma_load_box(dst, &map_v, v_row, v_plane, full_v(vs));
                tma_load_box(dst + kPSlab / 2, &map_v, v_row, v_plane + 1, full_v(vs));
            }
            v_pending = false;
            if (++vs == kPVStages) { vs = 0; vpar ^= 1u; }
        };
        int32_t r = blockIdx.x;
        const int64_t max_len = (int64_t)p.bt_stride * p.page_size;
        while (ok && r < W) {
            int32_t r_next = 0;
            if (lane == 0) r_next = atomicAdd(p.hdr + kHdrClaim, 1);
            // unit r = (sequence b, block qb of 32 query tokens, KV head g); the blocks of a sequence are
            // taken last first (they have the most steps)
            const int32_t b = find_sequence(p.tiles_prefix, p.batch, r, p.hkv);
            const int32_t local = r - p.hkv * p.tiles_prefix[b];
            const int32_t nqb = p.tiles_prefix[b + 1] - p.tiles_prefix[b];
            const int32_t qb = nqb - 1 - local / p.hkv, g = local % p.hkv;
            int64_t len = p.seq_lens[b];
            len = len < 0 ? 0 : (len > max_len ? max_len : len);
            int32_t q_len = f.q_start[b + 1] - f.q_start[b];
            if (q_len > (int32_t)len) q_len = (int32_t)len;                     // flagged by the plan
            const int32_t tok0 = qb * f.block;
            const int32_t n = min(f.block, q_len - tok0);
            const int32_t pos0 = (int32_t)len - q_len + tok0;
            const int32_t tok_end = pos0 + n;                                   // tokens some row sees
            const int32_t nsteps = (tok_end + kPStep - 1) / kPStep;
            const int32_t qrow0 = f.q_start[b] + tok0;
            const int32_t* table = p.block_table + (int64_t)b * p.bt_stride;
            const int32_t page_end = (tok_end + page_mask) >> p.page_shift;
            int32_t chunk_base = 0;
            int32_t pg = (lane < page_end) ? __ldg(table + lane) : 0;
            int32_t pg_next = (32 + lane < page_end) ? __ldg(table + 32 + lane) : 0;
            for (int32_t s = 0; ok && s < nsteps; ++s) {
                const int32_t step0 = s * kPStep;
                const int32_t first_page = step0 >> p.page_shift;
                if (first_page >= chunk_base + 32) {
                    chunk_base += 32;
                    pg = pg_next;
                    pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                }
                const int32_t nvalid = min(kPStep, tok_end - step0);
                const int32_t nbox = (nvalid + R - 1) >> p.box_shift;           // boxes of the step that are read
                // lane q's box: tokens step0 + q R ..; with 128-token pages two boxes share a page
                const int32_t box_tok = step0 + (lane & 7) * R;
                int32_t my_page = __shfl_sync(0xffffffffu, pg, ((box_tok >> p.page_shift) - chunk_base) & 31);
                const bool bad = (lane < nbox) && (my_page < 0 || my_page >= p.num_pages);
                if (__any_sync(0xffffffffu, bad)) {
                    if (lane == 0) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagBadPage);
                    if (my_page < 0 || my_page >= p.num_pages) my_page = 0;
                }
                const int32_t my_row = pool_row(p, my_page, g, box_tok & page_mask);
                const int32_t my_plane = pool_plane(p, g);
                ok = warp_wait(empty_k(ks), kpar ^ 1u, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    PMeta& m = meta[it % kPMetaRing];
                    m.n = n; m.idx = s; m.cnt = nsteps; m.row = qrow0; m.g = g;
                    m.diag = min(pos0 - step0, 1 << 20); m.nvalid = nvalid;
                    mbar_arrive(meta_full(it % kPMetaRing));
                    mbar_arrive_expect_tx(full_k(ks), (uint32_t)nbox * 2u * box_bytes);
                }
                __syncwarp();
                if (lane < nbox) {
                    // K of a step is one K-major slab per 64-dim half: [half][128 tokens][128 B]
                    const uint32_t dst = smem_base + ks * kPStageBytes + (uint32_t)(lane * R) * 128u;
                    tma_load_box(dst, &map_k, my_row, my_plane, full_k(ks));
                    tma_load_box(dst + kPSlab, &map_k, my_row, my_plane + 1, full_k(ks));
                }
                // V of the previous step, before anything that waits for the issuing warp: at a unit's first step the
                // wait below ends with the previous unit's last Q.K^T, and that unit's last products need this V
                if (v_pending) { issue_v(); if (!ok) break; }
                if (s == 0) {
                    // the unit's query rows: token j's 8 rows go to rows 8 (j % 16) .. + 7 of both halves of tile j / 16
                    ok = warp_wait(q_empty, (segs & 1u) ^ 1u, abort_flag);
                    if (!ok) break;
                    if (lane == 0) mbar_arrive_expect_tx(q_full, (uint32_t)n * kGroup * kRowBytes);
                    __syncwarp();
                    if (lane < n) {
                        const int32_t qrow = (qrow0 + lane) * p.hq + g * p.group;
                        const uint32_t dst = smem_base + SM::kQOff + (uint32_t)(lane >> 4) * kPQTileBytes +
                                             (uint32_t)(lane & 15) * 1024u;
                        tma_load_box(dst, &map_q, qrow, 0, q_full);
                        tma_load_box(dst + kPSlab, &map_q, qrow, 1, q_full);
                    }
                    q_inflight = true;
                    ++segs;
                }
                v_row = my_row; v_plane = my_plane; v_nbox = nbox; v_pending = true;
                ++it;
                if (++ks == kPKStages) { ks = 0; kpar ^= 1u; }
            }
            r = __shfl_sync(0xffffffffu, r_next, 0);
        }
        if (ok && v_pending) issue_v();                          // the last step's V
        if (ok) ok = warp_wait(empty_k(ks), kpar ^ 1u, abort_flag);
        if (ok && lane == 0) {
            meta[it % kPMetaRing].n = 0;                         // no more work
            mbar_arrive(meta_full(it % kPMetaRing));
            mbar_arrive(full_k(ks));                             // the issuing warp reads records through the K barriers
        }
        if (!ok && lane == 0) {
            wait_failed(p, abort_flag, 51);
            // let the copies still in flight land before the CTA's shared memory is released
            volatile int32_t never = 0;
            for (uint32_t j = it > (uint32_t)kPKStages ? it - kPKStages : 0u; j < it; ++j)
                mbar_wait(full_k(j % kPKStages), (j / kPKStages) & 1u, &never);
            const uint32_t vt = v_pending ? it - 1 : it;         // V steps requested so far
            for (uint32_t j = vt > (uint32_t)kPVStages ? vt - kPVStages : 0u; j < vt; ++j)
                mbar_wait(full_v(j % kPVStages), (j / kPVStages) & 1u, &never);
            if (q_inflight) mbar_wait(q_full, (segs - 1) & 1u, &never);
        }
        __syncwarp();
    } else if (warp == kPMmaWarp) {
        // =========================================================== issuing warp (one lane issues)
        // One thread issues the products of both tiles, in a fixed order that puts the tiles half a step apart:
        //     Q.K^T_A(j)   P.V_B(j-1)   Q.K^T_B(j)   P.V_A(j)   Q.K^T_A(j+1)   ...
        // so that tile A's rows are in their softmax while the pipe works for tile B and the other way round.
        // (With an issuing warp per tile nothing keeps the tiles apart: they drift into lockstep within a
        // dozen steps, collide on the tensor pipe and on the special-function unit, and each of these then
        // idles two thirds of the time.)  tcgen05.mma instructions of one thread execute in the order issued,
        // so the next Q.K^T of a tile, which overwrites the P it was just multiplied with, needs no wait for
        // that product.  The whole warp runs the loop so that addresses and descriptors stay warp-uniform.
        constexpr uint32_t idesc_qk = umma_idesc_bf16(kPRows, kPStep, false, false);
        constexpr uint32_t idesc_pv = umma_idesc_bf16(kPRows, kD, false, true);
        bool ok = true;
        int site = 0;
        uint32_t kp[2] = {0, 0};                                 // steps taken per tile (parity of p_full)
        uint32_t segs = 0;                                       // units ended
        // o_free(t) is arrived at only by tiles that had live rows in the unit (a tile without any runs ahead
        // of this warp, from record to record, and would put the barrier more than one phase ahead)
        uint32_t ofree[2] = {0, 0};                              // phases of o_free(t) consumed
        int32_t prev_n = 0;                                      // live tokens of the previous unit
        int ks = 0, vs = 0;
        uint32_t kpar = 0, vpar = 0;
        // tile B's product of the previous step, still to be issued
        bool pend = false, pend_first = false, pend_last = false, pend_wait_v = false;
        int pend_vs = 0;
        uint32_t pend_vpar = 0;
        int32_t pend_cols = 0, pend_nvalid = 0;
        // P.V of tile t over V stage `st`: waits for V and for the tile's probabilities
        auto issue_pv = [&](int t, int st, uint32_t stpar, int32_t ncols, int32_t nvalid, bool first, bool wait_v) -> bool {
            // (a satisfied wait still costs this warp some 200 clocks, and it is the busiest role: V is waited
            // for once per step, by the tile that reads it first)
            if (wait_v && !warp_wait(full_v(st), stpar, abort_flag)) { site = 56; return false; }
            const uint32_t v_addr = smem_base + SM::kVOff + st * kPStageBytes;
            const int32_t used = ncols > 64 ? kPStep : 64;       // token rows this tile's product reads
            if (nvalid < used) {
                // rows past the last token may hold anything (NaN included, or another step's data where no
                // page was read) and a zero probability does not silence them inside an MMA: clear them in
                // both halves first
                for (int i = lane; i < (used - nvalid) * 16; i += 32) {
                    const int rowi = nvalid + (i >> 4), c16 = i & 15;
                    const uint32_t addr = v_addr + (uint32_t)(rowi >> 6) * kPSlab + (uint32_t)(c16 >> 3) * (kPSlab / 2) +
                                          (uint32_t)(rowi & 63) * 128u + (uint32_t)((c16 & 7) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }
            if (!warp_wait(p_full(t), kp[t] & 1u, abort_flag)) { site = 57; return false; }
            ++kp[t];
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t s_col = tmem_base + 128u * t, o_col = tmem_base + kPTmemO + 128u * t;
                // tokens 0..63: P in columns [0, 32) of S_t; tokens 64..127: P in columns [64, 96)
                #pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    // the first product of a unit overwrites the accumulator
                    umma_ts(o_col, s_col + kk * 8, umma_smem_desc(v_addr + kk * 2048, kPSlab / 2, 1024), idesc_pv,
                            (first && kk == 0) ? 0u : 1u);
                if (ncols > 64) {
                    #pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_ts(o_col, s_col + 64 + kk * 8, umma_smem_desc(v_addr + kPSlab + kk * 2048, kPSlab / 2, 1024),
                                idesc_pv, 1u);
                }
            }
            __syncwarp();
            return true;
        };
        auto issue_qk = [&](int t, int st) {
            const uint32_t k_addr = smem_base + st * kPStageBytes;
            const uint32_t q_addr = smem_base + SM::kQOff + t * kPQTileBytes;
            if (lane == 0) {
                #pragma unroll
                for (int k16 = 0; k16 < 8; ++k16) {
                    const uint32_t off = (uint32_t)(k16 >> 2) * kPSlab + (uint32_t)(k16 & 3) * 32u;
                    umma_ss(tmem_base + 128u * t, umma_smem_desc(q_addr + off, 16, 1024),
                            umma_smem_desc(k_addr + off, 16, 1024), idesc_qk, k16 > 0);
                }
                umma_commit(s_full(t));            // (the K stage is released by a softmax thread that sees this)
            }
            __syncwarp();
        };
        auto flush_pending = [&]() -> bool {
            if (!pend) return true;
            if (!issue_pv(1, pend_vs, pend_vpar, pend_cols, pend_nvalid, pend_first, pend_wait_v)) return false;
            if (lane == 0) {
                umma_commit(empty_v(pend_vs));                   // both tiles are done with that step's V
                if (pend_last) umma_commit(pv_done(1));
            }
            __syncwarp();
            pend = false;
            return true;
        };
        // A step's record, and what each tile sees of the step
        struct Rec { int32_t n, idx, cnt, nvalid, diag, cols_a, cols_b; };
        // (the record was written before its K barrier was armed: having waited for K makes it visible, and
        // the end marker arrives the same way)
        auto fetch = [&](uint32_t it, Rec& r) -> bool {
            if (!warp_wait(full_k(ks), kpar, abort_flag)) { site = 54; return false; }
            const PMeta* mt = &meta[it % kPMetaRing];
            r.n = mt->n; r.idx = mt->idx; r.cnt = mt->cnt; r.nvalid = mt->nvalid; r.diag = mt->diag;
            r.cols_a = r.n ? tile_cols(r.n, 0, r.diag, r.nvalid) : 0;
            r.cols_b = r.n ? tile_cols(r.n, 1, r.diag, r.nvalid) : 0;
            return true;
        };
        for (uint32_t it = 0; ok; ++it) {
            Rec cur;
            if (!fetch(it, cur)) { ok = false; break; }
            if (cur.n == 0) break;
            if (cur.idx == 0) {
                // a unit starts: its queries must have landed; the previous unit's rows must have been read out
                // of O_A and their threads must be past the exchange of their sums (this unit's first step
                // reuses the exchange buffer)
                if (!warp_wait(q_full, segs & 1u, abort_flag)) { ok = false; site = 53; break; }
                if (tile_tokens(prev_n, 0) > 0) {
                    if (!warp_wait(o_free(0), ofree[0] & 1u, abort_flag)) { ok = false; site = 55; break; }
                    ++ofree[0];
                }
            }
            tc_fence_after_sync();
            if (cur.cols_a > 0) issue_qk(0, ks);
            if (!flush_pending()) { ok = false; break; }
            if (cur.idx == 0 && tile_tokens(prev_n, 1) > 0) {
                if (!warp_wait(o_free(1), ofree[1] & 1u, abort_flag)) { ok = false; site = 58; break; }
                ++ofree[1];
            }
            if (cur.cols_b > 0) issue_qk(1, ks);
            if (cur.idx == cur.cnt - 1 && lane == 0) umma_commit(q_empty);   // the last read of the unit's queries
            if (cur.cols_a > 0) {
                if (!issue_pv(0, vs, vpar, cur.cols_a, cur.nvalid, cur.idx == 0, true)) { ok = false; break; }
                if (lane == 0 && tile_last(cur.n, 0, cur.diag, cur.idx, cur.cnt)) umma_commit(pv_done(0));
                __syncwarp();
            }
            if (cur.cols_b > 0) {
                pend = true; pend_first = cur.idx == 0; pend_last = tile_last(cur.n, 1, cur.diag, cur.idx, cur.cnt);
                pend_vs = vs; pend_vpar = vpar; pend_cols = cur.cols_b; pend_nvalid = cur.nvalid;
                pend_wait_v = cur.cols_a == 0;
            } else {
                if (lane == 0) umma_commit(empty_v(vs));         // tile B does not read this step's V
                __syncwarp();
            }
            if (cur.idx == cur.cnt - 1) { ++segs; prev_n = cur.n; }
            if (++ks == kPKStages) { ks = 0; kpar ^= 1u; }
            if (++vs == kPVStages) { vs = 0; vpar ^= 1u; }
        }
        if (ok && !flush_pending()) ok = false;
        if (!ok && lane == 0) wait_failed(p, abort_flag, site);
        __syncwarp();
    } else if (warp < 16) {
        // =========================================================== softmax warps (thread = row x half of tile t)
        const int t = warp >> 3, h = (warp >> 2) & 1;
        const int row = ((warp & 3) << 5) | lane;
        const int j = row >> 3, head = row & 7;                  // token inside the tile, head of this row
        const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t s_mine = lane_base + 128u * t + 64u * h;  // this thread's 64 scores; its P goes over the first 32
        const uint32_t o_mine = lane_base + kPTmemO + 128u * t + 64u * h;   // the 64 columns of O it looks after
        float* x_mine = xch + (t * 2 + h) * kPRows + row;
        const float* x_other = xch + (t * 2 + (h ^ 1)) * kPRows + row;
        const uint32_t xbar = xch_bar(4 * t + (warp & 3));
        const bool first_thread = (tid & 255) == 0;              // one thread per tile
        const float sc = p.scale_log2e;
        const bool sc_neg = sc < 0.f;
        // The scale used for a row's probabilities is 2^-m_ref, where m_ref trails the true running maximum
        // by at most kSlack (in base-2 units): P stays below 2^kSlack, which bf16 and the fp32 sums hold
        // without loss, and O has to be rescaled in TMEM only when a step raises the maximum by more than that.
        // Both threads of a row hold the same m_ref; l is the sum over this thread's half only.
        constexpr float kSlack = 8.f;
        float m_ref = -INFINITY, l = 0.f;
        uint32_t k = 0, k_unit = 0, kx = 0, units = 0;           // steps taken in all / of this unit; exchanges; units taken part in
        int ks = 0;
        bool ok = true;
        int site = 0;
        for (uint32_t it = 0; ok; ++it) {
            if (!warp_wait(meta_full(it % kPMetaRing), (it / kPMetaRing) & 1u, abort_flag)) { ok = false; site = 60; break; }
            const PMeta mt = meta[it % kPMetaRing];
            if (mt.n == 0) break;
            const int32_t nt = tile_tokens(mt.n, t);
            const int32_t ncols = tile_cols(mt.n, t, mt.diag, mt.nvalid);
            const bool warp_live = (warp & 3) * 4 < nt;          // this warp (and its partner) holds rows of a live token
            if (ncols > 0) {
                if (!warp_wait(s_full(t), k & 1u, abort_flag)) { ok = false; site = 61; break; }
                // Q.K^T of this step is complete for this tile, and tile B's is issued after tile A's: the tile
                // that is last to read the K stage releases it
                if (first_thread && t == (tile_cols(mt.n, 1, mt.diag, mt.nvalid) > 0 ? 1 : 0)) mbar_arrive(empty_k(ks));
                tc_fence_after_sync();
                if (warp_live) {
                    const bool mine = h == 0 || ncols > 64;      // this half has columns that some row sees
                    const int limit = mt.diag + t * kPTileTok + j - 64 * h;   // this row sees columns 0 .. limit of the half
                    const bool masked = limit < 63;              // causal diagonal (or ragged last step)
                    // The 64 scores are read from TMEM twice, 32 at a time: once for the maximum, once for the
                    // exponentials.  Holding all 64 across the exchange below takes more registers than a thread
                    // of this kernel has (640 threads), and what spills goes to a local memory that the
                    // 227 KB of shared memory leave almost no L1 for.
                    float mx = -INFINITY;
                    if (mine) {
                        float e0 = sc_neg ? INFINITY : -INFINITY;    // extreme of raw score (x sign of the scale)
                        #pragma unroll
                        for (int part = 0; part < 2; ++part) {
                            uint32_t raw[32];
                            tmem_ld32(s_mine + 32 * part, raw);
                            tmem_wait_ld();
                            if (masked) {
                                // hidden K rows may hold anything: they leave the maximum by a select
                                #pragma unroll
                                for (int e = 0; e < 32; ++e)
                                    if (32 * part + e > limit) raw[e] = __float_as_uint(sc_neg ? INFINITY : -INFINITY);
                            }
                            float e1 = __uint_as_float(raw[0]);
                            if (!sc_neg) {
                                #pragma unroll
                                for (int e = 1; e < 31; e += 4) {
                                    asm("max.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[e])), "f"(__uint_as_float(raw[e + 1])));
                                    asm("max.f32 %0, %0, %1, %2;" : "+f"(e1) : "f"(__uint_as_float(raw[e + 2])), "f"(__uint_as_float(raw[e + 3])));
                                }
                                asm("max.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[29])), "f"(__uint_as_float(raw[30])));
                                asm("max.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(e1), "f"(__uint_as_float(raw[31])));
                            } else {
                                #pragma unroll
                                for (int e = 1; e < 31; e += 4) {
                                    asm("min.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[e])), "f"(__uint_as_float(raw[e + 1])));
                                    asm("min.f32 %0, %0, %1, %2;" : "+f"(e1) : "f"(__uint_as_float(raw[e + 2])), "f"(__uint_as_float(raw[e + 3])));
                                }
                                asm("min.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[29])), "f"(__uint_as_float(raw[30])));
                                asm("min.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(e1), "f"(__uint_as_float(raw[31])));
                            }
                        }
                        mx = e0 * sc;                            // (+-inf x scale of the matching sign: -inf when all is hidden)
                    }
                    // the row's maximum over the step: this half's and the partner's
                    *x_mine = mx;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(xbar);
                    if (!warp_wait(xbar, kx & 1u, abort_flag)) { ok = false; site = 62; }
                    ++kx;
                    mx = fmaxf(mx, *x_other);
                    // a row that has seen nothing so far (m_ref = -inf, l = 0, its O row zero or about to be
                    // overwritten) takes this step's maximum as its reference without any rescaling
                    const bool fresh = m_ref == -INFINITY;
                    const bool need = !fresh && mx > m_ref + kSlack;
                    const float m_use = (fresh || need) ? mx : m_ref;
                    const float alpha = need ? fast_exp2(m_ref - mx) : 1.f;
                    const float neg_m = (m_use == -INFINITY) ? 0.f : -m_use;   // still nothing seen: P = 0
                    const bool rescale = __any_sync(0xffffffffu, need);
                    float sum = 0.f;
                    if (mine) {
                        // the row's 64 probabilities of this half as bf16 pairs: the A operand of this half's P.V
                        float sum1 = 0.f;
                        #pragma unroll
                        for (int part = 0; part < 2; ++part) {
                            uint32_t raw[32];
                            tmem_ld32(s_mine + 32 * part, raw);
                            tmem_wait_ld();
                            uint32_t pk[16];
                            #pragma unroll
                            for (int e = 0; e < 16; ++e) {
                                float p0 = fast_exp2(fmaf(__uint_as_float(raw[2 * e]), sc, neg_m));
                                float p1 = fast_exp2(fmaf(__uint_as_float(raw[2 * e + 1]), sc, neg_m));
                                if (masked) {
                                    if (32 * part + 2 * e > limit) p0 = 0.f;
                                    if (32 * part + 2 * e + 1 > limit) p1 = 0.f;
                                }
                                sum += p0; sum1 += p1;
                                pk[e] = pack_bf16(p0, p1);
                            }
                            // (part 1's scores sit in columns 32 .. 63: part 0's probabilities, columns 0 .. 15, do not touch them)
                            tmem_st16(s_mine + 16 * part, pk);
                        }
                        sum += sum1;
                    }
                    if (rescale) {
                        // O_t holds everything up to the previous step, whose product is complete: this step's
                        // Q.K^T was issued after it.  Each thread of the row scales its 64 columns.
                        #pragma unroll
                        for (int cblk = 0; cblk < 2; ++cblk) {
                            uint32_t o[32];
                            tmem_ld32(o_mine + cblk * 32, o);
                            tmem_wait_ld();
                            #pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st32(o_mine + cblk * 32, o);
                        }
                    }
                    if (mine || rescale) tmem_wait_st();
                    l = fmaf(l, alpha, sum);
                    m_ref = m_use;
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(t));
                if (!ok) break;
                ++k; ++k_unit;
            }
            if (++ks == kPKStages) ks = 0;

            if (mt.idx == mt.cnt - 1) {
                // ---- the unit ends with this step: normalise and write this tile's rows of out / lse, each
                //      thread of a row 64 of the 128 columns
                bool live = false;
                float inv = 0.f;
                int64_t out_row = 0;
                if (k_unit > 0) {
                    // (the issuing warp commits to this barrier once per unit, after the tile's last product)
                    if (!warp_wait(pv_done(t), units & 1u, abort_flag)) { ok = false; site = 63; break; }
                    ++units;
                    tc_fence_after_sync();
                    if (warp_live) {
                        *x_mine = l;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(xbar);
                        if (!warp_wait(xbar, kx & 1u, abort_flag)) { ok = false; site = 64; }
                        ++kx;
                        const float l_row = l + *x_other;
                        inv = 1.f / l_row;
                        out_row = (int64_t)(mt.row + t * kPTileTok + j) * p.hq + mt.g * p.group + head;
                        live = j < nt && head < p.group && in_bounds(p.hdr, out_row, p.out_rows, 203);
                        if (live && h == 0) p.lse[out_row] = (m_ref + log2f(l_row)) * 0.6931471805599453f;
                        #pragma unroll
                        for (int cblk = 0; cblk < 2; ++cblk) {
                            uint32_t o[32];
                            tmem_ld32(o_mine + cblk * 32, o);
                            tmem_wait_ld();
                            if (cblk == 1) {
                                // everything this thread needs of O_t and of the exchange buffer is in registers:
                                // the next unit's first Q.K^T may be issued
                                tc_fence_before_sync();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(o_free(t));
                            }
                            if (live) {
                                uint4* od = reinterpret_cast<uint4*>(p.out + out_row * kD + 64 * h + cblk * 32);
                                #pragma unroll
                                for (int e = 0; e < 32; e += 8) {
                                    float v[8];
                                    #pragma unroll
                                    for (int q = 0; q < 8; ++q) v[q] = __uint_as_float(o[e + q]) * inv;
                                    od[e >> 3] = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]),
                                                            pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
                                }
                            }
                        }
                    }
                }
                if (nt > 0 && !(k_unit > 0 && warp_live)) {      // (a tile without live rows does not take part)
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(o_free(t));
                }
                if (!ok) break;
                m_ref = -INFINITY; l = 0.f; k_unit = 0;
            }
        }
        if (!ok && lane == 0) wait_failed(p, abort_flag, site);
        __syncwarp();
    }

    // ---- common exit: every role arrives here, then the allocating warp releases the TMEM
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kPMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kPTmemCols);
    }
}

// ------------------------------------------------------------------ host side

int prefill_pair_block() { return 2 * kPTileTok; }

cudaError_t launch_prefill_pair(const DecodeParams& p, const PrefillParams& f, cudaStream_t stream) {
    CUtensorMap mk, mv, mq;
    const uint64_t pool_rows = (uint64_t)p.num_pages * p.page_size * (p.token_major ? 1 : p.hkv);
    const uint32_t planes = p.token_major ? 2 * p.hkv : 2;
    if (!make_rows_map(&mk, p.k_pages, pool_rows, p.box_rows, 1, planes) ||
        !make_rows_map(&mv, p.v_pages, pool_rows, p.box_rows, 1, planes) ||
        !make_rows_map(&mq, p.q, (uint64_t)f.total_q * p.hq, kGroup, 1))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(prefill_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PSmem::kBytes);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.grid_ctas);
    cfg.blockDim = dim3(kPThreads);
    cfg.dynamicSmemBytes = PSmem::kBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_pair_kernel, p, f, mk, mv, mq);
}

}  // namespace concur
