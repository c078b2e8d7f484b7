// Attention of many query rows against one stream of K/V tiles on the 5th-generation tensor
// cores: the prefix pass of the shared-prefix (cascade) step and, with a causal mask, prefill.
// The description below is written for the prefix pass; what prefill changes is listed at TCfg.
//
// A unit is (group, KV head): the tiles that all siblings of a group have in common.  Each
// 64-token K/V tile is streamed from HBM once and multiplied with the query rows of all
// sharing siblings at once: n siblings x 8 heads of the GQA group = up to 80 rows, held as
// the 128-row A operand of tcgen05.mma (rows beyond 8n are never written out).  This is the
// one place of the decode step that is a dense contraction (80 flop per KV byte at ten
// siblings), so it runs on tcgen05 with its accumulators in tensor memory:
//
//   S[128 x 64]   = Q[128 x 128] . K_tile^T            (8 MMAs of K = 16; S in TMEM)
//   online softmax, one thread per row: thread t owns TMEM lane t = (sibling t / 8, head t % 8);
//                 it reads its 64 scores with tcgen05.ld, keeps the reference maximum and the sum
//                 in registers, and writes P = 2^(S - m) as packed bf16 back into TMEM
//   O[128 x 128] += P[128 x 64] . V_tile[64 x 128]     (4 MMAs of K = 16; O in TMEM, V is the
//                 MN-major B operand exactly as TMA laid it down)
//
// P never leaves TMEM (it is the A operand of P.V in the TS form).  The queries are the A operand of
// Q.K^T in the SS form, read straight from the staging buffer the TMA copies fill -- 8-row groups of
// 128-byte swizzled rows, which is the K-major operand layout as it stands.  (An earlier version
// copied them into TMEM once per segment; that saved 32 KB of operand reads per tile, which the
// tensor pipe does not miss, but tied the first product of a segment to the moment softmax group
// A had finished the previous segment.  With P in shared memory as well, the pipe spent ~1,100
// clocks per tile fetching operands.)
//
// One softmax warp per SM sub-partition is a serial chain (TMEM load, maximum, 64 exponentials
// at 4 per clock, pack, store, fences) of about 1,900 clocks per tile, which is below the HBM
// rate.  So there are TWO softmax warpgroups that take alternate tiles, each with its own
// P columns and O accumulator (TMEM columns: three score buffers, P_A, P_B, O_A, O_B); while one group
// is in its exponentials the other loads its scores.  At the end of a segment the two
// (m, l, O) states of every row are merged by their log-sum-exp, each group writing half of
// the output columns.
//
// A row's O is rescaled in TMEM (tcgen05.ld / st) only when a tile raises its maximum by more
// than a fixed slack over the reference its probabilities are scaled with, so in the steady
// state the softmax threads never touch O.
//
// Warp roles: warps 0-3 softmax group A, warps 4-7 softmax group B (a warp may touch the TMEM
// lanes 32 (w % 4) .. + 31), warp 8 TMA producer, warp 9 issues the Q.K^T MMAs (one thread) and
// owns the TMEM allocation, warp 10 issues the P.V MMAs.  One issuing thread for both was the
// bottleneck (about 90 clocks per tcgen05.mma and as much again in barrier waits and commits,
// all serial); the two products depend on different events (K landed and score buffer read,
// against P written and V landed), so each gets its own thread.  Tile i's scores go to score buffer
// i % 3, so Q.K^T of tile i is issued as soon as the scores of tile i - 3 (the other group's) have
// been read: a group's next scores are computed while it still works on its current tile.
//
// Input / output contract is that of the plan: a segment (the part of a unit inside one range)
// ends with one normalised fp32 partial (out, base-2 lse) per sibling in rows `row .. row + n`
// of pre_o / pre_lse, which the cascade combine kernel merges with the suffix partials.
//
// Every wait is bounded (see mbar_wait); a wait that runs out raises the CTA-wide abort flag,
// all roles fall through to the common exit and the TMEM allocation is released there.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"
#include "tensor_map.cuh"

namespace concur {

namespace {

// Two uses of the same pipeline.  Prefix pass of the cascade step: a row group is a sibling (up to
// kMaxShare = 10), every tile is whole and fully visible.  Prefill: a row group is a query token
// (16 per unit), the tiles on the diagonal are masked causally and the last one may be ragged.
constexpr int kTRows = 128;                               // MMA M

template <bool kPrefill>
struct TCfg {
    static constexpr int kShare = kPrefill ? 16 : kMaxShare;          // row groups (of 8 heads) per unit
    static constexpr int kKStages = kPrefill ? 4 : 5;                 // K ring: a stage is free again after Q.K^T
    static constexpr int kVStages = kPrefill ? 5 : 6;                 // V ring: a stage is free again after P.V
    static constexpr int kQRows = kShare * kGroup;                    // query rows that are really loaded
    static constexpr int kQHalfBytes = kQRows * 128;
    static constexpr int kQBytes = 2 * kQHalfBytes;                   // per staging buffer
    // Q.K^T reads its A operand straight from a staging buffer, always 128 rows of each half; where
    // fewer rows are staged the read runs on into what follows the half.  Behind the last half that
    // must still be this kernel's own, defined shared memory: a zeroed pad.
    static constexpr int kQPad = kTRows * 128 > kQHalfBytes ? kTRows * 128 - kQHalfBytes : 0;
    // A quarter of a tile's exponentials (the second of every other pair) is computed on the FMA pipe
    // in the prefix pass: measured 5 % faster there (0.212 -> 0.200 ms on a 16,384-token prompt shared by
    // ten).  Prefill, whose softmax threads are bound by instruction issue rather than by the
    // special-function unit, lost 3 % with a quarter and 10 % with a half, and keeps them all on that unit.
    static constexpr int kPolyEvery = kPrefill ? 0 : 2;           // 0: none
};
constexpr int kTVLag = 2;                                 // V of tile t is requested with K of tile t + 2
constexpr int kTMetaRing = 16;                            // tile records; readers trail the producer by < 8
constexpr int kTProducerWarp = 8;
constexpr int kTMmaWarp = 9;                              // issues Q.K^T, owns the TMEM allocation
constexpr int kTPvWarp = 10;                              // issues P.V
constexpr int kTThreads = 11 * 32;
constexpr int kTHalfBytes = kTile * 128;                  // 8 KB: 64 tokens x one 64-dim half
constexpr int kTTileBytes = 2 * kTHalfBytes;              // 16 KB: one K or V tile
// TMEM columns (512): three score buffers S_0 [64,128), S_1 [128,192), S_2 [0,64) used by tile
// it % 3; P_A [192,224), P_B [224,256) as packed bf16; O_A [256,384), O_B [384,512)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemP = 192, kTmemO = 256;
__host__ __device__ constexpr uint32_t tmem_s_col(uint32_t sb) { return sb == 2 ? 0u : 64u + 64u * sb; }


struct TMeta {
    int32_t n;            // live row groups (siblings / query tokens) of the segment; 0 = no more work
    int32_t idx, cnt;     // index of the tile in its segment, tiles of the segment
    int32_t qsel;         // query buffer of the segment
    int32_t row;          // prefix pass: first partial row of the segment; prefill: first query token
    int32_t g;            // KV head
    int32_t pages[4];     // physical pages of the tile (64 / P of them)
    int32_t nvalid;       // tokens of the tile that exist and that some row may see (1..64)
    int32_t diag;         // row group i sees columns c <= diag + i of the tile (>= 63: all of them)
    int32_t row_in_page;  // first row of the tile inside its page (non-zero only for pages of more than 64 tokens)
    int32_t pad[3];
};
static_assert(sizeof(TMeta) == 64, "one record per 64 bytes");

// Shared memory, from a 1024-byte aligned base.
template <bool kPrefill>
struct TSmem {
    using Cfg = TCfg<kPrefill>;
    static constexpr int kTKStages = Cfg::kKStages, kTVStages = Cfg::kVStages;
    static constexpr int kVOff = kTKStages * kTTileBytes;
    static constexpr int kQOff = kVOff + kTVStages * kTTileBytes;         // two staging buffers of the queries
    static constexpr int kXchOff = kQOff + 2 * Cfg::kQBytes + Cfg::kQPad; // [2 groups][128 rows] (m, l)
    static constexpr int kMetaOff = kXchOff + 2 * kTRows * 8;
    static constexpr int kBarOff = kMetaOff + kTMetaRing * (int)sizeof(TMeta);
    // full_k, empty_k per K stage; full_v, empty_v per V stage; meta_full per record; then pairs:
    // pairs q_full, q_empty, p_full, pv_done; xch_a, xch_b; triples s_full, s_free
    static constexpr int kNumBars = 2 * kTKStages + 2 * kTVStages + kTMetaRing + 20;
    static constexpr int kTmemPtrOff = kBarOff + kNumBars * 8;
    static constexpr int kAbortOff = kTmemPtrOff + 8;
    static constexpr int kTotal = kAbortOff + 8;
    static constexpr int kBytes = kTotal + 1024;
};
static_assert(TSmem<false>::kQOff % 1024 == 0 && TSmem<true>::kQOff % 1024 == 0 &&
              TCfg<false>::kQHalfBytes % 1024 == 0 && TCfg<true>::kQHalfBytes % 1024 == 0,
              "operand slabs must be 1024-byte aligned");
static_assert(TSmem<false>::kBytes <= 232448 && TSmem<true>::kBytes <= 232448, "exceeds the 227 KB a CTA may use");
// Extents of what the tensor-core descriptors read, against what the CTA owns.  (A 128-row operand read over
// 80 staged rows once ran 1.6 KB past the CTA's allocation; this is the arithmetic that would have caught it.)
//   Q.K^T, A operand: 128 rows x 128 B from the start of each half of a query buffer, the K = 16 steps up to 96 B
//   further in: the last buffer's second half must still have 128 rows of the CTA's memory behind it.
template <bool kPrefill>
constexpr int q_read_end() {
    return TSmem<kPrefill>::kQOff + TCfg<kPrefill>::kQBytes + TCfg<kPrefill>::kQHalfBytes + kTRows * 128;
}
static_assert(q_read_end<false>() <= TSmem<false>::kXchOff && q_read_end<true>() <= TSmem<true>::kXchOff,
              "the 128-row query operand read must end inside the query buffers and their pad");
//   Q.K^T, B operand: 64 token rows x 128 B per half of a K stage; P.V, B operand: per K = 16 step 16 token
//   rows (2,048 B) of both halves of a V stage.
static_assert(kTHalfBytes == kTile * 128 && 2 * kTHalfBytes == kTTileBytes && 4 * 2048 == kTHalfBytes,
              "a K or V stage is two 64-row halves; four 16-token steps span a half");
static_assert(TSmem<false>::kVOff == TCfg<false>::kKStages * kTTileBytes && TSmem<true>::kVOff == TCfg<true>::kKStages * kTTileBytes &&
              TSmem<false>::kQOff == TSmem<false>::kVOff + TCfg<false>::kVStages * kTTileBytes &&
              TSmem<true>::kQOff == TSmem<true>::kVOff + TCfg<true>::kVStages * kTTileBytes,
              "K ring, V ring and query buffers follow one another without overlap");
static_assert(64 + 64 + 64 + 32 + 32 + 128 + 128 == (int)kTmemCols, "three score buffers, two P tiles, two accumulators fill the 512 columns");

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1, int32_t c2,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}

}  // namespace

template <bool kPrefill>
__global__ void __launch_bounds__(kTThreads, 1)
attn_tc_kernel(DecodeParams p, CascadeParams c, PrefillParams f, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q) {
    using SM = TSmem<kPrefill>;
    using Cfg = TCfg<kPrefill>;
    constexpr int kTKStages = Cfg::kKStages, kTVStages = Cfg::kVStages;
    constexpr int kTQHalfBytes = Cfg::kQHalfBytes, kTQBytes = Cfg::kQBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    TMeta* meta = reinterpret_cast<TMeta*>(smem + SM::kMetaOff);
    float2* xch = reinterpret_cast<float2*>(smem + SM::kXchOff);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(smem + SM::kAbortOff);
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(smem + SM::kTmemPtrOff);
    const uint32_t bar_base = smem_base + SM::kBarOff;
    constexpr int kB0 = 2 * kTKStages + 2 * kTVStages + kTMetaRing;
    auto full_k = [&](int s) { return bar_base + 8u * s; };
    auto empty_k = [&](int s) { return bar_base + 8u * (kTKStages + s); };
    auto full_v = [&](int s) { return bar_base + 8u * (2 * kTKStages + s); };
    auto empty_v = [&](int s) { return bar_base + 8u * (2 * kTKStages + kTVStages + s); };
    auto meta_full = [&](int s) { return bar_base + 8u * (2 * kTKStages + 2 * kTVStages + s); };
    auto q_full = [&](int i) { return bar_base + 8u * (kB0 + i); };
    auto q_empty = [&](int i) { return bar_base + 8u * (kB0 + 2 + i); };
    auto s_full = [&](int i) { return bar_base + 8u * (kB0 + 14 + i); };   // per score buffer (3)
    auto s_free = [&](int i) { return bar_base + 8u * (kB0 + 17 + i); };
    auto p_full = [&](int i) { return bar_base + 8u * (kB0 + 8 + i); };
    auto pv_done = [&](int i) { return bar_base + 8u * (kB0 + 10 + i); };
    const uint32_t xch_a = bar_base + 8u * (kB0 + 12);               // both groups have published (m, l)
    const uint32_t xch_b = xch_a + 8u;                               // both groups have read both O

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int32_t P = p.box_rows;            // rows per box: the unit of the shared-memory tile layout

    // unused query rows must at least be defined once
    for (int i = tid; i < (2 * kTQBytes + Cfg::kQPad) / 16; i += kTThreads)
        reinterpret_cast<uint4*>(smem + SM::kQOff)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int s = 0; s < kTKStages; ++s) { mbar_init(full_k(s), 1); mbar_init(empty_k(s), 1); }
        for (int s = 0; s < kTVStages; ++s) { mbar_init(full_v(s), 1); mbar_init(empty_v(s), 1); }
        for (int s = 0; s < kTMetaRing; ++s) mbar_init(meta_full(s), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(q_full(i), 1);
            mbar_init(q_empty(i), 1);                            // one commit after the segment's last Q.K^T
            mbar_init(p_full(i), 128);
            mbar_init(pv_done(i), 1);
        }
        for (int i = 0; i < 3; ++i) { mbar_init(s_full(i), 1); mbar_init(s_free(i), 128); }
        mbar_init(xch_a, 256);
        mbar_init(xch_b, 256);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == kTMmaWarp) tmem_alloc(smem_base + SM::kTmemPtrOff, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr;
    // everything above (shared-memory set-up, TMEM allocation) overlaps the plan kernel when launched as
    // its programmatic dependent; the plan's outputs are read only below this wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // prefix pass: flat tile space and ranges of the cascade plan; prefill: W = number of units
    const int32_t W = kPrefill ? p.hdr[kHdrTotalTiles] : c.chdr[kHdrTotalTiles];
    const int32_t R = kPrefill ? 0 : c.chdr[kHdrNumRanges];

    if (warp == kTProducerWarp) {
        // =========================================================== producer warp
        uint32_t it = 0, vt = 0, seg = 0;                      // K tiles, V tiles, segments issued
        bool ok = true;
        const int32_t npages = kTile >> p.box_shift;           // boxes per tile
        const int32_t page_mask = p.page_size - 1;
        const uint32_t page_bytes = (uint32_t)P * 128u;        // one half of one page
        // V of tile u (lane 0 only): its pages are still in the tile's record
        auto issue_v = [&](uint32_t u) {
            const TMeta& m = meta[u % kTMetaRing];
            const int vs = u % kTVStages;
            ok = mbar_wait(empty_v(vs), ((u / kTVStages) & 1u) ^ 1u, abort_flag);
            if (!ok) return;
            const uint32_t vdst = smem_base + SM::kVOff + vs * kTTileBytes;
            const int32_t npg = (m.nvalid + P - 1) >> p.box_shift;       // boxes of the tile that are read
            if (npages == 1) {
                // page = tile: one box {64, 64, 2} lands as [half][row][128 B], the operand layout
                mbar_arrive_expect_tx(full_v(vs), kTTileBytes);
                tma_load_3d(vdst, &map_v, 0, pool_row(p, m.pages[0], m.g, m.row_in_page), pool_plane(p, m.g), full_v(vs));
            } else {
                mbar_arrive_expect_tx(full_v(vs), npg * 2 * page_bytes);
                #pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (q < npg) {
                        const int32_t prow = pool_row(p, m.pages[q], m.g, m.row_in_page), pl = pool_plane(p, m.g);
                        tma_load_3d(vdst + q * page_bytes, &map_v, 0, prow, pl, full_v(vs));
                        tma_load_3d(vdst + kTHalfBytes + q * page_bytes, &map_v, 0, prow, pl + 1, full_v(vs));
                    }
            }
            ++vt;
        };
        // One segment: tiles [tile0, tile1) of KV head g through the table row `table`, for `n` row
        // groups whose query rows are (qbase + j) * Hq + g * G.  pos0 / pos_last: positions of the
        // first and last row group (prefill; the prefix pass sees every token of its tiles).
        auto stream_segment = [&](const int32_t* table, int32_t g, int32_t tile0, int32_t tile1, int32_t n,
                                  int32_t row, int32_t qbase, int32_t pos0, int32_t pos_last) {
            const int32_t qsel = seg & 1;
            const int32_t tok_end = min(tile1 * kTile, pos_last + 1);
            const int32_t page_end = (tok_end + page_mask) >> p.page_shift;
            int32_t chunk_base = (tile0 * kTile) >> p.page_shift;
            int32_t pg = (chunk_base + lane < page_end) ? __ldg(table + chunk_base + lane) : 0;
            int32_t pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
            for (int32_t t = tile0; ok && t < tile1; ++t) {
                const int32_t first_page = (t * kTile) >> p.page_shift;
                const int32_t row_in_page = (t * kTile) & page_mask;
                if (first_page >= chunk_base + 32) {
                    chunk_base += 32;
                    pg = pg_next;
                    pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                }
                const int32_t nvalid = min(kTile, tok_end - t * kTile);
                const int32_t npg = (nvalid + P - 1) >> p.box_shift;           // boxes of the tile that are read
                const int ks = it % kTKStages;
                int32_t my_page = __shfl_sync(0xffffffffu, pg, (first_page - chunk_base + (lane & 3)) & 31);
                const bool bad = (lane < npg) && (my_page < 0 || my_page >= p.num_pages);
                if (__any_sync(0xffffffffu, bad)) {
                    if (lane == 0) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagBadPage);
                    if (my_page < 0 || my_page >= p.num_pages) my_page = 0;
                }
                const int32_t pages[4] = {__shfl_sync(0xffffffffu, my_page, 0), __shfl_sync(0xffffffffu, my_page, 1),
                                          __shfl_sync(0xffffffffu, my_page, 2), __shfl_sync(0xffffffffu, my_page, 3)};
                if (lane == 0) {
                    if (t == tile0) {
                        // the segment's query rows: row group j's 8 rows go to rows 8j .. 8j + 7 of both halves
                        ok = mbar_wait(q_empty(qsel), ((seg >> 1) & 1u) ^ 1u, abort_flag);
                        if (ok) {
                            mbar_arrive_expect_tx(q_full(qsel), n * kGroup * kRowBytes);
                            const uint32_t qdst = smem_base + SM::kQOff + qsel * kTQBytes;
                            for (int j = 0; j < n; ++j) {
                                const int32_t qrow = (qbase + j) * p.hq + g * p.group;
                                tma_load_3d(qdst + j * 1024, &map_q, 0, qrow, 0, q_full(qsel));
                                tma_load_3d(qdst + kTQHalfBytes + j * 1024, &map_q, 0, qrow, 1, q_full(qsel));
                            }
                        }
                    }
                    if (ok) ok = mbar_wait(empty_k(ks), ((it / kTKStages) & 1u) ^ 1u, abort_flag);
                    if (ok) {
                        TMeta& m = meta[it % kTMetaRing];
                        m.n = n; m.idx = t - tile0; m.cnt = tile1 - tile0; m.qsel = qsel; m.row = row; m.g = g;
                        m.pages[0] = pages[0]; m.pages[1] = pages[1]; m.pages[2] = pages[2]; m.pages[3] = pages[3];
                        m.nvalid = nvalid; m.row_in_page = row_in_page;
                        m.diag = kPrefill ? min(pos0 - t * kTile, 1 << 20) : (1 << 20);
                        mbar_arrive(meta_full(it % kTMetaRing));
                        const uint32_t kdst = smem_base + ks * kTTileBytes;
                        if (npages == 1) {
                            mbar_arrive_expect_tx(full_k(ks), kTTileBytes);
                            tma_load_3d(kdst, &map_k, 0, pool_row(p, pages[0], g, row_in_page), pool_plane(p, g), full_k(ks));
                        } else {
                            mbar_arrive_expect_tx(full_k(ks), npg * 2 * page_bytes);
                            #pragma unroll
                            for (int q = 0; q < 4; ++q)
                                if (q < npg) {
                                    const int32_t prow = pool_row(p, pages[q], g, row_in_page), pl = pool_plane(p, g);
                                    tma_load_3d(kdst + q * page_bytes, &map_k, 0, prow, pl, full_k(ks));
                                    tma_load_3d(kdst + kTHalfBytes + q * page_bytes, &map_k, 0, prow, pl + 1, full_k(ks));
                                }
                        }
                        if (it >= (uint32_t)kTVLag) issue_v(it - kTVLag);
                    }
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (ok) ++it;
            }
            ++seg;
        };
        int32_t r = blockIdx.x;
        if constexpr (!kPrefill) {
            while (ok && r < R) {
                int32_t r_next = 0;
                if (lane == 0) r_next = atomicAdd(c.chdr + kHdrClaim, 1);
                const int32_t x0 = range_begin(W, R, r), x1 = range_begin(W, R, r + 1);
                int32_t x = x0;
                while (ok && x < x1) {
                    // the prefix unit (group i, KV head g) that holds flat tile x
                    const int32_t i = find_sequence(c.ptiles_prefix, c.num_groups, x, p.hkv);
                    const int32_t t_i = c.ptiles_prefix[i + 1] - c.ptiles_prefix[i];
                    const int32_t base = p.hkv * c.ptiles_prefix[i];
                    const int32_t g = (x - base) / t_i;
                    const int32_t unit_start = base + g * t_i;
                    const int32_t tile0 = x - unit_start;
                    const int32_t tile1 = min(x1, unit_start + t_i) - unit_start;
                    x += tile1 - tile0;
                    const int32_t b0 = c.group_start[i];
                    const int32_t n = min(c.group_start[i + 1] - b0, kMaxShare);
                    const int32_t split = r - range_of(W, R, unit_start);
                    const int32_t row = c.unit_rowbase[i * p.hkv + g] + split * n;
                    // shared tiles are whole; they are read through the first sibling's table row
                    stream_segment(p.block_table + (int64_t)b0 * p.bt_stride, g, tile0, tile1, n, row, b0,
                                   1 << 28, tile1 * kTile - 1);
                }
                r = __shfl_sync(0xffffffffu, r_next, 0);
            }
        } else {
            // prefill: unit r = (sequence b, block of 16 query tokens, KV head g); the blocks of a
            // sequence are taken last first (they have the most tiles); a unit is never split
            const int64_t max_len = (int64_t)p.bt_stride * p.page_size;
            while (ok && r < W) {
                int32_t r_next = 0;
                if (lane == 0) r_next = atomicAdd(p.hdr + kHdrClaim, 1);
                const int32_t b = find_sequence(p.tiles_prefix, p.batch, r, p.hkv);
                const int32_t local = r - p.hkv * p.tiles_prefix[b];
                const int32_t nqb = p.tiles_prefix[b + 1] - p.tiles_prefix[b];
                const int32_t qb = nqb - 1 - local / p.hkv, g = local % p.hkv;
                int64_t len = p.seq_lens[b];
                len = len < 0 ? 0 : (len > max_len ? max_len : len);
                int32_t q_len = f.q_start[b + 1] - f.q_start[b];
                if (q_len > (int32_t)len) q_len = (int32_t)len;                 // flagged by the plan
                const int32_t tok0 = qb * Cfg::kShare;
                const int32_t n = min(Cfg::kShare, q_len - tok0);
                const int32_t pos0 = (int32_t)len - q_len + tok0;
                const int32_t pos_last = pos0 + n - 1;
                stream_segment(p.block_table + (int64_t)b * p.bt_stride, g, 0, pos_last / kTile + 1, n,
                               f.q_start[b] + tok0, f.q_start[b] + tok0, pos0, pos_last);
                r = __shfl_sync(0xffffffffu, r_next, 0);
            }
        }
        if (lane == 0) {
            while (ok && vt < it) issue_v(vt);                 // the last tiles' V
            if (ok) {
                const int ks = it % kTKStages;
                ok = mbar_wait(empty_k(ks), ((it / kTKStages) & 1u) ^ 1u, abort_flag);
                if (ok) {
                    meta[it % kTMetaRing].n = 0;               // no more work
                    mbar_arrive(meta_full(it % kTMetaRing));
                    mbar_arrive(full_k(ks));                   // the Q.K^T warp reads records through the K barriers
                }
            }
            if (!ok) {
                wait_failed(p, abort_flag, 31);
                // let the copies still in flight land before the CTA's shared memory is released
                volatile int32_t never = 0;
                for (uint32_t j = it > (uint32_t)kTKStages ? it - kTKStages : 0u; j < it; ++j)
                    mbar_wait(full_k(j % kTKStages), (j / kTKStages) & 1u, &never);
                for (uint32_t j = vt > (uint32_t)kTVStages ? vt - kTVStages : 0u; j < vt; ++j)
                    mbar_wait(full_v(j % kTVStages), (j / kTVStages) & 1u, &never);
            }
        }
    } else if (warp == kTMmaWarp) {
        // =========================================================== Q.K^T warp (one lane issues)
        // The whole warp runs the loop so that addresses and descriptors stay warp-uniform; the
        // MMAs and commits are issued by lane 0.  The tile's record was written before its K
        // barrier was armed, so waiting for K makes it visible; the end marker arrives the same way.
        {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kTRows, kTile, false, false);
            bool ok = true;
            int site = 0;
            uint32_t segs = 0;
            for (uint32_t it = 0; ok; ++it) {
                const int ks = it % kTKStages;
                if (!mbar_wait(full_k(ks), (it / kTKStages) & 1u, abort_flag)) { ok = false; site = 43; break; }
                const TMeta* mt = &meta[it % kTMetaRing];
                const int32_t idx = mt->idx, cnt = mt->cnt;
                if (mt->n == 0) break;
                if (idx == 0) {                               // a segment starts: its queries must have landed
                    if (!mbar_wait(q_full(mt->qsel), (segs >> 1) & 1u, abort_flag)) { ok = false; site = 33; break; }
                    ++segs;
                }
                // Three score buffers for two groups: tile `it` uses buffer it % 3, whose previous user
                // was tile it - 3 of the other group.  So this product does not wait for its own
                // group to have read the scores of its previous tile (it - 2): those sit in another
                // buffer, and a group's next scores are computed while it still works on the current
                // ones, however late it started on them.
                const uint32_t sb = it % 3u;
                if (!mbar_wait(s_free(sb), ((it / 3u) & 1u) ^ 1u, abort_flag)) { ok = false; site = 34; break; }
                tc_fence_after_sync();
                const uint32_t k_addr = smem_base + ks * kTTileBytes;
                const uint32_t q_addr = smem_base + SM::kQOff + mt->qsel * kTQBytes;
                if (lane == 0) {
                    #pragma unroll
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const uint32_t koff = (uint32_t)(k16 & 3) * 32u;
                        const uint64_t a = umma_smem_desc(q_addr + (k16 >> 2) * kTQHalfBytes + koff, 16, 1024);
                        const uint64_t b = umma_smem_desc(k_addr + (k16 >> 2) * kTHalfBytes + koff, 16, 1024);
                        umma_ss(tmem_base + tmem_s_col(sb), a, b, idesc_qk, k16 > 0);
                    }
                    umma_commit(s_full(sb));       // (the K stage is released by the softmax group that sees this)
                    if (idx == cnt - 1) umma_commit(q_empty(mt->qsel));   // the segment's last read of its queries
                }
                __syncwarp();
            }
            if (!ok && lane == 0) wait_failed(p, abort_flag, site);
        }
        __syncwarp();
    } else if (warp == kTPvWarp) {
        // =========================================================== P.V warp (one lane issues)
        {
            constexpr uint32_t idesc_pv = umma_idesc_bf16(kTRows, kD, false, true);
            bool ok = true;
            int site = 0;
            for (uint32_t u = 0; ok; ++u) {
                const int g = u & 1u;
                if (!mbar_wait(meta_full(u % kTMetaRing), (u / kTMetaRing) & 1u, abort_flag)) { ok = false; site = 46; break; }
                const TMeta* mt = &meta[u % kTMetaRing];
                const int32_t idx = mt->idx, nvalid = mt->nvalid;
                if (mt->n == 0) break;
                const int vs = u % kTVStages;
                if (!mbar_wait(p_full(g), (u >> 1) & 1u, abort_flag)) { ok = false; site = 35; break; }
                if (!mbar_wait(full_v(vs), (u / kTVStages) & 1u, abort_flag)) { ok = false; site = 36; break; }
                const uint32_t v_addr = smem_base + SM::kVOff + vs * kTTileBytes;
                if (nvalid < kTile) {
                    // rows past the last token may hold anything (NaN included, or another tile's data
                    // where no page was read) and a zero probability does not silence them inside an
                    // MMA: clear them in both halves first
                    for (int i = lane; i < (kTile - nvalid) * 16; i += 32) {
                        const int rowi = nvalid + (i >> 4), c16 = i & 15;
                        const uint32_t addr = v_addr + (uint32_t)(c16 >> 3) * kTHalfBytes + (uint32_t)rowi * 128u +
                                              (uint32_t)((c16 & 7) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
                tc_fence_after_sync();
                if (lane == 0) {
                    #pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t b = umma_smem_desc(v_addr + kk * 2048, kTHalfBytes, 1024);
                        // a group's first tile of a segment overwrites its accumulator
                        umma_ts(tmem_base + kTmemO + g * kD, tmem_base + kTmemP + g * 32 + kk * 8, b, idesc_pv,
                                (idx < 2 && kk == 0) ? 0u : 1u);
                    }
                    umma_commit(empty_v(vs));               // that V stage may be overwritten
                    umma_commit(pv_done(g));
                }
                __syncwarp();
            }
            if (!ok && lane == 0) wait_failed(p, abort_flag, site);
        }
        __syncwarp();
    } else {
        // =========================================================== softmax warps (thread = row)
        const int g = warp >> 2;                                 // group: tiles with (it & 1) == g
        const int row = tid & 127;
        const int j = row >> 3, head = row & 7;                  // sibling, head of this row
        const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t o_mine = lane_base + kTmemO + g * kD, o_other = lane_base + kTmemO + (g ^ 1) * kD;
        const float sc = p.scale_log2e;
        const bool sc_neg = sc < 0.f;
        // The scale used for a row's probabilities is 2^-m_ref, where m_ref trails the true running
        // maximum by at most kSlack (in base-2 units): P stays below 2^kSlack, which bf16 and the
        // fp32 sums hold without loss, and O has to be rescaled in TMEM only when a tile raises
        // the maximum by more than that -- a handful of times per segment instead of per tile.
        constexpr float kSlack = 8.f;
        float m_ref = -INFINITY, l = 0.f;
        uint32_t k = 0, segs = 0;                                // tiles this group has taken; segments ended
        bool ok = true;
        int site = 0;
        for (uint32_t it = 0; ok; ++it) {
            if (!mbar_wait(meta_full(it % kTMetaRing), (it / kTMetaRing) & 1u, abort_flag)) { ok = false; site = 37; break; }
            const TMeta mt = meta[it % kTMetaRing];
            if (mt.n == 0) break;
            const bool warp_live = (warp & 3) * 4 < mt.n;        // this warp holds rows of a sharing sibling
            const bool mine = (int)(it & 1u) == g;
            if (mine) {
                const bool first = mt.idx < 2;                   // this group's first tile of the segment
                const uint32_t sb = it % 3u;                     // the score buffer of this tile
                if (!mbar_wait(s_full(sb), (it / 3u) & 1u, abort_flag)) { ok = false; site = 38; break; }
                // Q.K^T of this tile is complete, so its K stage may be overwritten.  The release is a
                // plain arrival from a thread that learns of the completion anyway: a second
                // tcgen05.commit would cost the issuing thread about as much as an MMA.
                if (row == 0) mbar_arrive(empty_k(it % kTKStages));
                tc_fence_after_sync();
                uint32_t pk[32];                                 // the row's 64 probabilities, bf16 pairs
                float sum = 0.f, alpha = 1.f, m_use = m_ref;
                bool need = false;
                if (warp_live) {
                    uint32_t raw[2][32];
                    tmem_ld32(lane_base + tmem_s_col(sb), raw[0]);
                    tmem_ld32(lane_base + tmem_s_col(sb) + 32, raw[1]);
                    tmem_wait_ld();
                    tc_fence_before_sync();
                    mbar_arrive(s_free(sb));
                    float scl = sc;                              // what the values in raw[] still have to be multiplied by
                    bool neg = sc_neg;
                    if (kPrefill && mt.diag + j < kTile - 1) {
                        // causal diagonal (or ragged last tile): this row sees columns 0 .. diag + j only.
                        // Scale first, then replace what is hidden by -inf with a select: hidden K rows
                        // may hold anything.
                        const int limit = mt.diag + j;
                        #pragma unroll
                        for (int e = 0; e < 64; ++e) {
                            const float v = __uint_as_float(raw[e >> 5][e & 31]) * sc;
                            raw[e >> 5][e & 31] = __float_as_uint(e <= limit ? v : -INFINITY);
                        }
                        scl = 1.f; neg = false;
                    }
                    // extreme raw score of the tile (two chains); the scale may be negative
                    float e0 = __uint_as_float(raw[0][0]), e1 = __uint_as_float(raw[1][0]);
                    if (!neg) {
                        #pragma unroll
                        for (int e = 1; e < 31; e += 2) {
                            asm("max.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[0][e])), "f"(__uint_as_float(raw[0][e + 1])));
                            asm("max.f32 %0, %0, %1, %2;" : "+f"(e1) : "f"(__uint_as_float(raw[1][e])), "f"(__uint_as_float(raw[1][e + 1])));
                        }
                        asm("max.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[0][31])), "f"(__uint_as_float(raw[1][31])));
                        e0 = fmaxf(e0, e1);
                    } else {
                        #pragma unroll
                        for (int e = 1; e < 31; e += 2) {
                            asm("min.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[0][e])), "f"(__uint_as_float(raw[0][e + 1])));
                            asm("min.f32 %0, %0, %1, %2;" : "+f"(e1) : "f"(__uint_as_float(raw[1][e])), "f"(__uint_as_float(raw[1][e + 1])));
                        }
                        asm("min.f32 %0, %0, %1, %2;" : "+f"(e0) : "f"(__uint_as_float(raw[0][31])), "f"(__uint_as_float(raw[1][31])));
                        e0 = fminf(e0, e1);
                    }
                    const float mx = e0 * scl;
                    need = !first && (mx > m_ref + kSlack);
                    m_use = (first || need) ? mx : m_ref;
                    if (need) alpha = fast_exp2(m_ref - mx);
                    const float neg_m = (m_use == -INFINITY) ? 0.f : -m_use;   // a row that sees nothing yet: P = 0
                    float sum1 = 0.f;
                    #pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int t0 = 2 * e;
                        // every kPolyEvery-th pair takes its second exponential off the special-function unit
                        const float p0 = fast_exp2(fmaf(__uint_as_float(raw[t0 >> 5][t0 & 31]), scl, neg_m));
                        const float x1 = fmaf(__uint_as_float(raw[(t0 + 1) >> 5][(t0 + 1) & 31]), scl, neg_m);
                        const float p1 = (Cfg::kPolyEvery > 0 && e % (Cfg::kPolyEvery > 0 ? Cfg::kPolyEvery : 1) == 0) ? exp2_fma(x1) : fast_exp2(x1);
                        sum += p0; sum1 += p1;
                        pk[e] = pack_bf16(p0, p1);
                    }
                    sum += sum1;
                } else {
                    tc_fence_before_sync();
                    mbar_arrive(s_free(sb));
                }
                // this group's previous P.V must be complete before its P tile is overwritten and
                // before a rescale touches O; the probabilities above were computed while it ran
                if (k > 0) {
                    if (!mbar_wait(pv_done(g), (k - 1) & 1u, abort_flag)) { ok = false; site = 39; break; }
                    tc_fence_after_sync();
                }
                if (warp_live) {
                    if (__any_sync(0xffffffffu, need)) {
                        #pragma unroll
                        for (int cblk = 0; cblk < 4; ++cblk) {
                            uint32_t o[32];
                            tmem_ld32(o_mine + cblk * 32, o);
                            tmem_wait_ld();
                            #pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st32(o_mine + cblk * 32, o);
                        }
                        tmem_wait_st();
                    }
                    l = first ? sum : fmaf(l, alpha, sum);
                    m_ref = m_use;
                    tmem_st32(lane_base + kTmemP + g * 32, pk);  // the row's 64 probabilities, the A operand of P.V
                    tmem_wait_st();
                }
                tc_fence_before_sync();
                mbar_arrive(p_full(g));
                ++k;
            }

            if (mt.idx == mt.cnt - 1) {
                // ---- the segment ends with this tile: both groups meet, merge their two states of
                //      every row and write one normalised partial per sibling (half the columns each)
                const bool had = mine || mt.cnt >= 2;            // this group took a tile of the segment
                if (had) {
                    if (!mbar_wait(pv_done(g), (k - 1) & 1u, abort_flag)) { ok = false; site = 40; break; }
                    tc_fence_after_sync();
                }
                xch[g * kTRows + row] = make_float2(had ? m_ref : -INFINITY, had ? l : 0.f);
                mbar_arrive(xch_a);
                if (!mbar_wait(xch_a, segs & 1u, abort_flag)) { ok = false; site = 41; break; }
                if (warp_live) {
                    const float2 other = xch[(g ^ 1) * kTRows + row];
                    // Whether the other group took a tile of this segment is the same for every row
                    // (the TMEM loads below are warp-wide instructions and may depend on nothing
                    // else); whether a particular row of it saw any token is not, and is a select.
                    const bool had_other = !mine || mt.cnt >= 2;
                    const bool had2 = had_other && other.y > 0.f;
                    const float m1 = had ? m_ref : -INFINITY, l1 = had ? l : 0.f;
                    const float M = fmaxf(m1, other.x);
                    const float w1 = had ? fast_exp2(m1 - M) : 0.f, w2 = had2 ? fast_exp2(other.x - M) : 0.f;
                    const float L = l1 * w1 + other.y * w2;
                    const float inv = 1.f / L;
                    const float f1 = w1 * inv, f2 = w2 * inv;
                    // prefix pass: a normalised fp32 partial per sibling; prefill: the final rows of out / lse
                    const bool live = j < mt.n && (!kPrefill || head < p.group) &&
                                      (kPrefill ? in_bounds(p.hdr, (int64_t)(mt.row + j) * p.hq + mt.g * p.group + head, p.out_rows, 201)
                                                : in_bounds(p.hdr, mt.row + j, c.max_rows, 202));
                    float* dst = c.pre_o + ((int64_t)(mt.row + j) * kGroup + head) * kD + g * 64;
                    const int64_t out_row = (int64_t)(mt.row + j) * p.hq + mt.g * p.group + head;
                    #pragma unroll
                    for (int cblk = 0; cblk < 2; ++cblk) {
                        uint32_t oa[32], ob[32];
                        if (had) tmem_ld32(o_mine + g * 64 + cblk * 32, oa);
                        if (had_other) tmem_ld32(o_other + g * 64 + cblk * 32, ob);
                        tmem_wait_ld();
                        if (kPrefill && live) {
                            uint4* od = reinterpret_cast<uint4*>(p.out + out_row * kD + g * 64 + cblk * 32);
                            #pragma unroll
                            for (int e = 0; e < 32; e += 8) {
                                float v[8];
                                #pragma unroll
                                for (int q = 0; q < 8; ++q) {
                                    const float a = had ? __uint_as_float(oa[e + q]) * f1 : 0.f;
                                    v[q] = had2 ? fmaf(__uint_as_float(ob[e + q]), f2, a) : a;
                                }
                                od[e >> 3] = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]),
                                                        pack_bf16(v[6], v[7]));
                            }
                        }
                        if (!kPrefill && live) {
                            #pragma unroll
                            for (int e = 0; e < 32; e += 4) {
                                float4 v;
                                float* vp = reinterpret_cast<float*>(&v);
                                #pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    const float a = had ? __uint_as_float(oa[e + q]) * f1 : 0.f;
                                    vp[q] = had2 ? fmaf(__uint_as_float(ob[e + q]), f2, a) : a;
                                }
                                *reinterpret_cast<float4*>(dst + cblk * 32 + e) = v;
                            }
                        }
                    }
                    if (live && g == 0) {
                        if (kPrefill) p.lse[out_row] = (M + log2f(L)) * 0.6931471805599453f;
                        else c.pre_lse[(int64_t)(mt.row + j) * kGroup + head] = M + log2f(L);
                    }
                }
                // nobody's next P.V may overwrite an accumulator the other group is still reading
                tc_fence_before_sync();
                mbar_arrive(xch_b);
                if (!mbar_wait(xch_b, segs & 1u, abort_flag)) { ok = false; site = 42; break; }
                ++segs;
            }
        }
        if (!ok && lane == 0) wait_failed(p, abort_flag, site);
        __syncwarp();
    }

    // ---- common exit: every role arrives here, then the allocating warp releases the TMEM
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kTMmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------ host side

namespace {

template <bool kPrefill>
cudaError_t launch_attn_tc(const DecodeParams& p, const CascadeParams& c, const PrefillParams& f, uint64_t q_rows,
                           int grid, cudaStream_t stream) {
    CUtensorMap mk, mv, mq;
    const uint64_t pool_rows = (uint64_t)p.num_pages * p.page_size * (p.token_major ? 1 : p.hkv);
    const uint32_t planes = p.token_major ? 2 * p.hkv : 2;
    // a 64-token page is a whole tile: both halves come with one copy ([half][row][128 B])
    const uint32_t halves = p.box_rows == kTile ? 2 : 1;
    if (!make_rows_map(&mk, p.k_pages, pool_rows, p.box_rows, halves, planes) ||
        !make_rows_map(&mv, p.v_pages, pool_rows, p.box_rows, halves, planes) ||
        !make_rows_map(&mq, p.q, q_rows, kGroup, 1))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<kPrefill>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         TSmem<kPrefill>::kBytes);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kTThreads);
    cfg.dynamicSmemBytes = TSmem<kPrefill>::kBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, attn_tc_kernel<kPrefill>, p, c, f, mk, mv, mq);
}

constexpr int kPrefillPlanThreads = 1024;

}  // namespace

cudaError_t launch_prefix_tc(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream) {
    return launch_attn_tc<false>(p, c, PrefillParams{}, (uint64_t)p.batch * p.hq, c.grid_ctas, stream);
}

// ---- prefill plan: blocks of f.block query tokens per sequence and their prefix sums; one unit per
//      (sequence, block, KV head)
__global__ void __launch_bounds__(kPrefillPlanThreads) plan_prefill_kernel(DecodeParams p, PrefillParams f) {
    __shared__ int32_t warp_sums[kPrefillPlanThreads / 32];
    __shared__ int32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the attention kernel's prologue may start
    if (tid == 0) { carry_s = 0; p.tiles_prefix[0] = 0; }
    __syncthreads();
    const int64_t max_len = (int64_t)p.bt_stride * p.page_size;
    uint32_t flags = 0;
    for (int base = 0; base < p.batch; base += kPrefillPlanThreads) {
        const int b = base + tid;
        int32_t blocks = 0;
        if (b < p.batch) {
            int64_t len = p.seq_lens[b];
            if (len < 0) { len = 0; flags |= kFlagBadLen; }
            if (len > max_len) { len = max_len; flags |= kFlagBadLen; }
            int64_t q_len = (int64_t)f.q_start[b + 1] - f.q_start[b];
            if (q_len < 0) { q_len = 0; flags |= kFlagBadLen; }
            if (q_len > len) { q_len = len; flags |= kFlagBadLen; }      // more query tokens than cached tokens
            blocks = (int32_t)((q_len + f.block - 1) / f.block);
        }
        int32_t v = blocks;
        #pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t n = __shfl_up_sync(0xffffffffu, v, o);
            if (lane >= o) v += n;
        }
        if (lane == 31) warp_sums[warp] = v;
        __syncthreads();
        if (warp == 0) {
            int32_t w = warp_sums[lane];
            #pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t n = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += n;
            }
            warp_sums[lane] = w;
        }
        __syncthreads();
        const int32_t incl = v + (warp ? warp_sums[warp - 1] : 0) + carry_s;
        if (b < p.batch) p.tiles_prefix[b + 1] = incl;
        __syncthreads();
        if (tid == kPrefillPlanThreads - 1) carry_s = incl;
        __syncthreads();
    }
    if (flags) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), flags);
    if (tid == 0) {
        p.hdr[kHdrTotalTiles] = p.hkv * carry_s;         // units
        p.hdr[kHdrNumRanges] = p.hkv * carry_s;
        p.hdr[kHdrClaim] = p.grid_ctas;
    }
}

// pair != 0: the kernel with two query tiles per CTA (32-token blocks); else one tile (16-token blocks)
cudaError_t launch_prefill_tc(const DecodeParams& p, const PrefillParams& f_in, int pair, cudaStream_t stream) {
    PrefillParams f = f_in;
    f.block = pair ? prefill_pair_block() : TCfg<true>::kShare;
    plan_prefill_kernel<<<1, kPrefillPlanThreads, 0, stream>>>(p, f);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (pair) return launch_prefill_pair(p, f, stream);
    return launch_attn_tc<true>(p, CascadeParams{}, f, (uint64_t)f.total_q * p.hq, p.grid_ctas, stream);
}

}  // namespace concur
