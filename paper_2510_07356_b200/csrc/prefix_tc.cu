// Prefix pass of the shared-prefix (cascade) step on the 5th-generation tensor cores.
//
// A unit is (group, KV head): the tiles that all siblings of a group have in common.  Each
// 64-token K/V tile is streamed from HBM once and multiplied with the query rows of all
// sharing siblings at once: n siblings x 8 heads of the GQA group = up to 80 rows, held as
// the 128-row A operand of tcgen05.mma (rows beyond 8n are never written out).  This is the
// one place of the decode step that is a dense contraction (80 flop per KV byte at ten
// siblings), so it runs on tcgen05 with its accumulators in tensor memory:
//
//   S[128 x 64]   = Q[128 x 128] . K_tile^T            (8 MMAs of K = 16; S in TMEM, double-buffered)
//   online softmax, one thread per row: thread t owns TMEM lane t = (sibling t / 8, head t % 8);
//                 it reads its 64 scores with one tcgen05.ld, keeps the running maximum and sum in
//                 registers, and writes P = 2^(S - m) as bf16 into a swizzled shared-memory tile
//   O[128 x 128] += P[128 x 64] . V_tile[64 x 128]     (4 MMAs of K = 16; O in TMEM, V is the
//                 MN-major B operand exactly as TMA laid it down)
//   when a row's maximum moves, its O row is rescaled in TMEM (tcgen05.ld / st) before the
//   next P.V product is released.
//
// Warp roles: warps 0-3 softmax / rescale / epilogue (128 threads = 128 TMEM lanes), warp 4
// TMA producer, warp 5 issues the MMAs (one thread) and owns the TMEM allocation.  The MMA
// thread issues Q.K^T of tile i + 1 before P.V of tile i, so the tensor pipe works on the next
// scores while the softmax threads are busy with the current ones.
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

namespace concur {

namespace {

constexpr int kTStages = 5;
constexpr int kTProducerWarp = 4;
constexpr int kTMmaWarp = 5;
constexpr int kTThreads = 6 * 32;
constexpr int kTRows = 128;                               // MMA M
constexpr int kTHalfBytes = kTile * 128;                  // 8 KB: 64 tokens x one 64-dim half
constexpr int kTTileBytes = 2 * kTHalfBytes;              // 16 KB: one K or V tile
constexpr int kTStageBytes = 2 * kTTileBytes;             // K | V
constexpr int kTQRows = kMaxShare * kGroup;               // 80 query rows that are really loaded
constexpr int kTQHalfBytes = kTQRows * 128;               // 10 KB
constexpr int kTQBytes = 2 * kTQHalfBytes;                // 20 KB per buffer
constexpr int kTPBytes = kTRows * 128;                    // 16 KB: P tile, 128 rows x 64 tokens bf16
constexpr uint32_t kTmemCols = 256;                       // S0 [0,64)  S1 [64,128)  O [128,256)
constexpr uint32_t kTmemO = 128;

static_assert(kTQHalfBytes % 1024 == 0, "query halves must keep the swizzle phase");

struct TMeta {
    int32_t n;            // sharing siblings (2..kMaxShare); 0 = no more work
    int32_t first, last;  // first / last tile of its segment
    int32_t qsel;         // query buffer of the segment
    int32_t row;          // first partial row of the segment (one row per sibling)
    int32_t pad[3];
};

// Shared memory, from a 1024-byte aligned base.  The MMA reads 128 A rows; the query buffers
// hold 80, so the rows beyond them alias whatever follows (the other query buffer, the P tile):
// always inside this allocation, and only ever feeding accumulator rows that are not written out.
struct TSmem {
    static constexpr int kQOff = kTStages * kTStageBytes;                 // 2 x 20 KB
    static constexpr int kPOff = kQOff + 2 * kTQBytes;                    // 16 KB
    static constexpr int kMetaOff = kPOff + kTPBytes;
    static constexpr int kBarOff = kMetaOff + kTStages * (int)sizeof(TMeta);
    // full_k, full_v, empty per stage; q_full x2, q_empty x2; s_full x2, s_free x2; p_full; pv_done
    static constexpr int kNumBars = 3 * kTStages + 10;
    static constexpr int kTmemPtrOff = kBarOff + kNumBars * 8;
    static constexpr int kAbortOff = kTmemPtrOff + 8;
    static constexpr int kTotal = kAbortOff + 8;
    static constexpr int kBytes = kTotal + 1024;
};
static_assert(TSmem::kPOff % 1024 == 0 && TSmem::kQOff % 1024 == 0, "operand slabs must be 1024-byte aligned");
static_assert(TSmem::kQOff + kTQBytes + kTQHalfBytes + kTRows * 128 <= TSmem::kPOff + kTPBytes,
              "the 128-row view of the last query half must stay inside the allocation");
static_assert(TSmem::kBytes <= 232448, "exceeds the 227 KB a CTA may use");

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1, int32_t c2,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}

}  // namespace

__global__ void __launch_bounds__(kTThreads, 1)
prefix_tc_kernel(DecodeParams p, CascadeParams c, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    TMeta* meta = reinterpret_cast<TMeta*>(smem + TSmem::kMetaOff);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(smem + TSmem::kAbortOff);
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(smem + TSmem::kTmemPtrOff);
    const uint32_t bar_base = smem_base + TSmem::kBarOff;
    auto full_k = [&](int s) { return bar_base + 8u * s; };
    auto full_v = [&](int s) { return bar_base + 8u * (kTStages + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * kTStages + s); };
    auto q_full = [&](int i) { return bar_base + 8u * (3 * kTStages + i); };
    auto q_empty = [&](int i) { return bar_base + 8u * (3 * kTStages + 2 + i); };
    auto s_full = [&](int i) { return bar_base + 8u * (3 * kTStages + 4 + i); };
    auto s_free = [&](int i) { return bar_base + 8u * (3 * kTStages + 6 + i); };
    const uint32_t p_full = bar_base + 8u * (3 * kTStages + 8);
    const uint32_t pv_done = bar_base + 8u * (3 * kTStages + 9);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int32_t P = p.page_size;

    // unused query rows must at least be defined once
    for (int i = tid; i < (2 * kTQBytes + kTPBytes) / 16; i += kTThreads)
        reinterpret_cast<uint4*>(smem + TSmem::kQOff)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int s = 0; s < kTStages; ++s) {
            mbar_init(full_k(s), 1);
            mbar_init(full_v(s), 1);
            mbar_init(empty(s), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(q_full(i), 1);
            mbar_init(q_empty(i), 1);
            mbar_init(s_full(i), 1);
            mbar_init(s_free(i), 128);
        }
        mbar_init(p_full, 128);
        mbar_init(pv_done, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == kTMmaWarp) tmem_alloc(smem_base + TSmem::kTmemPtrOff, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr;
    const int32_t W = c.chdr[kHdrTotalTiles];
    const int32_t R = c.chdr[kHdrNumRanges];

    if (warp == kTProducerWarp) {
        // =========================================================== producer warp
        uint32_t it = 0, seg = 0;
        bool ok = true;
        const int pages_per_tile_shift = 6 - p.page_shift;
        const int32_t npages = kTile >> p.page_shift;
        const uint32_t page_bytes = (uint32_t)P * 128u;        // one half of one page
        int32_t r = blockIdx.x;
        while (ok && r < R) {
            int32_t r_next = 0;
            if (lane == 0) r_next = atomicAdd(c.chdr + kHdrClaim, 1);
            const int32_t x0 = range_begin(W, R, r), x1 = range_begin(W, R, r + 1);
            int32_t x = x0;
            while (ok && x < x1) {
                // the prefix unit (group i, KV head g) that holds flat tile x
                const int32_t i = find_sequence(c.ptiles_prefix, c.num_groups, x);
                const int32_t t_i = c.ptiles_prefix[i + 1] - c.ptiles_prefix[i];
                const int32_t base = kHkv * c.ptiles_prefix[i];
                const int32_t g = (x - base) / t_i;
                const int32_t unit_start = base + g * t_i;
                const int32_t tile0 = x - unit_start;
                const int32_t tile1 = min(x1, unit_start + t_i) - unit_start;
                x += tile1 - tile0;
                const int32_t b0 = c.group_start[i];
                const int32_t n = min(c.group_start[i + 1] - b0, kMaxShare);
                const int32_t split = r - range_of(W, R, unit_start);
                const int32_t row = c.unit_rowbase[i * kHkv + g] + split * n;
                const int32_t qsel = seg & 1;
                const int32_t* table = p.block_table + (int64_t)b0 * p.bt_stride;   // the first sibling's pages
                const int32_t page_end = tile1 << pages_per_tile_shift;
                int32_t chunk_base = tile0 << pages_per_tile_shift;
                int32_t pg = (chunk_base + lane < page_end) ? __ldg(table + chunk_base + lane) : 0;
                int32_t pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                for (int32_t t = tile0; ok && t < tile1; ++t) {
                    const int32_t first_page = t << pages_per_tile_shift;
                    if (first_page >= chunk_base + 32) {
                        chunk_base += 32;
                        pg = pg_next;
                        pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                    }
                    const int s = it % kTStages;
                    const uint32_t parity = (it / kTStages) & 1u;
                    int32_t my_page = __shfl_sync(0xffffffffu, pg, (first_page - chunk_base + (lane & 3)) & 31);
                    const bool bad = (lane < npages) && (my_page < 0 || my_page >= p.num_pages);
                    if (__any_sync(0xffffffffu, bad)) {
                        if (lane == 0) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagBadPage);
                        if (my_page < 0 || my_page >= p.num_pages) my_page = 0;
                    }
                    const int32_t pages[4] = {__shfl_sync(0xffffffffu, my_page, 0), __shfl_sync(0xffffffffu, my_page, 1),
                                              __shfl_sync(0xffffffffu, my_page, 2), __shfl_sync(0xffffffffu, my_page, 3)};
                    if (lane == 0) {
                        if (t == tile0) {
                            // the segment's query rows: sibling j's 8 rows go to rows 8j .. 8j + 7 of both halves
                            ok = mbar_wait(q_empty(qsel), ((seg >> 1) & 1u) ^ 1u, abort_flag);
                            if (ok) {
                                mbar_arrive_expect_tx(q_full(qsel), n * kGroup * kRowBytes);
                                const uint32_t qdst = smem_base + TSmem::kQOff + qsel * kTQBytes;
                                for (int j = 0; j < n; ++j) {
                                    const int32_t qrow = (b0 + j) * kHq + g * kGroup;
                                    tma_load_3d(qdst + j * 1024, &map_q, 0, qrow, 0, q_full(qsel));
                                    tma_load_3d(qdst + kTQHalfBytes + j * 1024, &map_q, 0, qrow, 1, q_full(qsel));
                                }
                            }
                        }
                        if (ok) ok = mbar_wait(empty(s), parity ^ 1u, abort_flag);
                        if (ok) {
                            TMeta& m = meta[s];
                            m.n = n; m.first = (t == tile0); m.last = (t == tile1 - 1); m.qsel = qsel; m.row = row;
                            const uint32_t kdst = smem_base + s * kTStageBytes;
                            const uint32_t vdst = kdst + kTTileBytes;
                            mbar_arrive_expect_tx(full_k(s), kTTileBytes);
                            #pragma unroll
                            for (int q = 0; q < 4; ++q)
                                if (q < npages) {
                                    const int32_t prow = (pages[q] * kHkv + g) * P;
                                    tma_load_3d(kdst + q * page_bytes, &map_k, 0, prow, 0, full_k(s));
                                    tma_load_3d(kdst + kTHalfBytes + q * page_bytes, &map_k, 0, prow, 1, full_k(s));
                                }
                            mbar_arrive_expect_tx(full_v(s), kTTileBytes);
                            #pragma unroll
                            for (int q = 0; q < 4; ++q)
                                if (q < npages) {
                                    const int32_t prow = (pages[q] * kHkv + g) * P;
                                    tma_load_3d(vdst + q * page_bytes, &map_v, 0, prow, 0, full_v(s));
                                    tma_load_3d(vdst + kTHalfBytes + q * page_bytes, &map_v, 0, prow, 1, full_v(s));
                                }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (ok) ++it;
                }
                ++seg;
            }
            r = __shfl_sync(0xffffffffu, r_next, 0);
        }
        if (lane == 0) {
            if (ok) {
                const int s = it % kTStages;
                ok = mbar_wait(empty(s), ((it / kTStages) & 1u) ^ 1u, abort_flag);
                if (ok) { meta[s].n = 0; mbar_arrive(full_k(s)); }
            }
            if (!ok) {
                wait_failed(p, abort_flag, 31);
                // let the copies still in flight land before the CTA's shared memory is released
                const uint32_t lo = it > (uint32_t)kTStages ? it - kTStages : 0u;
                for (uint32_t j = lo; j < it; ++j) {
                    volatile int32_t never = 0;
                    mbar_wait(full_k(j % kTStages), (j / kTStages) & 1u, &never);
                    mbar_wait(full_v(j % kTStages), (j / kTStages) & 1u, &never);
                }
            }
        }
    } else if (warp == kTMmaWarp) {
        // =========================================================== MMA warp (one thread issues)
        if (lane == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kTRows, kTile, false, false);
            constexpr uint32_t idesc_pv = umma_idesc_bf16(kTRows, kD, false, true);
            const uint32_t p_addr = smem_base + TSmem::kPOff;
            bool ok = true, have_prev = false;
            int ps = 0;
            uint32_t pparity = 0, pfirst = 0, segs = 0;
            int site = 0;
            for (uint32_t it = 0; ok; ++it) {
                const int s = it % kTStages;
                const uint32_t parity = (it / kTStages) & 1u;
                if (!mbar_wait(full_k(s), parity, abort_flag)) { ok = false; site = 32; break; }
                const TMeta mt = meta[s];
                const bool done = (mt.n == 0);
                auto issue_qk = [&]() {
                    if (mt.first) {
                        if (!mbar_wait(q_full(mt.qsel), (segs >> 1) & 1u, abort_flag)) { ok = false; site = 33; return; }
                        ++segs;
                    }
                    const int sb = it & 1u;
                    if (!mbar_wait(s_free(sb), ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; site = 34; return; }
                    tc_fence_after_sync();
                    const uint32_t q_addr = smem_base + TSmem::kQOff + mt.qsel * kTQBytes;
                    const uint32_t k_addr = smem_base + s * kTStageBytes;
                    #pragma unroll
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const uint32_t koff = (uint32_t)(k16 & 3) * 32u;
                        const uint64_t a = umma_smem_desc(q_addr + (k16 >> 2) * kTQHalfBytes + koff, 16, 1024);
                        const uint64_t b = umma_smem_desc(k_addr + (k16 >> 2) * kTHalfBytes + koff, 16, 1024);
                        umma_ss(tmem_base + sb * kTile, a, b, idesc_qk, k16 > 0);
                    }
                    umma_commit(s_full(sb));
                    if (mt.last) umma_commit(q_empty(mt.qsel));      // the segment's last read of its query buffer
                };
                auto issue_pv = [&]() {
                    if (!mbar_wait(p_full, (it - 1) & 1u, abort_flag)) { ok = false; site = 35; return; }
                    if (!mbar_wait(full_v(ps), pparity, abort_flag)) { ok = false; site = 36; return; }
                    tc_fence_after_sync();
                    const uint32_t v_addr = smem_base + ps * kTStageBytes + kTTileBytes;
                    #pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t a = umma_smem_desc(p_addr + kk * 32, 16, 1024);
                        const uint64_t b = umma_smem_desc(v_addr + kk * 2048, kTHalfBytes, 1024);
                        umma_ss(tmem_base + kTmemO, a, b, idesc_pv, (pfirst && kk == 0) ? 0u : 1u);
                    }
                    umma_commit(empty(ps));          // K and V of that stage may be overwritten
                    umma_commit(pv_done);
                };
                // scores of tile `it` first, so that they are computed while the softmax threads
                // work on tile it - 1; at a segment start the new queries may still be in flight,
                // so the pending P.V goes first there
                if (!done && !mt.first) issue_qk();
                if (ok && have_prev) issue_pv();
                if (ok && !done && mt.first) issue_qk();
                if (done) break;
                have_prev = true; ps = s; pparity = parity; pfirst = mt.first;
            }
            if (!ok) wait_failed(p, abort_flag, site);
        }
        __syncwarp();
    } else {
        // =========================================================== softmax warps (thread = row)
        const int j = tid >> 3, head = tid & 7;                  // sibling, head of this row
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        const uint32_t p_row = smem_base + TSmem::kPOff + (uint32_t)tid * 128u;
        const int sw = tid & 7;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        int site = 0;
        for (uint32_t it = 0; ok; ++it) {
            const int s = it % kTStages;
            const uint32_t parity = (it / kTStages) & 1u;
            if (!mbar_wait(full_k(s), parity, abort_flag)) { ok = false; site = 37; break; }
            const TMeta mt = meta[s];
            if (mt.n == 0) break;
            const int sb = it & 1u;
            if (mt.first) { m = -INFINITY; l = 0.f; }
            if (!mbar_wait(s_full(sb), (it >> 1) & 1u, abort_flag)) { ok = false; site = 38; break; }
            tc_fence_after_sync();
            uint32_t raw[2][32];
            tmem_ld32(lane_base + sb * kTile, raw[0]);
            tmem_ld32(lane_base + sb * kTile + 32, raw[1]);
            tmem_wait_ld();
            tc_fence_before_sync();
            mbar_arrive(s_free(sb));
            float mx = -INFINITY;
            #pragma unroll
            for (int h = 0; h < 2; ++h)
                #pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float v = __uint_as_float(raw[h][e]) * p.scale_log2e;
                    raw[h][e] = __float_as_uint(v);
                    mx = fmaxf(mx, v);
                }
            const float m_new = fmaxf(m, mx);
            const float alpha = fast_exp2(m - m_new);            // 0 on a segment's first tile
            const bool moved = (m_new != m) && !mt.first;
            // P.V of the previous tile must be complete: it reads the P tile written below, and a
            // rescale must see all of O
            if (it > 0) {
                if (!mbar_wait(pv_done, (it - 1) & 1u, abort_flag)) { ok = false; site = 39; break; }
                tc_fence_after_sync();
            }
            if (__any_sync(0xffffffffu, moved)) {
                const float a = moved ? alpha : 1.f;
                #pragma unroll
                for (int cblk = 0; cblk < 4; ++cblk) {
                    uint32_t o[32];
                    tmem_ld32(lane_base + kTmemO + cblk * 32, o);
                    tmem_wait_ld();
                    #pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * a);
                    tmem_st32(lane_base + kTmemO + cblk * 32, o);
                }
                tmem_wait_st();
            }
            m = m_new;
            float sum = 0.f;
            #pragma unroll
            for (int ch = 0; ch < 8; ++ch) {                     // 8 tokens = one 16-byte chunk of the P row
                uint32_t w[4];
                #pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int t0 = ch * 8 + 2 * e;
                    const float p0 = fast_exp2(__uint_as_float(raw[t0 >> 5][t0 & 31]) - m);
                    const float p1 = fast_exp2(__uint_as_float(raw[(t0 + 1) >> 5][(t0 + 1) & 31]) - m);
                    sum += p0 + p1;
                    w[e] = pack_bf16(p0, p1);
                }
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                             ::"r"(p_row + (uint32_t)((ch ^ sw) << 4)), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
            }
            l = fmaf(l, alpha, sum);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_before_sync();
            mbar_arrive(p_full);

            if (mt.last) {
                // ---- the segment's result: one normalised partial per sibling
                if (!mbar_wait(pv_done, it & 1u, abort_flag)) { ok = false; site = 40; break; }
                tc_fence_after_sync();
                const float inv = 1.f / l;
                const bool live = j < mt.n;
                float* dst = c.pre_o + ((int64_t)(mt.row + j) * kGroup + head) * kD;
                #pragma unroll
                for (int cblk = 0; cblk < 4; ++cblk) {
                    uint32_t o[32];
                    tmem_ld32(lane_base + kTmemO + cblk * 32, o);
                    tmem_wait_ld();
                    if (live) {
                        #pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            *reinterpret_cast<float4*>(dst + cblk * 32 + e) =
                                make_float4(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv,
                                            __uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
                    }
                }
                if (live) c.pre_lse[(int64_t)(mt.row + j) * kGroup + head] = m + log2f(l);
                tc_fence_before_sync();
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            sym = nullptr;
        return reinterpret_cast<EncodeTiledFn>(sym);
    }();
    return fn;
}

// Rows of 128 bf16 seen as {64 elements, rows, 2 halves}; a box is `box_rows` rows of ONE half
// and lands in shared memory as [row][128 B] with the 128-byte swizzle: one slab of a K-major
// (or, read along the rows, MN-major) tcgen05 operand.
bool make_half_row_map(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {64, rows, 2};
    const cuuint64_t strides[2] = {256, 128};
    const cuuint32_t box[3] = {64, box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_prefix_tc(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream) {
    CUtensorMap mk, mv, mq;
    const uint64_t pool_rows = (uint64_t)p.num_pages * kHkv * p.page_size;
    if (!make_half_row_map(&mk, p.k_pages, pool_rows, p.page_size) ||
        !make_half_row_map(&mv, p.v_pages, pool_rows, p.page_size) ||
        !make_half_row_map(&mq, p.q, (uint64_t)p.batch * kHq, kGroup))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(prefix_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TSmem::kBytes);
    if (e != cudaSuccess) return e;
    prefix_tc_kernel<<<c.grid_ctas, kTThreads, TSmem::kBytes, stream>>>(p, c, mk, mv, mq);
    return cudaGetLastError();
}

}  // namespace concur
