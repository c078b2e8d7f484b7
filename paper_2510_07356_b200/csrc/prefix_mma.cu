// Prefix pass of the shared-prefix (cascade) step, tensor-core kernel.
//
// A unit is (group, KV head): the tiles that all siblings of the group have in common.  They
// are streamed from HBM once (same TMA ring as the plain partial kernel) and multiplied with
// the query rows of all sharing siblings, so the contraction is no longer 16 x 8 x 128 per
// warp but 16 x 8n x 128 (n = 2..10 siblings):
//
//   phase 1  warp w owns tokens 16w..16w+15 of the tile:  S_j^T[16 x 8] = K . Q_j^T for every
//            sibling j (K fragments loaded once, reused for all j), per-warp column maxima
//   phase 2  all warps agree on the new running maximum per (sibling, head), rescale their
//            accumulators, and publish P = 2^(S - m) as bf16 in shared memory
//   phase 3  warp w owns output dims 32w..32w+31:  O_j^T[32 x 8] += V^T[32 x 64] . P_j^T[64 x 8]
//            (V fragments loaded once per tile, reused for all j)
//
// The accumulators are split by output dim, not by token, so a thread carries 8 floats per
// sibling instead of 32, which is what lets ten siblings fit in registers.  A segment ends with
// one normalised partial (out, base-2 lse) per sibling in the rows the plan assigned; the
// cascade combine kernel merges them with each sibling's suffix partials.
//
// Shared tiles are whole (the plan shares multiples of 64 tokens only): no masking here.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"

namespace concur {

namespace {

constexpr int kPStages = 4;
constexpr int kPConsumerWarps = 4;
constexpr int kPThreads = (kPConsumerWarps + 1) * 32;
constexpr int kPTileBytes = kTile * kRowBytes;            // 16 KB
constexpr int kPStageBytes = 2 * kPTileBytes;             // K | V
constexpr int kQTileBytes = kGroup * kRowBytes;           // 2 KB per sibling
constexpr int kPRowBytes = 144;                           // one (sibling, head) row of P: 64 bf16 + pad

struct PrefixMeta {
    int32_t n;            // sharing siblings (2..kMaxShare); 0 = no more work
    int32_t first, last;  // first / last tile of its segment
    int32_t qsel;         // which query buffer the segment uses
    int32_t row;          // first output row of the segment (one row per sibling)
    int32_t pad[3];
};

template <int NS>
struct PSmem {
    static constexpr int kQOff = kPStages * kPStageBytes;                    // 2 buffers x NS x 2 KB
    static constexpr int kPOff = kQOff + 2 * NS * kQTileBytes;               // NS x 8 rows x 144 B
    static constexpr int kWmaxOff = kPOff + NS * kGroup * kPRowBytes;        // [4 warps][NS][8] floats
    static constexpr int kLsumOff = kWmaxOff + kPConsumerWarps * NS * kGroup * 4;
    static constexpr int kMetaOff = kLsumOff + kPConsumerWarps * NS * kGroup * 4;
    static constexpr int kBarOff = kMetaOff + kPStages * (int)sizeof(PrefixMeta);
    // full_k, full_v, empty per stage; q_full x2, q_empty x2; sync_a, sync_b
    static constexpr int kAbortOff = kBarOff + (3 * kPStages + 6) * 8;
    static constexpr int kTotal = kAbortOff + 16;
    static constexpr int kBytes = kTotal + 1024;
};

}  // namespace

template <int NS>
__global__ void __launch_bounds__(kPThreads, 1)
prefix_mma_kernel(DecodeParams p, CascadeParams c, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q) {
    using L = PSmem<NS>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    float* wmax = reinterpret_cast<float*>(smem + L::kWmaxOff);
    float* lsum = reinterpret_cast<float*>(smem + L::kLsumOff);
    PrefixMeta* meta = reinterpret_cast<PrefixMeta*>(smem + L::kMetaOff);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(smem + L::kAbortOff);
    const uint32_t bar_base = smem_base + L::kBarOff;
    auto full_k = [&](int s) { return bar_base + 8u * s; };
    auto full_v = [&](int s) { return bar_base + 8u * (kPStages + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * kPStages + s); };
    auto q_full = [&](int i) { return bar_base + 8u * (3 * kPStages + i); };
    auto q_empty = [&](int i) { return bar_base + 8u * (3 * kPStages + 2 + i); };
    const uint32_t sync_a = bar_base + 8u * (3 * kPStages + 4);
    const uint32_t sync_b = sync_a + 8u;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int32_t P = p.box_rows;            // rows per box: the unit of the shared-memory tile layout

    if (tid == 0) {
        for (int s = 0; s < kPStages; ++s) {
            mbar_init(full_k(s), 1);
            mbar_init(full_v(s), 1);
            mbar_init(empty(s), kPConsumerWarps);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(q_full(i), 1); mbar_init(q_empty(i), kPConsumerWarps); }
        mbar_init(sync_a, kPConsumerWarps * 32);
        mbar_init(sync_b, kPConsumerWarps * 32);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int32_t W = c.chdr[kHdrTotalTiles];
    const int32_t R = c.chdr[kHdrNumRanges];

    if (warp == kPConsumerWarps) {
        // =========================================================== producer warp
        uint32_t it = 0, seg = 0;
        bool ok = true;
        const uint32_t box_bytes = (uint32_t)P * kRowBytes;
        const int32_t page_mask = p.page_size - 1;
        int32_t r = blockIdx.x;
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
                const int32_t n = min(c.group_start[i + 1] - b0, min(kMaxShare, NS));
                const int32_t split = r - range_of(W, R, unit_start);
                const int32_t row = c.unit_rowbase[i * p.hkv + g] + split * n;
                const int32_t qsel = seg & 1;
                const int32_t* table = p.block_table + (int64_t)b0 * p.bt_stride;   // the first sibling's pages
                const int32_t page_end = (tile1 * kTile + page_mask) >> p.page_shift;
                int32_t chunk_base = (tile0 * kTile) >> p.page_shift;
                int32_t pg = (chunk_base + lane < page_end) ? __ldg(table + chunk_base + lane) : 0;
                int32_t pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                for (int32_t t = tile0; ok && t < tile1; ++t) {
                    const int32_t first_page = (t * kTile) >> p.page_shift;
                    const int32_t row_in_page = (t * kTile) & page_mask;   // non-zero only for pages of more than 64 tokens
                    if (first_page >= chunk_base + 32) {
                        chunk_base += 32;
                        pg = pg_next;
                        pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                    }
                    const int32_t npages = kTile >> p.box_shift;          // boxes per tile
                    const int s = it % kPStages;
                    const uint32_t parity = (it / kPStages) & 1u;
                    int32_t my_page = __shfl_sync(0xffffffffu, pg, (first_page - chunk_base + (lane & 3)) & 31);
                    const bool bad = (lane < npages) && (my_page < 0 || my_page >= p.num_pages);
                    if (__any_sync(0xffffffffu, bad)) {
                        if (lane == 0) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagBadPage);
                        if (my_page < 0 || my_page >= p.num_pages) my_page = 0;
                    }
                    const int32_t pages[4] = {__shfl_sync(0xffffffffu, my_page, 0), __shfl_sync(0xffffffffu, my_page, 1),
                                              __shfl_sync(0xffffffffu, my_page, 2), __shfl_sync(0xffffffffu, my_page, 3)};
                    if (lane == 0) {
                        ok = mbar_wait(empty(s), parity ^ 1u, abort_flag);
                        if (ok && t == tile0) {
                            // the segment's query rows: one 2 KB swizzled tile per sibling
                            ok = mbar_wait(q_empty(qsel), ((seg >> 1) & 1u) ^ 1u, abort_flag);
                            if (ok) {
                                mbar_arrive_expect_tx(q_full(qsel), n * kQTileBytes);
                                const uint32_t qdst = smem_base + L::kQOff + qsel * NS * kQTileBytes;
                                for (int j = 0; j < n; ++j)
                                    tma_load_tile(qdst + j * kQTileBytes, &map_q, ((b0 + j) * p.hq + g * p.group), q_full(qsel));
                            }
                        }
                        if (ok) {
                            PrefixMeta& m = meta[s];
                            m.n = n; m.first = (t == tile0); m.last = (t == tile1 - 1); m.qsel = qsel; m.row = row;
                            const uint32_t kdst = smem_base + s * kPStageBytes;
                            const uint32_t vdst = kdst + kPTileBytes;
                            mbar_arrive_expect_tx(full_k(s), npages * box_bytes);
                            #pragma unroll
                            for (int q = 0; q < 4; ++q)
                                if (q < npages) tma_load_tile(kdst + q * box_bytes, &map_k, pool_row(p, pages[q], g, row_in_page), full_k(s), pool_plane(p, g));
                            mbar_arrive_expect_tx(full_v(s), npages * box_bytes);
                            #pragma unroll
                            for (int q = 0; q < 4; ++q)
                                if (q < npages) tma_load_tile(vdst + q * box_bytes, &map_v, pool_row(p, pages[q], g, row_in_page), full_v(s), pool_plane(p, g));
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
                const int s = it % kPStages;
                ok = mbar_wait(empty(s), ((it / kPStages) & 1u) ^ 1u, abort_flag);
                if (ok) { meta[s].n = 0; mbar_arrive(full_k(s)); }
            }
            if (!ok) {
                wait_failed(p, abort_flag, 21);
                const uint32_t lo = it > (uint32_t)kPStages ? it - kPStages : 0u;
                for (uint32_t j = lo; j < it; ++j) {
                    volatile int32_t never = 0;
                    mbar_wait(full_k(j % kPStages), (j / kPStages) & 1u, &never);
                    mbar_wait(full_v(j % kPStages), (j / kPStages) & 1u, &never);
                }
            }
        }
        return;
    }

    // =============================================================== consumer warps
    const int quad = lane & 3, qrow = lane >> 2;
    const float ninf = -INFINITY;
    const int tok0 = warp * 16;
    const uint32_t half_stride = (uint32_t)P * 128u;
    // K fragments of this warp's 16 tokens (phase 1)
    const uint32_t k_box_off = (uint32_t)(tok0 >> p.box_shift) * (uint32_t)P * kRowBytes;
    const int k_row = (tok0 & (P - 1)) + (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t k_row_off = k_box_off + (uint32_t)k_row * 128u;
    const int k_sel = lane >> 4;
    // Q fragments: tile [2 halves][8 heads][128 B]; ldmatrix.x4 covers two k-steps
    const int q_row = lane & 7, q_chunk = lane >> 3;
    // P rows for phase 3: ldmatrix.x4 covers tokens 32 tp .. 32 tp + 31 of one sibling
    const uint32_t p_lane_off = (uint32_t)(lane & 7) * kPRowBytes + (uint32_t)(lane >> 3) * 16u;
    const uint32_t pbase = smem_base + L::kPOff;

    float m[NS][2], l[NS][2], o[NS][2][4];
    #pragma unroll
    for (int j = 0; j < NS; ++j) {
        m[j][0] = m[j][1] = ninf; l[j][0] = l[j][1] = 0.f;
        #pragma unroll
        for (int db = 0; db < 2; ++db) o[j][db][0] = o[j][db][1] = o[j][db][2] = o[j][db][3] = 0.f;
    }
    uint32_t syncs = 0, segs = 0;

    auto fail = [&](int site) { if (lane == 0) wait_failed(p, abort_flag, site); };

    for (uint32_t it = 0;; ++it) {
        const int s = it % kPStages;
        const uint32_t parity = (it / kPStages) & 1u;
        if (!mbar_wait(full_k(s), parity, abort_flag)) { fail(22); return; }
        const PrefixMeta mt = meta[s];
        if (mt.n == 0) return;
        const uint32_t kbase = smem_base + s * kPStageBytes;
        const uint32_t vbase = kbase + kPTileBytes;
        const uint32_t qbase = smem_base + L::kQOff + mt.qsel * NS * kQTileBytes;
        if (mt.first) {
            if (!mbar_wait(q_full(mt.qsel), (segs >> 1) & 1u, abort_flag)) { fail(23); return; }
            #pragma unroll
            for (int j = 0; j < NS; ++j) {
                m[j][0] = m[j][1] = ninf; l[j][0] = l[j][1] = 0.f;
                #pragma unroll
                for (int db = 0; db < 2; ++db) o[j][db][0] = o[j][db][1] = o[j][db][2] = o[j][db][3] = 0.f;
            }
        }
        // ---- phase 1: S_j^T = K . Q_j^T for this warp's 16 tokens
        float sc[NS][4];
        #pragma unroll
        for (int j = 0; j < NS; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
        #pragma unroll
        for (int kp = 0; kp < 4; ++kp) {                 // pairs of 16-wide k-steps
            uint32_t a0[4], a1[4];
            {
                const int c0 = (2 * kp) * 2 + k_sel, c1 = (2 * kp + 1) * 2 + k_sel;
                ldmatrix_x4(kbase + k_row_off + (uint32_t)(c0 >> 3) * half_stride + (uint32_t)(((c0 & 7) ^ (k_row & 7)) << 4), a0);
                ldmatrix_x4(kbase + k_row_off + (uint32_t)(c1 >> 3) * half_stride + (uint32_t)(((c1 & 7) ^ (k_row & 7)) << 4), a1);
            }
            const int qc = kp * 4 + q_chunk;             // 16-byte chunk of the query row
            const uint32_t q_off = (uint32_t)(qc >> 3) * (kGroup * 128u) + (uint32_t)q_row * 128u +
                                   (uint32_t)(((qc & 7) ^ q_row) << 4);
            #pragma unroll
            for (int j = 0; j < NS; ++j) {
                if (j < mt.n) {
                    uint32_t qb[4];
                    ldmatrix_x4(qbase + j * kQTileBytes + q_off, qb);
                    mma_bf16(sc[j], a0, qb[0], qb[1]);
                    mma_bf16(sc[j], a1, qb[2], qb[3]);
                }
            }
        }
        // column maxima of this warp's block, per (sibling, head)
        #pragma unroll
        for (int j = 0; j < NS; ++j) {
            if (j < mt.n) {
                #pragma unroll
                for (int e = 0; e < 4; ++e) sc[j][e] *= p.scale_log2e;
                float b0 = fmaxf(sc[j][0], sc[j][2]), b1 = fmaxf(sc[j][1], sc[j][3]);
                #pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    b0 = fmaxf(b0, __shfl_xor_sync(0xffffffffu, b0, off));
                    b1 = fmaxf(b1, __shfl_xor_sync(0xffffffffu, b1, off));
                }
                if (qrow == 0) {
                    wmax[(warp * NS + j) * kGroup + 2 * quad] = b0;
                    wmax[(warp * NS + j) * kGroup + 2 * quad + 1] = b1;
                }
            }
        }
        mbar_arrive(sync_a);
        if (!mbar_wait(sync_a, syncs & 1u, abort_flag)) { fail(24); return; }
        // ---- phase 2: new running maxima, rescale, publish P
        #pragma unroll
        for (int j = 0; j < NS; ++j) {
            if (j < mt.n) {
                float n0 = m[j][0], n1 = m[j][1];
                #pragma unroll
                for (int w = 0; w < kPConsumerWarps; ++w) {
                    n0 = fmaxf(n0, wmax[(w * NS + j) * kGroup + 2 * quad]);
                    n1 = fmaxf(n1, wmax[(w * NS + j) * kGroup + 2 * quad + 1]);
                }
                const float a0 = fast_exp2(m[j][0] - n0), a1 = fast_exp2(m[j][1] - n1);
                m[j][0] = n0; m[j][1] = n1;
                const float p00 = fast_exp2(sc[j][0] - n0), p01 = fast_exp2(sc[j][1] - n1);
                const float p10 = fast_exp2(sc[j][2] - n0), p11 = fast_exp2(sc[j][3] - n1);
                l[j][0] = fmaf(l[j][0], a0, p00 + p10);
                l[j][1] = fmaf(l[j][1], a1, p01 + p11);
                #pragma unroll
                for (int db = 0; db < 2; ++db) { o[j][db][0] *= a0; o[j][db][1] *= a1; o[j][db][2] *= a0; o[j][db][3] *= a1; }
                // rows = heads, columns = this warp's tokens: transpose the two 8x8 blocks in registers
                const uint32_t t0 = movmatrix_trans(pack_bf16(p00, p01));
                const uint32_t t1 = movmatrix_trans(pack_bf16(p10, p11));
                const uint32_t dst = pbase + (uint32_t)(j * kGroup + qrow) * kPRowBytes + (uint32_t)(tok0 + 2 * quad) * 2u;
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst), "r"(t0) : "memory");
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst + 16u), "r"(t1) : "memory");
            }
        }
        mbar_arrive(sync_b);
        if (!mbar_wait(sync_b, syncs & 1u, abort_flag)) { fail(25); return; }
        ++syncs;
        if (!mbar_wait(full_v(s), parity, abort_flag)) { fail(26); return; }
        // ---- phase 3: O_j^T[32 dims of this warp] += V^T . P_j^T over the tile's 64 tokens
        #pragma unroll
        for (int tp = 0; tp < 2; ++tp) {                 // pairs of 16-token blocks
            uint32_t va[2][2][4];                        // [dim block][token block]
            #pragma unroll
            for (int db = 0; db < 2; ++db)
                #pragma unroll
                for (int tb = 0; tb < 2; ++tb) {
                    const int tok = (2 * tp + tb) * 16 + (lane & 7) + (lane >> 4) * 8;
                    const int chunk = (2 * warp + db) * 2 + ((lane >> 3) & 1);
                    const int rb = tok & (P - 1);
                    const uint32_t addr = vbase + (uint32_t)(tok >> p.box_shift) * (uint32_t)P * kRowBytes +
                                          (uint32_t)(chunk >> 3) * half_stride + (uint32_t)rb * 128u +
                                          (uint32_t)(((chunk & 7) ^ (rb & 7)) << 4);
                    ldmatrix_x4_trans(addr, va[db][tb]);
                }
            #pragma unroll
            for (int j = 0; j < NS; ++j) {
                if (j < mt.n) {
                    uint32_t pb[4];
                    ldmatrix_x4(pbase + (uint32_t)j * (kGroup * kPRowBytes) + p_lane_off + (uint32_t)tp * 64u, pb);
                    #pragma unroll
                    for (int db = 0; db < 2; ++db) {
                        mma_bf16(o[j][db], va[db][0], pb[0], pb[1]);
                        mma_bf16(o[j][db], va[db][1], pb[2], pb[3]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty(s));

        if (mt.last) {
            // ---- row sums over all tokens, then one normalised partial per sibling
            #pragma unroll
            for (int j = 0; j < NS; ++j) {
                if (j < mt.n) {
                    float l0 = l[j][0], l1 = l[j][1];
                    #pragma unroll
                    for (int off = 4; off < 32; off <<= 1) {
                        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
                    }
                    if (qrow == 0) {
                        lsum[(warp * NS + j) * kGroup + 2 * quad] = l0;
                        lsum[(warp * NS + j) * kGroup + 2 * quad + 1] = l1;
                    }
                }
            }
            mbar_arrive(sync_a);
            if (!mbar_wait(sync_a, syncs & 1u, abort_flag)) { fail(27); return; }
            #pragma unroll
            for (int j = 0; j < NS; ++j) {
                if (j < mt.n) {
                    float L0 = 0.f, L1 = 0.f;
                    #pragma unroll
                    for (int w = 0; w < kPConsumerWarps; ++w) {
                        L0 += lsum[(w * NS + j) * kGroup + 2 * quad];
                        L1 += lsum[(w * NS + j) * kGroup + 2 * quad + 1];
                    }
                    const float i0 = 1.f / L0, i1 = 1.f / L1;
                    if (!in_bounds(p.hdr, mt.row + j, c.max_rows, 301)) continue;
                    float* dst = c.pre_o + ((int64_t)(mt.row + j) * kGroup) * kD;
                    #pragma unroll
                    for (int db = 0; db < 2; ++db) {
                        const int d = warp * 32 + db * 16 + qrow;
                        dst[(2 * quad) * kD + d] = o[j][db][0] * i0;
                        dst[(2 * quad + 1) * kD + d] = o[j][db][1] * i1;
                        dst[(2 * quad) * kD + d + 8] = o[j][db][2] * i0;
                        dst[(2 * quad + 1) * kD + d + 8] = o[j][db][3] * i1;
                    }
                    if (warp == 0 && qrow == 0) {
                        c.pre_lse[(int64_t)(mt.row + j) * kGroup + 2 * quad] = m[j][0] + log2f(L0);
                        c.pre_lse[(int64_t)(mt.row + j) * kGroup + 2 * quad + 1] = m[j][1] + log2f(L1);
                    }
                }
            }
            mbar_arrive(sync_b);
            if (!mbar_wait(sync_b, syncs & 1u, abort_flag)) { fail(28); return; }
            ++syncs;
            __syncwarp();
            if (lane == 0) mbar_arrive(q_empty(mt.qsel));
            ++segs;
        }
    }
}

// ------------------------------------------------------------------ host side

namespace {

template <int NS>
cudaError_t launch_ns(const DecodeParams& p, const CascadeParams& c, const CUtensorMap& mk, const CUtensorMap& mv,
                      const CUtensorMap& mq, cudaStream_t stream) {
    cudaError_t e = cudaFuncSetAttribute(prefix_mma_kernel<NS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         PSmem<NS>::kBytes);
    if (e != cudaSuccess) return e;
    prefix_mma_kernel<NS><<<c.grid_ctas, kPThreads, PSmem<NS>::kBytes, stream>>>(p, c, mk, mv, mq);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefix_mma(const DecodeParams& p, const CascadeParams& c, cudaStream_t stream) {
    CUtensorMap mk, mv, mq;
    const uint64_t pool_rows = (uint64_t)p.num_pages * p.page_size * (p.token_major ? 1 : p.hkv);
    const uint32_t planes = p.token_major ? 2 * p.hkv : 2;
    if (!make_rows_map(&mk, p.k_pages, pool_rows, p.box_rows, 2, planes) ||
        !make_rows_map(&mv, p.v_pages, pool_rows, p.box_rows, 2, planes) ||
        !make_rows_map(&mq, p.q, (uint64_t)p.batch * p.hq, kGroup, 2))
        return cudaErrorInvalidValue;
    return launch_ns<kMaxShare>(p, c, mk, mv, mq, stream);
}

}  // namespace concur
