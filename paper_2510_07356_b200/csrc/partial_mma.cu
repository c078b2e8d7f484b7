// Split-KV partial kernel, tensor-core version (the default).
//
// One persistent CTA per SM: K and V tiles (64 tokens x 128 dims, 16 KB each) are streamed from the
// paged pools into a 5-stage shared-memory ring with TMA tensor copies (128-byte swizzle, one copy
// per (page, KV head) chunk).  Two sets of four consumer warps take alternate tiles; within a set
// each warp owns 16 tokens of the tile:
//
//   S^T[16 tok x 8 heads]  = K[16 tok x 128] . Q^T[128 x 8]        (8 mma.m16n8k16, bf16 -> fp32)
//   online softmax in fp32, base-2 domain, per-warp running max / sum
//   O^T[128 x 8 heads]    += V^T[128 x 16 tok] . P^T[16 tok x 8]   (8 mma.m16n8k16)
//
// so every K/V byte is fetched from HBM once and serves all 8 query heads of its GQA
// group.  Tokens sit on the MMA's M dimension and the 8 heads fill its N = 8 exactly; the
// probabilities go from accumulator layout to B-operand layout with two 8x8 register
// transposes.  When a segment (a run of tiles of one (sequence, KV head) unit inside a
// range of the plan) ends, the four warps' states are merged through shared memory and
// written either straight to out/lse (the segment was the whole unit) or to a partial
// slot; the CTA that finishes the last partial of a unit (an atomic ticket, no waiting)
// merges the unit's partials by their log-sum-exp and writes out/lse.
//
// The kernel is HBM-bound by design: ~32 issue slots per 8 KB of KV per warp; what matters
// is the depth of the TMA ring (192 KB in flight per SM) and that nothing stalls the
// producer (plan tables cached in shared memory, block-table entries prefetched 32 at a
// time, the next range claimed while the current one streams).
//
// Every wait is bounded: a wait that exceeds its limit sets CONCUR_FLAG_WAIT_LIMIT, raises
// a CTA-wide abort flag and every warp leaves; the producer first waits (bounded) for the
// copies it has in flight.
#include <cuda.h>

#include <atomic>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"

namespace concur {

namespace {

constexpr int kStages = 5;
constexpr int kSetWarps = 4;                           // warps of a consumer set: 16 tokens of a tile each
constexpr int kConsumerWarps = 2 * kSetWarps;          // set 0 (warps 0-3) takes even tiles, set 1 (warps 4-7) odd ones
constexpr int kProducerWarp = kConsumerWarps;          // warp 8
constexpr int kCombinerWarp = kConsumerWarps + 1;      // warp 9
constexpr int kCopyWarp0 = kConsumerWarps + 2;         // warps 10-13: helpers (copy issue; per-lane copies with small pages)
constexpr int kCopyWarps = 4;
constexpr int kThreads = (kConsumerWarps + 2 + kCopyWarps) * 32;
constexpr int kTileBytes = kTile * kRowBytes;             // 16 KB: one K or V tile
constexpr int kQBytes = kGroup * kRowBytes;               // 2 KB: the 8 query rows of a group
constexpr int kStageBytes = 2 * kTileBytes + kQBytes;     // K | V | Q
constexpr int kMergeStride = kD + 4;                      // floats per head row in the merge buffer
constexpr int kMergeBytes = kConsumerWarps * kGroup * kMergeStride * 4;
constexpr int kSmemBatch = 511;                           // sequences whose plan rows are cached in smem

struct StageMeta {
    int32_t b, g, slot;
    int32_t n_valid;       // valid tokens in the tile (1..64); 0 = no more work
    int32_t first;         // first tile of its segment
    int32_t last;          // bit 0: last tile of its segment; bit 1: parity of the tile's flat index
    int32_t unit_start;    // flat tile index of the unit's first tile
    int32_t tiles_b;       // tiles of the whole unit
    int32_t page[4];       // small pages: pool pages of the tile's boxes (for the copy helpers)
    int32_t new_row;       // fused append: row of the tile that is the sequence's new token, else -1
    int32_t new_page;      // ... and the pool page its slot is in (-1: not to be stored, the page id was bad)
    int32_t seg_new;       // fused append: 1 on a segment's first tile if the segment holds the unit's last tile
    int32_t row_in_page;   // first row of the tile inside its page (non-zero only for pages of more than 64 tokens)
};

// A finished partial segment handed from the consumer warps to the combiner warp.
struct CombineJob {
    int32_t b, g;
    int32_t unit_start, tiles_b;
    int32_t exit;          // 1 = the consumers are done; the combiner warp leaves
    int32_t pad[3];
};

struct Smem {
    // offsets from the 1024-aligned base
    static constexpr int kMergeOff = kStages * kStageBytes;
    static constexpr int kMlOff = kMergeOff + kMergeBytes;                       // [8 warps][8 heads][2]
    static constexpr int kPrefixOff = kMlOff + kConsumerWarps * kGroup * 2 * 4;  // [kSmemBatch + 1]
    static constexpr int kLenOff = kPrefixOff + (kSmemBatch + 1) * 4;            // [kSmemBatch + 1]
    static constexpr int kMetaOff = kLenOff + (kSmemBatch + 1) * 4;
    static constexpr int kBarOff = kMetaOff + kStages * (int)sizeof(StageMeta);  // full_k, full_v, empty, merge x2, job x2, sched
    static constexpr int kAbortOff = kBarOff + (4 * kStages + 4) * 8;            // abort flag
    static constexpr int kJobOff = kAbortOff + 16;                               // CombineJob
    static constexpr int kScanOff = kJobOff + 32;                                // per-warp totals of the tile scan
    static constexpr int kTotal = kScanOff + 128;
};
constexpr int kSmemBytes = Smem::kTotal + 1024;           // slack for the manual 1024-byte alignment
static_assert(kSmemBytes <= 232448, "exceeds the 227 KB a CTA may use");
// What the copies write and the fragment loads read stays inside the tile it belongs to, for every box
// size: a tile is 64 / P boxes of [2 halves][P rows][128 B]; the farthest byte a ldmatrix (or a lane copy,
// or the fused append's patch) touches is the last 16-byte piece of the last row of the second half of the
// last box.
constexpr int tile_extent(int P) { return (kTile / P - 1) * P * kRowBytes + P * 128 + (P - 1) * 128 + 7 * 16 + 16; }
static_assert(tile_extent(16) == kTileBytes && tile_extent(32) == kTileBytes && tile_extent(64) == kTileBytes,
              "a tile's boxes must fill exactly its 16 KB");
static_assert(2 * kTileBytes + kQBytes == kStageBytes && kGroup * kRowBytes == kQBytes, "stage = K tile | V tile | query rows");
static_assert(Smem::kMergeOff == kStages * kStageBytes && Smem::kMlOff - Smem::kMergeOff == kMergeBytes &&
              kMergeBytes >= kConsumerWarps * kGroup * kMergeStride * 4, "merge buffers follow the ring");
static_assert((int)sizeof(StageMeta) % 16 == 0 && Smem::kBarOff % 8 == 0, "records and barriers are aligned");

}  // namespace

__device__ __forceinline__ void partial_mma_body(const DecodeParams& p, const CUtensorMap& map_k,
                                                 const CUtensorMap& map_v, uint8_t* smem) {
    const uint32_t smem_base = smem_u32(smem);
    float* merge_o = reinterpret_cast<float*>(smem + Smem::kMergeOff);
    float* merge_ml = reinterpret_cast<float*>(smem + Smem::kMlOff);
    int32_t* sm_prefix = reinterpret_cast<int32_t*>(smem + Smem::kPrefixOff);
    int32_t* sm_len = reinterpret_cast<int32_t*>(smem + Smem::kLenOff);
    StageMeta* meta = reinterpret_cast<StageMeta*>(smem + Smem::kMetaOff);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(smem + Smem::kAbortOff);
    const uint32_t bar_base = smem_base + Smem::kBarOff;
    auto full_k = [&](int s) { return bar_base + 8u * s; };
    auto full_v = [&](int s) { return bar_base + 8u * (kStages + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
    const uint32_t merge_bar0 = bar_base + 8u * (3 * kStages);
    const uint32_t merge_bar1 = merge_bar0 + 8u;
    const uint32_t job_ready = merge_bar0 + 16u;      // consumers -> combiner: a job is posted
    const uint32_t job_taken = merge_bar0 + 24u;      // combiner -> consumers: the job slot is free again
    auto sched = [&](int s) { return merge_bar0 + 32u + 8u * s; };   // producer -> copy helpers: the stage's record is written
    volatile CombineJob* job_s = reinterpret_cast<volatile CombineJob*>(smem + Smem::kJobOff);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int32_t P = p.box_rows;            // rows per box: the unit of the shared-memory tile layout
    const int64_t max_len = (int64_t)p.bt_stride * p.page_size;
    const bool cached = p.batch <= kSmemBatch;
    // Small pages (16 or 32 tokens): a tile would be four or two TMA boxes per operand, and the copy
    // engine's cost per box caps the stream well below HBM speed.  There four helper warps copy a
    // quarter of the tile each (16 rows), 16 bytes per lane and instruction, into the same swizzled
    // layout; a tile's barrier then takes one arrival per copying lane (when that lane's copies have
    // landed) next to the producer's own.  (The producer used to copy one of the quarters itself; as
    // its time per tile is what the rate hangs on, giving that quarter to a fourth helper took 14 % off
    // a step with 16-token pages.)
    const bool lane_copy = p.lane_copy != 0;
    const uint64_t wait_ns = (uint64_t)p.wait_limit_ns;       // the roles' waits; the drain of copies in flight keeps 2 s
    constexpr uint32_t kCopyLanes = kCopyWarps * 32;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_k(s), lane_copy ? 1 + kCopyLanes : 1);
            mbar_init(full_v(s), lane_copy ? kCopyLanes : 1);
            mbar_init(sched(s), 1);
            mbar_init(empty(s), kConsumerWarps);       // the owning set when it is done, the other one when it has the record
        }
        mbar_init(merge_bar0, kConsumerWarps * 32);
        mbar_init(merge_bar1, kConsumerWarps * 32);
        mbar_init(job_ready, kConsumerWarps * 32);
        mbar_init(job_taken, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (p.group < kGroup) {
        // fewer than 8 heads per group: the query rows that no copy fills must at least be defined
        for (int i = tid; i < kStages * (kQBytes / 16); i += kThreads)
            reinterpret_cast<uint4*>(smem + (i / (kQBytes / 16)) * kStageBytes + 2 * kTileBytes)[i % (kQBytes / 16)] =
                make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // Launched as the plan kernel's programmatic dependent, this kernel may run before the plan has
    // finished.  In the plain step with a batch that fits the shared-memory tables it does not wait for
    // it: the tile counts, their prefix and the range count follow from seq_lens alone, so every CTA
    // works them out for itself (same arithmetic as the plan kernel) and starts streaming at once.
    // What does depend on the plan kernel is its resets -- the claim counter and the per-unit ticket
    // counters -- so each thread executes griddepcontrol.wait before its first atomic on either and
    // before its first global store.  In the other modes the wait comes first and the tables are read.
    const bool self_plan = cached && p.tok_offset == nullptr && !p.all_partial;
    bool plan_seen = !self_plan;
    int32_t W, R;
    // (opt-in) the next launch on the stream may begin while this one drains: its CTAs take the SMs this
    // launch's CTAs leave, fill their rings, and wait for this grid's end before their first claim or store
    if (p.overlap_next) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (self_plan) {
        int32_t* scan_ws = reinterpret_cast<int32_t*>(smem + Smem::kScanOff);
        if (tid == 0) sm_prefix[0] = 0;
        int32_t carry = 0, longest = 0;
        for (int base = 0; base < p.batch; base += kThreads) {
            const int b = base + tid;
            int32_t v = 0;
            if (b < p.batch) {
                const int64_t nn = p.seq_lens[b];
                const int32_t n = (int32_t)(nn < 0 ? 0 : (nn > max_len ? max_len : nn));
                // without a plan kernel, CTA 0 is the one that reports a length outside [0, stride * P]
                if (p.no_plan_launch && blockIdx.x == 0 && n != nn)
                    atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagBadLen);
                sm_len[b] = n;
                v = (n + kTile - 1) / kTile;
            }
            int32_t mx = v;
            #pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            #pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t up = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v += up;
            }
            if (lane == 31) { scan_ws[warp] = v; scan_ws[kThreads / 32 + warp] = mx; }
            __syncthreads();
            int32_t before = 0, total = 0;
            #pragma unroll
            for (int w2 = 0; w2 < kThreads / 32; ++w2) {
                const int32_t x = scan_ws[w2];
                total += x;
                if (w2 < warp) before += x;
                longest = max(longest, scan_ws[kThreads / 32 + w2]);
            }
            if (b < p.batch) sm_prefix[b + 1] = carry + before + v;
            carry += total;
            __syncthreads();
        }
        W = p.hkv * carry;
        R = plan_num_ranges(p, W, longest);
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        W = p.hdr[kHdrTotalTiles];
        R = p.hdr[kHdrNumRanges];
        if (cached) {
            for (int i = tid; i <= p.batch; i += kThreads) sm_prefix[i] = p.tiles_prefix[i];
            for (int i = tid; i < p.batch; i += kThreads) {
                int64_t n = p.seq_lens[i];
                sm_len[i] = (int32_t)(n < 0 ? 0 : (n > max_len ? max_len : n));
            }
        }
        __syncthreads();
    }
    auto see_plan = [&]() {
        if (!plan_seen) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            plan_seen = true;
        }
    };
    const int32_t* prefix = cached ? sm_prefix : p.tiles_prefix;
    // The next range nobody has.  After a plan kernel the counter starts at the grid size (CTA i began on
    // range i).  Without one there is nobody to reset a counter, so: with no more ranges than CTAs
    // there is nothing to claim and no counter is touched; otherwise the counter counts this launch's
    // claims from 0, and since every range that is streamed claims exactly once, the claim that draws
    // R - 1 is the launch's last and puts the counter back to 0 for the next launch.
    auto claim_range = [&]() -> int32_t {
        if (!p.no_plan_launch) return atomicAdd(p.hdr + kHdrClaim, 1);
        if (R <= (int32_t)gridDim.x) return R;
        const int32_t c = atomicAdd(p.hdr + kHdrClaimSelf, 1);
        if (c == R - 1) atomicExch(p.hdr + kHdrClaimSelf, 0);
        return (int32_t)gridDim.x + c;
    };

    // lane_copy: one instruction moves two 256-byte rows (lanes 0-15 the even row, 16-31 the odd
    // one), 16-byte piece c16 of a row each.  In a box's [half][row][128 B] layout with the
    // 128-byte swizzle, piece (half h, c) of row r sits at h*P*128 + r*128 + ((c ^ (r & 7)) << 4);
    // for r = r0 + 2j + hi (r0 a multiple of 8) that is the per-lane term below + r0*128 + 256 j,
    // with bits 4-6 xor-ed by (2j & 6).  Quarter w of a tile = its rows 16w .. 16w+15.
    auto copy_quarter = [&](int s, int w, int32_t n_valid, int32_t g, int32_t page) {
        const uint32_t hi = lane >> 4, c16 = lane & 15;
        const uint32_t soff = (c16 >> 3) * (uint32_t)P * 128u + hi * 128u + (((c16 & 7u) ^ hi) << 4);
        const uint32_t row_bytes = p.token_major ? (uint32_t)(p.hkv * kRowBytes) : (uint32_t)kRowBytes;
        const int32_t row0 = 16 * w;                              // first row of the quarter in its tile
        const bool live = row0 < ((n_valid + P - 1) & ~(P - 1));  // whole boxes are read, as the TMA path does
        const int32_t rb = row0 & (P - 1);                        // ... and in its page
        const uint32_t d0 = smem_base + s * kStageBytes + (uint32_t)(row0 >> p.box_shift) * ((uint32_t)P * kRowBytes) +
                            soff + (uint32_t)rb * 128u;
        const int64_t e0 = pool_elem(p, page, g, rb) * 2 + hi * row_bytes + c16 * 16u;
        #pragma unroll
        for (int op = 0; op < 2; ++op) {                          // K, then V
            if (live) {
                const uint8_t* src = reinterpret_cast<const uint8_t*>(op == 0 ? p.k_pages : p.v_pages) + e0;
                const uint32_t d = d0 + op * kTileBytes;
                #pragma unroll
                for (int j = 0; j < 8; ++j)
                    lane_copy16((d + j * 256u) ^ ((2u * j & 6u) << 4), src + (size_t)(2 * j) * row_bytes);
            }
            lane_copy_arrive(op == 0 ? full_k(s) : full_v(s));
        }
    };

    if (warp >= kCopyWarp0) {
        // =========================================================== helper warps
        if (!lane_copy) {
            // Pages of 64 tokens or more: the producer only keeps the books (ranges, segments, page ids, the
            // tile's record); the first helper issues the K copy (and a segment's query rows) of every tile
            // from that record, the second one the V copy.  Arming a barrier and issuing a tensor copy are
            // slow serial steps of one thread; with all of them in the producer its time per tile, not HBM,
            // set the kernel's rate (the step time times the SM clock was a constant).
            if (warp > kCopyWarp0 + 1) return;
            const bool is_k = warp == kCopyWarp0;
            const uint32_t box_bytes = (uint32_t)P * kRowBytes;
            uint32_t it = 0;
            bool ok = true;
            for (;; ++it) {
                const int s = it % kStages;
                ok = mbar_wait(sched(s), (it / kStages) & 1u, abort_flag, wait_ns);
                if (!ok) break;
                const int32_t n_valid = meta[s].n_valid;
                if (n_valid == 0) return;
                if (lane == 0) {
                    const int32_t npages = (n_valid + P - 1) >> p.box_shift;
                    const int32_t g = meta[s].g, rip = meta[s].row_in_page;
                    const uint32_t kdst = smem_base + s * kStageBytes;
                    if (is_k) {
                        const bool with_q = meta[s].first != 0;
                        const uint32_t q_bytes = (uint32_t)p.group * kRowBytes;
                        mbar_arrive_expect_tx(full_k(s), npages * box_bytes + (with_q ? q_bytes : 0u));
                        if (with_q)
                            bulk_load(kdst + 2 * kTileBytes, p.q + ((int64_t)meta[s].b * p.hq + g * p.group) * kD, q_bytes, full_k(s));
                        for (int i = 0; i < npages; ++i)
                            tma_load_tile(kdst + i * box_bytes, &map_k, pool_row(p, meta[s].page[i], g, rip), full_k(s), pool_plane(p, g));
                    } else {
                        mbar_arrive_expect_tx(full_v(s), npages * box_bytes);
                        for (int i = 0; i < npages; ++i)
                            tma_load_tile(kdst + kTileBytes + i * box_bytes, &map_v, pool_row(p, meta[s].page[i], g, rip), full_v(s), pool_plane(p, g));
                    }
                }
                __syncwarp();
            }
            // a wait gave up (here or elsewhere in the CTA): let this warp's copies in flight land before
            // the CTA's shared memory is released
            if (lane == 0) {
                wait_failed(p, abort_flag, 11);
                volatile int32_t never = 0;
                for (uint32_t j = it > (uint32_t)kStages ? it - kStages : 0u; j < it; ++j)
                    mbar_wait(is_k ? full_k(j % kStages) : full_v(j % kStages), (j / kStages) & 1u, &never);
            }
            return;
        }
        const int w = warp - kCopyWarp0;
        for (uint32_t it = 0;; ++it) {
            const int s = it % kStages;
            if (!mbar_wait(sched(s), (it / kStages) & 1u, abort_flag, wait_ns)) {
                if (lane == 0) wait_failed(p, abort_flag, 10);
                return;
            }
            const int32_t n_valid = meta[s].n_valid;
            if (n_valid == 0) return;
            copy_quarter(s, w, n_valid, meta[s].g, meta[s].page[(16 * w) >> p.box_shift]);
        }
    }

    if (warp == kProducerWarp) {
        // =========================================================== producer warp
        uint32_t it = 0;                       // tiles issued so far
        int32_t r = blockIdx.x;                // CTA i starts on range i; further ranges are claimed
        bool ok = true;
        const int32_t page_mask = p.page_size - 1;
        while (ok && r < R) {
            // the next range is claimed a few tiles before this one ends: late enough that no
            // CTA sits on work another could start, early enough to hide the atomic's latency
            int32_t r_next = 0;
            bool claimed = false;
            const int32_t x0 = range_begin(W, R, r);
            const int32_t x1 = range_begin(W, R, r + 1);
            int32_t x = x0;
            while (ok && x < x1) {
                const Segment sg = segment_at(prefix, p.batch, p.hkv, r, x0, x1, x, p.all_partial);
                x += sg.tile1 - sg.tile0;
                int32_t n;                // tokens of the sequence that this pass covers
                if (cached) n = sm_len[sg.b];
                else { int64_t nn = p.seq_lens[sg.b]; n = (int32_t)(nn < 0 ? 0 : (nn > max_len ? max_len : nn)); }
                // cascade mode: the first `off` tokens (a multiple of 64) belong to the prefix pass
                const int32_t off = p.tok_offset ? p.tok_offset[sg.b] : 0;
                n -= off;
                const int32_t* table = p.block_table + (int64_t)sg.b * p.bt_stride;
                // pages used by the segment (a page holds one or more boxes; a 128-token page two tiles)
                const int32_t page_end = (off + min(sg.tile1 * kTile, n) + page_mask) >> p.page_shift;
                int32_t chunk_base = (off + sg.tile0 * kTile) >> p.page_shift;
                // this lane's entry of the current 32-page chunk of the block table, and of the
                // chunk after it (fetched one chunk early so that its latency never stalls the ring)
                int32_t pg = (chunk_base + lane < page_end) ? __ldg(table + chunk_base + lane) : 0;
                int32_t pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                const int32_t unit_start = x - sg.tile1;      // x already points past the segment
                for (int32_t t = sg.tile0; ok && t < sg.tile1; ++t) {
                    // (a CTA that has not waited for the plan kernel yet first fills its ring)
                    if (!claimed && x1 - (unit_start + t) <= p.claim_ahead &&
                        (plan_seen || unit_start + t - x0 >= kStages || unit_start + t == x1 - 1)) {
                        see_plan();
                        if (lane == 0) r_next = claim_range();
                        claimed = true;
                    }
                    const int32_t tok_abs = off + t * kTile;               // first token of the tile in its sequence
                    const int32_t first_page = tok_abs >> p.page_shift;
                    const int32_t row_in_page = tok_abs & page_mask;       // non-zero only for pages of more than 64 tokens
                    if (first_page >= chunk_base + 32) {
                        chunk_base += 32;
                        pg = pg_next;
                        pg_next = (chunk_base + 32 + lane < page_end) ? __ldg(table + chunk_base + 32 + lane) : 0;
                    }
                    const int32_t n_valid = min(kTile, n - t * kTile);
                    const int32_t npages = (n_valid + P - 1) >> p.box_shift;      // boxes of the tile that are read
                    const int s = it % kStages;
                    const uint32_t parity = (it / kStages) & 1u;
                    // page ids of this tile, clamped into the pool
                    int32_t my_page = __shfl_sync(0xffffffffu, pg, (first_page - chunk_base + (lane & 3)) & 31);
                    bool bad = (lane < npages) && (my_page < 0 || my_page >= p.num_pages);
                    if (__any_sync(0xffffffffu, bad)) {
                        if (lane == 0) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagBadPage);
                        if (my_page < 0 || my_page >= p.num_pages) my_page = 0;
                    }
                    // (fused append: was the page of the tile's last token among the clamped ones?)
                    const bool new_page_bad = __shfl_sync(0xffffffffu, (int)bad, (n_valid - 1) >> p.box_shift) != 0;
                    const int32_t page0 = __shfl_sync(0xffffffffu, my_page, 0);
                    const int32_t page1 = __shfl_sync(0xffffffffu, my_page, 1);
                    const int32_t page2 = __shfl_sync(0xffffffffu, my_page, 2);
                    const int32_t page3 = __shfl_sync(0xffffffffu, my_page, 3);
                    if (lane == 0) {
                        ok = mbar_wait(empty(s), parity ^ 1u, abort_flag, wait_ns);
                        if (ok) {
                            StageMeta& m = meta[s];
                            m.b = sg.b; m.g = sg.g; m.slot = sg.slot; m.n_valid = n_valid;
                            m.first = (t == sg.tile0);
                            m.last = (t == sg.tile1 - 1 ? 1 : 0) | (((unit_start + t) & 1) << 1);
                            m.unit_start = unit_start; m.tiles_b = sg.tiles_b;
                            m.page[0] = page0; m.page[1] = page1; m.page[2] = page2; m.page[3] = page3;
                            // fused append: the sequence's last token sits in the unit's last tile
                            const bool new_here = p.k_new != nullptr && t == sg.tiles_b - 1;
                            const int32_t new_row = n_valid - 1;
                            const int32_t new_box = new_row >> p.box_shift;
                            const int32_t new_page = new_box == 0 ? page0 : (new_box == 1 ? page1 : (new_box == 2 ? page2 : page3));
                            m.new_row = new_here ? new_row : -1;
                            m.new_page = (new_here && !new_page_bad) ? new_page : -1;
                            m.seg_new = (p.k_new != nullptr && sg.tile1 == sg.tiles_b) ? 1 : 0;
                            m.row_in_page = row_in_page;
                            if (lane_copy) {
                                // small pages: the query rows by a bulk copy from here; the tile itself by the
                                // per-lane copies of the four helper warps
                                const uint32_t kdst = smem_base + s * kStageBytes;
                                const bool with_q = (t == sg.tile0);
                                const uint32_t q_bytes = (uint32_t)p.group * kRowBytes;
                                if (with_q) mbar_arrive_expect_tx(full_k(s), q_bytes);
                                else mbar_arrive(full_k(s));
                                if (with_q)
                                    bulk_load(kdst + 2 * kTileBytes, p.q + ((int64_t)sg.b * p.hq + sg.g * p.group) * kD,
                                              q_bytes, full_k(s));
                            }
                            mbar_arrive(sched(s));          // the helper warps may read the record (and issue the copies)
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (ok) ++it;
                }
            }
            // Whatever claim_ahead is, a range never ends without its successor claimed: a CTA that
            // streamed a range to its end and found no claim condition met (claim_ahead below 1) takes
            // its ticket here, so the loop always moves on to a range nobody else has.
            if (ok && !claimed) {
                see_plan();
                if (lane == 0) r_next = claim_range();
                claimed = true;
            }
            r = __shfl_sync(0xffffffffu, r_next, 0);
        }
        if (lane == 0) {
            if (ok) {
                // tell the consumers that there is no more work
                const int s = it % kStages;
                const uint32_t parity = (it / kStages) & 1u;
                ok = mbar_wait(empty(s), parity ^ 1u, abort_flag, wait_ns);
                if (ok) {
                    meta[s].n_valid = 0;
                    mbar_arrive_n(full_k(s), lane_copy ? 1 + kCopyLanes : 1);
                    mbar_arrive(sched(s));
                }
            }
            if (!ok) {
                wait_failed(p, abort_flag, 1);
                // let the copies still in flight land before the CTA's shared memory is released (small pages:
                // this warp's own; otherwise the helper warps issued them and wait for them)
                const uint32_t lo = it > (uint32_t)kStages ? it - kStages : 0u;
                for (uint32_t j = lane_copy ? lo : it; j < it; ++j) {
                    volatile int32_t never = 0;
                    mbar_wait(full_k(j % kStages), (j / kStages) & 1u, &never);
                    mbar_wait(full_v(j % kStages), (j / kStages) & 1u, &never);
                }
            }
        }
        return;
    }

    if (warp == kCombinerWarp) {
        // =========================================================== combiner warp
        // Takes the jobs the consumers post.  Each job is one finished partial of a unit that
        // the plan split over several ranges: an atomic ticket on the unit's counter tells
        // whether it was the unit's last one, and if so this warp merges the unit's partials
        //   L = log2 sum_s 2^{lse_s},  out = sum_s 2^{lse_s - L} out_s,  lse = L ln 2
        // with a running maximum, 4 dims per lane, all 8 heads in flight at once.
        const float ninf_c = -INFINITY;
        see_plan();
        if (p.no_plan_launch && blockIdx.x == 0) {
            // What the plan kernel would have written besides its tables: the results of sequences without
            // cached tokens, and (when this launch planned for itself) W, R and the range boundaries, which
            // the plan query reads back.
            if (self_plan) {
                if (lane == 0) { p.hdr[kHdrTotalTiles] = W; p.hdr[kHdrNumRanges] = R; }
                for (int32_t r = lane; r <= R; r += 32) p.range_start[r] = R > 0 ? range_begin(W, R, r) : 0;
            }
            for (int32_t b0 = 0; b0 < p.batch; b0 += 32) {
                const int32_t b = b0 + lane;
                int32_t n = 1;
                if (b < p.batch) n = cached ? sm_len[b] : max(0, p.seq_lens[b]);
                unsigned empties = __ballot_sync(0xffffffffu, n == 0);
                while (empties) {
                    const int e = b0 + (__ffs(empties) - 1);
                    empties &= empties - 1;
                    uint4* o = reinterpret_cast<uint4*>(p.out + (int64_t)e * p.hq * kD);
                    for (int i = lane; i < p.hq * kD / 8; i += 32) o[i] = make_uint4(0, 0, 0, 0);
                    for (int i = lane; i < p.hq; i += 32) p.lse[(int64_t)e * p.hq + i] = ninf_c;
                }
            }
        }
        for (uint32_t jobn = 0;; ++jobn) {
            if (!mbar_wait(job_ready, jobn & 1u, abort_flag, wait_ns)) {
                if (lane == 0) wait_failed(p, abort_flag, 8);
                return;
            }
            const int32_t jb = job_s->b, jg = job_s->g, ju = job_s->unit_start, jt = job_s->tiles_b;
            const int32_t jexit = job_s->exit;
            __syncwarp();
            if (lane == 0) mbar_arrive(job_taken);
            if (jexit) return;
            int32_t ticket = 0;
            if (!in_bounds(p.hdr, jb * p.hkv + jg, (int64_t)p.batch * p.hkv, 101)) continue;
            if (lane == 0)
                asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;"
                             : "=r"(ticket) : "l"(p.unit_done + jb * p.hkv + jg), "r"(1) : "memory");
            ticket = __shfl_sync(0xffffffffu, ticket, 0);
            __syncwarp();
            const int32_t r_lo = range_of(W, R, ju);
            const int32_t r_hi = range_of(W, R, ju + jt - 1);
            const int32_t splits = r_hi - r_lo + 1;
            if (ticket != splits - 1) continue;
            // every ticket of this unit has been drawn: the counter goes back to 0 for the next launch
            if (lane == 0) p.unit_done[jb * p.hkv + jg] = 0;
            // the unit's segment in range r is that range's first (slot 2r) unless the range
            // began before the unit did, which can only be the case for r_lo
            const int32_t slot_lo = 2 * r_lo + (range_begin(W, R, r_lo) < ju ? 1 : 0);
            float mx[kGroup], z[kGroup];
            float4 acc[kGroup];
            #pragma unroll
            for (int h = 0; h < kGroup; ++h) { mx[h] = ninf_c; z[h] = 0.f; acc[h] = make_float4(0.f, 0.f, 0.f, 0.f); }
            #pragma unroll 2
            for (int32_t i = 0; i < splits; ++i) {
                const int64_t slot = i ? 2 * (int64_t)(r_lo + i) : slot_lo;
                if (!in_bounds(p.hdr, slot, p.slot_cap, 102)) continue;
                const float4* lp = reinterpret_cast<const float4*>(p.part_lse + slot * kGroup);
                const float4 la = __ldcg(lp), lb = __ldcg(lp + 1);
                const float l8[kGroup] = {la.x, la.y, la.z, la.w, lb.x, lb.y, lb.z, lb.w};
                float4 v[kGroup];
                #pragma unroll
                for (int h = 0; h < kGroup; ++h)
                    v[h] = __ldcg(reinterpret_cast<const float4*>(p.part_o + (slot * kGroup + h) * kD) + lane);
                #pragma unroll
                for (int h = 0; h < kGroup; ++h) {
                    const float mn = fmaxf(mx[h], l8[h]);
                    const float a = fast_exp2(mx[h] - mn), wt = fast_exp2(l8[h] - mn);
                    mx[h] = mn;
                    z[h] = fmaf(z[h], a, wt);
                    acc[h].x = fmaf(acc[h].x, a, wt * v[h].x); acc[h].y = fmaf(acc[h].y, a, wt * v[h].y);
                    acc[h].z = fmaf(acc[h].z, a, wt * v[h].z); acc[h].w = fmaf(acc[h].w, a, wt * v[h].w);
                }
            }
            #pragma unroll
            for (int h = 0; h < kGroup; ++h) {
                if (h >= p.group) break;
                const float inv = 1.f / z[h];
                const int64_t row = (int64_t)jb * p.hq + jg * p.group + h;
                if (!in_bounds(p.hdr, row, p.out_rows, 103)) continue;
                uint2 packed;
                packed.x = pack_bf16(acc[h].x * inv, acc[h].y * inv);
                packed.y = pack_bf16(acc[h].z * inv, acc[h].w * inv);
                reinterpret_cast<uint2*>(p.out + row * kD)[lane] = packed;
                if (lane == 0) p.lse[row] = (mx[h] + log2f(z[h])) * 0.6931471805599453f;
            }
        }
    }

    // =============================================================== consumer warps
    const int quad = lane & 3;           // selects this thread's two heads: 2*quad, 2*quad + 1
    const int qrow = lane >> 2;          // row inside an 8-row fragment block
    const float ninf = -INFINITY;
    // per-lane pieces of the swizzled tile addresses (see the layout note at tma_load_tile):
    // a 64-token tile is 64/P boxes; a box is [2 halves][P rows][128 B], 16-byte chunks of a
    // row XOR-ed with (row & 7)
    // Two sets: a warp's work on a tile is one dependent chain (fragment loads, 8 MMAs, shuffles, exponentials,
    // transposes, 8 MMAs) with nothing of its own to overlap it with; two sets, each with its own running
    // state, halve the time the consumer side needs per tile.
    const int set = warp / kSetWarps;                             // this warp's set: tiles whose flat index has this parity
    const int tok0 = (warp % kSetWarps) * 16;                     // this warp's first token in the tile
    const uint32_t box_off = (uint32_t)(tok0 >> p.box_shift) * (uint32_t)P * kRowBytes;
    const uint32_t half_stride = (uint32_t)P * 128u;
    const int rb0 = tok0 & (P - 1);
    // K fragments (non-transposed): matrices (rows 0-7 | 8-15) x (k 0-7 | 8-15)
    const int k_row = rb0 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t k_row_off = box_off + (uint32_t)k_row * 128u;
    const int k_sel = lane >> 4;                                  // 16-byte chunk inside the 32-byte k-step
    // V fragments (transposed): matrices (tok 0-7 | 8-15) x (d 0-7 | 8-15), ordered for A = V^T
    const int v_row = rb0 + (lane & 7) + (lane >> 4) * 8;
    const uint32_t v_row_off = box_off + (uint32_t)v_row * 128u;
    const int v_sel = (lane >> 3) & 1;

    uint32_t qf[8][2];
    float m0 = ninf, m1 = ninf, l0 = 0.f, l1 = 0.f;
    float o[8][4];
    #pragma unroll
    for (int i = 0; i < 8; ++i) { qf[i][0] = qf[i][1] = 0u; o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    uint32_t merges = 0, jobs = 0;
    uint4 new_piece = make_uint4(0, 0, 0, 0);        // fused append: this lane's piece of the new token's K or V row

    for (uint32_t it = 0;; ++it) {
        const int s = it % kStages;
        const uint32_t parity = (it / kStages) & 1u;
        if (!mbar_wait(full_k(s), parity, abort_flag, wait_ns)) {
                if (lane == 0) wait_failed(p, abort_flag, 2);
                return;
        }
        const StageMeta mt = meta[s];
        if (mt.n_valid == 0) {
            // no more work: tell the combiner warp to leave once it has taken the last job.
            // All consumer threads meet first, so that no exit arrival can be counted into a
            // job phase that thread 0 (which may still be waiting to post it) has not joined.
            mbar_arrive(merge_bar0);
            if (!mbar_wait(merge_bar0, merges & 1u, abort_flag, wait_ns)) {
                if (lane == 0) wait_failed(p, abort_flag, 9);
                return;
            }
            if (tid == 0) {
                if (mbar_wait(job_taken, (jobs & 1u) ^ 1u, abort_flag, wait_ns)) job_s->exit = 1;
                else wait_failed(p, abort_flag, 7);
            }
            mbar_arrive(job_ready);
            return;
        }
        const uint32_t kbase = smem_base + s * kStageBytes;
        const uint32_t vbase = kbase + kTileBytes;
        // Both sets walk every tile's record: the segment's first tile carries its query rows (the set
        // that does not own that tile needs them for the next one) and starts both sets' states afresh,
        // and its last tile is where both meet for the merge.
        // Which set takes a tile follows from the tile's place in the flat tile space, not from how many tiles
        // this CTA happens to have seen: the grouping of a segment's sums, and with it every bit of the
        // result, is then the same from launch to launch whichever CTA claims which range.  (Consecutive
        // tiles still alternate; only at a jump to another range may one set get two tiles in a row.)
        const bool mine = ((mt.last >> 1) & 1) == set;
        if (mt.first) {
            const uint32_t* qs = reinterpret_cast<const uint32_t*>(smem + s * kStageBytes + 2 * kTileBytes);
            #pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                qf[ks][0] = qs[qrow * (kD / 2) + ks * 8 + quad];
                qf[ks][1] = qs[qrow * (kD / 2) + ks * 8 + quad + 4];
            }
            m0 = m1 = ninf; l0 = l1 = 0.f;
            #pragma unroll
            for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
            // fused append: this segment ends with the sequence's new token, whose rows come from k_new /
            // v_new; fetch them now (lanes 0-15 a 16-byte piece of the K row each, lanes 16-31 of the V row)
            // so that they are in registers by the time the last tile is
            if (mt.seg_new)
                new_piece = __ldg(reinterpret_cast<const uint4*>(
                    (lane < 16 ? p.k_new : p.v_new) + ((int64_t)mt.b * p.hkv + mt.g) * kD + (lane & 15) * 8));
        }
        const int valid = mine ? mt.n_valid - tok0 : 0;          // valid tokens among this warp's 16
        // Fused append (one tile per unit, none in any other call): the tile holds the sequence's new token.
        // The pool's slot has not been written yet, so the warp that owns the row puts the K row (here) and the
        // V row (below, once V has landed) where the copy left the slot's old contents, and stores both rows
        // into the pools for the steps to come.  patch_off: where the 16-byte piece (lane & 15) of the row sits
        // in a swizzled tile.
        bool patch = false;
        uint32_t patch_off = 0;
        if (mt.new_row >= 0 && mine) {
            patch = mt.new_row >= tok0 && mt.new_row < tok0 + 16;
            patch_off = (uint32_t)(mt.new_row >> p.box_shift) * (uint32_t)P * kRowBytes +
                        (uint32_t)((lane & 15) >> 3) * half_stride + (uint32_t)(mt.new_row & (P - 1)) * 128u +
                        (uint32_t)((((lane & 15) & 7) ^ (mt.new_row & 7)) << 4);
            if (patch) {
                if (lane < 16)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(kbase + patch_off), "r"(new_piece.x),
                                 "r"(new_piece.y), "r"(new_piece.z), "r"(new_piece.w) : "memory");
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (mt.new_page >= 0 && in_bounds(p.hdr, mt.new_page, p.num_pages, 106) &&
                    in_bounds(p.hdr, patch_off, kTileBytes - 15, 108)) {
                    see_plan();
                    const int32_t new_slot = (mt.row_in_page + mt.new_row) & (p.page_size - 1);
                    __nv_bfloat16* pool = lane < 16 ? const_cast<__nv_bfloat16*>(p.k_pages) : const_cast<__nv_bfloat16*>(p.v_pages);
                    *reinterpret_cast<uint4*>(pool + pool_elem(p, mt.new_page, mt.g, new_slot) + (lane & 15) * 8) = new_piece;
                }
            }
        }
        if (valid > 0) {
            // ---- S^T = K . Q^T  (two accumulator chains to shorten the dependency)
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
            #pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const int chunk = ks * 2 + k_sel;
                const uint32_t addr = kbase + k_row_off + (uint32_t)(chunk >> 3) * half_stride +
                                      (uint32_t)(((chunk & 7) ^ (k_row & 7)) << 4);
                uint32_t a[4];
                ldmatrix_x4(addr, a);
                if (ks & 1) mma_bf16(sb, a, qf[ks][0], qf[ks][1]);
                else mma_bf16(sa, a, qf[ks][0], qf[ks][1]);
            }
            // scores of tokens (qrow, qrow + 8) for heads (2 quad, 2 quad + 1), base-2 domain
            float s00 = (sa[0] + sb[0]) * p.scale_log2e, s01 = (sa[1] + sb[1]) * p.scale_log2e;
            float s10 = (sa[2] + sb[2]) * p.scale_log2e, s11 = (sa[3] + sb[3]) * p.scale_log2e;
            if (qrow >= valid) { s00 = ninf; s01 = ninf; }
            if (qrow + 8 >= valid) { s10 = ninf; s11 = ninf; }
            float bm0 = fmaxf(s00, s10), bm1 = fmaxf(s01, s11);
            #pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, off));
                bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, off));
            }
            const float n0 = fmaxf(m0, bm0), n1 = fmaxf(m1, bm1);
            if (__any_sync(0xffffffffu, (n0 != m0) || (n1 != m1))) {
                const float a0 = fast_exp2(m0 - n0), a1 = fast_exp2(m1 - n1);   // exp2(-inf) = 0 on first use
                l0 *= a0; l1 *= a1;
                #pragma unroll
                for (int i = 0; i < 8; ++i) { o[i][0] *= a0; o[i][1] *= a1; o[i][2] *= a0; o[i][3] *= a1; }
                m0 = n0; m1 = n1;
            }
            const float p00 = fast_exp2(s00 - m0), p01 = fast_exp2(s01 - m1);
            const float p10 = fast_exp2(s10 - m0), p11 = fast_exp2(s11 - m1);
            l0 += p00 + p10;
            l1 += p01 + p11;
            // P^T as the B operand: transpose the two 8x8 (token x head) blocks in registers
            const uint32_t pb0 = movmatrix_trans(pack_bf16(p00, p01));
            const uint32_t pb1 = movmatrix_trans(pack_bf16(p10, p11));

            if (!mbar_wait(full_v(s), parity, abort_flag, wait_ns)) {
                if (lane == 0) wait_failed(p, abort_flag, 3);
                return;
            }
            if (valid < 16) {
                // rows past the end of the sequence may hold anything (NaN included) and a zero
                // probability does not silence them inside an MMA: clear them first
                for (int i = lane; i < (16 - valid) * 16; i += 32) {
                    const int row = rb0 + valid + (i >> 4);
                    const int c = i & 15;
                    const uint32_t addr = vbase + box_off + (uint32_t)(c >> 3) * half_stride + (uint32_t)row * 128u +
                                          (uint32_t)((c & 7) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }
            if (patch) {
                if (lane >= 16)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(vbase + patch_off), "r"(new_piece.x),
                                 "r"(new_piece.y), "r"(new_piece.z), "r"(new_piece.w) : "memory");
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }
            // ---- O^T += V^T . P^T
            #pragma unroll
            for (int db = 0; db < 8; ++db) {
                const int chunk = db * 2 + v_sel;
                const uint32_t addr = vbase + v_row_off + (uint32_t)(chunk >> 3) * half_stride +
                                      (uint32_t)(((chunk & 7) ^ (v_row & 7)) << 4);
                uint32_t a[4];
                ldmatrix_x4_trans(addr, a);
                mma_bf16(o[db], a, pb0, pb1);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty(s));

        if (mt.last & 1) {
            // ---- merge the eight warps' states (both sets) and write the segment's result
            see_plan();
            #pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                l1 += __shfl_xor_sync(0xffffffffu, l1, off);
            }
            float* mo = merge_o + warp * (kGroup * kMergeStride);
            #pragma unroll
            for (int db = 0; db < 8; ++db) {
                const int d = db * 16 + qrow;
                mo[(2 * quad) * kMergeStride + d] = o[db][0];
                mo[(2 * quad + 1) * kMergeStride + d] = o[db][1];
                mo[(2 * quad) * kMergeStride + d + 8] = o[db][2];
                mo[(2 * quad + 1) * kMergeStride + d + 8] = o[db][3];
            }
            if (qrow == 0) {
                float* ml = merge_ml + (warp * kGroup + 2 * quad) * 2;
                ml[0] = m0; ml[1] = l0; ml[2] = m1; ml[3] = l1;
            }
            mbar_arrive(merge_bar0);
            if (!mbar_wait(merge_bar0, merges & 1u, abort_flag, wait_ns)) {
                if (lane == 0) wait_failed(p, abort_flag, 4);
                return;
            }
            // 256 consumer threads = 8 heads x 32 threads; a thread owns dims 4j .. 4j+3 of one head (a warp
            // reads 512 contiguous bytes of every state: conflict-free; 8- or 16-byte stores), so the
            // head's weights are computed once per thread instead of once per (thread, head).  A set
            // that took no tile of the segment contributes m = -inf, l = 0, O = 0: weight 0.
            {
                const int h = tid >> 5, j4 = (tid & 31) * 4;
                float2 ml[kConsumerWarps];
                float M = ninf;
                #pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    ml[w] = *reinterpret_cast<const float2*>(merge_ml + (w * kGroup + h) * 2);
                    M = fmaxf(M, ml[w].x);
                }
                float L = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                #pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float wt = fast_exp2(ml[w].x - M);
                    L = fmaf(ml[w].y, wt, L);
                    const float4 a = *reinterpret_cast<const float4*>(merge_o + (w * kGroup + h) * kMergeStride + j4);
                    acc.x = fmaf(a.x, wt, acc.x); acc.y = fmaf(a.y, wt, acc.y);
                    acc.z = fmaf(a.z, wt, acc.z); acc.w = fmaf(a.w, wt, acc.w);
                }
                const float inv = 1.f / L;
                acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
                const float lse2 = M + log2f(L);
                if (mt.slot < 0) {
                    if (h < p.group && in_bounds(p.hdr, (int64_t)mt.b * p.hq + mt.g * p.group + h, p.out_rows, 104)) {
                        const int64_t row = (int64_t)mt.b * p.hq + mt.g * p.group + h;
                        *reinterpret_cast<uint2*>(p.out + row * kD + j4) =
                            make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
                        if (j4 == 0) p.lse[row] = lse2 * 0.6931471805599453f;
                    }
                } else if (in_bounds(p.hdr, mt.slot, p.slot_cap, 105)) {
                    const int64_t row = (int64_t)mt.slot * kGroup + h;
                    *reinterpret_cast<float4*>(p.part_o + row * kD + j4) = acc;
                    if (j4 == 0) p.part_lse[row] = lse2;
                }
            }
            mbar_arrive(merge_bar1);
            if (!mbar_wait(merge_bar1, merges & 1u, abort_flag, wait_ns)) {
                if (lane == 0) wait_failed(p, abort_flag, 5);
                return;
            }
            if (mt.slot >= 0 && p.fuse_combine) {
                // hand the finished partial to the combiner warp; nobody here waits for it
                if (tid == 0) {
                    if (!mbar_wait(job_taken, (jobs & 1u) ^ 1u, abort_flag, wait_ns)) wait_failed(p, abort_flag, 6);
                    job_s->b = mt.b; job_s->g = mt.g; job_s->unit_start = mt.unit_start;
                    job_s->tiles_b = mt.tiles_b; job_s->exit = 0;
                }
                mbar_arrive(job_ready);       // releases this thread's partial stores to the combiner warp
                ++jobs;
            }
            ++merges;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
partial_mma_kernel(DecodeParams p, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    partial_mma_body(p, map_k, map_v, smem);
}

// ------------------------------------------------------------------ host side

cudaError_t launch_partial_mma(const DecodeParams& p, cudaStream_t stream, RowsMapCache* maps) {
    // the attribute is a property of the function on a device: setting it twice (two threads racing
    // through here) is harmless, so an atomic flag per device is all the ordering this needs
    static std::atomic<bool> attr_set[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
        e = cudaFuncSetAttribute(partial_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev < 64) attr_set[dev].store(true, std::memory_order_release);
    }
    // one box {64, rows of a box, 2} = the part of one (page, KV head) chunk that belongs to a tile
    const uint64_t pool_rows = (uint64_t)p.num_pages * p.page_size * (p.token_major ? 1 : p.hkv);
    const uint32_t planes = p.token_major ? 2 * p.hkv : 2;
    CUtensorMap local_k, local_v;
    const CUtensorMap *mk = &local_k, *mv = &local_v;
    if (maps) {
        mk = maps->get(p.k_pages, pool_rows, p.box_rows, 2, planes);
        mv = maps->get(p.v_pages, pool_rows, p.box_rows, 2, planes);
        if (!mk || !mv) return cudaErrorInvalidValue;
    } else if (!make_rows_map(&local_k, p.k_pages, pool_rows, p.box_rows, 2, planes) ||
               !make_rows_map(&local_v, p.v_pages, pool_rows, p.box_rows, 2, planes)) {
        return cudaErrorInvalidValue;
    }
    // Programmatic dependent launch: the kernel may start before the kernel ahead of it on the stream
    // has finished, if that kernel allows it.  After this library's plan kernel that is always wanted
    // (the prologue and the first tiles overlap the plan).  Without a plan kernel the kernel ahead is
    // the caller's, and this kernel reads seq_lens, q and the pools before it waits: only a caller who
    // has said that those are not that kernel's outputs gets the early start.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.grid_ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (!p.no_plan_launch || p.overlap_next) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, partial_mma_kernel, p, *mk, *mv);
}

}  // namespace concur
