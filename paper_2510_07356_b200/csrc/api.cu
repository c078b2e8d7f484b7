// C-ABI of the decode-attention library: handle, argument checks, workspace layout and
// the three stream-ordered launches (plan -> partial -> combine) of one decode step.
#include "../../include/concur_attn.h"

#include <new>

#include "common.cuh"
#include "tensor_map.cuh"

using namespace concur;

namespace {

constexpr int32_t kMaxRanges = 4736;          // capacity of the plan (148 SMs x 32)
constexpr int32_t kMaxBatchLimit = 65536;
constexpr size_t kAlign = 256;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct WorkspaceLayout {
    size_t hdr, prefix, range_start, unit_done, part_lse, part_o, total;
};

WorkspaceLayout layout_for(int32_t max_batch) {
    WorkspaceLayout w;
    size_t at = 0;
    w.hdr = at;          at += align_up(kHdrWords * sizeof(int32_t));
    w.prefix = at;       at += align_up(((size_t)max_batch + 1) * sizeof(int32_t));
    w.range_start = at;  at += align_up(((size_t)kMaxRanges + 1) * sizeof(int32_t));
    w.unit_done = at;    at += align_up((size_t)max_batch * kHkv * sizeof(int32_t));
    w.part_lse = at;     at += align_up((size_t)2 * kMaxRanges * kGroup * sizeof(float));
    w.part_o = at;       at += align_up((size_t)2 * kMaxRanges * kGroup * kD * sizeof(float));
    w.total = at;
    return w;
}

int check_config(const concur_attn_config_t* c) {
    if (!c) return CONCUR_ERR_INVALID_ARG;
    if ((c->kv_layout != CONCUR_KV_HEAD_MAJOR && c->kv_layout != CONCUR_KV_TOKEN_MAJOR) || c->device < 0)
        return CONCUR_ERR_INVALID_ARG;
    if (c->max_batch < 1 || c->max_batch > kMaxBatchLimit) return CONCUR_ERR_INVALID_ARG;
    if (c->max_pages_per_seq < 1) return CONCUR_ERR_INVALID_ARG;
    if (c->num_kv_heads < 1 || c->num_kv_heads > kHkv || c->head_dim != kD) return CONCUR_ERR_UNSUPPORTED;
    // 1 to 8 query heads per KV head
    if (c->num_q_heads < c->num_kv_heads || c->num_q_heads > kGroup * c->num_kv_heads ||
        c->num_q_heads % c->num_kv_heads != 0)
        return CONCUR_ERR_UNSUPPORTED;
    if (c->page_size != 16 && c->page_size != 32 && c->page_size != 64 && c->page_size != 128)
        return CONCUR_ERR_UNSUPPORTED;
    // the flat tile index space must fit int32
    const int64_t tiles_per_seq = ((int64_t)c->max_pages_per_seq * c->page_size + kTile - 1) / kTile;
    if (tiles_per_seq * c->max_batch * c->num_kv_heads >= (int64_t)1 << 31) return CONCUR_ERR_TOO_LARGE;
    return CONCUR_OK;
}

struct Staging {            // device copies of host tensors (concur_decode_attn_host)
    void* ptr = nullptr;
    size_t cap = 0;
};

class DeviceGuard {
public:
    explicit DeviceGuard(int device) {
        ok_ = cudaGetDevice(&prev_) == cudaSuccess;
        if (ok_ && prev_ != device) ok_ = cudaSetDevice(device) == cudaSuccess;
        switched_ = ok_ && prev_ != device;
    }
    ~DeviceGuard() { if (switched_) cudaSetDevice(prev_); }
    bool ok() const { return ok_; }
private:
    int prev_ = 0;
    bool ok_ = false, switched_ = false;
};

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

struct concur_attn {
    concur_attn_config_t cfg;
    int sm_count = 0;
    char* ws = nullptr;
    bool owns_ws = false;
    WorkspaceLayout lay;
    // options
    int32_t kernel = 0;
    int32_t forced_ranges = 0;
    int32_t grid_ctas = 0;
    int32_t ranges_per_cta = 0;
    int32_t min_range_tiles = 0;
    int32_t fuse_combine = 1;
    int32_t claim_ahead = 1 << 20;
    int32_t prefix_kernel = 0;
    int32_t prefill_kernel = 0;
    int32_t small_page_copy = 1;
    int64_t wait_limit_ns = 2000000000ll;
    cudaEvent_t ev_before = nullptr, ev_after = nullptr;
    Staging st_q, st_k, st_v, st_bt, st_len, st_out, st_lse;
    Staging cascade_ws;          // allocated on the first cascade call
    int32_t overlap_calls = 0;
    RowsMapCache maps;           // tensor maps of the pools seen recently
    // the plan concur_attn_plan left in the workspace, for concur_decode_attn_planned
    const int32_t* planned_lens = nullptr;
    int32_t planned_batch = -1, planned_stride = -1;
};

extern "C" {

size_t concur_attn_workspace_bytes(const concur_attn_config_t* cfg) {
    if (check_config(cfg) != CONCUR_OK) return 0;
    return layout_for(cfg->max_batch).total;
}

int concur_attn_create(const concur_attn_config_t* cfg, concur_attn_t** handle) {
    if (!handle) return CONCUR_ERR_INVALID_ARG;
    int rc = check_config(cfg);
    if (rc != CONCUR_OK) return rc;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device >= ndev) { cudaGetLastError(); return CONCUR_ERR_CUDA; }
    DeviceGuard guard(cfg->device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;

    concur_attn* h = new (std::nothrow) concur_attn;
    if (!h) return CONCUR_ERR_OOM;
    h->cfg = *cfg;
    h->lay = layout_for(cfg->max_batch);
    if (cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess) {
        delete h; return CONCUR_ERR_CUDA;
    }
    if (cfg->workspace) {
        if (!aligned(cfg->workspace, kAlign)) { delete h; return CONCUR_ERR_INVALID_ARG; }
        if (cfg->workspace_bytes < h->lay.total) { delete h; return CONCUR_ERR_TOO_LARGE; }
        h->ws = static_cast<char*>(cfg->workspace);
    } else {
        void* p = nullptr;
        if (cudaMalloc(&p, h->lay.total) != cudaSuccess) { cudaGetLastError(); delete h; return CONCUR_ERR_OOM; }
        h->ws = static_cast<char*>(p);
        h->owns_ws = true;
    }
    // the header and the per-unit ticket counters must start at zero (a launch without a plan kernel relies
    // on both); partial slots are written before they are read
    if (cudaMemset(h->ws, 0, h->lay.part_lse) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        if (h->owns_ws) cudaFree(h->ws);
        delete h; return CONCUR_ERR_CUDA;
    }
    *handle = h;
    return CONCUR_OK;
}

static int fill_params(concur_attn_t* h, DecodeParams& p, const void* q, const void* k_pages,
                       const void* v_pages, const int32_t* block_table, const int32_t* seq_lens,
                       float scale, void* out, float* lse, int32_t batch, int32_t num_pages,
                       int32_t stride) {
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_pages = static_cast<const __nv_bfloat16*>(k_pages);
    p.v_pages = static_cast<const __nv_bfloat16*>(v_pages);
    p.block_table = block_table;
    p.seq_lens = seq_lens;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.scale_log2e = scale * 1.4426950408889634f;
    p.batch = batch;
    p.num_pages = num_pages;
    p.bt_stride = stride;
    p.page_size = h->cfg.page_size;
    p.page_shift = h->cfg.page_size == 16 ? 4 : (h->cfg.page_size == 32 ? 5 : (h->cfg.page_size == 64 ? 6 : 7));
    p.box_rows = h->cfg.page_size < kTile ? h->cfg.page_size : kTile;
    p.box_shift = p.page_shift < 6 ? p.page_shift : 6;
    p.lane_copy = p.box_rows < kTile ? h->small_page_copy : 0;
    p.token_major = h->cfg.kv_layout == CONCUR_KV_TOKEN_MAJOR ? 1 : 0;
    p.hkv = h->cfg.num_kv_heads;
    p.hq = h->cfg.num_q_heads;
    p.group = h->cfg.num_q_heads / h->cfg.num_kv_heads;
    const int per_sm = h->kernel == 1 ? partial_scalar_ctas_per_sm() : 1;
    p.grid_ctas = h->grid_ctas > 0 ? h->grid_ctas : h->sm_count * per_sm;
    p.forced_ranges = h->forced_ranges;
    p.ranges_per_cta = h->ranges_per_cta;                 // 0: chosen per call from the amount of work
    p.min_range_tiles = h->min_range_tiles > 0 ? h->min_range_tiles : 2;
    p.max_ranges = kMaxRanges;
    p.slot_cap = 2 * kMaxRanges;
    p.out_rows = (int64_t)batch * h->cfg.num_q_heads;
    p.fuse_combine = h->fuse_combine;
    p.claim_ahead = h->claim_ahead;
    p.wait_limit_ns = h->wait_limit_ns;
    p.overlap_next = h->overlap_calls;
    p.hdr = reinterpret_cast<int32_t*>(h->ws + h->lay.hdr);
    p.tiles_prefix = reinterpret_cast<int32_t*>(h->ws + h->lay.prefix);
    p.range_start = reinterpret_cast<int32_t*>(h->ws + h->lay.range_start);
    p.unit_done = reinterpret_cast<int32_t*>(h->ws + h->lay.unit_done);
    p.part_lse = reinterpret_cast<float*>(h->ws + h->lay.part_lse);
    p.part_o = reinterpret_cast<float*>(h->ws + h->lay.part_o);
    p.tok_offset = nullptr;
    p.all_partial = 0;
    return CONCUR_OK;
}

static int check_call(concur_attn_t* h, const void* q, const void* k_pages, const void* v_pages,
                      const int32_t* block_table, const int32_t* seq_lens, void* out, float* lse,
                      int32_t batch, int32_t num_pages, int32_t stride, size_t ptr_align) {
    if (!h) return CONCUR_ERR_INVALID_ARG;
    if (batch < 0 || num_pages < 1 || stride < 1) return CONCUR_ERR_INVALID_ARG;
    if (batch > h->cfg.max_batch || stride > h->cfg.max_pages_per_seq) return CONCUR_ERR_TOO_LARGE;
    // pool rows are addressed with int32 coordinates
    if ((int64_t)num_pages * h->cfg.num_kv_heads * h->cfg.page_size >= (int64_t)1 << 31) return CONCUR_ERR_TOO_LARGE;
    if (batch == 0) return CONCUR_OK;
    if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !out || !lse) return CONCUR_ERR_INVALID_ARG;
    if (!aligned(q, ptr_align) || !aligned(k_pages, ptr_align) || !aligned(v_pages, ptr_align) ||
        !aligned(out, ptr_align) || !aligned(block_table, 4) || !aligned(seq_lens, 4) || !aligned(lse, 4))
        return CONCUR_ERR_INVALID_ARG;
    return CONCUR_OK;
}

// The sequences whose plan the tensor-core partial kernel keeps in shared memory and can therefore work
// out for itself (its kSmemBatch).
constexpr int32_t kSelfPlanBatch = 511;

// One launch instead of two: the tensor-core kernel with the merge fused needs no plan kernel when it
// plans for itself (batch <= kSelfPlanBatch) or when the tables of a matching concur_attn_plan call are
// in the workspace (`planned`).
static bool single_launch(const concur_attn_t* h, int32_t batch, bool planned) {
    return h->kernel == 0 && h->fuse_combine && (batch <= kSelfPlanBatch || planned);
}

static int enqueue(concur_attn_t* h, DecodeParams& p, cudaStream_t stream, bool planned = false) {
    p.no_plan_launch = single_launch(h, p.batch, planned) ? 1 : 0;
    // every launch but the one that reads them overwrites the tables a concur_attn_plan call left
    if (!(planned && p.batch > kSelfPlanBatch)) h->planned_batch = -1;
    if (!p.no_plan_launch && launch_plan(p, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    if (h->ev_before && cudaEventRecord(h->ev_before, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    cudaError_t e = h->kernel == 1 ? launch_partial_scalar(p, stream) : launch_partial_mma(p, stream, &h->maps);
    if (e != cudaSuccess) return CONCUR_ERR_CUDA;
    if (h->ev_after && cudaEventRecord(h->ev_after, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    // the tensor-core kernel merges split units itself; the scalar kernel leaves that to the
    // combine kernel
    if ((h->kernel == 1 || !h->fuse_combine) && launch_combine(p, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    return CONCUR_OK;
}

int concur_decode_attn(concur_attn_t* h, const void* q, const void* k_pages, const void* v_pages,
                       const int32_t* block_table, const int32_t* seq_lens, float scale, void* out,
                       float* lse, int32_t batch, int32_t num_pages, int32_t block_table_stride,
                       void* cuda_stream) {
    int rc = check_call(h, q, k_pages, v_pages, block_table, seq_lens, out, lse, batch, num_pages,
                        block_table_stride, 16);
    if (rc != CONCUR_OK || batch == 0) return rc;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    DecodeParams p = {};
    fill_params(h, p, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, batch, num_pages,
                block_table_stride);
    return enqueue(h, p, static_cast<cudaStream_t>(cuda_stream));
}

int concur_attn_plan(concur_attn_t* h, const int32_t* seq_lens, int32_t batch, int32_t block_table_stride,
                     void* cuda_stream) {
    if (!h) return CONCUR_ERR_INVALID_ARG;
    if (batch < 0 || block_table_stride < 1) return CONCUR_ERR_INVALID_ARG;
    if (batch > h->cfg.max_batch || block_table_stride > h->cfg.max_pages_per_seq) return CONCUR_ERR_TOO_LARGE;
    h->planned_batch = -1;
    if (batch == 0) return CONCUR_OK;
    if (!seq_lens || !aligned(seq_lens, 4)) return CONCUR_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    DecodeParams p = {};
    fill_params(h, p, nullptr, nullptr, nullptr, nullptr, seq_lens, 1.f, nullptr, nullptr, batch, 1,
                block_table_stride);
    if (launch_plan(p, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return CONCUR_ERR_CUDA;
    h->planned_lens = seq_lens;
    h->planned_batch = batch;
    h->planned_stride = block_table_stride;
    return CONCUR_OK;
}

int concur_decode_attn_planned(concur_attn_t* h, const void* q, const void* k_pages, const void* v_pages,
                               const int32_t* block_table, const int32_t* seq_lens, float scale, void* out,
                               float* lse, int32_t batch, int32_t num_pages, int32_t block_table_stride,
                               void* cuda_stream) {
    int rc = check_call(h, q, k_pages, v_pages, block_table, seq_lens, out, lse, batch, num_pages,
                        block_table_stride, 16);
    if (rc != CONCUR_OK || batch == 0) return rc;
    // small batches plan in-kernel and need no plan call; larger ones need the matching one
    const bool planned = h->planned_batch == batch && h->planned_stride == block_table_stride &&
                         h->planned_lens == seq_lens;
    if (batch > kSelfPlanBatch && !planned) return CONCUR_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    DecodeParams p = {};
    fill_params(h, p, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, batch, num_pages,
                block_table_stride);
    return enqueue(h, p, static_cast<cudaStream_t>(cuda_stream), planned);
}

int concur_decode_attn_append(concur_attn_t* h, const void* q, const void* k_new, const void* v_new, void* k_pages,
                              void* v_pages, const int32_t* block_table, const int32_t* seq_lens, float scale,
                              void* out, float* lse, int32_t batch, int32_t num_pages, int32_t block_table_stride,
                              void* cuda_stream) {
    int rc = check_call(h, q, k_pages, v_pages, block_table, seq_lens, out, lse, batch, num_pages,
                        block_table_stride, 16);
    if (rc != CONCUR_OK || batch == 0) return rc;
    if (!k_new || !v_new || !aligned(k_new, 16) || !aligned(v_new, 16)) return CONCUR_ERR_INVALID_ARG;
    // only the tensor-core kernel with the merge fused takes its last token from outside the pools
    if (h->kernel != 0 || !h->fuse_combine) return CONCUR_ERR_UNSUPPORTED;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    DecodeParams p = {};
    fill_params(h, p, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, batch, num_pages,
                block_table_stride);
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    return enqueue(h, p, static_cast<cudaStream_t>(cuda_stream));
}

int concur_kv_append(concur_attn_t* h, const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                     const int32_t* block_table, int32_t* seq_lens, int32_t batch, int32_t num_pages,
                     int32_t block_table_stride, void* cuda_stream) {
    return concur_kv_append_layer(h, k_new, v_new, k_pages, v_pages, block_table, seq_lens, batch, num_pages,
                                  block_table_stride, 1, cuda_stream);
}

int concur_kv_append_layer(concur_attn_t* h, const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                           const int32_t* block_table, int32_t* seq_lens, int32_t batch, int32_t num_pages,
                           int32_t block_table_stride, int32_t advance, void* cuda_stream) {
    if (!h || (advance != 0 && advance != 1)) return CONCUR_ERR_INVALID_ARG;
    if (batch < 0 || num_pages < 1 || block_table_stride < 1) return CONCUR_ERR_INVALID_ARG;
    if (batch > h->cfg.max_batch || block_table_stride > h->cfg.max_pages_per_seq) return CONCUR_ERR_TOO_LARGE;
    if ((int64_t)num_pages * h->cfg.num_kv_heads * h->cfg.page_size >= (int64_t)1 << 31) return CONCUR_ERR_TOO_LARGE;
    if (batch == 0) return CONCUR_OK;
    if (!k_new || !v_new || !k_pages || !v_pages || !block_table || !seq_lens) return CONCUR_ERR_INVALID_ARG;
    if (!aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(k_pages, 16) || !aligned(v_pages, 16) ||
        !aligned(block_table, 4) || !aligned(seq_lens, 4))
        return CONCUR_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    const int32_t P = h->cfg.page_size;
    const int32_t shift = P == 16 ? 4 : (P == 32 ? 5 : (P == 64 ? 6 : 7));
    if (launch_append(k_new, v_new, k_pages, v_pages, block_table, seq_lens,
                      reinterpret_cast<int32_t*>(h->ws + h->lay.hdr), batch, num_pages, block_table_stride, P,
                      shift, h->cfg.kv_layout == CONCUR_KV_TOKEN_MAJOR ? 1 : 0, h->cfg.num_kv_heads, advance,
                      static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return CONCUR_ERR_CUDA;
    return CONCUR_OK;
}

static int ensure(Staging& s, size_t bytes);

namespace {
constexpr int32_t kCascadeMaxBatch = 4096;
struct CascadeLayout {
    size_t chdr, tok_offset, seq_group, ptiles, rowbase, pre_lse, pre_o, part_lse, part_o, total;
    int32_t max_rows, max_slots;
};
CascadeLayout cascade_layout(int32_t max_batch, int sm_count) {
    CascadeLayout w;
    w.max_rows = kHkv * max_batch + kMaxShare * sm_count;     // whole units + one extra split per range
    w.max_slots = kMaxRanges + kHkv * max_batch;              // suffix partial slots r + u
    size_t at = 0;
    w.chdr = at;        at += align_up(kHdrWords * sizeof(int32_t));
    w.tok_offset = at;  at += align_up((size_t)max_batch * sizeof(int32_t));
    w.seq_group = at;   at += align_up((size_t)max_batch * sizeof(int32_t));
    w.ptiles = at;      at += align_up(((size_t)max_batch + 1) * sizeof(int32_t));
    w.rowbase = at;     at += align_up(((size_t)max_batch * kHkv + 1) * sizeof(int32_t));
    w.pre_lse = at;     at += align_up((size_t)w.max_rows * kGroup * sizeof(float));
    w.pre_o = at;       at += align_up((size_t)w.max_rows * kGroup * kD * sizeof(float));
    w.part_lse = at;    at += align_up((size_t)w.max_slots * kGroup * sizeof(float));
    w.part_o = at;      at += align_up((size_t)w.max_slots * kGroup * kD * sizeof(float));
    w.total = at;
    return w;
}
}  // namespace

int concur_decode_attn_cascade(concur_attn_t* h, const void* q, const void* k_pages, const void* v_pages,
                               const int32_t* block_table, const int32_t* seq_lens,
                               const int32_t* group_start, const int32_t* prefix_lens, float scale, void* out,
                               float* lse, int32_t batch, int32_t num_groups, int32_t num_pages,
                               int32_t block_table_stride, void* cuda_stream) {
    int rc = check_call(h, q, k_pages, v_pages, block_table, seq_lens, out, lse, batch, num_pages,
                        block_table_stride, 16);
    if (rc != CONCUR_OK || batch == 0) return rc;
    if (num_groups < 1 || num_groups > batch || !group_start || !prefix_lens || !aligned(group_start, 4) ||
        !aligned(prefix_lens, 4))
        return CONCUR_ERR_INVALID_ARG;
    if (h->cfg.max_batch > kCascadeMaxBatch) return CONCUR_ERR_UNSUPPORTED;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    const CascadeLayout lay = cascade_layout(h->cfg.max_batch, h->sm_count);
    if ((rc = ensure(h->cascade_ws, lay.total)) != CONCUR_OK) return rc;
    char* cw = static_cast<char*>(h->cascade_ws.ptr);

    DecodeParams p = {};
    fill_params(h, p, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, batch, num_pages,
                block_table_stride);
    CascadeParams c;
    c.group_start = group_start;
    c.prefix_lens = prefix_lens;
    c.num_groups = num_groups;
    c.grid_ctas = h->sm_count;
    c.max_rows = lay.max_rows;
    c.chdr = reinterpret_cast<int32_t*>(cw + lay.chdr);
    c.tok_offset = reinterpret_cast<int32_t*>(cw + lay.tok_offset);
    c.seq_group = reinterpret_cast<int32_t*>(cw + lay.seq_group);
    c.ptiles_prefix = reinterpret_cast<int32_t*>(cw + lay.ptiles);
    c.unit_rowbase = reinterpret_cast<int32_t*>(cw + lay.rowbase);
    c.pre_lse = reinterpret_cast<float*>(cw + lay.pre_lse);
    c.pre_o = reinterpret_cast<float*>(cw + lay.pre_o);
    // the suffix pass writes one partial per segment into the cascade's own slots
    p.part_lse = reinterpret_cast<float*>(cw + lay.part_lse);
    p.part_o = reinterpret_cast<float*>(cw + lay.part_o);
    p.slot_cap = lay.max_slots;
    p.tok_offset = c.tok_offset;
    p.all_partial = 1;
    p.fuse_combine = 0;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    h->planned_batch = -1;
    if (launch_plan_cascade(p, c, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    if (h->ev_before && cudaEventRecord(h->ev_before, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    if ((h->prefix_kernel == 1 ? launch_prefix_mma(p, c, stream) : launch_prefix_tc(p, c, stream)) != cudaSuccess)
        return CONCUR_ERR_CUDA;
    if (h->ev_after && cudaEventRecord(h->ev_after, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    cudaError_t e = h->kernel == 1 ? launch_partial_scalar(p, stream) : launch_partial_mma(p, stream, &h->maps);
    if (e != cudaSuccess) return CONCUR_ERR_CUDA;
    if (launch_combine_cascade(p, c, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    return CONCUR_OK;
}

int concur_prefill_attn(concur_attn_t* h, const void* q, const void* k_pages, const void* v_pages,
                        const int32_t* block_table, const int32_t* seq_lens, const int32_t* q_start, float scale,
                        void* out, float* lse, int32_t batch, int32_t total_q, int32_t num_pages,
                        int32_t block_table_stride, void* cuda_stream) {
    int rc = check_call(h, q, k_pages, v_pages, block_table, seq_lens, out, lse, batch, num_pages,
                        block_table_stride, 16);
    if (rc != CONCUR_OK || batch == 0) return rc;
    if (total_q < 0 || !q_start || !aligned(q_start, 4)) return CONCUR_ERR_INVALID_ARG;
    if ((int64_t)total_q * h->cfg.num_q_heads >= (int64_t)1 << 31) return CONCUR_ERR_TOO_LARGE;
    if (total_q == 0) return CONCUR_OK;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    DecodeParams p = {};
    fill_params(h, p, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, batch, num_pages,
                block_table_stride);
    p.grid_ctas = h->grid_ctas > 0 ? h->grid_ctas : h->sm_count;
    p.out_rows = (int64_t)total_q * h->cfg.num_q_heads;
    PrefillParams f;
    f.q_start = q_start;
    f.total_q = total_q;
    f.block = 0;                                                 // set by the launcher for the kernel it runs
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    h->planned_batch = -1;
    if (h->ev_before && cudaEventRecord(h->ev_before, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    if (launch_prefill_tc(p, f, h->prefill_kernel == 0, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    if (h->ev_after && cudaEventRecord(h->ev_after, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    return CONCUR_OK;
}

static int ensure(Staging& s, size_t bytes) {
    if (bytes <= s.cap) return CONCUR_OK;
    if (s.ptr) cudaFree(s.ptr);
    s.ptr = nullptr; s.cap = 0;
    if (cudaMalloc(&s.ptr, bytes) != cudaSuccess) { cudaGetLastError(); s.ptr = nullptr; return CONCUR_ERR_OOM; }
    s.cap = bytes;
    return CONCUR_OK;
}

int concur_decode_attn_host(concur_attn_t* h, const void* q, const void* k_pages, const void* v_pages,
                            const int32_t* block_table, const int32_t* seq_lens, float scale, void* out,
                            float* lse, int32_t batch, int32_t num_pages, int32_t block_table_stride,
                            void* cuda_stream) {
    int rc = check_call(h, q, k_pages, v_pages, block_table, seq_lens, out, lse, batch, num_pages,
                        block_table_stride, 2);
    if (rc != CONCUR_OK || batch == 0) return rc;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t q_bytes = (size_t)batch * h->cfg.num_q_heads * kD * 2;
    const size_t pool_bytes = (size_t)num_pages * h->cfg.num_kv_heads * h->cfg.page_size * kD * 2;
    const size_t bt_bytes = (size_t)batch * block_table_stride * 4;
    const size_t len_bytes = (size_t)batch * 4;
    const size_t lse_bytes = (size_t)batch * h->cfg.num_q_heads * 4;
    if ((rc = ensure(h->st_q, q_bytes)) || (rc = ensure(h->st_k, pool_bytes)) ||
        (rc = ensure(h->st_v, pool_bytes)) || (rc = ensure(h->st_bt, bt_bytes)) ||
        (rc = ensure(h->st_len, len_bytes)) || (rc = ensure(h->st_out, q_bytes)) ||
        (rc = ensure(h->st_lse, lse_bytes)))
        return rc;
    bool ok = true;
    ok &= cudaMemcpyAsync(h->st_q.ptr, q, q_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(h->st_k.ptr, k_pages, pool_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(h->st_v.ptr, v_pages, pool_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(h->st_bt.ptr, block_table, bt_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(h->st_len.ptr, seq_lens, len_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return CONCUR_ERR_CUDA; }
    DecodeParams p = {};
    fill_params(h, p, h->st_q.ptr, h->st_k.ptr, h->st_v.ptr, static_cast<const int32_t*>(h->st_bt.ptr),
                static_cast<const int32_t*>(h->st_len.ptr), scale, h->st_out.ptr,
                static_cast<float*>(h->st_lse.ptr), batch, num_pages, block_table_stride);
    rc = enqueue(h, p, stream);
    if (rc != CONCUR_OK) return rc;
    ok &= cudaMemcpyAsync(out, h->st_out.ptr, q_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(lse, h->st_lse.ptr, lse_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaStreamSynchronize(stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return CONCUR_ERR_CUDA; }
    return CONCUR_OK;
}

int concur_attn_status(concur_attn_t* h, void* cuda_stream, uint32_t* flags) {
    if (!h || !flags) return CONCUR_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t* word = reinterpret_cast<int32_t*>(h->ws + h->lay.hdr) + kHdrStatus;
    uint32_t v = 0;
    if (cudaMemcpyAsync(&v, word, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaMemsetAsync(word, 0, 4, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return CONCUR_ERR_CUDA;
    }
    // A kernel in which a wait gave up may have left the range counter and the units' ticket counters
    // half-way (only complete launches put them back to zero): start over.
    if ((v & kFlagWaitLimit) &&
        (cudaMemsetAsync(h->ws, 0, h->lay.part_lse, stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess)) {
        cudaGetLastError();
        return CONCUR_ERR_CUDA;
    }
    *flags = v;
    return CONCUR_OK;
}

int concur_attn_set_option(concur_attn_t* h, int32_t key, int64_t value) {
    if (!h || value < 0) return CONCUR_ERR_INVALID_ARG;
    switch (key) {
        case CONCUR_OPT_KERNEL:
            if (value > 1) return CONCUR_ERR_INVALID_ARG;
            h->kernel = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_NUM_RANGES:
            if (value > kMaxRanges) return CONCUR_ERR_INVALID_ARG;
            h->forced_ranges = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_GRID_CTAS:
            if (value > 65536) return CONCUR_ERR_INVALID_ARG;
            h->grid_ctas = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_RANGES_PER_CTA:
            if (value > 1024) return CONCUR_ERR_INVALID_ARG;
            h->ranges_per_cta = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_MIN_RANGE_TILES:
            if (value > (1 << 20)) return CONCUR_ERR_INVALID_ARG;
            h->min_range_tiles = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_FUSE_COMBINE:
            if (value > 1) return CONCUR_ERR_INVALID_ARG;
            h->fuse_combine = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_CLAIM_AHEAD:
            if (value > (1 << 20)) return CONCUR_ERR_INVALID_ARG;
            h->claim_ahead = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_PREFIX_KERNEL:
            if (value > 1) return CONCUR_ERR_INVALID_ARG;
            h->prefix_kernel = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_PREFILL_KERNEL:
            if (value > 1) return CONCUR_ERR_INVALID_ARG;
            h->prefill_kernel = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_SMALL_PAGE_COPY:
            if (value > 1) return CONCUR_ERR_INVALID_ARG;
            h->small_page_copy = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_OVERLAP_CALLS:
            if (value > 1) return CONCUR_ERR_INVALID_ARG;
            h->overlap_calls = (int32_t)value; return CONCUR_OK;
        case CONCUR_OPT_WAIT_LIMIT_NS:
            if (value > 60000000000ll) return CONCUR_ERR_INVALID_ARG;
            h->wait_limit_ns = value > 0 ? value : 2000000000ll; return CONCUR_OK;
        case CONCUR_OPT_EVENT_BEFORE_PARTIAL:
            h->ev_before = reinterpret_cast<cudaEvent_t>(static_cast<uintptr_t>(value)); return CONCUR_OK;
        case CONCUR_OPT_EVENT_AFTER_PARTIAL:
            h->ev_after = reinterpret_cast<cudaEvent_t>(static_cast<uintptr_t>(value)); return CONCUR_OK;
        default:
            return CONCUR_ERR_INVALID_ARG;
    }
}

int concur_attn_last_plan(concur_attn_t* h, void* cuda_stream, int32_t* num_ranges,
                          int32_t* total_tiles, int32_t* range_start, int32_t cap) {
    if (!h || !num_ranges || !total_tiles || cap < 0) return CONCUR_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok()) return CONCUR_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t hdr[kHdrWords];
    if (cudaMemcpyAsync(hdr, h->ws + h->lay.hdr, sizeof hdr, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) { cudaGetLastError(); return CONCUR_ERR_CUDA; }
    *num_ranges = hdr[kHdrNumRanges];
    *total_tiles = hdr[kHdrTotalTiles];
    if (range_start && cap > 0) {
        int32_t n = hdr[kHdrNumRanges] + 1;
        if (n > cap) n = cap;
        if (cudaMemcpyAsync(range_start, h->ws + h->lay.range_start, (size_t)n * 4, cudaMemcpyDeviceToHost,
                            stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) { cudaGetLastError(); return CONCUR_ERR_CUDA; }
    }
    return CONCUR_OK;
}

int concur_attn_destroy(concur_attn_t* h) {
    if (!h) return CONCUR_OK;
    DeviceGuard guard(h->cfg.device);
    Staging* all[] = {&h->st_q, &h->st_k, &h->st_v, &h->st_bt, &h->st_len, &h->st_out, &h->st_lse, &h->cascade_ws};
    for (Staging* s : all) if (s->ptr) cudaFree(s->ptr);
    if (h->owns_ws && h->ws) cudaFree(h->ws);
    delete h;
    return CONCUR_OK;
}

const char* concur_attn_strerror(int code) {
    switch (code) {
        case CONCUR_OK: return "ok";
        case CONCUR_ERR_INVALID_ARG: return "invalid argument";
        case CONCUR_ERR_UNSUPPORTED: return "unsupported geometry";
        case CONCUR_ERR_TOO_LARGE: return "size beyond the handle's limits";
        case CONCUR_ERR_CUDA: return "CUDA call failed";
        case CONCUR_ERR_OOM: return "out of device memory";
        default: return "unknown status";
    }
}

}  // extern "C"
