// concur_decode_attn_static: the decode-attention step for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need attention:
// a serving process that handed its whole device-memory budget to one arena at start-up and
// treats any later driver allocation as a fault, a plug-in running inside another runtime's
// callback where allocating calls are off limits, or code on a latency path that cannot
// afford the device-wide synchronisation cudaMalloc / cudaFree may imply.  The regular path
// needs a handle, and a handle owns (or is given) a workspace.  This entry point needs
// neither: its workspace is the fixed array below, which lives in the library's device image.
//
// The array's name means two different things.  In device code it is the array.  In host code
// it is only a host-side shadow symbol: handing `g_static_scratch` itself to a kernel would
// pass a host address.  The device address is obtained once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what the kernels get.
#include "../../include/concur_attn.h"

#include <mutex>

#include "common.cuh"

using namespace concur;

namespace {

constexpr int32_t kStaticMaxBatch = CONCUR_STATIC_MAX_BATCH;
constexpr int32_t kStaticMaxRanges = CONCUR_STATIC_MAX_RANGES;
constexpr int kMaxDevices = 64;

constexpr size_t round256(size_t x) { return (x + 255) / 256 * 256; }
constexpr size_t kOffHdr = 0;
constexpr size_t kOffPrefix = kOffHdr + round256(kHdrWords * sizeof(int32_t));
constexpr size_t kOffRangeStart = kOffPrefix + round256((kStaticMaxBatch + 1) * sizeof(int32_t));
constexpr size_t kOffUnitDone = kOffRangeStart + round256((kStaticMaxRanges + 1) * sizeof(int32_t));
constexpr size_t kOffPartLse = kOffUnitDone + round256((size_t)kStaticMaxBatch * kHkv * sizeof(int32_t));
constexpr size_t kOffPartO = kOffPartLse + round256((size_t)2 * kStaticMaxRanges * kGroup * sizeof(float));
constexpr size_t kStaticBytes = kOffPartO + round256((size_t)2 * kStaticMaxRanges * kGroup * kD * sizeof(float));

// About 4.3 MB, held by every GPU that loads the library until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

struct DeviceSetup {
    bool ready = false;
    char* scratch = nullptr;   // device address of g_static_scratch on this device
    int sm_count = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;      // two host threads may make a device's first call at the same time

// Once per device, with that device current: resolve the array's device address.
int setup_current_device(int dev, DeviceSetup** out) {
    if (dev < 0 || dev >= kMaxDevices) return CONCUR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[dev];
    if (!s.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return CONCUR_ERR_CUDA;
        }
        if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return CONCUR_ERR_CUDA;
        }
        s.scratch = static_cast<char*>(ptr);
        s.ready = true;
    }
    *out = &s;
    return CONCUR_OK;
}

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" int concur_decode_attn_static(const void* q, const void* k_pages, const void* v_pages,
                                         const int32_t* block_table, const int32_t* seq_lens, float scale,
                                         void* out, float* lse, int32_t batch, int32_t num_pages,
                                         int32_t block_table_stride, int32_t page_size, void* cuda_stream) {
    if (page_size != 16 && page_size != 32 && page_size != 64) return CONCUR_ERR_UNSUPPORTED;
    if (batch < 0 || num_pages < 1 || block_table_stride < 1) return CONCUR_ERR_INVALID_ARG;
    if (batch > kStaticMaxBatch) return CONCUR_ERR_TOO_LARGE;
    if ((int64_t)num_pages * kHkv * page_size >= (int64_t)1 << 31) return CONCUR_ERR_TOO_LARGE;
    const int64_t tiles_per_seq = ((int64_t)block_table_stride * page_size + kTile - 1) / kTile;
    if (tiles_per_seq * batch * kHkv >= (int64_t)1 << 31) return CONCUR_ERR_TOO_LARGE;
    if (batch == 0) return CONCUR_OK;
    if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !out || !lse) return CONCUR_ERR_INVALID_ARG;
    if (!aligned_to(q, 16) || !aligned_to(k_pages, 16) || !aligned_to(v_pages, 16) || !aligned_to(out, 16) ||
        !aligned_to(block_table, 4) || !aligned_to(seq_lens, 4) || !aligned_to(lse, 4))
        return CONCUR_ERR_INVALID_ARG;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CONCUR_ERR_CUDA; }
    DeviceSetup* s = nullptr;
    int rc = setup_current_device(dev, &s);
    if (rc != CONCUR_OK) return rc;

    DecodeParams p = {};
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
    p.bt_stride = block_table_stride;
    p.page_size = page_size;
    p.page_shift = page_size == 16 ? 4 : (page_size == 32 ? 5 : 6);
    p.box_rows = page_size;
    p.box_shift = p.page_shift;
    p.lane_copy = page_size < kTile ? 1 : 0;
    p.hkv = kHkv;
    p.hq = kHq;
    p.group = kGroup;
    p.grid_ctas = s->sm_count;
    p.forced_ranges = 0;
    p.ranges_per_cta = 0;
    p.min_range_tiles = 2;
    p.max_ranges = kStaticMaxRanges;
    p.slot_cap = 2 * kStaticMaxRanges;
    p.out_rows = (int64_t)batch * kHq;
    p.fuse_combine = 1;
    p.claim_ahead = 1 << 20;
    p.wait_limit_ns = 2000000000ll;
    // the plan kernel rewrites the tile count, the range count, the claim counter and the
    // per-unit counters at the start of every call, and every partial slot is written before
    // it is read, so nothing of the previous call's contents has to be cleared here
    p.hdr = reinterpret_cast<int32_t*>(s->scratch + kOffHdr);
    p.tiles_prefix = reinterpret_cast<int32_t*>(s->scratch + kOffPrefix);
    p.range_start = reinterpret_cast<int32_t*>(s->scratch + kOffRangeStart);
    p.unit_done = reinterpret_cast<int32_t*>(s->scratch + kOffUnitDone);
    p.part_lse = reinterpret_cast<float*>(s->scratch + kOffPartLse);
    p.part_o = reinterpret_cast<float*>(s->scratch + kOffPartO);

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (launch_plan(p, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    if (launch_partial_mma(p, stream) != cudaSuccess) return CONCUR_ERR_CUDA;
    return CONCUR_OK;
}
