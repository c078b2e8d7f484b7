// KV append: writes the new token's K and V rows of every sequence into its page slot and
// advances the sequence's length -- the write path of the paged cache, run once per decode
// step before the attention call.  A model has one pair of pools per layer and one set of
// lengths: the step's first append (advance = 1) writes at position len and makes it len + 1, the
// other layers' appends (advance = 0) write their rows into the same slot, position len - 1, and
// leave the lengths alone.
#include "common.cuh"

namespace concur {

constexpr int kAppendThreads = kHkv * (kRowBytes / 16);    // up to 8 heads x 16 sixteen-byte pieces

__global__ void __launch_bounds__(kAppendThreads) append_kernel(
        const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, uint4* k_pages, uint4* v_pages,
        const int32_t* __restrict__ block_table, int32_t* seq_lens, int32_t* hdr, int32_t num_pages,
        int32_t bt_stride, int32_t page_size, int32_t page_shift, int32_t token_major, int32_t hkv, int32_t advance) {
    const int b = blockIdx.x;
    const int g = threadIdx.x >> 4, piece = threadIdx.x & 15;
    const int64_t pos = (int64_t)seq_lens[b] - (advance ? 0 : 1);
    __syncthreads();                                   // everyone has read the length before it is advanced
    if (pos < 0 || pos >= (int64_t)bt_stride * page_size) {
        if (threadIdx.x == 0) atomicOr(reinterpret_cast<unsigned int*>(hdr + kHdrStatus), kFlagBadLen);
        return;                                        // no room in the table row: nothing is written
    }
    const int32_t page = block_table[(int64_t)b * bt_stride + (pos >> page_shift)];
    if (page < 0 || page >= num_pages) {
        if (threadIdx.x == 0) atomicOr(reinterpret_cast<unsigned int*>(hdr + kHdrStatus), kFlagBadPage);
        return;
    }
    const int32_t slot = (int32_t)(pos & (page_size - 1));
    if (g < hkv) {
        const int64_t row = token_major ? ((int64_t)page * page_size + slot) * hkv + g
                                        : ((int64_t)page * hkv + g) * page_size + slot;
        const int64_t src = ((int64_t)b * hkv + g) * (kRowBytes / 16) + piece;
        if (!in_bounds(hdr, row, (int64_t)num_pages * hkv * page_size, 601)) return;
        k_pages[row * (kRowBytes / 16) + piece] = k_new[src];
        v_pages[row * (kRowBytes / 16) + piece] = v_new[src];
    }
    if (threadIdx.x == 0 && advance) seq_lens[b] = (int32_t)pos + 1;
}

cudaError_t launch_append(const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                          const int32_t* block_table, int32_t* seq_lens, int32_t* hdr, int32_t batch,
                          int32_t num_pages, int32_t bt_stride, int32_t page_size, int32_t page_shift,
                          int32_t token_major, int32_t hkv, int32_t advance, cudaStream_t stream) {
    append_kernel<<<batch, kAppendThreads, 0, stream>>>(
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), static_cast<uint4*>(k_pages),
        static_cast<uint4*>(v_pages), block_table, seq_lens, hdr, num_pages, bt_stride, page_size, page_shift,
        token_major, hkv, advance);
    return cudaGetLastError();
}

}  // namespace concur
