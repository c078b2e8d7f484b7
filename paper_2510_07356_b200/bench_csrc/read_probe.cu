// Read-only HBM stream: the xor of every 32-bit word of a device buffer, read once with 16-byte
// loads that bypass L1.  A measurement aid: a decode-attention step is a read-only scan of the KV
// cache, so the rate of this kernel over the same pools is the closest plain-stream yardstick for
// the partial kernel (a device-to-device copy, the usual yardstick, also writes what it reads).
// The checksum makes the reads observable, and lets a test check that every word was read once.
//
// Built into its own shared library (libconcur_bench.so) for the benchmark: it is no step of the
// attention path and no part of the attention library's ABI.
#include <cuda_runtime.h>
#include <stdint.h>

#include "read_probe.h"

namespace concur {

namespace {

constexpr int kProbeThreads = 512;
constexpr int kProbeUnroll = 8;

__device__ __forceinline__ uint4 load_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kProbeThreads) read_probe_kernel(const uint4* __restrict__ buf, size_t n16,
                                                                   uint32_t* __restrict__ checksum) {
    const size_t stride = (size_t)gridDim.x * kProbeThreads;
    size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
    uint32_t acc = 0;
    for (; i + (kProbeUnroll - 1) * stride < n16; i += kProbeUnroll * stride) {
        uint4 v[kProbeUnroll];
        #pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) v[u] = load_stream16(buf + i + u * stride);
        #pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = load_stream16(buf + i);
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0 && acc) atomicXor(checksum, acc);
}

}  // namespace

}  // namespace concur

extern "C" int concur_bench_read_probe(const void* buf, size_t bytes, uint32_t* checksum, int32_t ctas,
                                       void* cuda_stream) {
    if (!buf || !checksum || ctas < 0 || ctas > 65536) return CONCUR_BENCH_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(buf) & 15u) || (bytes & 15u) || (reinterpret_cast<uintptr_t>(checksum) & 3u))
        return CONCUR_BENCH_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (ctas == 0) {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return CONCUR_BENCH_ERR_CUDA;
        }
        ctas = sms * 4;                       // four resident CTAs of 512 threads fill an SM's 2,048 thread slots
    }
    if (cudaMemsetAsync(checksum, 0, sizeof(uint32_t), stream) != cudaSuccess) {
        cudaGetLastError();
        return CONCUR_BENCH_ERR_CUDA;
    }
    if (bytes == 0) return CONCUR_BENCH_OK;
    concur::read_probe_kernel<<<ctas, concur::kProbeThreads, 0, stream>>>(static_cast<const uint4*>(buf), bytes / 16,
                                                                          checksum);
    if (cudaGetLastError() != cudaSuccess) return CONCUR_BENCH_ERR_CUDA;
    return CONCUR_BENCH_OK;
}
