/* Benchmark-side helper library (libconcur_bench.so); not part of the attention library's ABI. */
#ifndef CONCUR_BENCH_READ_PROBE_H_
#define CONCUR_BENCH_READ_PROBE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CONCUR_BENCH_OK 0
#define CONCUR_BENCH_ERR_INVALID_ARG (-1)
#define CONCUR_BENCH_ERR_CUDA (-4)

/* A read-only stream over a device buffer: reads `bytes` bytes at `buf` (device, 16-byte aligned,
 * `bytes` a multiple of 16) exactly once with 16-byte loads and leaves the xor of all their 32-bit
 * words in `*checksum` (device, 4-byte aligned; zeroed by the call first).  A decode step is a
 * read-only scan of the KV cache, so this kernel's rate over the same pools is the plain-stream
 * figure to hold the partial kernel against (a device copy also writes).  `ctas` = grid size, 0 =
 * four CTAs of 512 threads per SM of the current device.  Asynchronous on `cuda_stream`; allocates
 * nothing.  Misaligned or null arguments: CONCUR_BENCH_ERR_INVALID_ARG. */
int concur_bench_read_probe(const void* buf, size_t bytes, uint32_t* checksum, int32_t ctas, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
