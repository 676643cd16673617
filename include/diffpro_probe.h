/*
 * diffpro_probe.h -- measurement probes that accompany libdiffpro but are not part of it
 * (libdpprobe.so). They establish ceilings of the device that the benchmark reports its kernels
 * against; nothing in the product library calls them.
 */
#ifndef DIFFPRO_PROBE_H
#define DIFFPRO_PROBE_H
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif

enum { DP_PROBE_OK = 0, DP_PROBE_BAD_ARG = 1, DP_PROBE_ARCH = 2, DP_PROBE_CUDA = 3 };

/*
 * INT8 tensor-core ceiling (the rate of the instruction behind Step 5's INT8 x INT8 -> INT32 GEMM):
 * each of `ctas` CTAs issues `iters` groups of four back-to-back tcgen05 kind::i8 MMAs
 * (128 x tile_n x 32 each; tile_n a multiple of 16 up to 256) on operands resident in shared memory,
 * no global loads. Enqueues one kernel on `stream` (a cudaStream_t); ops = 2*128*tile_n*128*iters*ctas.
 * device_status: device int32, raised to nonzero if a bounded wait inside the kernel expires.
 * Needs compute capability 10.x (DP_PROBE_ARCH otherwise).
 */
int dp_probe_mma_i8(int32_t ctas, int32_t iters, int32_t tile_n, int32_t* device_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif
