// Measurement probe (its own shared object, libdpprobe.so; not part of the product library): the
// INT8 tensor-core ceiling of the device as seen by this library's own instruction stream. Each CTA fills one 128 x 128 (A) and one 256 x 128 (B) int8 operand tile in
// shared memory with pseudo-random bytes and issues `iters` k-blocks of four tcgen05.mma kind::i8
// (128 x tile_n x 32) each, alternating between two accumulator buffers; no global traffic.
#include "dp_common.cuh"
#include "../../include/diffpro_probe.h"

namespace dp {

__global__ void __launch_bounds__(128, 1) mma_i8_peak_kernel(int iters, int tile_n, int32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                 // 16 KB
  uint8_t* sB = smem + 128 * 128;     // 32 KB
  uint64_t* bar = reinterpret_cast<uint64_t*>(sB + 256 * 128);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5;

  uint32_t h = 0x9E3779B9u * (threadIdx.x + 1) + blockIdx.x;
  for (int i = threadIdx.x; i < (128 + 256) * 128 / 4; i += blockDim.x) {
    h = h * 1664525u + 1013904223u;
    reinterpret_cast<uint32_t*>(smem)[i] = h ^ (h >> 13);
  }
  fence_proxy_async_smem();
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) {
    const uint32_t idesc = idesc_i8(128, tile_n);
    const uint64_t adesc = smem_desc_sw128(smem_u32(sA));
    const uint64_t bdesc = smem_desc_sw128(smem_u32(sB));
    for (int it = 0; it < iters; ++it) {
      const uint32_t d = tmem_base + (it & 1) * 256;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) mma_i8_ss(d, adesc + 2 * k4, bdesc + 2 * k4, idesc, 1u);
    }
    mma_commit(bar);
    // bounded wait scaled to the work: ~2x the ideal duration plus slack
    const long long budget = (1ll << 24) + 2048ll * iters;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, 0)) {
      if (clock64() - t0 > budget) {
        *abort_flag = 1;
        break;
      }
    }
    if (*abort_flag && status != nullptr) atomicExch(status, DP_ERR_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace dp

extern "C" int dp_probe_mma_i8(int32_t ctas, int32_t iters, int32_t tile_n, int32_t* device_status, void* stream) {
  using namespace dp;
  if (ctas <= 0 || iters <= 0 || iters > (1 << 22) || tile_n < 16 || tile_n > 256 || (tile_n % 16)) return DP_PROBE_BAD_ARG;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return DP_PROBE_CUDA;
  if (major != 10) return DP_PROBE_ARCH;
  const size_t smem = 128 * 1024;  // more than half an SM: one CTA (and one TMEM allocation) per SM
  if (cudaFuncSetAttribute(mma_i8_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) !=
      cudaSuccess)
    return DP_PROBE_CUDA;
  cudaError_t e = launch(mma_i8_peak_kernel, dim3(ctas), dim3(128), smem, static_cast<cudaStream_t>(stream), false,
                         iters, tile_n, device_status);
  return e == cudaSuccess ? DP_PROBE_OK : DP_PROBE_CUDA;
}
