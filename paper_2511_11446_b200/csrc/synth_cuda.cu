// CUDA side of the seeded input generator (activations and integer weights), bit-identical to the
// numpy implementation in synth.py. Input generation only: none of the quantized-linear arithmetic
// lives here, and this file is built into its own shared object (libdpsynth.so).
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull;

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__device__ __forceinline__ int sum16(uint64_t h) {
  return static_cast<int>((h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + (h >> 48));
}
// Irwin-Hall (n = 8) standard normal of element i of stream `key`.
__device__ __forceinline__ float std_normal(uint64_t key, uint64_t i) {
  const uint64_t h0 = mix64(key + (2 * i + 1) * kGolden);
  const uint64_t h1 = mix64(key + (2 * i + 2) * kGolden);
  const int s = sum16(h0) + sum16(h1) - 262140;
  return __fmul_rn(static_cast<float>(s), static_cast<float>(1.0 / 53510.107));
}
__device__ __forceinline__ uint16_t bf16_rne(float f) {
  uint32_t u = __float_as_uint(f);
  return static_cast<uint16_t>((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

__global__ void activations_kernel(uint16_t* out, int64_t M, int64_t K, int64_t ld, uint64_t key,
                                   float sigma, const float* __restrict__ colscale) {
  const int64_t total = M * K;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t m = i / K, k = i - m * K;
    const float z = std_normal(key, static_cast<uint64_t>(i));
    out[m * ld + k] = bf16_rne(__fmul_rn(__fmul_rn(z, sigma), colscale[k]));
  }
}

// One block per output channel: max |z| over the row, then round-to-nearest integer codes.
__global__ void weights_kernel(int8_t* w, float* s_w, int64_t K, uint64_t key, float qmax) {
  __shared__ float red[32];
  const int64_t n = blockIdx.x;
  float amax = 0.0f;
  for (int64_t k = threadIdx.x; k < K; k += blockDim.x)
    amax = fmaxf(amax, fabsf(std_normal(key, static_cast<uint64_t>(n * K + k))));
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = 0.0f;
  for (int i = 0; i < (blockDim.x >> 5); ++i) amax = fmaxf(amax, red[i]);
  const float s = amax > 0.0f ? __fdiv_rn(amax, qmax) : 1.0f;
  for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {
    float r = rintf(__fdiv_rn(std_normal(key, static_cast<uint64_t>(n * K + k)), s));
    r = fminf(fmaxf(r, -qmax), qmax);
    w[n * K + k] = static_cast<int8_t>(r);
  }
  if (threadIdx.x == 0) s_w[n] = __fmul_rn(s, 0.02f);
}

}  // namespace

extern "C" int dps_activations(void* out_bf16, int64_t M, int64_t K, int64_t ld, uint64_t key,
                               float sigma, const float* colscale, void* stream) {
  if (M * K == 0) return 0;
  const int64_t total = M * K;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  activations_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<uint16_t*>(out_bf16), M, K, ld, key, sigma, colscale);
  return static_cast<int>(cudaGetLastError());
}

extern "C" int dps_weights(int8_t* w, float* s_w, int64_t N, int64_t K, uint64_t key, int bits,
                           void* stream) {
  if (N * K == 0) return 0;
  weights_kernel<<<static_cast<unsigned>(N), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      w, s_w, K, key, static_cast<float>((1 << (bits - 1)) - 1));
  return static_cast<int>(cudaGetLastError());
}
