// Dynamic activation quantization (Step 3, Eq. "daq"; b = 8, zero-point 0, clip threshold = the
// token's absolute maximum): bf16 [M][K] -> int8 codes + one fp32 scale per token.
//
// One warp owns one token. The row is read once with 16-byte loads and kept in registers; the
// absolute maximum is taken on the bf16 magnitude bits (monotone for finite values, so integer
// max is exact); the quantizer is one fused multiply-add per element: x * fl(127/a) + 1.5*2^23
// rounds the exact product once, half to even, and leaves the integer in the low mantissa bits.
// HBM-bound: 2 bytes read + 1 byte written per element.
#include "daq_device.cuh"

namespace dp {

constexpr int kDaqWarps = 8;

// MAXV = 16-byte vectors held per lane (row of up to 256*MAXV elements in registers).
template <int MAXV, bool EO>
__global__ void __launch_bounds__(kDaqWarps * 32)
daq_rows_kernel(const uint16_t* __restrict__ x, int64_t M, int K, int64_t ldx,
                int8_t* __restrict__ q, int64_t ldq, float* __restrict__ s_a,
                int32_t* __restrict__ rowsum, int tiled_kb, const UnpackJob job) {
  pdl_launch_dependents();
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kDaqWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_wait();
  if (static_cast<int>(blockIdx.x) >= job.first_block) {  // the launch's weight-expansion CTAs
    unpack_units(job, blockIdx.x - job.first_block);
    return;
  }
  if (row >= M) return;
  const int nvec = K >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(x + row * ldx);
  uint4 v[MAXV];
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) ld_nc_u32x4(xr + idx, v[i]);
    else v[i] = make_uint4(0, 0, 0, 0);
  }
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    m = absmax_bits2(m, v[i].x);
    m = absmax_bits2(m, v[i].y);
    m = absmax_bits2(m, v[i].z);
    m = absmax_bits2(m, v[i].w);
  }
  m = warp_max_u32(max(m & 0xFFFFu, m >> 16));
  float sc, inv;
  token_scale(m, sc, inv);
  const QRow qr(q, row, ldq, tiled_kb);
  int sum = 0;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) {
      uint2 o = quant_vec<EO>(v[i], inv);
      qr.store(idx, o);
      sum = __dp4a(static_cast<int>(o.x), 0x01010101, sum);
      sum = __dp4a(static_cast<int>(o.y), 0x01010101, sum);
    }
  }
  if (lane == 0) s_a[row] = sc;
  if (rowsum != nullptr) {
    sum = warp_sum_i32(sum);
    if (lane == 0) rowsum[row] = sum;
  }
}

// Any K (multiple of 8): two passes over the row, the second served by L1/L2.
template <bool EO>
__global__ void __launch_bounds__(kDaqWarps * 32)
daq_rows_2pass_kernel(const uint16_t* __restrict__ x, int64_t M, int K, int64_t ldx,
                      int8_t* __restrict__ q, int64_t ldq, float* __restrict__ s_a,
                      int32_t* __restrict__ rowsum, int tiled_kb, const UnpackJob job) {
  pdl_launch_dependents();
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kDaqWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_wait();
  if (static_cast<int>(blockIdx.x) >= job.first_block) {  // the launch's weight-expansion CTAs
    unpack_units(job, blockIdx.x - job.first_block);
    return;
  }
  if (row >= M) return;
  const int nvec = K >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(x + row * ldx);
  uint32_t m = 0;
  for (int idx = lane; idx < nvec; idx += 32) {
    uint4 v = xr[idx];
    m = absmax_bits2(absmax_bits2(absmax_bits2(absmax_bits2(m, v.x), v.y), v.z), v.w);
  }
  m = warp_max_u32(max(m & 0xFFFFu, m >> 16));
  float sc, inv;
  token_scale(m, sc, inv);
  const QRow qr(q, row, ldq, tiled_kb);
  int sum = 0;
  for (int idx = lane; idx < nvec; idx += 32) {
    uint2 o = quant_vec<EO>(xr[idx], inv);
    qr.store(idx, o);
    sum = __dp4a(static_cast<int>(o.x), 0x01010101, sum);
    sum = __dp4a(static_cast<int>(o.y), 0x01010101, sum);
  }
  if (lane == 0) s_a[row] = sc;
  if (rowsum != nullptr) {
    sum = warp_sum_i32(sum);
    if (lane == 0) rowsum[row] = sum;
  }
}

// ---- DAQ with a percentile clip and a-bit codes: robust_row in daq_device.cuh, one warp per token ----
template <int MAXV>
__global__ void __launch_bounds__(kDaqWarps * 32, MAXV <= 5 ? 3 : 2)  // register caps that keep 2-3 CTAs per SM
daq_rows_robust_kernel(const uint16_t* __restrict__ x, int64_t M, int K, int64_t ldx, int8_t* __restrict__ q,
                       int64_t ldq, float* __restrict__ s_a, int32_t* __restrict__ rowsum, int clip_rank,
                       float qmax, int tiled_kb, const UnpackJob job) {
  pdl_launch_dependents();
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kDaqWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_wait();
  if (static_cast<int>(blockIdx.x) >= job.first_block) {  // the launch's weight-expansion CTAs
    unpack_units(job, blockIdx.x - job.first_block);
    return;
  }
  if (row >= M) return;
  const QRow qr(q, row, ldq, tiled_kb);
  float sc;
  int sum;
  robust_row<MAXV>(x + row * ldx, K, lane, clip_rank, qmax, qr, sc, sum);
  if (lane == 0) s_a[row] = sc;
  if (rowsum != nullptr) {
    sum = warp_sum_i32(sum);
    if (lane == 0) rowsum[row] = sum;
  }
}

__global__ void __launch_bounds__(kDaqWarps * 32)
unpack_kernel(const UnpackJob job) {
  pdl_launch_dependents();
  pdl_wait();
  unpack_units(job, blockIdx.x);
}

template <bool EO>
static cudaError_t launch_daq_t(const uint16_t* xp, int64_t M, int k, int64_t ldx, int8_t* q, int64_t ldq,
                                float* s_a, int32_t* rowsum, int tiled_kb, cudaStream_t stream, bool pdl,
                                UnpackJob job) {
  const unsigned daq_blocks = static_cast<unsigned>((M + kDaqWarps - 1) / kDaqWarps);
  job.first_block = static_cast<int32_t>(daq_blocks);
  const unsigned extra = static_cast<unsigned>((job.units + kDaqWarps * 32 - 1) / (kDaqWarps * 32));
  const dim3 grid(daq_blocks + extra);
  const dim3 block(kDaqWarps * 32);
  if (k <= 256 * 5)
    return launch(daq_rows_kernel<5, EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, job);
  if (k <= 256 * 9)
    return launch(daq_rows_kernel<9, EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, job);
  if (k <= 256 * 18)
    return launch(daq_rows_kernel<18, EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, job);
  return launch(daq_rows_2pass_kernel<EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, job);
}

int launch_daq(const void* x, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq,
               float* s_a, int32_t* rowsum, int korder, bool tiled, cudaStream_t stream, bool pdl,
               const UnpackJob* unpack) {
  if (M == 0) return DP_OK;
  const uint16_t* xp = static_cast<const uint16_t*>(x);
  const int k = static_cast<int>(K);
  const int tiled_kb = tiled ? k / 128 : 0;
  UnpackJob job{nullptr, nullptr, 0, 0, 0};
  if (unpack != nullptr) job = *unpack;
  const cudaError_t e = korder == KORDER_EVEN_ODD
                            ? launch_daq_t<true>(xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, stream, pdl, job)
                            : launch_daq_t<false>(xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, stream, pdl, job);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "DAQ launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

int launch_daq_robust(const void* x, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq, float* s_a,
                      int32_t* rowsum, int clip_rank, int act_bits, bool tiled, cudaStream_t stream, bool pdl,
                      const UnpackJob* unpack) {
  if (M == 0) return DP_OK;
  const uint16_t* xp = static_cast<const uint16_t*>(x);
  const int k = static_cast<int>(K);
  const int tiled_kb = tiled ? k / 128 : 0;
  const float qmax = static_cast<float>((1 << (act_bits - 1)) - 1);
  UnpackJob job{nullptr, nullptr, 0, 0, 0};
  if (unpack != nullptr) job = *unpack;
  const unsigned daq_blocks = static_cast<unsigned>((M + kDaqWarps - 1) / kDaqWarps);
  job.first_block = static_cast<int32_t>(daq_blocks);
  const unsigned extra = static_cast<unsigned>((job.units + kDaqWarps * 32 - 1) / (kDaqWarps * 32));
  const dim3 grid(daq_blocks + extra), block(kDaqWarps * 32);
  cudaError_t e;
  if (k <= 256 * 5)
    e = launch(daq_rows_robust_kernel<5>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, clip_rank,
               qmax, tiled_kb, job);
  else if (k <= 256 * 9)
    e = launch(daq_rows_robust_kernel<9>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, clip_rank,
               qmax, tiled_kb, job);
  else
    e = launch(daq_rows_robust_kernel<18>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, clip_rank,
               qmax, tiled_kb, job);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "robust DAQ launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

int launch_unpack(const UnpackJob& job, cudaStream_t stream, bool pdl) {
  if (job.units == 0) return DP_OK;
  const dim3 grid(static_cast<unsigned>((job.units + kDaqWarps * 32 - 1) / (kDaqWarps * 32)));
  const cudaError_t e = launch(unpack_kernel, grid, dim3(kDaqWarps * 32), 0, stream, pdl, job);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "weight expansion launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp

extern "C" int dp_daq_quantize(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q,
                               int64_t ldq, float* s_a, int32_t* rowsum, dp_stream stream) {
  using namespace dp;
  if (M < 0 || K < 8 || K > 65536) return fail(DP_ERR_SHAPE, "dp_daq_quantize: bad M=%lld K=%lld",
                                                (long long)M, (long long)K);
  if (K % 8) return fail(DP_ERR_SHAPE, "dp_daq_quantize: K=%lld not a multiple of 8", (long long)K);
  if (M == 0) return DP_OK;
  if (!x_bf16 || !q || !s_a) return fail(DP_ERR_INVALID_ARG, "dp_daq_quantize: NULL pointer");
  if (ldx < K || ldq < K) return fail(DP_ERR_SHAPE, "dp_daq_quantize: leading dimension < K");
  if (!aligned16(x_bf16) || !aligned16(q) || (ldx % 8) || (ldq % 16) ||
      (reinterpret_cast<uintptr_t>(s_a) & 3u))
    return fail(DP_ERR_ALIGN, "dp_daq_quantize: pointers/pitches must be 16-byte aligned");
  int st = check_device();
  if (st != DP_OK) return st;
  return launch_daq(x_bf16, M, K, ldx, q, ldq, s_a, rowsum, KORDER_NATURAL, false,
                    static_cast<cudaStream_t>(stream), false);
}

extern "C" int dp_daq_quantize_robust(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q,
                                      int64_t ldq, float* s_a, int32_t* rowsum, int32_t clip_rank,
                                      int32_t act_bits, dp_stream stream) {
  using namespace dp;
  if (M < 0 || K < 8 || K > 4608 || (K % 8))
    return fail(DP_ERR_SHAPE, "dp_daq_quantize_robust: need M >= 0 and K a multiple of 8 in [8, 4608] (M=%lld K=%lld)",
                (long long)M, (long long)K);
  if (clip_rank < 1 || clip_rank > 64 || clip_rank > K)
    return fail(DP_ERR_INVALID_ARG, "dp_daq_quantize_robust: clip_rank=%d not in [1, min(K, 64)]", clip_rank);
  if (act_bits < 2 || act_bits > 8)
    return fail(DP_ERR_BITS, "dp_daq_quantize_robust: act_bits=%d not in [2, 8]", act_bits);
  if (M == 0) return DP_OK;
  if (!x_bf16 || !q || !s_a) return fail(DP_ERR_INVALID_ARG, "dp_daq_quantize_robust: NULL pointer");
  if (ldx < K || ldq < K) return fail(DP_ERR_SHAPE, "dp_daq_quantize_robust: leading dimension < K");
  if (!aligned16(x_bf16) || !aligned16(q) || (ldx % 8) || (ldq % 16) || (reinterpret_cast<uintptr_t>(s_a) & 3u))
    return fail(DP_ERR_ALIGN, "dp_daq_quantize_robust: pointers/pitches must be 16-byte aligned");
  int st = check_device();
  if (st != DP_OK) return st;
  return launch_daq_robust(x_bf16, M, K, ldx, q, ldq, s_a, rowsum, clip_rank, act_bits, false,
                           static_cast<cudaStream_t>(stream), false, nullptr);
}
