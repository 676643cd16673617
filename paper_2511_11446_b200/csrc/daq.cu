// Dynamic activation quantization (Step 3, Eq. "daq"; b = 8, zero-point 0, clip threshold = the
// token's absolute maximum): bf16 [M][K] -> int8 codes + one fp32 scale per token.
//
// One warp owns one token. The row is read once with 16-byte loads and kept in registers; the
// absolute maximum is taken on the bf16 magnitude bits (monotone for finite values, so integer
// max is exact); the quantizer is one fused multiply-add per element: x * fl(127/a) + 1.5*2^23
// rounds the exact product once, half to even, and leaves the integer in the low mantissa bits.
// HBM-bound: 2 bytes read + 1 byte written per element.
#include "dp_common.cuh"
#include "dp_internal.h"

namespace dp {

__device__ __forceinline__ uint32_t ld_nc_u32x4(const uint4* p, uint4& v) {
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return 0;
}

__device__ __forceinline__ uint32_t absmax_bits2(uint32_t m, uint32_t w) {
  return __vmaxu2(m, w & 0x7FFF7FFFu);
}

// Quantizes two bf16 packed in `w` (low half = even k) -> two int8 in the low bytes of result
// positions chosen by the caller.
__device__ __forceinline__ uint32_t quant_pair(uint32_t w, float inv) {
  const float magic = 12582912.0f;  // 1.5 * 2^23
  float lo = __uint_as_float(w << 16);
  float hi = __uint_as_float(w & 0xFFFF0000u);
  uint32_t a = __float_as_uint(__fmaf_rn(lo, inv, magic));
  uint32_t b = __float_as_uint(__fmaf_rn(hi, inv, magic));
  return __byte_perm(a, b, 0x0040);  // byte0 = a.byte0, byte1 = b.byte0
}

// Eight consecutive codes. EO = false: stored in order; EO = true: stored as k = 0,2,4,6,1,3,5,7.
template <bool EO>
__device__ __forceinline__ uint2 quant_vec(const uint4& v, float inv) {
  uint32_t p0 = quant_pair(v.x, inv), p1 = quant_pair(v.y, inv);
  uint32_t p2 = quant_pair(v.z, inv), p3 = quant_pair(v.w, inv);
  if constexpr (EO) {
    const uint32_t t0 = __byte_perm(p0, p1, 0x5140);  // k0 k2 k1 k3
    const uint32_t t1 = __byte_perm(p2, p3, 0x5140);  // k4 k6 k5 k7
    return make_uint2(__byte_perm(t0, t1, 0x5410), __byte_perm(t0, t1, 0x7632));
  } else {
    return make_uint2(__byte_perm(p0, p1, 0x5410), __byte_perm(p2, p3, 0x5410));
  }
}

// Scale and reciprocal of one token from its absmax magnitude bits (a bf16 pattern, sign cleared).
__device__ __forceinline__ void token_scale(uint32_t abits, float& s_a, float& inv) {
  float a = __uint_as_float(abits << 16);
  if (a < 7.888609052210118e-31f) {  // 2^-100: treat the token as all-zero
    s_a = 0.0f;
    inv = 0.0f;
  } else {
    s_a = __fdiv_rn(a, 127.0f);
    inv = __fdiv_rn(127.0f, a);
  }
}

__device__ __forceinline__ uint32_t warp_max_u32(uint32_t m) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  return m;
}
__device__ __forceinline__ int warp_sum_i32(int s) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  return s;
}

// Where the 8 codes of vector `idx` (k = 8 idx ..) of one token go. Row-major: q[row][k]. Tiled
// (tiled_kb = K / 128 > 0): the matrix is cut into 128-token x 128-code tiles of 16 KB, stored one
// after the other ([row tile][k block][128][128]), so that the GEMM's TMA loads of an activation tile
// read one contiguous 16 KB range instead of 128 rows a whole row pitch apart.
struct QRow {
  uint2* base;
  int tiled;
  __device__ __forceinline__ QRow(int8_t* q, int64_t row, int64_t ldq, int tiled_kb) : tiled(tiled_kb) {
    base = tiled_kb ? reinterpret_cast<uint2*>(q + ((row >> 7) * tiled_kb) * 16384 + (row & 127) * 128)
                    : reinterpret_cast<uint2*>(q + row * ldq);
  }
  __device__ __forceinline__ void store(int idx, uint2 v) const {
    if (tiled) base[(idx >> 4) * 2048 + (idx & 15)] = v;  // next k block: + 16384 bytes
    else base[idx] = v;
  }
};

constexpr int kDaqWarps = 8;

// MAXV = 16-byte vectors held per lane (row of up to 256*MAXV elements in registers).
template <int MAXV, bool EO>
__global__ void __launch_bounds__(kDaqWarps * 32)
daq_rows_kernel(const uint16_t* __restrict__ x, int64_t M, int K, int64_t ldx,
                int8_t* __restrict__ q, int64_t ldq, float* __restrict__ s_a,
                int32_t* __restrict__ rowsum, int tiled_kb) {
  pdl_launch_dependents();
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kDaqWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_wait();
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
                      int32_t* __restrict__ rowsum, int tiled_kb) {
  pdl_launch_dependents();
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kDaqWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_wait();
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

template <bool EO>
static cudaError_t launch_daq_t(const uint16_t* xp, int64_t M, int k, int64_t ldx, int8_t* q, int64_t ldq,
                                float* s_a, int32_t* rowsum, int tiled_kb, cudaStream_t stream, bool pdl) {
  const dim3 grid(static_cast<unsigned>((M + kDaqWarps - 1) / kDaqWarps));
  const dim3 block(kDaqWarps * 32);
  if (k <= 256 * 5)
    return launch(daq_rows_kernel<5, EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb);
  if (k <= 256 * 9)
    return launch(daq_rows_kernel<9, EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb);
  if (k <= 256 * 18)
    return launch(daq_rows_kernel<18, EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb);
  return launch(daq_rows_2pass_kernel<EO>, grid, block, 0, stream, pdl, xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb);
}

int launch_daq(const void* x, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq,
               float* s_a, int32_t* rowsum, int korder, bool tiled, cudaStream_t stream, bool pdl) {
  if (M == 0) return DP_OK;
  const uint16_t* xp = static_cast<const uint16_t*>(x);
  const int k = static_cast<int>(K);
  const int tiled_kb = tiled ? k / 128 : 0;
  const cudaError_t e = korder == KORDER_EVEN_ODD
                            ? launch_daq_t<true>(xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, stream, pdl)
                            : launch_daq_t<false>(xp, M, k, ldx, q, ldq, s_a, rowsum, tiled_kb, stream, pdl);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "DAQ launch failed: %s", cudaGetErrorString(e));
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
