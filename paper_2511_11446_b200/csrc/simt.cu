// CUDA-core path of the quantized linear for small row counts (adaLN modulation: M = batch).
//
// The whole layer in one launch: each CTA quantizes its (up to 8) tokens into shared memory
// (DAQ, Step 3 Eq. "daq"), then its warps stream packed weight rows from HBM, expand them to int8
// in registers, take dp4a dot products against the shared int8 tokens, and apply the dequant
// epilogue. The shape is bound by the weight bytes (M <= 32: 2..144 int8 ops per weight byte).
#include <cuda_bf16.h>

#include "dp_common.cuh"
#include "dp_internal.h"

namespace dp {

constexpr int kSimtRows = 8;     // tokens per CTA
constexpr int kSimtWarps = 8;
constexpr int kSimtChPerCta = 32;  // output channels per CTA

// 32 consecutive k of one weight row -> 8 words of 4 int8 (true values).
template <int BITS>
__device__ __forceinline__ void load_unit(const uint32_t* __restrict__ row, int unit,
                                          uint32_t (&w)[8]) {
  if constexpr (BITS == 8) {
    const uint4* p = reinterpret_cast<const uint4*>(row) + unit * 2;
    uint4 a = __ldg(p), b = __ldg(p + 1);
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
    w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
  } else if constexpr (BITS == 4) {
    uint4 a = __ldg(reinterpret_cast<const uint4*>(row) + unit);
    const uint32_t in[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t lo = in[i] & 0x0F0F0F0Fu, hi = (in[i] >> 4) & 0x0F0F0F0Fu;
      w[2 * i] = __vsub4(__byte_perm(lo, hi, 0x5140), 0x08080808u);
      w[2 * i + 1] = __vsub4(__byte_perm(lo, hi, 0x7362), 0x08080808u);
    }
  } else {
    const uint32_t* p = row + unit * 3;
    const uint32_t s0 = __ldg(p), s1 = __ldg(p + 1), s2 = __ldg(p + 2);
    const uint64_t lo64 = (static_cast<uint64_t>(s1) << 32) | s0;
    const uint64_t hi64 = (static_cast<uint64_t>(s2) << 32) | s1;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int bit = 12 * j;
      const uint32_t x = static_cast<uint32_t>(bit < 32 ? (lo64 >> bit) : (hi64 >> (bit - 32))) &
                         0xFFFu;
      uint32_t o = (x & 7u) | ((x & 0x38u) << 5) | ((x & 0x1C0u) << 10) | ((x & 0xE00u) << 15);
      w[j] = __vsub4(o, 0x04040404u);
    }
  }
}

template <int BITS>
__global__ void __launch_bounds__(kSimtWarps * 32)
simt_linear_kernel(SimtArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  int8_t* sq = reinterpret_cast<int8_t*>(smem);                       // [kSimtRows][K]
  float* ssa = reinterpret_cast<float*>(smem + kSimtRows * a.K);      // [kSimtRows]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * kSimtRows;
  const int K = a.K;
  pdl_launch_dependents();
  pdl_wait();

  // ---- prologue: this CTA's tokens -> int8 in shared memory (one warp per token) ----
  {
    const int64_t row = m0 + warp;
    uint2* dst = reinterpret_cast<uint2*>(sq + warp * K);
    const int nvec = K >> 3;
    if (row >= a.M) {
      for (int i = lane; i < nvec; i += 32) dst[i] = make_uint2(0, 0);
      if (lane == 0) ssa[warp] = 0.0f;
    } else if (a.s_a_in != nullptr) {
      const uint2* src = reinterpret_cast<const uint2*>(static_cast<const int8_t*>(a.x) + row * a.ldx);
      for (int i = lane; i < nvec; i += 32) dst[i] = src[i];
      if (lane == 0) ssa[warp] = a.s_a_in[row];
    } else {
      const uint4* xr = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(a.x) + row * a.ldx);
      uint32_t mx = 0;
      for (int i = lane; i < nvec; i += 32) {
        uint4 v = xr[i];
        mx = __vmaxu2(mx, v.x & 0x7FFF7FFFu);
        mx = __vmaxu2(mx, v.y & 0x7FFF7FFFu);
        mx = __vmaxu2(mx, v.z & 0x7FFF7FFFu);
        mx = __vmaxu2(mx, v.w & 0x7FFF7FFFu);
      }
      mx = max(mx & 0xFFFFu, mx >> 16);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
      const float amax = __uint_as_float(mx << 16);
      float sc = 0.0f, inv = 0.0f;
      if (!(amax < 7.888609052210118e-31f)) {  // 2^-100
        sc = __fdiv_rn(amax, 127.0f);
        inv = __fdiv_rn(127.0f, amax);
      }
      const float magic = 12582912.0f;
      for (int i = lane; i < nvec; i += 32) {
        uint4 v = xr[i];
        const uint32_t in[4] = {v.x, v.y, v.z, v.w};
        uint32_t b[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          b[2 * j] = __float_as_uint(__fmaf_rn(__uint_as_float(in[j] << 16), inv, magic)) & 0xFFu;
          b[2 * j + 1] =
              __float_as_uint(__fmaf_rn(__uint_as_float(in[j] & 0xFFFF0000u), inv, magic)) & 0xFFu;
        }
        dst[i] = make_uint2(b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24),
                            b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24));
      }
      if (lane == 0) ssa[warp] = sc;
    }
    if (blockIdx.x == 0 && row < a.M) {  // optional taps, written once per token
      if (a.dbg_sa != nullptr && lane == 0) a.dbg_sa[row] = ssa[warp];
      if (a.dbg_q != nullptr) {
        __syncwarp();
        uint2* dq = reinterpret_cast<uint2*>(a.dbg_q + row * a.dbg_ldq);
        for (int i = lane; i < nvec; i += 32) dq[i] = dst[i];
      }
    }
  }
  __syncthreads();

  // ---- weight streaming: warp w takes channels n0 + w, n0 + w + 8, ... ----
  const int units = K >> 5;
  const int row_words = (K * BITS) >> 5;
  const int n0 = blockIdx.x * kSimtChPerCta;
  for (int c = warp; c < kSimtChPerCta; c += kSimtWarps) {
    const int n = n0 + c;
    if (n >= a.N) break;
    const uint32_t* wrow = static_cast<const uint32_t*>(a.qweight) + static_cast<int64_t>(n) * row_words;
    int acc[kSimtRows];
#pragma unroll
    for (int m = 0; m < kSimtRows; ++m) acc[m] = 0;
    for (int u = lane; u < units; u += 32) {
      uint32_t w[8];
      load_unit<BITS>(wrow, u, w);
#pragma unroll
      for (int m = 0; m < kSimtRows; ++m) {
        const uint4* qp = reinterpret_cast<const uint4*>(sq + m * K + u * 32);
        const uint4 q0 = qp[0], q1 = qp[1];
        int s = acc[m];
        s = __dp4a(static_cast<int>(q0.x), static_cast<int>(w[0]), s);
        s = __dp4a(static_cast<int>(q0.y), static_cast<int>(w[1]), s);
        s = __dp4a(static_cast<int>(q0.z), static_cast<int>(w[2]), s);
        s = __dp4a(static_cast<int>(q0.w), static_cast<int>(w[3]), s);
        s = __dp4a(static_cast<int>(q1.x), static_cast<int>(w[4]), s);
        s = __dp4a(static_cast<int>(q1.y), static_cast<int>(w[5]), s);
        s = __dp4a(static_cast<int>(q1.z), static_cast<int>(w[6]), s);
        s = __dp4a(static_cast<int>(q1.w), static_cast<int>(w[7]), s);
        acc[m] = s;
      }
    }
    int mine = 0;
#pragma unroll
    for (int m = 0; m < kSimtRows; ++m) {
      int s = acc[m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
      if (lane == m) mine = s;
    }
    if (lane < kSimtRows && m0 + lane < a.M) {
      const int64_t row = m0 + lane;
      const float t = static_cast<float>(mine);
      const float sc = __fmul_rn(ssa[lane], a.s_w[n]);
      const float b = a.bias != nullptr ? __uint_as_float(static_cast<uint32_t>(a.bias[n]) << 16) : 0.0f;
      const float y = __fmaf_rn(t, sc, b);
      a.y[row * a.ldy + n] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
      if (a.dbg_acc != nullptr) a.dbg_acc[row * a.dbg_ldacc + n] = mine;
    }
  }
}

size_t simt_max_k() { return 16384; }

int launch_simt_linear(const SimtArgs& a, cudaStream_t stream, bool pdl) {
  if (a.M == 0) return DP_OK;
  const size_t smem = static_cast<size_t>(kSimtRows) * a.K + kSimtRows * sizeof(float);
  const dim3 grid((a.N + kSimtChPerCta - 1) / kSimtChPerCta,
                  static_cast<unsigned>((a.M + kSimtRows - 1) / kSimtRows));
  const dim3 block(kSimtWarps * 32);
  void (*kern)(SimtArgs) = a.bits == 8 ? simt_linear_kernel<8>
                           : a.bits == 4 ? simt_linear_kernel<4> : simt_linear_kernel<3>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "simt smem attribute: %s", cudaGetErrorString(e));
  }
  cudaError_t e = launch(kern, grid, block, smem, stream, pdl, a);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "simt launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
