// LayerNorm + adaLN modulation taken into dynamic activation quantization.
//
//   Step 3 of the paper keeps LayerNorms in higher precision and quantizes the activations of the
//   wrapped linears on the fly (Eq. "daq"). In a DiT block the qkv and fc1 linears are fed
//   LayerNorm(x) * (1 + scale) + shift with a per-sample adaLN scale and shift; run as separate
//   operators that is a normalization kernel writing bf16, and a quantization kernel reading it
//   back. Here one kernel reads the block's bf16 stream once and writes int8 codes and token scales:
//   the normalized, modulated values exist only in fp32 registers and are never rounded to bf16.
//
// Arithmetic (the oracle's, bit for bit): sums of x and x^2 of a token in double (the terms are bf16
// values and their squares; for activations whose magnitudes span less than ~2^13 every partial sum is
// exact, so the order of summation cannot matter; beyond that the sums differ from a sequential sum
// by double-precision roundings only), mean = S1 / K, var = S2 / K - mean^2, rstd = 1 / sqrt(var +
// eps), all in double with IEEE operations, then rounded to fp32; n = (x - mean) * rstd and
// h = fma(n, 1 + scale, shift) in fp32; DAQ of h as for bf16 inputs (absmax / 127, one rounding of
// the exact product with fl(127 / absmax), half to even).
//
// One warp owns one token; the row stays in registers as bf16 (16-byte loads); h is recomputed for
// the quantization pass only when the row is too long to keep it (same operations, same bits). Moves
// DAQ's bytes (2 read + 1 written per element) but is bound by the double-precision additions of the
// statistics (two per element; building the doubles with integer operations instead of the
// conversion instruction was slower): 34 us at M = 32768, K = 1152 against 19 us for DAQ alone.
#include "daq_device.cuh"

namespace dp {

constexpr int kLnWarps = 8;

struct LnArgs {
  const uint16_t* x;
  int64_t M, ldx;
  int K;
  const uint16_t* shift;  // [ceil(M / rows_per_sample)][K] or nullptr (then scale is nullptr too)
  const uint16_t* scale;
  int64_t rows_per_sample;
  float eps;
  int8_t* q;
  int64_t ldq;
  float* s_a;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// two bf16 packed in a word -> two fp32 packed in 64 bits
__device__ __forceinline__ uint64_t bf16x2_to_f32x2(uint32_t w) {
  return (static_cast<uint64_t>(w & 0xFFFF0000u) << 32) | static_cast<uint64_t>(w << 16);
}

// h of the two elements packed in w (modulation words sw, hw when MOD), as packed fp32 operations
// (each half rounded like the scalar instruction); nmean2 = (-mean, -mean), rstd2, one2 likewise.
template <bool MOD>
__device__ __forceinline__ uint64_t ln_pair(uint32_t w, uint32_t sw, uint32_t hw, uint64_t nmean2, uint64_t rstd2,
                                            uint64_t one2) {
  uint64_t h = f32x2_mul(f32x2_add(bf16x2_to_f32x2(w), nmean2), rstd2);  // x - mean is x + (-mean) exactly
  if constexpr (MOD) h = f32x2_fma(h, f32x2_add(one2, bf16x2_to_f32x2(sw)), bf16x2_to_f32x2(hw));
  return h;
}

template <int MAXV, bool MOD>
__global__ void __launch_bounds__(kLnWarps * 32) ln_modulate_daq_kernel(const LnArgs a) {
  pdl_launch_dependents();
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kLnWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  pdl_wait();
  if (row >= a.M) return;
  const int nvec = a.K >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(a.x + row * a.ldx);
  uint4 v[MAXV];
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) ld_nc_u32x4(xr + idx, v[i]);
    else v[i] = make_uint4(0, 0, 0, 0);
  }
  // ---- token statistics in double ----
  double s1 = 0.0, s2 = 0.0;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    if (lane + 32 * i >= nvec) continue;  // (padding vectors are zero: nothing to add)
    const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const double lo = static_cast<double>(bf16_lo(w[j])), hi = static_cast<double>(bf16_hi(w[j]));
      s1 = __dadd_rn(s1, lo);
      s1 = __dadd_rn(s1, hi);
      s2 = __fma_rn(lo, lo, s2);
      s2 = __fma_rn(hi, hi, s2);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s1 = __dadd_rn(s1, __shfl_xor_sync(0xFFFFFFFFu, s1, o));
    s2 = __dadd_rn(s2, __shfl_xor_sync(0xFFFFFFFFu, s2, o));
  }
  const double kd = static_cast<double>(a.K);
  const double mean_d = __ddiv_rn(s1, kd);
  double var_d = __dsub_rn(__ddiv_rn(s2, kd), __dmul_rn(mean_d, mean_d));
  if (var_d < 0.0) var_d = 0.0;
  const float mean = __double2float_rn(mean_d);
  const float rstd = __double2float_rn(__ddiv_rn(1.0, __dsqrt_rn(__dadd_rn(var_d, static_cast<double>(a.eps)))));
  // ---- h and its absmax (kept in registers when the row is short enough, else recomputed below) ----
  constexpr bool KEEP = MAXV <= 5;
  const uint4* shr = nullptr;
  const uint4* scr = nullptr;
  if constexpr (MOD) {
    const int64_t sample = row / a.rows_per_sample;
    shr = reinterpret_cast<const uint4*>(a.shift + sample * a.K);
    scr = reinterpret_cast<const uint4*>(a.scale + sample * a.K);
  }
  const uint64_t nmean2 = f32x2_pack(-mean, -mean), rstd2 = f32x2_pack(rstd, rstd), one2 = f32x2_pack(1.0f, 1.0f);
  uint64_t hk[KEEP ? MAXV * 4 : 1];
  auto h_of = [&](const int i, const int idx, uint64_t (&h)[4]) {
    uint4 sh = make_uint4(0, 0, 0, 0), sc = sh;
    if constexpr (MOD) {
      sh = __ldg(shr + idx);
      sc = __ldg(scr + idx);
    }
    h[0] = ln_pair<MOD>(v[i].x, sc.x, sh.x, nmean2, rstd2, one2);
    h[1] = ln_pair<MOD>(v[i].y, sc.y, sh.y, nmean2, rstd2, one2);
    h[2] = ln_pair<MOD>(v[i].z, sc.z, sh.z, nmean2, rstd2, one2);
    h[3] = ln_pair<MOD>(v[i].w, sc.w, sh.w, nmean2, rstd2, one2);
  };
  uint32_t amax_bits = 0;  // |h| as an integer: ordered like the value for finite h
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) {
      uint64_t h[4];
      h_of(i, idx, h);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        amax_bits = max(amax_bits, static_cast<uint32_t>(h[j]) & 0x7FFFFFFFu);
        amax_bits = max(amax_bits, static_cast<uint32_t>(h[j] >> 32) & 0x7FFFFFFFu);
        if constexpr (KEEP) hk[4 * i + j] = h[j];
      }
    }
  }
  amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
  const float amax = __uint_as_float(amax_bits);
  float sa = 0.0f, inv = 0.0f;
  if (!(amax < 7.888609052210118e-31f)) {  // 2^-100: below it the token is all-zero, as in the bf16 form
    sa = __fdiv_rn(amax, 127.0f);
    inv = __fdiv_rn(127.0f, amax);
  }
  // ---- quantize: fma(h, inv, 1.5 * 2^23) rounds the exact product once, half to even ----
  const uint64_t inv2 = f32x2_pack(inv, inv), magic2 = f32x2_pack(12582912.0f, 12582912.0f);
  uint2* qrow = reinterpret_cast<uint2*>(a.q + row * a.ldq);
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) {
      uint64_t h[4];
      if constexpr (KEEP) {
#pragma unroll
        for (int j = 0; j < 4; ++j) h[j] = hk[4 * i + j];
      } else {
        h_of(i, idx, h);
      }
      uint32_t p[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint64_t r = f32x2_fma(h[j], inv2, magic2);
        p[j] = __byte_perm(static_cast<uint32_t>(r), static_cast<uint32_t>(r >> 32), 0x0040);  // two codes in the low bytes
      }
      qrow[idx] = make_uint2(__byte_perm(p[0], p[1], 0x5410), __byte_perm(p[2], p[3], 0x5410));
    }
  }
  if (lane == 0) a.s_a[row] = sa;
}

template <int MAXV>
static cudaError_t launch_ln_v(const LnArgs& a, dim3 grid, cudaStream_t stream, bool pdl) {
  if (a.shift != nullptr) return launch(ln_modulate_daq_kernel<MAXV, true>, grid, dim3(kLnWarps * 32), 0, stream, pdl, a);
  return launch(ln_modulate_daq_kernel<MAXV, false>, grid, dim3(kLnWarps * 32), 0, stream, pdl, a);
}

int launch_ln_modulate_daq(const void* x, int64_t M, int64_t K, int64_t ldx, const void* shift, const void* scale,
                           int64_t rows_per_sample, float eps, int8_t* q, int64_t ldq, float* s_a,
                           cudaStream_t stream, bool pdl) {
  if (M == 0) return DP_OK;
  LnArgs a{static_cast<const uint16_t*>(x), M, ldx, static_cast<int>(K), static_cast<const uint16_t*>(shift),
           static_cast<const uint16_t*>(scale), rows_per_sample, eps, q, ldq, s_a};
  const dim3 grid(static_cast<unsigned>((M + kLnWarps - 1) / kLnWarps));
  cudaError_t e = K <= 256 * 5 ? launch_ln_v<5>(a, grid, stream, pdl) : launch_ln_v<18>(a, grid, stream, pdl);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "LayerNorm + DAQ launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
