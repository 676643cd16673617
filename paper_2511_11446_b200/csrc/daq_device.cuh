// Device-side pieces of dynamic activation quantization (Step 3, Eq. "daq"; b = 8, zero-point 0,
// clip threshold = the token's absolute maximum) shared by the stand-alone DAQ kernels and by the
// GEMM kernels that quantize their own activations.
#pragma once

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
    uint2* p = tiled ? base + (idx >> 4) * 2048 + (idx & 15) : base + idx;  // next k block: + 16384 bytes
    // read next by another kernel, through L2: no L1 allocation
    asm volatile("st.global.L1::no_allocate.v2.b32 [%0], {%1, %2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
  }
};

// One token by one warp, any K (multiple of 8): two passes over the row, the second served by
// L1/L2. Writes the codes through `qr` and returns the scale (valid in every lane).
template <bool EO>
__device__ __forceinline__ float daq_row_2pass(const uint16_t* __restrict__ x_row, int K, const QRow& qr, int lane) {
  const int nvec = K >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(x_row);
  uint32_t m = 0;
#pragma unroll 5
  for (int idx = lane; idx < nvec; idx += 32) {
    const uint4 v = xr[idx];
    m = absmax_bits2(absmax_bits2(absmax_bits2(absmax_bits2(m, v.x), v.y), v.z), v.w);
  }
  m = warp_max_u32(max(m & 0xFFFFu, m >> 16));
  float sc, inv;
  token_scale(m, sc, inv);
#pragma unroll 5
  for (int idx = lane; idx < nvec; idx += 32) qr.store(idx, quant_vec<EO>(xr[idx], inv));
  return sc;
}

// Two tokens by one warp at once (the loads of both are in flight together, which matters when the
// warp has several tokens to do and each costs a full memory round trip). has_b == false: only A.
template <bool EO>
__device__ __forceinline__ void daq_two_rows_2pass(const uint16_t* __restrict__ xa, const uint16_t* __restrict__ xb,
                                                   bool has_b, int K, const QRow& qa, const QRow& qb, int lane,
                                                   float& sc_a, float& sc_b) {
  const int nvec = K >> 3;
  const uint4* ra = reinterpret_cast<const uint4*>(xa);
  const uint4* rb = reinterpret_cast<const uint4*>(has_b ? xb : xa);
  uint32_t ma = 0, mb = 0;
#pragma unroll 5
  for (int idx = lane; idx < nvec; idx += 32) {
    const uint4 va = ra[idx], vb = rb[idx];
    ma = absmax_bits2(absmax_bits2(absmax_bits2(absmax_bits2(ma, va.x), va.y), va.z), va.w);
    mb = absmax_bits2(absmax_bits2(absmax_bits2(absmax_bits2(mb, vb.x), vb.y), vb.z), vb.w);
  }
  ma = max(ma & 0xFFFFu, ma >> 16);
  mb = max(mb & 0xFFFFu, mb >> 16);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ma = max(ma, __shfl_xor_sync(0xFFFFFFFFu, ma, o));
    mb = max(mb, __shfl_xor_sync(0xFFFFFFFFu, mb, o));
  }
  float inv_a, inv_b;
  token_scale(ma, sc_a, inv_a);
  token_scale(mb, sc_b, inv_b);
#pragma unroll 5
  for (int idx = lane; idx < nvec; idx += 32) {
    qa.store(idx, quant_vec<EO>(ra[idx], inv_a));
    if (has_b) qb.store(idx, quant_vec<EO>(rb[idx], inv_b));
  }
}

// ---- DAQ with a percentile clip and a-bit codes -------------------------------------------------------
// Eq. "daq" with tau = Percentile(|v|, p) below the maximum (nearest-rank reading: the clip_rank-th
// largest magnitude of the token, repeats counted) and alpha = tau / qmax, qmax = 2^(a-1) - 1 for the
// activation bits a of the step's time bin (Step 6). One warp per token, row in registers as above.
// The threshold is found by peeling maxima: each round takes the largest magnitude below the
// previous one together with its multiplicity until clip_rank values are covered (for p = 99.9: 2
// rounds at K = 1152, 5 at K = 4608). A lane keeps the maximum of each of its 8-element vectors, so
// a round is a max over those few numbers plus a rescan of only the vectors that held the peeled
// value. Values beyond tau are clipped to it before the multiplication and so land on +-qmax.
// Packed helpers on words of two 15-bit magnitudes (bit 15 of each half clear):
// number of halves equal to the value replicated in t2
__device__ __forceinline__ int count_eq2(uint32_t e, uint32_t t2) {
  const uint32_t z = ((e ^ t2) | 0x80008000u) - 0x00010001u;  // bit 15 of a half stays set unless the half was 0
  return __popc(~z & 0x80008000u);
}
// the halves that are below the bound replicated in b2 (<= 0x8000 per half), the others zeroed
__device__ __forceinline__ uint32_t keep_below2(uint32_t e, uint32_t b2) {
  const uint32_t ge = ((e | 0x80008000u) - b2) & 0x80008000u;  // bit 15 set where half >= bound; no borrow
  return e & ~(ge - (ge >> 15));
}
__device__ __forceinline__ uint32_t fold_max2(uint32_t m2) { return max(m2 & 0xFFFFu, m2 >> 16); }
// Two bf16 clipped to [-tau, tau] (tau2 = tau's magnitude bits in both halves): the magnitudes are
// 15-bit integers ordered like the values, so one packed minimum does it; then quantized as usual.
// Clipping first and rounding after is the equation's own order and cannot leave +-qmax.
__device__ __forceinline__ uint32_t quant_pair_clipped(uint32_t w, uint32_t tau2, float inv) {
  return quant_pair((w & 0x80008000u) | __vminu2(w & 0x7FFF7FFFu, tau2), inv);
}

// One token by one warp: x[K] bf16 (16-byte aligned) -> codes through `qr`, scale in `sc`, the lane's
// partial code sum in `sum`. K <= 256 * MAXV.
template <int MAXV>
__device__ __forceinline__ void robust_row(const uint16_t* __restrict__ x, int K, int lane, int clip_rank, float qmax,
                                           const QRow& qr, float& sc, int& sum) {
  const int nvec = K >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(x);
  uint4 v[MAXV];
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) ld_nc_u32x4(xr + idx, v[i]);
    else v[i] = make_uint4(0, 0, 0, 0);
  }
  // threshold: magnitude bits (bf16 pattern, sign cleared) of the clip_rank-th largest element
  uint32_t gmax[MAXV];  // per vector: its largest magnitude not yet peeled (padding vectors: 0)
#pragma unroll
  for (int i = 0; i < MAXV; ++i)
    gmax[i] = fold_max2(absmax_bits2(absmax_bits2(absmax_bits2(absmax_bits2(0u, v[i].x), v[i].y), v[i].z), v[i].w));
  uint32_t tau_bits = 0;
  int remaining = clip_rank;
  if (clip_rank == 2) {
    // The second largest magnitude (p = 99.9 at K = 1152) without peeling: a running (largest, second)
    // pair per packed half, three packed operations per two elements, then merged across the halves
    // and the warp; (a1, a2) + (b1, b2) = (max(a1, b1), max(min(a1, b1), max(a2, b2))) keeps repeats.
    uint32_t m1 = 0, m2 = 0;
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const uint32_t w[4] = {v[i].x & 0x7FFF7FFFu, v[i].y & 0x7FFF7FFFu, v[i].z & 0x7FFF7FFFu, v[i].w & 0x7FFF7FFFu};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        m2 = __vmaxu2(m2, __vminu2(m1, w[j]));
        m1 = __vmaxu2(m1, w[j]);
      }
    }
    uint32_t t1 = max(m1 & 0xFFFFu, m1 >> 16);
    uint32_t t2 = max(min(m1 & 0xFFFFu, m1 >> 16), max(m2 & 0xFFFFu, m2 >> 16));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const uint32_t u1 = __shfl_xor_sync(0xFFFFFFFFu, t1, o), u2 = __shfl_xor_sync(0xFFFFFFFFu, t2, o);
      t2 = max(min(t1, u1), max(t2, u2));
      t1 = max(t1, u1);
    }
    tau_bits = t2;
  }
  for (int round = 0; round < (clip_rank == 2 ? 0 : clip_rank); ++round) {
    uint32_t mx = 0;
#pragma unroll
    for (int i = 0; i < MAXV; ++i) mx = max(mx, gmax[i]);
    const uint32_t wmx = __reduce_max_sync(0xFFFFFFFFu, mx);
    tau_bits = wmx;
    if (wmx == 0) break;  // all that is left are zeros
    const uint32_t t2 = wmx | (wmx << 16);
    int cnt = 0;
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      if (gmax[i] == wmx) {  // this vector holds the value: count it and find the vector's next maximum
        const uint32_t w[4] = {v[i].x & 0x7FFF7FFFu, v[i].y & 0x7FFF7FFFu, v[i].z & 0x7FFF7FFFu,
                               v[i].w & 0x7FFF7FFFu};
        uint32_t m2 = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          cnt += count_eq2(w[j], t2);
          m2 = __vmaxu2(m2, keep_below2(w[j], t2));
        }
        gmax[i] = fold_max2(m2);
      }
    }
    const int wcnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    if (wcnt >= remaining) break;
    remaining -= wcnt;
  }
  const float tau = __uint_as_float(tau_bits << 16);
  float inv = 0.0f;
  sc = 0.0f;
  if (!(tau < 7.888609052210118e-31f)) {  // 2^-100, as in the absmax form
    sc = __fdiv_rn(tau, qmax);
    inv = __fdiv_rn(qmax, tau);
  }
  const uint32_t tau2 = tau_bits | (tau_bits << 16);
  sum = 0;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) {
      const uint32_t p0 = quant_pair_clipped(v[i].x, tau2, inv), p1 = quant_pair_clipped(v[i].y, tau2, inv);
      const uint32_t p2 = quant_pair_clipped(v[i].z, tau2, inv), p3 = quant_pair_clipped(v[i].w, tau2, inv);
      const uint2 o = make_uint2(__byte_perm(p0, p1, 0x5410), __byte_perm(p2, p3, 0x5410));
      qr.store(idx, o);
      sum = __dp4a(static_cast<int>(o.x), 0x01010101, sum);
      sum = __dp4a(static_cast<int>(o.y), 0x01010101, sum);
    }
  }
}

// Packed unit -> 8 words of 4 int8 (true values, k ascending).
template <int BITS>
__device__ __forceinline__ void expand_unit(const uint32_t (&pk)[BITS], uint32_t (&w)[8]) {
  if constexpr (BITS == 8) {
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = pk[i];
  } else if constexpr (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t lo = pk[i] & 0x0F0F0F0Fu, hi = (pk[i] >> 4) & 0x0F0F0F0Fu;
      w[2 * i] = __vsub4(__byte_perm(lo, hi, 0x5140), 0x08080808u);
      w[2 * i + 1] = __vsub4(__byte_perm(lo, hi, 0x7362), 0x08080808u);
    }
  } else {
    const uint64_t lo64 = (static_cast<uint64_t>(pk[1]) << 32) | pk[0];
    const uint64_t hi64 = (static_cast<uint64_t>(pk[2]) << 32) | pk[1];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int bit = 12 * j;
      const uint32_t x = static_cast<uint32_t>(bit < 32 ? (lo64 >> bit) : (hi64 >> (bit - 32))) & 0xFFFu;
      const uint32_t o = (x & 7u) | ((x & 0x38u) << 5) | ((x & 0x1C0u) << 10) | ((x & 0xE00u) << 15);
      w[j] = __vsub4(o, 0x04040404u);
    }
  }
}

// CTA `block` of an unpack job: one thread per unit of 32 codes (12 or 16 bytes in, 32 bytes out).
__device__ __forceinline__ void unpack_units(const UnpackJob& job, const int block) {
  const int64_t u = static_cast<int64_t>(block) * blockDim.x + threadIdx.x;
  if (u >= job.units) return;
  uint32_t w[8];
  if (job.bits == 4) {
    const uint4 v = reinterpret_cast<const uint4*>(job.packed)[u];
    const uint32_t pk[4] = {v.x, v.y, v.z, v.w};
    expand_unit<4>(pk, w);
  } else {
    const uint32_t* p = job.packed + u * 3;
    const uint32_t pk[3] = {p[0], p[1], p[2]};
    expand_unit<3>(pk, w);
  }
  st_global_v8(reinterpret_cast<uint4*>(job.out) + u * 2, w);  // 32 bytes, read next by the GEMM through L2
}

}  // namespace dp
