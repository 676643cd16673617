// CUDA-core path of the quantized linear for small row counts (adaLN modulation: M = batch).
//
// The whole layer in one launch, bound by the weight bytes (M <= 32: 2..144 int8 ops per weight
// byte). A CTA owns 32 output channels and up to 8 tokens. Eight lanes share one channel: each
// lane fetches its 32-code units of the packed weight row straight into registers, all loads of a
// pass issued back to back and BEFORE the CTA quantizes its tokens (DAQ, Step 3 Eq. "daq", one
// warp per token, codes to shared memory), so the HBM latency of the weights overlaps the
// prologue. The units are then expanded to int8 in registers, contracted against the shared int8
// tokens with dp4a, reduced over the eight lanes by a transpose-reduction (7 shuffles leave lane j
// with token j's sum) and sent through the dequant epilogue.
//
// For K <= 1152 (every adaLN layer) the contraction instead runs on warp-level int8 matrix
// instructions (m16n8k32: 16 channels x 8 tokens per warp), which removes almost all shared-memory
// reads and integer issue slots of the dp4a form and leaves the kernel bound by the weight stream:
// a warp owns 16 channels; lane (g, t) = (lane / 4, lane % 4) fetches the units 4j + t of rows g
// and g + 8, and because a dot product may visit k in any order as long as both operands agree,
// those registers serve directly as the A fragments while the B fragments are the same units of
// token g, read from shared memory (row pitch K + 8 keeps the 64-bit reads conflict-free).
#include <cuda_bf16.h>

#include "daq_device.cuh"

namespace dp {

constexpr int kSimtRows = 8;        // tokens per CTA
constexpr int kSimtWarps = 8;
constexpr int kSimtLanesPerCh = 8;  // lanes sharing one output channel
constexpr int kSimtChPerCta = kSimtWarps * (32 / kSimtLanesPerCh);
constexpr int kSimtSlots = 5;       // units a lane holds per pass (K = 1152: 36 units / 8 lanes)
constexpr int kMmaChPerWarp = 16;   // matrix-instruction form: channels per warp (the M of m16n8k32)
constexpr int kMmaChPerCta = kSimtWarps * kMmaChPerWarp;
constexpr int kMmaMaxK = 1152;
// 128-k steps whose packed units a lane keeps in flight at once (two rows each).
template <int BITS> __host__ __device__ constexpr int mma_batch() { return BITS == 8 ? 3 : (BITS == 4 ? 5 : 9); }

// Packed form of one unit (32 consecutive k of one weight row): BITS words.
template <int BITS>
__device__ __forceinline__ void fetch_unit(const uint32_t* __restrict__ row, int unit, uint32_t (&pk)[BITS]) {
  if constexpr (BITS == 8) {
    const uint4* p = reinterpret_cast<const uint4*>(row) + unit * 2;
    uint4 a, b;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "l"(p));
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p + 1));
    pk[0] = a.x; pk[1] = a.y; pk[2] = a.z; pk[3] = a.w;
    pk[4] = b.x; pk[5] = b.y; pk[6] = b.z; pk[7] = b.w;
  } else if constexpr (BITS == 4) {
    const uint4* p = reinterpret_cast<const uint4*>(row) + unit;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(pk[0]), "=r"(pk[1]), "=r"(pk[2]), "=r"(pk[3]) : "l"(p));
  } else {
    const uint32_t* p = row + unit * 3;
#pragma unroll
    for (int i = 0; i < 3; ++i)
      asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(pk[i]) : "l"(p + i));
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

// This CTA's tokens -> int8 in shared memory, one warp per token (rows `pitch` bytes apart), and
// their scales: DAQ here (Step 3, Eq. "daq"), or a copy when the caller passes quantized tokens.
__device__ __forceinline__ void stage_tokens(const SimtArgs& a, const int64_t m0, const int block_x,
                                             int8_t* sq, const int pitch, float* ssa) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = a.K;
  {
    const int64_t row = m0 + warp;
    uint2* dst = reinterpret_cast<uint2*>(sq + warp * pitch);
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
#pragma unroll 5
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
#pragma unroll 5
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
    if (block_x == 0 && row < a.M) {  // optional taps, written once per token
      if (a.dbg_sa != nullptr && lane == 0) a.dbg_sa[row] = ssa[warp];
      if (a.dbg_q != nullptr) {
        __syncwarp();
        uint2* dq = reinterpret_cast<uint2*>(a.dbg_q + row * a.dbg_ldq);
        for (int i = lane; i < nvec; i += 32) dq[i] = dst[i];
      }
    }
  }
}

template <int BITS>
__device__ __forceinline__ void simt_linear_body(const SimtArgs& a, const int block_x, const int block_y) {
  extern __shared__ __align__(16) uint8_t smem[];
  int8_t* sq = reinterpret_cast<int8_t*>(smem);                       // [kSimtRows][K]
  float* ssa = reinterpret_cast<float*>(smem + kSimtRows * a.K);      // [kSimtRows]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane & (kSimtLanesPerCh - 1);
  const int64_t m0 = static_cast<int64_t>(block_y) * kSimtRows;
  const int K = a.K;
  const int units = K >> 5;
  const int n = block_x * kSimtChPerCta + warp * (32 / kSimtLanesPerCh) + (lane >> 3);
  const bool n_ok = n < a.N;
  const uint32_t* wrow = static_cast<const uint32_t*>(a.qweight) +
                         static_cast<int64_t>(n_ok ? n : 0) * ((K * BITS) >> 5);
  pdl_launch_dependents();
  if (!a.early_w) pdl_wait();

  // ---- first pass of this lane's weight units: in flight across the prologue ----
  uint32_t pk[kSimtSlots][BITS];
#pragma unroll
  for (int i = 0; i < kSimtSlots; ++i) {
    const int u = sub + kSimtLanesPerCh * i;
    if (n_ok && u < units) fetch_unit<BITS>(wrow, u, pk[i]);
  }
  if (a.early_w) pdl_wait();  // the tokens come from the preceding kernel on the stream

  stage_tokens(a, m0, block_x, sq, K, ssa);
  __syncthreads();

  // ---- contraction: passes of kSimtSlots units per lane ----
  int acc[kSimtRows];
#pragma unroll
  for (int m = 0; m < kSimtRows; ++m) acc[m] = 0;
  for (int base = 0; base < units; base += kSimtLanesPerCh * kSimtSlots) {
    if (base != 0) {
#pragma unroll
      for (int i = 0; i < kSimtSlots; ++i) {
        const int u = base + sub + kSimtLanesPerCh * i;
        if (n_ok && u < units) fetch_unit<BITS>(wrow, u, pk[i]);
      }
    }
#pragma unroll
    for (int i = 0; i < kSimtSlots; ++i) {
      const int u = base + sub + kSimtLanesPerCh * i;
      if (n_ok && u < units) {
        uint32_t w[8];
        expand_unit<BITS>(pk[i], w);
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
    }
  }

  // ---- transpose-reduction over the 8 lanes of a channel: lane j ends with token j's sum ----
  {
    const bool hi4 = (sub & 4) != 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int send = hi4 ? acc[i] : acc[i + 4];
      const int keep = hi4 ? acc[i + 4] : acc[i];
      acc[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
    }
    const bool hi2 = (sub & 2) != 0;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int send = hi2 ? acc[i] : acc[i + 2];
      const int keep = hi2 ? acc[i + 2] : acc[i];
      acc[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 2);
    }
    const bool hi1 = (sub & 1) != 0;
    const int send = hi1 ? acc[0] : acc[1];
    const int keep = hi1 ? acc[1] : acc[0];
    acc[0] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 1);
  }
  const int64_t row = m0 + sub;
  if (n_ok && row < a.M) {
    const int mine = acc[0];
    const float t = static_cast<float>(mine);
    const float sc = __fmul_rn(ssa[sub], a.s_w[n]);
    const float b = a.bias != nullptr ? __uint_as_float(static_cast<uint32_t>(a.bias[n]) << 16) : 0.0f;
    const float y = __fmaf_rn(t, sc, b);
    a.y[row * a.ldy + n] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
    if (a.dbg_acc != nullptr) a.dbg_acc[row * a.dbg_ldacc + n] = mine;
  }
}

__device__ __forceinline__ void mma_m16n8k32_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Matrix-instruction form (K <= kMmaMaxK). Fragment roles of m16n8k32: A row = channel (g and g + 8),
// B column = token g, D element (row, column pair 2t, 2t + 1). The instruction's k index of a
// register is immaterial here: lane (g, t) supplies, for step s of its unit, words 2s and 2s + 1 of
// the unit as the (k-low, k-high) registers of BOTH operands, so every k meets its partner once.
template <int BITS>
__device__ __forceinline__ void simt_mma_body(const SimtArgs& a, const int block_x, const int block_y) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int K = a.K, pitch = K + 8;
  int8_t* sq = reinterpret_cast<int8_t*>(smem);                       // [kSimtRows][pitch]
  float* ssa = reinterpret_cast<float*>(smem + kSimtRows * pitch);    // [kSimtRows]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t m0 = static_cast<int64_t>(block_y) * kSimtRows;
  const int n0 = block_x * kMmaChPerCta + warp * kMmaChPerWarp;
  const bool n_ok = n0 < a.N;  // N is a multiple of 16: a warp's channels exist together
  const int64_t wpitch = (K * BITS) >> 5;
  const uint32_t* w_lo = static_cast<const uint32_t*>(a.qweight) + (n_ok ? n0 + g : 0) * wpitch;
  const uint32_t* w_hi = w_lo + (n_ok ? 8 * wpitch : 0);
  const int kj = K >> 7;
  constexpr int BJ = mma_batch<BITS>();
  uint32_t pk[BJ][2][BITS];
  pdl_launch_dependents();
  if (!a.early_w) pdl_wait();
  auto fetch_batch = [&](const int j0) {
#pragma unroll
    for (int i = 0; i < BJ; ++i) {
      if (n_ok && j0 + i < kj) {
        fetch_unit<BITS>(w_lo, 4 * (j0 + i) + t, pk[i][0]);
        fetch_unit<BITS>(w_hi, 4 * (j0 + i) + t, pk[i][1]);
      }
    }
  };
  fetch_batch(0);  // in flight across the prologue
  if (a.early_w) pdl_wait();
  stage_tokens(a, m0, block_x, sq, pitch, ssa);
  __syncthreads();

  int c[4] = {0, 0, 0, 0};
  const int8_t* qrow = sq + g * pitch + t * 32;
  for (int j0 = 0; j0 < kj; j0 += BJ) {
    if (j0 != 0) fetch_batch(j0);
#pragma unroll
    for (int i = 0; i < BJ; ++i) {
      if (n_ok && j0 + i < kj) {
        uint32_t wl[8], wh[8];
        expand_unit<BITS>(pk[i][0], wl);
        expand_unit<BITS>(pk[i][1], wh);
        const uint2* qp = reinterpret_cast<const uint2*>(qrow + (j0 + i) * 128);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const uint2 q = qp[s];
          mma_m16n8k32_s8(c, wl[2 * s], wh[2 * s], wl[2 * s + 1], wh[2 * s + 1], q.x, q.y);
        }
      }
    }
  }

  if (n_ok) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int n = n0 + g + 8 * h;
      const float sw = a.s_w[n];
      const float b = a.bias != nullptr ? __uint_as_float(static_cast<uint32_t>(a.bias[n]) << 16) : 0.0f;
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int tok = 2 * t + e;
        const int64_t row = m0 + tok;
        if (row < a.M) {
          const int mine = c[2 * h + e];
          const float y = __fmaf_rn(static_cast<float>(mine), __fmul_rn(ssa[tok], sw), b);
          a.y[row * a.ldy + n] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
          if (a.dbg_acc != nullptr) a.dbg_acc[row * a.dbg_ldacc + n] = mine;
        }
      }
    }
  }
}

template <int BITS, bool MMA>
__global__ void __launch_bounds__(kSimtWarps * 32)
simt_linear_kernel(SimtArgs a) {
  if constexpr (MMA) simt_mma_body<BITS>(a, blockIdx.x, blockIdx.y);
  else simt_linear_body<BITS>(a, blockIdx.x, blockIdx.y);
}

// Several layers of one shape (M, K, N) in one launch: blockIdx.z picks the layer. Used for the
// adaLN modulation linears of a timestep, which are mutually independent and, one at a time, far
// too small (3..8 MB of weights) to fill the GPU for longer than a launch takes.
// DAQ of every token of a group (one warp per token; grid = (ceil(M / 8), layers)).
__global__ void __launch_bounds__(kSimtWarps * 32)
daq_group_kernel(SimtGroupArgs g) {
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kSimtWarps + warp;
  pdl_wait();
  if (row >= g.M) return;
  const int layer = blockIdx.y;
  const uint16_t* x = static_cast<const uint16_t*>(g.layer[layer].x) + row * g.K;
  const QRow qr(g.q_scratch + static_cast<int64_t>(layer) * g.M * g.K, row, g.K, 0);
  const float sc = daq_row_2pass<false>(x, g.K, qr, lane);
  if (lane == 0) g.sa_scratch[static_cast<int64_t>(layer) * g.M + row] = sc;
}

template <bool MMA>
__global__ void __launch_bounds__(kSimtWarps * 32)
simt_group_kernel(SimtGroupArgs g) {
  SimtArgs a;
  const SimtGroupArgs::Layer& L = g.layer[blockIdx.z];
  a.x = L.x;
  a.ldx = g.K;
  a.s_a_in = nullptr;
  if (g.q_scratch != nullptr) {  // tokens already quantized by daq_group_kernel
    a.x = g.q_scratch + static_cast<int64_t>(blockIdx.z) * g.M * g.K;
    a.s_a_in = g.sa_scratch + static_cast<int64_t>(blockIdx.z) * g.M;
  }
  a.M = g.M;
  a.N = g.N;
  a.K = g.K;
  a.bits = L.bits;
  a.qweight = L.qweight;
  a.s_w = L.s_w;
  a.bias = L.bias;
  a.y = L.y;
  a.ldy = g.N;
  a.dbg_q = nullptr;
  a.dbg_ldq = 0;
  a.dbg_sa = nullptr;
  a.dbg_acc = nullptr;
  a.dbg_ldacc = 0;
  a.early_w = g.early_w;
  if constexpr (MMA) {
    if (L.bits == 8) simt_mma_body<8>(a, blockIdx.x, blockIdx.y);
    else if (L.bits == 4) simt_mma_body<4>(a, blockIdx.x, blockIdx.y);
    else simt_mma_body<3>(a, blockIdx.x, blockIdx.y);
  } else {
    if (L.bits == 8) simt_linear_body<8>(a, blockIdx.x, blockIdx.y);
    else if (L.bits == 4) simt_linear_body<4>(a, blockIdx.x, blockIdx.y);
    else simt_linear_body<3>(a, blockIdx.x, blockIdx.y);
  }
}

static bool simt_use_mma(int32_t K) { return K <= kMmaMaxK; }
static size_t simt_smem_bytes(int32_t K) {
  return static_cast<size_t>(kSimtRows) * (K + 8) + kSimtRows * sizeof(float);
}

size_t simt_max_k() { return 16384; }

size_t simt_group_scratch_bytes(int64_t M, int32_t K, int32_t n_layers) {
  const size_t q = (static_cast<size_t>(n_layers) * M * K + 255) & ~static_cast<size_t>(255);
  return q + ((sizeof(float) * n_layers * M + 255) & ~static_cast<size_t>(255));
}

int launch_simt_group(const SimtGroupArgs& g, cudaStream_t stream, bool pdl) {
  if (g.M == 0 || g.n_layers == 0) return DP_OK;
  if (g.q_scratch != nullptr) {
    const dim3 dgrid(static_cast<unsigned>((g.M + kSimtWarps - 1) / kSimtWarps), static_cast<unsigned>(g.n_layers));
    cudaError_t e = launch(daq_group_kernel, dgrid, dim3(kSimtWarps * 32), 0, stream, pdl, g);
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "grouped DAQ launch failed: %s", cudaGetErrorString(e));
  }
  const size_t smem = simt_smem_bytes(g.K);
  const bool mma = simt_use_mma(g.K);
  const int ch = mma ? kMmaChPerCta : kSimtChPerCta;
  const dim3 grid((g.N + ch - 1) / ch, static_cast<unsigned>((g.M + kSimtRows - 1) / kSimtRows),
                  static_cast<unsigned>(g.n_layers));
  const dim3 block(kSimtWarps * 32);
  void (*kern)(SimtGroupArgs) = mma ? simt_group_kernel<true> : simt_group_kernel<false>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "simt smem attribute: %s", cudaGetErrorString(e));
  }
  SimtGroupArgs args = g;
  if (!pdl) args.early_w = 0;
  if (g.q_scratch != nullptr && pdl) args.early_w = 1;  // the preceding kernel is the group's own DAQ
  cudaError_t e = launch(kern, grid, block, smem, stream, pdl, args);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "grouped simt launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

int launch_simt_linear(const SimtArgs& a, cudaStream_t stream, bool pdl) {
  if (a.M == 0) return DP_OK;
  const size_t smem = simt_smem_bytes(a.K);
  const bool mma = simt_use_mma(a.K);
  const int ch = mma ? kMmaChPerCta : kSimtChPerCta;
  const dim3 grid((a.N + ch - 1) / ch, static_cast<unsigned>((a.M + kSimtRows - 1) / kSimtRows));
  const dim3 block(kSimtWarps * 32);
  void (*kern)(SimtArgs);
  if (mma) kern = a.bits == 8 ? simt_linear_kernel<8, true> : a.bits == 4 ? simt_linear_kernel<4, true>
                                                                          : simt_linear_kernel<3, true>;
  else kern = a.bits == 8 ? simt_linear_kernel<8, false> : a.bits == 4 ? simt_linear_kernel<4, false>
                                                                       : simt_linear_kernel<3, false>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "simt smem attribute: %s", cudaGetErrorString(e));
  }
  SimtArgs args = a;
  if (!pdl) args.early_w = 0;
  cudaError_t e = launch(kern, grid, block, smem, stream, pdl, args);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "simt launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
