// Weight-streaming path of the quantized linear for small row counts (adaLN modulation: M = batch).
//
// The whole layer in one launch, bound by the weight bytes (M <= 32: 2..144 int8 ops per weight
// byte). Form for K > 1152: a CTA owns 32 output channels and up to 8 tokens. Eight lanes share one channel: each
// lane fetches its 32-code units of the packed weight row straight into registers, all loads of a
// pass issued back to back and BEFORE the CTA quantizes its tokens (DAQ, Step 3 Eq. "daq", one
// warp per token, codes to shared memory), so the HBM latency of the weights overlaps the
// prologue. The units are then expanded to int8 in registers, contracted against the shared int8
// tokens with dp4a, reduced over the eight lanes by a transpose-reduction (7 shuffles leave lane j
// with token j's sum) and sent through the dequant epilogue.
//
// For K <= 1152 (every adaLN layer) the contraction instead runs on warp-level int8 matrix
// instructions (m16n8k32 with the tokens as the 16 rows and 8 output channels as the columns), and
// the weights reach the SM as bulk asynchronous copies: eight consecutive weight rows are one
// contiguous run of the packed matrix, which each warp streams through a private ring of
// shared-memory stages (3- and 4-bit: one copy of eight whole rows per stage; 8-bit: one copy per
// row and third of K; completion counted in bytes on the stage's mbarrier), so
// HBM sees a few thousand long sequential streams and the bytes in flight do not depend on
// registers. Lane (g, t) = (lane / 4, lane % 4) reads the units 4j + t of row g from the stage and
// feeds them as B fragments: 8-bit codes as they are; packed 3- and 4-bit codes as UNSIGNED bytes
// that one mask (and at most a short shift) isolates where the field already sits, the power of two
// such a byte carries being common to an accumulator set and shifted out exactly at the end, the
// offset 2^(b-1) leaving as 2^(b-1) times the sum of the token's codes. Because a dot product may
// visit k in any order as long as both operands agree, the A fragments are the same units of tokens
// g and g + 8 from shared memory, staged in the k order the masks produce (row pitch K + 16 keeps
// those 128-bit reads conflict-free).
#include <cuda_bf16.h>

#include <algorithm>
#include <type_traits>

#include "daq_device.cuh"

namespace dp {

constexpr int kSimtRows = 8;        // tokens per CTA
constexpr int kSimtWarps = 8;
constexpr int kSimtLanesPerCh = 8;  // lanes sharing one output channel
constexpr int kSimtChPerCta = kSimtWarps * (32 / kSimtLanesPerCh);
constexpr int kSimtSlots = 5;       // units a lane holds per pass (K = 1152: 36 units / 8 lanes)
// Matrix-instruction form (K <= kMmaMaxK).
constexpr int kMmaMaxK = 1152;
constexpr int kMmaWarps = 8;
constexpr int kMmaRows = 16;          // tokens per CTA (the M of m16n8k32)
constexpr int kMmaCh = 8;             // output channels per block (the N of m16n8k32)
constexpr int kMmaMaxStages = 8;
constexpr int kMmaRingBytes = 9600;   // per warp
// 128-k steps per ring stage. Low-bit rows are short enough for a stage to hold eight whole rows,
// which are contiguous in the packed matrix: one copy per stage. 8-bit rows go in thirds, one copy
// per row, 16 bytes of padding per staged row so that the lanes' reads spread over all banks.
template <int BITS> __host__ __device__ constexpr int mma_chunk_j() { return BITS == 8 ? 3 : 9; }
constexpr int kMmaPitch8 = 3 * 128 + 16;

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

// Order in which a token's codes are laid out in shared memory for the matrix-instruction form. The
// contraction may visit k in any order as long as both operands agree, so the activations take the
// order in which cheap mask operations leave the weight codes of a packed unit:
//   ORDER_NATURAL  k ascending (8-bit weights, and the CUDA-core form);
//   ORDER_NIBBLE   within every 8 codes the even positions first, then the odd ones (4-bit: the low
//                  and the high nibbles of a packed word);
//   ORDER_PERIOD   within every 32 codes, word c (c = 0..7) holds positions c, 8 + c, 16 + c, 24 + c
//                  (3-bit: the fields at the same place of the four 3-byte periods of a packed unit).
enum { ORDER_NATURAL = 0, ORDER_NIBBLE = 1, ORDER_PERIOD = 2 };

template <int ORDER>
__device__ __forceinline__ void store_codes(int8_t* row, const int i, const uint2 v) {
  if constexpr (ORDER == ORDER_NATURAL) {
    reinterpret_cast<uint2*>(row)[i] = v;
  } else if constexpr (ORDER == ORDER_NIBBLE) {
    reinterpret_cast<uint2*>(row)[i] = make_uint2(__byte_perm(v.x, v.y, 0x6420), __byte_perm(v.x, v.y, 0x7531));
  } else {  // codes 8p .. 8p + 7 of a unit go to byte p of its eight words
    uint8_t* unit = reinterpret_cast<uint8_t*>(row) + (i >> 2) * 32 + (i & 3);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      unit[4 * c] = static_cast<uint8_t>(v.x >> (8 * c));
      unit[4 * (c + 4)] = static_cast<uint8_t>(v.y >> (8 * c));
    }
  }
}

// Token `warp` of this CTA -> int8 in shared memory, by one warp (rows `pitch` bytes apart), its
// scale and (srs != nullptr) the sum of its codes: DAQ here (Step 3, Eq. "daq"), or a copy when the
// caller passes quantized tokens.
template <int ORDER = ORDER_NATURAL>
__device__ __forceinline__ void stage_tokens(const SimtArgs& a, const int64_t m0, const int block_x,
                                             int8_t* sq, const int pitch, float* ssa, const int warp,
                                             int* srs = nullptr) {
  const int lane = threadIdx.x & 31;
  const int K = a.K;
  {
    const int64_t row = m0 + warp;
    int8_t* dst = sq + warp * pitch;
    const int nvec = K >> 3;
    const bool tap_q = block_x == 0 && row < a.M && a.dbg_q != nullptr;  // optional taps, written once per token
    uint2* dq = tap_q ? reinterpret_cast<uint2*>(a.dbg_q + row * a.dbg_ldq) : nullptr;
    int sum = 0;
    if (row >= a.M) {
      for (int i = lane; i < nvec; i += 32) reinterpret_cast<uint2*>(dst)[i] = make_uint2(0, 0);
      if (lane == 0) ssa[warp] = 0.0f;
    } else if (a.s_a_in != nullptr) {
      const uint2* src = reinterpret_cast<const uint2*>(static_cast<const int8_t*>(a.x) + row * a.ldx);
      for (int i = lane; i < nvec; i += 32) {
        const uint2 v = src[i];
        sum = __dp4a(static_cast<int>(v.x), 0x01010101, __dp4a(static_cast<int>(v.y), 0x01010101, sum));
        store_codes<ORDER>(dst, i, v);
        if (tap_q) dq[i] = v;
      }
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
        const uint2 w = make_uint2(b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24),
                                   b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24));
        sum = __dp4a(static_cast<int>(w.x), 0x01010101, __dp4a(static_cast<int>(w.y), 0x01010101, sum));
        store_codes<ORDER>(dst, i, w);
        if (tap_q) dq[i] = w;
      }
      if (lane == 0) ssa[warp] = sc;
    }
    if (srs != nullptr) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
      if (lane == 0) srs[warp] = sum;
    }
    if (block_x == 0 && row < a.M && a.dbg_sa != nullptr && lane == 0) a.dbg_sa[row] = ssa[warp];
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

  stage_tokens(a, m0, block_x, sq, K, ssa, warp);
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

// The same with unsigned 8-bit B (weight) operands.
__device__ __forceinline__ void mma_m16n8k32_s8u8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Packed unit `unit` of a staged weight row.
template <int BITS>
__device__ __forceinline__ void stage_unit(const uint8_t* row, int unit, uint32_t (&pk)[BITS]) {
  if constexpr (BITS == 8) {
    const uint4 u = reinterpret_cast<const uint4*>(row)[unit * 2], v = reinterpret_cast<const uint4*>(row)[unit * 2 + 1];
    pk[0] = u.x; pk[1] = u.y; pk[2] = u.z; pk[3] = u.w;
    pk[4] = v.x; pk[5] = v.y; pk[6] = v.z; pk[7] = v.w;
  } else if constexpr (BITS == 4) {
    const uint4 u = reinterpret_cast<const uint4*>(row)[unit];
    pk[0] = u.x; pk[1] = u.y; pk[2] = u.z; pk[3] = u.w;
  } else {
    const uint32_t* p = reinterpret_cast<const uint32_t*>(row) + unit * 3;
    pk[0] = p[0]; pk[1] = p[1]; pk[2] = p[2];
  }
}

// Bounded wait without the abort shortcut: lets copies already issued land before a warp that gave
// up leaves its ring.
__device__ __forceinline__ void mbar_drain(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > (1ll << 26)) return;
  }
}

// Matrix-instruction form (K <= kMmaMaxK). Fragment roles of m16n8k32: A row = token (g and g + 8),
// B column = channel g of the block, D element (token g or g + 8, channels 2t and 2t + 1). The
// instruction's k index of a register is immaterial here: lane (g, t) supplies, for step s of its
// unit, words 2s and 2s + 1 of the unit as the (k-low, k-high) registers of BOTH operands, so every
// k meets its partner exactly once.
template <int BITS>
__device__ __forceinline__ void simt_mma_body(const SimtArgs& a, const int block_x, const int block_y,
                                              const int grid_x) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int K = a.K, qpitch = K + 16;
  int8_t* sq = reinterpret_cast<int8_t*>(smem);                             // [kMmaRows][qpitch]
  float* ssa = reinterpret_cast<float*>(smem + kMmaRows * qpitch);          // [kMmaRows]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ssa + kMmaRows);
  int* srs = reinterpret_cast<int*>(ssa + kMmaRows + 4);                    // [kMmaRows] sums of the tokens' codes
  uint64_t* bars = reinterpret_cast<uint64_t*>(srs + kMmaRows);             // [kMmaWarps][kMmaMaxStages]
  uint8_t* ring = reinterpret_cast<uint8_t*>(bars + kMmaWarps * kMmaMaxStages);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t m0 = static_cast<int64_t>(block_y) * kMmaRows;
  const bool two = a.M - m0 > 8;  // tokens g + 8 exist
  constexpr int CJ = mma_chunk_j<BITS>();
  const int64_t rowbytes = (static_cast<int64_t>(K) * BITS) >> 3;
  const int pitch = BITS == 8 ? kMmaPitch8 : static_cast<int>(rowbytes);  // of a staged row
  const int stage = kMmaCh * pitch;
  const int S = min(kMmaMaxStages, kMmaRingBytes / stage);
  uint64_t* bar = bars + warp * kMmaMaxStages;
  uint8_t* myring = ring + warp * kMmaRingBytes;
  const uint8_t* wbase = static_cast<const uint8_t*>(a.qweight);
  const int kj = K >> 7;
  const int nc = (kj + CJ - 1) / CJ;  // 1 for the low-bit forms (K <= kMmaMaxK)
  // 8-channel blocks of this warp: blk0, blk0 + stride, ... The grid is sized to one wave, so a warp
  // streams several blocks back to back.
  const int nblocks = a.N / kMmaCh;
  const int stride = grid_x * kMmaWarps;
  const int blk0 = block_x * kMmaWarps + warp;
  const int total = blk0 < nblocks ? ((nblocks - blk0 + stride - 1) / stride) * nc : 0;

  if (threadIdx.x == 0) *abort_flag = 0;
  if (lane == 0) {
    for (int s = 0; s < S; ++s) mbar_init(&bar[s], 1);
    fence_barrier_init();
  }
  __syncwarp();
  pdl_launch_dependents();
  if (!a.early_w) pdl_wait();

  // Producer side of the ring (lane 0): item = (block, chunk); the copy of item i lands in stage i % S.
  int f_it = 0, f_c = 0, f_blk = blk0, f_s = 0;
  auto issue = [&]() {
    if (f_it < total) {
      const uint8_t* src = wbase + static_cast<int64_t>(f_blk) * kMmaCh * rowbytes;
      uint8_t* dst = myring + f_s * stage;
      if constexpr (BITS < 8) {
        if (lane == 0) {
          const uint32_t bytes = static_cast<uint32_t>(kMmaCh * rowbytes);
          mbar_arrive_expect_tx(&bar[f_s], bytes);
          bulk_load_1d(dst, src, bytes, &bar[f_s]);
        }
      } else {
        // one copy per row: issued by eight lanes at once (a bulk copy costs its issuing thread
        // 115-280 cycles; in sequence that was the longest phase of an 8-bit stage)
        const uint32_t bytes = static_cast<uint32_t>(min(CJ, kj - f_c * CJ) * 128);
        if (lane == 0) mbar_arrive_expect_tx(&bar[f_s], kMmaCh * bytes);
        __syncwarp();
        if (lane < kMmaCh)
          bulk_load_1d(dst + lane * kMmaPitch8, src + f_c * (CJ * 128) + lane * rowbytes, bytes, &bar[f_s]);
      }
      ++f_it;
      if (++f_s == S) f_s = 0;
      if (++f_c == nc) { f_c = 0; f_blk += stride; }
    }
  };
#pragma unroll 1
  for (int s = 0; s < S; ++s) issue();  // in flight across the prologue
  if (a.early_w) pdl_wait();
  // Scale and bias of channels 2t, 2t + 1: of the current block, and fetched one block ahead for the
  // next (a load issued at the top of the block it is needed in came back, under a saturated memory
  // system, a couple of thousand cycles later, and its first use stalled the warp for that long).
  float sw[2] = {0.0f, 0.0f}, bs[2] = {0.0f, 0.0f};
  float nsw[2] = {0.0f, 0.0f};
  uint32_t nbs[2] = {0u, 0u};
  auto fetch_scales = [&](const int blk) {
    if (blk < nblocks) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int n = blk * kMmaCh + 2 * t + e;
        nsw[e] = a.s_w[n];
        nbs[e] = a.bias != nullptr ? static_cast<uint32_t>(a.bias[n]) : 0u;
      }
    }
  };
  auto take_scales = [&]() {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      sw[e] = nsw[e];
      bs[e] = __uint_as_float(nbs[e] << 16);
    }
  };
  constexpr int ORDER = BITS == 4 ? ORDER_NIBBLE : BITS == 3 ? ORDER_PERIOD : ORDER_NATURAL;
  fetch_scales(blk0);  // of the first block: back by the time the tokens are staged
  for (int r = warp; r < (two ? kMmaRows : kMmaRows / 2); r += kMmaWarps)
    stage_tokens<ORDER>(a, m0, block_x, sq, qpitch, ssa, r, srs);
  __syncthreads();

  // One accumulator set per matrix instruction of a unit: consecutive instructions never wait on each
  // other's results. For packed weights the sets also differ in the power of two their operands
  // carry (see unit_step).
  constexpr int NC = 4;
  int c[NC][4];
#pragma unroll
  for (int i = 0; i < NC; ++i) c[i][0] = c[i][1] = c[i][2] = c[i][3] = 0;
  int c_c = 0, c_blk = blk0, st = 0;
  uint32_t ph = 0;
  const int8_t* qrow = sq + g * qpitch + t * 32;
  auto epilogue = [&]() {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int n = c_blk * kMmaCh + 2 * t + e;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int tok = g + 8 * h;
        const int64_t row = m0 + tok;
        if (row < a.M) {
          const int i = 2 * h + e;
          // Packed weights enter as unsigned fields u = w + 2^(BITS-1), each set carrying its power of
          // two (the shifts are exact), so the sum of the tokens' codes comes off at the end.
          int mine;
          if constexpr (BITS == 8) mine = c[0][i] + c[1][i] + c[2][i] + c[3][i];
          else if constexpr (BITS == 4) mine = c[0][i] + c[1][i] + ((c[2][i] + c[3][i]) >> 4) - 8 * srs[tok];
          else mine = c[0][i] + c[1][i] + (c[2][i] >> 2) + (c[3][i] >> 4) - 4 * srs[tok];
          const float y = __fmaf_rn(static_cast<float>(mine), __fmul_rn(ssa[tok], sw[e]), bs[e]);
          a.y[row * a.ldy + n] = __bfloat16_as_ushort(__float2bfloat16_rn(y));
          if (a.dbg_acc != nullptr) a.dbg_acc[row * a.dbg_ldacc + n] = mine;
        }
      }
    }
  };
  // One unit (32 codes of this lane's channel) of the staged chunk against tokens g (and g + 8 when
  // TWO). qu: the unit's 32 activation codes of token g in the k order of this bit width.
  auto unit_step = [&](const uint8_t* srow, const int8_t* qu, const int u, auto two_tag) {
    constexpr bool TWO = decltype(two_tag)::value;
    const uint4 l0 = *reinterpret_cast<const uint4*>(qu), l1 = *reinterpret_cast<const uint4*>(qu + 16);
    uint4 h0 = make_uint4(0u, 0u, 0u, 0u), h1 = h0;
    if constexpr (TWO) {
      h0 = *reinterpret_cast<const uint4*>(qu + 8 * qpitch);
      h1 = *reinterpret_cast<const uint4*>(qu + 8 * qpitch + 16);
    }
    uint32_t pk[BITS];
    stage_unit<BITS>(srow, u, pk);
    if constexpr (BITS == 8) {
      mma_m16n8k32_s8(c[0], l0.x, h0.x, l0.y, h0.y, pk[0], pk[1]);
      mma_m16n8k32_s8(c[1], l0.z, h0.z, l0.w, h0.w, pk[2], pk[3]);
      mma_m16n8k32_s8(c[2], l1.x, h1.x, l1.y, h1.y, pk[4], pk[5]);
      mma_m16n8k32_s8(c[3], l1.z, h1.z, l1.w, h1.w, pk[6], pk[7]);
    } else if constexpr (BITS == 4) {
      // A packed word's low nibbles are its even codes, its high nibbles its odd codes times 16: one
      // mask each, no shifts. Activation words (ORDER_NIBBLE): even, odd codes of word 0, of word 1, ...
      constexpr uint32_t LO = 0x0F0F0F0Fu, HI = 0xF0F0F0F0u;
      mma_m16n8k32_s8u8(c[0], l0.x, h0.x, l0.z, h0.z, pk[0] & LO, pk[1] & LO);
      mma_m16n8k32_s8u8(c[1], l1.x, h1.x, l1.z, h1.z, pk[2] & LO, pk[3] & LO);
      mma_m16n8k32_s8u8(c[2], l0.y, h0.y, l0.w, h0.w, pk[0] & HI, pk[1] & HI);
      mma_m16n8k32_s8u8(c[3], l1.y, h1.y, l1.w, h1.w, pk[2] & HI, pk[3] & HI);
    } else {
      // The 96-bit unit is four periods of three bytes, eight codes each. r0, r1, r2 collect the
      // periods' first, second, third bytes; then the field of code class j (codes j, 8 + j, 16 + j,
      // 24 + j: activation word j under ORDER_PERIOD) sits at the same bits of every byte:
      //   r0: class 0 bits 0-2, class 1 bits 3-5, class 2 (low two bits) bits 6-7
      //   r1: class 2 (high bit) bit 0, class 3 bits 1-3, class 4 bits 4-6, class 5 (low bit) bit 7
      //   r2: class 5 (high two bits) bits 0-1, class 6 bits 2-4, class 7 bits 5-7
      // Masked (and moved by a few bits where that makes two fields carry the same power of two),
      // each field is an unsigned operand byte worth its true value times 1, 4 or 16; the two parts of
      // the straddling classes 2 and 5 are put together first. The contraction is bound by the rate of
      // the matrix instructions, so the few extra logic operations that save a fifth instruction pay.
      const uint32_t x0 = __byte_perm(pk[0], pk[1], 0x0630), x1 = __byte_perm(pk[0], pk[1], 0x0741),
                     x2 = __byte_perm(pk[0], pk[1], 0x0052);
      const uint32_t r0 = __byte_perm(x0, pk[2], 0x5210), r1 = __byte_perm(x1, pk[2], 0x6210),
                     r2 = __byte_perm(x2, pk[2], 0x7410);
      const uint32_t f2 = ((r0 >> 6) & 0x03030303u) | ((r1 & 0x01010101u) << 2);
      const uint32_t f5 = ((r1 >> 7) & 0x01010101u) | ((r2 & 0x03030303u) << 1);
      // times 1: class 0 | class 2;  class 5 | class 7 (moved down)
      mma_m16n8k32_s8u8(c[0], l0.x, h0.x, l0.z, h0.z, r0 & 0x07070707u, f2);
      mma_m16n8k32_s8u8(c[1], l1.y, h1.y, l1.w, h1.w, f5, (r2 >> 5) & 0x07070707u);
      // times 4: class 3 (moved up one bit) | class 6
      mma_m16n8k32_s8u8(c[2], l0.w, h0.w, l1.z, h1.z, (r1 & 0x0E0E0E0Eu) << 1, r2 & 0x1C1C1C1Cu);
      // times 16: class 1 (moved up one bit) | class 4
      mma_m16n8k32_s8u8(c[3], l0.y, h0.y, l1.x, h1.x, (r0 & 0x38383838u) << 1, r1 & 0x70707070u);
    }
  };
  int it = 0;
  for (; it < total; ++it) {
    if (c_c == 0) {
      take_scales();
      fetch_scales(c_blk + stride);
    }
    if (!mbar_wait(&bar[st], ph, abort_flag)) break;
    const int nj = min(CJ, kj - c_c * CJ);
    const uint8_t* srow = myring + st * stage + g * pitch;
    const int8_t* qc = qrow + c_c * (CJ * 128);
    if (nj == CJ && !two) {  // the common case, free of per-unit tests
#pragma unroll
      for (int jj = 0; jj < CJ; ++jj) unit_step(srow, qc + jj * 128, 4 * jj + t, std::false_type{});
    } else if (two) {
#pragma unroll
      for (int jj = 0; jj < CJ; ++jj)
        if (jj < nj) unit_step(srow, qc + jj * 128, 4 * jj + t, std::true_type{});
    } else {
#pragma unroll
      for (int jj = 0; jj < CJ; ++jj)
        if (jj < nj) unit_step(srow, qc + jj * 128, 4 * jj + t, std::false_type{});
    }
    __syncwarp();  // every lane has consumed the stage: refill it
    issue();
    if (++c_c == nc) {
      epilogue();
#pragma unroll
      for (int i = 0; i < NC; ++i) c[i][0] = c[i][1] = c[i][2] = c[i][3] = 0;
      c_c = 0;
      c_blk += stride;
    }
    if (++st == S) { st = 0; ph ^= 1u; }
  }
  // A warp that gave up lets the copies it still has in flight land before the CTA may exit.
  for (; it < f_it; ++it) {
    mbar_drain(&bar[st], ph);
    if (++st == S) { st = 0; ph ^= 1u; }
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && a.status != nullptr) atomicExch(a.status, DP_ERR_TIMEOUT);
}

template <int BITS, bool MMA>
__global__ void __launch_bounds__(kSimtWarps * 32, MMA ? 2 : 0)
simt_linear_kernel(SimtArgs a) {
  if constexpr (MMA) simt_mma_body<BITS>(a, blockIdx.x, blockIdx.y, gridDim.x);
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

// The same under a DAQ policy (percentile clip, a-bit codes): rows of up to 1280 elements in registers.
__global__ void __launch_bounds__(kSimtWarps * 32)
daq_group_robust_kernel(SimtGroupArgs g) {
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kSimtWarps + warp;
  pdl_wait();
  if (row >= g.M) return;
  const int layer = blockIdx.y;
  const uint16_t* x = static_cast<const uint16_t*>(g.layer[layer].x) + row * g.K;
  const QRow qr(g.q_scratch + static_cast<int64_t>(layer) * g.M * g.K, row, g.K, 0);
  float sc;
  int sum;
  robust_row<5>(x, g.K, lane, g.daq_rank, static_cast<float>((1 << (g.daq_bits - 1)) - 1), qr, sc, sum);
  if (lane == 0) g.sa_scratch[static_cast<int64_t>(layer) * g.M + row] = sc;
}

template <bool MMA>
__global__ void __launch_bounds__(kSimtWarps * 32, MMA ? 2 : 0)
simt_group_kernel(SimtGroupArgs g) {
  SimtArgs a;
  int layer = blockIdx.z, block_x = blockIdx.x, grid_x = gridDim.x;
  if constexpr (MMA) {  // grid.x enumerates (layer, CTA of the layer)
    layer = 0;
    while (static_cast<int>(blockIdx.x) >= g.cta_begin[layer + 1]) ++layer;
    block_x = blockIdx.x - g.cta_begin[layer];
    grid_x = g.cta_begin[layer + 1] - g.cta_begin[layer];
  }
  const SimtGroupArgs::Layer& L = g.layer[layer];
  a.x = L.x;
  a.ldx = g.K;
  a.s_a_in = nullptr;
  if (g.q_scratch != nullptr) {  // tokens already quantized by daq_group_kernel
    a.x = g.q_scratch + static_cast<int64_t>(layer) * g.M * g.K;
    a.s_a_in = g.sa_scratch + static_cast<int64_t>(layer) * g.M;
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
  a.status = g.status;
  if constexpr (MMA) {
    if (L.bits == 8) simt_mma_body<8>(a, block_x, blockIdx.y, grid_x);
    else if (L.bits == 4) simt_mma_body<4>(a, block_x, blockIdx.y, grid_x);
    else simt_mma_body<3>(a, block_x, blockIdx.y, grid_x);
  } else {
    if (L.bits == 8) simt_linear_body<8>(a, blockIdx.x, blockIdx.y);
    else if (L.bits == 4) simt_linear_body<4>(a, blockIdx.x, blockIdx.y);
    else simt_linear_body<3>(a, blockIdx.x, blockIdx.y);
  }
}

static bool simt_use_mma(int32_t K) { return K <= kMmaMaxK; }
static size_t simt_smem_bytes(int32_t K) {
  if (!simt_use_mma(K)) return static_cast<size_t>(kSimtRows) * K + kSimtRows * sizeof(float);
  return static_cast<size_t>(kMmaRows) * (K + 16) + kMmaRows * sizeof(float) + 16 + kMmaRows * sizeof(int) +
         sizeof(uint64_t) * kMmaWarps * kMmaMaxStages + static_cast<size_t>(kMmaWarps) * kMmaRingBytes;
}

// grid.x of the matrix-instruction form: all CTAs of the launch resident at once (one wave), each
// warp walking its strided share of the 8-channel blocks.
template <typename Kern>
static int mma_grid_x(Kern kern, size_t smem, int32_t N, int64_t other_ctas) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kMmaWarps * 32, smem) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  const int64_t slots = static_cast<int64_t>(num_sms()) * per_sm;
  const int64_t full = (N / kMmaCh + kMmaWarps - 1) / kMmaWarps;
  return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(full, slots / std::max<int64_t>(1, other_ctas))));
}

static_assert(kMmaWarps == kSimtWarps, "both forms launch kSimtWarps warps");

size_t simt_max_k() { return 16384; }

size_t simt_group_scratch_bytes(int64_t M, int32_t K, int32_t n_layers) {
  const size_t q = (static_cast<size_t>(n_layers) * M * K + 255) & ~static_cast<size_t>(255);
  return q + ((sizeof(float) * n_layers * M + 255) & ~static_cast<size_t>(255));
}

int launch_simt_group(const SimtGroupArgs& g, cudaStream_t stream, bool pdl) {
  if (g.M == 0 || g.n_layers == 0) return DP_OK;
  if (g.q_scratch != nullptr) {
    const dim3 dgrid(static_cast<unsigned>((g.M + kSimtWarps - 1) / kSimtWarps), static_cast<unsigned>(g.n_layers));
    const bool robust = g.daq_rank > 1 || g.daq_bits < 8;
    if (robust && g.K > 1280) return fail(DP_ERR_SHAPE, "grouped DAQ policy: K=%d above 1280", g.K);
    cudaError_t e = robust ? launch(daq_group_robust_kernel, dgrid, dim3(kSimtWarps * 32), 0, stream, pdl, g)
                           : launch(daq_group_kernel, dgrid, dim3(kSimtWarps * 32), 0, stream, pdl, g);
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "grouped DAQ launch failed: %s", cudaGetErrorString(e));
  }
  const size_t smem = simt_smem_bytes(g.K);
  const bool mma = simt_use_mma(g.K);
  const int rows = mma ? kMmaRows : kSimtRows;
  const int64_t m_groups = (g.M + rows - 1) / rows;
  dim3 grid((g.N + kSimtChPerCta - 1) / kSimtChPerCta, static_cast<unsigned>(m_groups),
            static_cast<unsigned>(g.n_layers));
  const dim3 block(kSimtWarps * 32);
  void (*kern)(SimtGroupArgs) = mma ? simt_group_kernel<true> : simt_group_kernel<false>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "simt smem attribute: %s", cudaGetErrorString(e));
  }
  SimtGroupArgs args = g;
  if (mma) {
    // One wave: the resident-CTA slots are shared out in proportion to the time a CTA of each
    // bit-width needs per channel block (measured: the 8-bit form is bound by its copies, the 3-bit
    // form by the expansion arithmetic), every layer getting at least one CTA.
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kMmaWarps * 32, smem) != cudaSuccess || per_sm < 1)
      per_sm = 1;
    const int64_t slots = std::max<int64_t>(g.n_layers, static_cast<int64_t>(num_sms()) * per_sm / m_groups);
    const int full = (g.N / kMmaCh + kMmaWarps - 1) / kMmaWarps;
    double cost[kSimtGroupMax], total = 0.0;
    for (int l = 0; l < g.n_layers; ++l) {
      cost[l] = g.layer[l].bits == 8 ? 1.75 : g.layer[l].bits == 4 ? 1.0 : 1.1;
      total += cost[l];
    }
    int begin = 0;
    double acc = 0.0;
    for (int l = 0; l < g.n_layers; ++l) {  // cumulative rounding: the counts sum to `slots`
      args.cta_begin[l] = begin;
      acc += cost[l];
      const int end = static_cast<int>(acc / total * static_cast<double>(slots) + 0.5);
      begin = std::min(begin + full, std::max(begin + 1, end));
    }
    args.cta_begin[g.n_layers] = begin;
    grid = dim3(static_cast<unsigned>(begin), static_cast<unsigned>(m_groups), 1);
  }
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
  const int rows = mma ? kMmaRows : kSimtRows;
  const int64_t m_groups = (a.M + rows - 1) / rows;
  dim3 grid((a.N + kSimtChPerCta - 1) / kSimtChPerCta, static_cast<unsigned>(m_groups));
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
  if (mma) grid.x = mma_grid_x(kern, smem, a.N, m_groups);
  SimtArgs args = a;
  if (!pdl) args.early_w = 0;
  cudaError_t e = launch(kern, grid, block, smem, stream, pdl, args);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "simt launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
