// Device-side pieces shared by the tensor-core GEMM kernels of libdiffpro: tile constants, kernel
// parameters, the in-shared-memory expansion of packed 3/4-bit weight tiles, and the dequant
// epilogue of one warp (tcgen05.ld -> fp32 sequence -> bf16 -> 32-byte stores, one token per thread).
#pragma once

#include <cuda_bf16.h>

#include "daq_device.cuh"

namespace dp {

constexpr int BM = 128;
constexpr int BK = 128;  // int8 elements = bytes = one 128-byte swizzle row
constexpr int kEpiWarp0 = 2, kEpiWarps = 8, kUnpackWarp0 = kEpiWarp0 + kEpiWarps, kUnpackWarps = 8;
constexpr int kUnpackThreads = kUnpackWarps * 32;
__host__ __device__ constexpr int gemm_threads(int bits) {
  return (kUnpackWarp0 + (bits == 8 ? 0 : kUnpackWarps)) * 32;
}
constexpr int kSmemBudget = 200 * 1024;
constexpr int kPStages = 3;

// bn below is the number of weight rows ONE CTA holds (BN for CG = 1, BN / 2 for a pair).
__host__ __device__ constexpr int p_stage_bytes(int bn, int bits) {
  return bits == 8 ? 0 : bn * (BK * bits / 8);
}
__host__ __device__ constexpr int ab_stage_bytes(int bn) { return BM * BK + bn * BK; }
__host__ __device__ constexpr int num_stages(int bn, int bits) {
  int n = (kSmemBudget - kPStages * p_stage_bytes(bn, bits)) / ab_stage_bytes(bn);
  return n > 8 ? 8 : n;
}
__host__ __device__ constexpr int tmem_cols(int bn) { return bn <= 64 ? 128 : bn <= 128 ? 256 : 512; }

struct GemmParams {
  const float* s_a;
  const float* s_w;
  const uint16_t* bias;
  uint16_t* y;
  int64_t ldy;
  int32_t* dbg_acc;
  int64_t dbg_ldacc;
  // Residual taken into the epilogue (res != nullptr): y = bf16(gate ? fma(gate, lin, res) : lin + res)
  // in fp32, lin the value otherwise rounded to bf16. res [M][ldr] bf16 (may be y itself); gate
  // [ceil(M / rows_per_gate)][N] bf16 or nullptr.
  const uint16_t* res;
  int64_t ldr;
  const uint16_t* gate;
  int64_t rows_per_gate;
  int64_t M;
  int32_t N, K;
  int32_t m_tiles, n_tiles;  // m_tiles counts row tiles of 128 * CG tokens
  // In-kernel DAQ (x != nullptr): the kernel quantizes the bf16 activations itself, into the tiled
  // scratch q_out / s_a_out that tmap_a and s_a refer to, and its CTAs tell each other through
  // sync[] (one counter per 128-token tile, then one exit counter; all zero between kernels) which
  // tiles are complete.
  const uint16_t* x;
  int64_t ldx;
  int8_t* q_out;
  float* s_a_out;
  int32_t* sync;
  int32_t sync_tiles;
  int32_t a_tiled;  // activations are stored as contiguous 128 x 128 tiles
  int32_t early_w;  // weights may be fetched before the preceding kernel on the stream has finished
  int32_t* status;
  // Two ranges a later launch will read soon (a plan's next layer's packed weights and its bf16 input):
  // each CTA sends its slices on the way into L2 while this kernel, which leaves HBM mostly idle at a
  // few thousand tokens, runs. Hints only (L2 is the point of coherence: a range rewritten after the
  // hint is simply current when it is read); nullptr: none.
  const uint8_t* pf[2] = {nullptr, nullptr};
  uint32_t pf_bytes[2] = {0, 0}, pf_slice[2] = {0, 0};
  int32_t dbg_skip_kb = -1;  // test hook (dp_debug_skip_stage_load): k-block whose loads are left out, or -1
};

// TMA coordinates of the activation tile (token row m_row, a multiple of 128; k block kb).
__device__ __forceinline__ void a_tile_coords(const GemmParams& p, int m_row, int kb, int& c0, int& c1) {
  if (p.a_tiled) {
    c0 = 0;
    c1 = ((m_row >> 7) * (p.K / BK) + kb) * BM;
  } else {
    c0 = kb * BK;
    c1 = m_row;
  }
}

// ---- in-kernel DAQ -------------------------------------------------------------------------------
// Every CTA of the grid quantizes an equal share of the tokens (its 8 epilogue warps, one token per
// warp at a time), publishes each finished token on the counter of its 128-token tile, and only
// then turns to its GEMM tiles; the TMA producer of a tile first waits for that tile's counter.
template <bool EO>
__device__ __forceinline__ void daq_phase(const GemmParams& p, int epi_warp, int lane) {
  const int64_t per_cta = (p.M + gridDim.x - 1) / gridDim.x;
  const int64_t r0 = static_cast<int64_t>(blockIdx.x) * per_cta;
  const int64_t r1 = r0 + per_cta < p.M ? r0 + per_cta : p.M;
  const int kb = p.K / BK;
  for (int64_t row = r0 + epi_warp; row < r1; row += 2 * kEpiWarps) {  // two tokens per round
    const int64_t row_b = row + kEpiWarps;
    const bool has_b = row_b < r1;
    const QRow qa(p.q_out, row, 0, kb), qb(p.q_out, has_b ? row_b : row, 0, kb);
    float sc_a, sc_b;
    daq_two_rows_2pass<EO>(p.x + row * p.ldx, p.x + row_b * p.ldx, has_b, p.K, qa, qb, lane, sc_a, sc_b);
    if (lane == 0) {
      p.s_a_out[row] = sc_a;
      if (has_b) p.s_a_out[row_b] = sc_b;
    }
    __syncwarp();
    if (lane == 0) {
      __threadfence();  // the tokens' codes and scales are visible device-wide before they are counted
      if (has_b && (row_b >> 7) == (row >> 7)) {
        atomicAdd(p.sync + (row >> 7), 2);
      } else {
        atomicAdd(p.sync + (row >> 7), 1);
        if (has_b) atomicAdd(p.sync + (row_b >> 7), 1);
      }
    }
  }
}
// One thread: until every token of 128-token tile `t` has been quantized (bounded).
__device__ __forceinline__ bool wait_tile_quantized(const GemmParams& p, int t, volatile int* abort_flag) {
  const int64_t left = p.M - static_cast<int64_t>(t) * BM;
  const int expect = left >= BM ? BM : static_cast<int>(left);
  if (expect <= 0) return true;  // a tile wholly past M: the loads read the fill value
  const long long t0 = clock64();
  uint32_t polls = 0;
  while (ld_acquire_gpu(p.sync + t) < expect) {
    if ((++polls & 15u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitBudgetCycles) {
        *abort_flag = 1;
        return false;
      }
    }
  }
  fence_proxy_async_all();  // the codes were written with ordinary stores and are read by TMA next
  return true;
}
// Last thing a CTA does (one thread, after all its roles have finished): count itself out; the last
// CTA of the grid returns every counter to zero for the next kernel.
__device__ __forceinline__ void daq_sync_exit(const GemmParams& p) {
  __threadfence();
  if (atomicAdd(p.sync + p.sync_tiles, 1) == static_cast<int>(gridDim.x) - 1) {
    for (int i = 0; i <= p.sync_tiles; ++i) p.sync[i] = 0;
    __threadfence();
  }
}

struct Ring {  // stage index + phase bit of a circular buffer
  int s = 0;
  uint32_t ph = 0;
  __device__ __forceinline__ void next(int n) {
    if (++s == n) {
      s = 0;
      ph ^= 1u;
    }
  }
};

// ---- in-smem weight expansion ------------------------------------------------------------------
// 4-bit: tile P is [BN][64 bytes]; each thread expands 8 bytes (16 codes) into one 16-byte chunk of
// the operand tile B = [BN][128 bytes], chunk position XOR-swizzled by (row & 7).
template <int BN, bool PERM>
__device__ __forceinline__ void unpack4_tile(const uint8_t* P, uint8_t* B, int tid) {
#pragma unroll
  for (int i = 0; i < (BN * 8 + kUnpackThreads - 1) / kUnpackThreads; ++i) {
    const int idx = tid + i * kUnpackThreads;
    if (BN * 8 % kUnpackThreads != 0 && idx >= BN * 8) break;
    const int row = idx >> 3, kc = idx & 7;
    const uint2 in = *reinterpret_cast<const uint2*>(P + row * 64 + kc * 8);
    uint4 o;
    const uint32_t lo0 = ((in.x << 4) & 0xF0F0F0F0u) ^ 0x80808080u;  // even fields
    const uint32_t hi0 = (in.x & 0xF0F0F0F0u) ^ 0x80808080u;         // odd fields
    const uint32_t lo1 = ((in.y << 4) & 0xF0F0F0F0u) ^ 0x80808080u;
    const uint32_t hi1 = (in.y & 0xF0F0F0F0u) ^ 0x80808080u;
    if constexpr (PERM) {
      o = make_uint4(lo0, hi0, lo1, hi1);
    } else {
      o.x = __byte_perm(lo0, hi0, 0x5140);
      o.y = __byte_perm(lo0, hi0, 0x7362);
      o.z = __byte_perm(lo1, hi1, 0x5140);
      o.w = __byte_perm(lo1, hi1, 0x7362);
    }
    *reinterpret_cast<uint4*>(B + row * 128 + ((kc ^ (row & 7)) << 4)) = o;
  }
}

// 3-bit: tile P is [BN][48 bytes]; each thread expands 3 words (32 codes) into two 16-byte chunks.
__device__ __forceinline__ uint32_t spread3(uint32_t v) {  // 4 fields of 3 bits -> top 3 bits of 4 bytes
  return (((v << 5) & 0x000000E0u) | ((v << 10) & 0x0000E000u) | ((v << 15) & 0x00E00000u) |
          ((v << 20) & 0xE0000000u)) ^ 0x80808080u;
}
template <int BN>
__device__ __forceinline__ void unpack3_tile(const uint8_t* P, uint8_t* B, int tid) {
#pragma unroll
  for (int i = 0; i < (BN * 4 + kUnpackThreads - 1) / kUnpackThreads; ++i) {
    const int idx = tid + i * kUnpackThreads;
    if (BN * 4 % kUnpackThreads != 0 && idx >= BN * 4) break;
    const int row = idx >> 2, g = idx & 3;
    const uint32_t* src = reinterpret_cast<const uint32_t*>(P + row * 48 + g * 12);
    const uint32_t s0 = src[0], s1 = src[1], s2 = src[2];
    uint4 o0, o1;
    o0.x = spread3(s0);                               // stream bits  0..11
    o0.y = spread3(s0 >> 12);                         //             12..23
    o0.z = spread3(__funnelshift_r(s0, s1, 24));      //             24..35
    o0.w = spread3(s1 >> 4);                          //             36..47
    o1.x = spread3(s1 >> 16);                         //             48..59
    o1.y = spread3(__funnelshift_r(s1, s2, 28));      //             60..71
    o1.z = spread3(s2 >> 8);                          //             72..83
    o1.w = spread3(s2 >> 20);                         //             84..95
    uint8_t* brow = B + row * 128;
    const int sw = row & 7;
    *reinterpret_cast<uint4*>(brow + (((2 * g) ^ sw) << 4)) = o0;
    *reinterpret_cast<uint4*>(brow + (((2 * g + 1) ^ sw) << 4)) = o1;
  }
}

// ---- epilogue with one token per thread ---------------------------------------------------------------
// A warp serves its tensor-memory quadrant (32 tokens, one per thread) over a range of accumulator
// columns in rounds of 16: tcgen05.ld.32x32b.x16 (the next round's read is in flight while this one
// is converted), the fp32 sequence of Step 5 on packed pairs (two independent IEEE operations per
// instruction: int32 -> fp32, sc = s_a * s_w[n], fma(t, sc, bias[n]), bf16 round-to-nearest-even),
// and ONE 32-byte global store per thread and round (st.global.v8: a full sector of the token's
// output row), so nothing is staged in shared memory and no warp-level synchronisation sits between
// the arithmetic and the stores. Weight scales and biases come from a private fp32 copy in shared
// memory, read as broadcast 16-byte loads: global loads in this loop, even of a few cached KB, cost
// a trip to L2 per round with only ten warps on the SM to hide it. What bounds an epilogue on B200
// is the chip's store throughput (4.4 TB/s measured: about 15 bytes per clock and SM), then
// instruction issue; arithmetic does not.
template <int SHIFT>
struct RowEpilogue {
  static constexpr int CW = 16;         // columns per round
  static constexpr int kMaxCols = 128;  // columns a warp may own (its private copy of scales and biases)
  static constexpr int kScaleBytes = 2 * kMaxCols * 4;
  int qd, lane, staged_col;
  float *tsw, *tbias;
  uint32_t acc_empty_addr[2];

  __device__ __forceinline__ void init(int warp, int lane_, float* scale_copy, uint32_t acc_empty0,
                                       uint32_t acc_empty1) {
    lane = lane_;
    qd = warp & 3;
    tsw = scale_copy;
    tbias = scale_copy + kMaxCols;
    acc_empty_addr[0] = acc_empty0;
    acc_empty_addr[1] = acc_empty1;
    staged_col = -1;
  }

  // Output columns col .. col + ncols - 1 (col and ncols multiples of 16, ncols at most 128), this
  // CTA's tokens cta_row0 .. +127; their accumulators start at tensor-memory column t_col (buffer
  // `buf`, published on acc_full with phase aph). False if the wait was aborted.
  // RES: the kernel takes the residual (and gate) of GemmParams into the output; without it those
  // members are ignored.
  template <bool RES = false>
  __device__ __forceinline__ bool tile(const GemmParams& p, int col, int ncols, int cta_row0, uint32_t tmem_base,
                                       uint32_t t_col, uint64_t* acc_full, uint32_t aph, int buf,
                                       volatile int* abort_flag) {
    const int64_t row = static_cast<int64_t>(cta_row0) + qd * 32 + lane;
    float sa = 0.0f;
    if (p.x == nullptr && row < p.M) sa = __ldg(p.s_a + row);  // from an earlier kernel: fetched while waiting
    if (col != staged_col) {
      float sv[4], bv[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = lane + 32 * j;
        sv[j] = c < ncols ? __ldg(p.s_w + col + c) : 0.0f;
        bv[j] = (c < ncols && p.bias != nullptr)
                    ? __uint_as_float(static_cast<uint32_t>(__ldg(p.bias + col + c)) << 16)
                    : 0.0f;
      }
      __syncwarp();  // the previous sub-block's reads of the copy are done
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        tsw[lane + 32 * j] = sv[j];
        tbias[lane + 32 * j] = bv[j];
      }
      __syncwarp();
      staged_col = col;
    }
    // Residual and gate of this thread's token, fetched one round ahead of their use (plain loads: the
    // residual may be the output buffer, whose 32 bytes this thread reads before it overwrites them).
    const bool has_res = RES && p.res != nullptr && row < p.M;
    const bool has_gate = has_res && p.gate != nullptr;
    const uint16_t* rrow = has_res ? p.res + row * p.ldr + col : nullptr;
    const uint16_t* grow = has_gate ? p.gate + (row / p.rows_per_gate) * p.N + col : nullptr;
    uint4 rn0 = make_uint4(0, 0, 0, 0), rn1 = rn0, gn0 = rn0, gn1 = rn0;
    if (has_res) {  // the later rounds' lines on their way into L2 while the accumulators are still being summed
      for (int b = 128; b < ncols * 2; b += 128) prefetch_l2(reinterpret_cast<const uint8_t*>(rrow) + b);
      rn0 = ld_global_v4(rrow);
      rn1 = ld_global_v4(rrow + 8);
    }
    if (has_gate) {
      gn0 = ld_global_v4(grow);
      gn1 = ld_global_v4(grow + 8);
    }
    bool ok = mbar_wait(acc_full, aph, abort_flag);
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (!ok) return false;
    tc_fence_after();
    if (p.x != nullptr) {  // scales written by other CTAs of this kernel: their tile is complete by now
      (void)ld_acquire_gpu(p.sync + (cta_row0 >> 7));
      if (row < p.M) sa = *reinterpret_cast<const volatile float*>(p.s_a + row);
    }
    const uint64_t sa2 = f32x2_pack(sa, sa);
    const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + t_col;
    const float4* sw4 = reinterpret_cast<const float4*>(tsw);
    const float4* tb4 = reinterpret_cast<const float4*>(tbias);
    uint16_t* yrow = p.y + row * p.ldy + col;
    // 32-byte stores need the token's row segment 32-byte aligned; else two 16-byte stores
    const bool wide = ((reinterpret_cast<uintptr_t>(p.y) | static_cast<uintptr_t>(p.ldy * 2)) & 31u) == 0;
    const int rounds = ncols / CW;
    uint32_t ra[16];
    tmem_ld_32x16(t_addr, ra);
    for (int c = 0; c < rounds; ++c) {
      const uint32_t rr[8] = {rn0.x, rn0.y, rn0.z, rn0.w, rn1.x, rn1.y, rn1.z, rn1.w};
      const uint32_t gg[8] = {gn0.x, gn0.y, gn0.z, gn0.w, gn1.x, gn1.y, gn1.z, gn1.w};
      if (RES && c + 1 < rounds) {
        if (has_res) {
          rn0 = ld_global_v4(rrow + (c + 1) * CW);
          rn1 = ld_global_v4(rrow + (c + 1) * CW + 8);
        }
        if (has_gate) {
          gn0 = ld_global_v4(grow + (c + 1) * CW);
          gn1 = ld_global_v4(grow + (c + 1) * CW + 8);
        }
      }
      tmem_ld_wait();
      uint32_t a[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) a[i] = ra[i];
      if (c + 1 < rounds) {
        tmem_ld_32x16(t_addr + (c + 1) * CW, ra);
      } else {  // this warp's last accumulators are in registers: hand the buffer back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_addr[buf]);
      }
      uint32_t w[8];
#pragma unroll
      for (int q = 0; q < 4; ++q) {  // four columns at a time
        const float4 sw = sw4[c * 4 + q];
        const float4 bb = tb4[c * 4 + q];
        uint64_t t01 = f32x2_pack(__int2float_rn(static_cast<int>(a[4 * q])),
                                  __int2float_rn(static_cast<int>(a[4 * q + 1])));
        uint64_t t23 = f32x2_pack(__int2float_rn(static_cast<int>(a[4 * q + 2])),
                                  __int2float_rn(static_cast<int>(a[4 * q + 3])));
        if constexpr (SHIFT != 0) {  // exact: the accumulator is a multiple of 2^SHIFT
          const uint64_t down = f32x2_pack(1.0f / (1 << SHIFT), 1.0f / (1 << SHIFT));
          t01 = f32x2_mul(t01, down);
          t23 = f32x2_mul(t23, down);
        }
        const uint64_t y01 = f32x2_fma(t01, f32x2_mul(sa2, f32x2_pack(sw.x, sw.y)), f32x2_pack(bb.x, bb.y));
        const uint64_t y23 = f32x2_fma(t23, f32x2_mul(sa2, f32x2_pack(sw.z, sw.w)), f32x2_pack(bb.z, bb.w));
        float y0, y1, y2, y3;
        f32x2_unpack(y01, y0, y1);
        f32x2_unpack(y23, y2, y3);
        if (RES && p.res != nullptr) {  // uniform over the grid
          const float r0 = __uint_as_float(rr[2 * q] << 16), r1 = __uint_as_float(rr[2 * q] & 0xFFFF0000u);
          const float r2 = __uint_as_float(rr[2 * q + 1] << 16), r3 = __uint_as_float(rr[2 * q + 1] & 0xFFFF0000u);
          if (p.gate != nullptr) {
            y0 = fmaf(__uint_as_float(gg[2 * q] << 16), y0, r0);
            y1 = fmaf(__uint_as_float(gg[2 * q] & 0xFFFF0000u), y1, r1);
            y2 = fmaf(__uint_as_float(gg[2 * q + 1] << 16), y2, r2);
            y3 = fmaf(__uint_as_float(gg[2 * q + 1] & 0xFFFF0000u), y3, r3);
          } else {
            y0 = __fadd_rn(y0, r0);
            y1 = __fadd_rn(y1, r1);
            y2 = __fadd_rn(y2, r2);
            y3 = __fadd_rn(y3, r3);
          }
        }
        const __nv_bfloat162 v01 = __floats2bfloat162_rn(y0, y1), v23 = __floats2bfloat162_rn(y2, y3);
        w[2 * q] = *reinterpret_cast<const uint32_t*>(&v01);
        w[2 * q + 1] = *reinterpret_cast<const uint32_t*>(&v23);
      }
      if (row < p.M) {
        if (p.dbg_acc != nullptr) {
          int32_t* arow = p.dbg_acc + row * p.dbg_ldacc + col + c * CW;
#pragma unroll
          for (int i = 0; i < 16; ++i) arow[i] = static_cast<int>(a[i]) >> SHIFT;
        }
        if (wide) {
          st_global_v8(yrow + c * CW, w);
        } else {
          uint4* y4 = reinterpret_cast<uint4*>(yrow + c * CW);
          y4[0] = make_uint4(w[0], w[1], w[2], w[3]);
          y4[1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
    }
    return true;
  }
};

}  // namespace dp
