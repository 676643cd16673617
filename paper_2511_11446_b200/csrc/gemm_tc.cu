// Tensor-core path of the quantized linear: Y = dequant(Xq . unpack(Wp)^T) + bias on sm_100a.
//
//   Step 5 / Implementation of the paper: INT8 x INT8 -> INT32 GEMM with per-output-channel weight
//   scales; Step 3: weights are GPTQ-style packed low-bit integers, expanded on the fly.
//
// One persistent CTA per SM walks a static list of 128 x BN output tiles. Warp roles:
//   warp 0      TMA producer: int8 activation tiles (128-byte-swizzled) and packed weight tiles
//   warp 1      MMA issuer: tcgen05.mma kind::i8, int32 accumulators in tensor memory (two
//               accumulator buffers, so a tile's epilogue overlaps the next tile's mainloop)
//   warps 2-5   epilogue: tcgen05.ld -> (float)acc * s_a[m]*s_w[n] + bias -> bf16 -> global
//   warps 6-9   unpack (3/4-bit only): packed tile in smem -> int8 operand tile in smem, written in
//               the swizzled layout the MMA descriptor expects, then fence.proxy.async
//
// Low-bit codes are expanded as w * 2^(8-b) (the two's-complement field moved to the top of the
// byte: two logic ops per word instead of a sign-extension); the accumulator is then an exact
// multiple of 2^(8-b) (|acc| <= 4608*127*128 < 2^31) and the epilogue multiplies by 2^-(8-b),
// which is exact in fp32, before the scale.
#include <cuda_bf16.h>

#include "dp_common.cuh"
#include "dp_internal.h"

namespace dp {

constexpr int BM = 128;
constexpr int BK = 128;  // int8 elements = bytes = one 128-byte swizzle row
constexpr int kGemmThreads = 320;
constexpr int kEpiWarp0 = 2, kUnpackWarp0 = 6;
constexpr int kSmemBudget = 200 * 1024;
constexpr int kPStages = 3;

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
  int64_t M;
  int32_t N, K;
  int32_t m_tiles, n_tiles;
  int32_t* status;
};

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
template <int BN>
__device__ __forceinline__ void unpack4_tile(const uint8_t* P, uint8_t* B, int tid) {
#pragma unroll 4
  for (int idx = tid; idx < BN * 8; idx += 128) {
    const int row = idx >> 3, kc = idx & 7;
    const uint2 in = *reinterpret_cast<const uint2*>(P + row * 64 + kc * 8);
    uint4 o;
    {
      const uint32_t lo = ((in.x << 4) & 0xF0F0F0F0u) ^ 0x80808080u;  // even fields
      const uint32_t hi = (in.x & 0xF0F0F0F0u) ^ 0x80808080u;         // odd fields
      o.x = __byte_perm(lo, hi, 0x5140);
      o.y = __byte_perm(lo, hi, 0x7362);
    }
    {
      const uint32_t lo = ((in.y << 4) & 0xF0F0F0F0u) ^ 0x80808080u;
      const uint32_t hi = (in.y & 0xF0F0F0F0u) ^ 0x80808080u;
      o.z = __byte_perm(lo, hi, 0x5140);
      o.w = __byte_perm(lo, hi, 0x7362);
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
#pragma unroll 2
  for (int idx = tid; idx < BN * 4; idx += 128) {
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

// ---- the kernel ----------------------------------------------------------------------------------
template <int BN, int BITS>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
               const GemmParams p) {
  constexpr int NS = num_stages(BN, BITS);
  constexpr int NP = kPStages;
  constexpr int A_BYTES = BM * BK, B_BYTES = BN * BK, P_BYTES = p_stage_bytes(BN, BITS);
  constexpr int TCOLS = tmem_cols(BN);
  constexpr int SHIFT = 8 - BITS;  // accumulator carries a factor 2^SHIFT

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = sA + NS * A_BYTES;
  uint8_t* sP = sB + NS * B_BYTES;
  uint8_t* tail = sP + NP * P_BYTES;
  uint64_t* full_a = reinterpret_cast<uint64_t*>(tail);
  uint64_t* bready = full_a + NS;
  uint64_t* empty = bready + NS;
  uint64_t* pfull = empty + NS;
  uint64_t* pempty = pfull + NP;
  uint64_t* acc_full = pempty + NP;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* s_scale = reinterpret_cast<float*>(tmem_slot + 4);  // [4 warps][BN] weight scales of the tile
  float* s_bias = s_scale + 4 * BN;                           // [4 warps][BN]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = p.K / BK;
  const int total_tiles = p.m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_a[i], 1);
      mbar_init(&bready[i], 128);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < NP; ++i) {
      mbar_init(&pfull[i], 1);
      mbar_init(&pempty[i], 128);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 128);
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_w);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TCOLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_launch_dependents();
  pdl_wait();  // everything below reads what the previous kernel on the stream produced

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      Ring st, ps;
      int issued = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m_blk = tile % p.m_tiles, n_blk = tile / p.m_tiles;
        for (int kb = 0; kb < KB; ++kb) {
          if (!(ok = mbar_wait(&empty[st.s], st.ph ^ 1u, abort_flag))) break;
          if constexpr (BITS == 8) {
            mbar_arrive_expect_tx(&full_a[st.s], A_BYTES + B_BYTES);
            tma_load_2d(sA + st.s * A_BYTES, &tmap_a, kb * BK, m_blk * BM, &full_a[st.s]);
            tma_load_2d(sB + st.s * B_BYTES, &tmap_w, kb * BK, n_blk * BN, &full_a[st.s]);
          } else {
            if (!(ok = mbar_wait(&pempty[ps.s], ps.ph ^ 1u, abort_flag))) break;
            mbar_arrive_expect_tx(&pfull[ps.s], P_BYTES);
            tma_load_2d(sP + ps.s * P_BYTES, &tmap_w, kb * (BK * BITS / 8), n_blk * BN, &pfull[ps.s]);
            mbar_arrive_expect_tx(&full_a[st.s], A_BYTES);
            tma_load_2d(sA + st.s * A_BYTES, &tmap_a, kb * BK, m_blk * BM, &full_a[st.s]);
            ps.next(NP);
          }
          st.next(NS);
          ++issued;
        }
      }
      if (!ok) {
        // drain: give copies still in flight a bounded time to land before the CTA exits
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_i8(BM, BN);
      Ring st;
      bool ok = true;
      int tcount = 0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
        const int buf = tcount & 1;
        const uint32_t aph = (tcount >> 1) & 1;
        if (!(ok = mbar_wait(&acc_empty[buf], aph ^ 1u, abort_flag))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * (TCOLS / 2);
        for (int kb = 0; kb < KB; ++kb) {
          if (!(ok = mbar_wait(&full_a[st.s], st.ph, abort_flag))) break;
          if constexpr (BITS != 8) {
            if (!(ok = mbar_wait(&bready[st.s], st.ph, abort_flag))) break;
          }
          tc_fence_after();
          const uint64_t adesc = smem_desc_sw128(smem_u32(sA + st.s * A_BYTES));
          const uint64_t bdesc = smem_desc_sw128(smem_u32(sB + st.s * B_BYTES));
#pragma unroll
          for (int k4 = 0; k4 < BK / 32; ++k4)  // 32 bytes of K per instruction: +2 in 16-byte units
            mma_i8_ss(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
          mma_commit(&empty[st.s]);
          st.next(NS);
        }
        if (ok) mma_commit(&acc_full[buf]);
      }
    }
  } else if (warp < kUnpackWarp0) {
    // ================= epilogue =================
    const int qd = warp & 3;  // TMEM lane quadrant this warp may read
    float* ts = s_scale + (warp - kEpiWarp0) * BN;  // this warp's private copy: no CTA-wide sync
    float* tb = s_bias + (warp - kEpiWarp0) * BN;
    bool ok = true;
    int tcount = 0;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int m_blk = tile % p.m_tiles, n_blk = tile / p.m_tiles;
      const int buf = tcount & 1;
      const uint32_t aph = (tcount >> 1) & 1;
      const int n0 = n_blk * BN;
      __syncwarp();
      for (int i = lane; i < BN; i += 32) {
        ts[i] = p.s_w[n0 + i];
        tb[i] = p.bias != nullptr ? __uint_as_float(static_cast<uint32_t>(p.bias[n0 + i]) << 16) : 0.0f;
      }
      __syncwarp();
      const int64_t row = static_cast<int64_t>(m_blk) * BM + qd * 32 + lane;
      const bool row_ok = row < p.M;
      const float sa = row_ok ? p.s_a[row] : 0.0f;
      ok = mbar_wait(&acc_full[buf], aph, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + buf * (TCOLS / 2);
      uint16_t* yrow = p.y + row * p.ldy + n0;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32(t_addr + c * 32, r);
        tmem_ld_wait();
        if (row_ok) {
          uint32_t o[16];
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float t0 = __int2float_rn(static_cast<int>(r[j]));
            float t1 = __int2float_rn(static_cast<int>(r[j + 1]));
            if constexpr (SHIFT != 0) {
              t0 = __fmul_rn(t0, 1.0f / (1 << SHIFT));
              t1 = __fmul_rn(t1, 1.0f / (1 << SHIFT));
            }
            const float y0 = __fmaf_rn(t0, __fmul_rn(sa, ts[c * 32 + j]), tb[c * 32 + j]);
            const float y1 = __fmaf_rn(t1, __fmul_rn(sa, ts[c * 32 + j + 1]), tb[c * 32 + j + 1]);
            const __nv_bfloat162 h = __floats2bfloat162_rn(y0, y1);
            o[j >> 1] = *reinterpret_cast<const uint32_t*>(&h);
          }
          uint4* dst = reinterpret_cast<uint4*>(yrow + c * 32);
          dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
          dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
          dst[2] = make_uint4(o[8], o[9], o[10], o[11]);
          dst[3] = make_uint4(o[12], o[13], o[14], o[15]);
          if (p.dbg_acc != nullptr) {
            int32_t* arow = p.dbg_acc + row * p.dbg_ldacc + n0 + c * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j) arow[j] = static_cast<int>(r[j]) >> SHIFT;
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
    }
  } else {
    // ================= unpack (3/4-bit weights) =================
    if constexpr (BITS != 8) {
      const int ut = threadIdx.x - kUnpackWarp0 * 32;
      Ring st, ps;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        for (int kb = 0; kb < KB; ++kb) {
          ok = mbar_wait(&pfull[ps.s], ps.ph, abort_flag) &&
               mbar_wait(&empty[st.s], st.ph ^ 1u, abort_flag);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          if constexpr (BITS == 4) unpack4_tile<BN>(sP + ps.s * P_BYTES, sB + st.s * B_BYTES, ut);
          else unpack3_tile<BN>(sP + ps.s * P_BYTES, sB + st.s * B_BYTES, ut);
          fence_proxy_async_smem();
          mbar_arrive(&bready[st.s]);
          mbar_arrive(&pempty[ps.s]);
          st.next(NS);
          ps.next(NP);
        }
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TCOLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicExch(p.status, DP_ERR_TIMEOUT);
}

// ---- host side -------------------------------------------------------------------------------------
template <int BN, int BITS>
constexpr size_t gemm_smem_bytes() {
  return 1024 + static_cast<size_t>(num_stages(BN, BITS)) * ab_stage_bytes(BN) +
         kPStages * p_stage_bytes(BN, BITS) + (3 * 8 + 2 * kPStages + 4) * 8 + 16 + 8 * BN * 4 + 64;
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                              CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                              CUtensorMapFloatOOBfill);
static EncodeFn g_encode = nullptr;
static int g_num_sms = 0;

template <int BN, int BITS>
static cudaError_t set_attr() {
  return cudaFuncSetAttribute(gemm_i8_kernel<BN, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(gemm_smem_bytes<BN, BITS>()));
}

int num_sms() { return g_num_sms; }

int gemm_init() {
  static int state = -1;  // -1 not tried, else status
  if (state >= 0) return state;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess)
    return fail(DP_ERR_CUDA, "cuTensorMapEncodeTiled not available: %s", cudaGetErrorString(e));
  g_encode = reinterpret_cast<EncodeFn>(fn);
  int dev = 0;
  DP_CUDA_OK(cudaGetDevice(&dev));
  DP_CUDA_OK(cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev));
#define DP_SET(BN)                               \
  DP_CUDA_OK((set_attr<BN, 8>()));               \
  DP_CUDA_OK((set_attr<BN, 4>()));               \
  DP_CUDA_OK((set_attr<BN, 3>()));
  DP_SET(64) DP_SET(128) DP_SET(192) DP_SET(256)
#undef DP_SET
  state = DP_OK;
  return state;
}

static int encode_2d(CUtensorMap* out, const void* base, uint64_t inner_bytes, uint64_t rows,
                     uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows, bool swizzle128) {
  const cuuint64_t dims[2] = {inner_bytes, rows};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides,
                        box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(DP_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return DP_OK;
}

int gemm_encode_a(CUtensorMap* out, const int8_t* q, int64_t M, int64_t K, int64_t ldq) {
  return encode_2d(out, q, K, M, ldq, BK, BM, true);
}

int gemm_encode_w(CUtensorMap* out, const void* qweight, int32_t N, int32_t K, int32_t bits,
                  int32_t bn) {
  const uint64_t row_bytes = static_cast<uint64_t>(K) * bits / 8;
  return encode_2d(out, qweight, row_bytes, N, row_bytes, BK * bits / 8, bn, bits == 8);
}

// Tile width: the widest of {256, 192, 128, 64} dividing N whose tile count keeps the last wave
// reasonably full; small problems take narrower tiles to spread over the SMs.
int gemm_pick_bn(int64_t M, int32_t N, int32_t K, int32_t bits) {
  (void)K;
  (void)bits;
  const int64_t m_tiles = (M + BM - 1) / BM;
  const int sms = g_num_sms > 0 ? g_num_sms : 148;
  const int cand[4] = {256, 192, 128, 64};
  int best = 0;
  double best_cost = 1e30;
  for (int i = 0; i < 4; ++i) {
    const int bn = cand[i];
    if (N % bn) continue;
    const int64_t tiles = m_tiles * (N / bn);
    const int64_t waves = (tiles + sms - 1) / sms;
    // time model: waves * (tile MMA time + fixed per-tile overhead), MMA time ~ bn
    const double cost = static_cast<double>(waves) * (bn + 24.0);
    if (cost < best_cost) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

template <int BN>
static cudaError_t launch_bn(const GemmProblem& g, const GemmParams& p, dim3 grid, cudaStream_t stream,
                             bool pdl) {
  const dim3 block(kGemmThreads);
  switch (g.bits) {
    case 8:
      return launch(gemm_i8_kernel<BN, 8>, grid, block, gemm_smem_bytes<BN, 8>(), stream, pdl, g.tmap_a,
                    g.tmap_w, p);
    case 4:
      return launch(gemm_i8_kernel<BN, 4>, grid, block, gemm_smem_bytes<BN, 4>(), stream, pdl, g.tmap_a,
                    g.tmap_w, p);
    default:
      return launch(gemm_i8_kernel<BN, 3>, grid, block, gemm_smem_bytes<BN, 3>(), stream, pdl, g.tmap_a,
                    g.tmap_w, p);
  }
}

int launch_gemm(const GemmProblem& g, cudaStream_t stream, bool pdl) {
  if (g.M == 0) return DP_OK;
  GemmParams p;
  p.s_a = g.s_a;
  p.s_w = g.s_w;
  p.bias = g.bias;
  p.y = g.y;
  p.ldy = g.ldy;
  p.dbg_acc = g.dbg_acc;
  p.dbg_ldacc = g.dbg_ldacc;
  p.M = g.M;
  p.N = g.N;
  p.K = g.K;
  p.m_tiles = static_cast<int32_t>((g.M + BM - 1) / BM);
  p.n_tiles = g.N / g.bn;
  p.status = g.status;
  const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
  const dim3 grid(static_cast<unsigned>(tiles < g_num_sms ? tiles : g_num_sms));
  cudaError_t e;
  switch (g.bn) {
    case 64: e = launch_bn<64>(g, p, grid, stream, pdl); break;
    case 128: e = launch_bn<128>(g, p, grid, stream, pdl); break;
    case 192: e = launch_bn<192>(g, p, grid, stream, pdl); break;
    case 256: e = launch_bn<256>(g, p, grid, stream, pdl); break;
    default: return fail(DP_ERR_INVALID_ARG, "unsupported tile width %d", g.bn);
  }
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "GEMM launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
