// Quantized linear with GROUP-WISE weight scales (and optional zero-points).
//
//   Step 2 of the paper: the GPTQ storage format of its plans keeps one scale and one zero-point per
//   output channel and group of g input channels (g in 32 .. 288), not one scale per channel. With
//   them the int32 accumulator can no longer be dequantized once at the end: every group's partial
//   sum has its own scale. Sequence (the oracle's, bit for bit):
//       acc_G = sum_{k in G} q[m,k] * (u[n,k] - z[n,G])                exact int32
//       t = 0;  for G in order:  t = fma((float)acc_G, s_w[n][G], t)    fp32
//       y = bf16_rne(fma(t, s_a[m], bias[n]))
//
// One persistent CTA per SM walks 128 x 128 output tiles. Warp 0: TMA producer (int8 activation and
// weight tiles, 128 bytes of K per stage). Warp 1: MMA issuer: tcgen05.mma kind::i8 in steps of 32
// bytes of K; the steps of one group accumulate in one of FOUR 128-column tensor-memory buffers, the
// next group starts in the next buffer (group boundaries need not fall on stage boundaries: g = 192
// or 288 span one and a half or two and a quarter stages). Warps 2-9: fold and epilogue, one token
// per thread and 64 columns per warp: per group tcgen05.ld, the zero-point correction
// (2^(b-1) - z[n,G]) * rowsum_G[m] in int32 (the tensor core multiplies by u - 2^(b-1)), one fma into
// 64 fp32 partial outputs held in registers, then the buffer goes back to the MMA issuer; after the
// last group the token scale, bias, bf16 rounding and 32-byte stores.
// The fold costs two instructions per output and group, so this kernel is bound by the fold, not the
// tensor core, the more so the smaller g is.
#include "gemm_device.cuh"

namespace dp {

constexpr int kGrpBN = 128;
constexpr int kGrpBufs = 4;
constexpr int kGrpStages = 6;
constexpr int kGrpThreads = kUnpackWarp0 * 32;

struct GrpParams {
  const float* s_a;       // [M]
  const float* s_w;       // [N][ng]
  const uint8_t* zeros;   // [N][ng] or null
  const int32_t* rowsum;  // [M][ng] (zero-points only)
  const uint16_t* bias;
  uint16_t* y;
  int64_t ldy;
  int64_t M;
  int32_t N, K, g, ng, half;  // half = 2^(bits-1)
  int32_t m_tiles, n_tiles, a_tiled;
  int32_t* status;
};

__global__ void __launch_bounds__(kGrpThreads, 1)
gemm_grp_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                const GrpParams p) {
  constexpr int NS = kGrpStages, A_BYTES = BM * BK, B_BYTES = kGrpBN * BK;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = sA + NS * A_BYTES;
  float* s_scale = reinterpret_cast<float*>(sB + NS * B_BYTES);  // per warp: [2][64] group scales, [2][64] zero-point terms, [64] biases
  uint64_t* full = reinterpret_cast<uint64_t*>(s_scale + kEpiWarps * 320);
  uint64_t* empty = full + NS;
  uint64_t* grp_full = empty + NS;
  uint64_t* grp_empty = grp_full + kGrpBufs;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(grp_empty + kGrpBufs);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = p.K / BK;
  const int total_tiles = p.m_tiles * p.n_tiles;
  const int spg = p.g >> 5;  // MMA steps (32 bytes of K) per group

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < kGrpBufs; ++i) {
      mbar_init(&grp_full[i], 1);
      mbar_init(&grp_empty[i], kEpiWarps);
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_w);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_launch_dependents();
  pdl_wait();  // activations, scales and the int8 weight copy come from the preceding kernels on the stream

  if (warp == 0) {
    if (lane == 0) {
      Ring st;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int n_blk = tile % p.n_tiles, m_row = (tile / p.n_tiles) * BM;
        for (int kb = 0; kb < KB; ++kb) {
          if (!(ok = mbar_spin_wait(&empty[st.s], st.ph ^ 1u, abort_flag))) break;
          mbar_arrive_expect_tx(&full[st.s], A_BYTES + B_BYTES);
          int c0, c1;
          if (p.a_tiled) {
            c0 = 0;
            c1 = ((m_row >> 7) * KB + kb) * BM;
          } else {
            c0 = kb * BK;
            c1 = m_row;
          }
          tma_load_2d(sA + st.s * A_BYTES, &tmap_a, c0, c1, &full[st.s]);
          tma_load_2d(sB + st.s * B_BYTES, &tmap_w, kb * BK, n_blk * kGrpBN, &full[st.s]);
          st.next(NS);
        }
      }
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_i8(BM, kGrpBN);
      Ring st;
      bool ok = true;
      uint32_t gcount = 0;  // groups issued so far: buffer = gcount % 4
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        int pos = 0;  // step inside the current group
        for (int kb = 0; kb < KB && ok; ++kb) {
          if (!(ok = mbar_spin_wait(&full[st.s], st.ph, abort_flag))) break;
          tc_fence_after();
          const uint64_t adesc = smem_desc_sw128(smem_u32(sA + st.s * A_BYTES));
          const uint64_t bdesc = smem_desc_sw128(smem_u32(sB + st.s * B_BYTES));
          for (int k4 = 0; k4 < BK / 32; ++k4) {
            const uint32_t buf = gcount % kGrpBufs;
            if (pos == 0) {  // a new group: its buffer must have been folded
              if (!(ok = mbar_wait(&grp_empty[buf], ((gcount / kGrpBufs) & 1u) ^ 1u, abort_flag))) break;
              tc_fence_after();
            }
            mma_i8_ss(tmem_base + buf * kGrpBN, adesc + 2 * k4, bdesc + 2 * k4, idesc, pos != 0 ? 1u : 0u);
            if (++pos == spg) {
              mma_commit(&grp_full[buf]);
              pos = 0;
              ++gcount;
            }
          }
          if (ok) mma_commit(&empty[st.s]);
          st.next(NS);
        }
      }
    }
  } else {
    // ================= fold + epilogue: quadrant (warp & 3), column half (ew >> 2) =================
    const int ew = warp - kEpiWarp0, qd = warp & 3;
    const int col0 = (ew >> 2) * 64;
    float* wsc = s_scale + ew * 320;                            // [2][64] scales of the current / next group
    int32_t* wdz = reinterpret_cast<int32_t*>(wsc + 128);       // [2][64] (2^(b-1) - z) of the same groups
    float* wb = wsc + 256;                                      // [64] biases
    const bool wide = ((reinterpret_cast<uintptr_t>(p.y) | static_cast<uintptr_t>(p.ldy * 2)) & 31u) == 0;
    const bool zp = p.zeros != nullptr;
    bool ok = true;
    uint32_t gcount = 0;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int n0 = (tile % p.n_tiles) * kGrpBN + col0;
      const int64_t row = static_cast<int64_t>(tile / p.n_tiles) * BM + qd * 32 + lane;
      const bool live = row < p.M;
      const float sa = live ? __ldg(p.s_a + row) : 0.0f;
      // this lane stages columns lane and lane + 32 of the warp's 64
      const float* swp = p.s_w + static_cast<int64_t>(n0 + lane) * p.ng;
      const uint8_t* zpp = zp ? p.zeros + static_cast<int64_t>(n0 + lane) * p.ng : nullptr;
      const int64_t hop = static_cast<int64_t>(32) * p.ng;
      __syncwarp();
      wb[lane] = p.bias != nullptr ? __uint_as_float(static_cast<uint32_t>(__ldg(p.bias + n0 + lane)) << 16) : 0.0f;
      wb[lane + 32] =
          p.bias != nullptr ? __uint_as_float(static_cast<uint32_t>(__ldg(p.bias + n0 + lane + 32)) << 16) : 0.0f;
      float s0 = __ldg(swp), s1 = __ldg(swp + hop);  // group 0
      int z0 = zp ? p.half - static_cast<int>(__ldg(zpp)) : 0, z1 = zp ? p.half - static_cast<int>(__ldg(zpp + hop)) : 0;
      int rs = (zp && live) ? __ldg(p.rowsum + row * p.ng) : 0;
      float t[64];
#pragma unroll
      for (int i = 0; i < 64; ++i) t[i] = 0.0f;
      for (int G = 0; G < p.ng && ok; ++G, ++gcount) {
        const int par = G & 1;
        wsc[par * 64 + lane] = s0;
        wsc[par * 64 + lane + 32] = s1;
        wdz[par * 64 + lane] = z0;
        wdz[par * 64 + lane + 32] = z1;
        __syncwarp();
        const int rs_g = rs;
        if (G + 1 < p.ng) {  // the next group's scales fly while this one is folded
          s0 = __ldg(swp + G + 1);
          s1 = __ldg(swp + hop + G + 1);
          if (zp) {
            z0 = p.half - static_cast<int>(__ldg(zpp + G + 1));
            z1 = p.half - static_cast<int>(__ldg(zpp + hop + G + 1));
            if (live) rs = __ldg(p.rowsum + row * p.ng + G + 1);
          }
        }
        const uint32_t buf = gcount % kGrpBufs;
        ok = mbar_wait(&grp_full[buf], (gcount / kGrpBufs) & 1u, abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + buf * kGrpBN + col0;
        const float4* sc4 = reinterpret_cast<const float4*>(wsc + par * 64);
        const int4* dz4 = reinterpret_cast<const int4*>(wdz + par * 64);
        uint32_t ra[16];
        tmem_ld_32x16(t_addr, ra);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          tmem_ld_wait();
          uint32_t a[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) a[i] = ra[i];
          if (c + 1 < 4) {
            tmem_ld_32x16(t_addr + (c + 1) * 16, ra);
          } else {  // the group's accumulators are in registers: the buffer may take the next group
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&grp_empty[buf]);
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float4 sc = sc4[c * 4 + q];
            int a0 = static_cast<int>(a[4 * q]), a1 = static_cast<int>(a[4 * q + 1]);
            int a2 = static_cast<int>(a[4 * q + 2]), a3 = static_cast<int>(a[4 * q + 3]);
            if (zp) {
              const int4 dz = dz4[c * 4 + q];
              a0 += dz.x * rs_g;
              a1 += dz.y * rs_g;
              a2 += dz.z * rs_g;
              a3 += dz.w * rs_g;
            }
            float* tt = t + c * 16 + 4 * q;
            tt[0] = __fmaf_rn(__int2float_rn(a0), sc.x, tt[0]);
            tt[1] = __fmaf_rn(__int2float_rn(a1), sc.y, tt[1]);
            tt[2] = __fmaf_rn(__int2float_rn(a2), sc.z, tt[2]);
            tt[3] = __fmaf_rn(__int2float_rn(a3), sc.w, tt[3]);
          }
        }
      }
      if (!ok) break;
      if (live) {
        uint16_t* yrow = p.y + row * p.ldy + n0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float2 bb = *reinterpret_cast<const float2*>(wb + c * 16 + 2 * q);
            const __nv_bfloat162 v = __floats2bfloat162_rn(__fmaf_rn(t[c * 16 + 2 * q], sa, bb.x),
                                                           __fmaf_rn(t[c * 16 + 2 * q + 1], sa, bb.y));
            w[q] = *reinterpret_cast<const uint32_t*>(&v);
          }
          if (wide) {
            st_global_v8(yrow + c * 16, w);
          } else {
            uint4* y4 = reinterpret_cast<uint4*>(yrow + c * 16);
            y4[0] = make_uint4(w[0], w[1], w[2], w[3]);
            y4[1] = make_uint4(w[4], w[5], w[6], w[7]);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicExch(p.status, DP_ERR_TIMEOUT);
}

// Per-group sums of a token's int8 codes, rowsum[m][G] = sum_{k in G} q[m,k] (the zero-point term of the
// fold), from the tiled scratch the DAQ launch wrote ([row tile][k block][128][128]) or a row-major q.
// One warp per token: a lane sums 16 consecutive codes per load (a group is a multiple of 32 codes,
// so the 16 belong to one group) and adds the partial sum to the group's counter in shared memory.
constexpr int kRowsumWarps = 8, kRowsumMaxGroups = 160;  // K <= 5120 at g = 32
__global__ void __launch_bounds__(kRowsumWarps * 32)
group_rowsum_kernel(const int8_t* __restrict__ q, int64_t M, int K, int64_t ldq, int tiled, int g, int ng,
                    int32_t* __restrict__ rowsum) {
  __shared__ int sums[kRowsumWarps][kRowsumMaxGroups];
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t m = static_cast<int64_t>(blockIdx.x) * kRowsumWarps + warp;
  for (int G = lane; G < ng; G += 32) sums[warp][G] = 0;
  __syncwarp();
  pdl_wait();
  if (m >= M) return;
  for (int k = lane * 16; k < K; k += 32 * 16) {
    const int8_t* src = tiled ? q + ((m >> 7) * (K >> 7) + (k >> 7)) * 16384 + (m & 127) * 128 + (k & 127)
                              : q + m * ldq + k;
    const uint4 v = *reinterpret_cast<const uint4*>(src);
    int s = __dp4a(static_cast<int>(v.x), 0x01010101, 0);
    s = __dp4a(static_cast<int>(v.y), 0x01010101, s);
    s = __dp4a(static_cast<int>(v.z), 0x01010101, s);
    s = __dp4a(static_cast<int>(v.w), 0x01010101, s);
    atomicAdd(&sums[warp][k / g], s);
  }
  __syncwarp();
  for (int G = lane; G < ng; G += 32) rowsum[m * ng + G] = sums[warp][G];
}

// ---- host side -------------------------------------------------------------------------------------
constexpr size_t grp_smem_bytes() {
  return 1024 + static_cast<size_t>(kGrpStages) * (BM + kGrpBN) * BK + kEpiWarps * 320 * 4 +
         (2 * kGrpStages + 2 * kGrpBufs + 1) * 8 + 64;
}

int gemm_grp_init_device() {
  DP_CUDA_OK(cudaFuncSetAttribute(gemm_grp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(grp_smem_bytes())));
  return DP_OK;
}

// q / s_a: the quantized activations (tiled scratch when a_tiled); w8: int8 [N][K] (true values
// u - 2^(bits-1)); rowsum: scratch int32 [M][K/g], used (and filled here) only with zero-points.
int launch_gemm_grp(const int8_t* q, int64_t ldq, bool a_tiled, const float* s_a, const int8_t* w8, int32_t bits,
                    int32_t g, const float* s_w, const uint8_t* zeros, const uint16_t* bias, int32_t* rowsum, int64_t M,
                    int32_t N, int32_t K, uint16_t* y, int64_t ldy, int32_t* status, cudaStream_t stream, bool pdl) {
  if (M == 0) return DP_OK;
  if (N % kGrpBN || g <= 0 || g % 32 || K % g)
    return fail(DP_ERR_SHAPE, "group-wise layer: need N %% 128 == 0, g %% 32 == 0, K %% g == 0 (N=%d K=%d g=%d)", N, K, g);
  const int ng = K / g;
  if (zeros != nullptr) {
    if (ng > kRowsumMaxGroups) return fail(DP_ERR_SHAPE, "group-wise zero-points: more than %d groups per row", kRowsumMaxGroups);
    const cudaError_t e = launch(group_rowsum_kernel, dim3(static_cast<unsigned>((M + kRowsumWarps - 1) / kRowsumWarps)),
                                 dim3(kRowsumWarps * 32), 0, stream, pdl, q, M, static_cast<int>(K), ldq,
                                 a_tiled ? 1 : 0, static_cast<int>(g), ng, rowsum);
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "group row-sum launch failed: %s", cudaGetErrorString(e));
  }
  CUtensorMap ta, tw;
  int st = a_tiled ? gemm_encode_a_tiled(&ta, q, M, K) : gemm_encode_a(&ta, q, M, K, ldq);
  if (st != DP_OK) return st;
  st = gemm_encode_w(&tw, w8, N, K, 8, kGrpBN, 1);
  if (st != DP_OK) return st;
  GrpParams p;
  p.s_a = s_a;
  p.s_w = s_w;
  p.zeros = zeros;
  p.rowsum = rowsum;
  p.bias = bias;
  p.y = y;
  p.ldy = ldy;
  p.M = M;
  p.N = N;
  p.K = K;
  p.g = g;
  p.ng = ng;
  p.half = 1 << (bits - 1);
  p.m_tiles = static_cast<int32_t>((M + BM - 1) / BM);
  p.n_tiles = N / kGrpBN;
  p.a_tiled = a_tiled ? 1 : 0;
  p.status = status;
  const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
  const int sms = num_sms() > 0 ? num_sms() : 148;
  const cudaError_t e = launch(gemm_grp_kernel, dim3(static_cast<unsigned>(tiles < sms ? tiles : sms)), dim3(kGrpThreads),
                               grp_smem_bytes(), stream, pdl, ta, tw, p);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "group-wise GEMM launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
