// Pass-through linear for layers the plan keeps in 16-bit precision: Y = X . W^T + bias, bf16 inputs
// and weights, fp32 accumulation on the tensor cores, bf16 output.
//
//   Step 1 tiering / Step 2 results of the paper: the most sensitive layers are frozen in FP16 (22 of
//   113 in its best plan) and run beside the INT8 ones, so a deployed plan (Algorithm 2, Phase B) must
//   be able to run them in the same call sequence. No DAQ, no weight scales.
//
// One persistent CTA per SM walks 128 x BN output tiles (column tiles of a row strip together). Warp 0:
// TMA producer (activation and weight tiles of 64 bf16 = 128-byte rows, 128-byte swizzle, straight
// from the caller's row-major matrices); warp 1: MMA issuer (tcgen05.mma kind::f16 with bf16 operands,
// fp32 accumulators in tensor memory, two buffers); warps 2-9: epilogue, one token per thread:
// tcgen05.ld -> + bias -> bf16 -> one 32-byte store per 16 columns.
#include "gemm_device.cuh"

namespace dp {

constexpr int kBfThreads = kUnpackWarp0 * 32;
constexpr int kBfBK = 128;  // bytes of K per k-block = 64 bf16

// Instruction descriptor, kind::f16: D = f32, A = B = bf16, both K-major, dense.
__host__ __device__ constexpr uint32_t idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}
__device__ __forceinline__ void mma_bf16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

struct BfParams {
  const uint16_t* bias;
  uint16_t* y;
  int64_t ldy;
  int64_t M;
  int32_t N, K;
  int32_t m_tiles, n_tiles;
  int32_t* status;
};

__host__ __device__ constexpr int bf_stages(int bn) { return (200 * 1024) / ((BM + bn) * kBfBK); }

template <int BN>
__global__ void __launch_bounds__(kBfThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                 const BfParams p) {
  constexpr int NS = bf_stages(BN) > 8 ? 8 : bf_stages(BN);
  constexpr int A_BYTES = BM * kBfBK, B_BYTES = BN * kBfBK;
  constexpr int TCOLS = tmem_cols(BN);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = sA + NS * A_BYTES;
  float* s_bias = reinterpret_cast<float*>(sB + NS * B_BYTES);  // per epilogue warp: fp32 copy of its columns' biases
  uint64_t* full = reinterpret_cast<uint64_t*>(s_bias + kEpiWarps * 128);
  uint64_t* empty = full + NS;
  uint64_t* acc_full = empty + NS;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = (p.K * 2) / kBfBK;
  const int total_tiles = p.m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], kEpiWarps);
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
  pdl_wait();  // the activations may come from the preceding kernel on the stream

  if (warp == 0) {
    if (lane == 0) {
      Ring st;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int n_blk = tile % p.n_tiles, m_row = (tile / p.n_tiles) * BM;
        for (int kb = 0; kb < KB; ++kb) {
          if (!(ok = mbar_spin_wait(&empty[st.s], st.ph ^ 1u, abort_flag))) break;
          mbar_arrive_expect_tx(&full[st.s], A_BYTES + B_BYTES);
          tma_load_2d(sA + st.s * A_BYTES, &tmap_a, kb * kBfBK, m_row, &full[st.s]);
          tma_load_2d(sB + st.s * B_BYTES, &tmap_w, kb * kBfBK, n_blk * BN, &full[st.s]);
          st.next(NS);
        }
      }
      if (!ok) {  // give copies still in flight a bounded time to land before the CTA exits
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(BM, BN);
      Ring st;
      bool ok = true;
      int tcount = 0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
        const int buf = tcount & 1;
        if (!(ok = mbar_wait(&acc_empty[buf], ((tcount >> 1) & 1u) ^ 1u, abort_flag))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * (TCOLS / 2);
        for (int kb = 0; kb < KB; ++kb) {
          if (!(ok = mbar_spin_wait(&full[st.s], st.ph, abort_flag))) break;
          tc_fence_after();
          const uint64_t adesc = smem_desc_sw128(smem_u32(sA + st.s * A_BYTES));
          const uint64_t bdesc = smem_desc_sw128(smem_u32(sB + st.s * B_BYTES));
#pragma unroll
          for (int k4 = 0; k4 < kBfBK / 32; ++k4)  // 16 bf16 = 32 bytes of K per instruction
            mma_bf16_ss(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
          mma_commit(&empty[st.s]);
          st.next(NS);
        }
        if (ok) mma_commit(&acc_full[buf]);
      }
    }
  } else {
    // ================= epilogue: quadrant (warp & 3), column half (ew >> 2) =================
    const int ew = warp - kEpiWarp0, qd = warp & 3;
    constexpr int NCOLS = BN >= 64 ? BN / 2 : BN;  // columns per warp
    const int col0 = (ew >> 2) * NCOLS;
    float* tb = s_bias + ew * 128;
    const bool wide = ((reinterpret_cast<uintptr_t>(p.y) | static_cast<uintptr_t>(p.ldy * 2)) & 31u) == 0;
    bool ok = true;
    int tcount = 0, staged = -1;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int buf = tcount & 1;
      const int n0 = (tile % p.n_tiles) * BN + col0;
      const int64_t row = static_cast<int64_t>(tile / p.n_tiles) * BM + qd * 32 + lane;
      if (n0 != staged) {
        __syncwarp();
        for (int c = lane; c < NCOLS; c += 32)
          tb[c] = p.bias != nullptr ? __uint_as_float(static_cast<uint32_t>(__ldg(p.bias + n0 + c)) << 16) : 0.0f;
        __syncwarp();
        staged = n0;
      }
      ok = mbar_wait(&acc_full[buf], (tcount >> 1) & 1u, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + buf * (TCOLS / 2) + col0;
      uint16_t* yrow = p.y + row * p.ldy + n0;
      uint32_t ra[16];
      tmem_ld_32x16(t_addr, ra);
      for (int c = 0; c < NCOLS / 16; ++c) {
        tmem_ld_wait();
        uint32_t a[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] = ra[i];
        if (c + 1 < NCOLS / 16) {
          tmem_ld_32x16(t_addr + (c + 1) * 16, ra);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
        uint32_t w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float2 bb = *reinterpret_cast<const float2*>(tb + c * 16 + 2 * q);
          const __nv_bfloat162 v = __floats2bfloat162_rn(__fadd_rn(__uint_as_float(a[2 * q]), bb.x),
                                                         __fadd_rn(__uint_as_float(a[2 * q + 1]), bb.y));
          w[q] = *reinterpret_cast<const uint32_t*>(&v);
        }
        if (row < p.M) {
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
    tmem_dealloc(tmem_base, TCOLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicExch(p.status, DP_ERR_TIMEOUT);
}

// ---- host side -------------------------------------------------------------------------------------
template <int BN>
constexpr size_t bf_smem_bytes() {
  return 1024 + static_cast<size_t>(bf_stages(BN) > 8 ? 8 : bf_stages(BN)) * (BM + BN) * kBfBK + kEpiWarps * 128 * 4 +
         (2 * 8 + 4) * 8 + 64;
}

int gemm_bf16_init_device() {
  DP_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(bf_smem_bytes<64>())));
  DP_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(bf_smem_bytes<128>())));
  DP_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(bf_smem_bytes<256>())));
  return DP_OK;
}

// x bf16 [M][ldx], w bf16 [N][K] (row-major, K contiguous), bias bf16 [N] or null, y bf16 [M][ldy].
// N % 64 == 0, K % 128 == 0 (checked by the caller), pointers 16-byte aligned.
int launch_gemm_bf16(const void* x, int64_t ldx, const void* w, const uint16_t* bias, int64_t M, int32_t N, int32_t K,
                     uint16_t* y, int64_t ldy, int32_t* status, cudaStream_t stream, bool pdl) {
  if (M == 0) return DP_OK;
  const int bn = N % 256 == 0 ? 256 : N % 128 == 0 ? 128 : 64;
  CUtensorMap ta, tw;
  int st = gemm_encode_bytes_2d(&ta, x, static_cast<uint64_t>(K) * 2, static_cast<uint64_t>(M),
                                static_cast<uint64_t>(ldx) * 2, kBfBK, BM);
  if (st != DP_OK) return st;
  st = gemm_encode_bytes_2d(&tw, w, static_cast<uint64_t>(K) * 2, static_cast<uint64_t>(N), static_cast<uint64_t>(K) * 2,
                            kBfBK, bn);
  if (st != DP_OK) return st;
  BfParams p;
  p.bias = bias;
  p.y = y;
  p.ldy = ldy;
  p.M = M;
  p.N = N;
  p.K = K;
  p.m_tiles = static_cast<int32_t>((M + BM - 1) / BM);
  p.n_tiles = N / bn;
  p.status = status;
  const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
  const int sms = num_sms() > 0 ? num_sms() : 148;
  const dim3 grid(static_cast<unsigned>(tiles < sms ? tiles : sms)), block(kBfThreads);
  cudaError_t e;
  if (bn == 256) e = launch(gemm_bf16_kernel<256>, grid, block, bf_smem_bytes<256>(), stream, pdl, ta, tw, p);
  else if (bn == 128) e = launch(gemm_bf16_kernel<128>, grid, block, bf_smem_bytes<128>(), stream, pdl, ta, tw, p);
  else e = launch(gemm_bf16_kernel<64>, grid, block, bf_smem_bytes<64>(), stream, pdl, ta, tw, p);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "bf16 GEMM launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
