// Activation-stationary tensor-core path of the quantized linear for K <= 1152.
//
//   Step 5 / Implementation of the paper: INT8 x INT8 -> INT32 GEMM with per-output-channel weight
//   scales, dequantised in the epilogue.
//
// A CTA pair (tcgen05 cta_group::2) takes a work unit = (strip of 256 tokens, slice of the output
// channels). Each CTA keeps ITS 128 tokens' int8 codes for the whole K resident in shared memory
// (up to 9 k-blocks of 16 KB, fetched once per strip) and the pair walks the slice in sub-blocks of
// `bns` channels: only weight tiles stream through the TMA ring, each CTA fetching half of a
// sub-block's rows (bns / 2 x 128 bytes per k-block), and the accumulators of consecutive
// sub-blocks alternate between two tensor-memory buffers so that a sub-block's epilogue runs under
// the next one's MMAs. Per MAC a CTA fetches 1 / (2 x 128) byte of weights and, amortised over the
// slice, 1 / slice-width byte of activations: a quarter to a third of what the streaming kernels
// move from L2, which is what bounds those at a few thousand tokens (a layer is then one or two
// waves of tiles and every CTA re-reads its operands).
// Units are numbered strip-major and cut into equal contiguous runs, one per pair: with few tokens
// (M = 2048: 8 strips x 9 slices = 72 units on 74 pairs) a layer is exactly one wave; with many,
// consecutive units of a pair share the strip and the resident activations are kept.
//
// Warp roles: warp 0 TMA producer (one thread), warp 1 MMA issuer (one thread of the pair's leader),
// warps 2-9 epilogue (two per 32-token quadrant of tensor memory, half of the sub-block's columns each;
// one token per thread).
// All loads are plain (non-multicast) TMA loads; both CTAs' bytes are counted on the leader's
// barriers; tcgen05.commit frees ring stages in both CTAs.
#include "gemm_device.cuh"

namespace dp {

constexpr int kAsMaxKB = 9;      // k-blocks of 128 a resident strip may have (K <= 1152)
constexpr int kAsMaxStages = 8;  // weight ring depth limit
constexpr int kAsRingBytes = 64 * 1024;
constexpr int kAsEpiWarps = kEpiWarps;  // two per 32-token quadrant of tensor memory, half of the columns each
constexpr int kAsThreads = (kEpiWarp0 + kAsEpiWarps) * 32;  // producer, MMA, epilogue warps

struct AsParams {
  int32_t bns;             // sub-block width in output channels (64, 128, 192 or 256)
  int32_t nsub;            // sub-blocks per slice
  int32_t n_slices;        // N / (bns * nsub)
  int32_t units;           // strips * n_slices
  int32_t units_per_pair;  // contiguous run of units per pair
  int32_t stages;          // weight ring depth
};

__global__ void __launch_bounds__(kAsThreads, 1)
gemm_as_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
               const GemmParams p, const AsParams ap) {
  constexpr int A_BYTES = BM * BK;
  constexpr int TCOLS = 512;
  const int B_BYTES = (ap.bns >> 1) * BK;  // this CTA's half of a sub-block's weight rows, one k-block
  const int NS = ap.stages;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                        // [KB][128 tokens][128] int8, 128-byte swizzled: the strip
  uint8_t* sB = sA + kAsMaxKB * A_BYTES;     // weight ring
  float* s_scale = reinterpret_cast<float*>(sB + kAsRingBytes);  // per-warp fp32 copies of weight scales and biases
  uint64_t* a_full = reinterpret_cast<uint64_t*>(sB + kAsRingBytes + kAsEpiWarps * RowEpilogue<0>::kScaleBytes);  // leader: both CTAs' k-block landed
  uint64_t* w_full = a_full + kAsMaxKB;                                      // leader: both CTAs' stage landed
  uint64_t* w_empty = w_full + kAsMaxStages;                                 // every MMA reading the stage completed
  uint64_t* acc_full = w_empty + kAsMaxStages;
  uint64_t* acc_empty = acc_full + 2;  // leader's copy collects both CTAs' epilogue warps
  uint64_t* a_free = acc_empty + 2;    // every MMA reading the resident strip completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(a_free + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = p.K / BK;
  const uint32_t rank = cluster_ctarank();
  const int unit0 = static_cast<int>(blockIdx.x >> 1) * ap.units_per_pair;
  const int unit1 = min(ap.units, unit0 + ap.units_per_pair);
  const int slice_w = ap.bns * ap.nsub;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kAsMaxKB; ++i) mbar_init(&a_full[i], 2);
    for (int i = 0; i < kAsMaxStages; ++i) {
      mbar_init(&w_full[i], 2);
      mbar_init(&w_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 2 * kAsEpiWarps);  // one arrival per epilogue warp of both CTAs
    }
    mbar_init(a_free, 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_w);
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, TCOLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();  // both CTAs' barriers exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_launch_dependents();

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      Ring st;
      bool ok = true;
      bool open = !p.early_w;  // false until griddepcontrol.wait has been executed
      if (open) pdl_wait();
      int cur_strip = -1, strips = 0;
      const uint32_t w_full0 = map_to_cta(&w_full[0], 0), a_full0 = map_to_cta(&a_full[0], 0);  // in the leader
      auto load_w = [&](int kb, int w_row) {
        const uint32_t bar = w_full0 + 8u * static_cast<uint32_t>(st.s);
        mbar_arrive_expect_tx_cluster(bar, static_cast<uint32_t>(B_BYTES));
        tma_load_2d_pair(sB + st.s * B_BYTES, &tmap_w, kb * BK, w_row, bar);
        st.next(NS);
      };
      auto load_a = [&](int kb, int m_row) {
        const uint32_t bar = a_full0 + 8u * static_cast<uint32_t>(kb);
        mbar_arrive_expect_tx_cluster(bar, A_BYTES);
        int c0, c1;
        a_tile_coords(p, m_row, kb, c0, c1);
        tma_load_2d_pair(sA + kb * A_BYTES, &tmap_a, c0, c1, bar);
      };
      for (int u = unit0; u < unit1 && ok; ++u) {
        const int strip = u / ap.n_slices, slice = u - strip * ap.n_slices;
        const bool new_strip = strip != cur_strip;
        const int m_row = strip * (2 * BM) + static_cast<int>(rank) * BM;
        if (new_strip) {
          // the resident strip may be overwritten once every MMA reading it has completed
          if (strips > 0 && !(ok = mbar_wait_cluster(a_free, (strips - 1) & 1u, abort_flag))) break;
          cur_strip = strip;
          ++strips;
        }
        for (int sub = 0; sub < ap.nsub && ok; ++sub) {
          const int w_row = slice * slice_w + sub * ap.bns + static_cast<int>(rank) * (ap.bns >> 1);
          const bool with_a = new_strip && sub == 0;
          const int lead = min(NS, KB);  // weight stages that can be in flight before any is consumed
          for (int kb = 0; kb < KB; ++kb) {
            if (!(ok = mbar_spin_wait(&w_empty[st.s], st.ph ^ 1u, abort_flag))) break;
            if (with_a && open && kb < lead) load_a(kb, m_row);
            load_w(kb, w_row);
            if (with_a && kb == lead - 1) {
              // weights (constants) may go first while the kernel that produces the activations drains
              if (!open) {
                pdl_wait();
                open = true;
                for (int k2 = 0; k2 < lead; ++k2) load_a(k2, m_row);
              }
              for (int k2 = lead; k2 < KB; ++k2) load_a(k2, m_row);
            }
          }
        }
      }
      if (!open) pdl_wait();
      if (!ok) {  // give copies still in flight a bounded time to land before the CTA exits
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) {
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ================= MMA issuer (leader) =================
      const uint32_t idesc = idesc_i8(2 * BM, ap.bns);
      const uint64_t a_desc0 = smem_desc_sw128(smem_u32(sA));
      const uint64_t b_desc0 = smem_desc_sw128(smem_u32(sB));
      const uint32_t b_step = static_cast<uint32_t>(B_BYTES) >> 4;
      Ring st;
      bool ok = true;
      int g = 0, cur_strip = -1, strips = 0;
      for (int u = unit0; u < unit1 && ok; ++u) {
        const int strip = u / ap.n_slices;
        const bool new_strip = strip != cur_strip;
        if (new_strip) {
          cur_strip = strip;
          ++strips;
        }
        for (int sub = 0; sub < ap.nsub && ok; ++sub, ++g) {
          const int buf = g & 1;
          if (!(ok = mbar_wait_cluster(&acc_empty[buf], ((g >> 1) & 1u) ^ 1u, abort_flag))) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * (TCOLS / 2);
          for (int kb = 0; kb < KB; ++kb) {
            if (new_strip && sub == 0) {
              if (!(ok = mbar_spin_wait(&a_full[kb], (strips - 1) & 1u, abort_flag))) break;
            }
            if (!(ok = mbar_spin_wait(&w_full[st.s], st.ph, abort_flag))) break;
            tc_fence_after();
            const uint64_t adesc = a_desc0 + static_cast<uint64_t>(kb * (A_BYTES >> 4));
            const uint64_t bdesc = b_desc0 + static_cast<uint64_t>(st.s * b_step);
#pragma unroll
            for (int k4 = 0; k4 < BK / 32; ++k4)
              mma_i8_ss_pair(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
            mma_commit_pair(&w_empty[st.s]);
            st.next(NS);
          }
          if (!ok) break;
          mma_commit_pair(&acc_full[buf]);
        }
        if (!ok) break;
        if (u + 1 < unit1 && (u + 1) / ap.n_slices != cur_strip) mma_commit_pair(a_free);
      }
    }
  } else {
    // ================= epilogue =================
    const int ew = warp - kEpiWarp0;
    RowEpilogue<0> epi;
    epi.init(warp, lane, s_scale + ew * (RowEpilogue<0>::kScaleBytes / 4), map_to_cta(&acc_empty[0], 0),
             map_to_cta(&acc_empty[1], 0));
    const int ncols = ap.bns >> 1, col0 = (ew >> 2) * ncols;  // this warp's half of a sub-block's columns
    bool ok = true;
    int g = 0;
    pdl_wait();  // s_a is written by the preceding kernel
    for (int u = unit0; u < unit1 && ok; ++u) {
      const int strip = u / ap.n_slices, slice = u - strip * ap.n_slices;
      for (int sub = 0; sub < ap.nsub && ok; ++sub, ++g) {
        const int buf = g & 1;
        ok = epi.tile(p, slice * slice_w + sub * ap.bns + col0, ncols,
                      strip * (2 * BM) + static_cast<int>(rank) * BM, tmem_base, buf * (TCOLS / 2) + col0,
                      &acc_full[buf], (g >> 1) & 1u, buf, abort_flag);
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  cluster_sync();  // neither CTA frees tensor memory or exits while the other may still touch it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TCOLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicExch(p.status, DP_ERR_TIMEOUT);
}

// ---- host side -------------------------------------------------------------------------------------
constexpr size_t as_smem_bytes() {
  return 1024 + static_cast<size_t>(kAsMaxKB) * BM * BK + kAsRingBytes +
         kAsEpiWarps * RowEpilogue<0>::kScaleBytes +
         (kAsMaxKB + 2 * kAsMaxStages + 5) * 8 + 64;
}

int gemm_as_init_device() {
  DP_CUDA_OK(cudaFuncSetAttribute(gemm_as_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  static_cast<int>(as_smem_bytes())));
  return DP_OK;
}

bool gemm_as_supported(int32_t N, int32_t K) { return K <= kAsMaxKB * BK && N % 64 == 0; }

// Sub-block width and sub-blocks per slice for this problem: among the widths that tile N, the
// (bns, nsub) with the least modelled time = waves of units over the pairs x (the slice's MMA time
// + a fixed per-unit cost for fetching the strip and draining the last sub-block), in k-block
// clocks of a 256-wide sub-block.
void gemm_as_config(int64_t M, int32_t N, int32_t K, int forced_bns, int* bns_out, int* nsub_out) {
  (void)K;
  const int64_t pairs = gemm_max_pairs() > 0 ? gemm_max_pairs() : 74;
  const int64_t strips = (M + 2 * BM - 1) / (2 * BM);
  const int widths[4] = {256, 192, 128, 64};
  double best = 1e30;
  *bns_out = 0;
  *nsub_out = 1;
  for (int i = 0; i < 4; ++i) {
    const int bns = widths[i];
    if (N % bns || (forced_bns && bns != forced_bns)) continue;
    for (int nsub = 1; nsub <= 8; ++nsub) {
      if ((N / bns) % nsub) continue;
      const int64_t units = strips * (N / (bns * nsub));
      const int64_t per_pair = (units + pairs - 1) / pairs;
      // a narrow sub-block keeps the tensor core less busy per weight byte; the last sub-block's
      // epilogue is exposed
      const double sub_time = bns + (bns < 128 ? 48.0 : bns < 256 ? 16.0 : 0.0);
      const double cost = static_cast<double>(per_pair) * (nsub * sub_time + 96.0 + 0.25 * bns);
      if (cost < best) {
        best = cost;
        *bns_out = bns;
        *nsub_out = nsub;
      }
    }
  }
}

int launch_gemm_as(const GemmProblem& g, cudaStream_t stream, bool pdl) {
  if (g.M == 0) return DP_OK;
  if (!gemm_as_supported(g.N, g.K) || g.bits != 8 || g.x != nullptr || !g.a_tiled)
    return fail(DP_ERR_SHAPE, "activation-stationary kernel: unsupported N=%d K=%d bits=%d", g.N, g.K, g.bits);
  int bns = 0, nsub = 1;
  gemm_as_config(g.M, g.N, g.K, g.bn, &bns, &nsub);
  if (bns == 0 || bns != g.bn)
    return fail(DP_ERR_SHAPE, "activation-stationary kernel: sub-block width %d does not tile N=%d", g.bn, g.N);
  GemmParams p;
  p.s_a = g.s_a;
  p.s_w = g.s_w;
  p.bias = g.bias;
  p.y = g.y;
  p.ldy = g.ldy;
  p.dbg_acc = g.dbg_acc;
  p.dbg_ldacc = g.dbg_ldacc;
  p.res = nullptr;  // the residual epilogue is built for the streaming kernels only
  p.ldr = 0;
  p.gate = nullptr;
  p.rows_per_gate = 1;
  p.M = g.M;
  p.N = g.N;
  p.K = g.K;
  p.m_tiles = static_cast<int32_t>((g.M + 2 * BM - 1) / (2 * BM));
  p.n_tiles = g.N / bns;
  p.a_tiled = 1;
  p.x = nullptr;
  p.ldx = 0;
  p.q_out = nullptr;
  p.s_a_out = nullptr;
  p.sync = nullptr;
  p.sync_tiles = 0;
  p.early_w = (pdl && g.early_w) ? 1 : 0;
  p.status = g.status;
  AsParams ap;
  ap.bns = bns;
  ap.nsub = nsub;
  ap.n_slices = g.N / (bns * nsub);
  ap.units = p.m_tiles * ap.n_slices;
  const int64_t pairs = gemm_max_pairs() > 0 ? gemm_max_pairs() : num_sms() / 2;
  ap.units_per_pair = static_cast<int32_t>((ap.units + pairs - 1) / pairs);
  const int stage_bytes = (bns / 2) * BK;
  ap.stages = kAsRingBytes / stage_bytes > kAsMaxStages ? kAsMaxStages : kAsRingBytes / stage_bytes;
  const dim3 grid(static_cast<unsigned>(2 * ((ap.units + ap.units_per_pair - 1) / ap.units_per_pair)));
  const cudaError_t e = launch_cluster(gemm_as_kernel, grid, dim3(kAsThreads), as_smem_bytes(), stream, pdl, 2u,
                                       g.tmap_a, g.tmap_w, p, ap);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "activation-stationary GEMM launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
