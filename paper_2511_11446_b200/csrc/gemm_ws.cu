// Weight-stationary tensor-core path of the quantized linear for K <= 1152 and many tokens.
//
//   Step 5 / Implementation of the paper: INT8 x INT8 -> INT32 GEMM with per-output-channel weight
//   scales; Step 3: packed low-bit weights expanded on the fly.
//
// A CTA pair (tcgen05 cta_group::2) takes a strip of BN output channels, each CTA holding BN / 2 of
// its weight rows for the WHOLE K in shared memory (up to 9 k-blocks of 128: 144 KB at BN = 256),
// fetched -- and, for 3/4-bit layers, expanded to int8 -- once. The pair then walks a run of
// 256-token row tiles of that strip and streams only the activation tiles (16 KB per k-block and
// CTA) through a short TMA ring. Per MAC a CTA therefore fetches a quarter of the bytes of the
// single-CTA streaming kernel, and the expansion cost of packed weights is paid once per strip
// instead of once per tile. Work items (strip, row tile) are numbered strip-major and cut into
// equal contiguous runs, one per pair; a run that crosses a strip boundary reloads the strip.
//
// Warp roles as in the streaming kernel: warp 0 TMA producer, warp 1 MMA issuer (leader CTA) or
// stage reporter (the other CTA), warps 2-9 epilogue, warps 10-17 weight expansion (3/4-bit).
// Packed tiles are staged through the (then idle) activation ring slots.
#include "gemm_device.cuh"

namespace dp {

constexpr int kWsMaxKB = 9;   // k-blocks of 128 a resident strip may have (K <= 1152)
// Activation ring depth: what is left of shared memory beside the resident strip.
__host__ __device__ constexpr int ws_stages(int bn) { return bn >= 256 ? 4 : 6; }

template <int BN, int BITS, bool PERM>
__global__ void __launch_bounds__(gemm_threads(BITS), 1)
gemm_ws_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
               const GemmParams p, const int items_per_pair) {
  constexpr int CG = 2;
  constexpr int BNL = BN / CG;  // weight rows held by this CTA
  constexpr int NS = ws_stages(BN);
  constexpr int A_BYTES = BM * BK, B_BYTES = BNL * BK, P_BYTES = p_stage_bytes(BNL, BITS);
  constexpr int TCOLS = 512;
  constexpr int SHIFT = 8 - BITS;
  static_assert(P_BYTES <= A_BYTES, "a packed tile must fit an activation ring slot");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sW = smem;                            // [KB][BNL][128] int8, 128-byte swizzled: the strip
  uint8_t* sA = sW + kWsMaxKB * B_BYTES;         // activation ring (and packed-tile staging)
  float* s_scale = reinterpret_cast<float*>(sA + NS * A_BYTES);  // per epilogue warp: fp32 copies of scales, biases
  uint64_t* full_a = reinterpret_cast<uint64_t*>(s_scale + kEpiWarps * (RowEpilogue<SHIFT>::kScaleBytes / 4));
  uint64_t* empty = full_a + NS;
  uint64_t* peer_ready = empty + NS;  // leader only
  uint64_t* pfull = peer_ready + NS;
  uint64_t* pempty = pfull + NS;
  uint64_t* acc_full = pempty + NS;
  uint64_t* acc_empty = acc_full + 2;  // leader's copy collects both CTAs' epilogue warps
  uint64_t* w_full = acc_empty + 2;    // this CTA's half of the strip is in place
  uint64_t* w_peer = w_full + 1;       // leader only: the other CTA's half is in place
  uint64_t* w_free = w_peer + 1;       // every MMA that reads the current strip has completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(w_free + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = p.K / BK;
  const uint32_t rank = cluster_ctarank();
  const int total_items = p.m_tiles * p.n_tiles;
  const int item0 = (blockIdx.x / CG) * items_per_pair;
  const int item1 = min(total_items, item0 + items_per_pair);
  // item -> (strip, row tile): strip-major
  auto strip_of = [&](int item) { return item / p.m_tiles; };
  auto mtile_of = [&](int item) { return item % p.m_tiles; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_a[i], CG);  // leader's copy: one arrival (+ bytes) from each CTA's producer
      mbar_init(&empty[i], 1);
      mbar_init(&peer_ready[i], 1);
      mbar_init(&pfull[i], 1);
      mbar_init(&pempty[i], kUnpackThreads);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], CG * kEpiWarps);
    }
    mbar_init(w_full, BITS == 8 ? 1 : kUnpackThreads);
    mbar_init(w_peer, 1);
    mbar_init(w_free, 1);
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
  if (!p.early_w) pdl_wait();

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      Ring st, pr;
      bool ok = true, a_open = !p.early_w || p.x != nullptr;
      int cur_strip = -1, strips = 0, ready_tile = -1;
      for (int item = item0; item < item1 && ok; ++item) {
        const int strip = strip_of(item);
        if (strip != cur_strip) {
          // the previous strip may be overwritten once every MMA reading it has completed; by then
          // every activation slot has been consumed as well
          if (strips > 0 && !(ok = mbar_wait(w_free, (strips - 1) & 1u, abort_flag))) break;
          const int w_row = strip * BN + static_cast<int>(rank) * BNL;
          if constexpr (BITS == 8) {
            mbar_arrive_expect_tx(w_full, KB * B_BYTES);
            for (int kb = 0; kb < KB; ++kb) tma_load_2d(sW + kb * B_BYTES, &tmap_w, kb * BK, w_row, w_full);
          } else {
            for (int kb = 0; kb < KB && ok; ++kb) {
              if (!(ok = mbar_wait(&pempty[pr.s], pr.ph ^ 1u, abort_flag))) break;
              mbar_arrive_expect_tx(&pfull[pr.s], P_BYTES);
              tma_load_2d(sA + pr.s * A_BYTES, &tmap_w, kb * (BK * BITS / 8), w_row, &pfull[pr.s]);
              pr.next(NS);
            }
            // activation tiles reuse these slots: wait until the expansion warps have read them all
            Ring d = pr;
            for (int i = 0; i < NS && ok; ++i) {
              ok = mbar_wait(&pempty[d.s], d.ph ^ 1u, abort_flag);
              d.next(NS);
            }
            if (!ok) break;
          }
          cur_strip = strip;
          ++strips;
        }
        if (!a_open) {  // activations come from the preceding kernel on the stream
          pdl_wait();
          a_open = true;
        }
        const int m_row = mtile_of(item) * (BM * CG) + static_cast<int>(rank) * BM;
        if (p.x != nullptr && (m_row >> 7) != ready_tile) {  // in-kernel DAQ: this tile's tokens are quantized
          if (p.early_w && ready_tile < 0) pdl_wait();  // until the preceding kernel has exited the counters
                                                       // still hold ITS tiles' counts
          if (!(ok = wait_tile_quantized(p, m_row >> 7, abort_flag))) break;
          ready_tile = m_row >> 7;
        }
        for (int kb = 0; kb < KB; ++kb) {
          if (!(ok = mbar_spin_wait(&empty[st.s], st.ph ^ 1u, abort_flag))) break;
          // both CTAs' activation tiles are counted on the LEADER's barrier: the MMA thread waits once
          const uint32_t bar = map_to_cta(&full_a[st.s], 0);
          mbar_arrive_expect_tx_cluster(bar, A_BYTES);
          int c0, c1;
          a_tile_coords(p, m_row, kb, c0, c1);
          tma_load_2d_pair(sA + st.s * A_BYTES, &tmap_a, c0, c1, bar);
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
      if (rank != 0) {
        // ================= pair follower: report each resident strip to the leader =================
        bool ok = true;
        int cur_strip = -1, strips = 0;
        for (int item = item0; item < item1 && ok; ++item) {
          if (strip_of(item) != cur_strip) {
            if (!(ok = mbar_wait(w_full, strips & 1u, abort_flag))) break;
            mbar_arrive_cluster(map_to_cta(w_peer, 0));
            cur_strip = strip_of(item);
            ++strips;
          }

        }
      } else {
        // ================= MMA issuer =================
        constexpr uint32_t idesc = idesc_i8(BM * CG, BN);
        Ring st;
        bool ok = true;
        int tcount = 0, cur_strip = -1, strips = 0;
        for (int item = item0; item < item1 && ok; ++item, ++tcount) {
          if (strip_of(item) != cur_strip) {
            if (!(ok = mbar_wait(w_full, strips & 1u, abort_flag))) break;
            if (!(ok = mbar_wait_cluster(w_peer, strips & 1u, abort_flag))) break;
            cur_strip = strip_of(item);
            ++strips;
          }
          const int buf = tcount & 1;
          const uint32_t aph = (tcount >> 1) & 1;
          if (!(ok = mbar_wait_cluster(&acc_empty[buf], aph ^ 1u, abort_flag))) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * (TCOLS / 2);
          for (int kb = 0; kb < KB; ++kb) {
            if (!(ok = mbar_spin_wait(&full_a[st.s], st.ph, abort_flag))) break;  // both CTAs' tiles landed
            tc_fence_after();
            const uint64_t adesc = smem_desc_sw128(smem_u32(sA + st.s * A_BYTES));
            const uint64_t bdesc = smem_desc_sw128(smem_u32(sW + kb * B_BYTES));
#pragma unroll
            for (int k4 = 0; k4 < BK / 32; ++k4)
              mma_i8_ss_pair(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
            mma_commit_pair(&empty[st.s]);
            st.next(NS);
          }
          if (!ok) break;
          mma_commit_pair(&acc_full[buf]);
          if (item + 1 < item1 && strip_of(item + 1) != cur_strip) mma_commit_pair(w_free);
        }
      }
    }
  } else if (warp < kUnpackWarp0) {
    // ================= epilogue: quadrant (warp & 3), column half (ew >> 2) =================
    const int ew = warp - kEpiWarp0;
    RowEpilogue<SHIFT> epi;
    epi.init(warp, lane, s_scale + ew * (RowEpilogue<SHIFT>::kScaleBytes / 4), map_to_cta(&acc_empty[0], 0),
             map_to_cta(&acc_empty[1], 0));
    constexpr int NCOLS = BN / 2;
    const int col0 = (ew >> 2) * NCOLS;
    if (p.x != nullptr) {  // quantize this CTA's share of the tokens first (all eight warps)
      if (p.early_w) pdl_wait();
      daq_phase<PERM>(p, ew, lane);
    }
    bool ok = true;
    int tcount = 0;
    if (p.early_w && p.x == nullptr) pdl_wait();  // s_a is written by the preceding kernel
    for (int item = item0; item < item1 && ok; ++item, ++tcount) {
      const int buf = tcount & 1;
      ok = epi.tile(p, strip_of(item) * BN + col0, NCOLS, mtile_of(item) * (BM * CG) + static_cast<int>(rank) * BM,
                    tmem_base, buf * (TCOLS / 2) + col0, &acc_full[buf], (tcount >> 1) & 1, buf, abort_flag);
    }
  } else {
    // ================= weight expansion (3/4-bit): once per strip =================
    if constexpr (BITS != 8) {
      const int ut = threadIdx.x - kUnpackWarp0 * 32;
      Ring pr;
      bool ok = true;
      int cur_strip = -1, strips = 0;
      for (int item = item0; item < item1 && ok; ++item) {
        if (strip_of(item) == cur_strip) continue;
        if (strips > 0) {
          ok = mbar_wait(w_free, (strips - 1) & 1u, abort_flag);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
        }
        for (int kb = 0; kb < KB; ++kb) {
          ok = mbar_wait(&pfull[pr.s], pr.ph, abort_flag);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          if constexpr (BITS == 4) unpack4_tile<BNL, PERM>(sA + pr.s * A_BYTES, sW + kb * B_BYTES, ut);
          else unpack3_tile<BNL>(sA + pr.s * A_BYTES, sW + kb * B_BYTES, ut);
          mbar_arrive(&pempty[pr.s]);
          pr.next(NS);
        }
        if (!ok) break;
        fence_proxy_async_smem();
        mbar_arrive(w_full);
        cur_strip = strip_of(item);
        ++strips;
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TCOLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicExch(p.status, DP_ERR_TIMEOUT);
  if (threadIdx.x == 0 && p.x != nullptr) daq_sync_exit(p);
}

// ---- host side -------------------------------------------------------------------------------------
template <int BN>
constexpr size_t ws_smem_bytes() {
  return 1024 + static_cast<size_t>(kWsMaxKB) * (BN / 2) * BK + ws_stages(BN) * BM * BK +
         kEpiWarps * RowEpilogue<0>::kScaleBytes + (5 * ws_stages(BN) + 4 + 3) * 8 + 32 + 64;
}

template <int BN, int BITS, bool PERM>
static cudaError_t ws_set_attr() {
  return cudaFuncSetAttribute(gemm_ws_kernel<BN, BITS, PERM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(ws_smem_bytes<BN>()));
}

int gemm_ws_init_device() {  // per device, from gemm_init_device
#define DP_SET(BN)                                \
  DP_CUDA_OK((ws_set_attr<BN, 8, false>()));      \
  DP_CUDA_OK((ws_set_attr<BN, 4, false>()));      \
  DP_CUDA_OK((ws_set_attr<BN, 4, true>()));       \
  DP_CUDA_OK((ws_set_attr<BN, 3, false>()));
  DP_SET(192) DP_SET(256)
#undef DP_SET
  return DP_OK;
}

bool gemm_ws_supported(int32_t N, int32_t K) { return K <= kWsMaxKB * BK && (N % 256 == 0 || N % 192 == 0); }
int gemm_ws_pick_bn(int32_t N) { return N % 256 == 0 ? 256 : 192; }

template <int BN>
static cudaError_t ws_launch_bn(const GemmProblem& g, const GemmParams& p, int items_per_pair, dim3 grid,
                                cudaStream_t stream, bool pdl) {
  const dim3 block(gemm_threads(g.bits));
  const size_t smem = ws_smem_bytes<BN>();
  switch (g.bits) {
    case 8:
      return launch_cluster(gemm_ws_kernel<BN, 8, false>, grid, block, smem, stream, pdl, 2u, g.tmap_a, g.tmap_w, p,
                            items_per_pair);
    case 4:
      if (g.korder == KORDER_EVEN_ODD)
        return launch_cluster(gemm_ws_kernel<BN, 4, true>, grid, block, smem, stream, pdl, 2u, g.tmap_a, g.tmap_w, p,
                              items_per_pair);
      return launch_cluster(gemm_ws_kernel<BN, 4, false>, grid, block, smem, stream, pdl, 2u, g.tmap_a, g.tmap_w, p,
                            items_per_pair);
    default:
      return launch_cluster(gemm_ws_kernel<BN, 3, false>, grid, block, smem, stream, pdl, 2u, g.tmap_a, g.tmap_w, p,
                            items_per_pair);
  }
}

// g.bn is 192 or 256, g.tmap_w has a box of g.bn / 2 rows (as for the pair streaming kernel).
int launch_gemm_ws(const GemmProblem& g, cudaStream_t stream, bool pdl) {
  if (g.M == 0) return DP_OK;
  if (!gemm_ws_supported(g.N, g.K) || g.N % g.bn)
    return fail(DP_ERR_SHAPE, "weight-stationary kernel: unsupported N=%d K=%d bn=%d", g.N, g.K, g.bn);
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
  p.n_tiles = g.N / g.bn;
  p.a_tiled = g.a_tiled;
  p.x = g.x;
  p.ldx = g.ldx;
  p.q_out = g.q_out;
  p.s_a_out = g.s_a_out;
  p.sync = g.sync;
  p.sync_tiles = static_cast<int32_t>((g.M + BM - 1) / BM);
  p.early_w = (pdl && g.early_w) ? 1 : 0;
  p.status = g.status;
  const int64_t items = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
  const int64_t pairs = gemm_max_pairs() > 0 ? gemm_max_pairs() : num_sms() / 2;
  const int per_pair = static_cast<int>((items + pairs - 1) / pairs);
  const dim3 grid(static_cast<unsigned>(2 * ((items + per_pair - 1) / per_pair)));
  const cudaError_t e = g.bn == 256 ? ws_launch_bn<256>(g, p, per_pair, grid, stream, pdl)
                                    : ws_launch_bn<192>(g, p, per_pair, grid, stream, pdl);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "weight-stationary GEMM launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
