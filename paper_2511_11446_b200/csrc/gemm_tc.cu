// Tensor-core path of the quantized linear: Y = dequant(Xq . unpack(Wp)^T) + bias on sm_100a.
//
//   Step 5 / Implementation of the paper: INT8 x INT8 -> INT32 GEMM with per-output-channel weight
//   scales; Step 3: weights are GPTQ-style packed low-bit integers, expanded on the fly.
//
// One persistent CTA per SM walks a static list of output tiles. CG = 1: a CTA owns 128 x BN tiles.
// CG = 2: the two CTAs of a thread-block cluster own a 256 x BN tile together (tcgen05 cta_group::2):
// each loads its own 128 token rows and only ITS half of the BN weight rows (plain TMA loads, no
// multicast), the pair's leader issues one MMA per 32 bytes of K that reads both CTAs' shared
// memory, and each CTA ends up with its 128 x BN accumulator in its own tensor memory. Per CTA this
// halves the weight bytes fetched, expanded and read by the tensor core for the same MACs.
// Warp roles:
//   warp 0      TMA producer: int8 activation tiles (128-byte-swizzled) and packed weight tiles
//   warp 1      MMA issuer: tcgen05.mma kind::i8, int32 accumulators in tensor memory (two
//               accumulator buffers, so a tile's epilogue overlaps the next tile's mainloop)
//   warps 2-9   epilogue: tcgen05.ld -> (float)acc * s_a[m]*s_w[n] + bias -> bf16 -> global; two warps
//               per 32-token TMEM quadrant, each taking half of the tile's columns, one token per
//               thread and one 32-byte store per 16 columns
//   warps 10-17 unpack (3/4-bit only): packed tile in smem -> int8 operand tile in smem, written in
//               the swizzled layout the MMA descriptor expects, then fence.proxy.async
//
// K order. The contraction over k does not care in which order the k's of a 128-wide block sit in
// the two operand tiles as long as both agree. With PERM the activations arrive (from the DAQ
// kernel of the same call) with every group of 8 codes stored as k = 0,2,4,6,1,3,5,7, which is the
// order two mask operations leave the nibbles of a 4-bit word in, so the expansion needs no byte
// shuffles.
//
// Low-bit codes are expanded as w * 2^(8-b) (the two's-complement field moved to the top of the
// byte: two logic ops per word instead of a sign-extension); the accumulator is then an exact
// multiple of 2^(8-b) (|acc| <= 4608*127*128 < 2^31) and the epilogue multiplies by 2^-(8-b),
// which is exact in fp32, before the scale.
#include "gemm_device.cuh"

namespace dp {

// ---- the kernel ----------------------------------------------------------------------------------
template <int BN, int BITS, bool PERM, int CG, bool RES = false>
__global__ void __launch_bounds__(gemm_threads(BITS), 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
               const GemmParams p) {
  constexpr int BNL = BN / CG;  // weight rows held by this CTA
  constexpr int NS = num_stages(BNL, BITS);
  constexpr int NP = kPStages;
  constexpr int A_BYTES = BM * BK, B_BYTES = BNL * BK, P_BYTES = p_stage_bytes(BNL, BITS);
  constexpr int TCOLS = tmem_cols(BN);
  constexpr int SHIFT = 8 - BITS;  // accumulator carries a factor 2^SHIFT

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = sA + NS * A_BYTES;
  uint8_t* sP = sB + NS * B_BYTES;
  float* s_scale = reinterpret_cast<float*>(sP + NP * P_BYTES);  // per epilogue warp: fp32 copies of its columns' scales, biases
  uint64_t* full_a = reinterpret_cast<uint64_t*>(s_scale + kEpiWarps * (RowEpilogue<SHIFT>::kScaleBytes / 4));
  uint64_t* bready = full_a + NS;
  uint64_t* empty = bready + NS;
  uint64_t* peer_ready = empty + NS;  // pair leader only: the other CTA's stage is loaded (and expanded)
  uint64_t* pfull = peer_ready + NS;
  uint64_t* pempty = pfull + NP;
  uint64_t* acc_full = pempty + NP;
  uint64_t* acc_empty = acc_full + 2;  // CG = 2: the leader's copy collects both CTAs' epilogue warps
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = p.K / BK;
  const int total_tiles = p.m_tiles * p.n_tiles;
  const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;  // 0 = leader of the pair
  const int first_tile = blockIdx.x / CG, tile_stride = gridDim.x / CG;
  // TMA loads of operand stages: in a pair both CTAs' bytes are counted on the leader's barrier
  auto stage_expect = [&](uint64_t* bar, uint32_t bytes) {
    if constexpr (CG == 2) mbar_arrive_expect_tx_cluster(map_to_cta(bar, 0), bytes);
    else mbar_arrive_expect_tx(bar, bytes);
  };
  auto stage_load = [&](void* dst, const CUtensorMap* tm, int c0, int c1, uint64_t* bar) {
    if constexpr (CG == 2) tma_load_2d_pair(dst, tm, c0, c1, map_to_cta(bar, 0));
    else tma_load_2d(dst, tm, c0, c1, bar);
  };

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_a[i], CG);  // pair: the leader's copy counts both CTAs' TMA loads
      mbar_init(&bready[i], kUnpackThreads);
      mbar_init(&empty[i], 1);
      mbar_init(&peer_ready[i], 1);
    }
    for (int i = 0; i < NP; ++i) {
      mbar_init(&pfull[i], 1);
      mbar_init(&pempty[i], kUnpackThreads);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], CG * kEpiWarps);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_w);
  }
  if (warp == 1) {
    if constexpr (CG == 2) {
      tmem_alloc_pair(tmem_slot, TCOLS);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(tmem_slot, TCOLS);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (CG == 2) cluster_sync();  // both CTAs' barriers exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_launch_dependents();
  if (threadIdx.x == kEpiWarp0 * 32) {  // an epilogue thread: idle until the first accumulators
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const uint32_t off = blockIdx.x * p.pf_slice[r];
      if (p.pf[r] != nullptr && off < p.pf_bytes[r]) {
        const uint32_t n = min(p.pf_slice[r], p.pf_bytes[r] - off);
        for (uint32_t o = 0; o < n; o += 32768u) bulk_prefetch_l2(p.pf[r] + off + o, min(32768u, n - o));
      }
    }
  }
  // Activations and their scales come from the preceding kernel on the stream: the roles that read
  // them wait for it (griddepcontrol.wait) right before their first such read. Weights are
  // constants; unless early_w is set, everything waits here.
  if (!p.early_w) pdl_wait();

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      Ring st, ps;
      bool ok = true;
      bool a_open = !p.early_w || p.x != nullptr;  // false until griddepcontrol.wait has been executed
      int ready_tile = -1;                          // in-kernel DAQ: last 128-token tile seen complete
      int deferred = 0;          // stages whose weight tile is in flight but whose A tile is not
      int def_kb[NS], def_m[NS], def_s[NS];
      for (int tile = first_tile; tile < total_tiles && ok; tile += tile_stride) {
        const int n_blk = tile % p.n_tiles;  // column tiles of one row strip run together
        const int m_row = (tile / p.n_tiles) * (BM * CG) + static_cast<int>(rank) * BM;
        const int w_row = n_blk * BN + static_cast<int>(rank) * BNL;
        bool a_ready = p.x == nullptr || (m_row >> 7) == ready_tile;
        for (int kb = 0; kb < KB; ++kb) {
          if constexpr (CG == 1 && BITS == 8) {
            // test hook: this stage gets no loads and no arrival, so its barrier never completes and
            // the bounded waits of the other roles run out
            if (kb == p.dbg_skip_kb && tile == first_tile) {
              st.next(NS);
              continue;
            }
          }
          if (!a_open && deferred == NS) {  // ring full of weight tiles: now wait for the activations
            pdl_wait();
            a_open = true;
            for (int d = 0; d < deferred; ++d) {
              int c0, c1;
              a_tile_coords(p, def_m[d], def_kb[d], c0, c1);
              stage_load(sA + def_s[d] * A_BYTES, &tmap_a, c0, c1, &full_a[def_s[d]]);
            }
            deferred = 0;
          }
          if (!(ok = mbar_spin_wait(&empty[st.s], st.ph ^ 1u, abort_flag))) break;
          if constexpr (BITS == 8) {
            stage_expect(&full_a[st.s], A_BYTES + B_BYTES);
            stage_load(sB + st.s * B_BYTES, &tmap_w, kb * BK, w_row, &full_a[st.s]);
          } else {
            if (!(ok = mbar_wait(&pempty[ps.s], ps.ph ^ 1u, abort_flag))) break;
            mbar_arrive_expect_tx(&pfull[ps.s], P_BYTES);
            tma_load_2d(sP + ps.s * P_BYTES, &tmap_w, kb * (BK * BITS / 8), w_row, &pfull[ps.s]);
            stage_expect(&full_a[st.s], A_BYTES);
            ps.next(NP);
          }
          if (a_open) {
            if (!a_ready) {  // weights of this stage are already in flight; now the tile's tokens
              if (p.early_w && ready_tile < 0) pdl_wait();  // until the preceding kernel has exited the
                                                           // counters still hold ITS tiles' counts
              if (!(ok = wait_tile_quantized(p, m_row >> 7, abort_flag))) break;
              ready_tile = m_row >> 7;
              a_ready = true;
            }
            int c0, c1;
            a_tile_coords(p, m_row, kb, c0, c1);
            stage_load(sA + st.s * A_BYTES, &tmap_a, c0, c1, &full_a[st.s]);
          } else {
            def_kb[deferred] = kb;
            def_m[deferred] = m_row;
            def_s[deferred] = st.s;
            ++deferred;
          }
          st.next(NS);
        }
      }
      if (!a_open) {  // fewer k-blocks than stages in the whole CTA
        pdl_wait();
        for (int d = 0; d < deferred; ++d) {
          int c0, c1;
          a_tile_coords(p, def_m[d], def_kb[d], c0, c1);
          stage_load(sA + def_s[d] * A_BYTES, &tmap_a, c0, c1, &full_a[def_s[d]]);
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
    if (lane == 0) {
      if (CG == 2 && rank != 0) {
        // ================= pair follower: report each expanded weight stage to the leader =================
        // (TMA loads of both CTAs are counted on the leader's barrier directly)
        if constexpr (BITS != 8) {
          Ring st;
          bool ok = true;
          for (int tile = first_tile; tile < total_tiles && ok; tile += tile_stride) {
            for (int kb = 0; kb < KB; ++kb) {
              if (!(ok = mbar_wait(&bready[st.s], st.ph, abort_flag))) break;
              mbar_arrive_cluster(map_to_cta(&peer_ready[st.s], 0));
              st.next(NS);
            }
          }
        }
      } else {
        // ================= MMA issuer =================
        constexpr uint32_t idesc = idesc_i8(BM * CG, BN);
        Ring st;
        bool ok = true;
        int tcount = 0;
        for (int tile = first_tile; tile < total_tiles && ok; tile += tile_stride, ++tcount) {
          const int buf = tcount & 1;
          const uint32_t aph = (tcount >> 1) & 1;
          if (!(ok = CG == 2 ? mbar_wait_cluster(&acc_empty[buf], aph ^ 1u, abort_flag)
                             : mbar_wait(&acc_empty[buf], aph ^ 1u, abort_flag)))
            break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * (TCOLS / 2);
          for (int kb = 0; kb < KB; ++kb) {
            if (!(ok = mbar_spin_wait(&full_a[st.s], st.ph, abort_flag))) break;
            if constexpr (BITS != 8) {
              if (!(ok = mbar_wait(&bready[st.s], st.ph, abort_flag))) break;
              if constexpr (CG == 2) {
                if (!(ok = mbar_wait_cluster(&peer_ready[st.s], st.ph, abort_flag))) break;
              }
            }
            tc_fence_after();
            const uint64_t adesc = smem_desc_sw128(smem_u32(sA + st.s * A_BYTES));
            const uint64_t bdesc = smem_desc_sw128(smem_u32(sB + st.s * B_BYTES));
#pragma unroll
            for (int k4 = 0; k4 < BK / 32; ++k4) {  // 32 bytes of K per instruction: +2 in 16-byte units
              if constexpr (CG == 2)
                mma_i8_ss_pair(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
              else
                mma_i8_ss(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
            }
            if constexpr (CG == 2) mma_commit_pair(&empty[st.s]);
            else mma_commit(&empty[st.s]);
            st.next(NS);
          }
          if (ok) {
            if constexpr (CG == 2) mma_commit_pair(&acc_full[buf]);
            else mma_commit(&acc_full[buf]);
          }
        }
      }
    }
  } else if (warp < kUnpackWarp0) {
    // ================= epilogue: quadrant (warp & 3), column half (ew >> 2) =================
    const int ew = warp - kEpiWarp0;
    RowEpilogue<SHIFT> epi;
    epi.init(warp, lane, s_scale + ew * (RowEpilogue<SHIFT>::kScaleBytes / 4),
             CG == 2 ? map_to_cta(&acc_empty[0], 0) : smem_u32(&acc_empty[0]),
             CG == 2 ? map_to_cta(&acc_empty[1], 0) : smem_u32(&acc_empty[1]));
    constexpr int NCOLS = BN / 2;
    const int col0 = (ew >> 2) * NCOLS;
    if (p.x != nullptr) {  // quantize this CTA's share of the tokens first (all eight warps)
      if (p.early_w) pdl_wait();  // x comes from the preceding kernel, whose GEMM may still read the scratch
      daq_phase<PERM>(p, ew, lane);
    }
    bool ok = true;
    int tcount = 0;
    if (p.early_w && p.x == nullptr) pdl_wait();  // s_a is written by the preceding kernel
    for (int tile = first_tile; tile < total_tiles && ok; tile += tile_stride, ++tcount) {
      const int buf = tcount & 1;
      ok = epi.template tile<RES>(p, (tile % p.n_tiles) * BN + col0, NCOLS,
                    (tile / p.n_tiles) * (BM * CG) + static_cast<int>(rank) * BM, tmem_base,
                    buf * (TCOLS / 2) + col0, &acc_full[buf], (tcount >> 1) & 1, buf, abort_flag);
    }
  } else {
    // ================= unpack (3/4-bit weights) =================
    if constexpr (BITS != 8) {
      const int ut = threadIdx.x - kUnpackWarp0 * 32;
      Ring st, ps;
      bool ok = true;
      for (int tile = first_tile; tile < total_tiles && ok; tile += tile_stride) {
        for (int kb = 0; kb < KB; ++kb) {
          ok = mbar_wait(&pfull[ps.s], ps.ph, abort_flag) &&
               mbar_wait(&empty[st.s], st.ph ^ 1u, abort_flag);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          if constexpr (BITS == 4) unpack4_tile<BNL, PERM>(sP + ps.s * P_BYTES, sB + st.s * B_BYTES, ut);
          else unpack3_tile<BNL>(sP + ps.s * P_BYTES, sB + st.s * B_BYTES, ut);
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
  if constexpr (CG == 2) cluster_sync();  // neither CTA frees tensor memory or exits while the other may still touch it
  if (warp == 1) {
    tc_fence_after();
    if constexpr (CG == 2) tmem_dealloc_pair(tmem_base, TCOLS);
    else tmem_dealloc(tmem_base, TCOLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicExch(p.status, DP_ERR_TIMEOUT);
  if (threadIdx.x == 0 && p.x != nullptr) daq_sync_exit(p);
}

// ---- host side -------------------------------------------------------------------------------------
template <int BN, int BITS, int CG>
constexpr size_t gemm_smem_bytes() {
  return 1024 + static_cast<size_t>(num_stages(BN / CG, BITS)) * ab_stage_bytes(BN / CG) +
         kPStages * p_stage_bytes(BN / CG, BITS) + kEpiWarps * RowEpilogue<0>::kScaleBytes +
         (4 * 8 + 2 * kPStages + 4) * 8 + 32 + 64;
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                              CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                              CUtensorMapFloatOOBfill);
static EncodeFn g_encode = nullptr;  // the driver's tensor-map encoder (one per process)

template <int BN, int BITS, bool PERM, int CG>
static cudaError_t set_attr() {
  if constexpr (BITS == 8) {  // the form with a residual in the epilogue exists for 8-bit operands only
    cudaError_t e = cudaFuncSetAttribute(gemm_i8_kernel<BN, 8, false, CG, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(gemm_smem_bytes<BN, 8, CG>()));
    if (e != cudaSuccess) return e;
  }
  return cudaFuncSetAttribute(gemm_i8_kernel<BN, BITS, PERM, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(gemm_smem_bytes<BN, BITS, CG>()));
}

int gemm_korder(int32_t bits) { return bits == 4 ? KORDER_EVEN_ODD : KORDER_NATURAL; }

// First use of device `dev` (current; called under the library's device lock): the kernels'
// shared-memory attributes, the SM count and how many CTA pairs of the widest pair kernel can be
// resident at once.
int gemm_init_device(int dev, int* num_sms_out, int* max_pairs_out) {
  if (g_encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess)
      return fail(DP_ERR_CUDA, "cuTensorMapEncodeTiled not available: %s", cudaGetErrorString(e));
    g_encode = reinterpret_cast<EncodeFn>(fn);
  }
  int sms = 0;
  DP_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
#define DP_SET(BN, CG)                               \
  DP_CUDA_OK((set_attr<BN, 8, false, CG>()));        \
  DP_CUDA_OK((set_attr<BN, 4, false, CG>()));        \
  DP_CUDA_OK((set_attr<BN, 4, true, CG>()));         \
  DP_CUDA_OK((set_attr<BN, 3, false, CG>()));
  DP_SET(64, 1) DP_SET(128, 1) DP_SET(192, 1) DP_SET(256, 1)
  DP_SET(128, 2) DP_SET(192, 2) DP_SET(256, 2)
#undef DP_SET
  int pairs = 0;
  {  // how many CTA pairs fit on the device at once (one CTA per SM)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(sms & ~1));
    cfg.blockDim = dim3(gemm_threads(4));
    cfg.dynamicSmemBytes = gemm_smem_bytes<256, 4, 2>();
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&pairs, gemm_i8_kernel<256, 4, true, 2>, &cfg);
    if (e != cudaSuccess) return fail(DP_ERR_CUDA, "cudaOccupancyMaxActiveClusters: %s", cudaGetErrorString(e));
  }
  int st = gemm_ws_init_device();
  if (st != DP_OK) return st;
  st = gemm_as_init_device();
  if (st != DP_OK) return st;
  st = gemm_bf16_init_device();
  if (st != DP_OK) return st;
  st = gemm_grp_init_device();
  if (st != DP_OK) return st;
  *num_sms_out = sms;
  *max_pairs_out = pairs;
  return DP_OK;
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

// Any row-major matrix seen as bytes: rows of inner_bytes at pitch_bytes, boxes of box_inner x box_rows
// bytes, 128-byte swizzle.
int gemm_encode_bytes_2d(CUtensorMap* out, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
                         uint32_t box_inner, uint32_t box_rows) {
  return encode_2d(out, base, inner_bytes, rows, pitch_bytes, box_inner, box_rows, true);
}

int gemm_encode_a(CUtensorMap* out, const int8_t* q, int64_t M, int64_t K, int64_t ldq) {
  return encode_2d(out, q, K, M, ldq, BK, BM, true);
}
int gemm_encode_a_tiled(CUtensorMap* out, const int8_t* q, int64_t M, int64_t K) {
  const uint64_t rows = static_cast<uint64_t>((M + BM - 1) / BM) * (K / BK) * BM;
  return encode_2d(out, q, BK, rows, BK, BK, BM, true);
}

// The box of the weight descriptor is what ONE CTA fetches per k-block: bn / cg rows.
int gemm_encode_w(CUtensorMap* out, const void* qweight, int32_t N, int32_t K, int32_t bits,
                  int32_t bn, int32_t cg) {
  const uint64_t row_bytes = static_cast<uint64_t>(K) * bits / 8;
  return encode_2d(out, qweight, row_bytes, N, row_bytes, BK * bits / 8, bn / cg, bits == 8);
}

// Tile shape: width from {256, 192, 128, 64} dividing N, rows 128 (one CTA) or 256 (a CTA pair),
// by a small time model: waves of tiles over the SMs (or pairs) times the tile's mainloop time plus
// a fixed per-tile cost; pairs move half the weight bytes per MAC and are preferred on ties.
void gemm_pick_tile(int64_t M, int32_t N, int32_t K, int32_t bits, uint32_t allow, int* bn_out, int* cg_out) {
  (void)K;
  (void)bits;
  const int sms = num_sms() > 0 ? num_sms() : 148;
  const int pairs = gemm_max_pairs() > 0 ? gemm_max_pairs() : sms / 2;
  const int cand[4] = {256, 192, 128, 64};
  int best_bn = 0, best_cg = 1;
  double best_cost = 1e30;
  for (int cg = 2; cg >= 1; --cg) {
    if (!(allow & (1u << cg))) continue;
    for (int i = 0; i < 4; ++i) {
      const int bn = cand[i];
      if (N % bn || (cg == 2 && bn < 128)) continue;
      const int64_t tiles = ((M + BM * cg - 1) / (BM * cg)) * (N / bn);
      const int64_t slots = cg == 2 ? pairs : sms;
      const int64_t waves = (tiles + slots - 1) / slots;
      const double cost = static_cast<double>(waves) * (bn + 24.0) * (cg == 2 ? 0.98 : 1.0);
      if (cost < best_cost) {
        best_cost = cost;
        best_bn = bn;
        best_cg = cg;
      }
    }
  }
  *bn_out = best_bn;
  *cg_out = best_cg;
}

template <int BN, int CG>
static cudaError_t launch_bn(const GemmProblem& g, const GemmParams& p, dim3 grid, cudaStream_t stream,
                             bool pdl) {
  const dim3 block(gemm_threads(g.bits));
  switch (g.bits) {
    case 8:
      if (g.res != nullptr)
        return launch_cluster(gemm_i8_kernel<BN, 8, false, CG, true>, grid, block, gemm_smem_bytes<BN, 8, CG>(), stream,
                              pdl, CG, g.tmap_a, g.tmap_w, p);
      return launch_cluster(gemm_i8_kernel<BN, 8, false, CG>, grid, block, gemm_smem_bytes<BN, 8, CG>(), stream,
                            pdl, CG, g.tmap_a, g.tmap_w, p);
    case 4:
      if (g.korder == KORDER_EVEN_ODD)
        return launch_cluster(gemm_i8_kernel<BN, 4, true, CG>, grid, block, gemm_smem_bytes<BN, 4, CG>(), stream,
                              pdl, CG, g.tmap_a, g.tmap_w, p);
      return launch_cluster(gemm_i8_kernel<BN, 4, false, CG>, grid, block, gemm_smem_bytes<BN, 4, CG>(), stream,
                            pdl, CG, g.tmap_a, g.tmap_w, p);
    default:
      return launch_cluster(gemm_i8_kernel<BN, 3, false, CG>, grid, block, gemm_smem_bytes<BN, 3, CG>(), stream,
                            pdl, CG, g.tmap_a, g.tmap_w, p);
  }
}

// Ranges a plan wants on their way into L2 (consumed by the calling thread's next launch_gemm).
static thread_local const void* g_pf_ptr[2] = {nullptr, nullptr};
static thread_local size_t g_pf_bytes[2] = {0, 0};
void gemm_set_next_reads(const void* w, size_t w_bytes, const void* x, size_t x_bytes) {
  g_pf_ptr[0] = w;
  g_pf_bytes[0] = w_bytes;
  g_pf_ptr[1] = x;
  g_pf_bytes[1] = x_bytes;
}

// dp_debug_skip_stage_load: consumed by the calling thread's next single-CTA 8-bit launch.
static thread_local int32_t g_skip_kb = -1;
void gemm_debug_skip_stage_load(int32_t kb) { g_skip_kb = kb < 0 ? -1 : kb; }

int launch_gemm(const GemmProblem& g, cudaStream_t stream, bool pdl) {
  if (g.M == 0) return DP_OK;
  if (g.res != nullptr && g.bits != 8) return fail(DP_ERR_INVALID_ARG, "residual epilogue: 8-bit operands only");
  const int cg = g.cg == 2 ? 2 : 1;
  GemmParams p;
  if (cg == 1 && g.bits == 8) {
    p.dbg_skip_kb = g_skip_kb;
    g_skip_kb = -1;
  }
  p.s_a = g.s_a;
  p.s_w = g.s_w;
  p.bias = g.bias;
  p.y = g.y;
  p.ldy = g.ldy;
  p.dbg_acc = g.dbg_acc;
  p.dbg_ldacc = g.dbg_ldacc;
  p.res = g.res;
  p.ldr = g.ldr;
  p.gate = g.gate;
  p.rows_per_gate = g.rows_per_gate;
  p.M = g.M;
  p.N = g.N;
  p.K = g.K;
  p.m_tiles = static_cast<int32_t>((g.M + BM * cg - 1) / (BM * cg));
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
  const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
  const int64_t slots = cg == 2 ? (gemm_max_pairs() > 0 ? gemm_max_pairs() : num_sms() / 2) : num_sms();
  const dim3 grid(static_cast<unsigned>((tiles < slots ? tiles : slots) * cg));
  for (int r = 0; r < 2; ++r) {
    if (g_pf_ptr[r] != nullptr && g_pf_bytes[r] >= 16 && g_pf_bytes[r] < (1ull << 31) &&
        (reinterpret_cast<uintptr_t>(g_pf_ptr[r]) & 15u) == 0) {
      p.pf[r] = static_cast<const uint8_t*>(g_pf_ptr[r]);
      p.pf_bytes[r] = static_cast<uint32_t>(g_pf_bytes[r] & ~static_cast<size_t>(15));
      p.pf_slice[r] = ((p.pf_bytes[r] + grid.x - 1) / grid.x + 15u) & ~15u;
    }
    g_pf_ptr[r] = nullptr;
  }
  cudaError_t e;
  if (cg == 2) {
    switch (g.bn) {
      case 128: e = launch_bn<128, 2>(g, p, grid, stream, pdl); break;
      case 192: e = launch_bn<192, 2>(g, p, grid, stream, pdl); break;
      case 256: e = launch_bn<256, 2>(g, p, grid, stream, pdl); break;
      default: return fail(DP_ERR_INVALID_ARG, "unsupported pair tile width %d", g.bn);
    }
  } else {
    switch (g.bn) {
      case 64: e = launch_bn<64, 1>(g, p, grid, stream, pdl); break;
      case 128: e = launch_bn<128, 1>(g, p, grid, stream, pdl); break;
      case 192: e = launch_bn<192, 1>(g, p, grid, stream, pdl); break;
      case 256: e = launch_bn<256, 1>(g, p, grid, stream, pdl); break;
      default: return fail(DP_ERR_INVALID_ARG, "unsupported tile width %d", g.bn);
    }
  }
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "GEMM launch failed: %s", cudaGetErrorString(e));
  return DP_OK;
}

}  // namespace dp
