// C-ABI entry points of libdiffpro: argument checks, kernel-variant dispatch, plan objects.
#include <stdarg.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <mutex>
#include <new>
#include <queue>
#include <vector>

#include "dp_common.cuh"
#include "dp_internal.h"

namespace dp {

// ---- error reporting ---------------------------------------------------------------------------
static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}
int fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return status;
}

// ---- per-device state ----------------------------------------------------------------------------
// Everything the library caches about a device (architecture check, SM count, resident CTA pairs,
// the kernels' shared-memory attributes, which CUDA keeps per device) is set up on the first call
// made with that device current, under a lock, and published with a release store, so that threads
// that use different devices, or race on their first call, see consistent state.
constexpr int kMaxDevices = 64;
struct DeviceInfo {
  int status;  // DP_OK or DP_ERR_ARCH
  int num_sms, max_pairs;
};
static DeviceInfo g_dev[kMaxDevices];
static std::atomic<int> g_dev_ready[kMaxDevices];
static std::mutex g_dev_mutex;

static int current_device(int* dev) {
  cudaError_t e = cudaGetDevice(dev);
  if (e != cudaSuccess) return fail(DP_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (*dev < 0 || *dev >= kMaxDevices) return fail(DP_ERR_INVALID_ARG, "device ordinal %d not supported", *dev);
  return DP_OK;
}

int check_device() {
  int dev = 0;
  int st = current_device(&dev);
  if (st != DP_OK) return st;
  if (!g_dev_ready[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!g_dev_ready[dev].load(std::memory_order_relaxed)) {
      DeviceInfo d = {DP_OK, 0, 0};
      int major = 0;
      cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
      if (e != cudaSuccess) return fail(DP_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
      if (major != 10) {
        d.status = DP_ERR_ARCH;
      } else {  // a failure here is reported and NOT cached: the next call tries again
        st = gemm_init_device(dev, &d.num_sms, &d.max_pairs);
        if (st != DP_OK) return st;
      }
      g_dev[dev] = d;
      g_dev_ready[dev].store(1, std::memory_order_release);
    }
  }
  if (g_dev[dev].status != DP_OK)
    return fail(g_dev[dev].status, "device %d is not compute capability 10.x; sm_100 required", dev);
  return DP_OK;
}

static const DeviceInfo* ready_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  return g_dev_ready[dev].load(std::memory_order_acquire) ? &g_dev[dev] : nullptr;
}
int num_sms() {
  const DeviceInfo* d = ready_device();
  return d ? d->num_sms : 0;
}
int gemm_max_pairs() {
  const DeviceInfo* d = ready_device();
  return d ? d->max_pairs : 0;
}

static size_t align256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }
// Bytes of the int8 activation scratch: whole 128-token tiles.
static size_t scratch_q_bytes(int64_t M, int32_t K) { return static_cast<size_t>((M + 127) / 128 * 128) * K; }

constexpr uint32_t kLinearFlags =
    DP_FLAG_FORCE_SIMT | DP_FLAG_FORCE_MMA | DP_FLAG_NO_PDL | DP_FLAG_TILE_N_MASK | DP_FLAG_CTA_PAIR |
    DP_FLAG_NO_CTA_PAIR | DP_FLAG_WEIGHT_STATIONARY | DP_FLAG_NO_WEIGHT_STATIONARY | DP_FLAG_UNPACK_FIRST |
    DP_FLAG_NO_UNPACK_FIRST | DP_FLAG_ACT_STATIONARY | DP_FLAG_NO_ACT_STATIONARY;
constexpr int64_t kWsMinRows = 8192;  // from here on a resident weight strip is reused often enough to pay
static int forced_bn(uint32_t flags) { return static_cast<int>((flags & DP_FLAG_TILE_N_MASK) >> 8) * 64; }

// Tile width and CTA-group size of the tensor-core kernel for this problem, honouring the tuning
// flags (validated by check_tile_flags).
// `bits` is the width the GEMM kernel sees (8 in the unpack-first form); `tiled_a`: the activations
// are the library's own tiled scratch (DAQ run by the call).
static void choose_tile(uint32_t flags, int64_t M, int32_t N, int32_t K, int32_t bits, bool tiled_a, int* bn,
                        int* cg, int* ws) {
  *ws = 0;
  // (callers clear tiled_a when the layer's scale / bias pointers lack the alignment that kernel's
  // vector loads need)
  const bool as_ok = tiled_a && bits == 8 && gemm_as_supported(N, K) &&
                     !(flags & (DP_FLAG_NO_ACT_STATIONARY | DP_FLAG_NO_CTA_PAIR | DP_FLAG_WEIGHT_STATIONARY));
  if (as_ok && (flags & DP_FLAG_ACT_STATIONARY)) {
    int nsub = 1;
    const int fb = forced_bn(flags);
    gemm_as_config(M, N, K, (fb != 0 && N % fb == 0) ? fb : 0, bn, &nsub);
    if (*bn != 0) {
      *cg = 2;
      *ws = 2;
      return;
    }
  }
  const bool ws_ok = gemm_ws_supported(N, K) && !(flags & (DP_FLAG_NO_WEIGHT_STATIONARY | DP_FLAG_NO_CTA_PAIR));
  // By default only with 256-channel strips: with 192-channel ones the resident strip leaves the
  // activation ring too shallow for the rate the tensor core then asks of it, and the streaming pair
  // kernel is 3-6 % faster (measured at M = 32768: qkv 139 -> 133 us, proj 67 -> 63).
  // (Packed weights expanded inside the GEMM keep it at either width: expanding a strip once instead
  // of once per tile is worth far more: qkv at 3 bits 121 us against 182.)
  if (ws_ok && ((flags & DP_FLAG_WEIGHT_STATIONARY) || (M >= kWsMinRows && (bits < 8 || gemm_ws_pick_bn(N) == 256)))) {
    const int fb = forced_bn(flags);
    *bn = ((fb == 192 || fb == 256) && N % fb == 0) ? fb : gemm_ws_pick_bn(N);
    *cg = 2;
    *ws = 1;
    return;
  }
  uint32_t allow = 0x6;
  if (flags & DP_FLAG_CTA_PAIR) allow = 0x4;
  if (flags & DP_FLAG_NO_CTA_PAIR) allow = 0x2;
  gemm_pick_tile(M, N, K, bits, allow, bn, cg);
  const int fb = forced_bn(flags);
  if (fb != 0 && N % fb == 0) {
    *bn = fb;
    if (fb < 128) *cg = 1;
    else if (allow == 0x4) *cg = 2;
    else if (allow == 0x2) *cg = 1;
  }
}
static int check_tile_flags(uint32_t flags, int32_t N) {
  const int fb = forced_bn(flags);
  if (fb != 0 && (fb > 256 || N % fb)) return fail(DP_ERR_SHAPE, "forced tile width %d does not divide N=%d", fb, N);
  if ((flags & DP_FLAG_CTA_PAIR) && (flags & DP_FLAG_NO_CTA_PAIR))
    return fail(DP_ERR_INVALID_ARG, "CTA_PAIR and NO_CTA_PAIR are exclusive");
  if ((flags & DP_FLAG_CTA_PAIR) && ((fb != 0 && fb < 128) || (N % 128 && N % 192)))
    return fail(DP_ERR_SHAPE, "CTA-pair tiles need a tile width of 128, 192 or 256 dividing N=%d", N);
  if ((flags & DP_FLAG_WEIGHT_STATIONARY) && (flags & (DP_FLAG_NO_WEIGHT_STATIONARY | DP_FLAG_NO_CTA_PAIR)))
    return fail(DP_ERR_INVALID_ARG, "WEIGHT_STATIONARY contradicts another flag");
  if ((flags & DP_FLAG_ACT_STATIONARY) &&
      (flags & (DP_FLAG_NO_ACT_STATIONARY | DP_FLAG_NO_CTA_PAIR | DP_FLAG_WEIGHT_STATIONARY)))
    return fail(DP_ERR_INVALID_ARG, "ACT_STATIONARY contradicts another flag");
  return DP_OK;
}

// Whether a packed layer runs in the unpack-first form: the flags decide; by default it does when
// the library quantizes the activations itself (a workspace exists and the expansion rides in the
// DAQ launch).
static bool want_unpack_first(uint32_t flags, int32_t bits, bool library_daq) {
  if (bits >= 8 || (flags & DP_FLAG_NO_UNPACK_FIRST)) return false;
  return (flags & DP_FLAG_UNPACK_FIRST) || library_daq;
}

// Rank from the top of the nearest-rank percentile p (in 1/1000 %) of K values: K - ceil(p K / 100) + 1.
static int clip_rank_of(int32_t p_e3, int32_t K) {
  const int64_t c = (static_cast<int64_t>(p_e3) * K + 99999) / 100000;
  return static_cast<int>(K - (c < 1 ? 1 : c) + 1);
}

constexpr int64_t kEarlyWeightsMaxRows = 512;  // see run_linear
constexpr int64_t kSimtMaxRows = 32;  // at or below this the CUDA-core streaming kernel is used

static bool use_simt(int64_t M, int32_t N, int32_t K, uint32_t flags) {
  if (flags & DP_FLAG_FORCE_SIMT) return true;
  if (N % 64 != 0) return true;  // tensor path tiles N by 64/128/192/256
  if (flags & DP_FLAG_FORCE_MMA) return false;
  (void)K;
  return M <= kSimtMaxRows;
}

// (kept for kernels with alignment needs beyond check_weight's; none at present)
static bool as_pointers_ok(const dp_weight*) { return true; }

static int check_weight(const dp_weight* w) {
  if (!w) return fail(DP_ERR_INVALID_ARG, "dp_weight is NULL");
  if (w->bits != 3 && w->bits != 4 && w->bits != 8 && w->bits != 16)
    return fail(DP_ERR_BITS, "bits=%d not in {3,4,8,16}", w->bits);
  if (w->N < 16 || w->K < 128 || (w->K % 128) || (w->N % 16))
    return fail(DP_ERR_SHAPE, "N=%d K=%d: need K %% 128 == 0, N %% 16 == 0", w->N, w->K);
  if (w->bits == 16 && (w->N % 64))
    return fail(DP_ERR_SHAPE, "N=%d: a 16-bit pass-through layer needs N %% 64 == 0", w->N);
  if (w->group_size < 0 || (w->group_size == 0 && w->zeros != nullptr))
    return fail(DP_ERR_INVALID_ARG, "dp_weight: negative group_size, or zero-points without groups");
  if (w->group_size > 0) {
    if (w->bits == 16) return fail(DP_ERR_BITS, "a 16-bit pass-through layer has no weight scales, hence no groups");
    if ((w->group_size % 32) || (w->K % w->group_size) || (w->N % 128))
      return fail(DP_ERR_SHAPE, "group-wise scales: need g %% 32 == 0, K %% g == 0, N %% 128 == 0 (g=%d K=%d N=%d)",
                  w->group_size, w->K, w->N);
  }
  if (!w->qweight || (!w->s_w && w->bits != 16)) return fail(DP_ERR_INVALID_ARG, "dp_weight has a NULL member");
  if (!aligned16(w->qweight) || (reinterpret_cast<uintptr_t>(w->s_w) & 3u) ||
      (w->bias && (reinterpret_cast<uintptr_t>(w->bias) & 1u)))
    return fail(DP_ERR_ALIGN, "dp_weight pointers misaligned");
  return DP_OK;
}

// One layer, all checks done. tmap_w may be a pre-encoded descriptor (plan) or nullptr.
// `chained`: the kernel preceding this layer's first launch on the stream is a launch of the same
// dp_plan_run call, so it cannot be a producer of this layer's weights and they may be prefetched
// while it drains.
static int run_linear(const dp_weight* w, const void* x, int64_t ldx, const float* s_a_in, int64_t M,
                      void* y, int64_t ldy, void* workspace, const dp_debug* dbg, int32_t* status,
                      uint32_t flags, cudaStream_t stream, const CUtensorMap* tmap_w, int bn, int cg, int ws,
                      const CUtensorMap* tmap_a_cached, bool chained, int32_t* daq_sync = nullptr,
                      int pre = -1, int daq_rank = 1, int daq_bits = 8, const dp_residual* res = nullptr) {
  const bool pdl = !(flags & DP_FLAG_NO_PDL);
  if (w->bits == 16)  // a layer the plan keeps in 16-bit precision: no DAQ, no scales (checked by the caller)
    return launch_gemm_bf16(x, ldx, w->qweight, static_cast<const uint16_t*>(w->bias), M, w->N, w->K,
                            static_cast<uint16_t*>(y), ldy, status, stream, pdl);
  // DAQ policy of a plan (dp_plan_set_daq): clip threshold below the maximum and/or fewer activation bits
  const bool robust = s_a_in == nullptr && (daq_rank > 1 || daq_bits < 8);
  if (w->group_size > 0) {
    // Group-wise scales: DAQ into the tiled scratch (packed weights expanded to int8 by the same
    // launch), the per-group code sums when there are zero-points, then the folding GEMM.
    uint8_t* ws8 = static_cast<uint8_t*>(workspace);
    int8_t* wq = static_cast<int8_t*>(workspace);
    float* wsa = reinterpret_cast<float*>(ws8 + align256(scratch_q_bytes(M, w->K)));
    size_t off = align256(scratch_q_bytes(M, w->K)) + align256(sizeof(float) * static_cast<size_t>(M));
    const int8_t* w8 = static_cast<const int8_t*>(w->qweight);
    UnpackJob job{nullptr, nullptr, 0, 0, 0};
    if (w->bits < 8) {
      int8_t* dst = reinterpret_cast<int8_t*>(ws8 + off);
      off += align256(static_cast<size_t>(w->N) * w->K);
      job = UnpackJob{static_cast<const uint32_t*>(w->qweight), dst, static_cast<int64_t>(w->N) * w->K / 32, w->bits, 0};
      w8 = dst;
    }
    int32_t* rowsum = w->zeros != nullptr ? reinterpret_cast<int32_t*>(ws8 + off) : nullptr;
    int st = robust ? launch_daq_robust(x, M, w->K, ldx, wq, w->K, wsa, nullptr, daq_rank, daq_bits, true, stream, pdl,
                                        w->bits < 8 ? &job : nullptr)
                    : launch_daq(x, M, w->K, ldx, wq, w->K, wsa, nullptr, KORDER_NATURAL, true, stream, pdl,
                                 w->bits < 8 ? &job : nullptr);
    if (st != DP_OK) return st;
    return launch_gemm_grp(wq, w->K, true, wsa, w8, w->bits, w->group_size, w->s_w, static_cast<const uint8_t*>(w->zeros),
                           static_cast<const uint16_t*>(w->bias), rowsum, M, w->N, w->K, static_cast<uint16_t*>(y), ldy,
                           status, stream, pdl);
  }
  if (use_simt(M, w->N, w->K, flags)) {
    if (static_cast<size_t>(w->K) > simt_max_k())
      return fail(DP_ERR_SHAPE, "K=%d too large for the small-M kernel", w->K);
    SimtArgs a;
    a.x = x;
    a.ldx = ldx;
    a.s_a_in = s_a_in;
    if (robust) {  // quantize into the workspace first; the kernel then takes the codes as they are
      int8_t* wq = static_cast<int8_t*>(workspace);
      float* wsa = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align256(scratch_q_bytes(M, w->K)));
      int st = launch_daq_robust(x, M, w->K, ldx, wq, w->K, wsa, nullptr, daq_rank, daq_bits, false, stream, pdl,
                                 nullptr);
      if (st != DP_OK) return st;
      a.x = wq;
      a.ldx = w->K;
      a.s_a_in = wsa;
    }
    a.M = M;
    a.N = w->N;
    a.K = w->K;
    a.bits = w->bits;
    a.qweight = w->qweight;
    a.s_w = w->s_w;
    a.bias = static_cast<const uint16_t*>(w->bias);
    a.y = static_cast<uint16_t*>(y);
    a.ldy = ldy;
    a.dbg_q = dbg ? dbg->q : nullptr;
    a.dbg_ldq = dbg ? dbg->ldq : 0;
    a.dbg_sa = dbg ? dbg->s_a : nullptr;
    a.dbg_acc = dbg ? dbg->acc : nullptr;
    a.dbg_ldacc = dbg ? dbg->ldacc : 0;
    a.early_w = chained ? 1 : 0;
    a.status = status;
    return launch_simt_linear(a, stream, pdl);
  }
  const int8_t* q;
  const float* s_a;
  int64_t ldq;
  int korder = KORDER_NATURAL;
  // Unpack-first variant: the packed weights are expanded once to int8 [N][K] in the workspace (by
  // extra CTAs of the DAQ launch) and the 8-bit kernel runs on that copy, instead of every CTA
  // expanding the weight tiles it needs in shared memory.
  if (pre < 0) pre = want_unpack_first(flags, w->bits, s_a_in == nullptr) ? 1 : 0;
  if (res != nullptr) pre = 1;  // its epilogue is built into the 8-bit streaming kernels
  if (robust) {  // that kernel writes codes in natural k order only: packed layers run on the int8 copy
    pre = 1;
    daq_sync = nullptr;
  }
  const bool unpack_first = pre > 0 && w->bits < 8;
  dp_weight w8 = *w;
  UnpackJob job{nullptr, nullptr, 0, 0, 0};
  if (unpack_first) {
    int8_t* dst = reinterpret_cast<int8_t*>(static_cast<uint8_t*>(workspace) + align256(scratch_q_bytes(M, w->K)) +
                                            align256(sizeof(float) * static_cast<size_t>(M)));
    job = UnpackJob{static_cast<const uint32_t*>(w->qweight), dst, static_cast<int64_t>(w->N) * w->K / 32, w->bits, 0};
    w8.bits = 8;
    w8.qweight = dst;
    w = &w8;
    tmap_w = nullptr;  // the caller's descriptor covers the packed matrix
    daq_sync = nullptr;
  }
  const bool tiled = s_a_in == nullptr;  // the library's own scratch: stored as contiguous 128 x 128 tiles
  const bool fused = s_a_in == nullptr && daq_sync != nullptr && dbg == nullptr;  // DAQ inside the GEMM kernel
  if (s_a_in == nullptr) {
    int8_t* wq = static_cast<int8_t*>(workspace);
    float* wsa = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align256(scratch_q_bytes(M, w->K)));
    korder = gemm_korder(w->bits);
    if (robust) {
      int st = launch_daq_robust(x, M, w->K, ldx, wq, w->K, wsa, nullptr, daq_rank, daq_bits, true, stream, pdl,
                                 unpack_first ? &job : nullptr);
      if (st != DP_OK) return st;
    } else if (!fused) {
      int st = launch_daq(x, M, w->K, ldx, wq, w->K, wsa, nullptr, korder, true, stream, pdl,
                          unpack_first ? &job : nullptr);
      if (st != DP_OK) return st;
    }
    q = wq;
    s_a = wsa;
    ldq = w->K;
  } else {
    q = static_cast<const int8_t*>(x);
    s_a = s_a_in;
    ldq = ldx;
    if (unpack_first) {
      int st = launch_unpack(job, stream, pdl);
      if (st != DP_OK) return st;
    }
  }
  GemmProblem g;
  g.korder = korder;
  g.a_tiled = tiled ? 1 : 0;
  g.early_w = fused ? (chained ? 1 : 0) : (s_a_in == nullptr ? 1 : 0);
  if (unpack_first) g.early_w = 0;  // the weights come from the kernel just before this one
  // Fetching weight tiles while the DAQ launch still runs pays only for small M: measured on B200,
  // it shortens a layer by ~0.3 us at M = 256 but lengthens it by 1-1.5 us at M = 2048..4096 (the
  // prefetch of every CTA competes with the DAQ launch for bandwidth, and the ring then starts with
  // a burst of activation loads instead of a steady stream); no effect at M = 32768.
  if (M > kEarlyWeightsMaxRows) g.early_w = 0;
  g.x = fused ? static_cast<const uint16_t*>(x) : nullptr;
  g.ldx = ldx;
  g.q_out = fused ? const_cast<int8_t*>(q) : nullptr;
  g.s_a_out = fused ? const_cast<float*>(s_a) : nullptr;
  g.sync = fused ? daq_sync : nullptr;
  if (tmap_a_cached != nullptr) {
    g.tmap_a = *tmap_a_cached;
  } else {
    int st = tiled ? gemm_encode_a_tiled(&g.tmap_a, q, M, w->K) : gemm_encode_a(&g.tmap_a, q, M, w->K, ldq);
    if (st != DP_OK) return st;
  }
  if (bn == 0) choose_tile(flags, M, w->N, w->K, w->bits, tiled && as_pointers_ok(w), &bn, &cg, &ws);
  if (ws == 2 && (!tiled || w->bits != 8 || fused || !as_pointers_ok(w)))
    return fail(DP_ERR_INVALID_ARG, "the activation-stationary kernel needs DAQ run by the call, 8-bit weights (or the "
                                    "unpack-first form)");
  // Its weight ring is small (64 KB per CTA): prefetching it while the DAQ launch drains costs that
  // launch no bandwidth worth speaking of, whatever M is.
  if (ws == 2 && s_a_in == nullptr && !unpack_first && pdl) g.early_w = 1;
  g.cg = cg;
  g.ws = ws;
  if (tmap_w != nullptr) {
    g.tmap_w = *tmap_w;
  } else {
    int st = gemm_encode_w(&g.tmap_w, w->qweight, w->N, w->K, w->bits, bn, cg);
    if (st != DP_OK) return st;
  }
  g.s_a = s_a;
  g.s_w = w->s_w;
  g.bias = static_cast<const uint16_t*>(w->bias);
  g.y = static_cast<uint16_t*>(y);
  g.ldy = ldy;
  g.dbg_acc = dbg ? dbg->acc : nullptr;
  g.dbg_ldacc = dbg ? dbg->ldacc : 0;
  if (res != nullptr) {
    g.res = static_cast<const uint16_t*>(res->residual);
    g.ldr = res->ldr;
    g.gate = static_cast<const uint16_t*>(res->gate);
    g.rows_per_gate = res->gate ? res->rows_per_gate : 1;
  }
  g.M = M;
  g.N = w->N;
  g.K = w->K;
  g.bits = w->bits;
  g.bn = bn;
  g.status = status;
  int st = ws == 2 ? launch_gemm_as(g, stream, pdl) : ws ? launch_gemm_ws(g, stream, pdl) : launch_gemm(g, stream, pdl);
  if (st != DP_OK) return st;
  if (dbg != nullptr) {
    if (dbg->q != nullptr) {
      if (tiled || korder != KORDER_NATURAL) {  // the scratch holds a tiled / permuted copy: quantize again
        st = launch_daq(x, M, w->K, ldx, dbg->q, dbg->ldq, const_cast<float*>(s_a), nullptr, KORDER_NATURAL,
                        false, stream, false);
        if (st != DP_OK) return st;
      } else {
        DP_CUDA_OK(cudaMemcpy2DAsync(dbg->q, dbg->ldq, q, ldq, w->K, M, cudaMemcpyDeviceToDevice, stream));
      }
    }
    if (dbg->s_a != nullptr)
      DP_CUDA_OK(cudaMemcpyAsync(dbg->s_a, s_a, sizeof(float) * M, cudaMemcpyDeviceToDevice, stream));
  }
  return DP_OK;
}

static int check_linear_args(const dp_weight* w, const void* x, int64_t ldx, const float* s_a_in,
                             int64_t M, void* y, int64_t ldy, void* workspace, size_t workspace_bytes,
                             const dp_debug* dbg, uint32_t flags) {
  int st = check_weight(w);
  if (st != DP_OK) return st;
  if (M < 0) return fail(DP_ERR_SHAPE, "M=%lld is negative", (long long)M);
  if (flags & ~kLinearFlags) return fail(DP_ERR_INVALID_ARG, "unknown flag bits 0x%x", flags);
  if (int tst = check_tile_flags(flags, w->N)) return tst;
  if ((flags & DP_FLAG_FORCE_SIMT) && (flags & DP_FLAG_FORCE_MMA))
    return fail(DP_ERR_INVALID_ARG, "FORCE_SIMT and FORCE_MMA are exclusive");
  if ((flags & DP_FLAG_UNPACK_FIRST) && (flags & DP_FLAG_NO_UNPACK_FIRST))
    return fail(DP_ERR_INVALID_ARG, "UNPACK_FIRST and NO_UNPACK_FIRST are exclusive");
  if (w->bits == 16 && (s_a_in != nullptr || dbg != nullptr))
    return fail(DP_ERR_INVALID_ARG, "a 16-bit pass-through layer takes bf16 activations and has no taps");
  if (w->group_size > 0 && (s_a_in != nullptr || dbg != nullptr))
    return fail(DP_ERR_INVALID_ARG, "a layer with group-wise scales takes bf16 activations and has no taps");
  if (M == 0) return DP_OK;
  if (!x || !y) return fail(DP_ERR_INVALID_ARG, "x or y is NULL");
  if (ldx < w->K || ldy < w->N) return fail(DP_ERR_SHAPE, "leading dimension smaller than the row");
  const int64_t xa = s_a_in ? 16 : 8;  // elements per 16 bytes
  if (!aligned16(x) || !aligned16(y) || (ldx % xa) || (ldy % 8))
    return fail(DP_ERR_ALIGN, "x/y pointers and pitches must be 16-byte aligned");
  if (dbg) {
    if (dbg->q && (!aligned16(dbg->q) || dbg->ldq < w->K || (dbg->ldq % 16)))
      return fail(DP_ERR_ALIGN, "dbg.q misaligned or too narrow");
    if (dbg->acc && (dbg->ldacc < w->N || (reinterpret_cast<uintptr_t>(dbg->acc) & 3u)))
      return fail(DP_ERR_ALIGN, "dbg.acc misaligned or too narrow");
  }
  if (w->group_size > 0) {
    const size_t need = dp_wq_linear_workspace_grouped(M, w);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
      return fail(DP_ERR_WORKSPACE, "workspace needs %zu bytes, 256-byte aligned (got %zu)", need, workspace_bytes);
    return DP_OK;
  }
  // scratch users: the library's own DAQ, and the int8 copy of the weights of the unpack-first form
  if (w->bits != 16 && !use_simt(M, w->N, w->K, flags) &&
      (s_a_in == nullptr || want_unpack_first(flags, w->bits, false))) {
    const size_t need = dp_wq_linear_workspace(M, w->N, w->K, w->bits, flags);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
      return fail(DP_ERR_WORKSPACE, "workspace needs %zu bytes, 256-byte aligned (got %zu)", need,
                  workspace_bytes);
  }
  return DP_OK;
}

}  // namespace dp

// ================================================================================================
using namespace dp;

extern "C" size_t dp_wq_linear_workspace(int64_t M, int32_t N, int32_t K, int32_t bits, uint32_t flags) {
  if (M <= 0 || K <= 0 || bits == 16) return 256;
  if (use_simt(M, N, K, flags)) return 256;
  size_t need = align256(scratch_q_bytes(M, K)) + align256(sizeof(float) * static_cast<size_t>(M));
  if (want_unpack_first(flags, bits, true)) need += align256(static_cast<size_t>(N) * K);
  return need;
}

extern "C" size_t dp_wq_linear_workspace_grouped(int64_t M, const dp_weight* w) {
  if (!w || M <= 0 || w->K <= 0 || w->group_size <= 0) return 256;
  size_t need = align256(scratch_q_bytes(M, w->K)) + align256(sizeof(float) * static_cast<size_t>(M));
  if (w->bits < 8) need += align256(static_cast<size_t>(w->N) * w->K);
  if (w->zeros != nullptr) need += align256(sizeof(int32_t) * static_cast<size_t>(M) * (w->K / w->group_size));
  return need;
}

extern "C" int dp_wq_linear(const dp_weight* w, const void* x, int64_t ldx, const float* s_a_in,
                            int64_t M, void* y_bf16, int64_t ldy, void* workspace,
                            size_t workspace_bytes, const dp_debug* dbg, int32_t* device_status,
                            uint32_t flags, dp_stream stream) {
  int st = check_linear_args(w, x, ldx, s_a_in, M, y_bf16, ldy, workspace, workspace_bytes, dbg, flags);
  if (st != DP_OK || M == 0) return st;
  st = check_device();
  if (st != DP_OK) return st;
  return run_linear(w, x, ldx, s_a_in, M, y_bf16, ldy, workspace, dbg, device_status, flags,
                    static_cast<cudaStream_t>(stream), nullptr, 0, 0, 0, nullptr, false);
}

extern "C" int dp_ln_modulate_daq(const void* x, int64_t M, int64_t K, int64_t ldx, const void* shift,
                                  const void* scale, int64_t rows_per_sample, float eps, int8_t* q, int64_t ldq,
                                  float* s_a, dp_stream stream) {
  if (M < 0 || K <= 0 || (K % 8) || K > 4608) return fail(DP_ERR_SHAPE, "dp_ln_modulate_daq: M=%lld K=%lld", (long long)M, (long long)K);
  if ((shift == nullptr) != (scale == nullptr))
    return fail(DP_ERR_INVALID_ARG, "dp_ln_modulate_daq: shift and scale come together");
  if (shift != nullptr && rows_per_sample < 1) return fail(DP_ERR_SHAPE, "rows_per_sample=%lld", (long long)rows_per_sample);
  if (!(eps >= 0.0f)) return fail(DP_ERR_INVALID_ARG, "dp_ln_modulate_daq: eps must be >= 0");
  if (M == 0) return DP_OK;
  if (!x || !q || !s_a) return fail(DP_ERR_INVALID_ARG, "dp_ln_modulate_daq: NULL argument");
  if (ldx < K || ldq < K) return fail(DP_ERR_SHAPE, "leading dimension smaller than the row");
  if (!aligned16(x) || !aligned16(q) || (ldx % 8) || (ldq % 16) || (reinterpret_cast<uintptr_t>(s_a) & 3u) ||
      (shift && (!aligned16(shift) || !aligned16(scale))))
    return fail(DP_ERR_ALIGN, "dp_ln_modulate_daq: pointers and pitches must be 16-byte aligned");
  int st = check_device();
  if (st != DP_OK) return st;
  return launch_ln_modulate_daq(x, M, K, ldx, shift, scale, shift ? rows_per_sample : 1, eps, q, ldq, s_a,
                                static_cast<cudaStream_t>(stream), false);
}

extern "C" int dp_wq_linear_residual(const dp_weight* w, const void* x_bf16, int64_t ldx, int64_t M,
                                     const dp_residual* r, void* y_bf16, int64_t ldy, void* workspace,
                                     size_t workspace_bytes, int32_t* device_status, uint32_t flags,
                                     dp_stream stream) {
  if (flags & DP_FLAG_FORCE_SIMT)
    return fail(DP_ERR_INVALID_ARG, "dp_wq_linear_residual runs tensor-core kernels only");
  if (flags & (DP_FLAG_WEIGHT_STATIONARY | DP_FLAG_ACT_STATIONARY))
    return fail(DP_ERR_INVALID_ARG, "dp_wq_linear_residual runs the streaming kernels only");
  flags = (flags & ~DP_FLAG_NO_UNPACK_FIRST) | DP_FLAG_FORCE_MMA | DP_FLAG_UNPACK_FIRST | DP_FLAG_NO_WEIGHT_STATIONARY |
          DP_FLAG_NO_ACT_STATIONARY;
  int st = check_linear_args(w, x_bf16, ldx, nullptr, M, y_bf16, ldy, workspace, workspace_bytes, nullptr, flags);
  if (st != DP_OK) return st;
  if (w->bits == 16 || w->group_size > 0)
    return fail(DP_ERR_INVALID_ARG, "dp_wq_linear_residual takes per-channel layers of 3, 4 or 8 bits");
  if (!r) return fail(DP_ERR_INVALID_ARG, "dp_residual is NULL");
  if (M == 0) return DP_OK;
  if (!r->residual) return fail(DP_ERR_INVALID_ARG, "dp_residual.residual is NULL");
  if (r->ldr < w->N) return fail(DP_ERR_SHAPE, "dp_residual.ldr smaller than the row");
  if (!aligned16(r->residual) || (r->ldr % 8) || (r->gate && !aligned16(r->gate)))
    return fail(DP_ERR_ALIGN, "residual / gate pointers and pitch must be 16-byte aligned");
  if (r->gate && r->rows_per_gate < 1) return fail(DP_ERR_SHAPE, "rows_per_gate=%lld", (long long)r->rows_per_gate);
  st = check_device();
  if (st != DP_OK) return st;
  return run_linear(w, x_bf16, ldx, nullptr, M, y_bf16, ldy, workspace, nullptr, device_status, flags,
                    static_cast<cudaStream_t>(stream), nullptr, 0, 0, 0, nullptr, false, nullptr, -1, 1, 8, r);
}

// ---- the linear for callers that cannot allocate ---------------------------------------------------
// Scratch of dp_wq_linear_static. In host code `g_static_scratch` is only a handle for the runtime:
// its device address comes from cudaGetSymbolAddress, once per device, and that address is what the
// kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[DP_STATIC_SCRATCH_BYTES];

// device address per device ordinal, nullptr = not yet queried (a cudaDeviceReset invalidates it:
// the library does not support resetting a device it has been used on)
static std::atomic<void*> g_static_scratch_ptr[kMaxDevices];

static int static_scratch_address(void** out) {
  int dev = 0;
  int st = current_device(&dev);
  if (st != DP_OK) return st;
  void* p = g_static_scratch_ptr[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DP_CUDA_OK(cudaGetSymbolAddress(&p, g_static_scratch));
    if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 255u))
      return fail(DP_ERR_CUDA, "static scratch has no usable device address on device %d", dev);
    g_static_scratch_ptr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return DP_OK;
}

extern "C" int dp_wq_linear_static(const dp_weight* w, const void* x_bf16, int64_t ldx, int64_t M,
                                   void* y_bf16, int64_t ldy, int32_t* device_status, uint32_t flags,
                                   dp_stream stream) {
  // The built-in scratch is sized for the activations only: weights are expanded inside the GEMM
  // unless the caller asks otherwise (and the copy fits).
  if (!(flags & DP_FLAG_UNPACK_FIRST)) flags |= DP_FLAG_NO_UNPACK_FIRST;
  int st = check_weight(w);
  if (st != DP_OK) return st;
  const size_t need = w->group_size > 0 ? dp_wq_linear_workspace_grouped(M, w)
                                        : dp_wq_linear_workspace(M, w->N, w->K, w->bits, flags);
  if (need > DP_STATIC_SCRATCH_BYTES)
    return fail(DP_ERR_WORKSPACE,
                "dp_wq_linear_static: M=%lld K=%d needs %zu bytes of scratch, the built-in array holds %u; "
                "use dp_wq_linear with a caller-provided workspace",
                (long long)M, w->K, need, (unsigned)DP_STATIC_SCRATCH_BYTES);
  st = check_device();
  if (st != DP_OK) return st;
  void* scratch = nullptr;
  st = static_scratch_address(&scratch);
  if (st != DP_OK) return st;
  st = check_linear_args(w, x_bf16, ldx, nullptr, M, y_bf16, ldy, scratch, DP_STATIC_SCRATCH_BYTES, nullptr, flags);
  if (st != DP_OK || M == 0) return st;
  return run_linear(w, x_bf16, ldx, nullptr, M, y_bf16, ldy, scratch, nullptr, device_status, flags,
                    static_cast<cudaStream_t>(stream), nullptr, 0, 0, 0, nullptr, false);
}

// ---- plans ---------------------------------------------------------------------------------------
struct PlanLayer {
  dp_weight w;
  int64_t M;
  bool simt;
  int bn, cg, ws;
  int pre;  // weights expanded to int8 scratch first, 8-bit kernel on the copy
  CUtensorMap tmap_w;
  size_t x_offset;  // byte offset of this layer's input inside one staged step (host-input path)
};
struct TmapACache {
  const void* ptr;
  int64_t M, K;
  CUtensorMap map;
};
struct dp_plan {
  std::vector<PlanLayer> layers;
  uint32_t flags;
  size_t workspace_bytes;
  size_t x_bytes;
  std::vector<TmapACache> a_cache;
  std::vector<std::vector<int>> groups;  // small-M layers of equal shape, run first in every step
  std::vector<char> grouped;             // per layer: member of a group
  int32_t* daq_sync;                     // device counters of the in-kernel DAQ (nullptr: DAQ in its own kernel)
  // DAQ policy (dp_plan_set_daq): clip percentile in 1/1000 %, 100000 = the maximum; activation bits
  // of the three time bins of [0, daq_timesteps)
  int32_t daq_p_e3, daq_timesteps, daq_bits[3];
  cudaStream_t copy_stream;
  cudaEvent_t ev_copied[2], ev_consumed[2], ev_entry;
};

// Times every kernel variant that can run this layer shape (the whole layer: DAQ + GEMM, as the
// plan will launch it) and returns the fastest. Plan creation only.
struct TunedShape {
  int64_t M;
  int32_t N, K, bits;
  int bn, cg, ws, pre;
};
static int autotune_shape(const dp_weight& w, int64_t M, uint32_t flags, bool allow_as, int* bn_out, int* cg_out,
                          int* ws_out, int* pre_out) {
  struct Cand {
    int bn, cg, ws, pre;
  };
  std::vector<Cand> cands;
  const int widths[4] = {64, 128, 192, 256};
  const int pre_lo = (flags & DP_FLAG_UNPACK_FIRST) ? 1 : 0;
  const int pre_hi = (w.bits < 8 && !(flags & (DP_FLAG_NO_UNPACK_FIRST | DP_FLAG_FUSED_DAQ))) ? 1 : 0;
  for (int pre = pre_lo < pre_hi ? pre_lo : pre_hi; pre <= pre_hi; ++pre)
    for (int i = 0; i < 4; ++i)
      if (w.N % widths[i] == 0) {
        cands.push_back({widths[i], 1, 0, pre});
        if (widths[i] >= 128) cands.push_back({widths[i], 2, 0, pre});
        if (widths[i] >= 192 && gemm_ws_supported(w.N, w.K)) cands.push_back({widths[i], 2, 1, pre});
        if (allow_as && as_pointers_ok(&w) && gemm_as_supported(w.N, w.K) && (w.bits == 8 || pre))
          cands.push_back({widths[i], 2, 2, pre});
      }
  void *x = nullptr, *y = nullptr, *ws = nullptr;
  cudaStream_t stream = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  const size_t xb = static_cast<size_t>(M) * w.K * 2, yb = static_cast<size_t>(M) * w.N * 2;
  const size_t wb = dp_wq_linear_workspace(M, w.N, w.K, w.bits, DP_FLAG_UNPACK_FIRST);
  cudaError_t e = cudaMalloc(&x, xb);
  if (e == cudaSuccess) e = cudaMalloc(&y, yb);
  if (e == cudaSuccess) e = cudaMalloc(&ws, wb);
  if (e == cudaSuccess) e = cudaMemset(x, 0x3c, xb);  // bf16 0x3c3c = 0.0115: finite, non-zero
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  int st = e == cudaSuccess ? DP_OK : fail(DP_ERR_CUDA, "autotune set-up: %s", cudaGetErrorString(e));
  float best = 1e30f;
  for (size_t c = 0; c < cands.size() && st == DP_OK; ++c) {
    CUtensorMap tw;
    st = gemm_encode_w(&tw, w.qweight, w.N, w.K, w.bits, cands[c].bn, cands[c].cg);
    const int warm = 2, reps = 8;
    for (int it = 0; it < warm + reps && st == DP_OK; ++it) {
      if (it == warm) cudaEventRecord(e0, stream);
      st = run_linear(&w, x, w.K, nullptr, M, y, w.N, ws, nullptr, nullptr, flags & DP_FLAG_NO_PDL, stream, &tw,
                      cands[c].bn, cands[c].cg, cands[c].ws, nullptr, it > 0, nullptr, cands[c].pre);
    }
    if (st != DP_OK) break;
    cudaEventRecord(e1, stream);
    e = cudaEventSynchronize(e1);
    float ms = 0.0f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e != cudaSuccess) {
      st = fail(DP_ERR_CUDA, "autotune timing: %s", cudaGetErrorString(e));
      break;
    }
    if (ms < best) {
      best = ms;
      *bn_out = cands[c].bn;
      *cg_out = cands[c].cg;
      *ws_out = cands[c].ws;
      *pre_out = cands[c].pre;
    }
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (stream) cudaStreamDestroy(stream);
  cudaFree(x);
  cudaFree(y);
  cudaFree(ws);
  return st;
}

extern "C" int dp_plan_create(const dp_weight* layers, int32_t n_layers, const int64_t* M_per_layer,
                              uint32_t flags, dp_plan** out) {
  if (!out) return fail(DP_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!layers || !M_per_layer || n_layers <= 0)
    return fail(DP_ERR_INVALID_ARG, "layers/M_per_layer NULL or n_layers <= 0");
  if (flags & ~(kLinearFlags | DP_FLAG_AUTOTUNE | DP_FLAG_GROUP_SMALL_M | DP_FLAG_FUSED_DAQ))
    return fail(DP_ERR_INVALID_ARG, "unknown flag bits 0x%x", flags);
  const bool autotune = (flags & DP_FLAG_AUTOTUNE) != 0;
  const bool group_small = (flags & DP_FLAG_GROUP_SMALL_M) != 0;
  const bool fused_daq = (flags & DP_FLAG_FUSED_DAQ) != 0;
  flags &= ~(DP_FLAG_AUTOTUNE | DP_FLAG_GROUP_SMALL_M | DP_FLAG_FUSED_DAQ);
  std::vector<TunedShape> tuned;
  int st = check_device();
  if (st != DP_OK) return st;
  dp_plan* p = new (std::nothrow) dp_plan();
  if (!p) return fail(DP_ERR_CUDA, "out of host memory");
  p->flags = flags;
  p->workspace_bytes = 256;
  p->x_bytes = 0;
  p->copy_stream = nullptr;
  p->daq_sync = nullptr;
  p->daq_p_e3 = 100000;
  p->daq_timesteps = 0;
  p->daq_bits[0] = p->daq_bits[1] = p->daq_bits[2] = 8;
  for (int i = 0; i < 2; ++i) p->ev_copied[i] = p->ev_consumed[i] = nullptr;
  p->ev_entry = nullptr;
  for (int32_t l = 0; l < n_layers; ++l) {
    st = check_weight(&layers[l]);
    if (st == DP_OK && M_per_layer[l] < 0) st = fail(DP_ERR_SHAPE, "layer %d: negative M", l);
    if (st != DP_OK) {
      delete p;
      return st;
    }
    PlanLayer L;
    L.w = layers[l];
    L.M = M_per_layer[l];
    L.simt = L.w.bits != 16 && L.w.group_size == 0 && use_simt(L.M, L.w.N, L.w.K, flags);
    L.bn = 0;
    L.cg = 1;
    L.ws = 0;
    L.pre = 0;
    memset(&L.tmap_w, 0, sizeof(L.tmap_w));
    if (L.simt && static_cast<size_t>(L.w.K) > simt_max_k()) {
      delete p;
      return fail(DP_ERR_SHAPE, "layer %d: K too large for the small-M kernel", l);
    }
    if (!L.simt && L.M > 0 && L.w.bits != 16 && L.w.group_size == 0) {
      uint32_t lf = flags;  // a pair request that this layer's N cannot honour falls back to the default
      // DAQ inside the GEMM kernel and a DAQ launch that also expands the weights exclude each other
      if ((lf & DP_FLAG_FUSED_DAQ) && !(lf & DP_FLAG_UNPACK_FIRST)) lf |= DP_FLAG_NO_UNPACK_FIRST;
      if ((lf & DP_FLAG_CTA_PAIR) && L.w.N % 128 && L.w.N % 192) lf &= ~DP_FLAG_CTA_PAIR;
      if ((lf & DP_FLAG_WEIGHT_STATIONARY) && !gemm_ws_supported(L.w.N, L.w.K)) lf &= ~DP_FLAG_WEIGHT_STATIONARY;
      L.pre = want_unpack_first(lf, L.w.bits, true) ? 1 : 0;
      choose_tile(lf, L.M, L.w.N, L.w.K, L.pre ? 8 : L.w.bits, !fused_daq && as_pointers_ok(&L.w), &L.bn, &L.cg, &L.ws);
      if (autotune) {
        const TunedShape* hit = nullptr;
        for (const TunedShape& t : tuned)
          if (t.M == L.M && t.N == L.w.N && t.K == L.w.K && t.bits == L.w.bits) hit = &t;
        if (hit == nullptr) {
          TunedShape t = {L.M, L.w.N, L.w.K, L.w.bits, L.bn, L.cg, L.ws, L.pre};
          st = autotune_shape(L.w, L.M, flags, !fused_daq, &t.bn, &t.cg, &t.ws, &t.pre);
          if (st != DP_OK) {
            delete p;
            return st;
          }
          tuned.push_back(t);
          hit = &tuned.back();
        }
        L.bn = hit->bn;
        L.cg = hit->cg;
        L.ws = hit->ws;
        L.pre = hit->pre;
      }
      st = gemm_encode_w(&L.tmap_w, L.w.qweight, L.w.N, L.w.K, L.w.bits, L.bn, L.cg);
      if (st != DP_OK) {
        delete p;
        return st;
      }
    }
    const size_t ws = L.w.group_size > 0
                          ? dp_wq_linear_workspace_grouped(L.M, &L.w)
                          : dp_wq_linear_workspace(L.M, L.w.N, L.w.K, L.w.bits,
                                                   (flags & ~(DP_FLAG_UNPACK_FIRST | DP_FLAG_NO_UNPACK_FIRST)) |
                                                       (L.pre ? DP_FLAG_UNPACK_FIRST : DP_FLAG_NO_UNPACK_FIRST));
    if (ws > p->workspace_bytes) p->workspace_bytes = ws;

    L.x_offset = p->x_bytes;
    p->x_bytes += align256(static_cast<size_t>(L.M) * L.w.K * 2);
    p->layers.push_back(L);
  }
  p->grouped.assign(p->layers.size(), 0);
  if (group_small) {
    for (size_t l = 0; l < p->layers.size(); ++l) {
      const PlanLayer& L = p->layers[l];
      if (!L.simt || L.M == 0) continue;
      std::vector<int>* home = nullptr;
      for (auto& g : p->groups) {
        const PlanLayer& G = p->layers[g[0]];
        if (G.M == L.M && G.w.N == L.w.N && G.w.K == L.w.K && g.size() < static_cast<size_t>(kSimtGroupMax)) home = &g;
      }
      if (home == nullptr) {
        p->groups.emplace_back();
        home = &p->groups.back();
      }
      home->push_back(static_cast<int>(l));
      p->grouped[l] = 1;
    }
    for (const auto& g : p->groups) {
      const PlanLayer& G = p->layers[g[0]];
      const size_t need = simt_group_scratch_bytes(G.M, G.w.K, static_cast<int32_t>(g.size()));
      if (need > p->workspace_bytes) p->workspace_bytes = need;
    }
  }
  cudaError_t e = cudaSuccess;
  if (fused_daq) {
    int64_t max_tiles = 0;
    for (const PlanLayer& L : p->layers)
      if (!L.simt && (L.M + 127) / 128 > max_tiles) max_tiles = (L.M + 127) / 128;
    if (max_tiles > 0) {
      const size_t bytes = sizeof(int32_t) * static_cast<size_t>(max_tiles + 1);
      e = cudaMalloc(reinterpret_cast<void**>(&p->daq_sync), bytes);
      if (e == cudaSuccess) e = cudaMemset(p->daq_sync, 0, bytes);
    }
  }
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_entry, cudaEventDisableTiming);
  for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
    e = cudaEventCreateWithFlags(&p->ev_copied[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_consumed[i], cudaEventDisableTiming);
  }
  if (e != cudaSuccess) {
    dp_plan_destroy(p);
    return fail(DP_ERR_CUDA, "plan stream/event creation: %s", cudaGetErrorString(e));
  }
  *out = p;
  return DP_OK;
}

extern "C" size_t dp_plan_workspace(const dp_plan* plan) { return plan ? plan->workspace_bytes : 0; }
extern "C" int dp_plan_set_daq(dp_plan* plan, int32_t clip_percentile_e3, int32_t n_timesteps,
                               const int32_t* act_bits_by_bin) {
  if (!plan) return fail(DP_ERR_INVALID_ARG, "dp_plan_set_daq: plan is NULL");
  if (clip_percentile_e3 < 1 || clip_percentile_e3 > 100000)
    return fail(DP_ERR_INVALID_ARG, "dp_plan_set_daq: percentile %d/1000 %% not in (0, 100]", clip_percentile_e3);
  if (n_timesteps < 0 || (n_timesteps > 0 && !act_bits_by_bin))
    return fail(DP_ERR_INVALID_ARG, "dp_plan_set_daq: bad n_timesteps / act_bits_by_bin");
  for (int b = 0; b < 3 && n_timesteps > 0; ++b)
    if (act_bits_by_bin[b] < 2 || act_bits_by_bin[b] > 8)
      return fail(DP_ERR_BITS, "dp_plan_set_daq: activation bits %d not in [2, 8]", act_bits_by_bin[b]);
  size_t need = plan->workspace_bytes;
  for (const PlanLayer& L : plan->layers) {
    if (L.M == 0 || L.w.bits == 16 || L.w.group_size > 0) continue;  // no DAQ / scratch already sized for any rule
    const int rank = clip_rank_of(clip_percentile_e3, L.w.K);
    if (rank > 64 || L.w.K > 4608)
      return fail(DP_ERR_SHAPE, "dp_plan_set_daq: a layer with K=%d would need clip rank %d (limits: K <= 4608, rank <= 64)",
                  L.w.K, rank);
    // every layer quantizes into the workspace under a policy; packed ones run on their int8 copy
    size_t ws = align256(scratch_q_bytes(L.M, L.w.K)) + align256(sizeof(float) * static_cast<size_t>(L.M));
    if (!L.simt && L.w.bits < 8) ws += align256(static_cast<size_t>(L.w.N) * L.w.K);
    if (ws > need) need = ws;
  }
  plan->workspace_bytes = need;
  plan->daq_p_e3 = clip_percentile_e3;
  plan->daq_timesteps = n_timesteps;
  for (int b = 0; b < 3; ++b) plan->daq_bits[b] = n_timesteps > 0 ? act_bits_by_bin[b] : 8;
  return DP_OK;
}
extern "C" int dp_plan_set_layer_flags(dp_plan* plan, int32_t layer, uint32_t flags) {
  if (!plan || layer < 0 || layer >= static_cast<int32_t>(plan->layers.size()))
    return fail(DP_ERR_INVALID_ARG, "dp_plan_set_layer_flags: bad plan or layer index");
  PlanLayer& L = plan->layers[layer];
  constexpr uint32_t kVariantFlags = DP_FLAG_TILE_N_MASK | DP_FLAG_CTA_PAIR | DP_FLAG_NO_CTA_PAIR |
                                     DP_FLAG_WEIGHT_STATIONARY | DP_FLAG_NO_WEIGHT_STATIONARY | DP_FLAG_UNPACK_FIRST |
                                     DP_FLAG_NO_UNPACK_FIRST | DP_FLAG_ACT_STATIONARY | DP_FLAG_NO_ACT_STATIONARY;
  if (flags & ~kVariantFlags) return fail(DP_ERR_INVALID_ARG, "dp_plan_set_layer_flags: flag bits 0x%x do not name a variant", flags);
  if (L.simt || L.M == 0 || L.w.bits == 16 || L.w.group_size > 0)
    return fail(DP_ERR_INVALID_ARG, "layer %d runs the small-M, the 16-bit or the group-wise kernel: it has no variants",
                layer);
  if (int st = check_tile_flags(flags, L.w.N)) return st;
  if ((flags & DP_FLAG_WEIGHT_STATIONARY) && !gemm_ws_supported(L.w.N, L.w.K))
    return fail(DP_ERR_SHAPE, "layer %d: the weight-stationary kernel does not take N=%d K=%d", layer, L.w.N, L.w.K);
  PlanLayer T = L;
  if ((flags & DP_FLAG_UNPACK_FIRST) && (flags & DP_FLAG_NO_UNPACK_FIRST))
    return fail(DP_ERR_INVALID_ARG, "UNPACK_FIRST and NO_UNPACK_FIRST are exclusive");
  T.pre = want_unpack_first(flags, T.w.bits, true) ? 1 : 0;
  choose_tile(flags, T.M, T.w.N, T.w.K, T.pre ? 8 : T.w.bits, plan->daq_sync == nullptr && as_pointers_ok(&T.w), &T.bn,
              &T.cg, &T.ws);
  if ((flags & DP_FLAG_ACT_STATIONARY) && T.ws != 2)
    return fail(DP_ERR_SHAPE, "layer %d: the activation-stationary kernel does not take this layer (N=%d K=%d, %d-bit "
                              "weights without the unpack-first form, or DAQ fused into the GEMM)",
                layer, L.w.N, L.w.K, L.w.bits);
  if (int st = gemm_encode_w(&T.tmap_w, T.w.qweight, T.w.N, T.w.K, T.w.bits, T.bn, T.cg)) return st;
  L = T;
  const size_t ws = dp_wq_linear_workspace(L.M, L.w.N, L.w.K, L.w.bits,
                                           L.pre ? DP_FLAG_UNPACK_FIRST : DP_FLAG_NO_UNPACK_FIRST);
  if (ws > plan->workspace_bytes) plan->workspace_bytes = ws;
  return DP_OK;
}
extern "C" int dp_plan_layer_unpack_first(const dp_plan* plan, int32_t layer, int32_t* unpack_first) {
  if (!plan || layer < 0 || layer >= static_cast<int32_t>(plan->layers.size()) || !unpack_first)
    return fail(DP_ERR_INVALID_ARG, "dp_plan_layer_unpack_first: bad plan, layer index or NULL output");
  const PlanLayer& L = plan->layers[layer];
  *unpack_first = (!L.simt && L.pre) ? 1 : 0;
  return DP_OK;
}
extern "C" int dp_plan_layer_variant(const dp_plan* plan, int32_t layer, int32_t* tile_n, int32_t* cta_group,
                                     int32_t* weight_stationary, int32_t* small_m) {
  if (!plan || layer < 0 || layer >= static_cast<int32_t>(plan->layers.size()))
    return fail(DP_ERR_INVALID_ARG, "dp_plan_layer_variant: bad plan or layer index");
  const PlanLayer& L = plan->layers[layer];
  if (tile_n) *tile_n = L.simt ? 0 : L.bn;
  if (cta_group) *cta_group = L.simt ? 0 : L.cg;
  if (weight_stationary) *weight_stationary = L.simt ? 0 : L.ws;
  if (small_m) *small_m = L.simt ? 1 : 0;
  return DP_OK;
}
extern "C" size_t dp_plan_x_bytes(const dp_plan* plan) { return plan ? plan->x_bytes : 0; }

extern "C" void dp_plan_destroy(dp_plan* plan) {
  if (!plan) return;
  for (int i = 0; i < 2; ++i) {
    if (plan->ev_copied[i]) cudaEventDestroy(plan->ev_copied[i]);
    if (plan->ev_consumed[i]) cudaEventDestroy(plan->ev_consumed[i]);
    if (i == 0 && plan->ev_entry) cudaEventDestroy(plan->ev_entry);
  }
  if (plan->copy_stream) cudaStreamDestroy(plan->copy_stream);
  if (plan->daq_sync) cudaFree(plan->daq_sync);
  delete plan;
}

// The int8 activations of every tensor-path layer live at the start of the workspace, so their TMA
// descriptor depends only on (workspace, M, K): encoded once and reused across layers and steps.
static const CUtensorMap* cached_tmap_a(dp_plan* plan, const void* ws, int64_t M, int64_t K, int* st) {
  for (const TmapACache& c : plan->a_cache)
    if (c.ptr == ws && c.M == M && c.K == K) return &c.map;
  TmapACache c;
  c.ptr = ws;
  c.M = M;
  c.K = K;
  *st = gemm_encode_a_tiled(&c.map, static_cast<const int8_t*>(ws), M, K);
  if (*st != DP_OK) return nullptr;
  if (plan->a_cache.size() > 64) plan->a_cache.clear();
  plan->a_cache.push_back(c);
  return &plan->a_cache.back().map;
}

static int plan_run_step(dp_plan* plan, int32_t t, const void* const* xs, void* const* ys, void* workspace,
                         int32_t* status, cudaStream_t stream, bool* chained) {
  const int n = static_cast<int>(plan->layers.size());
  // DAQ policy of this step: the activation bits of the time bin t falls into (thirds of the range)
  int act_bits = 8;
  if (plan->daq_timesteps > 0) {
    int64_t bin = static_cast<int64_t>(t < 0 ? 0 : t) * 3 / plan->daq_timesteps;
    act_bits = plan->daq_bits[bin > 2 ? 2 : bin];
  }
  const bool robust = plan->daq_p_e3 < 100000 || act_bits < 8;
  // a group whose rows are too long for the grouped policy DAQ (register-resident, K <= 1280) runs layer by layer
  auto group_splits = [&](int l) { return robust && plan->layers[l].w.K > 1280; };
  for (const std::vector<int>& grp : plan->groups) {
    const PlanLayer& G = plan->layers[grp[0]];
    if (group_splits(grp[0])) continue;
    SimtGroupArgs ga;
    ga.M = G.M;
    ga.N = G.w.N;
    ga.K = G.w.K;
    ga.n_layers = static_cast<int32_t>(grp.size());
    ga.early_w = *chained ? 1 : 0;
    ga.status = status;
    ga.daq_rank = robust ? clip_rank_of(plan->daq_p_e3, G.w.K) : 1;
    ga.daq_bits = act_bits;
    // Plain DAQ runs inside the grouped kernel: every CTA quantizes its layer's few tokens while its
    // first weight copies are in flight (a separate quantization launch in front cost a kernel
    // boundary and a DRAM round trip, 6-8 us of a 35 us group). The percentile / a-bit form keeps
    // its own launch into the workspace.
    ga.q_scratch = robust ? static_cast<int8_t*>(workspace) : nullptr;
    ga.sa_scratch = robust ? reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) +
                                                      align256(static_cast<size_t>(ga.n_layers) * ga.M * ga.K))
                           : nullptr;
    for (size_t i = 0; i < grp.size(); ++i) {
      const int l = grp[i];
      const PlanLayer& L = plan->layers[l];
      if (!xs[l] || !ys[l]) return fail(DP_ERR_INVALID_ARG, "layer %d: NULL x or y", l);
      if (!aligned16(xs[l]) || !aligned16(ys[l])) return fail(DP_ERR_ALIGN, "layer %d: x/y misaligned", l);
      ga.layer[i] = {xs[l], static_cast<uint16_t*>(ys[l]), L.w.qweight, L.w.s_w,
                     static_cast<const uint16_t*>(L.w.bias), L.w.bits};
    }
    int st = launch_simt_group(ga, stream, !(plan->flags & DP_FLAG_NO_PDL));
    if (st != DP_OK) return st;
    *chained = true;
  }
  for (int l = 0; l < n; ++l) {
    const PlanLayer& L = plan->layers[l];
    if (L.M == 0 || (plan->grouped[l] && !group_splits(l))) continue;
    if (!xs[l] || !ys[l]) return fail(DP_ERR_INVALID_ARG, "layer %d: NULL x or y", l);
    if (!aligned16(xs[l]) || !aligned16(ys[l])) return fail(DP_ERR_ALIGN, "layer %d: x/y misaligned", l);
    const CUtensorMap* ta = nullptr;
    if (!L.simt && L.w.bits != 16 && L.w.group_size == 0) {
      int st = DP_OK;
      ta = cached_tmap_a(plan, workspace, L.M, L.w.K, &st);
      if (st != DP_OK) return st;
    }
    // The next tensor-core layer's packed weights and its input start towards L2 while this layer's
    // GEMM runs. A hint, not a reordering: if that input is still to be written (by this layer, say),
    // the hint fetches bytes that the write then replaces in L2, and nothing is read before its turn.
    gemm_set_next_reads(nullptr, 0, nullptr, 0);
    for (int j = l + 1; j < n; ++j) {
      const PlanLayer& Nx = plan->layers[j];
      if (Nx.M == 0 || (plan->grouped[j] && !group_splits(j))) continue;
      const size_t wb = static_cast<size_t>(Nx.w.N) * Nx.w.K * Nx.w.bits / 8;
      const size_t xb = static_cast<size_t>(Nx.M) * Nx.w.K * 2;
      // (only what fits L2 beside this layer's own operands: at tens of thousands of tokens an input
      // is larger than that and the hint would only evict)
      if (!Nx.simt && xs[j] != nullptr) gemm_set_next_reads(Nx.w.qweight, wb, xb <= (32u << 20) ? xs[j] : nullptr, xb);
      break;
    }
    int st = run_linear(&L.w, xs[l], L.w.K, nullptr, L.M, ys[l], L.w.N, workspace, nullptr, status,
                        plan->flags, stream, L.simt ? nullptr : &L.tmap_w, L.bn, L.cg, L.ws, ta, *chained,
                        L.simt ? nullptr : plan->daq_sync, L.simt ? 0 : L.pre,
                        robust ? clip_rank_of(plan->daq_p_e3, L.w.K) : 1, act_bits);
    gemm_set_next_reads(nullptr, 0, nullptr, 0);
    if (st != DP_OK) return st;
    *chained = true;
  }
  return DP_OK;
}

static int check_plan_run(const dp_plan* plan, const int32_t* steps, int32_t n_steps,
                          int32_t start_index, const void* xp, const void* yp, void* workspace,
                          size_t workspace_bytes, uint32_t flags) {
  if (!plan || !xp || !yp) return fail(DP_ERR_INVALID_ARG, "plan, x_ptrs or y_ptrs is NULL");
  if (n_steps < 0 || start_index < 0 || start_index > n_steps || (n_steps > 0 && !steps))
    return fail(DP_ERR_INVALID_ARG, "bad steps/n_steps/start_index");
  if (flags & ~(DP_PLAN_SAME_X | DP_PLAN_SAME_Y)) return fail(DP_ERR_INVALID_ARG, "unknown plan-run flags");
  if (!workspace || workspace_bytes < plan->workspace_bytes || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return fail(DP_ERR_WORKSPACE, "plan workspace needs %zu bytes, 256-byte aligned", plan->workspace_bytes);
  return DP_OK;
}

extern "C" int dp_plan_run(const dp_plan* plan_c, const int32_t* steps, int32_t n_steps,
                           int32_t start_index, const void* const* x_ptrs, void* const* y_ptrs,
                           void* workspace, size_t workspace_bytes, int32_t* device_status,
                           uint32_t flags, dp_stream stream) {
  int st = check_plan_run(plan_c, steps, n_steps, start_index, x_ptrs, y_ptrs, workspace,
                          workspace_bytes, flags);
  if (st != DP_OK) return st;
  dp_plan* plan = const_cast<dp_plan*>(plan_c);
  const int64_t n = static_cast<int64_t>(plan->layers.size());
  bool chained = false;
  for (int32_t i = n_steps - 1 - start_index; i >= 0; --i) {  // reverse(K*)
    const void* const* xs = x_ptrs + ((flags & DP_PLAN_SAME_X) ? 0 : i * n);
    void* const* ys = y_ptrs + ((flags & DP_PLAN_SAME_Y) ? 0 : i * n);
    st = plan_run_step(plan, steps[i], xs, ys, workspace, device_status, static_cast<cudaStream_t>(stream), &chained);
    if (st != DP_OK) return st;
  }
  return DP_OK;
}

extern "C" int dp_plan_run_host(const dp_plan* plan_c, const int32_t* steps, int32_t n_steps,
                                const void* const* x_host, void* x_stage, size_t x_stage_bytes,
                                void* const* y_dev, int32_t d2h_layer, void* const* y_host,
                                void* workspace, size_t workspace_bytes, int32_t* device_status,
                                uint32_t flags, dp_stream stream_) {
  int st = check_plan_run(plan_c, steps, n_steps, 0, x_host, y_dev, workspace, workspace_bytes,
                          flags & DP_PLAN_SAME_X);
  if (st != DP_OK) return st;
  if (flags & ~DP_PLAN_SAME_X) return fail(DP_ERR_INVALID_ARG, "unknown plan-run flags");
  dp_plan* plan = const_cast<dp_plan*>(plan_c);
  const int64_t n = static_cast<int64_t>(plan->layers.size());
  if (!x_stage || x_stage_bytes < 2 * plan->x_bytes || (reinterpret_cast<uintptr_t>(x_stage) & 255u))
    return fail(DP_ERR_WORKSPACE, "x_stage needs %zu bytes, 256-byte aligned", 2 * plan->x_bytes);
  if (d2h_layer >= n || (d2h_layer >= 0 && !y_host))
    return fail(DP_ERR_INVALID_ARG, "bad d2h_layer / y_host");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  std::vector<const void*> xs(n);
  // The copy stream starts behind everything already enqueued on `stream`: an earlier call's last
  // steps (or any other work of the caller) may still be reading the staging halves.
  DP_CUDA_OK(cudaEventRecord(plan->ev_entry, stream));
  DP_CUDA_OK(cudaStreamWaitEvent(plan->copy_stream, plan->ev_entry, 0));
  int j = 0;
  for (int32_t i = n_steps - 1; i >= 0; --i, ++j) {
    const int h = j & 1;
    uint8_t* stage = static_cast<uint8_t*>(x_stage) + h * plan->x_bytes;
    if (j >= 2) DP_CUDA_OK(cudaStreamWaitEvent(plan->copy_stream, plan->ev_consumed[h], 0));
    const void* const* src = x_host + ((flags & DP_PLAN_SAME_X) ? 0 : i * n);
    for (int64_t l = 0; l < n; ++l) {
      const PlanLayer& L = plan->layers[l];
      xs[l] = stage + L.x_offset;
      if (L.M == 0) continue;
      if (!src[l]) return fail(DP_ERR_INVALID_ARG, "layer %lld: NULL host input", (long long)l);
      DP_CUDA_OK(cudaMemcpyAsync(stage + L.x_offset, src[l], static_cast<size_t>(L.M) * L.w.K * 2,
                                 cudaMemcpyHostToDevice, plan->copy_stream));
    }
    DP_CUDA_OK(cudaEventRecord(plan->ev_copied[h], plan->copy_stream));
    DP_CUDA_OK(cudaStreamWaitEvent(stream, plan->ev_copied[h], 0));
    bool chained = false;  // an event wait precedes every step's first launch
    st = plan_run_step(plan, steps[i], xs.data(), y_dev, workspace, device_status, stream, &chained);
    if (st != DP_OK) return st;
    DP_CUDA_OK(cudaEventRecord(plan->ev_consumed[h], stream));
    if (d2h_layer >= 0) {
      const PlanLayer& L = plan->layers[d2h_layer];
      DP_CUDA_OK(cudaMemcpyAsync(y_host[i], y_dev[d2h_layer], static_cast<size_t>(L.M) * L.w.N * 2,
                                 cudaMemcpyDeviceToHost, stream));
    }
  }
  return DP_OK;
}

// ---- Algorithm 2, Phase A --------------------------------------------------------------------------
namespace {
struct BitMove {
  double score;
  int32_t layer;
  bool operator<(const BitMove& o) const {  // max-heap on score, ties to the lower layer index
    return score < o.score || (score == o.score && layer > o.layer);
  }
};
}  // namespace

extern "C" int dp_plan_phase_a(const dp_phase_a_problem* q, int32_t* bitplan_out, uint8_t* kept_out,
                               double* totals_out, int32_t* feasible) {
  if (!q || !bitplan_out || !kept_out) return fail(DP_ERR_INVALID_ARG, "dp_plan_phase_a: NULL argument");
  if (q->n_steps <= 0 || q->n_layers <= 0 || !q->drift || !q->step_cost || !q->n_options || !q->opt_bits ||
      !q->opt_c_lat || !q->opt_c_mem || !q->sens || !(q->rho >= 0.0 && q->rho <= 1.0))
    return fail(DP_ERR_INVALID_ARG, "dp_plan_phase_a: bad problem description");
  const int32_t T = q->n_steps, L = q->n_layers;
  std::vector<int64_t> off(L + 1, 0);
  for (int32_t l = 0; l < L; ++l) {
    if (q->n_options[l] <= 0) return fail(DP_ERR_INVALID_ARG, "dp_plan_phase_a: layer %d has no bit option", l);
    off[l + 1] = off[l] + q->n_options[l];
  }
  const int32_t tail0 = T - static_cast<int32_t>(q->rho * T);  // steps tail0 .. T-1 are protected
  // prunable steps by ascending drift (ties: lower timestep first)
  std::vector<int32_t> order;
  for (int32_t t = 0; t < tail0; ++t) order.push_back(t);
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return q->drift[a] < q->drift[b]; });
  size_t next_step = 0;
  std::vector<int32_t> cur(L, 0);  // option index per layer
  double C_lat = 0.0, C_mem = 0.0;
  for (int32_t t = 0; t < T; ++t) {
    kept_out[t] = 1;
    C_lat += q->step_cost[t];
  }
  auto score_of = [&](int32_t l) {
    const int64_t i = off[l] + cur[l];
    return (q->opt_c_lat[i] - q->opt_c_lat[i + 1]) / (q->eps + q->sens[l]);
  };
  std::priority_queue<BitMove> heap;
  for (int32_t l = 0; l < L; ++l) {
    C_lat += q->opt_c_lat[off[l]];
    C_mem += q->opt_c_mem[off[l]];
    if (q->n_options[l] > 1) heap.push({score_of(l), l});
  }
  int ok = 1;
  while (C_lat > q->B_lat || C_mem > q->B_mem) {
    const bool has_step = next_step < order.size();
    // bit candidate: the best-scored move that leaves the memory within budget, else the best-scored
    // move; moves skipped while looking go back on the heap
    bool has_bit = !heap.empty();
    BitMove pick{0.0, -1};
    if (has_bit) {
      std::vector<BitMove> skipped;
      while (!heap.empty()) {
        const BitMove m = heap.top();
        const int64_t i = off[m.layer] + cur[m.layer];
        if (C_mem - (q->opt_c_mem[i] - q->opt_c_mem[i + 1]) <= q->B_mem) {
          pick = m;
          break;
        }
        skipped.push_back(m);
        heap.pop();
      }
      if (pick.layer < 0) pick = skipped.front();  // none satisfies the clause: the top move
      else heap.pop();
      for (const BitMove& m : skipped)
        if (m.layer != pick.layer) heap.push(m);
    }
    if (!has_step && !has_bit) {
      ok = 0;
      break;
    }
    const int32_t t = has_step ? order[next_step] : -1;
    const double s_step = has_step ? q->step_cost[t] / (q->eps + q->drift[t]) : 0.0;
    if (has_step && (!has_bit || s_step > pick.score)) {
      kept_out[t] = 0;
      C_lat -= q->step_cost[t];
      ++next_step;
      if (has_bit) heap.push(pick);
    } else {
      const int32_t l = pick.layer;
      const int64_t i = off[l] + cur[l];
      C_lat -= q->opt_c_lat[i] - q->opt_c_lat[i + 1];
      C_mem -= q->opt_c_mem[i] - q->opt_c_mem[i + 1];
      ++cur[l];
      if (cur[l] + 1 < q->n_options[l]) heap.push({score_of(l), l});
    }
  }
  for (int32_t l = 0; l < L; ++l) bitplan_out[l] = q->opt_bits[off[l] + cur[l]];
  if (totals_out) {
    totals_out[0] = C_lat;
    totals_out[1] = C_mem;
  }
  if (feasible) *feasible = ok;
  return DP_OK;
}

extern "C" int dp_layer_latency_us(const dp_weight* w, int64_t M, uint32_t flags, int32_t reps, float* us_out) {
  if (!us_out || reps <= 0 || reps > 10000) return fail(DP_ERR_INVALID_ARG, "dp_layer_latency_us: bad reps / us_out");
  int st = check_weight(w);
  if (st != DP_OK) return st;
  if (M <= 0) return fail(DP_ERR_SHAPE, "dp_layer_latency_us: M must be positive");
  if (flags & ~kLinearFlags) return fail(DP_ERR_INVALID_ARG, "unknown flag bits 0x%x", flags);
  if (int tst = check_tile_flags(flags, w->N)) return tst;
  st = check_device();
  if (st != DP_OK) return st;
  void *x = nullptr, *y = nullptr, *ws = nullptr;
  cudaStream_t stream = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  const size_t xb = static_cast<size_t>(M) * w->K * 2, yb = static_cast<size_t>(M) * w->N * 2;
  const size_t wb = w->group_size > 0 ? dp_wq_linear_workspace_grouped(M, w)
                                      : dp_wq_linear_workspace(M, w->N, w->K, w->bits, flags);
  cudaError_t e = cudaMalloc(&x, xb);
  if (e == cudaSuccess) e = cudaMalloc(&y, yb);
  if (e == cudaSuccess) e = cudaMalloc(&ws, wb);
  if (e == cudaSuccess) e = cudaMemset(x, 0x3c, xb);  // bf16 0x3c3c = 0.0115: finite, non-zero
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  st = e == cudaSuccess ? DP_OK : fail(DP_ERR_CUDA, "dp_layer_latency_us set-up: %s", cudaGetErrorString(e));
  for (int it = 0; it < 2 + reps && st == DP_OK; ++it) {
    if (it == 2) cudaEventRecord(e0, stream);
    st = check_linear_args(w, x, w->K, nullptr, M, y, w->N, ws, wb, nullptr, flags);
    if (st == DP_OK)
      st = run_linear(w, x, w->K, nullptr, M, y, w->N, ws, nullptr, nullptr, flags, stream, nullptr, 0, 0, 0, nullptr,
                      it > 0);
  }
  if (st == DP_OK) {
    cudaEventRecord(e1, stream);
    e = cudaEventSynchronize(e1);
    float ms = 0.0f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e != cudaSuccess) st = fail(DP_ERR_CUDA, "dp_layer_latency_us timing: %s", cudaGetErrorString(e));
    else *us_out = ms * 1000.0f / static_cast<float>(reps);
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (stream) cudaStreamDestroy(stream);
  cudaFree(x);
  cudaFree(y);
  cudaFree(ws);
  return st;
}

// ---- host helpers ----------------------------------------------------------------------------------
extern "C" int dp_pack_weights_host(const int8_t* w, int32_t N, int32_t K, int32_t bits, void* out) {
  if (!w || !out || N <= 0 || K <= 0) return fail(DP_ERR_INVALID_ARG, "dp_pack_weights_host: bad arguments");
  if (bits == 8) {
    memcpy(out, w, static_cast<size_t>(N) * K);
    return DP_OK;
  }
  if (bits != 3 && bits != 4) return fail(DP_ERR_BITS, "bits=%d not in {3,4,8}", bits);
  if (K % 32) return fail(DP_ERR_SHAPE, "K=%d not a multiple of 32", K);
  const int half = 1 << (bits - 1);
  uint32_t* o = static_cast<uint32_t*>(out);
  for (int64_t n = 0; n < N; ++n) {
    uint64_t buf = 0;
    int nb = 0;
    for (int64_t k = 0; k < K; ++k) {
      const int v = w[n * K + k];
      if (v < -half || v >= half)
        return fail(DP_ERR_INVALID_ARG, "weight %d at [%lld,%lld] outside the %d-bit range", v,
                    (long long)n, (long long)k, bits);
      buf |= static_cast<uint64_t>(v + half) << nb;
      nb += bits;
      if (nb >= 32) {
        *o++ = static_cast<uint32_t>(buf);
        buf >>= 32;
        nb -= 32;
      }
    }
  }
  return DP_OK;
}

extern "C" void dp_debug_skip_stage_load(int32_t k_block) { dp::gemm_debug_skip_stage_load(k_block); }

extern "C" int32_t dp_clip_rank(int32_t clip_percentile_e3, int32_t K) {
  if (clip_percentile_e3 < 1 || clip_percentile_e3 > 100000 || K < 1) return 0;
  return dp::clip_rank_of(clip_percentile_e3, K);
}

extern "C" const char* dp_status_string(int s) {
  switch (s) {
    case DP_OK: return "DP_OK";
    case DP_ERR_INVALID_ARG: return "DP_ERR_INVALID_ARG";
    case DP_ERR_SHAPE: return "DP_ERR_SHAPE";
    case DP_ERR_ALIGN: return "DP_ERR_ALIGN";
    case DP_ERR_BITS: return "DP_ERR_BITS";
    case DP_ERR_WORKSPACE: return "DP_ERR_WORKSPACE";
    case DP_ERR_ARCH: return "DP_ERR_ARCH";
    case DP_ERR_CUDA: return "DP_ERR_CUDA";
    case DP_ERR_TIMEOUT: return "DP_ERR_TIMEOUT";
    default: return "DP_ERR_UNKNOWN";
  }
}
extern "C" const char* dp_last_error(void) { return dp::g_err; }
extern "C" int dp_version(void) { return (0 << 16) | 1; }
