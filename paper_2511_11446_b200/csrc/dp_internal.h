// Internal interfaces between the translation units of libdiffpro (host side).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/diffpro.h"

namespace dp {

// Order in which the int8 codes of a token are stored along K in the activation scratch.
enum KOrder {
  KORDER_NATURAL = 0,   // q[k] at byte k
  KORDER_EVEN_ODD = 1   // every group of 8 codes stored as k = 0,2,4,6,1,3,5,7 (4-bit weight path)
};
// The order the tensor-core path wants for weights of this width when it runs DAQ itself.
int gemm_korder(int32_t bits);

// daq.cu
// Expansion of a packed weight matrix to int8 [N][K] (true values, k ascending) in global scratch,
// run by extra CTAs of a DAQ launch or on its own: `units` = N * K / 32 units of 32 codes.
struct UnpackJob {
  const uint32_t* packed;
  int8_t* out;
  int64_t units;
  int32_t bits;         // 3 or 4
  int32_t first_block;  // filled by the launcher: CTAs from here on unpack
};
int launch_daq(const void* x, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq,
               float* s_a, int32_t* rowsum, int korder, bool tiled, cudaStream_t stream, bool pdl,
               const UnpackJob* unpack = nullptr);
int launch_unpack(const UnpackJob& job, cudaStream_t stream, bool pdl);
// ln.cu -- LayerNorm + adaLN modulation + DAQ in one pass (K a multiple of 8, at most 4608)
int launch_ln_modulate_daq(const void* x, int64_t M, int64_t K, int64_t ldx, const void* shift, const void* scale,
                           int64_t rows_per_sample, float eps, int8_t* q, int64_t ldq, float* s_a,
                           cudaStream_t stream, bool pdl);
int launch_daq_robust(const void* x, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq, float* s_a,
                      int32_t* rowsum, int clip_rank, int act_bits, bool tiled, cudaStream_t stream, bool pdl,
                      const UnpackJob* unpack);

// simt.cu — CUDA-core weight-streaming linear for small M (DAQ fused in the CTA prologue).
struct SimtArgs {
  const void* x;        // bf16 [M][ldx] or int8 [M][ldx] when s_a_in != nullptr
  int64_t ldx;
  const float* s_a_in;  // nullptr -> DAQ inside the kernel
  int64_t M;
  int32_t N, K, bits;
  const void* qweight;
  const float* s_w;
  const uint16_t* bias;
  uint16_t* y;
  int64_t ldy;
  int8_t* dbg_q;
  int64_t dbg_ldq;
  float* dbg_sa;
  int32_t* dbg_acc;
  int64_t dbg_ldacc;
  int32_t early_w;  // weights may be fetched before the preceding kernel on the stream has finished
  int32_t* status;  // device word raised to DP_ERR_TIMEOUT when a bounded wait expires (may be null)
};
int launch_simt_linear(const SimtArgs& a, cudaStream_t stream, bool pdl);
// Up to kSimtGroupMax layers of one shape (bf16 inputs [M][K], outputs [M][N], both contiguous).
constexpr int kSimtGroupMax = 32;
struct SimtGroupArgs {
  struct Layer {
    const void* x;
    uint16_t* y;
    const void* qweight;
    const float* s_w;
    const uint16_t* bias;
    int32_t bits;
  } layer[kSimtGroupMax];
  int64_t M;
  int32_t N, K, n_layers;
  int32_t early_w;
  // Scratch for the group's int8 tokens [n_layers][M][K] and scales [n_layers][M]: when given, one
  // small kernel quantizes all tokens of the group first and the main kernel's CTAs only fetch the
  // codes; when null every CTA quantizes its tokens itself.
  int8_t* q_scratch;
  float* sa_scratch;
  int32_t* status;  // as SimtArgs::status
  int32_t daq_rank, daq_bits;  // the group's DAQ rule: (1, 8) = absmax, 8 bits; else percentile clip / a-bit codes
  // Matrix-instruction form: CTAs [cta_begin[l], cta_begin[l + 1]) of grid.x work on layer l (filled
  // by launch_simt_group: more CTAs for the layers that take longer).
  int32_t cta_begin[kSimtGroupMax + 1];
};
size_t simt_group_scratch_bytes(int64_t M, int32_t K, int32_t n_layers);
int launch_simt_group(const SimtGroupArgs& g, cudaStream_t stream, bool pdl);
size_t simt_max_k();

// gemm_tc.cu — tcgen05 kind::i8 GEMM with in-smem weight unpack and fused dequant epilogue.
struct GemmTile {  // kernel variant
  int bn;          // tile width in output channels: 64, 128, 192 or 256
};
struct GemmProblem {
  CUtensorMap tmap_a;  // int8 activations [M][K]
  CUtensorMap tmap_w;  // packed weights, byte view [N][K*bits/8]
  const float* s_a;    // [M]
  const float* s_w;    // [N]
  const uint16_t* bias;
  uint16_t* y;
  int64_t ldy;
  int32_t* dbg_acc;
  int64_t dbg_ldacc;
  const uint16_t* res = nullptr;  // residual (and gate) taken into the epilogue, see dp_wq_linear_residual
  int64_t ldr = 0;
  const uint16_t* gate = nullptr;
  int64_t rows_per_gate = 1;
  int64_t M;
  int32_t N, K, bits, bn;
  int32_t cg;       // 1: one CTA per 128-row tile; 2: a CTA pair per 256-row tile
  int32_t ws;       // 1: weight-stationary pair kernel (cg == 2, bn in {192, 256}); 2: activation-stationary
                    // pair kernel (bn = width of its column sub-blocks)
  int32_t korder;   // KOrder of the activations behind tmap_a
  int32_t a_tiled;  // the activations behind tmap_a are stored as 128 x 128 tiles (see gemm_encode_a_tiled)
  int32_t early_w;  // the preceding kernel on the stream is this call's own DAQ: weights may be
                    // fetched before it has finished
  int32_t* status;
  // In-kernel DAQ (x != nullptr): the GEMM kernel quantizes x into q_out / s_a_out (the buffers
  // behind tmap_a and s_a) itself; sync = zeroed counters, one per 128-token tile plus one.
  const uint16_t* x;
  int64_t ldx;
  int8_t* q_out;
  float* s_a_out;
  int32_t* sync;
};
// allow: bit 1 = single-CTA tiles permitted, bit 2 = CTA-pair tiles permitted
void gemm_pick_tile(int64_t M, int32_t N, int32_t K, int32_t bits, uint32_t allow, int* bn_out, int* cg_out);
int gemm_max_pairs();
int gemm_encode_a(CUtensorMap* out, const int8_t* q, int64_t M, int64_t K, int64_t ldq);
// int8 activations stored as [ceil(M/128)][K/128] tiles of 128 tokens x 128 codes (16 KB each).
int gemm_encode_a_tiled(CUtensorMap* out, const int8_t* q, int64_t M, int64_t K);
int gemm_encode_w(CUtensorMap* out, const void* qweight, int32_t N, int32_t K, int32_t bits,
                  int32_t bn, int32_t cg);
int launch_gemm(const GemmProblem& p, cudaStream_t stream, bool pdl);
void gemm_debug_skip_stage_load(int32_t kb);  // see dp_debug_skip_stage_load
// Two ranges (a plan's next layer's packed weights and its bf16 input) that the calling thread's next
// launch_gemm sends on their way into L2 while it runs; cleared by that launch. Hints: any valid
// device ranges of the caller's, or nullptr.
void gemm_set_next_reads(const void* w, size_t w_bytes, const void* x, size_t x_bytes);

// gemm_ws.cu -- weight-stationary CTA-pair kernel (K <= 1152, N a multiple of 192 or 256).
bool gemm_ws_supported(int32_t N, int32_t K);
int gemm_ws_pick_bn(int32_t N);
int launch_gemm_ws(const GemmProblem& p, cudaStream_t stream, bool pdl);
// Per-device set-up (kernel attributes, tensor-map encoder, SM and CTA-pair counts), called once per
// device by check_device() with that device current.
int gemm_init_device(int dev, int* num_sms_out, int* max_pairs_out);
int gemm_ws_init_device();
int gemm_as_init_device();
int gemm_bf16_init_device();
int gemm_grp_init_device();

// gemm_grp.cu -- layers with group-wise weight scales (and zero-points): folding tensor-core kernel.
int launch_gemm_grp(const int8_t* q, int64_t ldq, bool a_tiled, const float* s_a, const int8_t* w8, int32_t bits,
                    int32_t g, const float* s_w, const uint8_t* zeros, const uint16_t* bias, int32_t* rowsum, int64_t M,
                    int32_t N, int32_t K, uint16_t* y, int64_t ldy, int32_t* status, cudaStream_t stream, bool pdl);

// gemm_bf16.cu -- pass-through linear of 16-bit layers (bf16 x bf16 -> fp32 -> bf16, tcgen05 kind::f16).
int launch_gemm_bf16(const void* x, int64_t ldx, const void* w, const uint16_t* bias, int64_t M, int32_t N, int32_t K,
                     uint16_t* y, int64_t ldy, int32_t* status, cudaStream_t stream, bool pdl);
int gemm_encode_bytes_2d(CUtensorMap* out, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
                         uint32_t box_inner, uint32_t box_rows);

// gemm_as.cu -- activation-stationary CTA-pair kernel (K <= 1152, 8-bit weights, tiled activations).
bool gemm_as_supported(int32_t N, int32_t K);
// Sub-block width (forced_bns, or the model's choice when 0) and sub-blocks per slice; *bns_out = 0 if none fits.
void gemm_as_config(int64_t M, int32_t N, int32_t K, int forced_bns, int* bns_out, int* nsub_out);
int launch_gemm_as(const GemmProblem& p, cudaStream_t stream, bool pdl);

int num_sms();

}  // namespace dp
