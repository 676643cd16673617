/*
 * diffpro.h — C ABI of libdiffpro: the quantized linear layer of a deployed DiffPro plan
 * (arxiv 2511.11446) as hand-written CUDA for NVIDIA B200 (sm_100a).
 *
 * One call of the hot path =
 *   DAQ (Step 3, Eq. "daq": symmetric INT8, zero-point 0, scale tau/(2^(b-1)-1) with b = 8; here
 *        tau = per-token absmax over K, i.e. the p = 100, one-group case of the equation)
 *   -> unpack of the GPTQ-style packed b-bit weights (Step 1/Step 3: weights are stored packed;
 *        Algorithm 1 names the widths 3, 4 and 8)
 *   -> INT8 x INT8 -> INT32 GEMM with per-output-channel weight scales (Step 5; Implementation)
 *   -> dequantisation y = acc * s_a[m] * s_w[n] + bias[n], stored as bf16.
 * dp_plan_run is Phase B of Algorithm 2: for t in reverse(K*), run every wrapped linear per the
 * bit plan. dp_daq_quantize_robust / dp_plan_set_daq add the equation's percentile clip (p < 100)
 * and Phase B's activation bits per time bin.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller unless the name says `host`.
 *   - Nothing on the hot path (dp_daq_quantize, dp_wq_linear, dp_plan_run) allocates, frees or
 *     synchronises: work is enqueued on `stream` and the call returns.
 *   - Return value is a dp_status (0 = DP_OK). Argument errors are found on the host before any
 *     launch; nothing is enqueued in that case. dp_last_error() gives a thread-local detail string.
 *   - Data pointers must be 16-byte aligned and leading dimensions (in elements) must make every
 *     row start 16-byte aligned, else DP_ERR_ALIGN.
 *   - Only compute-capability 10.x devices are accepted (DP_ERR_ARCH). There is no CPU fallback.
 *   - Device-side waits are bounded; if one expires the kernel records DP_ERR_TIMEOUT in the
 *     `device_status` word (when given) and exits without trapping.
 */
#ifndef DIFFPRO_H_
#define DIFFPRO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum dp_status {
  DP_OK = 0,
  DP_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, negative size, bad flag        */
  DP_ERR_SHAPE = 2,       /* K not a multiple of 128, N not a multiple of 16, ld < row length  */
  DP_ERR_ALIGN = 3,       /* pointer or row pitch not 16-byte aligned                          */
  DP_ERR_BITS = 4,        /* weight bit-width not in {3,4,8,16}                                */
  DP_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than dp_*_workspace() says              */
  DP_ERR_ARCH = 6,        /* current device is not sm_100                                      */
  DP_ERR_CUDA = 7,        /* a CUDA runtime/driver call failed (see dp_last_error)             */
  DP_ERR_TIMEOUT = 8      /* written by a kernel into device_status when a bounded wait expired */
} dp_status;

/* A CUDA stream handle (cudaStream_t), passed as an opaque pointer so this header needs no CUDA. */
typedef void* dp_stream;

/*
 * Constant data of one quantized linear (device pointers, caller-owned, read-only).
 * Weights are symmetric per-output-channel b-bit integers w[n][k] in [-2^(b-1), 2^(b-1)-1]:
 *   bits == 8 : qweight is int8 [N][K], two's complement, row-major.
 *   bits == 4 : qweight is uint32 [N][K/8];  field k of row n = bits [4k, 4k+4) of the row's
 *               little-endian bit stream (8 values per 32-bit word), code u = w + 8.
 *   bits == 3 : qweight is uint32 [N][3K/32]; field k = bits [3k, 3k+3) of the row's bit stream
 *               (32 values per 3 words; fields 10 and 21 of each group straddle words), u = w + 4.
 *   bits == 16: a layer the plan keeps in 16-bit precision (Step 1's tiering sends the most sensitive
 *               layers there; the paper's best plans freeze about a fifth of them): qweight is bf16
 *               [N][K] row-major, s_w is ignored (may be NULL), the layer is y = x . W^T + bias with
 *               fp32 accumulation and no DAQ; N % 64 == 0.
 * s_w  : fp32 [N], one scale per output channel (Step 5).
 * bias : bf16 [N] or NULL.
 * Group-wise scales (Step 2: the GPTQ storage format of the paper's plans, groups of 32..288 input
 * channels with a scale and a zero-point each): group_size = g > 0 (g % 32 == 0, K % g == 0, bits in
 * {3, 4, 8}, N % 128 == 0) makes s_w fp32 [N][K/g], one scale per output channel and group of g
 * consecutive k, and `zeros` uint8 [N][K/g] or NULL the zero-points in code units (NULL = 2^(bits-1),
 * the symmetric code): the weight is s_w[n][k/g] * (u[n][k] - zeros[n][k/g]). The layer is then
 *     acc_G = sum_{k in group G} q[m,k] * (u[n,k] - z[n,G])            (exact int32)
 *     t = 0;  for G = 0 .. K/g - 1:  t = fma((float)acc_G, s_w[n][G], t)   (fp32, in this order)
 *     y = bf16_rne(fma(t, s_a[m], bias[n]))
 * group_size = 0: one scale per output channel, `zeros` must be NULL.
 * Requirements: K % 128 == 0, N % 16 == 0, N,K >= 128.
 */
typedef struct dp_weight {
  int32_t N;
  int32_t K;
  int32_t bits;
  int32_t group_size; /* 0 = one scale per output channel */
  const void* qweight;
  const float* s_w;
  const void* bias;
  const void* zeros;  /* group-wise layers only: uint8 [N][K/g] or NULL */
} dp_weight;

/* Optional taps for tests: any member may be NULL. */
typedef struct dp_debug {
  int8_t* q;      /* [M][ldq] receives the DAQ codes                     */
  int64_t ldq;
  float* s_a;     /* [M] receives the activation scales                  */
  int32_t* acc;   /* [M][ldacc] receives the raw int32 accumulators      */
  int64_t ldacc;
} dp_debug;

/* flags for dp_wq_linear / dp_plan_create */
#define DP_FLAG_NONE 0u
#define DP_FLAG_FORCE_SIMT 1u   /* route through the CUDA-core weight-streaming kernel (any M)   */
#define DP_FLAG_FORCE_MMA 2u    /* route through the tcgen05 kernel even for small M              */
#define DP_FLAG_NO_PDL 4u       /* do not use programmatic dependent launch between the kernels  */
/* Tuning/testing: force the tensor-core kernel's tile width in output channels (64, 128, 192 or
 * 256; must divide N) instead of letting the library choose. */
#define DP_FLAG_TILE_N(bn) ((uint32_t)((bn) / 64) << 8)
#define DP_FLAG_TILE_N_MASK 0x700u
/* Tuning/testing: force (or forbid) the tensor-core kernel variant in which the two CTAs of a
 * thread-block cluster share a 256-row tile (tile width 128, 192 or 256 only). */
#define DP_FLAG_CTA_PAIR 0x800u
#define DP_FLAG_NO_CTA_PAIR 0x1000u
/* Tuning/testing: force (or forbid) the weight-stationary CTA-pair kernel, which keeps a strip of
 * output channels resident in shared memory for the whole K (K <= 1152, N a multiple of 192). */
#define DP_FLAG_WEIGHT_STATIONARY 0x2000u
#define DP_FLAG_NO_WEIGHT_STATIONARY 0x4000u
/* Tuning/testing: force (or forbid) the activation-stationary CTA-pair kernel, which keeps the int8
 * codes of a 256-token strip resident in shared memory for the whole K and streams only weight
 * tiles (K <= 1152, N a multiple of 64, 8-bit weights or the unpack-first form, DAQ run by the
 * library). DP_FLAG_TILE_N then names the width of the column sub-blocks it walks. */
#define DP_FLAG_ACT_STATIONARY 0x200000u
#define DP_FLAG_NO_ACT_STATIONARY 0x400000u

/* dp_plan_create only: choose each layer's tensor-core kernel variant (tile width, single CTA /
 * CTA pair / weight-stationary) by timing the candidates on the device during plan creation
 * (allocates scratch, launches and synchronises; a few milliseconds per distinct layer shape)
 * instead of by the built-in cost model. */
#define DP_FLAG_AUTOTUNE 0x10000u
/* dp_plan_create only: the caller states that, within one timestep, the inputs of the plan's
 * small-M layers (M <= 32: in a DiT the adaLN modulation linears, which consume only the
 * timestep/class embedding) do not depend on any other layer's output. dp_plan_run then runs
 * those layers first in each step, equal shapes grouped into one launch; results are unchanged. */
#define DP_FLAG_GROUP_SMALL_M 0x20000u

/* dp_plan_create only: let the plan's tensor-core GEMM kernels quantize their activations
 * themselves instead of running DAQ as a kernel of its own in front of each GEMM: the CTAs share
 * the tokens, publish finished 128-token tiles on counters the plan owns, and start the tiles
 * whose tokens are ready. One launch per layer instead of two; results are identical. Off by
 * default: on B200 the two-kernel form is faster, because its small DAQ kernel is already resident
 * (programmatic dependent launch) while the previous GEMM drains. */
#define DP_FLAG_FUSED_DAQ 0x40000u

/* dp_wq_linear and dp_plan_create, packed bit-widths (3, 4) on the tensor-core path: where the
 * packed weights are expanded (the unpack of the GPTQ-style packed weights of Step 3). UNPACK_FIRST: once
 * per call to int8 [N][K] in the workspace (extra CTAs of the DAQ launch; a launch of its own when the activations arrive
 * quantized), the 8-bit kernel then runs on that copy. NO_UNPACK_FIRST: tile by tile in shared memory
 * inside the GEMM. The first form avoids repeating the expansion in every CTA that needs a weight
 * tile (M/128 of them) and was faster on B200 at every size measured except where the
 * weight-stationary kernel applies (there equal), so it is the default whenever the library runs DAQ
 * itself; with quantized activations (s_a given) the default is the in-GEMM form, which needs no
 * workspace. The copy lives only for the call, the weights stay packed in memory, results are
 * identical. Adds N*K bytes to the workspace (dp_wq_linear_workspace counts them unless
 * NO_UNPACK_FIRST is given). With DP_FLAG_AUTOTUNE the plan times both forms per layer shape.
 * Giving both flags is an error. */
#define DP_FLAG_UNPACK_FIRST 0x80000u
#define DP_FLAG_NO_UNPACK_FIRST 0x100000u

/* flags for dp_plan_run */
#define DP_PLAN_SAME_X 1u       /* x_ptrs has n_layers entries reused by every step              */
#define DP_PLAN_SAME_Y 2u       /* y_ptrs has n_layers entries reused (overwritten) every step   */

/*
 * Dynamic activation quantization of a bf16 matrix, one scale per row (token).
 *   Step 3, Eq. "daq" with b = 8, zero-point 0, tau = max_k |x[m,k]|:
 *     a      = max_k |x[m,k]|
 *     s_a[m] = a / 127                       (fp32, round to nearest)
 *     q[m,k] = clamp(RNE(x[m,k] * (127/a)), -127, 127)   (127/a is one fp32 division; the product
 *              is rounded once, half to even, to an integer)
 *     a < 2^-100 (incl. 0): s_a[m] = 0 and q[m,:] = 0.
 *   x      : bf16 [M][ldx], ldx >= K, ldx % 8 == 0
 *   q      : int8 [M][ldq], ldq >= K, ldq % 16 == 0
 *   s_a    : fp32 [M]
 *   rowsum : int32 [M] receives sum_k q[m,k], or NULL
 * K % 8 == 0, 8 <= K <= 65536. M == 0 is a no-op returning DP_OK. Non-finite inputs are outside
 * the contract.
 */
int dp_daq_quantize(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq,
                    float* s_a, int32_t* rowsum, dp_stream stream);

/*
 * The same with the equation's percentile clip and with fewer activation bits.
 *   Step 3, Eq. "daq": tau = Percentile(|v|, p); Step 6 / Algorithm 2 Phase B: the activation bits of
 *   a forward pass come from the time bin of its step. Reading: the percentile is the nearest-rank one
 *   over the K magnitudes of a token and is passed as its rank from the top,
 *     clip_rank = K - ceil(p K / 100) + 1     (p = 100 -> 1; p = 99.9 -> 2 at K = 1152, 5 at K = 4608),
 *   so tau = the clip_rank-th largest |x[m,k]|, repeats counted. With qmax = 2^(act_bits-1) - 1:
 *     s_a[m] = tau / qmax,   q[m,k] = clamp(RNE(x[m,k] * (qmax/tau)), -qmax, qmax)
 *   (values beyond tau land on the extreme codes, which is what clipping to [-tau, tau] before the
 *   division gives); tau < 2^-100: s_a[m] = 0, q[m,:] = 0. clip_rank = 1, act_bits = 8 is dp_daq_quantize.
 * Arguments and layouts as dp_daq_quantize; 1 <= clip_rank <= min(K, 64) (DP_ERR_INVALID_ARG),
 * 2 <= act_bits <= 8 (DP_ERR_BITS), K % 8 == 0 and 8 <= K <= 4608 (DP_ERR_SHAPE). The codes are
 * ordinary int8, so dp_wq_linear takes them with their scales as quantized activations.
 */
int dp_daq_quantize_robust(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq,
                           float* s_a, int32_t* rowsum, int32_t clip_rank, int32_t act_bits,
                           dp_stream stream);

/*
 * The rank, counted from the largest, of the nearest-rank percentile that dp_daq_quantize_robust takes
 * as clip_rank: K - ceil(p K / 100) + 1 for p = clip_percentile_e3 / 1000 percent (Eq. "daq":
 * tau = Percentile(|v|, p); 100000 -> 1, the maximum). Host arithmetic only; returns 0 when
 * clip_percentile_e3 is outside [1, 100000] or K < 1.
 */
int32_t dp_clip_rank(int32_t clip_percentile_e3, int32_t K);

/* Bytes of device scratch dp_wq_linear needs for this problem (holds the int8 activations and
 * their scales between the two kernels of the large-M path). Never 0; multiple of 256. */
size_t dp_wq_linear_workspace(int64_t M, int32_t N, int32_t K, int32_t bits, uint32_t flags);

/* The same for a layer with group-wise scales (w->group_size > 0): such a layer always runs on the
 * tensor cores, whatever M is, on an int8 copy of its weights, and with zero-points also needs the
 * tokens' per-group code sums: the bytes for all of that. */
size_t dp_wq_linear_workspace_grouped(int64_t M, const dp_weight* w);

/*
 * One quantized linear: y[M][N] = dequant( DAQ(x)[M][K] . unpack(w)[N][K]^T ) + bias.
 *   Step 5 / Implementation: INT8 x INT8 -> INT32, per-output-channel weight scale; epilogue
 *     t = (float)acc; sc = s_a[m] * s_w[n]; y = bf16_rne(fma(t, sc, bias[n]))     (all fp32).
 *   w        : host pointer to a dp_weight whose members are device pointers
 *   x, ldx   : s_a_in == NULL -> bf16 [M][ldx] (DAQ runs inside the call);
 *              s_a_in != NULL -> int8 [M][ldx] already quantized, with scales s_a_in fp32 [M]
 *   y, ldy   : bf16 [M][ldy], ldy >= N, ldy % 8 == 0
 *   workspace: >= dp_wq_linear_workspace(...) bytes, 256-byte aligned; contents undefined after
 *   dbg      : NULL or taps (slower path when dbg->acc is set)
 *   device_status : int32 device word or NULL; set to DP_ERR_TIMEOUT by a kernel whose wait expired
 * M == 0 is a no-op. Calls on the same stream are ordered; the workspace may be reused by the
 * next call on that stream. A layer with w->group_size > 0 needs dp_wq_linear_workspace_grouped bytes,
 * takes bf16 activations only (s_a_in NULL) and has no taps. For w->bits == 16 (pass-through layer) x is bf16, s_a_in and dbg must be
 * NULL, no workspace is used, and the output is bf16_rne(fp32 sum + bias) with the sum accumulated in
 * fp32 on the tensor cores (order unspecified: compare with a tolerance, not bit for bit).
 */
int dp_wq_linear(const dp_weight* w, const void* x, int64_t ldx, const float* s_a_in, int64_t M,
                 void* y_bf16, int64_t ldy, void* workspace, size_t workspace_bytes,
                 const dp_debug* dbg, int32_t* device_status, uint32_t flags, dp_stream stream);

/*
 * LayerNorm + adaLN modulation taken into DAQ (Step 3 keeps LayerNorms in higher precision and
 * quantizes the wrapped linears' activations on the fly, Eq. "daq"; in a DiT block the qkv and fc1
 * linears are fed LayerNorm(x) * (1 + scale) + shift with one scale and shift vector per sample).
 * One pass over the bf16 stream x [M][ldx] writes int8 codes q [M][ldq] and token scales s_a [M],
 * ready for dp_wq_linear(w, q, ldq, s_a, ...); the normalized values exist only in fp32:
 *
 *     mean, var   of the token's K values (var = E[x^2] - mean^2), in double, rounded to fp32
 *     rstd        = 1 / sqrt(var + eps), in double, rounded to fp32
 *     n[k]        = (x[k] - mean) * rstd                              fp32, two roundings
 *     h[k]        = fma(n[k], 1 + scale[s][k], shift[s][k])           fp32, s = m / rows_per_sample
 *     q, s_a      = Eq. "daq" on h (absmax / 127, round half to even), as dp_daq_quantize on bf16
 *
 * shift, scale: device bf16 [ceil(M / rows_per_sample)][K], 16-byte aligned, or both NULL (plain
 * LayerNorm without affine parameters). K a multiple of 8, at most 4608; x, q 16-byte aligned, ldx a
 * multiple of 8, ldq of 16. Enqueues one kernel. Errors: DP_ERR_INVALID_ARG, DP_ERR_SHAPE,
 * DP_ERR_ALIGN, DP_ERR_ARCH.
 */
int dp_ln_modulate_daq(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, const void* shift_bf16,
                       const void* scale_bf16, int64_t rows_per_sample, float eps, int8_t* q, int64_t ldq,
                       float* s_a, dp_stream stream);

/*
 * The residual connection around a wrapped linear, taken into its epilogue (Step 3 keeps residual
 * adds in higher precision; a DiT block adds its attention projection and MLP output to the token
 * stream scaled by an adaLN gate per sample and channel). With lin[m][n] the fp32 value that
 * dp_wq_linear rounds to bf16 (Step 5's dequantized output plus bias):
 *
 *     y[m][n] = bf16( gate ? fma(gate[m / rows_per_gate][n], lin, residual[m][n]) : lin + residual[m][n] )
 *
 * evaluated in fp32 with one rounding to bf16 at the end, so the layer's output never passes through
 * bf16 before the add and the stream is read and written once instead of three times.
 */
typedef struct dp_residual {
  const void* residual;  /* device: bf16 [M][ldr]; may be the output buffer itself (ldr == ldy): each
                            element is read before it is overwritten, by the same thread          */
  int64_t ldr;           /* elements between rows, >= N, multiple of 8; residual 16-byte aligned  */
  const void* gate;      /* device: bf16 [ceil(M / rows_per_gate)][N], 16-byte aligned, or NULL   */
  int64_t rows_per_gate; /* tokens that share a gate row (tokens per sample), >= 1; ignored without gate */
} dp_residual;

/*
 * dp_wq_linear(w, x_bf16, ldx, NULL, M, ...) with the epilogue above. Per-channel weight scales at
 * 3, 4 or 8 bits only (DP_ERR_INVALID_ARG for a 16-bit or group-wise layer); always runs a tensor-core
 * kernel (DP_FLAG_FORCE_SIMT is refused) on int8 operands: packed weights are expanded into the
 * workspace first (DP_FLAG_UNPACK_FIRST is implied, DP_FLAG_NO_UNPACK_FIRST ignored). Workspace:
 * dp_wq_linear_workspace(M, N, K, bits, flags | DP_FLAG_FORCE_MMA | DP_FLAG_UNPACK_FIRST). Other arguments, flags and errors as dp_wq_linear.
 */
int dp_wq_linear_residual(const dp_weight* w, const void* x_bf16, int64_t ldx, int64_t M, const dp_residual* r,
                          void* y_bf16, int64_t ldy, void* workspace, size_t workspace_bytes,
                          int32_t* device_status, uint32_t flags, dp_stream stream);

/*
 * dp_wq_linear for callers that cannot allocate device memory. (The paper has no counterpart: this
 * is a deployment convenience of the library, not a step of the method.)
 *
 * Some hosts of this code only hand a kernel library its input and output buffers and forbid it to
 * call cudaMalloc: a custom-op slot of an inference runtime that owns all device memory, a step
 * that runs while a stream is being captured into a CUDA graph, or a latency-critical loop where an
 * allocation would stall the device. For them the scratch that dp_wq_linear takes as `workspace`
 * (the int8 activations and their scales between its two kernels) lives inside the library, in one
 * fixed device array of DP_STATIC_SCRATCH_BYTES that every GPU loading the library holds until the
 * process exits. The call computes exactly what dp_wq_linear(w, x, ldx, NULL, M, y, ldy, ...) does.
 *
 *   - Problems whose dp_wq_linear_workspace(M, N, K, bits, flags) exceeds DP_STATIC_SCRATCH_BYTES are
 *     refused with DP_ERR_WORKSPACE and nothing is enqueued (M = 2048 tokens at K = 4608 fits).
 *   - The first call on each device looks up the array's device address (a cheap runtime query, no
 *     allocation); make that first call outside any stream capture.
 *   - All calls on a device share the one array, on every stream: two calls whose kernels may
 *     overlap on the GPU race on it. Issue them on one stream, or order them yourself.
 *   - The array keeps whatever the previous call left. Nothing in it has to start at zero: the
 *     quantization kernel overwrites every byte that reaches a stored output before the GEMM runs
 *     (rows past M of the last 128-token tile are read by the GEMM's tile loads but belong to
 *     outputs that are never stored).
 *   - No cudaMalloc, cudaFree or other allocating routine is called; x is always bf16 (the
 *     pre-quantized form of dp_wq_linear needs no scratch and is not offered here).
 */
#define DP_STATIC_SCRATCH_BYTES (10u << 20)
int dp_wq_linear_static(const dp_weight* w, const void* x_bf16, int64_t ldx, int64_t M, void* y_bf16,
                        int64_t ldy, int32_t* device_status, uint32_t flags, dp_stream stream);

/*
 * A deployed plan (Algorithm 2, Phase B, whose first step wraps every linear according to the bit
 * plan): n_layers quantized linears with their row counts. Creation validates every layer, chooses kernel variants, encodes
 * TMA descriptors and may allocate/synchronise; it is not on the timed path. The dp_weight array is
 * copied; the device buffers it points to must outlive the plan.
 */
typedef struct dp_plan dp_plan;
int dp_plan_create(const dp_weight* layers, int32_t n_layers, const int64_t* M_per_layer,
                   uint32_t flags, dp_plan** out);
size_t dp_plan_workspace(const dp_plan* plan);
/* Which kernel the plan runs layer `layer` with (for reports and for timing that kernel alone):
 * *tile_n = tile width in output channels, *cta_group = 1 or 2 CTAs per row tile,
 * *weight_stationary = 0, 1 (weight-stationary kernel) or 2 (activation-stationary kernel; *tile_n is
 * then its sub-block width), *small_m = 1 when the CUDA-core small-M kernel is used (the other three
 * are then 0). Any output pointer may be NULL. */
int dp_plan_layer_variant(const dp_plan* plan, int32_t layer, int32_t* tile_n, int32_t* cta_group,
                          int32_t* weight_stationary, int32_t* small_m);
/* *unpack_first = 1 when the plan runs layer `layer` in the DP_FLAG_UNPACK_FIRST form (the
 * variant dp_plan_layer_variant reports is then the 8-bit kernel's). No counterpart in the paper. */
int dp_plan_layer_unpack_first(const dp_plan* plan, int32_t layer, int32_t* unpack_first);
/* Replaces the kernel variant of layer `layer` by the one `flags` names (the tuning flags of
 * dp_wq_linear: DP_FLAG_TILE_N, [NO_]CTA_PAIR, [NO_]WEIGHT_STATIONARY, [NO_]ACT_STATIONARY, UNPACK_FIRST; anything left
 * open is chosen as dp_wq_linear would): lets a deployment keep the outcome of one
 * DP_FLAG_AUTOTUNE run and apply it to later plans. Host only; may raise dp_plan_workspace, so ask
 * again afterwards. Small-M layers and unknown bits are refused (DP_ERR_INVALID_ARG), tile widths
 * that do not fit the layer with DP_ERR_SHAPE; the plan is unchanged on error. Not to be called
 * while a dp_plan_run of the plan is being issued. No counterpart in the paper. */
int dp_plan_set_layer_flags(dp_plan* plan, int32_t layer, uint32_t flags);
/* DAQ policy of a plan (Eq. "daq" with its percentile clip; Step 6 and Algorithm 2 Phase B, where
 * the activation bits of a forward pass are looked up by the time bin of its step: early, middle or
 * late). From the next dp_plan_run on, every layer
 * quantizes its activations as dp_daq_quantize_robust does, with
 *   clip_rank = K - ceil(p K / 100) + 1,  p = clip_percentile_e3 / 1000 percent (100000 = the maximum),
 *   act_bits  = act_bits_by_bin[min(2, 3 t / n_timesteps)] for a step with timestep value t
 * (reading: the three bins are thirds of [0, n_timesteps), bin 0 holding the smallest timestep
 * values; n_timesteps = 0: 8 bits at every step, act_bits_by_bin may be NULL). Under a policy other
 * than (100000, 8 bits) packed layers run in the unpack-first form, grouped small-M layers keep their
 * shared launches for K <= 1280 (longer rows run one by one behind a quantization launch of their
 * own), and DP_FLAG_FUSED_DAQ is ignored. May raise
 * dp_plan_workspace: ask again afterwards. Limits: K <= 4608 and clip_rank <= 64 for every layer
 * (DP_ERR_SHAPE), bits in [2, 8] (DP_ERR_BITS); the plan is unchanged on error. Host only; not to
 * be called while a dp_plan_run of the plan is being issued. */
int dp_plan_set_daq(dp_plan* plan, int32_t clip_percentile_e3, int32_t n_timesteps,
                    const int32_t* act_bits_by_bin);
void dp_plan_destroy(dp_plan* plan);

/*
 * Algorithm 2, Phase B: for i = n_steps-1 down to start_index... the retained timesteps are visited
 * in REVERSE order of the `steps` array (the sampler walks reverse(K*)); for each visited step
 * every layer l = 0..n_layers-1 is run in order:
 *     y_ptrs[i*n_layers + l] = wq_linear(layers[l], x_ptrs[i*n_layers + l])
 * (index i drops out under DP_PLAN_SAME_X / DP_PLAN_SAME_Y). x is bf16 [M_l][K_l] contiguous,
 * y is bf16 [M_l][N_l] contiguous. `steps` holds the timestep labels (host array; only its order
 * and length matter to the linears). Visits i = n_steps-1-start_index, ..., 0, so a caller can
 * resume an interrupted schedule by passing the number of steps already done as start_index.
 * x_ptrs / y_ptrs are HOST arrays of device pointers. Enqueues only; capturable in a CUDA graph.
 * While a layer's GEMM runs, its kernel issues L2 prefetch hints for the next layer's packed weights
 * and (up to 32 MB) for the next layer's input buffer. These are hints on memory the call is going to
 * read anyway: no layer is computed before its turn, and an input that an earlier layer of the same
 * step still writes (x of one layer aliasing y of another) is read only after that write, as the
 * stream order says.
 */
int dp_plan_run(const dp_plan* plan, const int32_t* steps, int32_t n_steps, int32_t start_index,
                const void* const* x_ptrs, void* const* y_ptrs, void* workspace,
                size_t workspace_bytes, int32_t* device_status, uint32_t flags, dp_stream stream);

/*
 * Same as dp_plan_run but the activations live in HOST memory (pinned for speed): for every
 * visited step the inputs of all layers are copied host->device into `x_stage` (two alternating
 * halves so the copy of one step overlaps the compute of the previous one, on an internal copy
 * stream), the layers run, and the outputs named by d2h_layers are copied back to y_host.
 *   x_host  : host array [n_steps*n_layers] of host pointers (or [n_layers] with DP_PLAN_SAME_X)
 *   x_stage : device buffer of 2 * dp_plan_x_bytes(plan) bytes
 *   y_dev   : host array [n_layers] of device output buffers (overwritten every step)
 *   y_host  : host array [n_steps] of host pointers receiving layer `d2h_layer`'s output per step
 * Returns after enqueueing; the caller synchronises `stream`. The internal copy stream starts behind
 * everything already enqueued on `stream` when the call is made, so consecutive calls (or a
 * dp_plan_run on the same workspace) need no synchronisation in between.
 */
size_t dp_plan_x_bytes(const dp_plan* plan);
int dp_plan_run_host(const dp_plan* plan, const int32_t* steps, int32_t n_steps,
                     const void* const* x_host, void* x_stage, size_t x_stage_bytes,
                     void* const* y_dev, int32_t d2h_layer, void* const* y_host, void* workspace,
                     size_t workspace_bytes, int32_t* device_status, uint32_t flags,
                     dp_stream stream);

/*
 * Algorithm 2, Phase A: budgeted joint planning of the per-layer bit plan and the kept timesteps
 * (host arithmetic only; the latency table it consumes can be measured with dp_layer_latency_us).
 *   Tail  = the last floor(rho * n_steps) step indices, always kept.
 *   Init  : every layer at its first (largest) bit option, every step kept;
 *           C_lat = sum_t step_cost[t] + sum_l c_lat[l][0],  C_mem = sum_l c_mem[l][0].
 *   While C_lat > B_lat or C_mem > B_mem:
 *     step candidate = the prunable (non-tail, still kept) step of least drift,
 *                      S_step = step_cost[t] / (eps + drift[t]);
 *     bit candidate  = the best-scored move "layer l: option j -> j + 1" among the layers' next moves,
 *                      S_bit = (c_lat[l][j] - c_lat[l][j+1]) / (eps + sens[l]), restricted to moves after
 *                      which C_mem <= B_mem when such a move exists;
 *     if S_step > S_bit the step is dropped (C_lat -= step_cost[t]); else the move is applied
 *     (C_lat, C_mem updated, the layer's next move becomes available).
 * Readings where the listing is silent: costs are used exactly as supplied (one additive C_lat: the
 * caller decides whether c_lat is per step or summed over the schedule); when no move satisfies the
 * memory clause the best-scored move is taken anyway, since otherwise an overrun larger than one move
 * could never be repaired; ties go to the lower layer index / lower timestep, and S_step == S_bit
 * applies the bit move; the loop also ends when neither candidate exists (*feasible = 0).
 *   options     : n_options[l] entries per layer, flattened in layer order (offset = running sum):
 *                 opt_bits (descending), opt_c_lat, opt_c_mem
 *   bitplan_out : [n_layers] chosen bits;  kept_out : [n_steps] 1 = kept
 *   totals_out  : [2] final C_lat, C_mem (may be NULL);  feasible : may be NULL
 * All pointers are HOST pointers. DP_ERR_INVALID_ARG on NULL / non-positive sizes / rho outside [0, 1].
 */
typedef struct dp_phase_a_problem {
  int32_t n_steps;
  const double* drift;      /* D_e(t) */
  const double* step_cost;  /* c_step(t) */
  int32_t n_layers;
  const int32_t* n_options;
  const int32_t* opt_bits;
  const double* opt_c_lat;
  const double* opt_c_mem;
  const double* sens;       /* s_M(l) */
  double B_lat, B_mem, rho, eps;
} dp_phase_a_problem;
int dp_plan_phase_a(const dp_phase_a_problem* problem, int32_t* bitplan_out, uint8_t* kept_out, double* totals_out,
                    int32_t* feasible);

/*
 * One entry c_lat(l, b) of Phase A's latency table, measured with this library's kernels: the time of
 * one whole quantized linear (DAQ + weight expansion + GEMM, as dp_wq_linear runs it with `flags`) for
 * weight `w` (device pointers) at M tokens, in microseconds, averaged over `reps` back-to-back calls
 * after two warm-up calls. Allocates and frees its own device buffers and synchronises: a plan-time
 * call like dp_plan_create, not part of the hot path. (Algorithm 2's inputs c_lat(l, b); the paper
 * measures them with its own integer kernels.)
 */
int dp_layer_latency_us(const dp_weight* w, int64_t M, uint32_t flags, int32_t reps, float* us_out);

/*
 * Host helper: pack int8 weights w[N][K] (values in [-2^(b-1), 2^(b-1)-1]) into the layout
 * dp_weight documents. `out` is a host buffer of N*K*bits/8 bytes. Values out of range give
 * DP_ERR_INVALID_ARG.
 */
int dp_pack_weights_host(const int8_t* w, int32_t N, int32_t K, int32_t bits, void* out);

/*
 * Test hook for the bounded device waits (no counterpart in the paper). The next launch of the
 * single-CTA tensor-core kernel made by the calling thread leaves out, in every CTA, the loads of
 * k-block `k_block` of the CTA's first tile: nothing is issued for that pipeline stage, so nothing is
 * in flight and no address is touched, and the stage's barrier is never completed. The MMA role's
 * bounded wait on it runs out (about 0.15 s), every role of the CTA leaves its loop, tensor memory is
 * freed, the kernel exits normally and `device_status` of that call reads DP_ERR_TIMEOUT; the
 * outputs of the call are undefined. The hook clears itself when that launch is made; k_block < 0
 * clears it without a launch. Host state is per thread.
 */
void dp_debug_skip_stage_load(int32_t k_block);

const char* dp_status_string(int status);
const char* dp_last_error(void);
/* Library ABI version: (major << 16) | minor. */
int dp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DIFFPRO_H_ */
