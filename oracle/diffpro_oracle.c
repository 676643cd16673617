/*
 * diffpro_oracle.c — TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, CPU restatement of the quantized linear layer of a deployed DiffPro plan, written
 * from the paper's definitions so the CUDA library can be checked against it. It shares no code
 * with the CUDA path and must never be called from the product path; only the tests, the smoke
 * check and the benchmark's cpu-baseline leg use it.
 *
 * What each function follows:
 *   orc_daq        Step 3, Eq. "daq": tau = clip threshold, alpha = tau / (2^(b-1) - 1) with b = 8,
 *                  q = round(clip(v, -tau, tau) / alpha), zero-point 0. Reading taken here: tau is
 *                  the absolute maximum of one token's K activations (p = 100, one group); round is
 *                  half-to-even; the division by alpha is evaluated as a multiplication by
 *                  fl(127 / tau) whose exact product is rounded once.
 *   orc_daq_robust Step 3, Eq. "daq" with its percentile clip (p < 100) and Step 6 / Algorithm 2
 *                  Phase B's activation bits per time bin: tau = Percentile(|v|, p) read as the
 *                  nearest-rank percentile of one token's K magnitudes and passed as its rank from
 *                  the top (rank 1 = maximum, rank r = r-th largest counting repeats;
 *                  r = K - ceil(p K / 100) + 1), alpha = tau / (2^(a-1) - 1) for a activation bits,
 *                  values beyond tau clip to the extreme codes. rank 1, a = 8 is orc_daq.
 *   orc_pack/orc_unpack   "GPTQ packed" low-bit weights (Step 1 calibration text, Step 3): a
 *                  little-endian bit stream of b-bit offset-binary codes per output channel. The
 *                  paper fixes no layout; this is the layout the library's header documents.
 *   orc_gemm_i32   Step 5 / Implementation: INT8 x INT8 -> INT32 contraction over K.
 *   orc_epilogue   Step 5: per-output-channel weight scale (and the per-token DAQ scale) applied to
 *                  the int32 accumulator; bias add; bf16 output.
 *   orc_wq_linear  the four above in order.
 *   orc_plan_run   Algorithm 2, Phase B: for t in reverse(K*): forward every wrapped linear.
 *   orc_wq_linear_grouped  Step 2's storage format: group-wise weight scales (one scale, and optionally one
 *                  zero-point, per output channel and group of g consecutive input channels) in place
 *                  of one scale per output channel. Reading taken (the paper gives no arithmetic):
 *                  acc_G = sum over the group of q * (u - z) exactly in int32; t = 0, then for the
 *                  groups in order t = fma((float)acc_G, s_w[n][G], t); y = bf16(fma(t, s_a[m], bias)).
 *   orc_wq_linear_residual  the residual connection around a wrapped linear taken into its epilogue
 *                  (Step 3: residual adds stay in higher precision; a DiT block adds the projection
 *                  and MLP outputs to its stream scaled by an adaLN gate per sample and channel).
 *                  Reading: lin = fma((float)acc, s_a*s_w, bias) as in orc_epilogue, then in fp32
 *                  v = fma(gate, lin, res) (gate given) or v = lin + res, y = bf16(v).
 *   orc_ln_modulate_daq  the operator in front of a block's qkv and fc1 linears taken into their DAQ
 *                  (Step 3: LayerNorms stay in higher precision; a DiT block feeds those linears
 *                  LayerNorm(x) * (1 + scale) + shift with a per-sample adaLN scale and shift), so the
 *                  normalized activations are quantized without ever being rounded to bf16. Reading:
 *                  mean and variance (biased, E[x^2] - mean^2) of a token in double from the exact
 *                  sums of its bf16 values, rstd = 1 / sqrt(var + eps) in double, both rounded to
 *                  fp32; then in fp32 n = (x - mean) * rstd, h = fma(n, 1 + scale, shift); then Eq.
 *                  "daq" on h exactly as orc_daq does on bf16 values.
 *   orc_linear_bf16  the layers a plan keeps in 16-bit precision (Step 1 tiering; Step 2 results): the
 *                  plain linear y = x . W^T + bias on bf16 inputs, summed in double (every product of
 *                  two bf16 values is exact in double), rounded once to bf16.
 *   orc_phase_a    Algorithm 2, Phase A: the greedy budgeted joint planning of bits and kept steps,
 *                  step by step in the listing's order; the "heap" and the sorted list are plain
 *                  searches for the best-scored move and the least-drift step.
 *
 * Parity status: every function here is pinned by tests/test_oracle_*.py (brute force in exact
 * rational arithmetic, closed forms, invariants, library cross-checks). End-to-end image quality
 * (FID, drift MSE) is "parity unpinned": it needs the paper's checkpoints and datasets.
 *
 * Build: gcc -O2 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 * The only parallelism is an OpenMP loop over rows (tokens) or calls; there is no blocking,
 * fusion or reordering.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---- bf16 <-> fp32 ------------------------------------------------------------------------- */

/* bf16 is the upper half of an IEEE binary32, so widening is exact. */
static float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* Round-to-nearest-even narrowing of a binary32 to bf16. */
static uint16_t f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u); /* quiet NaN */
  uint32_t keep_lsb = (u >> 16) & 1u;
  u += 0x7FFFu + keep_lsb;
  return (uint16_t)(u >> 16);
}

uint16_t orc_f32_to_bf16(float f) { return f32_to_bf16(f); }
float orc_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }

/* ---- DAQ (Step 3, Eq. "daq") ---------------------------------------------------------------- */

/* One token: x[K] bf16 -> q[K] int8, *s_a, optional *rowsum. */
static void daq_row(const uint16_t* x, int64_t K, int8_t* q, float* s_a, int32_t* rowsum) {
  float tau = 0.0f; /* clip threshold = max |v| */
  for (int64_t k = 0; k < K; ++k) {
    float v = fabsf(bf16_to_f32(x[k]));
    if (v > tau) tau = v;
  }
  int32_t sum = 0;
  if (tau < 0x1p-100f) { /* alpha would be 0 or denormal: define the token as all-zero */
    *s_a = 0.0f;
    for (int64_t k = 0; k < K; ++k) q[k] = 0;
  } else {
    const float alpha = tau / 127.0f;     /* scale, 2^(b-1)-1 = 127 */
    const float inv_alpha = 127.0f / tau; /* one fp32 division per token */
    *s_a = alpha;
    for (int64_t k = 0; k < K; ++k) {
      /* bf16 (8-bit significand) times fp32 (24-bit) is exact in double; nearbyint under the
         default rounding mode rounds half to even. */
      double r = nearbyint((double)bf16_to_f32(x[k]) * (double)inv_alpha);
      if (r > 127.0) r = 127.0;
      if (r < -127.0) r = -127.0;
      q[k] = (int8_t)r;
      sum += (int32_t)q[k];
    }
  }
  if (rowsum) *rowsum = sum;
}

void orc_daq(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, int8_t* q, int64_t ldq,
             float* s_a, int32_t* rowsum) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    daq_row(x + m * ldx, K, q + m * ldq, s_a + m, rowsum ? rowsum + m : 0);
}

/* ---- LayerNorm + adaLN modulation in front of DAQ ----------------------------------------------- */

/*
 * x bf16 [M][ldx]; shift, scale bf16 [ceil(M / rows_per_sample)][K] (both NULL: no modulation); eps as
 * in torch's layer_norm. q int8 [M][ldq], s_a fp32 [M]; h (optional) fp32 [M][K]: the modulated
 * normalized activations that were quantized.
 */
void orc_ln_modulate_daq(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, const uint16_t* shift,
                         const uint16_t* scale, int64_t rows_per_sample, float eps, int8_t* q, int64_t ldq,
                         float* s_a, float* h_out) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    const uint16_t* xr = x + m * ldx;
    double s1 = 0.0, s2 = 0.0; /* exact: bf16 values and their squares, K of them, fit a double's significand */
    for (int64_t k = 0; k < K; ++k) {
      const double v = (double)bf16_to_f32(xr[k]);
      s1 += v;
      s2 += v * v;
    }
    const double mean_d = s1 / (double)K;
    double var_d = s2 / (double)K - mean_d * mean_d;
    if (var_d < 0.0) var_d = 0.0;
    const float mean = (float)mean_d;
    const float rstd = (float)(1.0 / sqrt(var_d + (double)eps));
    float* h = (float*)malloc((size_t)K * sizeof(float));
    const int64_t sample = m / rows_per_sample;
    float a = 0.0f;
    for (int64_t k = 0; k < K; ++k) {
      const float d = bf16_to_f32(xr[k]) - mean;
      const float n = d * rstd;
      float v = n;
      if (scale) {
        const float g = 1.0f + bf16_to_f32(scale[sample * K + k]);
        v = fmaf(n, g, bf16_to_f32(shift[sample * K + k]));
      }
      h[k] = v;
      if (fabsf(v) > a) a = fabsf(v);
      if (h_out) h_out[m * K + k] = v;
    }
    int8_t* qr = q + m * ldq;
    if (a < 0x1p-100f) {
      s_a[m] = 0.0f;
      for (int64_t k = 0; k < K; ++k) qr[k] = 0;
    } else {
      const float alpha = a / 127.0f;
      const float inv_alpha = 127.0f / a;
      s_a[m] = alpha;
      for (int64_t k = 0; k < K; ++k) {
        /* two fp32 values: the product is exact in double */
        double r = nearbyint((double)h[k] * (double)inv_alpha);
        if (r > 127.0) r = 127.0;
        if (r < -127.0) r = -127.0;
        qr[k] = (int8_t)r;
      }
    }
    free(h);
  }
}

/* ---- DAQ with percentile clip and a-bit codes (Eq. "daq", p < 100; Step 6) ------------------- */

static int cmp_float_desc(const void* a, const void* b) {
  const float fa = *(const float*)a, fb = *(const float*)b;
  return (fa < fb) - (fa > fb);
}

/* One token. clip_rank in [1, K]; act_bits in [2, 8]. */
static void daq_row_robust(const uint16_t* x, int64_t K, int clip_rank, int act_bits, int8_t* q, float* s_a,
                           int32_t* rowsum) {
  float* mag = (float*)malloc((size_t)K * sizeof(float));
  for (int64_t k = 0; k < K; ++k) mag[k] = fabsf(bf16_to_f32(x[k]));
  qsort(mag, (size_t)K, sizeof(float), cmp_float_desc);
  const float tau = mag[clip_rank - 1]; /* the clip_rank-th largest magnitude */
  free(mag);
  const float qmax = (float)((1 << (act_bits - 1)) - 1);
  int32_t sum = 0;
  if (tau < 0x1p-100f) {
    *s_a = 0.0f;
    for (int64_t k = 0; k < K; ++k) q[k] = 0;
  } else {
    const float alpha = tau / qmax;
    const float inv_alpha = qmax / tau;
    *s_a = alpha;
    for (int64_t k = 0; k < K; ++k) {
      /* clip(v, -tau, tau) / alpha and then round is the same as round and then clamp to +-qmax,
         because tau / alpha rounds to qmax; the product is exact in double as in daq_row */
      double r = nearbyint((double)bf16_to_f32(x[k]) * (double)inv_alpha);
      if (r > (double)qmax) r = (double)qmax;
      if (r < -(double)qmax) r = -(double)qmax;
      q[k] = (int8_t)r;
      sum += (int32_t)q[k];
    }
  }
  if (rowsum) *rowsum = sum;
}

/* Returns 0, or -1 on a bad clip_rank / act_bits (nothing is written then). */
int orc_daq_robust(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, int clip_rank, int act_bits, int8_t* q,
                   int64_t ldq, float* s_a, int32_t* rowsum) {
  if (clip_rank < 1 || clip_rank > K || act_bits < 2 || act_bits > 8) return -1;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    daq_row_robust(x + m * ldx, K, clip_rank, act_bits, q + m * ldq, s_a + m, rowsum ? rowsum + m : 0);
  return 0;
}

/* ---- packed weights ------------------------------------------------------------------------- */

/* Words per packed row. */
static int64_t row_words(int64_t K, int bits) { return (K * bits + 31) / 32; }

/* w[N][K] int8 in [-2^(b-1), 2^(b-1)-1] -> packed. Returns 0, or 1 + index of the first value
   that is out of range. bits == 8 copies the bytes. */
int64_t orc_pack(const int8_t* w, int64_t N, int64_t K, int bits, void* out) {
  if (bits == 8) {
    memcpy(out, w, (size_t)(N * K));
    return 0;
  }
  const int half = 1 << (bits - 1);
  const int64_t rw = row_words(K, bits);
  uint32_t* o = (uint32_t*)out;
  memset(o, 0, (size_t)(N * rw) * 4);
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      int v = w[n * K + k];
      if (v < -half || v > half - 1) return 1 + n * K + k;
      uint32_t u = (uint32_t)(v + half); /* offset-binary code */
      for (int j = 0; j < bits; ++j) {   /* bit j of field k is stream bit bits*k + j */
        int64_t sbit = (int64_t)bits * k + j;
        if ((u >> j) & 1u) o[n * rw + sbit / 32] |= 1u << (sbit % 32);
      }
    }
  return 0;
}

void orc_unpack(const void* packed, int64_t N, int64_t K, int bits, int8_t* w) {
  if (bits == 8) {
    memcpy(w, packed, (size_t)(N * K));
    return;
  }
  const int half = 1 << (bits - 1);
  const int64_t rw = row_words(K, bits);
  const uint32_t* p = (const uint32_t*)packed;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      uint32_t u = 0;
      for (int j = 0; j < bits; ++j) {
        int64_t sbit = (int64_t)bits * k + j;
        u |= ((p[n * rw + sbit / 32] >> (sbit % 32)) & 1u) << j;
      }
      w[n * K + k] = (int8_t)((int)u - half);
    }
}

/* ---- integer GEMM (Step 5: INT8 x INT8 -> INT32) ---------------------------------------------- */

void orc_gemm_i32(const int8_t* q, int64_t ldq, const int8_t* w, int64_t M, int64_t N, int64_t K,
                  int32_t* acc, int64_t ldacc) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      int32_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += (int32_t)q[m * ldq + k] * (int32_t)w[n * K + k];
      acc[m * ldacc + n] = s;
    }
}

/* ---- dequant epilogue ------------------------------------------------------------------------ */

static uint16_t epilogue_one(int32_t acc, float s_a, float s_w, float bias) {
  float t = (float)acc;         /* int32 -> fp32, round to nearest */
  float sc = s_a * s_w;         /* combined scale, one rounding */
  float y = fmaf(t, sc, bias);  /* one rounding */
  return f32_to_bf16(y);
}

void orc_epilogue(const int32_t* acc, int64_t ldacc, const float* s_a, const float* s_w,
                  const uint16_t* bias, int64_t M, int64_t N, uint16_t* y, int64_t ldy) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n)
      y[m * ldy + n] =
          epilogue_one(acc[m * ldacc + n], s_a[m], s_w[n], bias ? bf16_to_f32(bias[n]) : 0.0f);
}

/* ---- the whole layer -------------------------------------------------------------------------- */

/*
 * x bf16 [M][ldx]; qweight packed per `bits`; outputs: y bf16 [M][ldy]; optional taps q_out
 * [M][K], s_a_out [M], acc_out [M][N]. scratch_w int8 [N][K], scratch_q int8 [M][K], scratch_sa
 * fp32 [M], scratch_acc int32 [M][N] are caller-provided work arrays.
 */
void orc_wq_linear(const uint16_t* x, int64_t ldx, int64_t M, int64_t N, int64_t K, int bits,
                   const void* qweight, const float* s_w, const uint16_t* bias, uint16_t* y,
                   int64_t ldy, int8_t* scratch_w, int8_t* scratch_q, float* scratch_sa,
                   int32_t* scratch_acc) {
  orc_daq(x, M, K, ldx, scratch_q, K, scratch_sa, 0);
  orc_unpack(qweight, N, K, bits, scratch_w);
  orc_gemm_i32(scratch_q, K, scratch_w, M, N, K, scratch_acc, N);
  orc_epilogue(scratch_acc, N, scratch_sa, s_w, bias, M, N, y, ldy);
}

/*
 * Selected outputs of the layer, for checks at sizes where the full product is too slow:
 * for p < npts, (m, n) = (pm[p], pn[p]); acc_out[p], y_out[p] are that element's accumulator and
 * bf16 output. Each point redoes the DAQ of its token and the unpack of its weight row.
 */
void orc_wq_linear_points(const uint16_t* x, int64_t ldx, int64_t N, int64_t K, int bits,
                          const void* qweight, const float* s_w, const uint16_t* bias,
                          const int64_t* pm, const int64_t* pn, int64_t npts, int32_t* acc_out,
                          uint16_t* y_out) {
  const int64_t rw = (bits == 8) ? 0 : row_words(K, bits);
#pragma omp parallel
  {
    int8_t* q = (int8_t*)malloc((size_t)K);
    int8_t* w = (int8_t*)malloc((size_t)K);
#pragma omp for schedule(static)
    for (int64_t p = 0; p < npts; ++p) {
      float s_a;
      daq_row(x + pm[p] * ldx, K, q, &s_a, 0);
      const void* row = (bits == 8) ? (const void*)((const int8_t*)qweight + pn[p] * K)
                                    : (const void*)((const uint32_t*)qweight + pn[p] * rw);
      orc_unpack(row, 1, K, bits, w);
      int32_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += (int32_t)q[k] * (int32_t)w[k];
      acc_out[p] = s;
      y_out[p] = epilogue_one(s, s_a, s_w[pn[p]], bias ? bf16_to_f32(bias[pn[p]]) : 0.0f);
    }
    free(q);
    free(w);
  }
}

/* ---- plan execution (Algorithm 2, Phase B) ---------------------------------------------------- */

typedef struct orc_layer {
  int64_t M, N, K;
  int32_t bits;
  const void* qweight;
  const float* s_w;
  const uint16_t* bias; /* may be NULL */
} orc_layer;

/*
 * kept[n_kept] is the retained-timestep list K* in ascending order; the sampler visits it in
 * reverse. x_ptrs/y_ptrs are indexed [i * n_layers + l] with i the index into kept[].
 * Scratch arrays are sized for the largest layer.
 */
void orc_plan_run(const orc_layer* layers, int32_t n_layers, const int32_t* kept, int32_t n_kept,
                  const uint16_t* const* x_ptrs, uint16_t* const* y_ptrs, int8_t* scratch_w,
                  int8_t* scratch_q, float* scratch_sa, int32_t* scratch_acc) {
  (void)kept; /* labels only: the linears depend on t through their inputs */
  for (int32_t i = n_kept - 1; i >= 0; --i)
    for (int32_t l = 0; l < n_layers; ++l) {
      const orc_layer* L = &layers[l];
      orc_wq_linear(x_ptrs[(int64_t)i * n_layers + l], L->K, L->M, L->N, L->K, L->bits, L->qweight,
                    L->s_w, L->bias, y_ptrs[(int64_t)i * n_layers + l], L->N, scratch_w, scratch_q,
                    scratch_sa, scratch_acc);
    }
}

/* ---- residual (and gate) in the epilogue -------------------------------------------------------- */

/*
 * As orc_wq_linear, then y[m][n] = bf16( gate ? fma(gate[m / rows_per_gate][n], lin, res[m][n]) : lin + res[m][n] )
 * with lin the fp32 value orc_epilogue rounds to bf16. res bf16 [M][ldr]; gate bf16
 * [ceil(M / rows_per_gate)][N] or NULL.
 */
void orc_wq_linear_residual(const uint16_t* x, int64_t ldx, int64_t M, int64_t N, int64_t K, int bits,
                            const void* qweight, const float* s_w, const uint16_t* bias, const uint16_t* res,
                            int64_t ldr, const uint16_t* gate, int64_t rows_per_gate, uint16_t* y, int64_t ldy,
                            int8_t* scratch_w, int8_t* scratch_q, float* scratch_sa, int32_t* scratch_acc) {
  orc_daq(x, M, K, ldx, scratch_q, K, scratch_sa, 0);
  orc_unpack(qweight, N, K, bits, scratch_w);
  orc_gemm_i32(scratch_q, K, scratch_w, M, N, K, scratch_acc, N);
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      const float t = (float)scratch_acc[m * N + n];
      const float sc = scratch_sa[m] * s_w[n];
      const float lin = fmaf(t, sc, bias ? bf16_to_f32(bias[n]) : 0.0f);
      const float r = bf16_to_f32(res[m * ldr + n]);
      const float v = gate ? fmaf(bf16_to_f32(gate[(m / rows_per_gate) * N + n]), lin, r) : lin + r;
      y[m * ldy + n] = f32_to_bf16(v);
    }
}

/* ---- group-wise weight scales (Step 2: "row/group-wise quantization with scale + zero-point") ---- */

/*
 * x bf16 [M][ldx]; qweight packed per `bits` (offset-binary codes u, as everywhere); group size g
 * (K % g == 0); s_w fp32 [N][K/g]; zeros uint8 [N][K/g] or NULL (NULL = the symmetric code
 * z = 2^(bits-1), i.e. w = u - z is the two's-complement value the per-channel path uses);
 * bias bf16 [N] or NULL -> y bf16 [M][ldy]. Scratch as orc_wq_linear.
 */
void orc_wq_linear_grouped(const uint16_t* x, int64_t ldx, int64_t M, int64_t N, int64_t K, int bits, int64_t g,
                           const void* qweight, const float* s_w, const uint8_t* zeros, const uint16_t* bias,
                           uint16_t* y, int64_t ldy, int8_t* scratch_w, int8_t* scratch_q, float* scratch_sa) {
  const int64_t ng = K / g;
  const int half = 1 << (bits - 1);
  orc_daq(x, M, K, ldx, scratch_q, K, scratch_sa, 0);
  orc_unpack(qweight, N, K, bits, scratch_w); /* w = u - 2^(bits-1) */
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      float t = 0.0f;
      for (int64_t G = 0; G < ng; ++G) {
        int32_t acc = 0;
        const int z = zeros ? (int)zeros[n * ng + G] : half;
        for (int64_t k = G * g; k < (G + 1) * g; ++k) {
          const int u = (int)scratch_w[n * K + k] + half; /* the stored code */
          acc += (int32_t)scratch_q[m * K + k] * (int32_t)(u - z);
        }
        t = fmaf((float)acc, s_w[n * ng + G], t);
      }
      y[m * ldy + n] = f32_to_bf16(fmaf(t, scratch_sa[m], bias ? bf16_to_f32(bias[n]) : 0.0f));
    }
}

/* ---- pass-through linear of 16-bit layers ------------------------------------------------------ */

/* Round-to-nearest-even narrowing of a double to bf16 (one rounding: via the exactly representable
   neighbours, not through float). */
static uint16_t f64_to_bf16(double v) {
  float f = (float)v; /* may double-round: repaired below by comparing the two candidates in double */
  uint32_t u;
  memcpy(&u, &f, 4);
  uint32_t lo = u & 0xFFFF0000u; /* candidate toward zero */
  uint32_t hi = lo + 0x10000u;   /* candidate away from zero */
  float flo, fhi;
  memcpy(&flo, &lo, 4);
  memcpy(&fhi, &hi, 4);
  /* (float)v can land one bf16 step beyond the bracket only when v rounds up to hi exactly: then
     lo == hi's pattern and the loop below still picks the nearer of the two neighbours of v */
  if (fabs((double)flo) > fabs(v)) { /* v's magnitude is below lo: step the bracket down */
    hi = lo;
    lo = lo - 0x10000u;
    memcpy(&flo, &lo, 4);
    memcpy(&fhi, &hi, 4);
  }
  const double dl = fabs(v - (double)flo), dh = fabs((double)fhi - v);
  if (dl < dh || (dl == dh && ((lo >> 16) & 1u) == 0)) return (uint16_t)(lo >> 16);
  return (uint16_t)(hi >> 16);
}

/*
 * x bf16 [M][ldx], w bf16 [N][K], bias bf16 [N] or NULL -> y bf16 [M][ldy]; optional exact[M][N]
 * (the double-precision value before the final rounding) and mag[M][N] = sum_k |x w| (for error
 * bounds of implementations that accumulate in lower precision).
 */
void orc_linear_bf16(const uint16_t* x, int64_t ldx, const uint16_t* w, const uint16_t* bias, int64_t M,
                     int64_t N, int64_t K, uint16_t* y, int64_t ldy, double* exact, double* mag) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      double s = 0.0, a = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        const double p = (double)bf16_to_f32(x[m * ldx + k]) * (double)bf16_to_f32(w[n * K + k]);
        s += p;
        a += fabs(p);
      }
      if (bias) s += (double)bf16_to_f32(bias[n]);
      y[m * ldy + n] = f64_to_bf16(s);
      if (exact) exact[m * N + n] = s;
      if (mag) mag[m * N + n] = a;
    }
}

/* ---- joint planning (Algorithm 2, Phase A) ---------------------------------------------------- */

/*
 * Inputs as in the algorithm: drift D_e(t) and step latency c_step(t) for t < n_steps; for layer l
 * its n_options[l] bit options (largest first) with c_lat, c_mem (flattened in layer order) and its
 * sensitivity s_M(l); budgets B_lat, B_mem; protected-tail fraction rho; epsilon.
 * Outputs: bitplan[l] = chosen bits, kept[t] = 1 if t is in K*, totals = {C_lat, C_mem}.
 * Returns 1 if both budgets are met at exit, 0 if the moves ran out first.
 * Readings (the listing is silent): one additive C_lat = sum of kept c_step + sum of current c_lat;
 * the bit candidate is the best-scored next move among those after which C_mem <= B_mem, or, when
 * there is none, the best-scored next move; ties: lower layer index, lower timestep; S_step must be
 * strictly larger than S_bit for the step to be dropped.
 */
int orc_phase_a(int32_t n_steps, const double* drift, const double* step_cost, int32_t n_layers,
                const int32_t* n_options, const int32_t* opt_bits, const double* opt_c_lat,
                const double* opt_c_mem, const double* sens, double B_lat, double B_mem, double rho,
                double eps, int32_t* bitplan, uint8_t* kept, double* totals) {
  int64_t* off = (int64_t*)malloc((size_t)(n_layers + 1) * sizeof(int64_t));
  int32_t* cur = (int32_t*)calloc((size_t)n_layers, sizeof(int32_t));
  off[0] = 0;
  for (int32_t l = 0; l < n_layers; ++l) off[l + 1] = off[l] + n_options[l];
  const int32_t n_tail = (int32_t)floor(rho * (double)n_steps); /* Tail = last floor(rho |T|) indices */
  double C_lat = 0.0, C_mem = 0.0;
  for (int32_t t = 0; t < n_steps; ++t) { /* K <- T */
    kept[t] = 1;
    C_lat += step_cost[t];
  }
  for (int32_t l = 0; l < n_layers; ++l) { /* Pi(l) <- max B_l */
    C_lat += opt_c_lat[off[l]];
    C_mem += opt_c_mem[off[l]];
  }
  int feasible = 1;
  while (C_lat > B_lat || C_mem > B_mem) {
    /* step candidate: first of R = prunable kept steps by ascending drift */
    int32_t ts = -1;
    for (int32_t t = 0; t < n_steps - n_tail; ++t)
      if (kept[t] && (ts < 0 || drift[t] < drift[ts])) ts = t;
    /* bit candidate: top of H_bit subject to the memory clause */
    int32_t lb = -1, lb_any = -1;
    double sb = 0.0, sb_any = 0.0;
    for (int32_t l = 0; l < n_layers; ++l) {
      if (cur[l] + 1 >= n_options[l]) continue; /* no cheaper option left */
      const int64_t i = off[l] + cur[l];
      const double score = (opt_c_lat[i] - opt_c_lat[i + 1]) / (eps + sens[l]);
      if (lb_any < 0 || score > sb_any) {
        lb_any = l;
        sb_any = score;
      }
      if (C_mem - (opt_c_mem[i] - opt_c_mem[i + 1]) <= B_mem && (lb < 0 || score > sb)) {
        lb = l;
        sb = score;
      }
    }
    if (lb < 0) {
      lb = lb_any;
      sb = sb_any;
    }
    if (ts < 0 && lb < 0) {
      feasible = 0;
      break;
    }
    const double s_step = ts >= 0 ? step_cost[ts] / (eps + drift[ts]) : 0.0;
    if (ts >= 0 && (lb < 0 || s_step > sb)) {
      kept[ts] = 0; /* K <- K \ {t*} */
      C_lat -= step_cost[ts];
    } else {
      const int64_t i = off[lb] + cur[lb];
      C_lat -= opt_c_lat[i] - opt_c_lat[i + 1];
      C_mem -= opt_c_mem[i] - opt_c_mem[i + 1];
      cur[lb] += 1; /* Pi(l*) <- b' */
    }
  }
  for (int32_t l = 0; l < n_layers; ++l) bitplan[l] = opt_bits[off[l] + cur[l]];
  totals[0] = C_lat;
  totals[1] = C_mem;
  free(off);
  free(cur);
  return feasible;
}
