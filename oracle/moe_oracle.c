/*
 * moe_oracle.c -- plain CPU statement of the MoE layer that prefill and decode
 * both execute (route -> dispatch layout -> grouped SwiGLU FFN -> combine).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA library is
 * measured against; it is never part of the product path and shares no code,
 * header, table or helper with it.  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference arm may build or call it.
 *
 * What it follows.  The paper (Section "DeepEP Communication-State Isolation",
 * subsection "Exposing a Safe Prefill Boundary") names the stages of a normal
 * dispatch -- expert notification, receive-count exchange, tensor allocation,
 * routed data movement -- and the evaluation section gives only shapes (top-8
 * routing over hundreds of experts).  The arithmetic itself is fixed by the
 * problem statement of this build:
 *
 *   out[t] = sum_{j<k} w[t,j] * FFN_{idx[t,j]}(x[t])  (+ FFN_shared(x[t]))
 *   FFN_e(v) = W_down,e * ( silu(W_gate,e v) .* (W_up,e v) ),  silu(z) = z / (1 + exp(-z))
 *   idx[t,:] = the k experts with the largest key = logit (+ selection bias),
 *              ties to the lower expert index, listed in descending key order
 *   w[t,:]   = softmax over the k selected (unbiased) logits, times routed_scale
 *
 * The grouped (permuted) execution reaches exactly this result, so the oracle
 * is the definition written out; the integer stages (counts, exclusive scan,
 * stable permutation) are written out too because their values are part of
 * the contract.
 *
 * Precision.  Inputs are bf16 (activations, weights) and fp32 (logits, bias).
 * The selection key is ONE fp32 add, because it decides integers and the GPU
 * takes the same decision in the same precision.  Everything else accumulates
 * in fp64 and is returned as fp32.  `emulate_bf16` additionally rounds the
 * activation `a`, the expert outputs `y` and the shared-expert output to bf16
 * (round-to-nearest-even) where a bf16 pipeline stores them; it exists to
 * separate storage rounding from bugs and is never the comparison target.
 *
 * Loops are in definition order.  `#pragma omp` spreads independent outputs
 * over cores and lets the compiler vectorise a dot product (which changes
 * rounding order only); nothing is blocked, fused or reordered beyond that.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NONFINITE 2
#define ORACLE_ERR_BAD_INDEX 3
#define ORACLE_ERR_ALLOC 4

/* ------------------------------------------------------------------ bf16 */

static inline float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

/* fp32 -> bf16, round to nearest, ties to even (finite inputs). */
static inline uint16_t f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

static inline double round_to_bf16(double v) { return (double)bf16_to_f32(f32_to_bf16((float)v)); }

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Exposed so the tests can pin the two conversions against a library. */
void oracle_bf16_to_f32(const uint16_t* in, int64_t n, float* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_f32(in[i]);
}
void oracle_f32_to_bf16(const float* in, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16(in[i]);
}

/* ----------------------------------------------------------------- route
 * Top-k routing over given router logits (stage a1).
 *   key[e] = logits[t,e] + bias[e]   (one fp32 add; bias NULL => key = logits)
 *   order  = key descending, expert index ascending on equal keys (IEEE ==, so
 *            -0.0 and +0.0 tie)
 *   w[t,j] = routed_scale * exp(l_j - m) / sum_j exp(l_j - m) over the k
 *            selected UNBIASED logits l_j, m their maximum, summed in j order.
 * logits [T,E] fp32 row-major, idx [T,k] int32, w [T,k] fp32.
 */
int oracle_route(const float* logits, const float* bias, int32_t T, int32_t E, int32_t k,
                 float routed_scale, int32_t* idx, float* w) {
  if (T < 0 || E <= 0 || k <= 0 || k > E) return ORACLE_ERR_ARG;
  int status = ORACLE_OK;
#pragma omp parallel for schedule(static)
  for (int32_t t = 0; t < T; ++t) {
    float* key = (float*)malloc((size_t)E * sizeof(float));
    char* taken = (char*)calloc((size_t)E, 1);
    if (!key || !taken) {
      status = ORACLE_ERR_ALLOC;
      free(key);
      free(taken);
      continue;
    }
    const float* l = logits + (int64_t)t * E;
    for (int32_t e = 0; e < E; ++e) {
      volatile float s = bias ? l[e] + bias[e] : l[e]; /* volatile: a real fp32 add, no excess precision */
      key[e] = s;
      if (!isfinite(key[e]) || !isfinite(l[e])) status = ORACLE_ERR_NONFINITE;
    }
    for (int32_t j = 0; j < k; ++j) {
      int32_t best = -1;
      for (int32_t e = 0; e < E; ++e) { /* ascending e + strict > keeps the lower index on ties */
        if (taken[e]) continue;
        if (best < 0 || key[e] > key[best]) best = e;
      }
      taken[best] = 1;
      idx[(int64_t)t * k + j] = best;
    }
    double m = -INFINITY;
    for (int32_t j = 0; j < k; ++j) {
      double lj = (double)l[idx[(int64_t)t * k + j]];
      if (lj > m) m = lj;
    }
    double s = 0.0;
    for (int32_t j = 0; j < k; ++j) s += exp((double)l[idx[(int64_t)t * k + j]] - m);
    for (int32_t j = 0; j < k; ++j)
      w[(int64_t)t * k + j] = (float)((double)routed_scale * exp((double)l[idx[(int64_t)t * k + j]] - m) / s);
    free(key);
    free(taken);
  }
  return status;
}

/* ---------------------------------------------------------------- layout
 * Dispatch layout (stages a2-a4): per-expert token counts, their exclusive
 * scan, and the stable token-to-expert permutation.  Flat slot f = t*k + j.
 *   counts[e]    = #{ f : topk_idx[f] == e }
 *   offsets[0]   = 0, offsets[e+1] = offsets[e] + counts[e]
 *   visiting f = 0..N-1 in order:  p = offsets[e_f] + seen[e_f]++ ;
 *   perm[p] = f ; inv_perm[f] = p
 * counts [E], offsets [E+1], perm [N], inv_perm [N], all int32.
 */
int oracle_layout(const int32_t* topk_idx, int64_t N, int32_t E, int32_t* counts, int32_t* offsets,
                  int32_t* perm, int32_t* inv_perm) {
  if (N < 0 || N > 0x7fffffffLL || E <= 0) return ORACLE_ERR_ARG;
  for (int32_t e = 0; e < E; ++e) counts[e] = 0;
  for (int64_t f = 0; f < N; ++f) {
    int32_t e = topk_idx[f];
    if (e < 0 || e >= E) return ORACLE_ERR_BAD_INDEX;
    counts[e] += 1;
  }
  offsets[0] = 0;
  for (int32_t e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
  int32_t* seen = (int32_t*)calloc((size_t)E, sizeof(int32_t));
  if (!seen) return ORACLE_ERR_ALLOC;
  for (int64_t f = 0; f < N; ++f) {
    int32_t e = topk_idx[f];
    int32_t p = offsets[e] + seen[e];
    seen[e] += 1;
    perm[p] = (int32_t)f;
    inv_perm[f] = p;
  }
  free(seen);
  return ORACLE_OK;
}

/* --------------------------------------------------------------- permute
 * Routed data movement (stage a5): x_perm[p,:] = x[perm[p] / k, :], a bit copy.
 * x [T,H] bf16, x_perm [N,H] bf16.
 */
int oracle_permute(const uint16_t* x, const int32_t* perm, int64_t N, int32_t k, int32_t H,
                   uint16_t* x_perm) {
  if (N < 0 || k <= 0 || H <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < N; ++p)
    memcpy(x_perm + p * H, x + (int64_t)(perm[p] / k) * H, (size_t)H * sizeof(uint16_t));
  return ORACLE_OK;
}

/* ------------------------------------------------------------------- FFN
 * One expert's SwiGLU feed-forward on M rows (stages a6 + a7, or a8 for the
 * shared expert):
 *   g_i = sum_h x[r,h] * W_gate_up[i,h]        i in [0,I)
 *   u_i = sum_h x[r,h] * W_gate_up[I+i,h]
 *   a_i = g_i / (1 + exp(-g_i)) * u_i
 *   y_c = sum_i a_i * W_down[c,i]              c in [0,H)
 * x_rows [M,H] bf16; w_gate_up [2I,H] bf16 (rows 0..I-1 gate, I..2I-1 up);
 * w_down [H,I] bf16; act_out [M,I] fp32 or NULL; y_out [M,H] fp32.
 */
int oracle_ffn(const uint16_t* x_rows, int64_t M, const uint16_t* w_gate_up, const uint16_t* w_down,
               int32_t H, int32_t I, int32_t emulate_bf16, float* act_out, float* y_out) {
  if (M < 0 || H <= 0 || I <= 0) return ORACLE_ERR_ARG;
  if (M == 0) return ORACLE_OK;
  double* a = (double*)malloc((size_t)M * (size_t)I * sizeof(double));
  if (!a) return ORACLE_ERR_ALLOC;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t r = 0; r < M; ++r) {
    for (int32_t i = 0; i < I; ++i) {
      const uint16_t* xr = x_rows + r * H;
      const uint16_t* wg = w_gate_up + (int64_t)i * H;
      const uint16_t* wu = w_gate_up + ((int64_t)I + i) * H;
      double g = 0.0, u = 0.0;
#pragma omp simd reduction(+ : g, u)
      for (int32_t h = 0; h < H; ++h) {
        double xv = (double)bf16_to_f32(xr[h]);
        g += xv * (double)bf16_to_f32(wg[h]);
        u += xv * (double)bf16_to_f32(wu[h]);
      }
      double av = g / (1.0 + exp(-g)) * u;
      if (emulate_bf16) av = round_to_bf16(av);
      a[r * I + i] = av;
    }
  }
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t r = 0; r < M; ++r) {
    for (int32_t c = 0; c < H; ++c) {
      const double* ar = a + r * I;
      const uint16_t* wd = w_down + (int64_t)c * I;
      double y = 0.0;
#pragma omp simd reduction(+ : y)
      for (int32_t i = 0; i < I; ++i) y += ar[i] * (double)bf16_to_f32(wd[i]);
      if (emulate_bf16) y = round_to_bf16(y);
      y_out[r * H + c] = (float)y;
    }
  }
  if (act_out)
    for (int64_t q = 0; q < M * (int64_t)I; ++q) act_out[q] = (float)a[q];
  free(a);
  return ORACLE_OK;
}

/* Grouped expert FFN over the permuted rows: expert e owns rows
 * [offsets[e], offsets[e+1]) of x_perm and uses slab e of the weights.
 * w_gate_up [E,2I,H], w_down [E,H,I] bf16.  act_out [N,I] (or NULL), y_out [N,H] fp32.
 */
int oracle_grouped_ffn(const uint16_t* x_perm, const int32_t* offsets, int32_t E,
                       const uint16_t* w_gate_up, const uint16_t* w_down, int32_t H, int32_t I,
                       int32_t emulate_bf16, float* act_out, float* y_out) {
  for (int32_t e = 0; e < E; ++e) {
    int64_t r0 = offsets[e], M = (int64_t)offsets[e + 1] - offsets[e];
    if (M < 0) return ORACLE_ERR_ARG;
    int rc = oracle_ffn(x_perm + r0 * H, M, w_gate_up + (int64_t)e * 2 * I * H,
                        w_down + (int64_t)e * H * I, H, I, emulate_bf16,
                        act_out ? act_out + r0 * I : NULL, y_out + r0 * H);
    if (rc) return rc;
  }
  return ORACLE_OK;
}

/* --------------------------------------------------------------- combine
 * Weighted combine back to token order (stage a9):
 *   out[t,c] = sum_{j=0..k-1} w[t,j] * y[inv_perm[t*k+j], c]  (+ y_shared[t,c])
 * accumulated in ascending j, then the shared term.  y [N,H] fp32,
 * y_shared [T,H] fp32 or NULL, out [T,H] fp32.
 */
int oracle_combine(const float* y, const int32_t* inv_perm, const float* w, const float* y_shared,
                   int32_t T, int32_t k, int32_t H, float* out) {
  if (T < 0 || k <= 0 || H <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
  for (int32_t t = 0; t < T; ++t) {
    for (int32_t c = 0; c < H; ++c) {
      double acc = 0.0;
      for (int32_t j = 0; j < k; ++j) {
        int64_t p = inv_perm[(int64_t)t * k + j];
        acc += (double)w[(int64_t)t * k + j] * (double)y[p * H + c];
      }
      if (y_shared) acc += (double)y_shared[(int64_t)t * H + c];
      out[(int64_t)t * H + c] = (float)acc;
    }
  }
  return ORACLE_OK;
}

/* ----------------------------------------------------- layer, by definition
 * The dense definition for a chosen set of tokens, with no permutation:
 *   out[s,:] = sum_j w[t,j] * FFN_{idx[t,j]}(x[t,:]) (+ FFN_shared(x[t,:])),  t = tokens[s]
 * (tokens == NULL means s = t for s in [0, n_tokens)).  Routing results are
 * inputs, so this function and oracle_route / oracle_layout / oracle_grouped_ffn
 * / oracle_combine give two independent routes to the same output.
 * term_abs (optional, [n_tokens,H]) receives sum_j |w_j * y_j[c]| + |y_shared[c]|,
 * the magnitude that scales the forward-error bound of the sum.
 */
int oracle_layer_tokens(const uint16_t* x, const int32_t* topk_idx, const float* topk_w,
                        const int32_t* tokens, int32_t n_tokens, int32_t k, int32_t E, int32_t H,
                        int32_t I, const uint16_t* w_gate_up, const uint16_t* w_down,
                        const uint16_t* ws_gate_up, const uint16_t* ws_down, int32_t I_shared,
                        int32_t emulate_bf16, float* out, float* term_abs) {
  if (n_tokens < 0 || k <= 0 || E <= 0 || H <= 0 || I <= 0) return ORACLE_ERR_ARG;
  float* y = (float*)malloc((size_t)H * sizeof(float));
  double* acc = (double*)malloc((size_t)H * sizeof(double));
  double* mag = (double*)malloc((size_t)H * sizeof(double));
  if (!y || !acc || !mag) {
    free(y);
    free(acc);
    free(mag);
    return ORACLE_ERR_ALLOC;
  }
  int rc = ORACLE_OK;
  for (int32_t s = 0; s < n_tokens && rc == ORACLE_OK; ++s) {
    int64_t t = tokens ? tokens[s] : s;
    for (int32_t c = 0; c < H; ++c) acc[c] = mag[c] = 0.0;
    for (int32_t j = 0; j < k && rc == ORACLE_OK; ++j) {
      int32_t e = topk_idx[t * k + j];
      if (e < 0 || e >= E) {
        rc = ORACLE_ERR_BAD_INDEX;
        break;
      }
      rc = oracle_ffn(x + t * H, 1, w_gate_up + (int64_t)e * 2 * I * H, w_down + (int64_t)e * H * I, H,
                      I, emulate_bf16, NULL, y);
      double wj = (double)topk_w[t * k + j];
      for (int32_t c = 0; c < H; ++c) {
        acc[c] += wj * (double)y[c];
        mag[c] += fabs(wj * (double)y[c]);
      }
    }
    if (rc == ORACLE_OK && ws_gate_up && ws_down) {
      rc = oracle_ffn(x + t * H, 1, ws_gate_up, ws_down, H, I_shared, emulate_bf16, NULL, y);
      for (int32_t c = 0; c < H; ++c) {
        acc[c] += (double)y[c];
        mag[c] += fabs((double)y[c]);
      }
    }
    for (int32_t c = 0; c < H; ++c) {
      out[(int64_t)s * H + c] = (float)acc[c];
      if (term_abs) term_abs[(int64_t)s * H + c] = (float)mag[c];
    }
  }
  free(y);
  free(acc);
  free(mag);
  return rc;
}

/* ===================================================================== FP8
 * Precision variant: 8-bit weights and activations (the paper evaluates its
 * models in BF16 and in FP8, Section "Evaluation", "Methodology", but prints no
 * recipe).  The reading taken here, step by step:
 *
 *   format     OCP E4M3 ("e4m3fn"): 1 sign, 4 exponent (bias 7), 3 mantissa
 *              bits; no infinities; largest finite value 448; subnormals are
 *              multiples of 2^-9.
 *   weights    given as E4M3 codes with one fp32 scale per output channel
 *              (per weight row): W[r,:] = scale_w[r] * decode(code[r,:]).
 *   activation a bf16 row v[0..n) entering a GEMM is quantised per row:
 *                amax  = max( max_i |v_i|, 2^-100 )          (fp32; the floor
 *                        keeps an all-zero row finite: its codes are 0)
 *                scale = amax / 448,  inv = 448 / amax       (fp32 divisions)
 *                code_i = e4m3( v_i * inv )  (one fp32 multiply, then round
 *                         to nearest even, saturating at +-448)
 *   GEMM1      g_i = (sum_h dq_x[h] * dq_wg[i,h]) * scale_x * scale_w[i],
 *              u_i likewise with the up row, a_i = silu(g_i) * u_i,
 *              a stored as bf16 (round to nearest even)
 *   GEMM2      the bf16 row a is quantised as above, then
 *              y_c = (sum_i dq_a[i] * dq_wd[c,i]) * scale_a * scale_w[c]
 *
 * The quantisation decides integers (codes), so it is written in fp32 with
 * exactly the operations listed; the sums accumulate in fp64.
 */
static inline float e4m3_to_f32(uint8_t c) {
  int sign = c >> 7, ex = (c >> 3) & 15, man = c & 7;
  float v;
  if (ex == 15 && man == 7) return NAN;
  if (ex == 0) v = ldexpf((float)man, -9);
  else v = ldexpf(1.0f + (float)man / 8.0f, ex - 7);
  return sign ? -v : v;
}

static inline uint8_t f32_to_e4m3(float f) {
  if (f != f) return 0x7f;
  uint8_t sign = (uint8_t)(signbit(f) ? 0x80 : 0);
  float a = fabsf(f);
  if (a >= 448.0f) return (uint8_t)(sign | 0x7e); /* saturate (also everything that would round past 448) */
  if (a < ldexpf(1.0f, -6)) {                     /* subnormal range: multiples of 2^-9; 8 is the first normal */
    int q = (int)rintf(ldexpf(a, 9));
    return (uint8_t)(sign | q);
  }
  int e;
  (void)frexpf(a, &e);
  e -= 1; /* a = m * 2^e, m in [1,2) */
  int man = (int)rintf(ldexpf(a, 3 - e)) - 8; /* round m*8 to nearest even; exact scaling */
  if (man == 8) {
    man = 0;
    e += 1;
  }
  if (e > 8 || (e == 8 && man > 6)) return (uint8_t)(sign | 0x7e);
  return (uint8_t)(sign | ((e + 7) << 3) | man);
}

void oracle_e4m3_decode(const uint8_t* in, int64_t n, float* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = e4m3_to_f32(in[i]);
}
void oracle_e4m3_encode(const float* in, int64_t n, uint8_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = f32_to_e4m3(in[i]);
}

/* Per-row dynamic quantisation of bf16 rows: x [M,n] bf16 -> q [M,n] codes, scale [M] fp32. */
int oracle_quantize_rows(const uint16_t* x, int64_t M, int32_t n, uint8_t* q, float* scale) {
  if (M < 0 || n <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < M; ++r) {
    float amax = 0.0f;
    for (int32_t i = 0; i < n; ++i) {
      float a = fabsf(bf16_to_f32(x[r * n + i]));
      if (a > amax) amax = a;
    }
    if (amax < 0x1p-100f) amax = 0x1p-100f;
    float inv = 448.0f / amax;
    scale[r] = amax / 448.0f;
    for (int32_t i = 0; i < n; ++i) q[r * n + i] = f32_to_e4m3(bf16_to_f32(x[r * n + i]) * inv);
  }
  return ORACLE_OK;
}

/* GEMM1 + SwiGLU of the FP8 variant for one expert: xq [M,H] codes, sx [M]; wq [2I,H] codes (rows 0..I-1 gate,
 * I..2I-1 up), sw [2I]; act_out [M,I] bf16 bits. */
int oracle_gemm1_fp8(const uint8_t* xq, const float* sx, int64_t M, const uint8_t* wq, const float* sw,
                     int32_t H, int32_t I, uint16_t* act_out) {
  if (M < 0 || H <= 0 || I <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t r = 0; r < M; ++r) {
    for (int32_t i = 0; i < I; ++i) {
      const uint8_t* xr = xq + r * H;
      const uint8_t* wg = wq + (int64_t)i * H;
      const uint8_t* wu = wq + ((int64_t)I + i) * H;
      double g = 0.0, u = 0.0;
      for (int32_t h = 0; h < H; ++h) {
        double xv = (double)e4m3_to_f32(xr[h]);
        g += xv * (double)e4m3_to_f32(wg[h]);
        u += xv * (double)e4m3_to_f32(wu[h]);
      }
      g *= (double)sx[r] * (double)sw[i];
      u *= (double)sx[r] * (double)sw[I + i];
      act_out[r * I + i] = f32_to_bf16((float)(g / (1.0 + exp(-g)) * u));
    }
  }
  return ORACLE_OK;
}

/* GEMM2 of the FP8 variant for one expert: aq [M,I] codes, sa [M]; wq [H,I] codes, sw [H]; y_out [M,H] fp32. */
int oracle_gemm2_fp8(const uint8_t* aq, const float* sa, int64_t M, const uint8_t* wq, const float* sw,
                     int32_t H, int32_t I, float* y_out) {
  if (M < 0 || H <= 0 || I <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t r = 0; r < M; ++r) {
    for (int32_t c = 0; c < H; ++c) {
      const uint8_t* ar = aq + r * I;
      const uint8_t* wd = wq + (int64_t)c * I;
      double y = 0.0;
      for (int32_t i = 0; i < I; ++i) y += (double)e4m3_to_f32(ar[i]) * (double)e4m3_to_f32(wd[i]);
      y_out[r * H + c] = (float)(y * (double)sa[r] * (double)sw[c]);
    }
  }
  return ORACLE_OK;
}
