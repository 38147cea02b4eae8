/*
 * CPU oracle for the routed-expert MoE layer -- TEST INFRASTRUCTURE, not product.
 *
 * Plain, slow, fp64.  It states what the streamFFN path must compute: the paper
 * changes *when* expert work runs (Section 3.2: asynchronous EP, launch threshold,
 * final flush; Appendix "Grouped FFN invocations" and "Output return and combine"),
 * never *what* it computes, so the float result is the plain definition of a
 * top-k mixture-of-experts SwiGLU FFN:
 *
 *   out[t] = sum over slots j with ids[t,j] < E_local of
 *            w[t,j] * ( silu(x_t Wg[e]) (.) (x_t Wu[e]) ) Wd[e],      e = ids[t,j]
 *
 * with every routed contribution weighted by its routing coefficient exactly once
 * (Appendix "Output return and combine").  The FFN form itself (SwiGLU, no bias) is
 * fixed by the benchmark definition; the paper only says "FFN".
 *
 * Nothing here is shared with the CUDA path; only tests, the smoke check and the
 * CPU-baseline timing may call it.
 *
 * Parity pins (tests/test_oracle_*.py): per-token brute force in another language
 * and loop nest, dense-MLP special cases through library matmuls, closed forms of
 * silu, exhaustive codec tables.  No function here is "parity unpinned".
 *
 * Microscaling operands ("Evaluation Settings", models and environments: the routed-expert weights of two of the three
 * evaluated models are MXFP4): a block of 32 consecutive elements along the contraction
 * dimension shares one power-of-two scale stored as an 8-bit exponent (ue8m0); weights are
 * e2m1 elements, activations e4m3 elements.  The paper gives no quantisation rule; the one
 * taken here is "the smallest power of two that brings the block's largest magnitude
 * inside the element range", elements rounded to nearest even.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F64 = 0, ORACLE_BF16 = 1, ORACLE_FP8 = 2, ORACLE_MXFP4 = 3 };
enum { ORACLE_MIRROR_FP8_ACT = 1, ORACLE_MIRROR_MXFP8_ACT = 4 };

/* ---- codecs: exact decoders and the two round-to-nearest-even encoders ---- */

/* bf16 is the top 16 bits of an IEEE binary32. */
double oracle_bf16_to_f64(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* e4m3 "fn" variant: 1 sign, 4 exponent (bias 7), 3 mantissa; no infinities;
 * exponent 15 with mantissa 7 is NaN; largest finite 448. */
double oracle_e4m3_to_f64(uint8_t c) {
  int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0) v = ldexp((double)m, -9);          /* subnormal: m/8 * 2^-6 */
  else v = ldexp(1.0 + m / 8.0, e - 7);
  return s ? -v : v;
}

/* Round-to-nearest-even onto the e4m3fn grid, saturating at +-448. */
uint8_t oracle_f64_to_e4m3(double x) {
  uint8_t s = signbit(x) ? 0x80 : 0;
  double a = fabs(x);
  if (isnan(a)) return s | 0x7f;
  if (a >= 448.0) return s | 0x7e;
  if (a == 0.0) return s;
  int ex;
  frexp(a, &ex);             /* a = f * 2^ex, f in [0.5,1)  =>  a in [2^(ex-1), 2^ex) */
  int e = ex - 1;            /* unbiased exponent of the leading bit */
  if (e < -6) e = -6;        /* subnormal range shares the spacing of e = -6 */
  double ulp = ldexp(1.0, e - 3);
  double q = a / ulp;        /* exact: division by a power of two */
  double r = nearbyint(q);   /* default rounding mode = nearest even */
  double v = r * ulp;
  if (v >= 448.0) return s | 0x7e;
  /* re-encode v */
  if (v < ldexp(1.0, -6)) return s | (uint8_t)(int)(v / ldexp(1.0, -9));
  frexp(v, &ex);
  e = ex - 1;
  int m = (int)((v / ldexp(1.0, e) - 1.0) * 8.0);
  return s | (uint8_t)(((e + 7) << 3) | m);
}

/* Round-to-nearest-even of a double onto the bf16 grid (via binary32, which is
 * exact for the diagnostic use here: inputs are well inside float range). */
uint16_t oracle_f64_to_bf16(double x) {
  float f = (float)x;
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

/* e2m1: 1 sign, 2 exponent (bias 1), 1 mantissa bit; magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6.
 * The code sits in the low four bits of the byte. */
double oracle_e2m1_to_f64(uint8_t c) {
  int s = (c >> 3) & 1, e = (c >> 1) & 3, m = c & 1;
  double v = (e == 0) ? 0.5 * m : ldexp(1.0 + 0.5 * m, e - 1);
  return s ? -v : v;
}

/* Round-to-nearest-even onto the e2m1 grid, saturating at +-6. */
uint8_t oracle_f64_to_e2m1(double x) {
  static const double grid[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};
  uint8_t s = signbit(x) ? 8 : 0;
  double a = fabs(x);
  if (isnan(a) || a >= 6.0) return s | 7;
  int best = 0;
  for (int c = 1; c < 8; ++c) {
    double d0 = fabs(a - grid[best]), d1 = fabs(a - grid[c]);
    if (d1 < d0 || (d1 == d0 && (c & 1) == 0)) best = c;   /* ties: the code with an even mantissa */
  }
  return s | (uint8_t)best;
}

/* ue8m0: an unsigned power-of-two scale, value 2^(c-127); code 255 is NaN. */
double oracle_ue8m0_to_f64(uint8_t c) {
  if (c == 255) return NAN;
  return ldexp(1.0, (int)c - 127);
}

/* Block scale of a microscaling block: the smallest power of two s with
 * amax <= elem_max * s, as a ue8m0 code, where elem_max = 1.75*2^8 (e4m3, emax=8,
 * top mantissa 0.75) or 1.5*2^2 (e2m1).  amax is taken in binary32: with biased
 * exponent E and fraction f of amax, log2(s) = E - 127 - emax, one more when
 * f > top mantissa.  An all-zero block gets scale 1 (code 127); the code is clamped
 * to 0..254. */
uint8_t oracle_mx_scale_code(float amax, int emax, double top_mantissa) {
  if (amax == 0.0f) return 127;
  uint32_t u;
  memcpy(&u, &amax, 4);
  int E = (int)((u >> 23) & 0xff);
  double f = (double)(u & 0x7fffffu) / 8388608.0;
  int code = E - emax + (f > top_mantissa ? 1 : 0);
  if (code < 0) code = 0;
  if (code > 254) code = 254;
  return (uint8_t)code;
}

double oracle_silu(double x) { return x / (1.0 + exp(-x)); }

/* ---- element access in fp64 ---- */

typedef struct {
  int dtype;
  const void *data;
  const void *scale; /* fp8: fp32 block scales; mxfp4: ue8m0 codes */
} tensor_t;

/* activations: [T,H]; fp8 scales fp32 [T,H/128]; mxfp4: e4m3 codes, ue8m0 scales [T,H/32] */
static double x_at(const tensor_t *x, int64_t H, int64_t t, int64_t h) {
  int64_t i = t * H + h;
  switch (x->dtype) {
    case ORACLE_F64: return ((const double *)x->data)[i];
    case ORACLE_BF16: return oracle_bf16_to_f64(((const uint16_t *)x->data)[i]);
    case ORACLE_MXFP4:
      return oracle_e4m3_to_f64(((const uint8_t *)x->data)[i]) *
             oracle_ue8m0_to_f64(((const uint8_t *)x->scale)[t * (H / 32) + h / 32]);
    default:
      return oracle_e4m3_to_f64(((const uint8_t *)x->data)[i]) *
             (double)((const float *)x->scale)[t * (H / 128) + h / 128];
  }
}

/* weights: [E,R,C] row-major (R = contraction dimension); fp8 scales fp32 [E,R/128,C/128];
 * mxfp4: one e2m1 code per byte, ue8m0 scales [E,R/32,C] (32 consecutive r share a scale) */
static double w_at(const tensor_t *w, int64_t R, int64_t C, int64_t e, int64_t r, int64_t c) {
  int64_t i = (e * R + r) * C + c;
  switch (w->dtype) {
    case ORACLE_F64: return ((const double *)w->data)[i];
    case ORACLE_BF16: return oracle_bf16_to_f64(((const uint16_t *)w->data)[i]);
    case ORACLE_MXFP4:
      return oracle_e2m1_to_f64(((const uint8_t *)w->data)[i] & 15) *
             oracle_ue8m0_to_f64(((const uint8_t *)w->scale)[(e * (R / 32) + r / 32) * C + c]);
    default:
      return oracle_e4m3_to_f64(((const uint8_t *)w->data)[i]) *
             (double)((const float *)w->scale)[(e * (R / 128) + r / 128) * (C / 128) + c / 128];
  }
}

/* Re-quantisation of the intermediate for the fp8 configuration: per row and per
 * 128-wide block, scale = (float)(amax/448) (1 when the block is all zero), code =
 * RNE e4m3 of a/scale saturated at 448, value = code*scale.  The activation and
 * quantisation sit between the two expert GEMMs (Appendix "Grouped FFN invocations"). */
static void requant_fp8_row(double *a, int64_t I) {
  for (int64_t b = 0; b < I; b += 128) {
    int64_t n = (I - b < 128) ? (I - b) : 128;
    double amax = 0.0;
    for (int64_t i = 0; i < n; ++i) {
      double v = fabs(a[b + i]);
      if (v > amax) amax = v;
    }
    float s = (amax == 0.0) ? 1.0f : (float)((float)amax / 448.0f);
    for (int64_t i = 0; i < n; ++i) {
      double q = a[b + i] / (double)s;
      a[b + i] = oracle_e4m3_to_f64(oracle_f64_to_e4m3(q)) * (double)s;
    }
  }
}

/* Re-quantisation of the intermediate for the microscaling configuration: per row and
 * per 32-wide block, ue8m0 scale from the block's amax (rule above, e4m3 elements), code =
 * RNE e4m3 of a/scale (a division by a power of two), value = code*scale. */
static void requant_mxfp8_row(double *a, int64_t I) {
  for (int64_t b = 0; b < I; b += 32) {
    int64_t n = (I - b < 32) ? (I - b) : 32;
    double amax = 0.0;
    for (int64_t i = 0; i < n; ++i) {
      double v = fabs(a[b + i]);
      if (v > amax) amax = v;
    }
    double s = oracle_ue8m0_to_f64(oracle_mx_scale_code((float)amax, 8, 0.75));
    for (int64_t i = 0; i < n; ++i)
      a[b + i] = oracle_e4m3_to_f64(oracle_f64_to_e4m3(a[b + i] / s)) * s;
  }
}

/*
 * The layer, for a selection of tokens.
 *   ids  [T,k] global expert ids; ids >= E_local belong to another rank and are skipped
 *   w    [T,k] fp32 routing coefficients
 *   Wg,Wu [E_local,H,I];  Wd [E_local,I,H]
 *   sel  token indices to evaluate (NULL => 0..n_sel-1)
 *   out  [n_sel,H] fp64; a token with no local expert gives exact zeros
 * Returns 0, or -1 on a bad expert id (<0).
 */
int oracle_moe_forward(int dtype, int64_t T, int64_t H, int64_t I, int64_t E_local, int64_t k,
                       const void *X, const void *Xs, const int32_t *ids, const float *w,
                       const void *Wg, const void *Wgs, const void *Wu, const void *Wus,
                       const void *Wd, const void *Wds, const int64_t *sel, int64_t n_sel,
                       int mirror, double *out, int nthreads) {
  tensor_t tx = {dtype, X, Xs}, tg = {dtype, Wg, Wgs}, tu = {dtype, Wu, Wus}, td = {dtype, Wd, Wds};
  int bad = 0;
  (void)T;
#ifdef _OPENMP
  if (nthreads > 0) omp_set_num_threads(nthreads);
#else
  (void)nthreads;
#endif
#pragma omp parallel
  {
    double *x = (double *)malloc(sizeof(double) * H);
    double *g = (double *)malloc(sizeof(double) * I);
    double *u = (double *)malloc(sizeof(double) * I);
    double *y = (double *)malloc(sizeof(double) * H);
#pragma omp for schedule(dynamic, 1)
    for (int64_t s = 0; s < n_sel; ++s) {
      int64_t t = sel ? sel[s] : s;
      double *acc = out + s * H;
      for (int64_t h = 0; h < H; ++h) acc[h] = 0.0;
      for (int64_t h = 0; h < H; ++h) x[h] = x_at(&tx, H, t, h);
      for (int64_t j = 0; j < k; ++j) {
        int64_t e = ids[t * k + j];
        if (e < 0) { bad = 1; continue; }
        if (e >= E_local) continue;               /* another rank's expert */
        for (int64_t i = 0; i < I; ++i) g[i] = u[i] = 0.0;
        for (int64_t h = 0; h < H; ++h) {         /* h ascending for every i */
          double xv = x[h];
          for (int64_t i = 0; i < I; ++i) {
            g[i] += xv * w_at(&tg, H, I, e, h, i);
            u[i] += xv * w_at(&tu, H, I, e, h, i);
          }
        }
        for (int64_t i = 0; i < I; ++i) g[i] = oracle_silu(g[i]) * u[i];   /* a = silu(g) * u */
        if (mirror & ORACLE_MIRROR_FP8_ACT) requant_fp8_row(g, I);
        if (mirror & ORACLE_MIRROR_MXFP8_ACT) requant_mxfp8_row(g, I);
        for (int64_t h = 0; h < H; ++h) y[h] = 0.0;
        for (int64_t i = 0; i < I; ++i) {         /* i ascending for every h */
          double av = g[i];
          for (int64_t h = 0; h < H; ++h) y[h] += av * w_at(&td, I, H, e, i, h);
        }
        double wj = (double)w[t * k + j];
        for (int64_t h = 0; h < H; ++h) acc[h] += wj * y[h];
      }
    }
    free(x); free(g); free(u); free(y);
  }
  return bad ? -1 : 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
