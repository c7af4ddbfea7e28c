/*
 * Oracle: Caffe-semantics convolution layer forward on the CPU.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * tests and the bench's CPU-baseline leg compare the CUDA library against.  It
 * shares no code, header, table or helper with the CUDA path and the product
 * never calls it.
 *
 * What it computes (the paper gives no formula for any layer; it inherits every
 * layer from BVLC Caffe, Section 2.2, and discusses the FP16 value range in
 * Section 3.1).  With x, w, bias holding IEEE binary16 values taken as reals:
 *
 *   P = floor((H + 2*pad_h - dil_h*(R-1) - 1) / stride_h) + 1      (Q likewise)
 *   grp(k) = k / (K/g)
 *   v[n,k,p,q] = bias[k]
 *              + sum_{c'<C/g} sum_{r<R} sum_{s<S}
 *                  X(n, grp(k)*(C/g)+c', p*stride_h-pad_h+r*dil_h,
 *                                        q*stride_w-pad_w+s*dil_w) * w[k,c',r,s]
 *   X = x inside the image, 0 outside (zero padding, no kernel flip)
 *   y = round_to_nearest_even_fp16( relu ? max(v,0) : v )
 *
 * The sum is carried in an fp64 accumulator in the fixed order bias, c', r, s
 * (a product of two binary16 numbers is exact in fp64), and rounded once.
 *
 * Entry points
 *   ref_conv_naive   the definition as a literal loop nest (small problems)
 *   ref_conv_fast    the same additions in the same order per output element,
 *                    arranged row-wise and spread over (n,k) with OpenMP; must
 *                    be bit-identical to ref_conv_naive
 *   ref_conv_points  the definition evaluated at a list of output coordinates
 *                    (sampled checks on problems too large to compute whole)
 *   ref_out_dim      the output-size formula
 *   ref_half_to_double / ref_double_to_half   binary16 conversion used above
 *   ref_cast_f32_to_f16   the weight-file converter's arithmetic (Section 3.4): every binary32
 *                    value rounded to the nearest binary16, ties to even; counts the finite
 *                    inputs that no finite binary16 can hold (they become infinities)
 *   ref_inner_product  the inner-product (fully connected) layer, named in Section 3.1 as
 *                    the other layer whose long sums overflow FP16:
 *                    y[n,k] = round( relu?( bias[k] + sum_c x[n,c] * w[k,c] ) ), fp64 sum
 *   ref_batchnorm    the batch-norm layer of Section 3.1 as its plain definition: per channel
 *                    over the N*H*W values, mean = sum x / M, var = sum (x - mean)^2 / M (the
 *                    biased variance), y = round( (x - mean) / sqrt(var + eps) ), all in fp64
 *                    (the grouped mean and the shift before squaring that the section describes
 *                    are ways of reaching these same numbers in narrow arithmetic); with stored
 *                    statistics the mean and variance are inputs
 *   ref_bn_fold      stored statistics and an optional per-channel scale and shift folded into
 *                    the weights and bias of the convolution before the batch norm
 *
 * Parity pins: every function here is pinned by the CPU tests (hand-worked
 * examples, closed forms, matmul / correlate2d restatements, invariants).
 * Unpinned by choice: NaN propagation.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct ref_conv_params {
  int32_t n, c, h, w;
  int32_t k, r, s;
  int32_t pad_h, pad_w, stride_h, stride_w, dil_h, dil_w;
  int32_t group;
} ref_conv_params;

/* ---- binary16 <-> double ------------------------------------------------ */

/* value of a binary16 bit pattern: (-1)^s * 2^(e-15) * (1 + m/1024), or the
   subnormal (-1)^s * 2^-14 * (m/1024) when e == 0 */
double ref_half_to_double(uint16_t bits) {
  int sign = bits >> 15;
  int e = (bits >> 10) & 0x1f;
  int m = bits & 0x3ff;
  double v;
  if (e == 0x1f) {
    v = m ? NAN : INFINITY;
  } else if (e == 0) {
    v = ldexp((double)m, -24);
  } else {
    v = ldexp((double)(1024 + m), e - 25);
  }
  return sign ? -v : v;
}

/* round a double to the nearest binary16, ties to even; overflow goes to inf
   (|v| >= 65520, the midpoint above the largest finite value 65504) */
uint16_t ref_double_to_half(double v) {
  uint16_t sign = signbit(v) ? 0x8000u : 0u;
  double a = fabs(v);
  if (isnan(v)) return (uint16_t)(sign | 0x7e00u);
  if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u);
  if (a == 0.0) return sign;
  int ex;
  (void)frexp(a, &ex);          /* a = f * 2^ex, f in [0.5,1): exponent of a is ex-1 */
  int e = ex - 1;
  if (e < -14) e = -14;         /* subnormal range shares the quantum of 2^-14 */
  /* spacing of representable values near a is 2^(e-10); a/quantum is exact */
  double q = ldexp(a, 10 - e);
  double rq = nearbyint(q);     /* default rounding mode: nearest, ties to even */
  /* rq is an integer in [0, 2048]; 2048 means the next binade */
  long mant = (long)rq;
  if (mant == 2048) { mant = 1024; e += 1; }
  if (mant < 1024) {
    /* subnormal (e == -14) or zero */
    return (uint16_t)(sign | (uint16_t)mant);
  }
  if (e > 15) return (uint16_t)(sign | 0x7c00u);
  return (uint16_t)(sign | (uint16_t)((e + 15) << 10) | (uint16_t)(mant - 1024));
}

/* ---- shape ------------------------------------------------------------- */

static int64_t floor_div(int64_t a, int64_t b) { /* b > 0 */
  int64_t q = a / b;
  if ((a % b) != 0 && a < 0) q -= 1;
  return q;
}

/* output extent along one axis; may be <= 0 for an invalid layer */
int64_t ref_out_dim(int64_t in, int64_t kernel, int64_t pad, int64_t stride, int64_t dil) {
  return floor_div(in + 2 * pad - dil * (kernel - 1) - 1, stride) + 1;
}

/* 0 if the parameters describe a valid layer, else nonzero */
int ref_conv_check(const ref_conv_params* p) {
  if (!p) return 1;
  if (p->n < 1 || p->c < 1 || p->h < 1 || p->w < 1 || p->k < 1 || p->r < 1 || p->s < 1) return 1;
  if (p->group < 1 || p->stride_h < 1 || p->stride_w < 1 || p->dil_h < 1 || p->dil_w < 1) return 1;
  if (p->pad_h < 0 || p->pad_w < 0) return 1;
  if (p->c % p->group || p->k % p->group) return 1;
  if (ref_out_dim(p->h, p->r, p->pad_h, p->stride_h, p->dil_h) < 1) return 1;
  if (ref_out_dim(p->w, p->s, p->pad_w, p->stride_w, p->dil_w) < 1) return 1;
  return 0;
}

/* ---- the definition, one output element -------------------------------- */

static double conv_at(const ref_conv_params* p, const uint16_t* x, const uint16_t* w,
                      const uint16_t* bias, int64_t n, int64_t k, int64_t op, int64_t oq) {
  const int64_t cg = p->c / p->group, kg = p->k / p->group;
  const int64_t grp = k / kg;
  double acc = bias ? ref_half_to_double(bias[k]) : 0.0;
  for (int64_t cc = 0; cc < cg; ++cc) {
    const int64_t ch = grp * cg + cc;
    for (int64_t r = 0; r < p->r; ++r) {
      const int64_t ih = op * p->stride_h - p->pad_h + r * p->dil_h;
      for (int64_t s = 0; s < p->s; ++s) {
        const int64_t iw = oq * p->stride_w - p->pad_w + s * p->dil_w;
        if (ih < 0 || ih >= p->h || iw < 0 || iw >= p->w) continue; /* X = 0 */
        const double xv = ref_half_to_double(x[((n * p->c + ch) * p->h + ih) * p->w + iw]);
        const double wv = ref_half_to_double(w[((k * cg + cc) * p->r + r) * p->s + s]);
        acc += xv * wv;
      }
    }
  }
  return acc;
}

static uint16_t finish(double v, int relu) {
  if (relu && v < 0.0) v = 0.0;
  return ref_double_to_half(v);
}

int ref_conv_naive(const ref_conv_params* p, const uint16_t* x, const uint16_t* w,
                   const uint16_t* bias, uint16_t* y, int relu) {
  if (ref_conv_check(p) || !x || !w || !y) return 1;
  const int64_t P = ref_out_dim(p->h, p->r, p->pad_h, p->stride_h, p->dil_h);
  const int64_t Q = ref_out_dim(p->w, p->s, p->pad_w, p->stride_w, p->dil_w);
  for (int64_t n = 0; n < p->n; ++n)
    for (int64_t k = 0; k < p->k; ++k)
      for (int64_t op = 0; op < P; ++op)
        for (int64_t oq = 0; oq < Q; ++oq)
          y[((n * p->k + k) * P + op) * Q + oq] = finish(conv_at(p, x, w, bias, n, k, op, oq), relu);
  return 0;
}

/* coords: npoints rows of (n, k, p, q); out: npoints binary16 results */
int ref_conv_points(const ref_conv_params* p, const uint16_t* x, const uint16_t* w,
                    const uint16_t* bias, int relu, const int64_t* coords, int64_t npoints,
                    uint16_t* out) {
  if (ref_conv_check(p) || !x || !w || !out || (!coords && npoints)) return 1;
  const int64_t P = ref_out_dim(p->h, p->r, p->pad_h, p->stride_h, p->dil_h);
  const int64_t Q = ref_out_dim(p->w, p->s, p->pad_w, p->stride_w, p->dil_w);
  int bad = 0;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < npoints; ++i) {
    const int64_t n = coords[4 * i], k = coords[4 * i + 1], op = coords[4 * i + 2], oq = coords[4 * i + 3];
    if (n < 0 || n >= p->n || k < 0 || k >= p->k || op < 0 || op >= P || oq < 0 || oq >= Q) {
#pragma omp atomic write
      bad = 1;
      continue;
    }
    out[i] = finish(conv_at(p, x, w, bias, n, k, op, oq), relu);
  }
  return bad;
}

/* ---- same additions, arranged by rows ---------------------------------- */

/* For every (n,k) the accumulator plane starts at bias[k]; then for c', r, s in
   that order the tap's contribution is added to every output element it reaches.
   Each output element therefore receives exactly the additions of conv_at in the
   same order (taps that fall in the padding are skipped in both). */
int ref_conv_fast(const ref_conv_params* p, const uint16_t* x, const uint16_t* w,
                  const uint16_t* bias, uint16_t* y, int relu) {
  if (ref_conv_check(p) || !x || !w || !y) return 1;
  const int64_t P = ref_out_dim(p->h, p->r, p->pad_h, p->stride_h, p->dil_h);
  const int64_t Q = ref_out_dim(p->w, p->s, p->pad_w, p->stride_w, p->dil_w);
  const int64_t cg = p->c / p->group, kg = p->k / p->group;
  const int64_t xelems = (int64_t)p->n * p->c * p->h * p->w;
  /* binary16 -> float is exact; float -> double in the loop is exact too */
  float* xf = (float*)malloc(sizeof(float) * (size_t)xelems);
  if (!xf) return 2;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < xelems; ++i) xf[i] = (float)ref_half_to_double(x[i]);

  int fail = 0;
#pragma omp parallel
  {
    double* acc = (double*)malloc(sizeof(double) * (size_t)(P * Q));
    if (!acc) {
#pragma omp atomic write
      fail = 1;
    }
#pragma omp barrier
    if (!fail) {
#pragma omp for collapse(2) schedule(dynamic, 1)
      for (int64_t n = 0; n < p->n; ++n) {
        for (int64_t k = 0; k < p->k; ++k) {
          const int64_t grp = k / kg;
          const double b = bias ? ref_half_to_double(bias[k]) : 0.0;
          for (int64_t i = 0; i < P * Q; ++i) acc[i] = b;
          for (int64_t cc = 0; cc < cg; ++cc) {
            const float* xplane = xf + ((n * p->c + grp * cg + cc) * p->h) * (int64_t)p->w;
            for (int64_t r = 0; r < p->r; ++r) {
              for (int64_t s = 0; s < p->s; ++s) {
                const double wv = ref_half_to_double(w[((k * cg + cc) * p->r + r) * p->s + s]);
                /* columns q with 0 <= q*stride_w - pad_w + s*dil_w < W */
                const int64_t off = s * p->dil_w - p->pad_w;
                int64_t qlo = off >= 0 ? 0 : (-off + p->stride_w - 1) / p->stride_w;
                int64_t qhi = floor_div(p->w - 1 - off, p->stride_w);
                if (qhi > Q - 1) qhi = Q - 1;
                if (qlo > qhi) continue;
                for (int64_t op = 0; op < P; ++op) {
                  const int64_t ih = op * p->stride_h - p->pad_h + r * p->dil_h;
                  if (ih < 0 || ih >= p->h) continue;
                  const float* xrow = xplane + ih * p->w + off;
                  double* arow = acc + op * Q;
                  const int64_t sw = p->stride_w;
                  for (int64_t oq = qlo; oq <= qhi; ++oq) arow[oq] += (double)xrow[oq * sw] * wv;
                }
              }
            }
          }
          uint16_t* yplane = y + (n * p->k + k) * P * Q;
          for (int64_t i = 0; i < P * Q; ++i) yplane[i] = finish(acc[i], relu);
        }
      }
    }
    free(acc);
  }
  free(xf);
  return fail ? 2 : 0;
}

/* ---- FP32 -> FP16 cast (the converter's arithmetic, Section 3.4) --------- */

/* dst[i] = binary16 nearest to src[i] (ties to even; |v| >= 65520 -> inf; NaN -> a quiet NaN
   of the same sign).  Returns the number of FINITE inputs whose result is infinite. */
int64_t ref_cast_f32_to_f16(const float* src, uint16_t* dst, int64_t count) {
  int64_t overflow = 0;
  for (int64_t i = 0; i < count; ++i) {
    const double v = (double)src[i];  /* exact */
    const uint16_t h = ref_double_to_half(v);
    dst[i] = h;
    if (isfinite(v) && (h & 0x7fffu) == 0x7c00u) ++overflow;
  }
  return overflow;
}

/* ---- inner product (fully connected) layer ------------------------------ */

/* x[N][C], w[K][C], bias[K] or NULL, y[N][K]; the sum runs bias first, then c ascending */
void ref_inner_product(int64_t n, int64_t c, int64_t k, const uint16_t* x, const uint16_t* w,
                       const uint16_t* bias, uint16_t* y, int relu) {
  for (int64_t in = 0; in < n; ++in) {
    for (int64_t ik = 0; ik < k; ++ik) {
      double acc = bias ? ref_half_to_double(bias[ik]) : 0.0;
      for (int64_t ic = 0; ic < c; ++ic)
        acc += ref_half_to_double(x[in * c + ic]) * ref_half_to_double(w[ik * c + ic]);
      y[in * k + ik] = finish(acc, relu);
    }
  }
}

/* ---- batch norm (Section 3.1) -------------------------------------------- */

/* x[N][C][HW] -> y of the same shape.  use_stored == 0: mean[c] and var[c] are computed from x
   and written; otherwise they are read.  No scale or shift (Caffe keeps those in a separate
   layer). */
void ref_batchnorm(int64_t n, int64_t c, int64_t hw, const uint16_t* x, double eps, int use_stored,
                   double* mean, double* var, uint16_t* y) {
  const double m = (double)(n * hw);
  for (int64_t ic = 0; ic < c; ++ic) {
    if (!use_stored) {
      double sum = 0.0;
      for (int64_t in = 0; in < n; ++in)
        for (int64_t i = 0; i < hw; ++i) sum += ref_half_to_double(x[(in * c + ic) * hw + i]);
      mean[ic] = sum / m;
      double sq = 0.0;
      for (int64_t in = 0; in < n; ++in)
        for (int64_t i = 0; i < hw; ++i) {
          const double d = ref_half_to_double(x[(in * c + ic) * hw + i]) - mean[ic];
          sq += d * d;
        }
      var[ic] = sq / m;
    }
    const double inv = 1.0 / sqrt(var[ic] + eps);
    for (int64_t in = 0; in < n; ++in)
      for (int64_t i = 0; i < hw; ++i) {
        const int64_t at = (in * c + ic) * hw + i;
        y[at] = ref_double_to_half((ref_half_to_double(x[at]) - mean[ic]) * inv);
      }
  }
}

/* a_k = gamma_k / sqrt(var_k + eps) (gamma = 1 if NULL); w'[k][j] = round(w[k][j] * a_k);
   b'[k] = round((b[k] - mean_k) * a_k + beta_k) (b = 0 if bias is NULL, beta = 0 if NULL):
   conv(x, w') + b' equals gamma * (conv(x, w) + b - mean) / sqrt(var + eps) + beta up to the
   rounding of w' and b'. */
void ref_bn_fold(int64_t k, int64_t per_k, const uint16_t* w, const uint16_t* bias, const double* mean,
                 const double* var, const double* gamma, const double* beta, double eps, uint16_t* w_out,
                 uint16_t* b_out) {
  for (int64_t ik = 0; ik < k; ++ik) {
    const double a = (gamma ? gamma[ik] : 1.0) / sqrt(var[ik] + eps);
    for (int64_t j = 0; j < per_k; ++j)
      w_out[ik * per_k + j] = ref_double_to_half(ref_half_to_double(w[ik * per_k + j]) * a);
    const double b = bias ? ref_half_to_double(bias[ik]) : 0.0;
    b_out[ik] = ref_double_to_half((b - mean[ik]) * a + (beta ? beta[ik] : 0.0));
  }
}

int ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
