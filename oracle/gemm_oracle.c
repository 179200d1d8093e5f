/*
 * CPU oracle for the dense GEMM hot path -- TEST INFRASTRUCTURE, NOT PRODUCT.
 *
 * Only the tests, the smoke check and the benchmark's cpu_baseline / reference
 * arm may call this file.  It shares no code with the CUDA library and is never
 * a fallback for it.
 *
 * What it computes is the textbook definition the paper's case study names
 * ("GEMM", Section 5.4) written out as a plain triple loop:
 *
 *     y(b,i,j) = act( alpha * sum_{k=0}^{K-1} opA(b,i,k) * opB(b,k,j)
 *                     + beta * C_in(b,i,j) + bias[j] )        (bias[i] when bias_per_row)
 *
 * act: identity, ReLU, GELU (exact erf form), GELU (tanh form) or SiLU;
 *
 * evaluated in IEEE double, k ascending, one output at a time, no blocking,
 * no reassociation (build without -ffast-math).  Inputs arrive as the very bit
 * patterns the GPU receives (uint16 for bf16 / fp16, float for fp32) and are
 * decoded exactly; a product of two significands of at most 11 bits is exact in
 * double, so the only rounding is the fp64 summation (relative error about
 * K * 2^-53 of sum |a||b|).
 *
 * Row-major storage convention:
 *   transa = 0: A is M x K, element (i,k) at A[i*lda + k];  transa = 1: A is
 *   stored K x M, element (i,k) at A[k*lda + i].
 *   transb = 0: B is K x N, element (k,j) at B[k*ldb + j];  transb = 1: B is
 *   stored N x K, element (k,j) at B[j*ldb + k].
 *   C / D is M x N, element (i,j) at C[i*ldc + j].
 *   Batch b adds b*stride_{a,b,c} elements.
 *
 * Parity pins (tests/test_oracle_pins.py): exhaustive codec round trips and
 * hand values, identity / permutation matrices, all-ones inputs (= K), rank-1
 * closed form, hand-computed tiny cases, alpha/beta special cases, batched ==
 * loop of singles, textbook values of the normal CDF for GELU, closed forms of
 * the logistic function for SiLU and the tanh GELU (plus the library's fp64
 * routines), row bias == column bias of the transposed product, and numpy's
 * fp64 matmul on small shapes.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

enum { OR_BF16 = 0, OR_F16 = 1, OR_F32 = 2, OR_FP8_E4M3 = 3, OR_FP8_E5M2 = 4 };
/* even values: no bias; odd values: the same activation with a bias added first */
enum { OR_EPI_NONE = 0, OR_EPI_BIAS = 1, OR_EPI_RELU = 2, OR_EPI_BIAS_RELU = 3,
       OR_EPI_GELU_ERF = 4, OR_EPI_BIAS_GELU_ERF = 5, OR_EPI_GELU_TANH = 6, OR_EPI_BIAS_GELU_TANH = 7,
       OR_EPI_SILU = 8, OR_EPI_BIAS_SILU = 9 };

typedef struct {
  int64_t M, N, K;
  int32_t transa, transb;
  int32_t ab_dtype;      /* OR_BF16, OR_F16 (uint16 patterns) or OR_FP8_E4M3, OR_FP8_E5M2 (uint8 patterns) */
  int32_t c_dtype;       /* dtype of C_in (read only when beta != 0) */
  int64_t lda, ldb, ldc;
  int64_t stride_a, stride_b, stride_c;
  int32_t epilogue;
  int32_t bias_per_row;  /* 0: bias[N], one value per output column; 1: bias[M], one value per output row */
} oracle_desc_t;

/* ---- codecs: bit pattern -> double (exact) ------------------------------ */

double oracle_bf16_to_f64(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

double oracle_f16_to_f64(uint16_t h) {
  int sign = (h >> 15) & 1;
  int e = (h >> 10) & 0x1F;
  int m = h & 0x3FF;
  double v;
  if (e == 0) {
    v = ldexp((double)m, -24);                 /* subnormal: m * 2^-24 */
  } else if (e == 31) {
    v = m ? NAN : INFINITY;
  } else {
    v = ldexp((double)(m | 0x400), e - 25);    /* (1.m) * 2^(e-15) */
  }
  return sign ? -v : v;
}

/* 8-bit floats (the OCP FP8 formats the fifth-generation tensor cores take).
 * E4M3: 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinities: exponent field 15 is an ordinary binade
 * (largest finite value 1.75 * 2^8 = 448) except that mantissa 7 there is NaN.
 * E5M2: 1 sign, 5 exponent (bias 15), 2 mantissa bits; IEEE-like, exponent field 31 is infinity / NaN. */
double oracle_e4m3_to_f64(uint8_t h) {
  int sign = (h >> 7) & 1, e = (h >> 3) & 0xF, m = h & 0x7;
  double v;
  if (e == 15 && m == 7) v = NAN;
  else if (e == 0) v = ldexp((double)m, -9);            /* subnormal: m/8 * 2^-6 */
  else v = ldexp((double)(m | 0x8), e - 10);           /* (1.m) * 2^(e-7) */
  return sign ? -v : v;
}
double oracle_e5m2_to_f64(uint8_t h) {
  int sign = (h >> 7) & 1, e = (h >> 2) & 0x1F, m = h & 0x3;
  double v;
  if (e == 31) v = m ? NAN : INFINITY;
  else if (e == 0) v = ldexp((double)m, -16);           /* subnormal: m/4 * 2^-14 */
  else v = ldexp((double)(m | 0x4), e - 17);           /* (1.m) * 2^(e-15) */
  return sign ? -v : v;
}

/* ---- codecs: double -> bit pattern, round to nearest even --------------- */
/* Generic RNE onto a binary format with `mbits` stored mantissa bits, exponent
 * bias `bias` and `ebits` exponent bits.  Works directly from the double, so
 * there is no intermediate fp32 rounding. */
static uint32_t rne_encode(double x, int mbits, int ebits, int bias) {
  uint32_t sign = signbit(x) ? 1u : 0u;
  uint32_t emax_field = (1u << ebits) - 1u;
  if (isnan(x)) return (sign << (mbits + ebits)) | (emax_field << mbits) | (1u << (mbits - 1));
  double a = fabs(x);
  if (isinf(a)) return (sign << (mbits + ebits)) | (emax_field << mbits);
  if (a == 0.0) return sign << (mbits + ebits);
  int ex;
  (void)frexp(a, &ex);                 /* a = f * 2^ex, f in [0.5,1) */
  int e = ex - 1;                      /* a = (1.x) * 2^e            */
  int emin = 1 - bias;                 /* smallest normal exponent   */
  int q = (e < emin ? emin : e) - mbits;   /* exponent of one ulp at this magnitude */
  double scaled = ldexp(a, -q);        /* exact: power-of-two scaling */
  double r = nearbyint(scaled);        /* default rounding mode = RNE */
  /* r is an integer < 2^(mbits+2); re-normalise */
  uint64_t mant = (uint64_t)r;
  int64_t efield;
  if (e < emin) {                      /* subnormal range: mant in [0, 2^mbits] */
    efield = 0;
    if (mant >> mbits) { efield = 1; mant -= (1ull << mbits); }
  } else {
    efield = e + bias;
    if (mant >> (mbits + 1)) { mant >>= 1; efield += 1; }   /* rounded up to next binade */
    mant -= (1ull << mbits);
  }
  if (efield >= (int64_t)emax_field) return (sign << (mbits + ebits)) | (emax_field << mbits); /* overflow -> Inf */
  return (sign << (mbits + ebits)) | ((uint32_t)efield << mbits) | (uint32_t)mant;
}

uint16_t oracle_f64_to_bf16(double x) { return (uint16_t)rne_encode(x, 7, 8, 127); }
uint16_t oracle_f64_to_f16(double x)  { return (uint16_t)rne_encode(x, 10, 5, 15); }
float    oracle_f64_to_f32(double x)  { return (float)x; }   /* C conversion is RNE */

/* ---- activation in fp64 -------------------------------------------------- */
/* GELU with the exact error function: x * Phi(x), Phi the standard normal CDF.
 * erfc form keeps relative accuracy in the negative tail. */
double oracle_gelu_erf(double t) { return 0.5 * t * erfc(-t * 0.70710678118654752440); }
/* The same function through erf; the pins require both forms to agree. */
double oracle_gelu_erf_alt(double t) { return 0.5 * t * (1.0 + erf(t * 0.70710678118654752440)); }

/* The logistic function 1 / (1 + e^-t), evaluated on the side where the exponential cannot overflow. */
double oracle_logistic(double t) {
  if (t >= 0.0) return 1.0 / (1.0 + exp(-t));
  double e = exp(t);
  return e / (1.0 + e);
}
/* SiLU (swish): t * logistic(t). */
double oracle_silu(double t) { return t * oracle_logistic(t); }
/* GELU, tanh form: 0.5 t (1 + tanh u) with u = sqrt(2/pi) (t + 0.044715 t^3).  Evaluated as t * logistic(2u),
 * the same function (0.5 (1 + tanh u) = 1 / (1 + e^-2u)) without the cancellation of 1 + tanh u in the negative
 * tail; the pins compare it with the tanh expression. */
double oracle_gelu_tanh(double t) {
  double u = 0.79788456080286535588 * (t + 0.044715 * t * t * t);
  return t * oracle_logistic(2.0 * u);
}

int oracle_max_threads(void);

static double load_ab(const void* p, int dtype, int64_t idx) {
  if (dtype == OR_FP8_E4M3) return oracle_e4m3_to_f64(((const uint8_t*)p)[idx]);
  if (dtype == OR_FP8_E5M2) return oracle_e5m2_to_f64(((const uint8_t*)p)[idx]);
  const uint16_t* h = (const uint16_t*)p;
  return dtype == OR_BF16 ? oracle_bf16_to_f64(h[idx]) : oracle_f16_to_f64(h[idx]);
}

static double load_c(const void* p, int dtype, int64_t idx) {
  if (dtype == OR_F32) return (double)((const float*)p)[idx];
  return load_ab(p, dtype, idx);
}

/*
 * Evaluate the definition on the cross product batches x rows x cols.
 * Outputs (each nb*nr*nc doubles, [batch][row][col] order):
 *   y      unrounded fp64 result
 *   bound  |alpha| * sum_k |a||b| + |beta| * |C_in| + |bias|   (tolerance scale)
 * `bound` may be NULL.  `threads` <= 0 lets OpenMP decide.  Returns 0, or -1
 * on a bad argument.
 */
int oracle_gemm(const oracle_desc_t* d, const void* A, const void* B, const void* C_in,
                const float* bias, float alpha, float beta,
                const int64_t* batches, int64_t nb, const int64_t* rows, int64_t nr,
                const int64_t* cols, int64_t nc, double* y, double* bound, int threads) {
  if (!d || !A || !B || !y || !batches || !rows || !cols) return -1;
  if (d->epilogue < OR_EPI_NONE || d->epilogue > OR_EPI_BIAS_SILU) return -1;
  int has_bias = d->epilogue & 1;
  int relu = d->epilogue == OR_EPI_RELU || d->epilogue == OR_EPI_BIAS_RELU;
  int gelu = d->epilogue == OR_EPI_GELU_ERF || d->epilogue == OR_EPI_BIAS_GELU_ERF;
  int gelu_tanh = d->epilogue == OR_EPI_GELU_TANH || d->epilogue == OR_EPI_BIAS_GELU_TANH;
  int silu = d->epilogue == OR_EPI_SILU || d->epilogue == OR_EPI_BIAS_SILU;
  if (has_bias && !bias) return -1;
  if (beta != 0.0f && !C_in) return -1;
  const int64_t K = d->K;
  const double dalpha = (double)alpha, dbeta = (double)beta;
  int64_t total = nb * nr * nc;
  int nthreads = threads > 0 ? threads : oracle_max_threads();
  (void)nthreads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 64) num_threads(nthreads)
#endif
  for (int64_t o = 0; o < total; ++o) {
    int64_t b = batches[o / (nr * nc)];
    int64_t i = rows[(o / nc) % nr];
    int64_t j = cols[o % nc];
    int64_t a0 = b * d->stride_a, b0 = b * d->stride_b;
    double acc = 0.0, absdot = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      double av = load_ab(A, d->ab_dtype, a0 + (d->transa ? k * d->lda + i : i * d->lda + k));
      double bv = load_ab(B, d->ab_dtype, b0 + (d->transb ? j * d->ldb + k : k * d->ldb + j));
      acc += av * bv;
      absdot += fabs(av) * fabs(bv);
    }
    double t = dalpha * acc;
    double bnd = fabs(dalpha) * absdot;
    if (beta != 0.0f) {
      double cv = load_c(C_in, d->c_dtype, b * d->stride_c + i * d->ldc + j);
      t += dbeta * cv;
      bnd += fabs(dbeta) * fabs(cv);
    }
    if (has_bias) {
      double bv = (double)bias[d->bias_per_row ? i : j];
      t += bv;
      bnd += fabs(bv);
    }
    if (relu) t = t > 0.0 ? t : 0.0;
    if (gelu) t = oracle_gelu_erf(t);
    if (gelu_tanh) t = oracle_gelu_tanh(t);
    if (silu) t = oracle_silu(t);
    y[o] = t;
    if (bound) bound[o] = bnd;
  }
  return 0;
}

/* Round an array of fp64 results to the output dtype's bit patterns (RNE).
 * out is uint16[n] for bf16 / fp16 and float[n] for fp32. */
int oracle_round_to(const double* y, int64_t n, int dtype, void* out) {
  if (!y || !out) return -1;
  for (int64_t i = 0; i < n; ++i) {
    if (dtype == OR_BF16) ((uint16_t*)out)[i] = oracle_f64_to_bf16(y[i]);
    else if (dtype == OR_F16) ((uint16_t*)out)[i] = oracle_f64_to_f16(y[i]);
    else ((float*)out)[i] = oracle_f64_to_f32(y[i]);
  }
  return 0;
}

/* Decode an array of 16-bit patterns to double (used by the tests to compare a
 * GPU output buffer with y in a common domain). */
int oracle_decode(const void* in, int64_t n, int dtype, double* out) {
  if (!in || !out) return -1;
  for (int64_t i = 0; i < n; ++i) out[i] = load_c(in, dtype, i);
  return 0;
}

int oracle_max_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
