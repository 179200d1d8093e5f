/*
 * Seeded, counter-based synthetic input generators.  Shared as DATA by the
 * oracle side and the CUDA side of every test: this file holds none of the
 * GEMM arithmetic, only "element index -> value" hashing and the rounding of
 * the drawn value to the storage type.
 *
 * Element `i` of tensor `tensor_id` under `seed` is a pure function of
 * (seed, tensor_id, i), so buffers can be filled in parallel and a sub-range
 * can be regenerated anywhere.
 *
 *   h(c)     = splitmix64 finaliser of (seed + tensor_id * GOLDEN + c)
 *   uniform  = (h >> 11) * 2^-53            in [0,1)
 *   normal   = sqrt(-2 ln(1-u1)) cos(2 pi u2),  u1 = uniform(i), u2 = uniform(i + 2^62)
 *   integer  = lo + h mod (hi - lo + 1)
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

enum { G_BF16 = 0, G_F16 = 1, G_F32 = 2, G_FP8_E4M3 = 3, G_FP8_E5M2 = 4 };

static inline uint64_t mix(uint64_t seed, uint64_t tensor_id, uint64_t c) {
  uint64_t z = seed + tensor_id * 0x9E3779B97F4A7C15ull + c;
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

static inline double unif(uint64_t h) { return (double)(h >> 11) * (1.0 / 9007199254740992.0); }

static inline uint16_t f32_to_bf16_bits(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);   /* NaN */
  u += 0x7FFFu + ((u >> 16) & 1u);                                           /* RNE */
  return (uint16_t)(u >> 16);
}

static inline uint16_t f32_to_f16_bits(float f) {
  _Float16 h = (_Float16)f;   /* hardware / soft-float conversion, round to nearest even */
  uint16_t b;
  memcpy(&b, &h, 2);
  return b;
}

/* Nearest 8-bit float (ties to even) with `mbits` mantissa bits and exponent bias `bias`; magnitudes beyond the
 * largest finite value saturate to it, NaN becomes zero: the generators only ever emit finite numbers. */
static inline uint8_t f64_to_fp8_bits(double v, int mbits, int bias, double max_finite) {
  uint8_t sign = signbit(v) ? 0x80 : 0;
  double a = fabs(v);
  if (!(a == a) || a == 0.0) return sign;
  if (a > max_finite) a = max_finite;
  int ex;
  (void)frexp(a, &ex);
  int e = ex - 1, emin = 1 - bias;
  int q = (e < emin ? emin : e) - mbits;            /* exponent of one unit in the last place here */
  double r = ldexp(nearbyint(ldexp(a, -q)), q);     /* default rounding mode: to nearest, ties to even */
  if (r == 0.0) return sign;
  (void)frexp(r, &ex);
  e = ex - 1;
  if (e < emin) return (uint8_t)(sign | (unsigned)ldexp(r, mbits - emin));                 /* subnormal */
  unsigned mant = (unsigned)ldexp(r, mbits - e) - (1u << mbits);
  return (uint8_t)(sign | ((unsigned)(e + bias) << mbits) | mant);
}

static inline void store(void* out, int64_t i, int dtype, double v) {
  if (dtype == G_FP8_E4M3) { ((uint8_t*)out)[i] = f64_to_fp8_bits(v, 3, 7, 448.0); return; }
  if (dtype == G_FP8_E5M2) { ((uint8_t*)out)[i] = f64_to_fp8_bits(v, 2, 15, 57344.0); return; }
  float f = (float)v;
  if (dtype == G_BF16) ((uint16_t*)out)[i] = f32_to_bf16_bits(f);
  else if (dtype == G_F16) ((uint16_t*)out)[i] = f32_to_f16_bits(f);
  else ((float*)out)[i] = f;
}

void gen_uniform(uint64_t seed, uint64_t tensor_id, int64_t n, double lo, double hi, int dtype, void* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) store(out, i, dtype, lo + (hi - lo) * unif(mix(seed, tensor_id, (uint64_t)i)));
}

void gen_normal(uint64_t seed, uint64_t tensor_id, int64_t n, double mean, double std, int dtype, void* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    double u1 = unif(mix(seed, tensor_id, (uint64_t)i));
    double u2 = unif(mix(seed, tensor_id, (uint64_t)i + (1ull << 62)));
    double z = sqrt(-2.0 * log(1.0 - u1)) * cos(6.28318530717958647692 * u2);
    store(out, i, dtype, mean + std * z);
  }
}

void gen_integer(uint64_t seed, uint64_t tensor_id, int64_t n, int64_t lo, int64_t hi, int dtype, void* out) {
  uint64_t span = (uint64_t)(hi - lo + 1);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) store(out, i, dtype, (double)(lo + (int64_t)(mix(seed, tensor_id, (uint64_t)i) % span)));
}

/* Bit-pattern helpers for tests that build inputs by hand. */
void gen_encode(const float* in, int64_t n, int dtype, void* out) {
  for (int64_t i = 0; i < n; ++i) store(out, i, dtype, (double)in[i]);
}

uint64_t gen_hash(uint64_t seed, uint64_t tensor_id, uint64_t c) { return mix(seed, tensor_id, c); }
