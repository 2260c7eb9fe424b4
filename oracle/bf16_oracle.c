/*
 * bfloat16 storage for the ApproxIFER oracle  --  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * The paper (arXiv 2109.09868) does not fix the precision in which queries and predictions are stored.  For the
 * library's bfloat16 payload variants the reading taken is: a stored bfloat16 value IS the real number it
 * denotes (widening is exact), the encoder / decoder formulas of Section 3 are evaluated on those numbers in
 * fp64 exactly as for fp32 payloads (approxifer_oracle.c, untouched), and the result is rounded ONCE to the
 * nearest bfloat16, ties to even.  This file holds only the two conversions; the formulas stay where they are.
 *
 * bfloat16 = 1 sign bit, 8 exponent bits (bias 127), 7 fraction bits: the upper half of an IEEE-754 binary32.
 * The conversions below are written from that definition with integer and exactly-representable fp64
 * arithmetic; they use no float-to-bfloat16 routine of any library.
 *
 * Pins (tests/test_oracle_bf16_pins.py): hand-written bit patterns (ties to even in both directions, the
 * smallest subnormal and half of it, the largest finite value and the overflow threshold, signed zeros,
 * infinities, NaN); round trip over all 65,536 bit patterns; every midpoint between neighbouring bfloat16
 * values, built exactly in fp64, goes to the neighbour with the even fraction; monotonicity.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

/* The real number a bfloat16 bit pattern denotes (NaN patterns give a NaN). */
double oracle_bf16_to_double(uint16_t b) {
  const int sign = (b >> 15) & 1;
  const int e = (b >> 7) & 0xff;
  const int f = b & 0x7f;
  double v;
  if (e == 0xff) {
    v = f ? NAN : INFINITY;
  } else if (e == 0) {
    v = ldexp((double)f, -126 - 7); /* subnormal: f * 2^-133 */
  } else {
    v = ldexp((double)(128 + f), e - 127 - 7); /* (1 + f/128) * 2^(e-127) */
  }
  return sign ? -v : v;
}

/* Nearest bfloat16 to x, ties to the even fraction; overflow to infinity; NaN to the quiet NaN 0x7fc0 with x's sign. */
uint16_t oracle_double_to_bf16(double x) {
  const uint16_t sign = signbit(x) ? 0x8000u : 0u;
  if (isnan(x)) return (uint16_t)(sign | 0x7fc0u);
  double a = fabs(x);
  if (isinf(a)) return (uint16_t)(sign | 0x7f80u);
  if (a == 0.0) return sign;
  int e2;
  (void)frexp(a, &e2); /* a = m * 2^e2, 0.5 <= m < 1  =>  floor(log2 a) = e2 - 1 */
  int e = e2 - 1;
  if (e < -126) e = -126; /* subnormal range: fixed quantum 2^-133 */
  /* q = a / 2^(e-7) is exact in fp64 (a power-of-two scaling of a 53-bit number); 128 <= q < 256 for normal a */
  const double q = ldexp(a, 7 - e);
  double r = floor(q);
  const double frac = q - r; /* exact */
  if (frac > 0.5 || (frac == 0.5 && fmod(r, 2.0) == 1.0)) r += 1.0;
  /* r in [0, 256]; r = 256 means the next binade (or, from the subnormal range, the smallest normal) */
  int64_t ri = (int64_t)r;
  int be; /* biased exponent */
  if (e == -126 && ri < 128) {
    be = 0; /* stays subnormal: fraction field = ri */
    return (uint16_t)(sign | (uint16_t)ri);
  }
  if (ri == 256) {
    ri = 128;
    e += 1;
  }
  be = e + 127;
  if (be >= 0xff) return (uint16_t)(sign | 0x7f80u); /* rounds beyond the largest finite value */
  return (uint16_t)(sign | (uint16_t)(be << 7) | (uint16_t)(ri - 128));
}

void oracle_bf16_widen(int64_t n, const uint16_t *in, float *out) {
  for (int64_t i = 0; i < n; ++i) out[i] = (float)oracle_bf16_to_double(in[i]); /* exact: every bfloat16 is a binary32 */
}

void oracle_bf16_round(int64_t n, const double *in, uint16_t *out) {
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_double_to_bf16(in[i]);
}
