/*
 * CPU oracle for the dense BLAS level-1 / level-2 family -- TEST INFRASTRUCTURE ONLY.
 * Not part of the product: only the test-suite, the smoke check and the bench's CPU-baseline
 * leg may build or call it.  It shares no code with the CUDA library.
 *
 * Instantiates blas_oracle_impl.h for the two precisions of Section 6.2.2 ("float (s),
 * double (d)").  Sums are accumulated in double for the s routines and in long double for
 * the d routines, then rounded once.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC blas_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>

#define T float
#define W double
#define P s
#define WSQRT sqrt
#include "blas_oracle_impl.h"
#undef T
#undef W
#undef P
#undef WSQRT

#define T double
#define W long double
#define P d
#define WSQRT sqrtl
#include "blas_oracle_impl.h"
#undef T
#undef W
#undef P
#undef WSQRT

/* dsdot (in the paper's level-1 set, Section 6.2.1): the dot product of two float vectors with
 * every product and the sum taken in extended precision: sum_i (wide)x_i * (wide)y_i.  A product of
 * two floats is exact in double already; the sum runs in long double and is rounded to double
 * once.  absterms = sum_i |x_i y_i|. */
static int64_t ds_vidx(int64_t i, int64_t n, int64_t inc) { return inc > 0 ? i * inc : (i - (n - 1)) * inc; }

void oracle_dsdot(int64_t n, const float* x, int64_t incx, const float* y, int64_t incy, double* result,
                  double* absterms) {
  long double acc = 0, aabs = 0;
  for (int64_t i = 0; i < n; ++i) {
    long double p = (long double)x[ds_vidx(i, n, incx)] * (long double)y[ds_vidx(i, n, incy)];
    acc += p;
    aabs += p < 0 ? -p : p;
  }
  *result = (double)acc;
  if (absterms) *absterms = (double)aabs;
}

/* sdsdot: sb + the same extended-precision sum, rounded to float once at the end.
 * absterms = |sb| + sum_i |x_i y_i|. */
void oracle_sdsdot(int64_t n, float sb, const float* x, int64_t incx, const float* y, int64_t incy, float* result,
                   double* absterms) {
  long double acc = (long double)sb, aabs = sb < 0 ? -(long double)sb : (long double)sb;
  for (int64_t i = 0; i < n; ++i) {
    long double p = (long double)x[ds_vidx(i, n, incx)] * (long double)y[ds_vidx(i, n, incy)];
    acc += p;
    aabs += p < 0 ? -p : p;
  }
  *result = (float)acc;
  if (absterms) *absterms = (double)aabs;
}

/* Size of the wide accumulator type of the d routines, so callers can size scratch_w. */
int oracle_wide_bytes(void) { return (int)sizeof(long double); }
