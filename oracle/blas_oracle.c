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

/* Size of the wide accumulator type of the d routines, so callers can size scratch_w. */
int oracle_wide_bytes(void) { return (int)sizeof(long double); }
