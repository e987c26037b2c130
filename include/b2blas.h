/*
 * b2blas -- dense BLAS level-1 / level-2 routines as hand-written sm_100a CUDA kernels.
 *
 * The routine family is the one the paper's linear-algebra scheduling library produces
 * (Section 6.2: "most of the kernels in BLAS levels 1 and 2"): level 1 in Section 6.2.1
 * (asum, axpy, dot, rot, scal, swap, copy; nrm2 and iamax are named there as the two the
 * paper could not express), level 2 in Section 6.2.2 (gemv, ger, symv, trmv, trsv; options
 * s/d, transpose t/n, lower/upper, unit/non-unit) and Figure 9b ("stride-1 and stride-any").
 * Calls follow the BLAS problem statement.
 *
 * General rules for every entry point
 *   - Prefix s = float, d = double.  All vector / matrix / result pointers are DEVICE
 *     pointers owned by the caller; scalars (alpha, beta, c, s) are passed by value from the
 *     host.  The library allocates no device memory and keeps no state between calls.
 *   - Calls are asynchronous on ctx->stream; outputs are valid once the stream has been
 *     synchronised.  Two calls that share one workspace must be ordered on one stream.
 *   - Vectors: logical element i of a vector with increment inc is at v[i*inc] for inc > 0
 *     and at v[(i-(n-1))*inc] for inc < 0.  inc == 0 is an error.  Input and output vectors
 *     must not overlap (except where the routine is in place by definition).
 *   - Matrices: order B2_ROW_MAJOR: A(i,j) = a[i*lda + j], lda >= max(1, #columns);
 *     order B2_COL_MAJOR: A(i,j) = a[j*lda + i], lda >= max(1, #rows).
 *   - Return value: 0 on success; -k when argument number k is invalid (1-based, not
 *     counting ctx; nothing is launched); a positive B2_STATUS_* code otherwise.
 *   - n == 0 (or m == 0 or n == 0 for matrices) is a successful no-op; reductions then
 *     write 0 to *result.
 */
#ifndef B2BLAS_H
#define B2BLAS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  B2_ROW_MAJOR = 101, B2_COL_MAJOR = 102,
  B2_NO_TRANS = 111, B2_TRANS = 112,
  B2_UPPER = 121, B2_LOWER = 122,
  B2_NON_UNIT = 131, B2_UNIT = 132
};

enum {
  B2_STATUS_OK = 0,
  B2_STATUS_LAUNCH_FAILED = 1,       /* a CUDA launch or memset was rejected (error consumed)   */
  B2_STATUS_WORKSPACE_TOO_SMALL = 2, /* ctx->workspace_bytes below what this call needs          */
  B2_STATUS_NOT_IMPLEMENTED = 3,
  B2_STATUS_TIMEOUT = 4,             /* only ever written to *ctx->device_status (bounded waits) */
  B2_STATUS_BAD_CONTEXT = 5,         /* ctx NULL, workspace NULL / misaligned                    */
  B2_STATUS_TOO_LARGE = 6            /* problem size above the fixed limit of a *_noalloc call   */
};

/*
 * Per-call context, filled by the caller.
 *   stream          cudaStream_t to launch on (NULL = legacy default stream).
 *   workspace       device memory, 256-byte aligned, at least b2_workspace_min_bytes() bytes.
 *                   Its first 4096 bytes are a control block that must be zero before the
 *                   first call (b2_workspace_reset does that); every call that completes
 *                   leaves it zero again.  The rest holds per-call partial results.
 *   workspace_bytes size of that memory.  Larger workspaces allow finer work splitting for
 *                   level-2 calls; b2_workspace_bytes() is a comfortable default.
 *   device_status   optional device int.  trsv writes B2_STATUS_TIMEOUT there if a bounded
 *                   wait on another thread block ran out (the call's output is then invalid).
 *                   Never written otherwise; the caller zeroes it.  A timed-out call leaves
 *                   the control block dirty: call b2_workspace_reset before the workspace is
 *                   used again.  A trsv call that finds the control block dirty solves
 *                   nothing and writes B2_STATUS_TIMEOUT again.  (symv / trmv write the same
 *                   value only with the optional TMA tile delivery switched on, if a wait
 *                   for a copy into shared memory ran out; they keep no state.)
 *   wait_limit      polling iterations before a trsv wait gives up; 0 = library default.
 */
typedef struct b2_ctx {
  void* stream;
  void* workspace;
  size_t workspace_bytes;
  int* device_status;
  unsigned long long wait_limit;
} b2_ctx;

size_t b2_workspace_min_bytes(void); /* control block + level-1 partials                   */
/* Recommended size (256 MiB): a default, not a bound.  It serves every call on matrices up to
 * 32768 x 32768 and vectors of any length without B2_STATUS_WORKSPACE_TOO_SMALL; the exact
 * need of one call is b2_workspace_query's. */
size_t b2_workspace_bytes(void);
/* Smallest workspace size with which no routine of this library returns
 * B2_STATUS_WORKSPACE_TOO_SMALL on an m x n matrix (vectors of max(m, n) elements; level-1
 * calls: pass m = n = 1) of elem_bytes-sized elements (4 or 8).  Larger workspaces only allow
 * finer work splitting.  Returns 0 for a negative size or another element size. */
size_t b2_workspace_query(int64_t m, int64_t n, size_t elem_bytes);
int b2_workspace_reset(const b2_ctx* ctx); /* async memset of the control block to zero     */
const char* b2_status_string(int status);
int b2_version(void);
/* Number of kernels this library has launched in this process so far (not thread-safe). */
unsigned long long b2_launch_count(void);

/* Bounds-checking build of the library (compiled with -DB2_DEBUG_BOUNDS into a separate file; no
 * counterpart in the paper: it stands in for a memory checker).  In that build every kernel
 * tests the addresses it touches against the extents of the call's arguments; an access
 * outside them is skipped and counted, nothing traps.  b2_debug_bounds_report synchronises the
 * device and writes {violations since the last report, first offending address, its size in
 * bytes} to out3 (host memory).  b2_debug_bounds_shrink(bytes) is the checker's own test hook:
 * it cuts `bytes` off the end of every extent, so that accesses which are in fact in bounds are
 * reported.  Both return B2_STATUS_NOT_IMPLEMENTED in the ordinary build.  Not thread-safe. */
int b2_debug_bounds_report(unsigned long long* out3);
int b2_debug_bounds_shrink(int bytes);

/* Tuning hooks (process-wide, not thread-safe): work-splitting parameters of the kernels,
 * indexed by the Knob enumeration of the sources.  Defaults are the tuned values; changing
 * them never changes what a routine computes, only how the work is cut.
 * b2_set_tuning returns 0, or -1 for an unknown knob. */
int b2_set_tuning(int knob, int64_t value);
int64_t b2_get_tuning(int knob);

/* ---- level 1 (Section 6.2.1) ------------------------------------------------------------ */

/* axpy (Figure 4a): y_i <- alpha*x_i + y_i.  alpha == 0 returns without touching y. */
int b2_saxpy(const b2_ctx* ctx, int64_t n, float alpha, const float* x, int64_t incx, float* y, int64_t incy);
int b2_daxpy(const b2_ctx* ctx, int64_t n, double alpha, const double* x, int64_t incx, double* y, int64_t incy);

/* scal: x_i <- alpha*x_i, one IEEE multiply per element (bit-exact against any plain loop). */
int b2_sscal(const b2_ctx* ctx, int64_t n, float alpha, float* x, int64_t incx);
int b2_dscal(const b2_ctx* ctx, int64_t n, double alpha, double* x, int64_t incx);

/* copy: y_i <- x_i. */
int b2_scopy(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, float* y, int64_t incy);
int b2_dcopy(const b2_ctx* ctx, int64_t n, const double* x, int64_t incx, double* y, int64_t incy);

/* swap: x_i <-> y_i. */
int b2_sswap(const b2_ctx* ctx, int64_t n, float* x, int64_t incx, float* y, int64_t incy);
int b2_dswap(const b2_ctx* ctx, int64_t n, double* x, int64_t incx, double* y, int64_t incy);

/* rot: (x_i, y_i) <- (c*x_i + s*y_i, c*y_i - s*x_i). */
int b2_srot(const b2_ctx* ctx, int64_t n, float* x, int64_t incx, float* y, int64_t incy, float c, float s);
int b2_drot(const b2_ctx* ctx, int64_t n, double* x, int64_t incx, double* y, int64_t incy, double c, double s);

/* rotm (Section 6.2.1 lists rotm among the level-1 kernels; the definition is the BLAS one):
 * the modified Givens rotation (x_i, y_i) <- (h11*x_i + h12*y_i, h21*x_i + h22*y_i).
 *   param   HOST pointer to 5 values {flag, h11, h21, h12, h22}; it is read before the call
 *           returns.  flag -1: all four entries from param; flag 0: h11 = h22 = 1 implied
 *           (param[1], param[4] not read); flag 1: h12 = 1, h21 = -1 implied (param[2],
 *           param[3] not read); flag -2: H = I, nothing is launched.
 * Errors: -1 n, -2 x, -3 incx, -4 y, -5 incy, -6 param (NULL or a flag outside {-2,-1,0,1}). */
int b2_srotm(const b2_ctx* ctx, int64_t n, float* x, int64_t incx, float* y, int64_t incy, const float* param);
int b2_drotm(const b2_ctx* ctx, int64_t n, double* x, int64_t incx, double* y, int64_t incy, const double* param);

/* dot: *result <- sum_i x_i*y_i.  Reductions are deterministic: same inputs, same bits. */
int b2_sdot(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, const float* y, int64_t incy, float* result);
int b2_ddot(const b2_ctx* ctx, int64_t n, const double* x, int64_t incx, const double* y, int64_t incy, double* result);

/* dsdot (Section 6.2.1 lists dsdot among the level-1 kernels): float vectors, every product and
 * the sum in double: *result <- sum_i (double)x_i * (double)y_i, a DEVICE double.
 * sdsdot: *result <- (float)(sb + that double sum), a DEVICE float, rounded once; it keeps the
 * double sum in ctx->workspace behind the block partials and runs one extra one-thread kernel.
 * Errors: dsdot as b2_sdot; sdsdot -1 n, -3 x, -4 incx, -5 y, -6 incy, -7 result. */
int b2_dsdot(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, const float* y, int64_t incy, double* result);
int b2_sdsdot(const b2_ctx* ctx, int64_t n, float sb, const float* x, int64_t incx, const float* y, int64_t incy,
              float* result);

/* sdot without any caller-provided or allocated scratch (the paper has no counterpart: this
 * entry point exists for deployment reasons only).  Same result contract as b2_sdot, but no
 * b2_ctx: the per-block partial sums and the ticket word sit in a fixed array inside the
 * library's device image (4352 bytes; every GPU that loads the library carries it until the
 * process exits).  It is meant for callers that cannot obtain device memory at the point of
 * the call -- a plug-in running inside a host application whose allocator owns the whole GPU
 * heap, a control loop whose rules forbid allocation after start-up because cudaMalloc may
 * block and synchronise the device, a code path that runs after an out-of-memory condition.
 * The entry point calls no cudaMalloc / cudaFree and no allocating library routine.
 *   stream   cudaStream_t to launch on (NULL = legacy default stream).
 *   n        0 <= n <= 2^30; larger n returns B2_STATUS_TOO_LARGE and launches nothing.
 *   others   as b2_sdot (device pointers, non-zero increments).
 * The first call on each device looks up the device address of the array; make that first
 * call outside any stream capture.  All calls share the one array: it still holds the last
 * call's partials, the ticket word is cleared by every call before its kernel, and two calls
 * that may overlap on the GPU (different streams, no ordering) race on it -- serialise them. */
int b2_sdot_noalloc(void* stream, int64_t n, const float* x, int64_t incx, const float* y, int64_t incy,
                    float* result);

/* asum: *result <- sum_i |x_i|. */
int b2_sasum(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, float* result);
int b2_dasum(const b2_ctx* ctx, int64_t n, const double* x, int64_t incx, double* result);

/* nrm2: *result <- sqrt(sum_i x_i^2), plain sum of squares (no overflow rescaling). */
int b2_snrm2(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, float* result);
int b2_dnrm2(const b2_ctx* ctx, int64_t n, const double* x, int64_t incx, double* result);

/* iamax: *result <- smallest 0-based i with |x_i| = max_k |x_k| (0 when n == 0). */
int b2_isamax(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, int64_t* result);
int b2_idamax(const b2_ctx* ctx, int64_t n, const double* x, int64_t incx, int64_t* result);

/* ---- level 2 (Section 6.2.2) ------------------------------------------------------------ */

/* gemv (Section 2 inset, Figure 7a / 7c): y <- alpha*op(A)*x + beta*y, A is m x n.
 * trans = B2_NO_TRANS: x has n elements, y has m; B2_TRANS: x has m, y has n.
 * beta == 0: y is written without being read. */
int b2_sgemv(const b2_ctx* ctx, int order, int trans, int64_t m, int64_t n, float alpha, const float* a, int64_t lda,
             const float* x, int64_t incx, float beta, float* y, int64_t incy);
int b2_dgemv(const b2_ctx* ctx, int order, int trans, int64_t m, int64_t n, double alpha, const double* a, int64_t lda,
             const double* x, int64_t incx, double beta, double* y, int64_t incy);

/* ger: A <- alpha*x*y^T + A, A is m x n, x has m elements, y has n.  alpha == 0: no-op. */
int b2_sger(const b2_ctx* ctx, int order, int64_t m, int64_t n, float alpha, const float* x, int64_t incx,
            const float* y, int64_t incy, float* a, int64_t lda);
int b2_dger(const b2_ctx* ctx, int order, int64_t m, int64_t n, double alpha, const double* x, int64_t incx,
            const double* y, int64_t incy, double* a, int64_t lda);

/* syr (Section 6.2.2, "symmetric rank-1 update"): A <- alpha*x*x^T + A on the uplo triangle
 * (with the diagonal) of the symmetric n x n matrix A; the other triangle is neither read nor
 * written.  alpha == 0: no-op.  Elementwise two-term sums: same tolerance class as ger. */
int b2_ssyr(const b2_ctx* ctx, int order, int uplo, int64_t n, float alpha, const float* x, int64_t incx, float* a,
            int64_t lda);
int b2_dsyr(const b2_ctx* ctx, int order, int uplo, int64_t n, double alpha, const double* x, int64_t incx, double* a,
            int64_t lda);

/* syr2 (Section 6.2.2, "symmetric rank-2 update"): A <- alpha*(x*y^T + y*x^T) + A on the uplo
 * triangle; otherwise as syr. */
int b2_ssyr2(const b2_ctx* ctx, int order, int uplo, int64_t n, float alpha, const float* x, int64_t incx,
             const float* y, int64_t incy, float* a, int64_t lda);
int b2_dsyr2(const b2_ctx* ctx, int order, int uplo, int64_t n, double alpha, const double* x, int64_t incx,
             const double* y, int64_t incy, double* a, int64_t lda);

/* symv: y <- alpha*A*x + beta*y, A symmetric n x n; only the uplo triangle (with the
 * diagonal) is referenced, the other triangle is never used. */
int b2_ssymv(const b2_ctx* ctx, int order, int uplo, int64_t n, float alpha, const float* a, int64_t lda,
             const float* x, int64_t incx, float beta, float* y, int64_t incy);
int b2_dsymv(const b2_ctx* ctx, int order, int uplo, int64_t n, double alpha, const double* a, int64_t lda,
             const double* x, int64_t incx, double beta, double* y, int64_t incy);

/* trmv: x <- op(A)*x in place, A triangular (uplo), diag = B2_UNIT: the diagonal is taken
 * as 1 and not referenced.  The other triangle is never used. */
int b2_strmv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const float* a, int64_t lda,
             float* x, int64_t incx);
int b2_dtrmv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const double* a, int64_t lda,
             double* x, int64_t incx);

/* trsv: solve op(A)*x = b in place (b passed in x), same options as trmv.  Blocked
 * substitution; thread blocks wait (bounded, see b2_ctx) on the blocks they depend on. */
int b2_strsv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const float* a, int64_t lda,
             float* x, int64_t incx);
int b2_dtrsv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const double* a, int64_t lda,
             double* x, int64_t incx);

#ifdef __cplusplus
}
#endif
#endif /* B2BLAS_H */
