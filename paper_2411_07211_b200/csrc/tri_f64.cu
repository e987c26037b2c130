// double instantiations of symv / trmv.
#include "tri_impl.cuh"
extern "C" {
int b2_dsymv(const b2_ctx* ctx, int order, int uplo, int64_t n, double alpha, const double* a, int64_t lda,
             const double* x, int64_t incx, double beta, double* y, int64_t incy) {
  return b2::symv_impl<double>(ctx, order, uplo, n, alpha, a, lda, x, incx, beta, y, incy);
}
int b2_dtrmv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const double* a, int64_t lda,
             double* x, int64_t incx) {
  return b2::trmv_impl<double>(ctx, order, uplo, trans, diag, n, a, lda, x, incx);
}
}
