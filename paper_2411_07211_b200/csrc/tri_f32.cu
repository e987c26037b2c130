// float instantiations of symv / trmv.
#include "tri_impl.cuh"
extern "C" {
int b2_ssymv(const b2_ctx* ctx, int order, int uplo, int64_t n, float alpha, const float* a, int64_t lda,
             const float* x, int64_t incx, float beta, float* y, int64_t incy) {
  return b2::symv_impl<float>(ctx, order, uplo, n, alpha, a, lda, x, incx, beta, y, incy);
}
int b2_strmv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const float* a, int64_t lda,
             float* x, int64_t incx) {
  return b2::trmv_impl<float>(ctx, order, uplo, trans, diag, n, a, lda, x, incx);
}
}
