// syr / syr2: symmetric rank-1 and rank-2 updates of the stored triangle (Section 6.2.2:
// "symmetric rank-1 update" and "symmetric rank-2 update" are among the level-2 kernels the
// paper's library covers).
//   syr  : A_ij <- alpha * x_i * x_j + A_ij
//   syr2 : A_ij <- alpha * (x_i * y_j + y_i * x_j) + A_ij        for (i, j) in the uplo triangle.
// Like ger this is a streaming read-modify-write of the matrix, 2s bytes per stored element;
// only the iteration space differs: tiles outside the triangle are skipped, tiles that the
// diagonal crosses are masked element by element, tiles inside take 128-bit packs.  Each lane
// keeps alpha * x_j (and alpha * y_j) for its columns in registers down a band of rows.
#include "common.cuh"

namespace b2 {

constexpr int kSyrCU = 2;    // packs per lane and row
constexpr int kSyrRows = 8;  // rows per warp and block

// Canonical row-major view: `lower` means the stored triangle has column <= row there.
template <typename T, int V, bool TWO>
__global__ void __launch_bounds__(kThreads) syr_kernel(T* __restrict__ a, int64_t lda, int64_t n,
                                                       const T* __restrict__ x, int64_t incx,
                                                       const T* __restrict__ y, int64_t incy, T alpha, bool lower,
                                                       int ntc) {
  constexpr int TC = 32 * V * kSyrCU;      // columns per block
  constexpr int RBLK = kWarps * kSyrRows;  // rows per block
  using P = Pack<T, V>;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t c0 = (int64_t)(blockIdx.x % ntc) * TC;
  const int64_t r0 = (int64_t)(blockIdx.x / ntc) * RBLK;
  // nothing of this tile inside the triangle?
  if (lower ? c0 > r0 + RBLK - 1 : c0 + TC - 1 < r0) return;
  const bool interior = lower ? c0 + TC - 1 <= r0 : c0 >= r0 + RBLK - 1;  // every element inside
  T xj[kSyrCU][V], yj[kSyrCU][V];
#pragma unroll
  for (int u = 0; u < kSyrCU; ++u)
#pragma unroll
    for (int e = 0; e < V; ++e) {
      const int64_t j = c0 + (u * 32 + lane) * V + e;
      xj[u][e] = j < n ? alpha * __ldg(x + j * incx) : T(0);
      yj[u][e] = (TWO && j < n) ? alpha * __ldg(y + j * incy) : T(0);
    }
#pragma unroll
  for (int ru = 0; ru < kSyrRows; ++ru) {
    const int64_t i = r0 + warp * kSyrRows + ru;
    if (i >= n) break;
    const T xi = __ldg(x + i * incx);
    const T yi = TWO ? __ldg(y + i * incy) : T(0);
#pragma unroll
    for (int u = 0; u < kSyrCU; ++u) {
      const int64_t cv = c0 + (u * 32 + lane) * V;
      T* ap = a + i * lda + cv;
      if (V > 1 && cv + V <= n && (interior || (lower ? cv + V - 1 <= i : cv >= i))) {
        P av = ld_cs<T, V>(ap);
#pragma unroll
        for (int e = 0; e < V; ++e) {
          // syr: alpha*x_i*x_j; syr2: x_i*(alpha*y_j) + y_i*(alpha*x_j)
          if (TWO) av.v[e] = yi * xj[u][e] + (xi * yj[u][e] + av.v[e]);
          else av.v[e] = xi * xj[u][e] + av.v[e];
        }
        st_cs<T, V>(ap, av);
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const int64_t j = cv + e;
          if (j < n && (lower ? j <= i : j >= i)) {
            if (TWO) ap[e] = yi * xj[u][e] + (xi * yj[u][e] + ap[e]);
            else ap[e] = xi * xj[u][e] + ap[e];
          }
        }
      }
    }
  }
}

template <typename T, int V, bool TWO>
static int syr_launch(const Launch& l, T* a, int64_t lda, int64_t n, const T* x, int64_t incx, const T* y,
                      int64_t incy, T alpha, bool lower) {
  constexpr int TC = 32 * V * kSyrCU;
  constexpr int RBLK = kWarps * kSyrRows;
  const int64_t ntc = (n + TC - 1) / TC, nrs = (n + RBLK - 1) / RBLK;
  if (ntc * nrs > 0x7fffffff) return B2_STATUS_NOT_IMPLEMENTED;
  syr_kernel<T, V, TWO><<<(unsigned)(ntc * nrs), kThreads, 0, l.stream>>>(a, lda, n, x, incx, y, incy, alpha, lower,
                                                                         (int)ntc);
  return check_launch();
}

template <typename T, bool TWO>
static int syr_impl(const b2_ctx* ctx, int order, int uplo, int64_t n, T alpha, const T* x, int64_t incx, const T* y,
                    int64_t incy, T* a, int64_t lda) {
  // argument positions after ctx: syr (order, uplo, n, alpha, x, incx, a, lda); syr2 adds (y, incy) after incx
  if (order != B2_ROW_MAJOR && order != B2_COL_MAJOR) return -1;
  if (uplo != B2_UPPER && uplo != B2_LOWER) return -2;
  if (n < 0) return -3;
  if (incx == 0) return -6;
  if (n > 0 && (x == nullptr || !aligned_to(x, sizeof(T)))) return -5;
  if (TWO) {
    if (incy == 0) return -8;
    if (n > 0 && (y == nullptr || !aligned_to(y, sizeof(T)))) return -7;
  }
  if (n > 0 && (a == nullptr || !aligned_to(a, sizeof(T)))) return TWO ? -9 : -7;
  if (lda < (n > 1 ? n : 1)) return TWO ? -10 : -8;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (n == 0 || alpha == T(0)) return B2_STATUS_OK;
  // canonical row-major view: a column-major upper triangle is a row-major lower one; the
  // update itself is symmetric in (i, j), so nothing else changes
  const bool lower = (uplo == B2_LOWER) == (order == B2_ROW_MAJOR);
  const T* xb = vec_base(x, n, incx);
  const T* yb = TWO ? vec_base(y, n, incy) : xb;
  constexpr int V = VecLen<T>::value;
  if (aligned_to(a, 16) && lda % V == 0) return syr_launch<T, V, TWO>(l, a, lda, n, xb, incx, yb, incy, alpha, lower);
  return syr_launch<T, 1, TWO>(l, a, lda, n, xb, incx, yb, incy, alpha, lower);
}

}  // namespace b2

extern "C" {
int b2_ssyr(const b2_ctx* ctx, int order, int uplo, int64_t n, float alpha, const float* x, int64_t incx, float* a,
            int64_t lda) {
  return b2::syr_impl<float, false>(ctx, order, uplo, n, alpha, x, incx, nullptr, 1, a, lda);
}
int b2_dsyr(const b2_ctx* ctx, int order, int uplo, int64_t n, double alpha, const double* x, int64_t incx, double* a,
            int64_t lda) {
  return b2::syr_impl<double, false>(ctx, order, uplo, n, alpha, x, incx, nullptr, 1, a, lda);
}
int b2_ssyr2(const b2_ctx* ctx, int order, int uplo, int64_t n, float alpha, const float* x, int64_t incx,
             const float* y, int64_t incy, float* a, int64_t lda) {
  return b2::syr_impl<float, true>(ctx, order, uplo, n, alpha, x, incx, y, incy, a, lda);
}
int b2_dsyr2(const b2_ctx* ctx, int order, int uplo, int64_t n, double alpha, const double* x, int64_t incx,
             const double* y, int64_t incy, double* a, int64_t lda) {
  return b2::syr_impl<double, true>(ctx, order, uplo, n, alpha, x, incx, y, incy, a, lda);
}
}
