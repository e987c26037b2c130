// gemv entry points: y <- alpha*op(A)*x + beta*y (Section 2 inset and Figure 7 of the paper).
// Row-major N is the row-dot kind, row-major T the column-sum kind; a column-major call is
// the transposed row-major problem (A^T stored row-major), so N and T swap kinds.
#include "level2.cuh"
#include "skinny.cuh"

namespace b2 {

using GemvRow = Kind<true, false, TRI_FULL, false, false>;
using GemvCol = Kind<false, true, TRI_FULL, false, false>;

template <typename T>
static int gemv_impl(const b2_ctx* ctx, int order, int trans, int64_t m, int64_t n, T alpha, const T* a, int64_t lda,
                     const T* x, int64_t incx, T beta, T* y, int64_t incy) {
  if (order != B2_ROW_MAJOR && order != B2_COL_MAJOR) return -1;
  if (trans != B2_NO_TRANS && trans != B2_TRANS) return -2;
  if (m < 0) return -3;
  if (n < 0) return -4;
  const int64_t minor = order == B2_ROW_MAJOR ? n : m;
  if (m > 0 && n > 0 && (a == nullptr || !aligned_to(a, sizeof(T)))) return -6;
  if (lda < (minor > 1 ? minor : 1)) return -7;
  const int64_t lenx = trans == B2_NO_TRANS ? n : m, leny = trans == B2_NO_TRANS ? m : n;
  if (incx == 0) return -9;
  if (lenx > 0 && leny > 0 && (x == nullptr || !aligned_to(x, sizeof(T)))) return -8;
  if (incy == 0) return -12;
  if (leny > 0 && (y == nullptr || !aligned_to(y, sizeof(T)))) return -11;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (m == 0 || n == 0) return B2_STATUS_OK;
  B2_DBG_RANGE(l, a, (size_t)(((order == B2_ROW_MAJOR ? m : n) - 1) * lda + minor) * sizeof(T));
  B2_DBG_VEC(l, x, lenx, incx);
  B2_DBG_VEC(l, y, leny, incy);
  B2_DBG_COMMIT(l);
  if (alpha == T(0)) return scale_y<T>(l, y, incy, leny, beta);

  L2Args<T> args = {};
  args.a = a;
  args.lda = lda;
  args.rows = order == B2_ROW_MAJOR ? m : n;  // canonical row-major view
  args.cols = order == B2_ROW_MAJOR ? n : m;
  args.alpha = alpha;
  args.beta = beta;
  args.y = vec_base(y, leny, incy);
  args.incy = incy;
  const bool rowdot = (order == B2_ROW_MAJOR) == (trans == B2_NO_TRANS);
  if (rowdot) {
    args.xc = vec_base(x, lenx, incx);
    args.incxc = incx;
    if (knob(kKnobNarrowBlock) && block_narrow_applies(a, lda, args.rows, args.cols))
      return block_rowdot<T>(l, a, args.rows, args.cols, args.xc, incx, alpha, beta, args.y, incy);
    if (skinny_applies(a, lda, args.rows, args.cols, true))
      return skinny_rowdot<T>(l, a, args.rows, args.cols, args.xc, incx, alpha, beta, args.y, incy);
    return l2_dispatch<T, GemvRow, true>(l, args, plan_rowout(args, true), true);
  }
  args.xr = vec_base(x, lenx, incx);
  args.incxr = incx;
  if (knob(kKnobNarrowBlock) && wide_applies<T>(args.rows, args.cols)) {
    const int64_t want = (args.cols + kThreads - 1) / kThreads, cap = (int64_t)sm_count() * 8;
    launch_chained(wide_colsum_kernel<T>, dim3((unsigned)(want < cap ? want : cap)), dim3(kThreads), 0, l.stream, a, lda, (int)args.rows, args.cols, args.xr,
                                                                                   incx, alpha, beta, args.y, incy);
    return check_launch();
  }
  if (knob(kKnobNarrowBlock) && block_narrow_applies(a, lda, args.rows, args.cols)) {
    const int ppr = (int)(args.cols / VecLen<T>::value), K = kThreads / ppr;
    const int64_t nsteps = (args.rows + (int64_t)K * kBlockUnroll - 1) / ((int64_t)K * kBlockUnroll);
    const int64_t cap = (int64_t)sm_count() * 4;
    const int grid = (int)(nsteps < cap ? nsteps : cap);
    if ((size_t)grid * args.cols * sizeof(T) <= l.scratch_bytes) {
      args.colpart = reinterpret_cast<T*>(l.scratch);
      args.nrs = grid;  // one partial row per block; the finalize kernel adds all of them
      args.ncs = 1;
      args.nct = 1;
      args.ctiles_per_cta = 1;
      args.rows_per_cta = args.rows;
      args.direct = 0;
      launch_chained(block_colsum_kernel<T>, dim3(grid), dim3(kThreads), 0, l.stream, a, args.rows, ppr, args.xr, incx, args.colpart, nsteps);
      if (int st = check_launch()) return st;
      launch_finalize<T, GemvCol, 32>(l, args, 1, (int)args.cols, args.cols);
      return check_launch();
    }
  }
  if (skinny_colsum_applies(a, lda, args.rows, args.cols)) {
    const int ppr = (int)(args.cols / VecLen<T>::value);
    const int64_t rows_per_step = (int64_t)(32 / ppr) * kColsumGroup;
    const int64_t nsteps = (args.rows + rows_per_step - 1) / rows_per_step;
    const int64_t want = (nsteps + kWarps - 1) / kWarps, cap = (int64_t)sm_count() * 4;
    const int grid = (int)(want < cap ? want : cap);
    if ((size_t)grid * args.cols * sizeof(T) <= l.scratch_bytes) {
      args.colpart = reinterpret_cast<T*>(l.scratch);
      args.nrs = grid;  // one partial row per block; the finalize kernel adds all of them
      args.ncs = 1;
      args.nct = 1;
      args.ctiles_per_cta = 1;
      args.rows_per_cta = args.rows;
      args.direct = 0;
      launch_chained(skinny_colsum_kernel<T>, dim3(grid), dim3(kThreads), 0, l.stream, a, args.rows, ppr, args.xr, incx, args.colpart, nsteps);
      if (int st = check_launch()) return st;
      launch_finalize<T, GemvCol, 32>(l, args, 1, (int)args.cols, args.cols);
      return check_launch();
    }
  }
  return l2_dispatch<T, GemvCol, true>(l, args, plan_colout(args, true, knob(kKnobGemvTRows)), true);
}

}  // namespace b2

extern "C" {
int b2_sgemv(const b2_ctx* ctx, int order, int trans, int64_t m, int64_t n, float alpha, const float* a, int64_t lda,
             const float* x, int64_t incx, float beta, float* y, int64_t incy) {
  return b2::gemv_impl<float>(ctx, order, trans, m, n, alpha, a, lda, x, incx, beta, y, incy);
}
int b2_dgemv(const b2_ctx* ctx, int order, int trans, int64_t m, int64_t n, double alpha, const double* a, int64_t lda,
             const double* x, int64_t incx, double beta, double* y, int64_t incy) {
  return b2::gemv_impl<double>(ctx, order, trans, m, n, alpha, a, lda, x, incx, beta, y, incy);
}
}
