// symv and trmv entry-point bodies (Section 6.2.2, "Triangular Matrix"): both run on the
// level-2 tile kernel restricted to one triangle of the canonical row-major view.
//   symv : row sums over the stored triangle (with the diagonal) plus column sums over its
//          strictly off-diagonal part -- each stored element is loaded once and used twice.
//   trmv : row sums (op(A) rows contiguous) or column sums (op(A) rows strided), the
//          diagonal replaced by 1 for diag = unit.  The result goes to partials first and is
//          written over x by the finalize kernel, after every block has finished reading x.
#pragma once
#include "level2.cuh"
#include "tri_tile.cuh"

namespace b2 {

template <typename T>
static int check_square(int order, int64_t n, const T* a, int64_t lda, int arg_order, int arg_n, int arg_a,
                        int arg_lda) {
  if (order != B2_ROW_MAJOR && order != B2_COL_MAJOR) return -arg_order;
  if (n < 0) return -arg_n;
  if (n > 0 && (a == nullptr || !aligned_to(a, sizeof(T)))) return -arg_a;
  if (lda < (n > 1 ? n : 1)) return -arg_lda;
  return 0;
}

template <typename T>
static L2Plan plan_tri(const L2Args<T>& a) {
  const int V = (aligned_to(a.a, 16) && a.lda % VecLen<T>::value == 0) ? VecLen<T>::value : 1;
  const int64_t nv = (a.cols + V - 1) / V;
  L2Plan p;
  p.shape = (nv >= 512 && knob(kKnobTriWide)) ? SHAPE_WIDE : SHAPE_MID;
  p.ctiles_per_cta = 1;
  p.rows_per_cta = knob(kKnobTriRows);
  return p;
}

template <typename T>
static int symv_impl(const b2_ctx* ctx, int order, int uplo, int64_t n, T alpha, const T* a, int64_t lda, const T* x,
                     int64_t incx, T beta, T* y, int64_t incy) {
  if (int e = check_square(order, n, a, lda, 1, 3, 5, 6)) return e;
  if (uplo != B2_UPPER && uplo != B2_LOWER) return -2;
  if (incx == 0) return -8;
  if (n > 0 && (x == nullptr || !aligned_to(x, sizeof(T)))) return -7;
  if (incy == 0) return -11;
  if (n > 0 && (y == nullptr || !aligned_to(y, sizeof(T)))) return -10;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (n == 0) return B2_STATUS_OK;
  B2_DBG_RANGE(l, a, (size_t)((n - 1) * lda + n) * sizeof(T));
  B2_DBG_VEC(l, x, n, incx);
  B2_DBG_VEC(l, y, n, incy);
  B2_DBG_COMMIT(l);
  if (alpha == T(0)) return scale_y<T>(l, y, incy, n, beta);
  L2Args<T> args = {};
  args.a = a;
  args.lda = lda;
  args.rows = args.cols = n;
  args.xc = args.xr = vec_base(x, n, incx);
  args.incxc = args.incxr = incx;
  args.alpha = alpha;
  args.beta = beta;
  args.y = vec_base(y, n, incy);
  args.incy = incy;
  // the stored triangle as it sits in the row-major view of the buffer
  const bool upper = (order == B2_ROW_MAJOR) == (uplo == B2_UPPER);
  // The tile kernel with the shared-memory ring (16-byte aligned matrices) is the faster one while
  // the triangle is small (n = 4096: 13 us against 19 us in float); from about 64 MiB of triangle
  // on the general tile kernel streams faster (n = 32768 float: 320 us against 357 us).  Knob value
  // 2 forces the ring kernel at every size (tests).
  // (double, upper triangle: that kind of the general kernel spills 132 bytes per thread at its
  // 64 registers and streams 10-15 % slower than the ring kernel at every size -- n = 32768:
  // 780 us against 684 us)
  const bool small = (double)n * (double)n * sizeof(T) / 2 <= 64.0 * 1024 * 1024;
  if (knob(kKnobTriTile) == 2 || (knob(kKnobTriTile) == 1 && (small || (sizeof(T) == 8 && upper)))) {
    bool handled = false;
    const int st = upper ? tt::tri_tile_run<T, true, true, TRI_UPPER, false, true>(l, a, lda, n, args.xc, incx, alpha, beta,
                                                                                  args.y, incy, &handled)
                         : tt::tri_tile_run<T, true, true, TRI_LOWER, false, true>(l, a, lda, n, args.xc, incx, alpha, beta,
                                                                                  args.y, incy, &handled);
    if (handled) return st;
  }
  const L2Plan plan = plan_tri(args);
  if (upper) return l2_dispatch<T, Kind<true, true, TRI_UPPER, false, true>, false>(l, args, plan, false);
  return l2_dispatch<T, Kind<true, true, TRI_LOWER, false, true>, false>(l, args, plan, false);
}

template <typename T, bool ROW, int TRI>
static int trmv_kind(const Launch& l, const L2Args<T>& args, bool unit) {
  // The tile kernel with the shared-memory ring serves trmv where it measured faster than the
  // general tile kernel: float row sums with a strided x (knob value 2: always, for the tests).
  const bool ring = knob(kKnobTriTile) == 2 || (knob(kKnobTriTile) == 1 && sizeof(T) == 4 && ROW && args.incxc != 1);
  if (ring) {
    bool handled = false;
    const int st =
        unit ? tt::tri_tile_run<T, ROW, !ROW, TRI, true, false>(l, args.a, args.lda, args.rows, args.xc, args.incxc, T(1), T(0),
                                                               args.y, args.incy, &handled)
             : tt::tri_tile_run<T, ROW, !ROW, TRI, false, false>(l, args.a, args.lda, args.rows, args.xc, args.incxc, T(1), T(0),
                                                                args.y, args.incy, &handled);
    if (handled) return st;
  }
  const L2Plan plan = ROW ? plan_rowout(args, false) : plan_colout(args, false, knob(kKnobTriRows));
  if (unit) return l2_dispatch<T, Kind<ROW, !ROW, TRI, true, false>, false>(l, args, plan, false);
  return l2_dispatch<T, Kind<ROW, !ROW, TRI, false, false>, false>(l, args, plan, false);
}

template <typename T>
static int trmv_impl(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const T* a, int64_t lda,
                     T* x, int64_t incx) {
  if (int e = check_square(order, n, a, lda, 1, 5, 6, 7)) return e;
  if (uplo != B2_UPPER && uplo != B2_LOWER) return -2;
  if (trans != B2_NO_TRANS && trans != B2_TRANS) return -3;
  if (diag != B2_NON_UNIT && diag != B2_UNIT) return -4;
  if (incx == 0) return -9;
  if (n > 0 && (x == nullptr || !aligned_to(x, sizeof(T)))) return -8;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (n == 0) return B2_STATUS_OK;
  B2_DBG_RANGE(l, a, (size_t)((n - 1) * lda + n) * sizeof(T));
  B2_DBG_VEC(l, x, n, incx);
  B2_DBG_COMMIT(l);
  L2Args<T> args = {};
  args.a = a;
  args.lda = lda;
  args.rows = args.cols = n;
  args.xc = args.xr = vec_base(x, n, incx);
  args.incxc = args.incxr = incx;
  args.alpha = T(1);
  args.beta = T(0);
  args.y = vec_base(x, n, incx);
  args.incy = incx;
  const bool upper = (order == B2_ROW_MAJOR) == (uplo == B2_UPPER);
  const bool row = (order == B2_ROW_MAJOR) == (trans == B2_NO_TRANS);
  const bool unit = diag == B2_UNIT;
  if (row) return upper ? trmv_kind<T, true, TRI_UPPER>(l, args, unit) : trmv_kind<T, true, TRI_LOWER>(l, args, unit);
  return upper ? trmv_kind<T, false, TRI_UPPER>(l, args, unit) : trmv_kind<T, false, TRI_LOWER>(l, args, unit);
}

}  // namespace b2
