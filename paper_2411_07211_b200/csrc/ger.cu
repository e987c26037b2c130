// ger: A <- alpha*x*y^T + A (Section 6.2.2; the paper's Figure 7 caption notes that ger shares
// the gemv schedule).  Pure streaming read-modify-write of A: each lane keeps alpha*y_j for
// its columns in registers and reuses them down a band of rows, x_i is a broadcast load.
#include "level2.cuh"
#include "skinny.cuh"

namespace b2 {

template <typename T, int V, class S>
__global__ void __launch_bounds__(kThreads) ger_kernel(T* __restrict__ a, int64_t lda, int64_t rows, int64_t cols,
                                                       const T* __restrict__ xr, int64_t incxr,
                                                       const T* __restrict__ yc, int64_t incyc, T alpha,
                                                       int64_t rows_per_cta, int nct) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int LPR = S::LPR, CU = S::CU, RU = S::RU, G = S::G, RB = S::RB;
  constexpr int TC = LPR * V * CU;
  using P = Pack<T, V>;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane / LPR, q = lane % LPR;
  const int ct = blockIdx.x % nct;
  const int64_t rs = blockIdx.x / nct;
  const int64_t r_begin = rs * rows_per_cta, r_end = min(rows, r_begin + rows_per_cta);
  const int64_t c0 = (int64_t)ct * TC;
  T yv[CU][V];
#pragma unroll
  for (int u = 0; u < CU; ++u)
#pragma unroll
    for (int e = 0; e < V; ++e) {
      const int64_t j = c0 + (u * LPR + q) * V + e;
      yv[u][e] = j < cols ? alpha * __ldg(yc + j * incyc) : T(0);
    }
  for (int64_t rb = r_begin; rb < r_end; rb += RB) {
    int64_t rowi[RU];
    T xv[RU];
#pragma unroll
    for (int ru = 0; ru < RU; ++ru) {
      rowi[ru] = rb + (ru * kWarps + warp) * G + g;
      xv[ru] = rowi[ru] < r_end ? __ldg(xr + rowi[ru] * incxr) : T(0);
    }
    if (rb + RB <= r_end && c0 + TC <= cols) {
      P av[RU][CU];
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u) av[ru][u] = ld_cs<T, V>(a + rowi[ru] * lda + c0 + (u * LPR + q) * V);
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u) {
#pragma unroll
          for (int e = 0; e < V; ++e) av[ru][u].v[e] = xv[ru] * yv[u][e] + av[ru][u].v[e];
          st_cs<T, V>(a + rowi[ru] * lda + c0 + (u * LPR + q) * V, av[ru][u]);
        }
    } else if (V > 1 && (c0 + TC <= cols || (cols - c0) % V == 0)) {
      // only the matrix edge cuts this tile, on pack boundaries (narrow matrices, short row
      // bands): the loads still go out together, each under its own row / pack predicate.
      // (Element-wise tiles, V == 1, stay on the plain path below: single-element streaming
      // stores to rows that start off a sector boundary measured twice as slow.)
      const int64_t npk = (min(cols, c0 + TC) - c0) / V;  // packs of this tile that exist
      P av[RU][CU];
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u)
          if (rowi[ru] < r_end && u * LPR + q < npk) av[ru][u] = ld_cs<T, V>(a + rowi[ru] * lda + c0 + (u * LPR + q) * V);
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u)
          if (rowi[ru] < r_end && u * LPR + q < npk) {
#pragma unroll
            for (int e = 0; e < V; ++e) av[ru][u].v[e] = xv[ru] * yv[u][e] + av[ru][u].v[e];
            st_cs<T, V>(a + rowi[ru] * lda + c0 + (u * LPR + q) * V, av[ru][u]);
          }
    } else {
#pragma unroll
      for (int ru = 0; ru < RU; ++ru) {
        if (rowi[ru] >= r_end) continue;
#pragma unroll
        for (int u = 0; u < CU; ++u) {
          const int64_t cv = c0 + (u * LPR + q) * V;
          T* ap = a + rowi[ru] * lda + cv;
          if (V > 1 && cv + V <= cols) {
            P av = ld_cs<T, V>(ap);
#pragma unroll
            for (int e = 0; e < V; ++e) av.v[e] = xv[ru] * yv[u][e] + av.v[e];
            st_cs<T, V>(ap, av);
          } else {
#pragma unroll
            for (int e = 0; e < V; ++e)
              if (cv + e < cols) ap[e] = xv[ru] * yv[u][e] + ap[e];
          }
        }
      }
    }
  }
}

template <typename T, int V, class S>
static int ger_launch(const Launch& l, T* a, int64_t lda, int64_t rows, int64_t cols, const T* xr, int64_t incxr,
                      const T* yc, int64_t incyc, T alpha) {
  constexpr int TC = S::template tc<V>();
  const int nct = (int)((cols + TC - 1) / TC);
  const int64_t rows_per_cta = (int64_t)S::RB * knob(kKnobGerRows);
  const int64_t nrs = (rows + rows_per_cta - 1) / rows_per_cta;
  if (nrs * nct > 0x7fffffff) return B2_STATUS_NOT_IMPLEMENTED;
  launch_chained(ger_kernel<T, V, S>, dim3((unsigned)(nrs * nct)), dim3(kThreads), 0, l.stream, a, lda, rows, cols, xr, incxr, yc, incyc, alpha,
                                                                        rows_per_cta, nct);
  return check_launch();
}

template <typename T, int V>
static int ger_shape(const Launch& l, T* a, int64_t lda, int64_t rows, int64_t cols, const T* xr, int64_t incxr,
                     const T* yc, int64_t incyc, T alpha) {
  const int64_t nv = (cols + V - 1) / V;
  if (nv >= 128) return ger_launch<T, V, ShapeWide>(l, a, lda, rows, cols, xr, incxr, yc, incyc, alpha);
  if (nv > 16) return ger_launch<T, V, ShapeMid>(l, a, lda, rows, cols, xr, incxr, yc, incyc, alpha);
  if (nv > 8) return ger_launch<T, V, ShapeHalf>(l, a, lda, rows, cols, xr, incxr, yc, incyc, alpha);
  return ger_launch<T, V, ShapeQuarter>(l, a, lda, rows, cols, xr, incxr, yc, incyc, alpha);
}

template <typename T>
static int ger_impl(const b2_ctx* ctx, int order, int64_t m, int64_t n, T alpha, const T* x, int64_t incx, const T* y,
                    int64_t incy, T* a, int64_t lda) {
  if (order != B2_ROW_MAJOR && order != B2_COL_MAJOR) return -1;
  if (m < 0) return -2;
  if (n < 0) return -3;
  if (incx == 0) return -6;
  if (m > 0 && n > 0 && (x == nullptr || !aligned_to(x, sizeof(T)))) return -5;
  if (incy == 0) return -8;
  if (m > 0 && n > 0 && (y == nullptr || !aligned_to(y, sizeof(T)))) return -7;
  if (m > 0 && n > 0 && (a == nullptr || !aligned_to(a, sizeof(T)))) return -9;
  const int64_t minor = order == B2_ROW_MAJOR ? n : m;
  if (lda < (minor > 1 ? minor : 1)) return -10;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (m == 0 || n == 0 || alpha == T(0)) return B2_STATUS_OK;
  B2_DBG_RANGE(l, a, (size_t)(((order == B2_ROW_MAJOR ? m : n) - 1) * lda + minor) * sizeof(T));
  B2_DBG_VEC(l, x, m, incx);
  B2_DBG_VEC(l, y, n, incy);
  B2_DBG_COMMIT(l);
  // canonical row-major view: row vector index = slow dimension of the buffer
  const bool rm = order == B2_ROW_MAJOR;
  const int64_t rows = rm ? m : n, cols = rm ? n : m;
  const T* xr = rm ? vec_base(x, m, incx) : vec_base(y, n, incy);
  const int64_t incxr = rm ? incx : incy;
  const T* yc = rm ? vec_base(y, n, incy) : vec_base(x, m, incx);
  const int64_t incyc = rm ? incy : incx;
  constexpr int V = VecLen<T>::value;
  // (measured: the element-wise walk wins in double; in float the pack kernels stay ahead)
  if (knob(kKnobNarrowBlock) && sizeof(T) == 8 && wide_applies<T>(rows, cols)) {
    const int64_t want = (cols + kThreads - 1) / kThreads, cap = (int64_t)sm_count() * 8;
    launch_chained(wide_ger_kernel<T>, dim3((unsigned)(want < cap ? want : cap)), dim3(kThreads), 0, l.stream, a, lda, (int)rows, cols, xr, incxr, yc, incyc,
                                                                                alpha);
    return check_launch();
  }
  if (skinny_applies(a, lda, rows, cols, false)) return skinny_ger<T>(l, a, rows, cols, xr, incxr, yc, incyc, alpha);
  if (aligned_to(a, 16) && lda % V == 0) return ger_shape<T, V>(l, a, lda, rows, cols, xr, incxr, yc, incyc, alpha);
  return ger_shape<T, 1>(l, a, lda, rows, cols, xr, incxr, yc, incyc, alpha);
}

}  // namespace b2

extern "C" {
int b2_sger(const b2_ctx* ctx, int order, int64_t m, int64_t n, float alpha, const float* x, int64_t incx,
            const float* y, int64_t incy, float* a, int64_t lda) {
  return b2::ger_impl<float>(ctx, order, m, n, alpha, x, incx, y, incy, a, lda);
}
int b2_dger(const b2_ctx* ctx, int order, int64_t m, int64_t n, double alpha, const double* x, int64_t incx,
            const double* y, int64_t incy, double* a, int64_t lda) {
  return b2::ger_impl<double>(ctx, order, m, n, alpha, x, incx, y, incy, a, lda);
}
}
