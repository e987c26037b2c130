// syr / syr2: symmetric rank-1 and rank-2 updates of the stored triangle (Section 6.2.2:
// "symmetric rank-1 update" and "symmetric rank-2 update" are among the level-2 kernels the
// paper's library covers).
//   syr  : A_ij <- alpha * x_i * x_j + A_ij
//   syr2 : A_ij <- alpha * (x_i * y_j + y_i * x_j) + A_ij        for (i, j) in the uplo triangle.
// Like ger this is a streaming read-modify-write of the matrix, 2s bytes per stored element;
// only the iteration space differs: the grid holds just the tiles that meet the triangle, a
// tile inside it takes 128-bit packs unconditionally, a tile that the diagonal crosses takes
// them where a whole pack is inside and single elements where the diagonal cuts one.  Each lane
// keeps alpha * x_j (and alpha * y_j) for its columns in registers down a band of rows.
#include "common.cuh"

namespace b2 {

// Tile shape: CU packs per lane and row (a warp covers 32 * V * CU columns of a row), RU rows per
// warp; CU * RU = 8 packs of every lane are in flight together.  Small tiles keep the tail of
// the grid short.  syr2 in float holds alpha*x_j and alpha*y_j for 4 * CU columns per lane, so it
// takes the narrow shape to stay within the registers of three resident blocks.
template <typename T, bool TWO>
struct SyrShape {
  static constexpr int CU = (TWO && sizeof(T) == 4) ? 2 : 4;
  static constexpr int RU = 8 / CU;
};

// Blocks enumerate only the tiles that meet the triangle.  Tiles are kSyrRows x TC; a "super
// row" is TC rows (m = TC / kSyrRows row tiles).  The first m * nct blocks take the tiles that
// the diagonal crosses (the slow, masked ones: started first, they do not end up as the tail of
// the grid), one per row tile.  The others take the tiles strictly inside: super row s + 1
// (counted from the narrow end of the triangle) has s + 1 of them per row tile, so interior
// block b lies there when m*s*(s+1)/2 <= b < m*(s+1)*(s+2)/2.
__device__ __forceinline__ void syr_tile_of_block(unsigned b, int m, int nct, bool lower, int64_t* row_tile,
                                                  int* col_tile, bool* on_diagonal) {
  const unsigned ndiag = (unsigned)m * (unsigned)nct;
  if (b < ndiag) {
    *row_tile = b;
    *col_tile = (int)(b / (unsigned)m);
    *on_diagonal = true;
    return;
  }
  b -= ndiag;
  const unsigned q = b / (unsigned)m;
  int s = (int)((sqrtf(8.0f * (float)q + 1.0f) - 1.0f) * 0.5f);
  while ((unsigned)(s + 1) * (unsigned)(s + 2) / 2 <= q) ++s;
  while ((unsigned)s * (unsigned)(s + 1) / 2 > q) --s;
  const unsigned rem = b - (unsigned)m * ((unsigned)s * (unsigned)(s + 1) / 2);
  const int rt_in = (int)(rem / (unsigned)(s + 1)), ctl = (int)(rem % (unsigned)(s + 1));
  const int super_row = lower ? s + 1 : nct - 2 - s;
  *row_tile = (int64_t)super_row * m + rt_in;
  *col_tile = lower ? ctl : nct - 1 - ctl;
  *on_diagonal = false;
}

// Canonical row-major view: `lower` means the stored triangle has column <= row there.
template <typename T, int V, bool TWO>
__global__ void __launch_bounds__(kThreads, TWO ? 3 : 4) syr_kernel(T* __restrict__ a, int64_t lda, int64_t n,
                                                       const T* __restrict__ x, int64_t incx,
                                                       const T* __restrict__ y, int64_t incy, T alpha, bool lower,
                                                       int nct) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int kSyrCU = SyrShape<T, TWO>::CU, kSyrRU = SyrShape<T, TWO>::RU;
  constexpr int kSyrRows = kWarps * kSyrRU;  // rows per block
  constexpr int TC = 32 * V * kSyrCU;        // columns per block
  constexpr int M = TC / kSyrRows;
  static_assert(TC % kSyrRows == 0, "a super row is a whole number of row tiles");
  using P = Pack<T, V>;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int64_t row_tile;
  int col_tile;
  bool diag;
  syr_tile_of_block(blockIdx.x, M, nct, lower, &row_tile, &col_tile, &diag);
  const int64_t c0 = (int64_t)col_tile * TC, r0 = row_tile * kSyrRows;
  if (r0 >= n) return;  // the last super row may be ragged
  const bool whole = !diag && r0 + kSyrRows <= n && c0 + TC <= n;  // every element inside, none ragged
  // the matrix loads of a whole tile go out before anything else: nothing they need depends
  // on the vectors (plain L2 loads: what is loaded is stored back at once, and evict-first loads
  // measured 4 % slower)
  T* ap[kSyrRU];
  P av[kSyrRU][kSyrCU];
  if (whole) {
#pragma unroll
    for (int ru = 0; ru < kSyrRU; ++ru) {
      ap[ru] = a + (r0 + ru * kWarps + warp) * lda + c0 + lane * V;
#pragma unroll
      for (int u = 0; u < kSyrCU; ++u) av[ru][u] = ld_cg<T, V>(ap[ru] + u * 32 * V);
    }
  }
  // alpha*x_j, alpha*y_j for the tile's columns and x_i, y_i for its rows pass through shared
  // memory: one global load per element and block instead of one per element and warp
  __shared__ __align__(16) T sxj[TC], syj[TWO ? TC : 1], sxi[kSyrRows], syi[TWO ? kSyrRows : 1];
  for (int t = threadIdx.x; t < TC; t += kThreads) {
    const int64_t j = c0 + t;
    sxj[t] = j < n ? alpha * __ldg(x + j * incx) : T(0);
    if (TWO) syj[t] = j < n ? alpha * __ldg(y + j * incy) : T(0);
  }
  if (threadIdx.x < kSyrRows) {
    const int64_t i = r0 + threadIdx.x;
    sxi[threadIdx.x] = i < n ? __ldg(x + i * incx) : T(0);
    if (TWO) syi[threadIdx.x] = i < n ? __ldg(y + i * incy) : T(0);
  }
  __syncthreads();
  T xj[kSyrCU][V], yj[kSyrCU][V];
#pragma unroll
  for (int u = 0; u < kSyrCU; ++u) {
    const P px = *reinterpret_cast<const P*>(&sxj[(u * 32 + lane) * V]);
    const P py = TWO ? *reinterpret_cast<const P*>(&syj[(u * 32 + lane) * V]) : P{};
#pragma unroll
    for (int e = 0; e < V; ++e) {
      xj[u][e] = px.v[e];
      yj[u][e] = TWO ? py.v[e] : T(0);
    }
  }
  if (whole) {
#pragma unroll
    for (int ru = 0; ru < kSyrRU; ++ru) {
      const T xi = sxi[ru * kWarps + warp];
      const T yi = TWO ? syi[ru * kWarps + warp] : T(0);
#pragma unroll
      for (int u = 0; u < kSyrCU; ++u) {
#pragma unroll
        for (int e = 0; e < V; ++e) {
          // syr: x_i*(alpha*x_j); syr2: y_i*(alpha*x_j) + x_i*(alpha*y_j)
          if (TWO) av[ru][u].v[e] = yi * xj[u][e] + (xi * yj[u][e] + av[ru][u].v[e]);
          else av[ru][u].v[e] = xi * xj[u][e] + av[ru][u].v[e];
        }
        st_cs<T, V>(ap[ru] + u * 32 * V, av[ru][u]);
      }
    }
    return;
  }
  // a tile that the diagonal or the matrix edge cuts: row by row; a pack that lies inside whole
  // is still moved as one, a pack that is cut goes element by element.  Columns are counted
  // from c0 here: jr in [0, TC), the matrix ends at ncols, row i has its diagonal at jd.
  const int ncols = (int)min((int64_t)TC, n - c0);
  for (int rr = warp; rr < kSyrRows; rr += kWarps) {
    const int64_t i = r0 + rr;
    if (i >= n) break;
    const int jd = (int)max((int64_t)-1, min((int64_t)TC, i - c0));
    const int lo = lower ? 0 : jd, hi = lower ? min(jd + 1, ncols) : ncols;  // columns [lo, hi) are inside
    const T xi = sxi[rr];
    const T yi = TWO ? syi[rr] : T(0);
    T* arow = a + i * lda + c0;
#pragma unroll
    for (int u = 0; u < kSyrCU; ++u) {
      const int jr = (u * 32 + lane) * V;
      if (V > 1 && jr >= lo && jr + V <= hi) {
        P av = ld_cg<T, V>(arow + jr);
#pragma unroll
        for (int e = 0; e < V; ++e) {
          if (TWO) av.v[e] = yi * xj[u][e] + (xi * yj[u][e] + av.v[e]);
          else av.v[e] = xi * xj[u][e] + av.v[e];
        }
        st_cs<T, V>(arow + jr, av);
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e)
          if (jr + e >= lo && jr + e < hi) {
            if (TWO) arow[jr + e] = yi * xj[u][e] + (xi * yj[u][e] + arow[jr + e]);
            else arow[jr + e] = xi * xj[u][e] + arow[jr + e];
          }
      }
    }
  }
}

template <typename T, int V, bool TWO>
static int syr_launch(const Launch& l, T* a, int64_t lda, int64_t n, const T* x, int64_t incx, const T* y,
                      int64_t incy, T alpha, bool lower) {
  constexpr int TC = 32 * V * SyrShape<T, TWO>::CU;
  constexpr int M = TC / (kWarps * SyrShape<T, TWO>::RU);
  const int64_t nct = (n + TC - 1) / TC;
  const int64_t blocks = M * (nct * (nct + 1) / 2);
  if (blocks > 0x7fffffff) return B2_STATUS_NOT_IMPLEMENTED;
  launch_chained(syr_kernel<T, V, TWO>, dim3((unsigned)blocks), dim3(kThreads), 0, l.stream, a, lda, n, x, incx, y, incy, alpha, lower,
                                                                     (int)nct);
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
  B2_DBG_RANGE(l, a, (size_t)((n - 1) * lda + n) * sizeof(T));
  B2_DBG_VEC(l, x, n, incx);
  if (TWO) B2_DBG_VEC(l, y, n, incy);
  B2_DBG_COMMIT(l);
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
