/*
 * CPU oracle for the dense BLAS level-1 / level-2 family -- TEST INFRASTRUCTURE ONLY.
 *
 * This file is included twice by blas_oracle.c, once per precision:
 *     T = float,  W = double        (prefix s)
 *     T = double, W = long double   (prefix d)
 * T is the storage type of the routine, W the wide type every sum is accumulated in.
 * Each output is rounded to T exactly once, at the end.  Loops run in index order;
 * there is no blocking, vectorisation, reordering or fusion, so each function can be
 * checked by eye against the definition it cites.
 *
 * Definitions followed: the paper adopts the BLAS problem statement by reference
 * (Section 6.2: "most of the kernels in BLAS levels 1 and 2"; options listed in
 * Section 6.2.2: precisions s/d, transpose t/n, lower/upper, unit/non-unit; Figure 9b:
 * "stride-1 and stride-any") and prints object code for axpy (Figure 4a),
 * gemv non-transposed (Section 2 inset, Figure 7a) and gemv transposed (Figure 7c).
 *
 * Conventions:
 *   - vectors: logical element i of a vector v with increment inc lives at
 *     v[i*inc] when inc > 0 and at v[(i-(n-1))*inc] when inc < 0 (BLAS walk order).
 *   - matrices: order 101 = row-major  (A(i,j) = a[i*lda + j]),
 *               order 102 = column-major (A(i,j) = a[j*lda + i]).
 *   - "absterms" outputs receive, per output element, the sum of the absolute values
 *     of the terms that were added to form it (accumulated in W, returned as double);
 *     tests scale their tolerance by it.  A NULL absterms pointer is skipped.
 *
 * Parity unpinned (documented, out of contract): NaN/Inf propagation, overflow-safe
 * scaling in nrm2, behaviour when input and output vectors alias.
 */

/* OR_PAR / OR_PAR_SUM: empty in the oracle proper.  The bench's all-cores baseline builds a
 * second copy of this file with ORACLE_OMP defined, where they put an OpenMP "parallel for" on
 * the outermost independent loop (a reduction clause for the three sums, which then add in
 * another order); that copy is only ever timed, never compared against. */
#ifndef OR_PAR
#ifdef ORACLE_OMP
#define OR_PAR _Pragma("omp parallel for schedule(static)")
#define OR_STR(...) #__VA_ARGS__
#define OR_PAR_SUM(...) _Pragma(OR_STR(omp parallel for schedule(static) reduction(+ : __VA_ARGS__)))
#else
#define OR_PAR
#define OR_PAR_SUM(...)
#endif
#endif

#define OR_CAT2(a, b) a##b
#define OR_CAT(a, b) OR_CAT2(a, b)
#define FN(name) OR_CAT(OR_CAT(oracle_, P), name)

static inline int64_t OR_CAT(P, _vidx)(int64_t i, int64_t n, int64_t inc) {
  return inc > 0 ? i * inc : (i - (n - 1)) * inc;
}
#define VIDX OR_CAT(P, _vidx)

static inline W OR_CAT(P, _wabs)(W v) { return v < 0 ? -v : v; }
#define WABS OR_CAT(P, _wabs)

static inline int64_t OR_CAT(P, _midx)(int order, int64_t i, int64_t j, int64_t lda) {
  return order == 101 ? i * lda + j : j * lda + i;
}
#define MIDX OR_CAT(P, _midx)

/* ---------------------------------------------------------------- level 1 */

/* axpy, Figure 4a: y[i] += a * x[i].  alpha == 0 returns without touching y. */
void FN(axpy)(int64_t n, T alpha, const T* x, int64_t incx, T* y, int64_t incy, double* absterms) {
  if (alpha == (T)0) {
    if (absterms)
      for (int64_t i = 0; i < n; ++i) absterms[i] = (double)WABS((W)y[VIDX(i, n, incy)]);
    return;
  }
  OR_PAR
  for (int64_t i = 0; i < n; ++i) {
    W p = (W)alpha * (W)x[VIDX(i, n, incx)];
    W yi = (W)y[VIDX(i, n, incy)];
    if (absterms) absterms[i] = (double)(WABS(p) + WABS(yi));
    y[VIDX(i, n, incy)] = (T)(p + yi);
  }
}

/* scal (Section 6.2.1 "scale"): x[i] = alpha * x[i], ONE multiply in type T. */
void FN(scal)(int64_t n, T alpha, T* x, int64_t incx) {
  OR_PAR
  for (int64_t i = 0; i < n; ++i) {
    volatile T prod = alpha * x[VIDX(i, n, incx)];
    x[VIDX(i, n, incx)] = prod;
  }
}

/* copy: y[i] = x[i]. */
void FN(copy)(int64_t n, const T* x, int64_t incx, T* y, int64_t incy) {
  OR_PAR
  for (int64_t i = 0; i < n; ++i) y[VIDX(i, n, incy)] = x[VIDX(i, n, incx)];
}

/* swap: x[i] <-> y[i]. */
void FN(swap)(int64_t n, T* x, int64_t incx, T* y, int64_t incy) {
  OR_PAR
  for (int64_t i = 0; i < n; ++i) {
    T t = x[VIDX(i, n, incx)];
    x[VIDX(i, n, incx)] = y[VIDX(i, n, incy)];
    y[VIDX(i, n, incy)] = t;
  }
}

/* rot: (x_i, y_i) <- (c x_i + s y_i, c y_i - s x_i), both from the old pair. */
void FN(rot)(int64_t n, T* x, int64_t incx, T* y, int64_t incy, T c, T s,
             double* absterms_x, double* absterms_y) {
  OR_PAR
  for (int64_t i = 0; i < n; ++i) {
    W xi = (W)x[VIDX(i, n, incx)], yi = (W)y[VIDX(i, n, incy)];
    W cx = (W)c * xi, sy = (W)s * yi, cy = (W)c * yi, sx = (W)s * xi;
    x[VIDX(i, n, incx)] = (T)(cx + sy);
    y[VIDX(i, n, incy)] = (T)(cy - sx);
    if (absterms_x) absterms_x[i] = (double)(WABS(cx) + WABS(sy));
    if (absterms_y) absterms_y[i] = (double)(WABS(cy) + WABS(sx));
  }
}

/* rotm: the modified Givens rotation (the paper's level-1 set, Section 6.2.1, includes rotm;
 * the definition is the BLAS one).  (x_i, y_i) <- (h11 x_i + h12 y_i, h21 x_i + h22 y_i), both
 * from the old pair, with H selected by flag = param[0]:
 *   flag = -1 : H = [h11 h12; h21 h22]   all four from param
 *   flag =  0 : H = [  1 h12; h21   1]   the diagonal is implied, param[1] and param[4] unread
 *   flag =  1 : H = [h11   1;  -1 h22]   the off-diagonal is implied, param[2] and param[3] unread
 *   flag = -2 : H = I                    nothing is read or written
 * param = {flag, h11, h21, h12, h22}.  An implied 1 or -1 means no multiplication: that term is
 * the element itself (or its negation). */
void FN(rotm)(int64_t n, T* x, int64_t incx, T* y, int64_t incy, const T* param,
              double* absterms_x, double* absterms_y) {
  const T flag = param[0];
  if (flag == (T)-2) return;
  for (int64_t i = 0; i < n; ++i) {
    W xi = (W)x[VIDX(i, n, incx)], yi = (W)y[VIDX(i, n, incy)];
    W xx, xy, yx, yy; /* the four terms: x' = xx + xy, y' = yx + yy */
    if (flag == (T)-1) {
      xx = (W)param[1] * xi; xy = (W)param[3] * yi;
      yx = (W)param[2] * xi; yy = (W)param[4] * yi;
    } else if (flag == (T)0) {
      xx = xi;               xy = (W)param[3] * yi;
      yx = (W)param[2] * xi; yy = yi;
    } else { /* flag == 1 */
      xx = (W)param[1] * xi; xy = yi;
      yx = -xi;              yy = (W)param[4] * yi;
    }
    x[VIDX(i, n, incx)] = (T)(xx + xy);
    y[VIDX(i, n, incy)] = (T)(yx + yy);
    if (absterms_x) absterms_x[i] = (double)(WABS(xx) + WABS(xy));
    if (absterms_y) absterms_y[i] = (double)(WABS(yx) + WABS(yy));
  }
}

/* dot: sum_i x_i y_i. */
void FN(dot)(int64_t n, const T* x, int64_t incx, const T* y, int64_t incy, T* result,
             double* absterms) {
  W acc = 0, aabs = 0;
  OR_PAR_SUM(acc, aabs)
  for (int64_t i = 0; i < n; ++i) {
    W p = (W)x[VIDX(i, n, incx)] * (W)y[VIDX(i, n, incy)];
    acc += p;
    aabs += WABS(p);
  }
  *result = (T)acc;
  if (absterms) *absterms = (double)aabs;
}

/* asum: sum_i |x_i|. */
void FN(asum)(int64_t n, const T* x, int64_t incx, T* result, double* absterms) {
  W acc = 0;
  OR_PAR_SUM(acc)
  for (int64_t i = 0; i < n; ++i) acc += WABS((W)x[VIDX(i, n, incx)]);
  *result = (T)acc;
  if (absterms) *absterms = (double)acc;
}

/* nrm2: sqrt(sum_i x_i^2); absterms receives sum_i x_i^2 (before the root). */
void FN(nrm2)(int64_t n, const T* x, int64_t incx, T* result, double* absterms) {
  W acc = 0;
  OR_PAR_SUM(acc)
  for (int64_t i = 0; i < n; ++i) {
    W v = (W)x[VIDX(i, n, incx)];
    acc += v * v;
  }
  *result = (T)WSQRT(acc);
  if (absterms) *absterms = (double)acc;
}

/* iamax: smallest 0-based i with |x_i| = max_k |x_k|; n == 0 gives 0.
 * Scan in index order, replace only on strict '>' (first maximum wins). */
void FN(iamax)(int64_t n, const T* x, int64_t incx, int64_t* result) {
  int64_t best_i = 0;
  if (n > 0) {
    T best = x[VIDX(0, n, incx)];
    if (best < 0) best = -best;
    for (int64_t i = 1; i < n; ++i) {
      T v = x[VIDX(i, n, incx)];
      if (v < 0) v = -v;
      if (v > best) {
        best = v;
        best_i = i;
      }
    }
  }
  *result = best_i;
}

/* ---------------------------------------------------------------- level 2 */

/* gemv (Section 2 inset / Figure 7a: y[i] += A[i,j]*x[j]; Figure 7c: y[j] += x[i]*A[i,j]),
 * with BLAS scaling: y <- alpha*op(A)*x + beta*y.  A is m x n.
 * trans 111: op(A) = A, x has n elements, y has m; trans 112: op(A) = A^T, x has m, y has n.
 * beta == 0: y is written without being read.  absterms has one entry per y element. */
void FN(gemv)(int order, int trans, int64_t m, int64_t n, T alpha, const T* a, int64_t lda,
              const T* x, int64_t incx, T beta, T* y, int64_t incy, double* absterms) {
  int64_t leny = trans == 111 ? m : n;
  int64_t lenx = trans == 111 ? n : m;
  OR_PAR
  for (int64_t r = 0; r < leny; ++r) {
    W acc = 0, aabs = 0;
    if (alpha != (T)0) {
      for (int64_t k = 0; k < lenx; ++k) {
        W aij = trans == 111 ? (W)a[MIDX(order, r, k, lda)] : (W)a[MIDX(order, k, r, lda)];
        W p = (W)alpha * (aij * (W)x[VIDX(k, lenx, incx)]);
        acc += p;
        aabs += WABS(p);
      }
    }
    if (beta != (T)0) {
      W by = (W)beta * (W)y[VIDX(r, leny, incy)];
      acc += by;
      aabs += WABS(by);
    }
    y[VIDX(r, leny, incy)] = (T)acc;
    if (absterms) absterms[r] = (double)aabs;
  }
}

/* ger: A[i,j] += alpha * x[i] * y[j], A is m x n.  alpha == 0 leaves A untouched.
 * absterms (optional) is a dense m*n array in (i*n + j) order regardless of storage order. */
void FN(ger)(int order, int64_t m, int64_t n, T alpha, const T* x, int64_t incx, const T* y,
             int64_t incy, T* a, int64_t lda, double* absterms) {
  OR_PAR
  for (int64_t i = 0; i < m; ++i) {
    for (int64_t j = 0; j < n; ++j) {
      W aij = (W)a[MIDX(order, i, j, lda)];
      if (alpha == (T)0) {
        if (absterms) absterms[i * n + j] = (double)WABS(aij);
        continue;
      }
      W p = (W)alpha * ((W)x[VIDX(i, m, incx)] * (W)y[VIDX(j, n, incy)]);
      a[MIDX(order, i, j, lda)] = (T)(p + aij);
      if (absterms) absterms[i * n + j] = (double)(WABS(p) + WABS(aij));
    }
  }
}

/* syr: A[i,j] += alpha * x[i] * x[j] for the (i,j) of the uplo triangle (121 upper: i <= j,
 * 122 lower: i >= j), A symmetric n x n with that triangle stored; the other triangle is never
 * touched.  alpha == 0 leaves A untouched.  One of the symmetric rank-1 updates of Section 6.2.2
 * ("symmetric rank-1 update"); the BLAS problem statement the paper adopts defines it.
 * absterms (optional) is a dense n*n array in (i*n + j) order; entries outside the triangle
 * are left as they are. */
void FN(syr)(int order, int uplo, int64_t n, T alpha, const T* x, int64_t incx, T* a, int64_t lda,
             double* absterms) {
  for (int64_t i = 0; i < n; ++i) {
    for (int64_t j = 0; j < n; ++j) {
      int stored = uplo == 121 ? (i <= j) : (i >= j);
      if (!stored) continue;
      W aij = (W)a[MIDX(order, i, j, lda)];
      if (alpha == (T)0) {
        if (absterms) absterms[i * n + j] = (double)WABS(aij);
        continue;
      }
      W p = (W)alpha * ((W)x[VIDX(i, n, incx)] * (W)x[VIDX(j, n, incx)]);
      a[MIDX(order, i, j, lda)] = (T)(p + aij);
      if (absterms) absterms[i * n + j] = (double)(WABS(p) + WABS(aij));
    }
  }
}

/* syr2: A[i,j] += alpha * (x[i]*y[j] + y[i]*x[j]) on the uplo triangle; same conventions as syr. */
void FN(syr2)(int order, int uplo, int64_t n, T alpha, const T* x, int64_t incx, const T* y,
              int64_t incy, T* a, int64_t lda, double* absterms) {
  for (int64_t i = 0; i < n; ++i) {
    for (int64_t j = 0; j < n; ++j) {
      int stored = uplo == 121 ? (i <= j) : (i >= j);
      if (!stored) continue;
      W aij = (W)a[MIDX(order, i, j, lda)];
      if (alpha == (T)0) {
        if (absterms) absterms[i * n + j] = (double)WABS(aij);
        continue;
      }
      W p1 = (W)alpha * ((W)x[VIDX(i, n, incx)] * (W)y[VIDX(j, n, incy)]);
      W p2 = (W)alpha * ((W)y[VIDX(i, n, incy)] * (W)x[VIDX(j, n, incx)]);
      a[MIDX(order, i, j, lda)] = (T)(p1 + p2 + aij);
      if (absterms) absterms[i * n + j] = (double)(WABS(p1) + WABS(p2) + WABS(aij));
    }
  }
}

/* Element (i,j) of a symmetric matrix of which only the uplo triangle is stored
 * (121 upper: i <= j stored, 122 lower: i >= j stored).  The other triangle is never read. */
static inline W OR_CAT(P, _sym_elem)(int order, int uplo, const T* a, int64_t lda, int64_t i,
                                     int64_t j) {
  int stored = uplo == 121 ? (i <= j) : (i >= j);
  return stored ? (W)a[MIDX(order, i, j, lda)] : (W)a[MIDX(order, j, i, lda)];
}

/* symv: y <- alpha*A*x + beta*y with A symmetric n x n, one triangle stored. */
void FN(symv)(int order, int uplo, int64_t n, T alpha, const T* a, int64_t lda, const T* x,
              int64_t incx, T beta, T* y, int64_t incy, double* absterms) {
  OR_PAR
  for (int64_t i = 0; i < n; ++i) {
    W acc = 0, aabs = 0;
    if (alpha != (T)0) {
      for (int64_t j = 0; j < n; ++j) {
        W aij = OR_CAT(P, _sym_elem)(order, uplo, a, lda, i, j);
        W p = (W)alpha * (aij * (W)x[VIDX(j, n, incx)]);
        acc += p;
        aabs += WABS(p);
      }
    }
    if (beta != (T)0) {
      W by = (W)beta * (W)y[VIDX(i, n, incy)];
      acc += by;
      aabs += WABS(by);
    }
    y[VIDX(i, n, incy)] = (T)acc;
    if (absterms) absterms[i] = (double)aabs;
  }
}

/* Element (i,j) of op(A) for a triangular A (uplo 121 upper / 122 lower, diag 131 non-unit /
 * 132 unit).  Outside the triangle it is 0 and on a unit diagonal it is 1, in both cases
 * WITHOUT reading memory.  *nonzero tells the caller whether the position is structural. */
static inline W OR_CAT(P, _tri_op_elem)(int order, int uplo, int trans, int diag, const T* a,
                                        int64_t lda, int64_t i, int64_t j, int* nonzero) {
  int64_t r = trans == 111 ? i : j; /* position inside A itself */
  int64_t c = trans == 111 ? j : i;
  int inside = uplo == 121 ? (r <= c) : (r >= c);
  *nonzero = inside;
  if (!inside) return 0;
  if (r == c && diag == 132) return 1;
  return (W)a[MIDX(order, r, c, lda)];
}
#define TRI_OP OR_CAT(P, _tri_op_elem)

/* trmv: x <- op(A) x.  Computed from a snapshot of x, stored at the end.
 * scratch_w must hold n values of W (caller passes n*sizeof(long double) bytes to be safe). */
void FN(trmv)(int order, int uplo, int trans, int diag, int64_t n, const T* a, int64_t lda, T* x,
              int64_t incx, double* absterms, void* scratch_w) {
  W* out = (W*)scratch_w;
  OR_PAR
  for (int64_t i = 0; i < n; ++i) {
    W acc = 0, aabs = 0;
    for (int64_t j = 0; j < n; ++j) {
      int nz;
      W e = TRI_OP(order, uplo, trans, diag, a, lda, i, j, &nz);
      if (!nz) continue;
      W p = e * (W)x[VIDX(j, n, incx)];
      acc += p;
      aabs += WABS(p);
    }
    out[i] = acc;
    if (absterms) absterms[i] = (double)aabs;
  }
  for (int64_t i = 0; i < n; ++i) x[VIDX(i, n, incx)] = (T)out[i];
}

/* trsv: solve op(A) x = b in place (b is passed in x).  op(A) lower triangular => forward
 * substitution x_i = (b_i - sum_{j<i} op(A)_ij x_j) / op(A)_ii; upper => backward.
 * The running solution is kept in W (scratch_w, n values) and rounded to T at the end.
 * absterms_i = |b_i| + sum_j |op(A)_ij x_j| (the magnitude of row i's balance). */
void FN(trsv)(int order, int uplo, int trans, int diag, int64_t n, const T* a, int64_t lda, T* x,
              int64_t incx, double* absterms, void* scratch_w) {
  W* sol = (W*)scratch_w;
  int eff_lower = (uplo == 122) != (trans == 112);
  for (int64_t step = 0; step < n; ++step) {
    int64_t i = eff_lower ? step : n - 1 - step;
    W bi = (W)x[VIDX(i, n, incx)];
    W acc = bi, aabs = WABS(bi);
    int64_t j0 = eff_lower ? 0 : i + 1, j1 = eff_lower ? i : n;
    for (int64_t j = j0; j < j1; ++j) {
      int nz;
      W e = TRI_OP(order, uplo, trans, diag, a, lda, i, j, &nz);
      W p = e * sol[j];
      acc -= p;
      aabs += WABS(p);
    }
    int nz;
    W d = TRI_OP(order, uplo, trans, diag, a, lda, i, i, &nz);
    sol[i] = acc / d;
    if (absterms) absterms[i] = (double)aabs;
  }
  for (int64_t i = 0; i < n; ++i) x[VIDX(i, n, incx)] = (T)sol[i];
}

/* Row-wise residual of a candidate solution xs of op(A) x = b, evaluated in W:
 *   resid_i = | b_i - sum_j op(A)_ij xs_j |,   scale_i = |b_i| + sum_j |op(A)_ij xs_j|. */
void FN(trsv_residual)(int order, int uplo, int trans, int diag, int64_t n, const T* a,
                       int64_t lda, const T* b, int64_t incb, const T* xs, int64_t incx,
                       double* resid, double* scale) {
  for (int64_t i = 0; i < n; ++i) {
    W bi = (W)b[VIDX(i, n, incb)];
    W acc = bi, aabs = WABS(bi);
    for (int64_t j = 0; j < n; ++j) {
      int nz;
      W e = TRI_OP(order, uplo, trans, diag, a, lda, i, j, &nz);
      if (!nz) continue;
      W p = e * (W)xs[VIDX(j, n, incx)];
      acc -= p;
      aabs += WABS(p);
    }
    resid[i] = (double)WABS(acc);
    scale[i] = (double)aabs;
  }
}

#undef TRI_OP
#undef MIDX
#undef WABS
#undef VIDX
#undef FN
#undef OR_CAT
#undef OR_CAT2
