// Level-2 matrix-vector template layer (Section 6.2.2 of the paper).
//
// One tile kernel serves gemv (N and T), symv and trmv in every option combination.  The
// matrix is always seen in its canonical row-major view (rows x cols, row stride lda; a
// column-major call is the transposed row-major problem).  A thread block owns a band of
// rows and a range of column tiles and may produce
//   ROWOUT: rowacc_i = sum_j A_ij * xc_j   (each row is a contiguous dot product), and/or
//   COLOUT: colacc_j = sum_i A_ij * xr_i   (column sums accumulated in registers),
// restricted to the upper / lower triangle for the triangular kinds.  This is the paper's
// level-2 recipe restated for a GPU: several rows are processed at once so the x values sit in
// registers and are reused (unroll-and-jam), triangular bounds are rounded to tile
// boundaries so full tiles run unmasked and only diagonal tiles are predicated, and narrow
// matrices get shapes whose whole row fits the lanes of a warp (the "skinny" case).
//
// Blocks write either the final result (when no other block contributes to the same
// output) or a partial into the workspace; l2_finalize then adds the partials in a fixed
// order and applies alpha / beta.  No atomics: results are bit-reproducible.
#pragma once

#include <algorithm>

#include "common.cuh"

namespace b2 {

enum { TRI_FULL = 0, TRI_UPPER = 1, TRI_LOWER = 2 };

template <bool ROWOUT_, bool COLOUT_, int TRI_, bool UNIT_, bool SYM_>
struct Kind {
  static constexpr bool ROWOUT = ROWOUT_, COLOUT = COLOUT_, UNIT = UNIT_, SYM = SYM_;
  static constexpr int TRI = TRI_;
};

// LPR lanes cover one row segment, so a warp covers G = 32/LPR rows per step; each lane owns
// CU packs of V columns; RU row steps are in flight per warp.
// NCT: column tiles a block of a COLOUT kind walks per row step (their column sums stay in
// registers side by side, the row sums run across all of them).
template <int LPR_, int CU_, int RU_, int NCT_ = 1>
struct Shape {
  static constexpr int LPR = LPR_, CU = CU_, RU = RU_, G = 32 / LPR_, NCT = NCT_;
  static constexpr int MINB = NCT_ == 1 ? 4 : 3;  // resident blocks per SM the register budget aims at
  static constexpr int RB = kWarps * G * RU_;  // rows per block step
  template <int V>
  static constexpr int tc() {
    return LPR_ * V * CU_;
  }
};

template <typename T>
struct L2Args {
  const T* a;
  int64_t lda, rows, cols;
  const T* xc;  // vector indexed by column (ROWOUT), base per vec_base()
  int64_t incxc;
  const T* xr;  // vector indexed by row (COLOUT)
  int64_t incxr;
  T* rowpart;  // [ncs][rows]
  T* colpart;  // [nrs][cols]
  int64_t rows_per_cta;
  int ctiles_per_cta, nct, nrs, ncs;
  int direct;  // 1: blocks write alpha*acc + beta*y straight to y
  int xc_vec;  // xc is 16-byte aligned with increment 1 (value 1) or 2 (value 2): read it in packs
  T alpha, beta;
  T* y;
  int64_t incy;
};

// Which parts of the tile grid hold any element of the triangle.  Used identically by the
// tile kernel (to skip work) and by the finalize kernel (to know which partials exist).
template <int TRI>
__host__ __device__ __forceinline__ bool region_active(int64_t r0, int64_t r1, int64_t c0, int64_t c1) {
  if (TRI == TRI_UPPER) return c1 - 1 >= r0;  // some (i, j) with j >= i
  if (TRI == TRI_LOWER) return c0 <= r1 - 1;  // some (i, j) with j <= i
  return true;
}
// Tile lies strictly inside the triangle (no diagonal element, no masking needed).
template <int TRI>
__device__ __forceinline__ bool region_strictly_inside(int64_t r0, int64_t r1, int64_t c0, int64_t c1) {
  if (TRI == TRI_UPPER) return c0 >= r1;
  if (TRI == TRI_LOWER) return c1 <= r0;
  return true;
}

template <typename T, int V, class K, class S>
__global__ void __launch_bounds__(kThreads, S::MINB) l2_tile_kernel(const L2Args<T> p) {
  constexpr int LPR = S::LPR, CU = S::CU, RU = S::RU, G = S::G, RB = S::RB;
  constexpr int TC = LPR * V * CU;
  constexpr int NCT = K::COLOUT ? S::NCT : 1;
  using P = Pack<T, V>;
  grid_dep_wait();
  grid_dep_launch();  // the next kernel of the stream (often this call's finalize pass) may be scheduled early

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane / LPR, q = lane % LPR;
  // Blocks start in index order.  In an upper triangle the bottom-right blocks are the ones that the
  // matrix edge cuts (the last column tile, ragged when n is not a multiple of the tile, is there the
  // LONGEST column); started last and running alone they would be the tail (measured in double at
  // n = 8190, column sums: 74 us against 48), so the order is reversed and the last block to start
  // is the small one in the top-left corner.
  const unsigned bidx = K::TRI == TRI_UPPER ? gridDim.x - 1u - blockIdx.x : blockIdx.x;
  const int cs = (int)(bidx % (unsigned)p.ncs);
  const int64_t rs = bidx / (unsigned)p.ncs;
  const int64_t r_begin = rs * p.rows_per_cta;
  const int64_t r_end = min(p.rows, r_begin + p.rows_per_cta);
  const int ct_begin = cs * p.ctiles_per_cta;
  const int ct_end = min(p.nct, ct_begin + p.ctiles_per_cta);
  const int64_t c_lo = (int64_t)ct_begin * TC, c_hi = min(p.cols, (int64_t)ct_end * TC);
  if (!region_active<K::TRI>(r_begin, r_end, c_lo, c_hi)) return;

  T colacc[NCT][CU][V];
  T xcv[NCT][CU][V];
  int xcv_ct[NCT];  // column tile whose x values are in xcv[c]
#pragma unroll
  for (int c = 0; c < NCT; ++c) {
    xcv_ct[c] = -1;
#pragma unroll
    for (int u = 0; u < CU; ++u)
#pragma unroll
      for (int e = 0; e < V; ++e) colacc[c][u][e] = T(0), xcv[c][u][e] = T(0);
  }

  // Address arithmetic is hoisted: inside a tile everything is a 32-bit local index or a
  // pointer bumped by a precomputed stride.
  const int lrow0 = warp * G + g;                            // first local row of this thread
  const int64_t rstride = (int64_t)kWarps * G * p.lda;       // elements between a thread's rows
  const int64_t xstride = (int64_t)kWarps * G * p.incxr;
  const T* a_cta = p.a + (r_begin + lrow0) * p.lda + q * V;  // row r_begin + lrow0, column q*V

  for (int64_t rb = r_begin; rb < r_end; rb += RB) {
    const int64_t rb_end = min(rb + RB, r_end);
    if (!region_active<K::TRI>(rb, rb_end, c_lo, c_hi)) continue;
    const int nr = (int)(rb_end - rb);  // rows of this batch
    const T* a_rb = a_cta + (rb - r_begin) * p.lda;
    T rowacc[RU], xrv[RU];
#pragma unroll
    for (int ru = 0; ru < RU; ++ru) {
      rowacc[ru] = T(0);
      xrv[ru] = T(0);
    }
    if (K::COLOUT) {
      const T* xp = p.xr + (rb + lrow0) * p.incxr;
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
        if (lrow0 + ru * kWarps * G < nr) xrv[ru] = __ldg(xp + ru * xstride);
    }
    // COLOUT kinds: slot c holds column tile ct_begin + c; ROWOUT-only kinds: one slot, any
    // number of column tiles.
#pragma unroll
    for (int c = 0; c < NCT; ++c) {
    const int ct_lo = K::COLOUT ? ct_begin + c : ct_begin;
    const int ct_hi = K::COLOUT ? min(ct_lo + 1, ct_end) : ct_end;
    for (int ct = ct_lo; ct < ct_hi; ++ct) {
      const int64_t c0 = (int64_t)ct * TC, c1 = min(p.cols, c0 + TC);
      if (!region_active<K::TRI>(rb, rb_end, c0, c1)) continue;
      if (K::ROWOUT && xcv_ct[c] != ct) {
        xcv_ct[c] = ct;
        if (V > 1 && p.xc_vec == 1 && c0 + TC <= p.cols) {
#pragma unroll
          for (int u = 0; u < CU; ++u) {
            const P xv = ld_ro<T, V>(p.xc + c0 + (u * LPR + q) * V);
#pragma unroll
            for (int e = 0; e < V; ++e) xcv[c][u][e] = xv.v[e];
          }
        } else if (V > 1 && p.xc_vec == 2 && c0 + TC < p.cols) {
          // increment 2: the V values sit in two consecutive packs (even positions); the odd
          // position after the last value exists because the tile is not the vector's last
#pragma unroll
          for (int u = 0; u < CU; ++u) {
            const T* xp = p.xc + 2 * (c0 + (u * LPR + q) * V);
            const P x0 = ld_ro<T, V>(xp), x1 = ld_ro<T, V>(xp + V);
#pragma unroll
            for (int e = 0; e < V; ++e) xcv[c][u][e] = (2 * e < V) ? x0.v[(2 * e) % V] : x1.v[(2 * e) % V];
          }
        } else {
#pragma unroll
          for (int u = 0; u < CU; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) {
              const int64_t j = c0 + (u * LPR + q) * V + e;
              xcv[c][u][e] = j < p.cols ? __ldg(p.xc + j * p.incxc) : T(0);
            }
        }
      }
      const bool fast = (rb + RB <= r_end) && (c0 + TC <= p.cols) &&
                        region_strictly_inside<K::TRI>(rb, rb + RB, c0, c0 + TC);
      if (fast) {
        P av[RU][CU];
        const T* at = a_rb + c0;
#pragma unroll
        for (int ru = 0; ru < RU; ++ru)
#pragma unroll
          for (int u = 0; u < CU; ++u) av[ru][u] = ld_nc<T, V>(at + ru * rstride + u * (LPR * V));
#pragma unroll
        for (int ru = 0; ru < RU; ++ru)
#pragma unroll
          for (int u = 0; u < CU; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) {
              if (K::ROWOUT) rowacc[ru] = av[ru][u].v[e] * xcv[c][u][e] + rowacc[ru];
              if (K::COLOUT) colacc[c][u][e] = av[ru][u].v[e] * xrv[ru] + colacc[c][u][e];
            }
      } else if (K::TRI == TRI_FULL && (V == 1 || (c1 - c0) % V == 0)) {
        // gemv: a tile that the matrix edge cuts (fewer rows than RB, or a row that ends on a
        // pack boundary before the tile does): the loads still go out together, each under its
        // own row / pack predicate.  Narrow matrices (fewer columns than one tile) and short
        // ones (fewer rows than one step) live entirely here.  A masked pack is zero and meets
        // a zero x value, so it adds nothing.
        const int npk = (int)(c1 - c0) / V;  // packs of this tile that exist
        P av[RU][CU];
        const T* at = a_rb + c0;
#pragma unroll
        for (int ru = 0; ru < RU; ++ru) {
          const bool rok = lrow0 + ru * kWarps * G < nr;
#pragma unroll
          for (int u = 0; u < CU; ++u) {
#pragma unroll
            for (int e = 0; e < V; ++e) av[ru][u].v[e] = T(0);
            if (rok && u * LPR + q < npk) av[ru][u] = ld_nc<T, V>(at + ru * rstride + u * (LPR * V));
          }
        }
#pragma unroll
        for (int ru = 0; ru < RU; ++ru)
#pragma unroll
          for (int u = 0; u < CU; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) {
              if (K::ROWOUT) rowacc[ru] = av[ru][u].v[e] * xcv[c][u][e] + rowacc[ru];
              if (K::COLOUT) colacc[c][u][e] = av[ru][u].v[e] * xrv[ru] + colacc[c][u][e];
            }
      } else {
        // Diagonal tiles and column edges inside a pack: local 32-bit indices; d = (first column)
        // - (first row), so element (li, lj) lies on the diagonal when d + lj == li.  All loads
        // of the tile go out together, each under its own predicate (a pack wholly outside the
        // triangle or the matrix is not read), and only then are the elements masked: loads
        // issued one by one between the branches made such a tile last several memory latencies.
        const int64_t d64 = c0 - rb;
        const int d = (int)(d64 > (1 << 24) ? (1 << 24) : d64 < -(1 << 24) ? -(1 << 24) : d64);
        const int nc = (int)(c1 - c0);
        const T* at = a_rb + c0;
        P av[RU][CU];
#pragma unroll
        for (int ru = 0; ru < RU; ++ru) {
          const int li = lrow0 + ru * kWarps * G;
#pragma unroll
          for (int u = 0; u < CU; ++u) {
            const int lc = (u * LPR + q) * V;
            bool use = li < nr && lc < nc;
            if (K::TRI == TRI_UPPER) use = use && d + lc + V - 1 >= li;
            if (K::TRI == TRI_LOWER) use = use && d + lc <= li;
            av[ru][u] = ld_nc_if<T, V>(at + ru * rstride + u * (LPR * V), use && (V == 1 || lc + V <= nc));
          }
        }
        if (V > 1 && nc % V != 0) {  // the rows end inside a pack: that pack element by element
#pragma unroll
          for (int ru = 0; ru < RU; ++ru) {
            const int li = lrow0 + ru * kWarps * G;
#pragma unroll
            for (int u = 0; u < CU; ++u) {
              const int lc = (u * LPR + q) * V;
              bool use = li < nr && lc < nc && lc + V > nc;
              if (K::TRI == TRI_UPPER) use = use && d + lc + V - 1 >= li;
              if (K::TRI == TRI_LOWER) use = use && d + lc <= li;
              const T* ap = at + ru * rstride + u * (LPR * V);
#pragma unroll
              for (int e = 0; e < V; ++e)
                if (use && lc + e < nc) av[ru][u].v[e] = __ldg(ap + e);
            }
          }
        }
#pragma unroll
        for (int ru = 0; ru < RU; ++ru) {
          const int li = lrow0 + ru * kWarps * G;
#pragma unroll
          for (int u = 0; u < CU; ++u) {
            const int lc = (u * LPR + q) * V;
#pragma unroll
            for (int e = 0; e < V; ++e) {
              const int lj = lc + e;
              bool in = li < nr && lj < nc;
              if (K::TRI == TRI_UPPER) in = in && d + lj >= li;
              if (K::TRI == TRI_LOWER) in = in && d + lj <= li;
              const bool dg = (K::TRI != TRI_FULL) && (d + lj == li);
              const T v = (K::UNIT && dg) ? T(1) : av[ru][u].v[e];
              // (a select, not a product with zero: x may hold infinities where the triangle ends)
              if (K::ROWOUT) rowacc[ru] = in ? v * xcv[c][u][e] + rowacc[ru] : rowacc[ru];
              if (K::COLOUT && !(K::SYM && dg)) colacc[c][u][e] = in ? v * xrv[ru] + colacc[c][u][e] : colacc[c][u][e];
            }
          }
        }
      }
    }
    }  // slot c
    if (K::ROWOUT) {  // all RU row sums in one transposing butterfly
      constexpr int LPV = LPR / RU;  // lanes left per row after the reduction
      const T s = multi_group_sum<LPR, RU>(rowacc, lane);
      const int64_t i = rb + ((q / LPV) * kWarps + warp) * G + g;
      if (q % LPV == 0 && i < r_end) {
        if (p.direct) {
          T* yp = p.y + i * p.incy;
          B2_STORE(yp, p.beta != T(0) ? p.alpha * s + p.beta * *yp : p.alpha * s);
        } else {
          p.rowpart[(int64_t)cs * p.rows + i] = s;
        }
      }
    }
  }

  if constexpr (K::COLOUT) {  // NCT column tiles per block for these kinds
    __shared__ T sm[kWarps][NCT * TC];
#pragma unroll
    for (int c = 0; c < NCT; ++c)
#pragma unroll
      for (int u = 0; u < CU; ++u)
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const T s = cross_group_sum<LPR>(colacc[c][u][e]);
          if (g == 0) sm[warp][c * TC + (u * LPR + q) * V + e] = s;
        }
    __syncthreads();
    for (int t = threadIdx.x; t < NCT * TC; t += kThreads) {
      const int64_t j = c_lo + t;
      if (j >= p.cols) break;
      T s = sm[0][t];
#pragma unroll
      for (int w = 1; w < kWarps; ++w) s += sm[w][t];
      if (p.direct) {
        T* yp = p.y + j * p.incy;
        B2_STORE(yp, p.beta != T(0) ? p.alpha * s + p.beta * *yp : p.alpha * s);
      } else {
        p.colpart[rs * p.cols + j] = s;
      }
    }
  }
}

// Adds the partials of each output in a fixed order and writes y = alpha*sum + beta*y.
// A block handles 256/SLICES consecutive outputs; SLICES threads share one output and split
// its list of partials (slice k takes partials k, k+SLICES, ...), then combine through shared
// memory in slice order.  Launched as a programmatic dependent of the tile kernel.
template <typename T, class K, int SLICES>
__global__ void __launch_bounds__(kThreads) l2_finalize(const L2Args<T> p, int RB, int TC) {
  constexpr int OUTB = kThreads / SLICES;
  __shared__ T sm[SLICES][OUTB];
  grid_dep_wait();
  grid_dep_launch();
  const int o = threadIdx.x % OUTB, slice = threadIdx.x / OUTB;
  const int64_t nout = K::ROWOUT ? p.rows : p.cols;
  const int64_t i = (int64_t)blockIdx.x * OUTB + o;
  T s = T(0);
  if (i < nout) {
    if (K::ROWOUT) {
      const int64_t rs = i / p.rows_per_cta;
      const int64_t r_end = min(p.rows, (rs + 1) * p.rows_per_cta);
      const int64_t rb = (i / RB) * RB;  // rows_per_cta is a multiple of RB
      const int64_t rb_end = min(rb + RB, r_end);
      // four partials per trip, their loads issued together (a load behind each test would
      // cost one L2 round trip per partial); added in the same order as one by one
      if constexpr (K::TRI == TRI_FULL) {  // every partial exists: a plain loop, which the compiler pipelines
        for (int cs = slice; cs < p.ncs; cs += SLICES) s += __ldcg(p.rowpart + (int64_t)cs * p.rows + i);
      } else
      for (int cs0 = slice; cs0 < p.ncs; cs0 += 4 * SLICES) {
        T v[4];
        bool act[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int cs = cs0 + k * SLICES;
          const int64_t c_lo = (int64_t)cs * p.ctiles_per_cta * TC;
          const int64_t c_hi = min(p.cols, c_lo + (int64_t)p.ctiles_per_cta * TC);
          act[k] = cs < p.ncs && region_active<K::TRI>(rb, rb_end, c_lo, c_hi);
          v[k] = act[k] ? __ldcg(p.rowpart + (int64_t)cs * p.rows + i) : T(0);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (act[k]) s += v[k];
      }
    }
    if (K::COLOUT) {
      const int64_t span = (int64_t)TC * p.ctiles_per_cta;  // columns of one block
      const int64_t c_lo = (i / span) * span, c_hi = min(p.cols, c_lo + span);
      if constexpr (K::TRI == TRI_FULL) {
        for (int64_t rs = slice; rs < p.nrs; rs += SLICES) s += __ldcg(p.colpart + rs * p.cols + i);
      } else
      for (int64_t rs0 = slice; rs0 < p.nrs; rs0 += 4 * SLICES) {
        T v[4];
        bool act[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int64_t rs = rs0 + k * SLICES;
          const int64_t r_begin = rs * p.rows_per_cta, r_end = min(p.rows, r_begin + p.rows_per_cta);
          act[k] = rs < p.nrs && region_active<K::TRI>(r_begin, r_end, c_lo, c_hi);
          v[k] = act[k] ? __ldcg(p.colpart + rs * p.cols + i) : T(0);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (act[k]) s += v[k];
      }
    }
  }
  if (SLICES > 1) {
    sm[slice][o] = s;
    __syncthreads();
    if (slice != 0) return;
#pragma unroll
    for (int k = 1; k < SLICES; ++k) s += sm[k][o];
  }
  if (i < nout) {
    T* yp = p.y + i * p.incy;
    B2_STORE(yp, p.beta != T(0) ? p.alpha * s + p.beta * *yp : p.alpha * s);
  }
}

// y <- beta*y (alpha == 0 shortcut); beta == 0 writes zeros without reading.
template <typename T>
__global__ void __launch_bounds__(kThreads) l2_scale_y(T* y, int64_t incy, int64_t n, T beta) {
  grid_dep_wait();
  grid_dep_launch();
  const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (i < n) y[i * incy] = beta == T(0) ? T(0) : beta * y[i * incy];
}

// ------------------------------------------------------------------------------- host side
struct L2Plan {
  int shape;             // index into the shape table
  int64_t rows_per_cta;  // multiple of the shape's RB
  int ctiles_per_cta;
};

template <typename T, class K, int SLICES>
static void launch_finalize(const Launch& l, const L2Args<T>& args, int RB, int TC, int64_t nout) {
  constexpr int OUTB = kThreads / SLICES;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((nout + OUTB - 1) / OUTB));
  cfg.blockDim = dim3(kThreads);
  cfg.stream = l.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = knob(kKnobUsePdl) ? 1 : 0;
  cudaLaunchKernelEx(&cfg, l2_finalize<T, K, SLICES>, args, RB, TC);
}

// Launches the tile kernel (+ finalize when partials are needed) for one shape.
template <typename T, int V, class K, class S>
static int l2_launch_shape(const Launch& l, L2Args<T> args, int64_t rows_per_cta, int ctiles_per_cta,
                           bool allow_direct) {
  constexpr int TC = S::template tc<V>();
  constexpr int RB = S::RB;
  args.nct = (int)((args.cols + TC - 1) / TC);
  args.xc_vec = (K::ROWOUT && V > 1 && aligned_to(args.xc, 16)) ? (args.incxc == 1 ? 1 : args.incxc == 2 ? 2 : 0) : 0;
  if (K::COLOUT) ctiles_per_cta = S::NCT;
  if (ctiles_per_cta < 1) ctiles_per_cta = 1;
  if (ctiles_per_cta > args.nct) ctiles_per_cta = args.nct;
  rows_per_cta = ((rows_per_cta + RB - 1) / RB) * RB;
  if (rows_per_cta < RB) rows_per_cta = RB;
  for (;;) {  // shrink the number of partials until they fit the workspace
    args.rows_per_cta = rows_per_cta;
    args.ctiles_per_cta = ctiles_per_cta;
    args.nrs = (int)((args.rows + rows_per_cta - 1) / rows_per_cta);
    args.ncs = (args.nct + ctiles_per_cta - 1) / ctiles_per_cta;
    const bool single = (!K::ROWOUT || args.ncs == 1) && (!K::COLOUT || args.nrs == 1) && !(K::ROWOUT && K::COLOUT);
    args.direct = allow_direct && single;
    if (args.direct) break;
    size_t need = 0;
    if (K::ROWOUT) need += (size_t)args.ncs * args.rows * sizeof(T);
    const size_t row_bytes = (need + 255) / 256 * 256;
    if (K::COLOUT) need = row_bytes + (size_t)args.nrs * args.cols * sizeof(T);
    if (need <= l.scratch_bytes) {
      args.rowpart = reinterpret_cast<T*>(l.scratch);
      args.colpart = reinterpret_cast<T*>(l.scratch + row_bytes);
      break;
    }
    // (a block of a column-sum kind walks exactly S::NCT column tiles -- their sums sit in its
    // registers -- so only its row band can grow; a row-dot kind merges column splits)
    bool changed = false;
    if (K::ROWOUT && !K::COLOUT && ctiles_per_cta < args.nct) ctiles_per_cta *= 2, changed = true;
    if (ctiles_per_cta > args.nct) ctiles_per_cta = args.nct;
    if (K::COLOUT && rows_per_cta < args.rows) rows_per_cta *= 2, changed = true;
    if (!changed) return B2_STATUS_WORKSPACE_TOO_SMALL;
  }
  const int64_t nblocks = (int64_t)args.nrs * args.ncs;
  if (nblocks > 0x7fffffff) return B2_STATUS_NOT_IMPLEMENTED;
  launch_chained(l2_tile_kernel<T, V, K, S>, dim3((unsigned)nblocks), dim3(kThreads), 0, l.stream, args);
  if (int st = check_launch()) return st;
  if (!args.direct) {
    const int64_t nout = K::ROWOUT ? args.rows : args.cols;
    const int nparts = (K::ROWOUT ? args.ncs : 0) + (K::COLOUT ? args.nrs : 0);
    if (nparts >= 512) launch_finalize<T, K, 32>(l, args, RB, TC, nout);
    else if (nparts >= 12) launch_finalize<T, K, 8>(l, args, RB, TC, nout);
    else launch_finalize<T, K, 1>(l, args, RB, TC, nout);
    if (int st = check_launch()) return st;
  }
  return B2_STATUS_OK;
}

// Shape table shared by all kinds.
using ShapeWide = Shape<32, 4, 2>;    // 2 KiB row segments, 16 rows per step
using ShapeMid = Shape<32, 1, 8>;     // 512 B row segments, 64 rows per step
using ShapeHalf = Shape<16, 1, 8>;    // 256 B row segments, 128 rows per step
using ShapeQuarter = Shape<8, 1, 8>;  // 128 B row segments, 256 rows per step
enum { SHAPE_WIDE = 0, SHAPE_MID = 1, SHAPE_HALF = 2, SHAPE_QUARTER = 3 };

inline int shape_rb(int shape) {
  switch (shape) {
    case SHAPE_WIDE: return ShapeWide::RB;
    case SHAPE_MID: return ShapeMid::RB;
    case SHAPE_HALF: return ShapeHalf::RB;
    default: return ShapeQuarter::RB;
  }
}
inline int shape_packs_per_row(int shape) {  // packs of one row segment
  switch (shape) {
    case SHAPE_WIDE: return 128;
    case SHAPE_MID: return 32;
    case SHAPE_HALF: return 16;
    default: return 8;
  }
}

// NARROW = false drops the two narrow shapes (kinds that never use them compile faster).
template <typename T, int V, class K, bool NARROW>
static int l2_launch(const Launch& l, const L2Args<T>& args, const L2Plan& plan, bool allow_direct) {
  if (plan.shape == SHAPE_WIDE)
    return l2_launch_shape<T, V, K, ShapeWide>(l, args, plan.rows_per_cta, plan.ctiles_per_cta, allow_direct);
  if constexpr (NARROW) {
    if (plan.shape == SHAPE_HALF)
      return l2_launch_shape<T, V, K, ShapeHalf>(l, args, plan.rows_per_cta, plan.ctiles_per_cta, allow_direct);
    if (plan.shape == SHAPE_QUARTER)
      return l2_launch_shape<T, V, K, ShapeQuarter>(l, args, plan.rows_per_cta, plan.ctiles_per_cta, allow_direct);
  }
  return l2_launch_shape<T, V, K, ShapeMid>(l, args, plan.rows_per_cta, plan.ctiles_per_cta, allow_direct);
}

// Picks the pack width: 16-byte packs need a 16-byte aligned base and row stride.
template <typename T, class K, bool NARROW>
static int l2_dispatch(const Launch& l, const L2Args<T>& args, const L2Plan& plan, bool allow_direct) {
  constexpr int V = VecLen<T>::value;
  if (aligned_to(args.a, 16) && args.lda % V == 0) return l2_launch<T, V, K, NARROW>(l, args, plan, allow_direct);
  return l2_launch<T, 1, K, NARROW>(l, args, plan, allow_direct);
}

// Plans.  ROWOUT-only kinds: one row step per block, several column tiles per block so that a
// block streams about `tile_bytes`; the remaining column splits become partials.
template <typename T>
static L2Plan plan_rowout(const L2Args<T>& a, bool narrow_ok) {
  const int V = (aligned_to(a.a, 16) && a.lda % VecLen<T>::value == 0) ? VecLen<T>::value : 1;
  const int64_t nv = (a.cols + V - 1) / V;
  L2Plan p;
  p.shape = nv >= 128 ? SHAPE_WIDE : (nv > 16 || !narrow_ok) ? SHAPE_MID : nv > 8 ? SHAPE_HALF : SHAPE_QUARTER;
  const int64_t tile_bytes = (int64_t)shape_rb(p.shape) * shape_packs_per_row(p.shape) * V * sizeof(T);
  int64_t cpc = knob(kKnobGemvNTileBytes) / tile_bytes;
  if (cpc < 1) cpc = 1;
  // A matrix of a few long rows (at most 8 row steps) would get one partial per column split
  // and a finalize pass that adds thousands of them per row: there the splits are limited to
  // about eight resident blocks per SM in all.
  const int64_t nrs = (a.rows + shape_rb(p.shape) - 1) / shape_rb(p.shape);
  if (nrs <= 8) {
    const int64_t nct = (nv + shape_packs_per_row(p.shape) - 1) / shape_packs_per_row(p.shape);
    const int64_t want_ncs = std::max<int64_t>(1, (int64_t)sm_count() * 8 / nrs);
    cpc = std::max(cpc, (nct + want_ncs - 1) / want_ncs);
  }
  p.ctiles_per_cta = (int)cpc;
  p.rows_per_cta = shape_rb(p.shape);
  return p;
}
// COLOUT kinds: one column tile per block, tall row bands; the bands become partials.
template <typename T>
static L2Plan plan_colout(const L2Args<T>& a, bool narrow_ok, int64_t rows_per_cta) {
  const int V = (aligned_to(a.a, 16) && a.lda % VecLen<T>::value == 0) ? VecLen<T>::value : 1;
  const int64_t nv = (a.cols + V - 1) / V;
  L2Plan p;
  p.shape = (nv > 16 || !narrow_ok) ? SHAPE_MID : nv > 8 ? SHAPE_HALF : SHAPE_QUARTER;
  // element-wise rows (not 16-byte aligned): a 32-element column tile makes tiny blocks, take 128
  if (V == 1 && nv >= 128) p.shape = SHAPE_WIDE;
  p.ctiles_per_cta = 1;
  if ((a.rows + rows_per_cta - 1) / rows_per_cta > 1024) rows_per_cta = (a.rows + 1023) / 1024;
  p.rows_per_cta = rows_per_cta;
  return p;
}

template <typename T>
static int scale_y(const Launch& l, T* y, int64_t incy, int64_t n, T beta) {
  if (beta == T(1) || n == 0) return B2_STATUS_OK;
  launch_chained(l2_scale_y<T>, dim3((unsigned)((n + kThreads - 1) / kThreads)), dim3(kThreads), 0, l.stream, vec_base(y, n, incy), incy, n, beta);
  return check_launch();
}

}  // namespace b2
