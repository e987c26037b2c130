// Narrow-matrix kernels for gemv (row-dot kind) and ger (Section 6.2.2 of the paper: a separate
// schedule for matrices whose row is a few vector registers long, with the reused vector staged
// once and static sizes up to 88 floats / 44 doubles).
//
// Setting: the canonical row-major view has many rows and a row of PPR 16-byte packs, PPR <= 22,
// stored without padding (lda == cols), so the whole matrix is ONE contiguous stream of packs and
// a pack never straddles two rows.  The general tile kernel gives each row its own group of 8,
// 16 or 32 lanes; at 10 or 11 packs per row a third of the lanes idle.  Here a warp instead takes
// "chunks" of 32 rows = 32 * PPR consecutive packs and reads them with PPR fully coalesced
// instructions: lane l, instruction k holds pack k*32 + l of the chunk, which belongs to row
// (k*32 + l) / PPR and column pack (k*32 + l) % PPR.  Neither quotient is computed by a division:
// both advance by fixed steps from one instruction to the next.
//   row-dot: each pack is multiplied with its slice of x (shared memory) into one partial, the
//            partials go to shared memory in stream order, and lane l then adds the PPR
//            partials of row l -- a segmented sum without any cross-lane traffic.
//   ger:     lane l holds alpha * x of row l of the chunk; a pack gets its row's value by a
//            shuffle and its slice of y from shared memory.
#pragma once

#include "common.cuh"

namespace b2 {

constexpr int kSkinnyMaxPpr = 22;       // 88 floats / 44 doubles per row
constexpr int kSkinnyGroup = 11;        // packs of a lane in flight together: a chunk is one or two groups
constexpr int64_t kSkinnyMinRows = 2048;

// True when the flat-stream kernels apply and pay: few packs per row, no padding, aligned base,
// and a row length that leaves more than 30 % of the lanes idle in the general kernel (which
// gives a row 8, 16 or 32 lanes).  Measured on 2^20-row matrices: at 10 and 22 packs per row the
// flat kernels win (float row-dot 0.71 -> 0.80 and 0.87 -> 0.92 of the copy rate, ger 0.72 ->
// 0.83), at 12 packs (75 % of the lanes busy) they lose.  The double row-dot is slower flat at
// every width measured (0.51 against 0.63): it stays on the general kernel.
template <typename T>
static bool skinny_applies(const T* a, int64_t lda, int64_t rows, int64_t cols, bool rowdot) {
  constexpr int V = VecLen<T>::value;
  if (rowdot && sizeof(T) == 8) return false;
  if (rows < kSkinnyMinRows || cols != lda || cols % V != 0 || !aligned_to(a, 16)) return false;
  const int64_t ppr = cols / V;
  if (ppr < 1 || ppr > kSkinnyMaxPpr) return false;
  const int64_t lanes = ppr <= 8 ? 8 : ppr <= 16 ? 16 : 32;
  return 10 * ppr < 7 * lanes;
}

// y_i <- alpha * sum_j a_ij x_j + beta * y_i over a flat pack stream.  x, y: vec_base() bases.
template <typename T>
__global__ void __launch_bounds__(kThreads, 3) skinny_rowdot_kernel(const T* __restrict__ a, int64_t rows, int ppr,
                                                                    const T* __restrict__ x, int64_t incx, T alpha,
                                                                    T beta, T* __restrict__ y, int64_t incy,
                                                                    int64_t nchunks) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int V = VecLen<T>::value;
  using P = Pack<T, V>;
  __shared__ __align__(16) T xs[kSkinnyMaxPpr * V];
  __shared__ T part[kWarps][(kSkinnyMaxPpr + 1) * 32];  // row r at r * (ppr | 1): an odd pitch spreads the banks
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = threadIdx.x; t < ppr * V; t += kThreads) xs[t] = __ldg(x + t * incx);
  __syncthreads();
  const int cstep = 32 % ppr, rstep = 32 / ppr;  // per instruction: column pack += cstep (mod ppr), row += rstep (+ carry)
  const int c_first = lane % ppr, r_first = lane / ppr;
  const int pitch = ppr | 1;
  for (int64_t chunk = (int64_t)blockIdx.x * kWarps + warp; chunk < nchunks; chunk += (int64_t)gridDim.x * kWarps) {
    const int64_t row0 = chunk * 32;
    const int nrows = (int)min((int64_t)32, rows - row0);
    const int npacks = nrows * ppr;  // packs of this chunk that exist
    const P* src = reinterpret_cast<const P*>(a) + row0 * ppr;
    int c = c_first, r = r_first;
    for (int k0 = 0; k0 < ppr; k0 += kSkinnyGroup) {
      P av[kSkinnyGroup];
#pragma unroll
      for (int g = 0; g < kSkinnyGroup; ++g) {
        const int pos = (k0 + g) * 32 + lane;
        av[g] = ld_nc_if<T, V>(reinterpret_cast<const T*>(src + pos), k0 + g < ppr && pos < npacks);
      }
#pragma unroll
      for (int g = 0; g < kSkinnyGroup; ++g) {
        const int pos = (k0 + g) * 32 + lane;
        if (k0 + g < ppr) {
          T s = T(0);
          if (pos < npacks) {
            const P xv = *reinterpret_cast<const P*>(&xs[c * V]);
#pragma unroll
            for (int e = 0; e < V; ++e) s = av[g].v[e] * xv.v[e] + s;
          }
          part[warp][r * pitch + c] = s;
          c += cstep;
          r += rstep;
          if (c >= ppr) {
            c -= ppr;
            r += 1;
          }
        }
      }
    }
    __syncwarp();
    if (lane < nrows) {
      T s = T(0);
      for (int k = 0; k < ppr; ++k) s += part[warp][lane * pitch + k];
      T* yp = y + (row0 + lane) * incy;
      *yp = beta != T(0) ? alpha * s + beta * *yp : alpha * s;
    }
    __syncwarp();  // part is rewritten by the next chunk
  }
}

// a_ij <- alpha * x_i * y_j + a_ij over a flat pack stream.  xr indexed by row, yc by column.
template <typename T>
__global__ void __launch_bounds__(kThreads, 3) skinny_ger_kernel(T* __restrict__ a, int64_t rows, int ppr,
                                                                 const T* __restrict__ xr, int64_t incxr,
                                                                 const T* __restrict__ yc, int64_t incyc, T alpha,
                                                                 int64_t nchunks) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int V = VecLen<T>::value;
  using P = Pack<T, V>;
  __shared__ __align__(16) T ys[kSkinnyMaxPpr * V];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = threadIdx.x; t < ppr * V; t += kThreads) ys[t] = __ldg(yc + t * incyc);
  __syncthreads();
  const int cstep = 32 % ppr, rstep = 32 / ppr;  // per instruction: column pack += cstep (mod ppr), row += rstep (+ carry)
  const int c_first = lane % ppr, r_first = lane / ppr;
  for (int64_t chunk = (int64_t)blockIdx.x * kWarps + warp; chunk < nchunks; chunk += (int64_t)gridDim.x * kWarps) {
    const int64_t row0 = chunk * 32;
    const int nrows = (int)min((int64_t)32, rows - row0);
    const int npacks = nrows * ppr;
    P* dst = reinterpret_cast<P*>(a) + row0 * ppr;
    const T xrow = lane < nrows ? alpha * __ldg(xr + (row0 + lane) * incxr) : T(0);
    int c = c_first, r = r_first;
    for (int k0 = 0; k0 < ppr; k0 += kSkinnyGroup) {
      P av[kSkinnyGroup];
#pragma unroll
      for (int g = 0; g < kSkinnyGroup; ++g) {
        const int pos = (k0 + g) * 32 + lane;
        if (k0 + g < ppr && pos < npacks) av[g] = ld_cg<T, V>(reinterpret_cast<const T*>(dst + pos));
      }
#pragma unroll
      for (int g = 0; g < kSkinnyGroup; ++g) {
        const int pos = (k0 + g) * 32 + lane;
        if (k0 + g < ppr) {  // uniform over the warp: the shuffle below is executed by all lanes
          const T xi = __shfl_sync(0xffffffffu, xrow, r & 31);
          if (pos < npacks) {
            const P yv = *reinterpret_cast<const P*>(&ys[c * V]);
#pragma unroll
            for (int e = 0; e < V; ++e) av[g].v[e] = xi * yv.v[e] + av[g].v[e];
            st_cs<T, V>(reinterpret_cast<T*>(dst + pos), av[g]);
          }
          c += cstep;
          r += rstep;
          if (c >= ppr) {
            c -= ppr;
            r += 1;
          }
        }
      }
    }
  }
}

// Column sums of a narrow matrix (the gemv kind whose output has one entry per column):
// colpart[block][j] = sum over the block's rows of a_ij * x_i.  A lane's column must not change
// from load to load (its sums live in registers), so here a row gets exactly PPR lanes: a warp
// instruction covers G = 32 / PPR whole rows with its first G * PPR lanes -- 30 of 32 lanes at 10
// packs per row, where power-of-two row groups would use 20.  The loads of one instruction are
// still one contiguous run of packs.  Each block leaves one partial row; the general finalize
// kernel adds the partials in a fixed order and applies alpha / beta.
constexpr int kColsumGroup = 8;  // instructions of a lane in flight together

template <typename T>
__global__ void __launch_bounds__(kThreads, 4) skinny_colsum_kernel(const T* __restrict__ a, int64_t rows, int ppr,
                                                                    const T* __restrict__ xr, int64_t incxr,
                                                                    T* __restrict__ colpart, int64_t nsteps) {
  constexpr int V = VecLen<T>::value;
  using P = Pack<T, V>;
  __shared__ T sm[kWarps][32 * V];
  grid_dep_wait();
  grid_dep_launch();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = 32 / ppr;
  const bool active = lane < G * ppr;
  const int g = lane / ppr;  // row of this lane inside an instruction (valid when active)
  const int64_t rows_per_step = (int64_t)G * kColsumGroup;
  T acc[V];
#pragma unroll
  for (int e = 0; e < V; ++e) acc[e] = T(0);
  for (int64_t step = (int64_t)blockIdx.x * kWarps + warp; step < nsteps; step += (int64_t)gridDim.x * kWarps) {
    const int64_t row0 = step * rows_per_step;
    const P* src = reinterpret_cast<const P*>(a) + row0 * ppr + lane;
    P av[kColsumGroup];
    T xv[kColsumGroup];
#pragma unroll
    for (int k = 0; k < kColsumGroup; ++k) {
      const int64_t row = row0 + k * G + g;
      const bool ok = active && row < rows;
      av[k] = ld_nc_if<T, V>(reinterpret_cast<const T*>(src + (int64_t)k * G * ppr), ok);
      xv[k] = ok ? __ldg(xr + row * incxr) : T(0);
    }
#pragma unroll
    for (int k = 0; k < kColsumGroup; ++k)
#pragma unroll
      for (int e = 0; e < V; ++e) acc[e] = av[k].v[e] * xv[k] + acc[e];
  }
  // lanes g * ppr + q (all g, all warps) hold partial sums of column pack q
#pragma unroll
  for (int e = 0; e < V; ++e) sm[warp][lane * V + e] = active ? acc[e] : T(0);
  __syncthreads();
  for (int j = threadIdx.x; j < ppr * V; j += kThreads) {
    const int q = j / V, e = j % V;
    T s = T(0);
    for (int w = 0; w < kWarps; ++w)
      for (int gg = 0; gg < G; ++gg) s += sm[w][(gg * ppr + q) * V + e];
    colpart[(int64_t)blockIdx.x * (ppr * V) + j] = s;
  }
}

// Exact-width row groups pay when they keep clearly more lanes busy than the general kernel's
// power-of-two groups (a margin of 15 % of the warp).
template <typename T>
static bool skinny_colsum_applies(const T* a, int64_t lda, int64_t rows, int64_t cols) {
  constexpr int V = VecLen<T>::value;
  if (rows < kSkinnyMinRows || cols != lda || cols % V != 0 || !aligned_to(a, 16)) return false;
  const int64_t ppr = cols / V;
  if (ppr < 1 || ppr > 16) return false;
  const int64_t lanes = ppr <= 8 ? 8 : 16;          // the general kernel's row group
  const int64_t busy = (32 / ppr) * ppr;            // lanes busy here, of 32
  return 100 * busy >= 100 * 32 * ppr / lanes + 15 * 32;
}

// Block-wide forms of the two gemv kinds for any row length up to kBlockMaxPpr packs: a row gets
// exactly PPR THREADS of the block (not lanes of one warp), so K = 256 / PPR whole rows are one
// contiguous run of K * PPR packs per step -- 240 of 256 threads at 20 packs per row, where a warp
// on its own would use 20 of its 32 lanes.  A thread's column pack never changes: its slice of x
// (row-dot) or its column sums (column kind) stay in registers.  kBlockUnroll steps are in flight.
constexpr int kBlockMaxPpr = 64;
constexpr int kBlockUnroll = 8;

// y_i <- alpha * sum_j a_ij x_j + beta * y_i.  Per pack one partial; the PPR partials of a row meet
// in shared memory (odd pitch), where one thread per row adds them in column order.
template <typename T>
__global__ void __launch_bounds__(kThreads, 3) block_rowdot_kernel(const T* __restrict__ a, int64_t rows, int ppr,
                                                                   const T* __restrict__ x, int64_t incx, T alpha,
                                                                   T beta, T* __restrict__ y, int64_t incy,
                                                                   int64_t nsteps) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int V = VecLen<T>::value, U = kBlockUnroll;
  using P = Pack<T, V>;
  extern __shared__ __align__(16) unsigned char block_smem[];
  T* part = reinterpret_cast<T*>(block_smem);  // [U][K * pitch]
  const int t = (int)threadIdx.x, K = kThreads / ppr, G = K * ppr, pitch = ppr | 1;
  const bool active = t < G;
  const int c = t % ppr, r = t / ppr;
  T xv[V];
#pragma unroll
  for (int e = 0; e < V; ++e) xv[e] = active ? __ldg(x + (int64_t)(c * V + e) * incx) : T(0);
  const int64_t rows_per_step = (int64_t)K * U;
  for (int64_t step = blockIdx.x; step < nsteps; step += gridDim.x) {
    const int64_t row0 = step * rows_per_step;
    const P* src = reinterpret_cast<const P*>(a) + row0 * ppr + t;
    P av[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      // (double: the branch-free load, 0.82 -> 0.92 of the copy rate at 40 columns; float measured
      // 5 % faster with the branch, which the compiler there turns into a predicate itself)
      if constexpr (sizeof(T) == 8) {
        av[u] = ld_nc_if<T, V>(reinterpret_cast<const T*>(src + (int64_t)u * G), active && row0 + u * K + r < rows);
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e) av[u].v[e] = T(0);
        if (active && row0 + u * K + r < rows) av[u] = ld_nc<T, V>(reinterpret_cast<const T*>(src + (int64_t)u * G));
      }
    }
    if (active) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        T s = T(0);
#pragma unroll
        for (int e = 0; e < V; ++e) s = av[u].v[e] * xv[e] + s;
        part[(u * K + r) * pitch + c] = s;
      }
    }
    __syncthreads();
    for (int j = t; j < K * U; j += kThreads) {
      const int64_t row = row0 + j;  // (slot j = u * K + r holds row row0 + u * K + r)
      if (row < rows) {
        T s = T(0);
        for (int q = 0; q < ppr; ++q) s += part[j * pitch + q];
        T* yp = y + row * incy;
        B2_STORE(yp, beta != T(0) ? alpha * s + beta * *yp : alpha * s);
      }
    }
    __syncthreads();  // part is rewritten by the next step
  }
}

// colpart[block][j] = sum over the block's rows of a_ij * x_i (the general finalize kernel adds
// the blocks' rows in a fixed order and applies alpha / beta).
template <typename T>
__global__ void __launch_bounds__(kThreads, 4) block_colsum_kernel(const T* __restrict__ a, int64_t rows, int ppr,
                                                                   const T* __restrict__ xr, int64_t incxr,
                                                                   T* __restrict__ colpart, int64_t nsteps) {
  constexpr int V = VecLen<T>::value, U = kBlockUnroll;
  using P = Pack<T, V>;
  __shared__ T sm[kThreads * V];
  grid_dep_wait();
  grid_dep_launch();
  const int t = (int)threadIdx.x, K = kThreads / ppr, G = K * ppr;
  const bool active = t < G;
  const int r = t / ppr;
  const int64_t rows_per_step = (int64_t)K * U;
  T acc[V];
#pragma unroll
  for (int e = 0; e < V; ++e) acc[e] = T(0);
  for (int64_t step = blockIdx.x; step < nsteps; step += gridDim.x) {
    const int64_t row0 = step * rows_per_step;
    const P* src = reinterpret_cast<const P*>(a) + row0 * ppr + t;
    P av[U];
    T xv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t row = row0 + u * K + r;
      av[u] = ld_nc_if<T, V>(reinterpret_cast<const T*>(src + (int64_t)u * G), active && row < rows);
      xv[u] = (active && row < rows) ? __ldg(xr + row * incxr) : T(0);
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int e = 0; e < V; ++e) acc[e] = av[u].v[e] * xv[u] + acc[e];
  }
  // threads rr * ppr + q (all rr) hold partial sums of column pack q
#pragma unroll
  for (int e = 0; e < V; ++e) sm[t * V + e] = active ? acc[e] : T(0);
  __syncthreads();
  for (int j = t; j < ppr * V; j += kThreads) {
    const int q = j / V, e = j % V;
    T s = T(0);
    for (int rr = 0; rr < K; ++rr) s += sm[(rr * ppr + q) * V + e];
    colpart[(int64_t)blockIdx.x * (ppr * V) + j] = s;
  }
}

// The block-wide kernels apply to unpadded, 16-byte aligned matrices of many narrow rows.
template <typename T>
static bool block_narrow_applies(const T* a, int64_t lda, int64_t rows, int64_t cols) {
  constexpr int V = VecLen<T>::value;
  if (rows < kSkinnyMinRows || cols != lda || cols % V != 0 || !aligned_to(a, 16)) return false;
  const int64_t ppr = cols / V;
  return ppr >= 1 && ppr <= kBlockMaxPpr;
}

template <typename T>
static int block_rowdot(const Launch& l, const T* a, int64_t rows, int64_t cols, const T* x, int64_t incx, T alpha,
                        T beta, T* y, int64_t incy) {
  const int ppr = (int)(cols / VecLen<T>::value), K = kThreads / ppr;
  const int64_t nsteps = (rows + (int64_t)K * kBlockUnroll - 1) / ((int64_t)K * kBlockUnroll);
  const int64_t cap = (int64_t)sm_count() * 3;
  const size_t smem = sizeof(T) * (size_t)kBlockUnroll * K * (ppr | 1);
  launch_chained(block_rowdot_kernel<T>, dim3((unsigned)(nsteps < cap ? nsteps : cap)), dim3(kThreads), smem, l.stream, a, rows, ppr, x, incx, alpha,
                                                                                          beta, y, incy, nsteps);
  return check_launch();
}

// The transposed shape: a canonical view of FEW (<= kWideMaxRows) very long rows -- what a narrow
// column-major matrix looks like.  A thread owns columns and walks down the few rows, so every
// load instruction of a warp is one contiguous run of a row whatever the alignment of the rows
// (an odd leading dimension puts every second row off the 16-byte boundary: element loads do not
// care), nothing is reduced across lanes, and x is staged once.  (The row-dot kind of this shape
// stays on the general kernel: a column-owning form of it measured no faster.)
constexpr int kWideMaxRows = 64;
constexpr int64_t kWideMinCols = 1 << 15;

template <typename T>
static bool wide_applies(int64_t rows, int64_t cols) {
  return rows >= 1 && rows <= kWideMaxRows && cols >= kWideMinCols;
}

// y_j <- alpha * sum_i a_ij x_i + beta * y_j (one output per column, written directly).
template <typename T>
__global__ void __launch_bounds__(kThreads) wide_colsum_kernel(const T* __restrict__ a, int64_t lda, int rows, int64_t cols,
                                                               const T* __restrict__ xr, int64_t incxr, T alpha, T beta,
                                                               T* __restrict__ y, int64_t incy) {
  grid_dep_wait();
  grid_dep_launch();
  __shared__ T xs[kWideMaxRows];
  if (threadIdx.x < rows) xs[threadIdx.x] = __ldg(xr + threadIdx.x * incxr);
  __syncthreads();
  for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < cols; j += (int64_t)gridDim.x * kThreads) {
    const T* col = a + j;
    T acc = T(0);
    int i = 0;
    for (; i + 8 <= rows; i += 8) {
      T v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = __ldg(col + (int64_t)(i + k) * lda);
#pragma unroll
      for (int k = 0; k < 8; ++k) acc = v[k] * xs[i + k] + acc;
    }
    for (; i < rows; ++i) acc = __ldg(col + (int64_t)i * lda) * xs[i] + acc;
    T* yp = y + j * incy;
    B2_STORE(yp, beta != T(0) ? alpha * acc + beta * *yp : alpha * acc);
  }
}

// a_ij <- alpha * x_i * y_j + a_ij, x indexed by the few rows, y by the many columns.
template <typename T>
__global__ void __launch_bounds__(kThreads) wide_ger_kernel(T* __restrict__ a, int64_t lda, int rows, int64_t cols,
                                                            const T* __restrict__ xr, int64_t incxr,
                                                            const T* __restrict__ yc, int64_t incyc, T alpha) {
  grid_dep_wait();
  grid_dep_launch();
  __shared__ T xs[kWideMaxRows];
  if (threadIdx.x < rows) xs[threadIdx.x] = alpha * __ldg(xr + threadIdx.x * incxr);
  __syncthreads();
  for (int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x; j < cols; j += (int64_t)gridDim.x * kThreads) {
    T* col = a + j;
    const T yj = __ldg(yc + j * incyc);
    int i = 0;
    for (; i + 8 <= rows; i += 8) {
      T v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = __ldcg(col + (int64_t)(i + k) * lda);
#pragma unroll
      for (int k = 0; k < 8; ++k) __stcs(col + (int64_t)(i + k) * lda, xs[i + k] * yj + v[k]);
    }
    for (; i < rows; ++i) __stcs(col + (int64_t)i * lda, xs[i] * yj + __ldcg(col + (int64_t)i * lda));
  }
}

template <typename T>
static int skinny_grid(int64_t nchunks) {
  const int64_t blocks = (nchunks + kWarps - 1) / kWarps;
  const int64_t cap = (int64_t)sm_count() * 3;  // one resident wave (three blocks per SM)
  return (int)(blocks < cap ? blocks : cap);
}

template <typename T>
static int skinny_rowdot(const Launch& l, const T* a, int64_t rows, int64_t cols, const T* x, int64_t incx, T alpha,
                         T beta, T* y, int64_t incy) {
  const int ppr = (int)(cols / VecLen<T>::value);
  const int64_t nchunks = (rows + 31) / 32;
  launch_chained(skinny_rowdot_kernel<T>, dim3(skinny_grid<T>(nchunks)), dim3(kThreads), 0, l.stream, a, rows, ppr, x, incx, alpha, beta, y,
                                                                             incy, nchunks);
  return check_launch();
}

template <typename T>
static int skinny_ger(const Launch& l, T* a, int64_t rows, int64_t cols, const T* xr, int64_t incxr, const T* yc,
                      int64_t incyc, T alpha) {
  const int ppr = (int)(cols / VecLen<T>::value);
  const int64_t nchunks = (rows + 31) / 32;
  launch_chained(skinny_ger_kernel<T>, dim3(skinny_grid<T>(nchunks)), dim3(kThreads), 0, l.stream, a, rows, ppr, xr, incxr, yc, incyc, alpha,
                                                                          nchunks);
  return check_launch();
}

}  // namespace b2
