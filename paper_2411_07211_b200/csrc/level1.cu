// BLAS level-1 kernels (Section 6.2.1 of the paper: single-loop O(n) operations).
//
// Two templates generate every variant:
//   * l1_map<T, Op>     : axpy, scal, copy, swap, rot      (elementwise, memory streaming)
//   * l1_reduce<T, Op>  : dot, asum, nrm2, iamax           (per-lane partial sums -> warp
//                         shuffle -> block -> deterministic second pass by the last block)
// each in a unit-stride flavour (128-bit coalesced packs, scalar head/tail peel when the
// pointers are not 16-byte aligned) and a strided flavour (any non-zero increment).
// The paper's level-1 recipe (Appendix D.1: vectorise, hoist invariants, interleave for ILP,
// predicated tail) maps onto: 128-bit packs, scalars in registers, NV independent packs in
// flight per thread, bounds-predicated last chunk.
#include "common.cuh"

namespace b2 {

// ------------------------------------------------------------------------------- map ops
// RX/RY: the op reads x / y; WX/WY: it writes x / y.
template <typename T>
struct AxpyOp {
  T a;
  static constexpr bool RX = true, RY = true, WX = false, WY = true;
  __device__ __forceinline__ void operator()(T& x, T& y) const { y = a * x + y; }
};
template <typename T>
struct ScalOp {
  T a;
  static constexpr bool RX = true, RY = false, WX = true, WY = false;
  __device__ __forceinline__ void operator()(T& x, T&) const { x = a * x; }  // one IEEE multiply
};
template <typename T>
struct CopyOp {
  static constexpr bool RX = true, RY = false, WX = false, WY = true;
  __device__ __forceinline__ void operator()(T& x, T& y) const { y = x; }
};
template <typename T>
struct SwapOp {
  static constexpr bool RX = true, RY = true, WX = true, WY = true;
  __device__ __forceinline__ void operator()(T& x, T& y) const {
    T t = x;
    x = y;
    y = t;
  }
};
template <typename T>
struct RotOp {
  T c, s;
  static constexpr bool RX = true, RY = true, WX = true, WY = true;
  __device__ __forceinline__ void operator()(T& x, T& y) const {
    T nx = c * x + s * y;
    T ny = c * y - s * x;
    x = nx;
    y = ny;
  }
};

// Modified Givens rotation: (x, y) <- (h11 x + h12 y, h21 x + h22 y).  The host has already
// written the entries the flag implies (1, -1) into the four coefficients; a product with
// +-1 is exact, so the implied forms lose nothing against skipping the multiplication.
template <typename T>
struct RotmOp {
  T h11, h12, h21, h22;
  static constexpr bool RX = true, RY = true, WX = true, WY = true;
  __device__ __forceinline__ void operator()(T& x, T& y) const {
    T nx = h11 * x + h12 * y;
    T ny = h21 * x + h22 * y;
    x = nx;
    y = ny;
  }
};

// Unit stride.  The vector region is [head, head + nvec*V); up to V-1 head and V-1 tail
// elements are handled one by one by the first threads of block 0.  Each thread keeps NV
// packs per array in flight.
template <typename T, class Op, int NV>
__global__ void __launch_bounds__(kThreads) l1_map_unit(Op op, T* __restrict__ x, T* __restrict__ y, int64_t n,
                                                        int64_t head, int64_t nvec, int64_t nchunks) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int V = VecLen<T>::value;
  using P = Pack<T, V>;
  T* xv = x + head;
  T* yv = y + head;
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    const int64_t v0 = chunk * (int64_t)(kThreads * NV) + threadIdx.x;
    P px[NV], py[NV];
    if (v0 + (int64_t)(NV - 1) * kThreads < nvec) {  // whole chunk inside: no predicates
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int64_t e = (v0 + (int64_t)k * kThreads) * V;
        if (Op::RX) px[k] = ld_cs<T, V>(xv + e);
        if (Op::RY) py[k] = ld_cs<T, V>(yv + e);
      }
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int64_t e = (v0 + (int64_t)k * kThreads) * V;
#pragma unroll
        for (int q = 0; q < V; ++q) op(px[k].v[q], py[k].v[q]);
        if (Op::WX) st_cs<T, V>(xv + e, px[k]);
        if (Op::WY) st_cs<T, V>(yv + e, py[k]);
      }
    } else {
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int64_t v = v0 + (int64_t)k * kThreads;
        if (v < nvec) {
          if (Op::RX) px[k] = ld_cs<T, V>(xv + v * V);
          if (Op::RY) py[k] = ld_cs<T, V>(yv + v * V);
        }
      }
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int64_t v = v0 + (int64_t)k * kThreads;
        if (v < nvec) {
#pragma unroll
          for (int q = 0; q < V; ++q) op(px[k].v[q], py[k].v[q]);
          if (Op::WX) st_cs<T, V>(xv + v * V, px[k]);
          if (Op::WY) st_cs<T, V>(yv + v * V, py[k]);
        }
      }
    }
  }
  if (blockIdx.x == 0) {  // scalar head [0, head) and tail [head + nvec*V, n)
    const int64_t tail0 = head + nvec * V;
    const int64_t ntail = n - tail0;
    int64_t i = -1;
    if ((int64_t)threadIdx.x < head) i = threadIdx.x;
    else if ((int64_t)threadIdx.x - head < ntail) i = tail0 + (threadIdx.x - head);
    if (i >= 0) {
      T a = T(0), b = T(0);
      if (Op::RX) a = x[i];
      if (Op::RY) b = y[i];
      op(a, b);
      if (Op::WX) x[i] = a;
      if (Op::WY) y[i] = b;
    }
  }
}

// Any stride: one element per thread and slot, NE slots in flight.  x and y are the bases
// from vec_base(), so logical element i is at x[i*incx] for either sign.
template <typename T, class Op, int NE>
__global__ void __launch_bounds__(kThreads) l1_map_strided(Op op, T* __restrict__ x, int64_t incx,
                                                           T* __restrict__ y, int64_t incy, int64_t n,
                                                           int64_t nchunks) {
  grid_dep_wait();
  grid_dep_launch();
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    const int64_t i0 = chunk * (int64_t)(kThreads * NE) + threadIdx.x;
    T a[NE], b[NE];
#pragma unroll
    for (int k = 0; k < NE; ++k) {
      const int64_t i = i0 + (int64_t)k * kThreads;
      a[k] = T(0);
      b[k] = T(0);
      if (i < n) {
        // An array that is written back must not be loaded evict-first: a strided store covers
        // only part of a sector, and the rest has to be still in L2 when it arrives, or the sector
        // is fetched from DRAM a second time (measured with L2 full of clean lines: swap with
        // increment 2 at 0.77 of the copy rate evict-first, 1.00 without).
        // a write-only strided target: start the fill of its sectors now, not when the store arrives
        if (!Op::RY && Op::WY) asm volatile("prefetch.global.L2 [%0];" ::"l"(y + i * incy));
        if (Op::RX) a[k] = Op::WX ? __ldcg(x + i * incx) : __ldcs(x + i * incx);
        if (Op::RY) b[k] = Op::WY ? __ldcg(y + i * incy) : __ldcs(y + i * incy);
      }
    }
#pragma unroll
    for (int k = 0; k < NE; ++k) {
      const int64_t i = i0 + (int64_t)k * kThreads;
      if (i < n) {
        op(a[k], b[k]);
        if (Op::WX) __stcs(x + i * incx, a[k]);
        if (Op::WY) __stcs(y + i * incy, b[k]);
      }
    }
  }
}

// ------------------------------------------------------------------------------- reduce ops
template <typename T>
struct DotOp {
  static constexpr bool kArgmax = false;
  static constexpr int kPacks = 4;  // 16-byte packs in flight per thread and array
  using Acc = T;
  using Out = T;
  using Slot = T;  // per-thread running value of the streaming loop
  __device__ __forceinline__ static Slot slot_init() { return T(0); }
  __device__ __forceinline__ static Acc slot_to_acc(Slot s, int64_t, int64_t) { return s; }
  static constexpr bool RY = true;
  __device__ __forceinline__ static Acc init() { return T(0); }
  __device__ __forceinline__ static void accum(Acc& a, T x, T y, int64_t) { a = x * y + a; }
  __device__ __forceinline__ static void slot_accum(Slot& a, T x, T y, int) { a = x * y + a; }
  __device__ __forceinline__ static Acc combine(Acc a, Acc b) { return a + b; }
  __device__ __forceinline__ static Acc shfl(Acc a, int m) { return shfl_xor(a, m); }
  __device__ __forceinline__ static Out finalize(Acc a) { return a; }
};
// dsdot: float inputs, every product and the whole sum in double (a product of two floats is
// exact in double, so the only rounding is the summation's).
struct DsdotOp {
  static constexpr bool kArgmax = false;
  static constexpr int kPacks = 4;
  using Acc = double;
  using Out = double;
  using Slot = double;
  __device__ __forceinline__ static Slot slot_init() { return 0.0; }
  __device__ __forceinline__ static Acc slot_to_acc(Slot s, int64_t, int64_t) { return s; }
  static constexpr bool RY = true;
  __device__ __forceinline__ static Acc init() { return 0.0; }
  __device__ __forceinline__ static void accum(Acc& a, float x, float y, int64_t) { a = (double)x * (double)y + a; }
  __device__ __forceinline__ static void slot_accum(Slot& a, float x, float y, int) { a = (double)x * (double)y + a; }
  __device__ __forceinline__ static Acc combine(Acc a, Acc b) { return a + b; }
  __device__ __forceinline__ static Acc shfl(Acc a, int m) { return shfl_xor(a, m); }
  __device__ __forceinline__ static Out finalize(Acc a) { return a; }
};
template <typename T>
struct AsumOp {
  static constexpr bool kArgmax = false;
  static constexpr int kPacks = 8;  // 16-byte packs in flight per thread and array
  using Acc = T;
  using Out = T;
  using Slot = T;  // per-thread running value of the streaming loop
  __device__ __forceinline__ static Slot slot_init() { return T(0); }
  __device__ __forceinline__ static Acc slot_to_acc(Slot s, int64_t, int64_t) { return s; }
  static constexpr bool RY = false;
  __device__ __forceinline__ static Acc init() { return T(0); }
  __device__ __forceinline__ static void accum(Acc& a, T x, T, int64_t) { a += fabs(x); }
  __device__ __forceinline__ static void slot_accum(Slot& a, T x, T, int) { a += fabs(x); }
  __device__ __forceinline__ static Acc combine(Acc a, Acc b) { return a + b; }
  __device__ __forceinline__ static Acc shfl(Acc a, int m) { return shfl_xor(a, m); }
  __device__ __forceinline__ static Out finalize(Acc a) { return a; }
};
template <typename T>
struct Nrm2Op {
  static constexpr bool kArgmax = false;
  static constexpr int kPacks = 8;  // 16-byte packs in flight per thread and array
  using Acc = T;
  using Out = T;
  using Slot = T;  // per-thread running value of the streaming loop
  __device__ __forceinline__ static Slot slot_init() { return T(0); }
  __device__ __forceinline__ static Acc slot_to_acc(Slot s, int64_t, int64_t) { return s; }
  static constexpr bool RY = false;
  __device__ __forceinline__ static Acc init() { return T(0); }
  __device__ __forceinline__ static void accum(Acc& a, T x, T, int64_t) { a = x * x + a; }
  __device__ __forceinline__ static void slot_accum(Slot& a, T x, T, int) { a = x * x + a; }
  __device__ __forceinline__ static Acc combine(Acc a, Acc b) { return a + b; }
  __device__ __forceinline__ static Acc shfl(Acc a, int m) { return shfl_xor(a, m); }
  __device__ __forceinline__ static Out finalize(Acc a) { return sqrt(a); }
};
template <typename T>
struct MaxIdx {
  T v;
  int64_t i;
};
// First index of the maximum magnitude: a candidate replaces the incumbent on a strictly
// larger magnitude, or on an equal magnitude with a smaller index.
template <typename T>
struct IamaxOp {
  static constexpr int kPacks = 8;
  static constexpr bool kArgmax = true;  // the kernels take the max-then-locate path
  using Acc = MaxIdx<T>;
  using Out = int64_t;
  static constexpr bool RY = false;
  __device__ __forceinline__ static Acc init() { return Acc{T(-1), INT64_MAX}; }
  __device__ __forceinline__ static void accum(Acc& a, T x, T, int64_t i) {
    const T m = fabs(x);
    if (m > a.v) {  // indices reach one accumulator in increasing order
      a.v = m;
      a.i = i;
    }
  }
  __device__ __forceinline__ static Acc combine(Acc a, Acc b) {
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
  }
  __device__ __forceinline__ static Acc shfl(Acc a, int m) { return Acc{shfl_xor(a.v, m), shfl_xor(a.i, m)}; }
  __device__ __forceinline__ static Out finalize(Acc a) { return a.i == INT64_MAX ? 0 : a.i; }
};

// L2-coherent read of another block's partial.
template <typename A>
__device__ __forceinline__ A ld_partial(const A* p) {
  return __ldcg(p);
}
template <typename T>
__device__ __forceinline__ MaxIdx<T> ld_partial(const MaxIdx<T>* p) {
  MaxIdx<T> r;
  r.v = __ldcg(&p->v);
  r.i = __ldcg(&p->i);
  return r;
}

// Block-wide combine in a fixed order; the result is valid in thread 0.
template <class Op>
__device__ __forceinline__ typename Op::Acc block_combine(typename Op::Acc a) {
  __shared__ typename Op::Acc sm[kWarps];
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) a = Op::combine(a, Op::shfl(a, m));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();  // sm may still be read from a previous use
  if (lane == 0) sm[warp] = a;
  __syncthreads();
  if (warp == 0) {
    a = lane < kWarps ? sm[lane] : Op::init();
#pragma unroll
    for (int m = kWarps / 2; m >= 1; m >>= 1) a = Op::combine(a, Op::shfl(a, m));
  }
  return a;
}

// Second pass: each block stores its partial, takes a ticket, and the block that draws the
// last ticket combines all partials in index order and writes the result.  It also puts the
// ticket counter back to zero for the next call.
template <class Op>
__device__ __forceinline__ void reduce_finish(typename Op::Acc acc, typename Op::Acc* partials, unsigned* ticket,
                                              typename Op::Out* result) {
  using Acc = typename Op::Acc;
  __shared__ bool is_last;
  acc = block_combine<Op>(acc);
  if (threadIdx.x == 0) {
    partials[blockIdx.x] = acc;
    __threadfence();
    const unsigned t = atomicAdd(ticket, 1u);
    is_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  Acc a = Op::init();
  for (unsigned b = threadIdx.x; b < gridDim.x; b += kThreads) a = Op::combine(a, ld_partial(&partials[b]));
  a = block_combine<Op>(a);
  if (threadIdx.x == 0) {
    *result = Op::finalize(a);
    *ticket = 0u;
  }
}

// Streaming pass of the sum-type reductions: NV*V independent running values per thread.
// The arg-max reduction (iamax) instead keeps ONE running maximum per thread: a max tree per
// chunk costs about one instruction per element, and only when a chunk raises the maximum is
// the first element that attains it located, while the chunk is still in registers.
// STEP = 2 serves increment 2: the kernel streams the whole span (n = its length) in 128-bit
// packs like a unit-stride vector and lets only the even span positions count -- DRAM moves
// whole sectors anyway, and a pack load costs a quarter of the instructions of four strided ones.
template <typename T, class Op, int NV, int STEP = 1>
__global__ void __launch_bounds__(kThreads) l1_reduce_unit(const T* __restrict__ x, const T* __restrict__ y, int64_t n,
                                                           int64_t head, int64_t nvec, int64_t nchunks,
                                                           typename Op::Acc* partials, unsigned* ticket,
                                                           typename Op::Out* result) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int V = VecLen<T>::value;
  using P = Pack<T, V>;
  using Acc = typename Op::Acc;
  const T* xv = x + head;
  const T* yv = y + head;
  const int hp = (int)(head & 1);  // STEP 2: pack element q is a vector element iff (q & 1) == hp (V is even)
  Acc a = Op::init();
  if constexpr (Op::kArgmax) {
    T best = T(-1);
    int64_t best_chunk = -1;
    int best_pos = 0;  // k*V + q inside that chunk
    for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
      const int64_t v0 = chunk * (int64_t)(kThreads * NV) + threadIdx.x;
      P px[NV];
      T m = T(-1);
      if (v0 + (int64_t)(NV - 1) * kThreads < nvec) {  // every pack of the thread exists: plain loads
#pragma unroll
        for (int k = 0; k < NV; ++k) px[k] = ld_nc<T, V>(xv + (v0 + (int64_t)k * kThreads) * V);
      } else {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
          const int64_t v = v0 + (int64_t)k * kThreads;
          px[k] = ld_nc_if<T, V>(xv + v * V, v < nvec);
        }
      }
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int64_t v = v0 + (int64_t)k * kThreads;
#pragma unroll
        for (int q = 0; q < V; ++q) {
          px[k].v[q] = (v < nvec && !(STEP == 2 && ((q ^ hp) & 1))) ? fabs(px[k].v[q]) : T(-1);
          m = fmax(m, px[k].v[q]);  // fmax drops NaN operands
        }
      }
      if (m > best) {  // strict: the earliest chunk wins ties; locate while the data is in registers
        best = m;
        best_chunk = chunk;
#pragma unroll
        for (int k = NV - 1; k >= 0; --k)
#pragma unroll
          for (int q = V - 1; q >= 0; --q)
            if (px[k].v[q] == m) best_pos = k * V + q;  // the lowest position is assigned last
      }
    }
    if (best_chunk >= 0) {
      const int k = best_pos / V, q = best_pos % V;
      a = Acc{best, (head + (best_chunk * (int64_t)(kThreads * NV) + threadIdx.x + (int64_t)k * kThreads) * V + q) / STEP};
    }
  } else {
    typename Op::Slot acc[NV][V];
#pragma unroll
    for (int k = 0; k < NV; ++k)
#pragma unroll
      for (int q = 0; q < V; ++q) acc[k][q] = Op::slot_init();
    for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
      const int64_t v0 = chunk * (int64_t)(kThreads * NV) + threadIdx.x;
      P px[NV], py[NV];
      if (v0 + (int64_t)(NV - 1) * kThreads < nvec) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
          const int64_t e = (v0 + (int64_t)k * kThreads) * V;
          px[k] = ld_nc<T, V>(xv + e);
          if (Op::RY) py[k] = ld_nc<T, V>(yv + e);
        }
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
          for (int q = 0; q < V; ++q)
            Op::slot_accum(acc[k][q], (STEP == 2 && ((q ^ hp) & 1)) ? T(0) : px[k].v[q],
                           (Op::RY && !(STEP == 2 && ((q ^ hp) & 1))) ? py[k].v[q] : T(0), 0);
      } else {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
          const int64_t v = v0 + (int64_t)k * kThreads;
          if (v < nvec) {
            px[k] = ld_nc<T, V>(xv + v * V);
            if (Op::RY) py[k] = ld_nc<T, V>(yv + v * V);
#pragma unroll
            for (int q = 0; q < V; ++q)
              Op::slot_accum(acc[k][q], (STEP == 2 && ((q ^ hp) & 1)) ? T(0) : px[k].v[q],
                           (Op::RY && !(STEP == 2 && ((q ^ hp) & 1))) ? py[k].v[q] : T(0), 0);
          }
        }
      }
    }
#pragma unroll
    for (int k = 0; k < NV; ++k)
#pragma unroll
      for (int q = 0; q < V; ++q) a = Op::combine(a, Op::slot_to_acc(acc[k][q], 0, 0));
  }
  if (blockIdx.x == 0) {  // scalar head and tail elements
    const int64_t tail0 = head + nvec * V;
    const int64_t ntail = n - tail0;
    int64_t i = -1;
    if ((int64_t)threadIdx.x < head) i = threadIdx.x;
    else if ((int64_t)threadIdx.x - head < ntail) i = tail0 + (threadIdx.x - head);
    if (i >= 0 && !(STEP == 2 && (i & 1))) {
      Acc e = Op::init();
      Op::accum(e, x[i], Op::RY ? y[i] : T(0), i / STEP);
      a = Op::combine(a, e);
    }
  }
  reduce_finish<Op>(a, partials, ticket, result);
}

template <typename T, class Op, int NE>
__global__ void __launch_bounds__(kThreads) l1_reduce_strided(const T* __restrict__ x, int64_t incx,
                                                              const T* __restrict__ y, int64_t incy, int64_t n,
                                                              int64_t nchunks, typename Op::Acc* partials,
                                                              unsigned* ticket, typename Op::Out* result) {
  grid_dep_wait();
  grid_dep_launch();
  using Acc = typename Op::Acc;
  Acc r = Op::init();
  if constexpr (Op::kArgmax) {
    T best = T(-1);
    int64_t best_chunk = -1;
    int best_pos = 0;
    for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
      const int64_t i0 = chunk * (int64_t)(kThreads * NE) + threadIdx.x;
      T a[NE];
#pragma unroll
      for (int k = 0; k < NE; ++k) {
        const int64_t i = i0 + (int64_t)k * kThreads;
        a[k] = i < n ? fabs(__ldg(x + i * incx)) : T(-1);
      }
      T m = T(-1);
#pragma unroll
      for (int k = 0; k < NE; ++k) m = fmax(m, a[k]);
      if (m > best) {
        best = m;
        best_chunk = chunk;
#pragma unroll
        for (int k = NE - 1; k >= 0; --k)
          if (a[k] == m) best_pos = k;
      }
    }
    if (best_chunk >= 0) r = Acc{best, best_chunk * (int64_t)(kThreads * NE) + threadIdx.x + (int64_t)best_pos * kThreads};
  } else {
    typename Op::Slot acc[NE];
#pragma unroll
    for (int k = 0; k < NE; ++k) acc[k] = Op::slot_init();
    for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
      const int64_t i0 = chunk * (int64_t)(kThreads * NE) + threadIdx.x;
      T a[NE], b[NE];
#pragma unroll
      for (int k = 0; k < NE; ++k) {
        const int64_t i = i0 + (int64_t)k * kThreads;
        a[k] = T(0);
        b[k] = T(0);
        if (i < n) {
          a[k] = __ldg(x + i * incx);
          if (Op::RY) b[k] = __ldg(y + i * incy);
        }
      }
#pragma unroll
      for (int k = 0; k < NE; ++k)
        if (i0 + (int64_t)k * kThreads < n) Op::slot_accum(acc[k], a[k], b[k], 0);
    }
#pragma unroll
    for (int k = 0; k < NE; ++k) r = Op::combine(r, Op::slot_to_acc(acc[k], 0, 0));
  }
  reduce_finish<Op>(r, partials, ticket, result);
}

// sdsdot's last step: result = (float)(sb + the double-accumulated dot), rounded once.
__global__ void sdsdot_finish(const double* __restrict__ acc, float sb, float* __restrict__ result) {
  grid_dep_wait();
  grid_dep_launch();
  *result = (float)((double)sb + *acc);
}

// ------------------------------------------------------------------------------- host side
static int grid_cap() { return sm_count() * (int)knob(kKnobL1BlocksPerSm); }

// One resident wave: as many blocks as really fit (the kernel grid-strides over the data), so
// no second, partly filled wave trails behind.  Only the blocks-per-SM figure of the kernel is
// cached (per device id); the SM count, the knob and the cap are read on every call.
struct WaveCache {
  int per_sm[64] = {0};
};
template <class Kernel>
static int one_wave(Kernel kernel, int cap, WaveCache& cache) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    (void)cudaGetLastError();
    return cap;
  }
  if (cache.per_sm[dev] == 0) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm <= 0) {
      (void)cudaGetLastError();
      return cap;
    }
    cache.per_sm[dev] = per_sm;
  }
  const int wave = cache.per_sm[dev] * sm_count();
  return wave < cap ? wave : cap;
}

template <typename T>
static bool same_head(const T* x, const T* y, bool use_y, int64_t* head) {
  constexpr int V = VecLen<T>::value;
  const int mx = (int)((reinterpret_cast<uintptr_t>(x) % 16) / sizeof(T));
  const int my = use_y ? (int)((reinterpret_cast<uintptr_t>(y) % 16) / sizeof(T)) : mx;
  *head = (V - mx) % V;
  return mx == my;
}

template <typename T, class Op>
static int run_map(const b2_ctx* ctx, Op op, int64_t n, T* x, int64_t incx, T* y, int64_t incy) {
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (n == 0) return B2_STATUS_OK;
  constexpr bool two = Op::RY || Op::WY;
  constexpr int V = VecLen<T>::value;
  B2_DBG_VEC(l, x, n, incx);
  if (two) B2_DBG_VEC(l, y, n, incy);
  B2_DBG_COMMIT(l);
  int64_t head = 0;
  if (incx == 1 && (!two || incy == 1) && same_head<T>(x, y, two, &head)) {
    constexpr int NV = two ? 4 : 8;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / V;
    const int64_t nchunks = (nvec + kThreads * NV - 1) / (kThreads * NV);
    const int64_t grid = nchunks < 1 ? 1 : (nchunks > (1 << 30) ? (1 << 30) : nchunks);
    launch_chained(l1_map_unit<T, Op, NV>, dim3((unsigned)grid), dim3(kThreads), 0, l.stream, op, x, two ? y : x, n, head, nvec, nchunks);
  } else {
    constexpr int NE = 8;
    const int64_t nchunks = (n + kThreads * NE - 1) / (kThreads * NE);
    const int64_t grid = nchunks > (1 << 30) ? (1 << 30) : nchunks;
    launch_chained(l1_map_strided<T, Op, NE>, dim3((unsigned)grid), dim3(kThreads), 0, l.stream, op, vec_base(x, n, incx), incx, two ? vec_base(y, n, incy) : x, two ? incy : 1, n, nchunks);
  }
  return check_launch();
}

template <typename T, class Op>
static int run_reduce(const b2_ctx* ctx, int64_t n, const T* x, int64_t incx, const T* y, int64_t incy,
                      typename Op::Out* result) {
  using Acc = typename Op::Acc;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (n == 0) {
    return cudaMemsetAsync(result, 0, sizeof(typename Op::Out), l.stream) == cudaSuccess ? B2_STATUS_OK
                                                                                        : B2_STATUS_LAUNCH_FAILED;
  }
  constexpr int V = VecLen<T>::value;
  if (n > ((int64_t)1 << 40)) return B2_STATUS_NOT_IMPLEMENTED;  // chunk ids are 32-bit
  B2_DBG_VEC(l, x, n, incx);
  if (Op::RY) B2_DBG_VEC(l, y, n, incy);
  B2_DBG_RANGE(l, result, sizeof(typename Op::Out));
  B2_DBG_COMMIT(l);
  const int cap = grid_cap();
  if (l.scratch_bytes < (size_t)cap * sizeof(Acc)) return B2_STATUS_WORKSPACE_TOO_SMALL;
  Acc* partials = reinterpret_cast<Acc*>(l.scratch);
  unsigned* ticket = l.ctl + kCtlReduceTicket;
  int64_t head = 0;
  if (incx == 1 && (!Op::RY || incy == 1) && same_head<T>(x, y, Op::RY, &head)) {
    constexpr int NV = Op::kPacks;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / V;
    const int64_t nchunks = (nvec + kThreads * NV - 1) / (kThreads * NV);
    static WaveCache wc;
    const int wave = one_wave(l1_reduce_unit<T, Op, NV>, cap, wc);
    const int64_t grid = nchunks < 1 ? 1 : (nchunks > wave ? wave : nchunks);
    launch_chained(l1_reduce_unit<T, Op, NV>, dim3((unsigned)grid), dim3(kThreads), 0, l.stream, x, Op::RY ? y : x, n, head, nvec, nchunks,
                                                                        partials, ticket, result);
  } else if (sizeof(T) == 4 && incx == 2 && (!Op::RY || incy == 2) && same_head<T>(x, y, Op::RY, &head)) {
    // (float only: for double, where a pack holds a single vector element, the strided kernel is the faster one)
    constexpr int NV = Op::kPacks;
    const int64_t span = 2 * n - 1;
    if (head > span) head = span;
    const int64_t nvec = (span - head) / V;
    const int64_t nchunks = (nvec + kThreads * NV - 1) / (kThreads * NV);
    static WaveCache wc;
    const int wave = one_wave(l1_reduce_unit<T, Op, NV, 2>, cap, wc);
    const int64_t grid = nchunks < 1 ? 1 : (nchunks > wave ? wave : nchunks);
    launch_chained(l1_reduce_unit<T, Op, NV, 2>, dim3((unsigned)grid), dim3(kThreads), 0, l.stream, x, Op::RY ? y : x, span, head, nvec, nchunks,
                                                                           partials, ticket, result);
  } else {
    constexpr int NE = Op::RY ? 8 : 16;
    const int64_t nchunks = (n + kThreads * NE - 1) / (kThreads * NE);
    static WaveCache wc;
    const int wave = one_wave(l1_reduce_strided<T, Op, NE>, cap, wc);
    const int64_t grid = nchunks > wave ? wave : nchunks;
    launch_chained(l1_reduce_strided<T, Op, NE>, dim3((unsigned)grid), dim3(kThreads), 0, l.stream, vec_base(x, n, incx), incx, Op::RY ? vec_base(y, n, incy) : x, Op::RY ? incy : 1, n, nchunks, partials, ticket,
        result);
  }
  return check_launch();
}

// Argument checks shared by the entry points; k-th argument numbers follow the header.
template <typename T>
static int check_vec(int64_t n, const T* p, int64_t inc, int argp, int arginc) {
  if (inc == 0) return -arginc;
  if (n > 0 && (p == nullptr || !aligned_to(p, sizeof(T)))) return -argp;
  return 0;
}

}  // namespace b2

using namespace b2;

#define B2_L1_TWO_VEC_CHECK()                                  \
  if (n < 0) return -1;                                        \
  if (int e = check_vec(n, x, incx, XP, XP + 1)) return e;     \
  if (int e = check_vec(n, y, incy, XP + 2, XP + 3)) return e;

// rotm: param is a HOST array {flag, h11, h21, h12, h22}; the flag decides which entries are read.
template <typename T>
static int rotm_impl(const b2_ctx* ctx, int64_t n, T* x, int64_t incx, T* y, int64_t incy, const T* param) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  if (param == nullptr) return -6;
  const T flag = param[0];
  RotmOp<T> op;
  if (flag == T(-1)) op = RotmOp<T>{param[1], param[3], param[2], param[4]};
  else if (flag == T(0)) op = RotmOp<T>{T(1), param[3], param[2], T(1)};
  else if (flag == T(1)) op = RotmOp<T>{param[1], T(1), T(-1), param[4]};
  else if (flag == T(-2)) {  // H = I: nothing to do
    Launch l;
    return make_launch(ctx, &l);
  } else return -6;
  return run_map<T>(ctx, op, n, x, incx, y, incy);
}
extern "C" {

int b2_saxpy(const b2_ctx* ctx, int64_t n, float alpha, const float* x, int64_t incx, float* y, int64_t incy) {
  constexpr int XP = 3;
  B2_L1_TWO_VEC_CHECK();
  if (alpha == 0.0f) {
    Launch l;
    return make_launch(ctx, &l);
  }
  return run_map<float>(ctx, AxpyOp<float>{alpha}, n, const_cast<float*>(x), incx, y, incy);
}
int b2_daxpy(const b2_ctx* ctx, int64_t n, double alpha, const double* x, int64_t incx, double* y, int64_t incy) {
  constexpr int XP = 3;
  B2_L1_TWO_VEC_CHECK();
  if (alpha == 0.0) {
    Launch l;
    return make_launch(ctx, &l);
  }
  return run_map<double>(ctx, AxpyOp<double>{alpha}, n, const_cast<double*>(x), incx, y, incy);
}

int b2_sscal(const b2_ctx* ctx, int64_t n, float alpha, float* x, int64_t incx) {
  if (n < 0) return -1;
  if (int e = check_vec(n, x, incx, 3, 4)) return e;
  return run_map<float>(ctx, ScalOp<float>{alpha}, n, x, incx, (float*)nullptr, 1);
}
int b2_dscal(const b2_ctx* ctx, int64_t n, double alpha, double* x, int64_t incx) {
  if (n < 0) return -1;
  if (int e = check_vec(n, x, incx, 3, 4)) return e;
  return run_map<double>(ctx, ScalOp<double>{alpha}, n, x, incx, (double*)nullptr, 1);
}

int b2_scopy(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, float* y, int64_t incy) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  return run_map<float>(ctx, CopyOp<float>{}, n, const_cast<float*>(x), incx, y, incy);
}
int b2_dcopy(const b2_ctx* ctx, int64_t n, const double* x, int64_t incx, double* y, int64_t incy) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  return run_map<double>(ctx, CopyOp<double>{}, n, const_cast<double*>(x), incx, y, incy);
}

int b2_sswap(const b2_ctx* ctx, int64_t n, float* x, int64_t incx, float* y, int64_t incy) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  return run_map<float>(ctx, SwapOp<float>{}, n, x, incx, y, incy);
}
int b2_dswap(const b2_ctx* ctx, int64_t n, double* x, int64_t incx, double* y, int64_t incy) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  return run_map<double>(ctx, SwapOp<double>{}, n, x, incx, y, incy);
}

int b2_srot(const b2_ctx* ctx, int64_t n, float* x, int64_t incx, float* y, int64_t incy, float c, float s) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  return run_map<float>(ctx, RotOp<float>{c, s}, n, x, incx, y, incy);
}
int b2_drot(const b2_ctx* ctx, int64_t n, double* x, int64_t incx, double* y, int64_t incy, double c, double s) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  return run_map<double>(ctx, RotOp<double>{c, s}, n, x, incx, y, incy);
}

int b2_sdot(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, const float* y, int64_t incy, float* result) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  if (result == nullptr) return -6;
  return run_reduce<float, DotOp<float>>(ctx, n, x, incx, y, incy, result);
}
int b2_ddot(const b2_ctx* ctx, int64_t n, const double* x, int64_t incx, const double* y, int64_t incy,
            double* result) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  if (result == nullptr) return -6;
  return run_reduce<double, DotOp<double>>(ctx, n, x, incx, y, incy, result);
}

int b2_srotm(const b2_ctx* ctx, int64_t n, float* x, int64_t incx, float* y, int64_t incy, const float* param) {
  return rotm_impl<float>(ctx, n, x, incx, y, incy, param);
}
int b2_drotm(const b2_ctx* ctx, int64_t n, double* x, int64_t incx, double* y, int64_t incy, const double* param) {
  return rotm_impl<double>(ctx, n, x, incx, y, incy, param);
}

int b2_dsdot(const b2_ctx* ctx, int64_t n, const float* x, int64_t incx, const float* y, int64_t incy,
             double* result) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  if (result == nullptr) return -6;
  return run_reduce<float, DsdotOp>(ctx, n, x, incx, y, incy, result);
}
int b2_sdsdot(const b2_ctx* ctx, int64_t n, float sb, const float* x, int64_t incx, const float* y, int64_t incy,
              float* result) {
  constexpr int XP = 3;
  B2_L1_TWO_VEC_CHECK();
  if (result == nullptr) return -7;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  // the double sum lands in the workspace, behind the block partials of the reduction
  const size_t off = ((size_t)grid_cap() * sizeof(double) + 255) / 256 * 256;
  if (l.scratch_bytes < off + sizeof(double)) return B2_STATUS_WORKSPACE_TOO_SMALL;
  double* acc = reinterpret_cast<double*>(l.scratch + off);
  if (int st = run_reduce<float, DsdotOp>(ctx, n, x, incx, y, incy, acc)) return st;
  launch_chained(sdsdot_finish, dim3(1), dim3(1), 0, l.stream, acc, sb, result);
  return check_launch();
}

#define B2_L1_ONE_VEC_REDUCE(NAME, T, OP, OUT)                                          \
  int NAME(const b2_ctx* ctx, int64_t n, const T* x, int64_t incx, OUT* result) {       \
    if (n < 0) return -1;                                                               \
    if (int e = check_vec(n, x, incx, 2, 3)) return e;                                  \
    if (result == nullptr) return -4;                                                   \
    return run_reduce<T, OP<T>>(ctx, n, x, incx, (const T*)nullptr, 1, result);         \
  }

B2_L1_ONE_VEC_REDUCE(b2_sasum, float, AsumOp, float)
B2_L1_ONE_VEC_REDUCE(b2_dasum, double, AsumOp, double)
B2_L1_ONE_VEC_REDUCE(b2_snrm2, float, Nrm2Op, float)
B2_L1_ONE_VEC_REDUCE(b2_dnrm2, double, Nrm2Op, double)
B2_L1_ONE_VEC_REDUCE(b2_isamax, float, IamaxOp, int64_t)
B2_L1_ONE_VEC_REDUCE(b2_idamax, double, IamaxOp, int64_t)

}  // extern "C"

// ------------------------------------------------------------------------- b2_sdot_noalloc
// A dot product for callers that own no device scratch and may not allocate any.  The
// partials and the ticket word that b2_sdot keeps in ctx->workspace live here in a fixed
// file-scope device array instead.  Layout: word 0 = ticket, partials from byte 256 on.
namespace b2 {
constexpr int kNoAllocMaxBlocks = 1024;
constexpr size_t kNoAllocScratchBytes = 256 + kNoAllocMaxBlocks * sizeof(float);
constexpr int64_t kNoAllocMaxN = (int64_t)1 << 30;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// In host code `g_noalloc_scratch` is only a handle: its device address has to be asked for,
// once per device, with that device current.
static int noalloc_scratch(unsigned char** out) {
  static unsigned char* cached[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return B2_STATUS_LAUNCH_FAILED;
  if (cached[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return B2_STATUS_LAUNCH_FAILED;
    }
    cached[dev] = static_cast<unsigned char*>(p);
  }
  *out = cached[dev];
  return B2_STATUS_OK;
}
}  // namespace b2

extern "C" int b2_sdot_noalloc(void* stream, int64_t n, const float* x, int64_t incx, const float* y, int64_t incy,
                               float* result) {
  constexpr int XP = 2;
  B2_L1_TWO_VEC_CHECK();
  if (result == nullptr) return -6;
  if (n > kNoAllocMaxN) return B2_STATUS_TOO_LARGE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n == 0)
    return cudaMemsetAsync(result, 0, sizeof(float), st) == cudaSuccess ? B2_STATUS_OK : B2_STATUS_LAUNCH_FAILED;
  unsigned char* scratch = nullptr;
  if (int rc = noalloc_scratch(&scratch)) return rc;
  unsigned* ticket = reinterpret_cast<unsigned*>(scratch);
  float* partials = reinterpret_cast<float*>(scratch + 256);
  // The array keeps whatever the previous call left; the ticket must start at zero.
  if (cudaMemsetAsync(ticket, 0, sizeof(unsigned), st) != cudaSuccess) return B2_STATUS_LAUNCH_FAILED;
  using Op = DotOp<float>;
  constexpr int V = VecLen<float>::value;
  int64_t head = 0;
  if (incx == 1 && incy == 1 && same_head<float>(x, y, true, &head)) {
    constexpr int NV = 4;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / V;
    const int64_t nchunks = (nvec + kThreads * NV - 1) / (kThreads * NV);
    const int64_t grid = nchunks < 1 ? 1 : (nchunks > kNoAllocMaxBlocks ? kNoAllocMaxBlocks : nchunks);
    l1_reduce_unit<float, Op, NV><<<(unsigned)grid, kThreads, 0, st>>>(x, y, n, head, nvec, nchunks, partials, ticket,
                                                                      result);
  } else {
    constexpr int NE = 8;
    const int64_t nchunks = (n + kThreads * NE - 1) / (kThreads * NE);
    const int64_t grid = nchunks > kNoAllocMaxBlocks ? kNoAllocMaxBlocks : nchunks;
    l1_reduce_strided<float, Op, NE><<<(unsigned)grid, kThreads, 0, st>>>(vec_base(x, n, incx), incx,
                                                                         vec_base(y, n, incy), incy, n, nchunks,
                                                                         partials, ticket, result);
  }
  return check_launch();
}
