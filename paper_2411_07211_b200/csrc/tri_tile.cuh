// symv and trmv on 16-byte aligned matrices: tile kernel with a shared-memory ring (Section 6.2.2, "Triangular
// Matrix": the same loop nest as gemv over a triangular iteration space, bounds rounded to the
// blocking factor so that full tiles run unmasked and only the tiles on the diagonal are masked).
//
// The canonical row-major view is cut into tiles of 128 rows x 32 packs (128 floats / 64 doubles).
// A 256-thread block is a 16 x 16 grid; thread (rg, cg) holds rows 8*rg .. 8*rg+7 and the two
// packs cg and cg + 16 of each (a half-warp covers 256 contiguous bytes of a row); the tile reaches
// the thread through asynchronous copies into shared memory, several half tiles ahead (see the
// kernel).  One pass over a tile serves
//   row sums  (ROW): sum_j A_ij x_j, kept in 8 registers while the block walks ALONG a block row and
//                    reduced over the 16 lanes of a row group once per unit, and / or
//   column sums (COL): sum_i A_ij x_i, per tile: one exchange between the two half-warps, then one
//                    store per warp into shared memory (no block-wide barrier per tile).
// symv uses both on the stored triangle (each element loaded once, used twice; the diagonal only
// in the row sum); trmv uses one of them with the diagonal taken as 1 for diag = unit.  A kind
// that has only column sums walks DOWN a block column instead, with the column sums in registers.
// Units (a few consecutive tiles) write partials to the workspace; tri_tile_finalize adds them in
// a fixed order, so results are bit-reproducible, and writes y (trmv: x, after every block has
// read it).
#pragma once

#include <cuda.h>  // CUtensorMap (types only: the encoder is fetched from the driver at run time)

#include "level2.cuh"

namespace b2 {
namespace tt {

// (measured: wider, flatter tiles -- 64 x 256 or 32 x 512 floats -- are slower here, they waste
// more of the tiles that the diagonal cuts and make the units coarser)
#ifndef B2_TT_RING
#define B2_TT_RING 3
#endif
constexpr int kRing = B2_TT_RING;  // tiles (64 KB each at 128 rows) in the shared-memory ring
#ifndef B2_TT_NR
#define B2_TT_NR 8
#endif
#ifndef B2_TT_UNITMAX
#define B2_TT_UNITMAX 4
#endif
#ifndef B2_TT_BPS
#define B2_TT_BPS 1
#endif
constexpr int kBlocksPerSm = B2_TT_BPS;
constexpr int kNR = B2_TT_NR;  // rows of a tile a thread holds
constexpr int kNP = 2;         // packs of each row a thread holds (16 lanes side by side, kNP groups of them)
constexpr int kTR = 16 * kNR;  // tile rows
constexpr int kUnitMax = B2_TT_UNITMAX;  // tiles per unit at most (1, 2 or 4)
constexpr int kMaxMajor = 2048;  // block rows (or column tiles) the unit table can hold

// Elements of the queue of x values: one slot per unit that can be in flight.  The producer runs
// up to kRing tiles ahead of the consumer and a unit may hold a single tile (the first or last
// unit of a row), so kRing + 1 units can be open at once; a slot is sized for the longest unit.
constexpr int kSlots = kRing + 1;
template <typename T, bool WALK_ROWS, bool ROWS_OF_X>
__host__ __device__ constexpr int kSlotElems() {
  constexpr int TC = 16 * kNP * VecLen<T>::value;
  // along the walking direction a slot holds unit * tile extent values, across it one tile extent
  constexpr int ext = ROWS_OF_X ? kTR : TC;
  constexpr bool along = ROWS_OF_X != WALK_ROWS;
  return kSlots * (along ? kUnitMax : 1) * ext;
}

// CAP: entries of the unit table.  The table travels in the kernel parameters; matrices of up to
// 128 block rows (columns) use the short form, whose parameter block is a tenth of the long one.
template <typename T, int CAP>
struct TileArgs {
  const T* a;
  int64_t lda, n;
  const T* x;  // base per vec_base()
  int64_t incx;
  T* rowpart;  // [groups][n]: ROW kinds, one row of partials per column group (ROW && COL: per unit column group)
  T* colpart;  // [groups][n]: COL kinds, one row of partials per block row (row walk) or row group (column walk)
  int nbr, nct;  // block rows, column tiles
  int unit;      // tiles per unit
  int ngroups;   // units per block row (row walk) / per block column (column walk)
  T alpha, beta;
  T* y;
  int64_t incy;
  int* status;  // device status word (may be null): a bounded wait that ran out reports here
  int prefix[CAP + 1];  // units before block row (column tile) i; the last entry is their total
};

// First and last column tile of block row I that meets the triangle.
template <int TRI, int TC>
__host__ __device__ __forceinline__ void row_range(int I, int64_t n, int nct, int* jlo, int* jhi) {
  const int64_t r0 = (int64_t)I * kTR, r1 = (r0 + kTR < n ? r0 + kTR : n) - 1;
  *jlo = TRI == TRI_UPPER ? (int)(r0 / TC) : 0;
  *jhi = TRI == TRI_LOWER ? (int)(r1 / TC) : nct - 1;
}
// First and last block row of column tile J that meets the triangle.
template <int TRI, int TC>
__host__ __device__ __forceinline__ void col_range(int J, int64_t n, int nbr, int* ilo, int* ihi) {
  const int64_t c0 = (int64_t)J * TC, c1 = (c0 + TC < n ? c0 + TC : n) - 1;
  *ilo = TRI == TRI_LOWER ? (int)(c0 / kTR) : 0;
  *ihi = TRI == TRI_UPPER ? (int)(c1 / kTR) : nbr - 1;
}

// Asynchronous 16-byte copy global -> shared memory of `bytes` (0 .. 16) bytes, the rest of the
// 16 zero-filled; element-sized copies for the vectors (bytes = 0: a zero).
__device__ __forceinline__ void cp_async16_full(void* dst, const void* src) {
  if (!B2_GUARD(src, 16)) {  // (bounds-checking build only: a zero-filled pack instead of the read)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, 0;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
    return;
  }
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(void* dst, const void* src, int bytes) {
  if (bytes > 0 && !B2_GUARD(src, (size_t)bytes)) bytes = 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(src),
               "r"(bytes)
               : "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_elem(void* dst, const void* src, bool valid) {
  if (valid && !B2_GUARD(src, (size_t)N)) valid = false;
  asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(src),
               "n"(N), "r"(valid ? N : 0)
               : "memory");
}
// Bulk asynchronous copies (one instruction per contiguous run, no per-thread load path) and the
// shared-memory barrier that counts their bytes.  Source and destination 16-byte aligned, size a
// multiple of 16; this GPU's own memory, no multicast.
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"((unsigned)__cvta_generic_to_shared(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
  unsigned done;
  asm volatile(
      "{\n\t.reg .pred q;\n\tmbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2;\n\tselp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(done)
      : "r"((unsigned)__cvta_generic_to_shared(bar)), "r"(parity)
      : "memory");
  return done != 0;
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   (unsigned)__cvta_generic_to_shared(dst)),
               "l"(src), "r"(bytes), "r"((unsigned)__cvta_generic_to_shared(bar))
               : "memory");
}
// One tiled TMA copy: the box of the tensor map at element coordinates (x, y) -> shared memory.
// x * element size must be a multiple of 16 bytes; what lies outside the tensor arrives as zeros.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, unsigned long long* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                   (unsigned)__cvta_generic_to_shared(dst)),
               "l"(map), "r"(x), "r"(y), "r"((unsigned)__cvta_generic_to_shared(bar))
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Persistent blocks (one per SM).  Block b takes the units b, b + gridDim, ... of the dense unit
// list and streams their tiles through a ring of kRing tiles in shared memory filled by
// asynchronous copies: every thread copies exactly the 16 packs it will later read itself, so the
// ring needs no barrier -- only the per-thread wait for its own copies -- and the copies of the
// next kRing - 1 tiles (also those of the block's next units) are in flight while a tile is
// multiplied.  Edge tiles use the same copies with a byte count that zero-fills what lies outside
// the matrix.  The x values of a unit travel the same way.
// BULK: a tile arrives as ONE tiled TMA copy (tensor map over the n x n matrix, box = one tile;
// what lies outside the matrix arrives as zeros), issued by one thread and counted by a
// shared-memory barrier per ring slot, and lies row-major in its slot; one block-wide barrier per
// tile keeps the refill of a slot behind its last reader.  Every wait on a barrier is bounded.
// (kTR separate row-sized bulk copies per tile measured three times SLOWER than the 16-byte
// per-thread copies: the fixed cost of a bulk copy is paid per 512 bytes.)
template <typename T, int CAP, bool ROW, bool COL, int TRI, bool UNIT, bool SYM, bool BULK = false>
__global__ void __launch_bounds__(kThreads, kBlocksPerSm) tri_tile_kernel(const TileArgs<T, CAP> p, const __grid_constant__ CUtensorMap tmap) {
  constexpr int V = VecLen<T>::value, TC = 16 * kNP * V, NR = kNR, HR = NR / 2, NP = kNP, TP = NR * NP;
  constexpr bool WALK_ROWS = ROW;  // column-sum-only kinds walk down a block column
  constexpr int XCU = WALK_ROWS ? kUnitMax * TC : TC;  // most column values a unit needs
  using P = Pack<T, V>;
  grid_dep_wait();
  grid_dep_launch();
  extern __shared__ __align__(128) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);             // [kRing][TP][kThreads] packs
  T* xr_q = reinterpret_cast<T*>(ring + kRing * TP * kThreads);  // [slots] row values of the units in flight
  constexpr int XRQ = COL ? kSlotElems<T, WALK_ROWS, true>() : 0, XCQ = ROW ? kSlotElems<T, WALK_ROWS, false>() : 0;
  T* xc_q = xr_q + XRQ;  // [slots] column values
  T* cbuf = xc_q + XCQ;  // [kWarps][XCU] column sums of the warps
  __shared__ unsigned long long full_bar[kRing];
  if (BULK) {
    if (threadIdx.x == 0) {
      for (int s = 0; s < kRing; ++s) mbar_init(&full_bar[s], 1u);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
  }
  unsigned bar_phase = 0;  // bit s: parity of the next completion of slot s
  bool dead = false;       // a bounded wait ran out: drain without touching the tiles

  const int ct = (int)threadIdx.x, warp = ct >> 5, lane = ct & 31;
  const int rg = ct >> 4, cg = ct & 15;
  const int nmajor = WALK_ROWS ? p.nbr : p.nct;
  const int nunits = p.prefix[nmajor];
  constexpr int nslots = kSlots;
  const int xr_stride = WALK_ROWS ? kTR : p.unit * kTR, xc_stride = WALK_ROWS ? p.unit * TC : TC;
  const int64_t row_step = p.lda;                              // elements between a thread's rows
  const int64_t thread_off = (int64_t)(rg * HR) * p.lda + V * cg;  // this thread's first pack inside a half tile
  const int64_t half_step = (int64_t)(kTR / 2) * p.lda;

  // A cursor walks the block's sequence of tiles; the units come in increasing order, so the row
  // (column) a unit belongs to is found by moving forward through the unit table.
  struct Cursor {
    int u, major, g, t0, t1, t, slot;
    bool valid;
  };
  auto open_unit = [&](Cursor& c) {
    c.valid = c.u < nunits;
    if (!c.valid) return;
    while (p.prefix[c.major + 1] <= c.u) ++c.major;
    c.g = c.u - p.prefix[c.major];
    int rl, rh;
    if (WALK_ROWS) row_range<TRI, TC>(c.major, p.n, p.nct, &rl, &rh);
    else col_range<TRI, TC>(c.major, p.n, p.nbr, &rl, &rh);
    c.t0 = max(rl, (rl / p.unit + c.g) * p.unit);
    c.t1 = min(rh, (rl / p.unit + c.g) * p.unit + p.unit - 1);
    c.t = c.t0;
  };
  auto advance = [&](Cursor& c) {
    if (++c.t <= c.t1) return;
    c.u += (int)gridDim.x;
    c.slot = c.slot + 1 == nslots ? 0 : c.slot + 1;
    open_unit(c);
  };

  Cursor prod, cons;
  prod.u = cons.u = (int)blockIdx.x;
  prod.slot = cons.slot = 0;
  prod.major = cons.major = 0;
  open_unit(prod);
  open_unit(cons);
  int pstage = 0, cstage = 0;

  // one producer step: the copies of the next tile (and, with a unit's first one, of its x values)
  auto produce = [&]() {
    if (prod.valid) {
      const int I = WALK_ROWS ? prod.major : prod.t, J = WALK_ROWS ? prod.t : prod.major;
      const int64_t r0 = (int64_t)I * kTR, c0 = (int64_t)J * TC;
      if (prod.t == prod.t0) {
        const int64_t rb = (int64_t)(WALK_ROWS ? I : prod.t0) * kTR, cb = (int64_t)(WALK_ROWS ? prod.t0 : J) * TC;
        const int nrv = (WALK_ROWS ? 1 : prod.t1 - prod.t0 + 1) * kTR, ncv = (WALK_ROWS ? prod.t1 - prod.t0 + 1 : 1) * TC;
        if (COL)
          for (int t = ct; t < nrv; t += kThreads) {
            const bool ok = rb + t < p.n;
            cp_async_elem<sizeof(T)>(xr_q + prod.slot * xr_stride + t, p.x + (ok ? (rb + t) * p.incx : 0), ok);
          }
        if (ROW)
          for (int t = ct; t < ncv; t += kThreads) {
            const bool ok = cb + t < p.n;
            cp_async_elem<sizeof(T)>(xc_q + prod.slot * xc_stride + t, p.x + (ok ? (cb + t) * p.incx : 0), ok);
          }
      }
      uint4* dst = ring + (size_t)pstage * TP * kThreads + ct;
      const T* src = p.a + r0 * p.lda + c0 + thread_off;
      if (BULK) {
        if (ct == 0) {
          mbar_arrive_expect(&full_bar[pstage], (unsigned)(kTR * TC * sizeof(T)));
          tma_load_2d(ring + (size_t)pstage * TP * kThreads, &tmap, (int)c0, (int)r0, &full_bar[pstage]);
        }
      } else if (r0 + kTR <= p.n && c0 + TC <= p.n) {
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int a = 0; a < HR; ++a)
#pragma unroll
            for (int hb = 0; hb < NP; ++hb)
              cp_async16_full(dst + ((h * HR + a) * NP + hb) * kThreads, src + h * half_step + a * row_step + hb * 16 * V);
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int a = 0; a < HR; ++a) {
            const int64_t r = r0 + h * (kTR / 2) + rg * HR + a;
#pragma unroll
            for (int hb = 0; hb < NP; ++hb) {
              const int64_t left = (p.n - (c0 + V * cg + hb * 16 * V)) * (int64_t)sizeof(T);
              const int bytes = (r < p.n && left > 0) ? (int)(left < 16 ? left : 16) : 0;
              cp_async16(dst + ((h * HR + a) * NP + hb) * kThreads,
                         bytes ? src + h * half_step + a * row_step + hb * 16 * V : p.a, bytes);
            }
          }
      }
      advance(prod);
    }
    cp_async_commit();  // (an empty group when the sequence has ended: the group count stays uniform)
    pstage = pstage + 1 == kRing ? 0 : pstage + 1;
  };

  T racc[NR], cacc[NP][V];
#pragma unroll
  for (int a = 0; a < NR; ++a) racc[a] = T(0);
#pragma unroll
  for (int hb = 0; hb < NP; ++hb)
#pragma unroll
    for (int e = 0; e < V; ++e) cacc[hb][e] = T(0);

#pragma unroll 1
  for (int s = 0; s < kRing - 1; ++s) produce();
#pragma unroll 1
  while (cons.valid) {
    if (BULK) __syncthreads();  // every thread has left the slot that this trip's copies refill
    produce();
    cp_async_wait<kRing - 1>();  // this thread's copies of the oldest tile in flight have landed
    if (BULK && !dead) {  // ... and so has the tile itself (bounded: a wait that runs out is reported, the block drains)
      const unsigned parity = (bar_phase >> cstage) & 1u;
      bool ok = false;
      for (int spin = 0; spin < (1 << 22) && !ok; ++spin) ok = mbar_try_wait(&full_bar[cstage], parity);
      bar_phase ^= 1u << cstage;
      if (!ok) {
        dead = true;
        if (p.status) atomicExch(p.status, (int)B2_STATUS_TIMEOUT);
      }
    }
    const int I = WALK_ROWS ? cons.major : cons.t, J = WALK_ROWS ? cons.t : cons.major;
    const int I0 = WALK_ROWS ? I : cons.t0, J0 = WALK_ROWS ? cons.t0 : J;
    if (cons.t == cons.t0) __syncthreads();  // the unit's x values came from other threads' copies
    const int64_t r0 = (int64_t)I * kTR, c0 = (int64_t)J * TC;
    // the thread's packs of the tile: its own copies (one slot entry per pack and thread), or, in a
    // tile that came as whole rows, row (h, a) of its row group and the packs cg, cg + 16 of that row
    const uint4* src = ring + (size_t)cstage * TP * kThreads + (BULK ? (rg * HR) * (TC / V) + cg : ct);
    auto pack_at = [&](int h, int a, int hb) -> int {
      return BULK ? (h * (kTR / 2) + a) * (TC / V) + hb * 16 : ((h * HR + a) * NP + hb) * kThreads;
    };
    cstage = cstage + 1 == kRing ? 0 : cstage + 1;
    T xc[NP][V];
    if (ROW) {
      const T* xs = xc_q + cons.slot * xc_stride + (J - J0) * TC + V * cg;
#pragma unroll
      for (int hb = 0; hb < NP; ++hb) {
        const P pk = *reinterpret_cast<const P*>(xs + hb * 16 * V);
#pragma unroll
        for (int e = 0; e < V; ++e) xc[hb][e] = pk.v[e];
      }
    }
    // no element of the tile on or beyond the diagonal: nothing to mask (what lies outside the
    // matrix arrived as zeros)
    const bool inside = TRI == TRI_FULL || (TRI == TRI_LOWER ? c0 + TC - 1 < r0 : c0 > r0 + kTR - 1);
#pragma unroll
    for (int h = 0; h < 2; ++h) {  // the two halves of the tile (rows 0 .. 63, 64 .. 127)
      T m[HR][NP][V];
#pragma unroll
      for (int a = 0; a < HR; ++a)
#pragma unroll
        for (int hb = 0; hb < NP; ++hb) {
          const uint4 raw = dead ? make_uint4(0u, 0u, 0u, 0u) : src[pack_at(h, a, hb)];
          const P pk = *reinterpret_cast<const P*>(&raw);
#pragma unroll
          for (int e = 0; e < V; ++e) m[a][hb][e] = pk.v[e];
        }
      T xr[HR];
      if (COL) {
        const T* xs = xr_q + cons.slot * xr_stride + (I - I0) * kTR + h * (kTR / 2) + rg * HR;
#pragma unroll
        for (int a = 0; a < HR; ++a) xr[a] = xs[a];
      }
      if (inside) {
#pragma unroll
        for (int a = 0; a < HR; ++a)
#pragma unroll
          for (int hb = 0; hb < NP; ++hb)
#pragma unroll
            for (int e = 0; e < V; ++e) {
              if (ROW) racc[h * HR + a] = m[a][hb][e] * xc[hb][e] + racc[h * HR + a];
              if (COL) cacc[hb][e] = m[a][hb][e] * xr[a] + cacc[hb][e];
            }
      } else {
        // a tile on the diagonal: d = (column of the element) - (row of the element)
        const int dbase = (int)(c0 - r0) - h * (kTR / 2) + V * cg - rg * HR;
        const int nrows = (int)min((int64_t)(kTR / 2), p.n - r0 - h * (kTR / 2));
#pragma unroll
        for (int a = 0; a < HR; ++a)
#pragma unroll
          for (int hb = 0; hb < NP; ++hb)
#pragma unroll
            for (int e = 0; e < V; ++e) {
              const int d = dbase + hb * 16 * V + e - a;
              const bool in_tri = TRI == TRI_LOWER ? d <= 0 : d >= 0;
              T v = in_tri ? m[a][hb][e] : T(0);
              if (UNIT && d == 0) v = (rg * HR + a < nrows) ? T(1) : T(0);
              if (ROW) racc[h * HR + a] = v * xc[hb][e] + racc[h * HR + a];
              if (COL) cacc[hb][e] = ((SYM && d == 0) ? T(0) : v) * xr[a] + cacc[hb][e];
            }
      }
    }
    const bool unit_done = cons.t == cons.t1;
    if (COL && (WALK_ROWS || unit_done)) {
      // column sums: the two row groups of the warp, then shared memory; along a block row per tile
#pragma unroll
      for (int hb = 0; hb < NP; ++hb) {
        P pk;
#pragma unroll
        for (int e = 0; e < V; ++e) {
          pk.v[e] = cacc[hb][e] + shfl_xor(cacc[hb][e], 16);
          cacc[hb][e] = T(0);
        }
        if (lane < 16) *reinterpret_cast<P*>(cbuf + warp * XCU + (J - J0) * TC + V * cg + hb * 16 * V) = pk;
      }
    }
    if (unit_done) {
      const int64_t r_base = (int64_t)I0 * kTR, c_base = (int64_t)J0 * TC;
      if (ROW) {  // 8 row sums over the 16 lanes of a row group: lanes 2v and 2v + 1 end up with value v
        const T s = multi_group_sum<16, NR>(racc, lane);
        constexpr int LPV = 16 / NR;  // lanes that end up with the same value
        const int v = cg / LPV;
        const int64_t i = r_base + (v / HR) * (kTR / 2) + rg * HR + v % HR;
        if (cg % LPV == 0 && i < p.n) p.rowpart[(int64_t)cons.g * p.n + i] = s;
#pragma unroll
        for (int a = 0; a < NR; ++a) racc[a] = T(0);
      }
      if (COL) {
        const int ncols = (WALK_ROWS ? cons.t1 - cons.t0 + 1 : 1) * TC;
        __syncthreads();
        for (int t = ct; t < ncols; t += kThreads) {
          if (c_base + t >= p.n) break;
          T s = cbuf[t];
#pragma unroll
          for (int w = 1; w < kWarps; ++w) s += cbuf[w * XCU + t];
          p.colpart[(int64_t)(WALK_ROWS ? cons.major : cons.g) * p.n + c_base + t] = s;
        }
        __syncthreads();  // cbuf is written again by the next unit
      }
    }
    advance(cons);
  }
  cp_async_wait<0>();
  if (BULK && dead) {  // copies may still be on their way into this block's shared memory: give them time to land
    for (int s = 0; s < kRing; ++s)
      for (int spin = 0; spin < (1 << 16) && !mbar_try_wait(&full_bar[s], (bar_phase >> s) & 1u); ++spin) {
      }
  }
}

// y_i = alpha * (row partials of i + column partials of i) + beta * y_i, the partials added in a
// fixed order.  A block of 32 (16) warps serves 32 consecutive outputs (one per lane, so every load is
// a coalesced row segment of a partial array); warp w takes partials w, w + 32, ... -- a handful
// of independent loads, all in flight at once -- and warp 0 adds the 32 sums in warp order.
// (16 warps in double precision: the block's shared memory must fit beside a tile-kernel block
// that is still running, or the early launch waits for it to leave)
template <typename T>
__host__ __device__ constexpr int fin_warps() {
  return sizeof(T) == 8 ? 16 : 32;
}
template <typename T, int CAP, bool ROW, bool COL, int TRI>
__global__ void __launch_bounds__(fin_warps<T>() * 32) tri_tile_finalize(const TileArgs<T, CAP> p) {
  constexpr int V = VecLen<T>::value, TC = 16 * kNP * V, kFinWarps = fin_warps<T>();
  constexpr bool WALK_ROWS = ROW;
  __shared__ T part[kFinWarps][33];
  grid_dep_wait();
  grid_dep_launch();
  const int w = (int)(threadIdx.x >> 5), lane = (int)(threadIdx.x & 31);
  const int64_t i = (int64_t)blockIdx.x * 32 + lane;
  T s = T(0);
  if (i < p.n) {
    int nrow = 0;
    if (ROW) {  // the units of i's block row
      int lo, hi;
      row_range<TRI, TC>((int)(i / kTR), p.n, p.nct, &lo, &hi);
      nrow = hi / p.unit - lo / p.unit + 1;
    }
    int clo = 0, ncol = 0;
    if (COL) {
      int lo, hi;
      col_range<TRI, TC>((int)(i / TC), p.n, p.nbr, &lo, &hi);
      // along block rows: one partial per block row that meets i's column tile; down block
      // columns: one per unit of i's block column
      clo = WALK_ROWS ? lo : 0;
      ncol = WALK_ROWS ? hi - lo + 1 : hi / p.unit - lo / p.unit + 1;
    }
    T s0 = T(0), s1 = T(0), s2 = T(0), s3 = T(0);
    auto fetch = [&](int k) -> T {
      if (k >= nrow + ncol) return T(0);
      return k < nrow ? __ldcg(p.rowpart + (int64_t)k * p.n + i) : __ldcg(p.colpart + (int64_t)(clo + k - nrow) * p.n + i);
    };
    for (int k = w; k < nrow + ncol; k += 4 * kFinWarps) {
      const T v0 = fetch(k), v1 = fetch(k + kFinWarps), v2 = fetch(k + 2 * kFinWarps), v3 = fetch(k + 3 * kFinWarps);
      s0 += v0, s1 += v1, s2 += v2, s3 += v3;
    }
    s = (s0 + s1) + (s2 + s3);
  }
  part[w][lane] = s;
  __syncthreads();
  if (w == 0 && i < p.n) {
    T t = part[0][lane];
#pragma unroll
    for (int k = 1; k < kFinWarps; ++k) t += part[k][lane];
    T* yp = p.y + i * p.incy;
    B2_STORE(yp, p.beta != T(0) ? p.alpha * t + p.beta * *yp : p.alpha * t);
  }
}

// Shared memory of the tile kernel: the ring, the queues of x values, the warps' column sums.
template <typename T, bool ROW, bool COL>
constexpr size_t tile_smem_bytes() {
  constexpr int TC = 16 * kNP * VecLen<T>::value;
  constexpr bool WALK_ROWS = ROW;
  return (size_t)kRing * kNR * kNP * kThreads * 16 +
         sizeof(T) * (size_t)((COL ? kSlotElems<T, WALK_ROWS, true>() : 0) + (ROW ? kSlotElems<T, WALK_ROWS, false>() : 0) +
                              (COL ? kWarps * (WALK_ROWS ? kUnitMax * TC : TC) : 0));
}

// Tensor map of the n x n row-major matrix with boxes of one tile (kTR rows x tc columns).  The
// encoder lives in the driver; it is looked up once.  false: no encoder, or the matrix does not
// meet the map's rules (the caller then uses the 16-byte copies).
template <typename T>
static bool encode_tile_map(CUtensorMap* map, const T* a, int64_t lda, int64_t n, int tc) {
  using Encode = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static Encode encode = [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      fn = nullptr;
    }
    return reinterpret_cast<Encode>(fn);
  }();
  if (encode == nullptr) return false;
  if ((lda * sizeof(T)) % 16 != 0 || !aligned_to(a, 16)) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)n, (cuuint64_t)n};
  const cuuint64_t strides[1] = {(cuuint64_t)lda * sizeof(T)};
  const cuuint32_t box[2] = {(cuuint32_t)tc, (cuuint32_t)kTR};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapDataType dt = sizeof(T) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT64;
  return encode(map, dt, 2, const_cast<T*>(a), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launches both kernels.  *handled is false (nothing launched) when the matrix is not 16-byte
// aligned, too large for the unit table, or the partials do not fit the workspace: the caller
// then uses the general tile kernel.
template <typename T, int CAP, bool ROW, bool COL, int TRI, bool UNIT, bool SYM>
static int tri_tile_run_cap(const Launch& l, const T* a, int64_t lda, int64_t n, const T* x, int64_t incx, T alpha, T beta,
                            T* y, int64_t incy, bool* handled) {
  constexpr int V = VecLen<T>::value, TC = 16 * kNP * V;
  constexpr bool WALK_ROWS = ROW;
  const int64_t nbr = (n + kTR - 1) / kTR, nct = (n + TC - 1) / TC;
  TileArgs<T, CAP> args = {};
  args.a = a;
  args.lda = lda;
  args.n = n;
  args.x = x;
  args.incx = incx;
  args.nbr = (int)nbr;
  args.nct = (int)nct;
  // longer units mean fewer partials, fewer reductions and fewer block-wide barriers per tile; a
  // dozen units per block keep the tail short (measured at 4096 tiles on 148 blocks: units of 2
  // take symv from 57 / 53 us (upper / lower, float) to 50.5 us, units of 4 to 52 / 50 us)
  const int64_t tiles = nbr * nct / 2;
  const int64_t per_block = tiles / sm_count();
  args.unit = (per_block >= 48 && kUnitMax >= 4) ? 4 : (per_block >= 12 && kUnitMax >= 2) ? 2 : 1;
  const int64_t forced = knob(kKnobTriTileUnit);
  if ((forced == 1 || forced == 2 || forced == 4) && forced <= kUnitMax) args.unit = (int)forced;
  const int nmajor = WALK_ROWS ? args.nbr : args.nct;
  int ngroups = 0;
  for (int i = 0; i < nmajor; ++i) {
    int lo, hi;
    if (WALK_ROWS) row_range<TRI, TC>(i, n, args.nct, &lo, &hi);
    else col_range<TRI, TC>(i, n, args.nbr, &lo, &hi);
    const int ng = hi / args.unit - lo / args.unit + 1;
    args.prefix[i + 1] = args.prefix[i] + ng;
    ngroups = ng > ngroups ? ng : ngroups;
  }
  args.ngroups = ngroups;
  const size_t row_bytes = ROW ? ((size_t)ngroups * n * sizeof(T) + 255) / 256 * 256 : 0;
  const size_t col_bytes = COL ? (size_t)(WALK_ROWS ? args.nbr : ngroups) * n * sizeof(T) : 0;
  if (row_bytes + col_bytes > l.scratch_bytes) return B2_STATUS_OK;
  args.rowpart = reinterpret_cast<T*>(l.scratch);
  args.colpart = reinterpret_cast<T*>(l.scratch + row_bytes);
  args.alpha = alpha;
  args.beta = beta;
  args.y = y;
  args.incy = incy;
  args.status = l.device_status;
  constexpr size_t smem = tile_smem_bytes<T, ROW, COL>();
  // whole rows by bulk copies when every tile is full (and the rows' starts and lengths are then
  // multiples of 16 bytes, which those copies need)
  CUtensorMap tmap = {};
  bool bulk = knob(kKnobTriBulk) != 0 && n <= 0x7fffffff;
#ifdef B2_DEBUG_BOUNDS
  bulk = false;  // (a TMA copy cannot be tested address by address: the checking build keeps the 16-byte copies)
#endif
  if (bulk) bulk = encode_tile_map<T>(&tmap, a, lda, n, TC);
  auto kern = bulk ? tri_tile_kernel<T, CAP, ROW, COL, TRI, UNIT, SYM, true> : tri_tile_kernel<T, CAP, ROW, COL, TRI, UNIT, SYM, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    (void)cudaGetLastError();
    return B2_STATUS_OK;
  }
  *handled = true;
  const int nunits = args.prefix[nmajor];
  const int grid = nunits < sm_count() * kBlocksPerSm ? nunits : sm_count() * kBlocksPerSm;
  launch_chained(kern, dim3(grid), dim3(kThreads), smem, l.stream, args, tmap);
  if (int st = check_launch()) return st;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((n + 31) / 32));
  cfg.blockDim = dim3(fin_warps<T>() * 32);
  cfg.stream = l.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = knob(kKnobUsePdl) ? 1 : 0;
  cudaLaunchKernelEx(&cfg, tri_tile_finalize<T, CAP, ROW, COL, TRI>, args);
  return check_launch();
}

template <typename T, bool ROW, bool COL, int TRI, bool UNIT, bool SYM>
static int tri_tile_run(const Launch& l, const T* a, int64_t lda, int64_t n, const T* x, int64_t incx, T alpha, T beta,
                        T* y, int64_t incy, bool* handled) {
  constexpr int V = VecLen<T>::value, TC = 16 * kNP * V;
  *handled = false;
  if (!aligned_to(a, 16) || lda % V != 0) return B2_STATUS_OK;
  const int64_t nmajor = ROW ? (n + kTR - 1) / kTR : (n + TC - 1) / TC;
  if (nmajor > kMaxMajor) return B2_STATUS_OK;
  if (nmajor <= 128) return tri_tile_run_cap<T, 128, ROW, COL, TRI, UNIT, SYM>(l, a, lda, n, x, incx, alpha, beta, y, incy, handled);
  return tri_tile_run_cap<T, kMaxMajor, ROW, COL, TRI, UNIT, SYM>(l, a, lda, n, x, incx, alpha, beta, y, incy, handled);
}

}  // namespace tt
}  // namespace b2
