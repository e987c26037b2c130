// trsv, sub-block kernel: solve op(A) x = b in place (Section 6.2.2; same option space as trmv).
//
// The unknowns are cut into blocks of NB (128 float / 64 double).  In solve order (top-down for
// an effectively lower-triangular op(A), bottom-up for an upper one) block row k needs
//     x_k = inv(D_k) * (b_k - sum_{s<k} A_ks x_s),
// and the chain k-1 -> k is the only sequential part.  Persistent 256-thread blocks draw block
// rows in solve order.  A block
//   1. inverts its diagonal block D_k in shared memory long before the front arrives
//      (recursive doubling on 4x4 register tiles; the matrix is kept in symmetric storage so
//      that both operand orientations are contiguous) and leaves inv(D_k) there in the
//      layout of a matrix tile,
//   2. walks along its block row: tile A_ks sits in registers, distributed over a 16 x 16
//      thread grid (an RS x RS sub-block per thread), so a tile-times-vector product needs RS
//      vector elements per thread from shared memory and one RS-value reduction over the 16
//      lanes of a row group -- a few hundred cycles from "x_s is here" to "row sums updated";
//      two register sets take turns, one multiplied while the other receives the next tile,
//   3. treats inv(D_k) as one more tile whose vector is r = b - sum: the last trip through the
//      SAME loop body produces x_k.  That matters: a stretch of code that a block executes
//      once, after tens of microseconds of doing something else, costs microseconds of
//      instruction fetches on the critical path; everything between "x_{k-1} is visible" and
//      "x_k is published" is therefore code the block has been executing on every tile,
//      including the publishing stores (predicated off on the earlier trips).
// Values cross SMs as 64-bit words {32 payload bits, 32-bit call tag}: data and ready flag
// are one store, and the consumer polls the data itself.  Every wait is bounded: when a
// budget runs out the thread records B2_STATUS_TIMEOUT, raises an abort word in the control
// block and every block drains without publishing.  Tickets are drawn in solve order, so a
// block only waits for rows that running or finished blocks hold.
#include "trsv_front.cuh"

namespace b2 {
namespace tf {

constexpr int kT = 256;  // threads per block: a 16 x 16 grid of sub-block owners
constexpr int kBar = 1;

template <typename T>
struct Geo;
template <>
struct Geo<float> {
  static constexpr int NB = 128, V = 4;
};
template <>
struct Geo<double> {
  static constexpr int NB = 64, V = 2;
};

template <typename T>
struct FrontArgs {
  const T* a;
  int64_t lda, n;
  T* x;
  int64_t incx;
  unsigned long long* xbuf;  // solved x: WPE tagged words per unknown, padded to whole blocks
  unsigned* ctl;
  int nb;
  int pf_dist;  // tiles pulled into L2 ahead of use
  unsigned tag;
  unsigned long long wait_limit;
  int* device_status;
  int debug_skip;
  int pm_from;  // first row (solve order) that premultiplies its last tile
};


// ---------------------------------------------------------------------------------------
// Named barrier.  Polling loops in front of it let lanes leave at different iterations, so the
// warp is re-converged first and the form that counts threads (not whole warps) is used.
__device__ __forceinline__ void bar_sync(int id, int count) {
  __syncwarp();
  asm volatile("barrier.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// Polling load through a generic address: the words live in global memory (another cluster's
// row) or in this block's shared memory (a row of the same cluster, written by its block).
__device__ __forceinline__ void ld_word2(const unsigned long long* p, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.relaxed.gpu.v2.u64 {%0,%1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}
// Thread-block cluster pieces: rank, cluster-wide barrier, address of a peer's shared memory,
// (predicated) stores into it.
__device__ __forceinline__ unsigned cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned map_remote(const void* local_smem, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"((unsigned)__cvta_generic_to_shared(local_smem)), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_remote_u32(unsigned raddr, unsigned v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(raddr), "r"(v) : "memory");
}
__device__ __forceinline__ void st_remote_if(bool pred, unsigned raddr, unsigned long long v) {
  asm volatile("{ .reg .pred q; setp.ne.u32 q, %0, 0; @q st.shared::cluster.u64 [%1], %2; }" ::"r"((unsigned)pred),
               "r"(raddr), "l"(v)
               : "memory");
}
__device__ __forceinline__ void publish_remote_if(bool pred, unsigned raddr, float v, unsigned tag) {
  st_remote_if(pred, raddr, ((unsigned long long)tag << 32) | __float_as_uint(v));
}
__device__ __forceinline__ void publish_remote_if(bool pred, unsigned raddr, double v, unsigned tag) {
  const unsigned long long b = (unsigned long long)__double_as_longlong(v);
  st_remote_if(pred, raddr, ((unsigned long long)tag << 32) | (b & 0xffffffffull));
  st_remote_if(pred, raddr + 8, ((unsigned long long)tag << 32) | (b >> 32));
}
// Stores under a predicate instead of a branch: the instructions are fetched on every trip of
// the tile loop and take effect on the last one only.
__device__ __forceinline__ void st_word_if(bool pred, unsigned long long* p, unsigned long long v) {
  asm volatile("{ .reg .pred q; setp.ne.u32 q, %0, 0; @q st.relaxed.gpu.global.u64 [%1], %2; }" ::"r"((unsigned)pred),
               "l"(p), "l"(v)
               : "memory");
}
__device__ __forceinline__ void st_val_if(bool pred, float* p, float v) {
  asm volatile("{ .reg .pred q; setp.ne.u32 q, %0, 0; @q st.global.f32 [%1], %2; }" ::"r"((unsigned)pred), "l"(p), "f"(v)
               : "memory");
}
__device__ __forceinline__ void st_val_if(bool pred, double* p, double v) {
  asm volatile("{ .reg .pred q; setp.ne.u32 q, %0, 0; @q st.global.f64 [%1], %2; }" ::"r"((unsigned)pred), "l"(p), "d"(v)
               : "memory");
}
__device__ __forceinline__ unsigned ld_flag(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

template <typename T>
struct Words {
  static constexpr int N = sizeof(T) / 4;
};
__device__ __forceinline__ void publish_if(bool pred, unsigned long long* w, float v, unsigned tag) {
  st_word_if(pred, w, ((unsigned long long)tag << 32) | __float_as_uint(v));
}
__device__ __forceinline__ void publish_if(bool pred, unsigned long long* w, double v, unsigned tag) {
  const unsigned long long b = (unsigned long long)__double_as_longlong(v);
  st_word_if(pred, w, ((unsigned long long)tag << 32) | (b & 0xffffffffull));
  st_word_if(pred, w + 1, ((unsigned long long)tag << 32) | (b >> 32));
}
__device__ __forceinline__ float decode(const unsigned long long* w, float) { return __uint_as_float((unsigned)w[0]); }
__device__ __forceinline__ double decode(const unsigned long long* w, double) {
  return __longlong_as_double((long long)(((unsigned long long)(unsigned)w[1] << 32) | (unsigned)w[0]));
}

// Per-thread state of the bounded waits.
struct Waiter {
  unsigned long long budget;
  unsigned* abort_word;  // control block: raised by the first wait that runs out
  int* device_status;
  bool dead;             // this thread stopped waiting (its budget ran out, or the abort word is up)

  __device__ __forceinline__ void fail() {
    dead = true;
    atomicExch(abort_word, 1u);
    if (device_status) atomicExch(device_status, (int)B2_STATUS_TIMEOUT);
  }
  // w holds a first attempt at the four words ptr[0..3] (16-byte aligned); polls until the
  // words with their bit in `need` set carry this call's tag.
  __device__ __forceinline__ void finish(unsigned long long (&w)[4], const unsigned long long* ptr, unsigned need,
                                         unsigned tag, unsigned sleep_ns) {
    if (need == 0u) return;
    for (;;) {
      bool ok = true;
#pragma unroll
      for (int i = 0; i < 4; ++i) ok = ok && (!((need >> i) & 1u) || (unsigned)(w[i] >> 32) == tag);
      if (ok || dead) return;
      if (--budget == 0) {
        fail();
        return;
      }
      if ((budget & 15) == 0 && ld_flag(abort_word) != 0u) {
        dead = true;
        return;
      }
      if (sleep_ns) __nanosleep(sleep_ns);
      ld_word2(ptr, w[0], w[1]);
      ld_word2(ptr + 2, w[2], w[3]);
    }
  }
};

// 16-byte load through a generic address (global memory or shared memory), issued where it
// stands: the compiler must not sink it towards its first use.
template <typename T, int N>
__device__ __forceinline__ Pack<T, N> ld_generic(const T* p) {
  static_assert(sizeof(T) * N == 16, "16-byte packs");
  uint4 t;
  asm volatile("ld.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(t.x), "=r"(t.y), "=r"(t.z), "=r"(t.w) : "l"(p) : "memory");
  return *reinterpret_cast<Pack<T, N>*>(&t);
}

// Four consecutive elements through 16-byte shared-memory accesses.
__device__ __forceinline__ void ld4(const float* p, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x, v[1] = t.y, v[2] = t.z, v[3] = t.w;
}
__device__ __forceinline__ void ld4(const double* p, double (&v)[4]) {
  const double2 t0 = *reinterpret_cast<const double2*>(p), t1 = *reinterpret_cast<const double2*>(p + 2);
  v[0] = t0.x, v[1] = t0.y, v[2] = t1.x, v[3] = t1.y;
}
__device__ __forceinline__ void st4(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void st4(double* p, double a, double b, double c, double d) {
  *reinterpret_cast<double2*>(p) = make_double2(a, b);
  *reinterpret_cast<double2*>(p + 2) = make_double2(c, d);
}

// ---------------------------------------------------------------------------------------
// COLTYPE: op(A)'s rows are columns of the stored row-major view.  BACKWARD: solve bottom-up.
// CS: blocks per cluster (1 = no cluster).  With CS = 8 a cluster takes eight consecutive block
// rows; a solved block is also written straight into the shared memory of the blocks that
// hold the later rows of the cluster, so seven hand-overs out of eight skip the trip through
// L2 and the polling of global memory.
template <typename T, bool COLTYPE, bool BACKWARD, bool UNIT, int CS>
__global__ void __launch_bounds__(kT, 1) trsv_front_kernel(const FrontArgs<T> p) {
  grid_dep_wait();
  grid_dep_launch();
  constexpr int NB = Geo<T>::NB, V = Geo<T>::V, WPE = Words<T>::N;
  constexpr int RS = NB / 16;  // sub-block edge: 8 (float) / 4 (double)
  constexpr int E = RS * RS;
  constexpr int LPO = 16 / RS;                  // lanes per row owner
  constexpr int H = NB / 2;                     // distance between a thread's two chunks
  constexpr int SP = NB + 16 / (int)sizeof(T);  // row pitch of S (rows start 16-byte aligned)
  constexpr bool CANON_LOWER = (COLTYPE == BACKWARD);  // stored triangle in the row-major view
  using P = Pack<T, V>;
  constexpr bool PM = CS == 1;  // premultiply the last tile (see below)

  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* S = reinterpret_cast<T*>(smem_raw);       // diagonal block, then its inverse (symmetric storage)
  T* Tm = S + NB * SP;                          // products in flight during the inversion
  T* Wt = S;                                    // ... and finally the inverse in the tile loader's layout
  T* Ms = Tm + (NB / 2) * (NB / 2 + 4);         // inv(D_k) * A_{k,k-1} in the same layout (the tile of the last trip)
  T* xs = Ms + (PM ? NB * SP : 0);              // [2][NB] x values of the current / next tile
  T* rbuf = xs + 2 * NB;                        // r = b - sum, the vector of the final trip
  T* bvec = rbuf + NB;
  T* red = bvec + NB;                           // [kT / 32][NB] per-warp partial row sums (column-type views)
  // x of the earlier rows of this cluster: [CS][NB * WPE] words {payload, row + 1}, written by their blocks
  unsigned long long* xrecv = reinterpret_cast<unsigned long long*>(red + (kT / 32) * NB);
  __shared__ unsigned s_ticket[2];

  const int ct = (int)threadIdx.x, warp = ct >> 5, lane = ct & 31;
  const int rg = ct >> 4, cg = ct & 15;
  // Row-type views: a 16 x 16 thread grid, thread (rg, cg) holds an RS x RS sub-block and the row
  // sums run over the 16 lanes that share rg.  Column-type views (a tile of op(A) is the transpose
  // of a stored tile): lanes must run along the STORED rows or a load instruction touches 16 rows
  // for one sector each, so lane l holds rows V*l .. V*l+V-1 of op(A), warp w the columns
  // w*JT .. w*JT+JT-1 (JT stored rows, each read as one 512-byte run by the warp), and the row
  // sums run across the warps through `red`.
  constexpr int JT = NB / (kT / 32);
  static_assert(JT * V == E, "both layouts hold the same number of elements per thread");
  // the row (solve order inside the block) this thread may own
  const int ti = COLTYPE ? (ct & (NB - 1)) : ((cg / LPO) / V) * H + V * rg + ((cg / LPO) % V);
  const bool owner = COLTYPE ? ct < NB : (cg % LPO) == 0;

  Waiter wt;
  wt.budget = p.wait_limit ? p.wait_limit : (1ull << 22);
  wt.abort_word = p.ctl + kCtlTrsvAbort;
  wt.device_status = p.device_status;
  wt.dead = false;
  int parity = 0;
  const unsigned rank = CS > 1 ? cluster_rank() : 0u;
  if (CS > 1) {
    for (int i = ct; i < CS * NB * WPE; i += kT) xrecv[i] = 0ull;  // no stale word may look like a row of this call
    cluster_sync_all();
  }

  for (;;) {
    // one ticket per cluster = CS consecutive block rows in solve order
    if (rank == 0u && ct == 0) {
      unsigned kk = 0xffffffffu;
      if (!wt.dead && ld_flag(wt.abort_word) == 0u) kk = atomicAdd(p.ctl + kCtlTrsvTicket, 1u);
      // abort word up (raised in this call, or left by an earlier timed-out call on a workspace
      // that was not reset): nothing more is solved, and the caller must be able to see that
      else if (p.device_status) atomicExch(p.device_status, (int)B2_STATUS_TIMEOUT);
      if (CS > 1) {
        for (unsigned r = 0; r < (unsigned)CS; ++r) st_remote_u32(map_remote(&s_ticket[parity], r), kk);
      } else {
        s_ticket[parity] = kk;
      }
    }
    if (CS > 1) cluster_sync_all();
    else bar_sync(kBar, kT);
    const unsigned long long kk = (unsigned long long)s_ticket[parity] * CS + rank;
    parity ^= 1;
    if (kk - rank >= (unsigned long long)p.nb) break;  // the whole cluster leaves together
    if (kk >= (unsigned long long)p.nb) continue;     // this group has fewer than CS rows
    const int k = (int)kk;  // position in the solve order = number of source tiles
    const int g0 = k - (int)rank;  // first row of this cluster's group
    const int I = BACKWARD ? p.nb - 1 - k : k;
    const int64_t r0 = (int64_t)I * NB;
    const int nbI = (int)min((int64_t)NB, p.n - r0);
    auto sidx = [&](int i) { return BACKWARD ? nbI - 1 - i : i; };  // solve order <-> memory order (involution)
    auto blk = [&](int s) { return BACKWARD ? p.nb - 1 - s : s; };
    const bool row_ok = ti < nbI;
    const int mi = row_ok ? sidx(ti) : 0;  // memory-local row of this thread's unknown

    // tile s of this block row -> registers: m[a * RS + b] = op(A)(row sub_i(a), column sub_j(b)).
    // A thread's RS rows / columns are two chunks of V (one 16-byte pack), NB/2 apart: the packs
    // that the lanes of a warp load together then tile whole 32-byte sectors.
    // The tiles of the last two trips are inv(D_k) and inv(D_k) A_{k,k-1}, laid out in shared
    // memory (Wt, Ms) the way a matrix tile lies in global memory.
    // PM (premultiply): the last tile is replaced by inv(D_k) A_{k,k-1}, so that one product instead
    // of two stands between x_{k-1} and x_k -- at the price of two trips between x_{k-2} and
    // x_{k-1}.  It pays where the hand-over itself is slow (through L2), not inside a cluster.
    // (the first rows go without: the front reaches them before the product could be formed)
    const int nm = (PM && k > 0 && k >= p.pm_from) ? 1 : 0;
    const int yt = k - nm;  // the trip that applies inv(D_k) to b - sum
    // full tile at base (leading dimension ld, tile origin: own rows rr0, source columns c0)
    auto fill = [&](T (&m)[E], const T* base, int64_t ld, int64_t c0, int64_t rr0, bool smem) {
      if (!COLTYPE) {
#pragma unroll
        for (int a = 0; a < RS; ++a) {
          const int i = (a / V) * H + V * rg + (a % V);
          const T* src = base + (rr0 + (BACKWARD ? NB - 1 - i : i)) * ld + c0 + V * cg;
#pragma unroll
          for (int hb = 0; hb < RS / V; ++hb) {
            const P pk = smem ? *reinterpret_cast<const P*>(src + hb * H) : ld_nc<T, V>(src + hb * H);
#pragma unroll
            for (int e = 0; e < V; ++e) m[a * RS + hb * V + e] = pk.v[e];
          }
        }
      } else {
        // m[jj * V + e] = op(A)(row V*lane + e, column warp*JT + jj) = stored (c0 + column, rr0 + row')
        const int m0 = BACKWARD ? NB - V * lane - V : V * lane;  // ascending memory run of the pack
#pragma unroll
        for (int jj = 0; jj < JT; ++jj) {
          const T* src = base + (c0 + warp * JT + jj) * ld + rr0 + m0;
          const P pk = smem ? *reinterpret_cast<const P*>(src) : ld_nc<T, V>(src);
#pragma unroll
          for (int e = 0; e < V; ++e) m[jj * V + (BACKWARD ? V - 1 - e : e)] = pk.v[e];
        }
      }
    };
    auto load_tile = [&](T (&m)[E], int s, bool raw) {
      const bool inv = !raw && s >= yt;  // trip yt reads Wt, trip k > 0 reads Ms; `raw`: the matrix tile itself
      const int64_t c0 = inv ? 0 : (int64_t)blk(s) * NB;
      const int nbJ = inv ? NB : (int)min((int64_t)NB, p.n - c0);
      if (inv) {
        // (this branch runs once or twice per block row, one trip before its data is needed and
        // before that trip waits for its x: its instruction fetches are off the critical path)
        fill(m, s == yt ? Wt : Ms, SP, 0, 0, true);
      } else if (nbI == NB && nbJ == NB) {
        fill(m, p.a, p.lda, c0, r0, false);
      } else if (!COLTYPE) {
#pragma unroll
        for (int a = 0; a < RS; ++a)
#pragma unroll
          for (int b = 0; b < RS; ++b) {
            const int i = (a / V) * H + V * rg + (a % V), jc = (b / V) * H + V * cg + (b % V);
            const bool ok = i < nbI && jc < nbJ;
            const int64_t mrow = r0 + (ok ? sidx(i) : 0), mcol = c0 + jc;
            m[a * RS + b] = ok ? __ldg(p.a + mrow * p.lda + mcol) : T(0);
          }
      } else {
#pragma unroll
        for (int jj = 0; jj < JT; ++jj)
#pragma unroll
          for (int e = 0; e < V; ++e) {
            const int i = V * lane + e, jc = warp * JT + jj;
            const bool ok = i < nbI && jc < nbJ;
            const int64_t mrow = r0 + (ok ? sidx(i) : 0), mcol = c0 + jc;
            m[jj * V + e] = ok ? __ldg(p.a + mcol * p.lda + mrow) : T(0);
          }
      }
    };
    // One 128-byte line per thread and call: tile s towards L2 (full tiles only).
    auto prefetch_tile = [&](int s) {
      if (s >= k || nbI < NB) return;
      const int64_t c0 = (int64_t)blk(s) * NB;
      if (p.n - c0 < NB) return;
      constexpr int LPR = NB * (int)sizeof(T) / 128;  // lines per tile row
      for (int i = ct; i < NB * LPR; i += kT) {
        const T* ptr = p.a + ((COLTYPE ? c0 : r0) + i / LPR) * p.lda + (COLTYPE ? r0 : c0) + (i % LPR) * (128 / (int)sizeof(T));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
      }
    };

    // --- diagonal block -> S, solve order, symmetric storage (S[t][t'] = S[t'][t]); b -> bvec
    if (nbI < NB)
      for (int idx = ct; idx < NB * SP; idx += kT) S[idx] = T(0);
    if (ct < NB) {
      const T bv = ct < nbI ? p.x[(r0 + sidx(ct)) * p.incx] : T(0);
      bvec[ct] = bv;
      rbuf[ct] = bv;  // r = b when nothing precedes
    }
    if (nbI < NB) bar_sync(kBar, kT);
    {
      constexpr int PACKS = NB * NB / V;
      constexpr int PPT = PACKS / kT;  // packs per thread: 16 (float) / 8 (double)
      P v[PPT];
#pragma unroll
      for (int m = 0; m < PPT; ++m) {
        const int idx = m * kT + ct, pr = idx / (NB / V), pc = (idx % (NB / V)) * V;
        const bool use = pr < nbI && pc < nbI && (CANON_LOWER ? pc <= pr : pc + V - 1 >= pr);  // pack touches the triangle
        if (use && pc + V <= nbI) {
          v[m] = ld_nc<T, V>(p.a + (r0 + pr) * p.lda + r0 + pc);
        } else {
#pragma unroll
          for (int e = 0; e < V; ++e)
            v[m].v[e] = (use && pc + e < nbI) ? __ldg(p.a + (r0 + pr) * p.lda + r0 + pc + e) : T(0);
        }
      }
#pragma unroll
      for (int m = 0; m < PPT; ++m) {
        const int idx = m * kT + ct, pr = idx / (NB / V), pc0 = (idx % (NB / V)) * V;
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const int pc = pc0 + e;
          const bool in_tri = pr < nbI && pc < nbI && (CANON_LOWER ? pc <= pr : pc >= pr);
          if (in_tri) {
            const int sr = sidx(pr), sc = sidx(pc);
            const T val = (pr == pc && UNIT) ? T(1) : v[m].v[e];
            S[sr * SP + sc] = val;
            S[sc * SP + sr] = val;
          }
        }
      }
    }
    for (int s = ct; s < NB; s += kT)
      if (s >= nbI) S[s * SP + s] = T(1);
    prefetch_tile(k - 1);
    for (int s = 0; s < p.pf_dist; ++s) prefetch_tile(s);
    bar_sync(kBar, kT);

    // --- in-place inverse.  4x4 diagonal blocks by substitution (one column per thread) ...
    {
      T col[4];
      const int c = ct, d0 = (c / 4) * 4, lc = c % 4;
      if (ct < NB) {
        T e[4][4];
#pragma unroll
        for (int ls = 0; ls < 4; ++ls)
#pragma unroll
          for (int lt = 0; lt <= ls; ++lt) e[ls][lt] = S[(d0 + ls) * SP + d0 + lt];
#pragma unroll
        for (int ls = 0; ls < 4; ++ls) {
          T acc = (ls == lc) ? T(1) : T(0);
#pragma unroll
          for (int lt = 0; lt < ls; ++lt) acc -= e[ls][lt] * col[lt];
          col[ls] = acc / e[ls][ls];
        }
      }
      bar_sync(kBar, kT);
      if (ct < NB) {
#pragma unroll
        for (int ls = 0; ls < 4; ++ls)
          if (ls >= lc) {
            S[(d0 + ls) * SP + c] = col[ls];
            S[c * SP + d0 + ls] = col[ls];
          }
      }
      bar_sync(kBar, kT);
    }
    // ... then, for h = 4 .. NB/2, every pair [A 0; C B] of h x h blocks gets its lower-left
    // block -inv(B) (C inv(A)).  Left operands are read through the mirrored half of S.
#pragma unroll 1
    for (int h = 4; h < NB; h *= 2) {
      const int tpr = h / 4, per_pair = tpr * tpr, total = (NB / (2 * h)) * per_pair;
      const int TP = h + 4;
      for (int e = ct; e < total; e += kT) {  // Tm = C * inv(A); lanes along the rows of Tm
        const int pr = e / per_pair, rem = e % per_pair, i0 = (rem % tpr) * 4, j0 = (rem / tpr) * 4;
        const int top = pr * 2 * h, bot = top + h;
        T acc[4][4];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = T(0);
#pragma unroll
        for (int dl = 0; dl < 4; ++dl) {  // inv(A) is zero above its diagonal
          const T* rowp = S + (top + j0 + dl) * SP;
          T cv[4], av[4];
          ld4(rowp + bot + i0, cv);
          ld4(rowp + top + j0, av);
#pragma unroll
          for (int ii = 0; ii < 4; ++ii)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
              if (jj <= dl) acc[ii][jj] = cv[ii] * av[jj] + acc[ii][jj];
        }
#pragma unroll 4
        for (int l = j0 + 4; l < h; ++l) {
          const T* rowp = S + (top + l) * SP;
          T cv[4], av[4];
          ld4(rowp + bot + i0, cv);
          ld4(rowp + top + j0, av);
#pragma unroll
          for (int ii = 0; ii < 4; ++ii)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = cv[ii] * av[jj] + acc[ii][jj];
        }
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
          st4(Tm + (pr * h + i0 + ii) * TP + j0, acc[ii][0], acc[ii][1], acc[ii][2], acc[ii][3]);
      }
      bar_sync(kBar, kT);
      for (int e = ct; e < total; e += kT) {  // X = -inv(B) * Tm; lanes along the columns of X
        const int pr = e / per_pair, rem = e % per_pair, j0 = (rem % tpr) * 4, i0 = (rem / tpr) * 4;
        const int top = pr * 2 * h, bot = top + h;
        T acc[4][4];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = T(0);
#pragma unroll 4
        for (int l = 0; l < i0; ++l) {
          T bv[4], tv[4];
          ld4(S + (bot + l) * SP + bot + i0, bv);
          ld4(Tm + (pr * h + l) * TP + j0, tv);
#pragma unroll
          for (int ii = 0; ii < 4; ++ii)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = bv[ii] * tv[jj] + acc[ii][jj];
        }
#pragma unroll
        for (int dl = 0; dl < 4; ++dl) {  // inv(B) is zero above its diagonal
          T bv[4], tv[4];
          ld4(S + (bot + i0 + dl) * SP + bot + i0, bv);
          ld4(Tm + (pr * h + i0 + dl) * TP + j0, tv);
#pragma unroll
          for (int ii = 0; ii < 4; ++ii)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
              if (ii >= dl) acc[ii][jj] = bv[ii] * tv[jj] + acc[ii][jj];
        }
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
          st4(S + (bot + i0 + ii) * SP + top + j0, -acc[ii][0], -acc[ii][1], -acc[ii][2], -acc[ii][3]);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
          st4(S + (top + j0 + jj) * SP + bot + i0, -acc[0][jj], -acc[1][jj], -acc[2][jj], -acc[3][jj]);
      }
      bar_sync(kBar, kT);
    }
    // --- Ms = inv(D_k) * A_{k,k-1}: with it, x_k = inv(D_k) (b - earlier tiles) - Ms x_{k-1}, and only
    // ONE tile-times-vector product stands between the arrival of x_{k-1} and x_k.
    if (nm) {
      {  // the tile, rows in solve order, through registers into Ms
        T t1[E];
        load_tile(t1, k - 1, true);
        if (!COLTYPE) {
#pragma unroll
          for (int a = 0; a < RS; ++a)
#pragma unroll
            for (int hb = 0; hb < RS / V; ++hb) {
              P pk;
#pragma unroll
              for (int e = 0; e < V; ++e) pk.v[e] = t1[a * RS + hb * V + e];
              *reinterpret_cast<P*>(Ms + ((a / V) * H + V * rg + (a % V)) * SP + hb * H + V * cg) = pk;
            }
        } else {
#pragma unroll
          for (int jj = 0; jj < JT; ++jj)
#pragma unroll
            for (int e = 0; e < V; ++e) Ms[(V * lane + e) * SP + warp * JT + jj] = t1[jj * V + e];
        }
      }
      bar_sync(kBar, kT);
      constexpr int JW = NB * NB / (4 * kT);  // columns per thread: 16 (float) / 4 (double), 4 rows
      constexpr int NJQ = NB / JW;            // threads along a row; a thread's chunks of 4 columns are 4 * NJQ apart
      const int i0 = (ct / NJQ) * 4, j0 = (ct % NJQ) * 4;
      T acc[4][JW];
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int jj = 0; jj < JW; ++jj) acc[ii][jj] = T(0);
#pragma unroll 2
      for (int l = 0; l < i0 + 4; ++l) {  // inv(D_k) is zero above its diagonal
        T wv[4];
        ld4(S + l * SP + i0, wv);  // column l of the inverse, through the mirrored half of S
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
          if (i0 + ii < l) wv[ii] = T(0);
#pragma unroll
        for (int u = 0; u < JW / 4; ++u) {
          T tv[4];
          ld4(Ms + l * SP + j0 + u * 4 * NJQ, tv);
#pragma unroll
          for (int ii = 0; ii < 4; ++ii)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[ii][u * 4 + e] = wv[ii] * tv[e] + acc[ii][u * 4 + e];
        }
      }
      bar_sync(kBar, kT);  // everybody has read the tile: overwrite it with the product, in the loader's layout
#pragma unroll
      for (int ii = 0; ii < 4; ++ii) {
        const int i = i0 + ii, mrow = BACKWARD ? NB - 1 - i : i;
        if (!COLTYPE) {
#pragma unroll
          for (int u = 0; u < JW / 4; ++u)
            st4(Ms + mrow * SP + j0 + u * 4 * NJQ, acc[ii][u * 4], acc[ii][u * 4 + 1], acc[ii][u * 4 + 2], acc[ii][u * 4 + 3]);
        } else {
#pragma unroll
          for (int jj = 0; jj < JW; ++jj) Ms[(j0 + (jj / 4) * 4 * NJQ + jj % 4) * SP + mrow] = acc[ii][jj];
        }
      }
    }
    bar_sync(kBar, kT);

    // --- the inverse, in place, into the layout in which load_tile reads a tile: zero above the
    // diagonal, rows (row-type views) or columns (column-type views) reversed for a bottom-up solve
    for (int idx = ct; idx < NB * NB / 2; idx += kT) {
      if (!BACKWARD) {  // only the masking: two elements per thread and step
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int e2 = idx + half * (NB * NB / 2), rho = e2 / NB, gam = e2 % NB;
          if (COLTYPE ? rho > gam : gam > rho) S[rho * SP + gam] = T(0);
        }
      } else if (!COLTYPE) {  // swap row rho with row NB-1-rho
        const int rho = idx / NB, gam = idx % NB, rho2 = NB - 1 - rho;
        const T va = S[rho * SP + gam], vb = S[rho2 * SP + gam];
        S[rho * SP + gam] = gam <= rho2 ? vb : T(0);
        S[rho2 * SP + gam] = gam <= rho ? va : T(0);
      } else {  // swap column gam with column NB-1-gam
        const int rho = idx / (NB / 2), gam = idx % (NB / 2), gam2 = NB - 1 - gam;
        const T va = S[rho * SP + gam], vb = S[rho * SP + gam2];
        S[rho * SP + gam] = rho <= gam2 ? vb : T(0);
        S[rho * SP + gam2] = rho <= gam ? va : T(0);
      }
    }
    bar_sync(kBar, kT);
    // --- along the block row.  Trips 0 .. k-2 multiply the tiles A_ks by x_s and add up; trip
    // yt = k-1 multiplies inv(D_k) by r = b - sum (y); trip k multiplies Ms by x_{k-1}: x_k = y - that.
    // (Row 0 has the single trip yt = 0 and x_0 = y.)
    // two register sets take turns: while one is multiplied, the other receives the next tile
    T tile_a[E], tile_b[E];
    load_tile(tile_a, 0, false);
    const T bi = bvec[ti];
    T racc = T(0), yreg = T(0);
    // warp 0 fetches the x values a trip needs: 4 tagged words per lane, first attempt one trip ahead
    unsigned long long xw[4] = {0, 0, 0, 0};
    unsigned xneed = 0, xtag = p.tag;
    const unsigned long long* xptr = p.xbuf;
    auto x_issue = [&](int s) {
      const int64_t xi = (int64_t)blk(s) * NB + V * lane;
      xneed = 0;
#pragma unroll
      for (int e = 0; e < V; ++e)
        if (xi + e < p.n) xneed |= ((1u << WPE) - 1u) << (e * WPE);
      const bool local = CS > 1 && s >= g0;  // a row of this cluster: its block writes into xrecv
      xptr = local ? xrecv + ((s - g0) * NB + V * lane) * WPE : p.xbuf + xi * WPE;
      xtag = local ? (unsigned)s + 1u : p.tag;
      if (xneed) {
        ld_word2(xptr, xw[0], xw[1]);
        ld_word2(xptr + 2, xw[2], xw[3]);
      }
    };
    if (warp == 0 && k > 0) x_issue(yt > 0 ? 0 : k - 1);  // (yt == 0 < k only with PM: the M trip's x)

    auto trip = [&](T (&cur)[E], T (&nxt)[E], int it) {
      const bool is_y = it == yt;
      const bool is_m = nm && it == k;
      const bool crit = it == k;  // the trip that ends with x_k
      const int srow = is_m ? k - 1 : it;      // the block whose x this trip multiplies (none on trip yt)
      T* xbuf_s = xs + (it & 1) * NB;
      // first of all, off the critical path: the next tile into the other register set and a
      // tile further ahead towards L2 -- in flight while this trip waits
      if (it < k) load_tile(nxt, it + 1, false);
      prefetch_tile(it + 1 + p.pf_dist);
      if (warp == 0 && !is_y) {
        const int dist = k - srow;  // rows between this block and the producer of the x
        wt.finish(xw, xptr, xneed, xtag, dist > 2 ? (unsigned)min((dist - 2) * 200, 2000) : 0u);
        P xv;
#pragma unroll
        for (int e = 0; e < V; ++e) xv.v[e] = ((xneed >> (e * WPE)) & 1u) ? decode(xw + e * WPE, T(0)) : T(0);
        *reinterpret_cast<P*>(xbuf_s + V * lane) = xv;
      }
      bar_sync(kBar, kT);
      const T* vec = is_y ? rbuf : xbuf_s;
      T s;
      if constexpr (!COLTYPE) {
        T xv[RS], part[RS];
#pragma unroll
        for (int hb = 0; hb < RS / V; ++hb) {
          const P pk = *reinterpret_cast<const P*>(vec + hb * H + V * cg);
#pragma unroll
          for (int e = 0; e < V; ++e) xv[hb * V + e] = pk.v[e];
        }
#pragma unroll
        for (int a = 0; a < RS; ++a) {
          part[a] = T(0);
#pragma unroll
          for (int bcol = 0; bcol < RS; ++bcol) part[a] = cur[a * RS + bcol] * xv[bcol] + part[a];
        }
        s = multi_group_sum<16, RS>(part, lane);
      } else {
        P part;
#pragma unroll
        for (int e = 0; e < V; ++e) part.v[e] = T(0);
#pragma unroll
        for (int q = 0; q < JT / V; ++q) {
          const P pk = *reinterpret_cast<const P*>(vec + warp * JT + q * V);  // the warp's columns: a broadcast
#pragma unroll
          for (int u = 0; u < V; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) part.v[e] = cur[(q * V + u) * V + e] * pk.v[u] + part.v[e];
        }
        *reinterpret_cast<P*>(red + warp * NB + V * lane) = part;
        bar_sync(kBar, kT);  // (the next trip writes red only after its own first barrier)
        s = T(0);
        if (ct < NB) {
#pragma unroll
          for (int w = 0; w < kT / 32; ++w) s += red[w * NB + ct];
        }
      }
      const T out = is_m ? yreg - s : s;
      if (is_y) yreg = s;
      if (it < yt) racc += s;
      if (owner && it < yt) rbuf[ti] = bi - racc;
      {  // publishing stores: fetched on every trip, performed on the last
        const bool real = crit && owner && row_ok && !wt.dead && k != p.debug_skip;
        if (CS > 1) {  // first of all to the blocks that hold the later rows of this cluster: they
                       // are one, two, ... steps away from needing it, and a trip takes most of a step
#pragma unroll
          for (int rr = 1; rr < CS; ++rr) {
            const unsigned target = min(rank + (unsigned)rr, (unsigned)CS - 1u);
            publish_remote_if(real && rank + (unsigned)rr < (unsigned)CS, map_remote(xrecv + ((int)rank * NB + mi) * WPE, target),
                              out, (unsigned)k + 1u);
          }
        }
        publish_if(real, p.xbuf + (r0 + mi) * WPE, out, p.tag);
        st_val_if(real, p.x + (r0 + mi) * p.incx, out);
      }
      // first attempt at the x words of the next trip that needs some
      if (warp == 0) {
        if (it + 1 < yt) x_issue(it + 1);
        else if (it + 1 == yt && nm) x_issue(k - 1);
      }
    };
    int ntrips = k + 1;
    asm volatile("" : "+r"(ntrips));  // loops of two trips, not peeled copies of the last ones
#pragma unroll 1
    for (int it = 0; it < ntrips; it += 2) {
      trip(tile_a, tile_b, it);
      if (it + 1 < ntrips) trip(tile_b, tile_a, it + 1);
    }
    bar_sync(kBar, kT);  // S, bvec, rbuf, xs are reused by the next block row
  }
  if (CS > 1) cluster_sync_all();  // no block leaves while a peer may still write into its shared memory
  // The last block out leaves the control block clean (not after an abort: the caller resets).
  if (ct == 0 && ld_flag(p.ctl + kCtlTrsvAbort) == 0u) {
    __threadfence();
    const unsigned d = atomicAdd(p.ctl + kCtlTrsvDone, 1u);
    if (d == gridDim.x - 1) {
      p.ctl[kCtlTrsvTicket] = 0u;
      p.ctl[kCtlTrsvDone] = 0u;
    }
  }
}

template <typename T>
constexpr size_t front_smem_bytes(int cs) {
  constexpr int NB = Geo<T>::NB;
  constexpr int SP = NB + 16 / (int)sizeof(T);
  return sizeof(T) * (size_t)((cs > 1 ? 1 : 2) * NB * SP + (NB / 2) * (NB / 2 + 4) + (4 + kT / 32) * NB) +
         (cs > 1 ? (size_t)cs * NB * Words<T>::N * 8 : 0);
}

constexpr int kCluster = 8;

// Launches the kernel; with clusters when the device can hold at least one (the grid is then a
// whole number of clusters, no more than can be resident), else block by block.
template <typename T, bool COLTYPE, bool BACKWARD, bool UNIT>
static int launch_one(const Launch& l, const FrontArgs<T>& args, int nb, bool want_cluster) {
  if (want_cluster) {
    constexpr size_t smem = front_smem_bytes<T>(kCluster);
    auto kern = trsv_front_kernel<T, COLTYPE, BACKWARD, UNIT, kCluster>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess) {
      cudaLaunchConfig_t cfg = {};
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = kCluster;
      at[0].val.clusterDim.y = 1;
      at[0].val.clusterDim.z = 1;
      cfg.gridDim = dim3(kCluster);
      cfg.blockDim = dim3(kT);
      cfg.dynamicSmemBytes = smem;
      cfg.stream = l.stream;
      cfg.attrs = at;
      cfg.numAttrs = 1;
      int max_clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&max_clusters, kern, &cfg) == cudaSuccess && max_clusters > 0) {
        const int groups = (nb + kCluster - 1) / kCluster;
        const int clusters = groups < max_clusters ? groups : max_clusters;
        cfg.gridDim = dim3(clusters * kCluster);
        const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, args);
        ++g_launch_count;
        if (e == cudaSuccess) return B2_STATUS_OK;
        (void)cudaGetLastError();
        return B2_STATUS_LAUNCH_FAILED;
      }
    }
    (void)cudaGetLastError();
  }
  constexpr size_t smem = front_smem_bytes<T>(1);
  auto kern = trsv_front_kernel<T, COLTYPE, BACKWARD, UNIT, 1>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    (void)cudaGetLastError();
    return B2_STATUS_LAUNCH_FAILED;
  }
  const int grid = nb < sm_count() ? nb : sm_count();
  launch_chained(kern, dim3(grid), dim3(kT), smem, l.stream, args);
  return check_launch();
}

template <typename T, bool COLTYPE, bool BACKWARD>
static int launch_diag(const Launch& l, const FrontArgs<T>& args, int nb, bool want_cluster, bool unit) {
  return unit ? launch_one<T, COLTYPE, BACKWARD, true>(l, args, nb, want_cluster)
              : launch_one<T, COLTYPE, BACKWARD, false>(l, args, nb, want_cluster);
}

}  // namespace tf

template <typename T>
int trsv_front_try(const Launch& l, bool coltype, bool backward, bool unit, int64_t n, const T* a, int64_t lda,
                   T* xbase, int64_t incx, unsigned tag, bool* handled) {
  using namespace tf;
  constexpr int NB = Geo<T>::NB, V = Geo<T>::V, WPE = Words<T>::N;
  *handled = false;
  if (!knob(kKnobTrsvFront)) return B2_STATUS_OK;
  // (knob value 1 keeps column-type views on the block-row kernel)
  if (coltype && knob(kKnobTrsvFront) < 2) return B2_STATUS_OK;
  if (!aligned_to(a, 16) || lda % V != 0) return B2_STATUS_OK;
  const int64_t nb64 = (n + NB - 1) / NB;
  if (nb64 > 0x3fffffff) return B2_STATUS_OK;
  const int nb = (int)nb64;
  const int grid = nb < sm_count() ? nb : sm_count();
  const size_t xbuf_words = (size_t)nb * NB * WPE;
  if (xbuf_words * 8 > l.scratch_bytes) return B2_STATUS_OK;
  FrontArgs<T> args = {};
  args.a = a;
  args.lda = lda;
  args.n = n;
  args.x = xbase;
  args.incx = incx;
  args.xbuf = reinterpret_cast<unsigned long long*>(l.scratch);
  args.ctl = l.ctl;
  args.nb = nb;
  {  // keep the prefetched-but-unused tiles of all blocks within a fraction of L2
    const int64_t tile_bytes = (int64_t)NB * NB * sizeof(T);
    // (measured at n = 11520 / 8192: one or two tiles ahead is best -- 142 / 167 us against 148 / 171 us
    // at eight ahead and 163 / 182 us with none -- so a nonzero budget always buys the first tile)
    int64_t d = knob(kKnobTrsvPrefetchBytes) / (tile_bytes * grid);
    if (d < 1 && knob(kKnobTrsvPrefetchBytes) > 0) d = 1;
    args.pf_dist = (int)(d < 0 ? 0 : d > 16 ? 16 : d);
  }
  args.tag = tag;
  args.wait_limit = l.wait_limit;
  args.device_status = l.device_status;
  args.debug_skip = (int)knob(kKnobTrsvDebugSkip);
  // the premultiplied last tile pays in double (64-row blocks: 167 us against 182 us) and costs in
  // float (143 / 141 us with it, 142 / 134 us without); a knob value >= 0 forces it from that row on
  {
    const int64_t pm = knob(kKnobTrsvPmFrom);
    args.pm_from = pm >= 0 ? (int)(pm > 0x3fffffff ? 0x3fffffff : pm) : (sizeof(T) == 8 ? 16 : 0x3fffffff);
  }
  *handled = true;
#ifdef B2_DEBUG_BOUNDS
  {  // (this translation unit has its own copy of the range table)
    Launch lc = l;
    B2_DBG_COMMIT(lc);
  }
#endif
  // (measured at n = 11520 / 8192: block by block with the premultiplied last tile is the
  // fastest form for both precisions -- float 156-162 us against 168-175 us in clusters of 8,
  // double 180 us against 216 us -- so clusters are off by default)
  const bool want_cluster = nb >= 2 && (knob(kKnobTrsvCluster) >= 2 || (knob(kKnobTrsvCluster) == 1 && sizeof(T) == 4));
  if (coltype)
    return backward ? launch_diag<T, true, true>(l, args, nb, want_cluster, unit)
                    : launch_diag<T, true, false>(l, args, nb, want_cluster, unit);
  return backward ? launch_diag<T, false, true>(l, args, nb, want_cluster, unit)
                  : launch_diag<T, false, false>(l, args, nb, want_cluster, unit);
}

template int trsv_front_try<float>(const Launch&, bool, bool, bool, int64_t, const float*, int64_t, float*, int64_t,
                                   unsigned, bool*);
template int trsv_front_try<double>(const Launch&, bool, bool, bool, int64_t, const double*, int64_t, double*, int64_t,
                                    unsigned, bool*);

}  // namespace b2
