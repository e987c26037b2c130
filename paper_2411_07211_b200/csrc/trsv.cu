// trsv: solve op(A) x = b in place (Section 6.2.2; same option space as trmv).
//
// Blocked substitution with a dependency-ordered diagonal-block solve.  The unknowns are cut
// into blocks of 128 (float) or 64 (double); thread blocks draw a ticket k = 0, 1, ... (the solve order: top-down for
// an effectively lower-triangular op(A), bottom-up for an upper one).  Block k
//   1. stages its diagonal block in shared memory and inverts it there, in place, by
//      recursive doubling (none of this depends on the solve),
//   2. streams the off-diagonal part of its block row (or block column when op(A)'s rows are
//      strided in memory) as tiles of 64 source unknowns in solve order; 16 compute warps keep the next
//      tile's matrix data in flight in registers and tiles further ahead are pulled into L2,
//      all BEFORE the x values they multiply exist,
//   3. receives those x values through a side buffer in the workspace in which every value is
//      published as 64-bit words {32 payload bits, 32-bit call tag}: data and "ready" flag
//      travel in one store, so the consumer polls the data itself and neither side needs a
//      fence or a second round trip through L2.  A 17th warp does nothing but poll (bounded)
//      and hands decoded values to the compute warps through a ring of shared-memory buffers
//      (named barriers), so polling latency never stalls the streaming warps, and only one warp
//      per block loads the hot words -- a herd of pollers would swamp the L2 slice that
//      holds them,
//   4. forms r = b - sum, multiplies by the inverted diagonal block, publishes its values
//      and writes them to the caller's x.
// The chain of dependent block solves makes the routine latency-bound: each step costs one L2
// store->load hand-over plus a block-sized matvec.  Tickets are drawn in launch order, so a block
// only ever waits for blocks that are already running: no co-residency assumption, no
// deadlock.  If the polls exceed the iteration limit the block records B2_STATUS_TIMEOUT in
// *device_status and leaves without publishing (its dependants then time out too).
//
// Accuracy note: the diagonal blocks are applied through their explicit inverses (computed in
// the working precision).  For diagonal blocks of moderate condition number this is as
// accurate as substitution; it is the usual trade for removing the dependent steps inside a block.
#include <atomic>

#include "common.cuh"
#include "trsv_front.cuh"

namespace b2 {

constexpr int kSB = 64;               // unknowns per source tile
constexpr int kCW = 16;               // compute warps
constexpr int kCT = kCW * 32;         // compute threads
constexpr int kTT = kCT + 32;         // + one polling warp
constexpr int kXB = 4;                // x buffers between the polling warp and the compute warps
constexpr int kBarFull = 1;           // named barriers kBarFull + b, kBarEmpty + b
constexpr int kBarEmpty = 1 + kXB;

__device__ __forceinline__ unsigned long long ld_word(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_word(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// Named barriers.  The polling loop in front of them lets lanes leave at different iterations, so
// the warp is re-converged first and the forms that count threads (not whole warps) are used.
__device__ __forceinline__ void bar_sync(int id, int count) {
  __syncwarp();
  asm volatile("barrier.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(int id, int count) {
  __syncwarp();
  asm volatile("barrier.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}

template <typename T>
struct TrsvArgs {
  const T* a;
  int64_t lda, n;
  T* x;  // base per vec_base()
  int64_t incx;
  unsigned long long* xbuf;  // published solution: 1 (float) or 2 (double) tagged words per unknown
  unsigned* ticket;
  int nb;   // blocks of trsv_block<T>() unknowns
  int nsb;  // 64-blocks (source tiles)
  unsigned tag;
  unsigned long long wait_limit;
  int* device_status;
  int debug_skip;
  int pf_dist;  // L2 prefetch distance in tiles
};

// Polling state of the polling warp's lanes: a total budget of polls for the whole kernel.
struct Poller {
  unsigned long long budget;
  volatile int* abort_flag;  // shared memory
  int* device_status;
  unsigned tag;
  unsigned backoff_ns;  // sleep after a miss (0 when the block is next in line)

  // Loads NW tagged words (null pointer = masked, counts as ready) with all loads in flight at
  // once, then re-reads only the ones whose tag is not this call's until all are ready.
  template <int NW>
  __device__ __forceinline__ void wait_words(unsigned long long (&w)[NW], const unsigned long long* const (&ptr)[NW]) {
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = ptr[i] ? ld_word(ptr[i]) : ((unsigned long long)tag << 32);
    for (;;) {
      bool ok = true;
#pragma unroll
      for (int i = 0; i < NW; ++i) ok = ok && ((unsigned)(w[i] >> 32) == tag);
      if (ok) break;
      if (budget == 0 || *abort_flag) {
        if (!*abort_flag) {
          *abort_flag = 1;
          if (device_status) atomicExch(device_status, (int)B2_STATUS_TIMEOUT);
        }
        break;
      }
      --budget;
      if (backoff_ns) __nanosleep(backoff_ns);
#pragma unroll
      for (int i = 0; i < NW; ++i)
        if ((unsigned)(w[i] >> 32) != tag) w[i] = ld_word(ptr[i]);
    }
  }
};

__device__ __forceinline__ void publish(unsigned long long* xb, int64_t i, float v, unsigned tag) {
  st_word(xb + i, ((unsigned long long)tag << 32) | __float_as_uint(v));
}
__device__ __forceinline__ void publish(unsigned long long* xb, int64_t i, double v, unsigned tag) {
  const unsigned long long b = (unsigned long long)__double_as_longlong(v);
  st_word(xb + 2 * i, ((unsigned long long)tag << 32) | (b & 0xffffffffull));
  st_word(xb + 2 * i + 1, ((unsigned long long)tag << 32) | (b >> 32));
}

// Tagged words of unknown i: 1 for float, 2 for double (low half first).
template <typename T>
struct Words {
  static constexpr int N = sizeof(T) / 4;
};
__device__ __forceinline__ float decode(const unsigned long long* w, float) { return __uint_as_float((unsigned)w[0]); }
__device__ __forceinline__ double decode(const unsigned long long* w, double) {
  return __longlong_as_double((long long)(((unsigned long long)(unsigned)w[1] << 32) | (unsigned)w[0]));
}

// COLTYPE: op(A)'s rows are columns of the stored row-major view.  BACKWARD: solve bottom-up.
// NB = unknowns per thread block: 128 for float, 64 for double (the diagonal-block work grows with
// NB^2 per unknown, and a 128 x 128 double block with its inverse would not fit in shared memory).
template <typename T, int NB, int V, bool COLTYPE, bool BACKWARD, bool UNIT>
__global__ void __launch_bounds__(kTT) trsv_kernel(const TrsvArgs<T> p) {
  grid_dep_wait();
  grid_dep_launch();
  // A tile is NB own unknowns x 64 source unknowns; in memory it is NB rows x 64 columns
  // (rows of op(A) contiguous) or 64 rows x NB columns (COLTYPE).
  constexpr int WS = NB + 8;        // row stride of W (16-byte row starts, conflict-free packs)
  constexpr int TPB = NB / kSB;     // source tiles a solved block publishes at once
  constexpr int TROWS = COLTYPE ? kSB : NB, TCOLS = COLTYPE ? NB : kSB;
  constexpr int LPR = (TCOLS / V) >= 32 ? 32 : TCOLS / V;
  constexpr int CU = TCOLS / (LPR * V);
  constexpr int G = 32 / LPR;
  constexpr int RU = TROWS / (kCW * G);
  constexpr bool CANON_LOWER = (COLTYPE == BACKWARD);  // stored triangle in the row-major view
  constexpr int WPE = Words<T>::N;
  using P = Pack<T, V>;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* W = reinterpret_cast<T*>(smem_raw);  // diagonal block in solve order, W[s*WS + t], then its inverse
  T* racc = W + NB * WS;                // r = b - (sum over solved blocks), per unknown (solve order)
  T* bvec = racc + NB;                   // right-hand side b (solve order)
  T* xsm = bvec + NB;                    // [kXB][kSB] x values handed over by the polling warp
  T* colsm = xsm + kXB * kSB;             // [kCW][NB], COLTYPE only
  __shared__ unsigned s_ticket;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool poller = warp == kCW;
  const int g = lane / LPR, q = lane % LPR;
  if (tid == 0) {
    s_ticket = atomicAdd(p.ticket, 1u);
    s_abort = 0;
  }
  __syncthreads();
  const int k = (int)s_ticket;  // position in the solve order
  if (k >= p.nb) {              // dirty control block (a previous call timed out and was not reset)
    if (tid == 0 && p.device_status) atomicExch(p.device_status, (int)B2_STATUS_TIMEOUT);
    return;
  }
  const int I = BACKWARD ? p.nb - 1 - k : k;  // block index in memory
  const int64_t r0 = (int64_t)I * NB;
  const int nbI = (int)min((int64_t)NB, p.n - r0);
  auto solve_idx = [&](int i) { return BACKWARD ? nbI - 1 - i : i; };
  // source tiles (64 unknowns each) in solve order: s -> global 64-block index
  const int nsrc = BACKWARD ? max(0, p.nsb - TPB * I - TPB) : TPB * I;
  auto src_block = [&](int s) { return BACKWARD ? p.nsb - 1 - s : s; };

  int lr[RU];
#pragma unroll
  for (int ru = 0; ru < RU; ++ru) lr[ru] = (ru * kCW + warp) * G + g;

  auto load_tile = [&](P (&av)[RU][CU], int s) {
    const int64_t c0 = (int64_t)src_block(s) * kSB;
    const int nbJ = (int)min((int64_t)kSB, p.n - c0);
    const int64_t rbase = COLTYPE ? c0 : r0, cbase = COLTYPE ? r0 : c0;
    const int nr = COLTYPE ? nbJ : nbI, nc = COLTYPE ? nbI : nbJ;
    if (nr == TROWS && nc == TCOLS) {
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u) av[ru][u] = ld_nc<T, V>(p.a + (rbase + lr[ru]) * p.lda + cbase + (u * LPR + q) * V);
    } else {
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u)
#pragma unroll
          for (int e = 0; e < V; ++e) {
            const int lc = (u * LPR + q) * V + e;
            av[ru][u].v[e] = (lr[ru] < nr && lc < nc) ? __ldg(p.a + (rbase + lr[ru]) * p.lda + cbase + lc) : T(0);
          }
    }
  };
  // Tiles further ahead are pulled into L2 while the block waits for the solve front, so DRAM
  // streams continuously instead of in bursts locked to the front (one 128-byte line per thread).
  auto prefetch_tile = [&](int s) {
    if (s >= nsrc) return;
    const int64_t c0 = (int64_t)src_block(s) * kSB;
    if (p.n - c0 < kSB || nbI < NB) return;  // ragged tiles are not worth it
    const int64_t rbase = COLTYPE ? c0 : r0, cbase = COLTYPE ? r0 : c0;
    constexpr int LINES = TCOLS * (int)sizeof(T) / 128;
    for (int i = tid; i < TROWS * LINES; i += kCT) {
      const T* ptr = p.a + (rbase + i / LINES) * p.lda + cbase + (i % LINES) * (128 / (int)sizeof(T));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
    }
  };

  // The first tile's matrix data goes in flight before anything else.
  P cur[RU][CU], nxt[RU][CU];
  if (!poller) {
    if (nsrc > 0) load_tile(nxt, 0);
    for (int s = 1; s < 1 + p.pf_dist; ++s) prefetch_tile(s);
  }

  // 1a. diagonal block -> W (zero elsewhere, identity on unused / unit diagonal); b -> bvec
  for (int idx = tid; idx < NB * WS; idx += kTT) W[idx] = T(0);
  if (tid < NB) {
    bvec[tid] = tid < nbI ? p.x[(r0 + solve_idx(tid)) * p.incx] : T(0);
    racc[tid] = bvec[tid];  // r = b when nothing precedes; entries past a ragged block stay zero
  }
  __syncthreads();
  for (int base = 0; base < NB * NB; base += 8 * kTT) {  // 8 independent loads in flight per thread
    T v[8];
    bool use[8];
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int idx = base + m * kTT + tid;
      const int pr = idx / NB, pc = idx % NB;  // position inside the stored block
      use[m] = idx < NB * NB && pr < nbI && pc < nbI && (CANON_LOWER ? (pc <= pr) : (pc >= pr)) &&
               !(UNIT && pr == pc);
      v[m] = use[m] ? __ldg(p.a + (r0 + pr) * p.lda + r0 + pc) : T(0);
    }
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int idx = base + m * kTT + tid;
      const int pr = idx / NB, pc = idx % NB;
      if (use[m]) {
        const int sr = solve_idx(pr), sc = solve_idx(pc);
        if (COLTYPE) W[sc * WS + sr] = v[m];
        else W[sr * WS + sc] = v[m];
      }
    }
  }
  for (int s = tid; s < NB; s += kTT)
    if (UNIT || s >= nbI) W[s * WS + s] = T(1);
  __syncthreads();

  // 1b. in-place inverse by recursive doubling.  4x4 diagonal blocks: one column per thread,
  // block held in registers, substitution on e_c.  Then, for h = 4 .. 64, every pair
  // [A 0; C B] of h x h blocks gets its lower-left block -B^-1 (C A^-1); the intermediate
  // C A^-1 is parked in the (unused) upper triangle at the transposed position.
  {
    T col[4];
    const int c = tid, d0 = (c / 4) * 4, lc = c % 4;
    if (tid < NB) {
      T e[4][4];
#pragma unroll
      for (int ls = 0; ls < 4; ++ls)
#pragma unroll
        for (int lt = 0; lt <= ls; ++lt) e[ls][lt] = W[(d0 + ls) * WS + d0 + lt];
#pragma unroll
      for (int ls = 0; ls < 4; ++ls) {
        T acc = (ls == lc) ? T(1) : T(0);
#pragma unroll
        for (int lt = 0; lt < ls; ++lt) acc -= e[ls][lt] * col[lt];
        col[ls] = acc / e[ls][ls];
      }
    }
    __syncthreads();
    if (tid < NB) {
#pragma unroll
      for (int ls = 0; ls < 4; ++ls) W[(d0 + ls) * WS + c] = col[ls];  // zero above the diagonal
    }
    __syncthreads();
  }
#pragma unroll 1
  for (int h = 4; h < NB; h *= 2) {  // 4x4 register tiles: 8 shared-memory loads per 16 multiply-adds
    const int tpr = h / 4, per_pair = tpr * tpr, total = (NB / (2 * h)) * per_pair;
    for (int e = tid; e < total; e += kTT) {  // Tm = C * A^-1  (A^-1 is zero above its diagonal)
      const int pr = e / per_pair, i0 = ((e % per_pair) / tpr) * 4, j0 = (e % tpr) * 4;
      const int top = pr * 2 * h, bot = top + h;
      T acc[4][4];
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = T(0);
#pragma unroll 4
      for (int l = j0; l < h; ++l) {
        T cv[4], av[4];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii) cv[ii] = W[(bot + i0 + ii) * WS + top + l];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) av[jj] = W[(top + l) * WS + top + j0 + jj];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = cv[ii] * av[jj] + acc[ii][jj];
      }
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) W[(top + j0 + jj) * WS + bot + i0 + ii] = acc[ii][jj];
    }
    __syncthreads();
    for (int e = tid; e < total; e += kTT) {  // X = -B^-1 * Tm, written over C (B^-1 zero above its diagonal)
      const int pr = e / per_pair, i0 = ((e % per_pair) / tpr) * 4, j0 = (e % tpr) * 4;
      const int top = pr * 2 * h, bot = top + h;
      T acc[4][4];
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = T(0);
#pragma unroll 4
      for (int l = 0; l < i0 + 4; ++l) {
        T bv[4], tv[4];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii) bv[ii] = W[(bot + i0 + ii) * WS + bot + l];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) tv[jj] = W[(top + j0 + jj) * WS + bot + l];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = bv[ii] * tv[jj] + acc[ii][jj];
      }
#pragma unroll
      for (int ii = 0; ii < 4; ++ii)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) W[(bot + i0 + ii) * WS + top + j0 + jj] = -acc[ii][jj];
    }
    __syncthreads();
    for (int e = tid; e < (NB / (2 * h)) * h * h; e += kTT) {  // scrub the parked intermediates
      const int pr = e / (h * h), i = (e % (h * h)) / h, j = e % h;
      W[(pr * 2 * h + j) * WS + pr * 2 * h + h + i] = T(0);
    }
    __syncthreads();
  }
  // The finished inverse: float blocks keep their share in registers (the matvec is then
  // free of shared-memory traffic), double blocks read it from shared memory in 16-byte packs.
  constexpr int VL = 16 / (int)sizeof(T);          // elements per pack
  constexpr int TPU = kCT / NB;                   // threads per unknown
  constexpr int NPK = NB / (TPU * VL);            // packs per thread
  constexpr bool WREG = sizeof(T) == 4;
  Pack<T, VL> wreg[WREG ? NPK : 1];
  if (WREG && !poller) {
    const int ms = tid / TPU, part = tid % TPU;
#pragma unroll
    for (int m = 0; m < NPK; ++m) wreg[m] = *reinterpret_cast<const Pack<T, VL>*>(&W[ms * WS + VL * (part + TPU * m)]);
  }

  // 2./3. off-diagonal tiles in solve order
  T rowacc[RU];
  T colacc[CU][V];
#pragma unroll
  for (int ru = 0; ru < RU; ++ru) rowacc[ru] = T(0);
#pragma unroll
  for (int u = 0; u < CU; ++u)
#pragma unroll
    for (int e = 0; e < V; ++e) colacc[u][e] = T(0);

  if (poller) {
    Poller poll;
    poll.budget = p.wait_limit ? p.wait_limit : (1ull << 20);
    poll.abort_flag = &s_abort;
    poll.device_status = p.device_status;
    poll.tag = p.tag;
    // A solved block publishes NB unknowns = TPB source tiles at once, so the tiles are polled TPB
    // at a time: one round trip through L2 serves them all.
    constexpr int EPL = TPB * kSB / 32;  // unknowns per lane and poll
    for (int s = 0; s < nsrc; s += TPB) {
#pragma unroll
      for (int t = 0; t < TPB; ++t)  // the compute warps are done with these buffers
        if (s + t < nsrc && s + t >= kXB) bar_sync(kBarEmpty + (s + t) % kXB, kTT);
      // blocks further from the front sleep between polls so that only the next in line spins
      const int last = min(s + TPB - 1, nsrc - 1);
      const int dist = k - (BACKWARD ? p.nb - 1 - src_block(last) / TPB : src_block(last) / TPB);
      poll.backoff_ns = dist > 1 ? (unsigned)min(dist - 1, 64) * 500u : 0u;
      unsigned long long w[EPL * WPE];
      const unsigned long long* wp[EPL * WPE];
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int el = lane * EPL + j, t = el / kSB, lc = el % kSB;  // tile of the group, position in it
        const int64_t u = (int64_t)src_block(min(s + t, nsrc - 1)) * kSB + lc;
        const bool valid = s + t < nsrc && u < p.n;
#pragma unroll
        for (int h = 0; h < WPE; ++h) wp[j * WPE + h] = valid ? p.xbuf + u * WPE + h : nullptr;
      }
      poll.wait_words(w, wp);
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int el = lane * EPL + j, t = el / kSB, lc = el % kSB;
        // (a tile past the end of the row has no buffer of its own: the slot it would map to may
        // still be read by the compute warps, four tiles behind)
        if (s + t < nsrc) xsm[((s + t) % kXB) * kSB + lc] = wp[j * WPE] ? decode(&w[j * WPE], T(0)) : T(0);
      }
      __threadfence_block();
#pragma unroll
      for (int t = 0; t < TPB; ++t)
        if (s + t < nsrc) bar_arrive(kBarFull + (s + t) % kXB, kTT);
    }
  } else {
#pragma unroll 1
    for (int s = 0; s < nsrc; ++s) {
      const int b = s % kXB;
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u) cur[ru][u] = nxt[ru][u];
      if (s + 1 < nsrc) {
        load_tile(nxt, s + 1);
        prefetch_tile(s + 1 + p.pf_dist);
      }
      bar_sync(kBarFull + b, kTT);  // x values of this tile are in xsm[b]
      const T* xg = xsm + b * kSB;
      if (COLTYPE) {
        T xr[RU];
#pragma unroll
        for (int ru = 0; ru < RU; ++ru) xr[ru] = xg[lr[ru]];
#pragma unroll
        for (int ru = 0; ru < RU; ++ru)
#pragma unroll
          for (int u = 0; u < CU; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) colacc[u][e] = cur[ru][u].v[e] * xr[ru] + colacc[u][e];
      } else {
        T xs[CU][V];
#pragma unroll
        for (int u = 0; u < CU; ++u)
#pragma unroll
          for (int e = 0; e < V; ++e) xs[u][e] = xg[(u * LPR + q) * V + e];
#pragma unroll
        for (int ru = 0; ru < RU; ++ru)
#pragma unroll
          for (int u = 0; u < CU; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) rowacc[ru] = cur[ru][u].v[e] * xs[u][e] + rowacc[ru];
      }
      if (s + kXB < nsrc) bar_arrive(kBarEmpty + b, kTT);  // only if the polling warp will wait for it
    }

    // per-unknown sums -> racc (solve order)
    if (COLTYPE) {
#pragma unroll
      for (int u = 0; u < CU; ++u)
#pragma unroll
        for (int e = 0; e < V; ++e) {
          const T s = cross_group_sum<LPR>(colacc[u][e]);
          if (g == 0) colsm[warp * NB + (u * LPR + q) * V + e] = s;
        }
    } else {
      constexpr int LPV = LPR / RU;  // lanes left per row after the reduction
      const T s = multi_group_sum<LPR, RU>(rowacc, lane);
      const int i = ((q / LPV) * kCW + warp) * G + g;
      if (q % LPV == 0 && i < nbI) racc[solve_idx(i)] = bvec[solve_idx(i)] - s;
    }
  }
  __syncthreads();
  if (COLTYPE) {
    if (tid < nbI) {
      T s = colsm[tid];
#pragma unroll
      for (int w = 1; w < kCW; ++w) s += colsm[w * NB + tid];
      racc[solve_idx(tid)] = bvec[solve_idx(tid)] - s;
    }
    __syncthreads();
  }
  if (s_abort) return;  // a wait ran out: publish nothing, dependants will time out too

  // 4. x = W * r: 4 threads per unknown, then publish and write back
  if (!poller) {
    const int s = tid / TPU, part = tid % TPU;
    T accv[VL];  // independent chains
#pragma unroll
    for (int e = 0; e < VL; ++e) accv[e] = T(0);
#pragma unroll
    for (int m = 0; m < NPK; ++m) {
      const int t0 = VL * (part + TPU * m);
      if (WREG) {
        const Pack<T, VL> rv = *reinterpret_cast<const Pack<T, VL>*>(&racc[t0]);
#pragma unroll
        for (int e = 0; e < VL; ++e) accv[e] = wreg[m].v[e] * rv.v[e] + accv[e];
      } else if (t0 <= s) {  // W is zero above the diagonal
        const Pack<T, VL> wv = *reinterpret_cast<const Pack<T, VL>*>(&W[s * WS + t0]);
        const Pack<T, VL> rv = *reinterpret_cast<const Pack<T, VL>*>(&racc[t0]);
#pragma unroll
        for (int e = 0; e < VL; ++e) accv[e] = wv.v[e] * rv.v[e] + accv[e];
      }
    }
    T acc = accv[0];
#pragma unroll
    for (int e = 1; e < VL; ++e) acc += accv[e];
#pragma unroll
    for (int m = 1; m < TPU; m <<= 1) acc += shfl_xor(acc, m);
    if (part == 0 && s < nbI && k != p.debug_skip) {
      const int i = solve_idx(s);
      publish(p.xbuf, r0 + i, acc, p.tag);
      p.x[(r0 + i) * p.incx] = acc;
    }
  }
  if (k == p.nb - 1 && tid == 0) *p.ticket = 0u;  // all tickets are drawn: leave the control block clean
}

template <typename T>
constexpr int trsv_block() {
  return sizeof(T) == 4 ? 128 : 64;
}
template <typename T, bool COLTYPE>
constexpr size_t trsv_smem_bytes() {
  constexpr int NB = trsv_block<T>();
  return sizeof(T) * (NB * (NB + 8) + 2 * NB + kXB * kSB + (COLTYPE ? kCW : 0) * NB);
}

template <typename T, int V, bool COLTYPE, bool BACKWARD, bool UNIT>
static int trsv_launch_one(const Launch& l, const TrsvArgs<T>& args) {
  constexpr size_t smem = trsv_smem_bytes<T, COLTYPE>();
  auto kern = trsv_kernel<T, trsv_block<T>(), V, COLTYPE, BACKWARD, UNIT>;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    (void)cudaGetLastError();
    return B2_STATUS_LAUNCH_FAILED;
  }
  launch_chained(kern, dim3(args.nb), dim3(kTT), smem, l.stream, args);
  return check_launch();
}

template <typename T, int V, bool COLTYPE, bool BACKWARD>
static int trsv_launch(const Launch& l, const TrsvArgs<T>& args, bool unit) {
  if (unit) return trsv_launch_one<T, V, COLTYPE, BACKWARD, true>(l, args);
  return trsv_launch_one<T, V, COLTYPE, BACKWARD, false>(l, args);
}

template <typename T, int V>
static int trsv_variant(const Launch& l, const TrsvArgs<T>& args, bool coltype, bool backward, bool unit) {
  if (coltype) return backward ? trsv_launch<T, V, true, true>(l, args, unit) : trsv_launch<T, V, true, false>(l, args, unit);
  return backward ? trsv_launch<T, V, false, true>(l, args, unit) : trsv_launch<T, V, false, false>(l, args, unit);
}

// Call tags: unique per call within the process, never 0, so that words left in the workspace
// by earlier calls can never look "ready".
static unsigned next_tag() {
  static std::atomic<unsigned> counter{0x2b7e1516u};
  unsigned t = counter.fetch_add(1u) + 1u;
  if (t == 0u) t = counter.fetch_add(1u) + 1u;
  return t;
}

template <typename T>
static int trsv_impl(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const T* a, int64_t lda,
                     T* x, int64_t incx) {
  if (order != B2_ROW_MAJOR && order != B2_COL_MAJOR) return -1;
  if (uplo != B2_UPPER && uplo != B2_LOWER) return -2;
  if (trans != B2_NO_TRANS && trans != B2_TRANS) return -3;
  if (diag != B2_NON_UNIT && diag != B2_UNIT) return -4;
  if (n < 0) return -5;
  if (n > 0 && (a == nullptr || !aligned_to(a, sizeof(T)))) return -6;
  if (lda < (n > 1 ? n : 1)) return -7;
  if (incx == 0) return -9;
  if (n > 0 && (x == nullptr || !aligned_to(x, sizeof(T)))) return -8;
  Launch l;
  if (int st = make_launch(ctx, &l)) return st;
  if (n == 0) return B2_STATUS_OK;
  B2_DBG_RANGE(l, a, (size_t)((n - 1) * lda + n) * sizeof(T));
  B2_DBG_VEC(l, x, n, incx);
  B2_DBG_COMMIT(l);
  // op(A) lower triangular <=> forward substitution
  const bool eff_lower = (uplo == B2_LOWER) != (trans == B2_TRANS);
  // rows of op(A) contiguous in memory <=> row-major N or column-major T
  const bool coltype = (order == B2_ROW_MAJOR) != (trans == B2_NO_TRANS);
  const bool unit = diag == B2_UNIT;
  const unsigned tag = next_tag();
  {
    bool handled = false;
    const int st = trsv_front_try<T>(l, coltype, !eff_lower, unit, n, a, lda, vec_base(x, n, incx), incx, tag, &handled);
    if (handled) return st;
  }
  constexpr int NB = trsv_block<T>();
  if ((n + NB - 1) / NB > 0x3fffffff) return B2_STATUS_NOT_IMPLEMENTED;
  const size_t xbuf_bytes = (size_t)n * 8 * (sizeof(T) / 4);
  if (l.scratch_bytes < xbuf_bytes) return B2_STATUS_WORKSPACE_TOO_SMALL;
  TrsvArgs<T> args = {};
  args.a = a;
  args.lda = lda;
  args.n = n;
  args.x = vec_base(x, n, incx);
  args.incx = incx;
  args.xbuf = reinterpret_cast<unsigned long long*>(l.scratch);
  args.ticket = l.ctl + kCtlTrsvTicket;
  args.nb = (int)((n + NB - 1) / NB);
  args.nsb = (int)((n + kSB - 1) / kSB);
  args.tag = tag;
  args.wait_limit = l.wait_limit;
  args.device_status = l.device_status;
  args.debug_skip = (int)knob(kKnobTrsvDebugSkip);
  {  // keep the prefetched-but-unused tiles of all blocks within a fraction of L2
    const int64_t tile_bytes = (int64_t)NB * kSB * sizeof(T);
    int64_t d = knob(kKnobTrsvPrefetchBytes) / (tile_bytes * args.nb);
    args.pf_dist = (int)(d < 0 ? 0 : d > 64 ? 64 : d);
  }
  constexpr int V = VecLen<T>::value;
  if (aligned_to(a, 16) && lda % V == 0) return trsv_variant<T, V>(l, args, coltype, !eff_lower, unit);
  return trsv_variant<T, 1>(l, args, coltype, !eff_lower, unit);
}

}  // namespace b2

extern "C" {
int b2_strsv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const float* a, int64_t lda,
             float* x, int64_t incx) {
  return b2::trsv_impl<float>(ctx, order, uplo, trans, diag, n, a, lda, x, incx);
}
int b2_dtrsv(const b2_ctx* ctx, int order, int uplo, int trans, int diag, int64_t n, const double* a, int64_t lda,
             double* x, int64_t incx) {
  return b2::trsv_impl<double>(ctx, order, uplo, trans, diag, n, a, lda, x, incx);
}
}
