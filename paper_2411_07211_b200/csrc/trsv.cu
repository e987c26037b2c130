// trsv: solve op(A) x = b in place (Section 6.2.2; same option space as trmv).
//
// Blocked substitution with a dependency-ordered diagonal-block solve.  The unknowns are cut
// into blocks of 64.  Thread blocks (512 threads) draw a ticket k = 0, 1, ... (the solve order: top-down for
// an effectively lower-triangular op(A), bottom-up for an upper one); block k
//   1. stages its 64x64 diagonal block in shared memory and inverts it there (recursive
//      doubling, all threads) -- none of this depends on the solve,
//   2. streams the off-diagonal tiles of its block row (or block column when op(A)'s rows are
//      strided in memory) in solve order, two tiles per step, with the matrix data of the next
//      step already in flight BEFORE it waits for the x values the current step multiplies,
//   3. takes those x values from a side buffer in the workspace in which every value is
//      published as 64-bit words {32 payload bits, 32-bit call tag}: data and "ready" flag
//      travel in one store, so a consumer polls the data itself (bounded; one warp polls for
//      the block) and neither side needs a fence or a second round trip through L2,
//   4. forms r = b - sum, multiplies by the inverted diagonal block (all threads), publishes
//      its 64 values and writes them to the caller's x.
// The chain of n/64 dependent steps makes the routine latency-bound; each step costs one
// L2 store->load hand-over plus a 64x64 matvec.  Tickets are drawn in launch order, so a block
// only ever waits for blocks that are already running: no co-residency assumption, no
// deadlock.  If the polls of a thread exceed the iteration limit the block records
// B2_STATUS_TIMEOUT in *device_status and leaves without publishing.
//
// Accuracy note: the diagonal blocks are applied through their explicit inverses (computed in
// the working precision).  For diagonal blocks of moderate condition number this is as
// accurate as substitution; it is the usual trade for removing 64 dependent steps per block.
#include <atomic>

#include "common.cuh"

namespace b2 {

constexpr int kNB = 64;
constexpr int kTT = 512;          // threads per trsv block
constexpr int kTW = kTT / 32;     // warps per trsv block
constexpr int kGRP = 2;           // source tiles handled per loop iteration

__device__ __forceinline__ unsigned long long ld_word(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_word(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

template <typename T>
struct TrsvArgs {
  const T* a;
  int64_t lda, n;
  T* x;  // base per vec_base()
  int64_t incx;
  unsigned long long* xbuf;  // published solution: 1 (float) or 2 (double) tagged words per unknown
  unsigned* ticket;
  int nb;
  unsigned tag;
  unsigned long long wait_limit;
  int* device_status;
  int debug_skip;
  int pf_dist;  // L2 prefetch distance in tiles
};

// Per-thread polling state: a total budget of polls for the whole kernel.
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
constexpr int kES = kNB + 1;  // row stride of E   (conflict-free column walks)
constexpr int kIS = kNB + 8;  // row stride of Einv (conflict-free for the 8-threads-per-row matvec)

template <typename T, int V, bool COLTYPE, bool BACKWARD, bool UNIT>
__global__ void __launch_bounds__(kTT) trsv_kernel(const TrsvArgs<T> p) {
  constexpr int LPR = (kNB / V) >= 32 ? 32 : kNB / V;
  constexpr int CU = kNB / (LPR * V);
  constexpr int G = 32 / LPR;
  constexpr int RU = kNB / (kTW * G);
  constexpr bool CANON_LOWER = (COLTYPE == BACKWARD);  // stored triangle in the row-major view
  using P = Pack<T, V>;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* E = reinterpret_cast<T*>(smem_raw);  // diagonal block in solve order, E[s*kES + t], t <= s
  T* Einv = E + kNB * kES;                // its inverse, Einv[s*kIS + t]
  T* racc = Einv + kNB * kIS;             // sum over solved blocks, per unknown (solve order)
  T* bvec = racc + kNB;                   // right-hand side b (solve order)
  T* xsm = bvec + kNB;                    // x values of the current tile group, double-buffered
  T* colsm = xsm + 2 * kGRP * kNB;        // [kTW][kNB], COLTYPE only
  __shared__ unsigned s_ticket;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
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
  const int64_t r0 = (int64_t)I * kNB;
  const int nbI = (int)min((int64_t)kNB, p.n - r0);
  auto solve_idx = [&](int i) { return BACKWARD ? nbI - 1 - i : i; };

  int lr[RU];
#pragma unroll
  for (int ru = 0; ru < RU; ++ru) lr[ru] = (ru * kTW + warp) * G + g;

  auto load_tile = [&](P (&av)[RU][CU], int s) {
    if (s >= k) {  // padding tile of the last group
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u)
#pragma unroll
          for (int e = 0; e < V; ++e) av[ru][u].v[e] = T(0);
      return;
    }
    const int J = BACKWARD ? p.nb - 1 - s : s;
    const int64_t c0 = (int64_t)J * kNB;
    const int nbJ = (int)min((int64_t)kNB, p.n - c0);
    const int64_t rbase = COLTYPE ? c0 : r0, cbase = COLTYPE ? r0 : c0;
    const int nr = COLTYPE ? nbJ : nbI, nc = COLTYPE ? nbI : nbJ;
    if (nr == kNB && nc == kNB) {
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
    if (s >= k) return;
    const int J = BACKWARD ? p.nb - 1 - s : s;
    const int64_t c0 = (int64_t)J * kNB;
    if (p.n - c0 < kNB || nbI < kNB) return;  // ragged tiles are not worth it
    const int64_t rbase = COLTYPE ? c0 : r0, cbase = COLTYPE ? r0 : c0;
    constexpr int LINES = kNB * (int)sizeof(T) / 128;
    if (tid < kNB * LINES) {
      const T* ptr = p.a + (rbase + tid / LINES) * p.lda + cbase + (tid % LINES) * (128 / (int)sizeof(T));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
    }
  };

  // The first tiles' matrix data go in flight before anything else.
  P cur[kGRP][RU][CU], nxt[kGRP][RU][CU];
#pragma unroll
  for (int t = 0; t < kGRP; ++t) load_tile(nxt[t], t);
  for (int s = kGRP; s < kGRP + p.pf_dist; ++s) prefetch_tile(s);

  // 1a. diagonal block -> E (zero elsewhere, identity on unused / unit diagonal); b -> bvec
  for (int idx = tid; idx < kNB * kES; idx += kTT) E[idx] = T(0);
  for (int idx = tid; idx < kNB * kIS; idx += kTT) Einv[idx] = T(0);
  if (tid < kNB) {
    bvec[tid] = tid < nbI ? p.x[(r0 + solve_idx(tid)) * p.incx] : T(0);
    racc[tid] = T(0);  // entries past a ragged block stay zero
  }
  __syncthreads();
  for (int idx = tid; idx < kNB * kNB; idx += kTT) {
    const int pr = idx / kNB, pc = idx % kNB;  // position inside the stored block
    if (pr < nbI && pc < nbI) {
      const bool in_tri = CANON_LOWER ? (pc <= pr) : (pc >= pr);
      if (in_tri && !(UNIT && pr == pc)) {
        const T v = __ldg(p.a + (r0 + pr) * p.lda + r0 + pc);
        const int sr = solve_idx(pr), sc = solve_idx(pc);
        if (COLTYPE) E[sc * kES + sr] = v;
        else E[sr * kES + sc] = v;
      }
    }
  }
  for (int s = tid; s < kNB; s += kTT)
    if (UNIT || s >= nbI) E[s * kES + s] = T(1);
  __syncthreads();

  // 1b. inverse of E by recursive doubling.  8x8 diagonal blocks are inverted by substitution
  // (one column per thread); then, for h = 8, 16, 32, every pair [A 0; C B] of h x h blocks gets
  // its lower-left block  -B^-1 (C A^-1).  The intermediate C A^-1 is parked in the unused
  // upper triangle of E (transposed position).
  if (tid < kNB) {
    const int c = tid, d0 = (c / 8) * 8;
    for (int s = c; s < d0 + 8; ++s) {
      T acc = (s == c) ? T(1) : T(0);
      for (int t = c; t < s; ++t) acc -= E[s * kES + t] * Einv[t * kIS + c];
      Einv[s * kIS + c] = acc / E[s * kES + s];
    }
  }
  __syncthreads();
#pragma unroll 1
  for (int h = 8; h < kNB; h *= 2) {
    const int per_pair = h * h, total = (kNB / (2 * h)) * per_pair;
    for (int e = tid; e < total; e += kTT) {  // Tm = C * A^-1
      const int pr = e / per_pair, i = (e % per_pair) / h, j = e % h;
      const int top = pr * 2 * h, bot = top + h;
      T acc = T(0);
      for (int l = j; l < h; ++l) acc = E[(bot + i) * kES + top + l] * Einv[(top + l) * kIS + top + j] + acc;
      E[(top + j) * kES + bot + i] = acc;
    }
    __syncthreads();
    for (int e = tid; e < total; e += kTT) {  // X = -B^-1 * Tm
      const int pr = e / per_pair, i = (e % per_pair) / h, j = e % h;
      const int top = pr * 2 * h, bot = top + h;
      T acc = T(0);
      for (int l = 0; l <= i; ++l) acc = Einv[(bot + i) * kIS + bot + l] * E[(top + j) * kES + bot + l] + acc;
      Einv[(bot + i) * kIS + top + j] = -acc;
    }
    __syncthreads();
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

  Poller poll;
  poll.budget = p.wait_limit ? p.wait_limit : (1ull << 20);
  poll.abort_flag = &s_abort;
  poll.device_status = p.device_status;
  poll.tag = p.tag;

  // Tiles are taken kGRP at a time: one poll round trip and one loop iteration then serve
  // kGRP tiles, which keeps a block with a long row ahead of the solve front.  The matrix data
  // of the next group is already in flight while this group's x values are awaited.
  constexpr int WPE = Words<T>::N;
  const int ngroups = (k + kGRP - 1) / kGRP;
#pragma unroll 1
  for (int gi = 0; gi < ngroups; ++gi) {
    const int s0 = gi * kGRP;
#pragma unroll
    for (int t = 0; t < kGRP; ++t)
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u) cur[t][ru][u] = nxt[t][ru][u];
    if (gi + 1 < ngroups) {
#pragma unroll
      for (int t = 0; t < kGRP; ++t) load_tile(nxt[t], s0 + kGRP + t);
#pragma unroll
      for (int t = 0; t < kGRP; ++t) prefetch_tile(s0 + kGRP + p.pf_dist + t);
    }
    // Warp 0 polls the group's tagged words on behalf of the block (one reader per block keeps
    // the L2 slice that holds the front's words from being swamped) and hands the decoded
    // values over through shared memory.  Blocks further from the front sleep between polls.
    T* xg = xsm + (gi & 1) * (kGRP * kNB);
    if (warp == 0) {
      const int dist = k - min(k - 1, s0 + kGRP - 1);
      poll.backoff_ns = dist > 1 ? (unsigned)min(dist - 1, 64) * 500u : 0u;
      constexpr int EPL = kGRP * kNB / 32;  // unknowns per lane
      unsigned long long w[EPL * WPE];
      const unsigned long long* wp[EPL * WPE];
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int el = lane * EPL + j, t = el / kNB, lc = el % kNB;
        const int s = s0 + t;
        const int J = BACKWARD ? p.nb - 1 - s : s;
        const int64_t c0 = (int64_t)J * kNB;
        const bool valid = s < k && c0 + lc < p.n;
#pragma unroll
        for (int h = 0; h < WPE; ++h) wp[j * WPE + h] = valid ? p.xbuf + (c0 + lc) * WPE + h : nullptr;
      }
      poll.wait_words(w, wp);
#pragma unroll
      for (int j = 0; j < EPL; ++j) xg[lane * EPL + j] = wp[j * WPE] ? decode(&w[j * WPE], T(0)) : T(0);
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < kGRP; ++t) {
      if (COLTYPE) {
        T xr[RU];
#pragma unroll
        for (int ru = 0; ru < RU; ++ru) xr[ru] = xg[t * kNB + lr[ru]];
#pragma unroll
        for (int ru = 0; ru < RU; ++ru)
#pragma unroll
          for (int u = 0; u < CU; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) colacc[u][e] = cur[t][ru][u].v[e] * xr[ru] + colacc[u][e];
      } else {
        T xs[CU][V];
#pragma unroll
        for (int u = 0; u < CU; ++u)
#pragma unroll
          for (int e = 0; e < V; ++e) xs[u][e] = xg[t * kNB + (u * LPR + q) * V + e];
#pragma unroll
        for (int ru = 0; ru < RU; ++ru)
#pragma unroll
          for (int u = 0; u < CU; ++u)
#pragma unroll
            for (int e = 0; e < V; ++e) rowacc[ru] = cur[t][ru][u].v[e] * xs[u][e] + rowacc[ru];
      }
    }
  }

  // per-unknown sums -> racc (solve order)
  if (COLTYPE) {
#pragma unroll
    for (int u = 0; u < CU; ++u)
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const T s = cross_group_sum<LPR>(colacc[u][e]);
        if (g == 0) colsm[warp * kNB + (u * LPR + q) * V + e] = s;
      }
    __syncthreads();
    if (tid < kNB) {
      T s = colsm[tid];
#pragma unroll
      for (int w = 1; w < kTW; ++w) s += colsm[w * kNB + tid];
      if (tid < nbI) racc[solve_idx(tid)] = s;
    }
  } else {
#pragma unroll
    for (int ru = 0; ru < RU; ++ru) {
      const T s = group_sum<LPR>(rowacc[ru]);
      if (q == 0 && lr[ru] < nbI) racc[solve_idx(lr[ru])] = s;
    }
  }
  __syncthreads();
  if (s_abort) return;  // a wait ran out: publish nothing, dependants will time out too

  // 4. x = Einv * (b - racc): kTT/64 threads per unknown, then publish and write back
  {
    constexpr int TPU = kTT / kNB;  // threads per unknown (8)
    const int s = tid / TPU, part = tid % TPU;
    T acc = T(0);
#pragma unroll
    for (int j = 0; j < kNB / TPU; ++j) {
      const int t = part + TPU * j;
      acc = Einv[s * kIS + t] * (bvec[t] - racc[t]) + acc;  // Einv is zero above the diagonal
    }
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

template <typename T, bool COLTYPE>
constexpr size_t trsv_smem_bytes() {
  return sizeof(T) * (kNB * kES + kNB * kIS + 2 * kNB + 2 * kGRP * kNB + (COLTYPE ? kTW : 1) * kNB);
}

template <typename T, int V, bool COLTYPE, bool BACKWARD, bool UNIT>
static int trsv_launch_one(const Launch& l, const TrsvArgs<T>& args) {
  constexpr size_t smem = trsv_smem_bytes<T, COLTYPE>();
  auto kern = trsv_kernel<T, V, COLTYPE, BACKWARD, UNIT>;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    (void)cudaGetLastError();
    return B2_STATUS_LAUNCH_FAILED;
  }
  kern<<<args.nb, kTT, smem, l.stream>>>(args);
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
  if ((n + kNB - 1) / kNB > 0x3fffffff) return B2_STATUS_NOT_IMPLEMENTED;
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
  args.nb = (int)((n + kNB - 1) / kNB);
  args.tag = next_tag();
  args.wait_limit = l.wait_limit;
  args.device_status = l.device_status;
  args.debug_skip = (int)knob(kKnobTrsvDebugSkip);
  {  // keep the prefetched-but-unused tiles of all blocks within a fraction of L2
    const int64_t tile_bytes = (int64_t)kNB * kNB * sizeof(T);
    int64_t d = knob(kKnobTrsvPrefetchBytes) / (tile_bytes * args.nb);
    args.pf_dist = (int)(d < 0 ? 0 : d > 64 ? 64 : d);
  }
  // op(A) lower triangular <=> forward substitution
  const bool eff_lower = (uplo == B2_LOWER) != (trans == B2_TRANS);
  // rows of op(A) contiguous in memory <=> row-major N or column-major T
  const bool coltype = (order == B2_ROW_MAJOR) != (trans == B2_NO_TRANS);
  const bool unit = diag == B2_UNIT;
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
