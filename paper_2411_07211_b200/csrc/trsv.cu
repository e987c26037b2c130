// trsv: solve op(A) x = b in place (Section 6.2.2; same option space as trmv).
//
// Blocked substitution with a dependency-ordered diagonal-block solve.  The unknowns are cut
// into blocks of 64.  Thread blocks draw a ticket k = 0, 1, ... (the solve order: top-down for
// an effectively lower-triangular op(A), bottom-up for an upper one); block k
//   1. stages its 64x64 diagonal block in shared memory,
//   2. streams the off-diagonal tiles of its block row (or block column when op(A)'s rows are
//      strided in memory) in solve order, prefetching each tile's matrix data BEFORE waiting
//      for the x values it multiplies (the matrix does not depend on the solve),
//   3. waits -- bounded -- until the `done` counter shows that the source block is solved,
//      reads its x values through L2 and accumulates,
//   4. solves its diagonal block in one warp and publishes: x written, fence, done = k + 1.
// Tickets are drawn in launch order, so a block only ever waits for blocks that are already
// running: no co-residency assumption, no deadlock.  If a wait still exceeds its iteration
// limit the block records B2_STATUS_TIMEOUT in *device_status and leaves without publishing.
#include "common.cuh"

namespace b2 {

constexpr int kNB = 64;

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

template <typename T>
struct TrsvArgs {
  const T* a;
  int64_t lda, n;
  T* x;  // base per vec_base()
  int64_t incx;
  unsigned* ticket;
  unsigned* done;
  int nb;
  unsigned long long wait_limit;
  int* device_status;
  int debug_skip;
};

// COLTYPE: op(A)'s rows are columns of the stored row-major view.  BACKWARD: solve bottom-up.
template <typename T, int V, bool COLTYPE, bool BACKWARD, bool UNIT>
__global__ void __launch_bounds__(kThreads) trsv_kernel(const TrsvArgs<T> p) {
  constexpr int LPR = (kNB / V) >= 32 ? 32 : kNB / V;
  constexpr int CU = kNB / (LPR * V);
  constexpr int G = 32 / LPR;
  constexpr int RU = kNB / (kWarps * G);
  constexpr bool CANON_LOWER = (COLTYPE == BACKWARD);  // stored triangle in the row-major view
  using P = Pack<T, V>;

  __shared__ T E[kNB][kNB + 1];   // diagonal block in solve order: E[s][t], t <= s
  __shared__ T racc[kNB];         // sum over solved blocks, per local unknown
  __shared__ T colsm[COLTYPE ? kWarps : 1][kNB];
  __shared__ unsigned s_ticket, s_done;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane / LPR, q = lane % LPR;
  if (tid == 0) {
    s_ticket = atomicAdd(p.ticket, 1u);
    s_abort = 0;
  }
  __syncthreads();
  const int k = (int)s_ticket;                      // position in the solve order
  const int I = BACKWARD ? p.nb - 1 - k : k;        // block index in memory
  const int64_t r0 = (int64_t)I * kNB;
  const int nbI = (int)min((int64_t)kNB, p.n - r0);
  auto solve_idx = [&](int i) { return BACKWARD ? nbI - 1 - i : i; };

  // 1. diagonal block -> E (zero elsewhere, identity on unused / unit diagonal)
  for (int idx = tid; idx < kNB * (kNB + 1); idx += kThreads) (&E[0][0])[idx] = T(0);
  __syncthreads();
  for (int idx = tid; idx < kNB * kNB; idx += kThreads) {
    const int pr = idx / kNB, pc = idx % kNB;  // position inside the stored block
    if (pr < nbI && pc < nbI) {
      const bool in_tri = CANON_LOWER ? (pc <= pr) : (pc >= pr);
      if (in_tri && !(UNIT && pr == pc)) {
        const T v = __ldg(p.a + (r0 + pr) * p.lda + r0 + pc);
        const int sr = solve_idx(pr), sc = solve_idx(pc);
        if (COLTYPE) E[sc][sr] = v;
        else E[sr][sc] = v;
      }
    }
  }
  for (int s = tid; s < kNB; s += kThreads)
    if (UNIT || s >= nbI) E[s][s] = T(1);

  // 2./3. off-diagonal tiles in solve order
  int lr[RU];
#pragma unroll
  for (int ru = 0; ru < RU; ++ru) lr[ru] = (ru * kWarps + warp) * G + g;
  T rowacc[RU];
  T colacc[CU][V];
#pragma unroll
  for (int ru = 0; ru < RU; ++ru) rowacc[ru] = T(0);
#pragma unroll
  for (int u = 0; u < CU; ++u)
#pragma unroll
    for (int e = 0; e < V; ++e) colacc[u][e] = T(0);

  auto load_tile = [&](P (&av)[RU][CU], int s) {
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

  unsigned known = 0;  // blocks known to be solved (uniform across the block)
  P nxt[RU][CU];
  if (k > 0) load_tile(nxt, 0);
  for (int s = 0; s < k; ++s) {
    P cur[RU][CU];
#pragma unroll
    for (int ru = 0; ru < RU; ++ru)
#pragma unroll
      for (int u = 0; u < CU; ++u) cur[ru][u] = nxt[ru][u];
    if (s + 1 < k) load_tile(nxt, s + 1);
    if (known <= (unsigned)s) {
      if (tid == 0) {
        const unsigned long long limit = p.wait_limit ? p.wait_limit : (1ull << 22);
        unsigned v = 0;
        unsigned long long it = 0;
        for (; it < limit; ++it) {
          v = ld_acquire(p.done);
          if (v > (unsigned)s) break;
        }
        if (it >= limit) {
          s_abort = 1;
          if (p.device_status) atomicExch(p.device_status, (int)B2_STATUS_TIMEOUT);
        }
        s_done = v;
      }
      __syncthreads();
      if (s_abort) return;
      known = s_done;
      __syncthreads();
    }
    const int J = BACKWARD ? p.nb - 1 - s : s;
    const int64_t c0 = (int64_t)J * kNB;
    const int nbJ = (int)min((int64_t)kNB, p.n - c0);
    if (COLTYPE) {
      T xr[RU];
#pragma unroll
      for (int ru = 0; ru < RU; ++ru) xr[ru] = lr[ru] < nbJ ? __ldcg(p.x + (c0 + lr[ru]) * p.incx) : T(0);
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
        for (int e = 0; e < V; ++e) {
          const int lc = (u * LPR + q) * V + e;
          xs[u][e] = lc < nbJ ? __ldcg(p.x + (c0 + lc) * p.incx) : T(0);
        }
#pragma unroll
      for (int ru = 0; ru < RU; ++ru)
#pragma unroll
        for (int u = 0; u < CU; ++u)
#pragma unroll
          for (int e = 0; e < V; ++e) rowacc[ru] = cur[ru][u].v[e] * xs[u][e] + rowacc[ru];
    }
  }

  // per-unknown sums -> racc
  if (COLTYPE) {
#pragma unroll
    for (int u = 0; u < CU; ++u)
#pragma unroll
      for (int e = 0; e < V; ++e) {
        const T s = cross_group_sum<LPR>(colacc[u][e]);
        if (g == 0) colsm[COLTYPE ? warp : 0][(u * LPR + q) * V + e] = s;
      }
    __syncthreads();
    if (tid < kNB) {
      T s = colsm[0][tid];
#pragma unroll
      for (int w = 1; w < (COLTYPE ? kWarps : 1); ++w) s += colsm[w][tid];
      racc[tid] = s;
    }
  } else {
#pragma unroll
    for (int ru = 0; ru < RU; ++ru) {
      const T s = group_sum<LPR>(rowacc[ru]);
      if (q == 0) racc[lr[ru]] = s;
    }
  }
  __syncthreads();

  // 4. diagonal solve in warp 0: lane owns unknowns `lane` and `32 + lane` of the solve order
  if (warp != 0) return;
  const int s0 = lane, s1 = 32 + lane;
  const int i0 = solve_idx(s0), i1 = solve_idx(s1);
  T v0 = s0 < nbI ? p.x[(r0 + i0) * p.incx] - racc[i0] : T(0);
  T v1 = s1 < nbI ? p.x[(r0 + i1) * p.incx] - racc[i1] : T(0);
  const T rd0 = T(1) / E[s0][s0], rd1 = T(1) / E[s1][s1];
  T x0 = T(0), x1 = T(0);
#pragma unroll 8
  for (int t = 0; t < 32; ++t) {
    const T xt = __shfl_sync(0xffffffffu, UNIT ? v0 : v0 * rd0, t);
    if (lane == t) x0 = xt;
    if (lane > t) v0 -= E[s0][t] * xt;
    v1 -= E[s1][t] * xt;
  }
#pragma unroll 8
  for (int t = 0; t < 32; ++t) {
    const T xt = __shfl_sync(0xffffffffu, UNIT ? v1 : v1 * rd1, t);
    if (lane == t) x1 = xt;
    if (lane > t) v1 -= E[s1][32 + t] * xt;
  }
  if (s0 < nbI) p.x[(r0 + i0) * p.incx] = x0;
  if (s1 < nbI) p.x[(r0 + i1) * p.incx] = x1;
  __threadfence();
  __syncwarp();
  if (lane == 0) {
    if (k == p.nb - 1) {  // everything is solved: leave the control block clean
      *p.ticket = 0u;
      st_release(p.done, 0u);
    } else if (k != p.debug_skip) {
      st_release(p.done, (unsigned)(k + 1));
    }
  }
}

template <typename T, int V, bool COLTYPE, bool BACKWARD>
static int trsv_launch(const Launch& l, const TrsvArgs<T>& args, bool unit) {
  if (unit) trsv_kernel<T, V, COLTYPE, BACKWARD, true><<<args.nb, kThreads, 0, l.stream>>>(args);
  else trsv_kernel<T, V, COLTYPE, BACKWARD, false><<<args.nb, kThreads, 0, l.stream>>>(args);
  return check_launch();
}

template <typename T, int V>
static int trsv_variant(const Launch& l, const TrsvArgs<T>& args, bool coltype, bool backward, bool unit) {
  if (coltype) return backward ? trsv_launch<T, V, true, true>(l, args, unit) : trsv_launch<T, V, true, false>(l, args, unit);
  return backward ? trsv_launch<T, V, false, true>(l, args, unit) : trsv_launch<T, V, false, false>(l, args, unit);
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
  TrsvArgs<T> args = {};
  args.a = a;
  args.lda = lda;
  args.n = n;
  args.x = vec_base(x, n, incx);
  args.incx = incx;
  args.ticket = l.ctl + kCtlTrsvTicket;
  args.done = l.ctl + kCtlTrsvDone;
  args.nb = (int)((n + kNB - 1) / kNB);
  args.wait_limit = l.wait_limit;
  args.device_status = l.device_status;
  args.debug_skip = (int)knob(kKnobTrsvDebugSkip);
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
