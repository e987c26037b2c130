// Shared device / host building blocks of the b2blas kernels (sm_100a).
//
// Everything in the library is generated from a few kernel templates; this header holds the
// pieces they share: 128-bit packs with streaming load / store flavours, warp and block
// reductions, the "last block finishes" ticket, launch helpers and the control-block layout.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "b2blas.h"

namespace b2 {

// ---------------------------------------------------------------------------------------
// Bounds-checking build (-DB2_DEBUG_BOUNDS; a separate library file, never the default).  Every
// entry point lists the byte ranges its kernels may touch (vector spans, matrix extents, result
// words, the workspace); the load / store helpers and intrinsics below then test each address
// against the list.  An access outside every range is NOT performed (a load gives zero): the
// kernel records a count, the first offending address and its size in a report the host can
// read, and carries on -- nothing traps, the context stays usable.
#ifdef B2_DEBUG_BOUNDS
struct DbgTable {
  unsigned long long lo[8], hi[8];
  int n;
  int shrink;  // test hook: bytes cut off the end of every range (makes in-bounds accesses look bad)
};
struct DbgReport {
  unsigned long long count, first_addr, first_bytes, pad;
};
static __device__ DbgTable g_dbg_table;    // one copy per translation unit, written before its kernels run
static __device__ DbgReport g_dbg_report;  // accumulated until the host collects it
__device__ __forceinline__ bool dbg_ok(const void* p, size_t bytes) {
  const unsigned long long a = (unsigned long long)p;
  for (int i = 0; i < g_dbg_table.n; ++i)
    if (a >= g_dbg_table.lo[i] && a + bytes <= g_dbg_table.hi[i] - (unsigned long long)g_dbg_table.shrink) return true;
  if (atomicAdd(&g_dbg_report.count, 1ull) == 0ull) {
    g_dbg_report.first_addr = a;
    g_dbg_report.first_bytes = bytes;
  }
  return false;
}
template <typename T>
__device__ __forceinline__ T dbg_ldg(const T* p) { return dbg_ok(p, sizeof(T)) ? __ldg(p) : T(); }
template <typename T>
__device__ __forceinline__ T dbg_ldcg(const T* p) { return dbg_ok(p, sizeof(T)) ? __ldcg(p) : T(); }
template <typename T>
__device__ __forceinline__ T dbg_ldcs(const T* p) { return dbg_ok(p, sizeof(T)) ? __ldcs(p) : T(); }
template <typename T>
__device__ __forceinline__ void dbg_stcs(T* p, T v) { if (dbg_ok(p, sizeof(T))) __stcs(p, v); }
#define __ldg(p) ::b2::dbg_ldg(p)
#define __ldcg(p) ::b2::dbg_ldcg(p)
#define __ldcs(p) ::b2::dbg_ldcs(p)
#define __stcs(p, v) ::b2::dbg_stcs(p, v)
#define B2_GUARD(p, bytes) ::b2::dbg_ok(p, bytes)
#else
#define B2_GUARD(p, bytes) true
#endif
// A plain store of a result element (checked in the bounds-checking build).
#define B2_STORE(ptr, value) do { if (B2_GUARD(ptr, sizeof(*(ptr)))) *(ptr) = (value); } while (0)

constexpr int kThreads = 256;  // every kernel uses 256-thread blocks (8 warps)
constexpr int kWarps = kThreads / 32;

// ---------------------------------------------------------------------------------------
// Control block at the start of ctx->workspace.  Zero between calls.
//   word 0      : ticket counter of the level-1 reductions
//   word 16     : ticket counter of trsv (next block-row to hand out)
//   word 17     : trsv "blocks finished" counter
//   word 19     : sub-block trsv: abort flag (stays up after a timeout until the workspace is reset)
// Scratch (partials, trsv flags) starts at kCtlBytes.
constexpr size_t kCtlBytes = 4096;
constexpr int kCtlReduceTicket = 0;
constexpr int kCtlTrsvTicket = 16;
constexpr int kCtlTrsvDone = 17;
constexpr int kCtlTrsvAbort = 19;  // sub-block trsv: raised when a bounded wait ran out

// ---------------------------------------------------------------------------------------
// 16-byte packs: 4 floats or 2 doubles.
template <typename T>
struct VecLen {
  static constexpr int value = 16 / sizeof(T);
};

template <typename T, int N>
struct alignas(sizeof(T) * N) Pack {
  T v[N];
};

// Streaming (evict-first) load of data that may be written later by this kernel.
template <typename T, int N>
__device__ __forceinline__ Pack<T, N> ld_cs(const T* p) {
  Pack<T, N> r = {};
  if (!B2_GUARD(p, sizeof(T) * N)) return r;
  if constexpr (sizeof(T) * N == 16) {
    uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
    r = *reinterpret_cast<Pack<T, N>*>(&t);
  } else {
    static_assert(N == 1, "packs are 16 bytes or one element");
    r.v[0] = __ldcs(p);
  }
  return r;
}

// Streaming load of data that this kernel writes back: L2 only, normal eviction priority, so
// that the line is still there when the store arrives (see ld_cs for the evict-first form).
template <typename T, int N>
__device__ __forceinline__ Pack<T, N> ld_cg(const T* p) {
  Pack<T, N> r = {};
  if (!B2_GUARD(p, sizeof(T) * N)) return r;
  if constexpr (sizeof(T) * N == 16) {
    uint4 t = __ldcg(reinterpret_cast<const uint4*>(p));
    r = *reinterpret_cast<Pack<T, N>*>(&t);
  } else {
    static_assert(N == 1, "packs are 16 bytes or one element");
    r.v[0] = __ldcg(p);
  }
  return r;
}

// Read-only streaming load (data not written by this kernel): non-coherent path, no L1
// allocation so the matrix stream does not evict the reused vectors.
template <typename T, int N>
__device__ __forceinline__ Pack<T, N> ld_nc(const T* p) {
  Pack<T, N> r = {};
  if (!B2_GUARD(p, sizeof(T) * N)) return r;
  if constexpr (sizeof(T) * N == 16) {
    uint4 t;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(t.x), "=r"(t.y), "=r"(t.z), "=r"(t.w)
                 : "l"(p));
    r = *reinterpret_cast<Pack<T, N>*>(&t);
  } else {
    static_assert(N == 1, "packs are 16 bytes or one element");
    r.v[0] = __ldg(p);
  }
  return r;
}

// The same load under a predicate, zeros otherwise, as ONE instruction sequence without a branch.
// (`if (c) v = ld_nc(p)` compiles to a branch around the load and a copy of the loaded registers
// where the paths meet; the copy waits for the load, so several such loads in a row go out one
// memory latency after the other.)
template <typename T, int N>
__device__ __forceinline__ Pack<T, N> ld_nc_if(const T* p, bool pred) {
  Pack<T, N> r = {};
  if (pred && !B2_GUARD(p, sizeof(T) * N)) pred = false;
  if constexpr (sizeof(T) * N == 16) {
    uint4 t;
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %5, 0;\n\tmov.u32 %0, 0;\n\tmov.u32 %1, 0;\n\tmov.u32 %2, 0;\n\tmov.u32 %3, 0;\n\t"
        "@q ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n\t}"
        : "=&r"(t.x), "=&r"(t.y), "=&r"(t.z), "=&r"(t.w)
        : "l"(p), "r"((unsigned)pred));
    r = *reinterpret_cast<Pack<T, N>*>(&t);
  } else {
    static_assert(N == 1, "packs are 16 bytes or one element");
    r.v[0] = pred ? __ldg(p) : T(0);
  }
  return r;
}

// Read-only load of reused data (the x vectors): cached in L1.
template <typename T, int N>
__device__ __forceinline__ Pack<T, N> ld_ro(const T* p) {
  Pack<T, N> r = {};
  if (!B2_GUARD(p, sizeof(T) * N)) return r;
  if constexpr (sizeof(T) * N == 16) {
    uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    r = *reinterpret_cast<Pack<T, N>*>(&t);
  } else {
    static_assert(N == 1, "packs are 16 bytes or one element");
    r.v[0] = __ldg(p);
  }
  return r;
}

template <typename T, int N>
__device__ __forceinline__ void st_cs(T* p, const Pack<T, N>& r) {
  if (!B2_GUARD(p, sizeof(T) * N)) return;
  if constexpr (sizeof(T) * N == 16) {
    __stcs(reinterpret_cast<uint4*>(p), *reinterpret_cast<const uint4*>(&r));
  } else {
    static_assert(N == 1, "packs are 16 bytes or one element");
    __stcs(p, r.v[0]);
  }
}

// ---------------------------------------------------------------------------------------
// Reductions.
template <typename T>
__device__ __forceinline__ T shfl_xor(T v, int mask) {
  return __shfl_xor_sync(0xffffffffu, v, mask);
}

// Sum over aligned groups of LANES lanes (LANES a power of two <= 32); every lane of the
// group receives the total.  Fixed butterfly order => deterministic.
template <int LANES, typename T>
__device__ __forceinline__ T group_sum(T v) {
#pragma unroll
  for (int m = LANES / 2; m >= 1; m >>= 1) v += shfl_xor(v, m);
  return v;
}

// Sums R values at once over each aligned group of LANES lanes (R a power of two <= LANES).
// The first log2(R) butterfly steps trade half of the values for the partner's other half, so
// the work shrinks with the lane span; plain butterflies finish the job.  Afterwards every
// lane holds the total of value index (lane % LANES) / (LANES / R).  Fixed order.
template <int LANES, int R, typename T>
__device__ __forceinline__ T multi_group_sum(T (&v)[R], int lane) {
  static_assert(R >= 1 && LANES >= R, "need at least one lane per value");
  int span = LANES;
#pragma unroll
  for (int n = R; n > 1; n >>= 1) {
    const int m = span >> 1, h = n >> 1;
    const bool up = (lane & m) != 0;
#pragma unroll
    for (int i = 0; i < h; ++i) {
      const T send = up ? v[i] : v[i + h];
      const T keep = up ? v[i + h] : v[i];
      v[i] = keep + shfl_xor(send, m);
    }
    span = m;
  }
#pragma unroll
  for (int m = (LANES / R) >> 1; m >= 1; m >>= 1) v[0] += shfl_xor(v[0], m);
  return v[0];
}

// Sum over the lanes that share (lane % LANES): the complementary butterfly.
template <int LANES, typename T>
__device__ __forceinline__ T cross_group_sum(T v) {
#pragma unroll
  for (int m = 16; m >= LANES; m >>= 1) v += shfl_xor(v, m);
  return v;
}

// Programmatic dependent launch (PDL): a dependent kernel may start while its predecessor
// drains; it must call grid_dep_wait() before touching the predecessor's outputs.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------------------------------
// Host helpers.
struct Launch {
  cudaStream_t stream;
  char* scratch;         // workspace past the control block
  size_t scratch_bytes;
  unsigned* ctl;         // control block as 32-bit words
  int* device_status;
  unsigned long long wait_limit;
#ifdef B2_DEBUG_BOUNDS
  unsigned long long dbg_lo[8], dbg_hi[8];  // byte ranges the kernels of this call may touch
  int dbg_n;
#endif
};

inline int make_launch(const b2_ctx* ctx, Launch* l) {
  if (ctx == nullptr || ctx->workspace == nullptr) return B2_STATUS_BAD_CONTEXT;
  if ((reinterpret_cast<uintptr_t>(ctx->workspace) & 255) != 0) return B2_STATUS_BAD_CONTEXT;
  if (ctx->workspace_bytes < kCtlBytes) return B2_STATUS_WORKSPACE_TOO_SMALL;
  l->stream = static_cast<cudaStream_t>(ctx->stream);
  l->ctl = static_cast<unsigned*>(ctx->workspace);
  l->scratch = static_cast<char*>(ctx->workspace) + kCtlBytes;
  l->scratch_bytes = ctx->workspace_bytes - kCtlBytes;
  l->device_status = ctx->device_status;
  l->wait_limit = ctx->wait_limit;
#ifdef B2_DEBUG_BOUNDS
  l->dbg_n = 0;
#endif
  return B2_STATUS_OK;
}

// Every kernel launch site calls this right after the launch; it also feeds the launch counter.
extern unsigned long long g_launch_count;
inline int check_launch() {
  ++g_launch_count;
  return cudaGetLastError() == cudaSuccess ? B2_STATUS_OK : B2_STATUS_LAUNCH_FAILED;
}

// Bounds-checking build: the ranges a call may touch, and their hand-over to this translation
// unit's device table (stream-ordered, before the kernels of the call).  No-ops otherwise.
#ifdef B2_DEBUG_BOUNDS
int dbg_shrink();  // test hook value (bytes)
void dbg_register_collector(void (*fn)(unsigned long long*));
inline void dbg_range(Launch& l, const void* p, size_t bytes) {
  if (p == nullptr || bytes == 0 || l.dbg_n >= 8) return;
  l.dbg_lo[l.dbg_n] = (unsigned long long)p;
  l.dbg_hi[l.dbg_n] = (unsigned long long)p + bytes;
  ++l.dbg_n;
}
template <typename T>
inline void dbg_vec(Launch& l, const T* p, int64_t n, int64_t inc) {  // p as the caller passes it
  if (n <= 0) return;
  const int64_t span = 1 + (n - 1) * (inc < 0 ? -inc : inc);
  dbg_range(l, p, (size_t)span * sizeof(T));
}
static void dbg_collect_this_unit(unsigned long long* out) {
  DbgReport r = {};
  if (cudaMemcpyFromSymbol(&r, g_dbg_report, sizeof(r)) != cudaSuccess) return;
  if (r.count && out[0] == 0) out[1] = r.first_addr, out[2] = r.first_bytes;
  out[0] += r.count;
  const DbgReport zero = {};
  cudaMemcpyToSymbol(g_dbg_report, &zero, sizeof(zero));
}
static void dbg_commit(Launch& l) {
  static bool registered = false;  // (one flag per translation unit, like the device symbols)
  if (!registered) {
    registered = true;
    dbg_register_collector(&dbg_collect_this_unit);
  }
  dbg_range(l, l.ctl, kCtlBytes + l.scratch_bytes);  // the workspace, whole
  DbgTable t = {};
  for (int i = 0; i < l.dbg_n && i < 8; ++i) t.lo[i] = l.dbg_lo[i], t.hi[i] = l.dbg_hi[i];
  t.n = l.dbg_n < 8 ? l.dbg_n : 8;
  t.shrink = dbg_shrink();
  cudaMemcpyToSymbolAsync(g_dbg_table, &t, sizeof(t), 0, cudaMemcpyHostToDevice, l.stream);
  --l.dbg_n;  // (a second commit of the same call adds the workspace again)
}
#define B2_DBG_VEC(l, p, n, inc) ::b2::dbg_vec(l, p, n, inc)
#define B2_DBG_RANGE(l, p, bytes) ::b2::dbg_range(l, p, bytes)
#define B2_DBG_COMMIT(l) ::b2::dbg_commit(l)
#else
#define B2_DBG_VEC(l, p, n, inc) ((void)0)
#define B2_DBG_RANGE(l, p, bytes) ((void)0)
#define B2_DBG_COMMIT(l) ((void)0)
#endif

// Number of SMs of the current device (cached per device id).
int sm_count();

// Tuning knobs (see b2_set_tuning).
enum Knob {
  kKnobL1BlocksPerSm = 0,
  kKnobGemvNTileBytes = 1,
  kKnobGemvTRows = 2,
  kKnobTriRows = 3,
  kKnobGerRows = 4,
  kKnobUsePdl = 5,
  kKnobTrsvDebugSkip = 6,  // test hook: solve-order block that never publishes (-1 = none)
  kKnobTriWide = 7,
  kKnobTrsvPrefetchBytes = 8,  // total L2 bytes trsv blocks may prefetch ahead of the front
  kKnobTrsvFront = 9,          // 0: block-row trsv kernel only; 1: sub-block kernel for row-type views; 2: for all views
  kKnobTrsvCluster = 10,       // sub-block trsv in clusters of 8 block rows: 0 never, 1 float only, 2 always
  kKnobTrsvPmFrom = 11,        // first block row whose last tile is premultiplied by the inverse diagonal block (-1: by precision)
  kKnobTriTile = 12,           // tile kernel with the shared-memory ring: 0 never, 1 symv and the trmv cases it wins, 2 symv and every trmv
  kKnobTriTileUnit = 13,       // tiles per unit of that kernel: 0 = by size, else 1, 2 or 4
  kKnobNarrowBlock = 14,       // gemv on unpadded narrow matrices: 1 = block-wide kernels, 0 = warp-wide / general ones
  kKnobTriBulk = 15,           // tile kernel with the shared-memory ring: 1 = a tile arrives as one tiled TMA copy (measured equal to the 16-byte copies; off by default)
  kKnobCount = 16
};
int64_t knob(int id);

// Launch with programmatic stream serialization: the grid may be scheduled while its predecessor
// in the stream drains.  Every kernel launched this way starts with grid_dep_wait() (nothing
// of the predecessor's memory is read or written before the predecessor has completed and
// flushed) followed by grid_dep_launch() (its own successor may be scheduled as soon as all
// of its blocks are resident), so the chain of completions stays transitive.
template <typename... KArgs, typename... Args>
inline void launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = knob(kKnobUsePdl) ? 1 : 0;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);  // (a failure is picked up by check_launch())
}


// Base pointer such that logical element i lives at base[i*inc] for either sign of inc.
template <typename T>
inline T* vec_base(T* p, int64_t n, int64_t inc) {
  return inc >= 0 ? p : p + (1 - n) * inc;
}

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace b2
