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
  Pack<T, N> r;
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
  Pack<T, N> r;
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
  Pack<T, N> r;
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

// Read-only load of reused data (the x vectors): cached in L1.
template <typename T, int N>
__device__ __forceinline__ Pack<T, N> ld_ro(const T* p) {
  Pack<T, N> r;
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
  return B2_STATUS_OK;
}

// Every kernel launch site calls this right after the launch; it also feeds the launch counter.
extern unsigned long long g_launch_count;
inline int check_launch() {
  ++g_launch_count;
  return cudaGetLastError() == cudaSuccess ? B2_STATUS_OK : B2_STATUS_LAUNCH_FAILED;
}

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
  kKnobTrsvPmFrom = 11,        // first block row whose last tile is premultiplied by the inverse diagonal block
  kKnobTriTile = 12,           // tile kernel with the shared-memory ring: 0 never, 1 symv and the trmv cases it wins, 2 symv and every trmv
  kKnobTriTileUnit = 13,       // tiles per unit of that kernel: 0 = by size, else 1, 2 or 4
  kKnobCount = 16
};
int64_t knob(int id);

// Base pointer such that logical element i lives at base[i*inc] for either sign of inc.
template <typename T>
inline T* vec_base(T* p, int64_t n, int64_t inc) {
  return inc >= 0 ? p : p + (1 - n) * inc;
}

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace b2
