// Library-wide pieces: workspace helpers, status strings, tuning knobs, device queries.
#include "common.cuh"

namespace b2 {

static int64_t g_knobs[kKnobCount] = {
    /* kKnobL1BlocksPerSm   */ 8,
    /* kKnobGemvNTileBytes  */ 64 * 1024,
    /* kKnobGemvTRows       */ 256,
    /* kKnobTriRows         */ 512,
    /* kKnobGerRows         */ 2,
    /* kKnobUsePdl          */ 1,
    /* kKnobTrsvDebugSkip   */ -1,
    /* kKnobTriWide         */ 0,
    /* kKnobTrsvPrefetchBytes */ 12 << 20,
    /* kKnobTrsvFront       */ 2,
    /* kKnobTrsvCluster     */ 0,
    /* kKnobTrsvPmFrom      */ -1,
    /* kKnobTriTile         */ 1,
    /* kKnobTriTileUnit     */ 0,
    /* kKnobNarrowBlock     */ 1,
    /* kKnobTriBulk         */ 0,
};

unsigned long long g_launch_count = 0;

#ifdef B2_DEBUG_BOUNDS
static int g_dbg_shrink = 0;
static void (*g_dbg_collectors[32])(unsigned long long*);
static int g_dbg_ncollectors = 0;
int dbg_shrink() { return g_dbg_shrink; }
void dbg_register_collector(void (*fn)(unsigned long long*)) {
  if (g_dbg_ncollectors < 32) g_dbg_collectors[g_dbg_ncollectors++] = fn;
}
#endif

int64_t knob(int id) { return (id >= 0 && id < kKnobCount) ? g_knobs[id] : 0; }

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace b2

extern "C" {

size_t b2_workspace_min_bytes(void) { return b2::kCtlBytes + 64 * 1024; }
size_t b2_workspace_bytes(void) { return (size_t)256 << 20; }

size_t b2_workspace_query(int64_t m, int64_t n, size_t elem_bytes) {
  if (m < 0 || n < 0 || (elem_bytes != 4 && elem_bytes != 8)) return 0;
  // level 1: one partial per block of the reduction grid; level 2 with every split merged: one
  // row of partials per output vector; symv, whose blocks produce row sums and column sums at
  // once: one row of partials per column tile of 32 packs; trsv: one or two
  // tagged 64-bit words per unknown
  const size_t vec = (size_t)(m > n ? m : n), sq = (size_t)(m < n ? m : n);
  const size_t tile_cols = 32 * (16 / elem_bytes);
  const size_t level2 = ((size_t)m + (size_t)n) * elem_bytes + 1024;
  const size_t symv = ((sq + tile_cols - 1) / tile_cols + 1) * sq * elem_bytes + 1024;
  const size_t trsv = vec * 8 * (elem_bytes / 4);
  size_t need = level2 > trsv ? level2 : trsv;
  if (symv > need) need = symv;
  return b2_workspace_min_bytes() + need;
}

int b2_workspace_reset(const b2_ctx* ctx) {
  b2::Launch l;
  if (int st = b2::make_launch(ctx, &l)) return st;
  return cudaMemsetAsync(ctx->workspace, 0, b2::kCtlBytes, l.stream) == cudaSuccess ? B2_STATUS_OK
                                                                                    : B2_STATUS_LAUNCH_FAILED;
}

const char* b2_status_string(int status) {
  if (status < 0) return "invalid argument (the negated value is its 1-based position after ctx)";
  switch (status) {
    case B2_STATUS_OK: return "ok";
    case B2_STATUS_LAUNCH_FAILED: return "CUDA launch failed";
    case B2_STATUS_WORKSPACE_TOO_SMALL: return "workspace too small";
    case B2_STATUS_NOT_IMPLEMENTED: return "not implemented";
    case B2_STATUS_TIMEOUT: return "a bounded device-side wait ran out";
    case B2_STATUS_TOO_LARGE: return "problem size above the fixed limit of this entry point";
    case B2_STATUS_BAD_CONTEXT: return "bad context (NULL, or workspace NULL / not 256-byte aligned)";
    default: return "unknown status";
  }
}

int b2_debug_bounds_report(unsigned long long* out3) {
#ifdef B2_DEBUG_BOUNDS
  if (out3 == nullptr) return -1;
  if (cudaDeviceSynchronize() != cudaSuccess) return B2_STATUS_LAUNCH_FAILED;
  out3[0] = out3[1] = out3[2] = 0;
  for (int i = 0; i < b2::g_dbg_ncollectors; ++i) b2::g_dbg_collectors[i](out3);
  return B2_STATUS_OK;
#else
  (void)out3;
  return B2_STATUS_NOT_IMPLEMENTED;
#endif
}

int b2_debug_bounds_shrink(int bytes) {
#ifdef B2_DEBUG_BOUNDS
  b2::g_dbg_shrink = bytes < 0 ? 0 : bytes;
  return B2_STATUS_OK;
#else
  (void)bytes;
  return B2_STATUS_NOT_IMPLEMENTED;
#endif
}

int b2_version(void) { return 100; }

unsigned long long b2_launch_count(void) { return b2::g_launch_count; }

int b2_set_tuning(int knob_id, int64_t value) {
  if (knob_id < 0 || knob_id >= b2::kKnobCount) return -1;
  b2::g_knobs[knob_id] = value;
  return 0;
}
int64_t b2_get_tuning(int knob_id) { return b2::knob(knob_id); }

}  // extern "C"
