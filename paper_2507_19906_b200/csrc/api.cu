// C-ABI layer: argument validation, workspace carving and launch sequencing.
// Everything that computes lives in the kernels; this file only marshals.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "../../include/calidrop.h"
#include "common.cuh"
#include "internal.h"

namespace calidrop {

namespace {

std::atomic<uint64_t> g_launches{0};
thread_local char g_err_text[256] = "";

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(cudaError_t e) {
  snprintf(g_err_text, sizeof g_err_text, "CUDA error: %s", cudaGetErrorString(e));
  return CALIDROP_CUDA_ERROR;
}

// Parameter checks shared by every entry point that reads the full struct.
int check_common(const calidrop_params* p) {
  if (!p) return CALIDROP_INVALID_ARG;
  if (p->B < 1 || p->Hq < 1 || p->Hkv < 1 || p->Hq % p->Hkv != 0) return CALIDROP_INVALID_ARG;
  if (p->D != kD) return CALIDROP_UNSUPPORTED;
  if (p->Hq / p->Hkv > kMaxG) return CALIDROP_UNSUPPORTED;
  if (p->n_cal < 1 || p->cap < 1) return CALIDROP_INVALID_ARG;
  if (!(p->softmax_scale >= 0.f) || !std::isfinite(p->softmax_scale)) return CALIDROP_INVALID_ARG;
  return CALIDROP_OK;
}

int check_compress(const calidrop_params* p) {
  int rc = check_common(p);
  if (rc != CALIDROP_OK) return rc;
  if (p->L < 1 || p->window < 1 || p->budget < 1) return CALIDROP_INVALID_ARG;
  if (p->pool < 1 || p->pool % 2 == 0) return CALIDROP_INVALID_ARG;
  if (p->n_cal > p->window) return CALIDROP_INVALID_ARG;
  if (p->budget < p->L && (p->budget <= p->window || p->L < p->window)) return CALIDROP_INVALID_ARG;
  const int n_kept = p->budget < p->L ? p->budget : p->L;
  if (p->cap < n_kept) return CALIDROP_INVALID_ARG;
  if (p->calib_size < -1) return CALIDROP_INVALID_ARG;
  return CALIDROP_OK;
}

float scale2_of(const calidrop_params* p) {
  const float s = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D);
  return s * kLog2e;
}

CompressGeom make_geom(const calidrop_params* p) {
  CompressGeom g{};
  g.B = p->B; g.Hq = p->Hq; g.Hkv = p->Hkv; g.G = p->Hq / p->Hkv;
  g.L = p->L; g.W = p->window; g.pool = p->pool; g.budget = p->budget; g.n_cal = p->n_cal; g.cap = p->cap;
  g.keep_all = p->budget >= p->L;
  g.n_cand = g.keep_all ? 0 : p->L - p->window;
  g.k_sel = g.keep_all ? 0 : p->budget - p->window;
  g.n_kept = g.keep_all ? p->L : p->budget;
  g.units = p->B * p->Hkv;
  g.bitmap_words = (p->L + 31) / 32;
  g.scale2 = scale2_of(p);
  // calibration size: how many of the n_cand - k_sel evicted candidates are calibrated
  const int n_evict = g.keep_all ? 0 : g.n_cand - g.k_sel;
  g.sized = !g.keep_all && p->calib_size != 0;
  g.n_calib = p->calib_size == 0 ? n_evict : (p->calib_size < 0 ? 0 : (p->calib_size < n_evict ? p->calib_size : n_evict));
  return g;
}

CompressWs make_ws(const CompressGeom& g) {
  CompressWs w{};
  size_t off = 0;
  const size_t n_cand = (size_t)(g.L > g.W ? g.L - g.W : 0);
  w.vote = off;    off = align_up(off + (size_t)g.units * n_cand * 4, 256);
  w.vote2 = off;   off = align_up(off + (g.G * g.W > 256 ? (size_t)g.units * n_cand * 4 : 0), 256);
  w.pooled = off;  off = align_up(off + (size_t)g.units * n_cand * 4, 256);
  w.row_lse = off; off = align_up(off + (size_t)g.B * g.Hq * g.W * 4, 256);
  w.bitmap = off;  off = align_up(off + (size_t)g.units * g.bitmap_words * 4, 256);
  w.bitmap2 = off; off = align_up(off + (g.sized ? (size_t)g.units * g.bitmap_words * 4 : 0), 256);
  w.calib_mask = g.sized ? w.bitmap2 : w.bitmap;
  w.n_tiles = (g.L + 127) / 128;
  w.stat_slots = w.n_tiles > 320 ? w.n_tiles : 320;
  w.stat_part = off; off = align_up(off + (size_t)g.B * g.Hq * g.W * w.stat_slots * 8, 256);
  w.status = off;    off = align_up(off + 4, 256);
  w.calib_o = w.calib_l = off;
  if (score_tc_supported(g) && calib_tc_supported(g)) {
    int gpb, n_cblocks, tpc, max_slots;
    size_t parts;
    calib_tc_plan(g, &gpb, &n_cblocks, &tpc, &max_slots, &parts);
    w.calib_o = off; off = align_up(off + parts * 128 * kD * 4, 256);
    w.calib_l = off; off = align_up(off + parts * kCalibGroups * 128 * 4, 256);
  }
  w.total = off;
  return w;
}

int device_supported() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  static int major_of[64];
  if (dev < 0 || dev >= 64) return 0;
  if (major_of[dev] == 0) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return 0;
    major_of[dev] = major;
  }
  return major_of[dev] == 10;
}

// Split-K factor of the decode launch: one CTA per SM at most (a CTA's ring takes most of an SM's
// shared memory), never fewer than 32 rows per split.
int decode_nsplit(int units_total, int n_kv) {
  int ns = kDecodeTargetCtas / units_total;
  if (ns < 1) ns = 1;
  if (ns > kDecodeMaxSplit) ns = kDecodeMaxSplit;
  const int by_rows = (n_kv + 31) / 32;
  if (ns > by_rows) ns = by_rows;
  return ns < 1 ? 1 : ns;
}

struct DecodeWs {
  size_t part_o, part_ml, part_best, counters, status, per_layer;
  int max_split;
};

DecodeWs make_decode_ws(const calidrop_params* p) {
  DecodeWs w{};
  const int units = p->B * p->Hkv;
  w.max_split = decode_nsplit(units, 1 << 30);
  size_t off = 0;
  w.counters = off; off = align_up(off + (size_t)units * 4 * kDecodeMaxLayers, 256);
  w.status = off;   off += 256;  // error word: nonzero after a bounded wait of the kernel ran out
  w.part_ml = off;  off = align_up(off + (size_t)units * w.max_split * kMaxG * 2 * 4, 256);
  w.part_best = off; off = align_up(off + (size_t)units * kMaxG * w.max_split * 8, 256);
  w.part_o = off;   off = align_up(off + (size_t)units * w.max_split * kMaxG * kD * 4, 256);
  w.per_layer = off;
  return w;
}

// Split plan and workspace carving of one decode-kernel launch over `cap_rows`-row caches.
DecodeCommon plan_decode(const calidrop_params* p, const DecodeWs& w, int n_layers, int kv_len, int n_kv,
                         bool has_new, int cap_rows, void* workspace) {
  DecodeCommon a{};
  a.B = p->B; a.Hq = p->Hq; a.Hkv = p->Hkv; a.G = p->Hq / p->Hkv; a.n_cal = p->n_cal; a.cap = cap_rows;
  a.kv_len = kv_len; a.n_kv = n_kv; a.has_new = has_new ? 1 : 0;
  a.units = p->B * p->Hkv; a.n_layers = n_layers;
  // the splits of a unit form one thread-block cluster: 1, 2, 4 or 8 CTAs
  int want = decode_nsplit(a.units * n_layers, n_kv);
  if (want > w.max_split) want = w.max_split;
  a.nsplit = 1;
  while (a.nsplit * 2 <= want && a.nsplit < 8) a.nsplit *= 2;
  // Few units with a long cache: several clusters per unit, combined through the workspace.  That
  // combine costs about 4 us (fences, a ticket, a round trip through L2), as much as a CTA needs
  // to stream a thousand rows, so a unit is split only while every CTA keeps at least 1024 rows.
  a.nclu = want / a.nsplit;
  const int rows_single = (n_kv + a.nsplit - 1) / a.nsplit;
  if (a.nclu > rows_single / 1024) a.nclu = rows_single / 1024;
  if (a.nclu < 1) a.nclu = 1;
  a.rows_per_split = (n_kv + a.nsplit * a.nclu - 1) / (a.nsplit * a.nclu);
  a.scale2 = scale2_of(p);
  a.theta1 = p->theta1; a.theta2 = p->theta2; a.always_apply = p->theta2 <= -1.0f;
  // The workspace is laid out array by array with the layer index outermost inside each
  // array, so it is carved for n_layers at once.
  char* base = (char*)workspace;
  const size_t nl = (size_t)n_layers;
  size_t off = 0;
  a.counters = (unsigned*)(base + off); off += align_up((size_t)a.units * 4 * kDecodeMaxLayers, 256);
  a.status = (unsigned*)(base + off);   off += 256;
  a.part_ml = (float*)(base + off);     off += align_up((size_t)a.units * a.nclu * kMaxG * 2 * 4 * nl, 256);
  a.part_best = (unsigned long long*)(base + off); off += align_up((size_t)a.units * a.nclu * kMaxG * 8 * nl, 256);
  a.part_o = (float*)(base + off);
  a.recal_slot = 0;
  return a;
}

// Built-in scratch of calidrop_decode_static.  In host code this name is only a handle for
// cudaGetSymbolAddress; the kernel must be given the device address that call returns.
static __device__ __align__(256) unsigned char g_static_decode_scratch[CALIDROP_STATIC_SCRATCH_BYTES];

// Device address of the built-in scratch on the current device (looked up once per device).
int static_scratch_ptr(void** out) {
  static void* ptr_of[64];
  static std::atomic<int> ready[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return CALIDROP_UNSUPPORTED;
  if (!ready[dev].load(std::memory_order_acquire)) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_decode_scratch);
    if (e != cudaSuccess) return cuda_fail(e);
    if (!ptr) return CALIDROP_CUDA_ERROR;
    ptr_of[dev] = ptr;   // racing first calls store the same value
    ready[dev].store(1, std::memory_order_release);
  }
  *out = ptr_of[dev];
  return CALIDROP_OK;
}

}  // namespace

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

}  // namespace calidrop

using namespace calidrop;

extern "C" {

size_t calidrop_compress_workspace_bytes(const calidrop_params* p) {
  if (check_compress(p) != CALIDROP_OK) return 0;
  return make_ws(make_geom(p)).total;
}

int calidrop_compress_workspace_layout(const calidrop_params* p, calidrop_compress_layout* out) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK || !out) return rc != CALIDROP_OK ? rc : CALIDROP_INVALID_ARG;
  CompressWs w = make_ws(make_geom(p));
  out->vote_offset = w.vote;
  out->pooled_offset = w.pooled;
  out->row_lse_offset = w.row_lse;
  out->status_offset = w.status;
  return CALIDROP_OK;
}

int calidrop_compress(const calidrop_params* p, const void* Q_obs, const void* K, const void* V,
                      const float* lse_obs, int32_t* kept_idx, void* K_kept, void* V_kept, float* O_c,
                      float* LSE_c, void* C_q, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK) return rc;
  const void* ptrs[] = {Q_obs, K, V, kept_idx, K_kept, V_kept, O_c, LSE_c, C_q, workspace};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return CALIDROP_INVALID_ARG;
  if (lse_obs && !aligned16(lse_obs)) return CALIDROP_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return CALIDROP_INVALID_ARG;
  const CompressGeom g = make_geom(p);
  const CompressWs ws = make_ws(g);
  if (workspace_bytes < ws.total) return CALIDROP_WORKSPACE_TOO_SMALL;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;
  // a sized calibration takes its second threshold in the cluster selection kernel
  if (g.sized && g.n_calib > 0 && !select_cluster_supported(g)) return CALIDROP_UNSUPPORTED;

  cudaStream_t st = (cudaStream_t)stream;
  char* wsp = (char*)workspace;
  cudaError_t e = cudaMemsetAsync(wsp + ws.status, 0, 4, st);
  if (e != cudaSuccess) return cuda_fail(e);
  // The contractions run on the tensor cores whenever the tiles cover the shape; the scalar
  // kernels remain for the rest (more than 512 window rows per kv head, budget >= L).
  const bool tc_path = score_tc_supported(g);
  const float* row_lse = lse_obs;
  if (!g.keep_all) {
    if (!row_lse) {
      e = tc_path ? launch_row_stats_tc(g, ws, Q_obs, K, wsp, st) : launch_row_stats(g, ws, Q_obs, K, wsp, st);
      if (e != cudaSuccess) return cuda_fail(e);
      row_lse = (const float*)(wsp + ws.row_lse);
    }
    e = tc_path ? launch_votes_tc(g, ws, Q_obs, K, row_lse, wsp, st) : launch_votes(g, ws, Q_obs, K, row_lse, wsp, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  e = select_cluster_supported(g) ? launch_pool_select_cluster(g, ws, wsp, kept_idx, st)
                                  : launch_pool_select(g, ws, wsp, kept_idx, st);
  if (e != cudaSuccess) return cuda_fail(e);
  // the compaction of the retained rows rides on the calibration's second kernel when that runs
  const bool calib_tc = tc_path && calib_tc_supported(g) && !(g.sized && g.n_calib == 0);
  if (!calib_tc) {
    e = launch_gather(g, K, V, kept_idx, K_kept, V_kept, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  const GatherArgs ga{(const uint4*)K, (const uint4*)V, kept_idx, (uint4*)K_kept, (uint4*)V_kept,
                      g.L, g.n_kept, g.cap, g.units};
  if (g.sized && g.n_calib == 0)
    e = launch_calib_none(g, Q_obs, O_c, LSE_c, C_q, st);
  else
    e = calib_tc ? launch_calib_tc(g, ws, Q_obs, K, V, row_lse, wsp, O_c, LSE_c, C_q, ga, st)
                 : launch_calib_direct(g, ws, Q_obs, K, V, wsp, O_c, LSE_c, C_q, st);
  if (e != cudaSuccess) return cuda_fail(e);
  return CALIDROP_OK;
}

int calidrop_calibrate(const calidrop_params* p, const void* Q_obs, const void* K, const void* V,
                       const float* lse_obs, const int32_t* kept_idx, void* K_kept, void* V_kept, float* O_c,
                       float* LSE_c, void* C_q, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK) return rc;
  const void* ptrs[] = {Q_obs, K, V, kept_idx, K_kept, V_kept, O_c, LSE_c, C_q, workspace};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return CALIDROP_INVALID_ARG;
  if (lse_obs && !aligned16(lse_obs)) return CALIDROP_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return CALIDROP_INVALID_ARG;
  if (p->calib_size != 0) return CALIDROP_INVALID_ARG;   // no votes here to rank the evicted rows by
  const CompressGeom g = make_geom(p);
  const CompressWs ws = make_ws(g);
  if (workspace_bytes < ws.total) return CALIDROP_WORKSPACE_TOO_SMALL;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;

  cudaStream_t st = (cudaStream_t)stream;
  char* wsp = (char*)workspace;
  cudaError_t e = cudaMemsetAsync(wsp + ws.status, 0, 4, st);
  if (e != cudaSuccess) return cuda_fail(e);
  const bool tc_path = score_tc_supported(g);
  // the calibration probabilities refer to the full-row softmax: its row LSE comes from the caller
  // or from the statistics pass of the scoring
  const float* row_lse = lse_obs;
  if (!g.keep_all && !row_lse) {
    e = tc_path ? launch_row_stats_tc(g, ws, Q_obs, K, wsp, st) : launch_row_stats(g, ws, Q_obs, K, wsp, st);
    if (e != cudaSuccess) return cuda_fail(e);
    row_lse = (const float*)(wsp + ws.row_lse);
  }
  e = launch_bitmap_from_indices(g, ws, wsp, kept_idx, st);
  if (e != cudaSuccess) return cuda_fail(e);
  const bool calib_tc = tc_path && calib_tc_supported(g);
  if (!calib_tc) {
    e = launch_gather(g, K, V, kept_idx, K_kept, V_kept, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  const GatherArgs ga{(const uint4*)K, (const uint4*)V, kept_idx, (uint4*)K_kept, (uint4*)V_kept,
                      g.L, g.n_kept, g.cap, g.units};
  e = calib_tc ? launch_calib_tc(g, ws, Q_obs, K, V, row_lse, wsp, O_c, LSE_c, C_q, ga, st)
               : launch_calib_direct(g, ws, Q_obs, K, V, wsp, O_c, LSE_c, C_q, st);
  if (e != cudaSuccess) return cuda_fail(e);
  return CALIDROP_OK;
}

size_t calidrop_accumulated_scores_workspace_bytes(const calidrop_params* p) {
  if (check_compress(p) != CALIDROP_OK) return 0;
  return align_up((size_t)p->B * p->Hq * p->L * 4, 256);
}

int calidrop_accumulated_scores(const calidrop_params* p, const void* Q_full, const void* K, float* scores,
                                void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK) return rc;
  const void* ptrs[] = {Q_full, K, scores, workspace};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return CALIDROP_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return CALIDROP_INVALID_ARG;
  if (workspace_bytes < calidrop_accumulated_scores_workspace_bytes(p)) return CALIDROP_WORKSPACE_TOO_SMALL;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;
  const CompressGeom g = make_geom(p);
  cudaError_t e = launch_accum_scores(p->B, p->Hq, p->Hkv, p->L, g.scale2, Q_full, K, (float*)workspace, scores,
                                      (cudaStream_t)stream);
  return e == cudaSuccess ? CALIDROP_OK : cuda_fail(e);
}

int calidrop_select_streaming(const calidrop_params* p, int32_t n_sink, int32_t* kept_idx, void* stream) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK) return rc;
  if (!kept_idx || !aligned16(kept_idx)) return CALIDROP_INVALID_ARG;
  const CompressGeom g = make_geom(p);
  const int recent_min = p->window < g.n_kept ? p->window : g.n_kept;
  if (n_sink < 0 || n_sink > g.n_kept - recent_min) return CALIDROP_INVALID_ARG;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;
  cudaError_t e = launch_streaming_indices(g, n_sink, kept_idx, (cudaStream_t)stream);
  return e == cudaSuccess ? CALIDROP_OK : cuda_fail(e);
}

int calidrop_select_from_scores(const calidrop_params* p, const float* scores, int32_t tail, int32_t* kept_idx,
                                void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK) return rc;
  if (!scores || !kept_idx || !workspace || !aligned16(scores) || !aligned16(kept_idx)) return CALIDROP_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return CALIDROP_INVALID_ARG;
  if (p->budget >= p->L || tail < p->window || tail >= p->budget) return CALIDROP_INVALID_ARG;
  const CompressGeom g0 = make_geom(p);
  const CompressWs ws = make_ws(g0);   // sized for window <= tail: the pooled scores of L - tail rows fit
  if (workspace_bytes < ws.total) return CALIDROP_WORKSPACE_TOO_SMALL;
  // the selection's geometry: `tail` rows are always kept, the rest compete
  CompressGeom g = g0;
  g.W = tail; g.n_cand = p->L - tail; g.k_sel = p->budget - tail; g.sized = 0; g.n_calib = 0;
  if (!select_cluster_supported(g)) return CALIDROP_UNSUPPORTED;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;
  cudaError_t e = launch_pool_select_scores(g, ws, (char*)workspace, scores, (size_t)p->L, kept_idx, (cudaStream_t)stream);
  return e == cudaSuccess ? CALIDROP_OK : cuda_fail(e);
}

int calidrop_gather_evicted(const calidrop_params* p, const void* K, const void* V, const int32_t* kept_idx,
                            int32_t* evict_idx, void* K_evict, void* V_evict, void* workspace,
                            size_t workspace_bytes, void* stream) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK) return rc;
  const void* ptrs[] = {K, V, kept_idx, evict_idx, K_evict, V_evict, workspace};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return CALIDROP_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return CALIDROP_INVALID_ARG;
  const CompressGeom g = make_geom(p);
  if (g.keep_all || g.n_calib == 0) return CALIDROP_INVALID_ARG;  // nothing is evicted / kept for calibration
  const CompressWs ws = make_ws(g);
  if (workspace_bytes < ws.total) return CALIDROP_WORKSPACE_TOO_SMALL;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  char* wsp = (char*)workspace;
  cudaError_t e = cudaSuccess;
  // sized calibration: the mask of the calibrated rows is the one calidrop_compress left in this workspace
  if (!g.sized) e = launch_bitmap_from_indices(g, ws, wsp, kept_idx, st);
  if (e != cudaSuccess) return cuda_fail(e);
  e = launch_evicted_indices(g, ws, wsp, evict_idx, st);
  if (e != cudaSuccess) return cuda_fail(e);
  const int n_evict = g.n_calib;
  e = launch_gather_rows(g, K, V, evict_idx, n_evict, n_evict, K_evict, V_evict, st);
  return e == cudaSuccess ? CALIDROP_OK : cuda_fail(e);
}

namespace {
// One asynchronous copy per tensor on the caller's copy stream, between the caller's two events.
int move_evicted(const calidrop_params* p, int32_t n_evict, const void* K_src, const void* V_src, void* K_dst,
                 void* V_dst, cudaMemcpyKind kind, void* copy_stream, void* wait_event, void* done_event) {
  int rc = check_common(p);
  if (rc != CALIDROP_OK) return rc;
  if (!K_src || !V_src || !K_dst || !V_dst || n_evict < 1) return CALIDROP_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)copy_stream;
  const size_t bytes = (size_t)p->B * p->Hkv * n_evict * kD * 2;
  cudaError_t e;
  if (wait_event && (e = cudaStreamWaitEvent(cs, (cudaEvent_t)wait_event, 0)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(K_dst, K_src, bytes, kind, cs)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(V_dst, V_src, bytes, kind, cs)) != cudaSuccess) return cuda_fail(e);
  if (done_event && (e = cudaEventRecord((cudaEvent_t)done_event, cs)) != cudaSuccess) return cuda_fail(e);
  return CALIDROP_OK;
}
}  // namespace

int calidrop_offload_evicted(const calidrop_params* p, int32_t n_evict, const void* K_evict, const void* V_evict,
                             void* K_host, void* V_host, void* copy_stream, void* wait_event, void* done_event) {
  return move_evicted(p, n_evict, K_evict, V_evict, K_host, V_host, cudaMemcpyDeviceToHost, copy_stream, wait_event,
                      done_event);
}

int calidrop_reload_evicted(const calidrop_params* p, int32_t n_evict, const void* K_host, const void* V_host,
                            void* K_evict, void* V_evict, void* copy_stream, void* wait_event, void* done_event) {
  return move_evicted(p, n_evict, K_host, V_host, K_evict, V_evict, cudaMemcpyHostToDevice, copy_stream, wait_event,
                      done_event);
}

int calidrop_recalibrate(const calidrop_params* p, const void* q, const void* K_evict, const void* V_evict,
                         int32_t n_evict, int32_t slot, float* O_c, float* LSE_c, void* C_q, void* workspace,
                         size_t workspace_bytes, void* stream) {
  int rc = check_common(p);
  if (rc != CALIDROP_OK) return rc;
  const void* req[] = {q, K_evict, V_evict, O_c, LSE_c, C_q, workspace};
  for (const void* r : req)
    if (!r || !aligned16(r)) return CALIDROP_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return CALIDROP_INVALID_ARG;
  if (n_evict < 1 || slot < 0 || slot >= p->n_cal) return CALIDROP_INVALID_ARG;
  const DecodeWs w = make_decode_ws(p);
  if (workspace_bytes < w.per_layer) return CALIDROP_WORKSPACE_TOO_SMALL;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;
  DecodeArgsT<1> args{};
  args.c = plan_decode(p, w, 1, n_evict, n_evict, false, n_evict, workspace);
  args.c.recal_slot = slot;
  args.layer[0] = DecodeLayerPtrs{q, nullptr, nullptr, const_cast<void*>(K_evict), const_cast<void*>(V_evict), O_c,
                                  LSE_c, C_q, nullptr, nullptr, nullptr};
  if (!make_decode_maps(args.c, args.layer[0], &args.maps[0])) return CALIDROP_CUDA_ERROR;
  cudaError_t e = launch_recalibrate(args, (cudaStream_t)stream);
  return e == cudaSuccess ? CALIDROP_OK : cuda_fail(e);
}

size_t calidrop_decode_workspace_bytes(const calidrop_params* p, int32_t kv_len_max) {
  if (check_common(p) != CALIDROP_OK || kv_len_max < 1) return 0;
  return make_decode_ws(p).per_layer;
}

size_t calidrop_decode_workspace_status_offset(const calidrop_params* p) {
  if (check_common(p) != CALIDROP_OK) return (size_t)-1;
  return make_decode_ws(p).status;
}

int calidrop_decode_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace) return CALIDROP_INVALID_ARG;
  cudaError_t e = cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream);
  return e == cudaSuccess ? CALIDROP_OK : cuda_fail(e);
}

int calidrop_decode_batched(const calidrop_params* p, int32_t n_layers, const calidrop_decode_layer* layers,
                            int32_t kv_len, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_common(p);
  if (rc != CALIDROP_OK) return rc;
  if (!layers || n_layers < 1 || n_layers > CALIDROP_MAX_LAYERS) return CALIDROP_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return CALIDROP_INVALID_ARG;
  if (kv_len < 0) return CALIDROP_INVALID_ARG;
  const bool has_new = layers[0].k_new != nullptr;
  const int n_kv = kv_len + (has_new ? 1 : 0);
  if (n_kv < 1 || n_kv > p->cap) return CALIDROP_INVALID_ARG;
  for (int i = 0; i < n_layers; ++i) {
    const calidrop_decode_layer& L = layers[i];
    const void* req[] = {L.q, L.K_kept, L.V_kept, L.O_c, L.LSE_c, L.C_q, L.out};
    for (const void* q : req)
      if (!q || !aligned16(q)) return CALIDROP_INVALID_ARG;
    if ((L.k_new != nullptr) != has_new || (L.v_new != nullptr) != has_new) return CALIDROP_INVALID_ARG;
    if (has_new && (!aligned16(L.k_new) || !aligned16(L.v_new))) return CALIDROP_INVALID_ARG;
  }
  const DecodeWs w = make_decode_ws(p);
  if (workspace_bytes < w.per_layer * (size_t)n_layers) return CALIDROP_WORKSPACE_TOO_SMALL;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;

  DecodeCommon a = plan_decode(p, w, n_layers, kv_len, n_kv, has_new, p->cap, workspace);
  cudaError_t e;
  if (n_layers == 1) {
    DecodeArgsT<1> args{};
    args.c = a;
    const calidrop_decode_layer& L = layers[0];
    args.layer[0] = DecodeLayerPtrs{L.q, L.k_new, L.v_new, L.K_kept, L.V_kept, L.O_c, L.LSE_c, L.C_q,
                                    L.out, L.lse_out, L.flags};
    if (!make_decode_maps(a, args.layer[0], &args.maps[0])) return CALIDROP_CUDA_ERROR;
    e = launch_decode(args, (cudaStream_t)stream);
  } else {
    static thread_local DecodeArgsT<kDecodeMaxLayers> args;
    args.c = a;
    for (int i = 0; i < n_layers; ++i) {
      const calidrop_decode_layer& L = layers[i];
      args.layer[i] = DecodeLayerPtrs{L.q, L.k_new, L.v_new, L.K_kept, L.V_kept, L.O_c, L.LSE_c, L.C_q,
                                      L.out, L.lse_out, L.flags};
      if (!make_decode_maps(a, args.layer[i], &args.maps[i])) return CALIDROP_CUDA_ERROR;
    }
    e = launch_decode(args, (cudaStream_t)stream);
  }
  return e == cudaSuccess ? CALIDROP_OK : cuda_fail(e);
}

int calidrop_decode(const calidrop_params* p, const void* q, const void* k_new, const void* v_new,
                    void* K_kept, void* V_kept, int32_t kv_len, const float* O_c, const float* LSE_c,
                    const void* C_q, void* out, float* lse_out, uint8_t* flags, void* workspace,
                    size_t workspace_bytes, void* stream) {
  calidrop_decode_layer L{q, k_new, v_new, K_kept, V_kept, O_c, LSE_c, C_q, out, lse_out, flags};
  return calidrop_decode_batched(p, 1, &L, kv_len, workspace, workspace_bytes, stream);
}

int calidrop_decode_static(const calidrop_params* p, const void* q, const void* k_new, const void* v_new,
                           void* K_kept, void* V_kept, int32_t kv_len, const float* O_c, const float* LSE_c,
                           const void* C_q, void* out, float* lse_out, uint8_t* flags, void* stream) {
  int rc = check_common(p);
  if (rc != CALIDROP_OK) return rc;
  const DecodeWs w = make_decode_ws(p);
  if (w.per_layer > (size_t)CALIDROP_STATIC_SCRATCH_BYTES) return CALIDROP_SCRATCH_LIMIT;
  // Everything calidrop_decode would reject is rejected here too, before the scratch is touched.
  const void* req[] = {q, K_kept, V_kept, O_c, LSE_c, C_q, out};
  for (const void* r : req)
    if (!r || !aligned16(r)) return CALIDROP_INVALID_ARG;
  if ((k_new != nullptr) != (v_new != nullptr)) return CALIDROP_INVALID_ARG;
  if (k_new && (!aligned16(k_new) || !aligned16(v_new))) return CALIDROP_INVALID_ARG;
  const int n_kv = kv_len + (k_new ? 1 : 0);
  if (kv_len < 0 || n_kv < 1 || n_kv > p->cap) return CALIDROP_INVALID_ARG;
  if (!device_supported()) return CALIDROP_UNSUPPORTED;
  void* scratch = nullptr;
  rc = static_scratch_ptr(&scratch);
  if (rc != CALIDROP_OK) return rc;
  // The arrival counters lead the carving; the rest of the scratch is written before it is read.
  cudaError_t e = cudaMemsetAsync(scratch, 0, w.part_ml, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e);
  return calidrop_decode(p, q, k_new, v_new, K_kept, V_kept, kv_len, O_c, LSE_c, C_q, out, lse_out, flags,
                         scratch, (size_t)CALIDROP_STATIC_SCRATCH_BYTES, stream);
}

int calidrop_compress_host(const calidrop_params* p, const void* Q_obs_h, const void* K_h, const void* V_h,
                           const float* lse_obs_h, int32_t* kept_idx_h, float* O_c_h, float* LSE_c_h,
                           void* Q_obs, void* K, void* V, float* lse_obs, int32_t* kept_idx, void* K_kept,
                           void* V_kept, float* O_c, float* LSE_c, void* C_q, void* workspace,
                           size_t workspace_bytes, void* stream) {
  int rc = check_compress(p);
  if (rc != CALIDROP_OK) return rc;
  if (!Q_obs_h || !K_h || !V_h || !kept_idx_h || !O_c_h || !LSE_c_h) return CALIDROP_INVALID_ARG;
  if (!Q_obs || !K || !V || !kept_idx || !K_kept || !V_kept || !O_c || !LSE_c || !C_q || !workspace)
    return CALIDROP_INVALID_ARG;
  if (lse_obs_h && !lse_obs) return CALIDROP_INVALID_ARG;
  if (workspace_bytes < calidrop_compress_workspace_bytes(p)) return CALIDROP_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t q_bytes = (size_t)p->B * p->Hq * p->window * kD * 2;
  const size_t kv_bytes = (size_t)p->B * p->Hkv * p->L * kD * 2;
  const size_t n_kept = p->budget < p->L ? p->budget : p->L;
  cudaError_t e;
  if ((e = cudaMemcpyAsync(Q_obs, Q_obs_h, q_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(K, K_h, kv_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(V, V_h, kv_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
  if (lse_obs_h) {
    e = cudaMemcpyAsync(lse_obs, lse_obs_h, (size_t)p->B * p->Hq * p->window * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  rc = calidrop_compress(p, Q_obs, K, V, lse_obs_h ? lse_obs : nullptr, kept_idx, K_kept, V_kept, O_c, LSE_c,
                         C_q, workspace, workspace_bytes, stream);
  if (rc != CALIDROP_OK) return rc;
  if ((e = cudaMemcpyAsync(kept_idx_h, kept_idx, (size_t)p->B * p->Hkv * n_kept * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(O_c_h, O_c, (size_t)p->B * p->Hq * p->n_cal * kD * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(LSE_c_h, LSE_c, (size_t)p->B * p->Hq * p->n_cal * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e);
  return CALIDROP_OK;
}

int calidrop_decode_host(const calidrop_params* p, const void* q_h, const void* k_new_h, const void* v_new_h,
                         void* out_h, float* lse_out_h, uint8_t* flags_h, void* q, void* k_new, void* v_new,
                         void* K_kept, void* V_kept, int32_t kv_len, const float* O_c, const float* LSE_c,
                         const void* C_q, void* out, float* lse_out, uint8_t* flags, void* workspace,
                         size_t workspace_bytes, void* stream) {
  int rc = check_common(p);
  if (rc != CALIDROP_OK) return rc;
  if (!q_h || !out_h || !q || !out) return CALIDROP_INVALID_ARG;
  if ((k_new_h != nullptr) != (v_new_h != nullptr)) return CALIDROP_INVALID_ARG;
  if (k_new_h && (!k_new || !v_new)) return CALIDROP_INVALID_ARG;
  if ((lse_out_h && !lse_out) || (flags_h && !flags)) return CALIDROP_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t q_bytes = (size_t)p->B * p->Hq * kD * 2;
  const size_t kv_bytes = (size_t)p->B * p->Hkv * kD * 2;
  cudaError_t e;
  if ((e = cudaMemcpyAsync(q, q_h, q_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
  if (k_new_h) {
    if ((e = cudaMemcpyAsync(k_new, k_new_h, kv_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(v_new, v_new_h, kv_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
  }
  rc = calidrop_decode(p, q, k_new_h ? k_new : nullptr, k_new_h ? v_new : nullptr, K_kept, V_kept, kv_len, O_c,
                       LSE_c, C_q, out, lse_out, flags, workspace, workspace_bytes, stream);
  if (rc != CALIDROP_OK) return rc;
  if ((e = cudaMemcpyAsync(out_h, out, q_bytes, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e);
  if (lse_out_h && (e = cudaMemcpyAsync(lse_out_h, lse_out, (size_t)p->B * p->Hq * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e);
  if (flags_h && (e = cudaMemcpyAsync(flags_h, flags, (size_t)p->B * p->Hq, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e);
  return CALIDROP_OK;
}

const char* calidrop_status_string(int status) {
  switch (status) {
    case CALIDROP_OK: return "ok";
    case CALIDROP_INVALID_ARG: return "invalid argument";
    case CALIDROP_UNSUPPORTED: return "unsupported configuration or device";
    case CALIDROP_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CALIDROP_CUDA_ERROR: return g_err_text[0] ? g_err_text : "CUDA error";
    case CALIDROP_SCRATCH_LIMIT: return "problem needs more scratch than the built-in static buffer holds";
    default: return "unknown status";
  }
}

int calidrop_version(void) { return 100; }

uint64_t calidrop_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
