// Internal launcher interface between the C-ABI layer (api.cu) and the kernels.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace calidrop {

// Geometry of one compress call, derived from calidrop_params on the host.
struct CompressGeom {
  int B, Hq, Hkv, G, L, W, pool, budget, n_cal, cap;
  int n_cand;   // L - W candidates per unit (0 when everything is kept)
  int k_sel;    // budget - W selected candidates
  int n_kept;   // min(budget, L)
  int keep_all; // budget >= L
  int units;    // B * Hkv
  int bitmap_words;  // ceil(L / 32) per unit
  float scale2;      // softmax scale * log2(e)
  // calibration size: n_calib of the evicted candidates take part in the calibration (all of them
  // unless `sized`); the masked passes then read the bitmap at ws.calib_mask
  int sized, n_calib;
};

// Workspace carving of compress (byte offsets, all 256-byte aligned).
struct CompressWs {
  size_t vote, vote2, pooled, row_lse, bitmap, stat_part, status, calib_o, calib_l, total;
  size_t bitmap2;     // sized calibration: bit set = the row is NOT one of the calibrated evicted rows
  size_t calib_mask;  // the bitmap the calibration passes mask with: bitmap, or bitmap2 when sized
  int n_tiles;     // 128-key tiles per unit (scalar statistics pass: one partial per tile)
  int stat_slots;  // (max, sum) partial slots per observation row in stat_part
};

struct DecodeLayerPtrs {
  const void* q;
  const void* k_new;
  const void* v_new;
  void* K;
  void* V;
  const float* O_c;
  const float* LSE_c;
  const void* C_q;
  void* out;
  float* lse_out;
  uint8_t* flags;
};

// TMA views of one layer's retained cache, [unit][row][128] bf16 with 128-byte swizzle: boxes of
// 64 rows for whole ring slots and of 16 rows for the ragged end of a split.  k64, v64 and k16 span
// the cache's capacity; v16 ends at row kv_len (rows beyond it arrive as zeros).
struct alignas(64) DecodeLayerMaps {
  CUtensorMap k64, v64, k16, v16;
};

constexpr int kCalibGroups = 4;  // softmax warpgroups of the calibration kernel: row-sum partials per slot
constexpr int kDecodeMaxLayers = 32;
constexpr int kDecodeMaxSplit = 64;
constexpr int kDecodeTargetCtas = 148;  // one CTA of a launch on each of the 148 SMs

struct DecodeCommon {
  int B, Hq, Hkv, G, n_cal, cap, kv_len, n_kv, has_new;
  int units, n_layers, rows_per_split;
  int nsplit;  // CTAs per cluster (1, 2, 4 or 8): the splits combined through distributed shared memory
  int nclu;    // clusters per (layer, unit); more than one only when few units share a long cache
  float scale2, theta1, theta2;
  int always_apply;
  // workspace arrays, used only when nclu > 1: per-cluster partials and the arrival counters
  float* part_o;                  // [layer][unit][nclu][8][128]
  float* part_ml;                 // [layer][unit][nclu][8][2]
  unsigned long long* part_best;  // [layer][unit][nclu][8] best (similarity, row) keys
  unsigned* counters;             // [layer][unit]
  unsigned* status;               // error word of the workspace: nonzero after a wait ran out
  int recal_slot;                 // launch_recalibrate only: the calibration row that is rewritten
};

// Kernel argument block for NL layers (1 for the single-layer entry points, 32 for the batched one:
// the block travels with every launch, so the common case keeps it small).
template <int NL>
struct DecodeArgsT {
  DecodeCommon c;
  DecodeLayerPtrs layer[NL];
  DecodeLayerMaps maps[NL];
};

// compress_simt.cu
cudaError_t launch_row_stats(const CompressGeom& g, const CompressWs& ws, const void* Q_obs,
                             const void* K, char* wsp, cudaStream_t st);
cudaError_t launch_votes(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                         const float* row_lse, char* wsp, cudaStream_t st);
cudaError_t launch_calib_direct(const CompressGeom& g, const CompressWs& ws, const void* Q_obs,
                                const void* K, const void* V, char* wsp, float* O_c, float* LSE_c,
                                void* C_q, cudaStream_t st);
// score_tc.cu / calib_tc.cu: the tcgen05 + TMA path
int pick_tile_splits(int groups, int n_tiles, int min_tiles);
bool score_tc_supported(const CompressGeom& g);
cudaError_t launch_row_stats_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                                char* wsp, cudaStream_t st);
cudaError_t launch_votes_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                            const float* row_lse, char* wsp, cudaStream_t st);
bool calib_tc_supported(const CompressGeom& g);
void calib_tc_plan(const CompressGeom& g, int* gpb, int* n_cblocks, int* tiles_per_cta, int* max_slots,
                   size_t* parts);
// The compaction of the retained rows (A5), as arguments: K_out[u, i, :] = K[u, idx[u, i], :], same
// for V.  The calibration's second kernel carries it along (blocks of its own beside the reduction's)
// when `idx` is not null: it only depends on the kept list, and as a kernel of its own between the
// selection and the calibration its 10 us at copy bandwidth were exposed.
struct GatherArgs {
  const uint4* K;
  const uint4* V;
  const int32_t* idx;   // [units, n_rows]
  uint4* K_out;         // [units, out_rows, 16]
  uint4* V_out;
  int L, n_rows, out_rows, units;
};
cudaError_t launch_calib_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                            const void* V, const float* row_lse, char* wsp, float* O_c, float* LSE_c, void* C_q,
                            const GatherArgs& gather, cudaStream_t st);
#ifdef __CUDACC__
// Rows [16 bx, 16 bx + 16) of unit `unit`: 16 lanes x 16 bytes per row, 256 threads.
__device__ __forceinline__ void gather_rows16(const GatherArgs& a, int bx, int unit, int tid) {
  const int i = bx * 16 + (tid >> 4);
  const int chunk = tid & 15;
  if (i >= a.n_rows) return;
  const int t = a.idx[(size_t)unit * a.n_rows + i];
  if (t < 0 || t >= a.L) return;   // a caller's list may hold anything: rows outside the prompt are skipped
  const size_t src = ((size_t)unit * a.L + t) * 16 + chunk;
  const size_t dst = ((size_t)unit * a.out_rows + i) * 16 + chunk;
  a.K_out[dst] = __ldg(a.K + src);
  a.V_out[dst] = __ldg(a.V + src);
}
#endif
// select.cu
cudaError_t launch_pool_select(const CompressGeom& g, const CompressWs& ws, char* wsp,
                               int32_t* kept_idx, cudaStream_t st);
// select_cluster.cu
bool select_cluster_supported(const CompressGeom& g);
cudaError_t launch_pool_select_cluster(const CompressGeom& g, const CompressWs& ws, char* wsp, int32_t* kept_idx,
                                       cudaStream_t st);
cudaError_t launch_pool_select_scores(const CompressGeom& g, const CompressWs& ws, char* wsp, const float* scores,
                                      size_t stride, int32_t* kept_idx, cudaStream_t st);
cudaError_t launch_streaming_indices(const CompressGeom& g, int n_sink, int32_t* kept_idx, cudaStream_t st);
cudaError_t launch_bitmap_from_indices(const CompressGeom& g, const CompressWs& ws, char* wsp,
                                       const int32_t* kept_idx, cudaStream_t st);
cudaError_t launch_gather_rows(const CompressGeom& g, const void* K, const void* V, const int32_t* idx, int n_rows,
                               int out_rows, void* K_out, void* V_out, cudaStream_t st);
cudaError_t launch_gather(const CompressGeom& g, const void* K, const void* V, const int32_t* kept_idx,
                          void* K_kept, void* V_kept, cudaStream_t st);
// accum_scores.cu
cudaError_t launch_accum_scores(int B, int Hq, int Hkv, int L, float scale2, const void* Q_full, const void* K,
                                float* lse2, float* scores, cudaStream_t st);
// decode.cu
// Fills the TMA views of one layer; false when the driver refuses the encoding.
bool make_decode_maps(const DecodeCommon& c, const DecodeLayerPtrs& L, DecodeLayerMaps* out);
cudaError_t launch_decode(const DecodeArgsT<1>& a, cudaStream_t st);
cudaError_t launch_decode(const DecodeArgsT<kDecodeMaxLayers>& a, cudaStream_t st);
// The same stream over the evicted KV (K, V of the layer = the compacted evicted rows), rewriting
// row recal_slot of O_c, LSE_c, C_q (Algorithm 2, lines 4-6).
cudaError_t launch_recalibrate(const DecodeArgsT<1>& a, cudaStream_t st);
cudaError_t launch_evicted_indices(const CompressGeom& g, const CompressWs& ws, char* wsp, int32_t* evict_idx,
                                   cudaStream_t st);
// Calibration size -1: no row is calibrated (O_c = 0, LSE_c = -inf, C_q = the calibration queries).
cudaError_t launch_calib_none(const CompressGeom& g, const void* Q_obs, float* O_c, float* LSE_c, void* C_q,
                              cudaStream_t st);

void count_launch(int n = 1);

#ifdef __CUDACC__
// Launch with the programmatic-serialisation attribute (see pdl_wait in common.cuh).
template <typename... Params, typename... Args>
cudaError_t launch_pdl(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}
#endif

}  // namespace calidrop
