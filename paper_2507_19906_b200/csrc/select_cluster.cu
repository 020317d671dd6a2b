// Pooling + per-(batch, kv-head) top-k on a thread-block cluster.
//
// The single-CTA selection of select.cu uses one SM per unit; with a few dozen units most of the
// GPU idles.  Here a cluster of eight CTAs shares a unit: CTA r owns the contiguous key range
// [r * chunk, (r + 1) * chunk), every thread keeps its ROWS keys (pooled votes as fp32 bit
// patterns) in registers, and the CTAs exchange only their 256-bin histograms and their counts
// through distributed shared memory.  The algorithm is the same exact radix select: four 8-bit
// passes find the bit pattern T of the k-th largest pooled vote and how many candidates equal to
// T still fit; an ordered compaction then emits, ascending, every candidate above T and the first
// need_eq candidates equal to T (ties go to the lowest index), plus the kept bitmap.
// Key (row i, thread tid) of CTA r is candidate r * chunk + i * 1024 + tid, so a warp covers 32
// consecutive candidates: loads coalesce and one ballot is one bitmap word.
#include <cooperative_groups.h>

#include "common.cuh"
#include "internal.h"

namespace calidrop {

namespace {

namespace cg = cooperative_groups;

constexpr int kClu = 8;
constexpr int kT = 1024;
constexpr int kW = kT / 32;

template <int ROWS, bool kSized>
__global__ void __cluster_dims__(kClu, 1, 1) __launch_bounds__(kT, ROWS <= 8 ? 2 : 1)  // two CTAs per SM where many units make more CTAs than SMs
pool_select_cluster_kernel(const float* __restrict__ vote, float* __restrict__ pooled,
                           uint32_t* __restrict__ bitmap, int32_t* __restrict__ kept_idx, int n_cand, int L,
                           int pool, int k_sel, int n_kept, int bitmap_words, uint32_t* __restrict__ mask2,
                           int n_calib, size_t vote_stride) {
  __shared__ unsigned hist[kW][256];
  __shared__ unsigned mine[2][256];   // this CTA's histogram of the current pass (double-buffered)
  __shared__ unsigned total[256];
  __shared__ unsigned sel_bin, sel_k;
  __shared__ unsigned cnt[2][2];      // this CTA's counts of keys > T and == T, for the two thresholds
  __shared__ unsigned wsum[ROWS * kW][2];

  pdl_trigger();
  pdl_wait();
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int unit = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = ROWS * kT;
  const float* v = vote + (size_t)unit * vote_stride;
  float* pl = pooled + (size_t)unit * n_cand;
  uint32_t* bm = bitmap + (size_t)unit * bitmap_words;
  int32_t* kept = kept_idx + (size_t)unit * n_kept;

  // 1. zero-padded average pool with a constant divisor; keys stay in registers
  unsigned key[ROWS];
  const int half = pool >> 1;
  const float fpool = (float)pool;
#pragma unroll
  for (int i = 0; i < ROWS; ++i) {
    const int t = rank * chunk + i * kT + tid;
    key[i] = 0u;
    if (t < n_cand) {
      float acc = 0.f;
      for (int d = -half; d <= half; ++d) {
        const int u = t + d;
        if (u >= 0 && u < n_cand) acc += v[u];
      }
      const float p = acc / fpool;
      pl[t] = p;
      key[i] = __float_as_uint(p);
    }
  }

  // 2. radix select, most significant byte first; the histograms of the eight CTAs are summed
  // through distributed shared memory.  Returns the bit pattern T of the kk-th largest pooled vote
  // and how many candidates equal to T are still taken (those at the lowest positions).
  auto radix_select = [&](unsigned kk, unsigned& T_out, unsigned& need_out) __attribute__((always_inline)) {
    unsigned prefix = 0, k = kk;
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < kW * 256; i += kT) (&hist[0][0])[i] = 0;
      __syncthreads();
#pragma unroll
      for (int i = 0; i < ROWS; ++i) {
        const int t = rank * chunk + i * kT + tid;
        const bool in = t < n_cand && ((pass == 0) || ((key[i] >> (shift + 8)) == prefix));
        if (in) atomicAdd(&hist[warp][(key[i] >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid < 256) {
        unsigned s = 0;
#pragma unroll 8
        for (int w = 0; w < kW; ++w) s += hist[w][tid];
        mine[pass & 1][tid] = s;
      }
      cluster.sync();
      if (tid < 256) {
        unsigned s = 0;
        for (int r = 0; r < kClu; ++r) s += cluster.map_shared_rank(&mine[pass & 1][0], r)[tid];
        total[tid] = s;
      }
      __syncthreads();
      if (warp == 0) {
        // lane 0 owns the 8 highest bins; walk bins downwards until k candidates are covered
        const int base = 255 - 8 * lane;
        unsigned c[8], s = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = total[base - j]; s += c[j]; }
        unsigned incl = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += n;
        }
        const unsigned ball = __ballot_sync(0xffffffffu, incl >= k);
        const int target = __ffs(ball) - 1;  // always found: the candidates number at least k
        if (lane == target) {
          unsigned run = incl - s;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (run + c[j] >= k) { sel_bin = (unsigned)(base - j); sel_k = k - run; break; }
            run += c[j];
          }
        }
      }
      __syncthreads();
      prefix = (prefix << 8) | sel_bin;
      k = sel_k;
    }
    // (the two passes that still use mine[] of this call lie at least two cluster barriers behind
    // when the next call writes them again)
    T_out = prefix;
    need_out = k;
  };
  unsigned T, need_eq;
  radix_select((unsigned)k_sel, T, need_eq);

  // 3. ordered compaction.  Per (row, warp): how many keys are above T / equal to T; the exclusive
  // scan of those counts in index order, over the cluster, gives every key the number of keys
  // above / equal to the threshold that precede it.
  unsigned gt_mask[ROWS], eq_mask[ROWS];
  unsigned before_gt = 0, before_eq = 0;  // keys of the lower-ranked CTAs
  auto scan_threshold = [&](unsigned Tx, int slot) __attribute__((always_inline)) {
#pragma unroll
    for (int i = 0; i < ROWS; ++i) {
      const int t = rank * chunk + i * kT + tid;
      const bool valid = t < n_cand;
      gt_mask[i] = __ballot_sync(0xffffffffu, valid && key[i] > Tx);
      eq_mask[i] = __ballot_sync(0xffffffffu, valid && key[i] == Tx);
      if (lane == 0) {
        wsum[i * kW + warp][0] = __popc(gt_mask[i]);
        wsum[i * kW + warp][1] = __popc(eq_mask[i]);
      }
    }
    __syncthreads();
    // exclusive scan of the ROWS * 32 warp counts in index order (row-major), by the first warp
    if (warp == 0) {
      unsigned run_gt = 0, run_eq = 0;
      for (int base = 0; base < ROWS * kW; base += 32) {
        const unsigned g0 = wsum[base + lane][0], e0 = wsum[base + lane][1];
        unsigned ig = g0, ie = e0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned a = __shfl_up_sync(0xffffffffu, ig, o);
          const unsigned b = __shfl_up_sync(0xffffffffu, ie, o);
          if (lane >= o) { ig += a; ie += b; }
        }
        wsum[base + lane][0] = run_gt + ig - g0;
        wsum[base + lane][1] = run_eq + ie - e0;
        run_gt += __shfl_sync(0xffffffffu, ig, 31);
        run_eq += __shfl_sync(0xffffffffu, ie, 31);
      }
      if (lane == 0) { cnt[slot][0] = run_gt; cnt[slot][1] = run_eq; }
    }
    cluster.sync();
    before_gt = before_eq = 0;
    for (int r = 0; r < rank; ++r) {
      const unsigned* c = cluster.map_shared_rank(&cnt[slot][0], r);
      before_gt += c[0];
      before_eq += c[1];
    }
  };
  // is key (row i, this thread) among the first `need` keys equal to Tx or above Tx ?
  const unsigned lt = (1u << lane) - 1u;
  auto taken = [&](int i, unsigned Tx, unsigned need) __attribute__((always_inline)) {
    const unsigned eq_before = before_eq + wsum[i * kW + warp][1] + __popc(eq_mask[i] & lt);
    return key[i] > Tx || (key[i] == Tx && eq_before < need);
  };

  scan_threshold(T, 0);
  unsigned take_bits = 0;   // bit i: this thread's key of row i was selected
#pragma unroll
  for (int i = 0; i < ROWS; ++i) {
    const int t = rank * chunk + i * kT + tid;
    const unsigned gt_before = before_gt + wsum[i * kW + warp][0] + __popc(gt_mask[i] & lt);
    const unsigned eq_before = before_eq + wsum[i * kW + warp][1] + __popc(eq_mask[i] & lt);
    bool take = false;
    if (t < n_cand) {
      take = taken(i, T, need_eq);
      if (take) kept[gt_before + min(eq_before, need_eq)] = t;
    } else if (t < L) {
      take = true;  // observation-window rows are always kept
    }
    take_bits |= (take ? 1u : 0u) << i;
    const unsigned word = __ballot_sync(0xffffffffu, take);
    const int t0 = rank * chunk + i * kT + warp * 32;
    if (lane == 0 && t0 < L) bm[t0 >> 5] = word;
  }
  // the window rows close the kept list
  if (rank == 0)
    for (int j = tid; j < L - n_cand; j += kT) kept[k_sel + j] = n_cand + j;

  // 4. calibration size: the next n_calib candidates in the same order, i.e. those among the first
  // k_sel + n_calib that were not selected.  mask2: bit set = the row is NOT one of them.
  if (kSized) {
    uint32_t* bm2 = mask2 + (size_t)unit * bitmap_words;
    unsigned T2, need2;
    __syncthreads();   // wsum and the flags of step 3 have been read by every thread of this CTA
    radix_select((unsigned)(k_sel + n_calib), T2, need2);
    scan_threshold(T2, 1);
#pragma unroll
    for (int i = 0; i < ROWS; ++i) {
      const int t = rank * chunk + i * kT + tid;
      const bool member = t < n_cand && !((take_bits >> i) & 1u) && taken(i, T2, need2);
      const unsigned word = ~__ballot_sync(0xffffffffu, member);
      const int t0 = rank * chunk + i * kT + warp * 32;
      if (lane == 0 && t0 < L) bm2[t0 >> 5] = word;
    }
  }
  cluster.sync();  // no CTA leaves while another may still read its shared memory
}

template <int ROWS>
void launch_rows(const CompressGeom& g, const CompressWs& ws, char* wsp, const float* scores, size_t stride,
                 int32_t* kept_idx, cudaStream_t st) {
  // (the cluster shape is the kernel's own attribute; the launch adds programmatic serialisation)
  if (g.sized && g.n_calib > 0)
    launch_pdl(pool_select_cluster_kernel<ROWS, true>, dim3(kClu, g.units), dim3(kT), 0, st, scores,
               (float*)(wsp + ws.pooled), (uint32_t*)(wsp + ws.bitmap), kept_idx, g.n_cand, g.L, g.pool, g.k_sel, g.n_kept,
               g.bitmap_words, (uint32_t*)(wsp + ws.bitmap2), g.n_calib, stride);
  else
    launch_pdl(pool_select_cluster_kernel<ROWS, false>, dim3(kClu, g.units), dim3(kT), 0, st, scores,
               (float*)(wsp + ws.pooled), (uint32_t*)(wsp + ws.bitmap), kept_idx, g.n_cand, g.L, g.pool, g.k_sel, g.n_kept,
               g.bitmap_words, (uint32_t*)nullptr, 0, stride);
}

}  // namespace

// The cluster kernel keeps at most 32 keys per thread: 8 CTAs x 1024 threads x 32.
bool select_cluster_supported(const CompressGeom& g) { return !g.keep_all && g.L <= kClu * kT * 32; }

// Selection from per-candidate scores [units][stride] (the window votes of the workspace, or a
// caller's scores).
cudaError_t launch_pool_select_scores(const CompressGeom& g, const CompressWs& ws, char* wsp, const float* scores,
                                      size_t stride, int32_t* kept_idx, cudaStream_t st) {
  const int rows = (g.L + kClu * kT - 1) / (kClu * kT);
  if (rows <= 1) launch_rows<1>(g, ws, wsp, scores, stride, kept_idx, st);
  else if (rows <= 2) launch_rows<2>(g, ws, wsp, scores, stride, kept_idx, st);
  else if (rows <= 4) launch_rows<4>(g, ws, wsp, scores, stride, kept_idx, st);
  else if (rows <= 8) launch_rows<8>(g, ws, wsp, scores, stride, kept_idx, st);
  else if (rows <= 16) launch_rows<16>(g, ws, wsp, scores, stride, kept_idx, st);
  else launch_rows<32>(g, ws, wsp, scores, stride, kept_idx, st);
  count_launch(1);
  return cudaGetLastError();
}

cudaError_t launch_pool_select_cluster(const CompressGeom& g, const CompressWs& ws, char* wsp, int32_t* kept_idx,
                                       cudaStream_t st) {
  return launch_pool_select_scores(g, ws, wsp, (const float*)(wsp + ws.vote), (size_t)g.n_cand, kept_idx, st);
}

// Sink-plus-recent index rule: the first n_sink rows and the last n_kept - n_sink.
__global__ void streaming_indices_kernel(int32_t* __restrict__ kept_idx, int L, int n_kept, int n_sink) {
  const int unit = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_kept) kept_idx[(size_t)unit * n_kept + i] = i < n_sink ? i : L - (n_kept - i);
}

cudaError_t launch_streaming_indices(const CompressGeom& g, int n_sink, int32_t* kept_idx, cudaStream_t st) {
  streaming_indices_kernel<<<dim3((g.n_kept + 255) / 256, g.units), 256, 0, st>>>(kept_idx, g.L, g.n_kept, n_sink);
  count_launch(1);
  return cudaGetLastError();
}

}  // namespace calidrop
