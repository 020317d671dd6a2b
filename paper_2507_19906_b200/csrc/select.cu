// Pooling of the votes, per-(batch, kv-head) top-k selection with a deterministic
// lowest-index tie rule, and gather-compaction of the kept K/V rows.
//
// Selection is an exact radix select on the fp32 bit patterns of the pooled votes (they are
// non-negative, so unsigned order equals numeric order): four 8-bit histogram passes find the
// value T of the k-th largest candidate and how many candidates equal to T still fit; one
// ordered compaction pass then emits, in ascending position, every candidate above T plus the
// first `need_eq` candidates equal to T.  No sort is needed because ascending position is
// the storage order of the kept rows.
#include "common.cuh"
#include "internal.h"

namespace calidrop {

namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

__global__ void __launch_bounds__(kSelThreads)
pool_select_kernel(const float* __restrict__ vote, float* __restrict__ pooled,
                   uint32_t* __restrict__ bitmap, int32_t* __restrict__ kept_idx, int n_cand, int L,
                   int pool, int k_sel, int n_kept, int bitmap_words) {
  __shared__ unsigned hist[kSelWarps][256];
  __shared__ unsigned total[256];
  __shared__ unsigned sel_bin, sel_k;
  __shared__ unsigned warp_gt[kSelWarps], warp_eq[kSelWarps];

  const int unit = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* v = vote + (size_t)unit * n_cand;
  float* pl = pooled + (size_t)unit * n_cand;
  uint32_t* bm = bitmap + (size_t)unit * bitmap_words;
  int32_t* kept = kept_idx + (size_t)unit * n_kept;

  // 1. zero-padded average pool with a constant divisor
  const int half = pool >> 1;
  const float fpool = (float)pool;
  for (int t = tid; t < n_cand; t += kSelThreads) {
    float acc = 0.f;
    for (int d = -half; d <= half; ++d) {
      int u = t + d;
      if (u >= 0 && u < n_cand) acc += v[u];
    }
    pl[t] = acc / fpool;
  }
  __syncthreads();
  const uint32_t* keys = reinterpret_cast<const uint32_t*>(pl);

  // 2. radix select, most significant byte first
  unsigned prefix = 0, k = (unsigned)k_sel;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < kSelWarps * 256; i += kSelThreads) (&hist[0][0])[i] = 0;
    __syncthreads();
    for (int t = tid; t < n_cand; t += kSelThreads) {
      const unsigned key = keys[t];
      const bool in = (pass == 0) || ((key >> (shift + 8)) == prefix);
      if (in) atomicAdd(&hist[warp][(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 256) {
      unsigned s = 0;
#pragma unroll 8
      for (int w = 0; w < kSelWarps; ++w) s += hist[w][tid];
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
    __syncthreads();
  }
  const unsigned T = prefix;     // bit pattern of the k-th largest pooled vote
  const unsigned need_eq = k;    // how many candidates equal to T are taken (lowest positions)

  // 3. ordered compaction: thread i owns positions [i*per, (i+1)*per), per a multiple of 32
  int per = (L + kSelThreads - 1) / kSelThreads;
  per = (per + 31) & ~31;
  const int t_begin = tid * per;
  unsigned cnt_gt = 0, cnt_eq = 0;
  for (int i = 0; i < per; ++i) {
    const int t = t_begin + i;
    if (t < n_cand) {
      const unsigned key = keys[t];
      cnt_gt += key > T;
      cnt_eq += key == T;
    }
  }
  unsigned inc_gt = cnt_gt, inc_eq = cnt_eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned a = __shfl_up_sync(0xffffffffu, inc_gt, o);
    unsigned b = __shfl_up_sync(0xffffffffu, inc_eq, o);
    if (lane >= o) { inc_gt += a; inc_eq += b; }
  }
  if (lane == 31) { warp_gt[warp] = inc_gt; warp_eq[warp] = inc_eq; }
  __syncthreads();
  unsigned before_gt = inc_gt - cnt_gt, before_eq = inc_eq - cnt_eq;
  for (int w = 0; w < warp; ++w) { before_gt += warp_gt[w]; before_eq += warp_eq[w]; }

  unsigned pos = before_gt + min(before_eq, need_eq);
  unsigned eq_seen = before_eq;
  for (int i0 = 0; i0 < per; i0 += 32) {
    const int tw = t_begin + i0;
    if (tw >= L) break;
    uint32_t word = 0;
    for (int i = 0; i < 32; ++i) {
      const int t = tw + i;
      bool take = false;
      if (t < n_cand) {
        const unsigned key = keys[t];
        if (key > T) {
          take = true;
        } else if (key == T) {
          take = eq_seen < need_eq;
          ++eq_seen;
        }
        if (take) kept[pos++] = t;
      } else if (t < L) {
        take = true;  // observation-window rows are always kept
      }
      word |= (take ? 1u : 0u) << i;
    }
    bm[tw >> 5] = word;
  }
  // the window rows close the kept list
  for (int j = tid; j < L - n_cand; j += kSelThreads) kept[k_sel + j] = n_cand + j;
}

// budget >= L: every row is kept.
__global__ void keep_all_kernel(uint32_t* __restrict__ bitmap, int32_t* __restrict__ kept_idx, int L,
                                int bitmap_words) {
  const int unit = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < L) kept_idx[(size_t)unit * L + t] = t;
  if (t < bitmap_words) bitmap[(size_t)unit * bitmap_words + t] = 0xffffffffu;
}

// Kept bitmap of a caller-supplied kept list: the listed rows plus the observation-window rows
// [n_cand, L), which count as kept whatever the list says.  The bitmap is zeroed beforehand.
__global__ void bitmap_from_indices_kernel(const int32_t* __restrict__ kept_idx, uint32_t* __restrict__ bitmap,
                                           int n_kept, int n_cand, int L, int bitmap_words) {
  const int unit = blockIdx.y;
  const int32_t* kept = kept_idx + (size_t)unit * n_kept;
  uint32_t* bm = bitmap + (size_t)unit * bitmap_words;
  const int n = n_kept + (L - n_cand);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int t = i < n_kept ? kept[i] : n_cand + (i - n_kept);
    if (t >= 0 && t < L) atomicOr(&bm[t >> 5], 1u << (t & 31));
  }
}

// K_kept[u, i, :] = K[u, kept_idx[u, i], :], same for V; 16 lanes x 16 bytes per row.
__global__ void __launch_bounds__(256) gather_kernel(const GatherArgs a) {
  gather_rows16(a, blockIdx.x, blockIdx.y, threadIdx.x);
}

}  // namespace

cudaError_t launch_pool_select(const CompressGeom& g, const CompressWs& ws, char* wsp,
                               int32_t* kept_idx, cudaStream_t st) {
  if (g.keep_all) {
    const int n = g.L > g.bitmap_words ? g.L : g.bitmap_words;
    dim3 grid((n + 255) / 256, g.units);
    keep_all_kernel<<<grid, 256, 0, st>>>((uint32_t*)(wsp + ws.bitmap), kept_idx, g.L, g.bitmap_words);
  } else {
    pool_select_kernel<<<g.units, kSelThreads, 0, st>>>(
        (const float*)(wsp + ws.vote), (float*)(wsp + ws.pooled), (uint32_t*)(wsp + ws.bitmap), kept_idx,
        g.n_cand, g.L, g.pool, g.k_sel, g.n_kept, g.bitmap_words);
  }
  count_launch(1);
  return cudaGetLastError();
}

// Ascending list of the evicted candidates of a unit: the zero bits of its kept bitmap below n_cand.
// One CTA per unit; thread i owns a contiguous run of bitmap words, so a block-wide exclusive scan of
// the per-thread counts gives every thread the position of its first index.
__global__ void __launch_bounds__(kSelThreads)
evicted_indices_kernel(const uint32_t* __restrict__ bitmap, int32_t* __restrict__ evict_idx, int n_cand, int n_evict,
                       int bitmap_words) {
  __shared__ unsigned warp_sum[kSelThreads / 32];
  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t* bm = bitmap + (size_t)unit * bitmap_words;
  int32_t* out = evict_idx + (size_t)unit * n_evict;
  const int n_words = (n_cand + 31) >> 5;
  const int wpt = (n_words + kSelThreads - 1) / kSelThreads;
  const int w0 = tid * wpt, w1 = min(n_words, w0 + wpt);
  auto zeros_of = [&](int w) {
    uint32_t z = ~bm[w];
    const int rem = n_cand - (w << 5);
    if (rem < 32) z &= (1u << rem) - 1u;
    return z;
  };
  // entries that no zero bit fills (a kept list with fewer candidates than expected leaves fewer
  // evicted rows than n_evict) hold -1, which the gather skips
  for (int i = tid; i < n_evict; i += kSelThreads) out[i] = -1;
  __syncthreads();
  unsigned cnt = 0;
  for (int w = w0; w < w1; ++w) cnt += __popc(zeros_of(w));
  unsigned incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    unsigned v = lane < kSelThreads / 32 ? warp_sum[lane] : 0u, iv = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned n = __shfl_up_sync(0xffffffffu, iv, o);
      if (lane >= o) iv += n;
    }
    if (lane < kSelThreads / 32) warp_sum[lane] = iv - v;
  }
  __syncthreads();
  unsigned pos = warp_sum[warp] + incl - cnt;
  for (int w = w0; w < w1; ++w) {
    uint32_t z = zeros_of(w);
    while (z) {
      const int b = __ffs(z) - 1;
      z &= z - 1;
      if (pos < (unsigned)n_evict) out[pos] = (w << 5) + b;
      ++pos;
    }
  }
}

cudaError_t launch_evicted_indices(const CompressGeom& g, const CompressWs& ws, char* wsp, int32_t* evict_idx,
                                   cudaStream_t st) {
  // the zero bits below n_cand of the kept bitmap, or of the calibration mask when the calibration is sized
  evicted_indices_kernel<<<g.units, kSelThreads, 0, st>>>((const uint32_t*)(wsp + ws.calib_mask), evict_idx, g.n_cand,
                                                          g.n_calib, g.bitmap_words);
  count_launch(1);
  return cudaGetLastError();
}

// No calibrated rows: zeros, -inf and the calibration queries.  One warp per (b, hq, c).
__global__ void __launch_bounds__(128)
calib_none_kernel(const __nv_bfloat16* __restrict__ Q_obs, float* __restrict__ O_c, float* __restrict__ LSE_c,
                  __nv_bfloat16* __restrict__ C_q, int rows, int W, int n_cal) {
  const int lane = threadIdx.x & 31, row = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int c = row % n_cal, bhq = row / n_cal;
  reinterpret_cast<float4*>(O_c + (size_t)row * kD)[lane] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (lane == 0) LSE_c[row] = -INFINITY;
  reinterpret_cast<uint2*>(C_q + (size_t)row * kD)[lane] =
      reinterpret_cast<const uint2*>(Q_obs + ((size_t)bhq * W + (W - n_cal + c)) * kD)[lane];
}

cudaError_t launch_calib_none(const CompressGeom& g, const void* Q_obs, float* O_c, float* LSE_c, void* C_q,
                              cudaStream_t st) {
  const int rows = g.B * g.Hq * g.n_cal;
  calib_none_kernel<<<(rows + 3) / 4, 128, 0, st>>>((const __nv_bfloat16*)Q_obs, O_c, LSE_c, (__nv_bfloat16*)C_q, rows,
                                                   g.W, g.n_cal);
  count_launch(1);
  return cudaGetLastError();
}

cudaError_t launch_bitmap_from_indices(const CompressGeom& g, const CompressWs& ws, char* wsp,
                                       const int32_t* kept_idx, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(wsp + ws.bitmap, 0, (size_t)g.units * g.bitmap_words * 4, st);
  if (e != cudaSuccess) return e;
  const int n = g.n_kept + (g.L - g.n_cand);
  int blocks = (n + 255) / 256;
  if (blocks > 64) blocks = 64;
  bitmap_from_indices_kernel<<<dim3(blocks, g.units), 256, 0, st>>>(kept_idx, (uint32_t*)(wsp + ws.bitmap), g.n_kept,
                                                                    g.n_cand, g.L, g.bitmap_words);
  count_launch(1);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const CompressGeom& g, const void* K, const void* V, const int32_t* idx, int n_rows,
                               int out_rows, void* K_out, void* V_out, cudaStream_t st) {
  dim3 grid((n_rows + 15) / 16, g.units);
  const GatherArgs a{(const uint4*)K, (const uint4*)V, idx, (uint4*)K_out, (uint4*)V_out, g.L, n_rows, out_rows, g.units};
  gather_kernel<<<grid, 256, 0, st>>>(a);
  count_launch(1);
  return cudaGetLastError();
}

cudaError_t launch_gather(const CompressGeom& g, const void* K, const void* V, const int32_t* kept_idx,
                          void* K_kept, void* V_kept, cudaStream_t st) {
  return launch_gather_rows(g, K, V, kept_idx, g.n_kept, g.cap, K_kept, V_kept, st);
}

}  // namespace calidrop
