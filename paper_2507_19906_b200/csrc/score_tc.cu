// Window scoring on the tensor cores (tcgen05 MMA, accumulator in TMEM, operands fed by TMA).
//
// Two kernels over one skeleton.  A CTA owns one (batch, kv-head) unit and a contiguous range of
// 128-key tiles; the unit's G*W observation rows stay resident in shared memory, the key tiles
// stream through a TMA ring.  Warp roles: warps 0-3 read the accumulator out of TMEM (one TMEM
// lane per thread), warp 4 is the TMA producer, warp 5 allocates TMEM and issues the MMAs.
//
//   statistics (kVotes = false):  S = Q K^T, query rows on the TMEM lanes.  Thread r keeps the
//       running (max, sum) of exp2(scale2 * s) over the keys row r may see (causal inside the
//       window).  Per-split partials are combined into the natural-log row LSE by
//       row_lse_reduce_kernel.  Skipped altogether when the caller supplies the row LSE.
//   votes (kVotes = true):  S^T = K Q^T, KEYS on the TMEM lanes, so the vote of a key,
//       sum over rows of exp2(scale2 * s - lse2[row]), is a per-thread sum over the accumulator's
//       columns: no cross-thread reduction and fp32 probabilities throughout.  Candidate keys
//       (t < L - W) are seen by every window row, so this pass needs no mask.
//
// Both passes are co-limited by the tensor pipe and the exponential unit (one exp2 per logit).
#include "internal.h"
#include "tc_common.cuh"

namespace calidrop {

namespace {

using namespace tc;

constexpr int kThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kMaxRows = 512;  // G * W handled by the tiles

struct ScoreArgs {
  int Hq, G, W, L, n_cand, GW;
  int n_blocks;    // blocks of observation rows
  int block_rows;  // rows per block: 128 for the statistics, a multiple of 32 (<= 256) for the votes
  int n_tiles;     // key tiles to cover
  int n_splits;
  int stages;      // depth of the key-tile ring (2 or 3)
  float scale2;
  const float* row_lse;  // votes: natural-log LSE of every observation row [B, Hq, W]
  float* vote;           // votes: out [units, n_cand]
  float2* stat_part;     // statistics: out [row][split] (max, sum) in the log2 domain
  unsigned* status;
};

template <bool kVotes>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                const ScoreArgs a) {
  constexpr int NBUF = kVotes ? 2 : 4;        // accumulator ring in TMEM
  constexpr int BUFCOLS = kVotes ? 256 : 128;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[16];
  __shared__ uint32_t tmem_slot;
  __shared__ Ctl ctl;
  __shared__ __align__(16) float nlse2_s[kVotes ? kMaxRows : 4];          // -log2-domain LSE per row (-inf: padding)
  __shared__ float2 ml_s[kVotes ? 1 : 4][kVotes ? 1 : 128];  // running (max, sum) per row block

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, unit = blockIdx.y;
  const int tile0 = (int)((long long)a.n_tiles * split / a.n_splits);
  const int tile1 = (int)((long long)a.n_tiles * (split + 1) / a.n_splits);
  const int nt = tile1 - tile0;
  const int n_jobs = nt * a.n_blocks;  // one job = one (key tile, row block) accumulator

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_half_bytes = (uint32_t)a.block_rows * kLineBytes;
  const uint32_t q_blk_bytes = 2u * q_half_bytes;
  const uint32_t q_base = smem_base;
  const uint32_t k_base = q_base + (uint32_t)a.n_blocks * q_blk_bytes;

  const uint32_t bar0 = smem_u32(bars);
  const uint32_t q_full = bar0;
  auto full_k = [&](int s) { return bar0 + 8u * (1 + s); };
  auto empty_k = [&](int s) { return bar0 + 8u * (4 + s); };
  auto t_full = [&](int b) { return bar0 + 8u * (7 + b); };
  auto t_empty = [&](int b) { return bar0 + 8u * (11 + b); };

  if (tid == 0) {
    ctl.abort = 0;
    ctl.status = a.status;
    mbar_init(q_full, 1);
    for (int s = 0; s < 3; ++s) { mbar_init(full_k(s), 1); mbar_init(empty_k(s), 1); }
    for (int b = 0; b < 4; ++b) { mbar_init(t_full(b), 1); mbar_init(t_empty(b), 128); }
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  const int hq0 = (unit / (a.Hq / a.G)) * a.Hq + (unit % (a.Hq / a.G)) * a.G;  // first query head of the unit
  if (kVotes) {
    for (int r = tid; r < kMaxRows; r += kThreads)
      nlse2_s[r] = r < a.GW ? -a.row_lse[(size_t)hq0 * a.W + r] * kLog2e : -INFINITY;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&q_map);
      tma_prefetch_desc(&k_map);
      mbar_arrive_expect_tx(q_full, (uint32_t)a.n_blocks * q_blk_bytes);
      for (int blk = 0; blk < a.n_blocks; ++blk)
        for (int half = 0; half < 2; ++half)
          tma_load_3d(q_base + blk * q_blk_bytes + half * q_half_bytes, &q_map, q_full, half * kHalfCols,
                      blk * a.block_rows, unit);
      for (int i = 0; i < nt; ++i) {
        const int s = i % a.stages;
        if (!mbar_wait(&ctl, empty_k(s), ((i / a.stages) & 1) ^ 1, 11u)) break;
        mbar_arrive_expect_tx(full_k(s), kKvTileBytes);
        for (int half = 0; half < 2; ++half)
          tma_load_3d(k_base + s * kKvTileBytes + half * (kKvTileBytes / 2), &k_map, full_k(s), half * kHalfCols,
                      (tile0 + i) * kTileKeys, unit);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(128, kVotes ? a.block_rows : 128, false, false);
      bool ok = mbar_wait(&ctl, q_full, 0, 12u);
      for (int j = 0; ok && j < n_jobs; ++j) {
        const int i = j / a.n_blocks, blk = j - i * a.n_blocks;
        const int s = i % a.stages, buf = j % NBUF;
        if (blk == 0 && !mbar_wait(&ctl, full_k(s), (i / a.stages) & 1, 13u)) break;
        if (!mbar_wait(&ctl, t_empty(buf), ((j / NBUF) & 1) ^ 1, 14u)) break;
        tc_fence_after_sync();
        const uint32_t d = tmem_base + (uint32_t)(buf * BUFCOLS);
        const uint32_t kt = k_base + (uint32_t)s * kKvTileBytes, qt = q_base + (uint32_t)blk * q_blk_bytes;
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint64_t kd = kmajor_desc(kt, kKvTileBytes / 2, kk);
          const uint64_t qd = kmajor_desc(qt, q_half_bytes, kk);
          umma_ss(d, kVotes ? kd : qd, kVotes ? qd : kd, idesc, kk > 0 ? 1u : 0u);
        }
        umma_commit(t_full(buf));
        if (blk == a.n_blocks - 1) umma_commit(empty_k(s));
      }
    }
  } else {
    // ------------------------------------------------------------ accumulator consumers
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
    float acc = 0.f;  // votes: running vote of this thread's key
    if (!kVotes) {
      for (int blk = 0; blk < 4; ++blk) ml_s[blk][tid] = make_float2(-INFINITY, 0.f);
    }
    for (int j = 0; j < n_jobs; ++j) {
      const int i = j / a.n_blocks, blk = j - i * a.n_blocks;
      const int buf = j % NBUF;
      bool ok = mbar_wait(&ctl, t_full(buf), (j / NBUF) & 1, 15u);
      if (!__all_sync(0xffffffffu, ok)) break;
      tc_fence_after_sync();
      const int tbase = (tile0 + i) * kTileKeys;
      const uint32_t taddr = lane_addr + (uint32_t)(buf * BUFCOLS);
      uint32_t r[32];
      if (kVotes) {
        const float* nl = nlse2_s + blk * a.block_rows;
        for (int c0 = 0; c0 < a.block_rows; c0 += 32) {
          tmem_ld32(taddr + c0, r);
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            const float4 n4 = *reinterpret_cast<const float4*>(nl + c0 + e);
            acc += ex2_approx(fmaf(__uint_as_float(r[e + 0]), a.scale2, n4.x));
            acc += ex2_approx(fmaf(__uint_as_float(r[e + 1]), a.scale2, n4.y));
            acc += ex2_approx(fmaf(__uint_as_float(r[e + 2]), a.scale2, n4.z));
            acc += ex2_approx(fmaf(__uint_as_float(r[e + 3]), a.scale2, n4.w));
          }
        }
        tc_fence_before_sync();
        mbar_arrive(t_empty(buf));
        if (blk == a.n_blocks - 1) {
          const int key = tbase + tid;
          if (key < a.n_cand) a.vote[(size_t)unit * a.n_cand + key] = acc;
          acc = 0.f;
        }
      } else {
        float2 ml = ml_s[blk][tid];
        const int row = blk * 128 + tid;
        // local index of the last key this row may see inside the tile (causal inside the window)
        const int lim = min(a.L - 1, a.n_cand + row % a.W) - tbase;
        const bool full_tile = __all_sync(0xffffffffu, lim >= kTileKeys - 1);
#pragma unroll 1
        for (int c0 = 0; c0 < kTileKeys; c0 += 32) {
          tmem_ld32(taddr + c0, r);
          float cmax = -INFINITY;
          if (full_tile) {
#pragma unroll
            for (int e = 0; e < 32; ++e) cmax = fmaxf(cmax, __uint_as_float(r[e]));
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              if (c0 + e > lim) r[e] = 0xff800000u;  // -inf
              cmax = fmaxf(cmax, __uint_as_float(r[e]));
            }
          }
          const float m_new = fmaxf(ml.x, cmax * a.scale2);
          if (m_new > -INFINITY) {
            float sum = 0.f;
#pragma unroll
            for (int e = 0; e < 32; ++e) sum += ex2_approx(fmaf(__uint_as_float(r[e]), a.scale2, -m_new));
            ml.y = ml.y * ex2_approx(ml.x - m_new) + sum;
            ml.x = m_new;
          }
        }
        tc_fence_before_sync();
        mbar_arrive(t_empty(buf));
        ml_s[blk][tid] = ml;
      }
    }
    if (!kVotes && !ctl.abort) {
      for (int blk = 0; blk < a.n_blocks; ++blk) {
        const int row = blk * 128 + tid;
        if (row < a.GW) a.stat_part[((size_t)hq0 * a.W + row) * a.n_splits + split] = ml_s[blk][tid];
      }
    }
  }

  // ---------------------------------------------------------------- teardown (every path)
  if (ctl.abort) {
    for (int i = 0; i < 50; ++i) __nanosleep(20000);  // let TMA copies still in flight land
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem_base, kTmemCols);
}

// Combine the per-split statistics of every observation row into its natural-log LSE.
__global__ void row_lse_from_splits_kernel(const float2* __restrict__ stat_part, float* __restrict__ row_lse,
                                           int rows, int n_splits) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const float2* p = stat_part + (size_t)r * n_splits;
  float m = -INFINITY;
  for (int i = 0; i < n_splits; ++i) m = fmaxf(m, p[i].x);
  float l = 0.f;
  for (int i = 0; i < n_splits; ++i)
    if (p[i].x > -INFINITY) l += p[i].y * exp2f(p[i].x - m);
  row_lse[r] = (m + log2f(l)) * kLn2;
}

template <bool kVotes>
cudaError_t set_smem_limit(int bytes) {
  static int granted[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && granted[dev] >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(score_tc_kernel<kVotes>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && dev >= 0 && dev < 64) granted[dev] = bytes;
  return e;
}

}  // namespace

// Number of key-range splits per work group so that `groups * splits` CTAs fill whole waves of
// the 148 SMs (one CTA per SM) while every CTA keeps at least `min_tiles` tiles.
int pick_tile_splits(int groups, int n_tiles, int min_tiles) {
  const int kSms = 148;
  int max_s = n_tiles / (min_tiles > 0 ? min_tiles : 1);
  if (max_s < 1) max_s = 1;
  if (max_s > 64) max_s = 64;
  int best = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= max_s; ++s) {
    const long long ctas = (long long)groups * s;
    const long long waves = (ctas + kSms - 1) / kSms;
    const double eff = (double)ctas / (double)(waves * kSms);
    if (eff > best_eff + 0.02) { best_eff = eff; best = s; }
  }
  return best;
}

bool score_tc_supported(const CompressGeom& g) {
  return !g.keep_all && g.G * g.W <= kMaxRows && g.W <= 128 && g.n_cand >= 1;
}

// Statistics (row LSE) of the G*W observation rows of every unit, into ws.row_lse.
cudaError_t launch_row_stats_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                                char* wsp, cudaStream_t st) {
  const int GW = g.G * g.W;
  ScoreArgs a{};
  a.Hq = g.Hq; a.G = g.G; a.W = g.W; a.L = g.L; a.n_cand = g.n_cand; a.GW = GW;
  a.n_blocks = (GW + 127) / 128;
  a.block_rows = 128;
  a.n_tiles = (g.L + kTileKeys - 1) / kTileKeys;
  a.n_splits = pick_tile_splits(g.units, a.n_tiles, 4);
  if (a.n_splits > ws.n_tiles) a.n_splits = ws.n_tiles;
  a.stages = a.n_blocks <= 3 ? 3 : 2;
  a.scale2 = g.scale2;
  a.stat_part = (float2*)(wsp + ws.stat_part);
  a.status = (unsigned*)(wsp + ws.status);
  CUtensorMap qm, km;
  const uint64_t qd[2] = {(uint64_t)GW, (uint64_t)g.units}, qs[2] = {256, (uint64_t)GW * 256};
  const uint32_t qb[2] = {128, 1};
  const uint64_t kd[2] = {(uint64_t)g.L, (uint64_t)g.units}, ks[2] = {256, (uint64_t)g.L * 256};
  const uint32_t kb[2] = {(uint32_t)kTileKeys, 1};
  if (!make_tensor_map_bf16(&qm, Q_obs, 3, qd, qs, qb) || !make_tensor_map_bf16(&km, K, 3, kd, ks, kb))
    return cudaErrorInvalidValue;
  const int smem = a.n_blocks * 128 * 256 + a.stages * kKvTileBytes + 1024;
  cudaError_t e = set_smem_limit<false>(smem);
  if (e != cudaSuccess) return e;
  score_tc_kernel<false><<<dim3(a.n_splits, g.units), kThreads, smem, st>>>(qm, km, a);
  const int rows = g.B * g.Hq * g.W;
  row_lse_from_splits_kernel<<<(rows + 127) / 128, 128, 0, st>>>(a.stat_part, (float*)(wsp + ws.row_lse), rows,
                                                                 a.n_splits);
  count_launch(2);
  return cudaGetLastError();
}

// Votes of every candidate key, into ws.vote.
cudaError_t launch_votes_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                            const float* row_lse, char* wsp, cudaStream_t st) {
  const int GW = g.G * g.W;
  ScoreArgs a{};
  a.Hq = g.Hq; a.G = g.G; a.W = g.W; a.L = g.L; a.n_cand = g.n_cand; a.GW = GW;
  a.n_blocks = (GW + 255) / 256;
  a.block_rows = ((GW + a.n_blocks - 1) / a.n_blocks + 31) / 32 * 32;
  a.n_tiles = (g.n_cand + kTileKeys - 1) / kTileKeys;
  a.n_splits = pick_tile_splits(g.units, a.n_tiles, 4);
  a.stages = 3;
  a.scale2 = g.scale2;
  a.row_lse = row_lse;
  a.vote = (float*)(wsp + ws.vote);
  a.status = (unsigned*)(wsp + ws.status);
  CUtensorMap qm, km;
  const uint64_t qd[2] = {(uint64_t)GW, (uint64_t)g.units}, qs[2] = {256, (uint64_t)GW * 256};
  const uint32_t qb[2] = {(uint32_t)a.block_rows, 1};
  const uint64_t kd[2] = {(uint64_t)g.L, (uint64_t)g.units}, ks[2] = {256, (uint64_t)g.L * 256};
  const uint32_t kb[2] = {(uint32_t)kTileKeys, 1};
  if (!make_tensor_map_bf16(&qm, Q_obs, 3, qd, qs, qb) || !make_tensor_map_bf16(&km, K, 3, kd, ks, kb))
    return cudaErrorInvalidValue;
  const int smem = a.n_blocks * a.block_rows * 256 + a.stages * kKvTileBytes + 1024;
  cudaError_t e = set_smem_limit<true>(smem);
  if (e != cudaSuccess) return e;
  score_tc_kernel<true><<<dim3(a.n_splits, g.units), kThreads, smem, st>>>(qm, km, a);
  count_launch(1);
  return cudaGetLastError();
}

}  // namespace calidrop
