// Window scoring on the tensor cores (tcgen05 MMA, accumulator in TMEM, operands fed by TMA).
//
// Two kernels over one skeleton.  The work is the linear space of (virtual unit, key tile) pairs;
// it is cut into equal contiguous ranges, one per CTA, and at most one CTA per SM is launched, so
// a CTA streams a long run of key tiles through its TMA ring and pays its start-up once.  A
// virtual unit is a (batch, kv-head) unit, or for the statistics one half of its window rows when
// there are more than 256; its query rows stay resident in shared memory and are reloaded when
// the CTA's range crosses into the next virtual unit.
// Warp roles: four consumer warpgroups in two pairs read the accumulators out of TMEM (one TMEM
// lane per thread; pair p drains accumulator buffer p, each of its groups half of the columns), one
// warp is the TMA producer, one warp allocates TMEM and issues the MMAs.  Every MMA has N = 256 where the shape allows it: with both operands in
// shared memory, narrower tiles are limited by operand fetch, not by the tensor pipe.
//
//   statistics (kVotes = false):  S = Q K^T, 128 query rows on the TMEM lanes, 256 keys per tile.
//       Thread r keeps the running (max, sum) of exp2(scale2 * s) over the keys row r may see
//       (causal inside the window).  Per-CTA partials are combined into the natural-log row LSE by
//       row_lse_from_parts_kernel.  Skipped altogether when the caller supplies the row LSE.
//   votes (kVotes = true):  S^T = K Q^T, 128 KEYS on the TMEM lanes and up to 256 query rows as
//       columns, so the vote of a key, sum over rows of exp2(scale2 * s - lse2[row]), is a
//       per-thread sum over the accumulator's columns: no cross-thread reduction and fp32
//       probabilities throughout.  Candidate keys (t < L - W) are seen by every window row, so this
//       pass needs no mask.
#include "internal.h"
#include "tc_common.cuh"

namespace calidrop {

namespace {

using namespace tc;

constexpr int kGroups = 4;  // consumer warpgroups (4 warps each), two pairs; pair p drains accumulator buffer p
constexpr int kProducerWarp = kGroups * 4;
constexpr int kMmaWarp = kGroups * 4 + 1;
constexpr int kThreads = kGroups * 128 + 64;
constexpr int kTmemCols = 512;  // two accumulators of 256 columns
constexpr int kBufCols = 256;
constexpr int kNumBufs = 2;
constexpr int kMaxRows = 512;   // G * W handled by the tiles
constexpr int kSms = 148;

struct ScoreArgs {
  int Hq, G, W, L, n_cand, GW;
  int vu_per_unit;    // virtual units per (batch, kv-head) unit
  int vu_rows;        // window rows a virtual unit starts at: vu % vu_per_unit * vu_rows
  int n_blocks;       // row blocks (= accumulators) per key tile
  int block_rows;     // rows per block: 128 for the statistics, a multiple of 64 (<= 256) for the votes
  int n_tiles;        // key tiles per virtual unit
  int total_tiles;    // virtual units * n_tiles
  int tiles_per_cta;
  int stages;         // depth of the key-tile ring
  int max_slots;      // statistics: partial slots per row (CTAs that can share a virtual unit)
  float scale2;
  const float* row_lse;  // votes: natural-log LSE of every observation row [B, Hq, W]
  float* vote;           // votes: out [units, n_cand]
  float* vote2;          // with several row blocks per tile: the partial votes of warpgroup 1 (added to vote afterwards)
  float2* stat_part;     // statistics: out [row][slot][group] (max, sum) in the log2 domain
  unsigned* status;
};

// exp2 of 32 logits against one reference, four independent partial sums
__device__ __forceinline__ float sum_exp2_32(const uint32_t (&r)[32], float scale2, float neg_ref) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int e = 0; e < 32; e += 4) {
    s0 += ex2_approx(fmaf(__uint_as_float(r[e + 0]), scale2, neg_ref));
    s1 += ex2_approx(fmaf(__uint_as_float(r[e + 1]), scale2, neg_ref));
    s2 += ex2_approx(fmaf(__uint_as_float(r[e + 2]), scale2, neg_ref));
    s3 += ex2_approx(fmaf(__uint_as_float(r[e + 3]), scale2, neg_ref));
  }
  return (s0 + s1) + (s2 + s3);
}

__device__ __forceinline__ float max_32(const uint32_t (&r)[32]) {
  float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
  for (int e = 0; e < 32; e += 4) {
    m0 = fmaxf(m0, __uint_as_float(r[e + 0]));
    m1 = fmaxf(m1, __uint_as_float(r[e + 1]));
    m2 = fmaxf(m2, __uint_as_float(r[e + 2]));
    m3 = fmaxf(m3, __uint_as_float(r[e + 3]));
  }
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}


template <bool kVotes>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                const ScoreArgs a) {
  constexpr int TILE_KEYS = kVotes ? 128 : 256;
  constexpr uint32_t STAGE_BYTES = TILE_KEYS * 256;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[22];
  __shared__ uint32_t tmem_slot;
  __shared__ Ctl ctl;
  // votes: -lse2 of the columns this warp reads (128 per row block at most), one copy per warp
  __shared__ __align__(16) float nlse2_s[kVotes ? kGroups * 4 : 1][kVotes ? 256 : 4];
  __shared__ float vx[2][128];  // votes: partial vote of the second column half, per pair
  __shared__ float2 ml_s[kVotes ? 1 : kGroups][kVotes ? 1 : 2][kVotes ? 1 : 128];       // running (max, sum)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x;
  const int g_begin = cta * a.tiles_per_cta;
  const int g_end = min(a.total_tiles, g_begin + a.tiles_per_cta);
  const int nt = g_end - g_begin;
  const int Hkv = a.Hq / a.G;
  // (the position inside the tile space is tracked incrementally: no division per tile)
  const int vu_begin = g_begin / a.n_tiles, tile_begin = g_begin - vu_begin * a.n_tiles;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_half_bytes = (uint32_t)a.block_rows * kLineBytes;
  const uint32_t q_blk_bytes = 2u * q_half_bytes;
  const uint32_t q_base = smem_base;
  const uint32_t k_base = q_base + (uint32_t)a.n_blocks * q_blk_bytes;

  const uint32_t bar0 = smem_u32(bars);
  const uint32_t q_full = bar0, q_empty = bar0 + 8u;
  auto full_k = [&](int s) { return bar0 + 8u * (2 + s); };
  auto empty_k = [&](int s) { return bar0 + 8u * (6 + s); };
  auto t_full = [&](int b) { return bar0 + 8u * (10 + b); };
  auto t_empty = [&](int b) { return bar0 + 8u * (14 + b); };
  auto vx_full = [&](int b) { return bar0 + 8u * (18 + b); };
  auto vx_empty = [&](int b) { return bar0 + 8u * (20 + b); };

  if (tid == 0) {
    ctl.abort = 0;
    ctl.status = a.status;
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    for (int s = 0; s < 4; ++s) { mbar_init(full_k(s), 1); mbar_init(empty_k(s), 1); }
    for (int b = 0; b < kNumBufs; ++b) {
      mbar_init(t_full(b), 1); mbar_init(t_empty(b), 256);   // a buffer is drained by one pair of warpgroups
      mbar_init(vx_full(b), 128); mbar_init(vx_empty(b), 128);
    }
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  pdl_wait();   // everything above ran beside the previous kernel's end; global memory from here on

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&q_map);
      tma_prefetch_desc(&k_map);
      int cur_vu = -1, seg = 0, vu = vu_begin, tile = tile_begin, unit = vu_begin / a.vu_per_unit;
      for (int i = 0; i < nt; ++i, ++tile) {
        if (tile == a.n_tiles) { tile = 0; ++vu; unit = vu / a.vu_per_unit; }
        if (vu != cur_vu) {
          // the query rows of the next virtual unit replace the current ones once its MMAs are done
          if (seg > 0 && !mbar_wait(&ctl, q_empty, (seg - 1) & 1, (kVotes ? 36u : 16u) | ((unsigned)i << 8))) break;
          const int row0 = (vu - unit * a.vu_per_unit) * a.vu_rows;
          mbar_arrive_expect_tx(q_full, (uint32_t)a.n_blocks * q_blk_bytes);
          for (int blk = 0; blk < a.n_blocks; ++blk)
            for (int half = 0; half < 2; ++half)
              tma_load_3d(q_base + blk * q_blk_bytes + half * q_half_bytes, &q_map, q_full, half * kHalfCols,
                          row0 + blk * a.block_rows, unit);
          cur_vu = vu;
          ++seg;
        }
        const int s = i % a.stages;
        if (!mbar_wait(&ctl, empty_k(s), ((i / a.stages) & 1) ^ 1, (kVotes ? 31u : 11u) | ((unsigned)i << 8))) break;
        mbar_arrive_expect_tx(full_k(s), STAGE_BYTES);
        for (int half = 0; half < 2; ++half)
          tma_load_3d(k_base + s * STAGE_BYTES + half * (STAGE_BYTES / 2), &k_map, full_k(s), half * kHalfCols,
                      tile * TILE_KEYS, unit);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(128, kVotes ? a.block_rows : TILE_KEYS, false, false);
      // Descriptors are built once per buffer; a k-step adds a constant to the address field (the
      // issuing thread's own instructions between two MMAs are what limits the issue rate).
      const uint64_t dq0 = smem_desc_sw128(q_base, 16u, 1024u);
      const uint64_t dk0 = smem_desc_sw128(k_base, 16u, 1024u);
      int cur_vu = -1, seg = 0, j = 0, vu = vu_begin, tile = tile_begin;
      for (int i = 0; i < nt; ++i, ++tile) {
        if (tile == a.n_tiles) { tile = 0; ++vu; }
        if (vu != cur_vu) {
          if (!mbar_wait(&ctl, q_full, seg & 1, (kVotes ? 32u : 12u) | ((unsigned)i << 8))) break;
          cur_vu = vu;
          ++seg;
        }
        const int s = i % a.stages;
        if (!mbar_wait(&ctl, full_k(s), (i / a.stages) & 1, (kVotes ? 33u : 13u) | ((unsigned)i << 8))) break;
        bool ok = true;
        const uint64_t kd = desc_advance(dk0, (uint32_t)s * STAGE_BYTES);
        for (int blk = 0; blk < a.n_blocks; ++blk, ++j) {
          const int buf = j & (kNumBufs - 1);
          if (!mbar_wait(&ctl, t_empty(buf), ((j / kNumBufs) & 1) ^ 1, (kVotes ? 34u : 14u) | ((unsigned)j << 8))) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t d = tmem_base + (uint32_t)(buf * kBufCols);
          const uint64_t qd = desc_advance(dq0, (uint32_t)blk * q_blk_bytes);
          // the second halves (k-steps 4..7) start half a tile further on
          const uint64_t kd2 = desc_advance(kd, STAGE_BYTES / 2), qd2 = desc_advance(qd, q_half_bytes);
          umma_ss_imm<0>(d, kVotes ? kd : qd, kVotes ? qd : kd, idesc);
#pragma unroll
          for (int kk = 1; kk < 4; ++kk)
            umma_ss_imm<1>(d, desc_advance(kVotes ? kd : qd, kk * 32u), desc_advance(kVotes ? qd : kd, kk * 32u), idesc);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma_ss_imm<1>(d, desc_advance(kVotes ? kd2 : qd2, kk * 32u), desc_advance(kVotes ? qd2 : kd2, kk * 32u), idesc);
          umma_commit(t_full(buf));
        }
        if (!ok) break;
        umma_commit(empty_k(s));
        const bool last_of_vu = (i == nt - 1) || (tile == a.n_tiles - 1);
        if (last_of_vu) umma_commit(q_empty);
      }
    }
  } else {
    // ------------------------------------------------------------ accumulator consumers
    // Thread ct of warpgroup grp owns TMEM lane ct.  The four groups form two pairs; the jobs (key
    // tile, row block) alternate between the pairs: pair p drains accumulator buffer p, i.e. every
    // job whose index has parity p, each of its two groups half of the columns.  The pairs run half
    // a job apart: while one waits for the MMAs of its next job (which cannot start before the
    // last columns of the current one have been read), the other, two warps per scheduler, keeps the
    // exponential unit busy; one warp per scheduler alone reaches less than half of that unit's rate.
    // (Measured at config 3, votes: two groups on the same job 110 us, the groups stalling together
    // at every job boundary; two groups on alternate jobs 100 us; four accumulators of 128 columns
    // 110 us, the narrower MMAs costing more than the wait they hide.)
    const int grp = warp >> 2, ct = tid & 127;
    const int pair = grp >> 1, half = grp & 1;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    int cur_vu = -1, j = 0;
    bool ok = true;
    float vsum = 0.f;

    // statistics: store this group's partial (max, sum) of every row of the virtual unit `vu`
    auto flush_stats = [&](int vu) {
      const int unit = vu / a.vu_per_unit;
      const int hq0 = (unit / Hkv) * a.Hq + (unit % Hkv) * a.G;
      const int row0 = (vu - unit * a.vu_per_unit) * a.vu_rows;
      const int slot = cta - (vu * a.n_tiles) / a.tiles_per_cta;
      for (int blk = 0; blk < a.n_blocks; ++blk) {
        const int row = row0 + blk * 128 + ct;
        if (row < a.GW)
          a.stat_part[(((size_t)hq0 * a.W + row) * a.max_slots + slot) * kGroups + grp] = ml_s[grp][blk][ct];
      }
    };

    int vu = vu_begin, tile = tile_begin, unit = vu_begin / a.vu_per_unit;
    int row0 = (vu - unit * a.vu_per_unit) * a.vu_rows;
    for (int i = 0; i < nt && ok; ++i, ++tile) {
      if (tile == a.n_tiles) {
        tile = 0; ++vu; unit = vu / a.vu_per_unit;
        row0 = (vu - unit * a.vu_per_unit) * a.vu_rows;
      }
      if (vu != cur_vu) {
        if (kVotes) {
          // this warp's copy of -lse2 of the unit's window rows (-inf for the padding rows); warps
          // keep their own copy so that no barrier wider than a warp is needed here
          const int hq0 = (unit / Hkv) * a.Hq + (unit % Hkv) * a.G;
          const int cwh = a.block_rows >> 1;   // this group's columns of a row block: [half * cwh, +cwh)
          __syncwarp();
          for (int idx = lane; idx < 256; idx += 32) {
            const int blk = idx >> 7, c = idx & 127;
            const int r = blk * a.block_rows + half * cwh + c;
            nlse2_s[warp][idx] = (blk < a.n_blocks && c < cwh && r < a.GW) ? -a.row_lse[(size_t)hq0 * a.W + r] * kLog2e
                                                                         : -INFINITY;
          }
          __syncwarp();
        } else {
          if (cur_vu >= 0) flush_stats(cur_vu);
          for (int blk = 0; blk < 2; ++blk) ml_s[grp][blk][ct] = make_float2(-INFINITY, 0.f);
        }
        cur_vu = vu;
      }
      const int tbase = tile * TILE_KEYS;
      for (int blk = 0; blk < a.n_blocks; ++blk, ++j) {
        if ((j & 1) != pair) continue;
        const int buf = j & (kNumBufs - 1);
        const uint32_t lane_addr = lane_base + (uint32_t)(buf * kBufCols);
        ok = mbar_wait(&ctl, t_full(buf), (j / kNumBufs) & 1, (kVotes ? 35u : 15u) | ((unsigned)j << 8));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        uint32_t ra[32], rb[32];
        if (kVotes) {
          const int cw = a.block_rows >> 1;  // columns (query rows) of this group: a multiple of 32
          const float* nl = nlse2_s[warp] + blk * 128;
          const uint32_t tcol = lane_addr + (uint32_t)(half * cw);
          float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;  // running vote of this thread's key
          auto add32 = [&](const uint32_t (&r)[32], int c0) {
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              const float4 n4 = *reinterpret_cast<const float4*>(nl + c0 + e);
              acc0 += ex2_approx(fmaf(__uint_as_float(r[e + 0]), a.scale2, n4.x));
              acc1 += ex2_approx(fmaf(__uint_as_float(r[e + 1]), a.scale2, n4.y));
              acc2 += ex2_approx(fmaf(__uint_as_float(r[e + 2]), a.scale2, n4.z));
              acc3 += ex2_approx(fmaf(__uint_as_float(r[e + 3]), a.scale2, n4.w));
            }
          };
          // chunks of 32 columns alternate between the two register sets (cw is a multiple of 32)
          tmem_ld32_issue(tcol, ra);
#pragma unroll 1
          for (int c0 = 0; c0 < cw; c0 += 64) {
            tmem_ld_wait(ra);
            const bool more_b = c0 + 32 < cw;
            if (more_b) tmem_ld32_issue(tcol + c0 + 32, rb);
            else { tc_fence_before_sync(); mbar_arrive(t_empty(buf)); }   // all of it is in registers
            add32(ra, c0);
            if (more_b) {
              tmem_ld_wait(rb);
              if (c0 + 64 < cw) tmem_ld32_issue(tcol + c0 + 64, ra);
              else { tc_fence_before_sync(); mbar_arrive(t_empty(buf)); }
              add32(rb, c0 + 32);
            }
          }
          // the two halves of the key's vote meet in shared memory; the first group stores the sum
          const float part = (acc0 + acc1) + (acc2 + acc3);
          const int jp = j >> 1;   // index of the job among this pair's jobs
          if (half == 1) {
            ok = mbar_wait(&ctl, vx_empty(pair), (jp & 1) ^ 1, 37u | ((unsigned)j << 8));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            vx[pair][ct] = part;
            mbar_arrive(vx_full(pair));
          } else {
            ok = mbar_wait(&ctl, vx_full(pair), jp & 1, 38u | ((unsigned)j << 8));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            vsum += part + vx[pair][ct];
            mbar_arrive(vx_empty(pair));
            // the vote of the key over this pair's row blocks of the tile; stored after the last of them
            if (blk + 2 >= a.n_blocks) {
              const int key = tbase + ct;
              float* out = (a.n_blocks > 1 && pair == 1) ? a.vote2 : a.vote;
              if (key < a.n_cand) out[(size_t)unit * a.n_cand + key] = vsum;
              vsum = 0.f;
            }
          }
        } else {
          float2 ml = ml_s[grp][blk][ct];
          const int row = row0 + blk * 128 + ct;
          // local index of the last key this row may see inside the tile (causal inside the window)
          const int lim = min(a.L - 1, a.n_cand + row % a.W) - tbase;
          const bool full_tile = __all_sync(0xffffffffu, lim >= TILE_KEYS - 1);
          auto fold32 = [&](uint32_t (&r)[32], int c0) {
            if (!full_tile) {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (c0 + e > lim) r[e] = 0xff800000u;  // -inf
            }
            const float m_new = fmaxf(ml.x, max_32(r) * a.scale2);
            if (m_new > -INFINITY) {
              ml.y = ml.y * ex2_approx(ml.x - m_new) + sum_exp2_32(r, a.scale2, -m_new);
              ml.x = m_new;
            }
          };
          const int cbeg = half * (TILE_KEYS / 2), cend = cbeg + TILE_KEYS / 2;  // this group's keys of the tile
          tmem_ld32_issue(lane_addr + cbeg, ra);
#pragma unroll 1
          for (int c0 = cbeg; c0 < cend; c0 += 64) {
            tmem_ld_wait(ra);
            tmem_ld32_issue(lane_addr + c0 + 32, rb);
            fold32(ra, c0);
            tmem_ld_wait(rb);
            if (c0 + 64 < cend) {
              tmem_ld32_issue(lane_addr + c0 + 64, ra);
            } else {
              tc_fence_before_sync();
              mbar_arrive(t_empty(buf));  // the accumulator is in registers: hand the buffer back early
            }
            fold32(rb, c0 + 32);
          }
          ml_s[grp][blk][ct] = ml;
        }
      }
    }
    if (!kVotes && ok && cur_vu >= 0 && !ctl.abort) flush_stats(cur_vu);
  }

  // ---------------------------------------------------------------- teardown (every path)
  if (ctl.abort) {
    for (int i = 0; i < 50; ++i) __nanosleep(20000);  // let TMA copies still in flight land
  }
  tc_fence_before_sync();
  __syncthreads();
  // Every warp of the CTA is done: the next kernel's CTAs may set themselves up while this one winds
  // down.  (A trigger that any thread reaches earlier counts for the whole CTA: with the idle lanes of
  // the producer and issuing warps passing it at the kernel's top, the successors' CTAs sat beside
  // the running ones for the kernel's whole length and the compress step was 12 % slower.)
  pdl_trigger();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

// Combine the partial statistics of every observation row into its natural-log LSE.  The
// partials of a row are those of the CTAs whose tile range overlaps the row's virtual unit.
__global__ void row_lse_from_parts_kernel(const float2* __restrict__ stat_part, float* __restrict__ row_lse,
                                          int rows, int GW, int vu_per_unit, int n_tiles, int tiles_per_cta,
                                          int max_slots) {
  pdl_trigger();
  pdl_wait();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const int unit = r / GW, row = r - unit * GW;
  const int vu = unit * vu_per_unit + row / 256;
  const int first = (vu * n_tiles) / tiles_per_cta, last = ((vu + 1) * n_tiles - 1) / tiles_per_cta;
  const int n = (last - first + 1) * kGroups;
  const float2* p = stat_part + (size_t)r * max_slots * kGroups;
  float m = -INFINITY;
  for (int i = 0; i < n; ++i) m = fmaxf(m, p[i].x);
  float l = 0.f;
  for (int i = 0; i < n; ++i)
    if (p[i].x > -INFINITY) l += p[i].y * exp2f(p[i].x - m);
  row_lse[r] = (m + log2f(l)) * kLn2;
}

__global__ void add_votes_kernel(float* __restrict__ vote, const float* __restrict__ vote2, size_t n) {
  pdl_trigger();
  pdl_wait();
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) vote[i] += vote2[i];
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

// Equal contiguous tile ranges over at most one CTA per SM.
void partition_tiles(ScoreArgs& a, int virtual_units) {
  a.total_tiles = virtual_units * a.n_tiles;
  const int ctas = a.total_tiles < kSms ? a.total_tiles : kSms;
  a.tiles_per_cta = (a.total_tiles + ctas - 1) / ctas;
}

}  // namespace

// Number of key-range splits per work group so that `groups * splits` CTAs fill whole waves of
// the 148 SMs (one CTA per SM) while every CTA keeps at least `min_tiles` tiles.
int pick_tile_splits(int groups, int n_tiles, int min_tiles) {
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
  a.vu_per_unit = (GW + 255) / 256;
  a.vu_rows = 256;
  a.n_blocks = GW <= 128 ? 1 : 2;
  a.block_rows = 128;
  a.n_tiles = (g.L + 255) / 256;
  partition_tiles(a, g.units * a.vu_per_unit);
  a.max_slots = (a.n_tiles + a.tiles_per_cta - 1) / a.tiles_per_cta + 1;
  if (a.max_slots * kGroups > ws.stat_slots) return cudaErrorInvalidValue;
  a.stages = 2;  // 64 KB tiles of 256 keys
  a.scale2 = g.scale2;
  a.stat_part = (float2*)(wsp + ws.stat_part);
  a.status = (unsigned*)(wsp + ws.status);
  CUtensorMap qm, km;
  const uint64_t qd[2] = {(uint64_t)GW, (uint64_t)g.units}, qs[2] = {256, (uint64_t)GW * 256};
  const uint32_t qb[2] = {128, 1};
  const uint64_t kd[2] = {(uint64_t)g.L, (uint64_t)g.units}, ks[2] = {256, (uint64_t)g.L * 256};
  const uint32_t kb[2] = {256, 1};
  if (!make_tensor_map_bf16(&qm, Q_obs, 3, qd, qs, qb) || !make_tensor_map_bf16(&km, K, 3, kd, ks, kb))
    return cudaErrorInvalidValue;
  const int smem = a.n_blocks * 128 * 256 + a.stages * 256 * 256 + 1024;
  cudaError_t e = set_smem_limit<false>(smem);
  if (e != cudaSuccess) return e;
  const int grid = (a.total_tiles + a.tiles_per_cta - 1) / a.tiles_per_cta;
  e = launch_pdl(score_tc_kernel<false>, dim3(grid), dim3(kThreads), (size_t)smem, st, qm, km, a);
  if (e != cudaSuccess) return e;
  const int rows = g.B * g.Hq * g.W;
  e = launch_pdl(row_lse_from_parts_kernel, dim3((rows + 127) / 128), dim3(128), 0, st, (const float2*)a.stat_part,
                 (float*)(wsp + ws.row_lse), rows, GW, a.vu_per_unit, a.n_tiles, a.tiles_per_cta, a.max_slots);
  count_launch(2);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// Votes of every candidate key, into ws.vote.
cudaError_t launch_votes_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                            const float* row_lse, char* wsp, cudaStream_t st) {
  const int GW = g.G * g.W;
  ScoreArgs a{};
  a.Hq = g.Hq; a.G = g.G; a.W = g.W; a.L = g.L; a.n_cand = g.n_cand; a.GW = GW;
  a.vu_per_unit = 1;
  a.vu_rows = 0;
  // One accumulator of up to 256 row columns per (key tile, row block); with several row blocks
  // per tile each warpgroup sums the blocks it drains and the two partial votes are added afterwards.
  a.n_blocks = (GW + 255) / 256;
  a.block_rows = ((GW + a.n_blocks - 1) / a.n_blocks + 63) / 64 * 64;
  a.n_tiles = (g.n_cand + kTileKeys - 1) / kTileKeys;
  partition_tiles(a, g.units);
  const int q_bytes = a.n_blocks * a.block_rows * 256;
  a.stages = q_bytes <= 65536 ? 4 : (q_bytes <= 98304 ? 3 : 2);
  a.scale2 = g.scale2;
  a.row_lse = row_lse;
  a.vote = (float*)(wsp + ws.vote);
  a.vote2 = (float*)(wsp + ws.vote2);
  a.status = (unsigned*)(wsp + ws.status);
  CUtensorMap qm, km;
  const uint64_t qd[2] = {(uint64_t)GW, (uint64_t)g.units}, qs[2] = {256, (uint64_t)GW * 256};
  const uint32_t qb[2] = {(uint32_t)a.block_rows, 1};
  const uint64_t kd[2] = {(uint64_t)g.L, (uint64_t)g.units}, ks[2] = {256, (uint64_t)g.L * 256};
  const uint32_t kb[2] = {(uint32_t)kTileKeys, 1};
  if (!make_tensor_map_bf16(&qm, Q_obs, 3, qd, qs, qb) || !make_tensor_map_bf16(&km, K, 3, kd, ks, kb))
    return cudaErrorInvalidValue;
  const int smem = q_bytes + a.stages * kKvTileBytes + 1024;
  cudaError_t e = set_smem_limit<true>(smem);
  if (e != cudaSuccess) return e;
  const int grid = (a.total_tiles + a.tiles_per_cta - 1) / a.tiles_per_cta;
  e = launch_pdl(score_tc_kernel<true>, dim3(grid), dim3(kThreads), (size_t)smem, st, qm, km, a);
  if (e != cudaSuccess) return e;
  count_launch(1);
  if (a.n_blocks > 1) {
    const size_t n = (size_t)g.units * g.n_cand;
    e = launch_pdl(add_votes_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, a.vote, (const float*)a.vote2, n);
    if (e != cudaSuccess) return e;
    count_launch(1);
  }
  return cudaGetLastError();
}

}  // namespace calidrop
