// Votes and the calibration sums in ONE pass over the keys (Algorithm 1, line 3 and lines 5-8), for
// the case in which every window query is a calibration query (n_cal = W).
//
// The probability p[r][t] = exp(q_r.k_t * scale - lse_r) of window row r and candidate key t serves
// two results: its sum over the rows is the key's vote (line 3), and once the kept set is known the
// calibration term of row r is the sum of p[r][t] v_t over the EVICTED keys (lines 5-8).  The
// evicted set is only known after the top-k, which needs every vote; but the evicted keys are the
// candidates minus the selected ones, so
//     sum over evicted = sum over ALL candidates - sum over the selected candidates.
// This kernel forms the first sum (O_all = P V and the row sums l_all over every candidate key)
// while it computes the votes, i.e. K is streamed once for both results and V once; the second sum
// runs afterwards over the few selected rows, which by then lie compacted in K_kept / V_kept (this
// same kernel on those, without the votes), and calib_combine_kernel subtracts.  Because both sums
// come from the same instruction sequence, a selected key has bit-identical logits and hence the
// same bf16-rounded probability in both, so its terms cancel exactly; what remains is the fp32
// accumulation error of the two sums, relative to the evicted share of the softmax mass.  (With
// the second sum taken by calib_tc_kernel, whose MMA has the operands the other way round, single
// probabilities differed by one bf16 step, which showed in O_c at 4e-2 when the key was a heavy one.)
//
// Work is the linear space of (kv unit, 128-key tile) pairs, cut into equal contiguous ranges; the
// CTAs of the row blocks of a unit (a row block = whole query heads, at most 128 window rows) walk
// the same range together so that a K/V tile fetched for one is an L2 hit for the others.  Per tile:
//     MMA 1   S^T = K Q^T        128 keys on the TMEM lanes, the block's rows as columns
//     threads p = exp2(scale2 * s - lse2[row]) in fp32 (zero for keys outside the candidates);
//             thread t sums its key's vote over the columns and keeps the running row sums;
//             p rounded to bf16 goes to shared memory as P^T [key][row], the layout of an
//             MN-major B operand (what a TMA box with the 128-byte swizzle would have written)
//     MMA 2   O^T += V^T P^T     head dimension on the lanes, rows as columns; V^T is the V tile read
//                                as an MN-major A operand
// The k-steps of S(i+2) are interleaved with those of P.V(i): MMAs that accumulate into one
// tensor-memory tile execute one after the other, two independent chains keep the pipe busy.
// Warp roles: two consumer warpgroups (both work on every tile, 64 row columns each), two TMA
// producer warps (Q and K; V), one warp that allocates TMEM and issues the MMAs.
// Tensor memory: S buffers at columns 0 and 128, O^T at 256.
#include <type_traits>

#include "internal.h"
#include "tc_common.cuh"

namespace calidrop {

namespace {

using namespace tc;

constexpr int kGroups = 2;
constexpr int kProducerWarp = kGroups * 4;
constexpr int kMmaWarp = kGroups * 4 + 1;
constexpr int kVProducerWarp = kGroups * 4 + 2;
constexpr int kThreads = kGroups * 128 + 96;
constexpr int kTmemCols = 512;
constexpr uint32_t kColO = 256;
constexpr int kStages = 2;                 // K ring and V ring alike
constexpr int kTileBytes = kKvTileBytes;   // 32 KB
constexpr int kNumBars = 20;
// dynamic shared memory: Q block, two P^T buffers, K ring, V ring (1024-byte aligned), then the
// barriers, the -lse2 table, the control block and the TMEM slot
constexpr int kMiscBytes = kNumBars * 8 + 128 * 4 + 32;
constexpr int kSmemBytes = (3 + 2 * kStages) * kTileBytes + 1024 + kMiscBytes;
static_assert(kSmemBytes <= 232448, "shared memory of score_pv_kernel exceeds one SM");
constexpr int kSms = 148;
constexpr int kPrefetchTiles = 6;          // L2 prefetch distance of the producer, in key tiles

struct PvArgs {
  int Hq, G, W, L, n_cand;
  int gpb;        // query heads per row block
  int n_cblocks;  // row blocks per unit
  int n_tiles;    // key tiles per unit
  int total_tiles, tiles_per_cta, max_slots;
  float scale2;
  const float* row_lse;   // [B, Hq, W] natural log
  float* vote;            // [n_cblocks][2][units][n_cand]: the partial votes of the halves of every row block
  size_t vote_stride;     // units * n_cand
  float* o_part;          // [virtual unit][slot][128 rows][128]
  float* l_part;          // [virtual unit][slot][8 warps][64 rows]
  unsigned* status;
};

__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap* map, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(c0), "r"(c1),
               "r"(c2)
               : "memory");
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  // (no memory clobber: the compiler may move its own loads across it; the proxy fence that
  // follows the last store is volatile too and stays behind every one of them)
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w));
}

__global__ void __launch_bounds__(kThreads, 1)
score_pv_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                const __grid_constant__ CUtensorMap v_map, const PvArgs a) {
  extern __shared__ unsigned char smem_raw[];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x / a.n_cblocks, cb = blockIdx.x % a.n_cblocks;
  const int g_begin = cta * a.tiles_per_cta;
  const int g_end = min(a.total_tiles, g_begin + a.tiles_per_cta);
  const int nt = g_end - g_begin;
  const int Hkv = a.Hq / a.G;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* const smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t q_base = smem_base;
  const uint32_t p_base = q_base + kTileBytes;
  const uint32_t k_base = p_base + 2 * kTileBytes;
  const uint32_t v_base = k_base + kStages * kTileBytes;
  unsigned char* const misc = smem_al + (3 + 2 * kStages) * kTileBytes;
  unsigned long long* const bars = reinterpret_cast<unsigned long long*>(misc);
  float* const nlse2_s = reinterpret_cast<float*>(misc + kNumBars * 8);       // [128]
  Ctl* const ctl = reinterpret_cast<Ctl*>(nlse2_s + 128);
  uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(ctl + 1);

  const uint32_t bar0 = smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  const uint32_t o_full = bar(0), o_empty = bar(1), q_full = bar(2), q_empty = bar(3), tbl_full = bar(4);
  auto full_k = [&](int s) { return bar(6 + s); };
  auto empty_k = [&](int s) { return bar(8 + s); };
  auto full_v = [&](int s) { return bar(10 + s); };
  auto empty_v = [&](int s) { return bar(12 + s); };
  auto s_full = [&](int b) { return bar(14 + b); };
  auto p_full = [&](int b) { return bar(16 + b); };
  auto p_empty = [&](int b) { return bar(18 + b); };

  if (tid == 0) {
    ctl->abort = 0;
    ctl->status = a.status;
    mbar_init(o_full, 1);
    mbar_init(o_empty, kGroups * 128);
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    mbar_init(tbl_full, 128);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_k(s), 1); mbar_init(empty_k(s), 1);
      mbar_init(full_v(s), 1); mbar_init(empty_v(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(s_full(b), 1); mbar_init(p_full(b), kGroups * 128); mbar_init(p_empty(b), 1);
    }
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  // The query block's box may cover fewer than 128 rows: clear the block once so that the rows no
  // TMA box writes hold zeros.
  for (int i = tid; i < kTileBytes / 16; i += kThreads) reinterpret_cast<uint4*>(smem_al)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // first tile of a run of tiles of one unit inside this CTA's range
  const int unit_begin = g_begin / a.n_tiles, tile_begin = g_begin - unit_begin * a.n_tiles;
  auto seg_first = [&](int i, int tile) { return i == 0 || tile == 0; };
  auto seg_last = [&](int i, int tile) { return i == nt - 1 || tile == a.n_tiles - 1; };

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------ TMA producer of Q and K
    // (K and V have a producer each: a K slot frees when its S is done, a V slot only when its P.V
    // is, and one thread serving both in turn would hold every K load back behind a V slot)
    if (lane == 0) {
      tma_prefetch_desc(&q_map);
      tma_prefetch_desc(&k_map);
      int seg = 0, tile = tile_begin, unit = unit_begin;
      // position of the tile kPrefetchTiles ahead, for the L2 prefetch (first row block only)
      int pf_tile = tile_begin, pf_unit = unit_begin, pf_i = 0;
      for (int i = 0; i < nt; ++i, ++tile) {
        if (tile == a.n_tiles) { tile = 0; ++unit; }
        if (cb == 0) {
          while (pf_i < nt && pf_i <= i + kPrefetchTiles) {
            if (pf_tile == a.n_tiles) { pf_tile = 0; ++pf_unit; }
            if (pf_i >= kStages) {   // the first tiles are fetched straight away
              for (int half = 0; half < 2; ++half)
                tma_prefetch_l2_3d(&k_map, half * kHalfCols, pf_tile * kTileKeys, pf_unit);
            }
            ++pf_i; ++pf_tile;
          }
        }
        if (seg_first(i, tile)) {
          // the Q block of the next unit replaces the current one once its MMAs are done
          if (seg > 0 && !mbar_wait(ctl, q_empty, (seg - 1) & 1, 40u | ((unsigned)i << 8))) break;
          const int g0 = cb * a.gpb;
          mbar_arrive_expect_tx(q_full, 2u * (uint32_t)(a.gpb * a.W) * kLineBytes);  // the whole box counts
          for (int half = 0; half < 2; ++half)
            tma_load_4d(q_base + half * (kTileBytes / 2), &q_map, q_full, half * kHalfCols, 0, g0, unit);
          ++seg;
        }
        const int s = i % kStages;
        if (!mbar_wait(ctl, empty_k(s), ((i / kStages) & 1) ^ 1, 41u | ((unsigned)i << 8))) break;
        mbar_arrive_expect_tx(full_k(s), kTileBytes);
        for (int half = 0; half < 2; ++half)
          tma_load_3d(k_base + s * kTileBytes + half * (kTileBytes / 2), &k_map, full_k(s), half * kHalfCols,
                      tile * kTileKeys, unit);
      }
    }
  } else if (warp == kVProducerWarp) {
    // ------------------------------------------------------------ TMA producer of V
    if (lane == 0) {
      tma_prefetch_desc(&v_map);
      int tile = tile_begin, unit = unit_begin;
      int pf_tile = tile_begin, pf_unit = unit_begin, pf_i = 0;
      for (int i = 0; i < nt; ++i, ++tile) {
        if (tile == a.n_tiles) { tile = 0; ++unit; }
        if (cb == 0) {
          while (pf_i < nt && pf_i <= i + kPrefetchTiles) {
            if (pf_tile == a.n_tiles) { pf_tile = 0; ++pf_unit; }
            if (pf_i >= kStages) {
              for (int half = 0; half < 2; ++half)
                tma_prefetch_l2_3d(&v_map, half * kHalfCols, pf_tile * kTileKeys, pf_unit);
            }
            ++pf_i; ++pf_tile;
          }
        }
        const int s = i % kStages;
        if (!mbar_wait(ctl, empty_v(s), ((i / kStages) & 1) ^ 1, 42u | ((unsigned)i << 8))) break;
        mbar_arrive_expect_tx(full_v(s), kTileBytes);
        for (int half = 0; half < 2; ++half)
          tma_load_3d(v_base + s * kTileBytes + half * (kTileBytes / 2), &v_map, full_v(s), half * kHalfCols,
                      tile * kTileKeys, unit);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ MMA issuer
    // At the start of a unit S(i) and S(i+1) are issued (k-steps interleaved); from then on P.V(i)
    // is issued together with S(i+2) as soon as P(i) is complete (which also means S(i) has been
    // read out of its buffer).  S never runs ahead across a change of unit: its Q block is only
    // loaded once the current unit's MMAs are done.
    if (lane == 0) {
      const uint32_t idesc_s = umma_idesc(128, 128, false, false);  // S^T: A = K tile, B = Q block, K-major
      const uint32_t idesc_o = umma_idesc(128, 128, true, true);    // O^T: A = V^T, B = P^T, MN-major
      const uint32_t tmem_o = tmem_base + kColO;
      int seg = 0;
      bool ok = true;
      // Descriptors of every operand buffer, built once; a k-step adds a constant to the address field.
      const uint64_t dq = smem_desc_sw128(q_base, 16u, 1024u);
      static_assert(kStages == 2, "the ring slots are picked by the parity of the tile index");
      const uint64_t dk0 = smem_desc_sw128(k_base, 16u, 1024u), dk1 = desc_advance(dk0, kTileBytes);
      const uint64_t dv0 = smem_desc_sw128(v_base, kTileBytes / 2, 1024u), dv1 = desc_advance(dv0, kTileBytes);
      const uint64_t dp0 = smem_desc_sw128(p_base, kTileBytes / 2, 1024u), dp1 = desc_advance(dp0, kTileBytes);
      // S(i): eight k-steps, K-major operands
      auto s_steps = [&](int i) {
        const uint32_t d = tmem_base + (uint32_t)((i & 1) * 128);
        const uint64_t kd = (i & 1) ? dk1 : dk0;
        umma_ss_imm<0>(d, kd, dq, idesc_s);
#pragma unroll
        for (int kk = 1; kk < kD / 16; ++kk)
          umma_ss_imm<1>(d, desc_advance(kd, kmajor_step_bytes(kTileBytes / 2, kk)),
                         desc_advance(dq, kmajor_step_bytes(kTileBytes / 2, kk)), idesc_s);
      };
      // P.V(i) with or without S(i2) interleaved: 16 keys per step; both P.V operands have the keys
      // as K (MN-major), 64-element blocks along M / N half a tile apart, groups of 8 keys 1024 bytes apart
      auto batch = [&](int i, auto first_tag, auto with_s_tag) {
        constexpr bool kFirst = decltype(first_tag)::value, kWithS = decltype(with_s_tag)::value;
        const uint64_t vd = (i & 1) ? dv1 : dv0, pd = (i & 1) ? dp1 : dp0;
        const uint32_t d = tmem_base + (uint32_t)((i & 1) * 128);   // S(i+2) reuses the buffer of S(i)
        const uint64_t kd = (i & 1) ? dk1 : dk0;                    // and K(i+2) the ring slot of K(i)
#pragma unroll
        for (int kk = 0; kk < kTileKeys / 16; ++kk) {
          const uint32_t koff = (uint32_t)kk * 16u * kLineBytes;
          if (kFirst && kk == 0) umma_ss_imm<0>(tmem_o, vd, pd, idesc_o);
          else umma_ss_imm<1>(tmem_o, desc_advance(vd, koff), desc_advance(pd, koff), idesc_o);
          if (kWithS) {
            if (kk == 0) umma_ss_imm<0>(d, kd, dq, idesc_s);
            else umma_ss_imm<1>(d, desc_advance(kd, kmajor_step_bytes(kTileBytes / 2, kk)),
                                desc_advance(dq, kmajor_step_bytes(kTileBytes / 2, kk)), idesc_s);
          }
        }
      };
      auto wait_k = [&](int i) { return mbar_wait(ctl, full_k(i % kStages), (i / kStages) & 1, 44u | ((unsigned)i << 8)); };
      auto s_done = [&](int i) { umma_commit(s_full(i & 1)); umma_commit(empty_k(i % kStages)); };
      int tile = tile_begin;
      for (int i = 0; ok && i < nt; ++i, ++tile) {
        if (tile == a.n_tiles) tile = 0;
        const bool first = seg_first(i, tile), last = seg_last(i, tile);
        if (first) {
          // new unit: its Q block must have landed, and O of the previous unit must have been read
          // out before the first P.V overwrites it
          ok = mbar_wait(ctl, q_full, seg & 1, 43u | ((unsigned)i << 8));
          if (ok && seg > 0) ok = mbar_wait(ctl, o_empty, (seg - 1) & 1, 45u | ((unsigned)i << 8));
          ++seg;
          if (!ok) break;
          const bool two = !last;
          ok = wait_k(i) && (!two || wait_k(i + 1));
          if (!ok) break;
          tc_fence_after_sync();
          s_steps(i);
          if (two) s_steps(i + 1);
          s_done(i);
          if (two) s_done(i + 1);
        }
        // P.V(i), together with S(i+2) when that tile belongs to the same unit
        const bool with_s = !last && !seg_last(i + 1, tile + 1);
        if (!mbar_wait(ctl, p_full(i & 1), (i >> 1) & 1, 46u | ((unsigned)i << 8))) break;
        if (!mbar_wait(ctl, full_v(i % kStages), (i / kStages) & 1, 47u | ((unsigned)i << 8))) break;
        if (with_s && !wait_k(i + 2)) break;
        tc_fence_after_sync();
        if (with_s) {
          if (first) batch(i, std::true_type{}, std::true_type{});
          else batch(i, std::false_type{}, std::true_type{});
        } else {
          if (first) batch(i, std::true_type{}, std::false_type{});
          else batch(i, std::false_type{}, std::false_type{});
        }
        if (with_s) s_done(i + 2);
        umma_commit(empty_v(i % kStages));
        umma_commit(p_empty(i & 1));
        if (last) {
          umma_commit(o_full);
          umma_commit(q_empty);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ consumers (one key each)
    // Thread ct of either group owns TMEM lane ct = key ct of the tile; group grp takes the columns
    // (window rows of the block) [64 grp, 64 grp + 64).
    const int grp = warp >> 2, ct = tid & 127;
    const uint32_t lane_bits = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_bits + (uint32_t)(grp * 64);
    const uint32_t p_line = (uint32_t)(grp * (kTileBytes / 2) + ct * kLineBytes);  // this key's line of the group's row block
    const uint32_t p_xor = (uint32_t)(ct & 7);
    float lrow[64];
#pragma unroll
    for (int c = 0; c < 64; ++c) lrow[c] = 0.f;
    int cur_unit = -1, seg = 0, rows = 0;
    bool ok = true;

    // Read out O^T and the row sums of the unit that just ended (each group half of the rows).
    // o_full also tells that every MMA that read the Q block or a P buffer has completed.
    auto store_partial = [&](int unit) -> bool {
      bool w = mbar_wait(ctl, o_full, (seg - 1) & 1, 50u);
      w = __all_sync(0xffffffffu, w);
      if (!w) return false;
      tc_fence_after_sync();
      const int slot = cta - (unit * a.n_tiles) / a.tiles_per_cta;
      const size_t part = (size_t)(unit * a.n_cblocks + cb) * a.max_slots + slot;
      float* obase = a.o_part + part * 128 * kD + ct;   // element (row r, head-dim ct) at r * 128 + ct
#pragma unroll 1
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t ov[32];
        tmem_ld32(tmem_base + lane_bits + kColO + (uint32_t)(grp * 64 + c0), ov);
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int r = grp * 64 + c0 + e;
          if (r < rows) obase[(size_t)r * kD] = __uint_as_float(ov[e]);
        }
      }
      // row sums: across the 32 keys of the warp; the warps' partials are added by the combine kernel
      float* lbase = a.l_part + (part * 8 + warp) * 64;
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        const float s = warp_sum(lrow[c]);
        if (lane == (c & 31)) lbase[c] = s;
        lrow[c] = 0.f;
      }
      tc_fence_before_sync();
      mbar_arrive(o_empty);
      return true;
    };

    int tile = tile_begin, unit = unit_begin;
    for (int i = 0; i < nt; ++i, ++tile) {
      if (tile == a.n_tiles) { tile = 0; ++unit; }
      if (unit != cur_unit) {
        if (cur_unit >= 0) {
          ok = store_partial(cur_unit);
          if (!ok) break;
        }
        // -lse2 of the block's rows (-inf for the rows the block does not have): written by group 0,
        // one entry per thread; every reader is past the previous unit's last tile by now
        const int hq0 = (unit / Hkv) * a.Hq + (unit % Hkv) * a.G;
        const int g0 = cb * a.gpb;
        rows = min(a.gpb, a.G - g0) * a.W;
        if (grp == 0) {
          nlse2_s[ct] = ct < rows ? -a.row_lse[(size_t)(hq0 + g0) * a.W + ct] * kLog2e : -INFINITY;
          mbar_arrive(tbl_full);
        }
        ok = mbar_wait(ctl, tbl_full, seg & 1, 51u | ((unsigned)i << 8));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        cur_unit = unit;
        ++seg;
      }
      const int buf = i & 1;
      const int key = tile * kTileKeys + ct;
      const bool key_ok = key < a.n_cand;
      const bool tile_full = (tile + 1) * kTileKeys <= a.n_cand;   // no key of the tile needs masking
      ok = mbar_wait(ctl, s_full(buf), (i >> 1) & 1, 48u | ((unsigned)i << 8));
      if (ok) ok = mbar_wait(ctl, p_empty(buf), ((i >> 1) & 1) ^ 1, 49u | ((unsigned)i << 8));
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t p_addr = p_base + (uint32_t)(buf * kTileBytes) + p_line;
      const float4* nl = reinterpret_cast<const float4*>(nlse2_s + grp * 64);
      float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
      // probabilities of 32 row columns: votes, row sums, bf16 pairs into this key's line of P^T
      auto soft32 = [&](const uint32_t (&sv)[32], auto c0_tag, auto masked_tag) {
        constexpr int c0 = decltype(c0_tag)::value;
        constexpr bool masked = decltype(masked_tag)::value;
        float pr[32];
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 n4 = nl[(c0 + e) >> 2];
          pr[e + 0] = ex2_approx(fmaf(__uint_as_float(sv[e + 0]), a.scale2, n4.x));
          pr[e + 1] = ex2_approx(fmaf(__uint_as_float(sv[e + 1]), a.scale2, n4.y));
          pr[e + 2] = ex2_approx(fmaf(__uint_as_float(sv[e + 2]), a.scale2, n4.z));
          pr[e + 3] = ex2_approx(fmaf(__uint_as_float(sv[e + 3]), a.scale2, n4.w));
        }
        if (masked) {
#pragma unroll
          for (int e = 0; e < 32; ++e) pr[e] = key_ok ? pr[e] : 0.f;
        }
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          acc0 += pr[e + 0]; acc1 += pr[e + 1]; acc2 += pr[e + 2]; acc3 += pr[e + 3];
          lrow[c0 + e + 0] += pr[e + 0]; lrow[c0 + e + 1] += pr[e + 1];
          lrow[c0 + e + 2] += pr[e + 2]; lrow[c0 + e + 3] += pr[e + 3];
        }
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          const uint32_t chunk = (uint32_t)((c0 + e) >> 3);
          st_shared_v4(p_addr + ((chunk ^ p_xor) << 4), pack_bf16(pr[e + 0], pr[e + 1]), pack_bf16(pr[e + 2], pr[e + 3]),
                       pack_bf16(pr[e + 4], pr[e + 5]), pack_bf16(pr[e + 6], pr[e + 7]));
        }
      };
      uint32_t ra[32], rb[32];
      tmem_ld32_issue(s_addr + (uint32_t)(buf * 128), ra);
      tmem_ld_wait(ra);
      tmem_ld32_issue(s_addr + (uint32_t)(buf * 128 + 32), rb);
      if (tile_full) {
        soft32(ra, std::integral_constant<int, 0>{}, std::false_type{});
        tmem_ld_wait(rb);
        soft32(rb, std::integral_constant<int, 32>{}, std::false_type{});
      } else {
        soft32(ra, std::integral_constant<int, 0>{}, std::true_type{});
        tmem_ld_wait(rb);
        soft32(rb, std::integral_constant<int, 32>{}, std::true_type{});
      }
      fence_proxy_async_smem();   // the P^T stores must be visible to the MMA's shared-memory reads
      tc_fence_before_sync();
      mbar_arrive(p_full(buf));
      // each group stores the partial vote of its half of the rows; sum_vote_parts_kernel adds them
      if (key_ok && a.vote)
        a.vote[(size_t)(cb * kGroups + grp) * a.vote_stride + (size_t)unit * a.n_cand + key] = (acc0 + acc1) + (acc2 + acc3);
    }
    if (ok && cur_unit >= 0) store_partial(cur_unit);
  }

  // ---------------------------------------------------------------- teardown (every path)
  if (ctl->abort) {
    for (int i = 0; i < 50; ++i) __nanosleep(20000);  // let TMA copies still in flight land
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

// vote[i] = sum of the partial votes (two per row block), in order.
__global__ void sum_vote_parts_kernel(float* __restrict__ vote, size_t n, int parts) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = vote[i];
  for (int p = 1; p < parts; ++p) s += vote[(size_t)p * n + i];
  vote[i] = s;
}

// The subtraction loses accuracy when the evicted keys carry little of a row's softmax mass: the
// fp32 accumulation error of the sum over all candidates (about 1e-5 of it, measured) is divided by
// that share.  Rows below this share have their unit listed for the masked pass over the evicted
// keys themselves (calib_tc_kernel in work-list mode), which rewrites the unit's rows.
constexpr float kMinEvictedShare = 1.0f / 64.0f;

// One warp per (batch, query head, window row): the sums over all candidates (score_pv_kernel)
// minus the sums over the selected ones (the same kernel on the compacted rows), each added up over
// its CTAs' partials in a fixed order; then O_c = O / l, LSE_c = lse + log l, C_q = the query.
// redo = {block counter, n_work, unit_flag[units], unit_pos[units], work_list[units]}, zeroed by the
// caller: rows that need the masked pass flag their unit, and the block that finishes last turns
// the flags into the ascending list of those units.
__global__ void __launch_bounds__(128)
calib_combine_kernel(const __nv_bfloat16* __restrict__ Q_obs, const float* __restrict__ row_lse,
                     const float* __restrict__ o_all, const float* __restrict__ l_all, int n_tiles_all,
                     int tpc_all, int slots_all, const float* __restrict__ o_sel, const float* __restrict__ l_sel,
                     int n_tiles_sel, int tpc_sel, int slots_sel, float* __restrict__ O_c,
                     float* __restrict__ LSE_c, __nv_bfloat16* __restrict__ C_q, int B, int Hq, int G, int W, int gpb,
                     int n_cblocks, int* __restrict__ redo) {
  __shared__ bool is_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.x * 4 + warp;  // (b, hq, c), n_cal = W
  const int units = B * (Hq / G);
  int* const unit_flag = redo + 2;
  if (row < B * Hq * W) {
    const int c = row % W, bhq = row / W;
    const int b = bhq / Hq, hq = bhq % Hq;
    const int Hkv = Hq / G, h = hq / G, g = hq % G;
    const int unit = b * Hkv + h, cb = g / gpb, r = (g % gpb) * W + c;
    const int vu = unit * n_cblocks + cb;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    {
      const int first = (unit * n_tiles_all) / tpc_all, last = ((unit + 1) * n_tiles_all - 1) / tpc_all;
      const size_t part0 = (size_t)vu * slots_all;
      for (int s = 0; s <= last - first; ++s) {
        const float4 v = *reinterpret_cast<const float4*>(o_all + ((part0 + s) * 128 + r) * kD + 4 * lane);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        for (int w = 0; w < 4; ++w) l += l_all[((part0 + s) * 8 + (r >> 6) * 4 + w) * 64 + (r & 63)];
      }
    }
    float4 sel = make_float4(0.f, 0.f, 0.f, 0.f);
    float ls = 0.f;
    {
      const int first = (unit * n_tiles_sel) / tpc_sel, last = ((unit + 1) * n_tiles_sel - 1) / tpc_sel;
      const size_t part0 = (size_t)vu * slots_sel;
      for (int s = 0; s <= last - first; ++s) {
        const float4 v = *reinterpret_cast<const float4*>(o_sel + ((part0 + s) * 128 + r) * kD + 4 * lane);
        sel.x += v.x; sel.y += v.y; sel.z += v.z; sel.w += v.w;
        for (int w = 0; w < 4; ++w) ls += l_sel[((part0 + s) * 8 + (r >> 6) * 4 + w) * 64 + (r & 63)];
      }
    }
    const float l_cand = l;
    l -= ls;
    if (lane == 0 && !(l >= kMinEvictedShare * l_cand)) atomicOr(&unit_flag[unit], 1);
    float4 out = make_float4(0.f, 0.f, 0.f, 0.f);
    float lse = -INFINITY;
    if (l > 0.f) {
      const float inv = 1.f / l;
      out = make_float4((acc.x - sel.x) * inv, (acc.y - sel.y) * inv, (acc.z - sel.z) * inv, (acc.w - sel.w) * inv);
      lse = row_lse[(size_t)bhq * W + c] + logf(l);
    }
    reinterpret_cast<float4*>(O_c + (size_t)row * kD)[lane] = out;
    if (lane == 0) LSE_c[row] = lse;
    reinterpret_cast<uint2*>(C_q + (size_t)row * kD)[lane] =
        reinterpret_cast<const uint2*>(Q_obs + (size_t)row * kD)[lane];
  }
  // the last block to finish lists the flagged units (no block waits for another)
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = atomicAdd(reinterpret_cast<unsigned*>(redo), 1u) == gridDim.x - 1;
  __syncthreads();
  if (is_last && warp == 0) {
    __threadfence();
    int* const unit_pos = unit_flag + units;
    int* const work_list = unit_pos + units;
    int count = 0;
    for (int base = 0; base < units; base += 32) {
      const int u = base + lane;
      const bool f = u < units && __ldcg(unit_flag + u) != 0;
      const unsigned ball = __ballot_sync(0xffffffffu, f);
      const int pos = count + __popc(ball & ((1u << lane) - 1u));
      if (u < units) unit_pos[u] = f ? pos : -1;
      if (f) work_list[pos] = u;
      count += __popc(ball);
    }
    if (lane == 0) redo[1] = count;
  }
}

}  // namespace

// The one-pass form needs every window row to be a calibration row, whole heads in a 128-row
// block, and more evicted than selected candidates (otherwise summing the evicted keys directly is
// both cheaper and free of the subtraction).
bool score_pv_supported(const CompressGeom& g) {
  return !g.keep_all && g.n_cal == g.W && g.W <= 128 && g.k_sel >= 1 && g.n_cand - g.k_sel > g.k_sel;
}

// One pass of score_pv_kernel over rows [0, n_keys) of every unit of K / V (a unit's rows are
// `unit_rows` apart): the partial (O, l) sums into o_part / l_part and, when `vote` is not null, the
// votes of those keys.
static cudaError_t launch_pv_pass(const CompressGeom& g, const void* Q_obs, const void* K, const void* V, int n_keys,
                                  size_t unit_rows, const float* row_lse, float* vote, float* o_part, float* l_part,
                                  unsigned* status, cudaStream_t st) {
  PvArgs a{};
  a.Hq = g.Hq; a.G = g.G; a.W = g.W; a.L = g.L; a.n_cand = n_keys;
  size_t parts;
  calib_tc_plan(g, n_keys, &a.gpb, &a.n_cblocks, &a.tiles_per_cta, &a.max_slots, &parts);
  a.n_tiles = (n_keys + kTileKeys - 1) / kTileKeys;
  a.total_tiles = g.units * a.n_tiles;
  a.scale2 = g.scale2;
  a.row_lse = row_lse;
  a.vote = vote;
  a.vote_stride = (size_t)g.units * n_keys;
  a.o_part = o_part;
  a.l_part = l_part;
  a.status = status;
  CUtensorMap qm, km, vm;
  // window rows: [head dim][j < W][g < G][unit]
  const uint64_t qd[3] = {(uint64_t)g.W, (uint64_t)g.G, (uint64_t)g.units};
  const uint64_t qs[3] = {256, (uint64_t)g.W * 256, (uint64_t)g.G * g.W * 256};
  const uint32_t qb[3] = {(uint32_t)g.W, (uint32_t)a.gpb, 1};
  if (!make_tensor_map_bf16(&qm, Q_obs, 4, qd, qs, qb)) return cudaErrorInvalidValue;
  // rows at or beyond n_keys are never used (their probabilities are masked), so the maps end there
  const uint64_t kd[2] = {(uint64_t)n_keys, (uint64_t)g.units}, ks[2] = {256, (uint64_t)unit_rows * 256};
  const uint32_t kb[2] = {(uint32_t)kTileKeys, 1};
  if (!make_tensor_map_bf16(&km, K, 3, kd, ks, kb) || !make_tensor_map_bf16(&vm, V, 3, kd, ks, kb))
    return cudaErrorInvalidValue;
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(score_pv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const int grid = (a.total_tiles + a.tiles_per_cta - 1) / a.tiles_per_cta * a.n_cblocks;
  score_pv_kernel<<<grid, kThreads, kSmemBytes, st>>>(qm, km, vm, a);
  count_launch(1);
  if (vote) {
    const size_t n = a.vote_stride;
    sum_vote_parts_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(vote, n, a.n_cblocks * kGroups);
    count_launch(1);
  }
  return cudaGetLastError();
}

// Votes of every candidate key (into ws.vote) and the sums over all candidates.
cudaError_t launch_score_pv(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                            const void* V, const float* row_lse, char* wsp, cudaStream_t st) {
  return launch_pv_pass(g, Q_obs, K, V, g.n_cand, (size_t)g.L, row_lse, (float*)(wsp + ws.vote),
                        (float*)(wsp + ws.calib_o), (float*)(wsp + ws.pv_l), (unsigned*)(wsp + ws.status), st);
}

// The sums over the selected rows, rows [0, k_sel) of every unit of the kept cache: the same kernel,
// hence the same logits and the same bf16 probabilities as in the pass over all candidates.
cudaError_t launch_score_pv_selected(const CompressGeom& g, const CompressWs& ws, const void* Q_obs,
                                     const void* K_kept, const void* V_kept, const float* row_lse, char* wsp,
                                     cudaStream_t st) {
  return launch_pv_pass(g, Q_obs, K_kept, V_kept, g.k_sel, (size_t)g.cap, row_lse, nullptr, (float*)(wsp + ws.sel_o),
                        (float*)(wsp + ws.sel_l), (unsigned*)(wsp + ws.status), st);
}

cudaError_t launch_calib_combine(const CompressGeom& g, const CompressWs& ws, const void* Q_obs,
                                 const float* row_lse, char* wsp, float* O_c, float* LSE_c, void* C_q,
                                 cudaStream_t st) {
  int gpb, n_cblocks, tpc_all, slots_all, tpc_sel, slots_sel;
  size_t parts;
  calib_tc_plan(g, g.n_cand, &gpb, &n_cblocks, &tpc_all, &slots_all, &parts);
  calib_tc_plan(g, g.k_sel, &gpb, &n_cblocks, &tpc_sel, &slots_sel, &parts);
  const int total = g.B * g.Hq * g.W;
  calib_combine_kernel<<<(total + 3) / 4, 128, 0, st>>>(
      (const __nv_bfloat16*)Q_obs, row_lse, (const float*)(wsp + ws.calib_o), (const float*)(wsp + ws.pv_l),
      (g.n_cand + kTileKeys - 1) / kTileKeys, tpc_all, slots_all, (const float*)(wsp + ws.sel_o),
      (const float*)(wsp + ws.sel_l), (g.k_sel + kTileKeys - 1) / kTileKeys, tpc_sel, slots_sel, O_c, LSE_c,
      (__nv_bfloat16*)C_q, g.B, g.Hq, g.G, g.W, gpb, n_cblocks, (int*)(wsp + ws.redo));
  count_launch(1);
  return cudaGetLastError();
}

}  // namespace calidrop
