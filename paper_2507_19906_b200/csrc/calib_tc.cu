// Calibration term on the tensor cores (Algorithm 1, lines 5-8): for every calibration query
// row, the softmax-weighted sum of the EVICTED values and the log of its normaliser.
//
// Work is the linear space of (virtual unit, 128-key tile) pairs, a virtual unit being one block
// of up to 128 calibration rows (whole query heads, n_cal rows each) of a (batch, kv-head) unit;
// it is cut into equal contiguous ranges, one per CTA, at most one CTA per SM.  Per tile:
//     MMA 1   S = Q_c K^T       query rows on the TMEM lanes; Q_c block resident in shared memory
//                               (reloaded per virtual unit), the K tile comes from TMA
//     threads p = exp2(scale2 * s - lse2[row]), zero for kept keys (bitmap) and for keys outside
//             the candidates; row sums l kept in fp32; p rounded to bf16 and stored into tensor
//             memory as the A operand of
//     MMA 2   O += P V          V tile from TMA, read as the MN-major B operand
// lse2[row] is the row's LSE over ALL the keys it sees (from the statistics pass or the caller), so
// every p <= 1 and no running maximum or rescaling is needed: the partial (O, l) of the key ranges
// simply add up.  calib_reduce_kernel sums them in a fixed order and writes O_c = O / l,
// LSE_c = lse + log l, C_q.
// Warp roles: two softmax warpgroups (group g takes the tiles with local index i % 2 == g), two TMA
// producer warps (Q_c and K; V), and two MMA-issuing warps, one for S and one for P.V: a single
// thread's dependent scalar instructions cost several cycles each, and with the waits and commits of
// both chains on one thread the issue, not the tensor pipe, set the pace (a lone chain of eight
// 128x128x16 MMAs runs at the pipe's 64 cycles each once its descriptors are prepared; no
// interleaving of chains is needed).
// Tensor memory: three S/P buffers of 128 columns at 0, 128, 256 and O at 384.  Tile i lives in buffer
// i % 3: S(i) arrives there, and its probabilities, rounded to bf16, overwrite the first 64 columns in
// place (a thread stores the P of 32 keys only after the S of those columns is in its registers).  A
// buffer is free again when the P.V that read it has completed; with three of them S(i+2) is ready
// when its group has finished tile i, and a group never waits for the P.V of its own previous tile
// (with two S buffers and a P buffer per group it did, for about a third of its time).
#include <type_traits>

#include "internal.h"
#include "tc_common.cuh"

namespace calidrop {

namespace {

using namespace tc;

constexpr int kGroups = kCalibGroups;  // softmax warpgroups: two pairs; a pair shares a tile, half of its keys each
constexpr int kProducerWarp = kGroups * 4;       // TMA: Q_c blocks and K tiles
constexpr int kMmaWarp = kGroups * 4 + 1;        // allocates TMEM, issues the S MMAs
constexpr int kPvWarp = kGroups * 4 + 2;         // issues the P.V MMAs
constexpr int kVProducerWarp = kGroups * 4 + 3;  // TMA: V tiles
constexpr int kThreads = kGroups * 128 + 128;
static_assert(kGroups == 4, "two pairs of softmax groups");
constexpr int kTmemCols = 512;
constexpr int kBufs = 3;                   // S/P buffers of 128 columns
constexpr uint32_t kColO = kBufs * 128;
constexpr int kStages = kBufs;             // K ring and V ring: slot t % 3 feeds buffer t % 3
constexpr int kTileBytes = kKvTileBytes;   // 32 KB
constexpr int kSmemBytes = (1 + 2 * kStages) * kTileBytes + 1024;  // Q_c block, K ring, V ring
constexpr int kSms = 148;

struct CalibArgs {
  int Hq, G, W, L, n_cand, n_cal;
  int gpb;        // query heads per row block
  int n_cblocks;  // row blocks (virtual units) per unit
  int n_tiles;    // key tiles per virtual unit
  int total_tiles, tiles_per_cta, max_slots;
  int bitmap_words;
  float scale2;
  const float* row_lse;    // [B, Hq, W] natural log
  const uint32_t* bitmap;  // [units][bitmap_words], bit set = kept
  float* o_part;           // [virtual unit][slot][128][128]
  float* l_part;           // [virtual unit][slot][group][128]
  unsigned* status;
};

__global__ void __launch_bounds__(kThreads, 1)
calib_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                const __grid_constant__ CUtensorMap v_map, const CalibArgs a) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[26];
  __shared__ uint32_t tmem_slot;
  __shared__ Ctl ctl;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // CTAs come in groups of n_cblocks: the members of a group walk the same (kv unit, key tile)
  // range at the same pace, one calibration row block each, so that a K/V tile fetched for one
  // of them is still in L2 when the others ask for it and crosses the HBM interface once.
  const int cta = blockIdx.x / a.n_cblocks, cb = blockIdx.x % a.n_cblocks;
  const int g_begin = cta * a.tiles_per_cta;
  const int g_end = min(a.total_tiles, g_begin + a.tiles_per_cta);
  const int nt = g_end - g_begin;
  const int Hkv = a.Hq / a.G;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_base = smem_base;
  const uint32_t k_base = q_base + kTileBytes;
  const uint32_t v_base = k_base + kStages * kTileBytes;
  unsigned char* const smem_al = smem_raw + (smem_base - smem_u32(smem_raw));

  const uint32_t bar0 = smem_u32(bars);
  const uint32_t o_full = bar0, o_empty = bar0 + 8u, q_full = bar0 + 8u * 23, q_empty = bar0 + 8u * 24;
  auto full_k = [&](int s) { return bar0 + 8u * (2 + s); };
  auto full_v = [&](int s) { return bar0 + 8u * (8 + s); };
  auto s_full = [&](int b) { return bar0 + 8u * (14 + b); };
  auto p_full = [&](int b) { return bar0 + 8u * (17 + b); };
  auto buf_free = [&](int b) { return bar0 + 8u * (20 + b); };  // the P.V that read buffer b has completed

  if (tid == 0) {
    ctl.abort = 0;
    ctl.status = a.status;
    mbar_init(o_full, 1);
    mbar_init(o_empty, kGroups * 128);
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_k(s), 1);
      mbar_init(full_v(s), 1);
    }
    for (int b = 0; b < kBufs; ++b) {
      mbar_init(s_full(b), 1); mbar_init(p_full(b), 256); mbar_init(buf_free(b), 1);
    }
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  // The query block's box may cover fewer than 128 rows: clear the block once so that the rows no
  // TMA box writes hold zeros.
  for (int i = tid; i < kTileBytes / 16; i += kThreads) reinterpret_cast<uint4*>(smem_al)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  pdl_wait();   // everything above ran beside the previous kernel's end; global memory from here on

  // first tile of a run of tiles of one virtual unit inside this CTA's range
  // (the position inside the tile space is tracked incrementally: no division per tile)
  const int unit_begin = g_begin / a.n_tiles, tile_begin = g_begin - unit_begin * a.n_tiles;
  const int vu_begin = unit_begin * a.n_cblocks + cb;

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------ TMA producer of Q_c and K
    // (K and V have a producer each: a K slot frees when its S is done, a V slot only when its P.V
    // is, and one thread serving both in turn would hold every K load back behind a V slot)
    if (lane == 0) {
      tma_prefetch_desc(&q_map);
      tma_prefetch_desc(&k_map);
      int seg = 0, vu = vu_begin, tile = tile_begin, unit = unit_begin;
      for (int i = 0; i < nt; ++i, ++tile) {
        if (tile == a.n_tiles) { tile = 0; ++unit; vu += a.n_cblocks; }
        if (i == 0 || tile == 0) {
          // the Q_c block of the next virtual unit replaces the current one once its MMAs are done
          if (seg > 0 && !mbar_wait(&ctl, q_empty, (seg - 1) & 1, 20u | ((unsigned)i << 8))) break;
          const int g0 = (vu - unit * a.n_cblocks) * a.gpb;
          mbar_arrive_expect_tx(q_full, 2u * (uint32_t)(a.gpb * a.n_cal) * kLineBytes);
          for (int half = 0; half < 2; ++half)
            tma_load_4d(q_base + half * (kTileBytes / 2), &q_map, q_full, half * kHalfCols, 0, g0, unit);
          ++seg;
        }
        const int s = i % kStages;
        // slot s is free when S(i-3), which read it, is done: the barrier that hands S to the softmax group
        if (!mbar_wait(&ctl, s_full(s), ((i / kStages) & 1) ^ 1, 21u | ((unsigned)i << 8))) break;
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
      for (int i = 0; i < nt; ++i, ++tile) {
        if (tile == a.n_tiles) { tile = 0; ++unit; }
        const int s = i % kStages;
        // slot s is free when the P.V of tile i-3 is done: the barrier that frees its S/P buffer
        if (!mbar_wait(&ctl, buf_free(s), ((i / kStages) & 1) ^ 1, 22u | ((unsigned)i << 8))) break;
        mbar_arrive_expect_tx(full_v(s), kTileBytes);
        for (int half = 0; half < 2; ++half)
          tma_load_3d(v_base + s * kTileBytes + half * (kTileBytes / 2), &v_map, full_v(s), half * kHalfCols,
                      tile * kTileKeys, unit);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ issuer of the S MMAs
    // The MMAs have two issuing threads, one for S = Q_c K^T and one for O += P V.  One thread for
    // both was the bottleneck of this kernel: besides its sixteen MMAs a tile it has three waits and
    // five commits to go through, each of them some hundred cycles of dependent scalar instructions
    // for a single thread (measured: 2900 cycles a tile against 1024 of tensor-pipe time, the softmax
    // groups waiting for S half of the time).  The two chains touch different accumulators; what
    // orders them is the barriers, not the issue order.
    // S(t) goes into buffer t % 3 as soon as the P.V of tile t-3 has completed (buf_free).  S never
    // runs ahead across a change of virtual unit: its Q_c block is only loaded once the current unit's
    // S MMAs are done.
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(128, 128, false, false);     // S: A = Q_c, B = K tile, K-major
      // Descriptors are built once per buffer and a k-step adds a constant to the address field: the
      // issuing thread's own instructions between two MMAs are what limits the issue rate.
      const uint64_t dq = smem_desc_sw128(q_base, 16u, 1024u);
      const uint64_t dk0 = smem_desc_sw128(k_base, 16u, 1024u);
      // The loop is kept short on purpose: between two tiles this one thread runs dependent scalar
      // instructions at several cycles each, and whatever it spends there the tensor pipe idles.
      // b = t % 3 is the tile's buffer and its K slot, ph = (t / 3) & 1 their phase.
      int seg = 0, tile = tile_begin, b = 0;
      uint32_t ph = 0;
      bool first = true;
      for (int t = 0; t < nt; ++t) {
        if (first) {
          // new virtual unit: its Q_c block must have landed
          if (!mbar_wait(&ctl, q_full, seg & 1, 23u | ((unsigned)t << 8))) break;
          ++seg;
        }
        if (t >= kBufs && !mbar_wait(&ctl, buf_free(b), ph ^ 1u, 29u | ((unsigned)t << 8))) break;
        if (!mbar_wait(&ctl, full_k(b), ph, 24u | ((unsigned)t << 8))) break;
        tc_fence_after_sync();
        const uint32_t d = tmem_base + (uint32_t)(b * 128);
        const uint64_t kd = desc_advance(dk0, (uint32_t)b * kTileBytes);
        umma_ss_imm<0>(d, dq, kd, idesc);
#pragma unroll
        for (int kk = 1; kk < kD / 16; ++kk)
          umma_ss_imm<1>(d, desc_advance(dq, kmajor_step_bytes(kTileBytes / 2, kk)),
                         desc_advance(kd, kmajor_step_bytes(kTileBytes / 2, kk)), idesc);
        umma_commit(s_full(b));   // to the softmax group, and to the K producer: the slot is free
        ++tile;
        first = tile == a.n_tiles;
        if (first) tile = 0;
        // every S of the unit has been issued by its last tile: Q_c may be replaced once they are done
        if (first || t == nt - 1) umma_commit(q_empty);
        if (++b == kBufs) { b = 0; ph ^= 1u; }
      }
    }
  } else if (warp == kPvWarp) {
    // ------------------------------------------------------------ issuer of the P.V MMAs
    if (lane == 0) {
      const uint32_t idesc_o = umma_idesc(128, 128, false, true);    // O: A = P (TMEM), B = V tile, MN-major
      const uint32_t tmem_o = tmem_base + kColO;
      // V tile with the keys as K, i.e. MN-major: blocks of 64 head-dim elements are half a tile
      // apart, groups of 8 keys 1024 bytes apart
      const uint64_t dv0 = smem_desc_sw128(v_base, kTileBytes / 2, 1024u);
      // P.V(i): A = P in tensor memory, 16 keys = 8 columns per step
      auto pv_steps = [&](int b, auto first_tag) {
        constexpr bool kFirst = decltype(first_tag)::value;
        const uint64_t vd = desc_advance(dv0, (uint32_t)b * kTileBytes);
        const uint32_t pa = tmem_base + (uint32_t)(b * 128);
        if (kFirst) umma_ts_imm<0>(tmem_o, pa, vd, idesc_o);
        else umma_ts_imm<1>(tmem_o, pa, vd, idesc_o);
#pragma unroll
        for (int kk = 1; kk < kTileKeys / 16; ++kk)   // the P of keys 64..127 sits at columns 64..95
          umma_ts_imm<1>(tmem_o, pa + (uint32_t)((kk >> 2) * 64 + (kk & 3) * 8),
                         desc_advance(vd, (uint32_t)kk * 16u * kLineBytes), idesc_o);
      };
      int seg = 0, tile = tile_begin, b = 0;
      uint32_t ph = 0;
      bool first = true;
      for (int i = 0; i < nt; ++i) {
        if (first) {
          // O of the previous unit must have been read out before the first P.V overwrites it
          if (seg > 0 && !mbar_wait(&ctl, o_empty, (seg - 1) & 1, 25u | ((unsigned)i << 8))) break;
          ++seg;
        }
        if (!mbar_wait(&ctl, p_full(b), ph, 26u | ((unsigned)i << 8))) break;
        if (!mbar_wait(&ctl, full_v(b), ph, 27u | ((unsigned)i << 8))) break;
        tc_fence_after_sync();
        if (first) pv_steps(b, std::true_type{});
        else pv_steps(b, std::false_type{});
        umma_commit(buf_free(b));   // to the S issuer, and to the V producer: the slot is free
        ++tile;
        first = tile == a.n_tiles;
        if (first) tile = 0;
        if (first || i == nt - 1) umma_commit(o_full);
        if (++b == kBufs) { b = 0; ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax threads (one row each)
    const int grp = warp >> 2, r = tid & 127;
    const int pair = grp >> 1, half = grp & 1;
    const uint32_t lane_bits = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t lane_addr = tmem_base + lane_bits;
    float l0 = 0.f, l1 = 0.f, nlse2 = -INFINITY;
    int seg = 0;
    bool ok = true, valid = false;

    // Read out O and the row sums of the virtual unit that just ended (each group a quarter of O's
    // columns).  o_full also tells that every MMA that read Q_c or P has completed.
    auto store_partial = [&](int vu) -> bool {
      bool w = mbar_wait(&ctl, o_full, (seg - 1) & 1, 30u);
      w = __all_sync(0xffffffffu, w);
      if (!w) return false;
      tc_fence_after_sync();
      const int slot = cta - ((vu / a.n_cblocks) * a.n_tiles) / a.tiles_per_cta;
      const size_t part = (size_t)vu * a.max_slots + slot;
      float* orow = a.o_part + (part * 128 + r) * kD;
      {
        const int c0 = grp * 32;
        uint32_t ov[32];
        tmem_ld32(tmem_base + lane_bits + kColO + c0, ov);
        if (valid) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<uint4*>(orow + c0 + e) = make_uint4(ov[e], ov[e + 1], ov[e + 2], ov[e + 3]);
        }
      }
      if (valid) a.l_part[(part * kGroups + grp) * 128 + r] = l0 + l1;
      tc_fence_before_sync();
      mbar_arrive(o_empty);
      return true;
    };
    // This thread's row of the virtual unit: is there one, and its -lse2.
    auto load_q = [&](int vu) {
      const int unit = vu / a.n_cblocks, cb = vu - unit * a.n_cblocks;
      const int hq0 = (unit / Hkv) * a.Hq + (unit % Hkv) * a.G;
      const int g0 = cb * a.gpb;
      const int rows = min(a.gpb, a.G - g0) * a.n_cal;
      valid = r < rows;
      nlse2 = -INFINITY;
      if (valid) {
        const int g = g0 + r / a.n_cal, c = r - (r / a.n_cal) * a.n_cal;
        nlse2 = -a.row_lse[(size_t)(hq0 + g) * a.W + (a.W - a.n_cal + c)] * kLog2e;
      }
    };

    const uint32_t* bm_all = a.bitmap;
    const int last_word = a.bitmap_words - 1;
    // The two kept-key words of this group's 64 keys of a tile (bit set = the key does not
    // contribute) are loaded RAW one own tile ahead: nothing may touch a loaded value before the tile
    // that uses it, or the thread waits for the load on the spot.  The index is clamped so that the
    // load is always valid.
    auto load_words = [&](int unit, int tile, uint32_t (&raw)[2]) {
      const uint32_t* bm = bm_all + (size_t)unit * a.bitmap_words;
      const int w0 = tile * (kTileKeys / 32) + 2 * half;
#pragma unroll
      for (int q = 0; q < 2; ++q) raw[q] = __ldg(bm + min(w0 + q, last_word));
    };
    // keys at or beyond n_cand do not contribute either; only a unit's last tile has any
    auto tail_mask = [&](int tile, uint32_t (&w)[2]) {
      const int tbase = tile * kTileKeys + 64 * half;
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int kb = tbase + 32 * q;
        w[q] |= kb >= a.n_cand ? 0xffffffffu : (kb + 32 > a.n_cand ? 0xffffffffu << (a.n_cand - kb) : 0u);
      }
    };
    // probabilities of 32 keys -> bf16 pairs -> 16 columns at paddr.  The
    // kept-key word is the same for every row of the tile, so the test on it is uniform; most
    // words have no kept key (the kept keys are a few per cent and come in runs).
    auto soft32 = [&](uint32_t (&sv)[32], uint32_t paddr, uint32_t w) {
#pragma unroll
      for (int e = 0; e < 32; ++e)
        sv[e] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(sv[e]), a.scale2, nlse2)));
      if (w != 0u) {
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if ((w >> e) & 1u) sv[e] = 0u;
      }
      uint32_t packed[16];
#pragma unroll
      for (int e = 0; e < 32; e += 2) {
        l0 += __uint_as_float(sv[e]);
        l1 += __uint_as_float(sv[e + 1]);
        packed[e >> 1] = pack_bf16(__uint_as_float(sv[e]), __uint_as_float(sv[e + 1]));
      }
      tmem_st16(paddr, packed);
    };

    // The CTA's tile range is a sequence of segments (the tiles of one virtual unit).  Pair p takes
    // the tiles whose local index has parity p, each of its groups 64 of the tile's keys; every group
    // opens and closes every segment, also one in which its pair has no tile.  Two pairs, half a tile
    // apart, keep up to four warps per scheduler on the exponential unit: one warp per scheduler alone
    // reaches less than half of that unit's rate (measured: a group alone took 2400 cycles for the
    // 128 x 128 exponentials of a tile, 18 cycles per warp instruction against the unit's 8).
    uint32_t next_raw[2] = {0u, 0u};
    if (pair < nt) {
      int t0 = tile_begin + pair, u0 = unit_begin;
      while (t0 >= a.n_tiles) { t0 -= a.n_tiles; ++u0; }
      load_words(u0, t0, next_raw);
    }
    int seg_first = 0, seg_tile0 = tile_begin, seg_unit = unit_begin, seg_vu = vu_begin;
    while (seg_first < nt) {
      const int seg_end = seg_first + min(nt - seg_first, a.n_tiles - seg_tile0);
      l0 = l1 = 0.f;
      load_q(seg_vu);
      ++seg;
#pragma unroll 1
      for (int i = seg_first + ((seg_first ^ pair) & 1); i < seg_end; i += 2) {
        const int tile = seg_tile0 + (i - seg_first);
        uint32_t word[2] = {next_raw[0], next_raw[1]};
        if (i + 2 < nt) {
          int t2 = tile + 2, u2 = seg_unit;
          while (t2 >= a.n_tiles) { t2 -= a.n_tiles; ++u2; }
          load_words(u2, t2, next_raw);
        }
        if (tile == a.n_tiles - 1) tail_mask(tile, word);
        const int b = i % kBufs;
        // S(i) of this group's keys; their P goes to the first 32 of the same 64 columns, which this
        // group alone reads, each 16 columns only after the S they held is in registers
        const uint32_t taddr = lane_addr + (uint32_t)(b * 128 + half * 64);
        ok = mbar_wait(&ctl, s_full(b), (i / kBufs) & 1, 28u | ((unsigned)i << 8));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        uint32_t ra[32], rb[32];
        tmem_ld32_issue(taddr, ra);
        tmem_ld_wait(ra);
        tmem_ld32_issue(taddr + 32, rb);   // arrives while the first 32 keys are worked on
        soft32(ra, taddr, word[0]);
        tmem_ld_wait(rb);
        soft32(rb, taddr + 16, word[1]);
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive(p_full(b));
      }
      if (!ok) break;
      ok = store_partial(seg_vu);
      if (!ok) break;
      seg_first = seg_end;
      seg_tile0 = 0;
      ++seg_unit;
      seg_vu += a.n_cblocks;
    }
  }

  // ---------------------------------------------------------------- teardown (every path)
  if (ctl.abort) {
    for (int i = 0; i < 50; ++i) __nanosleep(20000);  // let TMA copies still in flight land
  }
  tc_fence_before_sync();
  __syncthreads();
  pdl_trigger();   // every warp is done: the next kernel's CTAs may set themselves up while this one winds down
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

// One warp per (batch, query head, calibration row): sum the partials of the CTAs that shared the
// row's virtual unit, in order, then O_c = O / l, LSE_c = lse + log l (zeros and -inf when nothing
// was evicted), C_q = the query.  The blocks beyond the reduction's compact the retained rows.
__global__ void __launch_bounds__(256)
calib_reduce_kernel(const __nv_bfloat16* __restrict__ Q_obs, const float* __restrict__ row_lse,
                    const float* __restrict__ o_part, const float* __restrict__ l_part,
                    float* __restrict__ O_c, float* __restrict__ LSE_c, __nv_bfloat16* __restrict__ C_q, int B,
                    int Hq, int G, int W, int n_cal, int gpb, int n_cblocks, int n_tiles, int tiles_per_cta,
                    int max_slots, int reduce_blocks, const GatherArgs gather) {
  pdl_trigger();
  pdl_wait();
  if ((int)blockIdx.x >= reduce_blocks) {
    const int gb = (int)blockIdx.x - reduce_blocks, per_unit = (gather.n_rows + 15) / 16;
    gather_rows16(gather, gb % per_unit, gb / per_unit, threadIdx.x);
    return;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.x * 8 + warp;  // (b, hq, c)
  if (row >= B * Hq * n_cal) return;
  const int c = row % n_cal, bhq = row / n_cal;
  const int b = bhq / Hq, hq = bhq % Hq;
  const int Hkv = Hq / G, h = hq / G, g = hq % G;
  const int unit = b * Hkv + h, cb = g / gpb, r = (g % gpb) * n_cal + c;
  const int vu = unit * n_cblocks + cb;
  const int first = (unit * n_tiles) / tiles_per_cta, last = ((unit + 1) * n_tiles - 1) / tiles_per_cta;
  const size_t part0 = (size_t)vu * max_slots;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float l = 0.f;
  for (int s = 0; s <= last - first; ++s) {
    const float4 v = *reinterpret_cast<const float4*>(o_part + ((part0 + s) * 128 + r) * kD + 4 * lane);
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    for (int grp = 0; grp < kGroups; ++grp) l += l_part[((part0 + s) * kGroups + grp) * 128 + r];
  }
  const int qrow = W - n_cal + c;
  float4 out = make_float4(0.f, 0.f, 0.f, 0.f);
  float lse = -INFINITY;
  if (l > 0.f) {
    const float inv = 1.f / l;
    out = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    lse = row_lse[(size_t)bhq * W + qrow] + logf(l);
  }
  reinterpret_cast<float4*>(O_c + (size_t)row * kD)[lane] = out;
  if (lane == 0) LSE_c[row] = lse;
  reinterpret_cast<uint2*>(C_q + (size_t)row * kD)[lane] =
      reinterpret_cast<const uint2*>(Q_obs + ((size_t)bhq * W + qrow) * kD)[lane];
}

}  // namespace

bool calib_tc_supported(const CompressGeom& g) { return !g.keep_all && g.n_cal <= 128 && g.n_cand >= 1; }

// Row blocks per unit and the tile partition; `parts` = partial (O, l) slots the workspace holds.
void calib_tc_plan(const CompressGeom& g, int* gpb, int* n_cblocks, int* tiles_per_cta, int* max_slots,
                   size_t* parts) {
  int per = 128 / g.n_cal;
  if (per < 1) per = 1;
  if (per > g.G) per = g.G;
  *gpb = per;
  *n_cblocks = (g.G + per - 1) / per;
  const int n_tiles = (g.n_cand + kTileKeys - 1) / kTileKeys;
  // the (kv unit, tile) space is shared out over groups of n_cblocks CTAs
  const int total = g.units * n_tiles;
  int groups = kSms / *n_cblocks;
  if (groups < 1) groups = 1;
  if (groups > total) groups = total;
  *tiles_per_cta = (total + groups - 1) / groups;
  *max_slots = (n_tiles + *tiles_per_cta - 1) / *tiles_per_cta + 1;
  *parts = (size_t)g.units * *n_cblocks * *max_slots;
}

cudaError_t launch_calib_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                            const void* V, const float* row_lse, char* wsp, float* O_c, float* LSE_c, void* C_q,
                            const GatherArgs& gather, cudaStream_t st) {
  CalibArgs a{};
  a.Hq = g.Hq; a.G = g.G; a.W = g.W; a.L = g.L; a.n_cand = g.n_cand; a.n_cal = g.n_cal;
  size_t parts;
  calib_tc_plan(g, &a.gpb, &a.n_cblocks, &a.tiles_per_cta, &a.max_slots, &parts);
  a.n_tiles = (g.n_cand + kTileKeys - 1) / kTileKeys;
  a.total_tiles = g.units * a.n_tiles;
  a.bitmap_words = g.bitmap_words;
  a.scale2 = g.scale2;
  a.row_lse = row_lse;
  a.bitmap = (const uint32_t*)(wsp + ws.calib_mask);
  a.o_part = (float*)(wsp + ws.calib_o);
  a.l_part = (float*)(wsp + ws.calib_l);
  a.status = (unsigned*)(wsp + ws.status);
  CUtensorMap qm, km, vm;
  // calibration rows: [head dim][c < n_cal][g < G][unit], starting at observation row W - n_cal
  const uint64_t qd[3] = {(uint64_t)g.n_cal, (uint64_t)g.G, (uint64_t)g.units};
  const uint64_t qs[3] = {256, (uint64_t)g.W * 256, (uint64_t)g.G * g.W * 256};
  const uint32_t qb[3] = {(uint32_t)g.n_cal, (uint32_t)a.gpb, 1};
  const char* q0 = (const char*)Q_obs + (size_t)(g.W - g.n_cal) * 256;
  if (!make_tensor_map_bf16(&qm, q0, 4, qd, qs, qb)) return cudaErrorInvalidValue;
  const uint64_t kd[2] = {(uint64_t)g.L, (uint64_t)g.units}, ks[2] = {256, (uint64_t)g.L * 256};
  const uint32_t kb[2] = {(uint32_t)kTileKeys, 1};
  if (!make_tensor_map_bf16(&km, K, 3, kd, ks, kb) || !make_tensor_map_bf16(&vm, V, 3, kd, ks, kb))
    return cudaErrorInvalidValue;
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(calib_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  const int grid = (a.total_tiles + a.tiles_per_cta - 1) / a.tiles_per_cta * a.n_cblocks;
  e = launch_pdl(calib_tc_kernel, dim3(grid), dim3(kThreads), (size_t)kSmemBytes, st, qm, km, vm, a);
  if (e != cudaSuccess) return e;
  const int total = g.B * g.Hq * g.n_cal;
  const int reduce_blocks = (total + 7) / 8;
  const int gather_blocks = gather.idx ? gather.units * ((gather.n_rows + 15) / 16) : 0;
  e = launch_pdl(calib_reduce_kernel, dim3(reduce_blocks + gather_blocks), dim3(256), 0, st,
                 (const __nv_bfloat16*)Q_obs, row_lse, (const float*)a.o_part, (const float*)a.l_part, O_c, LSE_c,
                 (__nv_bfloat16*)C_q, g.B, g.Hq, g.G, g.W, g.n_cal, a.gpb, a.n_cblocks, a.n_tiles, a.tiles_per_cta,
                 a.max_slots, reduce_blocks, gather);
  if (e != cudaSuccess) return e;
  count_launch(2);
  return cudaGetLastError();
}

}  // namespace calidrop
