// Calibration term on the tensor cores (Algorithm 1, lines 5-8): for every calibration query
// row, the softmax-weighted sum of the EVICTED values and the log of its normaliser.
//
// A CTA owns one (batch, kv-head) unit, one block of up to 128 calibration rows (whole query
// heads, n_cal rows each) and a contiguous range of 128-key tiles.  Per tile:
//     MMA 1   S = Q_c K^T                (query rows on the TMEM lanes, K tile from TMA)
//     threads p = exp2(scale2 * s - lse2[row]), zero for kept keys (bitmap) and for keys outside
//             the candidates; row sums l kept in fp32; p rounded to bf16 into shared memory in the
//             K-major operand layout
//     MMA 2   O += P V                   (V tile from TMA, read as the MN-major B operand)
// lse2[row] is the row's LSE over ALL the keys it sees (from the statistics pass or the caller), so
// every p <= 1 and no running maximum or rescaling is needed: the partial (O, l) of the key
// ranges simply add up.  calib_reduce_kernel sums them in a fixed order and writes
// O_c = O / l, LSE_c = lse + log l, C_q.
// Warp roles as in the scoring kernels: warps 0-3 softmax, warp 4 TMA producer, warp 5 MMA issuer.
#include "internal.h"
#include "tc_common.cuh"

namespace calidrop {

namespace {

using namespace tc;

constexpr int kGroups = 2;  // softmax warpgroups; group g owns S buffer g and P buffer g (tiles i % 2 == g)
constexpr int kProducerWarp = kGroups * 4;
constexpr int kMmaWarp = kGroups * 4 + 1;
constexpr int kThreads = kGroups * 128 + 64;
constexpr int kTmemCols = 512;
constexpr int kTileBytes = kKvTileBytes;  // 32 KB: Q block, K tile, V tile and P tile alike
constexpr int kSmemBytes = 7 * kTileBytes + 1024;

struct CalibArgs {
  int Hq, G, W, L, n_cand, n_cal;
  int gpb;        // query heads per row block
  int n_cblocks;  // row blocks per unit
  int n_tiles, n_splits;
  int bitmap_words;
  float scale2;
  const float* row_lse;    // [B, Hq, W] natural log
  const uint32_t* bitmap;  // [units][bitmap_words], bit set = kept
  float* o_part;           // [unit][block][split][128][128]
  float* l_part;           // [unit][block][split][group][128]
  unsigned* status;
};

__global__ void __launch_bounds__(kThreads, 1)
calib_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                const __grid_constant__ CUtensorMap v_map, const CalibArgs a) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[20];
  __shared__ uint32_t tmem_slot;
  __shared__ Ctl ctl;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, cb = blockIdx.y, unit = blockIdx.z;
  const int tile0 = (int)((long long)a.n_tiles * split / a.n_splits);
  const int tile1 = (int)((long long)a.n_tiles * (split + 1) / a.n_splits);
  const int nt = tile1 - tile0;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_base = smem_base;
  const uint32_t k_base = q_base + kTileBytes;
  const uint32_t v_base = k_base + 2 * kTileBytes;
  const uint32_t p_base = v_base + 2 * kTileBytes;
  unsigned char* const smem_al = smem_raw + (smem_base - smem_u32(smem_raw));

  const uint32_t bar0 = smem_u32(bars);
  const uint32_t q_full = bar0, o_full = bar0 + 8u;
  auto full_k = [&](int s) { return bar0 + 8u * (2 + s); };
  auto empty_k = [&](int s) { return bar0 + 8u * (4 + s); };
  auto full_v = [&](int s) { return bar0 + 8u * (6 + s); };
  auto empty_v = [&](int s) { return bar0 + 8u * (8 + s); };
  auto s_full = [&](int s) { return bar0 + 8u * (10 + s); };
  auto s_empty = [&](int s) { return bar0 + 8u * (12 + s); };
  auto p_full = [&](int s) { return bar0 + 8u * (14 + s); };
  auto p_empty = [&](int s) { return bar0 + 8u * (16 + s); };

  if (tid == 0) {
    ctl.abort = 0;
    ctl.status = a.status;
    mbar_init(q_full, 1);
    mbar_init(o_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(full_k(s), 1); mbar_init(empty_k(s), 1);
      mbar_init(full_v(s), 1); mbar_init(empty_v(s), 1);
      mbar_init(s_full(s), 1); mbar_init(s_empty(s), 128);
      mbar_init(p_full(s), 128); mbar_init(p_empty(s), 1);
    }
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  // The query block's box may cover fewer than 128 rows: clear the block first so that the rows
  // the TMA does not write hold zeros.
  if (warp < 4) {
    uint4* qz = reinterpret_cast<uint4*>(smem_al);
    for (int i = tid; i < kTileBytes / 16; i += 128) qz[i] = make_uint4(0u, 0u, 0u, 0u);
    // (only the first warpgroup clears; the barrier below orders it before the TMA)
    fence_proxy_async_smem();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  const uint32_t tmem_o = tmem_base + 256u;

  const int Hkv = a.Hq / a.G;
  const int hq0 = (unit / Hkv) * a.Hq + (unit % Hkv) * a.G;
  const int g0 = cb * a.gpb;
  const int ng = min(a.gpb, a.G - g0);
  const int rows = ng * a.n_cal;  // valid rows of this block

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&q_map);
      tma_prefetch_desc(&k_map);
      tma_prefetch_desc(&v_map);
      const uint32_t q_half = (uint32_t)(a.gpb * a.n_cal) * kLineBytes;  // bytes one box writes
      mbar_arrive_expect_tx(q_full, 2u * q_half);
      for (int half = 0; half < 2; ++half)
        tma_load_4d(q_base + half * (kTileBytes / 2), &q_map, q_full, half * kHalfCols, 0, g0, unit);
      for (int i = 0; i < nt; ++i) {
        const int s = i & 1;
        const uint32_t ph = ((i >> 1) & 1) ^ 1;
        if (!mbar_wait(&ctl, empty_k(s), ph, 21u)) break;
        mbar_arrive_expect_tx(full_k(s), kTileBytes);
        for (int half = 0; half < 2; ++half)
          tma_load_3d(k_base + s * kTileBytes + half * (kTileBytes / 2), &k_map, full_k(s), half * kHalfCols,
                      (tile0 + i) * kTileKeys, unit);
        if (!mbar_wait(&ctl, empty_v(s), ph, 22u)) break;
        mbar_arrive_expect_tx(full_v(s), kTileBytes);
        for (int half = 0; half < 2; ++half)
          tma_load_3d(v_base + s * kTileBytes + half * (kTileBytes / 2), &v_map, full_v(s), half * kHalfCols,
                      (tile0 + i) * kTileKeys, unit);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = umma_idesc(128, 128, false, false);
      const uint32_t idesc_o = umma_idesc(128, 128, false, true);
      bool ok = mbar_wait(&ctl, q_full, 0, 23u);
      auto issue_s = [&](int i) -> bool {
        const int s = i & 1;
        const uint32_t ph = (i >> 1) & 1;
        if (!mbar_wait(&ctl, full_k(s), ph, 24u)) return false;
        if (!mbar_wait(&ctl, s_empty(s), ph ^ 1, 25u)) return false;
        tc_fence_after_sync();
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk)
          umma_ss(tmem_base + (uint32_t)(s * 128), kmajor_desc(q_base, kTileBytes / 2, kk),
                  kmajor_desc(k_base + s * kTileBytes, kTileBytes / 2, kk), idesc_s, kk > 0 ? 1u : 0u);
        umma_commit(s_full(s));
        umma_commit(empty_k(s));
        return true;
      };
      if (ok && nt > 0) ok = issue_s(0);
      for (int i = 0; ok && i < nt; ++i) {
        if (i + 1 < nt && !issue_s(i + 1)) { ok = false; break; }
        const int s = i & 1;
        const uint32_t ph = (i >> 1) & 1;
        if (!mbar_wait(&ctl, p_full(s), ph, 26u)) { ok = false; break; }
        if (!mbar_wait(&ctl, full_v(s), ph, 27u)) { ok = false; break; }
        tc_fence_after_sync();
#pragma unroll
        for (int kk = 0; kk < kTileKeys / 16; ++kk) {
          // A: P tile, K-major over the keys; B: V tile with the keys as K, i.e. MN-major: blocks of
          // 64 head-dim elements are half a tile apart, groups of 8 keys 1024 bytes apart.
          const uint64_t pd = kmajor_desc(p_base + s * kTileBytes, kTileBytes / 2, kk);
          const uint64_t vd = smem_desc_sw128(v_base + s * kTileBytes + (uint32_t)kk * 16u * kLineBytes,
                                              kTileBytes / 2, 1024u);
          umma_ss(tmem_o, pd, vd, idesc_o, (i > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(p_empty(s));
        umma_commit(empty_v(s));
      }
      if (ok) umma_commit(o_full);
    }
  } else {
    // ------------------------------------------------------------ softmax threads (one row each)
    const int grp = warp >> 2, r = tid & 127;
    const bool valid = r < rows;
    float nlse2 = -INFINITY;
    if (valid) {
      const int g = g0 + r / a.n_cal, c = r - (r / a.n_cal) * a.n_cal;
      nlse2 = -a.row_lse[(size_t)(hq0 + g) * a.W + (a.W - a.n_cal + c)] * kLog2e;
    }
    const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t* bm = a.bitmap + (size_t)unit * a.bitmap_words;
    float l0 = 0.f, l1 = 0.f;
    bool ok = true;
    for (int i = grp; i < nt; i += kGroups) {
      const int s = i & 1;  // == grp
      const uint32_t ph = (i >> 1) & 1;
      ok = mbar_wait(&ctl, s_full(s), ph, 28u) && mbar_wait(&ctl, p_empty(s), ph ^ 1, 29u);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const int tbase = (tile0 + i) * kTileKeys;
      const uint32_t p_row = p_base + s * kTileBytes + (uint32_t)r * kLineBytes;
      const uint32_t taddr = lane_addr + (uint32_t)(s * 128);
      // probabilities of 32 keys -> bf16 -> the P tile (K-major, 128-byte swizzle)
      auto soft32 = [&](const uint32_t (&sv)[32], int q4) {
        const int kbase = tbase + 32 * q4;
        uint32_t word = 0xffffffffu;  // bit set = this key does not contribute
        if (kbase < a.n_cand) {
          word = __ldg(bm + (kbase >> 5));
          if (kbase + 32 > a.n_cand) word |= 0xffffffffu << (a.n_cand - kbase);
        }
        uint32_t packed[16];
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float p0 = ex2_approx(fmaf(__uint_as_float(sv[e]), a.scale2, nlse2));
          float p1 = ex2_approx(fmaf(__uint_as_float(sv[e + 1]), a.scale2, nlse2));
          if ((word >> e) & 1u) p0 = 0.f;
          if ((word >> (e + 1)) & 1u) p1 = 0.f;
          l0 += p0;
          l1 += p1;
          packed[e >> 1] = pack_bf16(p0, p1);
        }
        const uint32_t half_off = (uint32_t)(q4 >> 1) * (kTileBytes / 2);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint32_t chunk = (uint32_t)((q4 & 1) * 4 + v) ^ (uint32_t)(r & 7);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(p_row + half_off + (chunk << 4)),
                       "r"(packed[4 * v]), "r"(packed[4 * v + 1]), "r"(packed[4 * v + 2]), "r"(packed[4 * v + 3])
                       : "memory");
        }
      };
      uint32_t ra[32], rb[32];
      tmem_ld32_issue(taddr, ra);
      tmem_ld_wait(ra);
      tmem_ld32_issue(taddr + 32, rb);
      soft32(ra, 0);
      tmem_ld_wait(rb);
      tmem_ld32_issue(taddr + 64, ra);
      soft32(rb, 1);
      tmem_ld_wait(ra);
      tmem_ld32_issue(taddr + 96, rb);
      soft32(ra, 2);
      tmem_ld_wait(rb);
      tc_fence_before_sync();
      mbar_arrive(s_empty(s));  // the logits are in registers: the next S tile may be issued
      soft32(rb, 3);
      fence_proxy_async_smem();
      mbar_arrive(p_full(s));
    }
    // epilogue: the accumulated O rows (each group stores half of the columns) and the row sums
    if (ok) {
      ok = nt == 0 || mbar_wait(&ctl, o_full, 0, 30u);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after_sync();
      const size_t part = ((size_t)unit * a.n_cblocks + cb) * a.n_splits + split;
      float* orow = a.o_part + (part * 128 + r) * kD;
#pragma unroll 1
      for (int c0 = grp * (kD / kGroups); c0 < (grp + 1) * (kD / kGroups); c0 += 32) {
        uint32_t ov[32];
        if (nt > 0) {
          tmem_ld32(tmem_o + ((uint32_t)((warp & 3) * 32) << 16) + c0, ov);
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) ov[e] = 0u;
        }
        if (valid) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<uint4*>(orow + c0 + e) = make_uint4(ov[e], ov[e + 1], ov[e + 2], ov[e + 3]);
        }
      }
      if (valid) a.l_part[(part * kGroups + grp) * 128 + r] = l0 + l1;
    }
  }

  // ---------------------------------------------------------------- teardown (every path)
  if (ctl.abort) {
    for (int i = 0; i < 50; ++i) __nanosleep(20000);  // let TMA copies still in flight land
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

// One warp per (batch, query head, calibration row): sum the key-range partials in order, then
// O_c = O / l, LSE_c = lse + log l (zeros and -inf when nothing was evicted), C_q = the query.
__global__ void __launch_bounds__(128)
calib_reduce_kernel(const __nv_bfloat16* __restrict__ Q_obs, const float* __restrict__ row_lse,
                    const float* __restrict__ o_part, const float* __restrict__ l_part,
                    float* __restrict__ O_c, float* __restrict__ LSE_c, __nv_bfloat16* __restrict__ C_q, int B,
                    int Hq, int G, int W, int n_cal, int gpb, int n_cblocks, int n_splits) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.x * 4 + warp;  // (b, hq, c)
  if (row >= B * Hq * n_cal) return;
  const int c = row % n_cal, bhq = row / n_cal;
  const int b = bhq / Hq, hq = bhq % Hq;
  const int Hkv = Hq / G, h = hq / G, g = hq % G;
  const int unit = b * Hkv + h, cb = g / gpb, r = (g % gpb) * n_cal + c;
  const size_t part0 = ((size_t)unit * n_cblocks + cb) * n_splits;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float l = 0.f;
  for (int s = 0; s < n_splits; ++s) {
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

void calib_tc_plan(const CompressGeom& g, int* gpb, int* n_cblocks, int* n_splits) {
  int per = 128 / g.n_cal;
  if (per < 1) per = 1;
  if (per > g.G) per = g.G;
  *gpb = per;
  *n_cblocks = (g.G + per - 1) / per;
  const int n_tiles = (g.n_cand + kTileKeys - 1) / kTileKeys;
  const int groups = g.units * *n_cblocks;
  int s = pick_tile_splits(groups, n_tiles, 4);
  const int cap = 592 / groups > 1 ? 592 / groups : 1;  // bounds the partial buffers
  if (s > cap) s = cap;
  *n_splits = s;
}

cudaError_t launch_calib_tc(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                            const void* V, const float* row_lse, char* wsp, float* O_c, float* LSE_c, void* C_q,
                            cudaStream_t st) {
  CalibArgs a{};
  a.Hq = g.Hq; a.G = g.G; a.W = g.W; a.L = g.L; a.n_cand = g.n_cand; a.n_cal = g.n_cal;
  calib_tc_plan(g, &a.gpb, &a.n_cblocks, &a.n_splits);
  a.n_tiles = (g.n_cand + kTileKeys - 1) / kTileKeys;
  a.bitmap_words = g.bitmap_words;
  a.scale2 = g.scale2;
  a.row_lse = row_lse;
  a.bitmap = (const uint32_t*)(wsp + ws.bitmap);
  a.o_part = (float*)(wsp + ws.calib_o);
  a.l_part = (float*)(wsp + ws.calib_l);
  a.status = (unsigned*)(wsp + ws.status);
  CUtensorMap qm, km, vm;
  // calibration rows: [head dim][c < n_cal][g < G][unit], starting at observation row W - n_cal
  const uint64_t qd[3] = {(uint64_t)g.n_cal, (uint64_t)g.G, (uint64_t)g.units};
  const uint64_t qs[3] = {256, (uint64_t)g.W * 256, (uint64_t)g.G * g.W * 256};
  const uint32_t qb[3] = {(uint32_t)g.n_cal, (uint32_t)a.gpb, 1};
  const char* q0 = (const char*)Q_obs + (size_t)(g.W - g.n_cal) * 256;
  const uint64_t kd[2] = {(uint64_t)g.L, (uint64_t)g.units}, ks[2] = {256, (uint64_t)g.L * 256};
  const uint32_t kb[2] = {(uint32_t)kTileKeys, 1};
  if (!make_tensor_map_bf16(&qm, q0, 4, qd, qs, qb) || !make_tensor_map_bf16(&km, K, 3, kd, ks, kb) ||
      !make_tensor_map_bf16(&vm, V, 3, kd, ks, kb))
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
  calib_tc_kernel<<<dim3(a.n_splits, a.n_cblocks, g.units), kThreads, kSmemBytes, st>>>(qm, km, vm, a);
  const int total = g.B * g.Hq * g.n_cal;
  calib_reduce_kernel<<<(total + 3) / 4, 128, 0, st>>>((const __nv_bfloat16*)Q_obs, row_lse, a.o_part, a.l_part, O_c,
                                                      LSE_c, (__nv_bfloat16*)C_q, g.B, g.Hq, g.G, g.W, g.n_cal,
                                                      a.gpb, a.n_cblocks, a.n_splits);
  count_launch(2);
  return cudaGetLastError();
}

}  // namespace calidrop
