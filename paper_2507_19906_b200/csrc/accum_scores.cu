// Accumulated attention scores of a prompt, the importance measure of the H2O eviction rule
// (Sections 4.1.2-4.1.3 apply the calibration on top of it): for every (batch, kv head) and every
// key t, the causal softmax attention that key receives, summed over the prompt's queries i >= t and
// over the query heads of the group.  Serving code gets these sums as a by-product of the prefill
// attention; this file computes them from Q and K for callers that have none, in two passes of
// 64 x 64 tiles on the warp-level tensor-core path (bf16 products, fp32 logits, statistics and sums):
//   pass 1  row statistics: lse2[b, hq, i] = log2 sum_{t <= i} exp2(s2[i, t]),  s2 = q.k * scale * log2(e)
//   pass 2  column sums:    score[b, h, t] = sum_{g < G} sum_{i >= t} exp2(s2[i, t] - lse2[i])
// Every key's sum is accumulated by one thread quad in a fixed order (no atomics), so the result is
// reproducible bit for bit.  The cost is that of the prefill attention itself (L^2 D flop per head),
// which is why it is not part of the compress step.
#include "common.cuh"
#include "internal.h"

namespace calidrop {

namespace {

constexpr int kTile = 64;          // queries and keys per tile
constexpr int kRowElems = kD + 8;  // padded shared-memory row (272 bytes): conflict-free 8 x 16-byte reads
constexpr int kThreads = 128;      // four warps, 16 tile rows each

// rows [row0, row0 + 64) of a [n_rows, 128] bf16 matrix into a padded tile; rows beyond n_rows are zeros
__device__ __forceinline__ void load_tile(__nv_bfloat16 (*dst)[kRowElems], const __nv_bfloat16* src, int row0,
                                          int n_rows, int tid) {
  for (int c = tid; c < kTile * 16; c += kThreads) {
    const int r = c >> 4, ch = c & 15;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + r < n_rows) v = __ldg(reinterpret_cast<const uint4*>(src + (size_t)(row0 + r) * kD) + ch);
    *reinterpret_cast<uint4*>(&dst[r][ch * 8]) = v;
  }
}

// A fragments (16 rows x 128) of the warp's rows of a tile: eight k-steps of four registers
__device__ __forceinline__ void load_a_frags(uint32_t (&a)[8][4], __nv_bfloat16 (*tile)[kRowElems], int warp, int lane) {
#pragma unroll
  for (int kk = 0; kk < 8; ++kk)
    ldmatrix_x4(smem_u32(&tile[warp * 16 + (lane & 15)][kk * 16 + (lane >> 4) * 8]), a[kk][0], a[kk][1], a[kk][2],
                a[kk][3]);
}

// C[16 x 64] = A[16 x 128] . T[64 x 128]^T for the rows of tile T as columns: eight 8-column blocks
__device__ __forceinline__ void tile_product(float (&c)[8][4], const uint32_t (&a)[8][4],
                                             __nv_bfloat16 (*tile)[kRowElems], int lane) {
#pragma unroll
  for (int n = 0; n < 8; ++n) c[n][0] = c[n][1] = c[n][2] = c[n][3] = 0.f;
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
    for (int n2 = 0; n2 < 4; ++n2) {
      // four 8 x 8 blocks: columns n2*16 .. +7 at k and k + 8, columns n2*16 + 8 .. +15 at k and k + 8
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4(smem_u32(&tile[n2 * 16 + (lane & 7) + ((lane >> 4) << 3)][kk * 16 + ((lane >> 3) & 1) * 8]), b0, b1,
                  b2, b3);
      mma_bf16_16816(c[2 * n2], a[kk][0], a[kk][1], a[kk][2], a[kk][3], b0, b1);
      mma_bf16_16816(c[2 * n2 + 1], a[kk][0], a[kk][1], a[kk][2], a[kk][3], b2, b3);
    }
  }
}

// pass 1: one CTA per (64-query block, batch * query head)
__global__ void __launch_bounds__(kThreads)
accum_row_lse_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                     float* __restrict__ lse2, int Hq, int G, int L, float scale2) {
  __shared__ __align__(16) __nv_bfloat16 qs[kTile][kRowElems];
  __shared__ __align__(16) __nv_bfloat16 ks[kTile][kRowElems];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, tq = lane & 3;
  const int bhq = blockIdx.y, b = bhq / Hq, hq = bhq % Hq, Hkv = Hq / G;
  const int q0 = blockIdx.x * kTile;
  const __nv_bfloat16* Qh = Q + (size_t)bhq * L * kD;
  const __nv_bfloat16* Kh = K + (size_t)(b * Hkv + hq / G) * L * kD;
  load_tile(qs, Qh, q0, L, tid);
  __syncthreads();
  uint32_t a[8][4];
  load_a_frags(a, qs, warp, lane);
  const int i0 = q0 + warp * 16 + gq, i1 = i0 + 8;  // this thread's two query rows
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  for (int k0 = 0; k0 <= q0 && k0 < L; k0 += kTile) {  // key tiles up to the diagonal one
    __syncthreads();
    load_tile(ks, Kh, k0, L, tid);
    __syncthreads();
    float c[8][4];
    tile_product(c, a, ks, lane);
    float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int t = k0 + n * 8 + 2 * tq + e;
        c[n][e] = (t <= i0 && t < L) ? c[n][e] * scale2 : -INFINITY;
        c[n][2 + e] = (t <= i1 && t < L) ? c[n][2 + e] * scale2 : -INFINITY;
        bm0 = fmaxf(bm0, c[n][e]);
        bm1 = fmaxf(bm1, c[n][2 + e]);
      }
    }
    bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 1)); bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 2));
    bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 1)); bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 2));
    const float n0 = fmaxf(m0, bm0), n1 = fmaxf(m1, bm1);
    float s0 = 0.f, s1 = 0.f;
    if (n0 > -INFINITY) {
#pragma unroll
      for (int n = 0; n < 8; ++n) s0 += ex2_approx(c[n][0] - n0) + ex2_approx(c[n][1] - n0);
      l0 = l0 * ex2_approx(m0 - n0) + s0;
      m0 = n0;
    }
    if (n1 > -INFINITY) {
#pragma unroll
      for (int n = 0; n < 8; ++n) s1 += ex2_approx(c[n][2] - n1) + ex2_approx(c[n][3] - n1);
      l1 = l1 * ex2_approx(m1 - n1) + s1;
      m1 = n1;
    }
  }
  // the four threads of a quad hold partial sums over their columns, all referred to the same maximum
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  if (tq == 0) {
    if (i0 < L) lse2[(size_t)bhq * L + i0] = m0 + log2f(l0);
    if (i1 < L) lse2[(size_t)bhq * L + i1] = m1 + log2f(l1);
  }
}

// pass 2: one CTA per (64-key tile, batch * kv head)
__global__ void __launch_bounds__(kThreads)
accum_col_sum_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                     const float* __restrict__ lse2, float* __restrict__ scores, int Hq, int G, int L,
                     float scale2) {
  __shared__ __align__(16) __nv_bfloat16 ks[kTile][kRowElems];
  __shared__ __align__(16) __nv_bfloat16 qs[kTile][kRowElems];
  __shared__ float ls[kTile];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, tq = lane & 3;
  const int unit = blockIdx.y, Hkv = Hq / G, b = unit / Hkv, h = unit % Hkv;
  const int k0 = blockIdx.x * kTile;
  load_tile(ks, K + (size_t)unit * L * kD, k0, L, tid);
  __syncthreads();
  uint32_t a[8][4];  // the warp's 16 keys as the rows of the product
  load_a_frags(a, ks, warp, lane);
  const int t0 = k0 + warp * 16 + gq, t1 = t0 + 8;  // this thread's two keys
  float acc0 = 0.f, acc1 = 0.f;
  for (int g = 0; g < G; ++g) {
    const int bhq = b * Hq + h * G + g;
    const __nv_bfloat16* Qh = Q + (size_t)bhq * L * kD;
    for (int q0 = k0; q0 < L; q0 += kTile) {  // query tiles from the diagonal one on
      __syncthreads();
      load_tile(qs, Qh, q0, L, tid);
      if (tid < kTile) ls[tid] = q0 + tid < L ? lse2[(size_t)bhq * L + q0 + tid] : INFINITY;
      __syncthreads();
      float c[8][4];
      tile_product(c, a, qs, lane);
#pragma unroll
      for (int n = 0; n < 8; ++n) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int col = n * 8 + 2 * tq + e, i = q0 + col;  // query i; rows beyond L have lse2 = +inf: p = 0
          const float lq = ls[col];
          if (i >= t0) acc0 += ex2_approx(c[n][e] * scale2 - lq);
          if (i >= t1) acc1 += ex2_approx(c[n][2 + e] * scale2 - lq);
        }
      }
    }
  }
  acc0 += __shfl_xor_sync(0xffffffffu, acc0, 1); acc0 += __shfl_xor_sync(0xffffffffu, acc0, 2);
  acc1 += __shfl_xor_sync(0xffffffffu, acc1, 1); acc1 += __shfl_xor_sync(0xffffffffu, acc1, 2);
  if (tq == 0) {
    if (t0 < L) scores[(size_t)unit * L + t0] = acc0;
    if (t1 < L) scores[(size_t)unit * L + t1] = acc1;
  }
}

}  // namespace

cudaError_t launch_accum_scores(int B, int Hq, int Hkv, int L, float scale2, const void* Q_full, const void* K,
                                float* lse2, float* scores, cudaStream_t st) {
  const int tiles = (L + kTile - 1) / kTile, G = Hq / Hkv;
  accum_row_lse_kernel<<<dim3(tiles, B * Hq), kThreads, 0, st>>>((const __nv_bfloat16*)Q_full, (const __nv_bfloat16*)K,
                                                                 lse2, Hq, G, L, scale2);
  accum_col_sum_kernel<<<dim3(tiles, B * Hkv), kThreads, 0, st>>>((const __nv_bfloat16*)Q_full,
                                                                  (const __nv_bfloat16*)K, lse2, scores, Hq, G, L,
                                                                  scale2);
  count_launch(2);
  return cudaGetLastError();
}

}  // namespace calidrop
