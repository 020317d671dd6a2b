// Scalar (CUDA-core) kernels of the compress-and-calibrate step:
//   * window scoring (softmax statistics of the observation rows, then the per-key votes),
//   * the direct evaluation of the calibration term over the evicted rows.
// One thread owns one key row in registers and walks the observation queries staged in
// shared memory, so every K row is read once per pass.
#include "common.cuh"
#include "internal.h"

namespace calidrop {

namespace {

constexpr int kTile = 128;     // keys per CTA (one per thread)
constexpr int kRowChunk = 32;  // observation rows staged in shared memory at a time

__device__ __forceinline__ void load_key_row(const __nv_bfloat16* row, float (&kf)[kD]) {
  const uint4* p = reinterpret_cast<const uint4*>(row);
#pragma unroll
  for (int i = 0; i < kD / 8; ++i) {
    uint4 v = __ldg(p + i);
    kf[8 * i + 0] = bf16_lo(v.x); kf[8 * i + 1] = bf16_hi(v.x);
    kf[8 * i + 2] = bf16_lo(v.y); kf[8 * i + 3] = bf16_hi(v.y);
    kf[8 * i + 4] = bf16_lo(v.z); kf[8 * i + 5] = bf16_hi(v.z);
    kf[8 * i + 6] = bf16_lo(v.w); kf[8 * i + 7] = bf16_hi(v.w);
  }
}

__device__ __forceinline__ float dot_smem_q(const float* q, const float (&kf)[kD]) {
  float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
  for (int d = 0; d < kD; d += 8) {
    float4 a = *reinterpret_cast<const float4*>(q + d);
    float4 b = *reinterpret_cast<const float4*>(q + d + 4);
    acc0 = fmaf(a.x, kf[d + 0], acc0); acc0 = fmaf(a.y, kf[d + 1], acc0);
    acc0 = fmaf(a.z, kf[d + 2], acc0); acc0 = fmaf(a.w, kf[d + 3], acc0);
    acc1 = fmaf(b.x, kf[d + 4], acc1); acc1 = fmaf(b.y, kf[d + 5], acc1);
    acc1 = fmaf(b.z, kf[d + 6], acc1); acc1 = fmaf(b.w, kf[d + 7], acc1);
  }
  return acc0 + acc1;
}

// MODE 0: per (row, key tile) partial softmax statistics (max and sum in the log2 domain).
// MODE 1: vote[t] = sum over rows of exp2(s * scale2 - lse2[row]).
template <int MODE>
__global__ void __launch_bounds__(kTile)
score_simt_kernel(const __nv_bfloat16* __restrict__ Q_obs, const __nv_bfloat16* __restrict__ K,
                  const float* __restrict__ row_lse, float* __restrict__ vote,
                  float2* __restrict__ stat_part, int Hq, int Hkv, int G, int W, int L, int n_cand,
                  int n_tiles, float scale2) {
  __shared__ __align__(16) float qs[kRowChunk][kD];
  __shared__ float lse2_s[kRowChunk];
  __shared__ float2 wpart[kTile / 32][kRowChunk];

  const int unit = blockIdx.y, tile = blockIdx.x;
  const int b = unit / Hkv, h = unit % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = tile * kTile + tid;
  const int R = G * W;
  const size_t row0 = (size_t)(b * Hq + h * G) * W;  // first observation row of this kv group
  const int t_limit = MODE == 0 ? L : n_cand;

  float kf[kD];
  if (t < t_limit) {
    load_key_row(K + ((size_t)unit * L + t) * kD, kf);
  } else {
#pragma unroll
    for (int d = 0; d < kD; ++d) kf[d] = 0.f;
  }

  float vote_acc = 0.f;
  for (int rc = 0; rc < R; rc += kRowChunk) {
    const int nr = min(kRowChunk, R - rc);
    __syncthreads();
    for (int i = tid; i < nr * (kD / 2); i += kTile) {
      int r = i / (kD / 2), dp = i % (kD / 2);
      uint32_t v = reinterpret_cast<const uint32_t*>(Q_obs + (row0 + rc + r) * kD)[dp];
      qs[r][2 * dp] = bf16_lo(v);
      qs[r][2 * dp + 1] = bf16_hi(v);
    }
    if (MODE == 1 && tid < nr) lse2_s[tid] = row_lse[row0 + rc + tid] * kLog2e;
    __syncthreads();

    for (int r = 0; r < nr; ++r) {
      float s2 = dot_smem_q(qs[r], kf) * scale2;
      if (MODE == 1) {
        if (t < n_cand) vote_acc += exp2f(s2 - lse2_s[r]);
      } else {
        const int j = (rc + r) % W;
        const bool visible = (t <= n_cand + j) && (t < L);
        float x = visible ? s2 : -INFINITY;
        float m = warp_max(x);
        float e = (visible && m > -INFINITY) ? exp2f(x - m) : 0.f;
        float l = warp_sum(e);
        if (lane == 0) wpart[warp][r] = make_float2(m, l);
      }
    }
    if (MODE == 0) {
      __syncthreads();
      if (tid < nr) {
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < kTile / 32; ++w) m = fmaxf(m, wpart[w][tid].x);
        float l = 0.f;
#pragma unroll
        for (int w = 0; w < kTile / 32; ++w) {
          float2 p = wpart[w][tid];
          if (p.x > -INFINITY) l += p.y * exp2f(p.x - m);
        }
        stat_part[(row0 + rc + tid) * n_tiles + tile] = make_float2(m, l);
      }
    }
  }
  if (MODE == 1 && t < n_cand) vote[(size_t)unit * n_cand + t] = vote_acc;
}

// Combine the per-tile statistics of every observation row into its natural-log LSE.
__global__ void row_lse_reduce_kernel(const float2* __restrict__ stat_part, float* __restrict__ row_lse,
                                      int rows, int n_tiles) {
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const float2* p = stat_part + (size_t)r * n_tiles;
  float m = -INFINITY;
  for (int i = 0; i < n_tiles; ++i) m = fmaxf(m, p[i].x);
  float l = 0.f;
  for (int i = 0; i < n_tiles; ++i)
    if (p[i].x > -INFINITY) l += p[i].y * exp2f(p[i].x - m);
  row_lse[r] = (m + log2f(l)) * kLn2;
}

// Direct evaluation of the calibration term (Algorithm 1, lines 5-8): one warp per
// (batch, query head, calibration row) streams every candidate key, skips the kept ones
// (bitmap), and keeps an online softmax over the evicted rest.  Lane i scores key t0 + i;
// for the value accumulation lane i owns output dims 4i .. 4i+3.
__global__ void __launch_bounds__(128)
calib_direct_kernel(const __nv_bfloat16* __restrict__ Q_obs, const __nv_bfloat16* __restrict__ K,
                    const __nv_bfloat16* __restrict__ V, const uint32_t* __restrict__ bitmap,
                    float* __restrict__ O_c, float* __restrict__ LSE_c, __nv_bfloat16* __restrict__ C_q,
                    int B, int Hq, int Hkv, int G, int W, int L, int n_cand, int n_cal, int bitmap_words,
                    float scale2) {
  __shared__ __align__(16) float qs[4][kD];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.x * 4 + warp;  // (b, hq, c)
  const int total = B * Hq * n_cal;
  if (row >= total) return;  // whole warp leaves together; no block-wide barrier below
  const int c = row % n_cal;
  const int bhq = row / n_cal;
  const int b = bhq / Hq, hq = bhq % Hq, h = hq / G;
  const int unit = b * Hkv + h;
  const __nv_bfloat16* q = Q_obs + ((size_t)bhq * W + (W - n_cal + c)) * kD;
  {
    uint2 v = reinterpret_cast<const uint2*>(q)[lane];
    qs[warp][4 * lane + 0] = bf16_lo(v.x); qs[warp][4 * lane + 1] = bf16_hi(v.x);
    qs[warp][4 * lane + 2] = bf16_lo(v.y); qs[warp][4 * lane + 3] = bf16_hi(v.y);
    reinterpret_cast<uint2*>(C_q + (size_t)row * kD)[lane] = v;
  }
  __syncwarp();
  const __nv_bfloat16* Ku = K + (size_t)unit * L * kD;
  const __nv_bfloat16* Vu = V + (size_t)unit * L * kD;
  const uint32_t* bm = bitmap + (size_t)unit * bitmap_words;

  float m = -INFINITY, l = 0.f;
  float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
  for (int t0 = 0; t0 < n_cand; t0 += 32) {
    const uint32_t kept = bm[t0 >> 5];
    const int t = t0 + lane;
    const bool evicted = (t < n_cand) && !((kept >> lane) & 1u);
    if (__ballot_sync(0xffffffffu, evicted) == 0u) continue;
    float s2 = -INFINITY;
    if (evicted) {
      float kf[kD];
      load_key_row(Ku + (size_t)t * kD, kf);
      s2 = dot_smem_q(qs[warp], kf) * scale2;
    }
    const float m_new = fmaxf(m, warp_max(s2));
    const float p = evicted ? exp2f(s2 - m_new) : 0.f;
    const float corr = (m > -INFINITY) ? exp2f(m - m_new) : 0.f;
    l = l * corr + warp_sum(p);
    o0 *= corr; o1 *= corr; o2 *= corr; o3 *= corr;
    m = m_new;
#pragma unroll 4
    for (int i = 0; i < 32; ++i) {
      const float pi = __shfl_sync(0xffffffffu, p, i);
      if (pi != 0.f) {  // warp-uniform
        uint2 v = __ldg(reinterpret_cast<const uint2*>(Vu + (size_t)(t0 + i) * kD) + lane);
        o0 = fmaf(pi, bf16_lo(v.x), o0); o1 = fmaf(pi, bf16_hi(v.x), o1);
        o2 = fmaf(pi, bf16_lo(v.y), o2); o3 = fmaf(pi, bf16_hi(v.y), o3);
      }
    }
  }
  float4 out = make_float4(0.f, 0.f, 0.f, 0.f);
  float lse = -INFINITY;
  if (l > 0.f) {
    const float inv = 1.f / l;
    out = make_float4(o0 * inv, o1 * inv, o2 * inv, o3 * inv);
    lse = (m + log2f(l)) * kLn2;
  }
  reinterpret_cast<float4*>(O_c + (size_t)row * kD)[lane] = out;
  if (lane == 0) LSE_c[row] = lse;
}

}  // namespace

cudaError_t launch_row_stats(const CompressGeom& g, const CompressWs& ws, const void* Q_obs,
                             const void* K, char* wsp, cudaStream_t st) {
  dim3 grid(ws.n_tiles, g.units);
  score_simt_kernel<0><<<grid, kTile, 0, st>>>(
      (const __nv_bfloat16*)Q_obs, (const __nv_bfloat16*)K, nullptr, nullptr,
      (float2*)(wsp + ws.stat_part), g.Hq, g.Hkv, g.G, g.W, g.L, g.n_cand, ws.n_tiles, g.scale2);
  const int rows = g.B * g.Hq * g.W;
  row_lse_reduce_kernel<<<(rows + 127) / 128, 128, 0, st>>>((const float2*)(wsp + ws.stat_part),
                                                            (float*)(wsp + ws.row_lse), rows, ws.n_tiles);
  count_launch(2);
  return cudaGetLastError();
}

cudaError_t launch_votes(const CompressGeom& g, const CompressWs& ws, const void* Q_obs, const void* K,
                         const float* row_lse, char* wsp, cudaStream_t st) {
  dim3 grid((g.n_cand + kTile - 1) / kTile, g.units);
  score_simt_kernel<1><<<grid, kTile, 0, st>>>((const __nv_bfloat16*)Q_obs, (const __nv_bfloat16*)K,
                                                row_lse, (float*)(wsp + ws.vote), nullptr, g.Hq, g.Hkv,
                                                g.G, g.W, g.L, g.n_cand, ws.n_tiles, g.scale2);
  count_launch(1);
  return cudaGetLastError();
}

cudaError_t launch_calib_direct(const CompressGeom& g, const CompressWs& ws, const void* Q_obs,
                                const void* K, const void* V, char* wsp, float* O_c, float* LSE_c,
                                void* C_q, cudaStream_t st) {
  const int total = g.B * g.Hq * g.n_cal;
  calib_direct_kernel<<<(total + 3) / 4, 128, 0, st>>>(
      (const __nv_bfloat16*)Q_obs, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V,
      (const uint32_t*)(wsp + ws.calib_mask), O_c, LSE_c, (__nv_bfloat16*)C_q, g.B, g.Hq, g.Hkv, g.G, g.W,
      g.L, g.n_cand, g.n_cal, g.bitmap_words, g.scale2);
  count_launch(1);
  return cudaGetLastError();
}

}  // namespace calidrop
