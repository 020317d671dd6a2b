// Decode-time attention over the compacted retained cache, merged with the calibration term.
//
// One launch covers: the append of the step's new K/V row, a split-K flash-decode over the
// retained rows with the G query heads of a kv group packed into one MMA tile (so every K/V
// byte is read once for all of them), the cosine similarity of the query with the stored
// calibration queries, the threshold gate, and the merge of Eq. 1-2.  The work is bound by
// HBM traffic (about 2G flop per byte), so the contraction uses the warp-level mma.sync path
// with G <= 8 rows of a 16-row tile; tcgen05 tiles (64 rows minimum) would add nothing here.
//
// Grid: (split, batch*kv-head, layer); the splits of one (unit, layer) form thread-block
// clusters of 1, 2, 4 or 8 CTAs.  Each CTA streams its slice of rows through shared memory with
// 16-byte cp.async copies (XOR-swizzled so ldmatrix is conflict-free), four warps each running
// an independent online softmax over interleaved 16-row blocks.  The splits are combined inside
// the cluster through distributed shared memory: every CTA finishes a slice of the 128 output
// dimensions for all heads of the group, so there is no global-memory round trip, no ticket and
// no CTA that works alone at the end.  Only when very few units share a long cache (fewer than
// 19 units per launch) does one cluster per unit leave most SMs idle; then a unit gets up to
// eight clusters, each writes its combined partial, its (max, sum) pair and its best similarity
// to the workspace, and the CTA that takes the last ticket of the unit's arrival counter merges
// them and resets the counter.
//
// A launch moves only tens of MB, so its latency chain matters as much as its bandwidth:
//   * the launch carries the programmatic-serialisation attribute and the kernel prefetches its
//     K/V slice into L2 before the dependency wait, so the HBM reads of one decode call overlap
//     the tail of whatever runs ahead of it in the stream;
//   * the K/V copies are issued first, the similarity work (which needs only q and C_q) runs while
//     they are in flight, and the cluster exchanges each CTA's best (similarity, row) pair early,
//     so the chosen O_c row is already being fetched while the partial outputs are combined.
#include <cooperative_groups.h>

#include "common.cuh"
#include "internal.h"

namespace calidrop {

namespace {

namespace cg = cooperative_groups;

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kBlkRows = 16;                           // rows per pipeline stage of one warp
constexpr int kStages = 3;
constexpr int kStageBytes = 2 * kBlkRows * kRowBytes;  // K block then V block
constexpr int kWarpSmem = kStages * kStageBytes;       // 24 KB
constexpr int kSmemBytes = kWarps * kWarpSmem;         // 192 KB -> one CTA per SM

constexpr int kWoStride = kD + 4;  // row stride of the per-warp partial outputs: heads land in distinct banks

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}

__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)(row * kRowBytes + ((chunk ^ (row & 7)) << 4));
}

struct RhoLoad {
  uint4 q0, q1, c0, c1;
};

__device__ __forceinline__ void rho_accumulate(const RhoLoad& r, float& dot, float& qq, float& cc) {
  const uint32_t qw[8] = {r.q0.x, r.q0.y, r.q0.z, r.q0.w, r.q1.x, r.q1.y, r.q1.z, r.q1.w};
  const uint32_t cw[8] = {r.c0.x, r.c0.y, r.c0.z, r.c0.w, r.c1.x, r.c1.y, r.c1.z, r.c1.w};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float a0 = bf16_lo(qw[j]), a1 = bf16_hi(qw[j]);
    const float b0 = bf16_lo(cw[j]), b1 = bf16_hi(cw[j]);
    dot = fmaf(a0, b0, fmaf(a1, b1, dot));
    qq = fmaf(a0, a0, fmaf(a1, a1, qq));
    cc = fmaf(b0, b0, fmaf(b1, b1, cc));
  }
}

// Order-preserving map of a float onto unsigned integers; with the row index in the low word,
// one 64-bit max picks the highest similarity and, among equals, the largest row index.
__device__ __forceinline__ unsigned long long rank_key(float rho, int c) {
  unsigned u = __float_as_uint(rho);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned)c;
}
__device__ __forceinline__ float rank_key_value(unsigned long long k) {
  unsigned u = (unsigned)(k >> 32);
  u = (u & 0x80000000u) ? (u & 0x7fffffffu) : ~u;
  return __uint_as_float(u);
}

__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Gate and merge of one output element (Eq. 1-2): (acc, M, Lsum) is the unnormalised partial of
// the retained cache in the log2 domain, best the chosen (similarity, calibration row) key.
__device__ __forceinline__ void merge_store(const DecodeArgs& a, const DecodeLayerPtrs& P, int hq, int d, float acc,
                                            float M, float Lsum, unsigned long long best, float lse_c, float oc) {
  const int cs = (int)(unsigned)(best & 0xffffffffull);
  const float rho = rank_key_value(best);
  float outv = acc / Lsum;       // O_a
  float lse2 = M + log2f(Lsum);  // LSE_a (log2 domain)
  const bool apply = (a.always_apply || rho > a.theta2) && (lse_c > -INFINITY);
  if (apply) {
    // alpha_i = e^{LSE_a - LSE}, alpha_j = e^{LSE_c - LSE}; out = alpha_i O_a + alpha_j O_c
    const float lc2 = lse_c * kLog2e;
    const float mx = fmaxf(lse2, lc2);
    const float ea = exp2f(lse2 - mx), ec = exp2f(lc2 - mx);
    const float tot = ea + ec;
    outv = (ea / tot) * outv + (ec / tot) * oc;
    lse2 = mx + log2f(tot);
  }
  reinterpret_cast<__nv_bfloat16*>(P.out)[(size_t)hq * kD + d] = __float2bfloat16_rn(outv);
  if (d == 0) {
    if (P.lse_out) P.lse_out[hq] = lse2 * kLn2;
    if (P.flags)
      P.flags[hq] = (uint8_t)((apply ? 1 : 0) | (rho < a.theta1 ? 2 : 0) | (a.n_cal <= 64 ? (cs << 2) : 0));
  }
}

__global__ void __launch_bounds__(kThreads, 1) decode_kernel(const __grid_constant__ DecodeArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ unsigned long long s_best[kMaxG];  // best (similarity, row) of this CTA's calibration rows

  cg::cluster_group cluster = cg::this_cluster();
  const int gs = blockIdx.x;             // split index over the whole unit
  const int split = gs % a.nsplit;       // rank inside the cluster
  const int clu = gs / a.nsplit;         // cluster of this unit
  const int n_gs = a.nsplit * a.nclu;
  const int unit = blockIdx.y, layer = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gq = lane >> 2, tq = lane & 3;  // MMA fragment coordinates
  const DecodeLayerPtrs& P = a.layer[layer];
  const int b = unit / a.Hkv, h = unit % a.Hkv;
  const int hq0 = b * a.Hq + h * a.G;  // first query head of this kv group

  const __nv_bfloat16* q = (const __nv_bfloat16*)P.q;
  const __nv_bfloat16* Cq = (const __nv_bfloat16*)P.C_q;
  const unsigned char* Kc = (const unsigned char*)P.K + (size_t)unit * a.cap * kRowBytes;
  const unsigned char* Vc = (const unsigned char*)P.V + (size_t)unit * a.cap * kRowBytes;
  const unsigned char* k_new = (const unsigned char*)P.k_new + (size_t)unit * kRowBytes;
  const unsigned char* v_new = (const unsigned char*)P.v_new + (size_t)unit * kRowBytes;

  const int r0 = min(a.n_kv, gs * a.rows_per_split);
  const int r1 = min(a.n_kv, r0 + a.rows_per_split);
  const int nblk = r1 > r0 ? (r1 - r0 + kBlkRows - 1) / kBlkRows : 0;
  const int my_blocks = nblk > warp ? (nblk - warp + kWarps - 1) / kWarps : 0;

  unsigned char* wsm = smem + warp * kWarpSmem;
  const uint32_t wsm_u32 = smem_u32(wsm);

  // ---- (0) overlap with the kernel ahead of this one in the stream.  Until the dependency wait
  // nothing the predecessor may have written is read and nothing is written; the only early work
  // is an L2 prefetch of this CTA's slice of the retained cache, which cannot observe stale data
  // (L2 is the point of coherence) and turns the later cp.async stream into L2 hits.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    const int n_old = min(r1, a.kv_len) - r0;  // rows already in the cache (the appended row is not)
    if (n_old > 0) {
      const unsigned bytes = (unsigned)n_old * kRowBytes;
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(Kc + (size_t)r0 * kRowBytes), "r"(bytes)
                   : "memory");
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(Vc + (size_t)r0 * kRowBytes), "r"(bytes)
                   : "memory");
    }
  }
  // calibration rows of this CTA: the contiguous range [c_begin, c_begin + n_c)
  const int c_per = (a.n_cal + n_gs - 1) / n_gs;
  const int c_begin = min(a.n_cal, gs * c_per);
  const int n_c = min(a.n_cal, c_begin + c_per) - c_begin;
  if (tid >= 32 && tid < 32 + a.G && n_c > 0) {  // same for the small operands of the similarity
    const int g = tid - 32;
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(Cq + ((size_t)(hq0 + g) * a.n_cal + c_begin) * kD),
                 "r"((unsigned)n_c * kRowBytes)
                 : "memory");
    if (g == 0)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(q + (size_t)hq0 * kD),
                   "r"((unsigned)a.G * kRowBytes)
                   : "memory");
  }
  if (tid < kMaxG) s_best[tid] = 0ull;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  __syncthreads();

  // ---- (1) loads of the similarity operands go out ahead of the K/V burst so that they are not
  // queued behind it: four lanes per (head, calibration row) pair, 32 pairs per pass, the first
  // two passes in flight at once
  constexpr int kPairsPerPass = kThreads / 4;
  const int pairs = n_c * a.G;
  const int sub = tid & 3;
  auto rho_load = [&](int pi, RhoLoad (&r)[2]) {
    r[0] = RhoLoad{}; r[1] = RhoLoad{};
    if (pi < pairs) {
      const int g = pi % a.G, c = c_begin + pi / a.G;
      const uint4* qp = reinterpret_cast<const uint4*>(q + (size_t)(hq0 + g) * kD + sub * 32);
      const uint4* cp = reinterpret_cast<const uint4*>(Cq + ((size_t)(hq0 + g) * a.n_cal + c) * kD + sub * 32);
      r[0].q0 = __ldg(qp); r[0].q1 = __ldg(qp + 1); r[0].c0 = __ldg(cp); r[0].c1 = __ldg(cp + 1);
      r[1].q0 = __ldg(qp + 2); r[1].q1 = __ldg(qp + 3); r[1].c0 = __ldg(cp + 2); r[1].c1 = __ldg(cp + 3);
    }
  };
  auto rho_finish = [&](int pi, const RhoLoad (&r)[2]) {
    float dot = 0.f, qq = 0.f, cc = 0.f;
    if (pi < pairs) { rho_accumulate(r[0], dot, qq, cc); rho_accumulate(r[1], dot, qq, cc); }
#pragma unroll
    for (int o = 1; o < 4; o <<= 1) {
      dot += __shfl_xor_sync(0xffffffffu, dot, o);
      qq += __shfl_xor_sync(0xffffffffu, qq, o);
      cc += __shfl_xor_sync(0xffffffffu, cc, o);
    }
    if (sub == 0 && pi < pairs) {
      const int g = pi % a.G, c = c_begin + pi / a.G;
      const float rho = (qq > 0.f && cc > 0.f) ? dot / (sqrtf(qq) * sqrtf(cc)) : 0.f;
      atomicMax(&s_best[g], rank_key(rho, c));
    }
  };
  RhoLoad rl0[2], rl1[2];
  rho_load(tid >> 2, rl0);
  rho_load(kPairsPerPass + (tid >> 2), rl1);

  // ---- (2) the K/V stream: issue one 16-row block (K and V) of this warp into a stage
  auto issue = [&](int i, int stage) {
    const int row_base = r0 + (warp + i * kWarps) * kBlkRows;
    const uint32_t dstK = wsm_u32 + stage * kStageBytes;
    const uint32_t dstV = dstK + kBlkRows * kRowBytes;
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int idx = it * 32 + lane;
      const int row = idx >> 4, chunk = idx & 15;
      const int rg = row_base + row;
      const bool valid = rg < r1;
      const bool fresh = a.has_new && rg == a.kv_len;
      const unsigned char* sk = fresh ? k_new + chunk * 16 : Kc + (size_t)(valid ? rg : 0) * kRowBytes + chunk * 16;
      const unsigned char* sv = fresh ? v_new + chunk * 16 : Vc + (size_t)(valid ? rg : 0) * kRowBytes + chunk * 16;
      cp_async_16(dstK + swz(row, chunk), sk, valid ? 16 : 0);
      cp_async_16(dstV + swz(row, chunk), sv, valid ? 16 : 0);
    }
  };
#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) {
    if (s < my_blocks) issue(s, s);
    cp_async_commit();
  }

  // ---- (3) query fragments (rows 0..G-1 of a 16-row A tile, the rest zero)
  uint32_t qa[kD / 16][2];
#pragma unroll
  for (int kk = 0; kk < kD / 16; ++kk) {
    qa[kk][0] = 0u; qa[kk][1] = 0u;
    if (gq < a.G) {
      const uint32_t* qr = reinterpret_cast<const uint32_t*>(q + (size_t)(hq0 + gq) * kD + kk * 16);
      qa[kk][0] = __ldg(qr + tq);
      qa[kk][1] = __ldg(qr + 4 + tq);
    }
  }

  // ---- (3b) append: the CTA whose slice holds row kv_len stores the new K/V row into the cache
  if (a.has_new && a.kv_len >= r0 && a.kv_len < r1 && warp == 0) {
    const int chunk = lane & 15;
    const unsigned char* src = (lane < 16 ? k_new : v_new) + chunk * 16;
    unsigned char* dst = (unsigned char*)(lane < 16 ? P.K : P.V) +
                         ((size_t)unit * a.cap + a.kv_len) * kRowBytes + chunk * 16;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  }

  // ---- (4) cosine similarities of this CTA's calibration rows; the best pair per head goes to
  // s_best (the K/V copies are in flight meanwhile)
  rho_finish(tid >> 2, rl0);
  rho_finish(kPairsPerPass + (tid >> 2), rl1);
  for (int base = 2 * kPairsPerPass; base < pairs; base += kPairsPerPass) {
    rho_load(base + (tid >> 2), rl0);
    rho_finish(base + (tid >> 2), rl0);
  }
  cluster_arrive();  // (A) this CTA's s_best is final

  // ---- (5) main loop.  The products are taken transposed, keys on the 16-row side of the MMA and
  // the (at most eight) heads on its 8-column side, so that no half of a tile is padding:
  //   S^T[16 keys x 8 heads]   = K_blk[16 x 128] . Q^T[128 x 8]          (8 MMAs)
  //   O^T[128 dims x 8 heads] += V_blk^T[128 x 16 keys] . P^T[16 x 8]     (8 MMAs)
  // A thread holds heads 2tq, 2tq+1 of keys gq, gq+8 (S^T) and of dims 16n+gq, 16n+gq+8 (O^T).
  float o[kD / 16][4];
#pragma unroll
  for (int n = 0; n < kD / 16; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // heads 2tq and 2tq+1
  const int mid = lane >> 3;

  for (int i = 0; i < my_blocks; ++i) {
    const int nxt = i + kStages - 1;
    if (nxt < my_blocks) issue(nxt, nxt % kStages);
    cp_async_commit();
    cp_async_wait<kStages - 1>();
    __syncwarp();

    const uint32_t sK = wsm_u32 + (i % kStages) * kStageBytes;
    const uint32_t sV = sK + kBlkRows * kRowBytes;
    const int row_base = r0 + (warp + i * kWarps) * kBlkRows;

    // S^T: two accumulators (even and odd k-steps) halve the dependent chain
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int kk = 0; kk < kD / 16; ++kk) {
      uint32_t a0, a1, a2, a3;
      ldmatrix_x4(sK + swz((lane & 7) + (mid & 1) * 8, kk * 2 + (mid >> 1)), a0, a1, a2, a3);
      if (kk & 1) mma_bf16_16816(sb, a0, a1, a2, a3, qa[kk][0], qa[kk][1]);
      else mma_bf16_16816(sa, a0, a1, a2, a3, qa[kk][0], qa[kk][1]);
    }
    // online softmax per head over the 16 keys of the block (keys gq and gq + 8 live here)
    const bool v0 = row_base + gq < r1, v1 = row_base + gq + 8 < r1;
    const float x00 = v0 ? (sa[0] + sb[0]) * a.scale2 : -INFINITY;
    const float x01 = v0 ? (sa[1] + sb[1]) * a.scale2 : -INFINITY;
    const float x10 = v1 ? (sa[2] + sb[2]) * a.scale2 : -INFINITY;
    const float x11 = v1 ? (sa[3] + sb[3]) * a.scale2 : -INFINITY;
    float bm0 = fmaxf(x00, x10), bm1 = fmaxf(x01, x11);
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, off));
      bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, off));
    }
    const float mn0 = fmaxf(m0, bm0), mn1 = fmaxf(m1, bm1);  // finite: the block's first key is valid
    const float corr0 = ex2_approx(m0 - mn0), corr1 = ex2_approx(m1 - mn1);
    const float p00 = ex2_approx(x00 - mn0), p01 = ex2_approx(x01 - mn1);
    const float p10 = ex2_approx(x10 - mn0), p11 = ex2_approx(x11 - mn1);
    l0 = l0 * corr0 + (p00 + p10);  // partial over this thread's keys, summed over gq at the end
    l1 = l1 * corr1 + (p01 + p11);
    m0 = mn0; m1 = mn1;
#pragma unroll
    for (int n = 0; n < kD / 16; ++n) { o[n][0] *= corr0; o[n][1] *= corr1; o[n][2] *= corr0; o[n][3] *= corr1; }
    // P^T as the B operand: transpose the two 8x8 (key, head) fragments inside the warp
    const uint32_t pb0 = movmatrix_trans(pack_bf16(p00, p01)), pb1 = movmatrix_trans(pack_bf16(p10, p11));
#pragma unroll
    for (int n = 0; n < kD / 16; ++n) {
      uint32_t a0, a1, a2, a3;
      ldmatrix_x4_trans(sV + swz((lane & 7) + (mid >> 1) * 8, n * 2 + (mid & 1)), a0, a1, a2, a3);
      mma_bf16_16816(o[n], a0, a1, a2, a3, pb0, pb1);
    }
    __syncwarp();  // the stage is refilled by the next iteration's cp.async
  }
  cp_async_wait<0>();
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
  }
  __syncthreads();  // all warps are done with their stages: reuse them for the combine

  // ---- (6) CTA combine of the four warps into this split's partial: xo[g][d], xml[g] = (m, l)
  float* wo = reinterpret_cast<float*>(smem);             // [warp][8][kWoStride]
  float* wml = wo + kWarps * kMaxG * kWoStride;            // [warp][8][2]
  float* xo = wml + kWarps * kMaxG * 2;                    // [8][128]
  float* xml = xo + kMaxG * kD;                            // [8][2]
  if (2 * tq < a.G) {
#pragma unroll
    for (int n = 0; n < kD / 16; ++n) {
      float* w0 = wo + (warp * kMaxG + 2 * tq) * kWoStride + n * 16 + gq;
      w0[0] = o[n][0]; w0[8] = o[n][2];
      w0[kWoStride] = o[n][1]; w0[kWoStride + 8] = o[n][3];
    }
    if (gq == 0) {
      wml[(warp * kMaxG + 2 * tq) * 2] = m0; wml[(warp * kMaxG + 2 * tq) * 2 + 1] = l0;
      wml[(warp * kMaxG + 2 * tq + 1) * 2] = m1; wml[(warp * kMaxG + 2 * tq + 1) * 2 + 1] = l1;
    }
  }
  __syncthreads();
  for (int d = tid; d < kD; d += kThreads) {
#pragma unroll
    for (int g = 0; g < kMaxG; ++g) {
      if (g >= a.G) break;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) M = fmaxf(M, wml[(w * kMaxG + g) * 2]);
      float Lsum = 0.f, acc = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float mw = wml[(w * kMaxG + g) * 2];
        const float sc = mw > -INFINITY ? ex2_approx(mw - M) : 0.f;
        Lsum += wml[(w * kMaxG + g) * 2 + 1] * sc;
        acc += wo[(w * kMaxG + g) * kWoStride + d] * sc;
      }
      xo[g * kD + d] = acc;
      if (d == 0) { xml[g * 2] = M; xml[g * 2 + 1] = Lsum; }
    }
  }
  cluster_wait();    // (A) every CTA's s_best can be read
  cluster_arrive();  // (B) this CTA's partial (xo, xml) is final

  // ---- (7) finish.  This CTA owns 128 / nsplit output dimensions of every head of the group.
  const int dpc = kD / a.nsplit;
  const int n_items = a.G * dpc;
  const bool single = a.nclu == 1;
  const int lu = layer * a.units + unit;
  for (int item0 = 0; item0 < n_items; item0 += kThreads) {
    const int item = item0 + tid;
    const bool act = item < n_items;
    const int g = act ? item / dpc : 0, d = split * dpc + (act ? item % dpc : 0);
    const int hq = hq0 + g;
    // the calibration row: best similarity over all CTAs, ties to the largest row index
    unsigned long long best = 0ull;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      if (s < a.nsplit) {
        const unsigned long long k = *cluster.map_shared_rank(&s_best[g], s);
        best = k > best ? k : best;
      }
    }
    float lse_c = 0.f, oc = 0.f;
    if (act && single) {  // in flight while the partials are exchanged
      const size_t crow = (size_t)hq * a.n_cal + (unsigned)(best & 0xffffffffull);
      lse_c = __ldg(P.LSE_c + crow);
      oc = __ldg(P.O_c + crow * kD + d);
    }
    if (item0 == 0) cluster_wait();  // (B) every CTA's partial can be read
    float ms[8], ls[8], os[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) {  // all remote reads in flight together
      ms[s] = -INFINITY; ls[s] = 0.f; os[s] = 0.f;
      if (s < a.nsplit) {
        const float2 ml2 = *reinterpret_cast<const float2*>(cluster.map_shared_rank(xml, s) + g * 2);
        ms[s] = ml2.x; ls[s] = ml2.y;
        os[s] = cluster.map_shared_rank(xo, s)[g * kD + d];
      }
    }
    float M = -INFINITY;
#pragma unroll
    for (int s = 0; s < 8; ++s) M = fmaxf(M, ms[s]);
    float Lsum = 0.f, acc = 0.f;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      const float sc = ms[s] > -INFINITY ? ex2_approx(ms[s] - M) : 0.f;
      Lsum = fmaf(ls[s], sc, Lsum);
      acc = fmaf(os[s], sc, acc);
    }
    if (single) {
      if (act) merge_store(a, P, hq, d, acc, M, Lsum, best, lse_c, oc);
    } else if (act) {
      // this cluster's partial goes to the workspace; (M, Lsum, best) are the same in all its CTAs
      const size_t pc = ((size_t)lu * a.nclu + clu) * kMaxG + g;
      a.part_o[pc * kD + d] = acc;
      if (d == 0) {
        a.part_ml[pc * 2] = M;
        a.part_ml[pc * 2 + 1] = Lsum;
        a.part_best[pc] = best;
      }
    }
  }
  cluster_arrive();  // (C) no CTA leaves while another may still read its shared memory
  if (!single) {
    // ---- (8) several clusters per unit: the CTA that takes the unit's last ticket merges them
    __shared__ unsigned s_ticket;
    __threadfence();
    __syncthreads();
    if (tid == 0) s_ticket = atomicAdd(&a.counters[lu], 1u);
    __syncthreads();
    if (s_ticket == (unsigned)(n_gs - 1)) {
      __threadfence();
      for (int gd = tid; gd < a.G * kD; gd += kThreads) {
        const int g = gd / kD, d = gd % kD;
        const size_t pu = (size_t)lu * a.nclu * kMaxG + g;
        unsigned long long best = 0ull;
        float ms[8], ls[8], os[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          ms[c] = -INFINITY; ls[c] = 0.f; os[c] = 0.f;
          if (c < a.nclu) {
            const size_t pc = pu + (size_t)c * kMaxG;
            const unsigned long long k = __ldcg(a.part_best + pc);
            best = k > best ? k : best;
            const float2 ml2 = __ldcg(reinterpret_cast<const float2*>(a.part_ml + pc * 2));
            ms[c] = ml2.x; ls[c] = ml2.y;
            os[c] = __ldcg(a.part_o + pc * kD + d);
          }
        }
        const int hq = hq0 + g;
        const size_t crow = (size_t)hq * a.n_cal + (unsigned)(best & 0xffffffffull);
        const float lse_c = __ldg(P.LSE_c + crow);
        const float oc = __ldg(P.O_c + crow * kD + d);
        float M = -INFINITY;
#pragma unroll
        for (int c = 0; c < 8; ++c) M = fmaxf(M, ms[c]);
        float Lsum = 0.f, acc = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const float sc = ms[c] > -INFINITY ? ex2_approx(ms[c] - M) : 0.f;
          Lsum = fmaf(ls[c], sc, Lsum);
          acc = fmaf(os[c], sc, acc);
        }
        merge_store(a, P, hq, d, acc, M, Lsum, best, lse_c, oc);
      }
      if (tid == 0) a.counters[lu] = 0u;  // ready for the next launch on this workspace
    }
  }
  cluster_wait();
}

}  // namespace

cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t st) {
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.nsplit * a.nclu, a.units, a.n_layers);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;  // the splits of a unit are one cluster
  attr[0].val.clusterDim.x = a.nsplit;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  e = cudaLaunchKernelEx(&cfg, decode_kernel, a);
  if (e != cudaSuccess) return e;
  count_launch(1);
  return cudaGetLastError();
}

}  // namespace calidrop
