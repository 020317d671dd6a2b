// Decode-time attention over the compacted retained cache, merged with the calibration term.
//
// One launch covers: the append of the step's new K/V row, a split-K flash-decode over the
// retained rows with the G query heads of a kv group packed into one MMA tile (so every K/V
// byte is read once for all of them), the cosine similarity of the query with the stored
// calibration queries, the threshold gate, and the merge of Eq. 1-2.  The work is bound by
// HBM traffic (about 2G flop per byte), so the contraction uses the warp-level mma.sync path;
// what matters is how the bytes get to the SM and how short the chain after the last byte is.
//
// Grid: (split, batch*kv-head, layer); the splits of one (unit, layer) form thread-block
// clusters of 1, 2, 4 or 8 CTAs.  A CTA has one producer warp and eight stream warps.  The
// producer moves the CTA's slice of K and V through a ring of six 64-row slots with TMA
// (128-byte swizzle, so ldmatrix is conflict-free and no load instruction per 16 bytes is
// spent on the stream); each slot is consumed by four stream warps, 16 rows each, with their
// own online softmax.  The products are taken transposed, keys on the 16-row side of the MMA and
// the (at most eight) heads on its 8-column side, so that no half of a tile is padding:
//   S^T[16 keys x 8 heads]   = K_blk[16 x 128] . Q^T[128 x 8]          (8 MMAs)
//   O^T[128 dims x 8 heads] += V_blk^T[128 x 16 keys] . P^T[16 x 8]     (8 MMAs)
// The splits are combined inside the cluster through distributed shared memory: every CTA
// finishes a slice of the 128 output dimensions for all heads of the group, and each CTA pushes
// its partial of a slice into the shared memory of the slice's owner with asynchronous stores that
// report their bytes to an mbarrier there, so that every CTA waits for its own data only and then
// reduces local data.  Only when very few units share a very long cache
// (more than 1024 rows per CTA even with a cluster of eight) does a unit get up to eight clusters;
// each writes its combined partial, its (max, sum) pair and its best similarity to the workspace, and
// the CTA that takes the last ticket of the unit's arrival counter merges them and resets the counter.
//
// A launch moves only tens of MB, so its latency chain matters as much as its bandwidth:
//   * the launch carries the programmatic-serialisation attribute and the kernel, first thing,
//     prefetches the head of its K/V slice into L2, ahead of the dependency wait; the ring takes
//     most of an SM's shared memory, so a launch has one CTA per SM at most;
//   * everything that does not need the predecessor's results (barrier setup, the address
//     arithmetic of all later loads) is done ahead of the wait as well;
//   * the similarity work (which needs only q and C_q) runs while the first slots are in flight,
//     and the cluster exchanges each CTA's best (similarity, row) pair early; the producer warp,
//     idle once the last slot is on its way, settles the calibration row meanwhile, and the chosen
//     O_c elements are fetched while the partial outputs are combined;
//   * the cache stream carries an evict-first L2 hint, the calibration state an evict-last hint.
#include <cooperative_groups.h>

#include "common.cuh"
#include "internal.h"
#include "tc_common.cuh"

namespace calidrop {

namespace {

namespace cg = cooperative_groups;

constexpr int kStreamWarps = 8;
constexpr int kThreads = (kStreamWarps + 1) * 32;  // the last warp is the producer
constexpr int kBlkRows = 16;                        // rows of one warp's MMA block
constexpr int kSlotRows = 64;                       // rows per ring slot: four blocks
constexpr int kSlotsWide = 6;    // ring of a launch with one CTA per SM at most: 192 KB
constexpr int kSlotsNarrow = 3;  // ring of a launch with more CTAs than SMs: 96 KB, two CTAs per SM
constexpr int kPlaneBytes = kSlotRows * 128;        // 64 rows x 64 columns of bf16 (one TMA box)
constexpr int kSlotBytes = 4 * kPlaneBytes;         // K low / K high / V low / V high column halves
constexpr int smem_bytes(int slots) { return slots * kSlotBytes + 1024; }  // + slack for the 1024-byte alignment
constexpr int kWoStride = kD + 4;  // row stride of the per-warp partial outputs: heads land in distinct banks
constexpr long long kWaitLimitCycles = 2000000000ll;  // about a second: a wait this long has failed

// Byte offset of 16-byte chunk `chunk` (0..15) of row `row` (0..63) inside the K or V part of a
// slot: two column halves, each a [64 rows][128 bytes] plane in the 128-byte swizzle TMA writes.
__device__ __forceinline__ uint32_t plane_off(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * kPlaneBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}

// ---- mbarrier / TMA helpers (every copy lands in the shared memory of the CTA that issued it)
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: when it runs out the CTA's abort flag is raised, the workspace's error word is
// set and every later wait of the CTA returns at once; the CTA still walks through all its
// barriers, so nothing hangs, but its output is not valid.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned* status, unsigned code) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = 0;
  unsigned polls = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++polls & 255u) == 0u) {
      if (*abort_flag) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      if (now - t0 > kWaitLimitCycles) {
        *abort_flag = 1;
        atomicCAS(status, 0u, code);
        return false;
      }
    }
  }
  return true;
}
// The same wait without the shortcut on the CTA's abort flag: only its own time limit ends it early.
// For waits that must be sat out even in a CTA that is giving up, because other CTAs still write
// into (or read from) this CTA's shared memory until the awaited phase completes.
__device__ __forceinline__ bool mbar_wait_sit_out(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  unsigned* status, unsigned code) {
  long long t0 = 0;
  unsigned polls = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++polls & 255u) == 0u) {
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      if (now - t0 > kWaitLimitCycles) {
        *abort_flag = 1;
        atomicCAS(status, 0u, code);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(pol)
      : "memory");
}

// L2 eviction policies.  The retained cache is read once per call and is far larger than what the
// next call on the same state finds in L2 again, so its lines are marked to go first; the
// calibration state (C_q, the chosen O_c rows, LSE_c) is small and read by every call, so its
// lines are marked to stay.  With that the similarity loads are L2 hits and do not queue behind
// the stream in the memory system.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint4 ldg_keep(const uint4* ptr, uint64_t pol) {
  uint4 v;
  asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr), "l"(pol));
  return v;
}
__device__ __forceinline__ float ldg_keep(const float* ptr, uint64_t pol) {
  float v;
  asm volatile("ld.global.nc.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(v) : "l"(ptr), "l"(pol));
  return v;
}

// Shared-memory address of `local` in CTA `rank` of the cluster, and an 8-byte store to such an
// address that reports its bytes to an mbarrier of the same CTA when it lands.
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void push_f32x2(uint32_t remote, float x, float y, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(remote),
               "f"(x), "f"(y), "r"(remote_bar)
               : "memory");
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
__device__ __forceinline__ void merge_store(const DecodeCommon& a, const DecodeLayerPtrs& P, int hq, int d, float acc,
                                            float M, float Lsum, unsigned long long best, float lse_c, float oc) {
  const int cs = (int)(unsigned)(best & 0xffffffffull);
  const float rho = rank_key_value(best);
  float outv = __fdividef(acc, Lsum);  // O_a
  float lse2 = M + __log2f(Lsum);      // LSE_a (log2 domain)
  const bool apply = (a.always_apply || rho > a.theta2) && (lse_c > -INFINITY);
  if (apply) {
    // alpha_i = e^{LSE_a - LSE}, alpha_j = e^{LSE_c - LSE}; out = alpha_i O_a + alpha_j O_c
    const float lc2 = lse_c * kLog2e;
    const float mx = fmaxf(lse2, lc2);
    const float ea = ex2_approx(lse2 - mx), ec = ex2_approx(lc2 - mx);
    const float inv = __fdividef(1.f, ea + ec);  // the sum is in [1, 2]
    outv = (ea * inv) * outv + (ec * inv) * oc;
    lse2 = mx + __log2f(ea + ec);
  }
  reinterpret_cast<__nv_bfloat16*>(P.out)[(size_t)hq * kD + d] = __float2bfloat16_rn(outv);
  if (d == 0) {
    if (P.lse_out) P.lse_out[hq] = lse2 * kLn2;
    if (P.flags)
      P.flags[hq] = (uint8_t)((apply ? 1 : 0) | (rho < a.theta1 ? 2 : 0) | (a.n_cal <= 64 ? (cs << 2) : 0));
  }
}

// Algorithm 2, lines 4-6, for the launches that recompute a calibration entry: the attention of the
// current query over the (reloaded) evicted KV is the new O_c row, its log-denominator the new LSE_c,
// and the query itself the new C_q row (the reading of line 4-5's "Q_-1" as the current query).
__device__ __forceinline__ void recal_store(const DecodeCommon& a, const DecodeLayerPtrs& P, int hq, int d, float acc,
                                            float M, float Lsum) {
  const size_t row = (size_t)hq * a.n_cal + a.recal_slot;
  const_cast<float*>(P.O_c)[row * kD + d] = acc / Lsum;
  reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(P.C_q))[row * kD + d] =
      reinterpret_cast<const __nv_bfloat16*>(P.q)[(size_t)hq * kD + d];
  if (d == 0) const_cast<float*>(P.LSE_c)[row] = (M + log2f(Lsum)) * kLn2;
}

// RECAL = false: the decode step.  RECAL = true: the same stream over the evicted KV, without the
// similarity and the gate, ending in recal_store.  kSlots: ring depth (six slots and one CTA per
// SM, or three slots and two CTAs per SM for launches of many short, independent slices, where the
// fixed chain of one CTA is what a second resident CTA can overlap).
template <int NL, bool RECAL, int kSlots>
__global__ void __launch_bounds__(kThreads, kSlots > 3 ? 1 : 2)
decode_kernel(const __grid_constant__ DecodeArgsT<NL> args) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long s_full[kSlots][2], s_empty[kSlots][2];
  __shared__ unsigned long long s_best[kMaxG];     // best (similarity, row) of this CTA's calibration rows
  __shared__ unsigned long long s_bestall[kMaxG];  // ... of the whole cluster
  __shared__ __align__(16) float s_xpart[kMaxG * kD];  // [source split][head][dim of this CTA's slice]
  __shared__ __align__(16) float s_xml[8][kMaxG][2];   // [source split][head] (max, sum)
  __shared__ __align__(8) unsigned long long s_push;  // counts the bytes pushed to this CTA by the cluster
  __shared__ int s_abort;
  __shared__ unsigned s_ticket;

  const DecodeCommon& a = args.c;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- (0) overlap with the kernel ahead of this one in the stream, first thing in the kernel: an
  // L2 prefetch of the head of this CTA's slice of the retained cache.  Until the dependency wait
  // nothing the predecessor may have written is read and nothing global is written; a prefetch
  // cannot observe stale data (L2 is the point of coherence) and turns the head of the later TMA
  // stream into L2 hits.  Only the head: about what HBM delivers until the dependency wait is
  // released.  A deeper prefetch queues so much in the memory system that the small, latency-
  // critical loads of q and C_q behind it come back late (measured: 3/8 of the slice is best).
  if (threadIdx.x == kStreamWarps * 32) {
    const int pr0 = min(a.n_kv, (int)blockIdx.x * a.rows_per_split);
    const int pr1 = min(a.n_kv, pr0 + a.rows_per_split);
    const int n_old = min(min(pr1, a.kv_len) - pr0, (3 * a.rows_per_split + 7) / 8);
    if (n_old > 0) {
      const uint64_t pol = policy_evict_first();
      const size_t off = ((size_t)blockIdx.y * a.cap + pr0) * kRowBytes;
      const unsigned bytes = (unsigned)n_old * kRowBytes;
      asm volatile("cp.async.bulk.prefetch.L2.global.L2::cache_hint [%0], %1, %2;" ::"l"(
                       (const unsigned char*)args.layer[blockIdx.z].K + off),
                   "r"(bytes), "l"(pol)
                   : "memory");
      asm volatile("cp.async.bulk.prefetch.L2.global.L2::cache_hint [%0], %1, %2;" ::"l"(
                       (const unsigned char*)args.layer[blockIdx.z].V + off),
                   "r"(bytes), "l"(pol)
                   : "memory");
    }
  }
  cg::cluster_group cluster = cg::this_cluster();
  const int gs = blockIdx.x;             // split index over the whole unit
  const int split = gs % a.nsplit;       // rank inside the cluster
  const int clu = gs / a.nsplit;         // cluster of this unit
  const int n_gs = a.nsplit * a.nclu;
  const int unit = blockIdx.y, layer = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gq = lane >> 2, tq = lane & 3;  // MMA fragment coordinates
  const DecodeLayerPtrs& P = args.layer[layer];
  const DecodeLayerMaps& TM = args.maps[layer];
  const int b = unit / a.Hkv, h = unit % a.Hkv;
  const int hq0 = b * a.Hq + h * a.G;  // first query head of this kv group

  const __nv_bfloat16* q = (const __nv_bfloat16*)P.q;
  const __nv_bfloat16* Cq = (const __nv_bfloat16*)P.C_q;

  const int r0 = min(a.n_kv, gs * a.rows_per_split);
  const int r1 = min(a.n_kv, r0 + a.rows_per_split);
  const int n_sb = (r1 - r0 + kSlotRows - 1) / kSlotRows;  // ring fills of this CTA

  const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* ring_ptr = smem_raw + (ring - smem_u32(smem_raw));
  volatile int* abort_flag = &s_abort;

  // calibration rows of this CTA: the contiguous range [c_begin, c_begin + n_c)
  const int c_per = (a.n_cal + n_gs - 1) / n_gs;
  const int c_begin = min(a.n_cal, gs * c_per);
  const int n_c = RECAL ? 0 : min(a.n_cal, c_begin + c_per) - c_begin;
  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s)
      for (int p = 0; p < 2; ++p) {
        mbar_init(smem_u32(&s_full[s][p]), 1);    // the producer's arrive with the byte count
        mbar_init(smem_u32(&s_empty[s][p]), 4);   // one lane of each of the slot's four warps
      }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_abort = 0;
  }
  if (warp == kStreamWarps && lane == 0) {
    // every CTA of the cluster (this one included) pushes its partial of this CTA's slice and its
    // (max, sum) pairs here: G * dpc * 4 + G * 8 bytes each
    mbar_init(smem_u32(&s_push), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect_tx(smem_u32(&s_push), (uint32_t)(a.nsplit * a.G * (kD / a.nsplit * 4 + 8)));
    asm volatile("prefetch.tensormap [%0];" ::"l"(&TM.k64) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&TM.v64) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&TM.k16) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&TM.v16) : "memory");
  }
  if (tid >= 32 && tid < 32 + a.G && n_c > 0) {  // same for the small operands of the similarity
    const int g = tid - 32;
    asm volatile("cp.async.bulk.prefetch.L2.global.L2::cache_hint [%0], %1, %2;" ::"l"(
                     Cq + ((size_t)(hq0 + g) * a.n_cal + c_begin) * kD),
                 "r"((unsigned)n_c * kRowBytes), "l"(pol_keep)
                 : "memory");
    if (g == 0)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(q + (size_t)hq0 * kD),
                   "r"((unsigned)a.G * kRowBytes)
                   : "memory");
  }
  if (tid < kMaxG) s_best[tid] = 0ull;
  // Address arithmetic of everything that is loaded right after the dependency wait, and of the
  // finish, is done here: a single warp runs a dependent chain of scalar instructions at a few
  // cycles each, and at this kernel's scale a hundred of them behind the wait are a measurable
  // part of a launch (0.4 us each for the similarity loads and for the O_c loads, measured).
  constexpr int kPairsPerPass = kThreads / 4;
  const int pairs = n_c * a.G;
  const int sub4 = tid & 3;
  const int pi0 = tid >> 2;
  const int pg0 = pi0 < pairs ? pi0 % a.G : 0, pc0 = c_begin + (pi0 < pairs ? pi0 / a.G : 0);
  const uint4* qp0 = reinterpret_cast<const uint4*>(q + (size_t)(hq0 + pg0) * kD + sub4 * 32);
  const uint4* cp0 = reinterpret_cast<const uint4*>(Cq + ((size_t)(hq0 + pg0) * a.n_cal + pc0) * kD + sub4 * 32);
  const uint32_t* qr0 = reinterpret_cast<const uint32_t*>(q + (size_t)(hq0 + min(gq, a.G - 1)) * kD) + tq;
  const int dpc = kD / a.nsplit, lg_dpc = 31 - __clz(dpc);  // nsplit is a power of two
  const int n_items = a.G * dpc;
  const bool single = a.nclu == 1;
  const bool early = !RECAL && single && n_items <= kThreads;  // one output element per thread at most
  const int eg = min(tid >> lg_dpc, a.G - 1), ed = split * dpc + (tid & (dpc - 1));
  const float* oc_base = P.O_c + (size_t)(hq0 + eg) * a.n_cal * kD + ed;
  const float* lsec_base = P.LSE_c + (size_t)(hq0 + eg) * a.n_cal;
  asm volatile("" ::"l"(qp0), "l"(cp0), "l"(qr0), "l"(oc_base), "l"(lsec_base), "r"(pg0), "r"(pc0));
  __syncthreads();  // barriers initialised, s_best cleared: nothing of this needs the predecessor
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // One ring fill: rows [r0 + sb * 64, ...) of K and V into slot sb % 3.  Whole slots take four
  // 64-row boxes; the ragged last slot takes 16-row boxes for the row groups that hold valid rows,
  // so a split never pulls more than 15 rows of its neighbour.  Only a 16-row box can reach past
  // row kv_len: the V map of those boxes ends at kv_len, so such V rows arrive as zeros (a zero
  // probability times whatever lies in the caller's memory could still be a NaN); the K rows
  // arrive as they lie in memory and their scores are masked.
  auto fill = [&](int sb) {
    const int s = sb % kSlots, k = sb / kSlots;
    const uint32_t bar = smem_u32(&s_full[s][k & 1]);
    const uint32_t dst = ring + s * kSlotBytes;
    const int row0 = r0 + sb * kSlotRows;
    const int nrows = min(kSlotRows, r1 - row0);
    if (nrows == kSlotRows) {
      mbar_expect_tx(bar, kSlotBytes);
      tma_load_3d(dst, &TM.k64, bar, 0, row0, unit, pol_stream);
      tma_load_3d(dst + kPlaneBytes, &TM.k64, bar, 64, row0, unit, pol_stream);
      tma_load_3d(dst + 2 * kPlaneBytes, &TM.v64, bar, 0, row0, unit, pol_stream);
      tma_load_3d(dst + 3 * kPlaneBytes, &TM.v64, bar, 64, row0, unit, pol_stream);
    } else {
      const int nb = (nrows + kBlkRows - 1) / kBlkRows;
      mbar_expect_tx(bar, (uint32_t)nb * 4u * kBlkRows * 128u);
      for (int j = 0; j < nb; ++j) {
        const uint32_t dj = dst + j * kBlkRows * 128;
        tma_load_3d(dj, &TM.k16, bar, 0, row0 + j * kBlkRows, unit, pol_stream);
        tma_load_3d(dj + kPlaneBytes, &TM.k16, bar, 64, row0 + j * kBlkRows, unit, pol_stream);
        tma_load_3d(dj + 2 * kPlaneBytes, &TM.v16, bar, 0, row0 + j * kBlkRows, unit, pol_stream);
        tma_load_3d(dj + 3 * kPlaneBytes, &TM.v16, bar, 64, row0 + j * kBlkRows, unit, pol_stream);
      }
    }
  };

  // ---- (1) cosine similarities of this CTA's calibration rows: four lanes per (head, row) pair,
  // 72 pairs per pass; the best pair per head goes to s_best while the first slots are in flight
  auto rho_load = [&](int pi, RhoLoad (&r)[2]) {
    r[0] = RhoLoad{}; r[1] = RhoLoad{};
    if (pi < pairs) {
      const int g = pi % a.G, c = c_begin + pi / a.G;
      const uint4* qp = reinterpret_cast<const uint4*>(q + (size_t)(hq0 + g) * kD + sub4 * 32);
      const uint4* cp = reinterpret_cast<const uint4*>(Cq + ((size_t)(hq0 + g) * a.n_cal + c) * kD + sub4 * 32);
      r[0].q0 = __ldg(qp); r[0].q1 = __ldg(qp + 1);
      r[0].c0 = ldg_keep(cp, pol_keep); r[0].c1 = ldg_keep(cp + 1, pol_keep);
      r[1].q0 = __ldg(qp + 2); r[1].q1 = __ldg(qp + 3);
      r[1].c0 = ldg_keep(cp + 2, pol_keep); r[1].c1 = ldg_keep(cp + 3, pol_keep);
    }
  };
  auto rho_finish = [&](int pi, int g, int c, const RhoLoad (&r)[2]) {
    float dot = 0.f, qq = 0.f, cc = 0.f;
    if (pi < pairs) { rho_accumulate(r[0], dot, qq, cc); rho_accumulate(r[1], dot, qq, cc); }
#pragma unroll
    for (int o = 1; o < 4; o <<= 1) {
      dot += __shfl_xor_sync(0xffffffffu, dot, o);
      qq += __shfl_xor_sync(0xffffffffu, qq, o);
      cc += __shfl_xor_sync(0xffffffffu, cc, o);
    }
    if (sub4 == 0 && pi < pairs) {
      const float rho = (qq > 0.f && cc > 0.f) ? dot / (sqrtf(qq) * sqrtf(cc)) : 0.f;
      atomicMax(&s_best[g], rank_key(rho, c));
    }
  };
  // query fragments of the stream warps (B operand of S^T, heads on the 8-column side): their
  // loads go out together with those of the similarity
  uint32_t qa[kD / 16][2];
#pragma unroll
  for (int kk = 0; kk < kD / 16; ++kk) {
    qa[kk][0] = 0u; qa[kk][1] = 0u;
    if (warp < kStreamWarps && gq < a.G) {
      qa[kk][0] = __ldg(qr0 + kk * 8);
      qa[kk][1] = __ldg(qr0 + kk * 8 + 4);
    }
  }
  RhoLoad rl[2];
  rl[0] = RhoLoad{}; rl[1] = RhoLoad{};
  if (pi0 < pairs) {
    rl[0].q0 = __ldg(qp0); rl[0].q1 = __ldg(qp0 + 1);
    rl[0].c0 = ldg_keep(cp0, pol_keep); rl[0].c1 = ldg_keep(cp0 + 1, pol_keep);
    rl[1].q0 = __ldg(qp0 + 2); rl[1].q1 = __ldg(qp0 + 3);
    rl[1].c0 = ldg_keep(cp0 + 2, pol_keep); rl[1].c1 = ldg_keep(cp0 + 3, pol_keep);
  }
  // the first ring fills go out behind the (small) similarity loads, not ahead of them
  if (warp == kStreamWarps) {
    if (lane == 0)
      for (int sb = 0; sb < min(n_sb, kSlots); ++sb) fill(sb);
    __syncwarp();
  }
  // The similarities are finished by the producer warp at once and by a stream warp after its first
  // slot, whose data is already there when the query arrives.  (A) then says this CTA's s_best is
  // final.  Publishing it to the cluster takes a release fence, which is slow while the stream is
  // in flight; the stream warps therefore only hand their updates to the producer warp through a
  // CTA barrier and arrive relaxed, and the producer warp, which has time, makes the one release
  // for the CTA.
  auto rho_rest = [&]() {
    rho_finish(pi0, pg0, pc0, rl);
    for (int base = kPairsPerPass; base < pairs; base += kPairsPerPass) {
      const int pi = base + pi0;
      rho_load(pi, rl);
      rho_finish(pi, pi < pairs ? pi % a.G : 0, c_begin + (pi < pairs ? pi / a.G : 0), rl);
    }
    if (warp != kStreamWarps) {
      asm volatile("barrier.cta.arrive 1, %0;" ::"n"(kThreads) : "memory");
      asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    }
  };

  float o[kD / 16][4];
#pragma unroll
  for (int n = 0; n < kD / 16; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // heads 2tq and 2tq+1

  if (warp == kStreamWarps) {
    rho_rest();
    // ---- (2) producer: refill a slot as soon as its four warps have released it
    if (lane == 0) {
      for (int sb = kSlots; sb < n_sb; ++sb) {
        const int s = sb % kSlots, kp = sb / kSlots - 1;  // the fill that occupies the slot
        if (!mbar_wait(smem_u32(&s_empty[s][kp & 1]), (kp >> 1) & 1, abort_flag, a.status, 0x100u + sb)) break;
        fill(sb);
      }
    }
    __syncwarp();
    // with the last fill under way the producer has nothing left to move: it settles the
    // calibration row (best similarity over the cluster, ties to the largest row index) while the
    // stream warps are still busy
    asm volatile("barrier.cta.sync 1, %0;" ::"n"(kThreads) : "memory");  // the stream warps' updates of s_best
    cluster_arrive();  // (A) with the release for the whole CTA
    cluster_wait();    //     every CTA's s_best can be read
    if (lane < a.G) {
      unsigned long long best = 0ull;
      for (int s = 0; s < a.nsplit; ++s) {
        const unsigned long long k = *cluster.map_shared_rank(&s_best[lane], s);
        best = k > best ? k : best;
      }
      s_bestall[lane] = best;
    }
  } else {
    // ---- (3) stream warps
    const int group = warp >> 2, sub = warp & 3;
    const int mid = lane >> 3;
    bool rho_done = false;
    for (int sb = group; sb < n_sb; sb += 2) {
      const int s = sb % kSlots, k = sb / kSlots;
      const bool ok = mbar_wait(smem_u32(&s_full[s][k & 1]), (k >> 1) & 1, abort_flag, a.status, 0x200u + sb);
      const int row_base = r0 + sb * kSlotRows + sub * kBlkRows;
      if (ok && row_base < r1) {
        const uint32_t sK = ring + s * kSlotBytes;
        const uint32_t sV = sK + 2 * kPlaneBytes;
        // D1: the warp that meets row kv_len takes it from k_new / v_new (the cache row has not
        // been written yet: what arrived for it is stale) and appends it to the cache
        if (a.has_new && a.kv_len >= row_base && a.kv_len < row_base + kBlkRows) {
          const int chunk = lane & 15;
          const int rs = a.kv_len - (r0 + sb * kSlotRows);  // row inside the slot
          const unsigned char* src = (const unsigned char*)(lane < 16 ? P.k_new : P.v_new) +
                                     (size_t)unit * kRowBytes + chunk * 16;
          const uint4 v = *reinterpret_cast<const uint4*>(src);
          unsigned char* dstg = (unsigned char*)(lane < 16 ? P.K : P.V) +
                                ((size_t)unit * a.cap + a.kv_len) * kRowBytes + chunk * 16;
          *reinterpret_cast<uint4*>(dstg) = v;
          *reinterpret_cast<uint4*>(ring_ptr + s * kSlotBytes + (lane < 16 ? 0 : 2 * kPlaneBytes) +
                                    plane_off(rs, chunk)) = v;
          __syncwarp();
        }
        // S^T: two accumulators (even and odd k-steps) halve the dependent chain
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4(sK + plane_off(sub * kBlkRows + (lane & 7) + (mid & 1) * 8, kk * 2 + (mid >> 1)), a0, a1, a2, a3);
          if (kk & 1) mma_bf16_16816(sb2, a0, a1, a2, a3, qa[kk][0], qa[kk][1]);
          else mma_bf16_16816(sa, a0, a1, a2, a3, qa[kk][0], qa[kk][1]);
        }
        // online softmax per head over the 16 keys of the block (keys gq and gq + 8 live here)
        const bool v0 = row_base + gq < r1, v1 = row_base + gq + 8 < r1;
        const float x00 = v0 ? (sa[0] + sb2[0]) * a.scale2 : -INFINITY;
        const float x01 = v0 ? (sa[1] + sb2[1]) * a.scale2 : -INFINITY;
        const float x10 = v1 ? (sa[2] + sb2[2]) * a.scale2 : -INFINITY;
        const float x11 = v1 ? (sa[3] + sb2[3]) * a.scale2 : -INFINITY;
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
          ldmatrix_x4_trans(sV + plane_off(sub * kBlkRows + (lane & 7) + (mid >> 1) * 8, n * 2 + (mid & 1)), a0, a1, a2, a3);
          mma_bf16_16816(o[n], a0, a1, a2, a3, pb0, pb1);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&s_empty[s][k & 1]));  // the slot may be refilled
      if (!rho_done) { rho_rest(); rho_done = true; }
    }
    if (!rho_done) rho_rest();
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, off);
      l1 += __shfl_xor_sync(0xffffffffu, l1, off);
    }
  }

  // ---- (4) the chosen O_c elements and LSE_c start their way while the partials are combined
  if (warp < kStreamWarps) cluster_wait();  // (A): the stream warps only pass it
  __syncthreads();  // all warps are done with the ring: reuse it for the combine
  // the common case has one output element per thread at most: its O_c element and LSE_c are
  // loaded now and arrive while the partials are combined
  if (!RECAL && (!single || n_items > kThreads)) {
    if (tid < a.G && single) {
      const size_t crow = (size_t)(hq0 + tid) * a.n_cal + (unsigned)(s_bestall[tid] & 0xffffffffull);
      const float* orow = P.O_c + crow * kD;
#pragma unroll
      for (int i = 0; i < 4; ++i) asm volatile("prefetch.global.L2 [%0];" ::"l"(orow + i * 32));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(P.LSE_c + crow));
    }
  }
  float lse_c_early = 0.f, oc_early = 0.f;
  if (early && tid < n_items) {
    const unsigned cs = (unsigned)(s_bestall[eg] & 0xffffffffull);
    lse_c_early = ldg_keep(lsec_base + cs, pol_keep);
    oc_early = ldg_keep(oc_base + (size_t)cs * kD, pol_keep);
  }

  // ---- (5) CTA combine of the eight stream warps, pushed to the owners of the output slices:
  // CTA r of the cluster owns dimensions [r * dpc, (r + 1) * dpc) of every head of the group
  float* wo = reinterpret_cast<float*>(ring_ptr);          // [warp][8][kWoStride]
  float* wml = wo + kStreamWarps * kMaxG * kWoStride;       // [warp][8][2]
  if (warp < kStreamWarps && 2 * tq < a.G) {
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
  // 256 threads: thread t owns dimensions 2 (t & 63) and 2 (t & 63) + 1 of head (t >> 6) + 4k, so the
  // scale factors of the eight warps are worked out once for two elements, which go to their owner
  // in one 8-byte store; all loads are done before the pushes (stores through generic pointers,
  // which the compiler will not move loads across)
  if (tid < 256) {
    const int d0 = 2 * (tid & 63);
    for (int g = tid >> 6; g < a.G; g += 4) {
      float mw[kStreamWarps], M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kStreamWarps; ++w) { mw[w] = wml[(w * kMaxG + g) * 2]; M = fmaxf(M, mw[w]); }
      float Lsum = 0.f, acc0 = 0.f, acc1 = 0.f;
#pragma unroll
      for (int w = 0; w < kStreamWarps; ++w) {
        const float sc = mw[w] > -INFINITY ? ex2_approx(mw[w] - M) : 0.f;
        const float2 wv = *reinterpret_cast<const float2*>(wo + (w * kMaxG + g) * kWoStride + d0);
        Lsum = fmaf(wml[(w * kMaxG + g) * 2 + 1], sc, Lsum);
        acc0 = fmaf(wv.x, sc, acc0);
        acc1 = fmaf(wv.y, sc, acc1);
      }
      const int own = d0 >> lg_dpc;  // dpc is even: both dimensions have the same owner
      push_f32x2(cluster_addr(smem_u32(s_xpart + (split * kMaxG + g) * dpc + (d0 - own * dpc)), own), acc0, acc1,
                 cluster_addr(smem_u32(&s_push), own));
      if ((tid & 63) < a.nsplit) {  // the (max, sum) pair of this split goes to every CTA of the cluster
        push_f32x2(cluster_addr(smem_u32(&s_xml[split][g][0]), tid & 63), M, Lsum,
                   cluster_addr(smem_u32(&s_push), tid & 63));
      }
    }
  }
  // (B) everything pushed to this CTA has arrived when its byte count is complete.  No cluster
  // barrier: a CTA waits for its own data only, and it cannot leave before the others have read its
  // s_best, because their pushes, which it waits for, come after those reads.  That argument needs
  // the wait to be sat out: a CTA whose earlier wait ran out (abort flag raised) must not skip it,
  // or its peers, which always reach their pushes, would read and write the shared memory of a
  // CTA that has left.  Only the wait's own time limit remains as the way out.
  mbar_wait_sit_out(smem_u32(&s_push), 0, abort_flag, a.status, 0x300u);

  // ---- (6) finish: reduce the splits for this CTA's output slice (local data only from here on,
  // so no CTA has to wait for another before it leaves)
  const int lu = layer * a.units + unit;
  for (int item = tid; item < n_items; item += kThreads) {
    const int g = item >> lg_dpc, dl = item & (dpc - 1), d = split * dpc + dl;
    const int hq = hq0 + g;
    const unsigned long long best = s_bestall[g];
    float ms[8], ls[8], xs[8], M = -INFINITY;
#pragma unroll
    for (int s = 0; s < 8; ++s) {  // all loads first (nsplit <= 8)
      const bool on = s < a.nsplit;
      ms[s] = on ? s_xml[s][g][0] : -INFINITY;
      ls[s] = on ? s_xml[s][g][1] : 0.f;
      xs[s] = on ? s_xpart[(s * kMaxG + g) * dpc + dl] : 0.f;
      M = fmaxf(M, ms[s]);
    }
    float Lsum = 0.f, acc = 0.f;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      const float sc = ms[s] > -INFINITY ? ex2_approx(ms[s] - M) : 0.f;
      Lsum = fmaf(ls[s], sc, Lsum);
      acc = fmaf(xs[s], sc, acc);
    }
    if (single) {
      if constexpr (RECAL) {
        recal_store(a, P, hq, d, acc, M, Lsum);
      } else {
        float lse_c = lse_c_early, oc = oc_early;
        if (!early) {
          const size_t crow = (size_t)hq * a.n_cal + (unsigned)(best & 0xffffffffull);
          lse_c = __ldg(P.LSE_c + crow);
          oc = __ldg(P.O_c + crow * kD + d);
        }
        merge_store(a, P, hq, d, acc, M, Lsum, best, lse_c, oc);
      }
    } else {
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
  if (!single) {
    // ---- (7) several clusters per unit: the CTA that takes the unit's last ticket merges them
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
        const float lse_c = RECAL ? 0.f : __ldg(P.LSE_c + crow);
        const float oc = RECAL ? 0.f : __ldg(P.O_c + crow * kD + d);
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
        if constexpr (RECAL) recal_store(a, P, hq, d, acc, M, Lsum);
        else merge_store(a, P, hq, d, acc, M, Lsum, best, lse_c, oc);
      }
      if (tid == 0) a.counters[lu] = 0u;  // ready for the next launch on this workspace
    }
  }
}

}  // namespace

bool make_decode_maps(const DecodeCommon& c, const DecodeLayerPtrs& L, DecodeLayerMaps* out) {
  // Three of the four maps cover all `cap` rows of the cache, whatever kv_len is, so one encoding
  // serves every step on a cache: a small per-thread table keyed by everything the encoding depends
  // on (the two base addresses, the capacity, the number of units) returns them on the following
  // calls (encoding all four on every call cost more host time than the kernel runs).  An entry can
  // never be stale: equal keys encode equal maps.  The fourth, V in 16-row boxes, is the only one
  // through which rows at or beyond kv_len can reach a product; it ends at kv_len, so the TMA unit
  // delivers zeros for those rows, and is encoded per call.
  struct Entry { const void* K; const void* V; int cap, units; DecodeLayerMaps maps; };
  constexpr int kEntries = 64;
  static thread_local Entry table[kEntries];
  static thread_local int next = 0;
  const uint64_t strides[2] = {(uint64_t)kRowBytes, (uint64_t)c.cap * kRowBytes};
  const uint32_t box64[2] = {(uint32_t)kSlotRows, 1}, box16[2] = {(uint32_t)kBlkRows, 1};
  const uint64_t dims_v16[2] = {(uint64_t)(c.kv_len > 0 ? c.kv_len : 1), (uint64_t)c.units};
  for (int i = 0; i < kEntries; ++i) {
    const Entry& e = table[i];
    if (e.K == L.K && e.V == L.V && e.cap == c.cap && e.units == c.units && e.K != nullptr) {
      *out = e.maps;
      return make_tensor_map_bf16(&out->v16, L.V, 3, dims_v16, strides, box16);
    }
  }
  const uint64_t dims[2] = {(uint64_t)c.cap, (uint64_t)c.units};
  if (!(make_tensor_map_bf16(&out->k64, L.K, 3, dims, strides, box64) &&
        make_tensor_map_bf16(&out->v64, L.V, 3, dims, strides, box64) &&
        make_tensor_map_bf16(&out->k16, L.K, 3, dims, strides, box16) &&
        make_tensor_map_bf16(&out->v16, L.V, 3, dims_v16, strides, box16)))
    return false;
  Entry& e = table[next];
  next = (next + 1) % kEntries;
  e.K = L.K; e.V = L.V; e.cap = c.cap; e.units = c.units; e.maps = *out;
  return true;
}

namespace {

template <int NL, bool RECAL, int kSlots>
cudaError_t launch_decode_s(const DecodeArgsT<NL>& a, cudaStream_t st) {
  constexpr int kSmemBytes = smem_bytes(kSlots);
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(decode_kernel<NL, RECAL, kSlots>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.c.nsplit * a.c.nclu, a.c.units, a.c.n_layers);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;  // the splits of a unit are one cluster
  attr[0].val.clusterDim.x = a.c.nsplit;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  e = cudaLaunchKernelEx(&cfg, decode_kernel<NL, RECAL, kSlots>, a);
  if (e != cudaSuccess) return e;
  count_launch(1);
  return cudaGetLastError();
}

// More CTAs than SMs and short slices (a stack of small caches in one launch): the narrow ring, so
// that two CTAs share an SM and one's fixed chain overlaps the other's stream.  Long slices keep the
// wide ring, which they need to stream at full rate (measured: 32 layers of 129-384 rows 115 -> 95 us
// with the narrow ring, 8 caches of 2049 rows 53 -> 57 us).
template <int NL, bool RECAL>
cudaError_t launch_decode_t(const DecodeArgsT<NL>& a, cudaStream_t st) {
  const long long ctas = (long long)a.c.nsplit * a.c.nclu * a.c.units * a.c.n_layers;
  const bool narrow = ctas > kDecodeTargetCtas && a.c.rows_per_split <= 8 * kSlotRows;
  return narrow ? launch_decode_s<NL, RECAL, kSlotsNarrow>(a, st) : launch_decode_s<NL, RECAL, kSlotsWide>(a, st);
}

}  // namespace

cudaError_t launch_decode(const DecodeArgsT<1>& a, cudaStream_t st) { return launch_decode_t<1, false>(a, st); }
cudaError_t launch_decode(const DecodeArgsT<kDecodeMaxLayers>& a, cudaStream_t st) {
  return launch_decode_t<kDecodeMaxLayers, false>(a, st);
}
cudaError_t launch_recalibrate(const DecodeArgsT<1>& a, cudaStream_t st) { return launch_decode_t<1, true>(a, st); }

}  // namespace calidrop
