/*
 * calidrop.h -- C ABI of the B200 (sm_100a) CaliDrop hot path.
 *
 * Two operations, after "CaliDrop: KV Cache Compression with Calibration":
 *
 *   calidrop_compress  end of prefill (Algorithm 1, lines 3-8): score the prompt's keys
 *                      with an observation window of recent queries, pool the scores, keep
 *                      a per-kv-head top-k budget of KV rows, compact them, and precompute
 *                      the calibration term (O_c, LSE_c, C_q) over the evicted rows.
 *   calidrop_decode    one decode step (Algorithm 2, lines 1-2 and 9-14): attention of the
 *                      new query over the retained cache, cosine similarity with the stored
 *                      calibration queries, threshold gate, and the merge of Eq. 1-2.
 *
 * Around them: calidrop_calibrate (the second half of calidrop_compress for a kept list chosen by
 * another eviction rule), calidrop_select_streaming and calidrop_select_from_scores (the kept lists
 * of two such rules: sinks plus recent rows, and top-k of accumulated scores, which
 * calidrop_accumulated_scores computes when the prefill does not supply them),
 * calidrop_gather_evicted, calidrop_offload_evicted, calidrop_reload_evicted and
 * calidrop_recalibrate (Algorithm 1 line 4 and Algorithm 2 lines 3-8: the evicted rows compacted,
 * moved to host memory and back beside the decode, and the recompute of a calibration entry from
 * them), calidrop_decode_batched (several layers in one launch) and calidrop_decode_static (no
 * caller workspace).  The field calib_size of the parameters is the calibration size of
 * Section 4.4.
 *
 * Conventions
 *   - Unless a comment says HOST, every tensor pointer is a DEVICE pointer to a contiguous,
 *     16-byte aligned buffer on the current device.  "bf16" buffers hold bfloat16 values.
 *   - The library allocates nothing and owns no buffer: all of them, including the workspaces,
 *     belong to the caller.  Two things outlast a call.  (1) calidrop_decode_static's built-in
 *     scratch array (see there).  (2) Small per-thread and per-device tables of derived values:
 *     whether a kernel's shared-memory attribute has been set on a device, the argument block of
 *     the batched decode, and the TMA descriptors of the caches the decode entry points have
 *     seen, keyed by the cache's addresses, capacity and unit count.  A descriptor is a pure
 *     function of its key, so a table entry is never stale and is never dereferenced by the
 *     library itself; freeing a cache needs no call into the library.
 *   - Every call validates its arguments on the host BEFORE enqueueing anything; a call that
 *     returns a non-zero status has had no effect.  Work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL is the default stream) and the call returns
 *     without synchronising.
 *   - Status codes: 0 = CALIDROP_OK, negative = error (see below).  No exceptions, no abort,
 *     no device trap.
 *   - Logits are q.k * softmax_scale with softmax_scale = 1/sqrt(D) when the field is 0.
 *     (Algorithm 1 prints the exponent of C_weight divided by d_k; Eq. 1-2 only hold with
 *     the attention's own 1/sqrt(d_k), which is what is used everywhere here.)
 *   - C_weight of Algorithm 1 is stored as its logarithm LSE_c; A_weight of Algorithm 2
 *     likewise as LSE_a.  alpha_i = exp(LSE_a - logaddexp(LSE_a, LSE_c)), which is Eq. 2.
 */
#ifndef CALIDROP_H_
#define CALIDROP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CALIDROP_OK 0
#define CALIDROP_INVALID_ARG (-1)         /* null/misaligned pointer, inconsistent sizes      */
#define CALIDROP_UNSUPPORTED (-2)         /* D != 128, Hq/Hkv > 8, device is not sm_100       */
#define CALIDROP_WORKSPACE_TOO_SMALL (-3)
#define CALIDROP_CUDA_ERROR (-4)          /* a launch or runtime call failed                  */
#define CALIDROP_SCRATCH_LIMIT (-5)       /* needs more than CALIDROP_STATIC_SCRATCH_BYTES    */

#define CALIDROP_MAX_LAYERS 32            /* layers per calidrop_decode_batched call          */
#define CALIDROP_STATIC_SCRATCH_BYTES (4u << 20)  /* built-in scratch of calidrop_decode_static */

typedef struct calidrop_params {
  int32_t B, Hq, Hkv, D;        /* D must be 128; Hq % Hkv == 0; G = Hq/Hkv <= 8              */
  int32_t L;                    /* prompt length; K, V are [B, Hkv, L, D]                      */
  int32_t window;               /* W >= 1: observation window = the last W prompt positions    */
  int32_t pool;                 /* odd >= 1: average-pool kernel over the votes                */
  int32_t budget;               /* retained prompt rows per kv head, INCLUDING the W window    */
                                /* rows; budget >= L keeps everything                          */
  int32_t n_cal;                /* 1..W calibration queries = the last n_cal window rows;      */
                                /* 1 is Algorithm 1 as printed (the last query only)           */
  int32_t cap;                  /* row capacity of K_kept/V_kept: >= min(budget,L) + appended  */
  float   softmax_scale;        /* 0 => 1/sqrt(D)                                              */
  float   theta1, theta2;       /* decode: rho < theta1 raises needs_recompute; rho > theta2   */
                                /* applies the calibration; theta2 <= -1 always applies it     */
  int32_t calib_size;           /* compress: the "calibration size" of the paper's Section 4.4 */
                                /* (Efficiency Optimization): 0 = every evicted row takes part */
                                /* in the calibration (Algorithm 1 as printed); m > 0 = only   */
                                /* the m evicted rows of highest pooled vote (ties: lowest     */
                                /* index), the rest are dropped for good; -1 = none (O_c = 0,  */
                                /* LSE_c = -inf).  A zero-initialised struct gives 0.          */
} calidrop_params;

/*
 * Bytes of scratch calidrop_compress needs for these parameters (0 if they are invalid).
 */
size_t calidrop_compress_workspace_bytes(const calidrop_params* p);

/*
 * Compress-and-calibrate (Algorithm 1, lines 3-8, with the SnapKV eviction rule the paper's
 * Sections 1 and 4.1.3 describe: observation window + pooled accumulated attention).
 *
 * Per (batch b, kv head h), with G query heads per kv head and candidates t in [0, L-W):
 *   a[g][j][t]  softmax row of window query j of head h*G+g (prompt position L-W+j) over
 *               the keys t <= L-W+j it can see;
 *   vote[t]   = sum_g sum_j a[g][j][t];
 *   pooled[t] = (1/pool) sum_{|d| <= pool/2} vote[t+d]   (zero padding, constant divisor);
 *   kept      = the budget-W candidates with the largest pooled[t] (ties: lowest index),
 *               in ascending order, followed by the window rows L-W .. L-1;
 *   E         = [0, L-W) \ kept, the evicted rows; with calib_size = m > 0 only the m of them
 *               with the largest pooled[t] (the candidates of rank budget-W .. budget-W+m-1 in the
 *               same order), with calib_size = -1 none;
 *   for c < n_cal, q_c = Q_obs[b, h*G+g, W-n_cal+c]:
 *     LSE_c[c] = log sum_{t in E} exp(q_c.k_t * scale),  O_c[c] = Att(q_c, K_E, V_E),
 *     C_q[c] = q_c.                                       (lines 5-8 of Algorithm 1)
 * budget >= L keeps all L rows (n_kept = L), LSE_c = -inf, O_c = 0.
 *
 *   Q_obs   in  [B, Hq, W, D] bf16   the last W prompt queries, as the attention sees them
 *   K, V    in  [B, Hkv, L, D] bf16
 *   lse_obs in  [B, Hq, W] f32 or NULL: natural-log softmax denominators of those W rows of
 *               the prefill attention (over keys t <= L-W+j, same scale).  Supplying them
 *               skips the pass that recomputes them.  Not validated.
 *   kept_idx out [B, Hkv, n_kept] i32, n_kept = min(budget, L)
 *   K_kept, V_kept out [B, Hkv, cap, D] bf16; rows 0..n_kept-1 are written (bit copies)
 *   O_c     out [B, Hq, n_cal, D] f32
 *   LSE_c   out [B, Hq, n_cal] f32
 *   C_q     out [B, Hq, n_cal, D] bf16
 *   workspace   scratch of at least calidrop_compress_workspace_bytes(p) bytes, 256-byte
 *               aligned; contents are undefined afterwards.  Two calls that overlap on the
 *               device must not share a workspace.
 *
 * Errors: INVALID_ARG for a null or misaligned pointer, Hq % Hkv != 0, window < 1,
 * even or non-positive pool, n_cal outside 1..W, budget <= window while budget < L,
 * L < window while budget < L, cap < n_kept; UNSUPPORTED for D != 128 or G > 8 or a device
 * that is not compute capability 10.x; WORKSPACE_TOO_SMALL; CUDA_ERROR.
 */
int calidrop_compress(const calidrop_params* p,
                      const void* Q_obs, const void* K, const void* V, const float* lse_obs,
                      int32_t* kept_idx, void* K_kept, void* V_kept,
                      float* O_c, float* LSE_c, void* C_q,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Gather and calibrate for a kept list chosen by the CALLER (Algorithm 1, line 3 "Select
 * KV_compress using eviction strategy", lets any eviction rule stand there; lines 5-8 are the same
 * for all of them): steps 2 and 3 of calidrop_compress with `kept_idx` as an INPUT, e.g. the
 * index rule of a sink-plus-recent cache or an accumulated-score rule computed elsewhere.
 *
 *   kept_idx in [B, Hkv, n_kept] i32, n_kept = min(budget, L), ascending per (b, kv head), each
 *            entry in [0, L), no duplicates.  The last `window` prompt rows count as kept whether
 *            the list names them or not (E = [0, L - window) minus the listed rows), so a list
 *            that is to be consistent with the gathered cache contains them.
 *   all other arguments, the workspace size and the errors: as for calidrop_compress.  The row
 *            LSE of the calibration queries is taken from lse_obs or, if that is NULL, computed by
 *            the statistics pass of the window scoring.  `pool` of `p` is not used.
 */
int calidrop_calibrate(const calidrop_params* p,
                       const void* Q_obs, const void* K, const void* V, const float* lse_obs,
                       const int32_t* kept_idx, void* K_kept, void* V_kept,
                       float* O_c, float* LSE_c, void* C_q,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * Kept lists of two other eviction rules, written on the device for calidrop_calibrate (the paper's
 * Section 4.1.2 applies CaliDrop on top of StreamingLLM, H2O and SnapKV alike; Section 4.1.3 gives
 * their settings: StreamingLLM with 32 sink tokens plus the most recent ones, H2O with half of the
 * budget for the heavy hitters of the accumulated attention score and half for the most recent).
 *
 * calidrop_select_streaming: kept = the first n_sink prompt rows and the last n_kept - n_sink ones,
 *   n_kept = min(budget, L).  INVALID_ARG unless 0 <= n_sink <= n_kept - min(window, n_kept) (the
 *   observation-window rows are part of the recent ones).
 * calidrop_select_from_scores: kept = the budget - tail rows of [0, L - tail) with the largest
 *   pooled score (zero-padded average pool of kernel `pool` of `p`, 1 for none; ties to the lowest
 *   index) and the last `tail` rows.  With the accumulated attention score of the prefill (its
 *   column sums over all queries, a by-product of the prefill attention, or the output of
 *   calidrop_accumulated_scores below) and tail = budget / 2 this is H2O's rule; with the window votes and tail = window it is
 *   the selection step of calidrop_compress.
 *     scores in [B, Hkv, L] f32, finite and non-negative (they are ordered by their bit patterns);
 *            entries at and beyond L - tail are not read
 *     tail   window <= tail < budget < L
 *     workspace: a calidrop_compress workspace for `p` (the pooled scores and a bitmap go there)
 *   UNSUPPORTED beyond 262144 prompt rows.
 *   kept_idx out [B, Hkv, n_kept] i32, ascending.
 * calidrop_accumulated_scores: H2O's importance measure (Section 4.1.2: the accumulated attention
 *   score) for callers whose prefill does not hand it over:
 *       scores[b, h, t] = sum over the G query heads of kv head h and over the prompt queries i >= t
 *                         of softmax_i(q_i . k / sqrt(D))[t]      (causal attention, column sums)
 *   in two tensor-core passes over Q and K (row statistics, then column sums; fp32 throughout, no
 *   atomics: bit-reproducible).  It costs as much as the prefill attention itself, L^2 D flop per
 *   head, and is therefore no part of calidrop_compress.
 *     Q_full in  [B, Hq, L, D] bf16, every prompt query (its last `window` rows are Q_obs)
 *     K      in  [B, Hkv, L, D] bf16
 *     scores out [B, Hkv, L] f32
 *     workspace: calidrop_accumulated_scores_workspace_bytes(p) bytes (the row statistics,
 *            4 B Hq L), 256-byte aligned; WORKSPACE_TOO_SMALL otherwise
 */
int calidrop_select_streaming(const calidrop_params* p, int32_t n_sink, int32_t* kept_idx, void* stream);
int calidrop_select_from_scores(const calidrop_params* p, const float* scores, int32_t tail, int32_t* kept_idx,
                                void* workspace, size_t workspace_bytes, void* stream);
size_t calidrop_accumulated_scores_workspace_bytes(const calidrop_params* p);
int calidrop_accumulated_scores(const calidrop_params* p, const void* Q_full, const void* K, float* scores,
                                void* workspace, size_t workspace_bytes, void* stream);

/*
 * The complement of calidrop_compress's gather: the evicted candidate rows, compacted, for the
 * caller to offload ("offload them to the CPU", Algorithm 1 line 4) and to hand back to
 * calidrop_recalibrate when a decode step raises needs_recompute.
 *
 *   kept_idx  in  [B, Hkv, n_kept] i32 as written by calidrop_compress (or given to calidrop_calibrate)
 *   evict_idx out [B, Hkv, n_evict] i32, n_evict = L - budget: the rows of [0, L - window) that
 *             kept_idx does not list, ascending
 *   K_evict, V_evict out [B, Hkv, n_evict, D] bf16: bit copies of those rows
 *   workspace as for calidrop_compress (its kept bitmap is rebuilt from kept_idx)
 * With calib_size = m > 0 the rows are the m calibrated ones (n_evict = min(m, L - budget)): which
 * they are depends on the votes, so `workspace` must then be the workspace of the calidrop_compress
 * call that wrote kept_idx (same parameters), not used for anything else in between; that call
 * leaves the list there.
 * INVALID_ARG also when budget >= L (nothing is evicted) or calib_size = -1 (nothing is kept for
 * calibration).
 */
int calidrop_gather_evicted(const calidrop_params* p, const void* K, const void* V, const int32_t* kept_idx,
                            int32_t* evict_idx, void* K_evict, void* V_evict,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Offload and reload of the compacted evicted rows ("Offload KV_evict" in Algorithm 1, line 4;
 * "reload" in Algorithm 2, line 4; Section 3.2: the evicted entries move to CPU memory and come
 * back when a recomputation is due).  Each call enqueues one asynchronous copy per tensor on
 * `copy_stream`, a stream of the caller's that is normally NOT the compute stream, so that the
 * transfer runs beside the decode steps:
 *   calidrop_offload_evicted   K_evict, V_evict (device) -> K_host, V_host (HOST)
 *   calidrop_reload_evicted    K_host, V_host (HOST) -> K_evict, V_evict (device)
 *
 *   K_evict, V_evict  device [B, Hkv, n_evict, D] bf16 (as written by calidrop_gather_evicted)
 *   K_host, V_host    HOST buffers of the same size; page-locked (cudaHostAlloc / cudaHostRegister)
 *                     if the copy is to be asynchronous with respect to the host
 *   wait_event        cudaEvent_t or NULL: copy_stream waits for it first (e.g. recorded on the
 *                     compute stream after calidrop_gather_evicted, or after the last use of the rows)
 *   done_event        cudaEvent_t or NULL: recorded on copy_stream behind the copies; the compute
 *                     stream waits for it (cudaStreamWaitEvent) before calidrop_recalibrate reads the rows
 * The library keeps neither the events nor the pointers.  Errors: INVALID_ARG (null pointer,
 * n_evict < 1), CUDA_ERROR.
 */
int calidrop_offload_evicted(const calidrop_params* p, int32_t n_evict, const void* K_evict, const void* V_evict,
                             void* K_host, void* V_host, void* copy_stream, void* wait_event, void* done_event);
int calidrop_reload_evicted(const calidrop_params* p, int32_t n_evict, const void* K_host, const void* V_host,
                            void* K_evict, void* V_evict, void* copy_stream, void* wait_event, void* done_event);

/*
 * Recompute one calibration entry with the current query (Algorithm 2, lines 4-6, taken when
 * rho < theta1; the printed "Q_-1" is read as the current query Q_t, which line 6 stores):
 * per (b, query head hq of kv head h)
 *   O_c[b, hq, slot, :] = attention of q[b, hq] over the evicted rows K_evict/V_evict[b, h, 0..n_evict),
 *   LSE_c[b, hq, slot]  = log of its softmax denominator,
 *   C_q[b, hq, slot, :] = q[b, hq].
 * The other calibration rows are left as they are; with n_cal = 1 this is the paper's update.
 * The caller then repeats the decode step (whose similarity with the new C_q row is 1).
 *
 *   q in [B, Hq, D] bf16; K_evict, V_evict in [B, Hkv, n_evict, D] bf16 (e.g. from
 *   calidrop_gather_evicted, reloaded); n_evict >= 1; slot in [0, n_cal);
 *   O_c, LSE_c, C_q in/out as written by calidrop_compress;
 *   workspace: a decode workspace (see calidrop_decode_workspace_bytes / _init).
 * The rows are streamed by the decode kernel (same split, same bounded waits, same error word).
 */
int calidrop_recalibrate(const calidrop_params* p, const void* q, const void* K_evict, const void* V_evict,
                         int32_t n_evict, int32_t slot, float* O_c, float* LSE_c, void* C_q,
                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * Offsets (bytes from the workspace base) of intermediate arrays of the last
 * calidrop_compress call that used this workspace, for diagnostics and tests:
 *   vote   [B, Hkv, L-W] f32, pooled [B, Hkv, L-W] f32, row_lse [B, Hq, W] f32 (natural log;
 *   not written when lse_obs was supplied), status u32.
 * status is 0 after a call whose kernels all ran to completion.  The tensor-core kernels wait
 * on their copy/MMA pipelines with a time limit; a wait that expires (which indicates a bug or
 * a failing device, not bad input) stores a non-zero code here and the kernel ends early, so
 * the call's outputs are then undefined.  A caller that wants the check reads the word after
 * synchronising the stream.
 * Returns CALIDROP_OK, or INVALID_ARG if the parameters are invalid.
 */
typedef struct calidrop_compress_layout {
  size_t vote_offset, pooled_offset, row_lse_offset, status_offset;
} calidrop_compress_layout;
int calidrop_compress_workspace_layout(const calidrop_params* p, calidrop_compress_layout* out);

/*
 * Bytes of scratch calidrop_decode needs when the retained cache holds at most kv_len_max
 * rows after the append (0 if the parameters are invalid).  For calidrop_decode_batched
 * multiply by the number of layers.
 */
size_t calidrop_decode_workspace_bytes(const calidrop_params* p, int32_t kv_len_max);

/*
 * Zero a decode workspace (asynchronously on `stream`).  A decode workspace must be zeroed
 * once before its first use; every decode call leaves it ready for the next one.  Calls
 * that overlap on the device must not share a workspace.
 */
int calidrop_decode_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Byte offset, from the base of a decode workspace, of its 32-bit error word (the same offset
 * for every layer count).  The decode kernel waits on its copy pipeline with a time limit; a
 * wait that expires (a bug or a failing device, not bad input) stores a non-zero code there and
 * the kernel runs to its end without hanging, with undefined outputs for that call.  The word
 * stays 0 otherwise.  Returns (size_t)-1 if the parameters are invalid.
 */
size_t calidrop_decode_workspace_status_offset(const calidrop_params* p);

/*
 * One decode step for one layer (Algorithm 2, lines 1-2 and 9-14).
 *
 * Per (b, query head hq of kv head h):
 *   if k_new != NULL the step's key/value rows are first stored at row kv_len of the cache;
 *   (O_a, LSE_a) = attention of q over cache rows [0, n_kv), n_kv = kv_len + (k_new ? 1 : 0),
 *                  with the log of its softmax denominator;            (line 1)
 *   rho_c = cos(q, C_q[c]) (0 if either norm is 0); c* = argmax_c rho_c, ties to the
 *           largest c; rho = rho_{c*};                                  (line 2)
 *   needs_recompute = rho < theta1  (lines 3-8, the reload of the evicted KV, are the
 *           caller's business: this call only raises the flag);
 *   if (rho > theta2 or theta2 <= -1) and LSE_c[c*] > -inf:             (lines 9-12, Eq. 1-2)
 *        LSE = logaddexp(LSE_a, LSE_c[c*]);
 *        out = exp(LSE_a - LSE) O_a + exp(LSE_c[c*] - LSE) O_c[c*];
 *   else out = O_a, LSE = LSE_a.                                        (lines 13-14)
 *
 *   q        in  [B, Hq, D] bf16
 *   k_new, v_new in [B, Hkv, D] bf16, or both NULL (no append)
 *   K_kept, V_kept in/out [B, Hkv, cap, D] bf16; row kv_len is written when k_new != NULL.
 *            The caller advances kv_len by one after an appending call.
 *   kv_len   rows valid before this call; kv_len + (k_new ? 1 : 0) must be in 1..cap
 *   O_c, LSE_c, C_q in: as written by calidrop_compress
 *   out      out [B, Hq, D] bf16
 *   lse_out  out [B, Hq] f32 or NULL: the log-denominator that `out` corresponds to
 *   flags    out [B, Hq] u8 or NULL: bit 0 calibration applied, bit 1 needs_recompute,
 *            bits 2..7 c* (only when n_cal <= 64)
 *   workspace    zero-initialised scratch (see calidrop_decode_workspace_init) of at least
 *            calidrop_decode_workspace_bytes(p, kv_len + 1) bytes, 256-byte aligned
 *
 * Only B, Hq, Hkv, D, n_cal, cap, softmax_scale, theta1, theta2 of `p` are read.
 * Errors as for calidrop_compress.
 */
int calidrop_decode(const calidrop_params* p,
                    const void* q, const void* k_new, const void* v_new,
                    void* K_kept, void* V_kept, int32_t kv_len,
                    const float* O_c, const float* LSE_c, const void* C_q,
                    void* out, float* lse_out, uint8_t* flags,
                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same decode step for n_layers independent layers of identical shape in ONE launch
 * (the attention layers of a model stack do not depend on each other inside this path once
 * their queries are known; a stack of small retained caches is otherwise launch-bound).
 * `layers` is a HOST array of n_layers entries whose members are the device pointers of
 * calidrop_decode, per layer.  n_layers must be in 1..CALIDROP_MAX_LAYERS.  The workspace
 * must hold n_layers * calidrop_decode_workspace_bytes(p, kv_len + 1) bytes.
 */
typedef struct calidrop_decode_layer {
  const void* q;
  const void* k_new;
  const void* v_new;
  void* K_kept;
  void* V_kept;
  const float* O_c;
  const float* LSE_c;
  const void* C_q;
  void* out;
  float* lse_out;
  uint8_t* flags;
} calidrop_decode_layer;

int calidrop_decode_batched(const calidrop_params* p, int32_t n_layers,
                            const calidrop_decode_layer* layers /* HOST */, int32_t kv_len,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * calidrop_decode for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the same decode step, not another operation.)
 *
 * Some hosts of this library hand it inputs and outputs but have no way to give it a
 * workspace: a plugin slot of an inference runtime whose memory planner was frozen before the
 * library was loaded, a callback that runs where cudaMalloc is forbidden (inside a stream
 * capture, or in a process whose device memory is owned entirely by another allocator), or
 * code that must not fail for lack of memory.  For them the split-K scratch of the decode
 * kernel lives in a fixed array of CALIDROP_STATIC_SCRATCH_BYTES (4 MiB) of device memory
 * that is part of the library image: every GPU that loads the library holds it until the
 * process exits, and this call, like the others, allocates and frees nothing.
 *
 * Arguments and results are exactly those of calidrop_decode without `workspace` and
 * `workspace_bytes`; the two entry points run the same kernel with the same split factor.
 *
 *   - Limit: calidrop_decode_workspace_bytes(p, kv_len + 1) must not exceed
 *     CALIDROP_STATIC_SCRATCH_BYTES (about B * Hkv <= 900 for n_cal = 64), otherwise the call
 *     returns CALIDROP_SCRATCH_LIMIT and does nothing.
 *   - The first call on each device looks the array's device address up and caches it.  Make
 *     that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last call left.  The
 *     part that must start at zero (the arrival counters and the error word of the bounded
 *     waits) is cleared on `stream` ahead of the kernel by every call.  The rest of the array is
 *     used only when a unit is split over several thread-block clusters (one or two units with
 *     tens of thousands of cached rows); otherwise the splits meet in shared memory.  Two calls that may overlap on the GPU (different streams without
 *     an ordering between them) race on the array; serialise them, or give the overlapping
 *     ones their own workspace through calidrop_decode.
 */
int calidrop_decode_static(const calidrop_params* p,
                           const void* q, const void* k_new, const void* v_new,
                           void* K_kept, void* V_kept, int32_t kv_len,
                           const float* O_c, const float* LSE_c, const void* C_q,
                           void* out, float* lse_out, uint8_t* flags, void* stream);

/*
 * End-to-end variants for callers whose tensors live in HOST memory (pinned memory makes the
 * copies asynchronous).  Inputs are copied to the caller's device buffers, the device
 * operation runs, and the results are copied back, all on `stream`; the call returns without
 * synchronising.  Arguments with the suffix _h are HOST pointers with the layouts of their
 * device counterparts; the device buffers and workspaces are as above.
 *
 * calidrop_compress_host copies Q_obs, K, V (and lse_obs_h if not NULL) in, and kept_idx,
 * O_c, LSE_c out; the compacted cache and C_q stay on the device for the decode steps.
 * calidrop_decode_host copies q, k_new, v_new in and out (and lse_out/flags if not NULL) out.
 */
int calidrop_compress_host(const calidrop_params* p,
                           const void* Q_obs_h, const void* K_h, const void* V_h,
                           const float* lse_obs_h,
                           int32_t* kept_idx_h, float* O_c_h, float* LSE_c_h,
                           void* Q_obs, void* K, void* V, float* lse_obs,
                           int32_t* kept_idx, void* K_kept, void* V_kept,
                           float* O_c, float* LSE_c, void* C_q,
                           void* workspace, size_t workspace_bytes, void* stream);

int calidrop_decode_host(const calidrop_params* p,
                         const void* q_h, const void* k_new_h, const void* v_new_h,
                         void* out_h, float* lse_out_h, uint8_t* flags_h,
                         void* q, void* k_new, void* v_new,
                         void* K_kept, void* V_kept, int32_t kv_len,
                         const float* O_c, const float* LSE_c, const void* C_q,
                         void* out, float* lse_out, uint8_t* flags,
                         void* workspace, size_t workspace_bytes, void* stream);

/* Human-readable text for a status code; for CALIDROP_CUDA_ERROR includes the last CUDA
 * error string seen by the calling thread. */
const char* calidrop_status_string(int status);

/* Library version: major * 10000 + minor * 100 + patch. */
int calidrop_version(void);

/* Number of kernels the library has launched from the calling process so far. */
uint64_t calidrop_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CALIDROP_H_ */
