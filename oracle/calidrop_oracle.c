/*
 * CPU oracle for CaliDrop's compress-and-calibrate step and calibrated decode attention.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64 restatement of
 * the method, used only by the tests, the smoke check and the bench's CPU-baseline leg.
 * It shares no code with the CUDA path.  The only parallelism is an OpenMP loop over the
 * independent (batch, kv-head) units; there is no tiling, no online softmax, no fusion.
 *
 * Inputs are bf16 bit patterns (uint16), widened exactly to double.
 *
 * What follows the paper, and what is this implementation's reading where the paper is silent:
 *   - Eq. 1-2 (attention decomposition): oracle_decode's merge.
 *   - Algorithm 1 lines 3-8 (select with an eviction strategy, calibrate with the last
 *     query over the evicted KV): oracle_compress / oracle_calibrate_given_indices.
 *   - Algorithm 2 lines 1-2, 9-14 (attention over the retained cache with its softmax
 *     denominator, cosine similarity, threshold gate, merge): oracle_decode.
 *   - The exponent scale is 1/sqrt(d_k) everywhere (Algorithm 1 prints "/d_k"; Eq. 1 only
 *     holds with the attention's own scale).  C_weight is kept as its logarithm.
 *   - The SnapKV scoring rule (Sections 1, 4.1.2, 4.1.3 give it in prose only): softmax of
 *     each observation-window query over all causally visible keys, votes summed over the
 *     window rows and over the query heads of a kv group, zero-padded average pooling with
 *     a constant divisor, top-(budget - window) by pooled vote with ties to the lower
 *     index, window rows always kept.  PARITY UNPINNED for these choices: the paper gives
 *     no formula, so the oracle is their definition (each step is still pinned to a
 *     textbook routine in the tests).
 *   - n_cal > 1 (several calibration queries, decode picks the most similar one, ties to
 *     the most recent) is an extension; n_cal = 1 is Algorithm 1 verbatim.
 *   - The "calibration size" of Section 4.4 (Efficiency Optimization; Fig. 3c): the evicted
 *     tokens are ranked by importance and only the first m are kept for calibration and
 *     offloading.  Importance is read as the pooled vote the eviction rule already ranks by,
 *     with the same tie rule (lower index first), so the calibrated set is the next m
 *     candidates after the selected ones in one and the same order.  PARITY UNPINNED for the
 *     choice of the importance measure (the paper names none); m >= |E| is Algorithm 1 as
 *     printed.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* s = scale * <q, k> over D entries. */
static double logit(const uint16_t* q, const uint16_t* k, int D, double scale) {
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += bf16_to_double(q[d]) * bf16_to_double(k[d]);
    return acc * scale;
}

/*
 * Softmax attention of one query over the key/value rows listed in idx[0..n) (idx == NULL:
 * rows 0..n-1).  Two passes: maximum, then sum.  Returns the log of the softmax
 * denominator (-inf and a zero output when n == 0).
 * Definition: Att(Q,K,V) = softmax(Q K^T / sqrt(d_k)) V, the first line of the proof of Eq. 1.
 */
static double attend_rows(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                          const int32_t* idx, int64_t n, int D, double scale, double* out) {
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (n <= 0) return -INFINITY;
    double* s = (double*)malloc((size_t)n * sizeof(double));
    double m = -INFINITY;
    for (int64_t i = 0; i < n; ++i) {
        int64_t t = idx ? idx[i] : i;
        s[i] = logit(q, K + t * D, D, scale);
        if (s[i] > m) m = s[i];
    }
    double denom = 0.0;
    for (int64_t i = 0; i < n; ++i) denom += exp(s[i] - m);
    for (int64_t i = 0; i < n; ++i) {
        int64_t t = idx ? idx[i] : i;
        double p = exp(s[i] - m) / denom;
        const uint16_t* v = V + t * D;
        for (int d = 0; d < D; ++d) out[d] += p * bf16_to_double(v[d]);
    }
    free(s);
    return m + log(denom);
}

/* Brute-force attention: nq queries [nq, D] over n rows of K, V [n, D]. */
void oracle_full_attention(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                           int nq, int64_t n, int D, double scale, double* out, double* lse) {
    for (int i = 0; i < nq; ++i)
        lse[i] = attend_rows(q + (int64_t)i * D, K, V, NULL, n, D, scale, out + (int64_t)i * D);
}

/*
 * Window scoring and vote reduction for one (batch, kv-head) unit.
 * Observation row j of query head g sits at prompt position L - W + j and sees keys
 * t <= L - W + j.  a[g][j][t] is its softmax row; vote[t] = sum_g sum_j a[g][j][t] for the
 * candidate keys t < L - W, accumulated in (g, j) order.  row_lse[g*W + j] receives the log
 * of the row's softmax denominator.
 */
static void unit_votes(const uint16_t* Qobs /* [G, W, D] */, const uint16_t* K /* [L, D] */,
                       int G, int W, int64_t L, int D, double scale,
                       double* vote /* [L - W] */, double* row_lse /* [G*W] */) {
    int64_t n_cand = L - W;
    for (int64_t t = 0; t < n_cand; ++t) vote[t] = 0.0;
    double* s = (double*)malloc((size_t)L * sizeof(double));
    for (int g = 0; g < G; ++g) {
        for (int j = 0; j < W; ++j) {
            const uint16_t* q = Qobs + ((int64_t)g * W + j) * D;
            int64_t visible = n_cand + j + 1; /* keys 0 .. L-W+j */
            double m = -INFINITY;
            for (int64_t t = 0; t < visible; ++t) {
                s[t] = logit(q, K + t * D, D, scale);
                if (s[t] > m) m = s[t];
            }
            double denom = 0.0;
            for (int64_t t = 0; t < visible; ++t) denom += exp(s[t] - m);
            for (int64_t t = 0; t < n_cand; ++t) vote[t] += exp(s[t] - m) / denom;
            row_lse[g * W + j] = m + log(denom);
        }
    }
    free(s);
}

/* Average pool, kernel `pool` (odd), stride 1, zero padding pool/2, divisor always pool. */
void oracle_pool(const double* vote, int64_t n, int pool, double* pooled) {
    int half = pool / 2;
    for (int64_t t = 0; t < n; ++t) {
        double acc = 0.0;
        for (int d = -half; d <= half; ++d) {
            int64_t u = t + d;
            if (u >= 0 && u < n) acc += vote[u];
        }
        pooled[t] = acc / (double)pool;
    }
}

typedef struct { double score; int32_t idx; } scored_t;

static int by_score_desc_then_index(const void* a, const void* b) {
    const scored_t* x = (const scored_t*)a;
    const scored_t* y = (const scored_t*)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

static int by_int(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

/* The k highest-scoring indices (ties to the lower index), returned in ascending order. */
void oracle_topk(const double* score, int64_t n, int64_t k, int32_t* out_sorted) {
    scored_t* a = (scored_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(scored_t));
    for (int64_t t = 0; t < n; ++t) { a[t].score = score[t]; a[t].idx = (int32_t)t; }
    qsort(a, (size_t)n, sizeof(scored_t), by_score_desc_then_index);
    for (int64_t i = 0; i < k; ++i) out_sorted[i] = a[i].idx;
    qsort(out_sorted, (size_t)k, sizeof(int32_t), by_int);
    free(a);
}

/*
 * Steps 6-7 for one unit given its kept list: copy the kept rows, then for every query
 * head of the group and every calibration row c (observation row W - n_cal + c) compute
 * LSE_c = log sum_{t in E} exp(q.k_t/sqrt(D)) and O_c = Att(q, K_E, V_E), with
 * E = [0, L-W) minus the kept candidates (Algorithm 1 lines 5-8, with the scale reading
 * stated in the header).
 */
static void unit_calibrate(const uint16_t* Qobs, const uint16_t* K, const uint16_t* V,
                           const int32_t* kept, int64_t n_kept,
                           const int32_t* calib_set, int64_t n_set, /* NULL: every evicted candidate */
                           int G, int W, int64_t L, int D, int n_cal, int64_t cap, double scale,
                           uint16_t* K_kept, uint16_t* V_kept,
                           double* O_c /* [G, n_cal, D] */, double* LSE_c /* [G, n_cal] */,
                           uint16_t* C_q /* [G, n_cal, D] */) {
    (void)cap;
    for (int64_t i = 0; i < n_kept; ++i) {
        memcpy(K_kept + i * D, K + (int64_t)kept[i] * D, (size_t)D * sizeof(uint16_t));
        memcpy(V_kept + i * D, V + (int64_t)kept[i] * D, (size_t)D * sizeof(uint16_t));
    }
    int64_t n_cand = L - W;
    if (n_cand < 0) n_cand = 0;
    char* is_kept = (char*)calloc((size_t)(L > 0 ? L : 1), 1);
    for (int64_t i = 0; i < n_kept; ++i) is_kept[kept[i]] = 1;
    int32_t* evicted = (int32_t*)malloc((size_t)(n_cand > 0 ? n_cand : 1) * sizeof(int32_t));
    int64_t n_e = 0;
    for (int64_t t = 0; t < n_cand; ++t)
        if (!is_kept[t]) evicted[n_e++] = (int32_t)t;
    if (calib_set) {   /* calibration size: only the listed evicted tokens take part */
        n_e = 0;
        for (int64_t i = 0; i < n_set; ++i)
            if (!is_kept[calib_set[i]]) evicted[n_e++] = calib_set[i];
    }
    for (int g = 0; g < G; ++g) {
        for (int c = 0; c < n_cal; ++c) {
            const uint16_t* q = Qobs + ((int64_t)g * W + (W - n_cal + c)) * D;
            int64_t o = (int64_t)g * n_cal + c;
            LSE_c[o] = attend_rows(q, K, V, evicted, n_e, D, scale, O_c + o * D);
            memcpy(C_q + o * D, q, (size_t)D * sizeof(uint16_t));
        }
    }
    free(evicted);
    free(is_kept);
}

/*
 * Compress-and-calibrate over all units.
 * Layouts: Q_obs [B,Hq,W,D], K,V [B,Hkv,L,D] (bf16 bits); kept_idx [B,Hkv,n_kept] with
 * n_kept = min(budget, L); K_kept,V_kept [B,Hkv,cap,D]; O_c [B,Hq,n_cal,D], LSE_c
 * [B,Hq,n_cal] (double); C_q [B,Hq,n_cal,D] (bf16 bits); vote, pooled [B,Hkv,L-W] and
 * row_lse [B,Hq,W] (double; may be NULL).
 * calib_size < 0: every evicted candidate is calibrated (Algorithm 1 as printed).  Otherwise only
 * the m = min(calib_size, number evicted) evicted candidates of highest pooled vote (ties to the
 * lower index) are; their ascending indices go to calib_idx [B,Hkv,m] when it is not NULL.
 * Returns 0, or -1 for arguments the method does not define (budget <= window < L).
 */
int oracle_compress(const uint16_t* Q_obs, const uint16_t* K, const uint16_t* V,
                    int B, int Hq, int Hkv, int64_t L, int D, int W, int pool, int64_t budget,
                    int n_cal, int64_t cap, double scale,
                    int32_t* kept_idx, uint16_t* K_kept, uint16_t* V_kept,
                    double* O_c, double* LSE_c, uint16_t* C_q,
                    double* vote_out, double* pooled_out, double* row_lse_out,
                    int64_t calib_size, int32_t* calib_idx) {
    if (Hq % Hkv != 0 || n_cal < 1 || n_cal > W || pool < 1 || pool % 2 == 0) return -1;
    int keep_all = budget >= L;
    if (!keep_all && (budget <= W || L < W)) return -1;
    int G = Hq / Hkv;
    int64_t n_kept = keep_all ? L : budget;
    int64_t n_cand = L - W;
    int64_t k_sel = budget - W;
    int units = B * Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        int b = u / Hkv, h = u % Hkv;
        const uint16_t* Ku = K + (int64_t)u * L * D;
        const uint16_t* Vu = V + (int64_t)u * L * D;
        const uint16_t* Qu = Q_obs + ((int64_t)b * Hq + (int64_t)h * G) * W * D;
        int32_t* kept = kept_idx + (int64_t)u * n_kept;
        int32_t* cset = NULL;
        int64_t m = 0;
        if (keep_all) {
            for (int64_t t = 0; t < L; ++t) kept[t] = (int32_t)t;
        } else {
            double* vote = (double*)malloc((size_t)n_cand * sizeof(double));
            double* pooled = (double*)malloc((size_t)n_cand * sizeof(double));
            double* row_lse = (double*)malloc((size_t)G * W * sizeof(double));
            unit_votes(Qu, Ku, G, W, L, D, scale, vote, row_lse);
            oracle_pool(vote, n_cand, pool, pooled);
            oracle_topk(pooled, n_cand, k_sel, kept);
            for (int j = 0; j < W; ++j) kept[k_sel + j] = (int32_t)(n_cand + j);
            if (calib_size >= 0) {
                /* the next m candidates in the same order: rank the candidates again with the
                 * selected ones pushed below every vote (votes are non-negative) */
                m = calib_size < n_cand - k_sel ? calib_size : n_cand - k_sel;
                double* rest = (double*)malloc((size_t)n_cand * sizeof(double));
                memcpy(rest, pooled, (size_t)n_cand * sizeof(double));
                for (int64_t i = 0; i < k_sel; ++i) rest[kept[i]] = -1.0;
                cset = (int32_t*)malloc((size_t)(m > 0 ? m : 1) * sizeof(int32_t));
                oracle_topk(rest, n_cand, m, cset);
                if (calib_idx) memcpy(calib_idx + (int64_t)u * m, cset, (size_t)m * sizeof(int32_t));
                free(rest);
            }
            if (vote_out) memcpy(vote_out + (int64_t)u * n_cand, vote, (size_t)n_cand * sizeof(double));
            if (pooled_out) memcpy(pooled_out + (int64_t)u * n_cand, pooled, (size_t)n_cand * sizeof(double));
            if (row_lse_out)
                memcpy(row_lse_out + ((int64_t)b * Hq + (int64_t)h * G) * W, row_lse,
                       (size_t)G * W * sizeof(double));
            free(vote); free(pooled); free(row_lse);
        }
        unit_calibrate(Qu, Ku, Vu, kept, n_kept, cset, m, G, W, L, D, n_cal, cap, scale,
                       K_kept + (int64_t)u * cap * D, V_kept + (int64_t)u * cap * D,
                       O_c + ((int64_t)b * Hq + (int64_t)h * G) * n_cal * D,
                       LSE_c + ((int64_t)b * Hq + (int64_t)h * G) * n_cal,
                       C_q + ((int64_t)b * Hq + (int64_t)h * G) * n_cal * D);
        free(cset);
    }
    return 0;
}

/* Steps 6-7 for an externally supplied kept list kept_idx [B,Hkv,n_kept]. */
int oracle_calibrate_given_indices(const uint16_t* Q_obs, const uint16_t* K, const uint16_t* V,
                                   int B, int Hq, int Hkv, int64_t L, int D, int W,
                                   int n_cal, int64_t cap, double scale,
                                   const int32_t* kept_idx, int64_t n_kept,
                                   uint16_t* K_kept, uint16_t* V_kept,
                                   double* O_c, double* LSE_c, uint16_t* C_q) {
    if (Hq % Hkv != 0 || n_cal < 1 || n_cal > W) return -1;
    int G = Hq / Hkv;
    int units = B * Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        int b = u / Hkv, h = u % Hkv;
        int64_t qoff = (int64_t)b * Hq + (int64_t)h * G;
        unit_calibrate(Q_obs + qoff * W * D, K + (int64_t)u * L * D, V + (int64_t)u * L * D,
                       kept_idx + (int64_t)u * n_kept, n_kept, NULL, 0, G, W, L, D, n_cal, cap, scale,
                       K_kept + (int64_t)u * cap * D, V_kept + (int64_t)u * cap * D,
                       O_c + qoff * n_cal * D, LSE_c + qoff * n_cal, C_q + qoff * n_cal * D);
    }
    return 0;
}

static double log_add_exp(double a, double b) {
    if (a == -INFINITY) return b;
    if (b == -INFINITY) return a;
    double m = a > b ? a : b;
    return m + log(exp(a - m) + exp(b - m));
}

/*
 * One decode step (Algorithm 2 lines 1-2 and 9-14; the recompute branch of lines 3-8 is
 * only flagged).  q [B,Hq,D]; k_new,v_new [B,Hkv,D] or NULL; K_kept,V_kept [B,Hkv,cap,D]
 * are updated in place at row kv_len when k_new is given; O_c [B,Hq,n_cal,D] and LSE_c
 * [B,Hq,n_cal] double; C_q [B,Hq,n_cal,D] bf16 bits.
 * Outputs (all optional except out): out [B,Hq,D], lse_out [B,Hq] (log-denominator
 * actually used), lse_a [B,Hq] (retained part only), rho [B,Hq,n_cal], flags [B,Hq]
 * (bit0 calibration applied, bit1 needs_recompute, bits 2..7 chosen row when n_cal <= 64).
 * force_c / force_apply [B,Hq] (or NULL): when >= 0, override the chosen calibration row /
 * the gate decision, so a caller can evaluate the oracle under another discrete choice.
 * Strict comparisons as printed: rho < theta1 flags a recompute, rho > theta2 applies the
 * calibration; theta2 <= -1 always applies it.
 */
void oracle_decode(const uint16_t* q, const uint16_t* k_new, const uint16_t* v_new,
                   uint16_t* K_kept, uint16_t* V_kept, int64_t kv_len,
                   const double* O_c, const double* LSE_c, const uint16_t* C_q,
                   int B, int Hq, int Hkv, int D, int n_cal, int64_t cap, double scale,
                   double theta1, double theta2,
                   const int32_t* force_c, const int32_t* force_apply,
                   double* out, double* lse_out, double* lse_a_out, double* rho_out,
                   uint8_t* flags_out) {
    int G = Hq / Hkv;
    int units = B * Hkv;
    int64_t n_kv = kv_len + (k_new ? 1 : 0);
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        uint16_t* Ku = K_kept + (int64_t)u * cap * D;
        uint16_t* Vu = V_kept + (int64_t)u * cap * D;
        if (k_new) {
            memcpy(Ku + kv_len * D, k_new + (int64_t)u * D, (size_t)D * sizeof(uint16_t));
            memcpy(Vu + kv_len * D, v_new + (int64_t)u * D, (size_t)D * sizeof(uint16_t));
        }
        int b = u / Hkv, h = u % Hkv;
        for (int g = 0; g < G; ++g) {
            int64_t hq = (int64_t)b * Hq + (int64_t)h * G + g;
            const uint16_t* qv = q + hq * D;
            double* o = out + hq * D;
            /* line 1: attention over the retained cache and its log-denominator */
            double lse_a = attend_rows(qv, Ku, Vu, NULL, n_kv, D, scale, o);
            /* line 2: cosine similarity with every stored calibration query */
            double qq = 0.0;
            for (int d = 0; d < D; ++d) qq += bf16_to_double(qv[d]) * bf16_to_double(qv[d]);
            int best = 0;
            double best_rho = -INFINITY;
            double* rho_all = (double*)malloc((size_t)n_cal * sizeof(double));
            for (int c = 0; c < n_cal; ++c) {
                const uint16_t* cq = C_q + (hq * n_cal + c) * D;
                double dot = 0.0, cc = 0.0;
                for (int d = 0; d < D; ++d) {
                    double x = bf16_to_double(cq[d]);
                    dot += bf16_to_double(qv[d]) * x;
                    cc += x * x;
                }
                double rho = (qq > 0.0 && cc > 0.0) ? dot / (sqrt(qq) * sqrt(cc)) : 0.0;
                rho_all[c] = rho;
                if (rho_out) rho_out[hq * n_cal + c] = rho;
                if (rho >= best_rho) { best_rho = rho; best = c; } /* ties: most recent row */
            }
            if (force_c && force_c[hq] >= 0) {
                best = force_c[hq];
                best_rho = rho_all[best];
            }
            free(rho_all);
            int needs_recompute = best_rho < theta1;
            int apply = (theta2 <= -1.0) || (best_rho > theta2);
            if (force_apply && force_apply[hq] >= 0) apply = force_apply[hq];
            double lse_c = LSE_c[hq * n_cal + best];
            double lse = lse_a;
            if (apply && lse_c > -INFINITY) {
                /* Eq. 1-2: alpha_i = e^{LSE_a - LSE}, alpha_j = e^{LSE_c - LSE} */
                lse = log_add_exp(lse_a, lse_c);
                double ai = exp(lse_a - lse), aj = exp(lse_c - lse);
                const double* oc = O_c + (hq * n_cal + best) * D;
                for (int d = 0; d < D; ++d) o[d] = ai * o[d] + aj * oc[d];
            } else {
                apply = 0;
            }
            if (lse_out) lse_out[hq] = lse;
            if (lse_a_out) lse_a_out[hq] = lse_a;
            if (flags_out)
                flags_out[hq] = (uint8_t)((apply ? 1 : 0) | (needs_recompute ? 2 : 0) |
                                          (n_cal <= 64 ? (best << 2) : 0));
        }
    }
}
