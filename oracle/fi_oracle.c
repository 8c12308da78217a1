/*
 * CPU oracle for the per-layer approximate-cache look-up of Freeze Inference
 * (arXiv 2002.02645).  TEST INFRASTRUCTURE ONLY: it is what the CUDA path is
 * checked against and what the benchmark times as the CPU baseline.  The
 * product never calls it.  It shares no code with the CUDA path.
 *
 * Everything is fp64 and follows the plain definition, one query at a time:
 *
 *   distance   D[n] = sum_j (q_j - c_nj)^2          Sec. 3: a neighbour tuple is (label, distance
 *                                                   to the input); squared L2, with the square
 *                                                   root applied on request (metric 1)
 *   neighbours the k smallest under the order (D, n) Sec. 3, the k-nearest-neighbour step of the
 *                                                   look-up API (ties: smaller index first)
 *   vote       for each label i among them:         Sec. 3, the confidence heuristic
 *                S_i = m_i / k
 *                C_i = S_i * sum_{j: label_j = i} w_j / d_j
 *              label = argmax_i C_i, conf = C_label ; w_j = 1 for a k-NN cache, w_j = the
 *              majority fraction f of a k-means cache entry, for which k = 1 gives the
 *              rule of Sec. 4: majority label of the closest centre, confidence f / distance
 *   hit        rule 0: conf > tau (strict)          Pseudocode 1, FreezeInference
 *              rule 1: d_win <= tau, d_win the smallest distance among the neighbours that carry
 *                      the winning label (for k = 1 the nearest-neighbour distance)
 *   compaction survivors keep their order           Sec. 5, rebuilding the batch after a layer
 *                                                   without the items frozen there
 *
 * Readings where the paper is silent: d = 0 gives 1/d = +inf, so an exact copy hits under rule 0
 * for every finite tau (observation O1 of Sec. 2); with fewer than k entries k_eff = min(k, N)
 * replaces k; an empty cache gives label -1, conf 0, miss; equal confidences are broken by the
 * larger m_i, then by the label whose nearest member comes first under (D, n).
 *
 * Parity pins (tests, marked "not gpu"): closed forms for k = 1 and for equal-distance
 * neighbours, a hand-evaluated vote, brute force by full sort in numpy on integer-coordinate
 * inputs, scaling / translation / permutation invariants, threshold monotonicity, compaction
 * invariants.  The paper prints no worked numeric example of a look-up, so none is pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* D[n] = sum_j (q_j - c_nj)^2, stored vectors widened to fp64 first */
static void sqdist_row_f32(const float *q, const float *x, int64_t n_entries, int64_t dim, double *D) {
    for (int64_t n = 0; n < n_entries; ++n) {
        const float *c = x + n * dim;
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (int64_t j = 0; j < dim; ++j) {
            double diff = (double)q[j] - (double)c[j];
            acc += diff * diff;
        }
        D[n] = acc;
    }
}

static void sqdist_row_bf16(const double *q, const uint16_t *x, int64_t n_entries, int64_t dim, double *D) {
    for (int64_t n = 0; n < n_entries; ++n) {
        const uint16_t *c = x + n * dim;
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (int64_t j = 0; j < dim; ++j) {
            uint32_t u = ((uint32_t)c[j]) << 16;
            float f;
            memcpy(&f, &u, sizeof f);
            double diff = q[j] - (double)f;
            acc += diff * diff;
        }
        D[n] = acc;
    }
}

/* Full squared-distance matrix [B x N]; dtype 0 = float32, 1 = bf16 bit patterns. */
void fio_sqdist(const void *queries, const void *cache, int dtype, int64_t batch, int64_t n_entries, int64_t dim,
                double *D) {
#pragma omp parallel
    {
        double *qd = (double *)malloc(sizeof(double) * (size_t)(dim > 0 ? dim : 1));
#pragma omp for schedule(dynamic, 1)
        for (int64_t b = 0; b < batch; ++b) {
            if (dtype == 0) {
                sqdist_row_f32((const float *)queries + b * dim, (const float *)cache, n_entries, dim, D + b * n_entries);
            } else {
                const uint16_t *q = (const uint16_t *)queries + b * dim;
                for (int64_t j = 0; j < dim; ++j) qd[j] = bf16_to_f64(q[j]);
                sqdist_row_bf16(qd, (const uint16_t *)cache, n_entries, dim, D + b * n_entries);
            }
        }
        free(qd);
    }
}

/* The kk smallest entries of D[0..N) under the total order (D, n); ascending.  kk <= N. */
void fio_select(const double *D, int64_t n_entries, int kk, double *out_d, int64_t *out_i) {
    int have = 0;
    for (int64_t n = 0; n < n_entries; ++n) {
        double v = D[n];
        if (have == kk && !(v < out_d[kk - 1])) continue; /* equal value, larger index: stays out */
        int pos = have < kk ? have : kk - 1;
        while (pos > 0 && v < out_d[pos - 1]) {
            out_d[pos] = out_d[pos - 1];
            out_i[pos] = out_i[pos - 1];
            --pos;
        }
        out_d[pos] = v;
        out_i[pos] = n;
        if (have < kk) ++have;
    }
}

/*
 * Vote, confidence and hit for one query from its k_eff neighbour tuples (ascending).
 * nd: squared distances; metric 0 uses them as d_j, metric 1 uses their square roots.
 */
void fio_vote(const double *nd, const int32_t *nlabel, const double *nweight, int k_eff, int metric, int rule, double tau,
              int32_t *label, double *conf, uint8_t *hit) {
    if (k_eff <= 0) {
        *label = -1;
        *conf = 0.0;
        *hit = 0;
        return;
    }
    int32_t best_label = -1;
    double best_c = 0.0, best_dwin = 0.0;
    int best_m = 0;
    for (int a = 0; a < k_eff; ++a) {
        int seen = 0;
        for (int e = 0; e < a; ++e) seen |= (nlabel[e] == nlabel[a]);
        if (seen) continue; /* label already scored at its first (nearest) occurrence */
        int m = 0;
        double sum = 0.0;
        for (int j = a; j < k_eff; ++j) {
            if (nlabel[j] != nlabel[a]) continue;
            double dj = metric == 1 ? sqrt(nd[j]) : nd[j];
            sum += nweight[j] / dj;
            ++m;
        }
        double share = (double)m / (double)k_eff;
        double c = share * sum;
        int better = best_label < 0 || c > best_c || (c == best_c && m > best_m);
        if (better) {
            best_label = nlabel[a];
            best_c = c;
            best_m = m;
            best_dwin = metric == 1 ? sqrt(nd[a]) : nd[a];
        }
    }
    *label = best_label;
    *conf = best_c;
    *hit = rule == 0 ? (uint8_t)(best_c > tau) : (uint8_t)(best_dwin <= tau);
}

/*
 * Look-up of a batch against one layer's cache.
 *   row_idx  nullable; query b is row row_idx[b] of `queries` (leading dimension `ld` elements)
 *   weights  nullable => 1.0
 *   out_nd / out_ni  [batch * k]: neighbour squared distances and indices, ascending, padded with +inf / -1
 *   out_next [batch]: squared distance of the (k+1)-th neighbour (+inf when there is none); the parity
 *                     harness uses it to find queries whose k-th / (k+1)-th gap is too small to call
 */
void fio_lookup(const void *queries, int64_t ld, const int32_t *row_idx, int64_t batch, const void *cache,
                const int32_t *labels, const float *weights, int dtype, int64_t n_entries, int64_t dim, int k, int metric,
                int rule, double tau, int32_t *out_label, double *out_conf, uint8_t *out_hit, double *out_nd,
                int64_t *out_ni, double *out_next) {
    int k_eff = (int64_t)k < n_entries ? k : (int)n_entries;
    int kk = (int64_t)(k + 1) < n_entries ? k + 1 : (int)n_entries;
#pragma omp parallel
    {
        double *D = (double *)malloc(sizeof(double) * (size_t)(n_entries > 0 ? n_entries : 1));
        double *qd = (double *)malloc(sizeof(double) * (size_t)(dim > 0 ? dim : 1));
        double *sd = (double *)malloc(sizeof(double) * (size_t)(k + 1));
        int64_t *si = (int64_t *)malloc(sizeof(int64_t) * (size_t)(k + 1));
        int32_t *sl = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k + 1));
        double *sw = (double *)malloc(sizeof(double) * (size_t)(k + 1));
#pragma omp for schedule(dynamic, 1)
        for (int64_t b = 0; b < batch; ++b) {
            int64_t r = row_idx ? (int64_t)row_idx[b] : b;
            if (dtype == 0) {
                sqdist_row_f32((const float *)queries + r * ld, (const float *)cache, n_entries, dim, D);
            } else {
                const uint16_t *q = (const uint16_t *)queries + r * ld;
                for (int64_t j = 0; j < dim; ++j) qd[j] = bf16_to_f64(q[j]);
                sqdist_row_bf16(qd, (const uint16_t *)cache, n_entries, dim, D);
            }
            fio_select(D, n_entries, kk, sd, si);
            for (int j = 0; j < k_eff; ++j) {
                sl[j] = labels[si[j]];
                sw[j] = weights ? (double)weights[si[j]] : 1.0;
            }
            fio_vote(sd, sl, sw, k_eff, metric, rule, tau, &out_label[b], &out_conf[b], &out_hit[b]);
            for (int j = 0; j < k; ++j) {
                out_nd[b * k + j] = j < k_eff ? sd[j] : INFINITY;
                out_ni[b * k + j] = j < k_eff ? si[j] : -1;
            }
            out_next[b] = kk > k_eff ? sd[k_eff] : INFINITY;
        }
        free(D);
        free(qd);
        free(sd);
        free(si);
        free(sl);
        free(sw);
    }
}

/*
 * Batch reconstruction: the requests of `active` (ids, in order) whose look-up missed, in the same order.
 * hit[i] belongs to active[i].  Returns the number of survivors.
 */
int64_t fio_compact(const int32_t *active, const uint8_t *hit, int64_t count, int32_t *miss) {
    int64_t m = 0;
    for (int64_t i = 0; i < count; ++i)
        if (!hit[i]) miss[m++] = active[i];
    return m;
}
