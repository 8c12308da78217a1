// Per-query finish of a look-up and the batch reconstruction.
//
// finalize_kernel (one CTA per query): merge the candidate lists that the distance kernels left per range of
// cache rows, optionally recompute the exact squared distance sum_j (q_j - c_j)^2 of each candidate in fp32
// (the GEMM's ||q||^2 + ||c||^2 - 2 q.c form cancels badly for close pairs), order by (distance, index), then
// apply the confidence heuristic of Sec. 3 (S_i = m_i/k, C_i = S_i * sum_j w_j/d_j, arg-max) and the hit rule of
// Pseudocode 1.
//
// finalize_rows_kernel: the same finish, one query per warp, for large batches of short rows.
//
// compact_kernel (one CTA): warp-ballot stream compaction of the misses, order kept (Sec. 5, rebuilding the
// batch after each layer), and the scatter of (label, confidence, stage) for the requests frozen here.
#include "fi_internal.cuh"

namespace fi {

namespace {

constexpr int kFinThreads = 256;
constexpr int kFinWarps = kFinThreads / 32;

// order-preserving integer image of a float (compares like the float, so an integer minimum is a float minimum)
__device__ __forceinline__ int32_t score_key(float f) {
    const int32_t b = __float_as_int(f);
    return b >= 0 ? b : b ^ 0x7FFFFFFF;
}
__device__ __forceinline__ float key_score(int32_t k) { return __int_as_float(k >= 0 ? k : k ^ 0x7FFFFFFF); }

struct FinalizeParams {
    const void *X;
    const int32_t *labels;
    const float *weights;
    int64_t n_entries;
    int dim;
    const void *Q;
    int64_t ldq;
    const int32_t *row_idx;
    int32_t batch_max;
    const int32_t *count_dev;
    const float *part_score;
    const int32_t *part_idx;
    int parts;
    int list_len;
    const GemmPlan *plan;
    int refine;
    int k;
    int metric;
    int rule;
    float tau;
    int32_t *out_label;
    float *out_conf;
    uint8_t *out_hit;
    float *out_topk_dist;
    int32_t *out_topk_idx;
    // certificate of the tensor-core path (refine = 1): is every cache row outside the candidate list provably farther
    // than the k-th neighbour?  eps bounds the relative error of a score against ||q||^2 + max ||c||^2.
    float eps;
    int32_t *cert;            // [0] queries without a certificate, [1] largest observed score error (float bits, relative
                              // to ||q||^2 + max ||c||^2), [2] length of the repair list, [3] max ||c||^2 (float bits)
    uint8_t *slot_cert;       // [batch] 1 = certified
    int32_t *repair_list;     // slots to look up again with exact distances (nullable: no repair)
    int repair_cap;
    const int32_t *out_slot;  // nullable: result b goes to output slot out_slot[b] (the repair pass)
};

__device__ __forceinline__ uint4 ld16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <typename T>
__device__ __forceinline__ float sqdiff16(uint4 q, uint4 x, float acc);
template <>
__device__ __forceinline__ float sqdiff16<float>(uint4 q, uint4 x, float acc) {
    float d0 = __uint_as_float(q.x) - __uint_as_float(x.x);
    float d1 = __uint_as_float(q.y) - __uint_as_float(x.y);
    float d2 = __uint_as_float(q.z) - __uint_as_float(x.z);
    float d3 = __uint_as_float(q.w) - __uint_as_float(x.w);
    acc = fmaf(d0, d0, acc);
    acc = fmaf(d1, d1, acc);
    acc = fmaf(d2, d2, acc);
    return fmaf(d3, d3, acc);
}
template <>
__device__ __forceinline__ float sqdiff16<uint16_t>(uint4 q, uint4 x, float acc) {
    uint32_t qw[4] = {q.x, q.y, q.z, q.w};
    uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float d0 = __uint_as_float(qw[i] << 16) - __uint_as_float(xw[i] << 16);
        float d1 = __uint_as_float(qw[i] & 0xFFFF0000u) - __uint_as_float(xw[i] & 0xFFFF0000u);
        acc = fmaf(d0, d0, acc);
        acc = fmaf(d1, d1, acc);
    }
    return acc;
}

template <typename T>
__device__ __forceinline__ float sqnorm16(uint4 q, float acc);
template <>
__device__ __forceinline__ float sqnorm16<float>(uint4 q, float acc) {
    acc = fmaf(__uint_as_float(q.x), __uint_as_float(q.x), acc);
    acc = fmaf(__uint_as_float(q.y), __uint_as_float(q.y), acc);
    acc = fmaf(__uint_as_float(q.z), __uint_as_float(q.z), acc);
    return fmaf(__uint_as_float(q.w), __uint_as_float(q.w), acc);
}
template <>
__device__ __forceinline__ float sqnorm16<uint16_t>(uint4 q, float acc) {
    uint32_t qw[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float a = __uint_as_float(qw[i] << 16), b = __uint_as_float(qw[i] & 0xFFFF0000u);
        acc = fmaf(a, a, acc);
        acc = fmaf(b, b, acc);
    }
    return acc;
}

// Certificate of one query on the tensor-core path.  The distance kernel ranks cache rows by an approximate score
// s^ = ||c||^2 - 2 q.c (bf16 products accumulated in fp32), whose error against the true s = d - ||q||^2 is taken
// to be at most E = eps (||q||^2 + max ||c||^2).  Its candidate list holds the `want` smallest scores, so every row
// outside the list has s^ >= s_last, hence a true distance >= s_last + ||q||^2 - E.  If the k-th exact distance found
// among the candidates is below that, no row outside the list can be among the k nearest: the neighbours are proven
// to be the exact ones.  (A list with fewer than `want` entries holds every row that counts.)
__device__ __forceinline__ bool certified(float d_k, float s_last, float qq, float c_max, float eps, bool list_full) {
    return !list_full || d_k < s_last + qq - eps * (qq + c_max);
}

__device__ __forceinline__ bool pair_less(float s, int i, float t, int j) { return s < t || (s == t && i < j); }

// One query, finished by all threads of a CTA together.
// kLong: rows of at least kLongRowChunks 16-byte chunks take the exact distances by slices of the row (below);
// kLong == 2: the same for candidate lists of at most four entries (k = 1), four candidates and two blocks of the row
// per step instead of eight candidates and one, so that as many loads are in flight
constexpr int kLongRowChunks = 1024;

template <typename T, int kLong>
__device__ __forceinline__ void finalize_query_cta(const FinalizeParams &p, int b, int parts, int list_len) {
    __shared__ float cand_s[kMaxK];
    __shared__ float cand_d[kMaxK];
    __shared__ int32_t cand_i[kMaxK];
    __shared__ int32_t cand_lab[kMaxK];
    __shared__ float cand_w[kMaxK];
    __shared__ int32_t red_k[kFinWarps];
    __shared__ int32_t red_i[kFinWarps];
    __shared__ float qq_sh;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int entries = parts * list_len;
    const float *ps = p.part_score + (int64_t)b * entries;
    const int32_t *pi = p.part_idx + (int64_t)b * entries;
    int want = p.refine ? list_len : p.k;
    if (want > kMaxK) want = kMaxK;
    const float kInf = __int_as_float(0x7F800000);

    // ---- merge: repeatedly take the smallest (score, index) pair above the previous pick.  Scores are compared
    // through their order-preserving integer images, so a warp's minimum is two warp-wide integer reductions
    // (score image, then index among the lanes that hold that score) instead of a shuffle tree.
    int32_t prev_k = (int32_t)0x80000000;
    int prev_i = -1;
    int cand_n = 0;
    // The distance GEMM leaves every list sorted by (score, index).  Up to 64 such lists are merged by warp 0 alone,
    // lane l holding the heads of lists l and l + 32: a round is two warp-wide integer minima and one lane stepping
    // its list, without any CTA-wide barrier.
    __shared__ int32_t cand_n_sh;
    const bool head_merge = p.refine != 0 && parts <= 64;
    if (head_merge) {
        // all entries of the lists come into shared memory in one round trip (every thread of the CTA fetches a few), so
        // that the merging warp steps through its lists without waiting on global memory between rounds
        __shared__ int32_t ent_k[64 * kMaxK];
        __shared__ int32_t ent_i[64 * kMaxK];
        for (int e = tid; e < entries; e += kFinThreads) {
            const int ii = pi[e];
            const bool live = ii >= 0 && ii < p.n_entries;   // else the list has ended (an index past the cache cannot occur; never follow one)
            ent_k[e] = live ? score_key(ps[e]) : 0x7FFFFFFF;
            ent_i[e] = live ? ii : 0x7FFFFFFF;
        }
        __syncthreads();
        if (warp == 0) {
            auto head = [&](int list, int h, int32_t &k, int32_t &i) {
                k = 0x7FFFFFFF;
                i = 0x7FFFFFFF;
                if (list < parts && h < list_len) {
                    k = ent_k[list * list_len + h];
                    i = ent_i[list * list_len + h];
                }
            };
            int h0 = 0, h1 = 0;
            int32_t k0, i0, k1, i1;
            head(lane, 0, k0, i0);
            head(lane + 32, 0, k1, i1);
            for (int r = 0; r < want; ++r) {
                const bool lower = k0 < k1 || (k0 == k1 && i0 < i1);
                const int32_t bk = lower ? k0 : k1, bi = lower ? i0 : i1;
                const int32_t mk = __reduce_min_sync(0xFFFFFFFFu, bk);
                const int32_t mi = __reduce_min_sync(0xFFFFFFFFu, bk == mk ? bi : 0x7FFFFFFF);
                if (mi == 0x7FFFFFFF) break;   // lists exhausted
                if (bk == mk && bi == mi) {    // a cache row sits in one list only: exactly one lane
                    if (lower) head(lane, ++h0, k0, i0);
                    else head(lane + 32, ++h1, k1, i1);
                }
                if (lane == 0) {
                    cand_s[r] = key_score(mk);
                    cand_i[r] = mi;
                }
                cand_n = r + 1;
            }
            if (lane == 0) cand_n_sh = cand_n;
        }
        __syncthreads();
        cand_n = cand_n_sh;
    }
    // up to kKeep entries per thread are fetched once and kept in registers for all rounds (a batch of 16 against 296
    // lists of 4 re-read them from L2 in every round before); longer inputs are read again in each round
    constexpr int kKeep = 8;
    const bool kept = !head_merge && entries <= kKeep * kFinThreads;
    int32_t ck[kKeep], ci[kKeep];
    if (kept) {
#pragma unroll
        for (int j = 0; j < kKeep; ++j) {
            const int e = tid + j * kFinThreads;
            ck[j] = 0x7FFFFFFF;
            ci[j] = 0x7FFFFFFF;
            if (e < entries) {
                const int i = pi[e];
                if (i >= 0 && i < p.n_entries) {   // else: empty slot (an index past the cache cannot occur; never follow one)
                    ck[j] = score_key(ps[e]);
                    ci[j] = i;
                }
            }
        }
    }
    for (int r = 0; r < want && !head_merge; ++r) {
        int32_t best_k = 0x7FFFFFFF;
        int best_i = 0x7FFFFFFF;
        if (kept) {
#pragma unroll
            for (int j = 0; j < kKeep; ++j) {
                const int32_t k = ck[j];
                const int i = ci[j];
                const bool above = r == 0 || k > prev_k || (k == prev_k && i > prev_i);
                if (i != 0x7FFFFFFF && above && (k < best_k || (k == best_k && i < best_i))) {
                    best_k = k;
                    best_i = i;
                }
            }
        } else {
            for (int e = tid; e < entries; e += kFinThreads) {
                const int i = pi[e];
                if (i < 0 || i >= p.n_entries) continue;   // empty slot (an index past the cache cannot occur; never follow one)
                const int32_t k = score_key(ps[e]);
                const bool above = r == 0 || k > prev_k || (k == prev_k && i > prev_i);
                if (above && (k < best_k || (k == best_k && i < best_i))) {
                    best_k = k;
                    best_i = i;
                }
            }
        }
        int32_t mk = __reduce_min_sync(0xFFFFFFFFu, best_k);
        int mi = __reduce_min_sync(0xFFFFFFFFu, best_k == mk ? best_i : 0x7FFFFFFF);
        if (lane == 0) {
            red_k[warp] = mk;
            red_i[warp] = mi;
        }
        __syncthreads();
        // every warp combines the warps' minima the same way
        best_k = lane < kFinWarps ? red_k[lane] : 0x7FFFFFFF;
        best_i = lane < kFinWarps ? red_i[lane] : 0x7FFFFFFF;
        mk = __reduce_min_sync(0xFFFFFFFFu, best_k);
        mi = __reduce_min_sync(0xFFFFFFFFu, best_k == mk ? best_i : 0x7FFFFFFF);
        __syncthreads();
        if (mi == 0x7FFFFFFF) break;   // lists exhausted
        if (tid == 0) {
            cand_s[r] = key_score(mk);
            cand_i[r] = mi;
        }
        prev_k = mk;
        prev_i = mi;
        cand_n = r + 1;
    }
    __syncthreads();

    // labels and weights of the candidates, fetched side by side while the distances are recomputed
    if (tid < cand_n) {
        cand_lab[tid] = p.labels[cand_i[tid]];
        cand_w[tid] = p.weights[cand_i[tid]];
    }
    // ---- exact distances of the candidates.  The row length is cut into blocks of 32 chunks of 16 bytes; warp w takes
    // every kFinWarps-th block and, for its blocks, reads the query once and up to eight candidate rows against it
    // (nine 16-byte loads in flight per lane).  A warp per candidate, each walking the whole row with four loads in
    // flight, was bound by the latency of its 32 dependent iterations.  (The packed fp32 subtract and multiply-add of
    // this architecture, two elements per instruction, were measured here too: slower, and 16 more registers.)
    // The partial sums are added in a fixed order (lanes by shuffle tree, then warps 0..7), so reruns are bit-identical.
    if (p.refine) {
        constexpr int kGroup = kLong == 2 ? 4 : 8;   // candidates per pass over the query
        constexpr int kBlocks = kLong == 2 ? 2 : 1;  // blocks of the row per step
        __shared__ float part[kFinWarps][kGroup + 1];
        const int64_t qr = p.row_idx ? (int64_t)p.row_idx[b] : (int64_t)b;
        const uint4 *q4 = reinterpret_cast<const uint4 *>(reinterpret_cast<const T *>(p.Q) + qr * p.ldq);
        const int chunks = p.dim / (16 / (int)sizeof(T));
        // short rows (fewer than 1,024 chunks: under 16 KiB): a warp per candidate, each walking the whole row, has less
        // to reduce and no barrier; the traffic argument above only bites on long rows
        if (!kLong) {
            const T *q = reinterpret_cast<const T *>(q4);
            for (int j = warp; j < cand_n; j += kFinWarps) {
                const T *x = reinterpret_cast<const T *>(p.X) + (int64_t)cand_i[j] * p.dim;
                float a0 = 0.f, a1 = 0.f, n0 = 0.f, n1 = 0.f;
                const bool with_norm = j == 0;   // ||q||^2 for the certificate rides along with the first candidate
                int c = lane;
                for (; c + 32 < chunks; c += 64) {
                    uint4 x0 = ld16(reinterpret_cast<const uint4 *>(x) + c);
                    uint4 x1 = ld16(reinterpret_cast<const uint4 *>(x) + c + 32);
                    uint4 q0 = ld16(reinterpret_cast<const uint4 *>(q) + c);
                    uint4 q1 = ld16(reinterpret_cast<const uint4 *>(q) + c + 32);
                    a0 = sqdiff16<T>(q0, x0, a0);
                    a1 = sqdiff16<T>(q1, x1, a1);
                    if (with_norm) {
                        n0 = sqnorm16<T>(q0, n0);
                        n1 = sqnorm16<T>(q1, n1);
                    }
                }
                for (; c < chunks; c += 32) {
                    const uint4 q0 = ld16(reinterpret_cast<const uint4 *>(q) + c);
                    a0 = sqdiff16<T>(q0, ld16(reinterpret_cast<const uint4 *>(x) + c), a0);
                    if (with_norm) n0 = sqnorm16<T>(q0, n0);
                }
                float a = a0 + a1, nq = n0 + n1;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
                    nq += __shfl_xor_sync(0xFFFFFFFFu, nq, o);
                }
                if (lane == 0) {
                    cand_d[j] = a;
                    if (with_norm) qq_sh = nq;
                }
            }
        } else {
            for (int j0 = 0; j0 < cand_n; j0 += kGroup) {
                const int nj = min(kGroup, cand_n - j0);
                const uint4 *x[kGroup];
#pragma unroll
                for (int u = 0; u < kGroup; ++u)
                    x[u] = reinterpret_cast<const uint4 *>(reinterpret_cast<const T *>(p.X) + (int64_t)cand_i[j0 + min(u, nj - 1)] * p.dim);
                float a[kGroup], nq = 0.f;
#pragma unroll
                for (int u = 0; u < kGroup; ++u) a[u] = 0.f;
                const bool with_norm = j0 == 0;   // ||q||^2 for the certificate rides along with the first pass
                for (int c = warp * 32 + lane; c < chunks; c += kBlocks * kFinWarps * 32) {
                    uint4 qv[kBlocks], xv[kBlocks][kGroup];
#pragma unroll
                    for (int s2 = 0; s2 < kBlocks; ++s2) {
                        const int cc = c + s2 * kFinWarps * 32;
                        if (cc < chunks) {
                            qv[s2] = ld16(q4 + cc);
#pragma unroll
                            for (int u = 0; u < kGroup; ++u)
                                if (u < nj) xv[s2][u] = ld16(x[u] + cc);
                        }
                    }
                    // (the sums grow block after block, as with one block per step)
#pragma unroll
                    for (int s2 = 0; s2 < kBlocks; ++s2) {
                        if (c + s2 * kFinWarps * 32 < chunks) {
#pragma unroll
                            for (int u = 0; u < kGroup; ++u)
                                if (u < nj) a[u] = sqdiff16<T>(qv[s2], xv[s2][u], a[u]);
                            if (with_norm) nq = sqnorm16<T>(qv[s2], nq);
                        }
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                    for (int u = 0; u < kGroup; ++u) a[u] += __shfl_xor_sync(0xFFFFFFFFu, a[u], o);
                    nq += __shfl_xor_sync(0xFFFFFFFFu, nq, o);
                }
                if (lane == 0) {
#pragma unroll
                    for (int u = 0; u < kGroup; ++u) part[warp][u] = a[u];
                    part[warp][kGroup] = nq;
                }
                __syncthreads();
                if (tid < nj || (tid == kGroup && with_norm)) {
                    float sum = 0.f;
#pragma unroll
                    for (int w = 0; w < kFinWarps; ++w) sum += part[w][tid];
                    if (tid < nj) cand_d[j0 + tid] = sum;
                    else qq_sh = sum;
                }
                __syncthreads();
            }
        }
    } else {
        if (tid < cand_n) cand_d[tid] = cand_s[tid];
    }
    __syncthreads();

    // ---- order by (distance, index), vote, hit
    if (tid == 0) {
        const int o = p.out_slot ? p.out_slot[b] : b;
        // the certificate needs the scores as the merge left them (cand_s keeps that order; the sort below moves only
        // distances, indices, labels and weights)
        float s_last = 0.f, err_max = 0.f;
        const float c_max = p.cert ? __int_as_float(p.cert[3]) : 0.f;
        if (p.refine && p.cert && cand_n > 0) {
            s_last = cand_s[cand_n - 1];
            const float denom = qq_sh + c_max;
            for (int a = 0; a < cand_n; ++a) err_max = fmaxf(err_max, fabsf(cand_s[a] + qq_sh - cand_d[a]));
            err_max = denom > 0.f ? err_max / denom : 0.f;
        }
        for (int a = 1; a < cand_n; ++a) {
            const float d = cand_d[a], w = cand_w[a];
            const int i = cand_i[a], l = cand_lab[a];
            int pos = a;
            while (pos > 0 && pair_less(d, i, cand_d[pos - 1], cand_i[pos - 1])) {
                cand_d[pos] = cand_d[pos - 1];
                cand_i[pos] = cand_i[pos - 1];
                cand_lab[pos] = cand_lab[pos - 1];
                cand_w[pos] = cand_w[pos - 1];
                --pos;
            }
            cand_d[pos] = d;
            cand_i[pos] = i;
            cand_lab[pos] = l;
            cand_w[pos] = w;
        }
        const int k_eff = cand_n < p.k ? cand_n : p.k;
        const int32_t *lab = cand_lab;
        const float *wgt = cand_w;
        int32_t best_label = -1;
        float best_c = 0.f, best_dwin = 0.f;
        int best_m = 0;
        for (int a = 0; a < k_eff; ++a) {
            bool seen = false;
            for (int e = 0; e < a; ++e) seen |= (lab[e] == lab[a]);
            if (seen) continue;   // scored at its nearest occurrence
            int m = 0;
            float sum = 0.f;
            for (int j = a; j < k_eff; ++j) {
                if (lab[j] != lab[a]) continue;
                float dj = p.metric == FI_METRIC_L2 ? sqrtf(cand_d[j]) : cand_d[j];
                sum += wgt[j] / dj;
                ++m;
            }
            float c = ((float)m / (float)k_eff) * sum;
            if (best_label < 0 || c > best_c || (c == best_c && m > best_m)) {
                best_label = lab[a];
                best_c = c;
                best_m = m;
                best_dwin = p.metric == FI_METRIC_L2 ? sqrtf(cand_d[a]) : cand_d[a];
            }
        }
        bool hit = k_eff > 0 && (p.rule == FI_HIT_CONF_GT ? best_c > p.tau : best_dwin <= p.tau);
        p.out_label[o] = best_label;
        p.out_conf[o] = best_c;
        p.out_hit[o] = hit ? 1 : 0;
        if (p.out_topk_dist)
            for (int j = 0; j < p.k; ++j) p.out_topk_dist[(int64_t)o * p.k + j] = j < k_eff ? cand_d[j] : kInf;
        if (p.out_topk_idx)
            for (int j = 0; j < p.k; ++j) p.out_topk_idx[(int64_t)o * p.k + j] = j < k_eff ? cand_i[j] : -1;
        if (p.cert && p.slot_cert) {
            bool ok = true;   // exact distances throughout (streaming lists, the repair pass): nothing to certify
            if (p.refine && k_eff > 0) {
                ok = certified(cand_d[k_eff - 1], s_last, qq_sh, c_max, p.eps, cand_n >= want);
                if (err_max > 0.f) atomicMax(p.cert + 1, __float_as_int(err_max));
            }
            p.slot_cert[o] = ok ? 1 : 0;
            if (!ok) {
                atomicAdd(p.cert, 1);
                if (p.repair_list) {
                    const int pos = atomicAdd(p.cert + 2, 1);
                    if (pos < p.repair_cap) p.repair_list[pos] = b;
                    else atomicAdd(p.cert + 4, 1);
                } else {
                    atomicAdd(p.cert + 4, 1);
                }
            }
        }
    }
    __syncthreads();   // the shared arrays may be reused for another query
}

// One query, finished by one warp: for short rows and few candidate entries (at most 32 x kWarpEntries), where a CTA per
// query spends its time on barriers and on launching CTAs.  Same steps as finalize_query_cta (the exact distances are
// summed in another order, each within fp32 rounding of the other): merge by repeated minimum (entries held in registers, lane l the entries l, l + 32, ...),
// exact distances (the warp walks one candidate row after the other), order by (distance, index), vote, hit rule.
constexpr int kWarpEntries = 16;

template <typename T>
__device__ __forceinline__ void finalize_query_warp(const FinalizeParams &p, int b, int parts, int list_len, float *sort_d,
                                                    int32_t *sort_i, int32_t *sort_lab, float *sort_w) {
    const int lane = threadIdx.x & 31;
    const int entries = parts * list_len;
    const float *ps = p.part_score + (int64_t)b * entries;
    const int32_t *pi = p.part_idx + (int64_t)b * entries;
    int want = p.refine ? list_len : p.k;
    if (want > kMaxK) want = kMaxK;
    const float kInf = __int_as_float(0x7F800000);

    // ---- merge; the r-th winner stays with lane r
    const int per_lane = (entries + 31) >> 5;
    int32_t key[kWarpEntries], idx[kWarpEntries];
#pragma unroll
    for (int j = 0; j < kWarpEntries; ++j) {
        key[j] = 0x7FFFFFFF;
        idx[j] = 0x7FFFFFFF;
        const int e = lane + 32 * j;
        if (j < per_lane && e < entries) {
            const int i = pi[e];
            if (i >= 0 && i < p.n_entries) {   // else: empty slot (an index past the cache cannot occur; never follow one)
                key[j] = score_key(ps[e]);
                idx[j] = i;
            }
        }
    }
    float my_d = kInf;       // lane r: score, later distance, of the r-th candidate
    float my_s = kInf;       // lane r: its score as the merge left it (for the certificate)
    int32_t my_i = 0x7FFFFFFF;
    int cand_n = 0;
    for (int r = 0; r < want; ++r) {
        int32_t bk = 0x7FFFFFFF, bi = 0x7FFFFFFF;
        int bj = 0;
#pragma unroll
        for (int j = 0; j < kWarpEntries; ++j) {
            if (j < per_lane && (key[j] < bk || (key[j] == bk && idx[j] < bi))) {
                bk = key[j];
                bi = idx[j];
                bj = j;
            }
        }
        const int32_t mk = __reduce_min_sync(0xFFFFFFFFu, bk);
        const int32_t mi = __reduce_min_sync(0xFFFFFFFFu, bk == mk ? bi : 0x7FFFFFFF);
        if (mi == 0x7FFFFFFF) break;   // lists exhausted
        if (bk == mk && bi == mi) {    // a cache row sits in one list only: exactly one lane
#pragma unroll
            for (int j = 0; j < kWarpEntries; ++j)
                if (j == bj) {
                    key[j] = 0x7FFFFFFF;
                    idx[j] = 0x7FFFFFFF;
                }
        }
        if (lane == r) {
            my_d = key_score(mk);
            my_i = mi;
        }
        cand_n = r + 1;
    }

    // label and weight of this lane's candidate, in flight while the distances are recomputed
    int32_t my_lab = -1;
    float my_w = 0.f;
    if (lane < cand_n) {
        my_lab = p.labels[my_i];
        my_w = p.weights[my_i];
    }
    my_s = my_d;
    float qq = 0.f;          // ||q||^2, every lane
    // ---- exact distances of the candidates, four rows at a time so that their loads overlap; two partial sums per row
    // and lane, then a shuffle tree
    if (p.refine) {
        const int64_t qr = p.row_idx ? (int64_t)p.row_idx[b] : (int64_t)b;
        const uint4 *q = reinterpret_cast<const uint4 *>(reinterpret_cast<const T *>(p.Q) + qr * p.ldq);
        const int chunks = p.dim / (16 / (int)sizeof(T));
        for (int j0 = 0; j0 < cand_n; j0 += 4) {
            const uint4 *x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int32_t cu = __shfl_sync(0xFFFFFFFFu, my_i, min(j0 + u, cand_n - 1));
                x[u] = reinterpret_cast<const uint4 *>(reinterpret_cast<const T *>(p.X) + (int64_t)cu * p.dim);
            }
            float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f}, n0 = 0.f, n1 = 0.f;
            const bool with_norm = j0 == 0;
            int c = lane;
            for (; c + 32 < chunks; c += 64) {
                const uint4 q0 = ld16(q + c), q1 = ld16(q + c + 32);
                if (with_norm) {
                    n0 = sqnorm16<T>(q0, n0);
                    n1 = sqnorm16<T>(q1, n1);
                }
                uint4 x0[4], x1[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    x0[u] = ld16(x[u] + c);
                    x1[u] = ld16(x[u] + c + 32);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    a0[u] = sqdiff16<T>(q0, x0[u], a0[u]);
                    a1[u] = sqdiff16<T>(q1, x1[u], a1[u]);
                }
            }
            for (; c < chunks; c += 32) {
                const uint4 q0 = ld16(q + c);
                if (with_norm) n0 = sqnorm16<T>(q0, n0);
                uint4 x0[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) x0[u] = ld16(x[u] + c);
#pragma unroll
                for (int u = 0; u < 4; ++u) a0[u] = sqdiff16<T>(q0, x0[u], a0[u]);
            }
            if (with_norm) {
                float nq = n0 + n1;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) nq += __shfl_xor_sync(0xFFFFFFFFu, nq, o);
                qq = nq;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float a = a0[u] + a1[u];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
                if (lane == j0 + u && j0 + u < cand_n) my_d = a;
            }
        }
    }

    // ---- order by (distance, index): every lane counts the candidates that come before its own
    int rank = 0;
    for (int j = 0; j < cand_n; ++j) {
        const float dj = __shfl_sync(0xFFFFFFFFu, my_d, j);
        const int32_t ij = __shfl_sync(0xFFFFFFFFu, my_i, j);
        rank += pair_less(dj, ij, my_d, my_i) ? 1 : 0;
    }
    if (lane < cand_n) {
        sort_d[rank] = my_d;
        sort_i[rank] = my_i;
        sort_lab[rank] = my_lab;
        sort_w[rank] = my_w;
    }
    __syncwarp();
    const int k_eff = cand_n < p.k ? cand_n : p.k;
    const float d = lane < cand_n ? sort_d[lane] : kInf;      // lane t: the t-th nearest candidate
    const int32_t ci = lane < cand_n ? sort_i[lane] : -1;
    const int32_t lab_sorted = lane < cand_n ? sort_lab[lane] : -1;
    const float w_sorted = lane < cand_n ? sort_w[lane] : 0.f;
    __syncwarp();

    // ---- vote (lanes 0 .. k_eff-1 hold the neighbours), hit
    int32_t lab = -1;
    float term = 0.f, dj = 0.f;
    if (lane < k_eff) {
        lab = lab_sorted;
        dj = p.metric == FI_METRIC_L2 ? sqrtf(d) : d;
        term = w_sorted / dj;
    }
    int m = 0;
    float sum = 0.f;
    bool first = true;
    for (int j = 0; j < k_eff; ++j) {
        const int32_t lj = __shfl_sync(0xFFFFFFFFu, lab, j);
        const float tj = __shfl_sync(0xFFFFFFFFu, term, j);
        if (lj == lab) {
            if (j < lane) first = false;   // scored at its nearest occurrence
            sum += tj;
            ++m;
        }
    }
    const float conf = ((float)m / (float)k_eff) * sum;
    int32_t best_label = -1;
    float best_c = 0.f, best_dwin = 0.f;
    int best_m = 0;
    for (int a = 0; a < k_eff; ++a) {
        const float ca = __shfl_sync(0xFFFFFFFFu, conf, a);
        const int ma = __shfl_sync(0xFFFFFFFFu, m, a);
        const int32_t la = __shfl_sync(0xFFFFFFFFu, lab, a);
        const float da = __shfl_sync(0xFFFFFFFFu, dj, a);
        const bool fa = __shfl_sync(0xFFFFFFFFu, first ? 1 : 0, a) != 0;
        if (fa && (best_label < 0 || ca > best_c || (ca == best_c && ma > best_m))) {
            best_label = la;
            best_c = ca;
            best_m = ma;
            best_dwin = da;
        }
    }
    const bool hit = k_eff > 0 && (p.rule == FI_HIT_CONF_GT ? best_c > p.tau : best_dwin <= p.tau);
    const int o = p.out_slot ? p.out_slot[b] : b;
    if (lane == 0) {
        p.out_label[o] = best_label;
        p.out_conf[o] = best_c;
        p.out_hit[o] = hit ? 1 : 0;
    }
    for (int j = lane; j < p.k; j += 32) {
        if (p.out_topk_dist) p.out_topk_dist[(int64_t)o * p.k + j] = j < k_eff ? d : kInf;
        if (p.out_topk_idx) p.out_topk_idx[(int64_t)o * p.k + j] = j < k_eff ? ci : -1;
    }
    if (p.cert && p.slot_cert) {
        // same certificate as in finalize_query_cta; lane r still holds the r-th merged score and its exact distance
        bool ok = true;
        if (p.refine && k_eff > 0) {
            const float c_max = __int_as_float(p.cert[3]);
            const float s_last = __shfl_sync(0xFFFFFFFFu, my_s, cand_n - 1);
            const float d_k = __shfl_sync(0xFFFFFFFFu, d, k_eff - 1);
            ok = certified(d_k, s_last, qq, c_max, p.eps, cand_n >= want);
            float err = lane < cand_n ? fabsf(my_s + qq - my_d) : 0.f;
#pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) err = fmaxf(err, __shfl_xor_sync(0xFFFFFFFFu, err, sh));
            const float denom = qq + c_max;
            if (lane == 0 && denom > 0.f && err > 0.f) atomicMax(p.cert + 1, __float_as_int(err / denom));
        }
        if (lane == 0) {
            p.slot_cert[o] = ok ? 1 : 0;
            if (!ok) {
                atomicAdd(p.cert, 1);
                if (p.repair_list) {
                    const int pos = atomicAdd(p.cert + 2, 1);
                    if (pos < p.repair_cap) p.repair_list[pos] = b;
                    else atomicAdd(p.cert + 4, 1);
                } else {
                    atomicAdd(p.cert + 4, 1);
                }
            }
        }
    }
}

// One CTA per query: long rows, where the exact distances need a CTA's worth of loads in flight.
template <typename T>
__global__ void __launch_bounds__(kFinThreads) finalize_kernel(FinalizeParams p) {
    const int count = p.count_dev ? min(*p.count_dev, p.batch_max) : p.batch_max;
    const int b = blockIdx.x;
    if (b >= count) return;
    const int parts = p.plan ? p.plan->lists : p.parts;
    const int list_len = p.plan ? p.plan->list_len : p.list_len;
    finalize_query_cta<T, 0>(p, b, parts, list_len);
}

// The same for long rows (16 KiB and more): the slice-wise exact distances hold eight candidates' partial sums per
// lane, so the kernel is compiled for four CTAs per SM instead of spilling at eight.
template <typename T>
__global__ void __launch_bounds__(kFinThreads, 4) finalize_long_kernel(FinalizeParams p) {
    const int count = p.count_dev ? min(*p.count_dev, p.batch_max) : p.batch_max;
    const int b = blockIdx.x;
    if (b >= count) return;
    const int parts = p.plan ? p.plan->lists : p.parts;
    const int list_len = p.plan ? p.plan->list_len : p.list_len;
    finalize_query_cta<T, 1>(p, b, parts, list_len);
}

// Long rows under lists of at most four entries (k = 1: the latency regime).
template <typename T>
__global__ void __launch_bounds__(kFinThreads, 4) finalize_long_few_kernel(FinalizeParams p) {
    const int count = p.count_dev ? min(*p.count_dev, p.batch_max) : p.batch_max;
    const int b = blockIdx.x;
    if (b >= count) return;
    const int parts = p.plan ? p.plan->lists : p.parts;
    const int list_len = p.plan ? p.plan->list_len : p.list_len;
    finalize_query_cta<T, 2>(p, b, parts, list_len);
}

// Short rows.  Large batches (k-means assignment, threshold calibration) whose candidate entries fit a warp's
// registers are finished one query per warp, kFinWarps consecutive queries per CTA: a CTA per query would spend its time
// on barriers and on CTA launches (40,000 queries: 0.26 -> 0.09 ms; 1,282 to 4,096 queries of 256 to 2,048 values: a
// four-stage cascade 1.513 -> 1.499 ms).  Batches below 1,024 keep the CTA per query, whose latency is shorter.  The grid always has one CTA per slot of the batch; the CTAs left without work return at once.
constexpr int kWarpModeMinBatch = 1024;

template <typename T>
__global__ void __launch_bounds__(kFinThreads, 4) finalize_rows_kernel(FinalizeParams p) {
    __shared__ float sort_d[kFinWarps][kMaxK];
    __shared__ int32_t sort_i[kFinWarps][kMaxK];
    __shared__ int32_t sort_lab[kFinWarps][kMaxK];
    __shared__ float sort_w[kFinWarps][kMaxK];
    const int count = p.count_dev ? min(*p.count_dev, p.batch_max) : p.batch_max;
    const int parts = p.plan ? p.plan->lists : p.parts;
    const int list_len = p.plan ? p.plan->list_len : p.list_len;
    if (count >= kWarpModeMinBatch && parts * list_len <= 32 * kWarpEntries) {
        const int warp = threadIdx.x >> 5;
        const int b = blockIdx.x * kFinWarps + warp;
        if (b < count) finalize_query_warp<T>(p, b, parts, list_len, sort_d[warp], sort_i[warp], sort_lab[warp], sort_w[warp]);
    } else if ((int)blockIdx.x < count) {
        finalize_query_cta<T, 0>(p, blockIdx.x, parts, list_len);
    }
}

// ---------------------------------------------------------------- K4: miss compaction
__global__ void __launch_bounds__(1024)
compact_kernel(const int32_t *__restrict__ active_idx, const int32_t *__restrict__ active_count, int32_t batch0,
               const int32_t *__restrict__ slot_label, const float *__restrict__ slot_conf,
               const uint8_t *__restrict__ slot_hit, int32_t stage, int32_t *__restrict__ miss_idx,
               int32_t *__restrict__ miss_count, int32_t *__restrict__ final_label, int32_t *__restrict__ exit_stage,
               float *__restrict__ final_conf) {
    __shared__ int32_t warp_total[32];
    __shared__ int32_t warp_base[32];
    __shared__ int32_t running;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int count = active_count ? min(*active_count, batch0) : batch0;
    if (tid == 0) running = 0;
    __syncthreads();
    for (int base = 0; base < count; base += 1024) {
        const int i = base + tid;
        const bool valid = i < count;
        int32_t id = 0;
        bool miss = false;
        if (valid) {
            id = active_idx ? active_idx[i] : i;
            miss = slot_hit[i] == 0;
            if (!miss) {
                final_label[id] = slot_label[i];
                final_conf[id] = slot_conf[i];
                exit_stage[id] = stage;
            }
        }
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, miss);
        const int before = __popc(ballot & ((1u << lane) - 1u));
        if (lane == 0) warp_total[warp] = __popc(ballot);
        __syncthreads();
        if (warp == 0) {
            int t = warp_total[lane];
            int incl = t;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += v;
            }
            warp_base[lane] = running + incl - t;
            __syncwarp();
            if (lane == 31) running += incl;
        }
        __syncthreads();
        if (miss) miss_idx[warp_base[warp] + before] = id;
        __syncthreads();
    }
    if (tid == 0) *miss_count = running;
}

__global__ void cascade_init_kernel(int32_t batch0, int32_t num_stages, int32_t *final_label, int32_t *exit_stage,
                                    float *final_conf) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < batch0; i += gridDim.x * blockDim.x) {
        final_label[i] = -1;
        exit_stage[i] = num_stages;
        final_conf[i] = 0.f;
    }
}

// ComputeThresholds (Pseudocode 1): running maximum of the confidences of wrong look-ups.  Confidences are
// non-negative, so their bit patterns order like the floats and atomicMax on the pattern is a float maximum.
__global__ void wrong_max_kernel(const int32_t *__restrict__ label, const float *__restrict__ conf,
                                 const int32_t *__restrict__ ref, int32_t n, int32_t *__restrict__ acc) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        if (label[i] != ref[i]) {
            atomicMax(acc, __float_as_int(fmaxf(conf[i], 0.f)));
            atomicAdd(acc + 1, 1);
        }
    }
}

// Cache rows sharded over several GPUs: each shard answers a look-up with its own k nearest entries (exact distances).
// neighbor_tuples_kernel turns a shard's neighbour indices into tuples that can travel: global index, label, weight.
__global__ void neighbor_tuples_kernel(const int32_t *__restrict__ topk_idx, int64_t n, int64_t size,
                                       int32_t index_offset, const int32_t *__restrict__ labels, const float *__restrict__ weights,
                                       int32_t *__restrict__ out_idx, int32_t *__restrict__ out_label,
                                       float *__restrict__ out_weight) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        int32_t li = topk_idx[i];
        if (li >= size) li = -1;   // not an index of this shard: treated as "no neighbour"
        out_idx[i] = li < 0 ? -1 : li + index_offset;
        out_label[i] = li < 0 ? -1 : labels[li];
        out_weight[i] = li < 0 ? 0.f : weights[li];
    }
}

// merge_vote_kernel: one thread per query merges the shards' tuples [shard][query][k] by (distance, global index),
// keeps the k nearest and applies the same vote and hit rule as finalize_kernel.  Every rank runs it on the same
// gathered tuples and gets the same answer.
__global__ void merge_vote_kernel(int shards, int batch, int k, const float *__restrict__ dist,
                                  const int32_t *__restrict__ idx, const int32_t *__restrict__ label,
                                  const float *__restrict__ weight, int metric, int rule, float tau,
                                  int32_t *__restrict__ out_label, float *__restrict__ out_conf,
                                  uint8_t *__restrict__ out_hit, float *__restrict__ out_dist,
                                  int32_t *__restrict__ out_idx) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const float kInf = __int_as_float(0x7F800000);
    float bd[kMaxK];
    int32_t bi[kMaxK], bl[kMaxK];
    float bw[kMaxK];
    int have = 0;
    for (int s = 0; s < shards; ++s) {
        const int64_t base = ((int64_t)s * batch + b) * k;
        for (int j = 0; j < k; ++j) {
            const int32_t gi = idx[base + j];
            if (gi < 0) continue;
            const float d = dist[base + j];
            if (have == k && !pair_less(d, gi, bd[k - 1], bi[k - 1])) continue;
            int pos = have < k ? have : k - 1;
            while (pos > 0 && pair_less(d, gi, bd[pos - 1], bi[pos - 1])) {
                bd[pos] = bd[pos - 1];
                bi[pos] = bi[pos - 1];
                bl[pos] = bl[pos - 1];
                bw[pos] = bw[pos - 1];
                --pos;
            }
            bd[pos] = d;
            bi[pos] = gi;
            bl[pos] = label[base + j];
            bw[pos] = weight[base + j];
            if (have < k) ++have;
        }
    }
    const int k_eff = have;
    int32_t best_label = -1;
    float best_c = 0.f, best_dwin = 0.f;
    int best_m = 0;
    for (int a = 0; a < k_eff; ++a) {
        bool seen = false;
        for (int e = 0; e < a; ++e) seen |= (bl[e] == bl[a]);
        if (seen) continue;
        int m = 0;
        float sum = 0.f;
        for (int j = a; j < k_eff; ++j) {
            if (bl[j] != bl[a]) continue;
            const float dj = metric == FI_METRIC_L2 ? sqrtf(bd[j]) : bd[j];
            sum += bw[j] / dj;
            ++m;
        }
        const float c = ((float)m / (float)k_eff) * sum;
        if (best_label < 0 || c > best_c || (c == best_c && m > best_m)) {
            best_label = bl[a];
            best_c = c;
            best_m = m;
            best_dwin = metric == FI_METRIC_L2 ? sqrtf(bd[a]) : bd[a];
        }
    }
    const bool hit = k_eff > 0 && (rule == FI_HIT_CONF_GT ? best_c > tau : best_dwin <= tau);
    out_label[b] = best_label;
    out_conf[b] = best_c;
    out_hit[b] = hit ? 1 : 0;
    if (out_dist)
        for (int j = 0; j < k; ++j) out_dist[(int64_t)b * k + j] = j < k_eff ? bd[j] : kInf;
    if (out_idx)
        for (int j = 0; j < k; ++j) out_idx[(int64_t)b * k + j] = j < k_eff ? bi[j] : -1;
}

}  // namespace

fi_status_t launch_neighbor_tuples(const fi_cache *c, const int32_t *topk_idx, int64_t n, int32_t index_offset,
                                   int32_t *out_idx, int32_t *out_label, float *out_weight, cudaStream_t stream) {
    if (n <= 0) return FI_OK;
    int grid = (int)((n + 255) / 256 < 2048 ? (n + 255) / 256 : 2048);
    neighbor_tuples_kernel<<<grid, 256, 0, stream>>>(topk_idx, n, c->size, index_offset, c->labels, c->weights, out_idx, out_label,
                                                     out_weight);
    count_launch();
    return check_launch("neighbor_tuples_kernel");
}

fi_status_t launch_merge_vote(int shards, int batch, int k, const float *dist, const int32_t *idx, const int32_t *label,
                              const float *weight, int metric, int rule, float tau, const fi_lookup_out_t &out,
                              cudaStream_t stream) {
    if (batch <= 0) return FI_OK;
    merge_vote_kernel<<<(batch + 127) / 128, 128, 0, stream>>>(shards, batch, k, dist, idx, label, weight, metric, rule, tau,
                                                              out.label, out.conf, out.hit, out.topk_dist, out.topk_idx);
    count_launch();
    return check_launch("merge_vote_kernel");
}

fi_status_t launch_wrong_max(const int32_t *label, const float *conf, const int32_t *ref, int32_t n, int32_t *acc,
                             cudaStream_t stream) {
    if (n <= 0) return FI_OK;
    int grid = (n + 255) / 256;
    if (grid > 1024) grid = 1024;
    wrong_max_kernel<<<grid, 256, 0, stream>>>(label, conf, ref, n, acc);
    count_launch();
    return check_launch("wrong_max_kernel");
}

fi_status_t launch_finalize(const fi_cache *c, const FinalizeArgs &a, cudaStream_t stream) {
    if (a.batch_max <= 0) return FI_OK;
    FinalizeParams p;
    p.X = c->rows;
    p.labels = c->labels;
    p.weights = c->weights;
    p.n_entries = c->size;
    p.dim = c->cfg.dim;
    p.Q = a.queries;
    p.ldq = a.ld_elems;
    p.row_idx = a.row_idx;
    p.batch_max = a.batch_max;
    p.count_dev = a.count_dev;
    p.part_score = c->part_score;
    p.part_idx = c->part_idx;
    p.parts = a.parts;
    p.list_len = a.list_len;
    p.plan = a.parts < 0 ? c->plan_dev : nullptr;
    p.refine = a.refine;
    p.k = c->cfg.k;
    p.metric = c->cfg.metric;
    p.rule = c->cfg.rule;
    p.tau = c->cfg.threshold;
    p.out_label = a.out.label;
    p.out_conf = a.out.conf;
    p.out_hit = a.out.hit;
    p.out_topk_dist = a.out.topk_dist;
    p.out_topk_idx = a.out.topk_idx;
    // score error model of the distance GEMM: each of its dim / 16 accumulation steps adds to an fp32 partial sum whose
    // magnitude is at most (||q||^2 + ||c||^2) / 2 and may drop up to one unit in its last place (relative 2^-23; the
    // accumulation truncates, the errors do not cancel), twice that for the factor -2 in the score; four more steps'
    // worth covers the rounding of ||c||^2 and of the final subtraction.  Measured on the five workloads the largest
    // error is about half of this bound at 8,192 to 65,536 values per row.
    p.eps = ((float)c->cfg.dim / 16.f + 4.f) * 1.1920929e-7f;   // (dim / 16 + 4) * 2^-23
    p.cert = c->cert_dev;
    p.slot_cert = c->slot_cert;
    p.repair_list = a.fill_repair_list ? c->repair_list : nullptr;
    p.repair_cap = kRepairCap;
    p.out_slot = a.out_slot;
    // short rows (up to 8 KiB) in batches large enough for the warp-per-query mode; everything else: a CTA per query
    // (the plain kernel needs fewer registers, so more of its CTAs are resident)
    const bool short_rows = (size_t)c->cfg.dim * c->elem_size <= 8192 && a.batch_max >= kWarpModeMinBatch;
    const int grid = a.batch_max;
    const bool few = gemm_list_len(c->cfg.k) <= 4;   // the tensor-core path's lists for k = 1
    const bool long_rows = a.refine && (size_t)c->cfg.dim * c->elem_size >= (size_t)kLongRowChunks * 16;
    if (c->cfg.dtype == FI_F32) {
        if (short_rows) finalize_rows_kernel<float><<<grid, kFinThreads, 0, stream>>>(p);
        else if (long_rows && few) finalize_long_few_kernel<float><<<grid, kFinThreads, 0, stream>>>(p);
        else if (long_rows) finalize_long_kernel<float><<<grid, kFinThreads, 0, stream>>>(p);
        else finalize_kernel<float><<<grid, kFinThreads, 0, stream>>>(p);
    } else {
        if (short_rows) finalize_rows_kernel<uint16_t><<<grid, kFinThreads, 0, stream>>>(p);
        else if (long_rows && few) finalize_long_few_kernel<uint16_t><<<grid, kFinThreads, 0, stream>>>(p);
        else if (long_rows) finalize_long_kernel<uint16_t><<<grid, kFinThreads, 0, stream>>>(p);
        else finalize_kernel<uint16_t><<<grid, kFinThreads, 0, stream>>>(p);
    }
    count_launch();
    return check_launch("finalize_kernel");
}

fi_status_t launch_compact(const fi_cache *c, const fi_cascade_state_t &st, cudaStream_t stream) {
    compact_kernel<<<1, 1024, 0, stream>>>(st.active_idx, st.active_count, st.batch0, c->slot_label, c->slot_conf,
                                           c->slot_hit, st.stage, st.miss_idx, st.miss_count, st.final_label,
                                           st.exit_stage, st.final_conf);
    count_launch();
    return check_launch("compact_kernel");
}

fi_status_t launch_cascade_init(const fi_cascade_state_t &st, int32_t num_stages, cudaStream_t stream) {
    if (st.batch0 <= 0) return FI_OK;
    int grid = (st.batch0 + 255) / 256;
    if (grid > 1024) grid = 1024;
    cascade_init_kernel<<<grid, 256, 0, stream>>>(st.batch0, num_stages, st.final_label, st.exit_stage, st.final_conf);
    count_launch();
    return check_launch("cascade_init_kernel");
}

}  // namespace fi
