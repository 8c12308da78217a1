// One Lloyd iteration for the k-means cache of Sec. 4: the entries of such a cache are <cluster centre, majority
// label, fraction of the majority label>.  The assignment step is the look-up itself (k = 1 against the current
// centres); this file holds the update step: per cluster the mean of its points, the majority label among the
// labels the model predicted for them, and that label's share.
//
// update_sum_kernel: grid (clusters, dimension chunks of 256 x 16 bytes, segments of the point range).  A CTA walks
// its segment of the assignment array 1,024 entries at a time (4 consecutive ones per thread), compacts the matching
// point ids in index order (per-thread counts, prefix over the CTA) and adds those rows into fp32 accumulators, one
// per value of the thread's 16 bytes, eight row loads in flight; update_mean_kernel adds the segments' sums in
// segment order.  Every sum runs in a fixed order, so results are bit-identical from run to run; integer work
// (counts, label histogram in shared memory) is exact.
#include "fi_internal.cuh"

namespace fi {
namespace {

constexpr int kKmThreads = 256;
constexpr int kKmPerThread = 4;                        // consecutive assignments a thread inspects per pass
constexpr int kKmPass = kKmThreads * kKmPerThread;     // assignments per pass of a CTA
constexpr int kKmMaxSegments = 64;                     // the point range is cut into at most this many segments
// a thread owns the values of one 16-byte piece of a row: 8 bf16 or 4 float; a CTA covers 256 such pieces
constexpr int kKmMaxClasses = 8192;        // label histogram held in shared memory

template <typename T>
struct Row8;
template <>
struct Row8<uint16_t> {   // bf16 bit patterns
    static constexpr int kVals = 8;
    static __device__ __forceinline__ void add(const uint16_t *p, float (&acc)[8]) {
        add(*reinterpret_cast<const uint4 *>(p), acc);
    }
    static __device__ __forceinline__ void add(const uint4 v, float (&acc)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc[2 * i] += __uint_as_float(w[i] << 16);
            acc[2 * i + 1] += __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ void store(uint16_t *p, const float (&m)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // round to nearest, ties to even
            uint32_t a = __float_as_uint(m[2 * i]), b = __float_as_uint(m[2 * i + 1]);
            a = (a + 0x7FFFu + ((a >> 16) & 1u)) >> 16;
            b = (b + 0x7FFFu + ((b >> 16) & 1u)) >> 16;
            w[i] = a | (b << 16);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    static __device__ __forceinline__ void copy(uint16_t *dst, const uint16_t *src) {
        *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
    }
};
template <>
struct Row8<float> {
    static constexpr int kVals = 4;
    static __device__ __forceinline__ void add(const float *p, float (&acc)[8]) {
        add(*reinterpret_cast<const uint4 *>(p), acc);
    }
    static __device__ __forceinline__ void add(const uint4 v, float (&acc)[8]) {
        acc[0] += __uint_as_float(v.x); acc[1] += __uint_as_float(v.y);
        acc[2] += __uint_as_float(v.z); acc[3] += __uint_as_float(v.w);
    }
    static __device__ __forceinline__ void store(float *p, const float (&m)[8]) {
        *reinterpret_cast<float4 *>(p) = make_float4(m[0], m[1], m[2], m[3]);
    }
    static __device__ __forceinline__ void copy(float *dst, const float *src) {
        *reinterpret_cast<float4 *>(dst) = *reinterpret_cast<const float4 *>(src);
    }
};

// Compaction of one pass: which of this thread's kKmPerThread consecutive points (from i0) belong to cluster c; the
// matching offsets (relative to the pass) go to match[] in index order.  Returns the pass's number of matches.
__device__ __forceinline__ int compact_pass(const int32_t *__restrict__ assign, int64_t i0, int64_t n, int c, int32_t *match,
                                            int32_t *warp_count, uint32_t &mine) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    mine = 0;
#pragma unroll
    for (int q = 0; q < kKmPerThread; ++q)
        if (i0 + q < n && assign[i0 + q] == c) mine |= 1u << q;
    const int cnt = __popc(mine);
    // exclusive prefix of the counts over the CTA: inside the warp by shuffles, across warps through shared memory
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) warp_count[warp] = incl;
    __syncthreads();
    int before = incl - cnt, all = 0;
#pragma unroll
    for (int w = 0; w < kKmThreads / 32; ++w) {
        before += w < warp ? warp_count[w] : 0;
        all += warp_count[w];
    }
    if (match) {
#pragma unroll
        for (int q = 0; q < kKmPerThread; ++q)
            if ((mine >> q) & 1u) match[before++] = tid * kKmPerThread + q;
    }
    return all;
}

// Step 1.  Grid (clusters, dimension chunks, segments of the point range).  CTA (c, y, s) adds the rows of cluster c
// among the points of segment s, in index order, and leaves the sums in partial[c][s][dim]: a big cluster is spread
// over as many CTAs as there are segments instead of being one CTA's serial chain.  The CTAs (c, 0, 0) also walk all
// points once for the integer work: the cluster's size, its label histogram, majority label and share.
template <typename T>
__global__ void __launch_bounds__(kKmThreads)
update_sum_kernel(const T *__restrict__ points, int64_t ld, const int32_t *__restrict__ point_labels,
                  const int32_t *__restrict__ assign, int64_t n, int dim, int num_classes, int64_t seg_len,
                  float *__restrict__ partial, int32_t *__restrict__ counts, int32_t *__restrict__ majority,
                  float *__restrict__ fraction) {
    extern __shared__ int32_t hist[];   // [num_classes], only in the CTAs (c, 0, 0)
    __shared__ int32_t match[kKmPass];
    __shared__ int32_t warp_count[kKmThreads / 32];
    __shared__ int32_t best_cnt[kKmThreads / 32], best_lab[kKmThreads / 32];

    const int c = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d0 = (blockIdx.y * kKmThreads + tid) * Row8<T>::kVals;   // this thread's 16 bytes of every row
    const bool has_dims = d0 < dim;                                    // dim is a multiple of kVals
    const bool do_labels = blockIdx.y == 0 && blockIdx.z == 0;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};

    const int64_t seg_lo = (int64_t)blockIdx.z * seg_len;
    const int64_t seg_hi = seg_lo + seg_len < n ? seg_lo + seg_len : n;
    for (int64_t base = seg_lo; base < seg_hi; base += kKmPass) {
        uint32_t mine;
        const int m = compact_pass(assign, base + (int64_t)tid * kKmPerThread, seg_hi, c, match, warp_count, mine);
        __syncthreads();
        if (has_dims) {
            // index order; the loads of eight rows are issued before their sums
            int j = 0;
            for (; j + 8 <= m; j += 8) {
                uint4 v[8];
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    v[e] = *reinterpret_cast<const uint4 *>(points + (base + match[j + e]) * ld + d0);
#pragma unroll
                for (int e = 0; e < 8; ++e) Row8<T>::add(v[e], acc);
            }
            for (; j < m; ++j) Row8<T>::add(points + (base + match[j]) * ld + d0, acc);
        }
        __syncthreads();
    }
    if (has_dims) {
        float *dst = partial + ((int64_t)c * gridDim.z + blockIdx.z) * dim + d0;
#pragma unroll
        for (int e = 0; e < Row8<T>::kVals; ++e) dst[e] = acc[e];
    }
    if (!do_labels) return;

    // ---- integer work over all points
    for (int l = tid; l < num_classes; l += kKmThreads) hist[l] = 0;
    __syncthreads();
    int total = 0;
    for (int64_t base = 0; base < n; base += kKmPass) {
        const int64_t i0 = base + (int64_t)tid * kKmPerThread;
        uint32_t mine;
        total += compact_pass(assign, i0, n, c, nullptr, warp_count, mine);
#pragma unroll
        for (int q = 0; q < kKmPerThread; ++q) {
            if ((mine >> q) & 1u) {
                const int32_t lab = point_labels[i0 + q];   // a label outside [0, num_classes) has no bin: it is not counted
                if ((uint32_t)lab < (uint32_t)num_classes) atomicAdd(&hist[lab], 1);
            }
        }
        __syncthreads();
    }
    // majority label: largest count, smaller label on ties
    int bc = -1, bl = -1;
    for (int l = tid; l < num_classes; l += kKmThreads) {
        const int h = hist[l];
        if (h > bc) {   // labels visited in ascending order per thread: ">" keeps the smaller one
            bc = h;
            bl = l;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const int oc = __shfl_xor_sync(0xFFFFFFFFu, bc, o), ol = __shfl_xor_sync(0xFFFFFFFFu, bl, o);
        if (oc > bc || (oc == bc && ol >= 0 && (bl < 0 || ol < bl))) {
            bc = oc;
            bl = ol;
        }
    }
    if (lane == 0) {
        best_cnt[warp] = bc;
        best_lab[warp] = bl;
    }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < kKmThreads / 32; ++w)
            if (best_cnt[w] > bc || (best_cnt[w] == bc && best_lab[w] >= 0 && (bl < 0 || best_lab[w] < bl))) {
                bc = best_cnt[w];
                bl = best_lab[w];
            }
        counts[c] = total;
        majority[c] = total > 0 ? bl : -1;
        fraction[c] = total > 0 ? (float)bc / (float)total : 0.f;
    }
}

// Step 2.  Grid (clusters, dimension chunks): the segments' sums are added in segment order (a fixed order: reruns are
// bit-identical), divided by the cluster's size and stored; an empty cluster keeps its centre.
template <typename T>
__global__ void __launch_bounds__(kKmThreads)
update_mean_kernel(const float *__restrict__ partial, int segments, const int32_t *__restrict__ counts, int dim,
                   const T *__restrict__ old_centres, T *__restrict__ new_centres) {
    const int c = blockIdx.x;
    const int d0 = (blockIdx.y * kKmThreads + threadIdx.x) * Row8<T>::kVals;
    if (d0 >= dim) return;
    T *dst = new_centres + (int64_t)c * dim + d0;
    const int total = counts[c];
    if (total <= 0) {
        Row8<T>::copy(dst, old_centres + (int64_t)c * dim + d0);
        return;
    }
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int sgm = 0; sgm < segments; ++sgm) {
        const float *src = partial + ((int64_t)c * segments + sgm) * dim + d0;
#pragma unroll
        for (int e = 0; e < Row8<T>::kVals; ++e) acc[e] += src[e];
    }
    float mean[8];
    const float cnt = (float)total;
#pragma unroll
    for (int e = 0; e < 8; ++e) mean[e] = acc[e] / cnt;
    Row8<T>::store(dst, mean);
}

}  // namespace

fi_status_t launch_kmeans_update(fi_cache *c, const void *points, int64_t ld, const int32_t *point_labels,
                                 const int32_t *assign, int64_t n, void *new_centres, int32_t *counts,
                                 int32_t *majority, float *fraction, cudaStream_t stream) {
    if (c->size <= 0) return FI_OK;
    if (c->cfg.num_classes > kKmMaxClasses) {
        set_error("fi_kmeans_step: at most %d classes", kKmMaxClasses);
        return FI_ERR_UNSUPPORTED;
    }
    // segments of whole passes, at most kKmMaxSegments of them
    const int64_t passes = (n + kKmPass - 1) / kKmPass;
    const int64_t per_seg = passes > kKmMaxSegments ? (passes + kKmMaxSegments - 1) / kKmMaxSegments : 1;
    const int segments = passes > 0 ? (int)((passes + per_seg - 1) / per_seg) : 1;
    const int64_t seg_len = per_seg * kKmPass;
    const size_t need = (size_t)c->size * (size_t)segments * (size_t)c->cfg.dim;
    if (c->km_partial_elems < need) {
        // grown on demand; the stream may still be reading the old buffer
        cudaError_t e = cudaStreamSynchronize(stream);
        if (e == cudaSuccess) {
            cudaFree(c->km_partial);
            c->km_partial = nullptr;
            c->km_partial_elems = 0;
            e = cudaMalloc(reinterpret_cast<void **>(&c->km_partial), need * sizeof(float));
        }
        if (e != cudaSuccess) {
            set_error("cannot allocate the k-means partial sums: %s", cudaGetErrorString(e));
            cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? FI_ERR_OOM : FI_ERR_CUDA;
        }
        c->km_partial_elems = need;
    }
    const int chunk = kKmThreads * (c->cfg.dtype == FI_F32 ? 4 : 8);
    const unsigned ychunks = (unsigned)((c->cfg.dim + chunk - 1) / chunk);
    dim3 grid((unsigned)c->size, ychunks, (unsigned)segments);
    dim3 grid2((unsigned)c->size, ychunks);
    const size_t smem = (size_t)c->cfg.num_classes * sizeof(int32_t);
    if (c->cfg.dtype == FI_F32) {
        update_sum_kernel<float><<<grid, kKmThreads, smem, stream>>>((const float *)points, ld, point_labels, assign, n,
                                                                    c->cfg.dim, c->cfg.num_classes, seg_len, c->km_partial,
                                                                    counts, majority, fraction);
        update_mean_kernel<float><<<grid2, kKmThreads, 0, stream>>>(c->km_partial, segments, counts, c->cfg.dim,
                                                                   (const float *)c->rows, (float *)new_centres);
    } else {
        update_sum_kernel<uint16_t><<<grid, kKmThreads, smem, stream>>>((const uint16_t *)points, ld, point_labels, assign,
                                                                       n, c->cfg.dim, c->cfg.num_classes, seg_len,
                                                                       c->km_partial, counts, majority, fraction);
        update_mean_kernel<uint16_t><<<grid2, kKmThreads, 0, stream>>>(c->km_partial, segments, counts, c->cfg.dim,
                                                                      (const uint16_t *)c->rows, (uint16_t *)new_centres);
    }
    count_launch(2);
    return check_launch("kmeans update kernels");
}

}  // namespace fi
