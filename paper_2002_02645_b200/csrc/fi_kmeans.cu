// One Lloyd iteration for the k-means cache of Sec. 4: the entries of such a cache are <cluster centre, majority
// label, fraction of the majority label>.  The assignment step is the look-up itself (k = 1 against the current
// centres); this file holds the update step: per cluster the mean of its points, the majority label among the
// labels the model predicted for them, and that label's share.
//
// update_kernel: grid (clusters, dimension chunks of 256 x 16 bytes).  A CTA walks the assignment array 256 entries at a
// time, compacts the matching point ids in index order (ballot + prefix) and adds those rows into fp32
// accumulators, one per value of the thread's 16 bytes.  Every sum runs in point-index order, so results are bit-identical from run to run;
// integer work (counts, label histogram in shared memory) is exact.
#include "fi_internal.cuh"

namespace fi {
namespace {

constexpr int kKmThreads = 256;
// a thread owns the values of one 16-byte piece of a row: 8 bf16 or 4 float; a CTA covers 256 such pieces
constexpr int kKmMaxClasses = 8192;        // label histogram held in shared memory

template <typename T>
struct Row8;
template <>
struct Row8<uint16_t> {   // bf16 bit patterns
    static constexpr int kVals = 8;
    static __device__ __forceinline__ void add(const uint16_t *p, float (&acc)[8]) {
        const uint4 v = *reinterpret_cast<const uint4 *>(p);
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
        const float4 a = *reinterpret_cast<const float4 *>(p);
        acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&m)[8]) {
        *reinterpret_cast<float4 *>(p) = make_float4(m[0], m[1], m[2], m[3]);
    }
    static __device__ __forceinline__ void copy(float *dst, const float *src) {
        *reinterpret_cast<float4 *>(dst) = *reinterpret_cast<const float4 *>(src);
    }
};

template <typename T>
__global__ void __launch_bounds__(kKmThreads)
update_kernel(const T *__restrict__ points, int64_t ld, const int32_t *__restrict__ point_labels,
              const int32_t *__restrict__ assign, int64_t n, int dim, int num_classes, const T *__restrict__ old_centres,
              T *__restrict__ new_centres, int32_t *__restrict__ counts, int32_t *__restrict__ majority,
              float *__restrict__ fraction) {
    extern __shared__ int32_t hist[];   // [num_classes], only in the CTAs of dimension chunk 0
    __shared__ int32_t match[kKmThreads];
    __shared__ int32_t warp_count[kKmThreads / 32];
    __shared__ int32_t n_match;
    __shared__ int32_t best_cnt[kKmThreads / 32], best_lab[kKmThreads / 32];

    const int c = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d0 = (blockIdx.y * kKmThreads + tid) * Row8<T>::kVals;   // this thread's 16 bytes of every row
    const bool has_dims = d0 < dim;                                    // dim is a multiple of kVals
    const bool do_labels = blockIdx.y == 0;
    if (do_labels)
        for (int l = tid; l < num_classes; l += kKmThreads) hist[l] = 0;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int total = 0;
    __syncthreads();

    for (int64_t base = 0; base < n; base += kKmThreads) {
        const int64_t i = base + tid;
        const bool mine = i < n && assign[i] == c;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, mine);
        if (lane == 0) warp_count[warp] = __popc(ballot);
        __syncthreads();
        int before = 0, all = 0;
#pragma unroll
        for (int w = 0; w < kKmThreads / 32; ++w) {
            before += w < warp ? warp_count[w] : 0;
            all += warp_count[w];
        }
        if (mine) {
            match[before + __popc(ballot & ((1u << lane) - 1u))] = (int32_t)(i - base);
            if (do_labels) {
                const int32_t lab = point_labels[i];   // a label outside [0, num_classes) has no bin: it is not counted
                if ((uint32_t)lab < (uint32_t)num_classes) atomicAdd(&hist[lab], 1);
            }
        }
        if (tid == 0) n_match = all;
        __syncthreads();
        const int m = n_match;
        if (has_dims)
            for (int j = 0; j < m; ++j) Row8<T>::add(points + (base + match[j]) * ld + d0, acc);   // index order
        total += m;
        __syncthreads();
    }

    if (has_dims) {
        T *dst = new_centres + (int64_t)c * dim + d0;
        if (total > 0) {
            float mean[8];
            const float inv_n = (float)total;
#pragma unroll
            for (int e = 0; e < 8; ++e) mean[e] = acc[e] / inv_n;
            Row8<T>::store(dst, mean);
        } else {
            Row8<T>::copy(dst, old_centres + (int64_t)c * dim + d0);   // an empty cluster keeps its centre
        }
    }
    if (do_labels) {
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
}

}  // namespace

fi_status_t launch_kmeans_update(const fi_cache *c, const void *points, int64_t ld, const int32_t *point_labels,
                                 const int32_t *assign, int64_t n, void *new_centres, int32_t *counts,
                                 int32_t *majority, float *fraction, cudaStream_t stream) {
    if (c->size <= 0) return FI_OK;
    if (c->cfg.num_classes > kKmMaxClasses) {
        set_error("fi_kmeans_step: at most %d classes", kKmMaxClasses);
        return FI_ERR_UNSUPPORTED;
    }
    const int chunk = kKmThreads * (c->cfg.dtype == FI_F32 ? 4 : 8);
    dim3 grid((unsigned)c->size, (unsigned)((c->cfg.dim + chunk - 1) / chunk));
    const size_t smem = (size_t)c->cfg.num_classes * sizeof(int32_t);
    if (c->cfg.dtype == FI_F32)
        update_kernel<float><<<grid, kKmThreads, smem, stream>>>((const float *)points, ld, point_labels, assign, n,
                                                                c->cfg.dim, c->cfg.num_classes, (const float *)c->rows,
                                                                (float *)new_centres, counts, majority, fraction);
    else
        update_kernel<uint16_t><<<grid, kKmThreads, smem, stream>>>((const uint16_t *)points, ld, point_labels, assign, n,
                                                                   c->cfg.dim, c->cfg.num_classes,
                                                                   (const uint16_t *)c->rows, (uint16_t *)new_centres,
                                                                   counts, majority, fraction);
    count_launch();
    return check_launch("kmeans update_kernel");
}

}  // namespace fi
