// Row norms, query gather, and the bandwidth-bound streaming look-up (small batches, float32 caches).
//
// The streaming kernel reads every cache row exactly once per group of up to 4 queries with 128-bit
// loads and evaluates the distance in its direct form, sum_j (q_j - c_j)^2, in fp32: differences of
// stored bf16 / fp32 values lose nothing to cancellation, so an exact copy gives exactly 0 and the
// candidate lists need no re-ranking afterwards.
#include "fi_internal.cuh"

namespace fi {

namespace {

constexpr int kStreamThreads = 256;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kRowsPerIter = 4;   // cache rows in flight per thread: 4 x 16 B loads
constexpr int kQB = 4;            // queries served by one pass over the rows
// A single request leaves the registers of three more accumulators per row free: eight rows in flight per thread
// instead of four, which is what the memory system needs from 768 threads per SM to run at its full rate.
constexpr int kRowsPerIterSingle = 8;

__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

template <typename T>
struct Elem;
template <>
struct Elem<float> {
    static constexpr int kPer16 = 4;
    __device__ static __forceinline__ float sqnorm(uint4 v) {
        float a = __uint_as_float(v.x), b = __uint_as_float(v.y), c = __uint_as_float(v.z), d = __uint_as_float(v.w);
        return a * a + b * b + c * c + d * d;
    }
    __device__ static __forceinline__ float sqdiff(uint4 q, uint4 x, float acc) {
        float d0 = __uint_as_float(q.x) - __uint_as_float(x.x);
        float d1 = __uint_as_float(q.y) - __uint_as_float(x.y);
        float d2 = __uint_as_float(q.z) - __uint_as_float(x.z);
        float d3 = __uint_as_float(q.w) - __uint_as_float(x.w);
        acc = fmaf(d0, d0, acc);
        acc = fmaf(d1, d1, acc);
        acc = fmaf(d2, d2, acc);
        acc = fmaf(d3, d3, acc);
        return acc;
    }
};
template <>
struct Elem<uint16_t> {   // bf16 bit patterns
    static constexpr int kPer16 = 8;
    __device__ static __forceinline__ float sqnorm(uint4 v) {
        float s = 0.f;
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float a = bf16lo(w[i]), b = bf16hi(w[i]);
            s = fmaf(a, a, s);
            s = fmaf(b, b, s);
        }
        return s;
    }
    __device__ static __forceinline__ float sqdiff(uint4 q, uint4 x, float acc) {
        uint32_t qw[4] = {q.x, q.y, q.z, q.w};
        uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float d0 = bf16lo(qw[i]) - bf16lo(xw[i]);
            float d1 = bf16hi(qw[i]) - bf16hi(xw[i]);
            acc = fmaf(d0, d0, acc);
            acc = fmaf(d1, d1, acc);
        }
        return acc;
    }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// ---------------------------------------------------------------- K0: squared norms of stored rows
template <typename T>
__global__ void row_norms_kernel(const T *__restrict__ rows, int64_t n, int dim, float *__restrict__ norms,
                                 int32_t *__restrict__ norm_max_bits) {
    int64_t row = (int64_t)blockIdx.x * (blockDim.x / 32) + (threadIdx.x / 32);
    if (row >= n) return;
    int lane = threadIdx.x & 31;
    const uint4 *p = reinterpret_cast<const uint4 *>(rows + row * dim);
    int chunks = dim / Elem<T>::kPer16;
    float s = 0.f;
    for (int c = lane; c < chunks; c += 32) s += Elem<T>::sqnorm(ld_stream16(p + c));
    s = warp_sum(s);
    if (lane == 0) {
        norms[row] = s;
        // norms are >= 0, so their bit patterns order like the values
        if (norm_max_bits && s == s) atomicMax(norm_max_bits, __float_as_int(s));
    }
}

// ---------------------------------------------------------------- gather rows of the active requests
__global__ void gather_rows_kernel(const char *__restrict__ src, int64_t ld_bytes, const int32_t *__restrict__ row_idx,
                                   const int32_t *__restrict__ count_dev, int32_t batch_max, char *__restrict__ dst,
                                   int row_bytes) {
    int count = count_dev ? min(*count_dev, batch_max) : batch_max;
    int chunks = row_bytes / 16;
    if (chunks <= 256) {
        // short rows: a row per warp (a CTA of 256 threads would leave most of them without a chunk)
        const int warps = blockDim.x >> 5, lane = threadIdx.x & 31;
        for (int b = blockIdx.x * warps + (threadIdx.x >> 5); b < count; b += gridDim.x * warps) {
            const uint4 *s = reinterpret_cast<const uint4 *>(src + (int64_t)row_idx[b] * ld_bytes);
            uint4 *d = reinterpret_cast<uint4 *>(dst + (int64_t)b * row_bytes);
            for (int c = lane; c < chunks; c += 32) d[c] = ld_stream16(s + c);
        }
        return;
    }
    for (int b = blockIdx.x; b < count; b += gridDim.x) {
        const uint4 *s = reinterpret_cast<const uint4 *>(src + (int64_t)row_idx[b] * ld_bytes);
        uint4 *d = reinterpret_cast<uint4 *>(dst + (int64_t)b * row_bytes);
        for (int c = threadIdx.x; c < chunks; c += blockDim.x) d[c] = ld_stream16(s + c);
    }
}

// ---------------------------------------------------------------- K5: streaming look-up
// grid = (parts, ceil(batch_max / QB)); CTA (p, g) scans the p-th range of cache rows for queries QB*g..QB*g+QB-1 and
// writes one sorted list of the k best (distance, index) pairs per query.  (QB, ROWS) = (4, 4), or (1, 8) for one request.
template <typename T, int QB, int ROWS>
__global__ void __launch_bounds__(kStreamThreads, QB == 1 ? 4 : 3)
stream_lookup_kernel(const T *__restrict__ X, int64_t n_entries, int dim, const T *__restrict__ Q, int64_t ldq,
                     const int32_t *__restrict__ row_idx, int32_t batch_max, const int32_t *__restrict__ count_dev,
                     int k, int parts, int q_in_smem, float *__restrict__ part_score, int32_t *__restrict__ part_idx) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ float red[kStreamWarps][ROWS * QB];
    __shared__ float best_d[QB][kMaxK];
    __shared__ int32_t best_i[QB][kMaxK];

    const int count = count_dev ? min(*count_dev, batch_max) : batch_max;
    const int q0 = blockIdx.y * QB;
    if (q0 >= count) return;
    const int nq = min(QB, count - q0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunks = dim / Elem<T>::kPer16;

    // query rows: in shared memory when they fit, else read in place (they stay in L1/L2)
    const uint4 *qrow[QB];
#pragma unroll
    for (int j = 0; j < QB; ++j) {
        int b = q0 + (j < nq ? j : 0);
        int64_t r = row_idx ? (int64_t)row_idx[b] : (int64_t)b;
        qrow[j] = reinterpret_cast<const uint4 *>(Q + r * ldq);
    }
    if (q_in_smem) {
        uint4 *sq = reinterpret_cast<uint4 *>(smem_raw);
        for (int j = 0; j < nq; ++j)
            for (int c = tid; c < chunks; c += kStreamThreads) sq[j * chunks + c] = qrow[j][c];
#pragma unroll
        for (int j = 0; j < QB; ++j) qrow[j] = sq + (j < nq ? j : 0) * chunks;
    }
    if (tid < QB * kMaxK) {
        best_d[tid / kMaxK][tid % kMaxK] = __int_as_float(0x7F800000);
        best_i[tid / kMaxK][tid % kMaxK] = -1;
    }
    __syncthreads();

    const int64_t r_begin = n_entries * blockIdx.x / parts;
    const int64_t r_end = n_entries * (blockIdx.x + 1) / parts;

    for (int64_t r = r_begin; r < r_end; r += ROWS) {
        float acc[ROWS][QB];
#pragma unroll
        for (int i = 0; i < ROWS; ++i)
#pragma unroll
            for (int j = 0; j < QB; ++j) acc[i][j] = 0.f;
        const uint4 *xrow[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            int64_t rr = r + i < r_end ? r + i : r_end - 1;   // tail: re-read the last row, result ignored
            xrow[i] = reinterpret_cast<const uint4 *>(X + rr * dim);
        }
        for (int c = tid; c < chunks; c += kStreamThreads) {
            uint4 xv[ROWS];
#pragma unroll
            for (int i = 0; i < ROWS; ++i) xv[i] = ld_stream16(xrow[i] + c);
#pragma unroll
            for (int j = 0; j < QB; ++j) {
                if (j < nq) {
                    uint4 qv = qrow[j][c];
#pragma unroll
                    for (int i = 0; i < ROWS; ++i) acc[i][j] = Elem<T>::sqdiff(qv, xv[i], acc[i][j]);
                }
            }
        }
        // block reduction of the 16 partial sums
#pragma unroll
        for (int i = 0; i < ROWS; ++i)
#pragma unroll
            for (int j = 0; j < QB; ++j) {
                float s = warp_sum(acc[i][j]);
                if (lane == 0) red[warp][i * QB + j] = s;
            }
        __syncthreads();
        if (tid < QB && tid < nq) {
            const int j = tid;
#pragma unroll
            for (int i = 0; i < ROWS; ++i) {
                if (r + i >= r_end) break;
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < kStreamWarps; ++w) s += red[w][i * QB + j];
                // insert (s, r+i) into the ascending list; rows arrive in ascending index, so "<" keeps the
                // smaller index first among equal distances
                if (s < best_d[j][k - 1]) {
                    int pos = k - 1;
                    while (pos > 0 && s < best_d[j][pos - 1]) {
                        best_d[j][pos] = best_d[j][pos - 1];
                        best_i[j][pos] = best_i[j][pos - 1];
                        --pos;
                    }
                    best_d[j][pos] = s;
                    best_i[j][pos] = (int32_t)(r + i);
                }
            }
        }
        __syncthreads();
    }
    // one list per (query, range)
    for (int t = tid; t < nq * k; t += kStreamThreads) {
        int j = t / k, e = t % k;
        int64_t o = ((int64_t)(q0 + j) * parts + blockIdx.x) * k + e;
        part_score[o] = best_d[j][e];
        part_idx[o] = best_i[j][e];
    }
}

}  // namespace

fi_status_t launch_row_norms(const void *rows, int dtype, int64_t n, int dim, float *norms, int32_t *norm_max_bits,
                             cudaStream_t stream) {
    if (n <= 0) return FI_OK;
    const int warps = 8;
    unsigned grid = (unsigned)((n + warps - 1) / warps);
    if (dtype == FI_F32)
        row_norms_kernel<float><<<grid, warps * 32, 0, stream>>>((const float *)rows, n, dim, norms, norm_max_bits);
    else
        row_norms_kernel<uint16_t><<<grid, warps * 32, 0, stream>>>((const uint16_t *)rows, n, dim, norms, norm_max_bits);
    count_launch();
    return check_launch("row_norms_kernel");
}

fi_status_t launch_gather_rows(const void *src, int64_t ld_elems, const int32_t *row_idx, int32_t batch_max,
                               const int32_t *count_dev, void *dst, int dim, size_t elem_size, cudaStream_t stream) {
    if (batch_max <= 0) return FI_OK;
    // (rows of up to 4 KiB go a row per warp, eight rows per CTA)
    const int row_chunks = (int)(dim * elem_size / 16);
    const int grid = row_chunks <= 256 ? (batch_max + 7) / 8 : batch_max;
    gather_rows_kernel<<<grid, 256, 0, stream>>>((const char *)src, ld_elems * (int64_t)elem_size, row_idx, count_dev,
                                                      batch_max, (char *)dst, (int)(dim * elem_size));
    count_launch();
    return check_launch("gather_rows_kernel");
}

fi_status_t launch_stream_lookup(const fi_cache *c, const void *queries, int64_t ld_elems, const int32_t *row_idx,
                                 int32_t batch_max, const int32_t *count_dev, int *parts_out, cudaStream_t stream) {
    const int k = c->cfg.k;
    const bool single = batch_max == 1;
    const int qb = single ? 1 : kQB, rows_per_iter = single ? kRowsPerIterSingle : kRowsPerIter;
    const int groups = (batch_max + qb - 1) / qb;
    const int q_rows = batch_max < qb ? batch_max : qb;   // query rows a CTA actually holds
    size_t q_bytes = (size_t)q_rows * c->cfg.dim * c->elem_size;
    int q_in_smem = q_bytes <= 160 * 1024;
    size_t dyn = q_in_smem ? q_bytes : 0;
    const void *kern = c->cfg.dtype == FI_F32
                           ? (single ? (const void *)stream_lookup_kernel<float, 1, kRowsPerIterSingle>
                                     : (const void *)stream_lookup_kernel<float, kQB, kRowsPerIter>)
                           : (single ? (const void *)stream_lookup_kernel<uint16_t, 1, kRowsPerIterSingle>
                                     : (const void *)stream_lookup_kernel<uint16_t, kQB, kRowsPerIter>);
    if (dyn > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kStreamThreads, dyn) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    // one wave of resident CTAs, but never more ranges than rows / rows per pass or than the scratch holds
    int parts = (per_sm * c->sm_count + groups - 1) / groups;
    int64_t max_parts_rows = (c->size + rows_per_iter - 1) / rows_per_iter;
    if (parts > max_parts_rows) parts = (int)max_parts_rows;
    int64_t max_parts_scratch = (int64_t)(c->part_entries / ((size_t)batch_max * (size_t)k));
    if (parts > max_parts_scratch) parts = (int)max_parts_scratch;
    if (parts < 1) parts = 1;
    *parts_out = parts;
    dim3 grid((unsigned)parts, (unsigned)groups);
    const void *rows = c->rows;
    int64_t n = c->size;
    int dim = c->cfg.dim, k_arg = k;
    float *part_score = c->part_score;
    int32_t *part_idx = c->part_idx;
    void *args[] = {&rows, &n, &dim, &queries, &ld_elems, &row_idx, &batch_max, &count_dev, &k_arg, &parts, &q_in_smem,
                    &part_score, &part_idx};
    cudaLaunchKernel(kern, grid, dim3(kStreamThreads), args, dyn, stream);   // (a failed launch is reported below)
    count_launch();
    return check_launch("stream_lookup_kernel");
}

}  // namespace fi
