// The C ABI declared in include/fi.h: argument checks, memory ownership, and the order in which the
// kernels of a look-up / cascade step are enqueued.  No arithmetic of the method lives here.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "fi_internal.cuh"

namespace fi {

namespace {
thread_local char g_err[512] = "";
std::atomic<long long> g_launches{0};

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

fi_status_t cuda_fail(cudaError_t e, const char *what) {
    set_error("%s: %s", what, cudaGetErrorString(e));
    cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? FI_ERR_OOM : FI_ERR_CUDA;
}

__global__ void fill_f32_kernel(float *p, int64_t n, float v) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = v;
}

template <typename T>
fi_status_t dev_alloc(T **p, size_t count, const char *what) {
    *p = nullptr;
    if (count == 0) count = 1;
    cudaError_t e = cudaMalloc(reinterpret_cast<void **>(p), count * sizeof(T));
    if (e != cudaSuccess) return cuda_fail(e, what);
    return FI_OK;
}

void free_all(fi_cache *c) {
    cudaFree(c->rows);
    cudaFree(c->labels);
    cudaFree(c->weights);
    cudaFree(c->norms);
    cudaFree(c->part_score);
    cudaFree(c->part_idx);
    cudaFree(c->q_compact);
    cudaFree(c->slot_label);
    cudaFree(c->slot_conf);
    cudaFree(c->slot_hit);
    cudaFree(c->plan_dev);
    cudaFree(c->row_bound);
    cudaFree(c->tail_dump);
    cudaFree(c->calib_acc);
    cudaFree(c->km_dist);
    cudaFree(c->km_partial);
    cudaFree(c->status_dev);
    cudaFree(c->cert_dev);
    cudaFree(c->slot_cert);
    cudaFree(c->repair_list);
    cudaFree(c->h2d_stage);
    for (int i = 0; i < kMaxPending; ++i)
        if (c->pend_ev[i]) cudaEventDestroy(c->pend_ev[i]);
    if (c->copy_ev) {
        for (int i = 0; i < kMaxHostStages; ++i) cudaEventDestroy(c->copy_ev[i]);
        delete[] c->copy_ev;
        c->copy_ev = nullptr;
    }
    if (c->copy_stream) {
        cudaStreamDestroy(c->copy_stream);
        c->copy_stream = nullptr;
    }
    if (c->prof_ev) {
        for (int i = 0; i < 2 * kProfSlots; ++i) cudaEventDestroy(c->prof_ev[i]);
        delete[] c->prof_ev;
        c->prof_ev = nullptr;
    }
}

// events around the distance kernel of one look-up
void prof_mark(fi_cache *c, int which, cudaStream_t stream) {
    if (!c->prof_on || !c->prof_ev) return;
    cudaEventRecord(c->prof_ev[2 * (c->prof_n % kProfSlots) + which], stream);
    if (which == 1) ++c->prof_n;
}

int resolve_path(const fi_cache *c, int batch_max) {
    if (c->size == 0) return FI_PATH_STREAM;   // nothing to contract with; the streaming kernel reports "no neighbour"
    if (c->cfg.path == FI_PATH_STREAM || c->cfg.path == FI_PATH_GEMM) return c->cfg.path;
    if (c->cfg.dtype == FI_F32 || batch_max <= kStreamMaxBatch) return FI_PATH_STREAM;
    return FI_PATH_GEMM;
}

// The candidate-list scratch is sized once, at create, for every batch up to max_batch against every cache size up to
// capacity (gemm_part_entries_bound); a look-up never allocates or synchronises.  A plan that would not fit is a bug of
// that bound and is refused instead of being run.
fi_status_t check_part_scratch(const fi_cache *c, size_t entries) {
    if (entries <= c->part_entries) return FI_OK;
    set_error("look-up scratch too small (%zu entries needed, %zu allocated at create)", entries, c->part_entries);
    return FI_ERR_CAPACITY;
}

fi_status_t lookup_impl(fi_cache *c, const void *queries, int64_t ld, const int32_t *row_idx, int32_t batch_max,
                        const int32_t *count_dev, const fi_lookup_out_t &out, cudaStream_t stream) {
    if (batch_max == 0) return FI_OK;
    refresh_view(c, stream);
    const int path = resolve_path(c, batch_max);
    FinalizeArgs fa;
    fa.queries = queries;
    fa.ld_elems = ld;
    fa.row_idx = row_idx;
    fa.batch_max = batch_max;
    fa.count_dev = count_dev;
    fa.out = out;
    fa.out_slot = nullptr;
    fa.fill_repair_list = false;
    fi_status_t st;
    if (path == FI_PATH_STREAM) {
        int parts = 1;
        prof_mark(c, 0, stream);
        st = launch_stream_lookup(c, queries, ld, row_idx, batch_max, count_dev, &parts, stream);
        if (st != FI_OK) return st;
        prof_mark(c, 1, stream);
        fa.parts = parts;
        fa.list_len = c->cfg.k;
        fa.refine = 0;
    } else {
        if (c->cfg.dtype != FI_BF16) {
            set_error("the tensor-core path needs a bf16 cache");
            return FI_ERR_UNSUPPORTED;
        }
        st = check_part_scratch(c, gemm_part_entries(batch_max, c->size, c->sm_count, c->cfg.k, c->cfg.dim));
        if (st != FI_OK) return st;
        const void *qsrc = queries;
        int64_t qld = ld;
        if (row_idx) {
            st = launch_gather_rows(queries, ld, row_idx, batch_max, count_dev, c->q_compact, c->cfg.dim, c->elem_size, stream);
            if (st != FI_OK) return st;
            qsrc = c->q_compact;
            qld = c->cfg.dim;
            fa.queries = qsrc;
            fa.ld_elems = qld;
            fa.row_idx = nullptr;
        } else if (batch_max < kMinMapRows) {
            // Measured: TMA loads through a map over fewer than four rows run the whole kernel 20 % slower (batches of 2
            // and 3 against 50,000 x 16,384: 319 us, of 4: 263 us).  Such batches are copied into the gather buffer and
            // loaded through a map over four of its rows; the rows past the batch hold whatever was there, their
            // results are never read.
            cudaError_t e = cudaMemcpy2DAsync(c->q_compact, (size_t)c->cfg.dim * c->elem_size, queries, (size_t)ld * c->elem_size,
                                              (size_t)c->cfg.dim * c->elem_size, (size_t)batch_max, cudaMemcpyDeviceToDevice, stream);
            if (e != cudaSuccess) return cuda_fail(e, "copying a small batch of queries");
            qsrc = c->q_compact;
            qld = c->cfg.dim;
        }
        const int32_t gemm_rows = qsrc == c->q_compact && batch_max < kMinMapRows ? kMinMapRows : batch_max;
        prof_mark(c, 0, stream);
        st = launch_gemm_select(c, qsrc, qld, gemm_rows, count_dev, stream);
        if (st != FI_OK) return st;
        prof_mark(c, 1, stream);
        fa.parts = -1;
        fa.list_len = -1;
        fa.refine = 1;
        if (c->repair_on) {
            // Exact repair: queries whose neighbours the certificate cannot prove are looked up again by the streaming
            // kernel (direct fp32 distances over the whole cache).  The list and its length stay on the device; the
            // kernels of the second pass return at once when the list is empty.
            fa.fill_repair_list = true;
            cudaError_t e = cudaMemsetAsync(c->cert_dev + 2, 0, sizeof(int32_t), stream);
            if (e != cudaSuccess) return cuda_fail(e, "clearing the repair list");
            st = launch_finalize(c, fa, stream);
            if (st != FI_OK) return st;
            int parts = 1;
            // the queries the distance GEMM read are indexed by slot (gathered copy, or the caller's rows as they are)
            st = launch_stream_lookup(c, fa.queries, fa.ld_elems, c->repair_list, kRepairCap, c->cert_dev + 2, &parts, stream);
            if (st != FI_OK) return st;
            FinalizeArgs fr = fa;
            fr.row_idx = nullptr;
            fr.batch_max = kRepairCap;
            fr.count_dev = c->cert_dev + 2;
            fr.parts = parts;
            fr.list_len = c->cfg.k;
            fr.refine = 0;
            fr.out_slot = c->repair_list;
            fr.fill_repair_list = false;
            return launch_finalize(c, fr, stream);
        }
    }
    return launch_finalize(c, fa, stream);
}

// The status words of `n` caches, fetched behind whatever is queued on `stream`; call before the stream is synchronised
// and hand the words to status_from_words afterwards.
cudaError_t fetch_status_words(fi_cache *const *caches, int n, int32_t *words, cudaStream_t stream) {
    cudaError_t e = cudaSuccess;
    for (int l = 0; l < n && e == cudaSuccess; ++l)
        e = cudaMemcpyAsync(words + l, caches[l]->status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, stream);
    return e;
}

// FI_ERR_TIMEOUT (and the words cleared) when a kernel of one of the caches gave up on a bounded wait: the results
// of that call are not to be trusted.
fi_status_t status_from_words(fi_cache *const *caches, int n, const int32_t *words, const char *who) {
    fi_status_t st = FI_OK;
    for (int l = 0; l < n; ++l) {
        if (words[l] == 0) continue;
        cudaMemset(caches[l]->status_dev, 0, sizeof(int32_t));
        if (st == FI_OK) {
            set_error("%s: a kernel gave up on a bounded wait (code %d, site %d, cache %d); the results are invalid", who,
                      words[l] & 0xFF, words[l] >> 8, l);
            st = FI_ERR_TIMEOUT;
        }
    }
    return st;
}

}  // namespace

// Entries a look-up enqueued now on `stream` may read.  Inserts retire in order: one counts when its event has completed
// (its rows, labels, weights and norms are then visible to every later launch) or when it was enqueued on `stream`
// itself (stream order); the first insert that is neither ends the prefix, whatever follows it.
void refresh_view(fi_cache *c, cudaStream_t stream) {
    while (c->pend_n > 0) {
        PendingInsert &p = c->pending[c->pend_head];
        if (cudaEventQuery(p.ev) != cudaSuccess) {
            cudaGetLastError();   // "not ready" is an answer, not a failure
            break;
        }
        c->committed = p.size_after;
        c->pend_head = (c->pend_head + 1) % kMaxPending;
        --c->pend_n;
    }
    int64_t view = c->committed;
    for (int i = 0; i < c->pend_n; ++i) {
        const PendingInsert &p = c->pending[(c->pend_head + i) % kMaxPending];
        if (p.stream != stream) break;
        view = p.size_after;
    }
    c->size = view;
}

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

fi_status_t check_launch(const char *what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, what);
    return FI_OK;
}

}  // namespace fi

using namespace fi;

// The projection object behind its opaque handle: the weight rows live in a cache object of their own (its rows are
// the B operand of the product, its per-row weights hold the bias), plus an output buffer for the cascade step.
struct fi_projection {
    fi_cache *w;
    int32_t in_dim, out_dim, max_batch, device;
    int32_t *zero_labels;   // [out_dim]
    float *zero_bias;       // [out_dim]
    void *y;                // [max_batch x out_dim] bf16, used by fi_cascade_step_projected
};

extern "C" {

fi_status_t fi_cache_create(const fi_cache_config_t *cfg, fi_cache_t **out) {
    if (out) *out = nullptr;
    if (!cfg || !out) {
        set_error("fi_cache_create: null argument");
        return FI_ERR_INVALID_ARG;
    }
    const bool bf16 = cfg->dtype == FI_BF16;
    if ((cfg->dtype != FI_F32 && !bf16) || cfg->dim <= 0 || cfg->dim % (bf16 ? 8 : 4) != 0 || cfg->capacity <= 0 ||
        cfg->capacity > kMaxEntries ||
        cfg->k < 1 || cfg->k > kMaxK || cfg->max_batch < 1 || cfg->num_classes < 1 ||
        (cfg->rule != FI_HIT_CONF_GT && cfg->rule != FI_HIT_DIST_LE) ||
        (cfg->metric != FI_METRIC_SQL2 && cfg->metric != FI_METRIC_L2) || cfg->path < FI_PATH_AUTO ||
        cfg->path > FI_PATH_GEMM) {
        set_error("fi_cache_create: invalid configuration (dim %d dtype %d capacity %lld k %d max_batch %d)", cfg->dim,
                  cfg->dtype, (long long)cfg->capacity, cfg->k, cfg->max_batch);
        return FI_ERR_INVALID_ARG;
    }
    if (cfg->path == FI_PATH_GEMM && !bf16) {
        set_error("fi_cache_create: the tensor-core path needs a bf16 cache");
        return FI_ERR_UNSUPPORTED;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) {
        cudaGetLastError();
        set_error("fi_cache_create: no CUDA device %d", cfg->device);
        return FI_ERR_CUDA;
    }
    DeviceGuard guard(cfg->device);
    if (!guard.ok) {
        set_error("fi_cache_create: cannot select device %d", cfg->device);
        return FI_ERR_CUDA;
    }
    fi_cache *c = new (std::nothrow) fi_cache();
    if (!c) {
        set_error("fi_cache_create: out of host memory");
        return FI_ERR_OOM;
    }
    memset(c, 0, sizeof *c);
    c->cfg = *cfg;
    c->elem_size = bf16 ? 2 : 4;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) {
        delete c;
        return cuda_fail(cudaGetLastError(), "fi_cache_create: device properties");
    }
    c->sm_count = prop.multiProcessorCount;
    c->sm_total = prop.multiProcessorCount;

    fi_status_t st = FI_OK;
    auto need = [&](fi_status_t s) {
        if (st == FI_OK) st = s;
    };
    unsigned char *rows = nullptr;
    need(dev_alloc(&rows, (size_t)cfg->capacity * cfg->dim * c->elem_size, "allocating cache rows"));
    c->rows = rows;
    if (st == FI_OK) need(dev_alloc(&c->labels, (size_t)cfg->capacity, "allocating labels"));
    if (st == FI_OK) need(dev_alloc(&c->weights, (size_t)cfg->capacity, "allocating weights"));
    if (st == FI_OK) need(dev_alloc(&c->norms, (size_t)cfg->capacity, "allocating norms"));
    // candidate lists: the streaming kernel cuts the rows into up to 16 ranges per SM for a group of 4 queries
    size_t entries = (size_t)16 * c->sm_count * 4 * cfg->k;
    if (entries < (size_t)cfg->max_batch * cfg->k * 2) entries = (size_t)cfg->max_batch * cfg->k * 2;
    if (bf16) {
        size_t g = gemm_part_entries_bound(cfg->max_batch, cfg->capacity, c->sm_count, cfg->k, cfg->dim);
        if (g > entries) entries = g;
    }
    if (st == FI_OK) need(dev_alloc(&c->part_score, entries, "allocating candidate scores"));
    if (st == FI_OK) need(dev_alloc(&c->part_idx, entries, "allocating candidate indices"));
    c->part_entries = entries;
    if (st == FI_OK && bf16) {
        unsigned char *qc = nullptr;
        // (at least kMinMapRows rows: see lookup_impl)
        need(dev_alloc(&qc, (size_t)(cfg->max_batch < kMinMapRows ? kMinMapRows : cfg->max_batch) * cfg->dim * c->elem_size,
                       "allocating the gathered-query buffer"));
        c->q_compact = qc;
    }
    if (st == FI_OK) need(dev_alloc(&c->slot_label, (size_t)cfg->max_batch, "allocating slot labels"));
    if (st == FI_OK) need(dev_alloc(&c->slot_conf, (size_t)cfg->max_batch, "allocating slot confidences"));
    if (st == FI_OK) need(dev_alloc(&c->slot_hit, (size_t)cfg->max_batch, "allocating slot hit flags"));
    if (st == FI_OK) need(dev_alloc(&c->plan_dev, 1, "allocating the plan"));
    if (st == FI_OK && bf16)
        need(dev_alloc(&c->row_bound, ((size_t)cfg->max_batch + 512) * gemm_list_len(cfg->k), "allocating the row bounds"));
    for (int i = 0; i < kMaxPending && st == FI_OK; ++i) {
        cudaError_t e = cudaEventCreateWithFlags(&c->pend_ev[i], cudaEventDisableTiming);
        if (e != cudaSuccess) st = cuda_fail(e, "creating the insert events");
    }
    if (st == FI_OK) need(dev_alloc(&c->status_dev, 1, "allocating the status word"));
    if (st == FI_OK) need(dev_alloc(&c->cert_dev, (size_t)kCertWords, "allocating the certificate block"));
    if (st == FI_OK) need(dev_alloc(&c->slot_cert, (size_t)cfg->max_batch, "allocating the certificate flags"));
    if (st == FI_OK) need(dev_alloc(&c->repair_list, (size_t)kRepairCap, "allocating the repair list"));
    if (st == FI_OK) {
        cudaError_t e = cudaMemset(c->cert_dev, 0, kCertWords * sizeof(int32_t));
        if (e == cudaSuccess) e = cudaMemset(c->slot_cert, 1, (size_t)cfg->max_batch);
        if (e != cudaSuccess) st = cuda_fail(e, "clearing the certificate block");
    }
    if (st == FI_OK) {
        cudaError_t e = cudaMemset(c->status_dev, 0, sizeof(int32_t));
        if (e != cudaSuccess) st = cuda_fail(e, "clearing the status word");
    }
    if (st == FI_OK && bf16) {
        // everything a look-up on the tensor-core path needs is set up here, so that no look-up ever allocates,
        // synchronises or re-encodes: partial-sum slots (shapes that can reach wave + tail mode), the kernels'
        // per-device attributes, and tensor maps over all `capacity` rows (rows not yet inserted read as zero and
        // are masked by the row count the kernels are given)
        const size_t units = gemm_tail_units(cfg->max_batch, cfg->dim, c->sm_count);
        if (units > 0) {
            need(dev_alloc(&c->tail_dump, units * 256 * 256, "allocating the partial-sum buffer of the distance GEMM"));
            if (st == FI_OK) c->tail_dump_units = units;
        }
        if (st == FI_OK) need(prepare_gemm_kernels(cfg->device));
        if (st == FI_OK) {
            cudaError_t e = cudaMemset(c->rows, 0, (size_t)cfg->capacity * cfg->dim * c->elem_size);
            if (e != cudaSuccess) st = cuda_fail(e, "clearing the cache rows");
        }
        if (st == FI_OK) need(ensure_tensor_maps(c));
    }
    if (st != FI_OK) {
        free_all(c);
        delete c;
        return st;
    }
    *out = c;
    return FI_OK;
}

fi_status_t fi_cache_destroy(fi_cache_t *c) {
    if (!c) return FI_OK;
    DeviceGuard guard(c->cfg.device);
    cudaDeviceSynchronize();
    free_all(c);
    cudaGetLastError();
    delete c;
    return FI_OK;
}

fi_status_t fi_cache_insert(fi_cache_t *c, const void *vecs, const int32_t *labels, const float *weights, int64_t n,
                            void *cuda_stream) {
    if (!c || n < 0 || (n > 0 && (!vecs || !labels))) {
        set_error("fi_cache_insert: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    if (n == 0) return FI_OK;
    if (c->enqueued + n > c->cfg.capacity) {
        set_error("fi_cache_insert: %lld entries do not fit (size %lld, capacity %lld)", (long long)n, (long long)c->enqueued,
                  (long long)c->cfg.capacity);
        return FI_ERR_CAPACITY;
    }
    if ((reinterpret_cast<uintptr_t>(vecs) & 15) != 0) {
        set_error("fi_cache_insert: vectors must be 16-byte aligned");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t row_bytes = (size_t)c->cfg.dim * c->elem_size;
    // a full ring of inserts in flight: wait for the oldest (the only place an insert blocks the host)
    if (c->pend_n == kMaxPending) {
        cudaError_t e0 = cudaEventSynchronize(c->pending[c->pend_head].ev);
        if (e0 != cudaSuccess) return cuda_fail(e0, "fi_cache_insert: waiting for an earlier insert");
        c->committed = c->pending[c->pend_head].size_after;
        c->pend_head = (c->pend_head + 1) % kMaxPending;
        --c->pend_n;
    }
    const int64_t at = c->enqueued;   // the new entries go behind everything enqueued so far
    unsigned char *dst = static_cast<unsigned char *>(c->rows) + (size_t)at * row_bytes;
    cudaError_t e = cudaMemcpyAsync(dst, vecs, (size_t)n * row_bytes, cudaMemcpyDeviceToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_insert: copying rows");
    e = cudaMemcpyAsync(c->labels + at, labels, (size_t)n * sizeof(int32_t), cudaMemcpyDeviceToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_insert: copying labels");
    if (weights) {
        e = cudaMemcpyAsync(c->weights + at, weights, (size_t)n * sizeof(float), cudaMemcpyDeviceToDevice, stream);
        if (e != cudaSuccess) return cuda_fail(e, "fi_cache_insert: copying weights");
    } else {
        int grid = (int)((n + 255) / 256 < 1024 ? (n + 255) / 256 : 1024);
        fill_f32_kernel<<<grid, 256, 0, stream>>>(c->weights + at, n, 1.0f);
        count_launch();
        fi_status_t st = check_launch("fill_f32_kernel");
        if (st != FI_OK) return st;
    }
    fi_status_t st = launch_row_norms(dst, c->cfg.dtype, n, c->cfg.dim, c->norms + at, c->cert_dev + 3, stream);
    if (st != FI_OK) return st;
    // the entries become visible to look-ups on other streams when this event has completed
    const int slot = (c->pend_head + c->pend_n) % kMaxPending;
    e = cudaEventRecord(c->pend_ev[slot], stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_insert: recording the completion event");
    c->enqueued = at + n;
    c->pending[slot] = PendingInsert{stream, c->pend_ev[slot], c->enqueued};
    ++c->pend_n;
    return FI_OK;
}

fi_status_t fi_cache_set_threshold(fi_cache_t *c, float tau) {
    if (!c) {
        set_error("fi_cache_set_threshold: null cache");
        return FI_ERR_INVALID_ARG;
    }
    c->cfg.threshold = tau;
    return FI_OK;
}

fi_status_t fi_cache_set_path(fi_cache_t *c, int32_t path) {
    if (!c || path < FI_PATH_AUTO || path > FI_PATH_GEMM) {
        set_error("fi_cache_set_path: invalid argument");
        return FI_ERR_INVALID_ARG;
    }
    if (path == FI_PATH_GEMM && c->cfg.dtype != FI_BF16) {
        set_error("fi_cache_set_path: the tensor-core path needs a bf16 cache");
        return FI_ERR_UNSUPPORTED;
    }
    c->cfg.path = path;
    return FI_OK;
}

int64_t fi_cache_size(const fi_cache_t *c) { return c ? c->enqueued : 0; }

int64_t fi_cache_lookup_view(const fi_cache_t *c) { return c ? c->size : 0; }

fi_status_t fi_cache_set_sm_limit(fi_cache_t *c, int32_t sms) {
    if (!c || sms < 0) {
        set_error("fi_cache_set_sm_limit: null cache or negative count");
        return FI_ERR_INVALID_ARG;
    }
    c->sm_limit = sms;
    c->sm_count = sms > 0 && sms < c->sm_total ? sms : c->sm_total;
    return FI_OK;
}

fi_status_t fi_cache_clear(fi_cache_t *c) {
    if (!c) {
        set_error("fi_cache_clear: null cache");
        return FI_ERR_INVALID_ARG;
    }
    c->size = 0;
    c->enqueued = 0;
    c->committed = 0;
    c->pend_n = 0;
    c->pend_head = 0;
    DeviceGuard guard(c->cfg.device);
    cudaMemsetAsync(c->cert_dev + 3, 0, sizeof(int32_t), nullptr);   // largest norm of the entries held: none now
    return FI_OK;
}

fi_status_t fi_kmeans_step(fi_cache_t *c, const void *points, int64_t ld_elems, const int32_t *point_labels, int64_t n,
                           int32_t *assign_out, void *new_centres, int32_t *counts, int32_t *majority_label,
                           float *fraction, void *cuda_stream) {
    if (!c || n < 0 || !new_centres || !counts || !majority_label || !fraction ||
        (n > 0 && (!points || !point_labels || !assign_out))) {
        set_error("fi_kmeans_step: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    refresh_view(c, static_cast<cudaStream_t>(cuda_stream));
    if (c->cfg.k != 1 || c->size <= 0) {
        set_error("fi_kmeans_step: the centres cache must have k = 1 and hold at least one centre");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (!c->km_dist) {
        fi_status_t st = dev_alloc(&c->km_dist, (size_t)c->cfg.max_batch, "allocating k-means scratch");
        if (st != FI_OK) return st;
    }
    // assignment: the nearest-centre index is the look-up's single neighbour
    fi_lookup_out_t out;
    out.label = c->slot_label;
    out.conf = c->slot_conf;
    out.hit = c->slot_hit;
    out.topk_dist = c->km_dist;
    const unsigned char *base = static_cast<const unsigned char *>(points);
    for (int64_t lo = 0; lo < n; lo += c->cfg.max_batch) {
        const int32_t b = (int32_t)((n - lo) < c->cfg.max_batch ? (n - lo) : c->cfg.max_batch);
        out.topk_idx = assign_out + lo;
        fi_status_t st = fi_cache_lookup_batch(c, base + (size_t)lo * ld_elems * c->elem_size, ld_elems, nullptr, b,
                                               nullptr, &out, cuda_stream);
        if (st != FI_OK) return st;
    }
    return launch_kmeans_update(c, points, ld_elems, point_labels, assign_out, n, new_centres, counts, majority_label,
                                fraction, stream);
}

fi_status_t fi_cache_lookup_batch(const fi_cache_t *cache, const void *queries, int64_t ld_elems, const int32_t *row_idx,
                                  int32_t batch_max, const int32_t *batch_count_dev, const fi_lookup_out_t *out,
                                  void *cuda_stream) {
    if (!cache || !out || batch_max < 0 || (batch_max > 0 && (!queries || !out->label || !out->conf || !out->hit))) {
        set_error("fi_cache_lookup_batch: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    if (batch_max > cache->cfg.max_batch) {
        set_error("fi_cache_lookup_batch: batch %d exceeds max_batch %d", batch_max, cache->cfg.max_batch);
        return FI_ERR_INVALID_ARG;
    }
    const int align_elems = 16 / (int)cache->elem_size;
    if (ld_elems < cache->cfg.dim || ld_elems % align_elems != 0 || (reinterpret_cast<uintptr_t>(queries) & 15) != 0) {
        set_error("fi_cache_lookup_batch: rows must start on 16-byte boundaries (ld %lld, dim %d)", (long long)ld_elems,
                  cache->cfg.dim);
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(cache->cfg.device);
    // the handle is const for the caller: the look-up does not change the cache's contents, only its scratch
    return lookup_impl(const_cast<fi_cache *>(cache), queries, ld_elems, row_idx, batch_max, batch_count_dev, *out,
                       static_cast<cudaStream_t>(cuda_stream));
}

fi_status_t fi_cascade_init(const fi_cascade_state_t *state, int32_t num_stages, int32_t device, void *cuda_stream) {
    if (!state || state->batch0 < 0 || num_stages < 0 ||
        (state->batch0 > 0 && (!state->final_label || !state->exit_stage || !state->final_conf))) {
        set_error("fi_cascade_init: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(device);
    return launch_cascade_init(*state, num_stages, static_cast<cudaStream_t>(cuda_stream));
}

fi_status_t fi_cascade_step(const fi_cache_t *cache, const void *stage_acts, int64_t ld_elems,
                            const fi_cascade_state_t *state, void *cuda_stream) {
    if (!cache || !state || state->batch0 < 0 || !state->miss_idx || !state->miss_count ||
        (state->batch0 > 0 && (!stage_acts || !state->final_label || !state->exit_stage || !state->final_conf))) {
        set_error("fi_cascade_step: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    if (state->batch0 > cache->cfg.max_batch) {
        set_error("fi_cascade_step: batch %d exceeds max_batch %d", state->batch0, cache->cfg.max_batch);
        return FI_ERR_INVALID_ARG;
    }
    if (state->miss_idx == state->active_idx) {
        set_error("fi_cascade_step: miss_idx must not alias active_idx");
        return FI_ERR_INVALID_ARG;
    }
    fi_cache *c = const_cast<fi_cache *>(cache);
    fi_lookup_out_t out;
    out.label = c->slot_label;
    out.conf = c->slot_conf;
    out.hit = c->slot_hit;
    out.topk_dist = nullptr;
    out.topk_idx = nullptr;
    fi_status_t st = fi_cache_lookup_batch(cache, stage_acts, ld_elems, state->active_idx, state->batch0,
                                           state->active_count, &out, cuda_stream);
    if (st != FI_OK) return st;
    DeviceGuard guard(cache->cfg.device);
    return launch_compact(c, *state, static_cast<cudaStream_t>(cuda_stream));
}

fi_status_t fi_cache_lookup_batch_host(const fi_cache_t *cache, const void *queries_host, int32_t batch,
                                       const fi_lookup_out_t *out_host, void *cuda_stream) {
    if (!cache || !out_host || batch < 0 ||
        (batch > 0 && (!queries_host || !out_host->label || !out_host->conf || !out_host->hit))) {
        set_error("fi_cache_lookup_batch_host: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    if (batch > cache->cfg.max_batch) {
        set_error("fi_cache_lookup_batch_host: batch %d exceeds max_batch %d", batch, cache->cfg.max_batch);
        return FI_ERR_INVALID_ARG;
    }
    if (batch == 0) return FI_OK;
    fi_cache *c = const_cast<fi_cache *>(cache);
    DeviceGuard guard(c->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int k = c->cfg.k;
    const size_t q_bytes = (size_t)batch * c->cfg.dim * c->elem_size;
    const size_t q_pad = (q_bytes + 255) & ~(size_t)255;
    const size_t out_bytes = (size_t)batch * (4 + 4 + 4 + 8 * (size_t)k);   // hit padded to 4 bytes per slot
    const size_t need = q_pad + out_bytes + 256;
    if (need > c->h2d_stage_bytes) {
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) return cuda_fail(e, "fi_cache_lookup_batch_host: synchronising");
        cudaFree(c->h2d_stage);
        c->h2d_stage = nullptr;
        c->h2d_stage_bytes = 0;
        e = cudaMalloc(&c->h2d_stage, need);
        if (e != cudaSuccess) return cuda_fail(e, "fi_cache_lookup_batch_host: allocating staging");
        c->h2d_stage_bytes = need;
    }
    unsigned char *base = static_cast<unsigned char *>(c->h2d_stage);
    fi_lookup_out_t dev;
    dev.label = reinterpret_cast<int32_t *>(base + q_pad);
    dev.conf = reinterpret_cast<float *>(base + q_pad + (size_t)batch * 4);
    dev.topk_dist = reinterpret_cast<float *>(base + q_pad + (size_t)batch * 8);
    dev.topk_idx = reinterpret_cast<int32_t *>(base + q_pad + (size_t)batch * 8 + (size_t)batch * k * 4);
    dev.hit = base + q_pad + (size_t)batch * 8 + (size_t)batch * k * 8;
    cudaError_t e = cudaMemcpyAsync(base, queries_host, q_bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_lookup_batch_host: copying queries");
    fi_status_t st = lookup_impl(c, base, c->cfg.dim, nullptr, batch, nullptr, dev, stream);
    if (st != FI_OK) return st;
    e = cudaMemcpyAsync(out_host->label, dev.label, (size_t)batch * 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host->conf, dev.conf, (size_t)batch * 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host->hit, dev.hit, (size_t)batch, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess && out_host->topk_dist)
        e = cudaMemcpyAsync(out_host->topk_dist, dev.topk_dist, (size_t)batch * k * 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess && out_host->topk_idx)
        e = cudaMemcpyAsync(out_host->topk_idx, dev.topk_idx, (size_t)batch * k * 4, cudaMemcpyDeviceToHost, stream);
    int32_t word = 0;
    if (e == cudaSuccess) e = fetch_status_words(&c, 1, &word, stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_lookup_batch_host: copying results");
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_lookup_batch_host: synchronising");
    return status_from_words(&c, 1, &word, "fi_cache_lookup_batch_host");
}

fi_status_t fi_cascade_run_host(fi_cache_t *const *caches, int32_t num_stages, const void *const *acts_host,
                                int32_t batch0, int32_t *final_label_host, int32_t *exit_stage_host,
                                float *final_conf_host, int32_t *stage_arrivals_host, void *cuda_stream) {
    if (!caches || !acts_host || num_stages < 1 || batch0 < 0 || !final_label_host || !exit_stage_host || !final_conf_host) {
        set_error("fi_cascade_run_host: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    for (int l = 0; l < num_stages; ++l) {
        if (!caches[l] || !acts_host[l] || caches[l]->cfg.device != caches[0]->cfg.device || batch0 > caches[l]->cfg.max_batch) {
            set_error("fi_cascade_run_host: stage %d: null cache or activations, other device, or batch above max_batch", l);
            return FI_ERR_INVALID_ARG;
        }
    }
    if (batch0 == 0) return FI_OK;
    fi_cache *c0 = caches[0];
    DeviceGuard guard(c0->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // device staging: activations of every stage, then the cascade state
    size_t act_off[kMaxHostStages];
    if (num_stages >= kMaxHostStages) {
        set_error("fi_cascade_run_host: at most %d stages", kMaxHostStages - 1);
        return FI_ERR_INVALID_ARG;
    }
    size_t total = 0;
    for (int l = 0; l < num_stages; ++l) {
        act_off[l] = total;
        total += ((size_t)batch0 * caches[l]->cfg.dim * caches[l]->elem_size + 255) & ~(size_t)255;
    }
    const size_t state_off = total;
    const size_t nb = (size_t)batch0;
    total += (5 * nb + (size_t)num_stages + 8) * 4 + 256;
    if (total > c0->h2d_stage_bytes) {
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) return cuda_fail(e, "fi_cascade_run_host: synchronising");
        cudaFree(c0->h2d_stage);
        c0->h2d_stage = nullptr;
        c0->h2d_stage_bytes = 0;
        e = cudaMalloc(&c0->h2d_stage, total);
        if (e != cudaSuccess) return cuda_fail(e, "fi_cascade_run_host: allocating staging");
        c0->h2d_stage_bytes = total;
    }
    if (!c0->copy_stream) {
        cudaError_t e = cudaStreamCreateWithFlags(&c0->copy_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(e, "fi_cascade_run_host: creating the upload stream");
    }
    if (!c0->copy_ev) {
        c0->copy_ev = new (std::nothrow) cudaEvent_t[kMaxHostStages];
        if (!c0->copy_ev) {
            set_error("fi_cascade_run_host: out of host memory");
            return FI_ERR_OOM;
        }
        for (int i = 0; i < kMaxHostStages; ++i) {
            cudaError_t e = cudaEventCreateWithFlags(&c0->copy_ev[i], cudaEventDisableTiming);
            if (e != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(c0->copy_ev[j]);
                delete[] c0->copy_ev;
                c0->copy_ev = nullptr;
                return cuda_fail(e, "fi_cascade_run_host: creating events");
            }
        }
    }
    unsigned char *base = static_cast<unsigned char *>(c0->h2d_stage);
    int32_t *ibase = reinterpret_cast<int32_t *>(base + state_off);
    int32_t *idx[2] = {ibase, ibase + nb};
    int32_t *final_label = ibase + 2 * nb;
    int32_t *exit_stage = ibase + 3 * nb;
    float *final_conf = reinterpret_cast<float *>(ibase + 4 * nb);
    int32_t *counts = ibase + 5 * nb;   // counts[l] = arrivals at stage l; counts[0] unused (= batch0)

    // Uploads go to their own stream in stage order, so stage l+1 arrives while stage l is looked up.  The
    // staging area is free: the previous call synchronised before returning.  The upload stream first waits
    // for whatever the caller already queued on the work stream (it may still be using the staging area).
    cudaEvent_t start_ev = c0->copy_ev[kMaxHostStages - 1];
    cudaError_t e = cudaEventRecord(start_ev, stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c0->copy_stream, start_ev, 0);
    for (int l = 0; l < num_stages && e == cudaSuccess; ++l) {
        e = cudaMemcpyAsync(base + act_off[l], acts_host[l], (size_t)batch0 * caches[l]->cfg.dim * caches[l]->elem_size,
                            cudaMemcpyHostToDevice, c0->copy_stream);
        if (e == cudaSuccess) e = cudaEventRecord(c0->copy_ev[l], c0->copy_stream);
    }
    if (e != cudaSuccess) {
        cudaStreamSynchronize(c0->copy_stream);
        return cuda_fail(e, "fi_cascade_run_host: copying activations");
    }

    fi_cascade_state_t st;
    memset(&st, 0, sizeof st);
    st.batch0 = batch0;
    st.final_label = final_label;
    st.exit_stage = exit_stage;
    st.final_conf = final_conf;
    fi_status_t rc = fi_cascade_init(&st, num_stages, c0->cfg.device, cuda_stream);
    if (rc != FI_OK) {
        cudaStreamSynchronize(c0->copy_stream);
        return rc;
    }
    for (int l = 0; l < num_stages; ++l) {
        st.stage = l;
        st.active_idx = l == 0 ? nullptr : idx[(l - 1) & 1];
        st.active_count = l == 0 ? nullptr : counts + l;
        st.miss_idx = idx[l & 1];
        st.miss_count = counts + l + 1;
        e = cudaStreamWaitEvent(stream, c0->copy_ev[l], 0);
        if (e != cudaSuccess) {
            cudaStreamSynchronize(c0->copy_stream);
            return cuda_fail(e, "fi_cascade_run_host: waiting for an upload");
        }
        rc = fi_cascade_step(caches[l], base + act_off[l], caches[l]->cfg.dim, &st, cuda_stream);
        if (rc != FI_OK) {
            cudaStreamSynchronize(c0->copy_stream);
            return rc;
        }
    }
    e = cudaMemcpyAsync(final_label_host, final_label, nb * 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(exit_stage_host, exit_stage, nb * 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(final_conf_host, final_conf, nb * 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess && stage_arrivals_host && num_stages > 0)
        e = cudaMemcpyAsync(stage_arrivals_host + 1, counts + 1, (size_t)num_stages * 4, cudaMemcpyDeviceToHost, stream);
    int32_t words[kMaxHostStages];
    if (e == cudaSuccess) e = fetch_status_words(caches, num_stages, words, stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cascade_run_host: copying results");
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cascade_run_host: synchronising");
    if (stage_arrivals_host) stage_arrivals_host[0] = batch0;
    return status_from_words(caches, num_stages, words, "fi_cascade_run_host");
}

fi_status_t fi_cache_compute_threshold(fi_cache_t *c, const void *val_acts, int64_t ld_elems, const int32_t *model_labels,
                                       int64_t n, float *tau_out, int64_t *wrong_out, void *cuda_stream) {
    if (!c || n < 0 || (n > 0 && (!val_acts || !model_labels))) {
        set_error("fi_cache_compute_threshold: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // two accumulator words (maximum as a bit pattern, count of wrong look-ups), allocated on first use
    if (!c->calib_acc) {
        fi_status_t st = dev_alloc(&c->calib_acc, 2, "allocating the calibration accumulator");
        if (st != FI_OK) return st;
    }
    cudaError_t e = cudaMemsetAsync(c->calib_acc, 0, 2 * sizeof(int32_t), stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_compute_threshold: clearing the accumulator");
    fi_lookup_out_t out;
    out.label = c->slot_label;
    out.conf = c->slot_conf;
    out.hit = c->slot_hit;
    out.topk_dist = nullptr;
    out.topk_idx = nullptr;
    const unsigned char *base = static_cast<const unsigned char *>(val_acts);
    for (int64_t lo = 0; lo < n; lo += c->cfg.max_batch) {
        const int32_t b = (int32_t)((n - lo) < c->cfg.max_batch ? (n - lo) : c->cfg.max_batch);
        fi_status_t st = fi_cache_lookup_batch(c, base + (size_t)lo * ld_elems * c->elem_size, ld_elems, nullptr, b,
                                               nullptr, &out, cuda_stream);
        if (st != FI_OK) return st;
        st = launch_wrong_max(c->slot_label, c->slot_conf, model_labels + lo, b, c->calib_acc, stream);
        if (st != FI_OK) return st;
    }
    int32_t host[2] = {0, 0};
    int32_t word = 0;
    e = cudaMemcpyAsync(host, c->calib_acc, sizeof host, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = fetch_status_words(&c, 1, &word, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_compute_threshold: reading the result");
    {
        const fi_status_t ws = status_from_words(&c, 1, &word, "fi_cache_compute_threshold");
        if (ws != FI_OK) return ws;   // the cache's threshold is left as it was
    }
    float tau;
    memcpy(&tau, &host[0], sizeof tau);
    c->cfg.threshold = tau;
    if (tau_out) *tau_out = tau;
    if (wrong_out) *wrong_out = host[1];
    return FI_OK;
}

fi_status_t fi_cache_neighbor_tuples(const fi_cache_t *c, const int32_t *topk_idx, int64_t n, int32_t index_offset,
                                     int32_t *global_idx, int32_t *label, float *weight, void *cuda_stream) {
    if (!c || n < 0 || (n > 0 && (!topk_idx || !global_idx || !label || !weight))) {
        set_error("fi_cache_neighbor_tuples: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    return launch_neighbor_tuples(c, topk_idx, n, index_offset, global_idx, label, weight,
                                  static_cast<cudaStream_t>(cuda_stream));
}

fi_status_t fi_merge_shard_lookups(int32_t shards, int32_t batch, int32_t k, const float *dist, const int32_t *global_idx,
                                   const int32_t *label, const float *weight, int32_t metric, int32_t rule,
                                   float threshold, const fi_lookup_out_t *out, void *cuda_stream) {
    if (shards < 1 || batch < 0 || k < 1 || k > kMaxK || !out ||
        (batch > 0 && (!dist || !global_idx || !label || !weight || !out->label || !out->conf || !out->hit)) ||
        (rule != FI_HIT_CONF_GT && rule != FI_HIT_DIST_LE) || (metric != FI_METRIC_SQL2 && metric != FI_METRIC_L2)) {
        set_error("fi_merge_shard_lookups: invalid argument");
        return FI_ERR_INVALID_ARG;
    }
    return launch_merge_vote(shards, batch, k, dist, global_idx, label, weight, metric, rule, threshold, *out,
                             static_cast<cudaStream_t>(cuda_stream));
}

fi_status_t fi_projection_destroy(fi_projection_t *p) {
    if (!p) return FI_OK;
    {
        DeviceGuard guard(p->device);
        cudaDeviceSynchronize();
        cudaFree(p->zero_labels);
        cudaFree(p->zero_bias);
        cudaFree(p->y);
        cudaGetLastError();
    }
    fi_cache_destroy(p->w);
    delete p;
    return FI_OK;
}

fi_status_t fi_projection_create(int32_t in_dim, int32_t out_dim, int32_t device, int32_t max_batch, fi_projection_t **out) {
    if (out) *out = nullptr;
    if (!out || in_dim < 8 || in_dim % 8 != 0 || out_dim < 16 || out_dim % 16 != 0 || max_batch < 1) {
        set_error("fi_projection_create: need in_dim a multiple of 8, out_dim a multiple of 16, max_batch >= 1");
        return FI_ERR_INVALID_ARG;
    }
    fi_projection *p = new (std::nothrow) fi_projection();
    if (!p) {
        set_error("fi_projection_create: out of host memory");
        return FI_ERR_OOM;
    }
    memset(p, 0, sizeof *p);
    p->in_dim = in_dim;
    p->out_dim = out_dim;
    p->max_batch = max_batch;
    p->device = device;
    fi_cache_config_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.dim = in_dim;
    cfg.dtype = FI_BF16;
    cfg.capacity = out_dim;
    cfg.num_classes = 1;
    cfg.k = 1;
    cfg.rule = FI_HIT_CONF_GT;
    cfg.metric = FI_METRIC_SQL2;
    cfg.device = device;
    cfg.max_batch = max_batch;
    cfg.path = FI_PATH_GEMM;
    fi_status_t st = fi_cache_create(&cfg, &p->w);
    if (st != FI_OK) {
        delete p;
        return st;
    }
    DeviceGuard guard(device);
    const size_t units = product_dump_units(max_batch, out_dim, p->w->sm_count);
    if (units > p->w->tail_dump_units) {
        cudaFree(p->w->tail_dump);
        p->w->tail_dump = nullptr;
        p->w->tail_dump_units = 0;
        st = dev_alloc(&p->w->tail_dump, units * 256 * 256, "allocating the projection's partial sums");
        if (st == FI_OK) p->w->tail_dump_units = units;
    }
    if (st == FI_OK) st = dev_alloc(&p->zero_labels, (size_t)out_dim, "allocating the projection's labels");
    if (st == FI_OK) st = dev_alloc(&p->zero_bias, (size_t)out_dim, "allocating the projection's zero bias");
    unsigned char *y = nullptr;
    if (st == FI_OK) st = dev_alloc(&y, (size_t)max_batch * out_dim * 2, "allocating the projection's output");
    p->y = y;
    if (st == FI_OK) {
        cudaError_t e = cudaMemset(p->zero_labels, 0, (size_t)out_dim * sizeof(int32_t));
        if (e == cudaSuccess) e = cudaMemset(p->zero_bias, 0, (size_t)out_dim * sizeof(float));
        if (e != cudaSuccess) st = cuda_fail(e, "fi_projection_create: clearing buffers");
    }
    if (st != FI_OK) {
        fi_projection_destroy(p);
        return st;
    }
    *out = p;
    return FI_OK;
}

fi_status_t fi_projection_set_weights(fi_projection_t *p, const void *weights, const float *bias, void *cuda_stream) {
    if (!p || !weights) {
        set_error("fi_projection_set_weights: null argument");
        return FI_ERR_INVALID_ARG;
    }
    fi_cache_clear(p->w);
    return fi_cache_insert(p->w, weights, p->zero_labels, bias ? bias : p->zero_bias, p->out_dim, cuda_stream);
}

fi_status_t fi_projection_poll_status(fi_projection_t *p) {
    if (!p) {
        set_error("fi_projection_poll_status: null projection");
        return FI_ERR_INVALID_ARG;
    }
    return fi_cache_poll_status(p->w);
}

fi_status_t fi_projection_apply(const fi_projection_t *p, const void *x, int64_t ld_elems, const int32_t *row_idx,
                                int32_t batch_max, const int32_t *batch_count_dev, void *y, int64_t ld_y,
                                void *cuda_stream) {
    if (!p || batch_max < 0 || (batch_max > 0 && (!x || !y))) {
        set_error("fi_projection_apply: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    refresh_view(p->w, static_cast<cudaStream_t>(cuda_stream));
    if (batch_max > p->max_batch || p->w->size != p->out_dim) {
        set_error("fi_projection_apply: batch %d exceeds max_batch %d, or the weights were never set", batch_max, p->max_batch);
        return FI_ERR_INVALID_ARG;
    }
    if (ld_elems < p->in_dim || ld_elems % 8 != 0 || (reinterpret_cast<uintptr_t>(x) & 15) != 0 || ld_y < p->out_dim) {
        set_error("fi_projection_apply: rows must start on 16-byte boundaries (ld %lld, in_dim %d; ld_y %lld, out_dim %d)",
                  (long long)ld_elems, p->in_dim, (long long)ld_y, p->out_dim);
        return FI_ERR_INVALID_ARG;
    }
    if (batch_max == 0) return FI_OK;
    DeviceGuard guard(p->device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    fi_cache *w = p->w;
    const void *src = x;
    int64_t ld = ld_elems;
    if (row_idx) {
        fi_status_t st = launch_gather_rows(x, ld_elems, row_idx, batch_max, batch_count_dev, w->q_compact, p->in_dim, 2, stream);
        if (st != FI_OK) return st;
        src = w->q_compact;
        ld = p->in_dim;
    }
    prof_mark(w, 0, stream);
    fi_status_t st = launch_gemm_project(w, src, ld, batch_max, batch_count_dev, y, ld_y, stream);
    if (st == FI_OK) prof_mark(w, 1, stream);
    return st;
}

fi_status_t fi_projection_set_profiling(fi_projection_t *p, int32_t enable) {
    if (!p) {
        set_error("fi_projection_set_profiling: null projection");
        return FI_ERR_INVALID_ARG;
    }
    return fi_cache_set_profiling(p->w, enable);
}

fi_status_t fi_projection_read_profile(fi_projection_t *p, float *total_ms, int32_t *launches) {
    if (!p) {
        set_error("fi_projection_read_profile: null projection");
        return FI_ERR_INVALID_ARG;
    }
    return fi_cache_read_profile(p->w, total_ms, launches);
}

fi_status_t fi_cascade_step_projected(const fi_cache_t *cache, const fi_projection_t *proj, const void *stage_acts,
                                      int64_t ld_elems, const fi_cascade_state_t *state, void *cuda_stream) {
    if (!cache || !proj || !state || state->batch0 < 0 || !state->miss_idx || !state->miss_count ||
        (state->batch0 > 0 && (!stage_acts || !state->final_label || !state->exit_stage || !state->final_conf))) {
        set_error("fi_cascade_step_projected: null or negative argument");
        return FI_ERR_INVALID_ARG;
    }
    if (cache->cfg.dtype != FI_BF16 || cache->cfg.dim != proj->out_dim || cache->cfg.device != proj->device) {
        set_error("fi_cascade_step_projected: the cache must be bf16, of the projection's output size and on its device");
        return FI_ERR_INVALID_ARG;
    }
    if (state->batch0 > cache->cfg.max_batch || state->batch0 > proj->max_batch) {
        set_error("fi_cascade_step_projected: batch %d exceeds max_batch", state->batch0);
        return FI_ERR_INVALID_ARG;
    }
    if (state->miss_idx == state->active_idx) {
        set_error("fi_cascade_step_projected: miss_idx must not alias active_idx");
        return FI_ERR_INVALID_ARG;
    }
    // slot i of the projected batch is the i-th active request: the look-up then needs no gather list
    fi_status_t st = fi_projection_apply(proj, stage_acts, ld_elems, state->active_idx, state->batch0, state->active_count,
                                         proj->y, proj->out_dim, cuda_stream);
    if (st != FI_OK) return st;
    fi_cache *c = const_cast<fi_cache *>(cache);
    fi_lookup_out_t out;
    out.label = c->slot_label;
    out.conf = c->slot_conf;
    out.hit = c->slot_hit;
    out.topk_dist = nullptr;
    out.topk_idx = nullptr;
    st = fi_cache_lookup_batch(cache, proj->y, proj->out_dim, nullptr, state->batch0, state->active_count, &out, cuda_stream);
    if (st != FI_OK) return st;
    DeviceGuard guard(cache->cfg.device);
    return launch_compact(c, *state, static_cast<cudaStream_t>(cuda_stream));
}

fi_status_t fi_cache_selftest_wait(fi_cache_t *c, int64_t limit_cycles, void *cuda_stream) {
    if (!c || limit_cycles < 1 || limit_cycles > 2000000000ll) {
        set_error("fi_cache_selftest_wait: null cache or limit outside 1..2e9 cycles");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    return launch_wait_selftest(c, (long long)limit_cycles, static_cast<cudaStream_t>(cuda_stream));
}

fi_status_t fi_cache_poll_status(fi_cache_t *c) {
    if (!c) {
        set_error("fi_cache_poll_status: null cache");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_poll_status: synchronising");
    int32_t word = 0;
    e = cudaMemcpy(&word, c->status_dev, sizeof word, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_poll_status: reading the status word");
    if (word != 0) {
        cudaMemset(c->status_dev, 0, sizeof word);
        set_error("a kernel gave up on a bounded wait (code %d, site %d)", word & 0xFF, word >> 8);
        return FI_ERR_TIMEOUT;
    }
    return FI_OK;
}

fi_status_t fi_cache_set_profiling(fi_cache_t *c, int32_t enable) {
    if (!c) {
        set_error("fi_cache_set_profiling: null cache");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    if (enable && !c->prof_ev) {
        c->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfSlots];
        if (!c->prof_ev) {
            set_error("fi_cache_set_profiling: out of host memory");
            return FI_ERR_OOM;
        }
        for (int i = 0; i < 2 * kProfSlots; ++i) {
            cudaError_t e = cudaEventCreate(&c->prof_ev[i]);
            if (e != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(c->prof_ev[j]);
                delete[] c->prof_ev;
                c->prof_ev = nullptr;
                return cuda_fail(e, "fi_cache_set_profiling: creating events");
            }
        }
    }
    c->prof_on = enable != 0;
    c->prof_n = 0;
    return FI_OK;
}

fi_status_t fi_cache_read_profile(fi_cache_t *c, float *total_ms, int32_t *launches) {
    if (!c || !total_ms || !launches) {
        set_error("fi_cache_read_profile: null argument");
        return FI_ERR_INVALID_ARG;
    }
    *total_ms = 0.f;
    *launches = 0;
    if (!c->prof_ev) return FI_OK;
    DeviceGuard guard(c->cfg.device);
    const int n = c->prof_n < kProfSlots ? c->prof_n : kProfSlots;
    for (int i = 0; i < n; ++i) {
        cudaError_t e = cudaEventSynchronize(c->prof_ev[2 * i + 1]);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]);
        if (e != cudaSuccess) return cuda_fail(e, "fi_cache_read_profile: reading events");
        *total_ms += ms;
    }
    *launches = n;
    c->prof_n = 0;
    return FI_OK;
}

fi_status_t fi_cache_set_repair(fi_cache_t *c, int32_t enable) {
    if (!c) {
        set_error("fi_cache_set_repair: null cache");
        return FI_ERR_INVALID_ARG;
    }
    c->repair_on = enable != 0;
    return FI_OK;
}

fi_status_t fi_cache_read_certificate(fi_cache_t *c, int64_t *uncertified, int64_t *unrepaired, float *max_score_error) {
    if (!c) {
        set_error("fi_cache_read_certificate: null cache");
        return FI_ERR_INVALID_ARG;
    }
    DeviceGuard guard(c->cfg.device);
    cudaError_t e = cudaDeviceSynchronize();
    int32_t w[kCertWords] = {0, 0, 0, 0, 0};
    if (e == cudaSuccess) e = cudaMemcpy(w, c->cert_dev, sizeof w, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemset(c->cert_dev, 0, 2 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(c->cert_dev + 4, 0, sizeof(int32_t));
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_read_certificate");
    if (uncertified) *uncertified = w[0];
    if (unrepaired) *unrepaired = w[4];
    if (max_score_error) memcpy(max_score_error, &w[1], sizeof(float));
    return FI_OK;
}

fi_status_t fi_cache_read_slot_certificates(fi_cache_t *c, uint8_t *flags_host, int32_t n) {
    if (!c || n < 0 || n > c->cfg.max_batch || (n > 0 && !flags_host)) {
        set_error("fi_cache_read_slot_certificates: null argument or more slots than max_batch");
        return FI_ERR_INVALID_ARG;
    }
    if (n == 0) return FI_OK;
    DeviceGuard guard(c->cfg.device);
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(flags_host, c->slot_cert, (size_t)n, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "fi_cache_read_slot_certificates");
    return FI_OK;
}

fi_status_t fi_gemm_plan_describe(int32_t count, int64_t n_entries, int32_t num_ctas, int32_t k, int32_t dim,
                                  int32_t max_batch, int32_t cta, int32_t *plan_out, int32_t *items_out,
                                  int32_t *n_items) {
    if (!plan_out || count <= 0 || n_entries <= 0 || num_ctas <= 0 || k <= 0 || dim <= 0 || max_batch < count) {
        set_error("fi_gemm_plan_describe: null or non-positive argument");
        return FI_ERR_INVALID_ARG;
    }
    const int tile_m = gemm_tile_m(max_batch, dim);
    const int num_kb = (dim + 63) / 64;
    const GemmPlan p = make_gemm_plan(count, n_entries, num_ctas, k, tile_m, num_kb);
    const int32_t v[17] = {p.count, p.m_tiles, p.mg, p.groups, p.parts, p.range16, p.list_len, p.tile_m, p.lists, p.mode,
                           p.n_tiles, p.tail_tiles, p.tail_slices, p.pieces, p.half, p.span_full, p.span_half};
    for (int i = 0; i < 17; ++i) plan_out[i] = v[i];
    if (n_items) *n_items = 0;
    int m, j, cm;
    if (p.mode == 3 && cta >= 0 && items_out && n_items && span_owner(p, cta, m, j, cm)) {
        const int s0 = span_begin(p, num_kb, j, cm), s1 = span_begin(p, num_kb, j + 1, cm);
        const int n = s1 > s0 ? (s1 - 1) / num_kb - s0 / num_kb + 1 : 0;
        for (int idx = 0; idx < n && idx < kMaxSpanItems; ++idx) {
            const int tile = s0 / num_kb + idx;
            int32_t *it = items_out + 6 * idx;
            it[0] = m;
            it[1] = tile;
            it[2] = idx == 0 ? s0 - tile * num_kb : 0;
            it[3] = s1 - tile * num_kb < num_kb ? s1 - tile * num_kb : num_kb;
            it[4] = p.half && m == p.m_tiles - 1 ? 1 : 2;
            it[5] = cta * kMaxSpanItems + idx;
        }
        *n_items = n;
    }
    return FI_OK;
}

int64_t fi_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

const char *fi_last_error(void) { return g_err; }

const char *fi_status_string(fi_status_t s) {
    switch (s) {
        case FI_OK: return "FI_OK";
        case FI_ERR_INVALID_ARG: return "FI_ERR_INVALID_ARG";
        case FI_ERR_CAPACITY: return "FI_ERR_CAPACITY";
        case FI_ERR_OOM: return "FI_ERR_OOM";
        case FI_ERR_CUDA: return "FI_ERR_CUDA";
        case FI_ERR_UNSUPPORTED: return "FI_ERR_UNSUPPORTED";
        case FI_ERR_TIMEOUT: return "FI_ERR_TIMEOUT";
    }
    return "FI_?";
}

}  // extern "C"
