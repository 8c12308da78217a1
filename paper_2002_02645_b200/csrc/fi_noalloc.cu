// Look-up entry point that allocates nothing.
//
// Some callers may not allocate device memory at the moment they need a look-up: a serving loop that has
// handed all of the GPU's memory to its own pool, code running between the capture and the replay of a CUDA
// graph, or a latency-critical path in which cudaMalloc (which may synchronise the device) is not acceptable.
// For them the streaming look-up is offered with its candidate-list scratch in a fixed array that is part of
// the library image: every GPU that loads the library holds these 4 MiB until the process exits.
#include <cstring>
#include <mutex>

#include "fi_internal.cuh"

namespace fi {
namespace {

constexpr int kNoAllocMaxBatch = 256;
constexpr size_t kNoAllocEntries = (size_t)kNoAllocMaxBatch * kMaxK * 64;   // 524,288 (score, index) pairs
constexpr size_t kNoAllocBytes = kNoAllocEntries * 8;                       // 4 MiB

// scratch of the streaming look-up: candidate scores, then candidate indices
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices];   // device address of the array on each device, filled on first use
int g_sm_count[kMaxDevices];

// Once per device, with that device current: the array's name is only a host-side handle, so ask the runtime
// for the address the kernels must be given.
fi_status_t scratch_for_device(int device, void **addr, int *sm_count) {
    if (device < 0 || device >= kMaxDevices) {
        set_error("fi_lookup_noalloc: device ordinal %d out of range", device);
        return FI_ERR_INVALID_ARG;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            set_error("fi_lookup_noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            cudaGetLastError();
            return FI_ERR_CUDA;
        }
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess || sms <= 0) {
            set_error("fi_lookup_noalloc: cannot read the SM count: %s", cudaGetErrorString(e));
            cudaGetLastError();
            return FI_ERR_CUDA;
        }
        g_sm_count[device] = sms;
        g_scratch_addr[device] = p;
    }
    *addr = g_scratch_addr[device];
    *sm_count = g_sm_count[device];
    return FI_OK;
}

}  // namespace
}  // namespace fi

using namespace fi;

extern "C" fi_status_t fi_lookup_noalloc(const void *cache_vecs, const int32_t *labels, const float *weights,
                                         int64_t n_entries, int32_t dim, int32_t dtype, int32_t k, int32_t rule,
                                         int32_t metric, float threshold, const void *queries, int64_t ld_elems,
                                         int32_t batch, const fi_lookup_out_t *out, void *cuda_stream) {
    if (!out || batch < 0 || n_entries < 0 || (batch > 0 && (!queries || !out->label || !out->conf || !out->hit)) ||
        (n_entries > 0 && (!cache_vecs || !labels || !weights))) {
        set_error("fi_lookup_noalloc: null or negative argument (weights are required here)");
        return FI_ERR_INVALID_ARG;
    }
    const bool bf16 = dtype == FI_BF16;
    if ((dtype != FI_F32 && !bf16) || dim <= 0 || dim % (bf16 ? 8 : 4) != 0 || k < 1 || k > kMaxK ||
        (rule != FI_HIT_CONF_GT && rule != FI_HIT_DIST_LE) || (metric != FI_METRIC_SQL2 && metric != FI_METRIC_L2)) {
        set_error("fi_lookup_noalloc: invalid dtype, dim, k, rule or metric");
        return FI_ERR_INVALID_ARG;
    }
    if (n_entries > kMaxEntries) {
        set_error("fi_lookup_noalloc: %lld entries exceed the int32 index range (at most %lld)", (long long)n_entries,
                  (long long)kMaxEntries);
        return FI_ERR_INVALID_ARG;
    }
    if (batch > kNoAllocMaxBatch) {
        set_error("fi_lookup_noalloc: batch %d exceeds the fixed scratch (at most %d requests per call)", batch,
                  kNoAllocMaxBatch);
        return FI_ERR_CAPACITY;
    }
    const int align_elems = bf16 ? 8 : 4;
    if (batch > 0 && (ld_elems < dim || ld_elems % align_elems != 0 || (reinterpret_cast<uintptr_t>(queries) & 15) != 0 ||
                      (n_entries > 0 && (reinterpret_cast<uintptr_t>(cache_vecs) & 15) != 0))) {
        set_error("fi_lookup_noalloc: rows must start on 16-byte boundaries");
        return FI_ERR_INVALID_ARG;
    }
    if (batch == 0) return FI_OK;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) {
        cudaGetLastError();
        set_error("fi_lookup_noalloc: no current CUDA device");
        return FI_ERR_CUDA;
    }
    void *scratch = nullptr;
    int sm_count = 0;
    fi_status_t st = scratch_for_device(device, &scratch, &sm_count);
    if (st != FI_OK) return st;

    // a cache view over the caller's arrays; nothing here is owned or freed
    fi_cache view;
    memset(&view, 0, sizeof view);
    view.cfg.dim = dim;
    view.cfg.dtype = dtype;
    view.cfg.capacity = n_entries;
    view.cfg.num_classes = 1;
    view.cfg.k = k;
    view.cfg.rule = rule;
    view.cfg.metric = metric;
    view.cfg.threshold = threshold;
    view.cfg.device = device;
    view.cfg.max_batch = kNoAllocMaxBatch;
    view.cfg.path = FI_PATH_STREAM;
    view.size = n_entries;
    view.sm_count = sm_count;
    view.elem_size = bf16 ? 2 : 4;
    view.rows = const_cast<void *>(cache_vecs);
    view.labels = const_cast<int32_t *>(labels);
    view.weights = const_cast<float *>(weights);
    view.part_score = static_cast<float *>(scratch);
    view.part_idx = reinterpret_cast<int32_t *>(static_cast<unsigned char *>(scratch) + kNoAllocEntries * 4);
    view.part_entries = kNoAllocEntries;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int parts = 1;
    st = launch_stream_lookup(&view, queries, ld_elems, nullptr, batch, nullptr, &parts, stream);
    if (st != FI_OK) return st;
    FinalizeArgs fa;
    fa.queries = queries;
    fa.ld_elems = ld_elems;
    fa.row_idx = nullptr;
    fa.batch_max = batch;
    fa.count_dev = nullptr;
    fa.parts = parts;
    fa.list_len = k;
    fa.refine = 0;
    fa.out = *out;
    return launch_finalize(&view, fa, stream);
}
