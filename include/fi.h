/*
 * fi.h — C ABI of the per-layer approximate cache of Freeze Inference (arXiv 2002.02645).
 *
 * One `fi_cache_t` is the cache of one DNN layer (Pseudocode 1: CACHE[layer], THRESHOLDS[layer]).
 * The online operations are the cache look-up API of Sec. 3 on a batch of requests and the
 * per-layer cascade step of Pseudocode 1 (FreezeInference) with the batch reconstruction that
 * Sec. 5 asks for.  All device work runs in CUDA kernels built for sm_100a; there is no CPU path.
 *
 * Conventions
 *   - Unless a parameter says "host", every data pointer is a DEVICE pointer on the cache's device,
 *     allocated and owned by the caller.  The library owns only what `fi_cache_create` allocates
 *     (rows, labels, weights, squared norms, scratch) and frees it in `fi_cache_destroy`.
 *   - `cuda_stream` is a `cudaStream_t` passed as `void*` (NULL = the legacy default stream).  Calls
 *     enqueue work on it and return without synchronising, except where stated.
 *   - Calls that use the same cache share its scratch memory and must be ordered on one stream
 *     (or otherwise serialised); different caches are independent.
 *   - Every failure is a returned status; nothing aborts, throws, or traps on the device.  A wait
 *     inside a kernel that runs out (bounded) sets a device status word, which `fi_cache_poll_status`
 *     reads.  `fi_last_error` gives a text for the last failure on the calling thread.
 *   - Vectors are row-major with contiguous elements: float32 (FI_F32) or bfloat16 (FI_BF16).
 *     Queries have the dtype of the cache.  bfloat16 rows must start on 16-byte boundaries
 *     (base pointer 16-byte aligned, leading dimension a multiple of 8 elements), and
 *     dim must be a multiple of 8 (bf16) or 4 (f32).
 */
#ifndef FI_H_
#define FI_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fi_cache fi_cache_t; /* opaque; one per layer */

typedef enum {
    FI_OK = 0,
    FI_ERR_INVALID_ARG = 1,
    FI_ERR_CAPACITY = 2,
    FI_ERR_OOM = 3,
    FI_ERR_CUDA = 4,
    FI_ERR_UNSUPPORTED = 5,
    FI_ERR_TIMEOUT = 6
} fi_status_t;

typedef enum { FI_F32 = 0, FI_BF16 = 1 } fi_dtype_t;

/* Hit rule.  FI_HIT_CONF_GT is the paper's: hit iff confidence > threshold, strict (Pseudocode 1,
 * FreezeInference; Sec. 2.1).  FI_HIT_DIST_LE: hit iff the smallest distance among the
 * neighbours that carry the winning label is <= threshold (for k = 1: nearest-neighbour distance). */
typedef enum { FI_HIT_CONF_GT = 0, FI_HIT_DIST_LE = 1 } fi_hit_rule_t;

/* The d_j of the confidence sum (Sec. 3): squared L2 distance, or its square root. */
typedef enum { FI_METRIC_SQL2 = 0, FI_METRIC_L2 = 1 } fi_metric_t;

/* Which kernels serve a look-up.  AUTO: the streaming kernel for single requests and for float32 caches,
 * the tensor-core distance GEMM otherwise (from 2 requests on the streaming kernel is bound by its ALU work).  The other two force a path (bf16 only for GEMM). */
typedef enum { FI_PATH_AUTO = 0, FI_PATH_STREAM = 1, FI_PATH_GEMM = 2 } fi_path_t;

typedef struct {
    int32_t dim;         /* vector length d */
    int32_t dtype;       /* fi_dtype_t */
    int64_t capacity;    /* maximum number of entries */
    int32_t num_classes; /* labels must lie in [0, num_classes) */
    int32_t k;           /* neighbours per look-up, 1..32 */
    int32_t rule;        /* fi_hit_rule_t */
    int32_t metric;      /* fi_metric_t */
    float threshold;     /* THRESHOLDS[layer] */
    int32_t device;      /* CUDA device ordinal */
    int32_t max_batch;   /* largest batch a look-up on this cache may carry (sizes the scratch) */
    int32_t path;        /* fi_path_t */
} fi_cache_config_t;

/* Results of a look-up, one entry per batch slot i (the i-th request of the batch). */
typedef struct {
    int32_t *label;      /* [batch] predicted label, -1 for an empty cache */
    float *conf;         /* [batch] confidence C of that label (+inf when a neighbour is at distance 0) */
    uint8_t *hit;        /* [batch] 1 = frozen here */
    float *topk_dist;    /* [batch*k] nullable; squared L2 distances of the k neighbours, ascending, +inf padded */
    int32_t *topk_idx;   /* [batch*k] nullable; their cache indices, -1 padded */
} fi_lookup_out_t;

/* State of a batch walking through the layers.  Request ids are 0..batch0-1. */
typedef struct {
    const int32_t *active_idx;   /* in : ids alive at this stage, ascending; NULL = all of 0..batch0-1 */
    const int32_t *active_count; /* in : how many; NULL = batch0 */
    int32_t *miss_idx;           /* out: ids alive at the next stage, ascending; [batch0] */
    int32_t *miss_count;         /* out: how many; [1] */
    int32_t *final_label;        /* [batch0] written for the requests frozen at this stage */
    int32_t *exit_stage;         /* [batch0] written with `stage` for them */
    float *final_conf;           /* [batch0] written with their confidence */
    int32_t stage;               /* index of this stage */
    int32_t batch0;              /* size of the original batch */
} fi_cascade_state_t;

/*
 * Create the (empty) cache of one layer: CACHE[layer] = {} and THRESHOLDS[layer] of Pseudocode 1.
 * Allocates capacity*dim elements plus labels, weights, norms and look-up scratch on cfg->device (the scratch:
 * candidate lists for max_batch requests, and for bf16 rows of 4,096 values and more under batches above 128 also
 * three 256 KiB slots of partial sums per SM, about 116 MB).
 * Synchronous.  Errors: INVALID_ARG (null, dim/k/capacity/max_batch out of range, dim not a multiple
 * of 8 (bf16) or 4 (f32)), OOM, CUDA.  On error *out is NULL.
 */
fi_status_t fi_cache_create(const fi_cache_config_t *cfg, fi_cache_t **out);

/* Free everything the cache owns.  Synchronises the device.  NULL is accepted. */
fi_status_t fi_cache_destroy(fi_cache_t *cache);

/*
 * Append n entries <vector, label[, weight]>: ConstructCache of Pseudocode 1 appends <IO[item][layer],
 * Y[item]>; with `weights` an entry is the k-means form of Sec. 4, <cluster centre, majority label,
 * fraction of the majority label>.  vecs: [n x dim] device, row-major, contiguous rows; labels: [n] device
 * int32; weights: [n] device float or NULL (= 1.0).  Also computes each row's squared norm.  Asynchronous
 * on the stream (which look-ups see the new entries: fi_cache_lookup_view below); label values are not range-checked on the host (they are opaque to the look-up).
 * Errors: CAPACITY when size + n > capacity (nothing is written), INVALID_ARG, CUDA.
 */
fi_status_t fi_cache_insert(fi_cache_t *cache, const void *vecs, const int32_t *labels, const float *weights,
                            int64_t n, void *cuda_stream);

/* Set THRESHOLDS[layer] (Pseudocode 1; Sec. 3.1 (ii) describes how the offline phase picks it). */
fi_status_t fi_cache_set_threshold(fi_cache_t *cache, float tau);

/* Choose the kernels later look-ups use (fi_path_t).  UNSUPPORTED for FI_PATH_GEMM on a float32 cache. */
fi_status_t fi_cache_set_path(fi_cache_t *cache, int32_t path);

/* Number of entries stored, counting every insert that has been enqueued. */
int64_t fi_cache_size(const fi_cache_t *cache);

/*
 * Inserting into a cache that is being looked up (Sec. 5, incremental cache update: entries are appended while the
 * cache serves requests).  An insert may run on one stream while look-ups of the same cache run on another.  A look-up
 * covers a PREFIX of the entries, fixed when it is enqueued: every insert that has completed by then, and every
 * insert enqueued earlier on the look-up's own stream, up to the first insert that is neither.  Rows behind that
 * prefix may be in the middle of being written; the kernels never read them (the row count travels as a kernel
 * argument; the tensor maps cover the whole capacity and never change).  Up to 16 inserts may be in flight per
 * cache; one more waits on the host for the oldest.
 * fi_cache_lookup_view: the number of entries the most recent look-up on this cache covered.
 * Look-ups of one cache still share its scratch and must be ordered among themselves.
 */
int64_t fi_cache_lookup_view(const fi_cache_t *cache);

/*
 * Limit the look-up kernels of this cache to `sms` persistent CTAs (0 = one per SM of the device, the default), so
 * that another stream's work, such as the next layer of the network (Sec. 5 pipelines cache look-ups with the
 * forward pass), finds free SMs while a look-up runs.  Takes effect from the next look-up.
 */
fi_status_t fi_cache_set_sm_limit(fi_cache_t *cache, int32_t sms);

/* Forget all entries (size becomes 0; capacity and configuration stay).  Asynchronous work already queued on the
 * cache must have been ordered before later inserts by the caller's stream. */
fi_status_t fi_cache_clear(fi_cache_t *cache);

/*
 * One Lloyd iteration towards the k-means cache of Sec. 4, whose entries are <cluster centre, majority label,
 * fraction of the majority label> (Sec. 2.1 clusters each block's outputs into 200 clusters and tags them this way).
 * `centres` is a cache that holds the current centres (its k must be 1).  Assignment step: every point goes to its
 * nearest centre under squared L2, ties to the smaller centre index (the look-up itself, in batches of max_batch).
 * Update step: per cluster the mean of its points, rounded to the cache's dtype; the number of points; the most
 * frequent of the points' labels (smaller label on ties) and its share.  A cluster without points keeps its
 * centre and gets label -1, share 0.
 *   points [n x ld_elems] device, dtype of the cache; point_labels [n] device int32 in [0, num_classes) (a label
 *   outside that range is left out of the majority count)
 *   assign_out [n] device int32; new_centres [size x dim] device, cache dtype; counts / majority_label [size]
 *   device int32; fraction [size] device float
 * Feeding (new_centres, majority_label, fraction) to fi_cache_clear + fi_cache_insert (as vecs, labels, weights)
 * gives the next iteration's centres, and after the last iteration the k-means cache itself.  At most 8,192
 * classes.  Asynchronous.
 */
fi_status_t fi_kmeans_step(fi_cache_t *centres, const void *points, int64_t ld_elems, const int32_t *point_labels,
                           int64_t n, int32_t *assign_out, void *new_centres, int32_t *counts,
                           int32_t *majority_label, float *fraction, void *cuda_stream);

/*
 * The cache look-up API of Sec. 3 for a batch: for each request the k nearest cached entries under squared
 * L2 (ties by smaller index), per label i among them S_i = m_i/k and C_i = S_i * sum_j w_j/d_j, the label
 * with the largest C_i and that C_i, and the hit flag under the cache's rule and threshold.  With
 * fewer than k entries, k_eff = min(k, size) replaces k.
 *   queries          [rows x ld_elems] device; request i is row row_idx[i] (or row i when row_idx is NULL)
 *   ld_elems         leading dimension in elements (>= dim)
 *   row_idx          [batch_max] device int32 or NULL
 *   batch_max        upper bound of the batch, 0..max_batch; sizes the launch
 *   batch_count_dev  [1] device int32 holding the actual batch (<= batch_max), or NULL = batch_max; read
 *                    by the kernels, never by the host, so a cascade needs no host round trip
 *   out              device arrays; slots >= the actual batch are left untouched
 * Asynchronous.  Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
fi_status_t fi_cache_lookup_batch(const fi_cache_t *cache, const void *queries, int64_t ld_elems,
                                  const int32_t *row_idx, int32_t batch_max, const int32_t *batch_count_dev,
                                  const fi_lookup_out_t *out, void *cuda_stream);

/* Start a cascade: final_label = -1, final_conf = 0, exit_stage = num_stages for all batch0 requests
 * (the value a request keeps when no layer freezes it: the model's output layer answers, Pseudocode 1). */
fi_status_t fi_cascade_init(const fi_cascade_state_t *state, int32_t num_stages, int32_t device, void *cuda_stream);

/*
 * One layer of FreezeInference (Pseudocode 1) for a whole batch: look up the activations of the requests
 * still alive in this layer's cache; a hit freezes the request (its label, confidence and stage are
 * recorded); the misses are compacted, order kept, into the batch of the next layer (Sec. 5: the batch
 * is rebuilt after each layer without the items frozen there).
 *   stage_acts  [batch0 x ld_elems] device: row r = activation of request r at this layer
 * Needs state->batch0 <= max_batch of the cache.  Asynchronous; the count stays on the device.
 */
fi_status_t fi_cascade_step(const fi_cache_t *stage_cache, const void *stage_acts, int64_t ld_elems,
                            const fi_cascade_state_t *state, void *cuda_stream);

/*
 * End-to-end variants with HOST buffers: copy the inputs to the device, run the same kernels, copy the
 * results back, and synchronise the stream before returning.
 * fi_cache_lookup_batch_host: queries [batch x dim] host, contiguous; out arrays are host pointers.
 * fi_cascade_run_host: acts[l] = [batch0 x dim_l] host activations of every request at stage l; runs
 * fi_cascade_init and num_stages steps; outputs [batch0] host arrays; stage_arrivals [num_stages+1] host,
 * nullable: number of requests that reached each stage, last entry = never frozen.
 */
fi_status_t fi_cache_lookup_batch_host(const fi_cache_t *cache, const void *queries_host, int32_t batch,
                                       const fi_lookup_out_t *out_host, void *cuda_stream);
fi_status_t fi_cascade_run_host(fi_cache_t *const *stage_caches, int32_t num_stages, const void *const *acts_host,
                                int32_t batch0, int32_t *final_label_host, int32_t *exit_stage_host,
                                float *final_conf_host, int32_t *stage_arrivals_host, void *cuda_stream);

/*
 * Look-up that allocates nothing (the paper has no counterpart: this entry point exists for callers that
 * cannot call cudaMalloc when they need an answer, e.g. a server whose own pool already holds all device
 * memory, or a latency path where an allocation, which may synchronise the device, is not acceptable).
 * Same result as fi_cache_lookup_batch on the streaming path, but on plain arrays instead of a cache
 * object, with the candidate-list scratch in a fixed 4 MiB array inside the library (every GPU that loads
 * the library holds it until the process exits).  Calls no cudaMalloc / cudaFree and no allocating routine.
 *   cache_vecs [n_entries x dim] device, contiguous rows, dtype fi_dtype_t; labels [n_entries] device;
 *   weights    [n_entries] device, REQUIRED here (pass ones for a plain k-NN cache);
 *   queries    [batch x ld_elems] device; out: device arrays as for fi_cache_lookup_batch;
 *   k 1..32; rule / metric / threshold as in fi_cache_config_t; runs on the current device.
 * Limits: batch <= 256 per call (FI_ERR_CAPACITY beyond; split larger batches).  The first call on a device
 * looks up the scratch array's device address (cudaGetSymbolAddress) and the SM count; make that first call
 * outside any stream capture.  All calls on a device share the one array and it keeps the previous call's
 * contents (every entry a call reads is first written by that call, so nothing needs clearing): calls that
 * overlap on the GPU (different streams without ordering) race on it and must be serialised by the caller.
 */
fi_status_t fi_lookup_noalloc(const void *cache_vecs, const int32_t *labels, const float *weights, int64_t n_entries,
                              int32_t dim, int32_t dtype, int32_t k, int32_t rule, int32_t metric, float threshold,
                              const void *queries, int64_t ld_elems, int32_t batch, const fi_lookup_out_t *out,
                              void *cuda_stream);

/*
 * ComputeThresholds of Pseudocode 1 for one layer (Sec. 3.1 (ii)): look up n validation activations in the
 * layer's cache and set THRESHOLDS[layer] to the largest confidence among the look-ups whose label differs from
 * the label the model itself predicted for that item (0 when no look-up is wrong), so that no validation item is frozen
 * with a wrong label.  The look-ups run in batches of at most max_batch; the maximum is formed on the device.
 *   val_acts   [n x ld_elems] device, dtype of the cache; model_labels [n] device int32 (Y[item])
 *   tau_out    host float, nullable: receives the threshold; wrong_out host int64, nullable: wrong look-ups
 * The cache's threshold is replaced by the result.  Synchronises the stream before returning.
 */
fi_status_t fi_cache_compute_threshold(fi_cache_t *cache, const void *val_acts, int64_t ld_elems,
                                       const int32_t *model_labels, int64_t n, float *tau_out, int64_t *wrong_out,
                                       void *cuda_stream);

/*
 * Cache rows sharded over several GPUs (the paper has one cache per layer on one machine; with entries split over
 * ranks, rank g holding global rows [offset_g, offset_g + size_g), the k nearest of the whole cache are among
 * the k nearest of every shard).  Step 1, on each rank after fi_cache_lookup_batch with topk outputs:
 * fi_cache_neighbor_tuples turns its neighbour indices [n = batch*k] into travelling tuples: global index
 * (local + index_offset, -1 stays -1), label and weight of each neighbour.  Step 2, after the ranks exchanged their
 * tuples and distances (e.g. one all-gather): fi_merge_shard_lookups merges [shards][batch][k] tuples per query
 * by (distance, global index), keeps k, and applies the vote and hit rule of Sec. 3 / Pseudocode 1 exactly as
 * fi_cache_lookup_batch does.  All pointers are device pointers on the current device; asynchronous.
 */
fi_status_t fi_cache_neighbor_tuples(const fi_cache_t *cache, const int32_t *topk_idx, int64_t n, int32_t index_offset,
                                     int32_t *global_idx, int32_t *label, float *weight, void *cuda_stream);
fi_status_t fi_merge_shard_lookups(int32_t shards, int32_t batch, int32_t k, const float *dist, const int32_t *global_idx,
                                   const int32_t *label, const float *weight, int32_t metric, int32_t rule,
                                   float threshold, const fi_lookup_out_t *out, void *cuda_stream);

/*
 * Dimensionality reduction in front of the look-up (Sec. 3: a one-layer network whose hidden layer has 1,024 nodes;
 * its hidden activations are what the caches hold and what a request is looked up with).  The trained weights are
 * the caller's; the library applies them:  y = max(0, W x + b), W [out_dim x in_dim] bf16 row-major, b [out_dim]
 * fp32 (null: zero), products accumulated in fp32 on the tensor cores, y rounded to bf16 (nearest even).  The paper
 * names no non-linearity; the rectifier is this library's reading.
 *   fi_projection_create: in_dim a multiple of 8, out_dim a multiple of 16; owns a copy of the weights, its scratch
 *     and one [max_batch x out_dim] output buffer.
 *   fi_projection_set_weights: device pointers; copies them (asynchronous on the stream).
 *   fi_projection_apply: x [batch_max x ld_elems] bf16 device, 16-byte aligned rows; row_idx (nullable) gathers rows of
 *     x as in fi_cache_lookup_batch; batch_count_dev (nullable) is the device-resident row count; y [batch_max x ld_y]
 *     bf16 device, 16-byte aligned, ld_y a multiple of 8; rows past the count are left untouched.  Asynchronous.
 *   fi_cascade_step_projected: fi_cascade_step with the projection applied to the surviving requests' activations
 *     first; `cache` holds projected vectors (dim = out_dim, bf16).
 *   fi_projection_poll_status: as fi_cache_poll_status, for the projection's own kernels (synchronises).
 * Errors: FI_ERR_INVALID_ARG for sizes, alignment, a batch above max_batch or weights never set.
 */
typedef struct fi_projection fi_projection_t;
fi_status_t fi_projection_create(int32_t in_dim, int32_t out_dim, int32_t device, int32_t max_batch, fi_projection_t **out);
fi_status_t fi_projection_destroy(fi_projection_t *proj);
fi_status_t fi_projection_set_weights(fi_projection_t *proj, const void *weights, const float *bias, void *cuda_stream);
fi_status_t fi_projection_poll_status(fi_projection_t *proj);
/* as fi_cache_set_profiling / fi_cache_read_profile, around the two kernels of fi_projection_apply */
fi_status_t fi_projection_set_profiling(fi_projection_t *proj, int32_t enable);
fi_status_t fi_projection_read_profile(fi_projection_t *proj, float *total_ms, int32_t *launches);
fi_status_t fi_projection_apply(const fi_projection_t *proj, const void *x, int64_t ld_elems, const int32_t *row_idx,
                                int32_t batch_max, const int32_t *batch_count_dev, void *y, int64_t ld_y,
                                void *cuda_stream);
fi_status_t fi_cascade_step_projected(const fi_cache_t *cache, const fi_projection_t *proj, const void *stage_acts,
                                      int64_t ld_elems, const fi_cascade_state_t *state, void *cuda_stream);

/*
 * Self-test of the failure path: enqueue a one-thread kernel that waits, with the given limit in SM cycles (at most
 * 2e9, about a second), on a barrier that nothing completes.  The wait runs out, the kernel sets the cache's status
 * word and returns; the next fi_cache_poll_status reports FI_ERR_TIMEOUT and the device stays usable.  Nothing
 * faults, traps or hangs.
 */
fi_status_t fi_cache_selftest_wait(fi_cache_t *cache, int64_t limit_cycles, void *cuda_stream);

/* Synchronise the device and return FI_ERR_TIMEOUT if a kernel of this cache gave up on a bounded wait
 * since the last poll (the word is cleared), FI_OK otherwise. */
fi_status_t fi_cache_poll_status(fi_cache_t *cache);

/*
 * Certificate of the tensor-core path (bf16 caches, batches of 2 and more; the paper has no counterpart: it looks up
 * with exact distances on the CPU).  The distance GEMM ranks cache rows by a score accumulated in fp32 on the tensor
 * cores and hands a short candidate list per request to the exact re-ranking.  With E = eps (||q||^2 + max ||c||^2),
 * eps = (dim / 16 + 4) * 2^-23, taken as the bound of a score's error (one dropped unit in the last place per
 * accumulation step of 16 columns), a request is CERTIFIED when the k-th exact
 * distance among its candidates is below (largest candidate score) + ||q||^2 - E: then no cache row outside the list
 * can be one of the k nearest, and the neighbours returned are the exact ones.  Look-ups on the streaming path use
 * exact distances throughout and are always certified.
 *   fi_cache_read_certificate: synchronises the device; returns and clears (nullable pointers are skipped) how many
 *     requests since the last read had no certificate, how many of those the repair pass did not look up again, and
 *     the largest score error observed on candidates, relative to ||q||^2 + max ||c||^2 (compare with eps).
 *   fi_cache_read_slot_certificates: synchronises; copies the flags of the cache's most recent look-up (1 = certified or
 *     repaired) for slots 0..n-1 to host memory.
 *   fi_cache_set_repair: with repair on, every look-up on the tensor-core path is followed by a second pass in which
 *     the streaming kernel looks the uncertified requests up again with exact distances (at most 64 per look-up; the
 *     list stays on the device, and the two extra kernels return at once when it is empty).  Off by default.
 */
fi_status_t fi_cache_set_repair(fi_cache_t *cache, int32_t enable);
fi_status_t fi_cache_read_certificate(fi_cache_t *cache, int64_t *uncertified, int64_t *unrepaired, float *max_score_error);
fi_status_t fi_cache_read_slot_certificates(fi_cache_t *cache, uint8_t *flags_host, int32_t n);

/*
 * Device timing of the distance kernel (the tensor-core GEMM or the streaming kernel) of later look-ups on
 * this cache: with profiling on, each look-up records a CUDA event before and after that kernel on the
 * caller's stream (up to 256 look-ups are kept; older ones are overwritten).  fi_cache_read_profile
 * synchronises on the recorded events, returns the summed kernel time in milliseconds and the number of
 * launches it covers, and clears the record.  Events are created on first use and freed by destroy.
 */
fi_status_t fi_cache_set_profiling(fi_cache_t *cache, int32_t enable);
fi_status_t fi_cache_read_profile(fi_cache_t *cache, float *total_ms, int32_t *launches);

/* Host only (no GPU call): how the distance GEMM of a look-up of `count` requests (in a call sized for `max_batch`)
 * against `n_entries` bf16 entries of `dim` values would be split over `num_ctas` CTAs.
 * plan_out[0..16] = count, query tiles, tiles per group, groups, cache-row ranges, rows per range / 16, list length,
 * rows per query tile, lists per query, mode (0 ranges, 1 wave + tail, 3 spans), cache-row tiles per query tile,
 * tiles left in pieces, pieces per tail tile, 0, half-full last query tile (0 / 1), CTAs per full query tile, CTAs
 * of the half-full one (the last three: spans mode).
 * If `cta` >= 0 and the mode is spans, items_out receives that CTA's pieces, six values each (query tile, cache-row
 * tile, first k-block, end k-block, 128-row MMAs, slot of the partial sums), and *n_items their number (at most 3);
 * in other modes *n_items = 0.  plan_out, items_out (18 values) and n_items are host pointers owned by the caller.
 * Errors: FI_ERR_INVALID_ARG for null plan_out or non-positive sizes.  Used by the tests of the host logic. */
fi_status_t fi_gemm_plan_describe(int32_t count, int64_t n_entries, int32_t num_ctas, int32_t k, int32_t dim,
                                  int32_t max_batch, int32_t cta, int32_t *plan_out, int32_t *items_out,
                                  int32_t *n_items);

/* Number of kernels this library has launched in the calling process (all caches). */
int64_t fi_launch_count(void);

/* Text of the last error on the calling thread ("" if none).  The pointer stays valid until the next call
 * of the library on this thread. */
const char *fi_last_error(void);

/* Name of a status code. */
const char *fi_status_string(fi_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* FI_H_ */
