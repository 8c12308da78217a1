// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fi.h"

namespace fi {

constexpr int kMaxK = 32;          // largest k of a look-up
constexpr long long kMaxEntries = 2147483647ll - 255;   // cache entries are indexed with int32 (tiles may overshoot by < 256)
constexpr int kStreamMaxBatch = 1; // batches up to this size take the streaming kernel under FI_PATH_AUTO (bf16)
constexpr int kTileM = 128;        // queries per MMA (= TMEM lanes); a CTA tile holds 128 or 256 queries
constexpr int kMaxHostStages = 64; // stages a host-driven cascade may have
constexpr int kRepairCap = 64;     // queries per look-up the exact repair pass can take
constexpr int kCertWords = 5;      // certificate block: uncertified, max score error (float bits), repair-list length,
                                   // max ||c||^2 (float bits), uncertified and not repaired
constexpr int kMaxPending = 16;    // inserts that may be in flight on a cache at once
constexpr int kMaxDevices = 64;    // device ordinals the per-device set-up tables cover
constexpr int kMinMapRows = 4;     // fewest rows a query tensor map is made over
constexpr int kProfSlots = 256;    // look-ups whose distance-kernel time is kept

// Candidates kept per query by the GEMM path before the exact re-ranking: k plus a margin of 3,
// rounded up to a list length the select kernel is compiled for.
__host__ __device__ inline int gemm_list_len(int k) {
    int want = k + 3;
    return want <= 4 ? 4 : want <= 8 ? 8 : want <= 16 ? 16 : 32;
}

// How the tiles of the distance GEMM are spread over the CTAs.  Query tiles (`tile_m` = 128 or 256 rows each) are
// taken in groups of `mg`; inside a group, CTA (m_local, q) owns query tile m_local and the q-th of `parts` equal
// ranges of cache rows, so CTAs with the same q stream the same cache rows at the same time (they meet in
// L2) and each query row ends up with one candidate list per range ("ranges" mode).
//
// When the whole problem is only a little more than one 256 x 256 tile per CTA (deep rows, few queries), cutting
// ranges would leave every CTA with two narrow tiles and the query tile read twice.  The "wave + tail" mode
// then gives each CTA one full tile over the whole row length, and the tiles left over are cut along the row
// length into `tail_slices` pieces, one per CTA; their partial sums go to memory and a small kernel adds them
// up and selects.
//
// When there is less than one 256 x 256 tile per CTA ("spans" mode), ranges would be narrow tiles under a query tile
// that every CTA reads in full.  Instead every query tile gets an equal share of the CTAs, and the (cache-row tile,
// k-block) pairs of that query tile, laid end to end, are cut into one span per CTA of its share: a CTA runs the
// k-blocks of its span (the end of one tile and the start of the next, at most kMaxSpanItems pieces), every piece
// leaves its partial sums in memory, and the same small kernel adds up the pieces of each tile and selects.  The
// spans of all query tiles have the same boundaries, so the CTAs that need the same cache rows read them at the same
// time; the query tiles are read at scattered times and have to stay in L2, which bounds their size.  A last query
// tile with at most 128 requests computes half (one of its two 128-row MMAs) and gets 3/4 of a share: its k-blocks
// still load the full cache-row tile.
struct GemmPlan {
    int32_t count;        // actual batch
    int32_t m_tiles;      // ceil(count / tile_m)
    int32_t mg;           // query tiles per group
    int32_t groups;       // ceil(m_tiles / mg)
    int32_t parts;        // cache-row ranges per query tile
    int32_t range16;      // rows per range, in units of 16 (the last range may be shorter)
    int32_t list_len;     // entries per candidate list
    int32_t tile_m;       // query rows per CTA tile
    int32_t lists;        // candidate lists per query
    int32_t mode;         // 0 = ranges, 1 = wave + tail, 2 = pieces only (plain product, no select), 3 = spans
    int32_t n_tiles;      // wave + tail, pieces, spans: cache-row tiles per query tile
    int32_t tail_tiles;   // wave + tail: tiles beyond the first wave; pieces, spans: all tiles
    int32_t tail_slices;  // wave + tail, pieces: pieces each of those tiles is cut into along the row length
    int32_t pieces;       // pieces: tail_tiles * tail_slices
    int32_t half;         // spans: 1 = the last query tile holds at most 128 requests
    int32_t span_full;    // spans: CTAs per full query tile
    int32_t span_half;    // spans: CTAs of the half query tile
};

constexpr int kMaxSpanItems = 3;   // pieces a span can consist of (spans are at most two tiles' k-blocks long)
constexpr int kMinSpanKb = 16;     // shortest span worth a CTA, in k-blocks

// Spans mode: which query tile CTA `cta` works for, its index among that tile's CTAs and their number (false: idle)
__host__ __device__ inline bool span_owner(const GemmPlan &p, int cta, int &m, int &j, int &cm) {
    const int mf = p.m_tiles - p.half, full_ctas = mf * p.span_full;
    if (cta < full_ctas) {
        m = cta / p.span_full;
        j = cta - m * p.span_full;
        cm = p.span_full;
        return true;
    }
    m = p.m_tiles - 1;
    j = cta - full_ctas;
    cm = p.span_half;
    return j < p.half * p.span_half;
}
// first CTA and number of CTAs of query tile m
__host__ __device__ inline void span_ctas_of(const GemmPlan &p, int m, int &first, int &cm) {
    const int mf = p.m_tiles - p.half;
    first = m < mf ? m * p.span_full : mf * p.span_full;
    cm = m < mf ? p.span_full : p.span_half;
}
// position, in (cache-row tile, k-block) pairs of one query tile, where the j-th of cm spans starts (j = cm: the end)
__host__ __device__ inline int span_begin(const GemmPlan &p, int num_kb, int j, int cm) {
    return j * (p.n_tiles * num_kb) / cm;
}

// `pair`: the workers are pairs of CTAs that share one tile of tile_m rows (half each; pair_lists epilogue warps, hence
// lists, per row; ranges only, range lengths a multiple of 32 rows); num_ctas is then the number of pairs.
__host__ __device__ inline GemmPlan make_gemm_plan(int count, long long n_entries, int num_ctas, int k, int tile_m,
                                                   int num_kb, bool pair = false, int pair_lists = 2) {
    GemmPlan p;
    p.count = count;
    p.m_tiles = (count + tile_m - 1) / tile_m;
    p.list_len = gemm_list_len(k);
    p.tile_m = tile_m;
    p.pieces = 0;
    p.lists = 0;
    p.mode = 0;
    p.n_tiles = p.tail_tiles = p.tail_slices = 0;
    p.half = p.span_full = p.span_half = 0;
    long long n16 = (n_entries + 15) / 16;
    if (p.m_tiles <= 0 || n16 <= 0) {
        p.mg = p.groups = p.parts = 1;
        p.range16 = 0;
        p.lists = pair ? pair_lists : tile_m == kTileM ? 2 : 1;
        return p;
    }
    if (tile_m == 2 * kTileM && num_kb >= 64 && !pair) {
        const long long nt = (n16 + 15) / 16;                 // tiles of at most 256 rows
        const long long total = (long long)p.m_tiles * nt;
        // Spans: less than a tile per CTA (a half tile counts 3/4: half the MMAs, 3/4 of the operand bytes), query
        // tiles of at most 16 MB together, and 32-bit span arithmetic.
        const int half = count - (p.m_tiles - 1) * tile_m <= kTileM ? 1 : 0;
        const int mf = p.m_tiles - half;
        if ((4 * mf + 3 * half) * nt <= 4 * num_ctas && (long long)p.m_tiles * num_kb <= 512 &&
            (long long)num_ctas * nt * num_kb < 2147483647ll) {
            const int len = (int)nt * num_kb;                       // pairs per query tile
            const int cap = len / kMinSpanKb > 0 ? len / kMinSpanKb : 1;
            int ch = half ? (mf ? num_ctas * 3 / (4 * mf + 3) : num_ctas) : 0;
            if (half && ch < 1) ch = 1;
            int cf = mf ? (num_ctas - ch) / mf : 0;
            if (ch > cap) ch = cap;
            if (cf > cap) cf = cap;
            // the longest span (len / c rounded up) may touch kMaxSpanItems tiles at most
            const bool fits = (!mf || (cf >= 1 && (len + cf - 1) / cf <= 2 * num_kb)) &&
                              (!half || (len + ch - 1) / ch <= 2 * num_kb);
            if (fits) {
                p.mode = 3;
                p.n_tiles = (int32_t)nt;
                p.tail_tiles = (int32_t)total;
                p.half = half;
                p.span_full = cf;
                p.span_half = ch;
                p.mg = p.m_tiles;
                p.groups = 1;
                p.parts = (int32_t)nt;
                p.range16 = 16;
                p.lists = (int32_t)nt;
                return p;
            }
        }
        if (total > num_ctas && total <= num_ctas + num_ctas / 2) {
            p.mode = 1;
            p.n_tiles = (int32_t)nt;
            p.tail_tiles = (int32_t)(total - num_ctas);
            int slices = num_ctas / p.tail_tiles;
            if (slices > num_kb) slices = num_kb;
            p.tail_slices = slices;
            p.mg = p.m_tiles;
            p.groups = 1;
            p.parts = (int32_t)nt;
            p.range16 = 16;
            p.lists = (int32_t)nt;
            return p;
        }
    }
    // Few cache rows (one tile spans them all) under many query tiles, e.g. assigning points to k-means centres:
    // cutting the rows into ranges would leave tiles a few rows wide, which the MMAs run at a fraction of their
    // rate while every CTA re-reads the query tiles.  The query tiles are dealt round-robin to all CTAs instead.
    if (n16 <= 16 && p.m_tiles >= num_ctas / 2 && !pair) {
        p.mg = p.m_tiles < num_ctas ? p.m_tiles : num_ctas;
        p.groups = (p.m_tiles + p.mg - 1) / p.mg;
        p.parts = 1;
        p.range16 = (int32_t)n16;
        p.lists = tile_m == kTileM ? 2 : 1;
        return p;
    }
    // Group size: the fewest MMA columns per CTA in total, except that on long ranges a larger group within 3 % of
    // that minimum is preferred: it means fewer, longer ranges, hence fewer candidate lists per query to warm up
    // and to merge, and more CTAs streaming the same cache rows at the same time.
    // (32-bit divisions: one thread of every CTA evaluates this at kernel start, and 64-bit ones cost microseconds)
    int best_mg = 1;
    int mg_max = p.m_tiles < 16 ? p.m_tiles : 16;
    if (mg_max > num_ctas) mg_max = num_ctas;
    // A group's query tiles are read again for every tile of cache rows, by CTAs on both dies, while the cache rows
    // stream through L2.  Over a cache that does not fit in L2 a group is kept under 48 MB of query tiles: measured on
    // 8,192 queries x 200,000 entries x 8,192 values, three groups of 11 tiles ran 1.3 % faster than two of 16 (the
    // traffic from memory stayed the same: cache-row tiles and query tiles together exceed what either die keeps).
    if (n_entries * (long long)num_kb * 128 > (96ll << 20)) {
        const int cap = (int)((48ll << 20) / ((long long)tile_m * num_kb * 128));
        if (mg_max > cap) mg_max = cap < 1 ? 1 : cap;
    }
    const int n16i = (int)n16;   // entries are indexed with int32, so n16 < 2^27
    long long cost[16], min_cost = -1;
    int eff[16];
    for (int mg = 1; mg <= mg_max; ++mg) {
        const int groups = (p.m_tiles + mg - 1) / mg;
        const int mg_eff = (p.m_tiles + groups - 1) / groups;
        int cand_parts = num_ctas / mg_eff;
        if (cand_parts > n16i) cand_parts = n16i;
        const int r = (n16i + cand_parts - 1) / cand_parts;
        cost[mg - 1] = (long long)groups * r;
        eff[mg - 1] = mg_eff;
        if (min_cost < 0 || cost[mg - 1] < min_cost) min_cost = cost[mg - 1];
    }
    for (int mg = 1; mg <= mg_max; ++mg) {
        const long long c = cost[mg - 1];
        // short ranges (under 4,096 rows per CTA) are latency-bound: exact minimum only
        if ((min_cost >= 256 ? c * 100 <= min_cost * 103 : c == min_cost) && eff[mg - 1] > best_mg) best_mg = eff[mg - 1];
    }
    p.mg = best_mg;
    p.groups = (p.m_tiles + p.mg - 1) / p.mg;
    int parts = num_ctas / p.mg;
    if (parts > n16i) parts = n16i;
    int r16 = (n16i + parts - 1) / parts;
    if (pair) r16 += r16 & 1;         // ranges of whole 32-row blocks: each CTA of a pair loads half of every tile
    parts = (n16i + r16 - 1) / r16;   // drop ranges that would be empty
    p.parts = (int32_t)parts;
    p.range16 = (int32_t)r16;
    // with 128-row tiles (and with pairs) two epilogue warps share each row and keep a list each
    p.lists = p.parts * (pair ? pair_lists : tile_m == kTileM ? 2 : 1);
    return p;
}

// Plan of a plain product Y = Q W^T (the projection in front of the look-up): every 256 x 256 tile of Y is cut
// along the row length into as many pieces as fill the CTAs once; piece p = tile * slices + slice goes to CTA
// p mod num_ctas and leaves its partial sums in slot p.
__host__ __device__ inline GemmPlan make_product_plan(int count, long long n_rows, int num_ctas, int tile_m, int num_kb) {
    GemmPlan p;
    p.count = count;
    p.m_tiles = (count + tile_m - 1) / tile_m;
    p.mg = p.m_tiles > 0 ? p.m_tiles : 1;
    p.groups = 1;
    p.range16 = 16;
    p.list_len = 0;
    p.tile_m = tile_m;
    p.lists = 0;
    p.mode = 2;
    const long long n16 = (n_rows + 15) / 16;
    p.n_tiles = (int32_t)((n16 + 15) / 16);
    p.parts = p.n_tiles;
    p.tail_tiles = p.m_tiles * p.n_tiles;
    // a piece shorter than 8 k-blocks costs more to store and add up again than its MMAs take
    int slices = p.tail_tiles > 0 ? num_ctas / p.tail_tiles : 1;
    if (slices > num_kb / 8) slices = num_kb / 8;
    if (slices < 1) slices = 1;
    p.tail_slices = slices;
    p.pieces = p.tail_tiles * slices;
    return p;
}

}  // namespace fi

// The cache object behind the opaque handle.
// An insert whose copies may still be running: the entries count for look-ups on other streams once `ev` has completed.
struct PendingInsert {
    cudaStream_t stream;
    cudaEvent_t ev;
    int64_t size_after;
};

struct fi_cache {
    fi_cache_config_t cfg;
    int64_t size;            // entries the look-up being enqueued covers (refresh_view): every insert that is complete or
                             // ordered before it on its stream, up to the first one that is neither
    int64_t enqueued;        // entries whose insert has been enqueued (what fi_cache_size reports)
    int64_t committed;       // entries of inserts known to be complete
    PendingInsert pending[fi::kMaxPending];   // oldest first, as a ring
    int pend_head, pend_n;
    cudaEvent_t pend_ev[fi::kMaxPending];     // one event per ring slot, created with the cache
    int sm_limit;            // CTAs the persistent kernels of a look-up may occupy (0 = all SMs)
    int sm_count;            // CTAs the persistent kernels launch (sm_total, or the caller's limit)
    int sm_total;            // SMs of the device
    size_t elem_size;
    // device storage owned by the cache
    void *rows;              // [capacity x dim]
    int32_t *labels;         // [capacity]
    float *weights;          // [capacity]
    float *norms;            // [capacity] squared norms of the stored values (fp32)
    // look-up scratch
    float *part_score;       // candidate lists
    int32_t *part_idx;
    size_t part_entries;     // capacity of the two arrays, in entries
    void *q_compact;         // [max_batch x dim] gathered queries for the GEMM path (bf16 caches)
    int32_t *slot_label;     // [max_batch] per-slot results of a cascade step
    float *slot_conf;
    uint8_t *slot_hit;
    float *tail_dump;        // partial sums of the tail tiles: [units][256 columns][256 rows], allocated on first need
    size_t tail_dump_units;
    int32_t *row_bound;      // [(max_batch + 256) x list_len] per-query slots whose maximum bounds the list_len-th best score, shared by all
                             // CTAs of a GEMM launch (order-preserving integer image of the float)
    fi::GemmPlan *plan_dev;  // written by the GEMM kernel, read by the finalize kernel
    int32_t *status_dev;     // device status word (bounded waits that ran out)
    int32_t *cert_dev;       // [kCertWords] certificate block of the tensor-core path (see FinalizeParams::cert)
    uint8_t *slot_cert;      // [max_batch] 1 = the slot's neighbours are proven exact (last look-up)
    int32_t *repair_list;    // [kRepairCap] slots the exact repair pass looks up again
    bool repair_on;
    int32_t *calib_acc;      // [2] threshold calibration: max wrong confidence (bit pattern), wrong count
    float *km_dist;          // [max_batch] k-means assignment scratch: nearest distances of one batch (unused output)
    float *km_partial;       // [size x segments x dim] k-means update: per-segment sums of the points of each cluster
    size_t km_partial_elems; // floats allocated there (grown on demand)
    // staging for the host-buffer entry points (allocated on first use)
    void *h2d_stage;
    size_t h2d_stage_bytes;
    cudaStream_t copy_stream;   // host-driven cascade: uploads of later stages run here, beside the look-ups
    cudaEvent_t *copy_ev;       // one "stage uploaded" event per stage (kMaxHostStages), created on first use
    // tensor maps over the cache rows (bf16 only): boxes of 64 and of 16 rows by 64 elements
    CUtensorMap tmap_rows64;
    CUtensorMap tmap_rows16;
    bool tmaps_ready;
    // optional device timing of the distance kernel
    bool prof_on;
    int prof_n;              // look-ups recorded since the last read
    cudaEvent_t *prof_ev;    // 2 * kProfSlots events, created on first use
};

namespace fi {

void set_error(const char *fmt, ...);
void count_launch(int n = 1);
fi_status_t check_launch(const char *what);

// ---- launchers (each enqueues on `stream`, returns a status) ----
// squared norms of n stored rows; norm_max_bits (nullable) is raised to the largest of them (float bit pattern)
fi_status_t launch_row_norms(const void *rows, int dtype, int64_t n, int dim, float *norms, int32_t *norm_max_bits,
                             cudaStream_t stream);

fi_status_t launch_gather_rows(const void *src, int64_t ld_elems, const int32_t *row_idx, int32_t batch_max,
                               const int32_t *count_dev, void *dst, int dim, size_t elem_size, cudaStream_t stream);

// streaming look-up: writes candidate lists [batch][parts][k] (exact fp32 squared distances); returns parts
fi_status_t launch_stream_lookup(const fi_cache *c, const void *queries, int64_t ld_elems, const int32_t *row_idx,
                                 int32_t batch_max, const int32_t *count_dev, int *parts_out, cudaStream_t stream);

// tensor-core distance GEMM with fused per-row select: writes candidate lists [batch][parts][list_len] of
// scores ||c||^2 - 2 q.c and the plan it used to c->plan_dev
fi_status_t launch_gemm_select(fi_cache *c, const void *queries_compact, int64_t ld_elems, int32_t batch_max,
                               const int32_t *count_dev, cudaStream_t stream);

// merge candidate lists, (optionally) recompute exact distances, vote, hit
struct FinalizeArgs {
    const void *queries;
    int64_t ld_elems;
    const int32_t *row_idx;
    int32_t batch_max;
    const int32_t *count_dev;
    int parts;              // lists per query, or -1: read from plan_dev
    int list_len;           // entries per list, or -1: read from plan_dev
    int refine;             // 1: scores are approximate, recompute sum (q-c)^2 for the candidates
    fi_lookup_out_t out;
    const int32_t *out_slot = nullptr;   // nullable: result b is written to output slot out_slot[b]
    bool fill_repair_list = false;       // uncertified slots are appended to the cache's repair list
};
fi_status_t launch_finalize(const fi_cache *c, const FinalizeArgs &a, cudaStream_t stream);

fi_status_t launch_compact(const fi_cache *c, const fi_cascade_state_t &st, cudaStream_t stream);
fi_status_t launch_cascade_init(const fi_cascade_state_t &st, int32_t num_stages, cudaStream_t stream);
// acc[0] = max(acc[0], conf[i]) as an integer image, acc[1] += 1, over the slots whose label differs from ref
fi_status_t launch_wrong_max(const int32_t *label, const float *conf, const int32_t *ref, int32_t n, int32_t *acc,
                             cudaStream_t stream);

// k-means update step (means, counts, majority label and its share) for the centres held in `c`
fi_status_t launch_kmeans_update(fi_cache *c, const void *points, int64_t ld, const int32_t *point_labels,
                                 const int32_t *assign, int64_t n, void *new_centres, int32_t *counts,
                                 int32_t *majority, float *fraction, cudaStream_t stream);

fi_status_t launch_neighbor_tuples(const fi_cache *c, const int32_t *topk_idx, int64_t n, int32_t index_offset,
                                   int32_t *out_idx, int32_t *out_label, float *out_weight, cudaStream_t stream);
fi_status_t launch_merge_vote(int shards, int batch, int k, const float *dist, const int32_t *idx, const int32_t *label,
                              const float *weight, int metric, int rule, float tau, const fi_lookup_out_t &out,
                              cudaStream_t stream);
// plain product on the tensor cores: y = max(0, q W^T + bias) rounded to bf16, W = the rows held in `w`, bias = its
// per-row weights; `units` = slots of partial sums `w->tail_dump` must hold (see product_dump_units)
fi_status_t launch_gemm_project(fi_cache *w, const void *queries_compact, int64_t ld_elems, int32_t batch_max,
                                const int32_t *count_dev, void *y, int64_t ld_y, cudaStream_t stream);
size_t product_dump_units(int max_batch, int64_t n_rows, int sm_count);
fi_status_t launch_wait_selftest(fi_cache *c, long long limit_cycles, cudaStream_t stream);
fi_status_t ensure_tensor_maps(fi_cache *c);
// sets c->size to the entries a look-up enqueued now on `stream` may read
void refresh_view(fi_cache *c, cudaStream_t stream);
size_t gemm_part_entries(int max_batch, int64_t capacity, int sm_count, int k, int dim);
// upper bound of gemm_part_entries over every batch <= max_batch and every cache size <= capacity
size_t gemm_part_entries_bound(int max_batch, int64_t capacity, int sm_count, int k, int dim);
// slots of 256 x 256 partial sums a cache's look-ups can need (wave + tail mode), 0 when that mode cannot occur
size_t gemm_tail_units(int max_batch, int dim, int sm_count);
// one-time, per-device set-up of every instantiation of the distance GEMM (shared-memory reservation, register check)
fi_status_t prepare_gemm_kernels(int device);
int gemm_tile_m(int batch_max, int dim);

}  // namespace fi
