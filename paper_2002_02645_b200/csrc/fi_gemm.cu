// Distance GEMM with fused per-row select for bf16 caches (sm_100a: TMA + tcgen05 + TMEM).
//
// Neighbour order under ||q - c||^2 = ||q||^2 + ||c||^2 - 2 q.c does not depend on ||q||^2, so the kernel ranks
// cache rows by the score  s = ||c||^2 - 2 q.c : S = Q X^T is a dense bf16 contraction with fp32 accumulation
// on the tensor cores; the distance matrix is never written to memory.  Each of the 4 epilogue warps reads
// accumulator tiles back from TMEM (one query row per thread) and keeps the `list_len` smallest scores of its
// row in registers.  The exact distances of those few candidates are recomputed afterwards (finalize_kernel).
//
// Roles inside a CTA of 384 threads (three warpgroups): warp 0 = TMA producer (one lane), warp 1 = TMEM owner and
// MMA issuer (one lane), warps 2..3 idle, warps 4..11 = epilogue.  Warpgroup 0 hands most of its registers to the
// epilogue warpgroups (setmaxnreg).  Shared-memory stages are handed over with mbarriers.  Two tile heights:
//   128 queries: accumulator double-buffered in TMEM (2 x 256 columns), so the select of one tile overlaps
//                the MMAs of the next; two epilogue warps per 32 rows, each taking every other 16-column chunk
//                and keeping its own list.  For short rows (few k-blocks per tile), where the select dominates.
//   256 queries: two 128-row MMAs share every cache-row stage, which halves the bytes the CTA pulls from L2
//                per flop (the kernel is bound by L2-to-SM bandwidth, not by the tensor pipe); the two
//                accumulators fill TMEM, so select and MMAs alternate; one epilogue warp per 32 rows.
// Select: a thread owns one query row.  Scores of two 16-column chunks are formed with independent FMAs and
// tested against the row's current k-th best through one min-tree; the few that pass are parked in a small
// per-thread queue in shared memory and inserted into the sorted register list once per tile, when all lanes
// of the warp insert together (inserting on the spot makes the whole warp walk the insert code whenever any
// one lane has a hit, which made the select 20x slower than the MMAs on short rows).  What a tile's scan needs
// from global memory (column norms, the row's shared bound) is fetched a tile ahead where the select is the
// critical path.
// Every wait is bounded: a wait that runs out sets the cache's status word and the CTA drains and returns.
#include <cuda_bf16.h>

#include <cstdlib>
#include <cstring>
#include <mutex>

#include "fi_internal.cuh"

namespace fi {

namespace {

constexpr int kBlockK = 64;                       // bf16 elements per k-block: 128 bytes, one swizzle row
constexpr int kMaxStages = 8;
constexpr int kMaxTileN = 256;                    // cache rows per tile (MMA N), multiple of 16
constexpr int kFirstTileN = 32;                   // cache rows of the short tile a long range opens with
constexpr int kABytes = kTileM * kBlockK * 2;     // 16 KiB
constexpr int kStageRegionBytes = 200 * 1024;     // operand ring; a stage is A (16 or 32 KiB) + B (tile width x 128 bytes)
constexpr int kMaxEpiWarps = 8;
constexpr int kTmemCols = 512;
constexpr long long kWaitLimitCycles = 8000000000ll;  // about 4 s of SM clocks: far beyond any tile, short enough to get the GPU back

struct __align__(8) SmemCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int32_t abort_flag;
    GemmPlan plan;
};

constexpr int kEpiThreads = kMaxEpiWarps * 32;
constexpr int kRoleThreads = 128;                  // warpgroup 0: TMA producer, MMA issuer, two idle warps
constexpr int kGemmThreads = kRoleThreads + kEpiThreads;
// Register split between the warpgroups (setmaxnreg): the kernel is launched with kLaunchRegs per thread, warpgroup
// 0 gives back all but kRoleRegs, the two epilogue warpgroups grow to kEpiRegs.  The shares must fit the launch's
// total, or the growing warps would wait for ever: checked here and again by the host against the compiled kernel.
constexpr int kLaunchRegs = 168;
constexpr int kRoleRegs = 56;
constexpr int kEpiRegs = 224;
static_assert(kRoleThreads * kRoleRegs + kEpiThreads * kEpiRegs <= kGemmThreads * kLaunchRegs, "register shares exceed the launch's total");
constexpr int kNormSmemBytes = kMaxEpiWarps * kMaxTileN * 4;   // 256 floats per epilogue warp
constexpr int kQueueCap = 7;                                    // pending candidates per epilogue thread
constexpr int kQueueStride = kEpiThreads * 8;                   // bytes between a thread's slots: (score, column) pairs
constexpr int kQueueSmemBytes = (kQueueCap + 1) * kQueueStride; // one more slot takes what does not fit
constexpr int kGemmSmemBytes =
    1024 /*alignment slack*/ + kStageRegionBytes + kNormSmemBytes + kQueueSmemBytes + (int)sizeof(SmemCtl);

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the abort flag and the status word) when the limit is reached or
// another thread of the CTA has already given up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, SmemCtl *ctl, int32_t *status, int where,
                                          long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try(bar, parity)) return true;
    // the SM's own cycle counter is a register read; the wait sits on the hand-over path of every stage and tile
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if ((++spins & 0xFF) == 0) {
            if (ctl->abort_flag) return false;
            if (clock64() - t0 > limit_cycles) {
                ctl->abort_flag = 1;
                atomicCAS(status, 0, (int32_t)(FI_ERR_TIMEOUT | (where << 8)));
                return false;
            }
        }
    }
}

// ---- pairs of CTAs (cluster of two) working on one tile with tcgen05 in cta_group::2
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.aligned;\nbarrier.cluster.wait.aligned;" ::: "memory");
}
// arrive on a barrier that may live in the other CTA of the pair (cluster address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of a pair: lands in this CTA's shared memory, completes bytes on a barrier of the leader CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster_addr, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}
// one MMA of the pair: D (256 x N, 128 rows in each CTA's TMEM) += A (128 rows per CTA) x B (N/2 rows per CTA)
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// completion of the pair's MMAs so far, signalled on the barrier at this address in BOTH CTAs
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(smem_u32(bar)),
                 "h"((uint16_t)3)
                 : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

// K-major operand tile in shared memory, rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                    // leading-dimension offset: unused for swizzled K-major
    d |= (uint64_t)(1024 >> 4) << 32;          // stride between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                    // 128-byte swizzle
    return d;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n
__device__ __forceinline__ uint32_t umma_instr_desc(int n, int m = kTileM) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 consecutive accumulator columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// wait for the loads; the registers are listed so that no use of them can move above the wait
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&v)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
                 :
                 : "memory");
}

// order-preserving integer image of a float, so that atomicMin on the image is a float minimum
__device__ __forceinline__ int32_t float_key(float f) {
    const int32_t b = __float_as_int(f);
    return b >= 0 ? b : b ^ 0x7FFFFFFF;
}
__device__ __forceinline__ float key_float(int32_t k) { return __int_as_float(k >= 0 ? k : k ^ 0x7FFFFFFF); }
// smallest of three (the compiler folds the pair into the three-input minimum of this architecture)
__device__ __forceinline__ float fmin3(float a, float b, float c) { return fminf(fminf(a, b), c); }

template <int KP>
struct TopList {
    float s[KP];
    int32_t i[KP];
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int e = 0; e < KP; ++e) {
            s[e] = __int_as_float(0x7F800000);
            i[e] = -1;
        }
    }
    // Equal scores keep their arrival order (smaller index first).  All comparisons are taken against the old
    // list first, so the selects of the KP positions do not depend on one another (a bubble pass would chain
    // them, and the two epilogue warps per scheduler cannot hide that latency).
    __device__ __forceinline__ void insert(float sc, int32_t idx) {
        bool below[KP];
#pragma unroll
        for (int e = 0; e < KP; ++e) below[e] = sc < s[e];
#pragma unroll
        for (int e = KP - 1; e > 0; --e) {
            s[e] = below[e] ? (below[e - 1] ? s[e - 1] : sc) : s[e];
            i[e] = below[e] ? (below[e - 1] ? i[e - 1] : idx) : i[e];
        }
        s[0] = below[0] ? sc : s[0];
        i[0] = below[0] ? idx : i[0];
    }
};

// One unit of work of a CTA: a tile of `w` cache rows starting at `col0` against query tile `m_tile`, over the
// k-blocks [kb0, kb1).  `select` tiles feed the per-row lists (reset before the first tile of a list, emitted
// after the last); the others store their partial sums for the tail kernel.
struct WorkItem {
    int m_tile, col0, w, kb0, kb1;
    int rows128;     // 128-row MMAs this item takes (256-row tiles: 1 when only the first 128 rows hold requests)
    int list;        // list index the rows' candidates go to (select tiles)
    int dump_slot;   // slot of the partial sums (tail pieces)
    bool select, reset, emit;
};

struct Schedule {
    GemmPlan plan;
    int cta, num_ctas, m_local, q, num_kb;
    long long n16;
    // ranges mode
    int col_begin, col_end, tiles, tile_w, first_w, my_groups, gran;
    // spans mode: this CTA's (cache-row tile, k-block) pairs [span0, span1) of query tile span_m
    int span0, span1, span_m;

    // gran: tile widths are multiples of it (16; 32 for pairs, whose CTAs each load half a tile in 16-row boxes)
    __device__ __forceinline__ void setup(const GemmPlan &p, int cta_, int num_ctas_, long long n_entries, int num_kb_,
                                          bool short_first_tile, int gran_ = 16) {
        plan = p;
        gran = gran_;
        cta = cta_;
        num_ctas = num_ctas_;
        num_kb = num_kb_;
        n16 = (n_entries + 15) / 16;
        m_local = cta % p.mg;
        q = cta / p.mg;
        col_begin = col_end = tiles = tile_w = first_w = my_groups = 0;
        if (p.mode == 0 && p.m_tiles > 0 && p.range16 > 0 && q < p.parts) {
            long long b = (long long)q * p.range16, e = b + p.range16;
            if (e > n16) e = n16;
            if (b > e) b = e;
            col_begin = (int)(b * 16);
            col_end = (int)(e * 16);
            const int cols = col_end - col_begin;
            // Where the select is the critical path (128-row tiles over short rows), long ranges open with a tile of
            // only kFirstTileN rows.  A list that starts empty takes in nearly every column it sees, one insertion
            // each; after a short first tile all lists of a query publish their first bounds, and the tiles that
            // follow are scanned against a bound that already covers (number of lists x kFirstTileN / 2) cache rows
            // instead of every list warming up on its own.  Elsewhere the extra tile would only lengthen the MMA
            // pipeline's serial part.
            first_w = short_first_tile && cols > 3 * kMaxTileN ? kFirstTileN : 0;
            const int rest_tiles = (cols - first_w + kMaxTileN - 1) / kMaxTileN;
            tile_w = rest_tiles > 0 ? (((cols - first_w + rest_tiles - 1) / rest_tiles + gran - 1) / gran) * gran : 0;
            tiles = rest_tiles + (first_w ? 1 : 0);
            my_groups = m_local < p.m_tiles ? (p.m_tiles - m_local + p.mg - 1) / p.mg : 0;
        }
        span0 = span1 = span_m = 0;
        int j, cm;
        if (p.mode == 3 && span_owner(p, cta, span_m, j, cm)) {
            span0 = span_begin(p, num_kb, j, cm);
            span1 = span_begin(p, num_kb, j + 1, cm);
        }
    }
    // widest tile this CTA will load (sizes the shared-memory stages)
    __device__ __forceinline__ int max_width() const { return plan.mode == 0 ? tile_w : kMaxTileN; }
    // ranges mode: first cache row and width of this CTA's t-th tile
    __device__ __forceinline__ int tile_col0(int t) const {
        return col_begin + (first_w && t ? first_w + (t - 1) * tile_w : t * tile_w);
    }
    __device__ __forceinline__ int tile_width(int t) const {
        if (first_w && t == 0) return first_w;
        // (a pair's last tile of the last range may reach up to 16 rows past the end of the cache: those columns score
        // +inf like every column past the entry count)
        const int rest = ((col_end - tile_col0(t) + gran - 1) / gran) * gran;
        return rest < tile_w ? rest : tile_w;
    }
    __device__ __forceinline__ int num_items() const {
        if (plan.m_tiles == 0 || n16 == 0) return 0;
        if (plan.mode == 0) return my_groups * tiles;
        if (plan.mode == 2) return cta < plan.pieces ? (plan.pieces - cta + num_ctas - 1) / num_ctas : 0;
        if (plan.mode == 3) return span1 > span0 ? (span1 - 1) / num_kb - span0 / num_kb + 1 : 0;
        return 1 + (cta < plan.tail_tiles * plan.tail_slices ? 1 : 0);
    }
    // wave + tail: the id-th tile in (cache-row tile, query tile) order; cache-row tiles are as even as 16-row
    // blocks allow
    __device__ __forceinline__ void tile_of(int id, WorkItem &it) const {
        const int n = id / plan.m_tiles;
        it.m_tile = id % plan.m_tiles;
        it.rows128 = 2;
        const long long b0 = n16 * n / plan.n_tiles, b1 = n16 * (n + 1) / plan.n_tiles;
        it.col0 = (int)(b0 * 16);
        it.w = (int)((b1 - b0) * 16);
        it.list = n;
    }
    // idx-th item; g and t are the caller's running (group, tile) counters in ranges mode (no divisions on the
    // hand-over path between tiles)
    __device__ __forceinline__ void item(int idx, int g, int t, WorkItem &it) const {
        it.dump_slot = 0;
        it.rows128 = 2;
        if (plan.mode == 0) {
            it.m_tile = g * plan.mg + m_local;
            it.col0 = tile_col0(t);
            it.w = tile_width(t);
            it.kb0 = 0;
            it.kb1 = num_kb;
            it.list = q;
            it.select = true;
            it.reset = t == 0;
            it.emit = t == tiles - 1;
            return;
        }
        if (plan.mode == 2) {
            const int piece = cta + idx * num_ctas;
            const int sl = piece % plan.tail_slices;
            tile_of(piece / plan.tail_slices, it);
            it.kb0 = (int)((long long)num_kb * sl / plan.tail_slices);
            it.kb1 = (int)((long long)num_kb * (sl + 1) / plan.tail_slices);
            it.select = it.reset = it.emit = false;
            it.dump_slot = piece;
            return;
        }
        if (plan.mode == 3) {
            const int n = span0 / num_kb + idx;
            tile_of(n * plan.m_tiles + span_m, it);
            it.rows128 = plan.half && span_m == plan.m_tiles - 1 ? 1 : 2;
            it.kb0 = idx == 0 ? span0 - n * num_kb : 0;
            it.kb1 = min(num_kb, span1 - n * num_kb);
            it.select = it.reset = it.emit = false;
            it.dump_slot = cta * kMaxSpanItems + idx;
            return;
        }
        if (idx == 0) {
            tile_of(cta, it);
            it.kb0 = 0;
            it.kb1 = num_kb;
            it.select = it.reset = it.emit = true;
            return;
        }
        const int j = cta / plan.tail_slices, sl = cta % plan.tail_slices;
        tile_of(num_ctas + j, it);
        it.kb0 = (int)((long long)num_kb * sl / plan.tail_slices);
        it.kb1 = (int)((long long)num_kb * (sl + 1) / plan.tail_slices);
        it.select = it.reset = it.emit = false;
        it.dump_slot = cta;
    }
};

// MSUB = 128-row MMAs per CTA tile (1 or 2).  PAIR (with MSUB = 1): the grid is launched as clusters of two CTAs that
// share every tile: 256 query rows (128 per CTA) against up to 256 cache rows, of which each CTA loads half; the MMAs
// are issued by the even CTA for both (tcgen05 cta_group::2) and leave each CTA its 128 rows of the accumulator, so the
// two accumulator buffers of a 128-row tile stay (the select overlaps the next tile's MMAs) while the operand bytes
// per flop are those of a 256 x 256 tile.  No load is multicast: each CTA fetches its own halves.
template <int KP, int MSUB, bool PAIR = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_select_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_x64,
                   const __grid_constant__ CUtensorMap tmap_x16, const float *__restrict__ norms, long long n_entries,
                   int dim, int batch_max, const int32_t *__restrict__ count_dev, int k,
                   float *__restrict__ part_score, int32_t *__restrict__ part_idx, GemmPlan *__restrict__ plan_out,
                   int32_t *row_bound, float *__restrict__ tail_dump, int32_t *__restrict__ status, int product_only) {
    constexpr int kTileRows = kTileM * MSUB * (PAIR ? 2 : 1);   // query rows per tile (of the CTA, or of the pair)
    constexpr int kATileBytes = kABytes * MSUB;
    const uint32_t rank = PAIR ? cluster_rank() : 0u;            // 0 = the CTA that issues the pair's MMAs
    const int worker = PAIR ? (int)blockIdx.x >> 1 : (int)blockIdx.x;
    const int num_workers = PAIR ? (int)gridDim.x >> 1 : (int)gridDim.x;
    constexpr int kAccBufs = MSUB == 1 ? 2 : 1;   // accumulator sets in TMEM
    constexpr int kSlots = KP;                    // bound slots per query row

    extern __shared__ unsigned char smem_raw[];
    // operand stages need 1024-byte alignment for the 128-byte swizzle
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *stage_base = smem;
    float *norm_smem = reinterpret_cast<float *>(smem + kStageRegionBytes);
    unsigned char *queue_smem = smem + kStageRegionBytes + kNormSmemBytes;
    SmemCtl *ctl = reinterpret_cast<SmemCtl *>(smem + kStageRegionBytes + kNormSmemBytes + kQueueSmemBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (dim + kBlockK - 1) / kBlockK;

    if (threadIdx.x == 0) {
        int count = count_dev ? min(*count_dev, batch_max) : batch_max;
        if (count < 0) count = 0;
        ctl->plan = product_only ? make_product_plan(count, n_entries, num_workers, kTileRows, num_kb)
                                 : make_gemm_plan(count, n_entries, num_workers, k, kTileRows, num_kb, PAIR, MSUB == 1 ? 2 : 1);
        ctl->abort_flag = 0;
        if (blockIdx.x == 0) *plan_out = ctl->plan;
    }
    __syncthreads();
    Schedule sched;
    sched.setup(ctl->plan, worker, num_workers, n_entries, num_kb, MSUB == 1 && num_kb <= 8, PAIR ? 32 : 16);
    const GemmPlan &plan = sched.plan;
    const int n_items = sched.num_items();
    if (n_items == 0) return;   // whole CTA, before any barrier
    // as many stages as fit: narrower tiles leave room for a deeper ring
    const int stage_bytes = kATileBytes + (PAIR ? sched.max_width() >> 1 : sched.max_width()) * (kBlockK * 2);
    const int num_stages = min(kMaxStages, kStageRegionBytes / stage_bytes);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&ctl->tmem_full[a], 1);
            mbar_init(&ctl->tmem_empty[a], PAIR ? 2 * kEpiThreads : kEpiThreads);   // a pair: both CTAs' epilogue threads
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        if (PAIR) {
            // the same warp of both CTAs, the same destination: the pair gets the same columns in both TMEMs
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                         "r"(kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                         "r"(kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();   // the other CTA's barriers are initialised before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    // Warpgroup 0 (all four warps at this one instruction) gives registers back before its warps take their roles;
    // the epilogue warpgroups claim theirs.
    if (warp < kRoleThreads / 32) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRoleRegs));
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t issued = 0, stage = 0, ph = 0;
            bool ok = true;
            // all k-blocks [kb0, kb1) of one tile
            auto load_tile = [&](int m_tile, int col0, int w, int kb0, int kb1, int rows128) {
                for (int kb = kb0; kb < kb1; ++kb, ++issued) {
                    if (!mbar_wait(&ctl->empty[stage], ph ^ 1, ctl, status, 1)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a_dst = smem_u32(stage_base + stage * stage_bytes);
                    const uint32_t b_dst = a_dst + kATileBytes;
                    if (PAIR) {
                        // this CTA's 128 query rows and its half of the tile's cache rows; the bytes of both CTAs are
                        // counted on the leader's barrier, which the leader alone arms
                        const int hw = w >> 1;
                        if (rank == 0) mbar_expect_tx(&ctl->full[stage], (uint32_t)(2 * kATileBytes + w * kBlockK * 2));
                        const uint32_t bar = map_to_rank(smem_u32(&ctl->full[stage]), 0);
#pragma unroll
                        for (int ms = 0; ms < MSUB; ++ms)
                            tma_load_2d_pair(a_dst + ms * kABytes, &tmap_q, bar, kb * kBlockK,
                                             m_tile * kTileRows + ((int)rank * MSUB + ms) * kTileM);
                        const int c0 = col0 + (int)rank * hw;
                        int r = 0;
                        for (; r + 64 <= hw; r += 64) tma_load_2d_pair(b_dst + r * (kBlockK * 2), &tmap_x64, bar, kb * kBlockK, c0 + r);
                        for (; r < hw; r += 16) tma_load_2d_pair(b_dst + r * (kBlockK * 2), &tmap_x16, bar, kb * kBlockK, c0 + r);
                    } else {
                        mbar_expect_tx(&ctl->full[stage], (uint32_t)((MSUB == 2 ? rows128 * kABytes : kATileBytes) + w * kBlockK * 2));
#pragma unroll
                        for (int ms = 0; ms < MSUB; ++ms)
                            if (ms < rows128)
                                tma_load_2d(a_dst + ms * kABytes, &tmap_q, &ctl->full[stage], kb * kBlockK,
                                            m_tile * kTileRows + ms * kTileM);
                        int r = 0;
                        for (; r + 64 <= w; r += 64)
                            tma_load_2d(b_dst + r * (kBlockK * 2), &tmap_x64, &ctl->full[stage], kb * kBlockK, col0 + r);
                        for (; r < w; r += 16)
                            tma_load_2d(b_dst + r * (kBlockK * 2), &tmap_x16, &ctl->full[stage], kb * kBlockK, col0 + r);
                    }
                    if (++stage == (uint32_t)num_stages) {
                        stage = 0;
                        ph ^= 1;
                    }
                }
            };
            if (plan.mode == 0) {
                for (int g = 0; g < sched.my_groups && ok; ++g)
                    for (int t = 0; t < sched.tiles && ok; ++t)
                        load_tile(g * plan.mg + sched.m_local, sched.tile_col0(t), sched.tile_width(t), 0, num_kb, MSUB);
            } else {
                for (int idx = 0; idx < n_items && ok; ++idx) {
                    WorkItem it;
                    sched.item(idx, 0, 0, it);
                    load_tile(it.m_tile, it.col0, it.w, it.kb0, it.kb1, it.rows128);
                }
            }
            if (!ok) {
                // gave up: let the copies already issued land before the CTA leaves
                uint32_t back = issued < (uint32_t)num_stages ? issued : (uint32_t)num_stages;
                uint32_t s2 = stage, p2 = ph;
                for (uint32_t j = 0; j < back; ++j) {
                    if (s2 == 0) {
                        s2 = num_stages;
                        p2 ^= 1;
                    }
                    --s2;
                    const long long t0 = clock64();
                    while (!mbar_try(&ctl->full[s2], p2))
                        if (clock64() - t0 > 40000000ll) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, ph = 0, tile_no = 0;
            bool ok = true;
            // all MMAs of one tile over the k-blocks [kb0, kb1)
            auto mma_tile = [&](int w, int kb0, int kb1, int rows128) {
                const uint32_t acc = tile_no % kAccBufs, acc_ph = (tile_no / kAccBufs) & 1;
                ++tile_no;
                if (!mbar_wait(&ctl->tmem_empty[acc], acc_ph ^ 1, ctl, status, 2)) {
                    ok = false;
                    return;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kMaxTileN;
                const uint32_t idesc = umma_instr_desc(w, PAIR ? 2 * kTileM : kTileM);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&ctl->full[stage], ph, ctl, status, 3)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(stage_base + stage * stage_bytes);
                    const uint64_t bdesc = umma_smem_desc(a_addr + kATileBytes);
#pragma unroll
                    for (int kk = 0; kk < kBlockK / 16; ++kk) {
                        if (PAIR) {
#pragma unroll
                            for (int ms = 0; ms < MSUB; ++ms)
                                umma_bf16_pair(d_tmem + ms * kMaxTileN, umma_smem_desc(a_addr + ms * kABytes) + 2 * kk,
                                               bdesc + 2 * kk, idesc, ((kb - kb0) | kk) != 0);
                        } else {
#pragma unroll
                            for (int ms = 0; ms < MSUB; ++ms)
                                if (ms < rows128)
                                    umma_bf16(d_tmem + ms * kMaxTileN, umma_smem_desc(a_addr + ms * kABytes) + 2 * kk,
                                              bdesc + 2 * kk, idesc, ((kb - kb0) | kk) != 0);
                        }
                    }
                    // frees the stage once these MMAs have read it (in both CTAs of a pair)
                    if (PAIR) umma_commit_pair(&ctl->empty[stage]);
                    else umma_commit(&ctl->empty[stage]);
                    if (++stage == (uint32_t)num_stages) {
                        stage = 0;
                        ph ^= 1;
                    }
                }
                if (ok) {
                    if (PAIR) umma_commit_pair(&ctl->tmem_full[acc]);
                    else umma_commit(&ctl->tmem_full[acc]);
                }
            };
            if (plan.mode == 0) {
                for (int g = 0; g < sched.my_groups && ok; ++g)
                    for (int t = 0; t < sched.tiles && ok; ++t)
                        mma_tile(sched.tile_width(t), 0, num_kb, MSUB);
            } else {
                for (int idx = 0; idx < n_items && ok; ++idx) {
                    WorkItem it;
                    sched.item(idx, 0, 0, it);
                    mma_tile(it.w, it.kb0, it.kb1, it.rows128);
                }
            }
        }
    } else if (warp >= kRoleThreads / 32) {
        // ------------------------------------------------------------ epilogue: per-row select
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kEpiRegs));
        const int ew = warp - kRoleThreads / 32;          // 0..7
        const int quarter = warp & 3;                     // TMEM lanes this warp may read: 32*quarter .. +31
        const int msub = MSUB == 2 ? (ew >> 2) : 0;       // which 128-row MMA this warp drains
        const int half = MSUB == 1 ? (ew >> 2) : 0;       // 128-row tiles: which 16-column chunks (even / odd)
        constexpr int kStep = MSUB == 1 ? 32 : 16;        // distance between this warp's chunks
        const int first = half * 16;
        const int row_in_tile = ((PAIR ? (int)rank * MSUB : 0) + msub) * kTileM + quarter * 32 + lane;
        const int te = threadIdx.x - kRoleThreads;        // 0..255, queue slot
        float *my_norm = norm_smem + ew * kMaxTileN;      // 256 floats: one buffer (256-row tiles) or two of 128
        // queue slots and norms are read and written through explicit shared-memory addresses
        const uint32_t q_base = smem_u32(queue_smem) + (uint32_t)te * 8u;
        TopList<KP> top;
        bool ok = true;

        // Bound shared by every CTA that scans cache rows for the same query.  A row has KP slots.
        // Ranges of 4 tiles or more (sharing 2): list l lowers slot (l + e) mod KP to its e-th best score.  The KP
        // slot values then belong to KP different cache rows (two slots filled by the same list hold different
        // entries of it; a stale entry is only larger than the current one), so their maximum bounds the KP-th
        // best score of the whole cache from above.  With many lists per query this is far tighter than any one
        // list's own KP-th best.
        // Ranges of 2 or 3 tiles (sharing 1): too short to pay for KP atomics per list; every list lowers slot 0 to
        // its KP-th best score, which is such a bound too.  Single tiles (sharing 0): nothing to share.
        // A score above the bound can be skipped by every list.  Scores equal to the bound are kept, so which
        // candidates reach the final merge never depends on the order in which CTAs publish.
        const int sharing = plan.mode != 0 || sched.tiles < 2 ? 0 : sched.tiles < 4 ? 1 : 2;
        float bound = __int_as_float(0x7F800000);

        // slot r of this thread's queue
        auto q_read = [&](int r, float &sc, int32_t &col) {
            uint32_t a, b;
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(a), "=r"(b) : "r"(q_base + (uint32_t)r * kQueueStride) : "memory");
            sc = __uint_as_float(a);
            col = (int32_t)b;
        };
        // append; what does not fit lands in the spare slot and is found again by rescanning the columns
        auto q_push = [&](int &cnt, float sc, int32_t col) {
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(q_base + (uint32_t)min(cnt, kQueueCap) * kQueueStride),
                         "r"(__float_as_uint(sc)), "r"(col)
                         : "memory");
            ++cnt;
        };
        // insert the first n queued candidates of every lane, all lanes together
        auto flush = [&](int n) {
            const int rounds = __reduce_max_sync(0xFFFFFFFFu, n);
            for (int r = 0; r < rounds; ++r) {
                if (r < n) {
                    float sc;
                    int32_t col;
                    q_read(r, sc, col);
                    if (sc < top.s[KP - 1] && sc <= bound) top.insert(sc, col);
                }
            }
        };
        // the same for one lane on its own (other lanes idle meanwhile)
        auto drain = [&](int n) {
            for (int r = 0; r < n; ++r) {
                float sc;
                int32_t col;
                q_read(r, sc, col);
                if (sc < top.s[KP - 1] && sc <= bound) top.insert(sc, col);
            }
        };

        uint32_t tile_no = 0;

        // What a tile's scan needs from global memory: the row's bound slots and the squared norms of the tile's
        // columns.  With 128-row tiles the epilogue is the critical path, so both are fetched a tile ahead (the slots
        // into registers before the previous tile's queue is drained, the norms by asynchronous copies into the
        // other half of the norm buffer while the previous tile is scanned); only a CTA's first tile, and 256-row
        // tiles (whose scan waits for the MMAs anyway and whose norms fill the buffer), fetch them on the spot.
        // (long lists keep too many slots to hold them in registers across a drain: those are read on the spot)
        constexpr bool kSlotsAhead = KP <= 8;
        int32_t slot_regs[kSlots];   // raw slot values of the next tile's row (slot_regs[0] alone when one slot is shared)
        bool fetched_ahead = false;

        // the row's slots, read past L1 (other SMs lower them)
        auto load_slots = [&](int m_tile, int sharing) {
            const int32_t *my_bound = row_bound + (long long)(m_tile * kTileRows + row_in_tile) * kSlots;
            if (sharing == 1) {
                asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(slot_regs[0]) : "l"(my_bound) : "memory");
            } else if (sharing == 2) {
#pragma unroll
                for (int e = 0; e < kSlots; e += 4)
                    asm volatile("ld.relaxed.gpu.global.v4.s32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(slot_regs[e]), "=r"(slot_regs[e + 1]), "=r"(slot_regs[e + 2]), "=r"(slot_regs[e + 3])
                                 : "l"(my_bound + e)
                                 : "memory");
            }
        };
        // the bound is the largest of the slots
        auto slots_bound = [&](int sharing) -> int32_t {
            if (sharing == 1) return slot_regs[0];
            if (sharing != 2) return 0x7F7F7F7F;
            int32_t key = (int32_t)0x80000000;
#pragma unroll
            for (int e = 0; e < kSlots; e += 4)
                key = max(max(key, max(slot_regs[e], slot_regs[e + 1])), max(slot_regs[e + 2], slot_regs[e + 3]));
            return key;
        };
        // squared norms of this warp's columns, chunk after chunk; rows past the end of the cache get +inf and
        // never enter a list
        // (a warp scans its chunks two at a time; an odd last chunk is paired with a chunk of +inf)
        auto stage_norms = [&](float *nrm, int col0, int w, bool async) {
            const int nch = (w - first + kStep - 1) / kStep;   // this warp's chunks
            const float inf = __int_as_float(0x7F800000);
            // four norms (16 bytes) per lane and round: a chunk is four lanes wide
            for (int u = lane; u < ((nch + 1) >> 1) * 8; u += 32) {
                const int c = first + (u >> 2) * kStep + (u & 3) * 4;
                const uint32_t dst = smem_u32(nrm + u * 4);
                const long long g = (long long)col0 + c;
                if ((u >> 2) >= nch || g >= n_entries) {
                    asm volatile("st.shared.v4.f32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "f"(inf) : "memory");
                } else if (g + 3 < n_entries) {
                    if (async) {
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(norms + g) : "memory");
                    } else {
                        const float4 v = __ldg(reinterpret_cast<const float4 *>(norms + g));
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                                     : "memory");
                    }
                } else {
                    // the cache ends inside these four columns
                    for (int e = 0; e < 4; ++e) nrm[u * 4 + e] = g + e < n_entries ? __ldg(norms + g + e) : inf;
                }
            }
        };

        // scan one accumulator tile into the running list of this thread's row; (nx_m_tile, nx_col0, nx_w) is the
        // tile this warp scans next (nx_w = 0: none)
        auto select_tile = [&](int m_tile, int col0, int w, int list, int sharing, int nx_m_tile, int nx_col0, int nx_w,
                               bool fresh_slots) {
            const uint32_t acc = tile_no % kAccBufs, acc_ph = (tile_no / kAccBufs) & 1;
            ++tile_no;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (acc + msub) * kMaxTileN;
            int32_t *my_bound = row_bound + (long long)(m_tile * kTileRows + row_in_tile) * kSlots;
            float *nrm = my_norm + acc * (kMaxTileN / 2);   // acc is 0 for 256-row tiles
            if (!fetched_ahead) {
                load_slots(m_tile, sharing);
                stage_norms(nrm, col0, w, false);
            } else {
                if (!kSlotsAhead) load_slots(m_tile, sharing);
                asm volatile("cp.async.wait_all;" ::: "memory");
            }
            __syncwarp();
            // the whole warp takes the same decision, so its lanes stay together for the TMEM loads
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(&ctl->tmem_full[acc], acc_ph, ctl, status, 4));
            if (!ok) return;
            tc_fence_after();
            if (fresh_slots) load_slots(m_tile, sharing);
            const int32_t bound_key = slots_bound(sharing);
            fetched_ahead = MSUB == 1 && nx_w > 0;
            if (fetched_ahead) stage_norms(my_norm + (acc ^ 1) * (kMaxTileN / 2), nx_col0, nx_w, true);
            bound = key_float(bound_key);
            float thr = fminf(top.s[KP - 1], bound);   // pre-filter: nothing above it can enter the list
            int cnt = 0;

            const uint32_t nrm_addr = smem_u32(nrm);
            const int nch = (w - first + kStep - 1) / kStep;   // this warp's chunks of 16 columns
            const int npairs = (nch + 1) >> 1;

            // Two chunks (32 columns) per step: all loads and the 32 score FMAs are independent, one min-tree
            // decides whether any column can enter the list.  The rare rest is lane-local: only the groups of four
            // columns that hold a passing score are walked, the passing columns are queued, and a lane whose queue
            // overflows inserts what it had queued, tightens its threshold and walks the step again.
            // TMEM loads of pair p; a missing second chunk reads the first again (its norms are +inf)
            auto issue = [&](uint32_t (&v0)[16], uint32_t (&v1)[16], int p) {
                const int ca = first + 2 * p * kStep;
                const int cb = 2 * p + 1 < nch ? ca + kStep : ca;
                __syncwarp();
                tmem_ld16(taddr + ca, v0);
                tmem_ld16(taddr + cb, v1);
            };
            // one register buffer: the loads of the next step are issued as soon as this step's scores are formed
            // and are in flight while they are examined
            uint32_t v0[16], v1[16];
            if (npairs > 0) issue(v0, v1, 0);
            for (int p = 0; p < npairs; ++p) {
                const int ca = first + 2 * p * kStep;                 // first chunk of the pair
                const int cb = ca + kStep;                            // second chunk (columns of +inf when past the tile)
                float sc[32];
                tmem_ld_wait(v0);
                tmem_ld_wait(v1);
#pragma unroll
                for (int q4 = 0; q4 < 8; ++q4) {
                    float n0, n1, n2, n3;
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                 : "=f"(n0), "=f"(n1), "=f"(n2), "=f"(n3)
                                 : "r"(nrm_addr + (uint32_t)(p * 32 + q4 * 4) * 4u));
                    const uint32_t *v = q4 < 4 ? &v0[q4 * 4] : &v1[(q4 - 4) * 4];
                    sc[q4 * 4 + 0] = fmaf(-2.f, __uint_as_float(v[0]), n0);
                    sc[q4 * 4 + 1] = fmaf(-2.f, __uint_as_float(v[1]), n1);
                    sc[q4 * 4 + 2] = fmaf(-2.f, __uint_as_float(v[2]), n2);
                    sc[q4 * 4 + 3] = fmaf(-2.f, __uint_as_float(v[3]), n3);
                }
                if (p + 1 < npairs) issue(v0, v1, p + 1);
                float gm[8];
#pragma unroll
                for (int g = 0; g < 8; ++g) gm[g] = fminf(fmin3(sc[4 * g], sc[4 * g + 1], sc[4 * g + 2]), sc[4 * g + 3]);
                const float mn = fminf(fmin3(gm[0], gm[1], gm[2]), fminf(fmin3(gm[3], gm[4], gm[5]), fminf(gm[6], gm[7])));
                if (mn <= thr) {
                    const int cnt0 = cnt;
                    auto walk = [&]() {
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            if (gm[g] <= thr) {
#pragma unroll
                                for (int jj = 0; jj < 4; ++jj) {
                                    const int j = 4 * g + jj;
                                    if (sc[j] <= thr) q_push(cnt, sc[j], col0 + (j < 16 ? ca + j : cb + j - 16));
                                }
                            }
                        }
                    };
                    // no threshold yet (the list is not full and no bound is known): every column passes, so
                    // queueing them would only overflow
                    bool direct = !(thr < __int_as_float(0x7F800000));
                    int pending = cnt0;
                    if (!direct) {
                        walk();
                        if (cnt > kQueueCap) {
                            drain(cnt0);
                            pending = 0;
                            thr = fminf(top.s[KP - 1], bound);
                            cnt = 0;
                            walk();
                            direct = cnt > kQueueCap;   // still too many: the list is filling up
                        }
                    }
                    if (direct) {
                        // insert column by column; arrival order, hence the tie order, is kept
                        drain(pending);
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (sc[j] < top.s[KP - 1] && sc[j] <= bound) top.insert(sc[j], col0 + (j < 16 ? ca + j : cb + j - 16));
                        cnt = 0;
                        thr = fminf(top.s[KP - 1], bound);
                    }
                }
            }
            __syncwarp();
            tc_fence_before();
            if (PAIR) mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->tmem_empty[acc]), 0));   // the leader's barrier
            else mbar_arrive(&ctl->tmem_empty[acc]);
            if (kSlotsAhead && fetched_ahead) load_slots(nx_m_tile, sharing);   // in flight while the queue is drained
            // after the accumulator is released: the MMAs of the next tile can start meanwhile
            if (__any_sync(0xFFFFFFFFu, cnt > 0)) flush(cnt);
            // publish this list where it changed
            if (cnt > 0 && sharing == 1) {
                if (top.s[KP - 1] < bound) atomicMin(my_bound, float_key(top.s[KP - 1]));
            } else if (cnt > 0 && sharing == 2) {
#pragma unroll
                for (int e = 0; e < KP; ++e)
                    if (top.s[e] <= bound) atomicMin(my_bound + ((list + e) & (KP - 1)), float_key(top.s[e]));
            }
            __syncwarp();
        };

        // write this thread's list as list number `list` of its row
        auto emit_list = [&](int m_tile, int list) {
            const int row = m_tile * kTileRows + row_in_tile;
            if (row < plan.count) {
                const long long o = ((long long)row * plan.lists + list) * KP;
#pragma unroll
                for (int e = 0; e < KP; ++e) {
                    part_score[o + e] = top.s[e];
                    part_idx[o + e] = top.i[e];
                }
            }
        };

        // a piece of a tile: store the partial sums, column-major so that the 32 rows of a warp coalesce
        auto dump_tile = [&](const WorkItem &it) {
            const uint32_t acc = tile_no % kAccBufs, acc_ph = (tile_no / kAccBufs) & 1;
            ++tile_no;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (acc + msub) * kMaxTileN;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(&ctl->tmem_full[acc], acc_ph, ctl, status, 5));
            if (!ok) return;
            tc_fence_after();
            float *dst = tail_dump + ((long long)it.dump_slot * kMaxTileN) * kTileRows + row_in_tile;
            // (the warps of a 128-row half that took no MMA only keep the barrier counts)
            for (int c0 = first; c0 < it.w && msub < it.rows128; c0 += kStep) {
                uint32_t v[16];
                __syncwarp();
                tmem_ld16(taddr + c0, v);
                tmem_ld_wait(v);
#pragma unroll
                for (int j = 0; j < 16; ++j) dst[(long long)(c0 + j) * kTileRows] = __uint_as_float(v[j]);
            }
            tc_fence_before();
            if (PAIR) mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->tmem_empty[acc]), 0));   // the leader's barrier
            else mbar_arrive(&ctl->tmem_empty[acc]);
            __syncwarp();
        };

        if (plan.mode == 0) {
            for (int g = 0; g < sched.my_groups && ok; ++g) {
                const int m_tile = g * plan.mg + sched.m_local;
                top.reset();
                for (int t = 0; t < sched.tiles && ok; ++t) {
                    const bool last_t = t + 1 == sched.tiles;
                    const int nx_t = last_t ? 0 : t + 1;
                    const int nx_w = last_t && g + 1 == sched.my_groups ? 0 : sched.tile_width(nx_t);
                    // while the lists of a query are young their bounds move fast: read the slots as late as possible
                    select_tile(m_tile, sched.tile_col0(t), sched.tile_width(t), MSUB == 1 ? sched.q * 2 + half : sched.q,
                                sharing, last_t ? m_tile + plan.mg : m_tile, sched.tile_col0(nx_t), nx_w, t < 3);
                }
                if (ok) emit_list(m_tile, MSUB == 1 ? sched.q * 2 + half : sched.q);
            }
        } else if (plan.mode == 1) {
            WorkItem it;
            sched.item(0, 0, 0, it);
            top.reset();
            select_tile(it.m_tile, it.col0, it.w, it.list, 0, 0, 0, 0, false);
            if (ok) emit_list(it.m_tile, it.list);
            if (ok && n_items > 1) {
                sched.item(1, 0, 0, it);
                dump_tile(it);
            }
        } else {
            for (int idx = 0; idx < n_items && ok; ++idx) {
                WorkItem it;
                sched.item(idx, 0, 0, it);
                dump_tile(it);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();   // neither CTA frees its TMEM or leaves while the other may still use it
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// Wave + tail and spans modes: add up the pieces of a tile in their order (the sum does not depend on timing), turn
// the dot products into scores and select per row.  A CTA takes 32 query rows of one tile and one warp per share of
// the tile's columns (a warp reads 128 contiguous bytes of the column-major partial sums per column; with a share of
// 16 columns per thread the loads of one piece are all in flight at once, and there are enough threads to cover the
// latency of memory).
//
// Lists of up to 8 entries (16 shares of 16 columns): no thread sorts anything.  The smallest scores of the 16 shares
// of a row are 16 different columns, so the KP-th smallest of them bounds the row's KP-th best score from above; it is
// found by counting (every thread ranks its own minimum among the row's 16).  The few columns at or below that bound
// (KP of them at least) go to a per-row queue in shared memory, every queued column ranks itself among the row's queue
// by (score, column) and the first KP write themselves to their place in the list.  A row whose queue overflows (many
// equal scores, or a tile so narrow that fewer than KP shares hold columns) is scanned again by one thread, column
// after column.
// Longer lists (8 or 4 shares): every thread keeps a list over its share, and the shares' lists of a row are merged
// pairwise, neighbours first, through shared memory, so equal scores keep the order a single scan would give them.
template <int KP>
struct PieceSplit {
    static constexpr int value = KP <= 8 ? 16 : KP == 16 ? 8 : 4;
};
constexpr int kPieceRowGroups = 2 * kTileM / 32;   // CTAs per tile
constexpr int kPieceQueue = 64;                    // queued columns per row (short lists)

template <int KP>
struct PieceSmem {
    static constexpr int kSplit = PieceSplit<KP>::value;
    // short lists: the shares' minima and the queues; long lists: the lists on their way through the merge
    static constexpr int kFloats = KP <= 8 ? kSplit * 32 + 2 * kPieceQueue * 32 : 2 * kSplit * KP * 32;
};

template <int KP>
__global__ void __launch_bounds__(32 * PieceSplit<KP>::value, KP <= 8 ? 2 : 1)
piece_select_kernel(const GemmPlan *__restrict__ plan_dev, int num_ctas, int num_kb, const float *__restrict__ dump,
                    const float *__restrict__ norms, long long n_entries, float *__restrict__ part_score,
                    int32_t *__restrict__ part_idx) {
    constexpr int kSplit = PieceSplit<KP>::value;
    constexpr int kRows = 2 * kTileM;
    constexpr int kShareCols = kMaxTileN / kSplit;
    __shared__ float smem_f[PieceSmem<KP>::kFloats];
    __shared__ int piece_info[4];   // slot of the first piece, slot of the second, CTA of the first, CTA of the last
    __shared__ int queue_len[32];
    __shared__ float row_thr[32];
    const GemmPlan plan = *plan_dev;
    if (plan.mode != 1 && plan.mode != 3) return;
    const int lane = threadIdx.x & 31, share = threadIdx.x >> 5;
    const int rg = blockIdx.x % kPieceRowGroups;
    const long long n16 = (n_entries + 15) / 16;
    const float inf = __int_as_float(0x7F800000);
    for (int t = blockIdx.x / kPieceRowGroups; t < plan.tail_tiles; t += gridDim.x / kPieceRowGroups) {
        int n, m_tile;
        if (plan.mode == 1) {
            const int id = num_ctas + t;
            n = id / plan.m_tiles;
            m_tile = id - n * plan.m_tiles;
        } else {
            m_tile = t / plan.n_tiles;
            n = t - m_tile * plan.n_tiles;
        }
        const int rows128 = plan.mode == 3 && plan.half && m_tile == plan.m_tiles - 1 ? 1 : 2;
        if (rg * 32 >= rows128 * kTileM || m_tile * kRows + rg * 32 >= plan.count) continue;   // whole CTA: no request here
        // the pieces of this tile: slot of piece j is j == 0 ? first : second + (j - 1) * stride
        int stride, pieces;
        __syncthreads();
        if (share == 0) {
            queue_len[lane] = 0;
            row_thr[lane] = inf;
        }
        if (plan.mode == 1) {
            stride = 1;
            pieces = plan.tail_slices;
            if (threadIdx.x == 0) {
                piece_info[0] = t * plan.tail_slices;
                piece_info[1] = t * plan.tail_slices + 1;
            }
            __syncthreads();
        } else {
            // spans are not empty and follow one another: the tile's pieces are those of the query tile's CTAs from
            // the one whose span holds the tile's first k-block to the one whose span holds its last
            stride = kMaxSpanItems;
            int first_cta, cm;
            span_ctas_of(plan, m_tile, first_cta, cm);
            const int p_lo = n * num_kb, p_hi = p_lo + num_kb;
            for (int j = threadIdx.x; j < cm; j += blockDim.x) {
                const int b0 = span_begin(plan, num_kb, j, cm), b1 = span_begin(plan, num_kb, j + 1, cm);
                if (b0 <= p_lo && p_lo < b1) {
                    piece_info[0] = (first_cta + j) * kMaxSpanItems + (n - b0 / num_kb);
                    piece_info[1] = (first_cta + j + 1) * kMaxSpanItems;
                    piece_info[2] = j;
                }
                if (b0 < p_hi && p_hi <= b1) piece_info[3] = j;
            }
            __syncthreads();
            pieces = piece_info[3] - piece_info[2] + 1;
        }
        const int slot0 = piece_info[0], slot1 = piece_info[1];
        const long long b0 = n16 * n / plan.n_tiles, b1 = n16 * (n + 1) / plan.n_tiles;
        const int col0 = (int)(b0 * 16), w = (int)((b1 - b0) * 16);
        const int row_in_tile = rg * 32 + lane;
        const int row = m_tile * kRows + row_in_tile;
        const long long out = ((long long)row * plan.lists + n) * KP;
        auto piece_ptr = [&](int pc, int c0) {
            return dump + ((long long)(pc == 0 ? slot0 : slot1 + (pc - 1) * stride) * kMaxTileN + c0) * kRows + row_in_tile;
        };
        // scores of the 16 columns from c0 on; two pieces' loads in flight, the sums still taken piece after piece
        auto scores16 = [&](int c0, float (&sc)[16]) {
            float dot[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) dot[j] = 0.f;
            int pc = 0;
            for (; pc + 2 <= pieces; pc += 2) {
                const float *pa = piece_ptr(pc, c0), *pb = piece_ptr(pc + 1, c0);
                float va[16], vb[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) va[j] = __ldg(pa + j * kRows);
#pragma unroll
                for (int j = 0; j < 16; ++j) vb[j] = __ldg(pb + j * kRows);
#pragma unroll
                for (int j = 0; j < 16; ++j) dot[j] = (dot[j] + va[j]) + vb[j];
            }
            if (pc < pieces) {
                const float *pa = piece_ptr(pc, c0);
#pragma unroll
                for (int j = 0; j < 16; ++j) dot[j] += __ldg(pa + j * kRows);
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int c = col0 + c0 + j;
                const float nrm = (long long)c < n_entries ? __ldg(norms + c) : inf;
                sc[j] = fmaf(-2.f, dot[j], nrm);
            }
        };
        if constexpr (KP <= 8) {
            float *mins = smem_f;                                                  // [share][row]
            float *queue_s = smem_f + kSplit * 32;                                 // [entry][row]
            int32_t *queue_i = reinterpret_cast<int32_t *>(queue_s + kPieceQueue * 32);
            const int c0 = share * 16;
            float sc[16];
            float mine = inf;
            if (c0 < w) {
                scores16(c0, sc);
#pragma unroll
                for (int j = 0; j < 16; ++j) mine = fminf(mine, sc[j]);
            }
            mins[share * 32 + lane] = mine;
            __syncthreads();
            // rank of this share's minimum among the row's 16 (equal minima: the lower share first)
            int below = 0;
#pragma unroll
            for (int s2 = 0; s2 < kSplit; ++s2) {
                const float o = mins[s2 * 32 + lane];
                below += (o < mine || (o == mine && s2 < share)) ? 1 : 0;
            }
            if (below == KP - 1) row_thr[lane] = mine;
            __syncthreads();
            const float thr = row_thr[lane];
            if (c0 < w) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (sc[j] <= thr && sc[j] < inf) {
                        const int e = atomicAdd(&queue_len[lane], 1);
                        if (e < kPieceQueue) {
                            queue_s[e * 32 + lane] = sc[j];
                            queue_i[e * 32 + lane] = col0 + c0 + j;
                        }
                    }
                }
            }
            __syncthreads();
            const int queued = queue_len[lane];
            if (row < plan.count) {
                if (queued <= kPieceQueue) {
                    for (int e = share; e < queued; e += kSplit) {
                        const float ms = queue_s[e * 32 + lane];
                        const int32_t mi = queue_i[e * 32 + lane];
                        int rank = 0;
                        for (int o = 0; o < queued; ++o) {
                            const float os = queue_s[o * 32 + lane];
                            rank += (os < ms || (os == ms && queue_i[o * 32 + lane] < mi)) ? 1 : 0;
                        }
                        if (rank < KP) {
                            part_score[out + rank] = ms;
                            part_idx[out + rank] = mi;
                        }
                    }
                    if (share < KP && share >= queued) {   // fewer columns than list entries
                        part_score[out + share] = inf;
                        part_idx[out + share] = -1;
                    }
                } else if (share == 0) {
                    TopList<KP> top;
                    top.reset();
                    for (int c1 = 0; c1 < w; c1 += 16) {
                        float s1[16];
                        scores16(c1, s1);
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (s1[j] < top.s[KP - 1]) top.insert(s1[j], col0 + c1 + j);
                    }
#pragma unroll
                    for (int e = 0; e < KP; ++e) {
                        part_score[out + e] = top.s[e];
                        part_idx[out + e] = top.i[e];
                    }
                }
            }
        } else {
            float *list_s = smem_f;                                                            // [share][entry][row]
            int32_t *list_i = reinterpret_cast<int32_t *>(smem_f + kSplit * KP * 32);
            TopList<KP> top;
            top.reset();
            for (int c0 = share * kShareCols; c0 < min(w, (share + 1) * kShareCols); c0 += 16) {
                float sc[16];
                scores16(c0, sc);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (sc[j] < top.s[KP - 1]) top.insert(sc[j], col0 + c0 + j);
            }
            // merge neighbours first: the incoming list always holds the higher columns
            for (int s2 = 1; s2 < kSplit; s2 <<= 1) {
                if ((share & (2 * s2 - 1)) == s2) {
#pragma unroll
                    for (int e = 0; e < KP; ++e) {
                        list_s[(share * KP + e) * 32 + lane] = top.s[e];
                        list_i[(share * KP + e) * 32 + lane] = top.i[e];
                    }
                }
                __syncthreads();
                if ((share & (2 * s2 - 1)) == 0) {
#pragma unroll
                    for (int e = 0; e < KP; ++e) {
                        const float sc = list_s[((share + s2) * KP + e) * 32 + lane];
                        if (sc < top.s[KP - 1]) top.insert(sc, list_i[((share + s2) * KP + e) * 32 + lane]);
                    }
                }
            }
            if (share == 0 && row < plan.count) {
#pragma unroll
                for (int e = 0; e < KP; ++e) {
                    part_score[out + e] = top.s[e];
                    part_idx[out + e] = top.i[e];
                }
            }
        }
    }
}

// Plain product, step 2: add up the pieces of every 256 x 256 tile in their order, add the bias, apply the
// rectifier and round to bf16 (round to nearest even).  Grid (tiles, 16 column groups), one row per thread; a thread
// writes 16 consecutive outputs of its row (32 bytes).
__global__ void __launch_bounds__(2 * kTileM)
product_reduce_kernel(const GemmPlan *__restrict__ plan_dev, const float *__restrict__ dump, const float *__restrict__ bias,
                      long long n_rows, __nv_bfloat16 *__restrict__ y, long long ld_y) {
    const GemmPlan plan = *plan_dev;
    if (plan.mode != 2) return;
    constexpr int kRows = 2 * kTileM;
    const long long n16 = (n_rows + 15) / 16;
    for (int tile = blockIdx.x; tile < plan.tail_tiles; tile += gridDim.x) {
        const int n = tile / plan.m_tiles, m_tile = tile % plan.m_tiles;
        const long long b0 = n16 * n / plan.n_tiles, b1 = n16 * (n + 1) / plan.n_tiles;
        const int col0 = (int)(b0 * 16), w = (int)((b1 - b0) * 16);
        const int c0 = blockIdx.y * 16;
        if (c0 >= w) continue;
        const float *base = dump + ((long long)tile * plan.tail_slices * kMaxTileN + c0) * kRows + threadIdx.x;
        float dot[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) dot[j] = 0.f;
        for (int sl = 0; sl < plan.tail_slices; ++sl) {
            const float *p = base + (long long)sl * kMaxTileN * kRows;
#pragma unroll
            for (int j = 0; j < 16; ++j) dot[j] += p[j * kRows];
        }
        const int row = m_tile * kRows + threadIdx.x;
        if (row >= plan.count) continue;
        __align__(16) __nv_bfloat16 out[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int c = col0 + c0 + j;
            const float v = (long long)c < n_rows ? dot[j] + __ldg(bias + c) : 0.f;
            out[j] = __float2bfloat16_rn(fmaxf(v, 0.f));
        }
        uint4 *dst = reinterpret_cast<uint4 *>(y + (long long)row * ld_y + col0 + c0);
        dst[0] = reinterpret_cast<const uint4 *>(out)[0];
        dst[1] = reinterpret_cast<const uint4 *>(out)[1];
    }
}

// Exercises the bounded wait on purpose: one thread waits on a barrier that nothing will ever complete, with a
// short limit, and must come back with the status word set instead of hanging.
__global__ void wait_selftest_kernel(long long limit_cycles, int32_t *status) {
    __shared__ SmemCtl ctl;
    if (threadIdx.x == 0) {
        ctl.abort_flag = 0;
        mbar_init(&ctl.full[0], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(&ctl.full[0], 0, &ctl, status, 9, limit_cycles);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 matrix [rows x dim], row pitch ld elements; box = box_rows x 64 elements, 128-byte swizzle, zero fill
fi_status_t encode_bf16_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t dim, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) {
        set_error("cuTensorMapEncodeTiled is not available from this driver");
        return FI_ERR_UNSUPPORTED;
    }
    cuuint64_t gdim[2] = {dim, rows > 0 ? rows : 1};
    cuuint64_t gstride[1] = {ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed with code %d (base %p rows %llu dim %llu ld %llu)", (int)r, base,
                  (unsigned long long)rows, (unsigned long long)dim, (unsigned long long)ld);
        return FI_ERR_CUDA;
    }
    return FI_OK;
}

// One-time set-up of a kernel instantiation: shared-memory reservation, and the proof that the register shares its
// warpgroups claim (setmaxnreg) fit what a launch of kGemmThreads threads is given.  Registers are handed out in
// units of 8 per thread; a kernel compiled to fewer registers than the split assumes must never be launched.
template <typename Kern>
fi_status_t prepare_gemm_kernel(Kern kern, const char *what) {
    cudaFuncAttributes attr;
    if (cudaFuncGetAttributes(&attr, kern) != cudaSuccess) {
        set_error("cannot query the attributes of the %s", what);
        cudaGetLastError();
        return FI_ERR_CUDA;
    }
    const int allocated = (attr.numRegs + 7) / 8 * 8;
    if (allocated * kGemmThreads < kRoleThreads * kRoleRegs + kEpiThreads * kEpiRegs) {
        set_error("%s: compiled to %d registers per thread, too few for its register split", what, attr.numRegs);
        return FI_ERR_UNSUPPORTED;
    }
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes) != cudaSuccess) {
        set_error("cannot reserve %d bytes of shared memory for the %s", kGemmSmemBytes, what);
        cudaGetLastError();
        return FI_ERR_CUDA;
    }
    return FI_OK;
}

template <int KP, int MSUB>
fi_status_t launch_kp(fi_cache *c, const CUtensorMap &tq, int32_t batch_max, const int32_t *count_dev, bool tail_possible,
                      cudaStream_t stream) {
    auto kern = gemm_select_kernel<KP, MSUB>;   // prepared for this device by prepare_gemm_kernels (fi_cache_create)
    // every bound starts at a huge finite value (0x7F7F7F7F as a float is 3.4e38)
    if (cudaMemsetAsync(c->row_bound, 0x7F, ((size_t)batch_max + 256) * KP * sizeof(int32_t), stream) != cudaSuccess) {
        set_error("cannot reset the row bounds");
        cudaGetLastError();
        return FI_ERR_CUDA;
    }
    kern<<<c->sm_count, kGemmThreads, kGemmSmemBytes, stream>>>(tq, c->tmap_rows64, c->tmap_rows16, c->norms,
                                                               (long long)c->size, c->cfg.dim, batch_max, count_dev,
                                                               c->cfg.k, c->part_score, c->part_idx, c->plan_dev,
                                                               c->row_bound, c->tail_dump, c->status_dev, 0);
    count_launch();
    fi_status_t st = check_launch("gemm_select_kernel");
    if (st != FI_OK || !tail_possible) return st;
    // the piece kernel reads the plan the GEMM wrote and returns at once when that plan left no pieces
    const int num_kb = (c->cfg.dim + kBlockK - 1) / kBlockK;
    piece_select_kernel<KP><<<kPieceRowGroups * c->sm_count, 32 * PieceSplit<KP>::value, 0, stream>>>(
        c->plan_dev, c->sm_count, num_kb, c->tail_dump, c->norms, (long long)c->size, c->part_score, c->part_idx);
    count_launch();
    return check_launch("piece_select_kernel");
}

// The pair kernel: clusters of two CTAs, one pair per two SMs.
template <int KP, int MSUB>
fi_status_t launch_pair_kp(fi_cache *c, const CUtensorMap &tq, int32_t batch_max, const int32_t *count_dev, cudaStream_t stream) {
    auto kern = gemm_select_kernel<KP, MSUB, true>;
    if (cudaMemsetAsync(c->row_bound, 0x7F, ((size_t)batch_max + 512) * KP * sizeof(int32_t), stream) != cudaSuccess) {
        set_error("cannot reset the row bounds");
        cudaGetLastError();
        return FI_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)(c->sm_count & ~1), 1, 1);
    cfg.blockDim = dim3(kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = kGemmSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float *norms = c->norms;
    long long n = (long long)c->size;
    int dim = c->cfg.dim, k = c->cfg.k, zero = 0;
    float *tail = c->tail_dump;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tq, c->tmap_rows64, c->tmap_rows16, norms, n, dim, (int)batch_max, count_dev, k,
                                       c->part_score, c->part_idx, c->plan_dev, c->row_bound, tail, c->status_dev, zero);
    count_launch();
    if (e != cudaSuccess) {
        set_error("gemm_select_kernel (pairs): %s", cudaGetErrorString(e));
        cudaGetLastError();
        return FI_ERR_CUDA;
    }
    return check_launch("gemm_select_kernel (pairs)");
}

template <int MSUB>
fi_status_t launch_pair(fi_cache *c, const CUtensorMap &tq, int32_t batch_max, const int32_t *count_dev, cudaStream_t stream) {
    switch (gemm_list_len(c->cfg.k)) {
        case 4: return launch_pair_kp<4, MSUB>(c, tq, batch_max, count_dev, stream);
        case 8: return launch_pair_kp<8, MSUB>(c, tq, batch_max, count_dev, stream);
        case 16: return launch_pair_kp<16, MSUB>(c, tq, batch_max, count_dev, stream);
        default: return launch_pair_kp<32, MSUB>(c, tq, batch_max, count_dev, stream);
    }
}

template <int MSUB>
fi_status_t launch_msub(fi_cache *c, const CUtensorMap &tq, int32_t batch_max, const int32_t *count_dev, bool tail_possible,
                        cudaStream_t stream) {
    switch (gemm_list_len(c->cfg.k)) {
        case 4: return launch_kp<4, MSUB>(c, tq, batch_max, count_dev, tail_possible, stream);
        case 8: return launch_kp<8, MSUB>(c, tq, batch_max, count_dev, tail_possible, stream);
        case 16: return launch_kp<16, MSUB>(c, tq, batch_max, count_dev, tail_possible, stream);
        default: return launch_kp<32, MSUB>(c, tq, batch_max, count_dev, tail_possible, stream);
    }
}

}  // namespace

// Query rows per CTA tile: 256 when the batch can fill it and a tile's k-loop is long enough (>= 16 k-blocks) to
// outweigh the select that can no longer overlap it (measured: at 16 k-blocks the halved operand traffic wins by 8 %,
// at 8 k-blocks the two are level); 128 otherwise.
int gemm_tile_m(int batch_max, int dim) { return (batch_max > kTileM && dim >= 16 * kBlockK) ? 2 * kTileM : kTileM; }

fi_status_t launch_wait_selftest(fi_cache *c, long long limit_cycles, cudaStream_t stream) {
    wait_selftest_kernel<<<1, 32, 0, stream>>>(limit_cycles, c->status_dev);
    count_launch();
    return check_launch("wait_selftest_kernel");
}

// The maps cover all `capacity` rows and are encoded once, at create: the kernels are told how many rows count
// (columns past that number get an infinite score), so appending entries never touches the maps.
fi_status_t ensure_tensor_maps(fi_cache *c) {
    if (c->tmaps_ready) return FI_OK;
    fi_status_t st = encode_bf16_map(&c->tmap_rows64, c->rows, (uint64_t)c->cfg.capacity, (uint64_t)c->cfg.dim, (uint64_t)c->cfg.dim, 64);
    if (st != FI_OK) return st;
    st = encode_bf16_map(&c->tmap_rows16, c->rows, (uint64_t)c->cfg.capacity, (uint64_t)c->cfg.dim, (uint64_t)c->cfg.dim, 16);
    if (st != FI_OK) return st;
    c->tmaps_ready = true;
    return FI_OK;
}

// Every instantiation of the distance GEMM is prepared once per device (the shared-memory reservation is a
// per-device attribute), under a lock, before the first cache on that device can launch one.
fi_status_t prepare_gemm_kernels(int device) {
    static std::mutex mu;
    static bool done[kMaxDevices] = {};
    if (device < 0 || device >= kMaxDevices) {
        set_error("device ordinal %d outside 0..%d", device, kMaxDevices - 1);
        return FI_ERR_INVALID_ARG;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (done[device]) return FI_OK;
    fi_status_t st = FI_OK;
    auto prep = [&](auto kern) {
        if (st == FI_OK) st = prepare_gemm_kernel(kern, "distance GEMM");
    };
    prep(gemm_select_kernel<4, 1>);
    prep(gemm_select_kernel<8, 1>);
    prep(gemm_select_kernel<16, 1>);
    prep(gemm_select_kernel<32, 1>);
    prep(gemm_select_kernel<4, 2>);
    prep(gemm_select_kernel<8, 2>);
    prep(gemm_select_kernel<16, 2>);
    prep(gemm_select_kernel<32, 2>);
    prep(gemm_select_kernel<4, 1, true>);
    prep(gemm_select_kernel<8, 1, true>);
    prep(gemm_select_kernel<16, 1, true>);
    prep(gemm_select_kernel<32, 1, true>);
    if (st == FI_OK) done[device] = true;
    return st;
}

size_t gemm_part_entries(int max_batch, int64_t capacity, int sm_count, int k, int dim) {
    size_t worst = 0;
    const int tile_m = gemm_tile_m(max_batch, dim);
    const int num_kb = (dim + kBlockK - 1) / kBlockK;
    int m_tiles_max = (max_batch + tile_m - 1) / tile_m;
    for (int mt = 1; mt <= m_tiles_max; ++mt) {
        GemmPlan p = make_gemm_plan(mt * tile_m, capacity, sm_count, k, tile_m, num_kb);
        size_t e = (size_t)mt * tile_m * (size_t)p.lists * (size_t)p.list_len;
        if (e > worst) worst = e;
    }
    return worst;
}

size_t gemm_part_entries_bound(int max_batch, int64_t capacity, int sm_count, int k, int dim) {
    // lists per query: at most one per range (ranges <= CTAs, and <= 16-row blocks of the cache), times two for
    // 128-row tiles (two epilogue warps per row); wave + tail and spans modes have one list per 256-row tile of the
    // cache, at most 1.5 x CTAs and 2 x CTAs of them
    const size_t n16 = (size_t)((capacity + 15) / 16);
    const size_t list_len = (size_t)gemm_list_len(k);
    auto entries = [&](int rows, int tile_m) {
        const size_t f = tile_m == kTileM ? 2 : 1;
        size_t lists = (size_t)sm_count * f;
        if (tile_m != kTileM && lists < (size_t)2 * sm_count) lists = (size_t)2 * sm_count;
        if (lists > n16 * f) lists = n16 * f;
        if (lists < f) lists = f;
        const size_t padded = (size_t)((rows + tile_m - 1) / tile_m) * tile_m;
        return padded * lists * list_len;
    };
    size_t worst = entries(max_batch < kTileM ? max_batch : (gemm_tile_m(max_batch, dim) == kTileM ? max_batch : kTileM), kTileM);
    if (gemm_tile_m(max_batch, dim) != kTileM) {
        const size_t e = entries(max_batch, 2 * kTileM);
        if (e > worst) worst = e;
    }
    return worst;
}

// slots of 256 x 256 partial sums: one per CTA in wave + tail mode, kMaxSpanItems per CTA in spans mode
size_t gemm_tail_units(int max_batch, int dim, int sm_count) {
    const int num_kb = (dim + kBlockK - 1) / kBlockK;
    return gemm_tile_m(max_batch, dim) == 2 * kTileM && num_kb >= 64 ? (size_t)sm_count * kMaxSpanItems : 0;
}

// Can a batch of at most batch_max requests against the current cache end up in a mode that leaves pieces (wave +
// tail, spans)?  The mode depends on the number of query tiles and on whether the last one is at most half full.
static bool tail_mode_possible(const fi_cache *c, int batch_max) {
    const int tile_m = gemm_tile_m(batch_max, c->cfg.dim);
    const int num_kb = (c->cfg.dim + kBlockK - 1) / kBlockK;
    const int m_tiles_max = (batch_max + tile_m - 1) / tile_m;
    for (int mt = 1; mt <= m_tiles_max; ++mt)
        for (int count : {mt * tile_m, mt * tile_m - tile_m / 2})
            if (make_gemm_plan(count, c->size, c->sm_count, c->cfg.k, tile_m, num_kb).mode != 0) return true;
    return false;
}

// Pairs of CTAs (tcgen05 cta_group::2).  Measured against single CTAs on one B200: a pair keeps two accumulator buffers
// under a 256-row tile, so the select overlaps the next tile's MMAs, which pays where a tile's k-loop is short enough for
// the select to be a large share of it and long enough for the hand-over between the two CTAs not to matter: rows of
// 1,024 to 2,048 values (100,000 entries, batch 4,096: -4 % and -13 %).  On shorter rows the hand-over costs more than
// the overlap gains, on longer rows the exposed select is a few per cent and the pair's MMAs run 5-8 % slower (one
// issuing thread and one full-barrier for two SMs), and shapes in wave + tail mode want one deep tile per CTA.
// (The kernel also runs with 256 query rows per CTA of a pair, a third fewer operand bytes per flop and one accumulator
// buffer; forced on, it lost 5 % on 8,192-value rows and more elsewhere, so no launch path instantiates it.)
// FICACHE_PAIR=0 / 1 in the environment overrides the choice (for A/B measurements).
static bool use_pair_kernel(const fi_cache *c, int batch_max) {
    static const int forced = [] {
        const char *e = getenv("FICACHE_PAIR");
        return e ? atoi(e) : -1;
    }();
    if (batch_max <= kTileM || c->sm_count < 2 || c->size < 512) return false;
    if (forced >= 0) return forced == 1;
    const int num_kb = (c->cfg.dim + kBlockK - 1) / kBlockK;
    return num_kb >= 16 && num_kb <= 32 && batch_max >= 8 * kTileM && c->size >= 32768 && !tail_mode_possible(c, batch_max);
}

fi_status_t launch_gemm_select(fi_cache *c, const void *queries_compact, int64_t ld_elems, int32_t batch_max,
                               const int32_t *count_dev, cudaStream_t stream) {
    if (batch_max <= 0) return FI_OK;
    if (c->size <= 0) {
        set_error("the distance GEMM needs a non-empty cache");
        return FI_ERR_INVALID_ARG;
    }
    fi_status_t st = ensure_tensor_maps(c);
    if (st != FI_OK) return st;
    if ((reinterpret_cast<uintptr_t>(queries_compact) & 15) != 0 || (ld_elems % 8) != 0) {
        set_error("bf16 queries must be 16-byte aligned with a leading dimension that is a multiple of 8");
        return FI_ERR_INVALID_ARG;
    }
    CUtensorMap tq;
    st = encode_bf16_map(&tq, queries_compact, (uint64_t)batch_max, (uint64_t)c->cfg.dim, (uint64_t)ld_elems, kTileM);
    if (st != FI_OK) return st;
    const bool tail_possible = tail_mode_possible(c, batch_max);
    if (tail_possible && c->tail_dump_units < (size_t)c->sm_count * kMaxSpanItems) {
        // slots of 256 x 256 partial sums, allocated at create for every cache whose shapes can get here
        set_error("the distance GEMM's partial-sum buffer is missing (%zu slots, %d needed)", c->tail_dump_units,
                  c->sm_count * kMaxSpanItems);
        return FI_ERR_CAPACITY;
    }
    if (use_pair_kernel(c, batch_max)) return launch_pair<1>(c, tq, batch_max, count_dev, stream);
    if (gemm_tile_m(batch_max, c->cfg.dim) == kTileM) return launch_msub<1>(c, tq, batch_max, count_dev, false, stream);
    return launch_msub<2>(c, tq, batch_max, count_dev, tail_possible, stream);
}

size_t product_dump_units(int max_batch, int64_t n_rows, int sm_count) {
    const int m_tiles = (max_batch + 2 * kTileM - 1) / (2 * kTileM);
    const int64_t n_tiles = ((n_rows + 15) / 16 + 15) / 16;
    const size_t tiles = (size_t)m_tiles * (size_t)n_tiles;
    return tiles > (size_t)sm_count ? tiles : (size_t)sm_count;   // pieces = tiles x floor(CTAs / tiles), or the tiles
}

fi_status_t launch_gemm_project(fi_cache *w, const void *queries_compact, int64_t ld_elems, int32_t batch_max,
                                const int32_t *count_dev, void *y, int64_t ld_y, cudaStream_t stream) {
    if (batch_max <= 0) return FI_OK;
    fi_status_t st = ensure_tensor_maps(w);
    if (st != FI_OK) return st;
    if ((reinterpret_cast<uintptr_t>(queries_compact) & 15) != 0 || (ld_elems % 8) != 0 ||
        (reinterpret_cast<uintptr_t>(y) & 15) != 0 || (ld_y % 8) != 0 || (w->size % 16) != 0) {
        set_error("projection: inputs and outputs must be 16-byte aligned, leading dimensions multiples of 8, outputs a multiple of 16");
        return FI_ERR_INVALID_ARG;
    }
    if (w->tail_dump_units < product_dump_units(batch_max, w->size, w->sm_count)) {
        set_error("projection: partial-sum buffer too small for a batch of %d", batch_max);
        return FI_ERR_INVALID_ARG;
    }
    CUtensorMap tq;
    st = encode_bf16_map(&tq, queries_compact, (uint64_t)batch_max, (uint64_t)w->cfg.dim, (uint64_t)ld_elems, kTileM);
    if (st != FI_OK) return st;
    auto kern = gemm_select_kernel<8, 2>;   // prepared for this device when the weights' cache object was created
    kern<<<w->sm_count, kGemmThreads, kGemmSmemBytes, stream>>>(tq, w->tmap_rows64, w->tmap_rows16, w->norms,
                                                               (long long)w->size, w->cfg.dim, batch_max, count_dev, 1,
                                                               w->part_score, w->part_idx, w->plan_dev, w->row_bound,
                                                               w->tail_dump, w->status_dev, 1);
    count_launch();
    st = check_launch("gemm_select_kernel (product)");
    if (st != FI_OK) return st;
    const int m_tiles = (batch_max + 2 * kTileM - 1) / (2 * kTileM);
    const int n_tiles = (int)(((w->size + 15) / 16 + 15) / 16);
    product_reduce_kernel<<<dim3(m_tiles * n_tiles, kMaxTileN / 16), 2 * kTileM, 0, stream>>>(
        w->plan_dev, w->tail_dump, w->weights, (long long)w->size, static_cast<__nv_bfloat16 *>(y), (long long)ld_y);
    count_launch();
    return check_launch("product_reduce_kernel");
}

}  // namespace fi
