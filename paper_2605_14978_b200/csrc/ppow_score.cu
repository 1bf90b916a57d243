// PPOW scoring pass: row-reduction kernels (the only HBM-heavy step: the bulk-copy pipeline kernel, with
// instances for rows of whole 16-byte units and for rows that start inside a unit, and a scalar kernel for
// tensors at different offsets within a unit), the per-window scan kernel, the one-launch kernel for small
// problems, and the host entry points ppow_score_windows(_traced) / ppow_score_workspace_bytes /
// ppow_score_kernel_launches / ppow_read_error_flags / ppow_timeline_read / ppow_selftest_wait_timeout.
#include "../../include/ppow.h"
#include "ppow_device.cuh"
#include "ppow_async.cuh"
#include "ppow_checked.cuh"

#include <math.h>

#include <atomic>

namespace ppow {

// Timeline build (-DPPOW_TIMELINE): every warp of the bulk-copy kernel leaves eleven 64-bit words behind --
// start, first data and end (%globaltimer, ns), items and tiles done, SM id, cycles spent waiting for copies,
// cycles spent in item ends, its total cycles, and of the item-end cycles those up to the end of the warp
// reduction and those from there to the opening of the next item; ppow_timeline_read copies them out.  Costs a
// few instructions per tile; the ordinary build has none of it.
#ifdef PPOW_TIMELINE
constexpr int TIMELINE_WARPS = 4096;
constexpr int TIMELINE_WORDS = 11;
__device__ unsigned long long g_timeline[TIMELINE_WARPS * TIMELINE_WORDS];
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ unsigned sm_id()
{
    unsigned t;
    asm volatile("mov.u32 %0, %smid;" : "=r"(t));
    return t;
}
#define PPOW_TL(...) __VA_ARGS__
#else
#define PPOW_TL(...)
#endif

constexpr int ROW_THREADS = 256;   // threads per CTA of the scalar row-reduction kernels
constexpr int UNROLL = 4;          // 16-byte units per lane per tensor in one tile (< 8: packed with the unit index)
constexpr int TILE_UNITS = 32 * UNROLL;       // 16-byte units per tile per tensor
constexpr int MAX_SHIFT = 5;       // a row is split into at most 2^5 work items
constexpr int PLAN_CLASSES = 5;    // row classes of the work plan: items of at most 64, 32, 16, 8, 4 tiles
// an item is at most 1/1 (rows shorter than 64 tiles) or 2/3 (longer rows) of a resident warp's share of the work
// still to hand out
constexpr size_t WS_HEADER_BYTES = 256;
constexpr size_t SMALL_ROW_BYTES = 4096;        // rows up to this long (at most two tiles) in
constexpr size_t SMALL_TOTAL_BYTES = 4u << 20;  // calls up to this many logit bytes take the one-launch kernel

// Workspace header (first WS_HEADER_BYTES of the workspace).
struct WsHeader {
    unsigned int next_item;    // work counter of the row-reduction kernels
    unsigned int error_flags;  // PPOW_FLAG_* bits
};

// Work plan: how the rows are cut into work items.  A row is `tiles` tiles long (a tile is TILE_UNITS
// 16-byte units of each tensor) and is cut into 2^shift items of whole tiles, item i of a row covering
// tiles [i*tiles >> shift, (i+1)*tiles >> shift).  Rows come in up to PLAN_CLASSES classes by row index:
// the first rows are cut into long items (every item ends with a warp reduction), the last rows into
// short ones, so that the warps, which take items in increasing order from a counter, run out of work
// at nearly the same time.  Items are numbered class by class, row by row; item i owns partials[i].
struct WorkPlan {
    uint32_t item_begin[PLAN_CLASSES + 1];   // first item of each class; [PLAN_CLASSES] = number of items
    int32_t row_begin[PLAN_CLASSES + 1];     // first row of each class; [PLAN_CLASSES] = N*K
    int32_t shift[PLAN_CLASSES];             // log2 of the items per row in the class
    int32_t tiles;                           // tiles per row
};

struct RowJob {
    const void *target, *draft;
    const int32_t *valid_len;
    RowPartial *partials;      // [plan.item_begin[PLAN_CLASSES]]
    WsHeader *header;
    WorkPlan plan;
    int32_t N, K, V;
    int32_t units_per_row;     // 16-byte units per row (bulk-copy kernel, rows of whole aligned units)
    int32_t tile_logits;       // logits per tile (scalar kernel: item boundaries in logits)
    int32_t shifted;           // bulk-copy kernel: rows are not whole 16-byte aligned units (odd V or an offset base)
    int32_t es_shift;          // log2 of the bytes per logit
    int64_t row_bytes;         // bytes per row
    uint32_t total_items;
    float s;                   // log2(e)/T
};

// (row, first tile, end tile) of a work item
__device__ __forceinline__ void locate_item(const WorkPlan &plan, uint32_t item, uint32_t &row, int32_t &t0, int32_t &t1)
{
    // selects, not indexing: the plan lives in the kernel's parameter space
    uint32_t ib = plan.item_begin[0];
    int32_t rb = plan.row_begin[0];
    int sh = plan.shift[0];
#pragma unroll
    for (int c = 1; c < PLAN_CLASSES; ++c) {
        const bool in = item >= plan.item_begin[c];
        ib = in ? plan.item_begin[c] : ib;
        rb = in ? plan.row_begin[c] : rb;
        sh = in ? plan.shift[c] : sh;
    }
    const uint32_t local = item - ib;
    const uint32_t seg = local & ((1u << sh) - 1u);
    row = (uint32_t)rb + (local >> sh);
    t0 = (int32_t)((seg * (uint32_t)plan.tiles) >> sh);
    t1 = (int32_t)(((seg + 1u) * (uint32_t)plan.tiles) >> sh);
}

// (first item, number of items) of a row
__device__ __forceinline__ void row_items(const WorkPlan &plan, uint32_t row, uint32_t &first, int &count)
{
    uint32_t ib = plan.item_begin[0];
    int32_t rb = plan.row_begin[0];
    int sh = plan.shift[0];
#pragma unroll
    for (int c = 1; c < PLAN_CLASSES; ++c) {
        const bool in = row >= (uint32_t)plan.row_begin[c];
        ib = in ? plan.item_begin[c] : ib;
        rb = in ? plan.row_begin[c] : rb;
        sh = in ? plan.shift[c] : sh;
    }
    first = ib + ((row - (uint32_t)rb) << sh);
    count = 1 << sh;
}

// ---- work distribution -----------------------------------------------------------------------
// A work item is one piece of one row, processed by one warp.  Every warp of the launch starts on the
// item with its own index (no round trip to memory before its first load); all further items are
// handed out by an atomic counter so that ragged windows (rows beyond valid_len are never read), warps
// that run at different speeds and the tail of the launch stay balanced (a static even split was
// measured 8 % slower).  Lane 0 fetches the id of a warp's next item while the warp is busy with the
// current one.

__device__ __forceinline__ bool item_is_valid(const RowJob &job, uint32_t item)
{
    if (job.valid_len == nullptr) return true;
    uint32_t row;
    int32_t t0, t1;
    locate_item(job.plan, item, row, t0, t1);
    const int32_t n = (int32_t)(row / (uint32_t)job.K), k = (int32_t)(row % (uint32_t)job.K);
    return k < __ldg(job.valid_len + n);
}

// Next item from the counter; `workers` = warps of the launch (their first items are not in the counter).
__device__ __forceinline__ uint32_t fetch_item(const RowJob &job, uint32_t workers)
{
    uint32_t it;
    do {
        it = workers + atomicAdd(&job.header->next_item, 1u);
    } while (it < job.total_items && !item_is_valid(job, it));
    return it;
}

// First item of a warp: its own index if that row is valid, else one from the counter (uniform across the warp).
__device__ __forceinline__ uint32_t first_item(const RowJob &job, uint32_t worker, uint32_t workers, int lane)
{
    uint32_t it = worker;
    if (it < job.total_items && !item_is_valid(job, it)) {
        if (lane == 0) it = fetch_item(job, workers);
        it = __shfl_sync(0xffffffffu, it, 0);
    }
    return it;
}

constexpr uint32_t BF16X2_NEG_INF = 0xff80ff80u;   // packed bf16 (-inf, -inf): neutral for the tile maximum

__device__ __forceinline__ int32_t warp_min_i32(int32_t v)
{
    int32_t r;
    asm volatile("redux.sync.min.s32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
    return r;
}

// ---- bulk-copy pipeline, one warp per work item (bf16, f16 or f32; both tensors at the same offset within a
// 16-byte unit) ----
// Each warp takes work items on its own (its first by its index, the rest from the work counter); no block
// barrier is used at all, so the warps of an SM drift apart.  The logits reach the warp through its own ring of
// PIPE_STAGES shared-memory stages filled by bulk copies (cp.async.bulk + mbarrier): while the warp
// computes on one tile, the copies of the next PIPE_STAGES - 1 tiles are in flight, across the end of
// an item into the next one.  Loads never pause for the arithmetic, the end-of-item reduction or the
// argmax re-read, and they hold no registers while in flight.
constexpr int PIPE_WARPS = 8;                 // warps per CTA
constexpr int PIPE_STAGES = 3;                // tiles per warp: one being computed on, two in flight
constexpr int PIPE_MIN_CTAS = 2;              // 2 CTAs * 8 warps * 3 stages * 4 KB = 192 KB of shared memory per SM
constexpr int TILE_BYTES = TILE_UNITS * 16;   // 2 KB per tensor
constexpr int ITEM_RING = 8;                  // > PIPE_STAGES + 1 item ids between producer and consumer
constexpr uint32_t WAIT_LIMIT = 1u << 20;     // probes of one mbarrier before the kernel gives up
constexpr size_t PIPE_SMEM_BYTES = (size_t)PIPE_WARPS * PIPE_STAGES * 2 * TILE_BYTES;

struct ItemCursor {
    uint32_t item;          // >= total_items: nothing left
    int32_t u, u1;          // next unit and end of the item, relative to the row's first unit
    int32_t units, head;    // units the row spans; logits of its first unit that belong to the row before (0 unless shifted)
    const uint4 *pa, *pb;   // first unit of the row in each tensor (16-byte aligned)
};

template <bool SHIFTED>
__device__ __forceinline__ void open_item(const RowJob &job, ItemCursor &c, uint32_t item)
{
    c.item = item;
    c.u = c.u1 = 0;
    c.units = c.head = 0;
    c.pa = c.pb = nullptr;
    if (item >= job.total_items) return;
    uint32_t row;
    int32_t t0, t1;
    locate_item(job.plan, item, row, t0, t1);
    if (!SHIFTED) {
        c.units = job.units_per_row;
        c.pa = reinterpret_cast<const uint4 *>(job.target) + (size_t)row * c.units;
        c.pb = reinterpret_cast<const uint4 *>(job.draft) + (size_t)row * c.units;
    } else {
        // A row that starts inside a 16-byte unit: the units are taken from the aligned address below its
        // start (both tensors have the same offset), `head` logits of the first unit and the logits past the
        // row's end in the last one are masked out when those units are read.
        const uintptr_t a = reinterpret_cast<uintptr_t>(job.target) + (size_t)row * (size_t)job.row_bytes;
        const uintptr_t b = reinterpret_cast<uintptr_t>(job.draft) + (size_t)row * (size_t)job.row_bytes;
        const int epu_shift = 4 - job.es_shift;
        c.head = (int32_t)((a & 15u) >> job.es_shift);
        c.units = (c.head + job.V + (1 << epu_shift) - 1) >> epu_shift;
        c.pa = reinterpret_cast<const uint4 *>(a & ~(uintptr_t)15);
        c.pb = reinterpret_cast<const uint4 *>(b & ~(uintptr_t)15);
    }
    c.u = t0 * TILE_UNITS;
    c.u1 = (t1 == job.plan.tiles) ? c.units : t1 * TILE_UNITS;   // the last item of a row takes what is left of it
}

// Storage formats of the bulk-copy kernel: how a 16-byte unit of logits is read.
struct FmtBf16 {
    static constexpr int EPU = 8;   // logits per unit
    static __device__ __forceinline__ uint4 none()   // a unit that never wins a maximum
    {
        return make_uint4(BF16X2_NEG_INF, BF16X2_NEG_INF, BF16X2_NEG_INF, BF16X2_NEG_INF);
    }
    static __device__ __forceinline__ float tile_max(const uint4 (&X)[UNROLL])
    {
        uint32_t m = max_bf16x2(max_bf16x2(X[0].x, X[0].y), max_bf16x2(X[0].z, X[0].w));
#pragma unroll
        for (int j = 1; j < UNROLL; ++j)
            m = max_bf16x2(m, max_bf16x2(max_bf16x2(X[j].x, X[j].y), max_bf16x2(X[j].z, X[j].w)));
        return fmaxf(bf16_lo(m), bf16_hi(m));
    }
    template <bool REV>
    static __device__ __forceinline__ void add_unit(RowAcc<REV> &acc, const uint4 &a, const uint4 &b, float2 s2,
                                                    float2 nra, float2 nrb)
    {
        acc.add_word(a.x, b.x, s2, nra, nrb);
        acc.add_word(a.y, b.y, s2, nra, nrb);
        acc.add_word(a.z, b.z, s2, nra, nrb);
        acc.add_word(a.w, b.w, s2, nra, nrb);
    }
    // position (0..EPU-1) of the first logit of the unit equal to `value`, or -1
    static __device__ __forceinline__ int first_equal(const uint4 &w4, float value)
    {
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
        int pos = -1;
#pragma unroll
        for (int q = 3; q >= 0; --q) {
            if (bf16_hi(w[q]) == value) pos = 2 * q + 1;
            if (bf16_lo(w[q]) == value) pos = 2 * q;
        }
        return pos;
    }
    static __device__ __forceinline__ void mask_unit(uint4 &w4, int lo, int hi) { UnitBf16::mask_unit(w4, lo, hi); }
};

struct FmtF16 {
    static constexpr int EPU = 8;
    static __device__ __forceinline__ uint4 none() { return make_uint4(0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u); }
    static __device__ __forceinline__ __half2 h2(uint32_t w) { return *reinterpret_cast<const __half2 *>(&w); }
    static __device__ __forceinline__ float tile_max(const uint4 (&X)[UNROLL])
    {
        __half2 m = __hmax2(__hmax2(h2(X[0].x), h2(X[0].y)), __hmax2(h2(X[0].z), h2(X[0].w)));
#pragma unroll
        for (int j = 1; j < UNROLL; ++j)
            m = __hmax2(m, __hmax2(__hmax2(h2(X[j].x), h2(X[j].y)), __hmax2(h2(X[j].z), h2(X[j].w))));
        const float2 f = __half22float2(m);
        return fmaxf(f.x, f.y);
    }
    template <bool REV>
    static __device__ __forceinline__ void add_unit(RowAcc<REV> &acc, const uint4 &a, const uint4 &b, float2 s2,
                                                    float2 nra, float2 nrb)
    {
        acc.add2(__half22float2(h2(a.x)), __half22float2(h2(b.x)), s2, nra, nrb);
        acc.add2(__half22float2(h2(a.y)), __half22float2(h2(b.y)), s2, nra, nrb);
        acc.add2(__half22float2(h2(a.z)), __half22float2(h2(b.z)), s2, nra, nrb);
        acc.add2(__half22float2(h2(a.w)), __half22float2(h2(b.w)), s2, nra, nrb);
    }
    static __device__ __forceinline__ int first_equal(const uint4 &w4, float value)
    {
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
        int pos = -1;
#pragma unroll
        for (int q = 3; q >= 0; --q) {
            const float2 f = __half22float2(h2(w[q]));
            if (f.y == value) pos = 2 * q + 1;
            if (f.x == value) pos = 2 * q;
        }
        return pos;
    }
    static __device__ __forceinline__ void mask_unit(uint4 &w4, int lo, int hi) { UnitF16::mask_unit(w4, lo, hi); }
};

struct FmtF32 {
    static constexpr int EPU = 4;
    static __device__ __forceinline__ uint4 none() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
    static __device__ __forceinline__ float tile_max(const uint4 (&X)[UNROLL])
    {
        float m = -INFINITY;
#pragma unroll
        for (int j = 0; j < UNROLL; ++j)
            m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(X[j].x), __uint_as_float(X[j].y)),
                               fmaxf(__uint_as_float(X[j].z), __uint_as_float(X[j].w))));
        return m;
    }
    template <bool REV>
    static __device__ __forceinline__ void add_unit(RowAcc<REV> &acc, const uint4 &a, const uint4 &b, float2 s2,
                                                    float2 nra, float2 nrb)
    {
        acc.add2(make_float2(__uint_as_float(a.x), __uint_as_float(a.y)),
                 make_float2(__uint_as_float(b.x), __uint_as_float(b.y)), s2, nra, nrb);
        acc.add2(make_float2(__uint_as_float(a.z), __uint_as_float(a.w)),
                 make_float2(__uint_as_float(b.z), __uint_as_float(b.w)), s2, nra, nrb);
    }
    static __device__ __forceinline__ int first_equal(const uint4 &w4, float value)
    {
        int pos = -1;
        if (__uint_as_float(w4.w) == value) pos = 3;
        if (__uint_as_float(w4.z) == value) pos = 2;
        if (__uint_as_float(w4.y) == value) pos = 1;
        if (__uint_as_float(w4.x) == value) pos = 0;
        return pos;
    }
    static __device__ __forceinline__ void mask_unit(uint4 &w4, int lo, int hi) { UnitF32::mask_unit(w4, lo, hi); }
};

// Which logits of unit `ui` of a shifted row belong to the row: [lo, hi).
struct RowEdges {
    int32_t head, span, units;   // span = head + V
    __device__ __forceinline__ bool touches(int32_t ui) const { return ui == 0 || ui == units - 1; }
    template <typename Fmt>
    __device__ __forceinline__ void mask(uint4 &w, int32_t ui) const
    {
        Fmt::mask_unit(w, ui == 0 ? head : 0, min(Fmt::EPU, span - ui * Fmt::EPU));
    }
};

// One tile out of shared memory.  `nu` = units of this lane that exist (UNROLL unless MASKED);
// MASKED tiles of a shifted row (`edges` != nullptr) also blank the logits of the row's first and last unit that
// belong to its neighbours.  refill() is called once every value of the stage sits in registers.
template <bool MASKED, bool REV, typename Fmt, typename Refill>
__device__ __forceinline__ void pipe_tile(const uint4 *sa, const uint4 *sb, int32_t u, int nu, RowAcc<REV> &acc,
                                          float s, Refill refill, const RowEdges *edges = nullptr)
{
    const int lane = threadIdx.x & 31;
    uint4 A[UNROLL], B[UNROLL];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) A[j] = (!MASKED || j < nu) ? sa[j * 32 + lane] : Fmt::none();
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) B[j] = (!MASKED || j < nu) ? sb[j * 32 + lane] : Fmt::none();
    if (MASKED && edges) {
#pragma unroll
        for (int j = 0; j < UNROLL; ++j) {
            if (j < nu && edges->touches(u + j * 32)) {
                edges->template mask<Fmt>(A[j], u + j * 32);
                edges->template mask<Fmt>(B[j], u + j * 32);
            }
        }
    }

    const float tmax_a = Fmt::tile_max(A), tmax_b = Fmt::tile_max(B);
    acc.guard(tmax_a, tmax_b, s);
    if (tmax_a > acc.max_a) {   // strict: an equal value seen later has a higher index
        acc.max_a = tmax_a;
        acc.best = u * 8 + nu;  // first unit of this lane in the tile and its unit count, packed
    }
    refill();   // the tile maxima consumed every word of the stage: it may be overwritten now
    const float2 s2 = make_float2(s, s);
    const float2 nra = make_float2(-acc.rho_a, -acc.rho_a), nrb = make_float2(-acc.rho_b, -acc.rho_b);
#pragma unroll
    for (int j = 0; j < UNROLL; ++j)
        if (!MASKED || j < nu) Fmt::add_unit(acc, A[j], B[j], s2, nra, nrb);
    acc.flush();
}

// SHIFTED: rows that start inside a 16-byte unit (instances of their own, so that the plain case pays nothing for it).
template <bool REV, typename Fmt, bool SHIFTED>
__global__ void __launch_bounds__(PIPE_WARPS * 32, PIPE_MIN_CTAS) row_reduce_pipe_kernel(const RowJob job)
{
    extern __shared__ __align__(128) unsigned char pipe_smem[];
    __shared__ __align__(8) uint64_t full_bar[PIPE_WARPS][PIPE_STAGES];
    __shared__ uint32_t item_ring[PIPE_WARPS][ITEM_RING];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    PPOW_TL(const unsigned long long tl_t0 = global_ns(); unsigned long long tl_t1 = 0; unsigned tl_items = 0, tl_tiles = 0;
            long long tl_wait = 0, tl_end = 0, tl_reduce = 0, tl_open = 0; const long long tl_c0 = clock64();)
    unsigned char *stages = pipe_smem + (size_t)warp * PIPE_STAGES * 2 * TILE_BYTES;
    const uint32_t stages_addr = smem_addr(stages);
    const uint32_t bars_addr = smem_addr(&full_bar[warp][0]);

    // the mbarriers of a warp are touched by that warp only (lane 0 arms them and issues the copies, every
    // lane waits on them): a warp-level barrier after their initialisation is all the set-up needs
    if (lane == 0) {
#pragma unroll
        for (int st = 0; st < PIPE_STAGES; ++st) mbar_init(bars_addr + 8 * st, 1);
        mbar_init_fence();
    }
    __syncwarp();

    // Producer side: P walks the items this warp takes and issues one tile per call.
    const uint32_t workers = gridDim.x * PIPE_WARPS;
    ItemCursor P, C;
    uint32_t produced = 0, consumed = 0;   // items opened by each side
    uint32_t pending = 0;                   // stages with a copy in flight
    uint32_t upcoming = 0;                  // (lane 0) id fetched ahead for the item after P's
    const uint32_t first = first_item(job, blockIdx.x * PIPE_WARPS + warp, workers, lane);
    if (lane == 0) item_ring[warp][0] = first;
    open_item<SHIFTED>(job, P, first);
    C = P;
    produced = consumed = 1;

    // copies of P's next tile into stage st
    auto issue = [&](int st) -> int32_t {
        const int32_t n = min(TILE_UNITS, P.u1 - P.u);
        // the tile lies inside its row, the row inside the tensors, the stage inside the warp's ring
        if (lane == 0 && PPOW_CHECK(n > 0 && P.u >= 0 && P.u + n <= P.units && st >= 0 && st < PIPE_STAGES &&
                                        reinterpret_cast<uintptr_t>(P.pa + P.u + n) <=
                                            ((reinterpret_cast<uintptr_t>(job.target) +
                                              (size_t)job.N * job.K * (size_t)job.row_bytes + 15u) & ~(uintptr_t)15),
                                    101, &job.header->error_flags)) {
            const uint32_t bar = bars_addr + 8 * st, dst = stages_addr + st * 2 * TILE_BYTES;
            mbar_arrive_expect_tx(bar, 2u * (uint32_t)n * 16u);
            bulk_load(dst, P.pa + P.u, (uint32_t)n * 16u, bar);
            bulk_load(dst + TILE_BYTES, P.pb + P.u, (uint32_t)n * 16u, bar);
        }
        pending |= 1u << st;
        return n;
    };
    // move P past n units; at the end of its item, on to the item fetched ahead (and fetch the one after)
    auto advance = [&](int32_t n) {
        P.u += n;
        if (P.u >= P.u1) {
            const uint32_t nx = __shfl_sync(0xffffffffu, upcoming, 0);
            if (lane == 0) {
                item_ring[warp][produced % ITEM_RING] = nx;
                if (nx < job.total_items) upcoming = fetch_item(job, workers);
            }
            ++produced;
            open_item<SHIFTED>(job, P, nx);
        }
    };
    auto produce = [&](int st) {
        if (P.item >= job.total_items) return;
        advance(issue(st));
    };

    // the first tile is on its way before the warp's first visit to the work counter
    if (P.item < job.total_items) {
        const int32_t n = issue(0);
        if (lane == 0) upcoming = fetch_item(job, workers);
        advance(n);
    }
#pragma unroll
    for (int st = 1; st < PIPE_STAGES; ++st) produce(st);

    uint32_t phases = 0;
    int st = 0;
    RowAcc<REV> acc;
    acc.reset();
    while (C.item < job.total_items) {
        const int32_t n = min(TILE_UNITS, C.u1 - C.u);
        // every lane waits (the tile becomes visible to the lanes that observed the phase); the vote keeps
        // the warp together if the limit is hit by only some of them
        PPOW_TL(const long long tl_w0 = clock64();)
        const bool arrived = __all_sync(0xffffffffu, mbar_wait_bounded(bars_addr + 8 * st, (phases >> st) & 1u, WAIT_LIMIT));
        PPOW_TL(tl_wait += clock64() - tl_w0; if (tl_t1 == 0) tl_t1 = global_ns(); ++tl_tiles;)
        if (!arrived) {
            // give up: report, wait (bounded) for the copies still aimed at this warp's stages, leave
            if (lane == 0) atomicOr(&job.header->error_flags, (unsigned)PPOW_FLAG_DEVICE_TIMEOUT);
#pragma unroll
            for (int q = 0; q < PIPE_STAGES; ++q)
                if (pending & (1u << q)) mbar_wait_bounded(bars_addr + 8 * q, (phases >> q) & 1u, WAIT_LIMIT);
            break;
        }
        phases ^= 1u << st;
        pending &= ~(1u << st);
        if (!PPOW_CHECK(st >= 0 && st < PIPE_STAGES && n > 0 && n <= TILE_UNITS, 104, &job.header->error_flags)) break;
        const uint4 *sa = reinterpret_cast<const uint4 *>(stages + st * 2 * TILE_BYTES);
        const uint4 *sb = reinterpret_cast<const uint4 *>(stages + st * 2 * TILE_BYTES + TILE_BYTES);
        auto refill = [&]() {
            __syncwarp();
            produce(st);
        };
        const RowEdges edges = {C.head, C.head + job.V, C.units};
        if (n == TILE_UNITS && (!SHIFTED || (C.u > 0 && C.u + n < C.units)))
            pipe_tile<false, REV, Fmt>(sa, sb, C.u + lane, UNROLL, acc, job.s, refill);
        else
            pipe_tile<true, REV, Fmt>(sa, sb, C.u + lane, min(UNROLL, (n - lane + 31) / 32), acc, job.s, refill,
                                      SHIFTED ? &edges : nullptr);
        C.u += n;

        if (C.u >= C.u1) {   // end of the item: warp reduction, argmax index, one partial
            PPOW_TL(const long long tl_e0 = clock64();)
            // The lanes that hold the item's maximum re-read the units of the tile that raised it, to find the
            // lowest vocabulary index.  The loads are issued as soon as the maximum is known, so that the rest
            // of the warp reduction covers their latency.
            const float my_max = acc.max_a;
            const float item_max = warp_max(my_max);
            const bool holder = my_max == item_max;
            const int32_t bu = acc.best >> 3, bn = acc.best & 7;
            const RowEdges done_edges = {C.head, C.head + job.V, C.units};
            uint4 cand[UNROLL];
#pragma unroll
            for (int j = 0; j < UNROLL; ++j)
                if (holder && j < bn &&
                    PPOW_CHECK(bu >= 0 && bu + j * 32 < C.units, 102, &job.header->error_flags))
                    cand[j] = __ldcs(C.pa + bu + j * 32);
                else
                    cand[j] = Fmt::none();
            RowPartial p = warp_reduce(acc);
            PPOW_TL(const long long tl_e1 = clock64(); tl_reduce += tl_e1 - tl_e0;)
            // the consumer moves on to its next item while the re-read is in flight
            const uint32_t done = C.item;
            acc.reset();
            __syncwarp();
            const uint32_t nx = item_ring[warp][consumed % ITEM_RING];
            ++consumed;
            open_item<SHIFTED>(job, C, nx);
            PPOW_TL(tl_open += clock64() - tl_e1;)
            int32_t arg = INT32_MAX;
            if (holder) {
#pragma unroll
                for (int j = 0; j < UNROLL; ++j) {
                    if (j < bn && arg == INT32_MAX) {
                        if (SHIFTED && done_edges.touches(bu + j * 32)) done_edges.template mask<Fmt>(cand[j], bu + j * 32);
                        const int pos = Fmt::first_equal(cand[j], my_max);
                        if (pos >= 0) arg = (bu + j * 32) * Fmt::EPU + pos - done_edges.head;
                    }
                }
            }
            arg = warp_min_i32(arg);
            if (lane == 0 && PPOW_CHECK(done < job.total_items, 103, &job.header->error_flags)) {
                p.argmax = arg;
                job.partials[done] = p;
            }
            PPOW_TL(++tl_items; tl_end += clock64() - tl_e0;)
        }
        st = (st + 1 == PIPE_STAGES) ? 0 : st + 1;
    }
    PPOW_TL(const unsigned tl_w = blockIdx.x * PIPE_WARPS + warp;
            if (lane == 0 && tl_w < TIMELINE_WARPS) {
                unsigned long long *o = g_timeline + (size_t)tl_w * TIMELINE_WORDS;
                o[0] = tl_t0; o[1] = tl_t1; o[2] = global_ns(); o[3] = tl_items; o[4] = tl_tiles; o[5] = sm_id();
                o[6] = (unsigned long long)tl_wait; o[7] = (unsigned long long)tl_end; o[8] = (unsigned long long)(clock64() - tl_c0);
                o[9] = (unsigned long long)tl_reduce; o[10] = (unsigned long long)tl_open;
            })
}

// ---- scalar path: any V, any alignment, any storage type ----------------------------------------

// One warp reduces logits [v0, v1) of a row with scalar coalesced loads: the loads of SCALAR_BATCH strides are
// issued together (a lane would otherwise have one pair of loads in flight per trip), then folded one by one.
constexpr int SCALAR_BATCH = 8;

template <typename T, bool REV>
__device__ __forceinline__ void reduce_span_scalar(const T *pa, const T *pb, int32_t v0, int32_t v1, int lane, float s,
                                                   RowAcc<REV> &acc, int32_t &arg)
{
    for (int32_t base = v0 + lane; base < v1; base += 32 * SCALAR_BATCH) {
        float a[SCALAR_BATCH], b[SCALAR_BATCH];
#pragma unroll
        for (int j = 0; j < SCALAR_BATCH; ++j) {
            const int32_t v = base + 32 * j;
            if (v < v1) {
                a[j] = load_logit<T>(pa, v);
                b[j] = load_logit<T>(pb, v);
            }
        }
#pragma unroll
        for (int j = 0; j < SCALAR_BATCH; ++j) {
            const int32_t v = base + 32 * j;
            if (v < v1) {
                acc.guard(a[j], b[j], s);
                if (a[j] > acc.max_a) { acc.max_a = a[j]; arg = v; }   // strict: first occurrence within the lane
                acc.add_pair(a[j], b[j], s);
                acc.flush();
            }
        }
    }
}

template <typename T, bool REV>
__global__ void __launch_bounds__(ROW_THREADS, 4) row_reduce_generic_kernel(const RowJob job)
{
    const int lane = threadIdx.x & 31;
    const uint32_t workers = gridDim.x * (ROW_THREADS / 32);
    uint32_t item = first_item(job, blockIdx.x * (ROW_THREADS / 32) + (threadIdx.x >> 5), workers, lane);

    while (item < job.total_items) {
        uint32_t next = 0;
        if (lane == 0) next = fetch_item(job, workers);   // consumed after this item

        uint32_t row;
        int32_t t0, t1;
        locate_item(job.plan, item, row, t0, t1);
        const int32_t v0 = t0 * job.tile_logits;
        const int32_t v1 = min(t1 * job.tile_logits, job.V);
        const T *pa = reinterpret_cast<const T *>(job.target) + (size_t)row * job.V;
        const T *pb = reinterpret_cast<const T *>(job.draft) + (size_t)row * job.V;

        RowAcc<REV> acc;
        acc.reset();
        int32_t arg = INT32_MAX;
        reduce_span_scalar<T, REV>(pa, pb, v0, v1, lane, job.s, acc, arg);
        const float my_max = acc.max_a;
        RowPartial p = warp_reduce(acc);
        arg = warp_min_i32(my_max == p.max_a ? arg : INT32_MAX);
        if (lane == 0 && PPOW_CHECK(item < job.total_items && v1 <= job.V && v0 >= 0, 105, &job.header->error_flags)) {
            p.argmax = arg;
            job.partials[item] = p;
        }
        item = __shfl_sync(0xffffffffu, next, 0);
    }
}

// ---- per-window scan: float64 epilogue per position, prefix scan, rewards, score --------------

struct ScanJob {
    const void *target, *draft;
    const int32_t *tokens;
    const float *uniforms;
    const int32_t *valid_len;
    const float *ref_logp;
    const RowPartial *partials;
    WsHeader *header;
    ppow_outputs out;
    WorkPlan plan;
    int32_t N, K, V, dtype, mode;
    float s;         // log2(e)/T as used by the row reduction
    float c, eta, eps;
    double ln_v;     // ln V
};

__device__ __forceinline__ double raw_logit(const void *base, int32_t dtype, size_t idx)
{
    if (dtype == PPOW_F32) return (double)__ldg(reinterpret_cast<const float *>(base) + idx);
    if (dtype == PPOW_F16) return (double)f16_to_f32(__ldg(reinterpret_cast<const uint16_t *>(base) + idx));
    return (double)__uint_as_float(((uint32_t)__ldg(reinterpret_cast<const uint16_t *>(base) + idx)) << 16);
}

constexpr int SCAN_THREADS = 128;

// A row's partial reductions merged against the largest references (float64).
struct RowSums {
    double Ra, Rb, Sa, Sb, E, D, B;
    float mx;
    int32_t arg;
};

// Folds the sums `p` of one part of a row into `m`, carrying the larger references: moving either side to a new
// reference is a multiplication by an exact power of two (references are whole numbers), so the order of the
// parts only matters to the rounding of the float64 additions.  A side that holds nothing (Sa == 0: every
// real part has a term near 2^0) is skipped.
__device__ __forceinline__ void fold_sums(RowSums &m, const RowSums &p)
{
    if (p.Sa == 0.0) return;
    if (m.Sa == 0.0) {
        m = p;
        return;
    }
    const double Ra = fmax(m.Ra, p.Ra), Rb = fmax(m.Rb, p.Rb);
    const double da0 = m.Ra - Ra, db0 = m.Rb - Rb;   // what is held so far: one of each pair is 0
    const double da1 = p.Ra - Ra, db1 = p.Rb - Rb;   // the new part
    const double fa0 = pow2_whole(da0), fb0 = pow2_whole(db0), fa1 = pow2_whole(da1), fb1 = pow2_whole(db1);
    m.E = fa0 * (m.E + da0 * m.Sa) + fa1 * (p.E + da1 * p.Sa);
    m.D = fa0 * (m.D + (da0 - db0) * m.Sa) + fa1 * (p.D + (da1 - db1) * p.Sa);
    m.B = fb0 * (m.B + (da0 - db0) * m.Sb) + fb1 * (p.B + (da1 - db1) * p.Sb);
    m.Sa = fa0 * m.Sa + fa1 * p.Sa;
    m.Sb = fb0 * m.Sb + fb1 * p.Sb;
    m.Ra = Ra;
    m.Rb = Rb;
    m.arg = p.mx > m.mx ? p.arg : (p.mx == m.mx ? min(m.arg, p.arg) : m.arg);
    m.mx = fmaxf(m.mx, p.mx);
}

__device__ __forceinline__ RowSums sums_of(const RowPartial &p)
{
    RowSums r = {(double)p.rho_a, (double)p.rho_b, p.Sa, p.Sb, p.E, p.D, p.B, p.max_a, p.argmax};
    return r;
}

// One lane merges parts start, start + stride, ... of a row, four loads at a time (a lane would otherwise
// wait for memory once per part).
__device__ __forceinline__ RowSums merge_partials(const RowPartial *pp, int parts, int start = 0, int stride = 1)
{
    RowSums m = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, -INFINITY, INT32_MAX};
    for (int i0 = start; i0 < parts; i0 += 4 * stride) {
        RowPartial q[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (i0 + j * stride < parts) q[j] = pp[i0 + j * stride];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (i0 + j * stride < parts) fold_sums(m, sums_of(q[j]));
    }
    return m;
}

__device__ __forceinline__ RowSums shfl_sums(const RowSums &m, int src_lane, bool xor_mode)
{
    RowSums r;
#define PPOW_SH(x) (xor_mode ? __shfl_xor_sync(0xffffffffu, (x), src_lane) : __shfl_sync(0xffffffffu, (x), src_lane))
    r.Ra = PPOW_SH(m.Ra); r.Rb = PPOW_SH(m.Rb); r.Sa = PPOW_SH(m.Sa); r.Sb = PPOW_SH(m.Sb);
    r.E = PPOW_SH(m.E); r.D = PPOW_SH(m.D); r.B = PPOW_SH(m.B); r.mx = PPOW_SH(m.mx); r.arg = PPOW_SH(m.arg);
#undef PPOW_SH
    return r;
}

// What the scan needs about the drafted token of one position: read ahead of the merge of the row's parts, so
// that these dependent loads (token id, then the two logits at that id) are in flight meanwhile.  Read for every
// position of the window, valid or not (the arrays hold K entries per window; a masked position's token is only
// looked at if it happens to be a vocabulary index, and is never scored), so that nothing here waits for the
// window's valid length.
struct TokenRead {
    int32_t tok;
    bool in_range;
    double a_tok, b_tok, u;
};

__device__ __forceinline__ TokenRead read_token(const ScanJob &job, const int32_t n, const int lane)
{
    TokenRead r = {0, false, 0.0, 0.0, 0.0};
    if (lane >= job.K) return r;
    const size_t row = (size_t)n * job.K + lane;
    r.tok = __ldg(job.tokens + row);
    r.in_range = r.tok >= 0 && r.tok < job.V &&
                 PPOW_CHECK(row < (size_t)job.N * job.K && row * job.V + r.tok < (size_t)job.N * job.K * job.V, 202,
                            &job.header->error_flags);
    if (r.in_range) {
        r.a_tok = raw_logit(job.target, job.dtype, row * job.V + r.tok);
        r.b_tok = raw_logit(job.draft, job.dtype, row * job.V + r.tok);
    }
    if (job.mode != PPOW_GREEDY) r.u = (double)__ldg(job.uniforms + row);
    return r;
}

// One warp scores window n, lane = position.  `m`: the merged reductions of this lane's row, `tr`: its drafted
// token (both unused by lanes beyond the window's valid length L).
__device__ __forceinline__ void scan_window(const ScanJob &job, const int32_t n, const int lane, const int32_t L,
                                            const RowSums &m, const TokenRead &tr)
{
    const int32_t K = job.K;
    const bool active = lane < L;
    const double LN2 = 0.69314718055994530942;

    double crit = 0.0, gap = 0.0, lp = 0.0, kl_rev = 0.0;
    float o_kl = 0.f, o_conf = 0.f, o_crit = 0.f, o_lp = 0.f, o_lq = 0.f, o_nabla = 0.f, o_lse_p = 0.f, o_lse_q = 0.f;
    int32_t o_arg = 0;
    int flag = 0;

    if (active) {
        const double Ra = m.Ra, Rb = m.Rb, Sa = m.Sa, Sb = m.Sb, E = m.E, D = m.D, Bv = m.B;
        const float mx = m.mx;
        const int32_t arg = m.arg;
        const double s = (double)job.s;
        const double l2Sa = log2(Sa), l2Sb = log2(Sb);
        const double H = (l2Sa - E / Sa) * LN2;                 // entropy of P, nats
        const double KL = (D / Sa - l2Sa + l2Sb) * LN2;         // KL(P || Q), nats
        kl_rev = (-Bv / Sb - l2Sb + l2Sa) * LN2;              // KL(Q || P), nats (meaningful only if B was accumulated)
        o_lse_p = (float)((Ra + l2Sa) * LN2);
        o_lse_q = (float)((Rb + l2Sb) * LN2);
        double C = 1.0 - H / job.ln_v;
        C = fmin(1.0, fmax(0.0, C));
        crit = C * KL;
        const double lmax2 = fma((double)mx, s, -Ra) - l2Sa;   // log2 P(argmax); explicit fma: same rounding as lp2

        const int32_t tok = tr.tok;
        double lq, lp2 = -INFINITY;
        if (!tr.in_range) {
            atomicOr(&job.header->error_flags, (unsigned)PPOW_FLAG_TOKEN_RANGE);
            lp = -INFINITY;
            lq = -INFINITY;
            flag = 0;
            o_nabla = INFINITY;
        } else {
            const double a_tok = tr.a_tok, b_tok = tr.b_tok;
            lp2 = fma(a_tok, s, -Ra) - l2Sa;
            lp = lp2 * LN2;
            lq = (fma(b_tok, s, -Rb) - l2Sb) * LN2;
            o_nabla = (float)(expm1(lp - lq) - (lp - lq));   // exp(d) - d - 1 without cancellation near d = 0
            if (job.mode == PPOW_GREEDY) {
                flag = (tok == arg);
            } else {
                const double alpha = fmin(1.0, exp(lp - lq));
                flag = (tr.u <= alpha);
            }
        }
        gap = (lmax2 - lp2) * LN2;   // differenced before scaling: exactly 0 when the token is the argmax
        o_kl = (float)KL; o_conf = (float)C; o_crit = (float)crit; o_lp = (float)lp; o_lq = (float)lq;
        o_arg = arg;
    }

    if (lane < K && PPOW_CHECK(n >= 0 && n < job.N && K <= 32, 203, &job.header->error_flags)) {
        const size_t row = (size_t)n * K + lane;
        if (job.out.accept_flag) job.out.accept_flag[row] = (uint8_t)flag;
        if (job.out.kl) job.out.kl[row] = o_kl;
        if (job.out.conf) job.out.conf[row] = o_conf;
        if (job.out.crit) job.out.crit[row] = o_crit;
        if (job.out.logp_tok) job.out.logp_tok[row] = o_lp;
        if (job.out.logq_tok) job.out.logq_tok[row] = o_lq;
        if (job.out.target_argmax) job.out.target_argmax[row] = o_arg;
        if (job.out.kl_rev) job.out.kl_rev[row] = (float)kl_rev;
        if (job.out.nabla) job.out.nabla[row] = o_nabla;
        if (job.out.lse_p) job.out.lse_p[row] = o_lse_p;
        if (job.out.lse_q) job.out.lse_q[row] = o_lse_q;
    }

    // accepted length = number of leading accepted positions (App. C.1)
    const unsigned accepted = __ballot_sync(0xffffffffu, flag != 0);
    const unsigned valid_mask = (L >= 32) ? 0xffffffffu : ((1u << L) - 1u);
    const unsigned rejected = (~accepted) & valid_mask;
    const int32_t k = rejected ? (__ffs(rejected) - 1) : L;

    const double sum_crit = warp_sum_f64(crit);
    const double sum_gap = warp_sum_f64(gap);
    const double sum_lp = warp_sum_f64(lp);
    const double sum_rev = warp_sum_f64(kl_rev);

    if (lane == 0) {
        float r_speed = 0.f, r_dist = 0.f, delta = 0.f, score = 0.f, rev_mean = 0.f;
        if (L > 0) {
            const double rs = (double)k / ((double)k * (double)job.c + 1.0);
            const double dl = job.ref_logp ? ((double)__ldg(job.ref_logp + n) - sum_lp) : sum_gap;
            r_speed = (float)rs;
            delta = (float)dl;
            r_dist = (k == 0 && dl < (double)job.eps) ? job.eta : 0.f;
            score = (float)(sum_crit / (double)L);
            rev_mean = (float)(sum_rev / (double)L);
        }
        job.out.accepted_len[n] = k;
        if (job.out.reward_speedup) job.out.reward_speedup[n] = r_speed;
        if (job.out.reward_dist) job.out.reward_dist[n] = r_dist;
        if (job.out.reward) job.out.reward[n] = r_speed + r_dist;
        if (job.out.delta) job.out.delta[n] = delta;
        if (job.out.score) job.out.score[n] = score;
        if (job.out.kl_rev_mean) job.out.kl_rev_mean[n] = rev_mean;
    }
}

__global__ void __launch_bounds__(SCAN_THREADS) window_scan_kernel(const ScanJob job)
{
    const int lane = threadIdx.x & 31;
    const int32_t n = (int32_t)((blockIdx.x * (unsigned)SCAN_THREADS + threadIdx.x) >> 5);
    if (n >= job.N) return;
    uint32_t first_part = 0;
    int parts = 0;
    // G lanes share the merge of one row's parts (rows near the end of the launch are cut into up to 32 items):
    // lanes [r*G, r*G + G) take parts sub, sub + G, ... of row r, fold their results together, and lane t, which
    // scores position t, fetches row t's sums from lane t*G
    int kp = 1;
    while (kp < job.K) kp <<= 1;
    const int G = 32 / kp, r = lane / G, sub = lane & (G - 1);
    int32_t L = job.valid_len ? __ldg(job.valid_len + n) : job.K;   // first needed after the merge
    const TokenRead tr = read_token(job, n, lane);                    // in flight while the parts are merged
    // every row of the window is merged, valid or not (a masked row's slots hold whatever an earlier call left
    // there; the result is dropped below), so that the loads do not wait for the valid length
    if (r < job.K) row_items(job.plan, (uint32_t)n * (uint32_t)job.K + (uint32_t)r, first_part, parts);
    if (!PPOW_CHECK((size_t)first_part + parts <= job.plan.item_begin[PLAN_CLASSES] && parts <= (1 << MAX_SHIFT), 204,
                    &job.header->error_flags))
        parts = 0;
    RowSums m = merge_partials(job.partials + first_part, parts, sub, G);
    for (int o = G >> 1; o > 0; o >>= 1) fold_sums(m, shfl_sums(m, o, true));
    m = shfl_sums(m, (lane * G) & 31, false);
    L = max(0, min(L, job.K));
    scan_window(job, n, lane, L, m, tr);
}

// ---- small problems: the whole pass in one launch ---------------------------------------------------
// When the logits of a call are a few megabytes the pass is bound by launches, not by memory: one CTA per
// window, warp t reduces position t's row (scalar coalesced loads, the same accumulators), the partials stay
// in shared memory and warp 0 scores the window.  No work counter, no partials in the workspace.
template <typename T, bool REV>
__global__ void __launch_bounds__(1024) score_small_kernel(const RowJob rj, const ScanJob sj)
{
    __shared__ RowPartial parts[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t n = (int32_t)blockIdx.x;
    int32_t L = rj.valid_len ? __ldg(rj.valid_len + n) : rj.K;
    L = max(0, min(L, rj.K));
    if (warp < L) {
        const size_t row = (size_t)n * rj.K + warp;
        const T *pa = reinterpret_cast<const T *>(rj.target) + row * rj.V;
        const T *pb = reinterpret_cast<const T *>(rj.draft) + row * rj.V;
        RowAcc<REV> acc;
        acc.reset();
        int32_t arg = INT32_MAX;
        reduce_span_scalar<T, REV>(pa, pb, 0, rj.V, lane, rj.s, acc, arg);
        const float my_max = acc.max_a;
        RowPartial p = warp_reduce(acc);
        arg = warp_min_i32(my_max == p.max_a ? arg : INT32_MAX);
        if (lane == 0 && PPOW_CHECK(warp < 32 && row < (size_t)rj.N * rj.K, 106, &rj.header->error_flags)) {
            p.argmax = arg;
            parts[warp] = p;
        }
    }
    __syncthreads();
    if (warp == 0) {
        const TokenRead tr = read_token(sj, n, lane);
        scan_window(sj, n, lane, L, merge_partials(&parts[lane < rj.K ? lane : 0], lane < L ? 1 : 0), tr);
    }
}

// ---- self-test of the bounded wait ----------------------------------------------------------------
// One warp waits on an mbarrier that nothing ever completes, with the same bounded wait and the same
// report as the bulk-copy kernel: the wait runs out, the warp sets PPOW_FLAG_DEVICE_TIMEOUT and returns.
__global__ void wait_timeout_selftest_kernel(WsHeader *header, uint32_t probes)
{
    __shared__ __align__(8) uint64_t bar;
    const uint32_t bar_addr = smem_addr(&bar);
    if (threadIdx.x == 0) {
        mbar_init(bar_addr, 1);
        mbar_init_fence();
    }
    __syncwarp();
    if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_addr, 0u, probes))) {
        if (threadIdx.x == 0) atomicOr(&header->error_flags, (unsigned)PPOW_FLAG_DEVICE_TIMEOUT);
    }
}

// ---- host side ----------------------------------------------------------------------------------

static bool params_ok(const ppow_params *p)
{
    if (!p) return false;
    if (p->N < 0 || p->K < 1 || p->V < 2) return false;
    if (p->dtype != PPOW_F32 && p->dtype != PPOW_BF16 && p->dtype != PPOW_F16) return false;
    if (p->mode != PPOW_GREEDY && p->mode != PPOW_STOCHASTIC) return false;
    if (!(p->temperature > 0.0f) || !isfinite(p->temperature)) return false;
    if (!(p->c >= 0.0f) || !isfinite(p->c)) return false;
    if (!isfinite(p->eta) || !isfinite(p->eps)) return false;
    if ((int64_t)p->N * p->K > (int64_t)1 << 26) return false;   // rows << MAX_SHIFT must fit 32 bits
    return true;
}

// The work plan depends only on (N, K, V, dtype), so that the workspace size is a pure function of the
// parameters.  Measured on B200 (per-warp timeline of the kernel): an item should be as long as the
// balance allows, because every item ends with a warp reduction worth more than half a tile of work; but
// the warps run at speeds that differ by +-20 % and finish their last items spread over one item's
// duration, which on a launch of a few hundred microseconds is 10-15 % of the time.  So the items shrink
// as the work runs out (guided self-scheduling, fixed ahead of time): a row whose distance from the last
// row leaves R tiles of work still to hand out is cut into items of at most R / (resident warps) tiles (a warp's
// share of what is left), rounded down to 64, 32, 16, 8 or 4.  Warps run at speeds that differ by +-20 % (by SM), so a slow warp
// that takes an item of a warp's whole remaining share ends late by a fifth of that item; on rows of 64 tiles
// and more, where an item end is cheap next to the item, the items therefore shrink half an item length earlier
// (measured: +2 % on a 256-window launch of the headline shape, within noise on the full workloads; on the short rows of the
// Vicuna-like workload the extra item ends cost 1 %, so those keep the whole share).
constexpr int64_t WORKER_WARPS = 148 * PIPE_MIN_CTAS * PIPE_WARPS;   // resident warps of the bulk-copy kernel on a B200

static int shift_for(int64_t tiles, int64_t item_tiles)
{
    int sh = 0;
    while (sh < MAX_SHIFT && ((tiles + ((int64_t)1 << sh) - 1) >> sh) > item_tiles && ((int64_t)2 << sh) <= tiles) ++sh;
    return sh;
}

static WorkPlan make_plan(const ppow_params *p)
{
    WorkPlan plan;
    const int64_t rows = (int64_t)p->N * p->K;
    const int64_t tile_logits = (int64_t)TILE_UNITS * (p->dtype == PPOW_F32 ? 4 : 8);
    const int64_t tiles = ((int64_t)p->V + tile_logits - 1) / tile_logits;   // per row
    plan.tiles = (int32_t)tiles;
    // class i holds items of at most 64 >> i tiles; it ends (and the next class starts) at the first row from
    // which fewer than margin * (64 >> i) * WORKER_WARPS tiles are still to come
    uint32_t item = 0;
    int64_t row = 0;
    for (int i = 0; i < PLAN_CLASSES; ++i) {
        int64_t end = rows;   // first row of the next class
        if (i + 1 < PLAN_CLASSES) {
            const int64_t margin_num = tiles >= 64 ? 3 : 2;   // halves: 3/2 of the item length for long rows, else 1
            const int64_t from_end = (margin_num * (int64_t)(64 >> i) * WORKER_WARPS / 2 + tiles - 1) / tiles;
            end = rows > from_end ? rows - from_end : 0;
        }
        if (end < row) end = row;
        plan.shift[i] = shift_for(tiles, 64 >> i);
        plan.item_begin[i] = item;
        plan.row_begin[i] = (int32_t)row;
        item += (uint32_t)((end - row) << plan.shift[i]);
        row = end;
    }
    plan.item_begin[PLAN_CLASSES] = item;
    plan.row_begin[PLAN_CLASSES] = (int32_t)row;
    return plan;
}

static bool takes_small_path(const ppow_params *p)
{
    const size_t esize = p->dtype == PPOW_F32 ? 4 : 2;
    return (size_t)p->V * esize <= SMALL_ROW_BYTES && 2 * (size_t)p->N * p->K * p->V * esize <= SMALL_TOTAL_BYTES;
}

// CTAs of a row kernel that are resident on the whole device at once.  Looked up once per (device, kernel)
// and remembered: the dynamic shared memory opt-in, the occupancy query and the SM count are host calls
// of several microseconds each, as much as a small problem's whole launch.  (Launch limits of a device are
// the only thing the library remembers between calls; concurrent first calls store the same value.)
constexpr int CACHE_DEVICES = 64, CACHE_KERNELS = 18;
static std::atomic<int> g_resident_ctas[CACHE_DEVICES][CACHE_KERNELS];

static int resident_ctas(int dev, int kernel_index, const void *kernel, int threads, size_t dyn_smem)
{
    const bool cached = dev >= 0 && dev < CACHE_DEVICES;
    if (cached) {
        const int v = g_resident_ctas[dev][kernel_index].load(std::memory_order_relaxed);
        if (v > 0) return v;
    }
    int sms = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (dyn_smem > 0 &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_smem) != cudaSuccess)
        return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, dyn_smem) != cudaSuccess || per_sm < 1)
        return 0;
    const int v = sms * per_sm;
    if (cached) g_resident_ctas[dev][kernel_index].store(v, std::memory_order_relaxed);
    return v;
}

}  // namespace ppow

using namespace ppow;

extern "C" size_t ppow_score_workspace_bytes(const ppow_params *params)
{
    if (!params_ok(params) || params->K > 32) return 0;
    return WS_HEADER_BYTES + (size_t)make_plan(params).item_begin[PLAN_CLASSES] * sizeof(RowPartial);
}

extern "C" int ppow_score_kernel_launches(const ppow_params *params)
{
    if (!params_ok(params) || params->K > 32 || params->N == 0) return 0;
    return takes_small_path(params) ? 1 : 2;
}

extern "C" ppow_status ppow_score_windows_traced(const ppow_params *params,
                                                 const void *draft_logits, const void *target_logits,
                                                 const int32_t *draft_tokens, const float *uniforms,
                                                 const int32_t *valid_len, const float *ref_logp,
                                                 const ppow_outputs *out,
                                                 void *workspace, size_t workspace_bytes, void *cuda_stream,
                                                 void *event_reduce_begin, void *event_reduce_end)
{
    if (!params_ok(params) || !out) return PPOW_ERR_INVALID_ARG;
    if (params->K > 32) return PPOW_ERR_UNSUPPORTED;
    if (params->N == 0) return PPOW_OK;
    if (!draft_logits || !target_logits || !draft_tokens || !out->accepted_len) return PPOW_ERR_INVALID_ARG;
    if (params->mode == PPOW_STOCHASTIC && !uniforms) return PPOW_ERR_INVALID_ARG;
    const size_t esize = params->dtype == PPOW_F32 ? 4 : 2;
    if (((uintptr_t)draft_logits % esize) || ((uintptr_t)target_logits % esize)) return PPOW_ERR_INVALID_ARG;
    const size_t need = ppow_score_workspace_bytes(params);
    if (!workspace || ((uintptr_t)workspace % 256) || workspace_bytes < need) return PPOW_ERR_WORKSPACE;

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    WsHeader *header = (WsHeader *)workspace;
    RowPartial *partials = (RowPartial *)((char *)workspace + WS_HEADER_BYTES);
    if (cudaMemsetAsync(header, 0, WS_HEADER_BYTES, stream) != cudaSuccess) return PPOW_ERR_CUDA;

    const WorkPlan plan = make_plan(params);
    const float s = (float)(1.4426950408889634074 / (double)params->temperature);

    RowJob rj;
    rj.target = target_logits; rj.draft = draft_logits; rj.valid_len = valid_len;
    rj.partials = partials; rj.header = header;
    rj.N = params->N; rj.K = params->K; rj.V = params->V;
    rj.plan = plan;
    rj.total_items = plan.item_begin[PLAN_CLASSES];
    rj.s = s;

    ScanJob sj;
    sj.target = target_logits; sj.draft = draft_logits; sj.tokens = draft_tokens; sj.uniforms = uniforms;
    sj.valid_len = valid_len; sj.ref_logp = ref_logp; sj.partials = partials; sj.header = header;
    sj.out = *out;
    sj.N = params->N; sj.K = params->K; sj.V = params->V; sj.dtype = params->dtype; sj.mode = params->mode;
    sj.plan = plan; sj.s = s; sj.c = params->c; sj.eta = params->eta; sj.eps = params->eps;
    sj.ln_v = log((double)params->V);
    const bool rev = out->kl_rev != nullptr || out->kl_rev_mean != nullptr;

    // a few megabytes of short rows: one launch for the whole pass (the events bracket that launch)
    if (takes_small_path(params)) {
        if (event_reduce_begin && cudaEventRecord((cudaEvent_t)event_reduce_begin, stream) != cudaSuccess)
            return PPOW_ERR_CUDA;
        rj.units_per_row = 0;
        rj.tile_logits = 0;
        const dim3 grid((unsigned)params->N), block((unsigned)params->K * 32u);
        if (params->dtype == PPOW_F32) {
            if (rev) score_small_kernel<float, true><<<grid, block, 0, stream>>>(rj, sj);
            else score_small_kernel<float, false><<<grid, block, 0, stream>>>(rj, sj);
        } else if (params->dtype == PPOW_F16) {
            if (rev) score_small_kernel<half_bits, true><<<grid, block, 0, stream>>>(rj, sj);
            else score_small_kernel<half_bits, false><<<grid, block, 0, stream>>>(rj, sj);
        } else {
            if (rev) score_small_kernel<uint16_t, true><<<grid, block, 0, stream>>>(rj, sj);
            else score_small_kernel<uint16_t, false><<<grid, block, 0, stream>>>(rj, sj);
        }
        if (cudaGetLastError() != cudaSuccess) return PPOW_ERR_CUDA;
        if (event_reduce_end && cudaEventRecord((cudaEvent_t)event_reduce_end, stream) != cudaSuccess)
            return PPOW_ERR_CUDA;
        return PPOW_OK;
    }

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PPOW_ERR_CUDA;

    // The bulk-copy kernel reads 16-byte aligned units.  Rows of whole aligned units are the plain case; rows that
    // start inside a unit (V not a multiple of the logits per unit, or a base pointer off a 16-byte boundary) are
    // read from the aligned address below their start with their first and last unit masked, which needs both
    // tensors at the same offset within a unit.  Tensors at different offsets take the scalar kernel.
    const int epu = params->dtype == PPOW_F32 ? FmtF32::EPU : FmtBf16::EPU;   // 8 logits per unit for both 16-bit types
    const bool vec_ok = ((uintptr_t)draft_logits % 16) == ((uintptr_t)target_logits % 16);
    rj.shifted = (params->V % epu != 0) || ((uintptr_t)target_logits % 16 != 0);
    rj.units_per_row = params->V / epu;
    rj.tile_logits = TILE_UNITS * epu;
    rj.es_shift = params->dtype == PPOW_F32 ? 2 : 1;
    rj.row_bytes = (int64_t)params->V * (int64_t)esize;
    // one warp per work item in every row kernel: a grid that fills the GPU, or fewer CTAs when there is little work.
    // The kernels that also accumulate the sum for KL(Q||P) run only when that output is asked for.
    const void *kernel;
    int threads = ROW_THREADS;
    size_t dyn_smem = 0;
    if (vec_ok) {
        const bool sh = rj.shifted != 0;
#define PPOW_PIPE(FMT) (rev ? (sh ? (const void *)row_reduce_pipe_kernel<true, FMT, true> : (const void *)row_reduce_pipe_kernel<true, FMT, false>) \
                            : (sh ? (const void *)row_reduce_pipe_kernel<false, FMT, true> : (const void *)row_reduce_pipe_kernel<false, FMT, false>))
        kernel = params->dtype == PPOW_BF16 ? PPOW_PIPE(FmtBf16) : params->dtype == PPOW_F16 ? PPOW_PIPE(FmtF16) : PPOW_PIPE(FmtF32);
#undef PPOW_PIPE
        threads = PIPE_WARPS * 32;
        dyn_smem = PIPE_SMEM_BYTES;
    } else if (params->dtype == PPOW_BF16) {
        kernel = rev ? (const void *)row_reduce_generic_kernel<uint16_t, true>
                     : (const void *)row_reduce_generic_kernel<uint16_t, false>;
    } else if (params->dtype == PPOW_F16) {
        kernel = rev ? (const void *)row_reduce_generic_kernel<half_bits, true>
                     : (const void *)row_reduce_generic_kernel<half_bits, false>;
    } else {
        kernel = rev ? (const void *)row_reduce_generic_kernel<float, true>
                     : (const void *)row_reduce_generic_kernel<float, false>;
    }
    const int kernel_index = (vec_ok ? (rj.shifted ? 12 : 6) : 0) + 2 * params->dtype + (rev ? 1 : 0);
    const int resident = resident_ctas(dev, kernel_index, kernel, threads, dyn_smem);
    if (resident < 1) return PPOW_ERR_CUDA;
    const unsigned warps_per_cta = (unsigned)threads / 32;
    const unsigned ctas_needed = (rj.total_items + warps_per_cta - 1) / warps_per_cta;
    unsigned grid = (unsigned)resident;
    if (grid > ctas_needed) grid = ctas_needed;

    if (event_reduce_begin && cudaEventRecord((cudaEvent_t)event_reduce_begin, stream) != cudaSuccess)
        return PPOW_ERR_CUDA;
    void *kargs[] = {(void *)&rj};
    if (cudaLaunchKernel(kernel, dim3(grid), dim3((unsigned)threads), kargs, dyn_smem, stream) != cudaSuccess ||
        cudaGetLastError() != cudaSuccess) {
        // a context that was torn down and rebuilt has lost the shared-memory opt-in: look the limits up again next time
        if (dev >= 0 && dev < CACHE_DEVICES) g_resident_ctas[dev][kernel_index].store(0, std::memory_order_relaxed);
        return PPOW_ERR_CUDA;
    }
    if (event_reduce_end && cudaEventRecord((cudaEvent_t)event_reduce_end, stream) != cudaSuccess)
        return PPOW_ERR_CUDA;

    const unsigned scan_grid = (unsigned)(((size_t)params->N * 32 + SCAN_THREADS - 1) / SCAN_THREADS);
    window_scan_kernel<<<scan_grid, SCAN_THREADS, 0, stream>>>(sj);
    if (cudaGetLastError() != cudaSuccess) return PPOW_ERR_CUDA;
    return PPOW_OK;
}

extern "C" ppow_status ppow_score_windows(const ppow_params *params,
                                          const void *draft_logits, const void *target_logits,
                                          const int32_t *draft_tokens, const float *uniforms,
                                          const int32_t *valid_len, const float *ref_logp,
                                          const ppow_outputs *out,
                                          void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return ppow_score_windows_traced(params, draft_logits, target_logits, draft_tokens, uniforms, valid_len,
                                     ref_logp, out, workspace, workspace_bytes, cuda_stream, nullptr, nullptr);
}

#ifdef PPOW_CHECKED
namespace ppow { int read_check_counters_score(unsigned int *f, unsigned int *s) { return read_check_counters(f, s); } }
#endif

extern "C" ppow_status ppow_timeline_read(uint64_t *words_host, size_t warps)
{
    if (!words_host) return PPOW_ERR_INVALID_ARG;
#ifdef PPOW_TIMELINE
    if (warps > (size_t)TIMELINE_WARPS) return PPOW_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return PPOW_ERR_CUDA;
    return cudaMemcpyFromSymbol(words_host, g_timeline, warps * TIMELINE_WORDS * sizeof(unsigned long long)) == cudaSuccess
               ? PPOW_OK
               : PPOW_ERR_CUDA;
#else
    (void)warps;
    return PPOW_ERR_UNSUPPORTED;   // not the timeline build
#endif
}

extern "C" ppow_status ppow_selftest_wait_timeout(void *workspace, size_t workspace_bytes, uint32_t probes,
                                                  void *cuda_stream)
{
    if (!workspace || ((uintptr_t)workspace % 256) || workspace_bytes < WS_HEADER_BYTES) return PPOW_ERR_WORKSPACE;
    if (probes < 1 || probes > (1u << 16)) return PPOW_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(workspace, 0, WS_HEADER_BYTES, stream) != cudaSuccess) return PPOW_ERR_CUDA;
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>((WsHeader *)workspace, probes);
    return cudaGetLastError() == cudaSuccess ? PPOW_OK : PPOW_ERR_CUDA;
}

extern "C" ppow_status ppow_read_error_flags(const void *workspace, uint32_t *flags_host, void *cuda_stream)
{
    if (!workspace || !flags_host) return PPOW_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const WsHeader *header = (const WsHeader *)workspace;
    unsigned int v = 0;
    if (cudaMemcpyAsync(&v, &header->error_flags, sizeof v, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return PPOW_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return PPOW_ERR_CUDA;
    *flags_host = v;
    return (v & PPOW_FLAG_DEVICE_TIMEOUT) ? PPOW_ERR_DEVICE_TIMEOUT : PPOW_OK;
}
