// The three kernels behind decode_attn(): plan (split schedule), partition (page gather by TMA,
// QK^T, online fp32 softmax, PV) and merge (log-sum-exp combine).  sm_100a only.
//
// Work model.  A "tile" is TILE_T consecutive tokens starting at a multiple of TILE_T.  Sequence b
// contributes nt_b tiles (those that intersect its attended range [lo_b, L_b)) for each of its Hkv
// KV heads.  All (b, kv head, tile) triples, in row-major order, form one line of `total` tiles.
// The line is cut into work units: its first part into one large unit per thread block (each block
// starts on its own, so no block waits for a ticket), the rest into many small units that the
// blocks take from an atomic ticket counter as they finish -- thread blocks do not all stream at
// the same speed, and the small units even out their finishing times.  A unit covers a run of
// (b, kv head) pairs; the pairs it covers completely are written straight to `out`, the (at most
// two) pairs it shares with neighbouring units go to a partial slot and are combined by the merge
// kernel.
#pragma once
#include "da_ptx.cuh"

namespace da {

constexpr int HEAD_DIM = 128;
constexpr int NCW = 4;                      // consumer warps per block; each owns 16 tokens of a tile
constexpr int TILE_T = 16 * NCW;            // tokens per pipeline stage, bf16 cache
constexpr int TILE_T8 = 32 * NCW;           // tokens per pipeline stage, 8-bit cache (a warp owns 32)
constexpr int KV_BYTES = TILE_T * 256;      // a K (or V) tile: TILE_T rows of 128 bf16, or TILE_T8 rows of 128 bytes
static_assert(TILE_T8 * 128 == KV_BYTES, "both cache types fill a stage");
constexpr float P8_SHIFT = 15.f;            // 8-bit cache: softmax weights are carried as 2^15 * p (f16 high + low)
constexpr int STAGE_BYTES = 2 * KV_BYTES;   // K tile followed by V tile
constexpr int NTHREADS = (NCW + 1) * 32;    // + one producer warp (with two column sets: 2 * NCW + 1 warps)
constexpr int PLAN_THREADS = 512;
constexpr int PLAN_SMEM_SEQS = 4096;
constexpr int MIN_TAIL_UNIT_TILES = 4;      // a ticketed unit is never cut smaller than this
constexpr int PLAN_BLOCKS = 16;             // the plan kernel's grid: each block cuts a slice of the units
constexpr int MERGE_WARP_SPLITS = 8;        // pairs cut into more splits are merged by a whole block
                                            // (a warp keeps eight partial rows in flight: one pass)
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

// Timeline build (-DDA_TIMELINE, a diagnostic library beside the normal one): the kernels leave
// %globaltimer stamps in g_timeline, which decode_attn_timeline() copies out.  Rows 0 .. 1023: thread
// blocks of the partition kernel -- column 0 entry, 1 past the wait for the plan, 2 first tile ready,
// 3 last tile consumed, 4 exit, 5 tiles consumed, 6 (b, kv head) items finished.  Rows TL_MERGE .. + 7:
// the merge kernel's first eight blocks -- 0 resident, 1 released by the partition kernel, 2 exit;
// row TL_MERGE + 8, column 2: the latest exit of any merge block.  Rows TL_PLAN .. + 7: the plan
// kernel's blocks -- 0 entry, 1 exit, 2 past the wait for the kernel before it in the stream, 3 lengths scanned, 4 cut made,
// 5 units written.  Rows TL_PREFIX .. + 5: thread block 0 of the prefix kernel, cycles (clock64) that one
// warp of each role spent in its phases, summed over the block's tiles -- softmax warp 0: 0 waiting for the
// scores, 1 loading them and agreeing on the row maximum, 2 weights (exp2, high/low parts, a rescale of O),
// 3 storing P and arriving, 4 after the last tile, 5 tiles, 6 cycles from entry to the end, 7 the same span
// in ns; score MMA warp: 0 waiting for the PV products, 1 for K, 2 issuing; the two PV MMA warps: 0 waiting for
// P, 1 for V, 2 issuing; the K and V loader warps: 0 waiting for a free buffer, 1 issuing the copies.
// In the normal build DA_TL() is empty and nothing is kept.
constexpr int TL_ROWS = 1064, TL_COLS = 8, TL_MERGE = 1024, TL_PLAN = 1036, TL_PREFIX = 1052;
#ifdef DA_TIMELINE
__device__ unsigned long long g_timeline[TL_ROWS][TL_COLS];
#define DA_TL(row, col) (g_timeline[(row)][(col)] = globaltimer_ns())
#define DA_TL_SET(row, col, value) (g_timeline[(row)][(col)] = (unsigned long long)(value))
#define DA_TL_MAX(row, col) atomicMax(&g_timeline[(row)][(col)], (unsigned long long)globaltimer_ns())
// phase counters: `acc` is a per-thread array, DA_PH(acc, slot, t) adds the cycles since t and restarts t
#define DA_PH_DECL(acc, t) long long acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; long long t = clock64()
#define DA_PH(acc, slot, t) do { const long long now_ = clock64(); acc[(slot)] += now_ - (t); (t) = now_; } while (0)
#define DA_PH_STORE(row, acc) do { for (int i_ = 0; i_ < 8; ++i_) g_timeline[(row)][i_] = (unsigned long long)acc[i_]; } while (0)
#else
#define DA_TL(row, col) ((void)0)
#define DA_TL_SET(row, col, value) ((void)0)
#define DA_TL_MAX(row, col) ((void)0)
#define DA_PH_DECL(acc, t) ((void)0)
#define DA_PH(acc, slot, t) ((void)0)
#define DA_PH_STORE(row, acc) ((void)0)
#endif

// flags of a tile's descriptor (written by the producer warp, read by the consumer warps)
constexpr int TILE_ITEM_END = 1;   // last tile this unit holds of its (b, kv head) pair
constexpr int TILE_WHOLE = 2;      // the unit holds every tile of the pair: write `out` directly
constexpr int TILE_STOP = 4;       // no more work for this block (carries no data)
constexpr int TILE_SPLITS_SHIFT = 8;   // direct mode: bits 8.. = blocks that share the tile's pair
constexpr int DIRECT_MAX_PAIRS = 512;  // direct mode: (sequence, KV head) pairs of a call (one counter each)

// A thread block's consumer warps form CSETS column sets of NCW warps.  Warp (set cs, token group tw) owns
// tokens WT * tw .. of every tile and the NT8 column tiles (8 query heads each) cs * NT8 .. of the KV
// group's (virtual) heads: one set of 1 or 2 column tiles serves up to 16 heads with two blocks per SM;
// two sets of 2 or 3 serve up to 32 or 48 (several new tokens per sequence) with one block per SM -- both
// sets read the same K and V tiles from shared memory, so K and V still cross HBM once.
template <int NT8, int CSETS>
struct PartCfg {
    static constexpr int NSTAGES = CSETS == 1 ? ((NT8 == 1) ? 3 : 2) : ((NT8 == 2) ? 4 : 3);
    static constexpr int HEADS_SET = NT8 * 8;                            // padded heads of one column set
    static constexpr int HEADS = CSETS * HEADS_SET;                      // padded heads per KV group
    static constexpr int THREADS = (NCW * CSETS + 1) * 32;               // consumer warps + one producer warp
    static constexpr int MIN_BLOCKS = CSETS == 1 ? 2 : 1;
    static constexpr int XBUF_BYTES = NCW * HEADS * HEAD_DIM * 4;        // cross-warp combine buffer
    static constexpr int STATS_BYTES = 2 * NCW * HEADS * 4;              // (m, l) per warp and head
    static constexpr int OFF_XBUF = NSTAGES * STAGE_BYTES;
    static constexpr int OFF_STATS = OFF_XBUF + XBUF_BYTES;
    static constexpr int OFF_META = OFF_STATS + STATS_BYTES;             // two int4 per stage
    static constexpr int OFF_BARS = OFF_META + NSTAGES * 32;             // full[NSTAGES], empty[NSTAGES], epi[2 * CSETS]
    static constexpr int OFF_FLAGS = OFF_BARS + (2 * NSTAGES + 2 * CSETS) * 8;   // abort flag
    static constexpr int SMEM_BYTES = OFF_FLAGS + 16;
    static_assert(SMEM_BYTES <= 232448, "a block must fit the 227 KB of shared memory an SM offers");
};

// What the plan kernel decides, read by the other two kernels.  Units 0 .. n_static-1 cut
// [0, static_w) into near-equal ranges (the first r_static of them one tile longer, q_static + 1);
// units n_static .. n_static+n_tail-1 cut [static_w, total) the same way.
struct PlanHeader {
    long long total;      // tiles over all (b, kv head) pairs
    long long static_w;   // tiles covered by the n_static large units (the rest: ticketed units)
    long long q_static, q_tail;   // floor(range / units) of the two cuts
    int r_static, r_tail;         // remainder of the two cuts
    int n_static;         // = thread blocks of the partition kernel
    int n_tail;           // ticketed units (0: none)
    int ticket;           // next ticketed unit to hand out (reset by the plan kernel)
    int kv_evict_first;   // K and V loads carry the L2 "evict first" policy (no pages seem to be shared)
    int pad[2];
};
// Split pairs found by plan block k: how many with <= MERGE_WARP_SPLITS splits, how many with more.
struct MergeCounts {
    int n_small[PLAN_BLOCKS];
    int n_big[PLAN_BLOCKS];
};

struct PartParams {
    const __nv_bfloat16 *q;
    int64_t q_sb, q_sh;
    const int32_t *block_table;
    int64_t bt_sb;
    void *out;
    int64_t o_sb, o_sh;
    float *lse;
    int64_t l_sb, l_sh;
    const int4 *seq_info;     // {lo, L, first_tile, num_tiles} per sequence
    const int4 *unit_work;    // {b, kv_head, first tile (relative to the pair's first), tiles} per unit
    PlanHeader *hdr;
    float *part_o;            // [2 * units][HEADS][128]
    float *part_lse;          // [2 * units][HEADS]
    int32_t *status;
    int32_t B, Hkv, G, P, box_rows, num_pages, out_bf16;
    int32_t log2_P;           // P = 1 << log2_P

    float scale_log2;         // scale * log2(e)
    const float *k_scale, *v_scale;   // 8-bit cache: per-KV-head factors (NULL: 1)
    // Several new tokens per sequence (Lq > 1, causal among them): query token qi of KV group g's head hd
    // is "virtual head" qi * G + hd of that group; Gv = Lq * G <= 16 of them share one pass over K and V.
    // Query qi sits at position L - Lq + qi and attends tokens below L - Lq + qi + 1.
    int32_t Lq, Gv;
    int64_t q_sq, o_sq, l_sq;         // strides of the query-token dimension (0 when Lq == 1)
    int32_t unit_cap;                 // rows of unit_work; the partial arrays hold 2 * unit_cap slots
    int64_t max_pages;                // entries in a block-table row
    // Direct mode (direct_splits > 0; small calls, one token per sequence): no plan and no merge kernel.
    // Block x takes piece x % direct_splits of pair x / direct_splits = (b, kv head), works its tiles out
    // from seq_lens[b] itself and writes a partial to slot x; the block that finishes a pair last (a counter
    // per pair, left at zero again) folds the pieces and writes the result.
    int32_t direct_splits, window;
    const int32_t *seq_lens;
    int64_t sl_stride;
    int32_t *pair_counters;           // [DIRECT_MAX_PAIRS], zero between calls
    int32_t *fold_counters;           // [unit_cap][2]: two-piece pairs folded by the second block to finish; zero between calls
};

struct PlanParams {
    const int32_t *seq_lens;
    int64_t sl_stride;
    int4 *seq_info;
    int32_t *prefix;          // [B+1] exclusive prefix of num_tiles
    int4 *unit_work;
    int4 *merge_small, *merge_big;      // per split pair {pair id b * Hkv + g, first slot, first unit, splits};
                                        // plan block k appends at [k * merge_seg, ...)
    MergeCounts *merge_counts;
    int32_t merge_seg;
    PlanHeader *hdr;
    int32_t *status;
    int32_t B, Hkv, P, window;
    int32_t tile_t;           // tokens per tile (TILE_T or TILE_T8)
    int32_t min_len;          // a non-empty sequence shorter than this is an error (the new tokens of an extend call)
    int32_t first_token;      // tokens before this one are not attended (the cascade's suffix pass)
    // L2 policy of the K/V loads: 0 normal, 1 evict first, 2 decide here -- evict first unless many
    // sequences start on the same physical page (a shared prefix is re-read from L2 by every sharer).
    int32_t kv_policy;
    const int32_t *block_table;   // only read for kv_policy 2 (may be NULL otherwise)
    int64_t bt_sb;
    int32_t n_static, n_tail_max, static_frac_q8;   // large units; most ticketed units; share of the
                                                    // line given to the large units, in 1/256
    int64_t max_pages;
    int32_t fold_pairs;       // pairs cut in two by neighbouring thread blocks' own ranges are folded by the partition kernel
};

struct MergeParams {
    const int4 *seq_info;
    const int32_t *prefix;
    const PlanHeader *hdr;
    const int4 *merge_small, *merge_big;
    const MergeCounts *merge_counts;
    int32_t merge_seg;
    const float *part_o;
    const float *part_lse;
    void *out;
    int64_t o_sb, o_sh;
    float *lse;
    int64_t l_sb, l_sh;
    int32_t B, Hkv, G, heads_pad, out_bf16;
    int32_t Lq, Gv;           // as in PartParams
    int64_t o_sq, l_sq;
    int32_t unit_cap;         // as in PartParams
    int32_t *status;
};

__device__ __forceinline__ void report_status(int32_t *status, int code, int a, int b, int c)
{
    if (atomicCAS(status, 0, code) == 0) {
        status[1] = a;
        status[2] = b;
        status[3] = c;
    }
}

// Bounds-check build (-DDA_BOUNDS_CHECK, part of the diagnostic library; compute-sanitizer's stand-in
// where that tool is not available): every index the kernels form into the plan arrays, the merge
// lists, the partial slots, the block table and the result tensors is compared with its extent first.
// An index outside it is recorded in the status record as {DA_DEV_BOUNDS, site, index, extent} and the
// access is skipped.  In the normal build DA_IN_RANGE() is `true` and costs nothing.
#ifdef DA_BOUNDS_CHECK
__device__ __forceinline__ bool in_range(int32_t *status, long long idx, long long extent, int site)
{
    if (idx >= 0 && idx < extent)
        return true;
    report_status(status, 4 /* DA_DEV_BOUNDS */, site, (int)idx, (int)extent);
    return false;
}
#define DA_IN_RANGE(status, idx, extent, site) ::da::in_range((status), (long long)(idx), (long long)(extent), (site))
#else
#define DA_IN_RANGE(status, idx, extent, site) true
#endif

// Start of range c of a cut with quotient q and remainder r.
__host__ __device__ __forceinline__ long long cut_start(long long q, int r, int c)
{
    return q * c + (c < r ? c : r);
}
// The range of that cut that holds offset w.
__host__ __device__ __forceinline__ int cut_owner(long long q, int r, long long w)
{
    const long long big = (long long)r * (q + 1);
    if (w < big)
        return (q + 1 < 0x7fffffffll && w < 0x7fffffffll) ? (int)((unsigned)w / (unsigned)(q + 1)) : (int)(w / (q + 1));
    const long long x = w - big;
    return r + ((q < 0x7fffffffll && x < 0x7fffffffll) ? (int)((unsigned)x / (unsigned)q) : (int)(x / q));
}
__host__ __device__ __forceinline__ long long unit_start(const PlanHeader &h, int u)
{
    if (u < h.n_static)
        return cut_start(h.q_static, h.r_static, u);
    if (u >= h.n_static + h.n_tail)
        return h.total;
    return h.static_w + cut_start(h.q_tail, h.r_tail, u - h.n_static);
}
__host__ __device__ __forceinline__ int unit_owner(const PlanHeader &h, long long w)
{
    if (w < h.static_w)
        return cut_owner(h.q_static, h.r_static, w);
    return h.n_static + cut_owner(h.q_tail, h.r_tail, w - h.static_w);
}
// Static units that hold tiles: with fewer tiles than thread blocks the last ones are empty.
__host__ __device__ __forceinline__ int static_units_in_use(const PlanHeader &h)
{
    return (int)(h.static_w < h.n_static ? h.static_w : h.n_static);
}
// How many units hold a piece of the pair whose tiles are [w0, w0 + nt) (nt > 0), and the first.
__host__ __device__ __forceinline__ int pair_splits(const PlanHeader &h, long long w0, int nt, int *u_first)
{
    const int uf = unit_owner(h, w0), ul = unit_owner(h, w0 + nt - 1);
    const int n_full = static_units_in_use(h);
    *u_first = uf;
    return (ul - uf + 1) - ((uf < n_full && ul >= h.n_static) ? h.n_static - n_full : 0);
}

// =====================================================================================  plan
// PLAN_BLOCKS blocks.  Every block computes, per sequence, the attended range, its tiles and the
// exclusive prefix of tiles (block 0 stores them), and the cut of the line into units; then each
// block works out, for its slice of the units, where the unit starts and whether it is the unit
// that makes a pair "split" (such pairs go to the merge lists).
__global__ void __launch_bounds__(PLAN_THREADS, 1) plan_kernel(PlanParams p)
{
    __shared__ int n_small_s, n_big_s;
    __shared__ int warp_tot[PLAN_THREADS / 32];
    __shared__ int running_s;
    __shared__ int prefix_s[PLAN_SMEM_SEQS + 1];   // copy of the prefix for the searches below
    __shared__ PlanHeader hdr_s;
    __shared__ int nonempty_s, same_start_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0)
        DA_TL(TL_PLAN + blockIdx.x, 0);
    grid_launch_dependents();   // the partition kernel may set up its blocks while the plan is made
    // The plan kernel is itself launched with programmatic serialization, so that its blocks can be
    // placed while the kernel before it in the stream drains: nothing is read or written before that
    // kernel is complete.
    grid_dependency_wait();
    if (tid == 0)
        DA_TL(TL_PLAN + blockIdx.x, 2);
    const bool writer = blockIdx.x == 0;
    if (tid == 0) {
        running_s = 0;
        n_small_s = 0;
        n_big_s = 0;
        nonempty_s = 0;
        same_start_s = 0;
    }
    __syncthreads();

    for (int base = 0; base < p.B; base += PLAN_THREADS) {
        const int b = base + tid;
        int lo = 0, L = 0, first = 0, nt = 0;
        if (b < p.B) {
            // Does this sequence start (after the tokens a cascade call skips) on the same page as the first
            // sequence, or as the one before it?  The three entries are asked for together with the length
            // (entry first_token / P exists in every row: the host checked it against max_pages); they are
            // compared, never used as page ids, and may be unspecified for sequences that end before them.
            const bool probe = writer && p.kv_policy == 2;
            int pg = 0, pg_first = 0, pg_prev = 0;
            if (probe) {
                const int64_t j = p.first_token / p.P;
                pg = __ldg(p.block_table + (int64_t)b * p.bt_sb + j);
                pg_first = __ldg(p.block_table + j);
                pg_prev = __ldg(p.block_table + (int64_t)(b > 0 ? b - 1 : 0) * p.bt_sb + j);
            }
            L = p.seq_lens[(int64_t)b * p.sl_stride];
            if (L < 0 || (int64_t)L > p.max_pages * (int64_t)p.P) {
                if (writer)
                    report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, 0, L);
                L = 0;
            }
            if (L > 0 && (L < p.first_token || L < p.min_len)) {
                if (writer)
                    report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, L < p.min_len ? 2 : 1, L);
                L = 0;
            }
            if (probe && L > p.first_token) {
                atomicAdd(&nonempty_s, 1);
                if (b > 0 && (pg == pg_first || pg == pg_prev))
                    atomicAdd(&same_start_s, 1);
            }
            lo = (p.window > 0 && p.window < L) ? L - p.window : 0;
            lo = max(lo, min(p.first_token, L));
            if (L > lo) {
                first = lo / p.tile_t;
                nt = (L - 1) / p.tile_t - first + 1;
            }
        }
        // block-wide exclusive scan of nt
        int incl = nt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o)
                incl += y;
        }
        if (lane == 31)
            warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int w = lane < PLAN_THREADS / 32 ? warp_tot[lane] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o)
                    w += y;
            }
            if (lane < PLAN_THREADS / 32)
                warp_tot[lane] = w;   // inclusive over warps
        }
        __syncthreads();
        const int run = running_s;
        const int excl = run + (warp ? warp_tot[warp - 1] : 0) + incl - nt;
        if (b < p.B) {
            if (writer) {
                p.seq_info[b] = make_int4(lo, L, first, nt);
                p.prefix[b] = excl;
            }
            if (b < PLAN_SMEM_SEQS)
                prefix_s[b] = excl;
        }
        __syncthreads();
        if (tid == PLAN_THREADS - 1)
            running_s = run + warp_tot[PLAN_THREADS / 32 - 1];
        __syncthreads();
    }
    const int tiles_per_head = running_s;
    const bool in_smem = p.B <= PLAN_SMEM_SEQS;
    if (tid == 0)
        DA_TL(TL_PLAN + blockIdx.x, 3);
    if (tid == 0) {
        if (writer)
            p.prefix[p.B] = tiles_per_head;
        if (in_smem)
            prefix_s[p.B] = tiles_per_head;
        // the cut: a share of the line to the large units, the rest to ticketed units of at least
        // MIN_TAIL_UNIT_TILES tiles each
        PlanHeader h;
        h.total = (long long)tiles_per_head * p.Hkv;
        h.n_static = p.n_static;
        long long tail_w = h.total * (256 - p.static_frac_q8) / 256;
        long long n_tail = tail_w / MIN_TAIL_UNIT_TILES;
        if (n_tail > p.n_tail_max)
            n_tail = p.n_tail_max;
        if (n_tail <= 0) {
            n_tail = 0;
            tail_w = 0;
        }
        h.n_tail = (int)n_tail;
        h.static_w = h.total - tail_w;
        h.q_static = h.static_w / h.n_static;
        h.r_static = (int)(h.static_w % h.n_static);
        h.q_tail = n_tail ? tail_w / n_tail : 0;
        h.r_tail = n_tail ? (int)(tail_w % n_tail) : 0;
        h.ticket = 0;
        h.kv_evict_first = p.kv_policy == 2 ? (4 * same_start_s < nonempty_s || nonempty_s < 2) : p.kv_policy;
        h.pad[0] = h.pad[1] = 0;
        hdr_s = h;
        if (writer)
            *p.hdr = h;
    }
    __syncthreads();   // this block's global writes are visible to itself after the barrier
    if (tid == 0)
        DA_TL(TL_PLAN + blockIdx.x, 4);
    // With more sequences than fit in shared memory the searches read block 0's global copy.
    // (Blocks cannot wait for one another, so in that case block 0 alone cuts all the units.)
    const int *prefix = in_smem ? prefix_s : p.prefix;
    const PlanHeader h = hdr_s;
    const int n_units = h.n_static + h.n_tail;
    const int n_full = static_units_in_use(h);
    const int units_max = p.n_static + p.n_tail_max;
    const int nblk = in_smem ? (int)gridDim.x : 1;
    const int slice = (units_max + nblk - 1) / nblk;
    const int u_begin = (int)blockIdx.x * slice;
    const int u_end = ((int)blockIdx.x < nblk) ? min(u_begin + slice, units_max) : u_begin;
    int4 *my_small = p.merge_small + (size_t)blockIdx.x * p.merge_seg;
    int4 *my_big = p.merge_big + (size_t)blockIdx.x * p.merge_seg;
    // room in this block's segment of the lists; a block that cuts all the units alone (nblk == 1) fills
    // the segments one after another, which the merge kernel's walk over the per-block counts reads back
    // as one contiguous list
    [[maybe_unused]] const int list_room = nblk == 1 ? p.merge_seg * PLAN_BLOCKS : p.merge_seg;
    // where tile w of the line lies: sequence, KV head, tile of the pair, tiles of the pair
    struct Where { int b, g, rel, nt; };
    auto locate = [&](long long w) {
        const int x = (w < 0x7fffffffll) ? (int)((unsigned)w / (unsigned)p.Hkv) : (int)(w / p.Hkv);
        // largest b with prefix[b] <= x; equal prefixes (empty sequences) resolve to the last
        int lo_i = 0, hi_i = p.B;   // invariant: prefix[lo_i] <= x < prefix[hi_i]
        while (hi_i - lo_i > 1) {
            const int mid = (lo_i + hi_i) >> 1;
            if (prefix[mid] <= x)
                lo_i = mid;
            else
                hi_i = mid;
        }
        Where r;
        r.b = lo_i;
        r.nt = prefix[r.b + 1] - prefix[r.b];
        const int rem = (int)(w - (long long)prefix[r.b] * p.Hkv);   // < Hkv * nt
        r.g = rem / r.nt;
        r.rel = rem - r.g * r.nt;
        return r;
    };
    // Does static unit v (0 < v < n_full) start inside a pair that began in unit v-1 and ends inside v?  Such a
    // pair has exactly two pieces, in two thread blocks' own ranges: the partition kernel folds it itself (the
    // block that finishes its piece second), so it is kept off the merge lists.  bit 0: yes; bit 2: the pair
    // is the FIRST item of unit v-1 (that unit starts at the pair's first tile).
    auto two_piece_start = [&](int v) {
        if (!p.fold_pairs || v <= 0 || v >= n_full)
            return 0;
        const long long vs = unit_start(h, v), ve = unit_start(h, v + 1);
        if (ve <= vs)
            return 0;
        const Where at = locate(vs);
        const long long w0 = vs - at.rel, prev_start = unit_start(h, v - 1);
        if (at.rel == 0 || prev_start > w0 || w0 + at.nt > ve)
            return 0;
        return 1 | (prev_start == w0 ? 4 : 0);
    };
    for (int u = u_begin + tid; u < u_end; u += PLAN_THREADS) {
        int4 uw = make_int4(0, 0, 0, 0);
        if (u < n_units) {
            const long long ws = unit_start(h, u), we = unit_start(h, u + 1);
            if (we > ws) {
                const Where at = locate(ws);
                const int b = at.b, nt = at.nt, g = at.g, rel = at.rel;
                // unit flags, above the KV head: 1 = my first item is the second piece of a two-piece pair,
                // 2 = my last item is the first piece of one, 4 = (with 1) my partner is its unit's first item
                const int mine = two_piece_start(u), next = two_piece_start(u + 1);
                uw = make_int4(b, g | ((mine | ((next & 1) << 1)) << 16), rel, (int)(we - ws));
                // A unit that starts inside a pair marks that pair as split.  The pair is listed once,
                // by the first such unit: the one whose predecessor holds the pair's first tile.
                if (rel > 0 && !(mine & 1)) {
                    const int prev = (u == h.n_static) ? n_full - 1 : u - 1;
                    const long long w0 = ws - rel, prev_start = unit_start(h, prev);
                    if (prev_start <= w0) {
                        int uf;
                        const int ns = pair_splits(h, w0, nt, &uf);
                        // the pair is the first item of unit `prev` only if that unit starts at it
                        const int4 e = make_int4(b * p.Hkv + g, 2 * prev + (prev_start == w0 ? 0 : 1), prev, ns);
                        if (ns > MERGE_WARP_SPLITS) {
                            const int at = atomicAdd(&n_big_s, 1);
                            if (DA_IN_RANGE(p.status, at, list_room, 1))
                                my_big[at] = e;
                        } else {
                            const int at = atomicAdd(&n_small_s, 1);
                            if (DA_IN_RANGE(p.status, at, list_room, 2))
                                my_small[at] = e;
                        }
                    }
                }
            }
        }
        if (DA_IN_RANGE(p.status, u, units_max, 3))
            p.unit_work[u] = uw;
    }
    __syncthreads();
    if (tid == 0) {
        DA_TL(TL_PLAN + blockIdx.x, 5);
        p.merge_counts->n_small[blockIdx.x] = n_small_s;
        p.merge_counts->n_big[blockIdx.x] = n_big_s;
        DA_TL(TL_PLAN + blockIdx.x, 1);
    }
}

// =====================================================================================  partition
// Layout of a K or V tile in shared memory.  One TMA box is box_rows token rows of one page, all
// 128 columns, written as two 64-column planes of box_rows 128-byte rows with the 128-byte swizzle
// (16-byte chunk index XORed with the row's low three bits).  A tile is TILE_T / box_rows such boxes
// back to back.  Row `row` of the tile therefore starts at row_offset(); its chunk c (0..15 along
// head_dim) is at  + (c >> 3) * plane_bytes + (((c & 7) ^ (row & 7)) << 4).
__device__ __forceinline__ uint32_t row_offset(int row, int box_rows)
{
    return (uint32_t)((row / box_rows) * (box_rows * 256) + (row % box_rows) * 128);
}

template <int NT8, bool KV8, int CSETS>
__global__ void __launch_bounds__((PartCfg<NT8, CSETS>::THREADS), (PartCfg<NT8, CSETS>::MIN_BLOCKS))
partition_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const PartParams p)
{
    using C = PartCfg<NT8, CSETS>;
    constexpr int HS = C::HEADS_SET;                   // padded heads of one column set
    constexpr int TT = KV8 ? TILE_T8 : TILE_T;        // tokens per tile
    constexpr uint32_t ROW_BYTES = KV8 ? 128u : 256u;  // one token row of one KV head
    constexpr int NSTAGES = C::NSTAGES;
    constexpr int HEADS = C::HEADS;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t smem_base = smem_u32(smem);
    float *xbuf = reinterpret_cast<float *>(smem + C::OFF_XBUF);
    float *st_m = reinterpret_cast<float *>(smem + C::OFF_STATS);
    float *st_l = st_m + NCW * HEADS;
    int4 *meta = reinterpret_cast<int4 *>(smem + C::OFF_META);   // [stage][2]
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAGS);
    const uint32_t bar_full = smem_base + C::OFF_BARS;
    const uint32_t bar_empty = bar_full + NSTAGES * 8;
    const uint32_t bar_epi0 = bar_empty + NSTAGES * 8;  // two barriers per column set for the consumers' epilogue

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0 && blockIdx.x < TL_MERGE)
        DA_TL(blockIdx.x, 0);

    if ((smem_base & 1023u) != 0) {   // the swizzle pattern is a function of the address bits
        if (tid == 0)
            report_status(p.status, 3, -1, (int)blockIdx.x, (int)smem_base);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < NSTAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, NCW * CSETS);
        }
        for (int s = 0; s < 2 * CSETS; ++s)
            mbar_init(bar_epi0 + 8 * s, NCW);
        mbar_fence_init();
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    grid_launch_dependents();   // lets the merge kernel's blocks become resident early
    __syncthreads();
    grid_dependency_wait();     // the plan (and everything before it in the stream) is complete
    if (tid == 0 && blockIdx.x < TL_MERGE)
        DA_TL(blockIdx.x, 1);

    if (warp == NCW * CSETS) {
        // ------------------------------------------------------------------ producer warp
        // Lane -> (box, K|V).  A box is box_rows token rows (all 128 columns) of one page.
        const int nboxes = TT / p.box_rows;
        const int box = lane >> 1, is_v = lane & 1;
        const bool active = lane < nboxes * 2;
        const uint32_t box_bytes = (uint32_t)p.box_rows * ROW_BYTES;
        const CUtensorMap *tm = is_v ? &tm_v : &tm_k;
        const bool direct = p.direct_splits > 0;
        const int n_static = direct ? 0 : p.hdr->n_static, n_units = direct ? 0 : n_static + p.hdr->n_tail;
        uint32_t it = 0;
        bool aborted = false;
        // K and V pass through L2 once (unless sequences share pages: then the caller may ask for the
        // normal priority, under which re-read pages stay in L2 longer)
        const uint64_t kv_policy = (!direct && p.hdr->kv_evict_first) ? l2_policy_evict_first() : l2_policy_evict_normal();

        // cursor over this block's tiles: unit u, pair (b, g), tile i of cnt
        // (a grid may hold more blocks than the plan has static ranges: the extra ones live on tickets alone)
        int u = (int)blockIdx.x < n_static ? (int)blockIdx.x : -1;
        int b = 0, g = 0, rel = 0, remaining = 0, cnt = 0, i = 0;
        int4 si = make_int4(0, 0, 0, 0);
        bool first_item = true;
        int direct_flags = 0, unit_flags = 0;
        const int box_tok = box * p.box_rows;   // this lane's first token within a tile
        const int32_t *bt_row = p.block_table;  // block-table row of the cursor's sequence (set in open_pair)
        auto take_ticket = [&]() {
            int t = 0;
            if (lane == 0)
                t = atomicAdd(&p.hdr->ticket, 1);
            t = __shfl_sync(0xffffffffu, t, 0) + n_static;
            return t < n_units ? t : -1;
        };
        if (!direct && (int)blockIdx.x >= n_static)
            u = take_ticket();
        auto open_unit = [&]() {   // make u a unit that has tiles, taking tickets past empty ones
            while (u >= 0) {
                if (!DA_IN_RANGE(p.status, u, p.unit_cap, 4))
                    return false;
                const int4 uw = p.unit_work[u];
                if (uw.w > 0) {
                    b = uw.x; g = uw.y & 0xffff; rel = uw.z; remaining = uw.w;
                    unit_flags = uw.y >> 16;
                    first_item = true;
                    return true;
                }
                u = take_ticket();
            }
            return false;
        };
        auto open_pair = [&]() {   // position on the next (b, g) pair that has tiles; false at the end
            for (;;) {
                while (remaining > 0) {
                    if (!DA_IN_RANGE(p.status, b, p.B, 5))
                        return false;
                    si = p.seq_info[b];
                    if (si.w > 0) {
                        cnt = min(si.w - rel, remaining);
                        i = 0;
                        bt_row = p.block_table + (int64_t)b * p.bt_sb;
                        return true;
                    }
                    ++b;   // an empty sequence (only reachable with g == 0)
                }
                u = take_ticket();   // this unit is finished
                if (!open_unit())
                    return false;
            }
        };
        struct Tile { int page, row, t0, g, b, lo, L, flags, slot, fold; bool need, valid; };
        auto fetch = [&](Tile &t) {   // describe the cursor's tile and start its block-table read
            t.t0 = (si.z + rel + i) * TT;
            const int tok0 = t.t0 + box_tok;
            t.need = active && tok0 < si.y && tok0 + p.box_rows > si.x;
            t.page = 0;
            t.row = tok0 & (p.P - 1);           // P is a power of two: no divisions in this loop
            if (t.need && !DA_IN_RANGE(p.status, tok0 >> p.log2_P, p.max_pages, 6))
                t.need = false;
            if (t.need)
                t.page = __ldg(bt_row + (tok0 >> p.log2_P));
            t.g = g; t.b = b; t.lo = si.x; t.L = si.y;
            t.flags = (i == cnt - 1 ? TILE_ITEM_END : 0) | (cnt == si.w ? TILE_WHOLE : 0) | direct_flags;
            t.slot = direct ? (int)blockIdx.x : 2 * u + (first_item ? 0 : 1);
            // A two-piece pair that this block and a neighbour share (the plan's unit flags): the item's last
            // tile tells the consumers which piece this is (1 first, 2 second) and the partner's slot.
            t.fold = 0;
            if (i == cnt - 1 && unit_flags) {
                if ((unit_flags & 1) && first_item && rel > 0)
                    t.fold = 2 | ((2 * (u - 1) + ((unit_flags & 4) ? 0 : 1)) << 2);
                else if ((unit_flags & 2) && remaining == cnt && cnt < si.w - rel)
                    t.fold = 1 | ((2 * (u + 1)) << 2);
            }
        };
        auto advance = [&]() {   // step to the next tile; false when the block has no more work
            if (++i == cnt) {
                if (direct)
                    return false;   // one piece of one pair per block
                remaining -= cnt;
                rel = 0;
                first_item = false;
                if (++g == p.Hkv) {
                    g = 0;
                    ++b;
                }
                return open_pair();
            }
            return true;
        };

        // Three tile records in rotation: a tile is described (and its block-table entry requested) two
        // tiles before its copies are issued, so that the entry has two tile periods to arrive, and no
        // record is ever copied (copying a register with a load in flight would wait for the load).
        bool cursor_ok;
        if (direct) {
            // this block's pair and piece; the sequence's attended range and tiles, as the plan kernel would
            // have worked them out
            const int pair = (int)blockIdx.x / p.direct_splits, piece = (int)blockIdx.x % p.direct_splits;
            b = pair / p.Hkv;
            g = pair % p.Hkv;
            int L = p.seq_lens[(int64_t)b * p.sl_stride];
            if (L < 0 || (int64_t)L > p.max_pages * (int64_t)p.P) {
                if (lane == 0 && g == 0 && piece == 0)
                    report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, 0, L);
                L = 0;
            }
            const int lo = (p.window > 0 && p.window < L) ? L - p.window : 0;
            const int first = lo / TT, nt = L > lo ? (L - 1) / TT - first + 1 : 0;
            const int pieces = min(p.direct_splits, nt);   // pieces that hold tiles: the first `pieces`
            si = make_int4(lo, L, first, nt);
            bt_row = p.block_table + (int64_t)b * p.bt_sb;
            cursor_ok = piece < pieces;
            if (cursor_ok) {
                rel = (int)((long long)nt * piece / pieces);
                cnt = (int)((long long)nt * (piece + 1) / pieces) - rel;
                direct_flags = pieces << TILE_SPLITS_SHIFT;
            } else if (nt == 0 && piece == 0) {
                // an empty sequence: out = 0, lse = -inf for the pair's heads (lane -> four output dims)
                for (int hd = 0; hd < p.G; ++hd) {
                    const int h_out = g * p.G + hd;
                    const int64_t at = (int64_t)b * p.o_sb + (int64_t)h_out * p.o_sh + 4 * lane;
                    if (p.out_bf16) {
                        uint16_t *o = reinterpret_cast<uint16_t *>(p.out) + at;
                        o[0] = o[1] = o[2] = o[3] = 0;
                    } else {
                        float *o = reinterpret_cast<float *>(p.out) + at;
                        o[0] = o[1] = o[2] = o[3] = 0.f;
                    }
                    if (lane == 0 && p.lse)
                        p.lse[(int64_t)b * p.l_sb + (int64_t)h_out * p.l_sh] = -INFINITY;
                }
            }
        } else {
            cursor_ok = open_unit() && open_pair();
        }
        auto fill = [&](Tile &t) {   // describe the cursor's tile, then move the cursor on
            t.valid = cursor_ok;
            if (cursor_ok) {
                fetch(t);
                cursor_ok = advance();
            }
        };
        auto issue = [&](Tile &cur) {   // the tile's descriptor and copies into the next free stage
            const int stage = it % NSTAGES;
            const uint32_t phase = (it / NSTAGES) & 1u;
            // A page id outside the pool: the load is skipped (the rows keep whatever the stage held) and
            // the tile is marked, so that the consumers write NaN for this (sequence, KV head) pair
            // instead of a finite result computed from stale rows.
            const bool bad_page = cur.need && (uint32_t)cur.page >= (uint32_t)p.num_pages;
            if (bad_page) {
                report_status(p.status, 1 /* DA_DEV_BAD_PAGE */, cur.b, (cur.t0 + box * p.box_rows) / p.P, cur.page);
                cur.need = false;
            }
            const uint32_t poisoned = __ballot_sync(0xffffffffu, bad_page);
            const uint32_t mask = __ballot_sync(0xffffffffu, cur.need);
            if (!mbar_wait_bounded(bar_empty + 8 * stage, phase ^ 1u, abort_flag))
                return false;
            // (diagnostic build only: one tile of block 0 can be left out altogether -- no arrival, no
            //  copies -- so that the consumers' bounded wait for it runs out)
            const bool withheld = DA_WITHHOLD(0, blockIdx.x, it);
            if (lane == 0 && !withheld) {
                meta[2 * stage] = make_int4(cur.b, cur.g, cur.t0, cur.flags);
                meta[2 * stage + 1] = make_int4(cur.lo, cur.L, cur.slot, (poisoned != 0u ? 1 : 0) | (cur.fold << 1));
                mbar_arrive_expect_tx(bar_full + 8 * stage, (uint32_t)__popc(mask) * box_bytes);
            }
            __syncwarp();
            if (cur.need && !withheld) {
                const uint32_t dst = smem_base + stage * STAGE_BYTES + is_v * KV_BYTES + box * box_bytes;
                if constexpr (KV8)
                    tma_load_4d_hint(dst, tm, 0, cur.row, cur.g, cur.page, bar_full + 8 * stage, kv_policy);
                else
                    tma_load_5d_hint(dst, tm, 0, cur.row, 0, cur.g, cur.page, bar_full + 8 * stage, kv_policy);
            }
            ++it;
            return true;
        };
        Tile t0, t1, t2;
        fill(t0);
        fill(t1);
        for (;;) {
            fill(t2);
            if (!t0.valid) break;
            if (!issue(t0)) { aborted = true; break; }
            fill(t0);
            if (!t1.valid) break;
            if (!issue(t1)) { aborted = true; break; }
            fill(t1);
            if (!t2.valid) break;
            if (!issue(t2)) { aborted = true; break; }
        }
        if (!aborted) {
            // tell the consumers that nothing follows
            const int stage = it % NSTAGES;
            const uint32_t phase = (it / NSTAGES) & 1u;
            if (mbar_wait_bounded(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) {
                if (lane == 0) {
                    meta[2 * stage] = make_int4(0, 0, 0, TILE_STOP);
                    mbar_arrive(bar_full + 8 * stage);
                }
            } else {
                aborted = true;
            }
        }
        if (aborted) {
            // Do not leave the block while copies may still land in its shared memory: wait (bounded)
            // for the most recent phase of every stage that was filled.
            if (lane == 0) {
                *abort_flag = 1;
                report_status(p.status, 3 /* DA_DEV_TIMEOUT */, -2, (int)blockIdx.x, (int)it);
                for (uint32_t k = 0; k < (uint32_t)NSTAGES && k < it; ++k) {
                    const uint32_t j = it - 1 - k;
                    const uint64_t t_begin = globaltimer_ns();
                    while (!mbar_try_wait(bar_full + 8 * (j % NSTAGES), (j / NSTAGES) & 1u)) {
                        if (globaltimer_ns() - t_begin > DA_WAIT_LIMIT_NS / 2)
                            break;
                    }
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    // They follow the tile descriptors the producer leaves with each stage.  A failed (timed-out)
    // wait raises the abort flag and leaves at once; every other wait then gives up quickly too.
    const int r = lane >> 2, c = lane & 3;
    const int tw = CSETS == 1 ? warp : warp % NCW;      // token group: this warp's rows of every tile
    const int cs = CSETS == 1 ? 0 : warp / NCW;         // column set
    const int col0 = cs * HS;                           // first (virtual) head of this warp's column tiles
    const uint32_t bar_epi = bar_epi0 + 16 * cs;
    uint32_t it = 0, items = 0;
    uint32_t ph_a = 0, ph_b = 0;   // completed phases of this column set's two epilogue barriers
    // per-lane offsets used by the ldmatrix address patterns
    const int k_row = 16 * tw + (lane & 7) + ((lane >> 3) & 1) * 8;     // K: matrices 1,3 are rows +8
    const int k_chunk = lane >> 4;                                      //    matrices 2,3 are chunk +1
    const int v_row = 16 * tw + (lane & 7) + (lane >> 4) * 8;           // V: matrices 2,3 are rows +8
    const int v_chunk = (lane >> 3) & 1;                                //    matrices 1,3 are chunk +1
    const uint32_t plane_bytes = (uint32_t)p.box_rows * 128u;
    const uint32_t k_off = row_offset(k_row, p.box_rows), v_off = row_offset(v_row, p.box_rows);
    const uint32_t k_sw = (uint32_t)(k_row & 7), v_sw = (uint32_t)(v_row & 7);

    // ---- 8-bit cache: a warp owns 32 tokens of a 128-token tile (rows of 128 bytes, 16-byte chunk index
    // XORed with the row's low three bits).  The codes are widened to f16 in registers (exactly: every
    // E4M3 value is an f16 value) and both products run as f16 mma with fp32 accumulation.  The warp's
    // scores form two 16-row tiles A and B; row x of tile A is warp-local token tok8(x), of tile B
    // 16 + tok8(x).  tok8 swaps rows 8-11 with 12-15 so that the eight rows of every ldmatrix phase,
    // for K and for the transposed V reads below, differ in their low three bits (no bank conflicts).
    //   K: one ldmatrix.x4 brings 16 rows x 32 dims as four registers of four codes (dims 4c..4c+3 of
    //      rows r / r+8, first and second 16 dims).  The low halves widen to the (k = 2c, 2c+1)
    //      fragment registers of one m16n8k16 step and the high halves to its (k = 2c+8, 2c+9)
    //      registers; Q's fragments are loaded in the same dim order, so the order does not matter.
    //   V: the transposed 8-bit ldmatrix takes one row address per k slot: lane j points slot j at the
    //      token whose weight sits in that slot of P's fragment (slots 4c+e <- block row 2c+e of the
    //      rows 0-7 block, 4c+2+e <- of the rows 8-15 block; tile A in slots 0-15, tile B in 16-31).
    auto tok8 = [](int x) { return x < 8 ? x : 8 + ((x + 4) & 7); };
    const int x8 = (lane & 7) + ((lane >> 3) & 1) * 8;          // QK ldmatrix: row of the 16-row tile
    const int k8_chunk = lane >> 4;                             //              16-byte half of the 32-dim step
    const int row_a8 = 32 * tw + tok8(x8), row_b8 = row_a8 + 16;
    const uint32_t ka8_off = (uint32_t)row_a8 * 128u, kb8_off = (uint32_t)row_b8 * 128u;
    const uint32_t ka8_sw = (uint32_t)(row_a8 & 7), kb8_sw = (uint32_t)(row_b8 & 7);
    const int slot_row = 8 * ((lane >> 1) & 1) + 2 * ((lane & 15) >> 2) + (lane & 1);   // PV: tile row of k slot `lane`
    const int row_v8 = 32 * tw + tok8(slot_row) + 16 * (lane >> 4);
    const uint32_t v8_off = (uint32_t)row_v8 * 128u, v8_sw = (uint32_t)(row_v8 & 7);
    const int t_a0 = tok8(r), t_a1 = tok8(r + 8);               // tokens of this lane's scores (tile B: + 16)

    auto give_up = [&](int where) {
        if (*abort_flag == 0) {
            *abort_flag = 1;
            report_status(p.status, 3 /* DA_DEV_TIMEOUT */, where, (int)blockIdx.x, (int)it);
        }
    };
    // Q^T fragments (B operand of S^T = K Q^T): lane holds head r, dims 16kk + 2c + {0,1} (+8)
    auto load_q = [&](uint32_t (&qf)[NT8][8][2], int b, int g) {
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            const int head = col0 + n * 8 + r;
            const int hv = head < p.Gv ? head : 0;
            const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
                p.q + (int64_t)b * p.q_sb + (int64_t)(hv / p.G) * p.q_sq + (int64_t)(g * p.G + hv % p.G) * p.q_sh);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                qf[n][kk][0] = head < p.Gv ? __ldg(qrow + 8 * kk + c) : 0u;
                qf[n][kk][1] = head < p.Gv ? __ldg(qrow + 8 * kk + 4 + c) : 0u;
            }
        }
    };

    // 8-bit cache: Q^T as f16 B fragments of S^T = K Q^T.  A head's query vector is scaled by a power
    // of two so that its largest magnitude lies in [2^14, 2^15) and rounded to f16; a bf16 has 8
    // significant bits and f16 carries 11 down to 2^-14, so the conversion is exact for every element
    // within 2^-28 of the head's largest (smaller ones are off by at most 2^-25 of the scaled value).
    // qf[n][i] is the fragment of k step i (16 dims): lane (r, c) holds head r, dims 16i + 4c .. + 3.
    // fh[n][e]: what turns the raw products of head 2c + e into log2-domain scores.
    // Two steps, so that the loads of the next item's vectors can fly while this item is combined:
    // load_q8_raw only issues the loads (bf16 pairs), q8_fragments turns them into the fragments.
    auto load_q8_raw = [&](uint32_t (&w)[NT8][8][2], float &ks, int b, int g) {
        ks = p.k_scale ? __ldg(p.k_scale + g) : 1.f;
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            const int head = col0 + n * 8 + r;
            const int hv = head < p.Gv ? head : 0;
            const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
                p.q + (int64_t)b * p.q_sb + (int64_t)(hv / p.G) * p.q_sq + (int64_t)(g * p.G + hv % p.G) * p.q_sh);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
                    w[n][i][hf] = head < p.Gv ? __ldg(qrow + 8 * i + 2 * c + hf) : 0u;
        }
    };
    auto q8_fragments = [&](uint32_t (&qf)[NT8][8][2], float (&fh)[NT8][2], const uint32_t (&w)[NT8][8][2], float ks) {
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            float amax = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
                    amax = fmaxf(amax, fmaxf(fabsf(bf16_lo_to_float(w[n][i][hf])), fabsf(bf16_hi_to_float(w[n][i][hf]))));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            // f = 2^(14 - exponent of amax), kept inside the normal fp32 range
            int fexp = 268 - (int)((__float_as_uint(amax) >> 23) & 0xffu);
            fexp = min(max(fexp, 1), 254);
            const float f = __uint_as_float((uint32_t)fexp << 23);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
                    qf[n][i][hf] = pack_f16(bf16_lo_to_float(w[n][i][hf]) * f, bf16_hi_to_float(w[n][i][hf]) * f);
            const float fin = (1.f / f) * ks * p.scale_log2;   // the same in all four lanes of head r
            fh[n][0] = __shfl_sync(0xffffffffu, fin, 8 * c);
            fh[n][1] = __shfl_sync(0xffffffffu, fin, 8 * c + 4);
        }
    };

    // the result row of (sequence b, virtual head `head` of KV group g): lane -> four output dims
    auto store_result = [&](int b, int g, int head, const float4 &val, float lse_nat) {
        const int qi = p.Lq > 1 ? head / p.G : 0;
        const int h_out = g * p.G + (head - qi * p.G);
        const int64_t at = (int64_t)b * p.o_sb + (int64_t)qi * p.o_sq + (int64_t)h_out * p.o_sh + 4 * lane;
        if (!DA_IN_RANGE(p.status, b, p.B, 7) || !DA_IN_RANGE(p.status, h_out, p.Hkv * p.G, 8) ||
            !DA_IN_RANGE(p.status, qi, p.Lq, 9))
            return;
        if (p.out_bf16) {
            __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(p.out) + at;
            const uint32_t lo = pack_bf16(val.x, val.y), hi = pack_bf16(val.z, val.w);
            if ((reinterpret_cast<uintptr_t>(o) & 7u) == 0) {
                *reinterpret_cast<uint2 *>(o) = make_uint2(lo, hi);
            } else {
                reinterpret_cast<uint16_t *>(o)[0] = (uint16_t)lo;
                reinterpret_cast<uint16_t *>(o)[1] = (uint16_t)(lo >> 16);
                reinterpret_cast<uint16_t *>(o)[2] = (uint16_t)hi;
                reinterpret_cast<uint16_t *>(o)[3] = (uint16_t)(hi >> 16);
            }
        } else {
            float *o = reinterpret_cast<float *>(p.out) + at;
            if ((reinterpret_cast<uintptr_t>(o) & 15u) == 0) {
                *reinterpret_cast<float4 *>(o) = val;
            } else {
                o[0] = val.x; o[1] = val.y; o[2] = val.z; o[3] = val.w;
            }
        }
        if (lane == 0 && p.lse)
            p.lse[(int64_t)b * p.l_sb + (int64_t)qi * p.l_sq + (int64_t)h_out * p.l_sh] = lse_nat;
    };

    uint32_t qf[NT8][8][2];
    float fh[NT8][2];
    // Direct mode: the block's pair follows from its index, so its query rows are asked for before the first
    // tile's descriptor arrives (the producer's length -> block table -> copy chain runs meanwhile).
    const bool q_early = p.direct_splits > 0;
    uint32_t qw[KV8 ? NT8 : 1][8][2];
    float ks_first = 1.f;
    if (q_early) {
        const int pair = (int)blockIdx.x / p.direct_splits;
        if constexpr (KV8)
            load_q8_raw(qw, ks_first, pair / p.Hkv, pair % p.Hkv);
        else
            load_q(qf, pair / p.Hkv, pair % p.Hkv);
    }
    if (!mbar_wait_bounded(bar_full, 0u, abort_flag)) {
        give_up(-3);
        return;
    }
    int4 m0 = meta[0], m1 = meta[1];
    if (tid == 0 && blockIdx.x < TL_MERGE)
        DA_TL(blockIdx.x, 2);
    if (m0.w & TILE_STOP)
        return;
    if constexpr (KV8) {
        if (!q_early)
            load_q8_raw(qw, ks_first, m0.x, m0.y);
        q8_fragments(qf, fh, qw, ks_first);
    } else {
        if (!q_early)
            load_q(qf, m0.x, m0.y);
#pragma unroll
        for (int n = 0; n < NT8; ++n)
            fh[n][0] = fh[n][1] = 0.f;
    }

    for (;;) {   // one (b, kv head) item per iteration
        const int b = m0.x, g = m0.y, lo = m1.x, L = m1.y, slot = m1.z;
        const bool whole = (m0.w & TILE_WHOLE) != 0;
        const int pieces = m0.w >> TILE_SPLITS_SHIFT;   // direct mode: blocks that share this pair (else 0)
        int fold = 0;             // a two-piece pair shared with a neighbouring block: piece (1, 2) | partner slot << 2
        bool poisoned = false;   // a tile of this item lost rows to a bad page id: the result is NaN
        float m_run[NT8][2], l_run[NT8][2], o[NT8][8][4];
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            m_run[n][0] = m_run[n][1] = -INFINITY;
            l_run[n][0] = l_run[n][1] = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                o[n][j][0] = o[n][j][1] = o[n][j][2] = o[n][j][3] = 0.f;
        }

        for (;;) {   // the item's tiles; (m0, m1) describe the tile in stage it % NSTAGES, already full
            const int stage = it % NSTAGES;
            constexpr int WT = KV8 ? 32 : 16;   // tokens of a tile that one warp owns
            const int a = m0.z + WT * tw;       // first token of this warp's rows
            const int v_lo = max(a, lo), v_hi = min(a + WT, L);
            const bool item_end = (m0.w & TILE_ITEM_END) != 0;
            poisoned |= (m1.w & 1) != 0;
            if (item_end)
                fold = m1.w >> 1;
            if constexpr (KV8) {
              if (v_lo < v_hi) {
                const uint32_t k_base = smem_base + stage * STAGE_BYTES;
                const uint32_t v_base = k_base + KV_BYTES;
                const bool ragged = (v_lo > a) || (v_hi < a + 32);
                if (ragged) {
                    // rows outside the attended range may hold NaN codes: clear those V rows (8 chunks each)
                    for (int e = lane; e < 256; e += 32) {
                        const int rr = e >> 3, ch = e & 7;
                        const int t = a + rr;
                        if (t < v_lo || t >= v_hi) {
                            const uint32_t addr = v_base + (uint32_t)(32 * tw + rr) * 128u + (ch << 4);
                            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
                        }
                    }
                    __syncwarp();
                }
                // ---- S^T = K Q^T for the two 16-token tiles; two accumulators each to shorten the chains
                float sa[NT8][4], sb[NT8][4];
                {
                    float aa[NT8][2][4], ab[NT8][2][4];
#pragma unroll
                    for (int n = 0; n < NT8; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            aa[n][0][e] = aa[n][1][e] = ab[n][0][e] = ab[n][1][e] = 0.f;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        uint32_t ca[4], cb[4];
                        ldmatrix_x4(ca, k_base + ka8_off + ((((uint32_t)(2 * kk + k8_chunk)) ^ ka8_sw) << 4));
                        ldmatrix_x4(cb, k_base + kb8_off + ((((uint32_t)(2 * kk + k8_chunk)) ^ kb8_sw) << 4));
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {   // the two 16-dim steps of this 32-dim load
                            uint32_t fa[4], fb[4];
                            fa[0] = e4m3x2_lo_to_f16x2(ca[2 * hf]);
                            fa[1] = e4m3x2_lo_to_f16x2(ca[2 * hf + 1]);
                            fa[2] = e4m3x2_hi_to_f16x2(ca[2 * hf]);
                            fa[3] = e4m3x2_hi_to_f16x2(ca[2 * hf + 1]);
                            fb[0] = e4m3x2_lo_to_f16x2(cb[2 * hf]);
                            fb[1] = e4m3x2_lo_to_f16x2(cb[2 * hf + 1]);
                            fb[2] = e4m3x2_hi_to_f16x2(cb[2 * hf]);
                            fb[3] = e4m3x2_hi_to_f16x2(cb[2 * hf + 1]);
#pragma unroll
                            for (int n = 0; n < NT8; ++n) {
                                mma_f16_16816(aa[n][hf], fa, qf[n][2 * kk + hf][0], qf[n][2 * kk + hf][1]);
                                mma_f16_16816(ab[n][hf], fb, qf[n][2 * kk + hf][0], qf[n][2 * kk + hf][1]);
                            }
                        }
                    }
#pragma unroll
                    for (int n = 0; n < NT8; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            sa[n][e] = (aa[n][0][e] + aa[n][1][e]) * fh[n][e & 1];
                            sb[n][e] = (ab[n][0][e] + ab[n][1][e]) * fh[n][e & 1];
                        }
                }
                // sa[n][0]: (token a + t_a0, head 2c) [1]: (t_a0, 2c+1) [2]: (t_a1, 2c) [3]: (t_a1, 2c+1); sb: tokens + 16
                if (ragged) {
                    const bool oa0 = (a + t_a0 >= v_lo) && (a + t_a0 < v_hi), oa1 = (a + t_a1 >= v_lo) && (a + t_a1 < v_hi);
                    const bool ob0 = (a + 16 + t_a0 >= v_lo) && (a + 16 + t_a0 < v_hi);
                    const bool ob1 = (a + 16 + t_a1 >= v_lo) && (a + 16 + t_a1 < v_hi);
#pragma unroll
                    for (int n = 0; n < NT8; ++n) {
                        if (!oa0) sa[n][0] = sa[n][1] = -INFINITY;
                        if (!oa1) sa[n][2] = sa[n][3] = -INFINITY;
                        if (!ob0) sb[n][0] = sb[n][1] = -INFINITY;
                        if (!ob1) sb[n][2] = sb[n][3] = -INFINITY;
                    }
                }
                if (p.Lq > 1 && a + 32 > L - p.Lq + 1) {
                    // several new tokens: the query of column (virtual head) v attends tokens below
                    // L - Lq + v / G + 1 only
#pragma unroll
                    for (int n = 0; n < NT8; ++n)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int lim = L - p.Lq + (col0 + n * 8 + 2 * c + e) / p.G + 1;
                            if (a + t_a0 >= lim) sa[n][e] = -INFINITY;
                            if (a + t_a1 >= lim) sa[n][2 + e] = -INFINITY;
                            if (a + 16 + t_a0 >= lim) sb[n][e] = -INFINITY;
                            if (a + 16 + t_a1 >= lim) sb[n][2 + e] = -INFINITY;
                        }
                }
                // ---- online softmax in the log2 domain: column (head) maxima over the 32 tokens
                float mx[NT8][2];
                bool grew = false;
#pragma unroll
                for (int n = 0; n < NT8; ++n) {
                    mx[n][0] = fmaxf(fmaxf(sa[n][0], sa[n][2]), fmaxf(sb[n][0], sb[n][2]));
                    mx[n][1] = fmaxf(fmaxf(sa[n][1], sa[n][3]), fmaxf(sb[n][1], sb[n][3]));
#pragma unroll
                    for (int o_ = 4; o_ < 32; o_ <<= 1) {
                        mx[n][0] = fmaxf(mx[n][0], __shfl_xor_sync(0xffffffffu, mx[n][0], o_));
                        mx[n][1] = fmaxf(mx[n][1], __shfl_xor_sync(0xffffffffu, mx[n][1], o_));
                    }
                    grew |= (mx[n][0] > m_run[n][0]) | (mx[n][1] > m_run[n][1]);
                }
                if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
                    for (int n = 0; n < NT8; ++n) {
                        float al[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float m_new = fmaxf(m_run[n][e], mx[n][e]);
                            al[e] = (m_run[n][e] == -INFINITY) ? 0.f : fast_exp2(m_run[n][e] - m_new);
                            m_run[n][e] = m_new;
                            l_run[n][e] *= al[e];
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            o[n][j][0] *= al[0];
                            o[n][j][1] *= al[1];
                            o[n][j][2] *= al[0];
                            o[n][j][3] *= al[1];
                        }
                    }
                }
                // ---- weights w = 2^15 * exp2(s - m) as f16 high and low parts (together ~22 bits of each
                //      weight; the factor 2^15 keeps weights down to 2^-39 of the largest representable),
                //      transposed into the B operand of O^T += V^T P^T.  ph[n][q]: block q = rows 0-7 / 8-15
                //      of tile A, then of tile B.
                uint32_t ph[NT8][4], pl[NT8][4];
#pragma unroll
                for (int n = 0; n < NT8; ++n) {
                    float w[8];
                    // (a column that has seen no token yet keeps m = -inf: exp2(-inf) = 0, not NaN)
                    const float mu[2] = {m_run[n][0] == -INFINITY ? 0.f : m_run[n][0] - P8_SHIFT,
                                         m_run[n][1] == -INFINITY ? 0.f : m_run[n][1] - P8_SHIFT};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        w[e] = fast_exp2(sa[n][e] - mu[e & 1]);
                        w[4 + e] = fast_exp2(sb[n][e] - mu[e & 1]);
                    }
                    l_run[n][0] += (w[0] + w[2]) + (w[4] + w[6]);
                    l_run[n][1] += (w[1] + w[3]) + (w[5] + w[7]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t hi = pack_f16(w[2 * q], w[2 * q + 1]);
                        const float2 hv = unpack_f16(hi);
                        const uint32_t lo = pack_f16(w[2 * q] - hv.x, w[2 * q + 1] - hv.y);
                        ph[n][q] = movmatrix_trans(hi);
                        pl[n][q] = movmatrix_trans(lo);
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t cv[4];
                    ldmatrix_b8_x2_trans(cv, v_base + v8_off + ((((uint32_t)j) ^ v8_sw) << 4));
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {   // tile A's 16 tokens, then tile B's
                        uint32_t vf[4];
                        vf[0] = e4m3x2_lo_to_f16x2(cv[2 * hf]);
                        vf[1] = e4m3x2_lo_to_f16x2(cv[2 * hf + 1]);
                        vf[2] = e4m3x2_hi_to_f16x2(cv[2 * hf]);
                        vf[3] = e4m3x2_hi_to_f16x2(cv[2 * hf + 1]);
#pragma unroll
                        for (int n = 0; n < NT8; ++n) {
                            mma_f16_16816(o[n][j], vf, ph[n][2 * hf], ph[n][2 * hf + 1]);
                            mma_f16_16816(o[n][j], vf, pl[n][2 * hf], pl[n][2 * hf + 1]);
                        }
                    }
                }
                if (ragged)
                    fence_proxy_async_smem();   // the zeroed rows will be overwritten by a later TMA load
              }
            } else
            if (v_lo < v_hi) {
                const uint32_t k_base = smem_base + stage * STAGE_BYTES;
                const uint32_t v_base = k_base + KV_BYTES;
                const bool ragged = (v_lo > a) || (v_hi < a + 16);
                if (ragged) {
                    // rows outside the attended range may hold NaN: a zero weight would not hide it
                    // in the PV product, so clear those V rows (both planes; 16 chunks of 16 B a row)
                    for (int e = lane; e < 256; e += 32) {
                        const int rr = e >> 4, ch = e & 15;
                        const int t = a + rr;
                        if (t < v_lo || t >= v_hi) {
                            const uint32_t addr = v_base + row_offset(16 * tw + rr, p.box_rows) +
                                                  (ch >> 3) * plane_bytes + ((ch & 7) << 4);
                            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
                        }
                    }
                    __syncwarp();
                }
                // ---- S^T = K Q^T: 16 tokens x HEADS, two accumulators to halve the dependency chain
                float s[NT8][4];
                {
                    float acc[NT8][2][4];
#pragma unroll
                    for (int n = 0; n < NT8; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            acc[n][0][e] = acc[n][1][e] = 0.f;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        uint32_t af[4];
                        // chunk 2kk + k_chunk: plane kk >> 2, position ((2kk + k_chunk) & 7) ^ (row & 7)
                        ldmatrix_x4(af, k_base + k_off + (kk >> 2) * plane_bytes +
                                            ((((2 * kk + k_chunk) & 7) ^ k_sw) << 4));
#pragma unroll
                        for (int n = 0; n < NT8; ++n)
                            mma_bf16_16816(acc[n][kk & 1], af, qf[n][kk][0], qf[n][kk][1]);
                    }
#pragma unroll
                    for (int n = 0; n < NT8; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            s[n][e] = (acc[n][0][e] + acc[n][1][e]) * p.scale_log2;
                }
                // s[n][0]: (token a+r, head 2c)  [1]: (a+r, 2c+1)  [2]: (a+r+8, 2c)  [3]: (a+r+8, 2c+1)
                if (ragged) {
                    const bool ok0 = (a + r >= v_lo) && (a + r < v_hi);
                    const bool ok1 = (a + r + 8 >= v_lo) && (a + r + 8 < v_hi);
#pragma unroll
                    for (int n = 0; n < NT8; ++n) {
                        if (!ok0) s[n][0] = s[n][1] = -INFINITY;
                        if (!ok1) s[n][2] = s[n][3] = -INFINITY;
                    }
                }
                if (p.Lq > 1 && a + 16 > L - p.Lq + 1) {
                    // several new tokens: the query of column (virtual head) v attends tokens below
                    // L - Lq + v / G + 1 only
#pragma unroll
                    for (int n = 0; n < NT8; ++n)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int lim = L - p.Lq + (col0 + n * 8 + 2 * c + e) / p.G + 1;
                            if (a + r >= lim) s[n][e] = -INFINITY;
                            if (a + r + 8 >= lim) s[n][2 + e] = -INFINITY;
                        }
                }
                // ---- online softmax in the log2 domain: column (head) maxima over the 16 tokens
                float mx[NT8][2];
                bool grew = false;
#pragma unroll
                for (int n = 0; n < NT8; ++n) {
                    mx[n][0] = fmaxf(s[n][0], s[n][2]);
                    mx[n][1] = fmaxf(s[n][1], s[n][3]);
#pragma unroll
                    for (int o_ = 4; o_ < 32; o_ <<= 1) {
                        mx[n][0] = fmaxf(mx[n][0], __shfl_xor_sync(0xffffffffu, mx[n][0], o_));
                        mx[n][1] = fmaxf(mx[n][1], __shfl_xor_sync(0xffffffffu, mx[n][1], o_));
                    }
                    grew |= (mx[n][0] > m_run[n][0]) | (mx[n][1] > m_run[n][1]);
                }
                if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
                    for (int n = 0; n < NT8; ++n) {
                        float al[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float m_new = fmaxf(m_run[n][e], mx[n][e]);
                            al[e] = (m_run[n][e] == -INFINITY) ? 0.f : fast_exp2(m_run[n][e] - m_new);
                            m_run[n][e] = m_new;
                            l_run[n][e] *= al[e];
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            o[n][j][0] *= al[0];
                            o[n][j][1] *= al[1];
                            o[n][j][2] *= al[0];
                            o[n][j][3] *= al[1];
                        }
                    }
                }
                // ---- P^T as the B operand of O^T += V^T P^T, split into bf16 high and low parts so
                //      that the product carries ~16 bits of each weight
                uint32_t ph[NT8][2], pl[NT8][2];
#pragma unroll
                for (int n = 0; n < NT8; ++n) {
                    float pv[4];
                    // (a column that has seen no token yet keeps m = -inf: exp2(-inf - 0) = 0, not NaN)
                    const float m0u = m_run[n][0] == -INFINITY ? 0.f : m_run[n][0];
                    const float m1u = m_run[n][1] == -INFINITY ? 0.f : m_run[n][1];
                    pv[0] = fast_exp2(s[n][0] - m0u);
                    pv[1] = fast_exp2(s[n][1] - m1u);
                    pv[2] = fast_exp2(s[n][2] - m0u);
                    pv[3] = fast_exp2(s[n][3] - m1u);
                    l_run[n][0] += pv[0] + pv[2];
                    l_run[n][1] += pv[1] + pv[3];
                    const uint32_t h01 = pack_bf16(pv[0], pv[1]);
                    const uint32_t h23 = pack_bf16(pv[2], pv[3]);
                    const uint32_t l01 = pack_bf16(pv[0] - bf16_lo_to_float(h01), pv[1] - bf16_hi_to_float(h01));
                    const uint32_t l23 = pack_bf16(pv[2] - bf16_lo_to_float(h23), pv[3] - bf16_hi_to_float(h23));
                    ph[n][0] = movmatrix_trans(h01);   // tokens 0-7  -> k = 2c, 2c+1, n = head r
                    ph[n][1] = movmatrix_trans(h23);   // tokens 8-15
                    pl[n][0] = movmatrix_trans(l01);
                    pl[n][1] = movmatrix_trans(l23);
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t vf[4];
                    ldmatrix_x4_trans(vf, v_base + v_off + (j >> 2) * plane_bytes +
                                              ((((2 * j + v_chunk) & 7) ^ v_sw) << 4));
#pragma unroll
                    for (int n = 0; n < NT8; ++n) {
                        mma_bf16_16816(o[n][j], vf, ph[n][0], ph[n][1]);
                        mma_bf16_16816(o[n][j], vf, pl[n][0], pl[n][1]);
                    }
                }
                if (ragged)
                    fence_proxy_async_smem();   // the zeroed rows will be overwritten by a later TMA load
            }
            __syncwarp();
            if (lane == 0)
                mbar_arrive(bar_empty + 8 * stage);
            ++it;
            if (tid == 0 && blockIdx.x < TL_MERGE)
                DA_TL(blockIdx.x, 3);
            // the next tile (of this item, or the first of the next one, or the stop mark)
            const int nstage = it % NSTAGES;
            if (!mbar_wait_bounded(bar_full + 8 * nstage, (it / NSTAGES) & 1u, abort_flag)) {
                give_up(-3);
                return;
            }
            m0 = meta[2 * nstage];
            m1 = meta[2 * nstage + 1];
            if (item_end)
                break;
        }

        // ---- the item is complete.  Start the next item's Q loads, then combine the four warps'
        //      (m, l, O) and write the pair's result or partial.
        const bool stop = (m0.w & TILE_STOP) != 0;
        uint32_t qn[NT8][8][2];
        float ks_next = 1.f;
        // 8-bit cache: this item's V factor (asked for here, used after the barrier below)
        const float vmul = (KV8 && p.v_scale) ? __ldg(p.v_scale + g) : 1.f;
        if (!stop) {
            if constexpr (KV8)
                load_q8_raw(qn, ks_next, m0.x, m0.y);
            else
                load_q(qn, m0.x, m0.y);
        }
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float l = l_run[n][e];
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                if (r == 0) {
                    // (8-bit cache: the weights were carried times 2^15, i.e. relative to m - 15)
                    st_m[tw * HEADS + col0 + n * 8 + 2 * c + e] = KV8 ? m_run[n][e] - P8_SHIFT : m_run[n][e];
                    st_l[tw * HEADS + col0 + n * 8 + 2 * c + e] = l;
                }
            }
            // xbuf[warp][head][d ^ 8*((head>>1)&3)] : conflict-free for these stores and the reads below
            float *xb = xbuf + (tw * HEADS + col0 + n * 8 + 2 * c) * HEAD_DIM;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int d0 = (16 * j + r) ^ (8 * c), d1 = (16 * j + r + 8) ^ (8 * c);
                xb[d0] = o[n][j][0];
                xb[HEAD_DIM + d0] = o[n][j][1];
                xb[d1] = o[n][j][2];
                xb[HEAD_DIM + d1] = o[n][j][3];
            }
        }
        __syncwarp();
        if (lane == 0)
            mbar_arrive(bar_epi);
        if (!mbar_wait_bounded(bar_epi, ph_a & 1u, abort_flag)) {
            give_up(-4);
            return;
        }
        ++ph_a;
        {
            // Warp w of a column set folds the set's heads w, w + 4, ...: lane -> output dims 4 lane .. 4 lane + 3.  A short loop
            // on purpose: this code runs once per item, so its instructions are fetched cold each time,
            // and a compact body costs far less than a long unrolled one.
            const uint64_t part_policy = l2_policy_evict_last();   // partial results wait in L2 for the merge kernel
#pragma unroll 1
            for (int head = col0 + tw; head < min(p.Gv, col0 + HS); head += NCW) {
                float mw[NCW], lw[NCW], f[NCW];
#pragma unroll
                for (int w = 0; w < NCW; ++w) {
                    mw[w] = st_m[w * HEADS + head];
                    lw[w] = st_l[w * HEADS + head];
                }
                const float *xrow = xbuf + head * HEAD_DIM + ((4 * lane) ^ (8 * ((head >> 1) & 3)));
                float4 x[NCW];
#pragma unroll
                for (int w = 0; w < NCW; ++w)
                    x[w] = *reinterpret_cast<const float4 *>(xrow + w * HEADS * HEAD_DIM);
                float M = mw[0];
#pragma unroll
                for (int w = 1; w < NCW; ++w)
                    M = fmaxf(M, mw[w]);
                float den = 0.f;
                float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w = 0; w < NCW; ++w) {
                    f[w] = fast_exp2(mw[w] - M);   // 0 for a warp that saw no token
                    den += lw[w] * f[w];
                    num.x += x[w].x * f[w];
                    num.y += x[w].y * f[w];
                    num.z += x[w].z * f[w];
                    num.w += x[w].w * f[w];
                }
                // (den = 0, or NaN when no warp saw a token: a piece in which this column's query attends
                //  nothing -- several new tokens only)
                const bool some = den > 0.f;
                const float inv = some ? (KV8 ? vmul / den : 1.f / den) : 0.f;
                float lse_nat = some ? (M + fast_log2(den)) * LN2 : -INFINITY;
                float4 val = some ? make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv)
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
                if (poisoned) {   // (a NaN partial makes the merged result NaN as well)
                    lse_nat = __int_as_float(0x7fc00000);
                    val = make_float4(lse_nat, lse_nat, lse_nat, lse_nat);
                }
                if (whole) {
                    store_result(b, g, head, val, lse_nat);
                } else {
                    if (!DA_IN_RANGE(p.status, slot, 2 * p.unit_cap, 10))
                        continue;
                    st_global_v4_hint(p.part_o + ((int64_t)slot * HEADS + head) * HEAD_DIM + 4 * lane, val, part_policy);
                    if (lane == 0)
                        st_global_f32_hint(p.part_lse + (int64_t)slot * HEADS + head, lse_nat, part_policy);
                }
            }
        }
        // A pair whose pieces are folded here rather than by the merge kernel: in direct mode every split pair
        // (`pieces` blocks share it), otherwise a pair cut in two by this block's range and a neighbour's
        // (`fold`).  The block that counts last on the pair's counter folds the pieces -- the merge kernel's
        // rule: M = max lse_k; w_k = exp(lse_k - M); out = sum w_k O_k / sum w_k; lse = M + ln sum w_k -- and
        // leaves the counter at zero for the next call.
        const bool counted = pieces > 1 || fold != 0;
        if (counted)
            __threadfence();   // this thread's partial stores are visible device-wide before the count below
        __syncwarp();
        if (lane == 0)
            mbar_arrive(bar_epi + 8);
        if (!mbar_wait_bounded(bar_epi + 8, ph_b & 1u, abort_flag)) {
            give_up(-5);
            return;
        }
        ++ph_b;
        if (counted) {
            volatile int *fold_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAGS + 4 + 4 * cs);
            int n_pieces, slot_a, slot_step;   // the pieces' slots: slot_a + k * slot_step
            int32_t *counter;
            if (fold) {
                const int partner = fold >> 2, first = (fold & 3) == 1;
                n_pieces = 2;
                slot_a = slot;
                slot_step = partner - slot;
                // one counter per boundary between two units (the earlier unit's index) and column set
                counter = p.fold_counters + (size_t)(first ? partner / 2 - 1 : partner / 2) * CSETS + cs;
            } else {
                const int pair = (int)blockIdx.x / p.direct_splits;
                n_pieces = pieces;
                slot_a = pair * p.direct_splits;
                slot_step = 1;
                counter = p.pair_counters + (DA_IN_RANGE(p.status, pair, DIRECT_MAX_PAIRS, 16) ? pair : 0);
            }
            if (tw == 0 && lane == 0) {
                const int last = atomicAdd(counter, 1) == n_pieces - 1;
                if (last)
                    *counter = 0;
                *fold_flag = last;
            }
            __syncwarp();
            if (lane == 0)
                mbar_arrive(bar_epi);
            if (!mbar_wait_bounded(bar_epi, ph_a & 1u, abort_flag)) {
                give_up(-6);
                return;
            }
            ++ph_a;
            if (*fold_flag) {
                __threadfence();   // the other blocks' partials were published before their counts
                for (int head = col0 + tw; head < min(p.Gv, col0 + HS); head += NCW) {
                    float lk[8], M = -INFINITY;
                    float4 ok_[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const bool on = k < n_pieces;
                        const int64_t sl = slot_a + (int64_t)k * slot_step;
                        lk[k] = on ? __ldcg(p.part_lse + sl * HEADS + head) : -INFINITY;
                        ok_[k] = on ? __ldcg(reinterpret_cast<const float4 *>(p.part_o + (sl * HEADS + head) * HEAD_DIM) + lane)
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
                        M = fmaxf(M, lk[k]);
                    }
                    float den = 0.f;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        // (a piece that saw no token has lse = -inf and weighs nothing; a NaN piece -- rows lost
                        //  to a bad page id -- makes the result NaN)
                        const float w = (k < n_pieces && lk[k] != -INFINITY) ? __expf(lk[k] - M) : 0.f;
                        den += w;
                        acc.x += w * ok_[k].x;
                        acc.y += w * ok_[k].y;
                        acc.z += w * ok_[k].z;
                        acc.w += w * ok_[k].w;
                    }
                    if (den == 0.f) {   // a column whose query attends none of the pair's tokens
                        store_result(b, g, head, make_float4(0.f, 0.f, 0.f, 0.f), -INFINITY);
                    } else {
                        const float inv = 1.f / den;
                        store_result(b, g, head, make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv), M + __logf(den));
                    }
                }
            }
        }
        ++items;
        if (stop) {
            if (tid == 0 && blockIdx.x < TL_MERGE) {
                DA_TL(blockIdx.x, 4);
                DA_TL_SET(blockIdx.x, 5, it);
                DA_TL_SET(blockIdx.x, 6, items);
            }
            return;
        }
        if constexpr (KV8) {
            q8_fragments(qf, fh, qn, ks_next);
        } else {
#pragma unroll
            for (int n = 0; n < NT8; ++n)
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    qf[n][kk][0] = qn[n][kk][0];
                    qf[n][kk][1] = qn[n][kk][1];
                }
        }
    }
}

// =====================================================================================  merge
// A fixed, small grid.  Its work comes from the lists of split pairs the plan kernel made (pairs
// that one unit covered were already written by the partition kernel) and from the empty
// sequences, which get out = 0 and lse = -inf.  For one (pair, head) with partials (O_s, lse_s):
//   M = max_s lse_s;  w_s = exp(lse_s - M);  out = sum_s w_s O_s / sum_s w_s;  lse = M + ln sum_s w_s.
// A warp takes up to 32 splits at once: lane s reads lse_s, the maximum and the sum of weights come
// from warp shuffles, then every lane accumulates its four head_dim columns over the splits (the
// loads do not depend on one another).  Pairs with more than 32 splits are folded by the eight
// warps of a block, 32 splits per warp and pass, and combined through shared memory.
constexpr int MERGE_LANES = HEAD_DIM / 4;
constexpr int MERGE_WARPS = 8;
constexpr int MERGE_THREADS = MERGE_WARPS * MERGE_LANES;
#ifndef DA_MERGE_BLOCKS_PER_SM
#define DA_MERGE_BLOCKS_PER_SM 3
#endif
constexpr int MERGE_BLOCKS_PER_SM = DA_MERGE_BLOCKS_PER_SM;   // resident blocks an SM holds (three: 78 registers a thread, no spills to speak of)

struct MergeAcc {
    float M, den;
    float4 acc;
};
// a <- a (+) b, both already weighted sums relative to their own maxima
__device__ __forceinline__ void merge_fold(MergeAcc &a, const MergeAcc &b)
{
    if (b.M == -INFINITY)
        return;
    const float m_new = fmaxf(a.M, b.M);
    const float sa = (a.M == -INFINITY) ? 0.f : __expf(a.M - m_new);
    const float sb = __expf(b.M - m_new);
    a.acc.x = a.acc.x * sa + b.acc.x * sb;
    a.acc.y = a.acc.y * sa + b.acc.y * sb;
    a.acc.z = a.acc.z * sa + b.acc.z * sb;
    a.acc.w = a.acc.w * sa + b.acc.w * sb;
    a.den = a.den * sa + b.den * sb;
    a.M = m_new;
}

__global__ void __launch_bounds__(MERGE_THREADS, MERGE_BLOCKS_PER_SM) merge_kernel(const MergeParams p)
{
    __shared__ MergeAcc s_part[MERGE_WARPS][MERGE_LANES];
    const int warp = threadIdx.x / MERGE_LANES, ln = threadIdx.x % MERGE_LANES, d = ln * 4;
    grid_launch_dependents();   // a following kernel launched the same way may place its blocks now
    if (threadIdx.x == 0 && blockIdx.x < 8)
        DA_TL(TL_MERGE + blockIdx.x, 0);
    grid_dependency_wait();     // partials and the plan are complete and visible
    if (threadIdx.x == 0 && blockIdx.x < 8)
        DA_TL(TL_MERGE + blockIdx.x, 1);
    const PlanHeader hdr = *p.hdr;
    const MergeCounts cnt = *p.merge_counts;
    const int n_full = static_units_in_use(hdr);
    const int gap = hdr.n_static - n_full;
    int n_small = 0, n_big = 0;
#pragma unroll
    for (int k = 0; k < PLAN_BLOCKS; ++k) {
        n_small += cnt.n_small[k];
        n_big += cnt.n_big[k];
    }
    // i-th entry of a list that the plan blocks filled segment by segment
    auto entry = [&](const int4 *list, const int (&per_block)[PLAN_BLOCKS], int i) {
        int k = 0;
#pragma unroll
        for (int j = 0; j < PLAN_BLOCKS - 1; ++j)
            if (k == j && i >= per_block[j]) {
                i -= per_block[j];
                ++k;
            }
        if (!DA_IN_RANGE(p.status, (long long)k * p.merge_seg + i, (long long)p.merge_seg * PLAN_BLOCKS, 11))
            return make_int4(0, 0, 0, 0);   // (no splits: the entry is skipped below)
        return list[(size_t)k * p.merge_seg + i];
    };
    auto store = [&](int b, int qi, int h, float4 v, float lse_val) {
        if (!DA_IN_RANGE(p.status, b, p.B, 12) || !DA_IN_RANGE(p.status, h, p.Hkv * p.G, 13) ||
            !DA_IN_RANGE(p.status, qi, p.Lq, 14))
            return;
        const int64_t at = (int64_t)b * p.o_sb + (int64_t)qi * p.o_sq + (int64_t)h * p.o_sh + d;
        if (p.out_bf16) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
            __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(p.out) + at;
            if ((reinterpret_cast<uintptr_t>(o) & 7u) == 0) {
                uint2 pk = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
                *reinterpret_cast<uint2 *>(o) = pk;
            } else {
                o[0] = lo.x; o[1] = lo.y; o[2] = hi.x; o[3] = hi.y;
            }
        } else {
            float *o = reinterpret_cast<float *>(p.out) + at;
            if ((reinterpret_cast<uintptr_t>(o) & 15u) == 0) {
                *reinterpret_cast<float4 *>(o) = v;
            } else {
                o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
            }
        }
        if (ln == 0 && p.lse)
            p.lse[(int64_t)b * p.l_sb + (int64_t)qi * p.l_sq + (int64_t)h * p.l_sh] = lse_val;
    };
    // splits [k0, min(k_end, k0 + 32)) of entry e (pair id, first slot, first unit, splits), one head
    auto warp_merge = [&](const int4 &e, int head, int k0, int k_end) {
        const int k = k0 + ln;
        const bool valid = k < k_end;
        int uu = e.z + k;
        if (e.z < n_full && uu >= n_full)
            uu += gap;   // skip the static units that hold no tiles
        int slot = (k == 0) ? e.y : 2 * uu;
        if (valid && !DA_IN_RANGE(p.status, slot, 2 * p.unit_cap, 15))
            slot = 0;
        const int n = min(k_end - k0, 32);
        auto row = [&](int sl) {
            return *reinterpret_cast<const float4 *>(p.part_o + ((int64_t)sl * p.heads_pad + head) * HEAD_DIM + d);
        };
        // the first eight partial rows are asked for together with the lse values (their addresses do
        // not depend on them): one round trip to memory less
        float4 o0[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int sl = __shfl_sync(0xffffffffu, slot, j);
            o0[j] = j < n ? row(sl) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const float l = valid ? p.part_lse[(int64_t)slot * p.heads_pad + head] : -INFINITY;
        MergeAcc a;
        a.M = l;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
            a.M = fmaxf(a.M, __shfl_xor_sync(0xffffffffu, a.M, o));
        const float w = valid ? __expf(l - a.M) : 0.f;
        a.den = w;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
            a.den += __shfl_xor_sync(0xffffffffu, a.den, o);
        a.acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float wj = __shfl_sync(0xffffffffu, w, j);   // 0 past the last split
            a.acc.x += wj * o0[j].x;
            a.acc.y += wj * o0[j].y;
            a.acc.z += wj * o0[j].z;
            a.acc.w += wj * o0[j].w;
        }
        // 8 independent loads in flight per lane and pass
        for (int s0 = 8; s0 < n; s0 += 8) {
            float4 o[8];
            float ws[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int s2 = s0 + j;
                ws[j] = __shfl_sync(0xffffffffu, w, s2 & 31);
                const int sl = __shfl_sync(0xffffffffu, slot, s2 & 31);
                o[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (s2 < n)
                    o[j] = row(sl);
                else
                    ws[j] = 0.f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                a.acc.x += ws[j] * o[j].x;
                a.acc.y += ws[j] * o[j].y;
                a.acc.z += ws[j] * o[j].z;
                a.acc.w += ws[j] * o[j].w;
            }
        }
        return a;
    };
    auto finish = [&](const int4 &e, int head, const MergeAcc &a) {
        const float inv = 1.f / a.den;
        // head = virtual head: query token head / G, head head % G of the pair's KV group
        store(e.x / p.Hkv, head / p.G, (e.x % p.Hkv) * p.G + head % p.G,
              make_float4(a.acc.x * inv, a.acc.y * inv, a.acc.z * inv, a.acc.w * inv), a.M + __logf(a.den));
    };

    // ---- pairs with many splits: one (pair, head) per block at a time, handed out from the last
    //      block down so that they rarely meet the warp-sized items below in the same block
    for (int item = (int)(gridDim.x - 1 - blockIdx.x); item < n_big * p.Gv; item += gridDim.x) {
        const int4 e = entry(p.merge_big, cnt.n_big, item / p.Gv);
        const int head = item % p.Gv;
#ifdef DA_BOUNDS_CHECK
        if (e.w == 0)
            continue;   // an entry the check above refused
#endif
        MergeAcc a = {-INFINITY, 0.f, make_float4(0.f, 0.f, 0.f, 0.f)};
        // the splits are dealt to the eight warps in equal chunks (of at least eight, the number of
        // rows a warp asks for at once), so that up to 64 splits cost one round trip to memory
        const int chunk = max(8, (e.w + MERGE_WARPS - 1) / MERGE_WARPS);
        const int k_end = min(e.w, (warp + 1) * chunk);
        for (int k0 = warp * chunk; k0 < k_end; k0 += 32)
            merge_fold(a, warp_merge(e, head, k0, k_end));
        s_part[warp][ln] = a;
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int k = 1; k < MERGE_WARPS; ++k)
                merge_fold(a, s_part[k][ln]);
            finish(e, head, a);
        }
        __syncthreads();
    }
    // ---- pairs with at most 32 splits: one (pair, head) per warp
    for (int item = blockIdx.x * MERGE_WARPS + warp; item < n_small * p.Gv; item += gridDim.x * MERGE_WARPS) {
        const int4 e = entry(p.merge_small, cnt.n_small, item / p.Gv);
        const int head = item % p.Gv;
#ifdef DA_BOUNDS_CHECK
        if (e.w == 0)
            continue;
#endif
        finish(e, head, warp_merge(e, head, 0, e.w));
    }
    // ---- empty sequences
    for (int b = blockIdx.x; b < p.B; b += gridDim.x) {
        if (p.seq_info[b].w != 0)
            continue;
        for (int h = warp; h < p.Lq * p.Hkv * p.G; h += MERGE_WARPS)
            store(b, h / (p.Hkv * p.G), h % (p.Hkv * p.G), make_float4(0.f, 0.f, 0.f, 0.f), -INFINITY);
    }
    if (threadIdx.x == 0) {
        if (blockIdx.x < 8)
            DA_TL(TL_MERGE + blockIdx.x, 2);
        DA_TL_MAX(TL_MERGE + 8, 2);
    }
}

// =====================================================================================  append
// The step before decode attention in a layer: the new token's K and V rows go into the paged cache
// at position L-1 (seq_lens already counts the new token).  One block per sequence; thread ->
// (K or V, kv head, 16-byte chunk of the row).  Pure byte moves, 16-byte vectors both ways.
struct AppendParams {
    const __nv_bfloat16 *k_new, *v_new;   // [B, Hkv, 128]
    int64_t kn_sb, kn_sh, vn_sb, vn_sh;
    __nv_bfloat16 *k_pages, *v_pages;     // strides in elements: page, head, token
    int64_t k_sp, k_sh, k_st, v_sp, v_sh, v_st;
    const int32_t *block_table;
    int64_t bt_sb;
    const int32_t *seq_lens;
    int64_t sl_stride;
    int32_t *status;
    int32_t B, Hkv, P, num_pages;
    int64_t max_pages;
};

__global__ void __launch_bounds__(256) append_kernel(const AppendParams p)
{
    const int b = blockIdx.x;
    const int L = p.seq_lens[(int64_t)b * p.sl_stride];
    if (L <= 0) {
        if (L < 0 && threadIdx.x == 0)
            report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, 0, L);
        return;
    }
    const int t = L - 1;
    if ((int64_t)(t / p.P) >= p.max_pages) {
        if (threadIdx.x == 0)
            report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, 0, L);
        return;
    }
    const int page = __ldg(p.block_table + (int64_t)b * p.bt_sb + t / p.P);
    if ((uint32_t)page >= (uint32_t)p.num_pages) {
        if (threadIdx.x == 0)
            report_status(p.status, 1 /* DA_DEV_BAD_PAGE */, b, t / p.P, page);
        return;
    }
    const int row = t % p.P;
    for (int e = threadIdx.x; e < 2 * p.Hkv * 16; e += blockDim.x) {
        const int c = e & 15, g = (e >> 4) % p.Hkv, is_v = e / (16 * p.Hkv);
        const __nv_bfloat16 *src = is_v ? p.v_new + (int64_t)b * p.vn_sb + (int64_t)g * p.vn_sh
                                        : p.k_new + (int64_t)b * p.kn_sb + (int64_t)g * p.kn_sh;
        __nv_bfloat16 *dst = is_v ? p.v_pages + (int64_t)page * p.v_sp + (int64_t)g * p.v_sh + (int64_t)row * p.v_st
                                  : p.k_pages + (int64_t)page * p.k_sp + (int64_t)g * p.k_sh + (int64_t)row * p.k_st;
        *reinterpret_cast<uint4 *>(dst + c * 8) = *reinterpret_cast<const uint4 *>(src + c * 8);
    }
}

// The same step for the 8-bit cache: each bf16 element is divided by its KV head's factor in fp32
// (one correctly rounded division) and rounded to the nearest E4M3 code (ties to even, saturating at
// +-448, NaN -> 0x7F) by the hardware conversion.  Thread -> (K or V, kv head, 8 elements).
struct Append8Params {
    const __nv_bfloat16 *k_new, *v_new;   // [B, Hkv, 128]
    int64_t kn_sb, kn_sh, vn_sb, vn_sh;
    uint8_t *k_pages, *v_pages;           // strides in bytes: page, head, token
    int64_t k_sp, k_sh, k_st, v_sp, v_sh, v_st;
    const float *k_scale, *v_scale;       // [Hkv] or NULL (1)
    const int32_t *block_table;
    int64_t bt_sb;
    const int32_t *seq_lens;
    int64_t sl_stride;
    int32_t *status;
    int32_t B, Hkv, P, num_pages;
    int64_t max_pages;
};

__global__ void __launch_bounds__(256) append8_kernel(const Append8Params p)
{
    const int b = blockIdx.x;
    const int L = p.seq_lens[(int64_t)b * p.sl_stride];
    if (L <= 0) {
        if (L < 0 && threadIdx.x == 0)
            report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, 0, L);
        return;
    }
    const int t = L - 1;
    if ((int64_t)(t / p.P) >= p.max_pages) {
        if (threadIdx.x == 0)
            report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, 0, L);
        return;
    }
    const int page = __ldg(p.block_table + (int64_t)b * p.bt_sb + t / p.P);
    if ((uint32_t)page >= (uint32_t)p.num_pages) {
        if (threadIdx.x == 0)
            report_status(p.status, 1 /* DA_DEV_BAD_PAGE */, b, t / p.P, page);
        return;
    }
    const int row = t % p.P;
    for (int e = threadIdx.x; e < 2 * p.Hkv * 16; e += blockDim.x) {
        const int c = e & 15, g = (e >> 4) % p.Hkv, is_v = e / (16 * p.Hkv);
        const __nv_bfloat16 *src = is_v ? p.v_new + (int64_t)b * p.vn_sb + (int64_t)g * p.vn_sh
                                        : p.k_new + (int64_t)b * p.kn_sb + (int64_t)g * p.kn_sh;
        uint8_t *dst = is_v ? p.v_pages + (int64_t)page * p.v_sp + (int64_t)g * p.v_sh + (int64_t)row * p.v_st
                            : p.k_pages + (int64_t)page * p.k_sp + (int64_t)g * p.k_sh + (int64_t)row * p.k_st;
        const float *sc = is_v ? p.v_scale : p.k_scale;
        const float factor = sc ? __ldg(sc + g) : 1.f;
        const uint4 in = *reinterpret_cast<const uint4 *>(src + c * 8);
        const uint32_t w[4] = {in.x, in.y, in.z, in.w};
        uint32_t codes[2];
#pragma unroll
        for (int h = 0; h < 2; ++h)
            codes[h] = pack_e4m3x4(__fdiv_rn(bf16_lo_to_float(w[2 * h]), factor), __fdiv_rn(bf16_hi_to_float(w[2 * h]), factor),
                                   __fdiv_rn(bf16_lo_to_float(w[2 * h + 1]), factor),
                                   __fdiv_rn(bf16_hi_to_float(w[2 * h + 1]), factor));
        *reinterpret_cast<uint2 *>(dst + c * 8) = make_uint2(codes[0], codes[1]);
    }
}

// =====================================================================================  host-input staging
// decode_attn_host_io: the three per-step inputs (q, block table, lengths) are read straight out of the
// caller's pinned, mapped host buffers by all SMs at once and written to the staging area -- one launch
// instead of three DMA copies, each of which costs several microseconds before its first byte moves.
struct StageParams {
    const uint8_t *src[3];
    uint8_t *dst[3];
    unsigned long long bytes[3];   // multiples of 4
};

__global__ void __launch_bounds__(256) stage_inputs_kernel(const StageParams p)
{
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, nthr = (size_t)gridDim.x * blockDim.x;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const uint8_t *s = p.src[r];
        uint8_t *d = p.dst[r];
        const size_t n = p.bytes[r];
        size_t done = 0;
        if (((reinterpret_cast<uintptr_t>(s) | reinterpret_cast<uintptr_t>(d)) & 15u) == 0) {
            const size_t n16 = n / 16;
            for (size_t i = tid; i < n16; i += nthr)
                reinterpret_cast<uint4 *>(d)[i] = reinterpret_cast<const uint4 *>(s)[i];
            done = n16 * 16;
        }
        for (size_t i = done / 4 + tid; i < n / 4; i += nthr)
            reinterpret_cast<uint32_t *>(d)[i] = reinterpret_cast<const uint32_t *>(s)[i];
    }
}

}  // namespace da
