// Host side of the C ABI declared in include/decode_attn.h: argument checks, the workspace
// layout, TMA descriptor creation and the three launches.  Nothing here allocates device memory.
#include "../../include/decode_attn.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>

#include "da_prefix.cuh"

namespace {

using namespace da;

constexpr int kVersion = 116;
constexpr int kMaxDevices = 64;
constexpr int kMaxGridBlocks = 4096;
constexpr int kMaxUnits = 8192;
constexpr int kMaxPrefixSplits = 4;
constexpr int kMaxGroup = 16;        // query heads per KV head
constexpr int kMaxStreamRows = 48;   // query rows per KV head (new tokens x heads) the streaming kernels take

std::mutex g_mu;
std::atomic<int> g_last_cuda_error{0};
std::atomic<int64_t> g_launches{0};
int64_t g_opt_grid_blocks = 0;   // 0 = two blocks per SM
int64_t g_opt_tail_units = 4;    // ticketed units per thread block (0: one static range per block only)
int64_t g_opt_static_frac = 224; // share of the work given to the static ranges, in 1/256
int64_t g_opt_kv_evict_first = 2; // L2 policy of the K and V loads: 0 normal, 1 evict first, 2 chosen by the plan kernel
int64_t g_opt_cascade_overlap = 1;  // the cascade's prefix pass beside its pass over the sequences' own tokens: 0 never,
                                    // 1 where the host's estimate favours it, 2 wherever the shapes allow
int64_t g_opt_cascade_prefix_sms = 0;   // SMs given to the prefix kernel then (0: a third of them)
int64_t g_opt_fold_pairs = 2;     // pairs cut in two by neighbouring blocks' own ranges are folded by the partition kernel:
                                  // 0 never, 1 always, 2 when the results go to host memory (decode_attn_host_io)
thread_local bool t_results_to_host = false;   // set by the host-buffer entry points around their call of run()
int64_t g_opt_direct_path = 1;    // small calls (every pair fits one wave of blocks) skip the plan and merge kernels
int64_t g_opt_extend_stream_rows = 16;   // decode_attn_extend: Lq * (Hq / Hkv) up to this many rows go through the
                                         // streaming (partition) kernel, more through the tcgen05 kernel; 0: never
cudaEvent_t g_ev_before = nullptr, g_ev_after = nullptr;
#ifdef DA_DIAG
int64_t g_host_wait_limit_us = 2000000, g_host_withhold[2] = {-1, -1};   // host copies of the device variables
#endif

struct DeviceState {
    void *ws = nullptr;
    size_t ws_bytes = 0;
    int sm_count = 0;
    bool attrs_set = false;
    // decode_attn_cascade with its two passes side by side: the second pass runs on a stream of the library's
    // own, forked from and joined to the caller's stream by these events (made at the first such call)
    cudaStream_t side_hi = nullptr, side_lo = nullptr;   // prefix kernel (highest priority); plan / partition / merge
    cudaEvent_t ev_fork = nullptr, ev_join_hi = nullptr, ev_join_lo = nullptr;
    bool side_failed = false;
};
DeviceState g_dev[kMaxDevices];

struct TmapKey {
    const void *ptr;
    int64_t shape[4];
    int64_t stride[4];
    int box_rows;
    int planes;   // 2: 5-D view, one box = both 64-column halves; 1: 4-D view, one box = one half;
                  // 0: 8-bit pool, 4-D view, one box = whole 128-byte rows
};
struct TmapEntry {
    TmapKey key;
    CUtensorMap map;
    bool used = false;
};
constexpr int kTmapCache = 16;
TmapEntry g_tmaps[kTmapCache];
int g_tmap_next = 0;

// Scratch for decode_attn_static_scratch(): part of the library image, so every GPU that loads the
// library holds these bytes until the process exits.  In host code this name is only a stand-in
// for the device object; its device address comes from cudaGetSymbolAddress (static_scratch_ptr).
constexpr size_t kStaticScratchBytes = 6u << 20;   // 6 MiB
constexpr int64_t kStaticMaxSeqs = 4096;
constexpr int kStaticMaxBlocks = 320;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
uint8_t *g_static_scratch_addr[kMaxDevices] = {};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int cuda_fail(cudaError_t e)
{
    g_last_cuda_error.store((int)e);
    return DA_ERR_CUDA;
}
#define DA_CUDA(call)                      \
    do {                                   \
        cudaError_t e_ = (call);           \
        if (e_ != cudaSuccess)             \
            return cuda_fail(e_);          \
    } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int current_device(int *dev, DeviceState **st)
{
    DA_CUDA(cudaGetDevice(dev));
    if (*dev < 0 || *dev >= kMaxDevices)
        return DA_ERR_UNSUPPORTED;
    *st = &g_dev[*dev];
    if ((*st)->sm_count == 0) {
        int n = 0;
        DA_CUDA(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, *dev));
        (*st)->sm_count = n;
    }
    return DA_OK;
}

int grid_blocks_for(const DeviceState *st)
{
    int64_t n = g_opt_grid_blocks > 0 ? g_opt_grid_blocks : 2 * (int64_t)st->sm_count;
    if (n < 1) n = 1;
    if (n > kMaxGridBlocks) n = kMaxGridBlocks;
    return (int)n;
}

// Ticketed units for a grid of nblocks (all units together stay within kMaxUnits).
int tail_units_for(int nblocks)
{
    int64_t t = g_opt_tail_units * (int64_t)nblocks;
    if (t + nblocks > kMaxUnits) t = kMaxUnits - nblocks;
    return t > 0 ? (int)t : 0;
}

// status record, the direct path's pair counters and the two-piece pairs' counters: zero between calls
constexpr size_t kWsHeadBytes = 256 + 2048 + (size_t)kMaxUnits * 2 * 4;

struct WsLayout {
    size_t status, counters, fold_counters, hdr, merge_counts, seq_info, prefix, unit_work, merge_small, merge_big, part_lse, part_o;
    int merge_seg;
    size_t stg_q, stg_bt, stg_sl, stg_out, stg_lse;
    size_t pre_o, pre_lse, suf_o, suf_lse, total;   // cascade scratch
};

// `units` = thread blocks of the partition kernel x (1 + ticketed units per block); `heads_pad` = most padded
// (virtual) heads per KV group whose partial results the slots must hold
WsLayout ws_layout(int64_t B, int64_t Hq, int64_t D, int64_t max_pages, int units, int heads_pad = kMaxStreamRows)
{
    WsLayout w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    w.status = take(16);
    w.counters = take((size_t)DIRECT_MAX_PAIRS * 4);
    w.fold_counters = take((size_t)kMaxUnits * 2 * 4);   // (a fixed size, so that the head does not move with the options)
    static_assert(DIRECT_MAX_PAIRS * 4 == 2048, "the cleared head holds the status record and the two counter arrays");
    w.hdr = take(sizeof(PlanHeader));
    w.merge_counts = take(sizeof(MergeCounts));
    w.merge_seg = (units + PLAN_BLOCKS - 1) / PLAN_BLOCKS;   // a plan block lists at most one pair per unit it cuts
    w.seq_info = take((size_t)B * 16);
    w.prefix = take((size_t)(B + 1) * 4);
    w.unit_work = take((size_t)units * 16);
    w.merge_small = take((size_t)w.merge_seg * PLAN_BLOCKS * 16);
    w.merge_big = take((size_t)w.merge_seg * PLAN_BLOCKS * 16);
    w.part_lse = take((size_t)2 * units * heads_pad * 4);
    w.part_o = take((size_t)2 * units * heads_pad * HEAD_DIM * 4);
    w.stg_q = take((size_t)B * Hq * D * 2);
    w.stg_bt = take((size_t)B * max_pages * 4);
    w.stg_sl = take((size_t)B * 4);
    w.stg_out = take((size_t)B * Hq * D * 4);
    w.stg_lse = take((size_t)B * Hq * 4);
    w.pre_o = take((size_t)kMaxPrefixSplits * B * Hq * D * 4);
    w.pre_lse = take((size_t)kMaxPrefixSplits * B * Hq * 4);
    w.suf_o = take((size_t)B * Hq * D * 4);
    w.suf_lse = take((size_t)B * Hq * 4);
    w.total = off;
    return w;
}

int get_encoder()
{
    if (g_encode)
        return DA_OK;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    DA_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || !fn)
        return cuda_fail(cudaErrorNotSupported);
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return DA_OK;
}

// A 5-D view {d within a 64-column half, token, half, kv head, page} of a K or V pool, box
// {64, box_rows, 2, 1, 1}, 128-byte swizzle.  Splitting head_dim into two halves keeps the inner box
// extent at the swizzle span (128 bytes) while one TMA operation still brings all 128 columns of
// box_rows tokens: in shared memory a box is two planes of box_rows 128-byte rows.
// planes = 2: the partition kernel's view, and the prefix kernel's view of V.  planes = 1: a 4-D view
// {d, token, kv head, page} with box {64, box_rows, 1, 1} (one 64-column half per box), the prefix
// kernel's view of K, whose score product wants each half of a tile contiguous.
int get_tmap(const da_tensor *t, int box_rows, int planes, CUtensorMap *out)
{
    TmapKey key;
    std::memset(&key, 0, sizeof key);
    key.ptr = t->data;
    for (int i = 0; i < 4; ++i) {
        key.shape[i] = t->shape[i];
        key.stride[i] = t->stride[i];
    }
    key.box_rows = box_rows;
    key.planes = planes;
    for (int i = 0; i < kTmapCache; ++i)
        if (g_tmaps[i].used && std::memcmp(&g_tmaps[i].key, &key, sizeof key) == 0) {
            *out = g_tmaps[i].map;
            return DA_OK;
        }
    int rc = get_encoder();
    if (rc != DA_OK)
        return rc;
    CUtensorMap m;
    CUresult r;
    if (planes == 0) {
        // 8-bit codes: {d, token, kv head, page}, strides in bytes, box {128, box_rows, 1, 1}: a row is
        // exactly the 128-byte swizzle span
        cuuint64_t gdim[4] = {(cuuint64_t)t->shape[3], (cuuint64_t)t->shape[2], (cuuint64_t)t->shape[1], (cuuint64_t)t->shape[0]};
        cuuint64_t gstr[3] = {(cuuint64_t)t->stride[2], (cuuint64_t)t->stride[1], (cuuint64_t)t->stride[0]};
        cuuint32_t box[4] = {128, (cuuint32_t)box_rows, 1, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, t->data, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else if (planes == 2) {
        cuuint64_t gdim[5] = {64, (cuuint64_t)t->shape[2], 2, (cuuint64_t)t->shape[1], (cuuint64_t)t->shape[0]};
        cuuint64_t gstr[4] = {(cuuint64_t)t->stride[2] * 2, 128, (cuuint64_t)t->stride[1] * 2, (cuuint64_t)t->stride[0] * 2};
        cuuint32_t box[5] = {64, (cuuint32_t)box_rows, 2, 1, 1};
        cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, t->data, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        cuuint64_t gdim[4] = {(cuuint64_t)t->shape[3], (cuuint64_t)t->shape[2], (cuuint64_t)t->shape[1], (cuuint64_t)t->shape[0]};
        cuuint64_t gstr[3] = {(cuuint64_t)t->stride[2] * 2, (cuuint64_t)t->stride[1] * 2, (cuuint64_t)t->stride[0] * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, t->data, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error.store((int)cudaErrorInvalidValue);
        return DA_ERR_CUDA;
    }
    TmapEntry &e = g_tmaps[g_tmap_next];
    g_tmap_next = (g_tmap_next + 1) % kTmapCache;
    e.key = key;
    e.map = m;
    e.used = true;
    *out = m;
    return DA_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Dims {
    int64_t B, Hq, Hkv, G, P, num_pages, max_pages;
};

int check_pool(const da_tensor *t, int32_t dtype = DA_BF16)
{
    if (!t->data) return DA_ERR_NULL;
    if (t->dtype != dtype) return DA_ERR_DTYPE;
    if (t->ndim != 4) return DA_ERR_SHAPE;
    if (t->shape[0] <= 0 || t->shape[1] <= 0 || t->shape[2] <= 0) return DA_ERR_SHAPE;
    if (t->shape[3] != HEAD_DIM) return DA_ERR_UNSUPPORTED;
    if (t->stride[3] != 1 || !aligned16(t->data)) return DA_ERR_STRIDE_ALIGN;
    const int64_t item = dtype == DA_FP8_E4M3 ? 1 : 2;
    for (int i = 0; i < 3; ++i)
        if (t->stride[i] <= 0 || (t->stride[i] * item) % 16 != 0 || t->stride[i] * item >= (1ll << 40))
            return DA_ERR_STRIDE_ALIGN;
    return DA_OK;
}

int validate(const da_tensor *q, const da_tensor *k, const da_tensor *v, const da_tensor *bt, const da_tensor *sl,
             const da_tensor *out, const da_tensor *lse, Dims *d, int32_t pool_dtype = DA_BF16)
{
    if (!q || !k || !v || !bt || !sl || !out) return DA_ERR_NULL;
    if (!q->data || !bt->data || !sl->data || !out->data) return DA_ERR_NULL;
    if (lse && !lse->data) return DA_ERR_NULL;
    if (q->dtype != DA_BF16 || bt->dtype != DA_I32 || sl->dtype != DA_I32) return DA_ERR_DTYPE;
    if (out->dtype != DA_F32 && out->dtype != DA_BF16) return DA_ERR_DTYPE;
    if (lse && lse->dtype != DA_F32) return DA_ERR_DTYPE;
    if (q->ndim != 3 || bt->ndim != 2 || sl->ndim != 1 || out->ndim != 3) return DA_ERR_SHAPE;
    if (lse && lse->ndim != 2) return DA_ERR_SHAPE;
    int rc = check_pool(k, pool_dtype);
    if (rc != DA_OK) return rc;
    rc = check_pool(v, pool_dtype);
    if (rc != DA_OK) return rc;
    for (int i = 0; i < 4; ++i)
        if (k->shape[i] != v->shape[i]) return DA_ERR_SHAPE;
    d->B = q->shape[0];
    d->Hq = q->shape[1];
    d->num_pages = k->shape[0];
    d->Hkv = k->shape[1];
    d->P = k->shape[2];
    d->max_pages = bt->shape[1];
    if (d->B < 0 || d->Hq <= 0 || d->Hkv <= 0 || d->num_pages <= 0 || d->max_pages <= 0) return DA_ERR_SHAPE;
    if (d->B > (1 << 24) || d->num_pages > 0x7fffffffll || d->max_pages > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
    if (q->shape[2] != HEAD_DIM) return DA_ERR_UNSUPPORTED;
    if (d->Hq % d->Hkv != 0) return DA_ERR_SHAPE;
    d->G = d->Hq / d->Hkv;
    if (d->G > kMaxGroup) return DA_ERR_UNSUPPORTED;
    if (d->P != 16 && d->P != 32 && d->P != 64 && d->P != 128) return DA_ERR_UNSUPPORTED;
    if (bt->shape[0] != d->B || sl->shape[0] != d->B) return DA_ERR_SHAPE;
    if (out->shape[0] != d->B || out->shape[1] != d->Hq || out->shape[2] != HEAD_DIM) return DA_ERR_SHAPE;
    if (lse && (lse->shape[0] != d->B || lse->shape[1] != d->Hq)) return DA_ERR_SHAPE;
    if (q->stride[2] != 1 || out->stride[2] != 1 || bt->stride[1] != 1) return DA_ERR_STRIDE_ALIGN;
    if ((q->stride[0] | q->stride[1]) & 1) return DA_ERR_STRIDE_ALIGN;   // rows read as 32-bit pairs
    if (reinterpret_cast<uintptr_t>(q->data) & 3u) return DA_ERR_STRIDE_ALIGN;
    return DA_OK;
}

template <int NT8, int CSETS>
int set_kernel_attrs()
{
    DA_CUDA(cudaFuncSetAttribute(partition_kernel<NT8, false, CSETS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 PartCfg<NT8, CSETS>::SMEM_BYTES));
    DA_CUDA(cudaFuncSetAttribute(partition_kernel<NT8, true, CSETS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 PartCfg<NT8, CSETS>::SMEM_BYTES));
    return DA_OK;
}

int set_all_kernel_attrs(DeviceState *st)
{
    if (st->attrs_set) return DA_OK;
    int rc = set_kernel_attrs<1, 1>();
    if (rc != DA_OK) return rc;
    rc = set_kernel_attrs<2, 1>();
    if (rc != DA_OK) return rc;
    rc = set_kernel_attrs<2, 2>();
    if (rc != DA_OK) return rc;
    rc = set_kernel_attrs<3, 2>();
    if (rc != DA_OK) return rc;
    DA_CUDA(cudaFuncSetAttribute(prefix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PF_SMEM_BYTES));
    // The prefix kernel's warps redistribute the block's registers among themselves (setmaxnreg): the shares
    // are written for a block launched with PF_REGS_LAUNCH registers a thread, and a block launched with
    // fewer would wait forever for the increase.  Refuse rather than launch.
    cudaFuncAttributes fa;
    DA_CUDA(cudaFuncGetAttributes(&fa, prefix_kernel));
    if (fa.numRegs < PF_REGS_LAUNCH) return DA_ERR_UNSUPPORTED;
    st->attrs_set = true;
    return DA_OK;
}

// The library's own stream and events for the cascade's side-by-side mode; false if they cannot be made
// (then the passes run one after the other).
bool ensure_side_stream(DeviceState *st)
{
    if (st->side_hi) return true;
    if (st->side_failed) return false;
    cudaStream_t hi = nullptr, lo = nullptr;
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
    int least = 0, greatest = 0;
    bool ok = cudaDeviceGetStreamPriorityRange(&least, &greatest) == cudaSuccess &&
              cudaStreamCreateWithPriority(&hi, cudaStreamNonBlocking, greatest) == cudaSuccess &&
              cudaStreamCreateWithPriority(&lo, cudaStreamNonBlocking, least) == cudaSuccess;
    for (int i = 0; ok && i < 3; ++i)
        ok = cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming) == cudaSuccess;
    if (ok) {
        st->side_hi = hi;
        st->side_lo = lo;
        st->ev_fork = ev[0];
        st->ev_join_hi = ev[1];
        st->ev_join_lo = ev[2];
        return true;
    }
    cudaGetLastError();   // not an error of the call being made
    for (cudaEvent_t e : ev)
        if (e) cudaEventDestroy(e);
    if (hi) cudaStreamDestroy(hi);
    if (lo) cudaStreamDestroy(lo);
    st->side_failed = true;
    return false;
}

// One instance of the partition kernel: NT8 column tiles of 8 heads per warp, CSETS column sets.
template <int NT8, int CSETS>
int launch_partition(cudaLaunchConfig_t &cfg, bool kv8, const CUtensorMap &tm_k, const CUtensorMap &tm_v, const PartParams &pa)
{
    cfg.blockDim = dim3((unsigned)PartCfg<NT8, CSETS>::THREADS);
    cfg.dynamicSmemBytes = PartCfg<NT8, CSETS>::SMEM_BYTES;
    if (kv8)
        DA_CUDA(cudaLaunchKernelEx(&cfg, partition_kernel<NT8, true, CSETS>, tm_k, tm_v, pa));
    else
        DA_CUDA(cudaLaunchKernelEx(&cfg, partition_kernel<NT8, false, CSETS>, tm_k, tm_v, pa));
    return DA_OK;
}

int launch_plan(const da_tensor *sl, int32_t window, int32_t first_token, const Dims &d, uint8_t *ws,
                const WsLayout &lay, int nblocks, int n_tail, cudaStream_t stream, int tile_t = TILE_T, int min_len = 0,
                const da_tensor *bt = nullptr)
{
    PlanParams pp;
    pp.seq_lens = static_cast<const int32_t *>(sl->data);
    pp.sl_stride = sl->stride[0];
    pp.seq_info = reinterpret_cast<int4 *>(ws + lay.seq_info);
    pp.prefix = reinterpret_cast<int32_t *>(ws + lay.prefix);
    pp.unit_work = reinterpret_cast<int4 *>(ws + lay.unit_work);
    pp.merge_small = reinterpret_cast<int4 *>(ws + lay.merge_small);
    pp.merge_big = reinterpret_cast<int4 *>(ws + lay.merge_big);
    pp.merge_counts = reinterpret_cast<MergeCounts *>(ws + lay.merge_counts);
    pp.merge_seg = lay.merge_seg;
    pp.hdr = reinterpret_cast<PlanHeader *>(ws + lay.hdr);
    pp.status = reinterpret_cast<int32_t *>(ws + lay.status);
    pp.B = (int32_t)d.B;
    pp.Hkv = (int32_t)d.Hkv;
    pp.P = (int32_t)d.P;
    pp.window = window;
    pp.tile_t = tile_t;
    pp.min_len = min_len;
    pp.first_token = first_token;
    pp.block_table = (bt && d.max_pages > 0) ? static_cast<const int32_t *>(bt->data) : nullptr;
    pp.bt_sb = bt ? bt->stride[0] : 0;
    pp.kv_policy = (int32_t)g_opt_kv_evict_first;
    // the plan kernel compares entry first_token / P of the rows: it must exist
    if (pp.kv_policy == 2 && (!pp.block_table || (int64_t)first_token / d.P >= d.max_pages)) pp.kv_policy = 1;
    pp.n_static = nblocks;
    pp.n_tail_max = n_tail;
    pp.static_frac_q8 = (int32_t)g_opt_static_frac;
    pp.max_pages = d.max_pages;
    pp.fold_pairs = g_opt_fold_pairs == 1 || (g_opt_fold_pairs == 2 && t_results_to_host);
    // Programmatic stream serialization: the blocks may be placed while the kernel before this one in
    // the stream finishes; the kernel waits on the device before it reads or writes anything.
    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)PLAN_BLOCKS);
    cfg.blockDim = dim3((unsigned)PLAN_THREADS);
    cfg.stream = stream;
    cfg.attrs = &pdl;
    cfg.numAttrs = 1;
    DA_CUDA(cudaLaunchKernelEx(&cfg, plan_kernel, pp));
    g_launches.fetch_add(1);
    return DA_OK;
}

// The three launches of the hot path, with every scratch array taken from `ws` as laid out by `lay`.
// Called with g_mu held.
int launch_path(DeviceState *st, const Dims &d, uint8_t *ws, const WsLayout &lay, int nblocks, int n_tail,
                const da_tensor *q,
                const da_tensor *k, const da_tensor *v, const da_tensor *bt, const da_tensor *sl, int32_t window,
                float scale, da_tensor *out, da_tensor *lse, cudaStream_t stream, int32_t first_token = 0,
                bool kv8 = false, const float *k_scale = nullptr, const float *v_scale = nullptr, int Lq = 1,
                int64_t q_sq = 0, int64_t o_sq = 0, int64_t l_sq = 0, int late_blocks = 0)
{
    // late_blocks: of the nblocks thread blocks, the last late_blocks get no range of their own and live on
    // tickets (they are expected to become resident late: the cascade's prefix kernel holds their SMs); the
    // partition kernel is then launched the ordinary way, so that it starts after the plan kernel has ended
    // and not while the prefix kernel's blocks may still be on their way to their SMs.
    int rc = set_all_kernel_attrs(st);
    if (rc != DA_OK) return rc;
    // Up to 16 (virtual) heads per KV group: one column set, two blocks per SM.  17 .. 48 (several new tokens
    // per sequence): two column sets in a block of nine warps, one block per SM.
    const int gv = (int)(Lq * d.G);
    const int csets = gv <= 16 ? 1 : 2;
    const int nt8 = gv <= 8 ? 1 : (gv <= 32 ? 2 : 3);
    if (csets == 2 && g_opt_grid_blocks <= 0) {
        nblocks = st->sm_count;
        n_tail = tail_units_for(nblocks);
    }
    const int tile_t = kv8 ? TILE_T8 : TILE_T;
    const int box_rows = d.P < tile_t ? (int)d.P : tile_t;
    CUtensorMap tm_k, tm_v;
    rc = get_tmap(k, box_rows, kv8 ? 0 : 2, &tm_k);
    if (rc != DA_OK) return rc;
    rc = get_tmap(v, box_rows, kv8 ? 0 : 2, &tm_v);
    if (rc != DA_OK) return rc;

    // Direct path: a call whose (sequence, KV head) pairs, each cut into a few pieces, fit one wave of thread
    // blocks is launched as ONE kernel -- every block works out its own piece from seq_lens, and the block that
    // finishes a pair last folds the pieces -- instead of plan + partition + merge, whose fixed costs (two
    // more launches, the plan's round trips) exceed the work of such a call.  The host cannot see the lengths:
    // it bounds a pair's tiles by the block-table row (and the window).
    int direct_splits = 0;
    if (g_opt_direct_path && g_opt_grid_blocks <= 0 && Lq == 1 && first_token == 0 && late_blocks == 0 &&
        d.B * d.Hkv <= DIRECT_MAX_PAIRS) {
        int64_t tiles_max = (d.max_pages * d.P + tile_t - 1) / tile_t;
        if (window > 0) tiles_max = std::min<int64_t>(tiles_max, (int64_t)window / tile_t + 2);
        const int64_t pairs = d.B * d.Hkv, wave = 2 * (int64_t)st->sm_count;
        int64_t s = std::min<int64_t>(8, std::max<int64_t>(1, tiles_max));       // one tile a piece where the wave has room
        s = std::min<int64_t>(s, wave / std::max<int64_t>(pairs, 1));
        if (s >= 1 && tiles_max <= 8 * s)   // at most eight tiles a piece: beyond that the planned split balances better
            direct_splits = (int)s;
    }
    if (direct_splits) {
        nblocks = (int)(d.B * d.Hkv) * direct_splits;   // <= two per SM <= the slots the workspace was sized for
        n_tail = 0;
    } else {
        rc = launch_plan(sl, window, first_token, d, ws, lay, nblocks - late_blocks, n_tail, stream, tile_t, Lq > 1 ? Lq : 0,
                         bt);
        if (rc != DA_OK) return rc;
    }

    PartParams pa;
    pa.q = static_cast<const __nv_bfloat16 *>(q->data);
    pa.q_sb = q->stride[0];
    pa.q_sh = q->stride[1];
    pa.block_table = static_cast<const int32_t *>(bt->data);
    pa.bt_sb = bt->stride[0];
    pa.out = out->data;
    pa.o_sb = out->stride[0];
    pa.o_sh = out->stride[1];
    pa.lse = lse ? static_cast<float *>(lse->data) : nullptr;
    pa.l_sb = lse ? lse->stride[0] : 0;
    pa.l_sh = lse ? lse->stride[1] : 0;
    pa.seq_info = reinterpret_cast<const int4 *>(ws + lay.seq_info);
    pa.unit_work = reinterpret_cast<const int4 *>(ws + lay.unit_work);
    pa.hdr = reinterpret_cast<PlanHeader *>(ws + lay.hdr);
    pa.part_o = reinterpret_cast<float *>(ws + lay.part_o);
    pa.part_lse = reinterpret_cast<float *>(ws + lay.part_lse);
    pa.status = reinterpret_cast<int32_t *>(ws + lay.status);
    pa.B = (int32_t)d.B;
    pa.Hkv = (int32_t)d.Hkv;
    pa.G = (int32_t)d.G;
    pa.P = (int32_t)d.P;
    pa.log2_P = d.P == 16 ? 4 : (d.P == 32 ? 5 : (d.P == 64 ? 6 : 7));
    pa.box_rows = box_rows;
    pa.num_pages = (int32_t)d.num_pages;
    pa.out_bf16 = out->dtype == DA_BF16;
    pa.scale_log2 = scale * LOG2E;
    pa.k_scale = k_scale;
    pa.v_scale = v_scale;
    pa.Lq = Lq;
    pa.Gv = (int32_t)(Lq * d.G);
    pa.q_sq = q_sq;
    pa.o_sq = o_sq;
    pa.l_sq = l_sq;
    pa.unit_cap = nblocks + n_tail;
    pa.max_pages = d.max_pages;
    pa.direct_splits = direct_splits;
    pa.window = window;
    pa.seq_lens = static_cast<const int32_t *>(sl->data);
    pa.sl_stride = sl->stride[0];
    pa.pair_counters = reinterpret_cast<int32_t *>(ws + lay.counters);
    pa.fold_counters = reinterpret_cast<int32_t *>(ws + lay.fold_counters);
    const bool timed = g_ev_before && g_ev_after;
    if (timed) DA_CUDA(cudaEventRecord(g_ev_before, stream));
    // Both dependent kernels are launched with programmatic stream serialization: their blocks may
    // become resident while the kernel before them still runs, and they wait on the device
    // (griddepcontrol.wait) before touching its results.
    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)nblocks);
    cfg.stream = stream;
    cfg.attrs = &pdl;
    cfg.numAttrs = late_blocks ? 0 : 1;
    if (csets == 1 && nt8 == 1)
        rc = launch_partition<1, 1>(cfg, kv8, tm_k, tm_v, pa);
    else if (csets == 1)
        rc = launch_partition<2, 1>(cfg, kv8, tm_k, tm_v, pa);
    else if (nt8 == 2)
        rc = launch_partition<2, 2>(cfg, kv8, tm_k, tm_v, pa);
    else
        rc = launch_partition<3, 2>(cfg, kv8, tm_k, tm_v, pa);
    if (rc != DA_OK) return rc;
    g_launches.fetch_add(1);
    if (timed) DA_CUDA(cudaEventRecord(g_ev_after, stream));
    if (direct_splits)
        return DA_OK;   // the partition kernel wrote the results itself

    MergeParams mp;
    mp.seq_info = pa.seq_info;
    mp.prefix = reinterpret_cast<const int32_t *>(ws + lay.prefix);
    mp.hdr = pa.hdr;
    mp.merge_small = reinterpret_cast<const int4 *>(ws + lay.merge_small);
    mp.merge_big = reinterpret_cast<const int4 *>(ws + lay.merge_big);
    mp.merge_counts = reinterpret_cast<const MergeCounts *>(ws + lay.merge_counts);
    mp.merge_seg = lay.merge_seg;
    mp.part_o = pa.part_o;
    mp.part_lse = pa.part_lse;
    mp.out = out->data;
    mp.o_sb = pa.o_sb;
    mp.o_sh = pa.o_sh;
    mp.lse = pa.lse;
    mp.l_sb = pa.l_sb;
    mp.l_sh = pa.l_sh;
    mp.B = pa.B;
    mp.Hkv = pa.Hkv;
    mp.G = pa.G;
    mp.heads_pad = csets * nt8 * 8;
    mp.out_bf16 = pa.out_bf16;
    mp.Lq = pa.Lq;
    mp.Gv = pa.Gv;
    mp.o_sq = o_sq;
    mp.l_sq = l_sq;
    mp.unit_cap = pa.unit_cap;
    mp.status = pa.status;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)(MERGE_BLOCKS_PER_SM * st->sm_count));
    cfg.blockDim = dim3((unsigned)MERGE_THREADS);
    cfg.dynamicSmemBytes = 0;
    DA_CUDA(cudaLaunchKernelEx(&cfg, merge_kernel, mp));
    g_launches.fetch_add(1);
    return DA_OK;
}

int run(const da_tensor *q, const da_tensor *k, const da_tensor *v, const da_tensor *bt, const da_tensor *sl,
        int32_t window, float scale, da_tensor *out, da_tensor *lse, cudaStream_t stream, bool kv8 = false,
        const float *k_scale = nullptr, const float *v_scale = nullptr)
{
    Dims d;
    int rc = validate(q, k, v, bt, sl, out, lse, &d, kv8 ? DA_FP8_E4M3 : DA_BF16);
    if (rc != DA_OK) return rc;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    const int nblocks = grid_blocks_for(st);
    const int n_tail = tail_units_for(nblocks);
    const WsLayout lay = ws_layout(d.B, d.Hq, HEAD_DIM, d.max_pages, nblocks + n_tail);
    if (!st->ws || st->ws_bytes < lay.stg_q) return DA_ERR_WORKSPACE;   // staging is only for host_io
    if (d.B == 0) return DA_OK;
    return launch_path(st, d, static_cast<uint8_t *>(st->ws), lay, nblocks, n_tail, q, k, v, bt, sl, window, scale,
                       out, lse, stream, 0, kv8, k_scale, v_scale);
}

// The device-side address of a pinned, mapped host buffer (NULL for pageable or unknown memory).
void *mapped_device_pointer(const void *host_ptr)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host_ptr) != cudaSuccess) {
        cudaGetLastError();   // not an error of the call being made
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

bool contiguous(const da_tensor *t)
{
    int64_t expect = 1;
    for (int i = t->ndim - 1; i >= 0; --i) {
        if (t->shape[i] != 1 && t->stride[i] != expect) return false;
        expect *= t->shape[i];
    }
    return true;
}

}  // namespace

extern "C" {

int decode_attn(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const da_tensor *block_table,
                const da_tensor *seq_lens, int32_t window, float scale, da_tensor *out, da_tensor *lse, void *stream)
{
    return run(q, k_pages, v_pages, block_table, seq_lens, window, scale, out, lse, static_cast<cudaStream_t>(stream));
}

int decode_attn_fp8kv(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const float *k_scale,
                      const float *v_scale, const da_tensor *block_table, const da_tensor *seq_lens, int32_t window,
                      float scale, da_tensor *out, da_tensor *lse, void *stream)
{
    return run(q, k_pages, v_pages, block_table, seq_lens, window, scale, out, lse, static_cast<cudaStream_t>(stream),
               true, k_scale, v_scale);
}

}  // extern "C"

namespace {
// decode_attn_cascade / decode_attn_fp8kv_cascade.  For the 8-bit cache the shared prefix is first widened,
// exactly, into a bf16 copy in the caller's scratch, which the tensor-core kernel then reads as a pool whose
// page i holds tokens [i P, (i+1) P); the per-KV-head factors enter in that kernel.
int run_cascade(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const da_tensor *block_table,
                const da_tensor *seq_lens, int32_t shared_prefix_tokens, float scale, da_tensor *out, da_tensor *lse,
                cudaStream_t stream, bool kv8, const float *k_scale, const float *v_scale, void *prefix_scratch,
                size_t prefix_scratch_bytes)
{
    if (shared_prefix_tokens <= 0)
        return run(q, k_pages, v_pages, block_table, seq_lens, 0, scale, out, lse, stream, kv8, k_scale, v_scale);
    Dims d;
    int rc = validate(q, k_pages, v_pages, block_table, seq_lens, out, lse, &d, kv8 ? DA_FP8_E4M3 : DA_BF16);
    if (rc != DA_OK) return rc;
    if (shared_prefix_tokens % PF_TOK != 0 || (int64_t)shared_prefix_tokens > d.max_pages * d.P) return DA_ERR_SHAPE;
    if (d.B * d.Hq > 0x7fffffffll / HEAD_DIM) return DA_ERR_UNSUPPORTED;
    const int64_t prefix_pages = (shared_prefix_tokens + d.P - 1) / d.P;
    const size_t half_copy = (size_t)prefix_pages * d.Hkv * d.P * HEAD_DIM * 2;   // bytes of the widened K (or V)
    if (kv8) {
        if (!prefix_scratch) return DA_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(prefix_scratch) & 255u) return DA_ERR_STRIDE_ALIGN;
        if (prefix_scratch_bytes < 2 * half_copy) return DA_ERR_WORKSPACE;
    }

    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    const int nblocks = grid_blocks_for(st);
    const int n_tail = tail_units_for(nblocks);
    const WsLayout lay = ws_layout(d.B, d.Hq, HEAD_DIM, d.max_pages, nblocks + n_tail);
    if (!st->ws || st->ws_bytes < lay.total) return DA_ERR_WORKSPACE;
    if (d.B == 0) return DA_OK;
    uint8_t *ws = static_cast<uint8_t *>(st->ws);

    // 1. attention of every query row over the shared prefix, on the tensor cores
    const int box_rows = d.P < PF_TOK ? (int)d.P : PF_TOK;
    da_tensor kw = *k_pages, vw = *v_pages;   // the pools the prefix kernel reads
    if (kv8) {
        // 1a. the prefix's E4M3 codes -> bf16 (exact), page i of the copy = prefix tokens [i P, (i+1) P)
        WidenParams wp;
        wp.k_pages = static_cast<const uint8_t *>(k_pages->data);
        wp.v_pages = static_cast<const uint8_t *>(v_pages->data);
        wp.k_sp = k_pages->stride[0]; wp.k_sh = k_pages->stride[1]; wp.k_st = k_pages->stride[2];
        wp.v_sp = v_pages->stride[0]; wp.v_sh = v_pages->stride[1]; wp.v_st = v_pages->stride[2];
        wp.block_table = static_cast<const int32_t *>(block_table->data);
        wp.bt_sb = 0;
        wp.seq_lens = nullptr;
        wp.sl_stride = 0;
        wp.pages_per_seq = (int32_t)prefix_pages;
        wp.seq0 = 0;
        wp.k_out = static_cast<__nv_bfloat16 *>(prefix_scratch);
        wp.v_out = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(prefix_scratch) + half_copy);
        wp.status = reinterpret_cast<int32_t *>(ws + lay.status);
        wp.Hkv = (int32_t)d.Hkv;
        wp.P = (int32_t)d.P;
        wp.num_pages = (int32_t)d.num_pages;
        widen_prefix_kernel<<<(unsigned)(prefix_pages * d.Hkv), 256, 0, stream>>>(wp);
        g_launches.fetch_add(1);
        DA_CUDA(cudaGetLastError());
        for (da_tensor *t : {&kw, &vw}) {
            t->dtype = DA_BF16;
            t->shape[0] = prefix_pages;
            t->stride[2] = HEAD_DIM;
            t->stride[1] = d.P * HEAD_DIM;
            t->stride[0] = d.Hkv * d.P * HEAD_DIM;
        }
        kw.data = wp.k_out;
        vw.data = wp.v_out;
    }
    rc = set_all_kernel_attrs(st);
    if (rc != DA_OK) return rc;
    CUtensorMap tm_k, tm_v;
    rc = get_tmap(&kw, box_rows, 1, &tm_k);
    if (rc != DA_OK) return rc;
    rc = get_tmap(&vw, box_rows, 2, &tm_v);   // (K: one plane per box; V: both)
    if (rc != DA_OK) return rc;
    PrefixParams pf;
    pf.k_scale = kv8 ? k_scale : nullptr;
    pf.v_scale = kv8 ? v_scale : nullptr;
    pf.identity_pages = kv8 ? (int32_t)prefix_pages : 0;
    pf.seq0 = 0;
    pf.q = static_cast<const __nv_bfloat16 *>(q->data);
    pf.q_sb = q->stride[0];
    pf.q_sq = 0;
    pf.q_sh = q->stride[1];
    pf.block_table = static_cast<const int32_t *>(block_table->data);
    pf.bt_sb = block_table->stride[0];
    pf.seq_lens = nullptr;
    pf.sl_stride = 0;
    pf.out = nullptr;
    pf.o_sb = pf.o_sq = pf.o_sh = 0;
    pf.lse = nullptr;
    pf.l_sb = pf.l_sq = pf.l_sh = 0;
    pf.out_bf16 = 0;
    pf.ext = 0;
    pf.Lq = 1;
    pf.max_pages = d.max_pages;
    pf.pre_o = reinterpret_cast<float *>(ws + lay.pre_o);
    pf.pre_lse = reinterpret_cast<float *>(ws + lay.pre_lse);
    pf.status = reinterpret_cast<int32_t *>(ws + lay.status);
    pf.B = (int32_t)d.B;
    pf.Hkv = (int32_t)d.Hkv;
    pf.G = (int32_t)d.G;
    pf.P = (int32_t)d.P;
    pf.box_rows = box_rows;
    pf.num_pages = kv8 ? (int32_t)prefix_pages : (int32_t)d.num_pages;
    pf.prefix_tiles = shared_prefix_tokens / PF_TOK;
    pf.row_tiles = (int32_t)((d.B * d.G + PF_ROWS - 1) / PF_ROWS);
    // (profile events, if set, bracket the prefix kernel in this entry point, not the partition kernel)
    cudaEvent_t ev_before = g_ev_before, ev_after = g_ev_after;
    const bool timed = ev_before && ev_after;
    // one block per SM at a time (its shared memory fills an SM): as many KV ranges as fit one wave
    const int64_t pairs = (int64_t)pf.row_tiles * pf.Hkv;
    int splits = (int)(st->sm_count / pairs);
    if (splits > kMaxPrefixSplits) splits = kMaxPrefixSplits;
    if (splits > pf.prefix_tiles) splits = pf.prefix_tiles;
    if (splits < 1) splits = 1;
    pf.splits = splits;
    pf.split0 = 0;
    pf.scale_log2 = scale * LOG2E;
    if (pairs * splits > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
    // Side by side or one after the other.  The prefix pass is bound by the tensor cores and the pass over the
    // sequences' own tokens by HBM, which a good half of the SMs saturate.  So, where the second is expected to
    // last at least as long as the first would on a third of the SMs, the two run side by side on two streams of
    // the library's own, forked from the caller's stream and joined to it before the final merge:
    //  * the prefix kernel at the highest priority, its KV ranges in two launches -- the first range alone
    //    (a block fills an SM's shared memory, so (row tiles x KV heads) SMs are taken and the others stay
    //    free), then the remaining ranges, whose blocks follow on the SMs the first launch leaves;
    //  * plan / partition / merge at the lowest priority.  The partition blocks find the other SMs; those that
    //    find no room are given no range of their own and join, on tickets, once no prefix block is waiting
    //    for an SM.  When the sequences' own parts turn out short, the waiting prefix blocks spread over the
    //    SMs that the partition blocks leave (priority decides who gets a free SM).
    // The partition kernel is launched to start only after the plan kernel has ended, microseconds after the
    // first prefix launch could start; should its blocks be placed first all the same, they take every SM and
    // the prefix kernel runs after them: slower, still correct.  The host cannot see the lengths: it takes
    // half of what the block-table rows can hold beyond the prefix as the typical sequence's own part.
    int first_splits = 0;   // KV ranges of the first prefix launch (0: one launch, passes one after the other)
    if (g_opt_cascade_overlap && !timed && g_opt_grid_blocks <= 0 && splits >= 2) {
        int64_t sa = g_opt_cascade_prefix_sms > 0 ? g_opt_cascade_prefix_sms / pairs : (splits + 1) / 3;
        sa = std::max<int64_t>(1, std::min<int64_t>(sa, splits - 1));
        const int64_t x = pairs * sa;
        const double flops = 4.0 * PF_ROWS * (double)pairs * shared_prefix_tokens * HEAD_DIM;
        const double t_prefix = flops / ((double)x * 4.4e12);                      // seconds, on x SMs
        const double own = 0.5 * (double)(d.max_pages * d.P - shared_prefix_tokens);
        const double t_own = (double)d.B * d.Hkv * own * (kv8 ? 256.0 : 512.0) / 7.0e12;
        if (x <= st->sm_count / 2 && (g_opt_cascade_overlap == 2 || t_own >= t_prefix) && ensure_side_stream(st))
            first_splits = (int)sa;
    }
    const int prefix_sms = first_splits ? (int)(pairs * first_splits) : 0;
    cudaStream_t pre_stream = stream, own_stream = stream;
    if (first_splits) {
        DA_CUDA(cudaEventRecord(st->ev_fork, stream));
        DA_CUDA(cudaStreamWaitEvent(st->side_hi, st->ev_fork, 0));
        DA_CUDA(cudaStreamWaitEvent(st->side_lo, st->ev_fork, 0));
        pre_stream = st->side_hi;
        own_stream = st->side_lo;
    }
    if (timed) DA_CUDA(cudaEventRecord(ev_before, stream));
    {
        const int n1 = first_splits ? first_splits : splits;
        prefix_kernel<<<(unsigned)(pairs * n1), PF_THREADS, PF_SMEM_BYTES, pre_stream>>>(tm_k, tm_v, pf);
        g_launches.fetch_add(1);
        cudaError_t e = cudaGetLastError();
        if (e == cudaSuccess && n1 < splits) {
            pf.split0 = n1;
            prefix_kernel<<<(unsigned)(pairs * (splits - n1)), PF_THREADS, PF_SMEM_BYTES, pre_stream>>>(tm_k, tm_v, pf);
            g_launches.fetch_add(1);
            e = cudaGetLastError();
        }
        if (first_splits) {   // (also after a failed launch: the caller's stream must not be left forked)
            cudaError_t e1 = cudaEventRecord(st->ev_join_hi, st->side_hi);
            if (e1 == cudaSuccess) e1 = cudaStreamWaitEvent(stream, st->ev_join_hi, 0);
            if (e == cudaSuccess) e = e1;
        }
        if (e != cudaSuccess) {
            if (first_splits && cudaEventRecord(st->ev_join_lo, st->side_lo) == cudaSuccess)
                cudaStreamWaitEvent(stream, st->ev_join_lo, 0);
            return cuda_fail(e);
        }
    }
    if (timed) DA_CUDA(cudaEventRecord(ev_after, stream));

    // 2. attention over the tokens past the prefix, per sequence, into fp32 scratch
    da_tensor so, sl;
    so.data = ws + lay.suf_o;
    so.dtype = DA_F32;
    so.ndim = 3;
    so.shape[0] = d.B; so.shape[1] = d.Hq; so.shape[2] = HEAD_DIM; so.shape[3] = 0;
    so.stride[0] = d.Hq * HEAD_DIM; so.stride[1] = HEAD_DIM; so.stride[2] = 1; so.stride[3] = 0;
    sl.data = ws + lay.suf_lse;
    sl.dtype = DA_F32;
    sl.ndim = 2;
    sl.shape[0] = d.B; sl.shape[1] = d.Hq; sl.shape[2] = sl.shape[3] = 0;
    sl.stride[0] = d.Hq; sl.stride[1] = 1; sl.stride[2] = sl.stride[3] = 0;
    g_ev_before = g_ev_after = nullptr;
    rc = launch_path(st, d, ws, lay, nblocks, n_tail, q, k_pages, v_pages, block_table, seq_lens, 0, scale, &so, &sl, own_stream,
                     shared_prefix_tokens, kv8, k_scale, v_scale, 1, 0, 0, 0, prefix_sms ? 2 * prefix_sms : 0);
    g_ev_before = ev_before;
    g_ev_after = ev_after;
    if (first_splits) {   // (also after a failed launch: the caller's stream must not be left forked)
        cudaError_t e1 = cudaEventRecord(st->ev_join_lo, st->side_lo);
        if (e1 == cudaSuccess) e1 = cudaStreamWaitEvent(stream, st->ev_join_lo, 0);
        if (rc == DA_OK) DA_CUDA(e1);
    }
    if (rc != DA_OK) return rc;

    // 3. fold prefix partials and suffix result
    CascadeMergeParams cm;
    cm.pre_o = pf.pre_o;
    cm.pre_lse = pf.pre_lse;
    cm.suf_o = reinterpret_cast<const float *>(ws + lay.suf_o);
    cm.suf_lse = reinterpret_cast<const float *>(ws + lay.suf_lse);
    cm.seq_info = reinterpret_cast<const int4 *>(ws + lay.seq_info);
    cm.out = out->data;
    cm.o_sb = out->stride[0];
    cm.o_sq = 0;
    cm.o_sh = out->stride[1];
    cm.lse = lse ? static_cast<float *>(lse->data) : nullptr;
    cm.l_sb = lse ? lse->stride[0] : 0;
    cm.l_sq = 0;
    cm.l_sh = lse ? lse->stride[1] : 0;
    cm.B = (int32_t)d.B;
    cm.Lq = 1;
    cm.Hq = (int32_t)d.Hq;
    cm.splits = splits;
    cm.out_bf16 = out->dtype == DA_BF16;
    cascade_merge_kernel<<<(unsigned)((d.B * d.Hq + 7) / 8), 256, 0, stream>>>(cm);
    g_launches.fetch_add(1);
    DA_CUDA(cudaGetLastError());
    return DA_OK;
}
}  // namespace

extern "C" {

int decode_attn_cascade(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                        const da_tensor *block_table, const da_tensor *seq_lens, int32_t shared_prefix_tokens, float scale,
                        da_tensor *out, da_tensor *lse, void *stream)
{
    return run_cascade(q, k_pages, v_pages, block_table, seq_lens, shared_prefix_tokens, scale, out, lse,
                       static_cast<cudaStream_t>(stream), false, nullptr, nullptr, nullptr, 0);
}

int decode_attn_fp8kv_cascade(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const float *k_scale,
                              const float *v_scale, const da_tensor *block_table, const da_tensor *seq_lens,
                              int32_t shared_prefix_tokens, float scale, da_tensor *out, da_tensor *lse,
                              void *prefix_scratch, size_t prefix_scratch_bytes, void *stream)
{
    return run_cascade(q, k_pages, v_pages, block_table, seq_lens, shared_prefix_tokens, scale, out, lse,
                       static_cast<cudaStream_t>(stream), true, k_scale, v_scale, prefix_scratch, prefix_scratch_bytes);
}

size_t decode_attn_fp8kv_cascade_scratch_bytes(int32_t shared_prefix_tokens, int32_t Hkv, int32_t P)
{
    if (shared_prefix_tokens <= 0 || Hkv <= 0 || P <= 0) return 0;
    const size_t pages = ((size_t)shared_prefix_tokens + P - 1) / P;
    return 2 * pages * Hkv * P * HEAD_DIM * 2;
}

int decode_attn_append(const da_tensor *k_new, const da_tensor *v_new, da_tensor *k_pages, da_tensor *v_pages,
                       const da_tensor *block_table, const da_tensor *seq_lens, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!k_new || !v_new || !k_pages || !v_pages || !block_table || !seq_lens) return DA_ERR_NULL;
    if (!k_new->data || !v_new->data || !block_table->data || !seq_lens->data) return DA_ERR_NULL;
    int rc = check_pool(k_pages);
    if (rc != DA_OK) return rc;
    rc = check_pool(v_pages);
    if (rc != DA_OK) return rc;
    for (int i = 0; i < 4; ++i)
        if (k_pages->shape[i] != v_pages->shape[i]) return DA_ERR_SHAPE;
    if (k_new->dtype != DA_BF16 || v_new->dtype != DA_BF16 || block_table->dtype != DA_I32 || seq_lens->dtype != DA_I32)
        return DA_ERR_DTYPE;
    if (k_new->ndim != 3 || v_new->ndim != 3 || block_table->ndim != 2 || seq_lens->ndim != 1) return DA_ERR_SHAPE;
    const int64_t B = k_new->shape[0], Hkv = k_pages->shape[1], P = k_pages->shape[2];
    if (k_new->shape[1] != Hkv || k_new->shape[2] != HEAD_DIM) return DA_ERR_SHAPE;
    for (int i = 0; i < 3; ++i)
        if (v_new->shape[i] != k_new->shape[i]) return DA_ERR_SHAPE;
    if (block_table->shape[0] != B || seq_lens->shape[0] != B || block_table->shape[1] <= 0) return DA_ERR_SHAPE;
    if (B < 0 || B > (1 << 24) || k_pages->shape[0] > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
    if (P != 16 && P != 32 && P != 64 && P != 128) return DA_ERR_UNSUPPORTED;
    const da_tensor *nw[2] = {k_new, v_new};
    for (const da_tensor *t : nw) {
        if (t->stride[2] != 1 || !aligned16(t->data) || (t->stride[0] * 2) % 16 != 0 || (t->stride[1] * 2) % 16 != 0)
            return DA_ERR_STRIDE_ALIGN;
    }
    if (block_table->stride[1] != 1) return DA_ERR_STRIDE_ALIGN;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    if (!st->ws || st->ws_bytes < 256) return DA_ERR_WORKSPACE;   // the status record lives there
    if (B == 0) return DA_OK;
    AppendParams ap;
    ap.k_new = static_cast<const __nv_bfloat16 *>(k_new->data);
    ap.v_new = static_cast<const __nv_bfloat16 *>(v_new->data);
    ap.kn_sb = k_new->stride[0];
    ap.kn_sh = k_new->stride[1];
    ap.vn_sb = v_new->stride[0];
    ap.vn_sh = v_new->stride[1];
    ap.k_pages = static_cast<__nv_bfloat16 *>(k_pages->data);
    ap.v_pages = static_cast<__nv_bfloat16 *>(v_pages->data);
    ap.k_sp = k_pages->stride[0];
    ap.k_sh = k_pages->stride[1];
    ap.k_st = k_pages->stride[2];
    ap.v_sp = v_pages->stride[0];
    ap.v_sh = v_pages->stride[1];
    ap.v_st = v_pages->stride[2];
    ap.block_table = static_cast<const int32_t *>(block_table->data);
    ap.bt_sb = block_table->stride[0];
    ap.seq_lens = static_cast<const int32_t *>(seq_lens->data);
    ap.sl_stride = seq_lens->stride[0];
    ap.status = reinterpret_cast<int32_t *>(st->ws);
    ap.B = (int32_t)B;
    ap.Hkv = (int32_t)Hkv;
    ap.P = (int32_t)P;
    ap.num_pages = (int32_t)k_pages->shape[0];
    ap.max_pages = block_table->shape[1];
    append_kernel<<<(unsigned)B, 256, 0, stream>>>(ap);
    g_launches.fetch_add(1);
    DA_CUDA(cudaGetLastError());
    return DA_OK;
}

int decode_attn_append_fp8kv(const da_tensor *k_new, const da_tensor *v_new, da_tensor *k_pages, da_tensor *v_pages,
                             const float *k_scale, const float *v_scale, const da_tensor *block_table,
                             const da_tensor *seq_lens, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!k_new || !v_new || !k_pages || !v_pages || !block_table || !seq_lens) return DA_ERR_NULL;
    if (!k_new->data || !v_new->data || !block_table->data || !seq_lens->data) return DA_ERR_NULL;
    int rc = check_pool(k_pages, DA_FP8_E4M3);
    if (rc != DA_OK) return rc;
    rc = check_pool(v_pages, DA_FP8_E4M3);
    if (rc != DA_OK) return rc;
    for (int i = 0; i < 4; ++i)
        if (k_pages->shape[i] != v_pages->shape[i]) return DA_ERR_SHAPE;
    if (k_new->dtype != DA_BF16 || v_new->dtype != DA_BF16 || block_table->dtype != DA_I32 || seq_lens->dtype != DA_I32)
        return DA_ERR_DTYPE;
    if (k_new->ndim != 3 || v_new->ndim != 3 || block_table->ndim != 2 || seq_lens->ndim != 1) return DA_ERR_SHAPE;
    const int64_t B = k_new->shape[0], Hkv = k_pages->shape[1], P = k_pages->shape[2];
    if (k_new->shape[1] != Hkv || k_new->shape[2] != HEAD_DIM) return DA_ERR_SHAPE;
    for (int i = 0; i < 3; ++i)
        if (v_new->shape[i] != k_new->shape[i]) return DA_ERR_SHAPE;
    if (block_table->shape[0] != B || seq_lens->shape[0] != B || block_table->shape[1] <= 0) return DA_ERR_SHAPE;
    if (B < 0 || B > (1 << 24) || k_pages->shape[0] > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
    if (P != 16 && P != 32 && P != 64 && P != 128) return DA_ERR_UNSUPPORTED;
    const da_tensor *nw[2] = {k_new, v_new};
    for (const da_tensor *t : nw) {
        if (t->stride[2] != 1 || !aligned16(t->data) || (t->stride[0] * 2) % 16 != 0 || (t->stride[1] * 2) % 16 != 0)
            return DA_ERR_STRIDE_ALIGN;
    }
    if (block_table->stride[1] != 1) return DA_ERR_STRIDE_ALIGN;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    if (!st->ws || st->ws_bytes < 256) return DA_ERR_WORKSPACE;   // the status record lives there
    if (B == 0) return DA_OK;
    Append8Params ap;
    ap.k_new = static_cast<const __nv_bfloat16 *>(k_new->data);
    ap.v_new = static_cast<const __nv_bfloat16 *>(v_new->data);
    ap.kn_sb = k_new->stride[0];
    ap.kn_sh = k_new->stride[1];
    ap.vn_sb = v_new->stride[0];
    ap.vn_sh = v_new->stride[1];
    ap.k_pages = static_cast<uint8_t *>(k_pages->data);
    ap.v_pages = static_cast<uint8_t *>(v_pages->data);
    ap.k_sp = k_pages->stride[0];
    ap.k_sh = k_pages->stride[1];
    ap.k_st = k_pages->stride[2];
    ap.v_sp = v_pages->stride[0];
    ap.v_sh = v_pages->stride[1];
    ap.v_st = v_pages->stride[2];
    ap.k_scale = k_scale;
    ap.v_scale = v_scale;
    ap.block_table = static_cast<const int32_t *>(block_table->data);
    ap.bt_sb = block_table->stride[0];
    ap.seq_lens = static_cast<const int32_t *>(seq_lens->data);
    ap.sl_stride = seq_lens->stride[0];
    ap.status = reinterpret_cast<int32_t *>(st->ws);
    ap.B = (int32_t)B;
    ap.Hkv = (int32_t)Hkv;
    ap.P = (int32_t)P;
    ap.num_pages = (int32_t)k_pages->shape[0];
    ap.max_pages = block_table->shape[1];
    append8_kernel<<<(unsigned)B, 256, 0, stream>>>(ap);
    g_launches.fetch_add(1);
    DA_CUDA(cudaGetLastError());
    return DA_OK;
}

}  // extern "C"

namespace {
// decode_attn_extend / decode_attn_fp8kv_extend
int run_extend(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const da_tensor *block_table,
               const da_tensor *seq_lens, float scale, da_tensor *out, da_tensor *lse, cudaStream_t stream, bool kv8,
               const float *k_scale, const float *v_scale, void *wide_scratch = nullptr, size_t wide_scratch_bytes = 0,
               bool has_scratch_arg = false, int32_t seq0 = 0)
{
    if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !out) return DA_ERR_NULL;
    if (!q->data || !block_table->data || !seq_lens->data || !out->data || (lse && !lse->data)) return DA_ERR_NULL;
    if (q->dtype != DA_BF16 || block_table->dtype != DA_I32 || seq_lens->dtype != DA_I32) return DA_ERR_DTYPE;
    if (out->dtype != DA_F32 && out->dtype != DA_BF16) return DA_ERR_DTYPE;
    if (lse && lse->dtype != DA_F32) return DA_ERR_DTYPE;
    if (q->ndim != 4 || out->ndim != 4 || block_table->ndim != 2 || seq_lens->ndim != 1 || (lse && lse->ndim != 3))
        return DA_ERR_SHAPE;
    int rc = check_pool(k_pages, kv8 ? DA_FP8_E4M3 : DA_BF16);
    if (rc != DA_OK) return rc;
    rc = check_pool(v_pages, kv8 ? DA_FP8_E4M3 : DA_BF16);
    if (rc != DA_OK) return rc;
    for (int i = 0; i < 4; ++i)
        if (k_pages->shape[i] != v_pages->shape[i]) return DA_ERR_SHAPE;
    const int64_t B = q->shape[0], Lq = q->shape[1], Hq = q->shape[2];
    const int64_t Hkv = k_pages->shape[1], P = k_pages->shape[2], max_pages = block_table->shape[1];
    if (q->shape[3] != HEAD_DIM) return DA_ERR_UNSUPPORTED;
    if (Hkv <= 0 || k_pages->shape[0] <= 0) return DA_ERR_SHAPE;   // (before Hkv divides anything)
    if (B < 0 || Lq <= 0 || Hq <= 0 || max_pages <= 0 || Hq % Hkv != 0) return DA_ERR_SHAPE;
    if (P != 16 && P != 32 && P != 64 && P != 128) return DA_ERR_UNSUPPORTED;
    if (B > (1 << 20) || Lq > (1 << 20) || k_pages->shape[0] > 0x7fffffffll || max_pages * P > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
    for (int i = 0; i < 4; ++i)
        if (out->shape[i] != q->shape[i]) return DA_ERR_SHAPE;
    if (lse && (lse->shape[0] != B || lse->shape[1] != Lq || lse->shape[2] != Hq)) return DA_ERR_SHAPE;
    if (block_table->shape[0] != B || seq_lens->shape[0] != B) return DA_ERR_SHAPE;
    if (q->stride[3] != 1 || out->stride[3] != 1 || block_table->stride[1] != 1) return DA_ERR_STRIDE_ALIGN;
    if ((q->stride[0] | q->stride[1] | q->stride[2]) & 1 || (reinterpret_cast<uintptr_t>(q->data) & 3u)) return DA_ERR_STRIDE_ALIGN;
    const int64_t G = Hq / Hkv;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    const int nblocks = grid_blocks_for(st);
    const WsLayout lay = ws_layout(B, Hq, HEAD_DIM, max_pages, nblocks + tail_units_for(nblocks));
    if (!st->ws || st->ws_bytes < lay.total) return DA_ERR_WORKSPACE;
    if (B == 0) return DA_OK;
    uint8_t *ws = static_cast<uint8_t *>(st->ws);
    rc = set_all_kernel_attrs(st);
    if (rc != DA_OK) return rc;
    if ((Lq * G <= g_opt_extend_stream_rows || kv8) && Lq * G <= kMaxStreamRows) {
        // A few new tokens (speculated tokens, short appends): their Lq * G query rows per KV head ride
        // through the streaming kernels as one wider group, K and V crossing HBM once as in decode_attn();
        // the tensor-core kernel below would fill only Lq * G of its 128 rows.
        Dims d;
        d.B = B; d.Hq = Hq; d.Hkv = Hkv; d.G = G; d.P = P; d.num_pages = k_pages->shape[0]; d.max_pages = max_pages;
        da_tensor q3 = *q, o3 = *out, l3;
        q3.ndim = 3; q3.shape[1] = Hq; q3.shape[2] = HEAD_DIM; q3.stride[1] = q->stride[2]; q3.stride[2] = 1;
        o3.ndim = 3; o3.shape[1] = Hq; o3.shape[2] = HEAD_DIM; o3.stride[1] = out->stride[2]; o3.stride[2] = 1;
        if (lse) {
            l3 = *lse;
            l3.ndim = 2; l3.shape[1] = Hq; l3.stride[1] = lse->stride[2];
        }
        const int n_tail = tail_units_for(nblocks);
        return launch_path(st, d, ws, lay, nblocks, n_tail, &q3, k_pages, v_pages, block_table, seq_lens, 0, scale, &o3,
                           lse ? &l3 : nullptr, stream, 0, kv8, k_scale, v_scale, (int)Lq, q->stride[1], out->stride[1],
                           lse ? lse->stride[1] : 0);
    }
    // The tensor-core kernel reads a bf16 cache.  Over the 8-bit cache, the pages every sequence attends are
    // first widened, exactly, into a bf16 copy in the caller's scratch -- page i of sequence b becomes page
    // b * max_pages + i of the copy, so the kernel needs no block table -- and the per-KV-head factors enter in
    // the kernel (k_scale with the score scale, v_scale with the result), as in the cascade.
    if (kv8 && !has_scratch_arg)
        return DA_ERR_UNSUPPORTED;
    const int box_rows = P < PF_TOK ? (int)P : PF_TOK;
    da_tensor kw = *k_pages, vw = *v_pages;   // the pools the kernel reads
    if (kv8) {
        const int64_t copy_pages = B * max_pages;
        if (copy_pages > 0x7fffffffll || copy_pages * Hkv > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
        const size_t half_copy = (size_t)copy_pages * Hkv * P * HEAD_DIM * 2;   // bytes of the widened K (or V)
        if (!wide_scratch) return DA_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(wide_scratch) & 255u) return DA_ERR_STRIDE_ALIGN;
        if (wide_scratch_bytes < 2 * half_copy) return DA_ERR_WORKSPACE;
        WidenParams wp;
        wp.k_pages = static_cast<const uint8_t *>(k_pages->data);
        wp.v_pages = static_cast<const uint8_t *>(v_pages->data);
        wp.k_sp = k_pages->stride[0]; wp.k_sh = k_pages->stride[1]; wp.k_st = k_pages->stride[2];
        wp.v_sp = v_pages->stride[0]; wp.v_sh = v_pages->stride[1]; wp.v_st = v_pages->stride[2];
        wp.block_table = static_cast<const int32_t *>(block_table->data);
        wp.bt_sb = block_table->stride[0];
        wp.seq_lens = static_cast<const int32_t *>(seq_lens->data);
        wp.sl_stride = seq_lens->stride[0];
        wp.pages_per_seq = (int32_t)max_pages;
        wp.seq0 = seq0;
        wp.k_out = static_cast<__nv_bfloat16 *>(wide_scratch);
        wp.v_out = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(wide_scratch) + half_copy);
        wp.status = reinterpret_cast<int32_t *>(ws + lay.status);
        wp.Hkv = (int32_t)Hkv;
        wp.P = (int32_t)P;
        wp.num_pages = (int32_t)k_pages->shape[0];
        widen_prefix_kernel<<<(unsigned)(copy_pages * Hkv), 256, 0, stream>>>(wp);
        g_launches.fetch_add(1);
        DA_CUDA(cudaGetLastError());
        for (da_tensor *t : {&kw, &vw}) {
            t->dtype = DA_BF16;
            t->shape[0] = copy_pages;
            t->stride[2] = HEAD_DIM;
            t->stride[1] = P * HEAD_DIM;
            t->stride[0] = Hkv * P * HEAD_DIM;
        }
        kw.data = wp.k_out;
        vw.data = wp.v_out;
    }
    CUtensorMap tm_k, tm_v;
    rc = get_tmap(&kw, box_rows, 1, &tm_k);
    if (rc != DA_OK) return rc;
    rc = get_tmap(&vw, box_rows, 2, &tm_v);   // (K: one plane per box; V: both)
    if (rc != DA_OK) return rc;

    PrefixParams pf;
    pf.k_scale = kv8 ? k_scale : nullptr;
    pf.v_scale = kv8 ? v_scale : nullptr;
    pf.identity_pages = kv8 ? (int32_t)max_pages : 0;
    pf.seq0 = seq0;
    pf.q = static_cast<const __nv_bfloat16 *>(q->data);
    pf.q_sb = q->stride[0];
    pf.q_sq = q->stride[1];
    pf.q_sh = q->stride[2];
    pf.block_table = static_cast<const int32_t *>(block_table->data);
    pf.bt_sb = block_table->stride[0];
    pf.seq_lens = static_cast<const int32_t *>(seq_lens->data);
    pf.sl_stride = seq_lens->stride[0];
    pf.pre_o = reinterpret_cast<float *>(ws + lay.pre_o);
    pf.pre_lse = reinterpret_cast<float *>(ws + lay.pre_lse);
    pf.out = out->data;
    pf.o_sb = out->stride[0];
    pf.o_sq = out->stride[1];
    pf.o_sh = out->stride[2];
    pf.lse = lse ? static_cast<float *>(lse->data) : nullptr;
    pf.l_sb = lse ? lse->stride[0] : 0;
    pf.l_sq = lse ? lse->stride[1] : 0;
    pf.l_sh = lse ? lse->stride[2] : 0;
    pf.status = reinterpret_cast<int32_t *>(ws + lay.status);
    pf.B = (int32_t)B;
    pf.Hkv = (int32_t)Hkv;
    pf.G = (int32_t)G;
    pf.P = (int32_t)P;
    pf.box_rows = box_rows;
    pf.num_pages = (int32_t)kw.shape[0];
    pf.out_bf16 = out->dtype == DA_BF16;
    pf.ext = 1;
    pf.Lq = (int32_t)Lq;
    pf.max_pages = max_pages;
    pf.prefix_tiles = 0;
    pf.row_tiles = (int32_t)((Lq * G + PF_ROWS - 1) / PF_ROWS);
    // KV ranges: as many as fill one wave, if their partials fit the scratch sized for the cascade
    // (kMaxPrefixSplits x B x Hq rows); long query blocks have enough thread blocks anyway.
    const long long base = (long long)B * Hkv * pf.row_tiles;
    int splits = (int)(st->sm_count / base);
    if (splits > kMaxPrefixSplits) splits = kMaxPrefixSplits;
    if ((long long)splits * Lq > kMaxPrefixSplits) splits = (int)(kMaxPrefixSplits / Lq);
    if (splits < 1) splits = 1;
    pf.splits = splits;
    pf.split0 = 0;
    pf.scale_log2 = scale * LOG2E;
    const long long grid = base * splits;
    if (grid > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
    const bool timed = g_ev_before && g_ev_after;
    if (timed) DA_CUDA(cudaEventRecord(g_ev_before, stream));
    prefix_kernel<<<(unsigned)grid, PF_THREADS, PF_SMEM_BYTES, stream>>>(tm_k, tm_v, pf);
    g_launches.fetch_add(1);
    DA_CUDA(cudaGetLastError());
    if (timed) DA_CUDA(cudaEventRecord(g_ev_after, stream));
    if (splits > 1) {
        CascadeMergeParams cm;
        cm.pre_o = pf.pre_o;
        cm.pre_lse = pf.pre_lse;
        cm.suf_o = nullptr;
        cm.suf_lse = nullptr;
        cm.seq_info = nullptr;
        cm.out = out->data;
        cm.o_sb = pf.o_sb;
        cm.o_sq = pf.o_sq;
        cm.o_sh = pf.o_sh;
        cm.lse = pf.lse;
        cm.l_sb = pf.l_sb;
        cm.l_sq = pf.l_sq;
        cm.l_sh = pf.l_sh;
        cm.B = (int32_t)B;
        cm.Lq = (int32_t)Lq;
        cm.Hq = (int32_t)Hq;
        cm.splits = splits;
        cm.out_bf16 = pf.out_bf16;
        cascade_merge_kernel<<<(unsigned)((B * Lq * Hq + 7) / 8), 256, 0, stream>>>(cm);
        g_launches.fetch_add(1);
        DA_CUDA(cudaGetLastError());
    }
    return DA_OK;
}
}  // namespace

extern "C" {

int decode_attn_extend(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const da_tensor *block_table,
                       const da_tensor *seq_lens, float scale, da_tensor *out, da_tensor *lse, void *stream)
{
    return run_extend(q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, static_cast<cudaStream_t>(stream), false,
                      nullptr, nullptr);
}

int decode_attn_fp8kv_extend(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const float *k_scale,
                             const float *v_scale, const da_tensor *block_table, const da_tensor *seq_lens, float scale,
                             da_tensor *out, da_tensor *lse, void *stream)
{
    return run_extend(q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, static_cast<cudaStream_t>(stream), true,
                      k_scale, v_scale);
}

int decode_attn_fp8kv_extend_wide(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages, const float *k_scale,
                                  const float *v_scale, const da_tensor *block_table, const da_tensor *seq_lens, float scale,
                                  da_tensor *out, da_tensor *lse, void *scratch, size_t scratch_bytes, void *stream)
{
    // A scratch buffer that holds the widened pages of some, not all, of the sequences: the call is made in
    // groups of as many sequences as fit, one after the other on the stream (the next group's copy follows the
    // kernel that read the last one's).  Everything else about the arguments is checked by the calls themselves.
    if (q && q->ndim == 4 && k_pages && k_pages->ndim == 4 && block_table && block_table->ndim == 2 && seq_lens &&
        seq_lens->ndim == 1 && out && out->ndim == 4 && (!lse || lse->ndim == 3) && scratch && q->data && out->data &&
        block_table->data && seq_lens->data && (!lse || lse->data)) {
        const int64_t B = q->shape[0], Lq = q->shape[1], Hq = q->shape[2];
        const int64_t Hkv = k_pages->shape[1], P = k_pages->shape[2], max_pages = block_table->shape[1];
        if (B > 1 && Lq > 0 && Hkv > 0 && Hq > 0 && Hq % Hkv == 0 && P > 0 && P <= 128 && max_pages > 0 &&
            max_pages <= 0x7fffffffll && Lq * (Hq / Hkv) > kMaxStreamRows && out->shape[0] == B &&
            block_table->shape[0] == B && seq_lens->shape[0] == B && (!lse || lse->shape[0] == B)) {
            const size_t per_seq = (size_t)max_pages * (size_t)Hkv * (size_t)P * HEAD_DIM * 2 * 2;
            if (scratch_bytes >= per_seq && scratch_bytes / per_seq < (size_t)B) {
                const int64_t group = (int64_t)(scratch_bytes / per_seq);
                auto rows = [](const da_tensor *t, int64_t b0, int64_t n, int64_t item) {
                    da_tensor v = *t;
                    v.data = static_cast<uint8_t *>(t->data) + b0 * t->stride[0] * item;
                    v.shape[0] = n;
                    return v;
                };
                for (int64_t b0 = 0; b0 < B; b0 += group) {
                    const int64_t n = std::min<int64_t>(group, B - b0);
                    da_tensor qg = rows(q, b0, n, 2), btg = rows(block_table, b0, n, 4), slg = rows(seq_lens, b0, n, 4);
                    da_tensor og = rows(out, b0, n, out->dtype == DA_BF16 ? 2 : 4), lg;
                    if (lse) lg = rows(lse, b0, n, 4);
                    const int rc = run_extend(&qg, k_pages, v_pages, &btg, &slg, scale, &og, lse ? &lg : nullptr,
                                              static_cast<cudaStream_t>(stream), true, k_scale, v_scale, scratch,
                                              scratch_bytes, true, (int32_t)b0);
                    if (rc != DA_OK) return rc;
                }
                return DA_OK;
            }
        }
    }
    return run_extend(q, k_pages, v_pages, block_table, seq_lens, scale, out, lse, static_cast<cudaStream_t>(stream), true,
                      k_scale, v_scale, scratch, scratch_bytes, true);
}

size_t decode_attn_fp8kv_extend_wide_scratch_bytes(int32_t B, int64_t max_pages, int32_t Hkv, int32_t P)
{
    if (B <= 0 || max_pages <= 0 || Hkv <= 0 || P <= 0) return 0;
    return (size_t)B * (size_t)max_pages * (size_t)Hkv * (size_t)P * HEAD_DIM * 2 * 2;
}

}  // extern "C"

namespace {
// decode_attn_host_io / decode_attn_fp8kv_host_io
int run_host_io(const da_tensor *q_host, const da_tensor *k_pages, const da_tensor *v_pages,
                const da_tensor *block_table_host, const da_tensor *seq_lens_host, int32_t window, float scale,
                da_tensor *out_host, da_tensor *lse_host, cudaStream_t stream, bool kv8, const float *k_scale,
                const float *v_scale)
{
    Dims d;
    int rc = validate(q_host, k_pages, v_pages, block_table_host, seq_lens_host, out_host, lse_host, &d,
                      kv8 ? DA_FP8_E4M3 : DA_BF16);
    if (rc != DA_OK) return rc;
    if (!contiguous(q_host) || !contiguous(block_table_host) || !contiguous(seq_lens_host) || !contiguous(out_host) ||
        (lse_host && !contiguous(lse_host)))
        return DA_ERR_STRIDE_ALIGN;
    uint8_t *ws;
    WsLayout lay;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        int dev;
        DeviceState *st;
        rc = current_device(&dev, &st);
        if (rc != DA_OK) return rc;
        const int nb = grid_blocks_for(st);
        lay = ws_layout(d.B, d.Hq, HEAD_DIM, d.max_pages, nb + tail_units_for(nb));
        if (!st->ws || st->ws_bytes < lay.total) return DA_ERR_WORKSPACE;
        ws = static_cast<uint8_t *>(st->ws);
    }
    if (d.B == 0) return DA_OK;
    const size_t out_item = out_host->dtype == DA_BF16 ? 2 : 4;
    // Inputs: from pinned, mapped host buffers one kernel gathers all three into the staging area;
    // from other memory, three copies.
    {
        const size_t nb[3] = {(size_t)d.B * d.Hq * HEAD_DIM * 2, (size_t)d.B * d.max_pages * 4, (size_t)d.B * 4};
        const void *hp[3] = {q_host->data, block_table_host->data, seq_lens_host->data};
        const size_t at[3] = {lay.stg_q, lay.stg_bt, lay.stg_sl};
        StageParams sp;
        bool all_mapped = true;
        for (int r = 0; r < 3; ++r) {
            sp.src[r] = static_cast<const uint8_t *>(mapped_device_pointer(hp[r]));
            sp.dst[r] = ws + at[r];
            sp.bytes[r] = nb[r];
            all_mapped = all_mapped && sp.src[r] != nullptr && (reinterpret_cast<uintptr_t>(sp.src[r]) & 3u) == 0;
        }
        if (all_mapped) {
            int dev = 0, sms = 148;
            DA_CUDA(cudaGetDevice(&dev));
            if (dev >= 0 && dev < kMaxDevices && g_dev[dev].sm_count > 0) sms = g_dev[dev].sm_count;
            stage_inputs_kernel<<<(unsigned)(2 * sms), 256, 0, stream>>>(sp);
            g_launches.fetch_add(1);
            DA_CUDA(cudaGetLastError());
        } else {
            for (int r = 0; r < 3; ++r)
                DA_CUDA(cudaMemcpyAsync(ws + at[r], hp[r], nb[r], cudaMemcpyHostToDevice, stream));
        }
    }
    da_tensor qd = *q_host, btd = *block_table_host, sld = *seq_lens_host, od = *out_host, ld;
    qd.data = ws + lay.stg_q;
    btd.data = ws + lay.stg_bt;
    sld.data = ws + lay.stg_sl;
    // Results: when the host buffers are pinned and mapped into the device's address space the kernels
    // write them directly (the stores travel while the rest of the batch is still streaming, and no
    // copy is queued after the kernels); otherwise they go to staging and are copied back.
    void *out_dev = mapped_device_pointer(out_host->data);
    void *lse_dev = lse_host ? mapped_device_pointer(lse_host->data) : nullptr;
    const bool direct = out_dev && (!lse_host || lse_dev);
    od.data = direct ? out_dev : ws + lay.stg_out;
    if (lse_host) {
        ld = *lse_host;
        ld.data = direct ? lse_dev : ws + lay.stg_lse;
    }
    t_results_to_host = direct;   // results written across PCIe: spread them over the kernel's run (option "fold_pairs")
    rc = run(&qd, k_pages, v_pages, &btd, &sld, window, scale, &od, lse_host ? &ld : nullptr, stream, kv8, k_scale, v_scale);
    t_results_to_host = false;
    if (rc != DA_OK) return rc;
    if (!direct) {
        DA_CUDA(cudaMemcpyAsync(out_host->data, ws + lay.stg_out, (size_t)d.B * d.Hq * HEAD_DIM * out_item, cudaMemcpyDeviceToHost, stream));
        if (lse_host)
            DA_CUDA(cudaMemcpyAsync(lse_host->data, ws + lay.stg_lse, (size_t)d.B * d.Hq * 4, cudaMemcpyDeviceToHost, stream));
    }
    return DA_OK;
}
}  // namespace

extern "C" {

int decode_attn_host_io(const da_tensor *q_host, const da_tensor *k_pages, const da_tensor *v_pages,
                        const da_tensor *block_table_host, const da_tensor *seq_lens_host, int32_t window, float scale,
                        da_tensor *out_host, da_tensor *lse_host, void *stream)
{
    return run_host_io(q_host, k_pages, v_pages, block_table_host, seq_lens_host, window, scale, out_host, lse_host,
                       static_cast<cudaStream_t>(stream), false, nullptr, nullptr);
}

int decode_attn_fp8kv_host_io(const da_tensor *q_host, const da_tensor *k_pages, const da_tensor *v_pages,
                              const float *k_scale, const float *v_scale, const da_tensor *block_table_host,
                              const da_tensor *seq_lens_host, int32_t window, float scale, da_tensor *out_host,
                              da_tensor *lse_host, void *stream)
{
    return run_host_io(q_host, k_pages, v_pages, block_table_host, seq_lens_host, window, scale, out_host, lse_host,
                       static_cast<cudaStream_t>(stream), true, k_scale, v_scale);
}

int decode_attn_static_scratch(const da_tensor *q, const da_tensor *k_pages, const da_tensor *v_pages,
                               const da_tensor *block_table, const da_tensor *seq_lens, int32_t window, float scale,
                               da_tensor *out, da_tensor *lse, int32_t *dev_status4, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Dims d;
    int rc = validate(q, k_pages, v_pages, block_table, seq_lens, out, lse, &d);
    if (rc != DA_OK) return rc;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    const int nblocks = grid_blocks_for(st);
    const WsLayout lay = ws_layout(d.B, d.Hq, HEAD_DIM, d.max_pages, nblocks, kMaxGroup);
    // beyond the fixed array: refuse, never spill into an allocation
    if (d.B > kStaticMaxSeqs || nblocks > kStaticMaxBlocks || lay.stg_q > kStaticScratchBytes)
        return DA_ERR_WORKSPACE;
    if (!g_static_scratch_addr[dev]) {
        // once per device, with that device current: the device address of the array
        void *p = nullptr;
        DA_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return cuda_fail(cudaErrorInvalidSymbol);
        g_static_scratch_addr[dev] = static_cast<uint8_t *>(p);
    }
    uint8_t *ws = g_static_scratch_addr[dev];
    // the array keeps the previous call's contents; only the status record has to start at zero
    DA_CUDA(cudaMemsetAsync(ws + lay.status, 0, 16, stream));
    if (d.B > 0) {
        // one static range per thread block, no ticketed units: keeps the partial slots within the array
        rc = launch_path(st, d, ws, lay, nblocks, 0, q, k_pages, v_pages, block_table, seq_lens, window, scale, out,
                         lse, stream);
        if (rc != DA_OK) return rc;
    }
    if (dev_status4)
        DA_CUDA(cudaMemcpyAsync(dev_status4, ws + lay.status, 16, cudaMemcpyDeviceToDevice, stream));
    return DA_OK;
}

size_t decode_attn_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t P, int64_t max_pages)
{
    (void)Hkv;
    (void)P;
    if (B < 0 || Hq <= 0 || D <= 0 || max_pages < 0) return 0;
    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    int nblocks = g_opt_grid_blocks > 0 ? (int)g_opt_grid_blocks : kMaxGridBlocks;
    if (g_opt_grid_blocks <= 0 && current_device(&dev, &st) == DA_OK)
        nblocks = grid_blocks_for(st);
    return ws_layout(B, Hq, D, max_pages, nblocks + tail_units_for(nblocks)).total;
}

int decode_attn_set_workspace(void *dev_ptr, size_t bytes)
{
    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    int rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    if (!dev_ptr) {
        st->ws = nullptr;
        st->ws_bytes = 0;
        return DA_OK;
    }
    if (reinterpret_cast<uintptr_t>(dev_ptr) & 255u) return DA_ERR_STRIDE_ALIGN;
    if (bytes < 256) return DA_ERR_WORKSPACE;
    DA_CUDA(cudaMemsetAsync(dev_ptr, 0, bytes < kWsHeadBytes ? bytes : kWsHeadBytes, 0));
    DA_CUDA(cudaStreamSynchronize(0));
    st->ws = dev_ptr;
    st->ws_bytes = bytes;
    return DA_OK;
}

int decode_attn_read_device_status(void *stream_, int32_t *host_status4)
{
    if (!host_status4) return DA_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    void *ws;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        int dev;
        DeviceState *st;
        int rc = current_device(&dev, &st);
        if (rc != DA_OK) return rc;
        if (!st->ws) return DA_ERR_WORKSPACE;
        ws = st->ws;
    }
    DA_CUDA(cudaMemcpyAsync(host_status4, ws, 16, cudaMemcpyDeviceToHost, stream));
    DA_CUDA(cudaMemsetAsync(ws, 0, 16, stream));
    DA_CUDA(cudaStreamSynchronize(stream));
    if (host_status4[0] == DA_DEV_TIMEOUT) {
        // a call that gave up may have left the direct path's pair counters part-way: start them at zero again
        std::lock_guard<std::mutex> lock(g_mu);
        int dev;
        DeviceState *st;
        if (current_device(&dev, &st) == DA_OK && st->ws == ws && st->ws_bytes >= kWsHeadBytes) {
            DA_CUDA(cudaMemsetAsync(static_cast<uint8_t *>(ws) + 256, 0, kWsHeadBytes - 256, stream));
            DA_CUDA(cudaStreamSynchronize(stream));
        }
    }
    return DA_OK;
}

int decode_attn_plan(const da_tensor *seq_lens, int32_t window, int32_t Hkv, int32_t P, int64_t max_pages,
                     int32_t *host_seq_info, int32_t *host_unit_work, int32_t *num_units, int32_t *num_static,
                     int32_t *tile_tokens, void *stream_)
{
    if (!seq_lens || !seq_lens->data || !host_seq_info || !host_unit_work || !num_units || !num_static || !tile_tokens)
        return DA_ERR_NULL;
    if (seq_lens->dtype != DA_I32) return DA_ERR_DTYPE;
    if (seq_lens->ndim != 1 || Hkv <= 0 || max_pages <= 0) return DA_ERR_SHAPE;
    if (P != 16 && P != 32 && P != 64 && P != 128) return DA_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::lock_guard<std::mutex> lock(g_mu);
    int dev;
    DeviceState *st;
    int rc = current_device(&dev, &st);
    if (rc != DA_OK) return rc;
    const int nblocks = grid_blocks_for(st);
    const int n_tail = tail_units_for(nblocks);
    Dims d;
    d.B = seq_lens->shape[0];
    d.Hkv = Hkv;
    d.P = P;
    d.max_pages = max_pages;
    const WsLayout lay = ws_layout(d.B, 1, HEAD_DIM, max_pages, nblocks + n_tail);
    if (!st->ws || st->ws_bytes < lay.part_lse) return DA_ERR_WORKSPACE;
    if (*num_units < nblocks + n_tail) return DA_ERR_SHAPE;
    *num_units = 0;
    *num_static = nblocks;
    *tile_tokens = TILE_T;
    if (d.B == 0) return DA_OK;
    uint8_t *ws = static_cast<uint8_t *>(st->ws);
    rc = launch_plan(seq_lens, window, 0, d, ws, lay, nblocks, n_tail, stream);
    if (rc != DA_OK) return rc;
    PlanHeader h;
    DA_CUDA(cudaMemcpyAsync(&h, ws + lay.hdr, sizeof h, cudaMemcpyDeviceToHost, stream));
    DA_CUDA(cudaMemcpyAsync(host_seq_info, ws + lay.seq_info, (size_t)d.B * 16, cudaMemcpyDeviceToHost, stream));
    DA_CUDA(cudaMemcpyAsync(host_unit_work, ws + lay.unit_work, (size_t)(nblocks + n_tail) * 16, cudaMemcpyDeviceToHost,
                            stream));
    DA_CUDA(cudaStreamSynchronize(stream));
    *num_units = h.n_static + h.n_tail;
    for (int u = 0; u < nblocks + n_tail; ++u)
        host_unit_work[4 * u + 1] &= 0xffff;   // (the kernels keep per-unit flags above the KV head)
    return DA_OK;
}

int decode_attn_set_option(const char *name, int64_t value)
{
    if (!name) return DA_ERR_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    if (std::strcmp(name, "grid_blocks") == 0) {
        if (value < 0 || value > kMaxGridBlocks) return DA_ERR_UNSUPPORTED;
        g_opt_grid_blocks = value;
        return DA_OK;
    }
    if (std::strcmp(name, "tail_units") == 0) {
        if (value < 0 || value > 64) return DA_ERR_UNSUPPORTED;
        g_opt_tail_units = value;
        return DA_OK;
    }
    if (std::strcmp(name, "static_frac") == 0) {
        if (value < 0 || value > 256) return DA_ERR_UNSUPPORTED;
        g_opt_static_frac = value;
        return DA_OK;
    }
    if (std::strcmp(name, "kv_evict_first") == 0) {
        if (value < 0 || value > 2) return DA_ERR_UNSUPPORTED;
        g_opt_kv_evict_first = value;
        return DA_OK;
    }
    if (std::strcmp(name, "direct_path") == 0) {
        if (value < 0 || value > 1) return DA_ERR_UNSUPPORTED;
        g_opt_direct_path = value;
        return DA_OK;
    }
    if (std::strcmp(name, "fold_pairs") == 0) {
        if (value < 0 || value > 2) return DA_ERR_UNSUPPORTED;
        g_opt_fold_pairs = value;
        return DA_OK;
    }
    if (std::strcmp(name, "cascade_overlap") == 0) {
        if (value < 0 || value > 2) return DA_ERR_UNSUPPORTED;
        g_opt_cascade_overlap = value;
        return DA_OK;
    }
    if (std::strcmp(name, "cascade_prefix_sms") == 0) {
        if (value < 0 || value > 1024) return DA_ERR_UNSUPPORTED;
        g_opt_cascade_prefix_sms = value;
        return DA_OK;
    }
    if (std::strcmp(name, "extend_stream_rows") == 0) {
        if (value < 0 || value > kMaxStreamRows) return DA_ERR_UNSUPPORTED;
        g_opt_extend_stream_rows = value;
        return DA_OK;
    }
#ifdef DA_DIAG
    // Diagnostic build only; each writes a device variable of the current device (synchronously).
    if (std::strcmp(name, "diag_wait_limit_us") == 0) {
        if (value < 1 || value > 2000000) return DA_ERR_UNSUPPORTED;
        const unsigned long long ns = (unsigned long long)value * 1000ull;
        DA_CUDA(cudaMemcpyToSymbol(da::g_diag_wait_limit_ns, &ns, sizeof ns));
        g_host_wait_limit_us = value;
        return DA_OK;
    }
    if (std::strcmp(name, "diag_withhold_partition_tile") == 0 || std::strcmp(name, "diag_withhold_prefix_tile") == 0) {
        if (value < -1 || value > 0x7fffffffll) return DA_ERR_UNSUPPORTED;
        const int which = std::strcmp(name, "diag_withhold_prefix_tile") == 0;
        const int v = (int)value;
        DA_CUDA(cudaMemcpyToSymbol(da::g_diag_withhold, &v, sizeof v, (size_t)which * sizeof(int)));
        g_host_withhold[which] = value;
        return DA_OK;
    }
#endif
    return DA_ERR_UNSUPPORTED;
}

int64_t decode_attn_get_option(const char *name)
{
    if (!name) return -1;
    std::lock_guard<std::mutex> lock(g_mu);
    if (std::strcmp(name, "grid_blocks") == 0) return g_opt_grid_blocks;
    if (std::strcmp(name, "tail_units") == 0) return g_opt_tail_units;
    if (std::strcmp(name, "static_frac") == 0) return g_opt_static_frac;
    if (std::strcmp(name, "kv_evict_first") == 0) return g_opt_kv_evict_first;
    if (std::strcmp(name, "extend_stream_rows") == 0) return g_opt_extend_stream_rows;
    if (std::strcmp(name, "direct_path") == 0) return g_opt_direct_path;
    if (std::strcmp(name, "fold_pairs") == 0) return g_opt_fold_pairs;
    if (std::strcmp(name, "cascade_overlap") == 0) return g_opt_cascade_overlap;
    if (std::strcmp(name, "cascade_prefix_sms") == 0) return g_opt_cascade_prefix_sms;
#ifdef DA_DIAG
    if (std::strcmp(name, "diag_wait_limit_us") == 0) return g_host_wait_limit_us;
    if (std::strcmp(name, "diag_withhold_partition_tile") == 0) return g_host_withhold[0];
    if (std::strcmp(name, "diag_withhold_prefix_tile") == 0) return g_host_withhold[1];
#endif
    return -1;
}

int decode_attn_set_profile_events(void *before, void *after)
{
    std::lock_guard<std::mutex> lock(g_mu);
    g_ev_before = static_cast<cudaEvent_t>(before);
    g_ev_after = static_cast<cudaEvent_t>(after);
    return DA_OK;
}

const char *decode_attn_strerror(int status)
{
    switch (status) {
    case DA_OK: return "ok";
    case DA_ERR_NULL: return "a required pointer is NULL";
    case DA_ERR_SHAPE: return "tensor ranks or extents disagree";
    case DA_ERR_DTYPE: return "wrong element type";
    case DA_ERR_STRIDE_ALIGN: return "non-contiguous last dimension, or a base/stride that is not suitably aligned";
    case DA_ERR_UNSUPPORTED: return "unsupported head_dim, page size, group size or option";
    case DA_ERR_WORKSPACE: return "no workspace registered for this device, or it is too small";
    case DA_ERR_CUDA: return "a CUDA call failed (see decode_attn_last_cuda_error)";
    default: return "unknown status";
    }
}

int decode_attn_timeline(unsigned long long *host_out, int64_t capacity, int32_t clear)
{
#ifdef DA_TIMELINE
    constexpr int64_t n = (int64_t)da::TL_ROWS * da::TL_COLS;
    if (!host_out) return DA_ERR_NULL;
    if (capacity < n) return DA_ERR_SHAPE;
    std::lock_guard<std::mutex> lock(g_mu);
    DA_CUDA(cudaMemcpyFromSymbol(host_out, da::g_timeline, (size_t)n * 8));   // waits for the device's work
    if (clear) {
        void *sym = nullptr;
        DA_CUDA(cudaGetSymbolAddress(&sym, da::g_timeline));
        DA_CUDA(cudaMemset(sym, 0, (size_t)n * 8));
    }
    return DA_OK;
#else
    (void)host_out; (void)capacity; (void)clear;
    return DA_ERR_UNSUPPORTED;
#endif
}

int decode_attn_last_cuda_error(void) { return g_last_cuda_error.load(); }
int decode_attn_version(void) { return kVersion; }
int64_t decode_attn_launch_count(void) { return g_launches.load(); }

}  // extern "C"
