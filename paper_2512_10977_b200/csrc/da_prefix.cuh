// Shared-prefix ("cascade") decode: when every sequence of the batch starts with the same pages --
// the agent sessions all begin with one long initial prompt -- the attention of all B * Hq query
// vectors over that prefix is one dense contraction per KV head: a (B*G) x T score matrix against
// K, softmax, times V.  That is tensor-core work, done here with tcgen05 (operands in shared memory
// by TMA, accumulators in tensor memory), instead of streaming the same pages once per sequence.
//
// prefix_kernel: one block = 128 query rows (row = b * G + head-in-group) of one KV head and one
// range of 128-token KV tiles.  Per tile:  S = Q K^T  (tcgen05.mma, M = N = K = 128, fp32 in TMEM)
// -> the sixteen softmax warps read their rows of S (four threads per row, 32 columns each), keep running
// max / sum in the log2 domain, write P = exp2(S - m) as bf16 high and low parts over their scores in tensor
// memory -> O += P_hi V + P_lo V (tcgen05.mma with the A operand in TMEM, accumulating in another TMEM
// region) -> the softmax threads rescale a row of O in TMEM only when its maximum has grown by more than
// 2^8 (rare).  Three more warps issue the MMAs -- one the score products, one the P_hi V products, one the
// P_lo V products into an accumulator of its own: a thread that issues a tcgen05.mma is held for about
// 70 ns, longer than the tensor core needs for a 128 x 128 x 16 product, so a single issuing thread keeps
// the pipe less than half busy; issued from several warps the same instructions run back to back -- and two
// more the TMA loads, one for K and one for V (issuing a tile's tensor copies is slow enough that one warp
// doing it all set the pace of the block).  Result: a normalised partial (O / l, lse) per (split, b, h),
// combined with the per-sequence suffix attention by cascade_merge_kernel.
#pragma once
#include "da_kernels.cuh"

namespace da {

constexpr int PF_ROWS = 128;                 // query rows per block (UMMA M)
constexpr int PF_TOK = 128;                  // tokens per KV tile (UMMA N for S, K for PV)
constexpr int PF_PLANE = PF_TOK * 128;       // one 64-column half of a 128-row tile: 128-byte rows
constexpr int PF_TILE = 2 * PF_PLANE;        // 32 KB: Q, a K tile, a V tile
constexpr int PF_TPR = 4;                    // softmax threads per row (each owns 128 / PF_TPR columns of a tile)
constexpr int PF_COLS = 128 / PF_TPR;
constexpr int PF_DRV = 4 * PF_TPR;           // warps 0..15: softmax; warp 16: issues the score MMAs (and owns the TMEM
constexpr int PF_PV = PF_DRV + 1;            // allocation); warps 17, 18: issue the P_hi V and the P_lo V MMAs;
constexpr int PF_LOADER = PF_DRV + 3;        // warp 19: issues the TMA loads of K, warp 20 those of V
constexpr int PF_THREADS = (PF_LOADER + 5) * 32;   // + one idle warp: whole warpgroups, for the register hand-over   // (one tensor copy costs its issuing warp ~90 cycles)
// Registers.  The block is launched with PF_REGS_LAUNCH a thread (the kernel's compiled count, checked on the
// host before the first launch); the sixteen softmax warps then take PF_REGS_SOFTMAX each and the other eight
// (two whole warpgroups) keep PF_REGS_OTHER: the sum must not exceed what the block was launched with, or the
// increase would wait for registers that never come.
constexpr int PF_REGS_LAUNCH = 80, PF_REGS_SOFTMAX = 96, PF_REGS_OTHER = 40;
static_assert(PF_DRV * PF_REGS_SOFTMAX + (PF_THREADS / 32 - PF_DRV) * PF_REGS_OTHER <= (PF_THREADS / 32) * PF_REGS_LAUNCH,
              "the register shares of the warps must fit what the block is launched with");
constexpr int PF_OFF_Q = 0;
constexpr float PF_RESCALE_LOG2 = 8.f;       // a row's reference maximum moves only when the maximum grew by more
constexpr uint32_t PF_WAIT_SLEEP_NS = 32;     // softmax warps yield while they wait: the driver warp shares their schedulers
constexpr int PF_NB = 3;                     // K and V buffers (tiles in flight)
constexpr int PF_OFF_K = PF_TILE;
constexpr int PF_OFF_V = (1 + PF_NB) * PF_TILE;
constexpr int PF_OFF_BARS = (1 + 2 * PF_NB) * PF_TILE;   // kfull[3], vfull[3], kfree[3], o[3], s[2], p[2], x[4]
constexpr int PF_OFF_MISC = PF_OFF_BARS + 160;  // TMEM base address, abort flag, "a page id was bad" flag
constexpr int PF_OFF_XCHG = PF_OFF_MISC + 16;   // row maxima / sums swapped between a row's two threads
constexpr int PF_SMEM_BYTES = PF_OFF_XCHG + PF_TPR * 128 * 4;   // 2 buffers of bf16 maxima, or one of fp32 sums
static_assert(PF_SMEM_BYTES <= 232448, "one block must fit the 227 KB of shared memory an SM offers");
constexpr int PF_TMEM_COLS = 512;            // S buffers in columns [0,128) and [128,256), O in [256,384) (the P_hi V
                                             // products) and [384,512) (the P_lo V products; added at the end).
constexpr int PF_TMEM_PH = 0;                // P(j) overwrites S(j) in place once both threads of a row have read
constexpr int PF_TMEM_PL = 64;               // their scores: high parts in the buffer's columns [0,64), low parts in
                                             // [64,128) -- 128 tokens as 64 columns of bf16 pairs, the A operand of
                                             // the PV product.  So P is double-buffered like S, and the softmax of
                                             // tile j+1 does not wait for the PV product of tile j.

// The kernel serves two callers.
//  * cascade (ext = 0): rows = all sequences' heads of one KV group, row = b * G + head; keys = the
//    shared prefix, named by row 0 of the block table; every row attends every prefix token.
//  * extend (ext = 1): one sequence per block; rows = its Lq new query tokens' heads of one KV
//    group, row = qi * G + head; keys = that sequence's own pages; query qi sits at position
//    L - Lq + qi and attends tokens 0 .. L - Lq + qi (causal).
struct PrefixParams {
    const __nv_bfloat16 *q;
    int64_t q_sb, q_sq, q_sh;     // strides of sequence, query token (extend), head
    const int32_t *block_table;
    int64_t bt_sb;
    const int32_t *seq_lens;      // extend only
    int64_t sl_stride;
    float *pre_o;                 // [splits][rows_total * Hkv][128] normalised partials (rows_total = B*Lq*G)
    float *pre_lse;               // [splits][rows_total * Hkv]
    void *out;                    // extend with one split writes the result directly
    int64_t o_sb, o_sq, o_sh;
    float *lse;
    int64_t l_sb, l_sq, l_sh;
    int32_t *status;
    int32_t B, Hkv, G, P, box_rows, num_pages, out_bf16;
    int32_t ext, Lq;
    int64_t max_pages;
    int32_t prefix_tiles;         // cascade: shared prefix length / PF_TOK
    int32_t splits;               // KV ranges per (row tile, head)
    int32_t split0;               // cascade: the first KV range of this launch (a call may launch the ranges in two groups)
    int32_t row_tiles;            // cascade: ceil(B*G / 128); extend: ceil(Lq*G / 128)
    float scale_log2;
    // The shared prefix of an 8-bit cache, widened to bf16 in scratch (widen_prefix_kernel): the pools are
    // then that scratch copy, whose page i holds tokens [i P, (i+1) P) (no block table), and the per-KV-head
    // factors enter here -- k_scale[g] with the score scale, v_scale[g] with the result.  NULL / 0 otherwise.
    const float *k_scale, *v_scale;
    int32_t identity_pages;       // > 0: page t / P of sequence b is page b * identity_pages + t / P of the pools
    int32_t seq0;                 // sequence number of row 0 in the caller's batch (a call may be made in groups): status records
};

// ---------------------------------------------------------------- tcgen05 wrappers
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4),
// descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor for kind::f16: fp32 accumulator, bf16 A and B, A K-major, B K- or
// MN-major, N and M in units of 8 and 16.
__device__ __forceinline__ uint32_t umma_idesc(int m, int n, bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// Arrive on `bar` once every tcgen05 operation this thread issued so far has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
        "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i)
        v[i] = __uint_as_float(r[i]);
}
// The same load without the wait, so that several can be in flight; tmem_ld_wait() ends them all.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
        "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 32 consecutive 32-bit columns of this thread's TMEM lane, written from registers.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
        "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
// 16 consecutive 32-bit columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D += A * B with the A operand in tensor memory (row i in lane i, two bf16 of K per column).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// The K pool is read here through a 4-D tiled map {d, token, head, page} with box {64, box_rows, 1, 1}:
// one box is one 64-column plane of box_rows token rows, so a plane of a tile is contiguous and
// its 8-row groups are 1024 bytes apart, which is what the matrix descriptors above assume; the V pool
// through the 5-D map of the partition kernel (both planes of box_rows rows per box).
// (The loads themselves are in da_ptx.cuh.)

__global__ void __launch_bounds__(PF_THREADS, 1)
prefix_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const PrefixParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];   // no static shared memory: keeps the base 1024-B aligned
    uint32_t &tmem_base_s = *reinterpret_cast<uint32_t *>(smem + PF_OFF_MISC);
    int &abort_s = *reinterpret_cast<int *>(smem + PF_OFF_MISC + 4);
    volatile int *poison_s = reinterpret_cast<volatile int *>(smem + PF_OFF_MISC + 8);
    const uint32_t sb = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // per K/V buffer (tile t uses buffer t % 3): K loaded, V loaded, K no longer needed (scores complete),
    // PV product complete; per S buffer (t & 1): scores complete; P written; row-maximum exchange
    const uint32_t bar_kfull = sb + PF_OFF_BARS, bar_vfull = bar_kfull + 24, bar_kfree = bar_kfull + 48, bar_o = bar_kfull + 72,
                   bar_s = bar_kfull + 96, bar_p = bar_kfull + 112, bar_x0 = bar_kfull + 128;   // s, p: one per S buffer; x: one per 32 rows
    volatile int *abort_flag = &abort_s;

    // block -> (row tile, kv head, [sequence,] split)
    const int rt = blockIdx.x % p.row_tiles;
    const int g = (blockIdx.x / p.row_tiles) % p.Hkv;
    int split = blockIdx.x / (p.row_tiles * p.Hkv) + p.split0;
    int bseq = 0, L = 0, kv_tiles = p.prefix_tiles;
    int R = p.B * p.G;               // rows in this block's row space
    if (p.ext) {
        bseq = split % p.B;
        split /= p.B;
        R = p.Lq * p.G;
        L = p.seq_lens[(int64_t)bseq * p.sl_stride];
        if (L < 0 || (L > 0 && L < p.Lq) || (int64_t)L > p.max_pages * (int64_t)p.P) {
            if (tid == 0)
                report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, bseq + p.seq0, 2, L);
            L = 0;
        }
        // causal: the block's last row attends tokens below L - Lq + qi_max + 1
        const int qi_max = min(p.Lq - 1, (rt * PF_ROWS + PF_ROWS - 1) / p.G);
        const int lim_max = L > 0 ? L - p.Lq + qi_max + 1 : 0;
        kv_tiles = (lim_max + PF_TOK - 1) / PF_TOK;
    }
    const int t_begin = (int)((long long)kv_tiles * split / p.splits);
    const int t_end = (int)((long long)kv_tiles * (split + 1) / p.splits);
    const int ntiles = t_end - t_begin;
    const int32_t *bt_row = p.block_table + (int64_t)bseq * p.bt_sb;
    // extend: from this token on some row of the block is masked (the first query's limit)
    const int mask_from = p.ext ? L - p.Lq + 1 : 0x7fffffff;

    if ((sb & 1023u) != 0) {
        if (tid == 0)
            report_status(p.status, 3, -6, (int)blockIdx.x, (int)sb);
        return;
    }
    if (tid == 0) {
        abort_s = 0;
        *poison_s = 0;
        for (int i = 0; i < PF_NB; ++i) {
            mbar_init(bar_kfull + 8 * i, 2);   // two loader warps per operand, each arrives with its bytes
            mbar_init(bar_vfull + 8 * i, 2);
            mbar_init(bar_kfree + 8 * i, 1);
            mbar_init(bar_o + 8 * i, 2);   // the two PV products of a tile, committed by their issuing warps
        }
        mbar_init(bar_s, 1);
        mbar_init(bar_s + 8, 1);
        // (one hand-over barrier per S buffer: a warp cannot arrive for tile j + 2 before the hand-over of tile j is
        //  complete -- those scores are only written after it -- so no arrival can be counted for the wrong tile,
        //  however far one warp runs ahead of another)
        mbar_init(bar_p, PF_DRV);
        mbar_init(bar_p + 8, PF_DRV);
        for (int i = 0; i < 4; ++i)
            mbar_init(bar_x0 + 8 * i, PF_TPR);   // the row-maximum exchange of one quarter of the rows: its PF_TPR warps
        mbar_fence_init();
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == PF_DRV)
        tmem_alloc(smem_u32(&tmem_base_s), PF_TMEM_COLS);
    // Q rows of this block into the swizzled K-major layout: row r, 16-byte chunk c (0..15 along d)
    // -> plane c >> 3, byte r * 128 + (((c & 7) ^ (r & 7)) << 4).  Rows past B * G are zero.
    for (int e = tid; e < PF_ROWS * 16; e += PF_THREADS) {
        const int r = e >> 4, c = e & 15;
        const int row = rt * PF_ROWS + r;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (row < R) {
            const int outer = row / p.G, hi = row % p.G;   // sequence (cascade) or query token (extend)
            const __nv_bfloat16 *src = p.q + (p.ext ? (int64_t)bseq * p.q_sb + (int64_t)outer * p.q_sq : (int64_t)outer * p.q_sb) +
                                       (int64_t)(g * p.G + hi) * p.q_sh + c * 8;
            if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
                val = *reinterpret_cast<const uint4 *>(src);
            } else {
                const uint32_t *s32p = reinterpret_cast<const uint32_t *>(src);
                val = make_uint4(s32p[0], s32p[1], s32p[2], s32p[3]);
            }
        }
        *reinterpret_cast<uint4 *>(smem + PF_OFF_Q + (c >> 3) * PF_PLANE + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = val;
    }
    fence_proxy_async_smem();   // Q is read by the tensor core through the async proxy
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    const uint32_t tmem_s = tmem, tmem_o = tmem + 256, tmem_o2 = tmem + 384;   // S(j) lives at tmem_s + 128 * (j & 1)

    if (warp >= PF_LOADER + 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PF_REGS_OTHER));   // the idle warp
    } else if (warp >= PF_LOADER) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PF_REGS_OTHER));
        // ------------------------------------------------------------------ loader warps: TMA
        // Warp PF_LOADER loads the K tiles, warp PF_LOADER + 1 the V tiles (issuing a tile's 16 tensor
        // copies takes a warp ~1500 cycles: one warp for both was the slowest stage of the block).
        // K: lane l < 2 * boxes issues one load per tile: box l >> 1 (box_rows tokens of one page), plane
        // l & 1 -- the score product reads a K tile as 128 rows of one 64-column plane after the other, so
        // a copy cannot span both planes.  V: lane l < boxes issues one load per tile, box l with both of
        // its planes (the pool seen as {64 columns, token, half, head, page}: half as many copies, and the
        // TMA unit's ~85 cycles per copy are what the loaders spend their time on); the tile is then its
        // boxes one after the other, each box_rows rows of the first 64 columns followed by box_rows rows
        // of the other 64, which suits the PV product: each of its steps reads 16 token rows, and the
        // distance between the planes is just its descriptor's leading offset.  Tiles 0..2 fill the three
        // buffers; after that K(t) follows the completion of the scores of tile t-3 (bar_kfree) and V(t)
        // the completion of the PV products of tile t-3 (bar_o).
        if (ntiles > 0) {
            const bool is_v = warp >= PF_LOADER + 2;
            const int half = (warp - PF_LOADER) & 1;            // each operand's copies are shared by two warps
            const int boxes = PF_TOK / p.box_rows;
            const int copies = is_v ? boxes : 2 * boxes, per_warp = max(1, copies / 2);
            const int ci = lane + half * per_warp;              // this lane's copy of the tile
            const int box = is_v ? ci : ci >> 1, pl = is_v ? 0 : ci & 1;
            const bool active = lane < per_warp && ci < copies;
            const uint32_t bar_full = is_v ? bar_vfull : bar_kfull;
            const uint32_t bar_free = is_v ? bar_o : bar_kfree;
            const CUtensorMap *tm = is_v ? &tm_v : &tm_k;
            bool ok = true;
            int issued = 0;
            auto read_page = [&](int j) {   // page id of this lane's box of tile j (0 for idle lanes)
                if (!active || j >= ntiles)
                    return 0;
                const int t = (t_begin + j) * PF_TOK + box * p.box_rows;
                if (p.ext && t >= L)
                    return 0;   // past the sequence's last page: the block table has no entry
                return p.identity_pages ? bseq * p.identity_pages + t / p.P : __ldg(bt_row + t / p.P);
            };
            auto load_tile = [&](int j, int page) {   // tile j into buffer j % 3
                const int buf = j % PF_NB;
                const uint32_t bar = bar_full + 8 * buf;
                // extend: boxes wholly past the sequence's end are not loaded (their rows are masked)
                const int t_tile = (t_begin + j) * PF_TOK;
                const int nbox = p.ext ? min(boxes, (L - t_tile + p.box_rows - 1) / p.box_rows) : boxes;
                const bool mine = active && box < nbox;
                const int t = t_tile + box * p.box_rows;
                if (mine && (uint32_t)page >= (uint32_t)p.num_pages) {
                    // A page id outside the pool.  The copy is made from just past the pool instead (the
                    // tensor map fills zeros there and still counts the bytes), and the block is marked:
                    // its rows are written as NaN, not as a finite result over zeroed keys.
                    if (!is_v && pl == 0)
                        report_status(p.status, 1 /* DA_DEV_BAD_PAGE */, bseq + p.seq0, t / p.P, page);
                    *poison_s = 1;
                    page = p.num_pages;
                }
                // (diagnostic build only: the K loader of block 0 can leave one tile out altogether)
                const bool withheld = !is_v && DA_WITHHOLD(1, blockIdx.x, j);
                const uint32_t n_mine = (uint32_t)__popc(__ballot_sync(0xffffffffu, mine));   // (also orders the mark above
                if (lane == 0 && !withheld)                                                    //  before lane 0's arrival)
                    mbar_arrive_expect_tx(bar, n_mine * (uint32_t)p.box_rows * (is_v ? 256u : 128u));
                __syncwarp();
                if (mine && !withheld) {
                    if (is_v)
                        tma_load_5d(sb + PF_OFF_V + (uint32_t)(buf * PF_TILE + box * p.box_rows * 256), tm, 0, t % p.P, 0, g, page, bar);
                    else
                        tma_load_4d(sb + PF_OFF_K + (uint32_t)(buf * PF_TILE + pl * PF_PLANE + box * p.box_rows * 128), tm,
                                    pl * 64, t % p.P, g, page, bar);
                }
                issued = j + 1;
            };
            int pg = read_page(0);
            DA_PH_DECL(ph, ph_t);
            for (int t = 0; ok && t < ntiles; ++t) {
                if (t >= PF_NB) {
                    ok = mbar_wait_bounded(bar_free + 8 * (t % PF_NB), (uint32_t)(((t - PF_NB) / PF_NB) & 1), abort_flag);
                    if (!ok)
                        break;
                }
                DA_PH(ph, 0, ph_t);
                const int pg_now = pg;
                pg = read_page(t + 1);   // fetched one tile ahead
                load_tile(t, pg_now);
                DA_PH(ph, 1, ph_t);
            }
            if (blockIdx.x == 0 && lane == 0 && half == 0)
                DA_PH_STORE(TL_PREFIX + 4 + (int)is_v, ph);
            if (!ok && lane == 0) {
                if (*abort_flag == 0) {
                    *abort_flag = 1;
                    report_status(p.status, 3 /* DA_DEV_TIMEOUT */, -9, (int)blockIdx.x, 0);
                }
            }
            if (*abort_flag && lane == 0) {
                // do not leave while copies may still land in shared memory: bounded wait for the
                // latest fill of each buffer
                for (int k = 0; k < PF_NB; ++k) {
                    const int jk = issued - 1 - k;
                    const uint64_t t0 = globaltimer_ns();
                    while (jk >= 0 && !mbar_try_wait(bar_full + 8 * (jk % PF_NB), (uint32_t)((jk / PF_NB) & 1))) {
                        if (globaltimer_ns() - t0 > DA_WAIT_LIMIT_NS / 2)
                            break;
                    }
                }
            }
        }
    } else if (warp == PF_DRV) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PF_REGS_OTHER));
        // ------------------------------------------------------------------ score MMA warp
        // All lanes wait together; lane 0 issues.  S(0), S(1), then S(j+2) into the S buffer of tile j as
        // soon as both PV products of tile j are complete (they read P(j) from that buffer) -- so the scores
        // of tile j+1 are ready before the softmax of j ends.  Nothing is computed per instruction that can
        // be computed once: the matrix descriptors of Q and of the first K buffer are built here, and a step
        // or a buffer only adds a constant to the descriptor's address field (bits 0-13, in 16-byte units).
        if (ntiles > 0) {
            bool ok = true;
            const uint64_t q_desc = umma_desc(sb + PF_OFF_Q, 16, 1024);
            const uint64_t k_desc = umma_desc(sb + PF_OFF_K, 16, 1024);
            const uint32_t idesc_s = umma_idesc(PF_ROWS, PF_TOK, false);
            static_assert(PF_OFF_V + PF_NB * PF_TILE <= (1 << 18), "descriptor addresses must stay inside 256 KB");
            auto mma_s = [&](int j) {   // S = Q K^T for tile j
                const uint64_t kd = k_desc + (uint64_t)(((j % PF_NB) * PF_TILE) >> 4);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * PF_PLANE + (kk & 3) * 32) >> 4);
                    umma_bf16(tmem_s + 128 * (j & 1), q_desc + off, kd + off, idesc_s, kk > 0);
                }
                umma_commit(bar_s + 8 * (j & 1));
                umma_commit(bar_kfree + 8 * (j % PF_NB));
            };
            auto kfull = [&](int j) {
                return mbar_wait_bounded(bar_kfull + 8 * (j % PF_NB), (uint32_t)((j / PF_NB) & 1), abort_flag);
            };
            for (int j = 0; ok && j < 2 && j < ntiles; ++j) {
                ok = kfull(j);
                if (ok) {
                    tc_fence_after();
                    if (lane == 0)
                        mma_s(j);
                    __syncwarp();
                }
            }
            DA_PH_DECL(ph, ph_t);
            for (int j = 0; ok && j + 2 < ntiles; ++j) {
                ok = mbar_wait_bounded(bar_o + 8 * (j % PF_NB), (uint32_t)((j / PF_NB) & 1), abort_flag);
                DA_PH(ph, 0, ph_t);
                ok = ok && kfull(j + 2);
                DA_PH(ph, 1, ph_t);
                if (!ok)
                    break;
                tc_fence_after();
                if (lane == 0)
                    mma_s(j + 2);
                __syncwarp();
                DA_PH(ph, 2, ph_t);
            }
            if (blockIdx.x == 0 && lane == 0)
                DA_PH_STORE(TL_PREFIX + 1, ph);
            if (!ok && lane == 0 && *abort_flag == 0) {
                *abort_flag = 1;
                report_status(p.status, 3 /* DA_DEV_TIMEOUT */, -7, (int)blockIdx.x, 0);
            }
        }
    } else if (warp == PF_PV || warp == PF_PV + 1) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PF_REGS_OTHER));
        // ------------------------------------------------------------------ PV MMA warps
        // Warp PF_PV accumulates P_hi V in tmem_o, warp PF_PV + 1 P_lo V in tmem_o2: for every tile, as soon
        // as P is written and V has landed.  A = P from tensor memory (16 tokens = 8 columns per step);
        // B = V stored [token][d]: MN-major, planes are the two halves of d (leading offset = plane),
        // 8-token groups 1024 B apart.
        if (ntiles > 0) {
            bool ok = true;
            const bool low = warp == PF_PV + 1;
            // a V tile is its boxes one after the other, each box its two 64-column planes of box_rows rows
            const uint64_t v_desc = umma_desc(sb + PF_OFF_V, (uint32_t)p.box_rows * 128u, 1024);
            const uint32_t idesc_o = umma_idesc(PF_ROWS, HEAD_DIM, true);
            const int log2_br = 31 - __clz(p.box_rows);
            const uint32_t acc = low ? tmem_o2 : tmem_o;
            DA_PH_DECL(ph, ph_t);
            for (int j = 0; ok && j < ntiles; ++j) {
                ok = mbar_wait_bounded(bar_p + 8 * (j & 1), (uint32_t)((j >> 1) & 1), abort_flag);
                DA_PH(ph, 0, ph_t);
                ok = ok && mbar_wait_bounded(bar_vfull + 8 * (j % PF_NB), (uint32_t)((j / PF_NB) & 1), abort_flag);
                DA_PH(ph, 1, ph_t);
                if (!ok)
                    break;
                tc_fence_after();
                if (lane == 0) {
                    const uint64_t vd = v_desc + (uint64_t)(((j % PF_NB) * PF_TILE) >> 4);
                    const uint32_t pa = tmem_s + 128 * (j & 1) + (low ? PF_TMEM_PL : PF_TMEM_PH);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        // tokens 16 kk .. 16 kk + 15: box (16 kk) / box_rows, row (16 kk) % box_rows of it
                        const uint32_t t16 = 16u * kk;
                        const uint32_t off = ((t16 >> log2_br) << (log2_br + 8)) + (t16 & ((uint32_t)p.box_rows - 1u)) * 128u;
                        umma_bf16_ts(acc, pa + kk * 8, vd + (uint64_t)(off >> 4), idesc_o, j > 0 || kk > 0);
                    }
                    umma_commit(bar_o + 8 * (j % PF_NB));
                }
                __syncwarp();
                DA_PH(ph, 2, ph_t);
            }
            if (blockIdx.x == 0 && lane == 0)
                DA_PH_STORE(TL_PREFIX + 2 + (int)low, ph);
            if (!ok && lane == 0 && *abort_flag == 0) {
                *abort_flag = 1;
                report_status(p.status, 3 /* DA_DEV_TIMEOUT */, -7, (int)blockIdx.x, 1 + (int)low);
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(PF_REGS_SOFTMAX));
        // ------------------------------------------------------------------ softmax warps
        // PF_TPR threads per row: warps w, w + 4, w + 8, ... read the same TMEM lanes (32 * (w % 4) ...),
        // each its own PF_COLS columns -- of S (tokens) and of O_tile (head_dim).
        static_assert(PF_COLS == 32, "the TMEM access shapes below are written for 32 columns a thread");
        const int r = 32 * (warp & 3) + lane;            // row of the tile = TMEM lane
        const int part = warp >> 2;                      // which columns
        const uint32_t lane_sel = (uint32_t)(32 * (warp & 3)) << 16;
        const uint32_t lane_base = lane_sel + (uint32_t)(part * PF_COLS);
        // row maxima are swapped as bf16 rounded UP, [2 buffers][PF_TPR parts][128 rows]: every thread of a
        // row reads the same four values, so they agree on one reference that is >= every score (the
        // result does not depend on which reference is used, only on its being common); the final sums
        // of weights go through the same bytes as fp32 [PF_TPR][128]
        __nv_bfloat16 *xchg = reinterpret_cast<__nv_bfloat16 *>(smem + PF_OFF_XCHG);
        // O accumulates in tensor memory across tiles, relative to a reference maximum m_run that is
        // moved only when a row's maximum has grown by more than PF_RESCALE_LOG2 (weights then stay
        // below 2^PF_RESCALE_LOG2, well inside what the bf16 high + low pair carries); moving it
        // means scaling that row of O, which after the first few tiles is rare.
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        // The scale enters inside the exponent (one fma per score).  A masked raw score must come out as
        // -inf after scaling whatever the scale's sign; a scale of exactly 0 would turn it into NaN
        // (inf * 0), so 0 is replaced by 1e-30, which changes no weight by more than 1e-24.
        const float sc_in = p.scale_log2 * (p.k_scale ? __ldg(p.k_scale + g) : 1.f);
        const float sc = sc_in == 0.f ? 1e-30f : sc_in;
        const float v_mul = p.v_scale ? __ldg(p.v_scale + g) : 1.f;
        const float neg_inf_raw = sc > 0.f ? -INFINITY : INFINITY;
        // extend: this row's query attends tokens below `limit` (0 for padding rows: nothing)
        const int rr = rt * PF_ROWS + r;
        const int limit = (p.ext && rr < R && L > 0) ? L - p.Lq + rr / p.G + 1 : 0;
        // extend, a tile that reaches past the sequence's end: those V rows were not loaded, or are a page's
        // unused tail, and may hold NaN, which a zero weight would not hide.  All softmax threads clear them
        // (both planes, 128 bytes a row) once V has landed, before the PV product reads them.
        auto clear_v_tail = [&](int j, int t_tile) {
            if (!mbar_wait_bounded(bar_vfull + 8 * (j % PF_NB), (uint32_t)((j / PF_NB) & 1), abort_flag, DA_WAIT_LIMIT_NS, PF_WAIT_SLEEP_NS))
                return false;
            const int first_bad = max(L - t_tile, 0);
            uint8_t *vb = smem + PF_OFF_V + (j % PF_NB) * PF_TILE;
            for (int e = tid; e < (PF_TOK - first_bad) * 16; e += PF_TPR * PF_ROWS) {
                const int row = first_bad + (e >> 4), ch = e & 15;
                const int bx = row / p.box_rows, rr_ = row % p.box_rows;   // box-major tile: see the loader warps
                *reinterpret_cast<uint4 *>(vb + bx * p.box_rows * 256 + (ch >> 3) * p.box_rows * 128 + rr_ * 128 + ((ch & 7) << 4)) =
                    make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async_smem();
            return true;
        };
        // A warp whose 32 rows all lie past the block's last query row (a few new tokens fill only the first
        // rows of the tile; the last row tile of a batch) computes nothing: it only keeps pace with the
        // barriers its fellows use -- the tail clearing and the hand-over of P.
        const bool has_rows = rt * PF_ROWS + 32 * (warp & 3) < R;
        DA_PH_DECL(ph, ph_t);
#ifdef DA_TIMELINE
        const long long ph_begin = ph_t;
        const unsigned long long ph_ns = globaltimer_ns();
#endif
        const uint32_t bar_x = bar_x0 + 8 * (warp & 3);   // shared with the other warps that hold these 32 rows
        for (int j = 0; !has_rows && j < ntiles; ++j) {
            const int t_tile = (t_begin + j) * PF_TOK;
            if (p.ext && t_tile + PF_TOK > L && !clear_v_tail(j, t_tile)) {
                ok = false;
                break;
            }
            __syncwarp();
            if (lane == 0)
                mbar_arrive(bar_p + 8 * (j & 1));
            // (no second arrival before every warp has made its first: wait for this tile's hand-over)
            if (!mbar_wait_bounded(bar_p + 8 * (j & 1), (uint32_t)((j >> 1) & 1), abort_flag, DA_WAIT_LIMIT_NS, PF_WAIT_SLEEP_NS)) {
                ok = false;
                break;
            }
        }
        for (int j = 0; has_rows && j < ntiles; ++j) {
            if (!mbar_wait_bounded(bar_s + 8 * (j & 1), (uint32_t)((j >> 1) & 1), abort_flag, DA_WAIT_LIMIT_NS, PF_WAIT_SLEEP_NS)) {
                ok = false;
                break;
            }
            DA_PH(ph, 0, ph_t);
            tc_fence_after();
            // this thread's raw scores (q.k) and the largest scaled one
            float sv[PF_COLS];
            {
                uint32_t v[PF_COLS];
                tmem_ld32_issue(tmem_s + 128 * (j & 1) + lane_base, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < PF_COLS; ++i)
                    sv[i] = __uint_as_float(v[i]);
            }
            const int t_tile = (t_begin + j) * PF_TOK;
            if (t_tile + PF_TOK > mask_from) {   // extend, near the end: causal mask by select (K rows past
                const int t_mine = t_tile + part * PF_COLS;   // the sequence's end may hold anything)
#pragma unroll
                for (int i = 0; i < PF_COLS; ++i)
                    if (t_mine + i >= limit)
                        sv[i] = neg_inf_raw;
            }
            // (three at a time; fifteen instructions, five deep, for 32 scores)
            float mx;
            if (sc > 0.f) {
                float t[11];
#pragma unroll
                for (int i = 0; i < 10; ++i)
                    t[i] = fmax3(sv[3 * i], sv[3 * i + 1], sv[3 * i + 2]);
                t[10] = fmaxf(sv[30], sv[31]);
                const float u0 = fmax3(t[0], t[1], t[2]), u1 = fmax3(t[3], t[4], t[5]), u2 = fmax3(t[6], t[7], t[8]);
                mx = fmax3(fmax3(u0, u1, u2), t[9], t[10]);
            } else {
                float t[11];
#pragma unroll
                for (int i = 0; i < 10; ++i)
                    t[i] = fmin3(sv[3 * i], sv[3 * i + 1], sv[3 * i + 2]);
                t[10] = fminf(sv[30], sv[31]);
                const float u0 = fmin3(t[0], t[1], t[2]), u1 = fmin3(t[3], t[4], t[5]), u2 = fmin3(t[6], t[7], t[8]);
                mx = fmin3(fmin3(u0, u1, u2), t[9], t[10]);
            }
            mx = (mx == neg_inf_raw) ? -INFINITY : mx * sc;
            // the row's threads must use one maximum: swap through shared memory ([row][part]: a thread
            // reads its row's four values with one 8-byte load)
            __nv_bfloat16 *xb = xchg + (j & 1) * (PF_TPR * 128);
            xb[r * PF_TPR + part] = __float2bfloat16_ru(mx);
            __syncwarp();
            if (lane == 0)
                mbar_arrive(bar_x);
            if (!mbar_wait_bounded(bar_x, (uint32_t)(j & 1), abort_flag, DA_WAIT_LIMIT_NS, PF_WAIT_SLEEP_NS)) {
                ok = false;
                break;
            }
            static_assert(PF_TPR == 4, "four bf16 maxima per row are read as one 8-byte word");
            {
                const uint2 four = *reinterpret_cast<const uint2 *>(xb + r * PF_TPR);
                const uint32_t m2 = bf16x2_max(four.x, four.y);
                mx = fmaxf(bf16_lo_to_float(m2), bf16_hi_to_float(m2));
            }
            DA_PH(ph, 1, ph_t);
            const bool moved = (m_run == -INFINITY) || (mx > m_run + PF_RESCALE_LOG2);
            const float m_new = moved ? mx : m_run;
            const float alpha = !moved ? 1.f : (m_run == -INFINITY ? 0.f : fast_exp2(m_run - m_new));
            // weights, their sum, and P as bf16 high + low parts (kept in registers for now)
            // (two scores per instruction where the arithmetic allows: scale and shift, the sum, the low part)
            uint32_t phi[PF_COLS / 2], plo[PF_COLS / 2];
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;   // a row with nothing to attend yet
            const uint64_t sc2 = f32x2(sc, sc), nm2 = f32x2(-m_use, -m_use);
            uint64_t lsum_a = f32x2(0.f, 0.f), lsum_b = lsum_a;
#pragma unroll
            for (int e = 0; e < PF_COLS / 2; ++e) {
                float x0, x1, l0, l1;
                f32x2_split(f32x2_fma(f32x2(sv[2 * e], sv[2 * e + 1]), sc2, nm2), x0, x1);
                const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                const uint64_t pp = f32x2(p0, p1);
                if (e & 1)
                    lsum_b = f32x2_add(lsum_b, pp);
                else
                    lsum_a = f32x2_add(lsum_a, pp);
                phi[e] = pack_bf16(p0, p1);
                f32x2_split(f32x2_sub(pp, f32x2(bf16_lo_to_float(phi[e]), bf16_hi_to_float(phi[e]))), l0, l1);
                plo[e] = pack_bf16(l0, l1);
            }
            float lsum;
            {
                float s0, s1;
                f32x2_split(f32x2_add(lsum_a, lsum_b), s0, s1);
                lsum = s0 + s1;
            }
            // a row of O may be rescaled only once the previous tile's PV product is complete
            // (tcgen05.ld / .st are warp-wide: all lanes go)
            if (j > 0 && __any_sync(0xffffffffu, moved)) {
                if (!mbar_wait_bounded(bar_o + 8 * ((j - 1) % PF_NB), (uint32_t)(((j - 1) / PF_NB) & 1), abort_flag, DA_WAIT_LIMIT_NS, PF_WAIT_SLEEP_NS)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
#pragma unroll 1
                for (int a = 0; a < 2; ++a) {
                    const uint32_t at = (a ? tmem_o2 : tmem_o) + lane_base;
                    uint32_t v[PF_COLS];
                    tmem_ld32_issue(at, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < PF_COLS; ++i)
                        v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                    tmem_st32(at, v);
                }
            }
            if (p.ext && t_tile + PF_TOK > L && !clear_v_tail(j, t_tile)) {
                ok = false;
                break;
            }
            DA_PH(ph, 2, ph_t);
            // P into tensor memory, over this tile's scores (every thread of the row has read its own: the
            // maximum exchange above came after the loads): this thread's 32 tokens are 16 columns of bf16 pairs
            tmem_st16(tmem_s + 128 * (j & 1) + PF_TMEM_PH + lane_sel + part * (PF_COLS / 2), phi);
            tmem_st16(tmem_s + 128 * (j & 1) + PF_TMEM_PL + lane_sel + part * (PF_COLS / 2), plo);
            tmem_st_wait();
            l_run = l_run * alpha + lsum;
            m_run = m_new;
            tc_fence_before();          // this thread's TMEM reads and writes precede the MMAs that follow
            __syncwarp();
            if (lane == 0)
                mbar_arrive(bar_p + 8 * (j & 1));     // one arrival per warp: 512 arrivals on one barrier cost hundreds of cycles
            DA_PH(ph, 3, ph_t);
        }
        uint32_t o_raw[PF_COLS];
        if (ok && ntiles > 0 && has_rows) {
            if (mbar_wait_bounded(bar_o + 8 * ((ntiles - 1) % PF_NB), (uint32_t)(((ntiles - 1) / PF_NB) & 1), abort_flag, DA_WAIT_LIMIT_NS, PF_WAIT_SLEEP_NS)) {
                tc_fence_after();
                uint32_t o_low[PF_COLS];
                tmem_ld32_issue(tmem_o + lane_base, o_raw);
                tmem_ld32_issue(tmem_o2 + lane_base, o_low);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < PF_COLS; ++i)   // the two products' sums: O = P_hi V + P_lo V
                    o_raw[i] = __float_as_uint(__uint_as_float(o_raw[i]) + __uint_as_float(o_low[i]));
            } else {
                ok = false;
            }
        }
        // the row's sum of weights is the sum of its threads' sums (all relative to m_run)
        float l_row = 0.f;
        if (ok && ntiles > 0 && has_rows) {
            // (every thread has read the last maxima before the last PV product could complete)
            float *xb = reinterpret_cast<float *>(smem + PF_OFF_XCHG);
            xb[part * 128 + r] = l_run;
            __syncwarp();
            if (lane == 0)
                mbar_arrive(bar_x);
            if (mbar_wait_bounded(bar_x, (uint32_t)(ntiles & 1), abort_flag, DA_WAIT_LIMIT_NS, PF_WAIT_SLEEP_NS)) {
#pragma unroll
                for (int q = 0; q < PF_TPR; ++q)
                    l_row += xb[q * 128 + r];
            } else {
                ok = false;
            }
        }
        if (!ok) {
            if (*abort_flag == 0) {
                *abort_flag = 1;
                report_status(p.status, 3 /* DA_DEV_TIMEOUT */, -8, (int)blockIdx.x, 0);
            }
        } else {
            if (rr < R) {
                const int outer = rr / p.G, hd = rr % p.G;   // sequence (cascade) or query token (extend)
                const bool any = ntiles > 0 && l_row > 0.f;
                // (every copy of this block was issued long before; a NaN sum of weights: NaN keys, e.g. the
                //  NaN-filled page of a widened 8-bit prefix whose page id was bad)
                const bool poisoned = *poison_s != 0 || l_row != l_row;
                const float nan = __int_as_float(0x7fc00000);
                const float inv = any ? v_mul / l_row : 0.f;
                const float lse_val = poisoned ? nan : (any ? (m_run + fast_log2(l_row)) * LN2 : -INFINITY);
                float vals[PF_COLS];
#pragma unroll
                for (int i = 0; i < PF_COLS; ++i)
                    vals[i] = poisoned ? nan : (any ? __uint_as_float(o_raw[i]) * inv : 0.f);
                const int h = g * p.G + hd;
                if (p.ext && p.splits == 1) {
                    const int64_t at = (int64_t)bseq * p.o_sb + (int64_t)outer * p.o_sq + (int64_t)h * p.o_sh + part * PF_COLS;
                    if (p.out_bf16) {
                        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + at;
#pragma unroll
                        for (int i = 0; i < PF_COLS; ++i)
                            dst[i] = __float2bfloat16_rn(vals[i]);
                    } else {
                        float *dst = reinterpret_cast<float *>(p.out) + at;
#pragma unroll
                        for (int i = 0; i < PF_COLS; ++i)
                            dst[i] = vals[i];
                    }
                    if (part == 0 && p.lse)
                        p.lse[(int64_t)bseq * p.l_sb + (int64_t)outer * p.l_sq + (int64_t)h * p.l_sh] = lse_val;
                } else {
                    const int Hq = p.Hkv * p.G;
                    const int64_t n_rows = (int64_t)p.B * (p.ext ? p.Lq : 1) * Hq;
                    const int64_t idx = p.ext ? ((int64_t)bseq * p.Lq + outer) * Hq + h : (int64_t)outer * Hq + h;
                    const int64_t at = (int64_t)split * n_rows + idx;
                    float *dst = p.pre_o + at * HEAD_DIM + part * PF_COLS;
#pragma unroll
                    for (int i = 0; i < PF_COLS; i += 4)
                        *reinterpret_cast<float4 *>(dst + i) = make_float4(vals[i], vals[i + 1], vals[i + 2], vals[i + 3]);
                    if (part == 0)
                        p.pre_lse[at] = lse_val;
                }
            }
        }
#ifdef DA_TIMELINE
        DA_PH(ph, 4, ph_t);
        if (blockIdx.x == 0 && tid == 0) {
            ph[5] = ntiles;
            ph[6] = ph_t - ph_begin;
            ph[7] = (long long)(globaltimer_ns() - ph_ns);
            DA_PH_STORE(TL_PREFIX, ph);
        }
#endif
    }
    tc_fence_before();
    __syncthreads();
    if (warp == PF_DRV)
        tmem_dealloc(tmem, PF_TMEM_COLS);
}

// =====================================================================================  8-bit prefix -> bf16
// The shared prefix of an 8-bit (E4M3) cache is widened ONCE per call into a bf16 copy that the tensor-core
// kernel above reads: every E4M3 value is a bf16 value, so the copy is exact; the per-KV-head factors stay
// out of it (PrefixParams::k_scale / v_scale).  One block per (prefix page, KV head); the copy is laid out
// [page index][head][token][128] for K, then the same for V.  A page id outside the pool sets the status
// record and fills that page with NaN, which makes every row of the result NaN (every row attends it).
struct WidenParams {
    const uint8_t *k_pages, *v_pages;     // strides in bytes: page, head, token
    int64_t k_sp, k_sh, k_st, v_sp, v_sh, v_st;
    const int32_t *block_table;           // cascade: row 0 names the prefix pages; extend: every row its sequence's
    int64_t bt_sb;
    const int32_t *seq_lens;              // extend: pages wholly past a sequence's end are left out; NULL: all pages
    int64_t sl_stride;
    __nv_bfloat16 *k_out, *v_out;         // [sequences][pages_per_seq][Hkv][P][128] each (cascade: one "sequence")
    int32_t *status;
    int32_t Hkv, P, num_pages;
    int32_t pages_per_seq;                // cascade: pages of the prefix; extend: width of the block table
    int32_t seq0;                         // sequence number of row 0 in the caller's batch (status records)
};

__global__ void __launch_bounds__(256) widen_prefix_kernel(const WidenParams p)
{
    const int g = blockIdx.x % p.Hkv;
    const int pi = (blockIdx.x / p.Hkv) % p.pages_per_seq, b = blockIdx.x / (p.Hkv * p.pages_per_seq);
    if (p.seq_lens) {
        const int L = __ldg(p.seq_lens + (int64_t)b * p.sl_stride);
        // (a length the attention kernel refuses counts as empty there too)
        if (L <= 0 || (int64_t)L > (int64_t)p.pages_per_seq * p.P || (int64_t)pi * p.P >= L)
            return;
    }
    const int page = __ldg(p.block_table + (int64_t)b * p.bt_sb + pi);
    const bool bad = (uint32_t)page >= (uint32_t)p.num_pages;
    if (bad && threadIdx.x == 0 && g == 0)
        report_status(p.status, 1 /* DA_DEV_BAD_PAGE */, b + p.seq0, pi, page);
    const int64_t slot = (int64_t)b * p.pages_per_seq + pi;   // page of the copy
    const int chunks = p.P * 8;   // 16 codes each
    for (int e = threadIdx.x; e < 2 * chunks; e += blockDim.x) {
        const int is_v = e >= chunks, c = (is_v ? e - chunks : e), tok = c >> 3, ch = c & 7;
        __nv_bfloat16 *dst = (is_v ? p.v_out : p.k_out) + ((slot * p.Hkv + g) * p.P + tok) * HEAD_DIM + ch * 16;
        uint32_t w[8];
        if (bad) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                w[i] = 0x7fc07fc0u;   // two bf16 NaN
        } else {
            const uint8_t *src = is_v ? p.v_pages + (int64_t)page * p.v_sp + (int64_t)g * p.v_sh + (int64_t)tok * p.v_st
                                      : p.k_pages + (int64_t)page * p.k_sp + (int64_t)g * p.k_sh + (int64_t)tok * p.k_st;
            const uint4 in = *reinterpret_cast<const uint4 *>(src + ch * 16);
            const uint32_t codes[4] = {in.x, in.y, in.z, in.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 lo = unpack_f16(e4m3x2_lo_to_f16x2(codes[i])), hi = unpack_f16(e4m3x2_hi_to_f16x2(codes[i]));
                w[2 * i] = pack_bf16(lo.x, lo.y);       // exact: four significant bits, exponents well inside bf16's
                w[2 * i + 1] = pack_bf16(hi.x, hi.y);
            }
        }
        reinterpret_cast<uint4 *>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<uint4 *>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
}

// =====================================================================================  cascade merge
// One warp per (b, h): fold the prefix partials (one per KV split) and the suffix result (computed
// by the plan / partition / merge kernels over tokens >= prefix into fp32 scratch) and write `out`
// and `lse`.  lse = -inf marks "no tokens" and contributes nothing.
struct CascadeMergeParams {
    const float *pre_o, *pre_lse;   // [splits][n][128], [splits][n]   with n = B * Lq * Hq
    const float *suf_o, *suf_lse;   // [n][128], [n]; may be NULL (extend: no separate suffix pass)
    const int4 *seq_info;           // the suffix pass's plan {lo, L, ..}: L == 0 marks a sequence that is empty or
                                    // was refused (shorter than the prefix) -> 0 / -inf; may be NULL
    void *out;
    int64_t o_sb, o_sq, o_sh;
    float *lse;
    int64_t l_sb, l_sq, l_sh;
    int32_t B, Lq, Hq, splits, out_bf16;
};

__global__ void __launch_bounds__(256) cascade_merge_kernel(const CascadeMergeParams p)
{
    const int warp = threadIdx.x >> 5, ln = threadIdx.x & 31, d = ln * 4;
    const int64_t idx = (int64_t)blockIdx.x * 8 + warp;
    const int64_t n = (int64_t)p.B * p.Lq * p.Hq;
    if (idx >= n)
        return;
    float M = p.suf_lse ? p.suf_lse[idx] : -INFINITY;
    for (int s = 0; s < p.splits; ++s)
        M = fmaxf(M, p.pre_lse[(int64_t)s * n + idx]);
    float den = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    auto fold = [&](float l, const float *o) {
        if (l == -INFINITY)
            return;
        const float w = __expf(l - M);
        const float4 v = *reinterpret_cast<const float4 *>(o + d);
        acc.x += w * v.x;
        acc.y += w * v.y;
        acc.z += w * v.z;
        acc.w += w * v.w;
        den += w;
    };
    if (p.suf_lse)
        fold(p.suf_lse[idx], p.suf_o + idx * HEAD_DIM);
    for (int s = 0; s < p.splits; ++s)
        fold(p.pre_lse[(int64_t)s * n + idx], p.pre_o + ((int64_t)s * n + idx) * HEAD_DIM);
    const int h = (int)(idx % p.Hq), qi = (int)((idx / p.Hq) % p.Lq), b = (int)(idx / ((int64_t)p.Hq * p.Lq));
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    float lse_val = -INFINITY;
    const bool empty = p.seq_info && p.seq_info[b].y == 0;
    if (empty) {
        // nothing to attend
    } else if (den > 0.f) {
        const float inv = 1.f / den;
        v = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        lse_val = M + __logf(den);
    } else if (den != den) {
        // a NaN partial (rows lost to a bad page id) makes the result NaN
        v = make_float4(den, den, den, den);
        lse_val = den;
    }
    const int64_t at = (int64_t)b * p.o_sb + (int64_t)qi * p.o_sq + (int64_t)h * p.o_sh + d;
    if (p.out_bf16) {
        __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(p.out) + at;
        o[0] = __float2bfloat16_rn(v.x);
        o[1] = __float2bfloat16_rn(v.y);
        o[2] = __float2bfloat16_rn(v.z);
        o[3] = __float2bfloat16_rn(v.w);
    } else {
        float *o = reinterpret_cast<float *>(p.out) + at;
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
    if (ln == 0 && p.lse)
        p.lse[(int64_t)b * p.l_sb + (int64_t)qi * p.l_sq + (int64_t)h * p.l_sh] = lse_val;
}

}  // namespace da
