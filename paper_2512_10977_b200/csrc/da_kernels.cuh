// The three kernels behind decode_attn(): plan (split schedule), partition (page gather by TMA,
// QK^T, online fp32 softmax, PV) and merge (log-sum-exp combine).  sm_100a only.
//
// Work model.  A "tile" is TILE_T consecutive tokens starting at a multiple of TILE_T.  Sequence b
// contributes nt_b tiles (those that intersect its attended range [lo_b, L_b)) for each of its Hkv
// KV heads.  All (b, kv head, tile) units are laid out in row-major order and cut into gridDim.x
// equal contiguous ranges, one per thread block, so every block streams the same number of bytes
// whatever the mix of sequence lengths.  A block's range covers a run of (b, kv head) pairs; the
// pairs it covers completely are written straight to `out`, the (at most two) pairs it shares with
// its neighbours go to a partial slot and are combined by the merge kernel.
#pragma once
#include "da_ptx.cuh"

namespace da {

constexpr int HEAD_DIM = 128;
constexpr int NCW = 4;                      // consumer warps per block; each owns 16 tokens of a tile
constexpr int TILE_T = 16 * NCW;            // tokens per pipeline stage
constexpr int KV_BYTES = TILE_T * 256;      // a K (or V) tile: TILE_T rows of 128 bf16
constexpr int STAGE_BYTES = 2 * KV_BYTES;   // K tile followed by V tile
constexpr int NTHREADS = (NCW + 1) * 32;    // + one producer warp
constexpr int PLAN_THREADS = 1024;
constexpr int PLAN_SMEM_SEQS = 4096;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

template <int NT8>
struct PartCfg {
    static constexpr int NSTAGES = (NT8 == 1) ? 3 : 2;
    static constexpr int HEADS = NT8 * 8;                                // padded heads per KV group
    static constexpr int XBUF_BYTES = NCW * HEADS * HEAD_DIM * 4;        // cross-warp combine buffer
    static constexpr int STATS_BYTES = 2 * NCW * HEADS * 4;              // (m, l) per warp and head
    static constexpr int OFF_XBUF = NSTAGES * STAGE_BYTES;
    static constexpr int OFF_STATS = OFF_XBUF + XBUF_BYTES;
    static constexpr int OFF_BARS = OFF_STATS + STATS_BYTES;             // full[NSTAGES], empty[NSTAGES]
    static constexpr int OFF_FLAGS = OFF_BARS + 2 * NSTAGES * 8;         // abort flag
    static constexpr int SMEM_BYTES = OFF_FLAGS + 16;
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
    const int4 *block_work;   // {b, kv_head, first tile (relative), tiles} per thread block
    float *part_o;            // [2*gridDim.x][HEADS][128]
    float *part_lse;          // [2*gridDim.x][HEADS]
    int32_t *status;
    int32_t B, Hkv, G, P, box_rows, num_pages, out_bf16;
    float scale_log2;         // scale * log2(e)
};

struct PlanParams {
    const int32_t *seq_lens;
    int64_t sl_stride;
    int4 *seq_info;
    int32_t *prefix;          // [B+1] exclusive prefix of num_tiles
    int4 *block_work;
    int32_t *status;
    int32_t B, Hkv, P, window, nblocks;
    int64_t max_pages;
};

struct MergeParams {
    const int4 *seq_info;
    const int32_t *prefix;
    const float *part_o;
    const float *part_lse;
    void *out;
    int64_t o_sb, o_sh;
    float *lse;
    int64_t l_sb, l_sh;
    int32_t B, Hkv, G, heads_pad, nblocks, out_bf16;
};

__device__ __forceinline__ void report_status(int32_t *status, int code, int a, int b, int c)
{
    if (atomicCAS(status, 0, code) == 0) {
        status[1] = a;
        status[2] = b;
        status[3] = c;
    }
}

// Start of block c's range when `total` units are cut into `n` contiguous near-equal ranges.
__host__ __device__ __forceinline__ int64_t range_start(int64_t total, int n, int c)
{
    const int64_t qq = total / n, rr = total % n;
    return qq * c + (c < rr ? c : rr);
}
// The block whose range holds unit w.
__host__ __device__ __forceinline__ int range_owner(int64_t total, int n, int64_t w)
{
    const int64_t qq = total / n, rr = total % n;
    const int64_t big = rr * (qq + 1);
    return (w < big) ? (int)(w / (qq + 1)) : (int)(rr + (w - big) / qq);
}

// =====================================================================================  plan
// One block.  Per sequence: attended range, tiles, exclusive prefix of tiles; per thread block of
// the partition kernel: where its range starts.
__global__ void __launch_bounds__(PLAN_THREADS, 1) plan_kernel(PlanParams p)
{
    __shared__ int warp_tot[PLAN_THREADS / 32];
    __shared__ int running_s;
    __shared__ int prefix_s[PLAN_SMEM_SEQS + 1];   // copy of the prefix for the searches below
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0)
        running_s = 0;
    __syncthreads();

    for (int base = 0; base < p.B; base += PLAN_THREADS) {
        const int b = base + tid;
        int lo = 0, L = 0, first = 0, nt = 0;
        if (b < p.B) {
            L = p.seq_lens[(int64_t)b * p.sl_stride];
            if (L < 0 || (int64_t)L > p.max_pages * (int64_t)p.P) {
                report_status(p.status, 2 /* DA_DEV_BAD_SEQLEN */, b, 0, L);
                L = 0;
            }
            lo = (p.window > 0 && p.window < L) ? L - p.window : 0;
            if (L > 0) {
                first = lo / TILE_T;
                nt = (L - 1) / TILE_T - first + 1;
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
            int w = warp_tot[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o)
                    w += y;
            }
            warp_tot[lane] = w;   // inclusive over warps
        }
        __syncthreads();
        const int run = running_s;
        const int excl = run + (warp ? warp_tot[warp - 1] : 0) + incl - nt;
        if (b < p.B) {
            p.seq_info[b] = make_int4(lo, L, first, nt);
            p.prefix[b] = excl;
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
    if (tid == 0) {
        p.prefix[p.B] = tiles_per_head;
        if (in_smem)
            prefix_s[p.B] = tiles_per_head;
    }
    __syncthreads();   // this block's global writes are visible to itself after the barrier
    const int *prefix = in_smem ? prefix_s : p.prefix;

    const int64_t total = (int64_t)tiles_per_head * p.Hkv;
    for (int c = tid; c < p.nblocks; c += PLAN_THREADS) {
        const int64_t ws = range_start(total, p.nblocks, c);
        const int64_t we = range_start(total, p.nblocks, c + 1);
        int4 bw = make_int4(0, 0, 0, 0);
        if (we > ws) {
            const int x = (int)(ws / p.Hkv);
            // largest b with prefix[b] <= x; equal prefixes (empty sequences) resolve to the last
            int lo_i = 0, hi_i = p.B;   // invariant: prefix[lo_i] <= x < prefix[hi_i]
            while (hi_i - lo_i > 1) {
                const int mid = (lo_i + hi_i) >> 1;
                if (prefix[mid] <= x)
                    lo_i = mid;
                else
                    hi_i = mid;
            }
            const int b = lo_i;
            const int nt = prefix[b + 1] - prefix[b];
            const int64_t rem = ws - (int64_t)prefix[b] * p.Hkv;
            bw = make_int4(b, (int)(rem / nt), (int)(rem % nt), (int)(we - ws));
        }
        p.block_work[c] = bw;
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

template <int NT8>
__global__ void __launch_bounds__(NTHREADS, 2)
partition_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const PartParams p)
{
    using C = PartCfg<NT8>;
    constexpr int NSTAGES = C::NSTAGES;
    constexpr int HEADS = C::HEADS;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t smem_base = smem_u32(smem);
    float *xbuf = reinterpret_cast<float *>(smem + C::OFF_XBUF);
    float *st_m = reinterpret_cast<float *>(smem + C::OFF_STATS);
    float *st_l = st_m + NCW * HEADS;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAGS);
    const uint32_t bar_full = smem_base + C::OFF_BARS;
    const uint32_t bar_empty = bar_full + NSTAGES * 8;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if ((smem_base & 1023u) != 0) {   // the swizzle pattern is a function of the address bits
        if (tid == 0)
            report_status(p.status, 3, -1, (int)blockIdx.x, (int)smem_base);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < NSTAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, NCW);
        }
        mbar_fence_init();
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    __syncthreads();

    const int4 bw = p.block_work[blockIdx.x];
    int b = bw.x, g = bw.y, rel = bw.z, remaining = bw.w;

    if (warp == NCW) {
        // ------------------------------------------------------------------ producer warp
        // Lane -> (box, K|V).  A box is box_rows token rows (all 128 columns) of one page.
        const int nboxes = TILE_T / p.box_rows;
        const int box = lane >> 1, is_v = lane & 1;
        const bool active = lane < nboxes * 2;
        const uint32_t box_bytes = (uint32_t)p.box_rows * 256u;
        const CUtensorMap *tm = is_v ? &tm_v : &tm_k;
        uint32_t it = 0;
        bool aborted = false;

        // state of the tile whose page id is being fetched ahead
        int4 si = make_int4(0, 0, 0, 0);
        int cnt = 0, i = 0;
        auto open_pair = [&]() {   // position on the next (b, g) pair that has tiles; false at the end
            while (remaining > 0) {
                si = p.seq_info[b];
                if (si.w > 0) {
                    cnt = min(si.w - rel, remaining);
                    i = 0;
                    return true;
                }
                ++b;   // an empty sequence (only reachable with g == 0)
            }
            return false;
        };
        auto fetch_page = [&](int &page, int &row, bool &need, int &t0_out, int &g_out, int &b_out) {
            const int t0 = (si.z + rel + i) * TILE_T;
            const int tok0 = t0 + box * p.box_rows;
            need = active && tok0 < si.y && tok0 + p.box_rows > si.x;
            page = 0;
            row = tok0 % p.P;
            if (need)
                page = __ldg(p.block_table + (int64_t)b * p.bt_sb + tok0 / p.P);
            t0_out = t0;
            g_out = g;
            b_out = b;
        };
        auto advance = [&]() {   // step to the next tile of this block's range
            if (++i == cnt) {
                remaining -= cnt;
                rel = 0;
                if (++g == p.Hkv) {
                    g = 0;
                    ++b;
                }
                return open_pair();
            }
            return true;
        };

        bool have = open_pair();
        int page = 0, row = 0, t0 = 0, gg = 0, bb = 0;
        bool need = false;
        if (have)
            fetch_page(page, row, need, t0, gg, bb);
        while (have) {
            // issue the next tile's block-table read before waiting for a free stage
            int n_page = 0, n_row = 0, n_t0 = 0, n_g = 0, n_b = 0;
            bool n_need = false;
            const bool n_have = advance();
            if (n_have)
                fetch_page(n_page, n_row, n_need, n_t0, n_g, n_b);

            const int stage = it % NSTAGES;
            const uint32_t phase = (it / NSTAGES) & 1u;
            if (need && (uint32_t)page >= (uint32_t)p.num_pages) {
                report_status(p.status, 1 /* DA_DEV_BAD_PAGE */, bb, (t0 + box * p.box_rows) / p.P, page);
                need = false;   // skip the load; the rows keep whatever the stage held
            }
            const uint32_t mask = __ballot_sync(0xffffffffu, need);
            if (!mbar_wait_bounded(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) {
                aborted = true;
                break;
            }
            if (lane == 0)
                mbar_arrive_expect_tx(bar_full + 8 * stage, (uint32_t)__popc(mask) * box_bytes);
            __syncwarp();
            if (need) {
                const uint32_t dst = smem_base + stage * STAGE_BYTES + is_v * KV_BYTES + box * box_bytes;
                tma_load_5d(dst, tm, 0, row, 0, gg, page, bar_full + 8 * stage);
            }
            ++it;
            have = n_have;
            page = n_page; row = n_row; need = n_need; t0 = n_t0; gg = n_g; bb = n_b;
        }
        if (aborted) {
            // Do not leave the block while copies may still land in its shared memory: wait (bounded)
            // for the most recent phase of every stage that was filled.
            if (lane == 0) {
                *abort_flag = 1;
                report_status(p.status, 3 /* DA_DEV_TIMEOUT */, -2, (int)blockIdx.x, (int)it);
                for (uint32_t k = 0; k < (uint32_t)NSTAGES && k < it; ++k) {
                    const uint32_t j = it - 1 - k;
                    const uint32_t t_start = 0;
                    (void)t_start;
                    const uint64_t t_begin = globaltimer_ns();
                    while (!mbar_try_wait(bar_full + 8 * (j % NSTAGES), (j / NSTAGES) & 1u)) {
                        if (globaltimer_ns() - t_begin > 1000000000ull)
                            break;
                    }
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    const int r = lane >> 2, c = lane & 3;
    uint32_t it = 0;
    bool first_item = true;
    // per-lane byte offsets used by the ldmatrix address patterns
    const int k_row = 16 * warp + (lane & 7) + ((lane >> 3) & 1) * 8;   // K: matrices 1,3 are rows +8
    const int k_chunk = lane >> 4;                                      //    matrices 2,3 are chunk +1
    const int v_row = 16 * warp + (lane & 7) + (lane >> 4) * 8;         // V: matrices 2,3 are rows +8
    const int v_chunk = (lane >> 3) & 1;                                //    matrices 1,3 are chunk +1
    const uint32_t plane_bytes = (uint32_t)p.box_rows * 128u;
    const uint32_t k_off = row_offset(k_row, p.box_rows), v_off = row_offset(v_row, p.box_rows);
    const uint32_t k_sw = (uint32_t)(k_row & 7), v_sw = (uint32_t)(v_row & 7);

    while (remaining > 0) {
        const int4 si = p.seq_info[b];
        if (si.w == 0) {
            ++b;
            continue;
        }
        const int lo = si.x, L = si.y;
        const int cnt = min(si.w - rel, remaining);
        const bool whole = (cnt == si.w);

        // Q^T fragments (B operand of S^T = K Q^T): lane holds head r, dims 16kk + 2c + {0,1} (+8)
        uint32_t qf[NT8][8][2];
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            const int head = n * 8 + r;
            const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
                p.q + (int64_t)b * p.q_sb + (int64_t)(g * p.G + (head < p.G ? head : 0)) * p.q_sh);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                qf[n][kk][0] = head < p.G ? __ldg(qrow + 8 * kk + c) : 0u;
                qf[n][kk][1] = head < p.G ? __ldg(qrow + 8 * kk + 4 + c) : 0u;
            }
        }
        float m_run[NT8][2], l_run[NT8][2], o[NT8][8][4];
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
            m_run[n][0] = m_run[n][1] = -INFINITY;
            l_run[n][0] = l_run[n][1] = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                o[n][j][0] = o[n][j][1] = o[n][j][2] = o[n][j][3] = 0.f;
        }

        for (int i = 0; i < cnt; ++i, ++it) {
            const int stage = it % NSTAGES;
            const uint32_t phase = (it / NSTAGES) & 1u;
            const int a = (si.z + rel + i) * TILE_T + 16 * warp;   // first token of this warp's rows
            const int v_lo = max(a, lo), v_hi = min(a + 16, L);
            if (!mbar_wait_bounded(bar_full + 8 * stage, phase, abort_flag)) {
                // results are void from here on; keep walking so that every barrier below is still met
                if (*abort_flag == 0) {
                    *abort_flag = 1;
                    report_status(p.status, 3 /* DA_DEV_TIMEOUT */, -3, (int)blockIdx.x, (int)it);
                }
            }
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
                            const uint32_t addr = v_base + row_offset(16 * warp + rr, p.box_rows) + (ch >> 3) * plane_bytes + ((ch & 7) << 4);
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
                    pv[0] = fast_exp2(s[n][0] - m_run[n][0]);
                    pv[1] = fast_exp2(s[n][1] - m_run[n][1]);
                    pv[2] = fast_exp2(s[n][2] - m_run[n][0]);
                    pv[3] = fast_exp2(s[n][3] - m_run[n][1]);
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
                    ldmatrix_x4_trans(vf, v_base + v_off + (j >> 2) * plane_bytes + ((((2 * j + v_chunk) & 7) ^ v_sw) << 4));
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
        }

        // ---- combine the four warps' (m, l, O) and write the pair's result or partial
#pragma unroll
        for (int n = 0; n < NT8; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float l = l_run[n][e];
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                if (r == 0) {
                    st_m[warp * HEADS + n * 8 + 2 * c + e] = m_run[n][e];
                    st_l[warp * HEADS + n * 8 + 2 * c + e] = l;
                }
            }
            // xbuf[warp][head][d ^ 8*((head>>1)&3)] : conflict-free for these stores and the reads below
            float *xb = xbuf + (warp * HEADS + n * 8 + 2 * c) * HEAD_DIM;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int d0 = (16 * j + r) ^ (8 * c), d1 = (16 * j + r + 8) ^ (8 * c);
                xb[d0] = o[n][j][0];
                xb[HEAD_DIM + d0] = o[n][j][1];
                xb[d1] = o[n][j][2];
                xb[HEAD_DIM + d1] = o[n][j][3];
            }
        }
        named_barrier_sync(1, NCW * 32);
        {
            const int d = tid;   // 0..127
            const int slot = 2 * (int)blockIdx.x + (first_item ? 0 : 1);
            for (int head = 0; head < p.G; ++head) {
                float M = st_m[head];
#pragma unroll
                for (int w = 1; w < NCW; ++w)
                    M = fmaxf(M, st_m[w * HEADS + head]);
                float den = 0.f, num = 0.f;
                const int dx = d ^ (8 * ((head >> 1) & 3));
#pragma unroll
                for (int w = 0; w < NCW; ++w) {
                    const float f = fast_exp2(st_m[w * HEADS + head] - M);   // 0 for a warp that saw no token
                    den += st_l[w * HEADS + head] * f;
                    num += xbuf[(w * HEADS + head) * HEAD_DIM + dx] * f;
                }
                const float val = num / den;
                const float lse_nat = (M + fast_log2(den)) * LN2;
                if (whole) {
                    const int h = g * p.G + head;
                    if (p.out_bf16)
                        reinterpret_cast<__nv_bfloat16 *>(p.out)[(int64_t)b * p.o_sb + (int64_t)h * p.o_sh + d] =
                            __float2bfloat16_rn(val);
                    else
                        reinterpret_cast<float *>(p.out)[(int64_t)b * p.o_sb + (int64_t)h * p.o_sh + d] = val;
                    if (d == 0 && p.lse)
                        p.lse[(int64_t)b * p.l_sb + (int64_t)h * p.l_sh] = lse_nat;
                } else {
                    p.part_o[((int64_t)slot * HEADS + head) * HEAD_DIM + d] = val;
                    if (d == 0)
                        p.part_lse[(int64_t)slot * HEADS + head] = lse_nat;
                }
            }
        }
        named_barrier_sync(1, NCW * 32);

        first_item = false;
        remaining -= cnt;
        rel = 0;
        if (++g == p.Hkv) {
            g = 0;
            ++b;
        }
    }
}

// =====================================================================================  merge
// One block per (sequence, KV head); thread = (head of the group, four head_dim columns).  Pairs
// that a single thread block covered were already written by the partition kernel; empty sequences
// get out = 0 and lse = -inf; the rest are combined from their partial slots, one split at a time:
//   M' = max(M, lse_s);  acc = acc * exp(M - M') + exp(lse_s - M') * O_s;  den likewise;
//   out = acc / den;  lse = M + ln den.
constexpr int MERGE_LANES = HEAD_DIM / 4;

__global__ void __launch_bounds__(16 * MERGE_LANES) merge_kernel(const MergeParams p)
{
    const int b = blockIdx.x / p.Hkv, g = blockIdx.x % p.Hkv;
    const int head = threadIdx.x / MERGE_LANES, d = (threadIdx.x % MERGE_LANES) * 4;
    if (head >= p.G)
        return;
    const int4 si = p.seq_info[b];
    const int tiles_before = p.prefix[b], tiles_all = p.prefix[p.B];
    const int nt = si.w;
    const int h = g * p.G + head;

    auto store = [&](float4 v, float lse_val) {
        const int64_t at = (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + d;
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
        if (d == 0 && p.lse)
            p.lse[(int64_t)b * p.l_sb + (int64_t)h * p.l_sh] = lse_val;
    };

    if (nt == 0) {
        store(make_float4(0.f, 0.f, 0.f, 0.f), -INFINITY);
        return;
    }
    const int64_t total = (int64_t)tiles_all * p.Hkv;
    const int64_t w0 = (int64_t)tiles_before * p.Hkv + (int64_t)g * nt;
    const int c_first = range_owner(total, p.nblocks, w0);
    const int c_last = range_owner(total, p.nblocks, w0 + nt - 1);
    if (c_first == c_last)
        return;
    // the pair is the first item of every block but possibly c_first, where it is the first item
    // only if that block's range starts exactly at the pair
    const int slot_first = 2 * c_first + (range_start(total, p.nblocks, c_first) == w0 ? 0 : 1);
    float M = -INFINITY, den = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int cc = c_first; cc <= c_last; ++cc) {
        const int slot = (cc == c_first) ? slot_first : 2 * cc;
        const float l = p.part_lse[(int64_t)slot * p.heads_pad + head];
        const float4 o = *reinterpret_cast<const float4 *>(p.part_o + ((int64_t)slot * p.heads_pad + head) * HEAD_DIM + d);
        const float m_new = fmaxf(M, l);
        const float sc = (M == -INFINITY) ? 0.f : __expf(M - m_new);
        const float w = __expf(l - m_new);
        acc.x = acc.x * sc + w * o.x;
        acc.y = acc.y * sc + w * o.y;
        acc.z = acc.z * sc + w * o.z;
        acc.w = acc.w * sc + w * o.w;
        den = den * sc + w;
        M = m_new;
    }
    const float inv = 1.f / den;
    store(make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv), M + __logf(den));
}

}  // namespace da
