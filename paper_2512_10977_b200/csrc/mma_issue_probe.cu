// Diagnostic, not part of the library: times back-to-back tcgen05.mma (kind::f16, bf16, M = 128, K = 16)
// instructions on one SM -- operands are zeros in shared / tensor memory, one thread block, one or two
// issuing warps -- and prints cycles and nanoseconds per instruction.  It answers two design questions of
// the tensor-core kernels here: what one issuing thread can sustain (the instruction holds its thread for a
// fixed time, whatever N is), and what a tcgen05 form of the decode kernels' 8- to 48-column products would
// cost per instruction.  Every wait is bounded; tensor memory is freed on every path.
//   python -m paper_2512_10977_b200.mma_probe
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#include "da_prefix.cuh"
using namespace da;

struct Cfg { int ts; int b_mn; int n; int reps; int ld_warps; int mode; };
struct Res { long long total, issue, ns; int ok; };

__device__ __forceinline__ uint32_t idesc_of(int m, int n, bool b_mn) { return umma_idesc(m, n, b_mn); }

__global__ void __launch_bounds__(192, 1) probe(Cfg c, Res *res)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint32_t tmem_base_s;
    __shared__ uint64_t bar_s, bar2_s;
    __shared__ int abort_s;
    __shared__ volatile int go_s, done_s;
    const uint32_t sb = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < 160 * 1024 / 16; i += blockDim.x)
        reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    const uint32_t bar = smem_u32(&bar_s);
    if (tid == 0) {
        abort_s = 0; go_s = 0; done_s = 0;
        mbar_init(bar, 1);
        mbar_init(smem_u32(&bar2_s), 1);
        mbar_fence_init();
    }
    if (warp == 4)
        tmem_alloc(smem_u32(&tmem_base_s), 512);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    if (warp == 4) {
        // zero the A region in TMEM (columns 256..383) so TS reads defined data: done by warps 0-3 below
    }
    if (warp < 4) {
        uint32_t z[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) z[i] = 0;
        const uint32_t lane_sel = (uint32_t)(32 * warp) << 16;
        for (int col = 0; col < 512; col += 32)
            tmem_st32(tmem + lane_sel + col, z);
        tmem_st_wait();
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    if (warp == 4 || (warp == 5 && c.mode == 2)) {
        const int second = warp == 5;
        const uint32_t mybar = second ? smem_u32(&bar2_s) : bar;
        const uint32_t d_tmem = tmem + (second ? 128 : 0);
        const uint64_t a_desc = umma_desc(sb, 16, 1024);
        const uint64_t b_desc_k = umma_desc(sb + 32768, 16, 1024);
        const uint64_t b_desc_mn = umma_desc(sb + 32768, 128 * 128, 1024);
        const uint32_t idesc = idesc_of(128, c.n, c.b_mn != 0);
        const int reps = c.mode == 2 ? c.reps / 2 : c.reps;
        long long t0 = 0, t1 = 0, t2 = 0;
        bool ok = true;
        const unsigned long long ns0 = globaltimer_ns();
        if (c.mode == 1) {
            // whole warp runs the loop; one elected lane issues
            go_s = 1;
            t0 = clock64();
            for (int r = 0; r < reps; ++r) {
                const int kk = r & 7;
                const uint64_t offa = (uint64_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
                const uint64_t bd = c.b_mn ? b_desc_mn + (uint64_t)((kk * 2048) >> 4)
                                           : b_desc_k + (uint64_t)(((kk >> 2) * (c.n * 128) + (kk & 3) * 32) >> 4);
                const uint64_t ad = a_desc + offa;
                const uint32_t acc = r > 0;
                if (c.ts)
                    asm volatile("{\n\t.reg .pred p, e;\n\tsetp.ne.b32 p, %4, 0;\n\telect.sync _|e, 0xffffffff;\n\t"
                                 "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem), "r"(tmem + 256 + kk * 8), "l"(bd), "r"(idesc), "r"(acc) : "memory");
                else
                    asm volatile("{\n\t.reg .pred p, e;\n\tsetp.ne.b32 p, %4, 0;\n\telect.sync _|e, 0xffffffff;\n\t"
                                 "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem), "l"(ad), "l"(bd), "r"(idesc), "r"(acc) : "memory");
            }
            t1 = clock64();
            if (lane == 0) umma_commit(mybar);
            __syncwarp();
            volatile int *af = &abort_s;
            ok = mbar_wait_bounded(mybar, 0u, af, 200000000ull, 0);
            t2 = clock64();
        } else if (lane == 0) {
            go_s = 1;
            t0 = clock64();
            for (int r = 0; r < reps; ++r) {
                const int kk = r & 7;
                if (c.ts) {
                    const uint64_t bd = c.b_mn ? b_desc_mn + (uint64_t)((kk * 2048) >> 4)
                                               : b_desc_k + (uint64_t)(((kk >> 2) * (c.n * 128) + (kk & 3) * 32) >> 4);
                    umma_bf16_ts(d_tmem, tmem + 256 + kk * 8, bd, idesc, r > 0);
                } else {
                    const uint64_t offa = (uint64_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
                    const uint64_t bd = c.b_mn ? b_desc_mn + (uint64_t)((kk * 2048) >> 4)
                                               : b_desc_k + (uint64_t)(((kk >> 2) * (c.n * 128) + (kk & 3) * 32) >> 4);
                    umma_bf16(d_tmem, a_desc + offa, bd, idesc, r > 0);
                }
            }
            t1 = clock64();
            umma_commit(mybar);
            volatile int *af = &abort_s;
            ok = mbar_wait_bounded(mybar, 0u, af, 200000000ull, 0);
            t2 = clock64();
        }
        if (lane == 0) {
            if (!second) done_s = 1;
            res[second].total = t2 - t0;
            res[second].issue = t1 - t0;
            res[second].ns = (long long)(globaltimer_ns() - ns0);
            res[second].ok = ok;
        }
        __syncwarp();
    } else if (warp < c.ld_warps) {
        // concurrent TMEM traffic like the softmax warps': loads of 32 columns in a loop while MMAs run
        while (!go_s) { }
        const uint32_t lane_sel = (uint32_t)(32 * warp) << 16;
        uint32_t acc = 0;
        int spins = 0;
        while (!done_s && ++spins < 2000000) {
            uint32_t v[32];
            tmem_ld32_issue(tmem + lane_sel + 384 + 32 * (spins & 3), v);
            tmem_ld_wait();
            acc += v[0] + v[31];
        }
        if (acc == 0x12345678u) res[blockIdx.x].ok = 7;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4)
        tmem_dealloc(tmem, 512);
}

int main()
{
    Res *res;
    cudaMalloc(&res, sizeof(Res) * 8);
    cudaFuncSetAttribute(probe, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    // {A from tensor memory, B MN-major, N, instructions, (unused), mode: 0 one thread issues, 1 the same inside a
    //  warp-uniform loop with elect.sync, 2 two warps issue half each into accumulators of their own}
    const Cfg cfgs[] = {
        {0, 0, 8, 256, 0, 0},   {0, 0, 16, 256, 0, 0},  {0, 0, 32, 256, 0, 0},  {0, 0, 48, 256, 0, 0},  {0, 0, 64, 256, 0, 0},
        {0, 0, 128, 256, 0, 0}, {0, 0, 192, 256, 0, 0}, {0, 0, 256, 256, 0, 0}, {0, 1, 128, 256, 0, 0}, {1, 1, 128, 256, 0, 0},
        {0, 0, 128, 256, 0, 1}, {1, 1, 128, 256, 0, 1},
        {0, 0, 16, 256, 0, 2},  {0, 0, 64, 256, 0, 2},  {0, 0, 128, 256, 0, 2}, {1, 1, 128, 256, 0, 2},
    };
    for (const Cfg &c : cfgs) {
        Res h = {0, 0, 0, 0};
        for (int rep = 0; rep < 3; ++rep) {
            probe<<<1, 192, 160 * 1024>>>(c, res);
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) { printf("CUDA error %s\n", cudaGetErrorString(e)); return 1; }
            cudaMemcpy(&h, res, sizeof h, cudaMemcpyDeviceToHost);
        }
        Res h2 = {0, 0, 0, 0};
        cudaMemcpy(&h2, res + 1, sizeof h2, cudaMemcpyDeviceToHost);
        printf("%s B %s-major N=%3d  %s : %6.1f cycles = %5.1f ns per instruction (issuing loop alone %6.1f cycles)%s\n",
               c.ts ? "A in TMEM, " : "A in smem, ", c.b_mn ? "MN" : "K ", c.n,
               c.mode == 0 ? "one issuing thread   " : (c.mode == 1 ? "one thread, elect.sync" : "two issuing warps    "),
               (double)h.total / c.reps, (double)h.ns / c.reps, (double)h.issue / (c.mode == 2 ? c.reps / 2 : c.reps),
               h.ok ? "" : "  [a wait ran out]");
    }
    return 0;
}
