// Stand-alone timing program: how fast can one SM issue tcgen05.mma (M = 128, K = 16, bf16) when the operands
// are already in shared memory?  It compares the two ways of writing the issuing loop:
//   * a single lane inside a branch, shared-memory descriptors rebuilt from a run-time ring slot per instruction;
//   * the whole warp in lock-step, descriptor low words advanced by adds, the instruction predicated on an
//     elected lane (the form the library's kernels use: umma_bf16_lohi in sb_tcgen05.cuh).
// Each variant is run without and with a (satisfied) mbarrier wait + tcgen05.fence per four MMAs, as a ring
// consumer has.  Prints cycles per MMA (clock64) and nanoseconds per MMA (%globaltimer), one line per case.
// Every wait is bounded.  Build: python -m paper_2112_15317_b200.build_ext ; run: paper_2112_15317_b200/mma_issue_rate
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#include "sb_tcgen05.cuh"

using namespace sb;

enum { LANE_BRANCH = 0, CONVERGED_WARP = 1 };

template <int N, int PATH, bool WAIT>
__global__ void __launch_bounds__(128) issue_kernel(long long* out, int iters, int stages)
{
    extern __shared__ uint8_t raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t ready[8], drained, done;
    __shared__ uint32_t slot;
    constexpr int STAGE = 16384 + N * 128;                       // A tile + B tile of one ring slot
    for (int i = threadIdx.x; i < 2 * STAGE / 16; i += 128) ((uint4*)smem)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        for (int i = 0; i < 8; ++i) mbar_init(&ready[i], 1);
        mbar_init(&drained, 1);
        mbar_init(&done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) { tmem_alloc(&slot, 512); tmem_relinquish(); }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = slot;
    constexpr uint32_t idesc = make_idesc(N, 0, 0);
    const uint32_t sa0 = smem_u32(smem);
    long long c0 = 0, c1 = 0;
    unsigned long long g0 = 0, g1 = 0;
    // a barrier that has never completed a phase reports parity 1 as complete: waiting on ready[] with parity 1
    // returns at once, like the full barrier of a ring slot whose data has already landed
    if (PATH == LANE_BRANCH) {
        if (threadIdx.x == 0) {
            c0 = clock64(); g0 = globaltimer_ns();
            for (int it = 0; it < iters; ++it) {
                const int s = it % stages;
                if (WAIT) { if (!mbar_wait(&ready[s & 7], 1)) break; tc_fence_after(); }
                const uint32_t a = sa0 + (uint32_t)(s & 1) * STAGE, b = a + 16384;     // two physical slots suffice for timing
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16(tmem, make_desc(a + kk * 32, 16), make_desc(b + kk * 32, 16), idesc, (it > 0 || kk > 0) ? 1u : 0u);
                umma_commit(&drained);
            }
            umma_commit(&done);
            mbar_wait(&done, 0);
            c1 = clock64(); g1 = globaltimer_ns();
        }
    } else if (threadIdx.x < 32) {
        const uint64_t d0 = make_desc(sa0, 16);
        const uint32_t hi = (uint32_t)(d0 >> 32), lo0 = (uint32_t)d0;
        const uint32_t elected = elect_one() ? 1u : 0u;
        c0 = clock64(); g0 = globaltimer_ns();
        int s = 0;
        uint32_t lo = lo0;
        for (int it = 0; it < iters; ++it) {
            if (WAIT) { if (!__all_sync(0xffffffffu, mbar_wait(&ready[s & 7], 1) ? 1 : 0)) break; tc_fence_after(); }
            const uint32_t blo = lo + (16384 >> 4);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma_bf16_lohi(tmem, lo + kk * 2, hi, blo + kk * 2, hi, idesc, (it > 0 || kk > 0) ? 1u : 0u, elected);
            if (elected) umma_commit(&drained);
            __syncwarp();
            ++s; lo += (uint32_t)STAGE >> 4;
            if (s == 2) { s = 0; lo = lo0; }
        }
        if (elected) umma_commit(&done);
        __syncwarp();
        mbar_wait(&done, 0);
        c1 = clock64(); g1 = globaltimer_ns();
    }
    if (threadIdx.x == 0) {
        out[blockIdx.x] = c1 - c0;
        out[gridDim.x + blockIdx.x] = (long long)(g1 - g0);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

template <int N, int PATH, bool WAIT>
static void run(const char* name, int iters, int ctas)
{
    long long* d = nullptr;
    if (cudaMalloc(&d, (size_t)ctas * 16) != cudaSuccess) { printf("cudaMalloc failed\n"); exit(1); }
    const size_t smem = 1024 + 2 * (16384 + N * 128);
    cudaFuncSetAttribute(issue_kernel<N, PATH, WAIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    for (int rep = 0; rep < 2; ++rep) issue_kernel<N, PATH, WAIT><<<ctas, 128, smem>>>(d, iters, 4);
    const cudaError_t e = cudaDeviceSynchronize();
    long long* h = (long long*)malloc((size_t)ctas * 16);
    cudaMemcpy(h, d, (size_t)ctas * 16, cudaMemcpyDeviceToHost);
    double cyc = 0, ns = 0;
    for (int i = 0; i < ctas; ++i) { cyc += (double)h[i]; ns += (double)h[ctas + i]; }
    const double mmas = 4.0 * iters;
    printf("%-46s N=%3d: %6.1f cycles/MMA  %6.1f ns/MMA  (ideal %3d cycles)  %s\n", name, N, cyc / ctas / mmas, ns / ctas / mmas, N / 2,
           cudaGetErrorString(e));
    free(h);
    cudaFree(d);
}

int main()
{
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess || prop.major != 10) { printf("needs an sm_100 GPU\n"); return 1; }
    const int ctas = prop.multiProcessorCount, iters = 256;
    run<256, LANE_BRANCH, false>("one lane in a branch", iters, ctas);
    run<128, LANE_BRANCH, false>("one lane in a branch", iters, ctas);
    run<64, LANE_BRANCH, false>("one lane in a branch", iters, ctas);
    run<256, LANE_BRANCH, true>("one lane in a branch + wait/fence per 4", iters, ctas);
    run<128, LANE_BRANCH, true>("one lane in a branch + wait/fence per 4", iters, ctas);
    run<64, LANE_BRANCH, true>("one lane in a branch + wait/fence per 4", iters, ctas);
    run<256, CONVERGED_WARP, false>("converged warp, elected lane", iters, ctas);
    run<128, CONVERGED_WARP, false>("converged warp, elected lane", iters, ctas);
    run<64, CONVERGED_WARP, false>("converged warp, elected lane", iters, ctas);
    run<256, CONVERGED_WARP, true>("converged warp, elected lane + wait/fence per 4", iters, ctas);
    run<128, CONVERGED_WARP, true>("converged warp, elected lane + wait/fence per 4", iters, ctas);
    run<64, CONVERGED_WARP, true>("converged warp, elected lane + wait/fence per 4", iters, ctas);
    return 0;
}
