// Input-layer 3x3 convolution (1, 3 or 4 input channels) on the tcgen05 tensor cores.
//
// With so few input channels the reduction of one output pixel is only 9*Cin values (27 for RGB), far
// below a 64-wide TMA box, so the im2col operand is built by the threads themselves: a "patch tile" of
// one 128-byte row per pixel holding k = tap*Cin + c for k < 9*Cin and zeros after, written straight into
// the 128-byte-swizzled shared-memory layout the MMA descriptors expect (16-byte chunk j of row r sits at
// r*128 + ((j ^ (r & 7)) << 4)).  The same tile serves both passes:
//   forward : D[pixel, cout] = patch[pixel, :] . W[cout, :]      A = patch tile (K-major), B = weights (K-major)
//   wgrad   : D[cout, k]     = sum_pixel dy[pixel, cout] * patch[pixel, k]
//                                                               A = dy tile (MN-major, by TMA), B = patch tile (MN-major)
// In the weight-gradient pass column 9*Cin of the patch tile holds 1 for every valid pixel, so the same MMA
// also produces the bias gradient (sum of dy over the pixels) in accumulator column 9*Cin.
//
// Both kernels keep several CTAs resident per SM (small tiles, 64 TMEM columns each): the gather of the
// patches is latency-bound and the CTAs hide one another's latency.  Every mbarrier wait is bounded and
// reports through the model's device status word.
#include "sb_umma.h"
#include "sb_tcgen05.cuh"

#include <cstdio>
#include <cstdlib>

namespace sb {

namespace {

constexpr int CI_THREADS = 128;

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <bool TAB>
__device__ __forceinline__ const __nv_bfloat16* image_ptr(const __nv_bfloat16* x, const PtrTab& tab, int b_per_rep, uint32_t n, size_t img_elems)
{
    if (!TAB) return x + (size_t)n * img_elems;
    const uint32_t rep = n / (uint32_t)b_per_rep;
    return (const __nv_bfloat16*)tab.p[rep] + (size_t)(n - rep * (uint32_t)b_per_rep) * img_elems;
}
// flat pixel index (< 2^31: checked by the launchers) -> column, row, image; 32-bit divisions only
__device__ __forceinline__ void pixel_coords(uint32_t P, int W, int H, int& w, int& h, uint32_t& n)
{
    const uint32_t q = P / (uint32_t)W;
    w = (int)(P - q * (uint32_t)W);
    n = q / (uint32_t)H;
    h = (int)(q - n * (uint32_t)H);
}

// k-values [k0, k0 + 8) of pixel (h, w) of image `img` as one 16-byte chunk; `ones_col` (or -1) is the k index that holds 1.
template <int CIN>
__device__ __forceinline__ uint4 patch_chunk(const __nv_bfloat16* img, int h, int w, int H, int W, int k0, int ones_col)
{
    uint32_t pk[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        uint32_t two[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int k = k0 + 2 * e + u;
            uint32_t bits = 0;
            if (k < 9 * CIN) {
                const int tap = k / CIN, c = k - tap * CIN;
                const int r3 = tap / 3, hh = h + r3 - 1, ww = w + (tap - 3 * r3) - 1;
                if (hh >= 0 && hh < H && ww >= 0 && ww < W)
                    bits = (uint32_t)__bfloat16_as_ushort(img[((size_t)hh * W + ww) * CIN + c]);
            } else if (k == ones_col) {
                bits = 0x3F80u;   // bf16 1.0
            }
            two[u] = bits;
        }
        pk[e] = two[0] | (two[1] << 16);
    }
    return make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

// Staged variant: the pixels a tile's 3x3 neighbourhoods touch are one contiguous range of the image (flat pixels
// [first - W - 1, last + W + 1], clipped to the image), so the CTA first copies that range into shared memory with
// coalesced 4-byte loads and the patch rows are gathered from there (27 two-byte global loads per pixel become ~7
// four-byte loads per thread).  `win` holds the elements from index e_start of the image on.
template <int CIN>
__device__ __forceinline__ uint4 patch_chunk_win(const __nv_bfloat16* win, long e_start, int h, int w, int H, int W, int k0, int ones_col)
{
    uint32_t pk[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        uint32_t two[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int k = k0 + 2 * e + u;
            uint32_t bits = 0;
            if (k < 9 * CIN) {
                const int tap = k / CIN, c = k - tap * CIN;
                const int r3 = tap / 3, hh = h + r3 - 1, ww = w + (tap - 3 * r3) - 1;
                if (hh >= 0 && hh < H && ww >= 0 && ww < W)
                    bits = (uint32_t)__bfloat16_as_ushort(win[((long)hh * W + ww) * CIN + c - e_start]);
            } else if (k == ones_col) {
                bits = 0x3F80u;   // bf16 1.0
            }
            two[u] = bits;
        }
        pk[e] = two[0] | (two[1] << 16);
    }
    return make_uint4(pk[0], pk[1], pk[2], pk[3]);
}
// Copies the window of `count` pixels starting at pixel p_in of the image `img` (H*W*CIN elements, an even number,
// 4-byte aligned) into `win`; returns the element index the window starts at.  Called by all CI_THREADS threads.
template <int CIN>
__device__ __forceinline__ long stage_window(const __nv_bfloat16* img, __nv_bfloat16* win, long p_in, int count, int H, int W)
{
    const long HW = (long)H * W;
    long lo = p_in - W - 1, hi = p_in + count + W + 1;
    if (lo < 0) lo = 0;
    if (hi > HW) hi = HW;
    const long e_start = (lo * CIN) & ~1L, e_end = hi * CIN;       // e_end <= H*W*CIN, which is even: whole words stay inside
    const int words = (int)((e_end - e_start + 1) / 2);
    const uint32_t* src = (const uint32_t*)(img + e_start);
    uint32_t* dst = (uint32_t*)win;
    for (int i = threadIdx.x; i < words; i += CI_THREADS) dst[i] = src[i];
    return e_start;
}
// Shared-memory bytes of the window for `count` pixels per tile; 0 = too large, gather from global memory instead.
static size_t window_bytes(int count, int W, int Cin)
{
    const size_t b = ((size_t)(count + 2 * W + 2) * Cin + 2) * 2;
    return b <= 24576 ? (b + 15) / 16 * 16 : 0;
}

// ------------------------------------------------------------------------------------------------
// Forward: persistent CTAs, one 128-pixel tile (flat pixel index) per iteration
// ------------------------------------------------------------------------------------------------
template <int CIN, bool TAB>
__global__ void __launch_bounds__(CI_THREADS)
conv_in_fwd_umma_kernel(const __grid_constant__ CUtensorMap mapY, int tma_out, const __nv_bfloat16* __restrict__ x, PtrTab tab, int b_per_rep,
                        const __nv_bfloat16* __restrict__ wt,
                        const float* __restrict__ bias, __nv_bfloat16* __restrict__ y, long npix, int H, int W, int Cout, int relu,
                        long n_tiles, uint32_t tmem_cols, uint32_t* status, int use_window)
{
    constexpr int KSTEPS = (9 * CIN + 15) / 16;      // 16-wide MMA k-steps that hold data
    constexpr int CHUNKS = 2 * KSTEPS;               // 16-byte chunks per row that hold data
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;                               // 128 rows x 128 B
    uint8_t* sB = smem + 16384;                       // Cout rows x 128 B
    float* s_bias = (float*)(sB + (size_t)Cout * 128);
    uint64_t* bar = (uint64_t*)(s_bias + Cout);
    uint32_t* tmem_slot = (uint32_t*)(bar + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    __nv_bfloat16* win = (__nv_bfloat16*)(((uintptr_t)(tmem_slot + 2) + 15) & ~(uintptr_t)15);   // input window (use_window)

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32, r = threadIdx.x;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        tmem_alloc(tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    pdl_prologue();
    // weights: row n = W[n, 0 .. 9*CIN) then zeros (only the chunks the MMA reads are written)
    for (int n = threadIdx.x; n < Cout; n += CI_THREADS) {
        const __nv_bfloat16* wr = wt + (size_t)n * 9 * CIN;
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int k = 8 * j + 2 * e;
                const uint32_t lo = k < 9 * CIN ? (uint32_t)__bfloat16_as_ushort(wr[k]) : 0u;
                const uint32_t hi = k + 1 < 9 * CIN ? (uint32_t)__bfloat16_as_ushort(wr[k + 1]) : 0u;
                pk[e] = lo | (hi << 16);
            }
            *(uint4*)(sB + n * 128 + ((j ^ (n & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        s_bias[n] = bias[n];
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t idesc = make_idesc(Cout, 0, 0);
    const size_t img_elems = (size_t)H * W * CIN;
    uint32_t phase = 0;

    const long HW = (long)H * W;
    for (long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const long P0 = tile * 128, P = P0 + r;
        const bool valid = P < npix;
        int w = 0, h = 0;
        const __nv_bfloat16* img = x;
        if (valid) {
            uint32_t n;
            pixel_coords((uint32_t)P, W, H, w, h, n);
            img = image_ptr<TAB>(x, tab, b_per_rep, n, img_elems);
        }
        // a tile that lies inside one image (uniform over the CTA) gathers from the staged window
        const uint32_t n0_img = (uint32_t)P0 / (uint32_t)HW;
        const long p_in = (long)((uint32_t)P0 - n0_img * (uint32_t)HW);
        const bool staged = use_window && p_in + 128 <= HW && P0 + 128 <= npix;
        if (tma_out) {
            // the previous tile's output was staged in sA: its TMA store must have read it before sA is rewritten
            if (threadIdx.x == 0) tma_store_wait_read();
            __syncthreads();
        }
        if (staged) {
            const __nv_bfloat16* img0 = image_ptr<TAB>(x, tab, b_per_rep, n0_img, img_elems);
            const long e_start = stage_window<CIN>(img0, win, p_in, 128, H, W);
            __syncthreads();
#pragma unroll
            for (int j = 0; j < CHUNKS; ++j)
                *(uint4*)(sA + r * 128 + ((j ^ (r & 7)) << 4)) = patch_chunk_win<CIN>(win, e_start, h, w, H, W, 8 * j, -1);
        } else {
#pragma unroll
            for (int j = 0; j < CHUNKS; ++j) {
                const uint4 v = valid ? patch_chunk<CIN>(img, h, w, H, W, 8 * j, -1) : make_uint4(0u, 0u, 0u, 0u);
                *(uint4*)(sA + r * 128 + ((j ^ (r & 7)) << 4)) = v;
            }
        }
        fence_async_smem();          // the tensor core reads shared memory through the async proxy
        __syncthreads();
        if (threadIdx.x == 0) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < KSTEPS; ++kk)
                umma_bf16(tmem_base, make_desc(smem_u32(sA) + kk * 32, 16), make_desc(smem_u32(sB) + kk * 32, 16), idesc, kk > 0 ? 1u : 0u);
            umma_commit(bar);
        }
        bool ok = true;
        if (lane == 0) ok = mbar_wait(bar, phase);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        phase ^= 1u;
        if (!ok) {
            if (lane == 0) { *abort_flag = 1; atomicMax(status, (uint32_t)DEV_TIMEOUT_EPI); }
        } else {
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
            __nv_bfloat16* yr = y + (size_t)P * Cout;
            for (int c0 = 0; c0 < Cout; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(taddr + c0, v);
                tmem_ld_wait();
                if (!valid) continue;
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float a = __uint_as_float(v[2 * j]) + s_bias[c0 + 2 * j], b = __uint_as_float(v[2 * j + 1]) + s_bias[c0 + 2 * j + 1];
                    if (relu) { if (!(a > 0.f)) a = 0.f; if (!(b > 0.f)) b = 0.f; }
                    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
                    pk[j] = *(uint32_t*)&t;
                }
                if (tma_out) {
                    // output row r = 128 bytes (64 channels), staged in the A tile's buffer (the MMA has consumed it) in
                    // the same 128-byte swizzle, so that one TMA store writes the tile's 16 KB in full lines
                    const int j0 = c0 >> 3;
                    *(uint4*)(sA + r * 128 + (((j0) ^ (r & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    *(uint4*)(sA + r * 128 + (((j0 + 1) ^ (r & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                } else {
                    ((uint4*)(yr + c0))[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    ((uint4*)(yr + c0))[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
            }
        }
        if (tma_out) fence_async_smem();
        tc_fence_before();
        __syncthreads();             // accumulator drained and A tile consumed before the next tile overwrites them
        if (*abort_flag) break;
        if (tma_out && threadIdx.x == 0) {
            tma_store_4d(&mapY, smem_u32(sA), 0, (int)P0, 0, 0);     // rows past the last pixel are clipped by the tensor map
            tma_store_commit();
        }
    }
    if (tma_out && threadIdx.x == 0) tma_store_wait_read();   // shared memory may be released once the stores have read it; the writes complete with the grid
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------------
// Weight + bias gradient: each CTA accumulates a contiguous range of 64-pixel chunks into one TMEM
// accumulator D[cout, k] and writes it as a partial buffer [Cout*9*CIN weights | Cout biases]
// ------------------------------------------------------------------------------------------------
template <int CIN, bool TAB>
__global__ void __launch_bounds__(CI_THREADS)
conv_in_wgrad_umma_kernel(const __grid_constant__ CUtensorMap mapDy, const __nv_bfloat16* __restrict__ x, PtrTab tab, int b_per_rep,
                          float* __restrict__ part, long npix, int H, int W, long stride_floats, long n_chunks, long chunks_per_cta,
                          uint32_t* status)
{
    constexpr int COUT = 64;
    constexpr int NK = 9 * CIN;                       // weight columns; column NK is the bias gradient
    constexpr int CHUNKS = (NK + 1 + 7) / 8;          // 16-byte chunks per row that hold data
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    // stage s: [dy tile: 64 pixel rows x 128 B (64 couts)] [patch tile: 64 pixel rows x 128 B]; the MMA's second
    // 64-row block of A (couts 64..127, unused) aliases the patch tile, which always holds finite values
    uint8_t* stage0 = smem;
    uint64_t* full = (uint64_t*)(smem + 2 * 16384);   // [2] dy tile landed
    uint64_t* done = full + 2;                        // [2] the MMAs that read the stage have completed
    uint64_t* fin = done + 2;                         // [1] accumulator complete
    uint32_t* tmem_slot = (uint32_t*)(fin + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const long c_begin = (long)blockIdx.x * chunks_per_cta;
    const long c_end = c_begin + chunks_per_cta < n_chunks ? c_begin + chunks_per_cta : n_chunks;
    const int n_iters = (int)(c_end - c_begin);
    if (n_iters <= 0) return;      // uniform over the CTA (the host sizes the grid so that this does not happen)

    if (threadIdx.x == 0) {
        mbar_init(&full[0], 1); mbar_init(&full[1], 1);
        mbar_init(&done[0], 1); mbar_init(&done[1], 1);
        mbar_init(fin, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        tmem_alloc(tmem_slot, 64);
        tmem_relinquish();
    }
    // the patch tile's unused chunks are zeroed once: their positions depend on the row only
    for (int e = threadIdx.x; e < 2 * 64 * 8; e += CI_THREADS) {
        const int s = e / 512, row = (e / 8) % 64, j = e % 8;
        if (j >= CHUNKS) *(uint4*)(stage0 + s * 16384 + 8192 + row * 128 + ((j ^ (row & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
    }
    pdl_prologue();
    if (threadIdx.x == 0) {
        mbar_expect_tx(&full[0], 8192u);
        tma_load_4d(&mapDy, stage0, &full[0], 0, (int)(c_begin * 64), 0, 0);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    constexpr uint32_t idesc = make_idesc(64, 1, 1);
    const size_t img_elems = (size_t)H * W * CIN;
    const int row = threadIdx.x >> 1, half = threadIdx.x & 1;     // two threads per pixel row

    // This thread's 16-byte chunks of the patch row of pixel chunk `it`, gathered into registers: the gather of chunk
    // it + 1 is issued before chunk it is stored and multiplied, so its load latency overlaps that work.
    constexpr int NJ = (CHUNKS + 1) / 2;
    auto gather = [&](int it, uint4 (&out)[NJ]) {
        const long P = (c_begin + it) * 64 + row;
        const bool valid = P < npix;
        int w = 0, h = 0;
        const __nv_bfloat16* img = x;
        if (valid) {
            uint32_t n;
            pixel_coords((uint32_t)P, W, H, w, h, n);
            img = image_ptr<TAB>(x, tab, b_per_rep, n, img_elems);
        }
#pragma unroll
        for (int jj = 0; jj < NJ; ++jj) {
            const int j = 2 * jj + half;
            out[jj] = (j < CHUNKS && valid) ? patch_chunk<CIN>(img, h, w, H, W, 8 * j, NK) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    uint4 cur[NJ], nxt[NJ];
    gather(0, cur);
#pragma unroll
    for (int jj = 0; jj < NJ; ++jj) nxt[jj] = make_uint4(0u, 0u, 0u, 0u);
    for (int it = 0; it < n_iters; ++it) {
        const int s = it & 1;
        uint8_t* sa = stage0 + s * 16384;
        uint8_t* sb = sa + 8192;
        if (it + 1 < n_iters) gather(it + 1, nxt);
        // (stage s is free: thread 0 waited for the MMAs of chunk it-2 before the barrier that ended iteration it-1)
#pragma unroll
        for (int jj = 0; jj < NJ; ++jj) {
            const int j = 2 * jj + half;
            if (j < CHUNKS) *(uint4*)(sb + row * 128 + ((j ^ (row & 7)) << 4)) = cur[jj];
        }
#pragma unroll
        for (int jj = 0; jj < NJ; ++jj) cur[jj] = nxt[jj];
        fence_async_smem();
        __syncthreads();
        if (threadIdx.x == 0) {
            if (!mbar_wait(&full[s], (uint32_t)((it / 2) & 1))) {
                *abort_flag = 1; atomicMax(status, (uint32_t)DEV_TIMEOUT_MMA);
            } else {
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16(tmem_base, make_desc(smem_u32(sa) + kk * 2048, 8192), make_desc(smem_u32(sb) + kk * 2048, 8192), idesc,
                              (it > 0 || kk > 0) ? 1u : 0u);
                umma_commit(&done[s]);
                if (it == n_iters - 1) umma_commit(fin);
                // the other stage: wait for the MMAs of chunk it-1 that read it, then fetch chunk it+1's dy tile into it
                if (it + 1 < n_iters) {
                    if (it >= 1 && !mbar_wait(&done[s ^ 1], (uint32_t)(((it - 1) / 2) & 1))) {
                        *abort_flag = 1; atomicMax(status, (uint32_t)DEV_TIMEOUT_TMA);
                    } else {
                        mbar_expect_tx(&full[s ^ 1], 8192u);
                        tma_load_4d(&mapDy, stage0 + (s ^ 1) * 16384, &full[s ^ 1], 0, (int)((c_begin + it + 1) * 64), 0, 0);
                    }
                }
            }
        }
        __syncthreads();
        if (*abort_flag) break;
    }
    __syncthreads();
    if (!*abort_flag) {
        bool ok = true;
        if (lane == 0) ok = mbar_wait(fin, 0);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) {
            if (lane == 0) { *abort_flag = 1; atomicMax(status, (uint32_t)DEV_TIMEOUT_EPI); }
        } else {
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
            const int cout = warp * 32 + lane;               // accumulator row; rows 64.. are the unused block
            float* pw = part + (size_t)blockIdx.x * stride_floats + (size_t)cout * NK;
            float* pb = part + (size_t)blockIdx.x * stride_floats + (size_t)COUT * NK + cout;
#pragma unroll
            for (int c0 = 0; c0 < 8 * CHUNKS; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(taddr + c0, v);                    // warp-collective
                tmem_ld_wait();
                if (cout < COUT) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (c0 + j < NK) pw[c0 + j] = __uint_as_float(v[j]);
                        else if (c0 + j == NK) *pb = __uint_as_float(v[j]);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 64);
    }
}

uint32_t pow2_cols(int n)
{
    uint32_t c = 32;
    while ((int)c < n) c *= 2;
    return c;
}

}  // namespace

bool conv_in_umma_supported(int Cin, int Cout) { return (Cin == 1 || Cin == 3 || Cin == 4) && Cout == 64; }

int conv_in_umma_wgrad_blocks(long npix)
{
    const long chunks = (npix + 63) / 64;
    long ctas = chunks / 4;                       // at least ~4 chunks per CTA
    if (ctas > 148 * 6) ctas = 148 * 6;           // six CTAs per SM overlap one another's gather / MMA / barrier chains (4: +15 % time)
    if (ctas < 1) ctas = 1;
    const long cpc = (chunks + ctas - 1) / ctas;
    return (int)((chunks + cpc - 1) / cpc);       // no empty trailing CTA
}

template <int CIN>
static cudaError_t launch_fwd_t(const ConvSimtArgs& a, const CUtensorMap* mapY, uint32_t* status, cudaStream_t st)
{
    const long npix = (long)a.B * a.H * a.W;
    if (npix + 128 >= (1L << 31)) return cudaErrorInvalidValue;     // the kernel's pixel arithmetic is 32-bit
    const long n_tiles = (npix + 127) / 128;
    // the staged gather needs images of an even number of elements (4-byte loads) and a window that fits
    static const bool no_window = tune("SB_CONV_IN_WINDOW", 1) == 0;
    const size_t wbytes = (!no_window && ((size_t)a.H * a.W * CIN) % 2 == 0) ? window_bytes(128, a.W, CIN) : 0;
    const size_t smem = 1024 + 16384 + (size_t)a.Cout * 128 + (size_t)a.Cout * 4 + 64 + wbytes;
    const int use_window = wbytes > 0 ? 1 : 0;
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
    const uint32_t cols = pow2_cols(a.Cout);
    // the output goes out by TMA store when the caller made a tensor map for it (64 channels: one 128-byte row per pixel)
    static const bool no_tma_out = tune("SB_CONV_IN_TMA_OUT", 1) == 0;
    const int tma_out = (mapY && a.Cout == 64 && !no_tma_out) ? 1 : 0;
    CUtensorMap dummy{};
    const CUtensorMap& my = tma_out ? *mapY : dummy;
    // persistent CTAs, as many as are resident at once (7 per SM for 64 output channels; their TMEM columns also fit:
    // 8 x 64): one CTA more per SM than fits means a second wave (measured 159 us with 7, 228 us with 8 at ImageNet size)
    long per_sm = (227L * 1024) / (long)(smem + 1024);       // shared memory (1 KB per CTA is reserved by the system)
    if (per_sm > 512 / (long)cols) per_sm = 512 / (long)cols;    // TMEM columns
    if (per_sm > 8) per_sm = 8;
    if (per_sm < 1) per_sm = 1;
    const int grid = (int)(n_tiles < 148L * per_sm ? n_tiles : 148L * per_sm);
    if (a.tab)
        return pdl_launch(conv_in_fwd_umma_kernel<CIN, true>, dim3(grid), dim3(CI_THREADS), smem, st, my, tma_out, (const __nv_bfloat16*)nullptr, tab, a.b_per_rep,
                          (const __nv_bfloat16*)a.w, a.bias, (__nv_bfloat16*)a.out, npix, a.H, a.W, a.Cout, a.relu, n_tiles, cols, status, use_window);
    return pdl_launch(conv_in_fwd_umma_kernel<CIN, false>, dim3(grid), dim3(CI_THREADS), smem, st, my, tma_out, (const __nv_bfloat16*)a.in, tab, a.b_per_rep,
                      (const __nv_bfloat16*)a.w, a.bias, (__nv_bfloat16*)a.out, npix, a.H, a.W, a.Cout, a.relu, n_tiles, cols, status, use_window);
}

cudaError_t launch_conv_in_fwd_umma(const ConvSimtArgs& a, const CUtensorMap* mapY, uint32_t* status, cudaStream_t st)
{
    switch (a.Cin) {
    case 1: return launch_fwd_t<1>(a, mapY, status, st);
    case 3: return launch_fwd_t<3>(a, mapY, status, st);
    case 4: return launch_fwd_t<4>(a, mapY, status, st);
    default: return cudaErrorInvalidValue;
    }
}

template <int CIN>
static cudaError_t launch_wgrad_t(const WgradSimtArgs& a, const CUtensorMap& mapDy, uint32_t* status, cudaStream_t st)
{
    const long npix = (long)a.B * a.H * a.W;
    if (npix + 128 >= (1L << 31)) return cudaErrorInvalidValue;     // the kernel's pixel arithmetic is 32-bit
    const long chunks = (npix + 63) / 64;
    const int grid = conv_in_umma_wgrad_blocks(npix);
    const long cpc = (chunks + grid - 1) / grid;
    const long stride = (long)a.Cout * 9 * CIN + a.Cout;
    const size_t smem = 1024 + 2 * 16384 + 128;
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
    if (a.tab)
        return pdl_launch(conv_in_wgrad_umma_kernel<CIN, true>, dim3(grid), dim3(CI_THREADS), smem, st, mapDy, (const __nv_bfloat16*)nullptr, tab,
                          a.b_per_rep, a.part, npix, a.H, a.W, stride, chunks, cpc, status);
    return pdl_launch(conv_in_wgrad_umma_kernel<CIN, false>, dim3(grid), dim3(CI_THREADS), smem, st, mapDy, (const __nv_bfloat16*)a.x, tab,
                      a.b_per_rep, a.part, npix, a.H, a.W, stride, chunks, cpc, status);
}

cudaError_t launch_conv_in_wgrad_umma(const WgradSimtArgs& a, const CUtensorMap& mapDy, uint32_t* status, cudaStream_t st)
{
    switch (a.Cin) {
    case 1: return launch_wgrad_t<1>(a, mapDy, status, st);
    case 3: return launch_wgrad_t<3>(a, mapDy, status, st);
    case 4: return launch_wgrad_t<4>(a, mapDy, status, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace sb
