// sb_conv_in_wgrad_static: weight and bias gradient of an input-layer 3x3 convolution (Cin of 1, 3
// or 4) whose scratch space is a fixed array compiled into the library, so the call needs no device
// allocation of any kind, neither by the caller (no arena) nor by the library.
//
// The model path computes the same gradient with split partial sums in the caller's arena.  This
// variant keeps the partial sums in g_scratch below: every GPU that loads the library carries those
// 2 MiB until the process exits.  All calls share the array and it keeps the last call's contents;
// nothing in it has to start at zero, because every partial buffer a launch reads was fully written
// by the same launch's first kernel.  Two calls that overlap on the GPU (different streams, or
// different host threads) would race on the array: callers serialise them.
#include "../../include/splitbrain.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdarg>
#include <cstdio>

namespace {

constexpr int STATIC_BLOCKS = 128;           // partial buffers (= thread blocks of the first kernel)
constexpr int STATIC_MAX_PER_BLOCK = 4096;   // floats per partial buffer: Cout*(9*Cin+1) must not exceed this
constexpr size_t SCRATCH_FLOATS = (size_t)STATIC_BLOCKS * STATIC_MAX_PER_BLOCK;   // 2 MiB

// In host code this name is only a handle for the runtime, not a device address: the address the
// kernels use is obtained per device with cudaGetSymbolAddress (see scratch_for_current_device).
static __device__ __align__(256) float g_scratch[SCRATCH_FLOATS];

constexpr int MAX_DEVICES = 64;
float* g_scratch_addr[MAX_DEVICES] = {nullptr};

thread_local char g_msg[256] = "";
sb_status fail(sb_status s, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_msg, sizeof(g_msg), fmt, ap);
    va_end(ap);
    return s;
}

// One-time set-up per device, with that device current: ask the runtime where g_scratch lives.
sb_status scratch_for_current_device(float** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(SB_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= MAX_DEVICES) return fail(SB_ERR_UNSUPPORTED, "device index %d out of range", dev);
    if (!g_scratch_addr[dev]) {
        float* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_scratch);
        if (e != cudaSuccess || !p) return fail(SB_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return SB_OK;
}

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Block = 64 output channels x 4 pixel lanes.  Per 64-pixel chunk the first 64 threads stage the
// 3x3xCIN input patches in shared memory; thread (k, q) then accumulates dy[pixel,k] * patch[pixel,:]
// over the pixels q, q+4, ...  Partial sums go to scratch[block][Cout*9*CIN (weights) + Cout (bias)].
template <typename T, int CIN>
__global__ void __launch_bounds__(256)
conv_in_wgrad_static_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ scratch,
                            long npix, int H, int W, int Cout, int per_block)
{
    constexpr int NJ = 9 * CIN;
    constexpr int PJ = (NJ + 3) / 4 * 4;
    __shared__ __align__(16) float s_patch[64][PJ];
    __shared__ float s_red[3][64][NJ + 1];
    const int k = threadIdx.x % 64, q = threadIdx.x / 64;
    const int k0 = blockIdx.y * 64;
    float acc[NJ], accb = 0.f;
#pragma unroll
    for (int j = 0; j < NJ; ++j) acc[j] = 0.f;
    const long nchunks = (npix + 63) / 64;
    for (long ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
        const long p0 = ch * 64;
        if (threadIdx.x < 64) {
            const long pix = p0 + threadIdx.x;
            const int w_ = (int)(pix % W);
            const long t = pix / W;
            const int h_ = (int)(t % H);
            const long n_ = t / H;
#pragma unroll
            for (int r = 0; r < 3; ++r)
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    const int hh = h_ + r - 1, ww = w_ + s - 1;
                    const bool in = pix < npix && hh >= 0 && hh < H && ww >= 0 && ww < W;
#pragma unroll
                    for (int c = 0; c < CIN; ++c)
                        s_patch[threadIdx.x][(r * 3 + s) * CIN + c] = in ? to_f(x[(((size_t)n_ * H + hh) * W + ww) * CIN + c]) : 0.f;
                }
        }
        __syncthreads();
        if (k0 + k < Cout) {
            for (int pp = q; pp < 64; pp += 4) {
                const long pix = p0 + pp;
                if (pix >= npix) break;
                const float d = to_f(dy[(size_t)pix * Cout + k0 + k]);
                accb += d;
#pragma unroll
                for (int j = 0; j < NJ; ++j) acc[j] = fmaf(d, s_patch[pp][j], acc[j]);
            }
        }
        __syncthreads();
    }
    if (q > 0) {
#pragma unroll
        for (int j = 0; j < NJ; ++j) s_red[q - 1][k][j] = acc[j];
        s_red[q - 1][k][NJ] = accb;
    }
    __syncthreads();
    if (q == 0 && k0 + k < Cout) {
        float* dst = scratch + (size_t)blockIdx.x * per_block;
#pragma unroll
        for (int j = 0; j < NJ; ++j) dst[(size_t)(k0 + k) * NJ + j] = acc[j] + s_red[0][k][j] + s_red[1][k][j] + s_red[2][k][j];
        dst[(size_t)Cout * NJ + k0 + k] = accb + s_red[0][k][NJ] + s_red[1][k][NJ] + s_red[2][k][NJ];
    }
}

// dw[i] / db[i] = sum over the partial buffers, in buffer order.
__global__ void __launch_bounds__(256)
reduce_static_kernel(const float* __restrict__ scratch, int blocks, int per_block, int n_w, float* __restrict__ dw, float* __restrict__ db)
{
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= per_block) return;
    float t = 0.f;
    for (int b = 0; b < blocks; ++b) t += scratch[(size_t)b * per_block + i];
    if (i < n_w) dw[i] = t; else db[i - n_w] = t;
}

template <typename T>
cudaError_t launch_static(const void* x, const void* dy, float* scratch, float* dw, float* db, int B, int H, int W, int Cin,
                          int Cout, cudaStream_t st)
{
    const long npix = (long)B * H * W;
    const long chunks = (npix + 63) / 64;
    const int blocks = (int)(chunks < STATIC_BLOCKS ? chunks : STATIC_BLOCKS);
    const int per_block = Cout * (9 * Cin + 1);
    dim3 grid(blocks, (Cout + 63) / 64);
    if (Cin == 1) conv_in_wgrad_static_kernel<T, 1><<<grid, 256, 0, st>>>((const T*)x, (const T*)dy, scratch, npix, H, W, Cout, per_block);
    else if (Cin == 3) conv_in_wgrad_static_kernel<T, 3><<<grid, 256, 0, st>>>((const T*)x, (const T*)dy, scratch, npix, H, W, Cout, per_block);
    else conv_in_wgrad_static_kernel<T, 4><<<grid, 256, 0, st>>>((const T*)x, (const T*)dy, scratch, npix, H, W, Cout, per_block);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    reduce_static_kernel<<<(per_block + 255) / 256, 256, 0, st>>>(scratch, blocks, per_block, Cout * 9 * Cin, dw, db);
    return cudaGetLastError();
}

}  // namespace

extern "C" sb_status sb_conv_in_wgrad_static(const void* x, const void* dy, float* dw, float* db, int32_t B, int32_t H, int32_t W,
                                              int32_t Cin, int32_t Cout, int32_t precision, void* stream)
{
    if (!x || !dy || !dw || !db) return fail(SB_ERR_INVALID_ARG, "null pointer argument");
    if (precision != SB_FP32 && precision != SB_BF16) return fail(SB_ERR_INVALID_ARG, "precision must be SB_FP32 or SB_BF16");
    if (B < 1 || H < 1 || W < 1 || Cout < 1) return fail(SB_ERR_SHAPE, "B, H, W and Cout must be positive");
    if (Cin != 1 && Cin != 3 && Cin != 4) return fail(SB_ERR_UNSUPPORTED, "Cin must be 1, 3 or 4 (got %d)", Cin);
    if ((long)Cout * (9 * Cin + 1) > STATIC_MAX_PER_BLOCK)
        return fail(SB_ERR_UNSUPPORTED, "Cout*(9*Cin+1) = %ld exceeds the built-in scratch limit of %d floats per partial buffer",
                    (long)Cout * (9 * Cin + 1), STATIC_MAX_PER_BLOCK);
    float* scratch = nullptr;
    sb_status s = scratch_for_current_device(&scratch);
    if (s != SB_OK) return s;
    cudaError_t e = precision == SB_BF16
                        ? launch_static<__nv_bfloat16>(x, dy, scratch, dw, db, B, H, W, Cin, Cout, (cudaStream_t)stream)
                        : launch_static<float>(x, dy, scratch, dw, db, B, H, W, Cin, Cout, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(SB_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
    return SB_OK;
}

extern "C" const char* sb_static_last_error(void) { return g_msg; }
