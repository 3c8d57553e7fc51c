// CUDA-core kernels of the SplitBrain training step for sm_100a.
//
//  * bandwidth-bound steps that every mode uses: 2x2 max-pool forward/backward, softmax
//    cross-entropy, SGD with momentum, column sums (bias gradients) and split reductions;
//  * float-accumulating FFMA versions of the contractions (3x3 conv forward / dgrad / wgrad and
//    a strided GEMM for the sharded FC layers).  They are the float mode, serve layers whose
//    channel count does not fit the tensor-core tiles (e.g. the 3-channel input layer), and are
//    the on-device cross-check of the tcgen05 kernels.
//
// T is the activation dtype (float or __nv_bfloat16); all sums are carried in float.
#include "sb_internal.h"

namespace sb {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// store 8 consecutive values (pointer 16-byte aligned for bf16, 32-byte for float)
__device__ __forceinline__ void store8(float* p, const float (&v)[8])
{
    ((float4*)p)[0] = make_float4(v[0], v[1], v[2], v[3]);
    ((float4*)p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8])
{
    uint32_t pk[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
        pk[j] = *(uint32_t*)&t;
    }
    *(uint4*)p = make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

static inline int cdiv(long a, long b) { return (int)((a + b - 1) / b); }

// =============================================================================================
// 3x3 convolution, forward and data gradient (direct, tiled through shared memory).
//   forward: y[n,h,w,o] = act(bias[o] + sum_{r,s,i} x[n,h+r-1,w+s-1,i] * W[o,r,s,i])
//   dgrad  : dx[n,h,w,o] = mask * sum_{r,s,i} dy[n,h-r+1,w-s+1,i] * W[i,r,s,o]
// Block: 8x8 output pixels x 32 output channels, 128 threads, 4 pixels x 4 channels per thread.
// =============================================================================================
constexpr int CV_TP = 8, CV_TC = 32, CV_CK = 16;

template <typename T, bool DGRAD, bool TAB>
__global__ void __launch_bounds__(128)
conv3x3_simt_kernel(const T* __restrict__ in, PtrTab tab, int b_per_rep, const T* __restrict__ wt,
                    const float* __restrict__ bias, T* __restrict__ out, const T* __restrict__ mask_ref,
                    int H, int W, int Cred, int Cres, int Cin, int relu)
{
    pdl_prologue();
    __shared__ float s_in[CV_TP + 2][CV_TP + 2][CV_CK + 1];
    __shared__ float s_w[9][CV_CK][CV_TC];
    const int tiles_w = (W + CV_TP - 1) / CV_TP;
    const int h0 = (blockIdx.x / tiles_w) * CV_TP, w0 = (blockIdx.x % tiles_w) * CV_TP;
    const int n = blockIdx.y;
    const int o0 = blockIdx.z * CV_TC;
    const int tid = threadIdx.x;
    const int cg = tid / 16, pg = tid % 16;
    const int prow = pg / 2, pcol = (pg % 2) * 4;
    const T* img = TAB ? (const T*)tab.p[n / b_per_rep] + (size_t)(n % b_per_rep) * H * W * Cred
                       : in + (size_t)n * H * W * Cred;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int c0 = 0; c0 < Cred; c0 += CV_CK) {
        for (int e = tid; e < (CV_TP + 2) * (CV_TP + 2) * CV_CK; e += 128) {
            int c = e % CV_CK, q = e / CV_CK;
            int ww = q % (CV_TP + 2), hh = q / (CV_TP + 2);
            int gh = h0 + hh - 1, gw = w0 + ww - 1, gc = c0 + c;
            float v = 0.f;
            if (gh >= 0 && gh < H && gw >= 0 && gw < W && gc < Cred) v = ldf(img + ((size_t)gh * W + gw) * Cred + gc);
            s_in[hh][ww][c] = v;
        }
        for (int e = tid; e < 9 * CV_CK * CV_TC; e += 128) {
            int o = e % CV_TC, q = e / CV_TC;
            int c = q % CV_CK, t = q / CV_CK;
            int go = o0 + o, gc = c0 + c;
            float v = 0.f;
            if (go < Cres && gc < Cred) {
                // weight tensor is [Cout][9][Cin]; forward: out=o, in=c ; dgrad: out index is Cin, reduce index is Cout
                size_t wi = DGRAD ? (((size_t)gc * 9 + t) * Cin + go) : (((size_t)go * 9 + t) * Cin + gc);
                v = ldf(wt + wi);
            }
            s_w[t][c][o] = v;
        }
        __syncthreads();
#pragma unroll
        for (int t = 0; t < 9; ++t) {
            const int r = t / 3, s = t % 3;
            const int dr = DGRAD ? (2 - r) : r, ds = DGRAD ? (2 - s) : s;
#pragma unroll 4
            for (int c = 0; c < CV_CK; ++c) {
                float xv[4], wv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) xv[i] = s_in[prow + dr][pcol + i + ds][c];
#pragma unroll
                for (int j = 0; j < 4; ++j) wv[j] = s_w[t][c][cg * 4 + j];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xv[i], wv[j], acc[i][j]);
            }
        }
        __syncthreads();
    }
    const int gh = h0 + prow;
    if (gh >= H) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int gw = w0 + pcol + i;
        if (gw >= W) continue;
        size_t pix = ((size_t)n * H + gh) * W + gw;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int go = o0 + cg * 4 + j;
            if (go >= Cres) continue;
            float v = acc[i][j];
            if (!DGRAD) {
                v += bias[go];
                if (relu && !(v > 0.f)) v = 0.f;
            } else if (mask_ref != nullptr) {
                if (!(ldf(mask_ref + pix * Cres + go) > 0.f)) v = 0.f;
            }
            stf(out + pix * Cres + go, v);
        }
    }
}

template <typename T>
static cudaError_t launch_conv_simt_t(const ConvSimtArgs& a, cudaStream_t st)
{
    const int Cred = a.dgrad ? a.Cout : a.Cin, Cres = a.dgrad ? a.Cin : a.Cout;
    dim3 grid(cdiv(a.H, CV_TP) * cdiv(a.W, CV_TP), a.B, cdiv(Cres, CV_TC));
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
    if (a.dgrad)
        SB_LAUNCH((conv3x3_simt_kernel<T, true, false>), grid, 128, 0, st, (const T*)a.in, tab, a.b_per_rep, (const T*)a.w, a.bias,
                                                                  (T*)a.out, (const T*)a.mask_ref, a.H, a.W, Cred, Cres, a.Cin, 0);
    else if (a.tab)
        SB_LAUNCH((conv3x3_simt_kernel<T, false, true>), grid, 128, 0, st, nullptr, tab, a.b_per_rep, (const T*)a.w, a.bias,
                                                                  (T*)a.out, nullptr, a.H, a.W, Cred, Cres, a.Cin, a.relu);
    else
        SB_LAUNCH((conv3x3_simt_kernel<T, false, false>), grid, 128, 0, st, (const T*)a.in, tab, a.b_per_rep, (const T*)a.w, a.bias,
                                                                   (T*)a.out, nullptr, a.H, a.W, Cred, Cres, a.Cin, a.relu);
    return cudaGetLastError();
}
cudaError_t launch_conv_simt(const ConvSimtArgs& a, bool bf16, cudaStream_t st)
{
    return bf16 ? launch_conv_simt_t<__nv_bfloat16>(a, st) : launch_conv_simt_t<float>(a, st);
}

// =============================================================================================
// 3x3 convolution weight gradient: part[s][k,t,c] = sum over split s's pixels of
// dy[pix,k] * x[pix shifted by tap t, c].  Block: 32 (k) x 32 (c) outputs of one tap, 256 threads.
// =============================================================================================
template <typename T, bool TAB>
__global__ void __launch_bounds__(256)
conv3x3_wgrad_simt_kernel(const T* __restrict__ x, PtrTab tab, int b_per_rep, const T* __restrict__ dy,
                          float* __restrict__ part, int B, int H, int W, int Cin, int Cout, int splits)
{
    pdl_prologue();
    __shared__ float s_dy[32][33];
    __shared__ float s_x[32][33];
    const int k0 = blockIdx.x * 32;
    const int ctiles = (Cin + 31) / 32;
    const int c0 = (blockIdx.y % ctiles) * 32, t = blockIdx.y / ctiles;
    const int r = t / 3, s = t % 3;
    const int sp = blockIdx.z;
    const int imgs = B / splits;
    const long pix_begin = (long)sp * imgs * H * W, pix_end = pix_begin + (long)imgs * H * W;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    for (long p0 = pix_begin; p0 < pix_end; p0 += 32) {
        for (int e = tid; e < 32 * 32; e += 256) {
            int j = e % 32, pp = e / 32;
            long pix = p0 + pp;
            float vd = 0.f, vx = 0.f;
            if (pix < pix_end) {
                if (k0 + j < Cout) vd = ldf(dy + pix * Cout + k0 + j);
                int w_ = (int)(pix % W);
                long q = pix / W;
                int h_ = (int)(q % H), n_ = (int)(q / H);
                int hh = h_ + r - 1, ww = w_ + s - 1;
                if (hh >= 0 && hh < H && ww >= 0 && ww < W && c0 + j < Cin) {
                    const T* img = TAB ? (const T*)tab.p[n_ / b_per_rep] + (size_t)(n_ % b_per_rep) * H * W * Cin
                                       : x + (size_t)n_ * H * W * Cin;
                    vx = ldf(img + ((size_t)hh * W + ww) * Cin + c0 + j);
                }
            }
            s_dy[pp][j] = vd;
            s_x[pp][j] = vx;
        }
        __syncthreads();
#pragma unroll 8
        for (int pp = 0; pp < 32; ++pp) {
            float a0 = s_dy[pp][ty * 2], a1 = s_dy[pp][ty * 2 + 1];
            float b0 = s_x[pp][tx * 2], b1 = s_x[pp][tx * 2 + 1];
            acc[0][0] = fmaf(a0, b0, acc[0][0]);
            acc[0][1] = fmaf(a0, b1, acc[0][1]);
            acc[1][0] = fmaf(a1, b0, acc[1][0]);
            acc[1][1] = fmaf(a1, b1, acc[1][1]);
        }
        __syncthreads();
    }
    float* dst = part + (size_t)sp * Cout * 9 * Cin;
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            int k = k0 + ty * 2 + i, c = c0 + tx * 2 + j;
            if (k < Cout && c < Cin) dst[((size_t)k * 9 + t) * Cin + c] = acc[i][j];
        }
}

cudaError_t launch_wgrad_simt(const WgradSimtArgs& a, bool bf16, cudaStream_t st)
{
    dim3 grid(cdiv(a.Cout, 32), cdiv(a.Cin, 32) * 9, a.splits);
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
#define SB_WG(T, TABF)                                                                                         \
    SB_LAUNCH((conv3x3_wgrad_simt_kernel<T, TABF>), grid, 256, 0, st, (const T*)a.x, tab, a.b_per_rep, (const T*)a.dy, \
                                                            a.part, a.B, a.H, a.W, a.Cin, a.Cout, a.splits)
    if (bf16) { if (a.tab) SB_WG(__nv_bfloat16, true); else SB_WG(__nv_bfloat16, false); }
    else      { if (a.tab) SB_WG(float, true); else SB_WG(float, false); }
#undef SB_WG
    return cudaGetLastError();
}

// =============================================================================================
// Column sums (bias gradients) and the reduction of split partial sums.
// =============================================================================================
template <typename T>
__global__ void __launch_bounds__(256)
colsum_kernel(const T* __restrict__ in, float* __restrict__ part, int M, int N, int splits)
{
    pdl_prologue();
    __shared__ float s[8][33];
    const int col = blockIdx.x * 32 + threadIdx.x % 32;
    const int lane_row = threadIdx.x / 32;
    const int sp = blockIdx.y;
    const long rows = M / splits, r0 = (long)sp * rows;
    float acc = 0.f;
    if (col < N)
        for (long r = lane_row; r < rows; r += 8) acc += ldf(in + (r0 + r) * N + col);
    s[lane_row][threadIdx.x % 32] = acc;
    __syncthreads();
    if (lane_row == 0 && col < N) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) t += s[i][threadIdx.x];
        part[(size_t)sp * N + col] = t;
    }
}
// bf16, N a multiple of 8: a thread owns 8 adjacent columns (one 16-byte load per row), 8 row lanes per block take rows
// r0 + lane_row, + 8, ... with four independent loads in flight and are combined in lane order (deterministic).
__global__ void __launch_bounds__(256)
colsum_vec_kernel(const uint4* __restrict__ in, float* __restrict__ part, int M, int N, int splits)
{
    pdl_prologue();
    __shared__ float s[8][32][9];
    const int nv = N / 8;
    const int vc = blockIdx.x * 32 + threadIdx.x % 32;
    const int lane_row = threadIdx.x / 32;
    const int sp = blockIdx.y;
    const long rows = (M + splits - 1) / splits, r0 = (long)sp * rows;
    const long r1 = r0 + rows < M ? r0 + rows : M;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (vc < nv) {
        long r = r0 + lane_row;
        for (; r + 24 < r1; r += 32) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = __ldg(in + (r + 8 * u) * nv + vc);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const __nv_bfloat16* h = (const __nv_bfloat16*)&v[u];
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[j] += __bfloat162float(h[j]);
            }
        }
        for (; r < r1; r += 8) {
            const uint4 v = __ldg(in + r * nv + vc);
            const __nv_bfloat16* h = (const __nv_bfloat16*)&v;
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += __bfloat162float(h[j]);
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) s[lane_row][threadIdx.x % 32][j] = acc[j];
    __syncthreads();
    if (lane_row == 0 && vc < nv) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float t = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) t += s[i][threadIdx.x][j];
            part[(size_t)sp * N + vc * 8 + j] = t;
        }
    }
}
cudaError_t launch_colsum(const void* in, bool bf16, float* part, int M, int N, int splits, cudaStream_t st)
{
    if (bf16 && N % 8 == 0 && (((uintptr_t)in) & 15) == 0) {
        dim3 vgrid(cdiv(N / 8, 32), splits);
        SB_LAUNCH((colsum_vec_kernel), vgrid, 256, 0, st, (const uint4*)in, part, M, N, splits);
        return cudaGetLastError();
    }
    dim3 grid(cdiv(N, 32), splits);
    if (bf16) SB_LAUNCH((colsum_kernel<__nv_bfloat16>), grid, 256, 0, st, (const __nv_bfloat16*)in, part, M, N, splits);
    else SB_LAUNCH((colsum_kernel<float>), grid, 256, 0, st, (const float*)in, part, M, N, splits);
    return cudaGetLastError();
}

__global__ void __launch_bounds__(256)
reduce_partials_kernel(const float* __restrict__ part, size_t stride, float* __restrict__ out, size_t n, int splits)
{
    pdl_prologue();
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float t = 0.f;
        for (int s = 0; s < splits; ++s) t += part[(size_t)s * stride + i];
        out[i] = t;
    }
}
__global__ void __launch_bounds__(256)
reduce_partials4_kernel(const float4* __restrict__ part, size_t stride4, float4* __restrict__ out, size_t n4, int splits)
{
    pdl_prologue();
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        // loads go out in batches of 8 (independent, all in flight together); the additions keep split order
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s0 = 0; s0 < splits; s0 += 8) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                v[u] = (s0 + u < splits) ? __ldg(part + (size_t)(s0 + u) * stride4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 8; ++u) { t.x += v[u].x; t.y += v[u].y; t.z += v[u].z; t.w += v[u].w; }
        }
        out[i] = t;
    }
}
// Many splits, few elements: 32 elements per block, LANES lanes share the splits of each element (lane l takes
// splits l, l + LANES, ... in order, four loads in flight) and are combined in lane order: a fixed order, so the
// result is deterministic.  LANES = 8, or 32 from 128 splits on (the input layer's per-block partial sums).
template <int LANES>
__device__ __forceinline__ float many_lane_sum(const float* __restrict__ part, size_t stride, size_t i, int lane, int splits)
{
    float t = 0.f;
    int sp = lane;
    for (; sp + 3 * LANES < splits; sp += 4 * LANES) {
        const float a = part[(size_t)sp * stride + i], b = part[(size_t)(sp + LANES) * stride + i];
        const float c = part[(size_t)(sp + 2 * LANES) * stride + i], d = part[(size_t)(sp + 3 * LANES) * stride + i];
        t += a; t += b; t += c; t += d;
    }
    for (; sp < splits; sp += LANES) t += part[(size_t)sp * stride + i];
    return t;
}
template <int LANES>
__global__ void __launch_bounds__(32 * LANES)
reduce_partials_many_kernel(const float* __restrict__ part, size_t stride, float* __restrict__ out, size_t n, int splits)
{
    pdl_prologue();
    __shared__ float s[LANES][33];
    const int e = threadIdx.x % 32, lane = threadIdx.x / 32;
    const size_t i = blockIdx.x * 32ull + e;
    s[lane][e] = i < n ? many_lane_sum<LANES>(part, stride, i, lane, splits) : 0.f;
    __syncthreads();
    if (lane == 0 && i < n) {
        float r = 0.f;
#pragma unroll
        for (int j = 0; j < LANES; ++j) r += s[j][e];
        out[i] = r;
    }
}
cudaError_t launch_reduce_partials(const float* part, size_t stride, float* out, size_t n, int splits, cudaStream_t st)
{
    if (splits >= 128 && n <= (1u << 20)) {
        SB_LAUNCH((reduce_partials_many_kernel<32>), cdiv((long)n, 32), 1024, 0, st, part, stride, out, n, splits);
    } else if (splits >= 32 && n <= (1u << 20)) {
        SB_LAUNCH((reduce_partials_many_kernel<8>), cdiv((long)n, 32), 256, 0, st, part, stride, out, n, splits);
    } else if (n % 4 == 0 && stride % 4 == 0 && (((uintptr_t)part | (uintptr_t)out) & 15) == 0) {
        int blocks = cdiv((long)(n / 4), 256);
        if (blocks > 148 * 8) blocks = 148 * 8;
        SB_LAUNCH((reduce_partials4_kernel), blocks, 256, 0, st, (const float4*)part, stride / 4, (float4*)out, n / 4, splits);
    } else {
        int blocks = cdiv((long)n, 256);
        if (blocks > 148 * 8) blocks = 148 * 8;
        SB_LAUNCH((reduce_partials_kernel), blocks, 256, 0, st, part, stride, out, n, splits);
    }
    return cudaGetLastError();
}

// =============================================================================================
// Split-reduction epilogue of the tensor-core GEMMs: out = epi(sum_s part[s]) with the splits added in
// order; epi = bias + ReLU (-> bf16 or float) or the ReLU mask (-> bf16).  Four columns per thread.
// =============================================================================================
template <int EPI>
__global__ void __launch_bounds__(256)
splitk_epilogue_kernel(const float* __restrict__ part, size_t split_stride, int splits, size_t n4, int N,
                       const float* __restrict__ bias, int relu, const __nv_bfloat16* __restrict__ ref,
                       void* __restrict__ out, int out_f32)
{
    pdl_prologue();
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const size_t e = i * 4;
        // loads go out in batches of 8 (independent, all in flight together); the additions keep split order
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s0 = 0; s0 < splits; s0 += 8) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                v[u] = (s0 + u < splits) ? __ldg((const float4*)(part + (size_t)(s0 + u) * split_stride + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 8; ++u) { t.x += v[u].x; t.y += v[u].y; t.z += v[u].z; t.w += v[u].w; }
        }
        if (EPI == EPI_BIAS_ACT) {
            const float4 b = *(const float4*)(bias + (e % (size_t)N));
            t.x += b.x; t.y += b.y; t.z += b.z; t.w += b.w;
            if (relu) {
                if (!(t.x > 0.f)) t.x = 0.f;
                if (!(t.y > 0.f)) t.y = 0.f;
                if (!(t.z > 0.f)) t.z = 0.f;
                if (!(t.w > 0.f)) t.w = 0.f;
            }
        } else if (ref != nullptr) {
            const uint2 r = *(const uint2*)(ref + e);
            const __nv_bfloat16* rb = (const __nv_bfloat16*)&r;
            if (!(__bfloat162float(rb[0]) > 0.f)) t.x = 0.f;
            if (!(__bfloat162float(rb[1]) > 0.f)) t.y = 0.f;
            if (!(__bfloat162float(rb[2]) > 0.f)) t.z = 0.f;
            if (!(__bfloat162float(rb[3]) > 0.f)) t.w = 0.f;
        }
        if (out_f32) {
            *(float4*)((float*)out + e) = t;
        } else {
            __nv_bfloat162 lo = __floats2bfloat162_rn(t.x, t.y), hi = __floats2bfloat162_rn(t.z, t.w);
            uint2 pk;
            pk.x = *(uint32_t*)&lo;
            pk.y = *(uint32_t*)&hi;
            *(uint2*)((__nv_bfloat16*)out + e) = pk;
        }
    }
}
cudaError_t launch_splitk_epilogue(const SplitKEpiArgs& a, cudaStream_t st)
{
    if (a.N % 4 != 0) return cudaErrorInvalidValue;
    const size_t n4 = (size_t)a.rows * a.N / 4;
    int blocks = cdiv((long)n4, 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (a.epi == EPI_BIAS_ACT)
        SB_LAUNCH((splitk_epilogue_kernel<EPI_BIAS_ACT>), blocks, 256, 0, st, a.part, a.split_stride, a.splits, n4, a.N, a.bias, a.relu, nullptr, a.out, a.out_f32);
    else
        SB_LAUNCH((splitk_epilogue_kernel<EPI_MASK>), blocks, 256, 0, st, a.part, a.split_stride, a.splits, n4, a.N, nullptr, 0, (const __nv_bfloat16*)a.ref, a.out, 0);
    return cudaGetLastError();
}

// =============================================================================================
// 2x2 max-pool, stride 2.  One thread per pooled pixel and VEC channels (16-byte accesses when the
// channel count allows).  Ties go to the first maximum in scan order (0,0),(0,1),(1,0),(1,1).
// =============================================================================================
template <typename T, int VEC> struct VecT;
template <> struct VecT<float, 4> { typedef float4 type; };
template <> struct VecT<float, 1> { typedef float type; };
template <> struct VecT<__nv_bfloat16, 8> { typedef uint4 type; };
template <> struct VecT<__nv_bfloat16, 1> { typedef __nv_bfloat16 type; };
template <int VEC> struct VecU8;
template <> struct VecU8<8> { typedef uint2 type; };
template <> struct VecU8<4> { typedef uint32_t type; };
template <> struct VecU8<1> { typedef uint8_t type; };

template <typename T, int VEC>
__global__ void __launch_bounds__(256)
maxpool_fwd_kernel(const T* __restrict__ x, T* __restrict__ p, uint8_t* __restrict__ idx, long total, int H, int W, int C)
{
    pdl_prologue();
    typedef typename VecT<T, VEC>::type V;
    typedef typename VecU8<VEC>::type VI;
    const int Ho = H / 2, Wo = W / 2, Cv = C / VEC;
    for (long e = blockIdx.x * (long)blockDim.x + threadIdx.x; e < total; e += (long)gridDim.x * blockDim.x) {
        int cv = (int)(e % Cv);
        long q = e / Cv;
        int wo = (int)(q % Wo);
        q /= Wo;
        int ho = (int)(q % Ho);
        long n = q / Ho;
        const T* base = x + (((size_t)n * H + 2 * ho) * W + 2 * wo) * C + (size_t)cv * VEC;
        V v[4];
        v[0] = *(const V*)(base);
        v[1] = *(const V*)(base + C);
        v[2] = *(const V*)(base + (size_t)W * C);
        v[3] = *(const V*)(base + (size_t)W * C + C);
        V outv;
        VI outi;
        T* ov = (T*)&outv;
        uint8_t* oi = (uint8_t*)&outi;
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            T bestv = ((const T*)&v[0])[k];
            float best = ldf(&bestv);
            int bi = 0;
#pragma unroll
            for (int j = 1; j < 4; ++j) {
                T cand = ((const T*)&v[j])[k];
                float f = ldf(&cand);
                if (f > best) { best = f; bi = j; bestv = cand; }
            }
            ov[k] = bestv;
            oi[k] = (uint8_t)bi;
        }
        size_t o = (size_t)e * VEC;
        *(V*)(p + o) = outv;
        *(VI*)(idx + o) = outi;
    }
}

template <typename T, int VEC>
__global__ void __launch_bounds__(256)
maxpool_bwd_kernel(const T* __restrict__ dp, const uint8_t* __restrict__ idx, const T* __restrict__ p,
                   T* __restrict__ dx, long total, int H, int W, int C)
{
    pdl_prologue();
    typedef typename VecT<T, VEC>::type V;
    typedef typename VecU8<VEC>::type VI;
    const int Ho = H / 2, Wo = W / 2, Cv = C / VEC;
    for (long e = blockIdx.x * (long)blockDim.x + threadIdx.x; e < total; e += (long)gridDim.x * blockDim.x) {
        int cv = (int)(e % Cv);
        long q = e / Cv;
        int wo = (int)(q % Wo);
        q /= Wo;
        int ho = (int)(q % Ho);
        long n = q / Ho;
        size_t o = (size_t)e * VEC;
        V g = *(const V*)(dp + o);
        VI iv = *(const VI*)(idx + o);
        const uint8_t* ii = (const uint8_t*)&iv;
        T* gp = (T*)&g;
        if (p != nullptr) {
            V pv = *(const V*)(p + o);
#pragma unroll
            for (int k = 0; k < VEC; ++k)
                if (!(ldf((const T*)&pv + k) > 0.f)) stf(gp + k, 0.f);
        }
        T* base = dx + (((size_t)n * H + 2 * ho) * W + 2 * wo) * C + (size_t)cv * VEC;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            V ov;
            T* op = (T*)&ov;
#pragma unroll
            for (int k = 0; k < VEC; ++k) {
                if (ii[k] == j) op[k] = gp[k]; else stf(op + k, 0.f);
            }
            *(V*)(base + (size_t)(j >> 1) * W * C + (size_t)(j & 1) * C) = ov;
        }
    }
}

static int ew_blocks(long total)
{
    long b = (total + 255) / 256;
    long cap = 148L * 16;
    return (int)(b < cap ? (b < 1 ? 1 : b) : cap);
}

cudaError_t launch_pool_fwd(const PoolArgs& a, bool bf16, cudaStream_t st)
{
    long pooled = (long)a.B * (a.H / 2) * (a.W / 2) * a.C;
    if (bf16) {
        if (a.C % 8 == 0) SB_LAUNCH((maxpool_fwd_kernel<__nv_bfloat16, 8>), ew_blocks(pooled / 8), 256, 0, st, (const __nv_bfloat16*)a.x, (__nv_bfloat16*)a.p, a.idx, pooled / 8, a.H, a.W, a.C);
        else SB_LAUNCH((maxpool_fwd_kernel<__nv_bfloat16, 1>), ew_blocks(pooled), 256, 0, st, (const __nv_bfloat16*)a.x, (__nv_bfloat16*)a.p, a.idx, pooled, a.H, a.W, a.C);
    } else {
        if (a.C % 4 == 0) SB_LAUNCH((maxpool_fwd_kernel<float, 4>), ew_blocks(pooled / 4), 256, 0, st, (const float*)a.x, (float*)a.p, a.idx, pooled / 4, a.H, a.W, a.C);
        else SB_LAUNCH((maxpool_fwd_kernel<float, 1>), ew_blocks(pooled), 256, 0, st, (const float*)a.x, (float*)a.p, a.idx, pooled, a.H, a.W, a.C);
    }
    return cudaGetLastError();
}
cudaError_t launch_pool_bwd(const PoolBwdArgs& a, bool bf16, cudaStream_t st)
{
    long pooled = (long)a.B * (a.H / 2) * (a.W / 2) * a.C;
    if (bf16) {
        if (a.C % 8 == 0) SB_LAUNCH((maxpool_bwd_kernel<__nv_bfloat16, 8>), ew_blocks(pooled / 8), 256, 0, st, (const __nv_bfloat16*)a.dp, a.idx, (const __nv_bfloat16*)a.p, (__nv_bfloat16*)a.dx, pooled / 8, a.H, a.W, a.C);
        else SB_LAUNCH((maxpool_bwd_kernel<__nv_bfloat16, 1>), ew_blocks(pooled), 256, 0, st, (const __nv_bfloat16*)a.dp, a.idx, (const __nv_bfloat16*)a.p, (__nv_bfloat16*)a.dx, pooled, a.H, a.W, a.C);
    } else {
        if (a.C % 4 == 0) SB_LAUNCH((maxpool_bwd_kernel<float, 4>), ew_blocks(pooled / 4), 256, 0, st, (const float*)a.dp, a.idx, (const float*)a.p, (float*)a.dx, pooled / 4, a.H, a.W, a.C);
        else SB_LAUNCH((maxpool_bwd_kernel<float, 1>), ew_blocks(pooled), 256, 0, st, (const float*)a.dp, a.idx, (const float*)a.p, (float*)a.dx, pooled, a.H, a.W, a.C);
    }
    return cudaGetLastError();
}

// =============================================================================================
// Softmax cross-entropy: one warp per row (shuffle max / sum), dZ = (softmax - onehot)/B.
// The last block to finish adds the row losses in row order, so the mean is deterministic.
// =============================================================================================
template <typename T>
__global__ void __launch_bounds__(256)
softmax_xent_kernel(const float* __restrict__ logits, PtrTab labels, int b_per_rep, float* __restrict__ row_loss,
                    float* __restrict__ loss, T* __restrict__ dZ, unsigned int* __restrict__ counter, int B, int C,
                    int scale_B, const float* __restrict__ loss_base, int loss_rows)
{
    pdl_prologue();
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int g = blockIdx.x * 8 + warp;
    if (g < B) {
        const float* z = logits + (size_t)g * C;
        const int y = ((const int32_t*)labels.p[g / b_per_rep])[g % b_per_rep];
        float m = -INFINITY;
        for (int c = lane; c < C; c += 32) m = fmaxf(m, z[c]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float s = 0.f;
        for (int c = lane; c < C; c += 32) s += expf(z[c] - m);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float lse = m + logf(s);
        const float invB = 1.0f / (float)scale_B;
        for (int c = lane; c < C; c += 32) {
            float pr = expf(z[c] - lse);
            stf(dZ + (size_t)g * C + c, (pr - (c == y ? 1.f : 0.f)) * invB);
        }
        if (lane == 0) row_loss[g] = (y >= 0 && y < C) ? lse - z[y] : 0.f;
    }
    __shared__ bool last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = (atomicAdd(counter, 1u) == gridDim.x - 1);
    __syncthreads();
    if (last && warp == 0) {
        __threadfence();
        float t = 0.f;
        for (int i0 = 0; i0 < loss_rows; i0 += 32) {   // fixed order: chunks of 32 rows, tree inside
            float v = (i0 + lane < loss_rows) ? ((volatile const float*)loss_base)[i0 + lane] : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            t += v;
        }
        if (lane == 0) { *loss = t / (float)loss_rows; *counter = 0u; }
    }
}
cudaError_t launch_softmax_xent(const XentArgs& a, bool bf16, cudaStream_t st)
{
    int blocks = cdiv(a.B, 8);
    const int scale_B = a.scale_B > 0 ? a.scale_B : a.B;
    const float* loss_base = a.loss_rows > 0 ? a.loss_base : a.row_loss;
    const int loss_rows = a.loss_rows > 0 ? a.loss_rows : a.B;
    if (bf16) SB_LAUNCH((softmax_xent_kernel<__nv_bfloat16>), blocks, 256, 0, st, a.logits, a.labels, a.b_per_rep, a.row_loss, a.loss, (__nv_bfloat16*)a.dZ, a.counter, a.B, a.C, scale_B, loss_base, loss_rows);
    else SB_LAUNCH((softmax_xent_kernel<float>), blocks, 256, 0, st, a.logits, a.labels, a.b_per_rep, a.row_loss, a.loss, (float*)a.dZ, a.counter, a.B, a.C, scale_B, loss_base, loss_rows);
    return cudaGetLastError();
}

// Modulo layer as a row permutation (see ModuloCopyArgs): one block column per row, 16-byte chunks.
__global__ void __launch_bounds__(256)
modulo_copy_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t row_vecs, int R, int b, int K, int scatter,
                   PtrTab labels, int has_labels, int32_t* __restrict__ labels_out)
{
    pdl_prologue();
    const int bk = b / K;
    const int nat = blockIdx.y;                                  // natural row index r*b + k*bk + i
    const int r = nat / b, k = (nat % b) / bk, i = nat % bk;
    const int sub = k * (R * bk) + r * bk + i;                   // sub-iteration order
    const uint4* s = src + (size_t)(scatter ? sub : nat) * row_vecs;
    uint4* d = dst + (size_t)(scatter ? nat : sub) * row_vecs;
    for (size_t v = blockIdx.x * (size_t)blockDim.x + threadIdx.x; v < row_vecs; v += (size_t)gridDim.x * blockDim.x) d[v] = s[v];
    if (has_labels && !scatter && blockIdx.x == 0 && threadIdx.x == 0) labels_out[sub] = ((const int32_t*)labels.p[r])[nat % b];
}
cudaError_t launch_modulo_copy(const ModuloCopyArgs& a, cudaStream_t st)
{
    if (a.row_bytes % 16 != 0 || a.K < 1 || a.b % a.K != 0) return cudaErrorInvalidValue;
    const size_t row_vecs = a.row_bytes / 16;
    int bx = (int)((row_vecs + 255) / 256);
    if (bx > 32) bx = 32;
    if (bx < 1) bx = 1;
    PtrTab tab{};
    if (a.labels) tab = *a.labels;
    SB_LAUNCH((modulo_copy_kernel), dim3(bx, a.R * a.b), 256, 0, st, (const uint4*)a.src, (uint4*)a.dst, row_vecs, a.R, a.b, a.K, a.scatter, tab,
              a.labels ? 1 : 0, a.labels_out);
    return cudaGetLastError();
}

// =============================================================================================
// Dropout [Listing 1, case DROPOUT | RELU]: a one-to-one layer on the (partitioned) width of the FC + ReLU layer below.
// Element (global batch row g, logical column c) is kept iff the first output word of Philox-4x32-10 (Salmon et al.,
// SC'11) at counter (e mod 2^32, e div 2^32, layer, iteration), e = g*width + c, under the 64-bit seed as key, is at
// least p * 2^32; kept elements are multiplied by 1/(1 - p).  state = {seed lo, seed hi, iteration, unused}.
// =============================================================================================
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1)
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}
// sub_bk > 0: the rows are those of sub-iteration sub_k of the modulo layer's schedule (replica r's sub_k-th slice of sub_bk rows,
// replica-major): buffer row j is batch row (j / sub_bk) * sub_b + sub_k * sub_bk + j % sub_bk, and the mask follows the batch row
template <typename T>
__global__ void __launch_bounds__(256)
dropout_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, size_t n, int width, const uint32_t* __restrict__ state, uint32_t layer,
                   uint32_t threshold, float scale, int sub_bk, int sub_b, int sub_k)
{
    pdl_prologue();
    const uint32_t k0 = state[0], k1 = state[1], it = state[2];
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        size_t e = i;
        if (sub_bk > 0) {
            const size_t j = i / (size_t)width, c = i - j * (size_t)width;
            const size_t g = (j / (size_t)sub_bk) * (size_t)sub_b + (size_t)sub_k * (size_t)sub_bk + j % (size_t)sub_bk;
            e = g * (size_t)width + c;
        }
        const uint32_t u = philox4x32_10_word0((uint32_t)e, (uint32_t)(e >> 32), layer, it, k0, k1);
        stf(y + i, u >= threshold ? ldf(x + i) * scale : 0.0f);
    }
}
// y = x * scale (the backward pass of the kept elements; the dropped ones arrive as zeros)
template <typename T>
__global__ void __launch_bounds__(256)
scale_kernel(const T* __restrict__ x, T* __restrict__ y, size_t n, float scale)
{
    pdl_prologue();
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) stf(y + e, ldf(x + e) * scale);
}
// mode 0: state = {v0, v1, v2, 0};  mode 1: ++iteration
__global__ void dropout_state_kernel(uint32_t* state, int mode, uint32_t v0, uint32_t v1, uint32_t v2)
{
    pdl_prologue();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    if (mode == 0) { state[0] = v0; state[1] = v1; state[2] = v2; state[3] = 0u; }
    else state[2] += 1u;
}
cudaError_t launch_dropout_fwd(const void* x, void* y, size_t rows, int width, const uint32_t* state, int layer, int units, bool bf16, cudaStream_t st,
                               int sub_bk, int sub_b, int sub_k)
{
    const size_t n = rows * (size_t)width;
    const uint32_t threshold = (uint32_t)units << 16;
    const float scale = 65536.0f / (float)(65536 - units);
    if (bf16) SB_LAUNCH((dropout_fwd_kernel<__nv_bfloat16>), ew_blocks((long)n), 256, 0, st, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, n, width, state, (uint32_t)layer, threshold, scale, sub_bk, sub_b, sub_k);
    else SB_LAUNCH((dropout_fwd_kernel<float>), ew_blocks((long)n), 256, 0, st, (const float*)x, (float*)y, n, width, state, (uint32_t)layer, threshold, scale, sub_bk, sub_b, sub_k);
    return cudaGetLastError();
}
cudaError_t launch_dropout_bwd(const void* dy, void* dx, size_t n, int units, bool bf16, cudaStream_t st)
{
    const float scale = 65536.0f / (float)(65536 - units);
    if (bf16) SB_LAUNCH((scale_kernel<__nv_bfloat16>), ew_blocks((long)n), 256, 0, st, (const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, n, scale);
    else SB_LAUNCH((scale_kernel<float>), ew_blocks((long)n), 256, 0, st, (const float*)dy, (float*)dx, n, scale);
    return cudaGetLastError();
}
cudaError_t launch_dropout_state(uint32_t* state, int mode, uint64_t seed, uint32_t iteration, cudaStream_t st)
{
    SB_LAUNCH((dropout_state_kernel), 1, 32, 0, st, state, mode, (uint32_t)seed, (uint32_t)(seed >> 32), iteration);
    return cudaGetLastError();
}

// =============================================================================================
// SGD with momentum over the whole (padded, 16-byte aligned) parameter arena:
// v <- mu*v + g ; w <- w - lr*v ; optional bf16 copy of the new w.
// =============================================================================================
template <bool SHADOW>
__device__ __forceinline__ void sgd_apply(float4& ww, float4& vv, const float4& gg, float lr, float mu, uint2* shadow_at)
{
    vv.x = fmaf(mu, vv.x, gg.x); vv.y = fmaf(mu, vv.y, gg.y); vv.z = fmaf(mu, vv.z, gg.z); vv.w = fmaf(mu, vv.w, gg.w);
    ww.x = fmaf(-lr, vv.x, ww.x); ww.y = fmaf(-lr, vv.y, ww.y); ww.z = fmaf(-lr, vv.z, ww.z); ww.w = fmaf(-lr, vv.w, ww.w);
    if (SHADOW) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(ww.x, ww.y), hi = __floats2bfloat162_rn(ww.z, ww.w);
        uint2 pk;
        pk.x = *(uint32_t*)&lo;
        pk.y = *(uint32_t*)&hi;
        *shadow_at = pk;
    }
}
// Grid-stride blocks with four independent 16-byte triples in flight per thread.  (Measured: the update does not
// hide behind the backward pass's tensor-core kernels whatever the grid size -- 16, 8, 4, 2 or 1 blocks per SM
// all give the same step time, and confined to 32 or 64 blocks the update overlaps but is itself too slow;
// streaming (evict-first) loads and stores make no difference either.  SB_SGD_BLOCKS_PER_SM changes the grid.)
template <bool SHADOW>
__global__ void __launch_bounds__(256)
sgd_kernel(float4* __restrict__ w, float4* __restrict__ v, const float4* __restrict__ g,
           uint2* __restrict__ shadow, size_t n4, float lr, float mu)
{
    pdl_prologue();
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n4; i += 4 * stride) {
        float4 ww[4], vv[4], gg[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { ww[u] = __ldcs(w + i + u * stride); vv[u] = __ldcs(v + i + u * stride); gg[u] = __ldcs(g + i + u * stride); }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            sgd_apply<SHADOW>(ww[u], vv[u], gg[u], lr, mu, SHADOW ? shadow + i + u * stride : nullptr);
            __stcs(v + i + u * stride, vv[u]);
            __stcs(w + i + u * stride, ww[u]);
        }
    }
    for (; i < n4; i += stride) {
        float4 ww = __ldcs(w + i), vv = __ldcs(v + i), gg = __ldcs(g + i);
        sgd_apply<SHADOW>(ww, vv, gg, lr, mu, SHADOW ? shadow + i : nullptr);
        __stcs(v + i, vv);
        __stcs(w + i, ww);
    }
}
// Ordered split reduce and update in one pass: g = sum_s part[s] (the same kernels' split order as
// launch_reduce_partials, so the gradient has the same bits), then the SGD step on w, v (and the bf16 copy) without
// the gradient ever being written to or read back from the gradient arena.
template <bool SHADOW>
__global__ void __launch_bounds__(256)
reduce_sgd4_kernel(const float4* __restrict__ part, size_t stride4, int splits, float4* __restrict__ w, float4* __restrict__ v,
                   uint2* __restrict__ shadow, size_t n4, float lr, float mu)
{
    pdl_prologue();
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 ww = w[i], vv = v[i];
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s0 = 0; s0 < splits; s0 += 8) {
            float4 pv[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                pv[u] = (s0 + u < splits) ? __ldg(part + (size_t)(s0 + u) * stride4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 8; ++u) { t.x += pv[u].x; t.y += pv[u].y; t.z += pv[u].z; t.w += pv[u].w; }
        }
        sgd_apply<SHADOW>(ww, vv, t, lr, mu, SHADOW ? shadow + i : nullptr);
        v[i] = vv;
        w[i] = ww;
    }
}
__device__ __forceinline__ void sgd_apply_scalar(float* w, float* v, float g, __nv_bfloat16* shadow, size_t i, float lr, float mu)
{
    const float vv = fmaf(mu, v[i], g), ww = fmaf(-lr, vv, w[i]);
    v[i] = vv;
    w[i] = ww;
    if (shadow) shadow[i] = __float2bfloat16_rn(ww);
}
template <int LANES>
__global__ void __launch_bounds__(32 * LANES)
reduce_sgd_many_kernel(const float* __restrict__ part, size_t stride, int splits, float* __restrict__ w, float* __restrict__ v,
                       __nv_bfloat16* __restrict__ shadow, size_t n, float lr, float mu)
{
    pdl_prologue();
    __shared__ float s[LANES][33];
    const int e = threadIdx.x % 32, lane = threadIdx.x / 32;
    const size_t i = blockIdx.x * 32ull + e;
    s[lane][e] = i < n ? many_lane_sum<LANES>(part, stride, i, lane, splits) : 0.f;
    __syncthreads();
    if (lane == 0 && i < n) {
        float r = 0.f;
#pragma unroll
        for (int j = 0; j < LANES; ++j) r += s[j][e];
        sgd_apply_scalar(w, v, r, shadow, i, lr, mu);
    }
}
__global__ void __launch_bounds__(256)
reduce_sgd_kernel(const float* __restrict__ part, size_t stride, int splits, float* __restrict__ w, float* __restrict__ v,
                  __nv_bfloat16* __restrict__ shadow, size_t n, float lr, float mu)
{
    pdl_prologue();
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float t = 0.f;
        for (int sp = 0; sp < splits; ++sp) t += part[(size_t)sp * stride + i];
        sgd_apply_scalar(w, v, t, shadow, i, lr, mu);
    }
}
cudaError_t launch_reduce_sgd(const float* part, size_t stride, size_t n, int splits, float* w, float* v, __nv_bfloat16* shadow,
                              float lr, float mu, cudaStream_t st)
{
    // (the same case split as launch_reduce_partials: each case sums in the same order there and here)
    if (splits >= 128 && n <= (1u << 20)) {
        SB_LAUNCH((reduce_sgd_many_kernel<32>), cdiv((long)n, 32), 1024, 0, st, part, stride, splits, w, v, shadow, n, lr, mu);
    } else if (splits >= 32 && n <= (1u << 20)) {
        SB_LAUNCH((reduce_sgd_many_kernel<8>), cdiv((long)n, 32), 256, 0, st, part, stride, splits, w, v, shadow, n, lr, mu);
    } else if (n % 4 == 0 && stride % 4 == 0 && (((uintptr_t)part | (uintptr_t)w | (uintptr_t)v) & 15) == 0 && (((uintptr_t)shadow) & 7) == 0) {
        int blocks = cdiv((long)(n / 4), 256);
        if (blocks > 148 * 8) blocks = 148 * 8;
        if (shadow) SB_LAUNCH((reduce_sgd4_kernel<true>), blocks, 256, 0, st, (const float4*)part, stride / 4, splits, (float4*)w, (float4*)v, (uint2*)shadow, n / 4, lr, mu);
        else SB_LAUNCH((reduce_sgd4_kernel<false>), blocks, 256, 0, st, (const float4*)part, stride / 4, splits, (float4*)w, (float4*)v, nullptr, n / 4, lr, mu);
    } else {
        int blocks = cdiv((long)n, 256);
        if (blocks > 148 * 8) blocks = 148 * 8;
        SB_LAUNCH((reduce_sgd_kernel), blocks, 256, 0, st, part, stride, splits, w, v, shadow, n, lr, mu);
    }
    return cudaGetLastError();
}

cudaError_t launch_sgd(float* w, float* v, const float* g, __nv_bfloat16* shadow, size_t n, float lr, float mu, cudaStream_t st)
{
    size_t n4 = n / 4;
    static const int per_sm = (int)tune("SB_SGD_BLOCKS_PER_SM", 16);
    long blocks = ((long)n4 + 255) / 256;
    if (blocks > 148L * per_sm) blocks = 148L * per_sm;
    if (blocks < 1) blocks = 1;
    if (shadow) SB_LAUNCH((sgd_kernel<true>), (int)blocks, 256, 0, st, (float4*)w, (float4*)v, (const float4*)g, (uint2*)shadow, n4, lr, mu);
    else SB_LAUNCH((sgd_kernel<false>), (int)blocks, 256, 0, st, (float4*)w, (float4*)v, (const float4*)g, nullptr, n4, lr, mu);
    return cudaGetLastError();
}

__global__ void __launch_bounds__(256)
to_bf16_kernel(const float4* __restrict__ w, uint2* __restrict__ shadow, size_t n4)
{
    pdl_prologue();
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 ww = w[i];
        __nv_bfloat162 lo = __floats2bfloat162_rn(ww.x, ww.y), hi = __floats2bfloat162_rn(ww.z, ww.w);
        uint2 pk;
        pk.x = *(uint32_t*)&lo;
        pk.y = *(uint32_t*)&hi;
        shadow[i] = pk;
    }
}
cudaError_t launch_to_bf16(const float* w, __nv_bfloat16* shadow, size_t n, cudaStream_t st)
{
    SB_LAUNCH((to_bf16_kernel), ew_blocks((long)(n / 4)), 256, 0, st, (const float4*)w, (uint2*)shadow, n / 4);
    return cudaGetLastError();
}

// =============================================================================================
// Input-layer convolution (Cin <= 4, e.g. RGB images): 9*Cin <= 36 products per output, far too
// thin for tensor-core tiles and bound by the output / dy traffic.  Each thread builds the
// 3x3xCin patch of its pixel in registers (forward) or the block stages patches in shared memory
// (weight gradient).
// =============================================================================================
template <typename T, int CIN, bool TAB>
__device__ __forceinline__ void load_patch(float (&patch)[9 * CIN], const T* __restrict__ x, const PtrTab& tab, int b_per_rep,
                                           long pix, int H, int W)
{
    const int w_ = (int)(pix % W);
    const long q = pix / W;
    const int h_ = (int)(q % H), n_ = (int)(q / H);
    const T* img = TAB ? (const T*)tab.p[n_ / b_per_rep] + (size_t)(n_ % b_per_rep) * H * W * CIN : x + (size_t)n_ * H * W * CIN;
#pragma unroll
    for (int r = 0; r < 3; ++r)
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            const int hh = h_ + r - 1, ww = w_ + s - 1;
            const bool in = hh >= 0 && hh < H && ww >= 0 && ww < W;
#pragma unroll
            for (int c = 0; c < CIN; ++c) patch[(r * 3 + s) * CIN + c] = in ? ldf(img + ((size_t)hh * W + ww) * CIN + c) : 0.f;
        }
}

// Forward: 8 consecutive threads share a pixel, each produces 8 output channels (16-byte stores that
// a warp lays down as contiguous 128-byte pixel rows).  Weights live in shared memory as [9*CIN][Cout].
template <typename T, int CIN, bool TAB>
__global__ void __launch_bounds__(256)
conv_in_fwd_kernel(const T* __restrict__ x, PtrTab tab, int b_per_rep, const T* __restrict__ wt, const float* __restrict__ bias,
                   T* __restrict__ y, long npix, int H, int W, int Cout, int relu)
{
    pdl_prologue();
    extern __shared__ float s_wf[];            // [9*CIN][Cout] then bias [Cout]
    float* s_b = s_wf + 9 * CIN * Cout;
    for (int e = threadIdx.x; e < 9 * CIN * Cout; e += 256) {
        int k = e % Cout, j = e / Cout;
        s_wf[e] = ldf(wt + (size_t)k * 9 * CIN + j);
    }
    for (int e = threadIdx.x; e < Cout; e += 256) s_b[e] = bias[e];
    __syncthreads();
    const int groups = Cout / 8;               // threads per pixel
    const long t = blockIdx.x * 256L + threadIdx.x;
    const long pix = t / groups;
    const int kg = (int)(t % groups) * 8;
    if (pix >= npix) return;
    float patch[9 * CIN];
    load_patch<T, CIN, TAB>(patch, x, tab, b_per_rep, pix, H, W);
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = s_b[kg + i];
#pragma unroll
    for (int j = 0; j < 9 * CIN; ++j) {
        const float4 w0 = *(const float4*)(s_wf + j * Cout + kg), w1 = *(const float4*)(s_wf + j * Cout + kg + 4);
        acc[0] = fmaf(patch[j], w0.x, acc[0]); acc[1] = fmaf(patch[j], w0.y, acc[1]);
        acc[2] = fmaf(patch[j], w0.z, acc[2]); acc[3] = fmaf(patch[j], w0.w, acc[3]);
        acc[4] = fmaf(patch[j], w1.x, acc[4]); acc[5] = fmaf(patch[j], w1.y, acc[5]);
        acc[6] = fmaf(patch[j], w1.z, acc[6]); acc[7] = fmaf(patch[j], w1.w, acc[7]);
    }
    if (relu) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (!(acc[i] > 0.f)) acc[i] = 0.f;
    }
    store8(y + (size_t)pix * Cout + kg, acc);
}

// Forward, 4 pixels per thread (W a multiple of 4): a thread owns 4 horizontally adjacent pixels and 8 output
// channels.  The 3 x 6 x CIN input window of the 4 pixels sits in registers, so each pair of 16-byte weight
// reads from shared memory feeds 32 FMAs (the 1-pixel kernel above is bound by those reads).
template <typename T, int CIN, bool TAB>
__global__ void __launch_bounds__(256)
conv_in_fwd4_kernel(const T* __restrict__ x, PtrTab tab, int b_per_rep, const T* __restrict__ wt, const float* __restrict__ bias,
                    T* __restrict__ y, long nquads, int H, int W, int Cout, int relu)
{
    pdl_prologue();
    extern __shared__ float s_wf[];            // [9*CIN][Cout] then bias [Cout]
    float* s_b = s_wf + 9 * CIN * Cout;
    for (int e = threadIdx.x; e < 9 * CIN * Cout; e += 256) {
        int k = e % Cout, j = e / Cout;
        s_wf[e] = ldf(wt + (size_t)k * 9 * CIN + j);
    }
    for (int e = threadIdx.x; e < Cout; e += 256) s_b[e] = bias[e];
    __syncthreads();
    const int groups = Cout / 8;
    const long t = blockIdx.x * 256L + threadIdx.x;
    const long quad = t / groups;
    const int kg = (int)(t % groups) * 8;
    if (quad >= nquads) return;
    const int wq = W / 4;
    const int w0 = (int)(quad % wq) * 4;
    const long q2 = quad / wq;
    const int h = (int)(q2 % H);
    const long n = q2 / H;
    const T* img = TAB ? (const T*)tab.p[n / b_per_rep] + (size_t)(n % b_per_rep) * H * W * CIN : x + (size_t)n * H * W * CIN;
    float win[3][6 * CIN];                     // rows h-1..h+1, columns w0-1..w0+4
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int hh = h + r - 1;
#pragma unroll
        for (int c6 = 0; c6 < 6; ++c6) {
            const int ww = w0 + c6 - 1;
            const bool in = hh >= 0 && hh < H && ww >= 0 && ww < W;
#pragma unroll
            for (int c = 0; c < CIN; ++c) win[r][c6 * CIN + c] = in ? ldf(img + ((size_t)hh * W + ww) * CIN + c) : 0.f;
        }
    }
    float acc[4][8];
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[p][i] = s_b[kg + i];
#pragma unroll
    for (int r = 0; r < 3; ++r)
#pragma unroll
        for (int sc = 0; sc < 3 * CIN; ++sc) {          // sc = s*CIN + c
            const int j = r * 3 * CIN + sc;
            const float4 w0v = *(const float4*)(s_wf + j * Cout + kg), w1v = *(const float4*)(s_wf + j * Cout + kg + 4);
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const float xv = win[r][p * CIN + sc];
                acc[p][0] = fmaf(xv, w0v.x, acc[p][0]); acc[p][1] = fmaf(xv, w0v.y, acc[p][1]);
                acc[p][2] = fmaf(xv, w0v.z, acc[p][2]); acc[p][3] = fmaf(xv, w0v.w, acc[p][3]);
                acc[p][4] = fmaf(xv, w1v.x, acc[p][4]); acc[p][5] = fmaf(xv, w1v.y, acc[p][5]);
                acc[p][6] = fmaf(xv, w1v.z, acc[p][6]); acc[p][7] = fmaf(xv, w1v.w, acc[p][7]);
            }
        }
    const size_t pix0 = ((size_t)n * H + h) * W + w0;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        if (relu) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (!(acc[p][i] > 0.f)) acc[p][i] = 0.f;
        }
        store8(y + (pix0 + p) * Cout + kg, acc[p]);
    }
}

// Weight + bias gradient: block = 64 output channels x 4 pixel lanes; per 64-pixel chunk the block stages
// the patches in shared memory, then thread (k, q) accumulates dy[pix,k] * patch[pix,:] over its pixels.
// part[block][k][9*CIN] and part_b[block][k] are reduced afterwards in block order.
template <typename T, int CIN, bool TAB>
__global__ void __launch_bounds__(256)
conv_in_wgrad_kernel(const T* __restrict__ x, PtrTab tab, int b_per_rep, const T* __restrict__ dy, float* __restrict__ part,
                     long npix, int H, int W, int Cout, long stride_floats)
{
    pdl_prologue();
    constexpr int PJ = (9 * CIN + 3) / 4 * 4;   // padded patch length (16-byte rows)
    __shared__ __align__(16) float s_patch[64][PJ];
    __shared__ float s_red[3][64][9 * CIN + 1];
    const int k = threadIdx.x % 64, q = threadIdx.x / 64;
    const int k0 = blockIdx.y * 64;
    float acc[9 * CIN], accb = 0.f;
#pragma unroll
    for (int j = 0; j < 9 * CIN; ++j) acc[j] = 0.f;
    const long nchunks = (npix + 63) / 64;
    for (long ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
        const long p0 = ch * 64;
        {
            // staging: thread (pixel pp, filter row r) writes the 3 taps x CIN values of that row; lane group 3
            // clears the padding columns
            const int pp = threadIdx.x % 64, r = threadIdx.x / 64;
            const long pix = p0 + pp;
            if (r < 3) {
                const int w_ = (int)(pix % W);
                const long t = pix / W;
                const int h_ = (int)(t % H);
                const long n_ = t / H;
                const int hh = h_ + r - 1;
                const bool row_in = pix < npix && hh >= 0 && hh < H;
                const T* img = nullptr;
                if (row_in)
                    img = (TAB ? (const T*)tab.p[n_ / b_per_rep] + (size_t)(n_ % b_per_rep) * H * W * CIN : x + (size_t)n_ * H * W * CIN) +
                          (size_t)hh * W * CIN;
#pragma unroll
                for (int sdx = 0; sdx < 3; ++sdx) {
                    const int ww = w_ + sdx - 1;
                    const bool in = row_in && ww >= 0 && ww < W;
#pragma unroll
                    for (int c = 0; c < CIN; ++c) s_patch[pp][(r * 3 + sdx) * CIN + c] = in ? ldf(img + (size_t)ww * CIN + c) : 0.f;
                }
            } else {
#pragma unroll
                for (int j = 9 * CIN; j < PJ; ++j) s_patch[pp][j] = 0.f;
            }
        }
        __syncthreads();
        if (k0 + k < Cout) {
            // this thread's 16 pixels of the chunk, 4 at a time so that 4 dy loads are in flight together
            for (int pg = 0; pg < 4; ++pg) {
                float d[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const long pix = p0 + q + 4 * (pg * 4 + u);
                    d[u] = pix < npix ? ldf(dy + (size_t)pix * Cout + k0 + k) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int pp = q + 4 * (pg * 4 + u);
                    accb += d[u];
                    float pv[PJ];
#pragma unroll
                    for (int j4 = 0; j4 < PJ / 4; ++j4) {
                        const float4 v = *(const float4*)&s_patch[pp][j4 * 4];
                        pv[j4 * 4] = v.x; pv[j4 * 4 + 1] = v.y; pv[j4 * 4 + 2] = v.z; pv[j4 * 4 + 3] = v.w;
                    }
#pragma unroll
                    for (int j = 0; j < 9 * CIN; ++j) acc[j] = fmaf(d[u], pv[j], acc[j]);
                }
            }
        }
        __syncthreads();
    }
    // fixed-order reduction over the 4 pixel lanes
    if (q > 0) {
#pragma unroll
        for (int j = 0; j < 9 * CIN; ++j) s_red[q - 1][k][j] = acc[j];
        s_red[q - 1][k][9 * CIN] = accb;
    }
    __syncthreads();
    if (q == 0 && k0 + k < Cout) {
        float* dst = part + (size_t)blockIdx.x * stride_floats;
#pragma unroll
        for (int j = 0; j < 9 * CIN; ++j) dst[(size_t)(k0 + k) * 9 * CIN + j] = acc[j] + s_red[0][k][j] + s_red[1][k][j] + s_red[2][k][j];
        dst[(size_t)Cout * 9 * CIN + k0 + k] = accb + s_red[0][k][9 * CIN] + s_red[1][k][9 * CIN] + s_red[2][k][9 * CIN];
    }
}

template <typename T, int CIN>
static cudaError_t launch_conv_in_fwd_t(const ConvSimtArgs& a, cudaStream_t st)
{
    const long npix = (long)a.B * a.H * a.W;
    const long threads = npix * (a.Cout / 8);
    const int blocks = (int)((threads + 255) / 256);
    const size_t smem = (size_t)(9 * CIN * a.Cout + a.Cout) * 4;
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
    if (a.W % 4 == 0) {
        const long nquads = npix / 4;
        const int qblocks = (int)((nquads * (a.Cout / 8) + 255) / 256);
        if (a.tab) SB_LAUNCH((conv_in_fwd4_kernel<T, CIN, true>), qblocks, 256, smem, st, nullptr, tab, a.b_per_rep, (const T*)a.w, a.bias, (T*)a.out, nquads, a.H, a.W, a.Cout, a.relu);
        else SB_LAUNCH((conv_in_fwd4_kernel<T, CIN, false>), qblocks, 256, smem, st, (const T*)a.in, tab, a.b_per_rep, (const T*)a.w, a.bias, (T*)a.out, nquads, a.H, a.W, a.Cout, a.relu);
        return cudaGetLastError();
    }
    if (a.tab) SB_LAUNCH((conv_in_fwd_kernel<T, CIN, true>), blocks, 256, smem, st, nullptr, tab, a.b_per_rep, (const T*)a.w, a.bias, (T*)a.out, npix, a.H, a.W, a.Cout, a.relu);
    else SB_LAUNCH((conv_in_fwd_kernel<T, CIN, false>), blocks, 256, smem, st, (const T*)a.in, tab, a.b_per_rep, (const T*)a.w, a.bias, (T*)a.out, npix, a.H, a.W, a.Cout, a.relu);
    return cudaGetLastError();
}
bool conv_in_supported(int Cin, int Cout) { return (Cin == 1 || Cin == 3 || Cin == 4) && Cout % 8 == 0 && Cout <= 256; }
cudaError_t launch_conv_in_fwd(const ConvSimtArgs& a, bool bf16, cudaStream_t st)
{
#define SB_CI(T) (a.Cin == 1 ? launch_conv_in_fwd_t<T, 1>(a, st) : a.Cin == 3 ? launch_conv_in_fwd_t<T, 3>(a, st) : launch_conv_in_fwd_t<T, 4>(a, st))
    return bf16 ? SB_CI(__nv_bfloat16) : SB_CI(float);
#undef SB_CI
}
int conv_in_wgrad_blocks(int B, int H, int W)
{
    long chunks = ((long)B * H * W + 63) / 64;
    return (int)(chunks < 148 * 4 ? chunks : 148 * 4);
}
template <typename T, int CIN>
static cudaError_t launch_conv_in_wgrad_t(const WgradSimtArgs& a, cudaStream_t st)
{
    const long npix = (long)a.B * a.H * a.W;
    dim3 grid(conv_in_wgrad_blocks(a.B, a.H, a.W), (a.Cout + 63) / 64);
    const long stride = (long)a.Cout * 9 * CIN + a.Cout;
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
    if (a.tab) SB_LAUNCH((conv_in_wgrad_kernel<T, CIN, true>), grid, 256, 0, st, nullptr, tab, a.b_per_rep, (const T*)a.dy, a.part, npix, a.H, a.W, a.Cout, stride);
    else SB_LAUNCH((conv_in_wgrad_kernel<T, CIN, false>), grid, 256, 0, st, (const T*)a.x, tab, a.b_per_rep, (const T*)a.dy, a.part, npix, a.H, a.W, a.Cout, stride);
    return cudaGetLastError();
}
// part: [conv_in_wgrad_blocks][Cout*9*Cin + Cout] floats (weights then bias), to be reduced in block order.
cudaError_t launch_conv_in_wgrad(const WgradSimtArgs& a, bool bf16, cudaStream_t st)
{
#define SB_CI(T) (a.Cin == 1 ? launch_conv_in_wgrad_t<T, 1>(a, st) : a.Cin == 3 ? launch_conv_in_wgrad_t<T, 3>(a, st) : launch_conv_in_wgrad_t<T, 4>(a, st))
    return bf16 ? SB_CI(__nv_bfloat16) : SB_CI(float);
#undef SB_CI
}

// =============================================================================================
// Narrow FC layers (out <= 16, e.g. the 10-class logits layer): too narrow for any GEMM tile.
//   forward : one block per batch row, threads split the reduction, block-wide shuffle reduce
//   wgrad   : one thread per input column, dY staged in shared memory
//   dgrad   : one thread per (row, input column)
// =============================================================================================
constexpr int NARROW_MAX = 16;

// Forward: one warp per batch row, 8 rows per block; a lane walks the reduction in steps of 8 values
// (one 16-byte load of X and of each weight row for bf16), then the warp shuffle-reduces its out_f sums.
template <typename T> struct Vec8;
template <> struct Vec8<float> { static constexpr int N = 4; typedef float4 V; };
template <> struct Vec8<__nv_bfloat16> { static constexpr int N = 8; typedef uint4 V; };

// Block = 2 batch rows x 4 reduction quarters (one warp each).  A lane issues all its 16-byte loads of X and
// of the out_f weight rows for its slice up front (many loads in flight: the kernel is pure latency), the warp
// shuffle-reduces, and the 4 quarters of a row are added in order through shared memory.
template <typename T, bool TAB, int KS, bool VEC>
__global__ void __launch_bounds__(64 * KS)
fc_narrow_fwd_kernel(const T* __restrict__ X, PtrTab tab, int tab_b, const T* __restrict__ Wt, const float* __restrict__ bias,
                     T* __restrict__ Y, float* __restrict__ Y32, int B, int in_f, int out_f, int relu)
{
    pdl_prologue();
    constexpr int VN = Vec8<T>::N;
    typedef typename Vec8<T>::V V;
    __shared__ float s_part[2][KS][NARROW_MAX];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int rl = warp / KS, ks = warp % KS;
    const int g = blockIdx.x * 2 + rl;
    const int kq = in_f / KS;                 // reduction elements of this warp (multiple of 32*VN or handled by the tail loop)
    float acc[NARROW_MAX];
#pragma unroll
    for (int j = 0; j < NARROW_MAX; ++j) acc[j] = 0.f;
    if (g < B) {
        const T* xr = (TAB ? (const T*)tab.p[g / tab_b] + (size_t)(g % tab_b) * in_f : X + (size_t)g * in_f) + (size_t)ks * kq;
        const T* wr = Wt + (size_t)ks * kq;
        if (VEC) {
            // 16-byte loads: the host only selects this variant when every row and every slice starts 16-byte aligned
            for (int k = lane * VN; k + VN <= kq; k += 32 * VN) {
                const V xv = *(const V*)(xr + k);
                V wv[NARROW_MAX];
#pragma unroll
                for (int j = 0; j < NARROW_MAX; ++j)
                    if (j < out_f) wv[j] = *(const V*)(wr + (size_t)j * in_f + k);
#pragma unroll
                for (int j = 0; j < NARROW_MAX; ++j)
                    if (j < out_f) {
#pragma unroll
                        for (int i = 0; i < VN; ++i) acc[j] = fmaf(ldf((const T*)&xv + i), ldf((const T*)&wv[j] + i), acc[j]);
                    }
            }
        } else {
            for (int k = lane; k < kq; k += 32) {
                const float xv = ldf(xr + k);
#pragma unroll
                for (int j = 0; j < NARROW_MAX; ++j)
                    if (j < out_f) acc[j] = fmaf(xv, ldf(wr + (size_t)j * in_f + k), acc[j]);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < NARROW_MAX; ++j) {
        float v = acc[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) s_part[rl][ks][j] = v;
    }
    __syncthreads();
    if (threadIdx.x < 2 * NARROW_MAX) {
        const int r2 = threadIdx.x / NARROW_MAX, j = threadIdx.x % NARROW_MAX;
        const int g2 = blockIdx.x * 2 + r2;
        if (g2 < B && j < out_f) {
            float v = bias[j];
#pragma unroll
            for (int q = 0; q < KS; ++q) v += s_part[r2][q][j];
            if (relu && !(v > 0.f)) v = 0.f;
            if (Y32) Y32[(size_t)g2 * out_f + j] = v;
            if (Y) stf(Y + (size_t)g2 * out_f + j, v);
        }
    }
}

// Weight + bias gradient: block = 32 input columns x 8 row lanes; lane l sums batch rows l, l+8, ... for its
// column, then the 8 lanes are combined in lane order through shared memory (deterministic).
template <typename T, bool TAB>
__global__ void __launch_bounds__(256)
fc_narrow_wgrad_kernel(const T* __restrict__ X, PtrTab tab, int tab_b, const T* __restrict__ dY, float* __restrict__ dW,
                       float* __restrict__ db, int B, int in_f, int out_f)
{
    pdl_prologue();
    extern __shared__ float s_dy[];   // [B][out_f], then the reduction buffer [8][32][NARROW_MAX]
    float* s_red = s_dy + B * out_f;
    for (int e = threadIdx.x; e < B * out_f; e += 256) s_dy[e] = ldf(dY + e);
    __syncthreads();
    const int col = threadIdx.x % 32, lane = threadIdx.x / 32;
    const int i = blockIdx.x * 32 + col;
    if (blockIdx.x == 0 && threadIdx.x < out_f) {
        float t = 0.f;
        for (int g = 0; g < B; ++g) t += s_dy[g * out_f + threadIdx.x];
        db[threadIdx.x] = t;
    }
    float acc[NARROW_MAX];
#pragma unroll
    for (int j = 0; j < NARROW_MAX; ++j) acc[j] = 0.f;
    if (i < in_f) {
        for (int g = lane; g < B; g += 8) {
            const T* xr = TAB ? (const T*)tab.p[g / tab_b] + (size_t)(g % tab_b) * in_f : X + (size_t)g * in_f;
            const float xv = ldf(xr + i);
#pragma unroll
            for (int j = 0; j < NARROW_MAX; ++j)
                if (j < out_f) acc[j] = fmaf(s_dy[g * out_f + j], xv, acc[j]);
        }
    }
#pragma unroll
    for (int j = 0; j < NARROW_MAX; ++j) s_red[(lane * 32 + col) * NARROW_MAX + j] = acc[j];
    __syncthreads();
    if (lane == 0 && i < in_f) {
#pragma unroll
        for (int j = 0; j < NARROW_MAX; ++j)
            if (j < out_f) {
                float t = 0.f;
#pragma unroll
                for (int l = 0; l < 8; ++l) t += s_red[(l * 32 + col) * NARROW_MAX + j];
                dW[(size_t)j * in_f + i] = t;
            }
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
fc_narrow_dgrad_kernel(const T* __restrict__ dY, const T* __restrict__ Wt, const T* __restrict__ ref, T* __restrict__ dX,
                       int in_f, int out_f)
{
    pdl_prologue();
    __shared__ float s_d[NARROW_MAX];
    const int g = blockIdx.y;
    if (threadIdx.x < out_f) s_d[threadIdx.x] = ldf(dY + (size_t)g * out_f + threadIdx.x);
    __syncthreads();
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= in_f) return;
    float acc = 0.f;
#pragma unroll
    for (int j = 0; j < NARROW_MAX; ++j)
        if (j < out_f) acc = fmaf(s_d[j], ldf(Wt + (size_t)j * in_f + i), acc);
    if (ref != nullptr && !(ldf(ref + (size_t)g * in_f + i) > 0.f)) acc = 0.f;
    stf(dX + (size_t)g * in_f + i, acc);
}

bool fc_narrow_supported(int out_f, int B) { return out_f <= NARROW_MAX && (size_t)B * out_f * 4 <= 24 * 1024; }

template <typename T>
static cudaError_t launch_fc_narrow_t(const FcNarrowArgs& a, cudaStream_t st)
{
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
    const int tb = a.tab_b > 0 ? a.tab_b : 1;
    if (a.pass == 0) {
        const int blocks = (a.B + 1) / 2;
        // 16-byte loads need every row (and every quarter of a row) to start on a 16-byte boundary
        const bool aligned_ptrs = (((uintptr_t)a.W | (uintptr_t)a.X) & 15) == 0 && !a.tab;
        const bool vec = aligned_ptrs && a.in_f % Vec8<T>::N == 0;
        const bool quarters = vec && a.in_f % (4 * Vec8<T>::N) == 0;
#define SB_NF(TABF, KS, VECF) SB_LAUNCH((fc_narrow_fwd_kernel<T, TABF, KS, VECF>), blocks, 64 * KS, 0, st,  \
            (const T*)a.X, tab, tb, (const T*)a.W, a.bias, (T*)a.Y, a.Y32, a.B, a.in_f, a.out_f, a.relu)
        if (quarters) SB_NF(false, 4, true);
        else if (vec) SB_NF(false, 1, true);
        else if (a.tab) SB_NF(true, 1, false);
        else SB_NF(false, 1, false);
#undef SB_NF
    } else if (a.pass == 1) {
        const size_t smem = (size_t)a.B * a.out_f * 4 + 8 * 32 * NARROW_MAX * 4;
        const int blocks = (a.in_f + 31) / 32;
        if (a.tab) SB_LAUNCH((fc_narrow_wgrad_kernel<T, true>), blocks, 256, smem, st, nullptr, tab, tb, (const T*)a.dY, a.dW, a.db, a.B, a.in_f, a.out_f);
        else SB_LAUNCH((fc_narrow_wgrad_kernel<T, false>), blocks, 256, smem, st, (const T*)a.X, tab, tb, (const T*)a.dY, a.dW, a.db, a.B, a.in_f, a.out_f);
    } else {
        dim3 grid((a.in_f + 255) / 256, a.B);
        SB_LAUNCH((fc_narrow_dgrad_kernel<T>), grid, 256, 0, st, (const T*)a.dY, (const T*)a.W, (const T*)a.ref, (T*)a.dX, a.in_f, a.out_f);
    }
    return cudaGetLastError();
}
cudaError_t launch_fc_narrow(const FcNarrowArgs& a, bool bf16, cudaStream_t st)
{
    return bf16 ? launch_fc_narrow_t<__nv_bfloat16>(a, st) : launch_fc_narrow_t<float>(a, st);
}

// =============================================================================================
// Strided FFMA GEMM for the sharded FC layers:  C[m,n] = sum_k A(m,k) * B(n,k).
// 64x64 tile, BK = 16, 256 threads, 4x4 outputs per thread.  blockIdx.z = shard for the
// partitions that own outputs; the K-partition (dgrad) walks the shards one after another.
// =============================================================================================
__device__ __forceinline__ int shard_lo(int j, int total, int shards) { return (int)(((long)j * total) / shards); }

template <typename T, int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ A, long sAm, long sAk, const T* __restrict__ Bm, long sBn, long sBk,
                 int M, int N, int K, void* __restrict__ Cv, long ldc, float* __restrict__ C32,
                 const float* __restrict__ bias, int relu, const T* __restrict__ ref, long ldref,
                 int shard_dim, int shards, PtrTab tab, int tab_mode, int tab_b)
{
    pdl_prologue();
    __shared__ float As[16][65];
    __shared__ float Bs[16][65];
    int m_lo = 0, m_hi = M, n_lo = 0, n_hi = N;
    if (shard_dim == 1) { n_lo = shard_lo(blockIdx.z, N, shards); n_hi = shard_lo(blockIdx.z + 1, N, shards); }
    if (shard_dim == 3) { m_lo = shard_lo(blockIdx.z, M, shards); m_hi = shard_lo(blockIdx.z + 1, M, shards); }
    const int m0 = m_lo + blockIdx.y * 64, n0 = n_lo + blockIdx.x * 64;
    if (m0 >= m_hi || n0 >= n_hi) return;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    const int kparts = (shard_dim == 2) ? shards : 1;
    for (int kp = 0; kp < kparts; ++kp) {
        const int k_lo = (shard_dim == 2) ? shard_lo(kp, K, shards) : 0;
        const int k_hi = (shard_dim == 2) ? shard_lo(kp + 1, K, shards) : K;
        for (int k0 = k_lo; k0 < k_hi; k0 += 16) {
            for (int e = tid; e < 64 * 16; e += 256) {
                int mm, kk;
                if (sAk == 1) { kk = e % 16; mm = e / 16; } else { mm = e % 64; kk = e / 64; }
                float v = 0.f;
                if (m0 + mm < m_hi && k0 + kk < k_hi) {
                    const int m = m0 + mm;
                    v = (tab_mode == 1) ? ldf((const T*)tab.p[m / tab_b] + (long)(m % tab_b) * sAm + (long)(k0 + kk) * sAk)
                                        : ldf(A + (long)m * sAm + (long)(k0 + kk) * sAk);
                }
                As[kk][mm] = v;
                int nn;
                if (sBk == 1) { kk = e % 16; nn = e / 16; } else { nn = e % 64; kk = e / 64; }
                v = 0.f;
                if (n0 + nn < n_hi && k0 + kk < k_hi) {
                    const int k = k0 + kk;
                    v = (tab_mode == 2) ? ldf((const T*)tab.p[k / tab_b] + (long)(n0 + nn) * sBn + (long)(k % tab_b) * sBk)
                                        : ldf(Bm + (long)(n0 + nn) * sBn + (long)k * sBk);
                }
                Bs[kk][nn] = v;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) {
                float a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
                for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
            __syncthreads();
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= m_hi) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int n = n0 + tx * 4 + j;
            if (n >= n_hi) continue;
            float v = acc[i][j];
            if (EPI == EPI_BIAS_ACT) {
                v += bias[n];
                if (relu && !(v > 0.f)) v = 0.f;
                if (C32) C32[(long)m * ldc + n] = v;
                if (Cv) stf((T*)Cv + (long)m * ldc + n, v);
            } else if (EPI == EPI_MASK) {
                if (ref != nullptr && !(ldf(ref + (long)m * ldref + n) > 0.f)) v = 0.f;
                stf((T*)Cv + (long)m * ldc + n, v);
            } else {
                ((float*)Cv)[(long)m * ldc + n] = v;
            }
        }
    }
}

template <typename T>
static cudaError_t launch_gemm_simt_t(const GemmSimtArgs& a, cudaStream_t st)
{
    int shards = a.shard_dim ? a.shards : 1;
    int Mmax = a.M, Nmax = a.N, gz = 1;
    if (a.shard_dim == 1) { Nmax = cdiv(a.N, shards); gz = shards; }
    if (a.shard_dim == 3) { Mmax = cdiv(a.M, shards); gz = shards; }
    dim3 grid(cdiv(Nmax, 64), cdiv(Mmax, 64), gz);
    PtrTab tab{};
    if (a.tab) tab = *a.tab;
    const int tab_mode = a.tab ? a.tab_mode : 0;
#define SB_GM(E)                                                                                                    \
    SB_LAUNCH((gemm_simt_kernel<T, E>), grid, 256, 0, st, (const T*)a.A, a.sAm, a.sAk, (const T*)a.B, a.sBn, a.sBk, a.M, a.N, a.K, \
                                                 a.C, a.ldc, a.C32, a.bias, a.relu, (const T*)a.ref, a.ldref, a.shard_dim, shards, \
                                                 tab, tab_mode, a.tab_b > 0 ? a.tab_b : 1)
    if (a.epi == EPI_BIAS_ACT) SB_GM(EPI_BIAS_ACT);
    else if (a.epi == EPI_MASK) SB_GM(EPI_MASK);
    else SB_GM(EPI_F32);
#undef SB_GM
    return cudaGetLastError();
}
cudaError_t launch_gemm_simt(const GemmSimtArgs& a, bool bf16, cudaStream_t st)
{
    return bf16 ? launch_gemm_simt_t<__nv_bfloat16>(a, st) : launch_gemm_simt_t<float>(a, st);
}

}  // namespace sb
