// Internal declarations shared by the host-side planner (sb_api.cu) and the kernel files.
// Nothing here is part of the public C ABI (see include/splitbrain.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include <cstdlib>
#include <utility>

namespace sb {

constexpr int MAX_PARTS = 64;  // upper bound on R and K

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  Every kernel of the library starts with pdl_prologue(): it waits until the
// kernels it depends on have completed (griddepcontrol.wait, a no-op for a normally launched kernel) and
// then lets the next kernel in the stream start launching (griddepcontrol.launch_dependents), so that the
// next kernel's launch latency and set-up overlap this kernel's execution.  Nothing is read from or written
// to global memory before the wait.  SB_PDL=0 in the environment launches everything the classic way.
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_prologue() { pdl_wait(); pdl_trigger(); }
#endif
// Tuning constants of the planner.  The shipped library uses the compiled-in defaults; a development build
// (-DSB_DEV_TUNING) lets an environment variable of the same name override each one for A/B measurements.
inline double tune(const char* name, double dflt)
{
#ifdef SB_DEV_TUNING
    const char* e = getenv(name);
    return e ? atof(e) : dflt;
#else
    (void)name;
    return dflt;
#endif
}
// (the calling thread can switch the attribute off for the launches it enqueues next: pdl_classic() = 1 ... = 0)
inline int& pdl_classic() { static thread_local int off = 0; return off; }
// Set by the calling thread around a launch whose predecessor in the stream is known not to have written the layer's weights
// (a kernel of the same forward or backward pass): the tensor-core kernel may then fetch weights before it waits for it.
inline int& weights_first() { static thread_local int on = 0; return on; }
inline bool pdl_enabled()
{
    static const bool on = [] { const char* e = getenv("SB_PDL"); return !(e && e[0] == '0'); }();
    return on && !pdl_classic();
}
template <typename... KArgs, typename... Args>
inline cudaError_t pdl_launch(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(std::forward<Args>(args))...);
}
#define SB_LAUNCH(kern, grid, block, smem, st, ...) (void)::sb::pdl_launch((kern), dim3(grid), dim3(block), (size_t)(smem), (st), __VA_ARGS__)


// Pointer table for per-replica caller buffers (inputs, labels): passed by value to kernels.
struct PtrTab {
    const void* p[MAX_PARTS];
};

// Device status word codes (written by kernels that give up on a bounded wait).
enum : uint32_t { DEV_OK = 0, DEV_TIMEOUT_TMA = 1, DEV_TIMEOUT_MMA = 2, DEV_TIMEOUT_EPI = 3, DEV_PAIR_TMEM = 4 };

// ---------------------------------------------------------------------------------------------
// CUDA-core ("SIMT") kernels: the float mode, odd channel counts, and the cross-check path.
// All launchers return the cudaError_t of the launch.  `bf16` selects the activation dtype
// (false: float, true: __nv_bfloat16) of every T-typed pointer.
// ---------------------------------------------------------------------------------------------

struct ConvSimtArgs {
    const void* in;       // [B,H,W,Cred] activation dtype (ignored when tab != nullptr)
    const PtrTab* tab;    // optional: R per-replica input pointers (host pointer to the table)
    int b_per_rep;
    const void* w;        // [Cout,3,3,Cin] activation dtype (float master or bf16 shadow)
    const float* bias;    // [Cout] (forward only)
    void* out;            // [B,H,W,Cres] activation dtype
    const void* mask_ref; // dgrad only, optional: zero the result where mask_ref <= 0 ([B,H,W,Cres])
    int B, H, W, Cin, Cout;
    int dgrad;            // 0: forward (+bias, ReLU if relu) ; 1: data gradient
    int relu;
};
cudaError_t launch_conv_simt(const ConvSimtArgs& a, bool bf16, cudaStream_t st);

struct WgradSimtArgs {
    const void* x;        // [B,H,W,Cin] (ignored when tab != nullptr)
    const PtrTab* tab;
    int b_per_rep;
    const void* dy;       // [B,H,W,Cout]
    float* part;          // [splits][Cout*9*Cin] partial sums (or the gradient itself if splits==1)
    int B, H, W, Cin, Cout;
    int splits;           // pixel-range splits; split s covers images [s*B/splits, (s+1)*B/splits)
};
cudaError_t launch_wgrad_simt(const WgradSimtArgs& a, bool bf16, cudaStream_t st);

// Input-layer convolution (Cin of 1, 3 or 4; Cout a multiple of 8): dedicated forward and weight+bias
// gradient kernels.  The gradient kernel writes conv_in_wgrad_blocks() partial buffers of
// Cout*9*Cin + Cout floats each (weights, then bias) into a.part, to be reduced in block order.
bool conv_in_supported(int Cin, int Cout);
cudaError_t launch_conv_in_fwd(const ConvSimtArgs& a, bool bf16, cudaStream_t st);
int conv_in_wgrad_blocks(int B, int H, int W);
cudaError_t launch_conv_in_wgrad(const WgradSimtArgs& a, bool bf16, cudaStream_t st);

// Narrow FC layer (out <= 16): pass 0 forward, 1 weight+bias gradient, 2 input gradient.
struct FcNarrowArgs {
    int pass;
    const void* X; const PtrTab* tab; int tab_b;   // [B,in] activations (or R per-replica buffers of tab_b rows)
    const void* W;                                 // [out,in] activation dtype
    const float* bias; void* Y; float* Y32; int relu;   // forward outputs (either may be null)
    const void* dY; float* dW; float* db;          // gradient inputs/outputs
    const void* ref; void* dX;                     // dgrad: optional ReLU mask source and output [B,in]
    int B, in_f, out_f;
};
bool fc_narrow_supported(int out_f, int B);
cudaError_t launch_fc_narrow(const FcNarrowArgs& a, bool bf16, cudaStream_t st);

// part[s][n] = sum over the rows of split s of in[row][n];  rows split evenly (M % splits == 0).
cudaError_t launch_colsum(const void* in, bool bf16, float* part, int M, int N, int splits, cudaStream_t st);
// out[i] = sum_{s<splits} part[s*stride + i], s ascending.
cudaError_t launch_reduce_partials(const float* part, size_t stride, float* out, size_t n, int splits, cudaStream_t st);
// the same ordered sum, consumed at once by the SGD step of the n parameters at w / v (shadow: their bf16 copies or nullptr)
cudaError_t launch_reduce_sgd(const float* part, size_t stride, size_t n, int splits, float* w, float* v, __nv_bfloat16* shadow,
                              float lr, float mu, cudaStream_t st);

struct PoolArgs {
    const void* x;  // [B,H,W,C]
    void* p;        // [B,H/2,W/2,C]
    uint8_t* idx;   // [B,H/2,W/2,C]
    int B, H, W, C;
};
cudaError_t launch_pool_fwd(const PoolArgs& a, bool bf16, cudaStream_t st);
struct PoolBwdArgs {
    const void* dp;      // [B,H/2,W/2,C] gradient w.r.t. the pooled output
    const uint8_t* idx;
    const void* p;       // pooled output (ReLU mask source) or nullptr for no mask
    void* dx;            // [B,H,W,C]
    int B, H, W, C;
};
cudaError_t launch_pool_bwd(const PoolBwdArgs& a, bool bf16, cudaStream_t st);

struct XentArgs {
    const float* logits;  // [B,C]
    PtrTab labels;        // R pointers to int32 [b]
    int b_per_rep;
    float* row_loss;      // [B]
    float* loss;          // [1] mean over rows
    void* dZ;             // [B,C] activation dtype: (softmax - onehot)/B
    unsigned int* counter; // zero-initialised word; left at zero
    int B, C;
    // Sub-batch use (modulo schedule): the rows above are a slice of a larger batch.  scale_B > 0 replaces B in the
    // 1/B of dZ; loss_rows > 0 makes the mean loss the sum of loss_base[0 .. loss_rows) divided by loss_rows.
    int scale_B = 0;
    const float* loss_base = nullptr;
    int loss_rows = 0;
};
cudaError_t launch_softmax_xent(const XentArgs& a, bool bf16, cudaStream_t st);

// Modulo layer as an explicit copy (sub-iteration schedule): R replicas of b rows, K slices of b/K rows each.
// gather : dst[k*(R*b/K) + r*(b/K) + i] = src[r*b + k*(b/K) + i]   (rows of `row_bytes` bytes, a multiple of 16)
// scatter: the inverse.  labels (optional, gather only): int32 per row, read through the per-replica table.
struct ModuloCopyArgs {
    const void* src;
    void* dst;
    size_t row_bytes;
    int R, b, K;
    int scatter;               // 0: gather, 1: scatter
    const PtrTab* labels;      // gather only: R pointers to int32 [b]; nullptr = no labels
    int32_t* labels_out;       // [R*b] in sub-iteration order
};
cudaError_t launch_modulo_copy(const ModuloCopyArgs& a, cudaStream_t st);

// Dropout layer on a [rows, width] activation matrix (units = drop probability * 65536): y = keep ? x / (1 - p) : 0 with the
// keep bit of logical element (row, column) drawn by a counter-based generator from `state` = {seed lo, seed hi, iteration}
// (device memory) and the layer index; backward: dx = dy / (1 - p) (dy arrives zero where the output was zero).
// sub_bk > 0: the rows are sub-iteration sub_k of the modulo schedule (sub_bk rows of each replica's sub_b); masks follow the batch rows
cudaError_t launch_dropout_fwd(const void* x, void* y, size_t rows, int width, const uint32_t* state, int layer, int units, bool bf16, cudaStream_t st,
                               int sub_bk = 0, int sub_b = 0, int sub_k = 0);
cudaError_t launch_dropout_bwd(const void* dy, void* dx, size_t n, int units, bool bf16, cudaStream_t st);
// mode 0: state <- {seed, iteration}; mode 1: iteration += 1
cudaError_t launch_dropout_state(uint32_t* state, int mode, uint64_t seed, uint32_t iteration, cudaStream_t st);

cudaError_t launch_sgd(float* w, float* v, const float* g, __nv_bfloat16* shadow, size_t n,
                       float lr, float mu, cudaStream_t st);
cudaError_t launch_to_bf16(const float* w, __nv_bfloat16* shadow, size_t n, cudaStream_t st);

enum { EPI_BIAS_ACT = 0, EPI_MASK = 1, EPI_F32 = 2 };
// Ordered sum of split-reduction partial sums [split][rows][N] followed by the GEMM epilogue
// (epi = EPI_BIAS_ACT or EPI_MASK below); N must be a multiple of 4.
struct SplitKEpiArgs {
    const float* part; size_t split_stride; int splits;
    long rows; int N;
    int epi; const float* bias; int relu; const void* ref;
    void* out; int out_f32;
};
cudaError_t launch_splitk_epilogue(const SplitKEpiArgs& a, cudaStream_t st);

// Strided GEMM  C[m,n] = sum_k A(m,k) * B(n,k)  with A(m,k) = A[m*sAm + k*sAk], B(n,k) = B[n*sBn + k*sBk].
struct GemmSimtArgs {
    const void* A; long sAm, sAk;
    const void* B; long sBn, sBk;
    int M, N, K;
    int epi;
    void* C; long ldc;        // activation dtype (EPI_BIAS_ACT, EPI_MASK) or float (EPI_F32)
    float* C32;               // EPI_BIAS_ACT: optional float copy of the result (logits), same ldc
    const float* bias;        // EPI_BIAS_ACT: [N]
    int relu;
    const void* ref; long ldref;  // EPI_MASK: optional, zero where ref <= 0
    // Model-shard partition of one GEMM dimension: 0 none, 1 = N (forward: each shard owns its
    // output columns), 2 = K (dgrad: sum over shards), 3 = M (wgrad: each shard owns its rows).
    int shard_dim, shards;
    // Optional replica gather by addressing: the rows of the activation matrix live in R separate
    // caller buffers of tab_b rows each.  tab_mode 1: A's m index is the row; 2: B's k index is.
    const PtrTab* tab; int tab_mode, tab_b;
};
cudaError_t launch_gemm_simt(const GemmSimtArgs& a, bool bf16, cudaStream_t st);

}  // namespace sb
