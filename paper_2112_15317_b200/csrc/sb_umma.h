// Interface between the host planner (sb_api.cu) and the tcgen05 tensor-core path (sb_umma.cu).
#pragma once

#include "../../include/splitbrain.h"
#include "sb_internal.h"
#include <cuda.h>

namespace sb {

// One planned tensor-core launch: tensor maps, tile geometry and epilogue pointers.
struct UmmaOp {
    bool enabled = false;
    alignas(64) CUtensorMap mapA;
    alignas(64) CUtensorMap mapB;
    alignas(64) CUtensorMap mapC;          // output tensor, for the TMA-store epilogue (when the op's tma_out is set);
                                           // FC weight gradient: the float master weights [out][in] (update folded in)
    alignas(64) CUtensorMap mapD;          // FC weight gradient: the momentum buffer, same shape
    alignas(16) unsigned char blob[512];   // kernel parameters, tile width and grid (see sb_umma.cu)
};
struct UmmaLayer {
    UmmaOp fwd, dgrad, wgrad;
    bool conv_in = false;                // input-layer conv on the tensor cores (wgrad.mapA then maps this layer's dy,
                                         // fwd.mapA its output for the TMA store)
    const void* bound_input = nullptr;   // layer 0 only: the input buffer the tensor maps currently point at
    bool pool_fused = false;             // conv layer followed by a 2x2 max-pool: the forward kernel also writes the pool layer's
                                         // output and argmax bytes from its staged output tile
};

// Read-only views of the model for the planner in sb_umma.cu.
struct ModelView {
    const sb_config* cfg;
    bool bf16;
    int B, n_layers, first_fc;
    float *Wm, *Gm, *Vm;
    __nv_bfloat16* Sm;
    float* ws;      // data-side scratch
    float* ws_wk[8];  // weight-side scratch regions, one per weight stream: layer i uses ws_wk[i % n_wstreams]
    int n_wstreams;   // 0: everything runs on the caller's stream (region 0)
    size_t ws_floats;
    uint32_t* status;
    char* input_grad;
    const PtrTab* x_tab;
    char* stage_x;        // contiguous [B, input] staging area inside the arena
};
struct LayerView {
    int kind, H, W, Cin, Cout, in_f, out_f;
    int K;                // FC: this layer's column shards
    bool relu;
    size_t p_w, p_b, n_w, n_b;
    char *act, *dact;
    unsigned char* pool_idx;   // pool layers: argmax bytes
    const char* in_act;   // previous layer's output (nullptr for layer 0)
    char* d_below;        // where the input gradient goes
    bool below_relu;
    UmmaLayer* um;
};
ModelView model_view(sb_model* m);
LayerView layer_view(sb_model* m, int i);
int64_t* launch_counter(sb_model* m);

// Scratch floats the tensor-core path needs (split partial sums); called during planning,
// before the arena exists (pointers in the views are null or unset).
sb_status umma_plan_scratch(sb_model* m, size_t* floats);
// Encodes tensor maps and decides, per layer and pass, whether the tensor-core kernel runs (layers first_layer..).
sb_status umma_plan_layers(sb_model* m, int first_layer);

sb_status umma_conv_fwd(sb_model* m, int layer, cudaStream_t st);
sb_status umma_conv_dgrad(sb_model* m, int layer, cudaStream_t st);
// Launches the weight-gradient kernel; *splits > 1 means it wrote split partial sums at *part
// (to be reduced in split order by the caller), else it wrote the gradient itself.
sb_status umma_conv_wgrad_launch(sb_model* m, int layer, cudaStream_t st, int* splits, float** part);
// false: the layer's weight-gradient kernel (CTA-pair variant) leaves the bias gradient to a column-sum kernel
bool umma_wgrad_bias_fused(sb_model* m, int layer);
// First-layer FC: points the tensor maps that read the network input at `x` ([B, in] contiguous, bf16).
sb_status umma_bind_input(sb_model* m, const void* x);
sb_status umma_fc_fwd(sb_model* m, int layer, cudaStream_t st);
sb_status umma_fc_dgrad(sb_model* m, int layer, cudaStream_t st);
sb_status umma_fc_wgrad(sb_model* m, int layer, cudaStream_t st);
// FC weight gradient with the SGD-momentum update applied in the kernel's epilogue (gradient never stored): possible when
// umma_fc_wgrad_can_update says so (unsplit reduction, staged epilogue, bias gradient in the same kernel)
bool umma_fc_wgrad_can_update(sb_model* m, int layer);
sb_status umma_fc_wgrad_update(sb_model* m, int layer, float lr, float mu, cudaStream_t st);

// Input-layer convolution (1, 3 or 4 input channels, 64 output channels, bf16) on the tensor cores.
bool conv_in_umma_supported(int Cin, int Cout);
// Partial buffers the weight-gradient kernel writes ([blocks][Cout*9*Cin + Cout] floats, reduced in block order).
int conv_in_umma_wgrad_blocks(long npix);
// mapY: optional tensor map of the output as [pixels][Cout] with a (64, 128) box (nullptr: plain stores)
cudaError_t launch_conv_in_fwd_umma(const ConvSimtArgs& a, const CUtensorMap* mapY, uint32_t* status, cudaStream_t st);
cudaError_t launch_conv_in_wgrad_umma(const WgradSimtArgs& a, const CUtensorMap& mapDy, uint32_t* status, cudaStream_t st);

const char* umma_last_error();
// One CTA that waits (bounded by limit_ns) on a barrier nothing completes, then reports through the status word.
cudaError_t launch_wait_probe(uint32_t* status, unsigned long long limit_ns, cudaStream_t st);
#ifdef SB_CTA_TIMING
// Development builds only: when set to a device buffer of 1024*16 uint64, every tensor-core CTA (first 1024 of a launch)
// records clock stamps at its phase boundaries.
void umma_set_timing_buffer(void* dev_ptr);
void umma_set_trace_buffer(void* dev_ptr);
#endif

}  // namespace sb
