// tcgen05 tensor-core path (placeholder: every layer falls back to the CUDA-core kernels).
#include "sb_umma.h"
namespace sb {
sb_status umma_plan_scratch(sb_model*, size_t* floats) { *floats = 0; return SB_OK; }
sb_status umma_plan_layers(sb_model*) { return SB_OK; }
sb_status umma_conv_fwd(sb_model*, int, cudaStream_t) { return SB_ERR_UNSUPPORTED; }
sb_status umma_conv_dgrad(sb_model*, int, cudaStream_t) { return SB_ERR_UNSUPPORTED; }
sb_status umma_conv_wgrad(sb_model*, int, cudaStream_t) { return SB_ERR_UNSUPPORTED; }
sb_status umma_fc_fwd(sb_model*, int, cudaStream_t) { return SB_ERR_UNSUPPORTED; }
sb_status umma_fc_dgrad(sb_model*, int, cudaStream_t) { return SB_ERR_UNSUPPORTED; }
sb_status umma_fc_wgrad(sb_model*, int, cudaStream_t) { return SB_ERR_UNSUPPORTED; }
}
