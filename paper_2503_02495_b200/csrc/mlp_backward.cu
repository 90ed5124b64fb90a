// uoe_mlp_backward (derivative of Eq. 38-40 with the selection held constant).
#include "kernels.cuh"

namespace uoe {
size_t mlp_bwd_workspace_bytes(const Dims& D) { (void)D; return 0; }
}  // namespace uoe

using namespace uoe;

extern "C" uoe_status uoe_mlp_backward(const uoe_problem* prob, const void* x, const void* W1, const void* W2,
                                       const void* W_r, const int32_t* expert_idx, const int32_t* patch_idx,
                                       const float* gate, const int32_t* expert_offsets, const float* p_samp,
                                       const float* p_patch, const void* saved_h, const void* dy, void* dx,
                                       float* dW1, float* dW2, float* dW_r, void* ws, size_t ws_bytes,
                                       void* cuda_stream) {
    (void)prob; (void)x; (void)W1; (void)W2; (void)W_r; (void)expert_idx; (void)patch_idx; (void)gate;
    (void)expert_offsets; (void)p_samp; (void)p_patch; (void)saved_h; (void)dy; (void)dx; (void)dW1; (void)dW2;
    (void)dW_r; (void)ws; (void)ws_bytes; (void)cuda_stream;
    return UOE_ERR_UNSUPPORTED;
}
