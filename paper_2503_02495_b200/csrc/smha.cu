// uoe_smha_forward (Eq. 27-30, 33-36).
#include "kernels.cuh"

namespace uoe {
size_t smha_fwd_workspace_bytes(const Dims& D) { (void)D; return 0; }
}  // namespace uoe

using namespace uoe;

extern "C" uoe_status uoe_smha_forward(const uoe_problem* prob, const void* x, const void* Wq, const void* Wk,
                                       const void* Wv, const void* Wo, const int32_t* expert_idx,
                                       const int32_t* patch_idx, const float* gate, const int32_t* expert_offsets,
                                       void* y, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
    (void)prob; (void)x; (void)Wq; (void)Wk; (void)Wv; (void)Wo; (void)expert_idx; (void)patch_idx; (void)gate;
    (void)expert_offsets; (void)y; (void)lse; (void)ws; (void)ws_bytes; (void)cuda_stream;
    return UOE_ERR_UNSUPPORTED;
}
