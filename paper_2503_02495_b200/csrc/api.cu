// Entry points that launch nothing: sizes, status text, status read-back, launch counter.
#include "kernels.cuh"

using namespace uoe;

extern "C" int64_t uoe_max_routed_rows(const uoe_problem* prob) {
    Dims D;
    if (make_dims(prob, D) != UOE_OK) return 0;
    return D.Rmax;
}

extern "C" size_t uoe_workspace_bytes(const uoe_problem* prob, int op) {
    Dims D;
    if (make_dims(prob, D) != UOE_OK) return 0;
    switch (op) {
        case UOE_OP_ROUTE: return route_workspace_bytes(D);
        case UOE_OP_MLP_FWD: return D.d_e > 0 ? mlp_fwd_workspace_bytes(D) : 0;
        case UOE_OP_MLP_BWD: return D.d_e > 0 ? mlp_bwd_workspace_bytes(D) : 0;
        case UOE_OP_SMHA_FWD: return D.H > 0 ? smha_fwd_workspace_bytes(D) : 0;
        default: return 0;
    }
}

extern "C" const char* uoe_status_string(int status) {
    switch (status) {
        case UOE_OK: return "ok";
        case UOE_ERR_INVALID_ARG: return "invalid argument";
        case UOE_ERR_UNSUPPORTED: return "unsupported problem";
        case UOE_ERR_WORKSPACE: return "workspace too small";
        case UOE_ERR_CUDA: return "CUDA call failed";
        case UOE_ERR_TIMEOUT: return "device wait timed out";
        case UOE_ERR_DEVICE_INDEX: return "routing index out of range";
        default: return "unknown status";
    }
}

extern "C" uoe_status uoe_read_device_status(void* ws, void* cuda_stream) {
    if (!ws) return UOE_ERR_INVALID_ARG;
    int v = 0;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(&v, ws, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return UOE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return UOE_ERR_CUDA;
    return (uoe_status)v;
}

extern "C" int64_t uoe_launch_count(void) { return g_launch_count; }
