// Entry points that launch nothing: sizes, status text, status read-back, launch counter.
#include "kernels.cuh"
#include "tmap.cuh"

#include <vector>

namespace uoe {
namespace {
struct ProfRec { const char* name; cudaEvent_t e0, e1; };
bool g_prof_on = false;
std::vector<ProfRec> g_prof;
}  // namespace

ProfScope::ProfScope(const char* name, cudaStream_t s) : slot(-1), stream(s) {
    if (!g_prof_on || !name) return;
    ProfRec r{name, nullptr, nullptr};
    if (cudaEventCreate(&r.e0) != cudaSuccess || cudaEventCreate(&r.e1) != cudaSuccess) return;
    cudaEventRecord(r.e0, s);
    g_prof.push_back(r);
    slot = (int)g_prof.size() - 1;
}
ProfScope::~ProfScope() {
    if (slot >= 0) cudaEventRecord(g_prof[slot].e1, stream);
}
}  // namespace uoe

using namespace uoe;

extern "C" void uoe_profile_enable(int on) {
    if (on) {
        for (auto& r : g_prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
        g_prof.clear();
    }
    g_prof_on = on != 0;
}

extern "C" int uoe_profile_count(void) { return (int)g_prof.size(); }

extern "C" uoe_status uoe_profile_get(int i, const char** name, float* ms) {
    if (i < 0 || i >= (int)g_prof.size() || !name || !ms) return UOE_ERR_INVALID_ARG;
    if (cudaEventSynchronize(g_prof[i].e1) != cudaSuccess) return UOE_ERR_CUDA;
    if (cudaEventElapsedTime(ms, g_prof[i].e0, g_prof[i].e1) != cudaSuccess) return UOE_ERR_CUDA;
    *name = g_prof[i].name;
    return UOE_OK;
}

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
        case UOE_OP_SMHA_BWD: return D.H > 0 ? smha_bwd_workspace_bytes(D) : 0;
        case UOE_OP_BALANCE_BWD: return balance_bwd_workspace_bytes(D);
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
        case UOE_ERR_STATIC_SCRATCH: return "problem too large for the built-in static scratch of uoe_route_static";
        default: return "unknown status";
    }
}

extern "C" uoe_status uoe_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream) {
    if (!ws || ws_bytes < kStatusBytes) return UOE_ERR_INVALID_ARG;
    const size_t bytes = ws_bytes < kControlBytes ? ws_bytes : kControlBytes;
    if (cudaMemsetAsync(ws, 0, bytes, (cudaStream_t)cuda_stream) != cudaSuccess) return UOE_ERR_CUDA;
    return UOE_OK;
}

extern "C" uoe_status uoe_read_device_status(void* ws, void* cuda_stream) {
    if (!ws) return UOE_ERR_INVALID_ARG;
    int v = 0;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(&v, ws, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return UOE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return UOE_ERR_CUDA;
    if (v != 0) {      // read and clear: the next anomaly can be recorded again
        if (cudaMemsetAsync(ws, 0, sizeof(int), s) != cudaSuccess) return UOE_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return UOE_ERR_CUDA;
    }
    return (uoe_status)v;
}

extern "C" int64_t uoe_launch_count(void) { return g_launch_count; }

extern "C" int64_t uoe_tensor_map_encodings(void) { return tmap_encode_count(); }
