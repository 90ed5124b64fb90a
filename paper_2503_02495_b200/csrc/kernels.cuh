// Internal launch interface between the entry points (route.cu, mlp.cu, smha.cu, api.cu) and the kernels.
#pragma once
#include "common.cuh"

namespace uoe {

size_t route_workspace_bytes(const Dims& D);
size_t mlp_fwd_workspace_bytes(const Dims& D);
size_t mlp_bwd_workspace_bytes(const Dims& D);
size_t smha_fwd_workspace_bytes(const Dims& D);

// Layout of the routing plan inside a workspace: where each (sample, expert) pair's rows start and,
// for every patch of every sample, which routed rows and gates feed it back (the inverse of Eq. 18).
struct PlanPtrs {
    int* pair_row;     // [B,k]    first routed row of (b, s)
    int* inv_row;      // [B,m,k]  first routed row of patch j in slot s, or -1
    float* inv_gate;   // [B,m,k]
    int* expert_end;   // [n]      first padding row of expert i's region
};
inline size_t plan_bytes(const Dims& D) {
    return align_up((size_t)D.B * D.k * 4, 1024) + 2 * align_up((size_t)D.B * D.m * D.k * 4, 1024) + 1024;
}
inline PlanPtrs plan_ptrs(const Dims& D, char* base) {
    PlanPtrs p;
    p.pair_row = (int*)base;
    base += align_up((size_t)D.B * D.k * 4, 1024);
    p.inv_row = (int*)base;
    base += align_up((size_t)D.B * D.m * D.k * 4, 1024);
    p.inv_gate = (float*)base;
    base += align_up((size_t)D.B * D.m * D.k * 4, 1024);
    p.expert_end = (int*)base;
    return p;
}

uoe_status launch_plan(const Dims& D, const int* expert_idx, const int* patch_idx, const float* gate,
                       const int* offsets, const PlanPtrs& P, int* status, cudaStream_t s);

// Eq. 18 / 24: copy the selected patches of `src` [B,L,d] into the routed buffer `dst` [rows,d];
// unused slots and the padding rows of each expert region are zero-filled.
// If tail is not null, rows [offsets[n], rows_max) of tail (rows of tail_row_bytes) are zero-filled too.
uoe_status launch_gather(const Dims& D, const void* src, const int* patch_idx, const int* offsets,
                         const PlanPtrs& P, void* dst, cudaStream_t s, void* tail = nullptr,
                         long long tail_row_bytes = 0);

// Eq. 20 / 26 / 36 / 40: y[b,t,:] = (residual ? x[b,t,:] : 0) + sum_s w_s * z[row_s(t),:], every output row
// written once, contributions added in ascending slot order.  w_s = gate if use_gate else 1.
uoe_status launch_combine(const Dims& D, const void* x, const void* z, const PlanPtrs& P, bool residual,
                          bool use_gate, void* y, cudaStream_t s);

// Grouped GEMM over the routed rows: C[r,:] = epilogue(A[r,:] @ W[e(r)]) where e(r) is the expert whose
// region holds row r.  W is [n, K, N] (b_kmajor = false: rows of K, N contiguous) or [n, N, K] (true).
struct GemmArgs {
    const void* A;          // [rows_max, K]
    const void* W;          // expert weights
    const void* bias;       // [n, N] or null (float32 path only)
    void* C;                // [rows_max, N]
    void* pre;              // optional [rows_max, N]: value before the activation
    const int* offsets;     // [n+1] device
    int n, K, N;
    int act;                // uoe_act applied in the epilogue (UOE_ACT_IDENTITY = none)
    bool b_kmajor;
    long long rows_max;     // host bound on offsets[n] (rows the buffers hold)
    // bf16 path only: up to three weight tensors of the same shape applied to the same A in one launch
    // (the q, k, v projections of Eq. 28-30); matrix q writes C (q = 0), C1, C2.
    int nmat = 1;
    const void* W1 = nullptr;
    const void* W2 = nullptr;
    void* C1 = nullptr;
    void* C2 = nullptr;
    const char* label = "gemm";   // name under which the launch is profiled
};
uoe_status launch_gemm_f32(const GemmArgs& g, cudaStream_t s);
uoe_status launch_gemm_bf16(const GemmArgs& g, int* status, cudaStream_t s);

}  // namespace uoe
