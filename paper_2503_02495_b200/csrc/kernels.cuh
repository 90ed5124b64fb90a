// Internal launch interface between the entry points (route.cu, mlp.cu, smha.cu, api.cu) and the kernels.
#pragma once
#include "common.cuh"

namespace uoe {

size_t route_workspace_bytes(const Dims& D);
size_t mlp_fwd_workspace_bytes(const Dims& D);
size_t mlp_bwd_workspace_bytes(const Dims& D);
size_t smha_fwd_workspace_bytes(const Dims& D);
size_t smha_bwd_workspace_bytes(const Dims& D);
size_t balance_bwd_workspace_bytes(const Dims& D);

// Layout of the routing plan inside a workspace: where each (sample, expert) pair's rows start and,
// for every patch of every sample, which routed rows and gates feed it back (the inverse of Eq. 18).
struct PlanPtrs {
    int* pair_row = nullptr;     // [B,k]    first routed row of (b, s)
    int* inv_row = nullptr;      // [B,m,k]  first routed row of patch j in slot s, or -1; when the router wrote the plan:
                                 //          the row's offset from pair_row[b,s] (inv_relative)
    float* inv_gate = nullptr;   // [B,m,k]
    int* expert_end = nullptr;   // [n]      first padding row of expert i's region
    float* row_gate = nullptr;   // [Rmax]   backward only: combine weight of each routed row (0 on pad-token rows and unused slots)
    float* row_valid = nullptr;  // [Rmax]   backward only: 1 on rows that hold a real token, else 0
    int* src_patch = nullptr;    // [Rmax/l_p] source patch (b*m + j) of every l_p-row block of the routed buffers, -1 = zero rows
    int* slot_pair = nullptr;    // [n,B]    plan written by the router kernel: pair (b*k + s) of the q-th sample in expert i's
                                 //          region (it replaces src_patch, which that plan does not fill)
    bool inv_relative = false;   // inv_row holds offsets from pair_row (plan written by the router kernel)
    // plan written by the router kernel, whole samples per expert (every chosen expert takes every patch that holds a
    // real token, Eq. 21-26): slot u of a pair is patch u, so inv_row, inv_gate and patch_idx are neither written nor
    // read; the combine takes its weights from the router's gate array [B,k,c]
    bool identity_patches = false;
    const float* gate = nullptr;
    // plan written by the router kernel only: a routed buffer whose first rows past the last expert region are
    // zero-filled (up to 128 of them, as many as a 128-row tile that starts inside the last region can reach)
    uint4* tail = nullptr;
    long long tail_row_vecs = 0, rows_max = 0;
};

// Device arrays that uoe_route writes (shapes as in uoe.h).
struct RoutingPtrs {
    int* expert_idx = nullptr;
    int* patch_idx = nullptr;
    float* gate = nullptr;
    float* p_samp = nullptr;
    float* p_patch = nullptr;
    int* expert_offsets = nullptr;
};

// uoe_route on a scratch area laid out as route_workspace_bytes describes (its control block zeroed once).  With
// `plan` the routing plan is written by the same kernels (inv_row relative to pair_row), so no plan kernel is needed;
// route_can_plan says whether the problem allows that.
bool route_can_plan(const Dims& D);
// Whether the router treats the problem as pure expert selection (whole samples per expert, Eq. 21-26): then a plan it
// writes has identity_patches set and holds no inverse map.
inline bool route_whole_samples(const Dims& D, uint32_t flags) {
    return !(flags & (UOE_FLAG_DYNAMIC_C | UOE_FLAG_GENERAL_PATH)) && D.c >= (D.Lv + D.l_p - 1) / D.l_p;
}
uoe_status route_run(const uoe_problem* prob, const void* x, const void* W_r, const RoutingPtrs& r, char* scratch,
                     cudaStream_t stream, const PlanPtrs* plan);
// Gathering through the GEMM's own TMA loads needs whole patches inside a 128-row tile, 8-row swizzle groups
// and 64-column K steps.
inline bool can_fuse_gather(const Dims& D) {
    return D.bf16 && D.l_p % 8 == 0 && 128 % D.l_p == 0 && D.d % 64 == 0;
}
inline size_t plan_bytes(const Dims& D, bool with_rows = false) {
    return align_up((size_t)D.B * D.k * 4, 1024) + 2 * align_up((size_t)D.B * D.m * D.k * 4, 1024) + 1024 +
           (with_rows ? 2 * align_up((size_t)D.Rmax * 4, 1024) : 0) + align_up((size_t)(D.Rmax / D.l_p + 1) * 4, 1024) +
           align_up((size_t)D.n * D.B * 4, 1024);
}
inline PlanPtrs plan_ptrs(const Dims& D, char* base, bool with_rows = false) {
    PlanPtrs p;
    p.pair_row = (int*)base;
    base += align_up((size_t)D.B * D.k * 4, 1024);
    p.inv_row = (int*)base;
    base += align_up((size_t)D.B * D.m * D.k * 4, 1024);
    p.inv_gate = (float*)base;
    base += align_up((size_t)D.B * D.m * D.k * 4, 1024);
    p.expert_end = (int*)base;
    base += 1024;
    p.row_gate = with_rows ? (float*)base : nullptr;
    base += with_rows ? align_up((size_t)D.Rmax * 4, 1024) : 0;
    p.row_valid = with_rows ? (float*)base : nullptr;
    base += with_rows ? align_up((size_t)D.Rmax * 4, 1024) : 0;
    p.src_patch = (int*)base;
    base += align_up((size_t)(D.Rmax / D.l_p + 1) * 4, 1024);
    p.slot_pair = (int*)base;
    return p;
}

// Where the rows of a gathered operand come from (Eq. 18 inside a kernel's own loads): either the table that the
// plan kernel writes (src_patch[row / l_p]) or, with the plan the router kernel writes, derived per row block from the
// pair that owns the block (slot_pair) and that pair's selected patches (patch_idx).
struct SrcMap {
    const int* src_patch = nullptr;
    const int* slot_pair = nullptr;    // [n,B]
    const int* patch_idx = nullptr;    // [B,k,c]
    const int* expert_end = nullptr;   // [n]
    int B = 0, k = 0, c = 0, m = 0, l_p = 0;
    int n_elig = -1;                   // >= 0: slot u of a pair is patch u for u < n_elig (whole samples per expert), patch_idx is not read
    __host__ __device__ bool on() const { return src_patch != nullptr || slot_pair != nullptr; }
};
inline SrcMap src_map_of(const Dims& D, const PlanPtrs& P, const int* patch_idx) {
    SrcMap g;
    if (P.inv_relative) { g.slot_pair = P.slot_pair; g.patch_idx = patch_idx; g.expert_end = P.expert_end; }
    else g.src_patch = P.src_patch;
    if (P.inv_relative && P.identity_patches) g.n_elig = (D.Lv + D.l_p - 1) / D.l_p;
    g.B = D.B; g.k = D.k; g.c = D.c; g.m = D.m; g.l_p = D.l_p;
    return g;
}
#ifdef __CUDACC__
// Source patch (index into the [Bm patches] view of the source tensor) of the l_p-row block that starts at routed row
// r inside the region of expert e (first row off_e); Bm (out of range: the loads return zeros) for padding rows and
// unused slots.
__device__ __forceinline__ int src_of(const SrcMap& g, int r, int e, int off_e, int Bm) {
    int src;
    if (g.src_patch) {
        src = g.src_patch[r / g.l_p];
    } else {
        src = -1;
        if (r < g.expert_end[e]) {
            const int rel = r - off_e, l_a = g.c * g.l_p;
            const int pair = g.slot_pair[(size_t)e * g.B + rel / l_a];
            const int u = (rel % l_a) / g.l_p;
            const int pj = g.n_elig >= 0 ? (u < g.n_elig ? u : -1) : g.patch_idx[(size_t)pair * g.c + u];
            if (pj >= 0 && pj < g.m) src = (pair / g.k) * g.m + pj;
        }
    }
    return src < 0 ? Bm : src;
}
#endif

// use_gate only matters for the per-row arrays of the backward (row_gate = gate or 1).
// If tail is not null, rows [offsets[n], Rmax) of tail (rows of tail_row_bytes) are zero-filled.
uoe_status launch_plan(const Dims& D, const int* expert_idx, const int* patch_idx, const float* gate,
                       const int* offsets, const PlanPtrs& P, int* status, cudaStream_t s, bool use_gate = true,
                       void* tail = nullptr, long long tail_row_bytes = 0);

// Eq. 18 / 24: copy the selected patches of `src` [B,L,d] into the routed buffer `dst` [rows,d];
// unused slots and the padding rows of each expert region are zero-filled.
// If tail is not null, rows [offsets[n], rows_max) of tail (rows of tail_row_bytes) are zero-filled too.
uoe_status launch_gather(const Dims& D, const void* src, const int* patch_idx, const int* offsets,
                         const PlanPtrs& P, void* dst, cudaStream_t s, void* tail = nullptr,
                         long long tail_row_bytes = 0);

// Eq. 20 / 26 / 36 / 40: y[b,t,:] = (residual ? x[b,t,:] : 0) + sum_s w_s * z[row_s(t),:], every output row
// written once, contributions added in ascending slot order.  w_s = gate if use_gate else 1.
// If rvec is not null (backward through the router), every real token of patch (b,j) also receives the
// vector rvec[b*m + j, :]  (float32 [B*m, d]).
uoe_status launch_combine(const Dims& D, const void* x, const void* z, const PlanPtrs& P, bool residual,
                          bool use_gate, void* y, cudaStream_t s, const float* rvec = nullptr);

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
    // bf16 path, backward epilogue (bwd = true): with u = A @ W (the gradient w.r.t. the activation output,
    // before the gate), h = bwd_h[r,:] the saved pre-activation:
    //   C  [r,:] = row_gate[r] * u * phi'(h)         (gradient w.r.t. the pre-activation)
    //   C1 [r,:] = row_gate[r] * phi(h)              (gated activation, operand of the weight gradient)
    //   dg_part[r, column tile] = row_valid[r] * sum over the tile's columns of u * phi(h)
    // bf16 path, gathered A (Eq. 18 inside the GEMM): if gather_x is not null, A is ignored and row block q of a
    // tile is loaded from patch src_patch[tile*128/l_p + q] of gather_x [Bm patches, l_p, K]
    const void* gather_x = nullptr;
    const int* src_patch = nullptr;
    int l_p = 0, Bm = 0;
    SrcMap map;             // if map.on(): used instead of src_patch (the router-written plan has no src_patch table)
    // bf16 path, forward epilogue: C[r,:] is multiplied, after the activation, by blk_scale[r / 128] (one combine weight
    // per 128-row block, Eq. 40 applied ahead of the second layer; `pre` keeps the unscaled pre-activation)
    const float* blk_scale = nullptr;
    bool bwd = false;
    const void* bwd_h = nullptr;
    const float* row_gate = nullptr;
    const float* row_valid = nullptr;
    float* dg_part = nullptr;
};

// Column-tile width the bf16 grouped GEMM uses for N output columns (dg_part has N / that many columns).
inline int gemm_bf16_bn(int N) { return (N % 256 == 0) ? 256 : (N % 128 == 0 ? 128 : 64); }

// Per-expert weight gradient over ragged row counts:  dW[e] [M, N] (float32, overwritten) =
// sum over the rows r of expert e's region of  P[r, 0:M]^T  Q[r, 0:N]   (P [rows, M], Q [rows, N], bf16).
// Rows of a region beyond its real rows must be zero in P or Q.
// `part`: scratch of wgrad_scratch_bytes(n, M, N, rows_max) bytes for the split-K partial outputs (may be null when
// that is 0; with null the contraction is never split).
size_t wgrad_scratch_bytes(int n, int M, int N, long long rows_max);
// Gathered operands (Eq. 18 inside the weight-gradient contraction): with gather_p (gather_q) the pointer P (Q) is
// the source tensor [Bm patches, l_p, M (N)] and routed row r is row r % l_p of patch src_patch[r / l_p]
// (-1 = zero rows).  Needs every 64-row K block to be whole slabs inside whole patches, with regions (multiples of
// 128 rows) starting on patch boundaries:
inline bool wgrad_can_gather(int l_p) { return l_p >= 16 && 128 % l_p == 0; }
struct WgradGather {
    bool gather_p = false, gather_q = false;
    const int* src_patch = nullptr;
    int l_p = 64, Bm = 0;
};
uoe_status launch_wgrad_bf16(const void* P, const void* Q, float* dW, const int* offsets, int n, int M, int N,
                             long long rows_max, const char* label, int* status, cudaStream_t s, float* part = nullptr,
                             const WgradGather& g = WgradGather());
uoe_status launch_gemm_f32(const GemmArgs& g, cudaStream_t s);

// Scratch of the router half of a backward pass (all float32).
struct RouterBwdScratch {
    float* G;       // [B*m, n]   gradient of the router logits per (sample, patch)
    float* pool;    // [B*m, d]   sums of the real rows of each patch
    float* rvec;    // [B*m, d]   W_r G: added to dx on every real token of the patch
    float* dgate;   // [B,k,c]
    float* wpart;   // partial sums of dW_r
};
size_t router_backward_scratch_bytes(const Dims& D);
RouterBwdScratch router_backward_scratch(const Dims& D, char* base);
// dgp: [rows, nt] float32, per-row partials of d(loss)/d(gate) (zero on rows that hold no real token).
uoe_status launch_router_backward(const Dims& D, const void* x, const void* W_r, const int* expert_idx,
                                  const int* patch_idx, const float* p_samp, const float* p_patch, const PlanPtrs& P,
                                  const float* dgp, int nt, const RouterBwdScratch& rs, float* dW_r, cudaStream_t stream);
uoe_status launch_gemm_bf16(const GemmArgs& g, int* status, cudaStream_t s);

// Eq. 38-39 in one kernel for narrow experts (bf16, d_e = 256, d <= 512): z = phi(A W1[e]) W2[e] with the hidden tile
// kept on chip.  A [rows, d] is a routed buffer, or gathered from gather_x through src_patch as in GemmArgs;
// pre (optional) [rows, 256] receives the pre-activation.
bool mlp_can_fuse(const Dims& D);
uoe_status launch_mlp_fused(const Dims& D, const void* A, const void* W1, const void* W2, void* z, void* pre,
                            const int* offsets, int act, const void* gather_x, const SrcMap& map, int* status,
                            cudaStream_t s, const void* b1 = nullptr, const void* b2 = nullptr);

// ---- forward halves behind the routing plan (shared by the per-half entry points and the block entry) ----
struct MlpFwdBufs { void* xg; void* a; void* z; };
// Second layer + combine walked by output patch (patches of 128 tokens): whether the problem and plan allow it, the
// per-block combine weights it needs the first layer to apply, and the launch itself.
bool gemm2_patch_can(const Dims& D, const PlanPtrs& P, const void* b2);
uoe_status launch_block_gate(const Dims& D, const PlanPtrs& P, bool use_gate, float* blk, cudaStream_t s);
// (w_kmajor: the weights are [n, d, d_e] and the product is a' W^T, the backward's dx; rvec [B*m, d]: added on real tokens)
uoe_status launch_gemm2_patch(const Dims& D, const void* a, const void* W2, const void* x, void* y, const int* offsets,
                              const PlanPtrs& P, bool residual, int* status, cudaStream_t s, bool w_kmajor = false,
                              const float* rvec = nullptr, const char* label = "gemm2");
struct SmhaFwdBufs { void *xg, *q, *k, *v, *o, *z; };
struct SmhaFwdOffsets { size_t xg, q, k, v, o, z; };
// bytes of the routed buffers of a forward half and their offsets (0 for a buffer the path does not need)
size_t mlp_fwd_buffer_bytes(const Dims& D, size_t* xg, size_t* a, size_t* z);
size_t smha_fwd_buffer_bytes(const Dims& D, SmhaFwdOffsets* o);
uoe_status mlp_forward_check(const uoe_problem* prob, Dims& D, const void* x, const void* W1, const void* W2,
                             const void* b1, const void* b2, const void* y, const void* saved_h);
uoe_status mlp_forward_run(const Dims& D, const uoe_problem* prob, const void* x, const void* W1, const void* W2,
                           const void* b1, const void* b2, const int* patch_idx, const int* expert_offsets,
                           const PlanPtrs& P, const MlpFwdBufs& bufs, void* y, void* saved_h, int* status,
                           cudaStream_t stream);
uoe_status smha_forward_check(const uoe_problem* prob, Dims& D, const void* x, const void* Wq, const void* Wk,
                              const void* Wv, const void* Wo, const void* y);
uoe_status smha_forward_run(const Dims& D, const uoe_problem* prob, const void* x, const void* Wq, const void* Wk,
                            const void* Wv, const void* Wo, const int* expert_idx, const int* patch_idx,
                            const int* expert_offsets, const PlanPtrs& P, const SmhaFwdBufs& bufs, void* y, float* lse,
                            int* status, cudaStream_t stream);

}  // namespace uoe
