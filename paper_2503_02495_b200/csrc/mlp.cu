// uoe_mlp_forward: UoME forward (Eq. 37-40) as plan -> gather (Eq. 18) -> grouped GEMM1 + phi (Eq. 38)
// -> grouped GEMM2 (Eq. 39) -> weighted combine (Eq. 20 / 40).  On the bf16 path the gather happens inside the
// first GEMM's loads, and for narrow experts (d_e = 256, d <= 512) both GEMMs are one kernel.
#include "kernels.cuh"

namespace uoe {

struct MlpFwdWs { size_t plan, xg, a, z, total; };

static MlpFwdWs mlp_fwd_ws(const Dims& D) {
    WsCarver w;
    w.take(kStatusBytes);
    MlpFwdWs r;
    r.plan = w.take(plan_bytes(D));
    r.xg = can_fuse_gather(D) ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);     // the GEMM gathers x itself
    r.a = mlp_can_fuse(D) ? 0 : w.take((size_t)D.Rmax * D.d_e * D.esize);          // the fused kernel keeps the hidden tile on chip
    r.z = w.take((size_t)D.Rmax * D.d * D.esize);
    r.total = w.off;
    return r;
}

size_t mlp_fwd_workspace_bytes(const Dims& D) { return mlp_fwd_ws(D).total; }

size_t mlp_fwd_buffer_bytes(const Dims& D, size_t* xg, size_t* a, size_t* z) {
    WsCarver w;
    *xg = can_fuse_gather(D) ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);
    *a = mlp_can_fuse(D) ? 0 : w.take((size_t)D.Rmax * D.d_e * D.esize);
    *z = w.take((size_t)D.Rmax * D.d * D.esize);
    return w.off;
}

}  // namespace uoe

// Everything of the UoME forward behind the routing plan: gather (unless the GEMM gathers), the two grouped GEMMs
// (or the one fused kernel), combine.
uoe_status uoe::mlp_forward_run(const Dims& D, const uoe_problem* prob, const void* x, const void* W1, const void* W2,
                                const void* b1, const void* b2, const int* patch_idx, const int* expert_offsets,
                                const PlanPtrs& P, const MlpFwdBufs& bufs, void* y, void* saved_h, int* status,
                                cudaStream_t stream) {
    uoe_status st;
    void *xg = bufs.xg, *a = bufs.a, *z = bufs.z;
    const bool fused = can_fuse_gather(D);
    if (!fused) {
        st = launch_gather(D, x, patch_idx, expert_offsets, P, xg, stream);
        if (st != UOE_OK) return st;
    }

    GemmArgs g1{xg, W1, b1, a, saved_h, expert_offsets, D.n, D.d, D.d_e, prob->act, false, D.Rmax};
    const SrcMap map = src_map_of(D, P, patch_idx);
    if (fused) { g1.gather_x = x; g1.map = map; g1.l_p = D.l_p; g1.Bm = D.B * D.m; }
    GemmArgs g2{a, W2, b2, z, nullptr, expert_offsets, D.n, D.d_e, D.d, UOE_ACT_IDENTITY, false, D.Rmax};
    g1.label = "gemm1_act";
    g2.label = "gemm2";
    if (!mlp_can_fuse(D) && gemm2_patch_can(D, P, b2)) {
        // patches of 128 tokens: the first layer applies the combine weights (one per 128-row block, kept where z would
        // be), the second layer is walked by output patch and writes y itself
        float* blk = (float*)z;
        st = launch_block_gate(D, P, (prob->flags & UOE_FLAG_GATE) != 0, blk, stream);
        if (st != UOE_OK) return st;
        g1.blk_scale = blk;
        st = launch_gemm_bf16(g1, status, stream);
        if (st != UOE_OK) return st;
        return launch_gemm2_patch(D, a, W2, x, y, expert_offsets, P, (prob->flags & UOE_FLAG_RESIDUAL) != 0, status, stream);
    }
    if (mlp_can_fuse(D)) {                    // narrow experts: both GEMMs in one kernel, the hidden tile stays on chip
        st = launch_mlp_fused(D, xg, W1, W2, z, saved_h, expert_offsets, prob->act, fused ? x : nullptr, map, status,
                              stream, b1, b2);
        if (st != UOE_OK) return st;
    } else if (D.bf16) {
        st = launch_gemm_bf16(g1, status, stream);
        if (st != UOE_OK) return st;
        st = launch_gemm_bf16(g2, status, stream);
        if (st != UOE_OK) return st;
    } else {
        st = launch_gemm_f32(g1, stream);
        if (st != UOE_OK) return st;
        st = launch_gemm_f32(g2, stream);
        if (st != UOE_OK) return st;
    }
    return launch_combine(D, x, z, P, (prob->flags & UOE_FLAG_RESIDUAL) != 0, (prob->flags & UOE_FLAG_GATE) != 0, y,
                          stream);
}

uoe_status uoe::mlp_forward_check(const uoe_problem* prob, Dims& D, const void* x, const void* W1, const void* W2,
                                  const void* b1, const void* b2, const void* y, const void* saved_h) {
    uoe_status st = make_dims(prob, D);
    if (st != UOE_OK) return st;
    if (!x || !W1 || !W2 || !y) return UOE_ERR_INVALID_ARG;
    if (D.d_e < 1) return UOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(W1) || !aligned16(W2) || !aligned16(y) || (saved_h && !aligned16(saved_h)))
        return UOE_ERR_INVALID_ARG;
    if ((D.d_e * D.esize) % 16 != 0) return UOE_ERR_UNSUPPORTED;
    if ((b1 && !aligned16(b1)) || (b2 && !aligned16(b2))) return UOE_ERR_INVALID_ARG;
    if (D.bf16 && (b1 || b2) && D.d_e % 64 != 0) return UOE_ERR_UNSUPPORTED;
    return UOE_OK;
}

using namespace uoe;

extern "C" uoe_status uoe_mlp_forward(const uoe_problem* prob, const void* x, const void* W1, const void* W2,
                                      const void* b1, const void* b2, const int32_t* expert_idx,
                                      const int32_t* patch_idx, const float* gate, const int32_t* expert_offsets,
                                      void* y, void* saved_h, void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims D;
    uoe_status st = mlp_forward_check(prob, D, x, W1, W2, b1, b2, y, saved_h);
    if (st != UOE_OK) return st;
    if (!expert_idx || !patch_idx || !gate || !expert_offsets || !ws || !aligned16(ws)) return UOE_ERR_INVALID_ARG;
    const MlpFwdWs W = mlp_fwd_ws(D);
    if (ws_bytes < W.total) return UOE_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    char* base = (char*)ws;
    int* status = (int*)base;
    const PlanPtrs P = plan_ptrs(D, base + W.plan);
    st = launch_plan(D, expert_idx, patch_idx, gate, expert_offsets, P, status, stream);
    if (st != UOE_OK) return st;
    const MlpFwdBufs bufs{base + W.xg, base + W.a, base + W.z};
    return mlp_forward_run(D, prob, x, W1, W2, b1, b2, patch_idx, expert_offsets, P, bufs, y, saved_h, status, stream);
}
