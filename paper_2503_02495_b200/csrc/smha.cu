// uoe_smha_forward: SMHA forward (Eq. 27-30, 32-36) as plan -> grouped q/k/v projections in one launch,
// gathering x inside the TMA loads (Eq. 27-30) -> optional RoPE (Eq. 32) -> attention over each pair's
// gathered tokens with the expert's output projection in the same kernel (Eq. 33-35; a separate grouped GEMM
// when an expert has several heads or d > 512) -> weighted combine (Eq. 36).
#include "kernels.cuh"

namespace uoe {

uoe_status launch_attention(const Dims& D, const void* q, const void* k, const void* v, void* o, float* lse,
                            const int* pair_row, const int* patch_idx, bool causal, int* status, cudaStream_t s,
                            const void* Wo = nullptr, const int* expert_idx = nullptr, void* z = nullptr);
bool attention_can_fuse_out(const Dims& D);

uoe_status launch_rope(const Dims& D, void* a, void* b, int ld, const int* pair_row, const int* patch_idx, bool inverse,
                       cudaStream_t s);

struct SmhaWs { size_t plan, xg, q, k, v, o, z, total; };

static SmhaWs smha_ws(const Dims& D) {
    WsCarver w;
    w.take(kStatusBytes);
    SmhaWs r;
    r.plan = w.take(plan_bytes(D));
    r.xg = can_fuse_gather(D) ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);     // the projection gathers x itself
    r.q = w.take((size_t)D.Rmax * D.d_g * D.esize);
    r.k = w.take((size_t)D.Rmax * D.d_g * D.esize);
    r.v = w.take((size_t)D.Rmax * D.d_g * D.esize);
    r.o = w.take((size_t)D.Rmax * D.d_g * D.esize);
    r.z = w.take((size_t)D.Rmax * D.d * D.esize);
    r.total = w.off;
    return r;
}

size_t smha_fwd_workspace_bytes(const Dims& D) { return smha_ws(D).total; }

size_t smha_fwd_buffer_bytes(const Dims& D, SmhaFwdOffsets* o) {
    WsCarver w;
    o->xg = can_fuse_gather(D) ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);
    o->q = w.take((size_t)D.Rmax * D.d_g * D.esize);
    o->k = w.take((size_t)D.Rmax * D.d_g * D.esize);
    o->v = w.take((size_t)D.Rmax * D.d_g * D.esize);
    o->o = w.take((size_t)D.Rmax * D.d_g * D.esize);
    o->z = w.take((size_t)D.Rmax * D.d * D.esize);
    return w.off;
}

}  // namespace uoe

// Everything of the SMHA forward behind the routing plan.  Rows of v past the last expert region must already be
// finite (the plan step zero-fills them): they may sit inside the last key tile of a pair.
uoe_status uoe::smha_forward_run(const Dims& D, const uoe_problem* prob, const void* x, const void* Wq, const void* Wk,
                                 const void* Wv, const void* Wo, const int* expert_idx, const int* patch_idx,
                                 const int* expert_offsets, const PlanPtrs& P, const SmhaFwdBufs& bufs, void* y,
                                 float* lse, int* status, cudaStream_t stream) {
    uoe_status st;
    void *xg = bufs.xg, *q = bufs.q, *k = bufs.k, *v = bufs.v, *o = bufs.o, *z = bufs.z;
    const bool fused = can_fuse_gather(D);
    if (!fused) {
        st = launch_gather(D, x, patch_idx, expert_offsets, P, xg, stream);
        if (st != UOE_OK) return st;
    }
    GemmArgs gq{xg, Wq, nullptr, q, nullptr, expert_offsets, D.n, D.d, D.d_g, UOE_ACT_IDENTITY, false, D.Rmax};
    if (fused) { gq.gather_x = x; gq.map = src_map_of(D, P, patch_idx); gq.l_p = D.l_p; gq.Bm = D.B * D.m; }
    gq.label = "qkv_proj";
    gq.nmat = 3; gq.W1 = Wk; gq.W2 = Wv; gq.C1 = k; gq.C2 = v;
    st = launch_gemm_bf16(gq, status, stream);
    if (st != UOE_OK) return st;
    st = launch_rope(D, q, k, D.d_g, P.pair_row, patch_idx, false, stream);      // Eq. 32 (nothing if d_rope = 0)
    if (st != UOE_OK) return st;
    const bool causal = (prob->flags & UOE_FLAG_CAUSAL) != 0;
    if (attention_can_fuse_out(D)) {          // Eq. 33-35 in one kernel: attention and the expert's output projection
        st = launch_attention(D, q, k, v, o, lse, P.pair_row, patch_idx, causal, status, stream, Wo, expert_idx, z);
        if (st != UOE_OK) return st;
    } else {
        st = launch_attention(D, q, k, v, o, lse, P.pair_row, patch_idx, causal, status, stream);
        if (st != UOE_OK) return st;
        GemmArgs go{o, Wo, nullptr, z, nullptr, expert_offsets, D.n, D.d_g, D.d, UOE_ACT_IDENTITY, false, D.Rmax};
        go.label = "out_proj";
        st = launch_gemm_bf16(go, status, stream);
        if (st != UOE_OK) return st;
    }
    return launch_combine(D, x, z, P, (prob->flags & UOE_FLAG_RESIDUAL) != 0, (prob->flags & UOE_FLAG_GATE) != 0, y,
                          stream);
}

uoe_status uoe::smha_forward_check(const uoe_problem* prob, Dims& D, const void* x, const void* Wq, const void* Wk,
                                   const void* Wv, const void* Wo, const void* y) {
    uoe_status st = make_dims(prob, D);
    if (st != UOE_OK) return st;
    if (!x || !Wq || !Wk || !Wv || !Wo || !y) return UOE_ERR_INVALID_ARG;
    if (D.H < 1 || D.d_g < 1) return UOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(Wq) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(Wo) || !aligned16(y))
        return UOE_ERR_INVALID_ARG;
    if (!D.bf16 || D.d_h != 64) return UOE_ERR_UNSUPPORTED;     // tensor-core path: bf16, 64-wide heads
    return UOE_OK;
}

using namespace uoe;

extern "C" uoe_status uoe_smha_forward(const uoe_problem* prob, const void* x, const void* Wq, const void* Wk,
                                       const void* Wv, const void* Wo, const int32_t* expert_idx,
                                       const int32_t* patch_idx, const float* gate, const int32_t* expert_offsets,
                                       void* y, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims D;
    uoe_status st = smha_forward_check(prob, D, x, Wq, Wk, Wv, Wo, y);
    if (st != UOE_OK) return st;
    if (!expert_idx || !patch_idx || !gate || !expert_offsets || !ws || !aligned16(ws)) return UOE_ERR_INVALID_ARG;
    const SmhaWs W = smha_ws(D);
    if (ws_bytes < W.total) return UOE_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    char* base = (char*)ws;
    int* status = (int*)base;
    const PlanPtrs P = plan_ptrs(D, base + W.plan);
    const SmhaFwdBufs bufs{base + W.xg, base + W.q, base + W.k, base + W.v, base + W.o, base + W.z};
    // rows of v past the last expert region are never written by the projection but may sit inside the
    // last key tile of a pair: the plan kernel makes them finite (zero)
    st = launch_plan(D, expert_idx, patch_idx, gate, expert_offsets, P, status, stream, true, bufs.v,
                     (long long)D.d_g * D.esize);
    if (st != UOE_OK) return st;
    return smha_forward_run(D, prob, x, Wq, Wk, Wv, Wo, expert_idx, patch_idx, expert_offsets, P, bufs, y, lse, status, stream);
}
