// uoe_block_forward: one Union-of-Experts transformer block (Section III-C, Fig. 2) in one call:
//   u = SMHA(x)   router (Eq. 13-17, 21-23) -> q/k/v projections -> attention -> output projection -> combine (Eq. 27-36)
//   y = UoME(u)   router on u               -> expert MLPs                                         -> combine (Eq. 37-40)
// One workspace serves both halves.  Each router writes its routing plan from the CTA that completes the selection
// (no plan kernel), both routers share one scratch area, and the routed buffers of the two halves share memory.
#include "kernels.cuh"

namespace uoe {
namespace {

struct BlockWs {
    size_t route, plan_att, plan_mlp, r_att, r_mlp, bufs, total;
    SmhaFwdOffsets so;
    size_t m_xg, m_a, m_z;
};

// device arrays of one router's outputs, carved from the workspace when the caller does not want them
size_t routing_bytes(const Dims& D) {
    return align_up((size_t)D.B * D.k * 4, 1024) + 2 * align_up((size_t)D.B * D.k * D.c * 4, 1024) +
           align_up((size_t)D.B * D.n * 4, 1024) + align_up((size_t)D.B * D.n * D.m * 4, 1024) + 1024;
}
RoutingPtrs routing_in(const Dims& D, char* base) {
    RoutingPtrs r;
    r.expert_idx = (int*)base;   base += align_up((size_t)D.B * D.k * 4, 1024);
    r.patch_idx = (int*)base;    base += align_up((size_t)D.B * D.k * D.c * 4, 1024);
    r.gate = (float*)base;       base += align_up((size_t)D.B * D.k * D.c * 4, 1024);
    r.p_samp = (float*)base;     base += align_up((size_t)D.B * D.n * 4, 1024);
    r.p_patch = (float*)base;    base += align_up((size_t)D.B * D.n * D.m * 4, 1024);
    r.expert_offsets = (int*)base;
    return r;
}

BlockWs block_ws(const Dims* Da, const Dims* Dm) {
    BlockWs r = {};
    WsCarver w;
    size_t rb = 0;
    if (Da) rb = route_workspace_bytes(*Da);
    if (Dm && route_workspace_bytes(*Dm) > rb) rb = route_workspace_bytes(*Dm);
    r.route = w.take(rb);                       // starts with the control block (status word, tickets)
    if (Da) { r.plan_att = w.take(plan_bytes(*Da)); r.r_att = w.take(routing_bytes(*Da)); }
    if (Dm) { r.plan_mlp = w.take(plan_bytes(*Dm)); r.r_mlp = w.take(routing_bytes(*Dm)); }
    size_t ba = 0, bm = 0;
    if (Da) ba = smha_fwd_buffer_bytes(*Da, &r.so);
    if (Dm) bm = mlp_fwd_buffer_bytes(*Dm, &r.m_xg, &r.m_a, &r.m_z);
    r.bufs = w.take(ba > bm ? ba : bm);         // the halves run one after the other: their routed buffers share memory
    r.total = w.off;
    return r;
}

RoutingPtrs routing_of(const uoe_routing* r) {
    RoutingPtrs p;
    p.expert_idx = r->expert_idx; p.patch_idx = r->patch_idx; p.gate = r->gate;
    p.p_samp = r->p_samp; p.p_patch = r->p_patch; p.expert_offsets = r->expert_offsets;
    return p;
}
bool routing_complete(const uoe_routing* r) {
    return r->expert_idx && r->patch_idx && r->gate && r->p_samp && r->p_patch && r->expert_offsets;
}

}  // namespace

size_t block_fwd_workspace_bytes(const Dims* Da, const Dims* Dm) { return block_ws(Da, Dm).total; }

}  // namespace uoe

using namespace uoe;

extern "C" size_t uoe_block_workspace_bytes(const uoe_problem* att, const uoe_problem* mlp) {
    Dims Da, Dm;
    if (!att && !mlp) return 0;
    if (att && (make_dims(att, Da) != UOE_OK || Da.H < 1)) return 0;
    if (mlp && (make_dims(mlp, Dm) != UOE_OK || Dm.d_e < 1)) return 0;
    return block_ws(att ? &Da : nullptr, mlp ? &Dm : nullptr).total;
}

extern "C" uoe_status uoe_block_forward(const uoe_problem* att, const uoe_problem* mlp, const void* x,
                                        const void* Wr_att, const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                                        const void* Wr_mlp, const void* W1, const void* W2,
                                        const uoe_routing* r_att, const uoe_routing* r_mlp, void* u, void* y,
                                        void* saved_h, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
    if (!att && !mlp) return UOE_ERR_INVALID_ARG;
    if (!x || !y || !ws || !aligned16(ws)) return UOE_ERR_INVALID_ARG;
    Dims Da, Dm;
    uoe_status st;
    // ---- everything is validated before the first launch ----
    if (att) {
        if (!Wr_att || !aligned16(Wr_att)) return UOE_ERR_INVALID_ARG;
        void* out_att = mlp ? u : y;
        if (!out_att) return UOE_ERR_INVALID_ARG;
        st = smha_forward_check(att, Da, x, Wq, Wk, Wv, Wo, out_att);
        if (st != UOE_OK) return st;
        if (r_att && !routing_complete(r_att)) return UOE_ERR_INVALID_ARG;
    }
    if (mlp) {
        if (!Wr_mlp || !aligned16(Wr_mlp)) return UOE_ERR_INVALID_ARG;
        st = mlp_forward_check(mlp, Dm, att ? u : x, W1, W2, nullptr, nullptr, y, saved_h);
        if (st != UOE_OK) return st;
        if (r_mlp && !routing_complete(r_mlp)) return UOE_ERR_INVALID_ARG;
    }
    if (att && mlp) {      // two halves of one block: same tokens, same width, same storage type
        if (Da.B != Dm.B || Da.L != Dm.L || Da.Lv != Dm.Lv || Da.d != Dm.d || Da.bf16 != Dm.bf16) return UOE_ERR_INVALID_ARG;
        if (u == x || u == y) return UOE_ERR_INVALID_ARG;
    }
    const BlockWs W = block_ws(att ? &Da : nullptr, mlp ? &Dm : nullptr);
    if (ws_bytes < W.total) return UOE_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    char* base = (char*)ws;
    int* status = (int*)base;
    char* scratch = base + W.route;
    char* bufs = base + W.bufs;

    const void* cur = x;
    if (att) {
        const RoutingPtrs R = r_att ? routing_of(r_att) : routing_in(Da, base + W.r_att);
        PlanPtrs P = plan_ptrs(Da, base + W.plan_att);
        const SmhaFwdBufs B{bufs + W.so.xg, bufs + W.so.q, bufs + W.so.k, bufs + W.so.v, bufs + W.so.o, bufs + W.so.z};
        if (route_can_plan(Da)) {
            P.inv_relative = true;
            P.identity_patches = route_whole_samples(Da, att->flags);
            P.gate = R.gate;
            P.tail = (uint4*)B.v; P.tail_row_vecs = (long long)Da.d_g * Da.esize / 16; P.rows_max = Da.Rmax;
            st = route_run(att, cur, Wr_att, R, scratch, stream, &P);
            if (st != UOE_OK) return st;
        } else {
            st = route_run(att, cur, Wr_att, R, scratch, stream, nullptr);
            if (st != UOE_OK) return st;
            st = launch_plan(Da, R.expert_idx, R.patch_idx, R.gate, R.expert_offsets, P, status, stream, true, B.v,
                             (long long)Da.d_g * Da.esize);
            if (st != UOE_OK) return st;
        }
        void* out_att = mlp ? u : y;
        st = smha_forward_run(Da, att, cur, Wq, Wk, Wv, Wo, R.expert_idx, R.patch_idx, R.expert_offsets, P, B, out_att, lse,
                              status, stream);
        if (st != UOE_OK) return st;
        cur = out_att;
    }
    if (mlp) {
        const RoutingPtrs R = r_mlp ? routing_of(r_mlp) : routing_in(Dm, base + W.r_mlp);
        PlanPtrs P = plan_ptrs(Dm, base + W.plan_mlp);
        if (route_can_plan(Dm)) {
            P.inv_relative = true;
            P.identity_patches = route_whole_samples(Dm, mlp->flags);
            P.gate = R.gate;
            st = route_run(mlp, cur, Wr_mlp, R, scratch, stream, &P);
            if (st != UOE_OK) return st;
        } else {
            st = route_run(mlp, cur, Wr_mlp, R, scratch, stream, nullptr);
            if (st != UOE_OK) return st;
            st = launch_plan(Dm, R.expert_idx, R.patch_idx, R.gate, R.expert_offsets, P, status, stream);
            if (st != UOE_OK) return st;
        }
        const MlpFwdBufs B{bufs + W.m_xg, bufs + W.m_a, bufs + W.m_z};
        st = mlp_forward_run(Dm, mlp, cur, W1, W2, nullptr, nullptr, R.patch_idx, R.expert_offsets, P, B, y, saved_h, status,
                             stream);
        if (st != UOE_OK) return st;
    }
    return UOE_OK;
}
