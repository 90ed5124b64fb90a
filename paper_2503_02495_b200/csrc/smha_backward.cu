// uoe_smha_backward: gradients of sum(y * dy) for y = uoe_smha_forward(x, ...) with the selection held constant
// (derivative of Eq. 27-36; with gating also of Eq. 14 and 21 through the gate weights).  The paper gives no
// backward text.  Nothing is saved by the forward: q, k, v, o and the log-sum-exp are recomputed here.
//
// In routed-row space, for the rows r of pair (b, i) with combine weight w_r (0 on pad-token rows):
//   q, k, v = x_g W^{q,k,v}_i ; o, lse = attention(q, k, v)              recomputed (Eq. 28-34)
//   do_raw  = dy_g W^o_i^T                                               grouped GEMM (K-major weights)
//   dgate(patch) = sum_r <do_raw_r, o_r> ;  do = w do_raw ; og = w o ;  delta_{r,h} = sum_{c in head h} do o
//   dq, dk, dv = attention backward(q, k, v, do, lse, delta)             -> one buffer [rows, 3 d_g]
//   dx_g = [dq dk dv] [W^q_i W^k_i W^v_i]^T                              one grouped GEMM, K = 3 d_g
//   d[W^q W^k W^v]_i = x_g^T [dq dk dv] ;  dW^o_i^T = dy_g^T og          ragged-K weight-gradient GEMMs
// then dx = dy + combine(dx_g) + router term, and the router gradients as in the UoME backward.
#include "kernels.cuh"

namespace uoe {

uoe_status launch_attention(const Dims& D, const void* q, const void* k, const void* v, void* o, float* lse,
                            const int* pair_row, const int* patch_idx, bool causal, int* status, cudaStream_t s,
                            const void* Wo = nullptr, const int* expert_idx = nullptr, void* z = nullptr);
bool attention_can_fuse_out(const Dims& D);
uoe_status launch_attention_backward(const Dims& D, const void* q, const void* k, const void* v, const void* dout,
                                     const float* lse, const float* delta, void* dq, void* dk, void* dv, int ld_out,
                                     const int* pair_row, const int* patch_idx, bool causal, int* status,
                                     cudaStream_t s);

uoe_status launch_rope(const Dims& D, void* a, void* b, int ld, const int* pair_row, const int* patch_idx, bool inverse,
                       cudaStream_t s);

namespace {

constexpr int kThreads = 256;

// Rows that no kernel writes but that can sit inside a 128-row MMA tile or inside an expert region's contraction
// range are made zero (a NaN there would poison a whole accumulator): segment i < n is the padding of expert i's
// region, [expert_end[i], offsets[i+1]); segment n is [offsets[n], rows_max).  Up to three [rows_max, width]
// buffers per launch.  grid (n + 1, splits).
__global__ void __launch_bounds__(kThreads)
zero_pad_rows_kernel(uint4* __restrict__ a, uint4* __restrict__ b, uint4* __restrict__ c, const int* __restrict__ expert_end,
                     const int* __restrict__ offsets, int n, long long rows_max, int row_vecs) {
    pdl_trigger();
    pdl_wait();
    const int seg = blockIdx.x;
    const long long r0 = seg < n ? expert_end[seg] : offsets[n];
    const long long r1 = seg < n ? offsets[seg + 1] : rows_max;
    const long long total = (r1 - r0) * row_vecs;
    const uint4 z = make_uint4(0, 0, 0, 0);
    for (long long q = (long long)blockIdx.y * kThreads + threadIdx.x; q < total; q += (long long)gridDim.y * kThreads) {
        a[r0 * row_vecs + q] = z;
        if (b) b[r0 * row_vecs + q] = z;
        if (c) c[r0 * row_vecs + q] = z;
    }
}

// One thread per (routed row, head):  dot = <do_raw, o> over the head's 64 columns;
//   delta[row, head] = w dot,  dg_part[row, head] = valid dot,  do = w do_raw (in place),  og = w o;
// rows with w = 0 (pad tokens, unused slots, region padding, where o may never have been written) get exact zeros.
__global__ void __launch_bounds__(kThreads)
attn_bwd_prep_kernel(__nv_bfloat16* __restrict__ dout, const __nv_bfloat16* __restrict__ o, __nv_bfloat16* __restrict__ og,
                     const float* __restrict__ row_gate, const float* __restrict__ row_valid, float* __restrict__ delta,
                     float* __restrict__ dg_part, const int* __restrict__ offsets, int n, int heads, int d_g) {
    pdl_trigger();
    pdl_wait();
    const long long idx = (long long)blockIdx.x * kThreads + threadIdx.x;
    const long long row = idx / heads;
    const int head = (int)(idx % heads);
    if (row >= offsets[n]) return;
    const float w = row_gate[row], valid = row_valid[row];
    uint4* dp = (uint4*)(dout + row * d_g + head * 64);
    const uint4* op = (const uint4*)(o + row * d_g + head * 64);
    uint4* gp = (uint4*)(og + row * d_g + head * 64);
    uint4 dv[8], ov[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) { dv[q] = dp[q]; ov[q] = op[q]; }
    float dot = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        float a[8], b[8];
        unpack16<__nv_bfloat16>(dv[q], a);
        unpack16<__nv_bfloat16>(ov[q], b);
#pragma unroll
        for (int v = 0; v < 8; ++v) {
            dot = fmaf(a[v], b[v], dot);
            a[v] = w != 0.f ? a[v] * w : 0.f;
            b[v] = w != 0.f ? b[v] * w : 0.f;
        }
        dp[q] = pack16<__nv_bfloat16>(a);
        gp[q] = pack16<__nv_bfloat16>(b);
    }
    delta[row * heads + head] = w != 0.f ? w * dot : 0.f;
    dg_part[row * heads + head] = valid != 0.f ? dot : 0.f;
}

// Wcat[e, r, :] = [Wq[e, r, :], Wk[e, r, :], Wv[e, r, :]]   ([n, d, d_g] x 3 -> [n, d, 3 d_g]), 16-byte pieces
__global__ void __launch_bounds__(kThreads)
concat_qkv_kernel(const uint4* __restrict__ Wq, const uint4* __restrict__ Wk, const uint4* __restrict__ Wv,
                  uint4* __restrict__ Wcat, long long rows, int vecs /* d_g / 8 */) {
    pdl_trigger();
    pdl_wait();
    const long long total = rows * 3 * vecs;
    for (long long q = (long long)blockIdx.x * kThreads + threadIdx.x; q < total; q += (long long)gridDim.x * kThreads) {
        const long long r = q / (3 * vecs);
        const int cidx = (int)(q % (3 * vecs)), which = cidx / vecs, v = cidx % vecs;
        const uint4* src = which == 0 ? Wq : (which == 1 ? Wk : Wv);
        Wcat[q] = src[r * vecs + v];
    }
}

// dWcat [n*d, 3 d_g] -> dWq, dWk, dWv [n*d, d_g];  dWoT [n, d, d_g] -> dWo [n, d_g, d]   (float32)
__global__ void __launch_bounds__(kThreads)
finalize_wgrads_kernel(const float* __restrict__ dWcat, const float* __restrict__ dWoT, float* __restrict__ dWq,
                       float* __restrict__ dWk, float* __restrict__ dWv, float* __restrict__ dWo, int n, int d, int d_g) {
    pdl_trigger();
    pdl_wait();
    const long long per = (long long)n * d * d_g;
    const long long total = 4 * per;
    for (long long q = (long long)blockIdx.x * kThreads + threadIdx.x; q < total; q += (long long)gridDim.x * kThreads) {
        const int which = (int)(q / per);
        const long long e = q % per;
        if (which < 3) {
            const long long r = e / d_g;
            const int cc = (int)(e % d_g);
            const float v = dWcat[r * 3 * d_g + which * d_g + cc];
            (which == 0 ? dWq : (which == 1 ? dWk : dWv))[e] = v;
        } else {                 // e indexes dWo [n, d_g, d]
            const int dd = (int)(e % d);
            const long long t = e / d;
            const int cc = (int)(t % d_g);
            const long long ex = t / d_g;
            dWo[e] = dWoT[(ex * d + dd) * d_g + cc];
        }
    }
}

struct SmhaBwdWs {
    size_t plan, xg, dyg, q, k, v, o, dout, og, dqkv, dxg, lse, delta, dgp, wcat, dwcat, dwot, router, wgpart, total;
};

SmhaBwdWs smha_bwd_ws(const Dims& D) {
    WsCarver w;
    w.take(kStatusBytes);
    SmhaBwdWs r;
    const int heads = D.d_g > 0 ? D.d_g / 64 : 1;
    const size_t rg = (size_t)D.Rmax * D.d_g * D.esize;
    r.plan = w.take(plan_bytes(D, true));
    const bool fused = can_fuse_gather(D) && wgrad_can_gather(D.l_p);      // x and dy gathered inside the consumers' TMA loads
    r.xg = fused ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);
    r.dyg = fused ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);
    r.q = w.take(rg); r.k = w.take(rg); r.v = w.take(rg); r.o = w.take(rg); r.dout = w.take(rg); r.og = w.take(rg);
    r.dqkv = w.take(3 * rg);
    r.dxg = w.take((size_t)D.Rmax * D.d * D.esize);
    r.lse = w.take((size_t)D.Rmax * heads * 4);
    r.delta = w.take((size_t)D.Rmax * heads * 4);
    r.dgp = w.take((size_t)D.Rmax * heads * 4);
    r.wcat = w.take((size_t)D.n * D.d * 3 * D.d_g * D.esize);
    r.dwcat = w.take((size_t)D.n * D.d * 3 * D.d_g * 4);
    r.dwot = w.take((size_t)D.n * D.d * D.d_g * 4);
    r.router = w.take(router_backward_scratch_bytes(D));
    {   // split-K partials, sized for the larger of the two weight gradients
        const size_t s1 = wgrad_scratch_bytes(D.n, D.d, 3 * D.d_g, D.Rmax), s2 = wgrad_scratch_bytes(D.n, D.d, D.d_g, D.Rmax);
        r.wgpart = w.take((s1 > s2 ? s1 : s2) + 1024);
    }
    r.total = w.off;
    return r;
}

}  // namespace

size_t smha_bwd_workspace_bytes(const Dims& D) { return smha_bwd_ws(D).total; }

}  // namespace uoe

using namespace uoe;

extern "C" uoe_status uoe_smha_backward(const uoe_problem* prob, const void* x, const void* Wq, const void* Wk,
                                        const void* Wv, const void* Wo, const void* W_r, const int32_t* expert_idx,
                                        const int32_t* patch_idx, const float* gate, const int32_t* expert_offsets,
                                        const float* p_samp, const float* p_patch, const void* dy, void* dx,
                                        float* dWq, float* dWk, float* dWv, float* dWo, float* dW_r, void* ws,
                                        size_t ws_bytes, void* cuda_stream) {
    Dims D;
    uoe_status st = make_dims(prob, D);
    if (st != UOE_OK) return st;
    if (!x || !Wq || !Wk || !Wv || !Wo || !W_r || !expert_idx || !patch_idx || !gate || !expert_offsets || !p_samp ||
        !p_patch || !dy || !dx || !dWq || !dWk || !dWv || !dWo || !dW_r || !ws)
        return UOE_ERR_INVALID_ARG;
    if (D.H < 1 || D.d_g < 1) return UOE_ERR_INVALID_ARG;
    const void* al[] = {x, Wq, Wk, Wv, Wo, dy, dx, dWq, dWk, dWv, dWo, ws};
    for (const void* p : al)
        if (!aligned16(p)) return UOE_ERR_INVALID_ARG;
    // tensor-core path only: bf16, 64-wide heads, model width that tiles the 128-row weight-gradient MMA
    if (!D.bf16 || D.d_h != 64 || D.d % 128 != 0) return UOE_ERR_UNSUPPORTED;
    if ((long long)D.B * D.k > 65535) return UOE_ERR_UNSUPPORTED;  // the attention grids carry the pairs on their z axis
    const SmhaBwdWs W = smha_bwd_ws(D);
    if (ws_bytes < W.total) return UOE_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const bool use_gate = (prob->flags & UOE_FLAG_GATE) != 0;
    const bool residual = (prob->flags & UOE_FLAG_RESIDUAL) != 0;
    const bool causal = (prob->flags & UOE_FLAG_CAUSAL) != 0;
    const int heads = D.d_g / 64;
    char* base = (char*)ws;
    int* status = (int*)base;
    const PlanPtrs P = plan_ptrs(D, base + W.plan, true);
    // rows of the per-row weights that belong to no pair (region padding) must read as zero
    UOE_CUDA_OK(cudaMemsetAsync(P.row_gate, 0, 2 * align_up((size_t)D.Rmax * 4, 1024), stream));
    void *xg = base + W.xg, *dyg = base + W.dyg, *q = base + W.q, *k = base + W.k, *v = base + W.v, *o = base + W.o;
    void *dout = base + W.dout, *og = base + W.og, *dqkv = base + W.dqkv, *dxg = base + W.dxg;
    float *lse = (float*)(base + W.lse), *delta = (float*)(base + W.delta), *dgp = (float*)(base + W.dgp);
    void* wcat = base + W.wcat;
    float *dwcat = (float*)(base + W.dwcat), *dwot = (float*)(base + W.dwot);
    const RouterBwdScratch rs = router_backward_scratch(D, base + W.router);
    const long long rowb = (long long)D.d_g * D.esize;

    st = launch_plan(D, expert_idx, patch_idx, gate, expert_offsets, P, status, stream, use_gate, v, rowb);
    if (st != UOE_OK) return st;
    // Eq. 18 for x and dy: either inside the TMA loads of the kernels that consume them, or as routed copies
    const bool fused = can_fuse_gather(D) && wgrad_can_gather(D.l_p);
    WgradGather gp;
    if (fused) {
        gp.gather_p = true; gp.src_patch = P.src_patch; gp.l_p = D.l_p; gp.Bm = D.B * D.m;
    } else {
        st = launch_gather(D, x, patch_idx, expert_offsets, P, xg, stream);
        if (st != UOE_OK) return st;
        st = launch_gather(D, dy, patch_idx, expert_offsets, P, dyg, stream);
        if (st != UOE_OK) return st;
    }
    {
        ProfScope ps("zero_pad_rows", stream);
        launch_k(zero_pad_rows_kernel, dim3(D.n + 1, 16), dim3(kThreads), 0, stream, (uint4*)q, (uint4*)k, (uint4*)dout,
                 (const int*)P.expert_end, expert_offsets, D.n, D.Rmax, (int)(rowb / 16));
        launch_k(zero_pad_rows_kernel, dim3(D.n + 1, 16), dim3(kThreads), 0, stream, (uint4*)dqkv, (uint4*)nullptr,
                 (uint4*)nullptr, (const int*)P.expert_end, expert_offsets, D.n, D.Rmax, (int)(3 * rowb / 16));
    }
    UOE_LAUNCHED();
    UOE_LAUNCHED();

    // ---- forward recomputation (Eq. 28-34) ----
    GemmArgs gq{xg, Wq, nullptr, q, nullptr, expert_offsets, D.n, D.d, D.d_g, UOE_ACT_IDENTITY, false, D.Rmax};
    if (fused) { gq.gather_x = x; gq.src_patch = P.src_patch; gq.l_p = D.l_p; gq.Bm = D.B * D.m; }
    gq.label = "qkv_proj";
    gq.nmat = 3; gq.W1 = Wk; gq.W2 = Wv; gq.C1 = k; gq.C2 = v;
    st = launch_gemm_bf16(gq, status, stream);
    if (st != UOE_OK) return st;
    st = launch_rope(D, q, k, D.d_g, P.pair_row, patch_idx, false, stream);      // Eq. 32 (nothing if d_rope = 0)
    if (st != UOE_OK) return st;
    st = launch_attention(D, q, k, v, o, lse, P.pair_row, patch_idx, causal, status, stream);
    if (st != UOE_OK) return st;

    // ---- out-projection backward ----
    GemmArgs gd{dyg, Wo, nullptr, dout, nullptr, expert_offsets, D.n, D.d, D.d_g, UOE_ACT_IDENTITY, true, D.Rmax};
    if (fused) { gd.gather_x = dy; gd.src_patch = P.src_patch; gd.l_p = D.l_p; gd.Bm = D.B * D.m; }
    gd.label = "bwd_do";
    st = launch_gemm_bf16(gd, status, stream);
    if (st != UOE_OK) return st;
    {
        ProfScope ps("attn_bwd_prep", stream);
        const long long items = D.Rmax * heads;
        launch_k(attn_bwd_prep_kernel, dim3((unsigned)((items + kThreads - 1) / kThreads)), dim3(kThreads), 0, stream,
                 (__nv_bfloat16*)dout, (const __nv_bfloat16*)o, (__nv_bfloat16*)og, (const float*)P.row_gate,
                 (const float*)P.row_valid, delta, dgp, expert_offsets, D.n, heads, D.d_g);
    }
    UOE_LAUNCHED();
    st = launch_wgrad_bf16(fused ? dy : dyg, og, dwot, expert_offsets, D.n, D.d, D.d_g, D.Rmax, "wgrad_Wo", status, stream,
                           wgrad_scratch_bytes(D.n, D.d, D.d_g, D.Rmax) ? (float*)(base + W.wgpart) : nullptr, gp);
    if (st != UOE_OK) return st;

    // ---- attention backward ----
    __nv_bfloat16* dq = (__nv_bfloat16*)dqkv;
    st = launch_attention_backward(D, q, k, v, dout, lse, delta, dq, dq + D.d_g, dq + 2 * D.d_g, 3 * D.d_g, P.pair_row,
                                   patch_idx, causal, status, stream);
    if (st != UOE_OK) return st;

    // gradients w.r.t. the rotated q, k -> w.r.t. the projections: rotate back
    st = launch_rope(D, dq, dq + D.d_g, 3 * D.d_g, P.pair_row, patch_idx, true, stream);
    if (st != UOE_OK) return st;

    // ---- projection backward: dx_g and the q/k/v weight gradients from the concatenated [dq dk dv] ----
    {
        ProfScope ps("concat_qkv", stream);
        launch_k(concat_qkv_kernel, dim3(128), dim3(kThreads), 0, stream, (const uint4*)Wq, (const uint4*)Wk, (const uint4*)Wv,
                 (uint4*)wcat, (long long)D.n * D.d, D.d_g / 8);
    }
    UOE_LAUNCHED();
    GemmArgs gx{dqkv, wcat, nullptr, dxg, nullptr, expert_offsets, D.n, 3 * D.d_g, D.d, UOE_ACT_IDENTITY, true, D.Rmax};
    gx.label = "bwd_dx_att";
    st = launch_gemm_bf16(gx, status, stream);
    if (st != UOE_OK) return st;
    st = launch_wgrad_bf16(fused ? x : xg, dqkv, dwcat, expert_offsets, D.n, D.d, 3 * D.d_g, D.Rmax, "wgrad_Wqkv", status, stream,
                           wgrad_scratch_bytes(D.n, D.d, 3 * D.d_g, D.Rmax) ? (float*)(base + W.wgpart) : nullptr, gp);
    if (st != UOE_OK) return st;
    {
        ProfScope ps("finalize_wgrads", stream);
        launch_k(finalize_wgrads_kernel, dim3(256), dim3(kThreads), 0, stream, (const float*)dwcat, (const float*)dwot, dWq, dWk,
                 dWv, dWo, D.n, D.d, D.d_g);
    }
    UOE_LAUNCHED();

    // ---- router ----
    if (use_gate) {
        st = launch_router_backward(D, x, W_r, expert_idx, patch_idx, p_samp, p_patch, P, dgp, heads, rs, dW_r, stream);
        if (st != UOE_OK) return st;
    } else {
        UOE_CUDA_OK(cudaMemsetAsync(dW_r, 0, (size_t)D.d * D.n * sizeof(float), stream));
    }
    return launch_combine(D, dy, dxg, P, residual, false, dx, stream, use_gate ? rs.rvec : nullptr);
}
