// uoe_mlp_backward: gradients of sum(y * dy) for y = uoe_mlp_forward(x, ...) with the selection held
// constant (derivative of Eq. 38-40; with gating also of Eq. 14 and 21 through the gate weights).
//
// In routed-row space, for a row r of expert i with combine weight w_r, saved pre-activation h_r:
//   u_r  = dy_r A^O_i^T                      grouped GEMM (K-major weights), epilogue produces
//   dh_r = w_r u_r * phi'(h_r)               -> buffer dh
//   ag_r = w_r phi(h_r)                      -> buffer ag
//   dgate(slab) = sum_r <u_r, phi(h_r)>      -> per-row partials, reduced per (sample, expert, patch)
//   dA^O_i = ag^T dy_g,  dA^I_i = x_g^T dh   ragged-K weight-gradient GEMMs
//   dx_g = dh A^I_i^T                        grouped GEMM, then combined back with unit weights
// Router: dgate -> dP_samp, dP_patch -> softmax Jacobians -> per-(sample, patch) logit gradient G, which
// feeds dW_r (through the pooled token sums) and one more term of dx.
#include "kernels.cuh"

namespace uoe {
namespace {

constexpr int kThreads = 256;

// dgate[b,s,u] = sum over the slab's rows and column tiles of the per-row partials; one warp per slab,
// fixed summation order.  grid ceil(B*k*c / 4), 128 threads.
__global__ void __launch_bounds__(128)
dgate_kernel(const float* __restrict__ dg_part, int nt, const int* __restrict__ pair_row,
             const int* __restrict__ patch_idx, int n_slabs, int c, int m, int l_p, float* __restrict__ dgate) {
    pdl_trigger();
    pdl_wait();
    const int slab = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (slab >= n_slabs) return;
    const int j = patch_idx[slab];
    float a = 0.f;
    if (j >= 0 && j < m) {
        const float* src = dg_part + ((size_t)pair_row[slab / c] + (size_t)(slab % c) * l_p) * nt;
        for (int q = lane; q < l_p * nt; q += 32) a += src[q];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) dgate[slab] = a;
}

// grid B, 128 threads, dynamic smem 2*n*m floats.  G[b,j,i] = dlogit_patch[b,i,j]/cnt_j + dlogit_samp[b,i]/L_valid.
__global__ void __launch_bounds__(128)
router_bwd_kernel(const float* __restrict__ dgate,
                  const int* __restrict__ expert_idx, const int* __restrict__ patch_idx,
                  const float* __restrict__ p_samp, const float* __restrict__ p_patch, int n, int k, int m, int c,
                  int l_p, int Lv, float* __restrict__ G) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ float sm[];
    float* pp = sm;                 // [n][m] patch gate
    float* dpp = sm + n * m;        // [n][m] its gradient
    __shared__ float ps[32], dps[32], dls[32];
    const int b = blockIdx.x, tid = threadIdx.x;
    for (int idx = tid; idx < n * m; idx += 128) { pp[idx] = p_patch[(size_t)b * n * m + idx]; dpp[idx] = 0.f; }
    if (tid < n) { ps[tid] = p_samp[(size_t)b * n + tid]; dps[tid] = 0.f; }
    __syncthreads();
    // gate = P_samp * P_patch: each chosen expert's slots are handled by one thread, in slot order
    if (tid < k) {
        const int i = expert_idx[(size_t)b * k + tid];
        float acc = 0.f;
        for (int u = 0; u < c; ++u) {
            const int j = patch_idx[((size_t)b * k + tid) * c + u];
            if (j < 0 || j >= m) continue;
            const float dg = dgate[((size_t)b * k + tid) * c + u];
            acc += dg * pp[i * m + j];
            dpp[i * m + j] = dg * ps[i];          // one (expert, patch) pair per slot: no other writer
        }
        dps[i] = acc;
    }
    __syncthreads();
    if (tid == 0) {                                       // softmax Jacobian of the sample gate (Eq. 21)
        float dot = 0.f;
        for (int i = 0; i < n; ++i) dot += ps[i] * dps[i];
        for (int i = 0; i < n; ++i) dls[i] = ps[i] * (dps[i] - dot);
    }
    __syncthreads();
    for (int j = tid; j < m; j += 128) {                  // softmax Jacobian of each patch gate (Eq. 14)
        const int cnt = max(0, min(l_p, Lv - j * l_p));
        float dot = 0.f;
        for (int i = 0; i < n; ++i) dot += pp[i * m + j] * dpp[i * m + j];
        for (int i = 0; i < n; ++i) {
            const float dlp = pp[i * m + j] * (dpp[i * m + j] - dot);
            G[((size_t)b * m + j) * n + i] = cnt > 0 ? dlp / (float)cnt + dls[i] / (float)Lv : 0.f;
        }
    }
}

// grid B*m * column chunks (chunk fastest, so concurrent CTAs read x linearly): sum of the real rows of each
// patch, float32 [B*m, d]
template <typename T>
__global__ void __launch_bounds__(kThreads)
pool_kernel(const T* __restrict__ x, float* __restrict__ pool, int L, int Lv, int d, int m, int l_p, int CT, int nchunks) {
    pdl_trigger();
    pdl_wait();
    constexpr int V = Vec16<T>::N;
    __shared__ float red[kThreads * V];
    const int bj = blockIdx.x / nchunks, chunk = blockIdx.x % nchunks, b = bj / m, j = bj % m;
    const int ct = threadIdx.x % CT, rt = threadIdx.x / CT, RT = kThreads / CT;
    const int col = (chunk * CT + ct) * V;
    const int rows = max(0, min(l_p, Lv - j * l_p));
    float cs[V];
#pragma unroll
    for (int v = 0; v < V; ++v) cs[v] = 0.f;
    if (col < d) {
        const T* base = x + ((size_t)b * L + (size_t)j * l_p) * d + col;
        int r = rt;
        for (; r + 7 * RT < rows; r += 8 * RT) {
            uint4 q[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) q[u] = ld_stream16(base + (size_t)(r + u * RT) * d);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float f[V];
                unpack16<T>(q[u], f);
#pragma unroll
                for (int v = 0; v < V; ++v) cs[v] += f[v];
            }
        }
        for (; r < rows; r += RT) {
            float f[V];
            unpack16<T>(ld_stream16(base + (size_t)r * d), f);
#pragma unroll
            for (int v = 0; v < V; ++v) cs[v] += f[v];
        }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) red[(rt * CT + ct) * V + v] = cs[v];
    __syncthreads();
    if (rt == 0 && col < d) {
        for (int q = 1; q < RT; ++q)
#pragma unroll
            for (int v = 0; v < V; ++v) cs[v] += red[(q * CT + ct) * V + v];
#pragma unroll
        for (int v = 0; v < V; ++v) pool[(size_t)bj * d + col + v] = cs[v];
    }
}

// rvec[bj, dd] = sum_i W_r[dd, i] * G[bj, i]: what the router path adds to dx for every real token of patch bj
template <typename T>
__global__ void __launch_bounds__(kThreads)
rvec_kernel(const T* __restrict__ W_r, const float* __restrict__ G, float* __restrict__ rvec, int d, int n) {
    pdl_trigger();
    pdl_wait();
    __shared__ float sG[32];
    const int bj = blockIdx.x;
    if (threadIdx.x < n) sG[threadIdx.x] = G[(size_t)bj * n + threadIdx.x];
    __syncthreads();
    constexpr int V = Vec16<T>::N;
    const bool vec_rows = (n % V) == 0;               // a row of W_r is a whole number of 16-byte pieces
    for (int dd = threadIdx.x; dd < d; dd += kThreads) {
        float a = 0.f;
        if (vec_rows) {
            const uint4* wr = (const uint4*)(W_r + (size_t)dd * n);
            for (int q = 0; q < n / V; ++q) {
                float f[V];
                unpack16<T>(wr[q], f);
#pragma unroll
                for (int v = 0; v < V; ++v) a = fmaf(f[v], sG[q * V + v], a);
            }
        } else {
            for (int i = 0; i < n; ++i) a = fmaf(to_f32(W_r[(size_t)dd * n + i]), sG[i], a);
        }
        rvec[(size_t)bj * d + dd] = a;
    }
}

// dW_r[dd, i] = sum over (b, j) of pool[bj, dd] * G[bj, i] in two fixed-order stages: grid (d/256, S) partial sums
// over S chunks of bj, then a sum over the chunks.
constexpr int kDwrSplit = 64;            // most splits (sizes the partial buffer)
// splits actually used: enough (column block, split) CTAs for two per SM, no more (every split writes d*n partials)
inline int dwr_split(int d) {
    const int col_blocks = (d + kThreads - 1) / kThreads;
    int s = (2 * 148 + col_blocks - 1) / col_blocks;
    return s < 4 ? 4 : (s > kDwrSplit ? kDwrSplit : s);
}
__global__ void __launch_bounds__(kThreads)
dwr_partial_kernel(const float* __restrict__ pool, const float* __restrict__ G, float* __restrict__ part, int BM, int d,
                   int n) {
    pdl_trigger();
    pdl_wait();
    __shared__ float sG[64 * 32];
    const int dd = blockIdx.x * kThreads + threadIdx.x;
    const int per = (BM + (int)gridDim.y - 1) / (int)gridDim.y;
    const int lo = blockIdx.y * per, hi = min(BM, lo + per);
    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.f;
    for (int b0 = lo; b0 < hi; b0 += 64) {
        const int nb = min(64, hi - b0);
        __syncthreads();
        for (int q = threadIdx.x; q < nb * n; q += kThreads) sG[q] = G[(size_t)b0 * n + q];
        __syncthreads();
        if (dd < d) {
            for (int q = 0; q < nb; ++q) {
                const float p = pool[(size_t)(b0 + q) * d + dd];
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i < n) acc[i] = fmaf(p, sG[q * n + i], acc[i]);
            }
        }
    }
    if (dd < d) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < n) part[((size_t)blockIdx.y * d + dd) * n + i] = acc[i];
    }
}
__global__ void __launch_bounds__(kThreads)
dwr_sum_kernel(const float* __restrict__ part, float* __restrict__ dW_r, int total, int nsplit) {
    pdl_trigger();
    pdl_wait();
    const int idx = blockIdx.x * kThreads + threadIdx.x;
    if (idx >= total) return;
    float a = 0.f;
    for (int s = 0; s < nsplit; ++s) a += part[(size_t)s * total + idx];
    dW_r[idx] = a;
}

// Gradient of the load-balancing loss (Eq. 42-44) with respect to the router logits.  grid B, 128 threads, dynamic
// shared memory n*m floats.  f_i (Eq. 43) is piecewise constant, so only P_i (Eq. 44) carries a gradient:
//   dL_b/dg_{i,j} = alpha f_i / l on the real patches;  G[b,j,i] = softmax Jacobian (Eq. 14) of that, / cnt_j.
__global__ void __launch_bounds__(128)
balance_bwd_kernel(const float* __restrict__ p_patch, const float* __restrict__ dloss, int Lv, int n, int k, int m,
                   int l_p, float alpha, float* __restrict__ G) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ float pp[];          // [n][m]
    __shared__ int cnts[32];
    const int b = blockIdx.x, tid = threadIdx.x;
    const int n_elig = (Lv + l_p - 1) / l_p;
    for (int idx = tid; idx < n * m; idx += 128) pp[idx] = p_patch[(size_t)b * n * m + idx];
    if (tid < 32) cnts[tid] = 0;
    __syncthreads();
    for (int j = tid; j < n_elig; j += 128) {      // Eq. 15 / 43: patch j counts for its k best experts
        for (int i = 0; i < n; ++i) {
            const float v = pp[i * m + j];
            int rank = 0;
            for (int q = 0; q < n; ++q) {
                const float w = pp[q * m + j];
                rank += (w > v) || (w == v && q < i);
            }
            if (rank < k) atomicAdd(&cnts[i], 1);
        }
    }
    __syncthreads();
    const float scale = dloss[b] * alpha * (float)n / ((float)k * (float)n_elig * (float)n_elig);     // dloss alpha (n / k l) / l
    for (int j = tid; j < m; j += 128) {
        const int cnt = max(0, min(l_p, Lv - j * l_p));
        float dot = 0.f;
        for (int i = 0; i < n; ++i) dot += pp[i * m + j] * scale * (float)cnts[i];
        for (int i = 0; i < n; ++i) {
            const float dl = pp[i * m + j] * (scale * (float)cnts[i] - dot);
            G[((size_t)b * m + j) * n + i] = cnt > 0 ? dl / (float)cnt : 0.f;
        }
    }
}

// dx[b, t, :] = rvec[b, patch of t, :] on real tokens, 0 on pad tokens (bf16).  grid B*m, 256 threads.
__global__ void __launch_bounds__(kThreads)
spread_rvec_kernel(const float* __restrict__ rvec, __nv_bfloat16* __restrict__ dx, int L, int Lv, int d, int m, int l_p) {
    pdl_trigger();
    pdl_wait();
    const int bj = blockIdx.x, b = bj / m, j = bj % m;
    const int vpr = d / 8;
    for (int idx = threadIdx.x; idx < l_p * vpr; idx += kThreads) {
        const int r = idx / vpr, cv = idx % vpr, t = j * l_p + r;
        float f[8];
#pragma unroll
        for (int v = 0; v < 8; ++v) f[v] = t < Lv ? rvec[(size_t)bj * d + cv * 8 + v] : 0.f;
        st_stream16(dx + ((size_t)b * L + t) * d + (size_t)cv * 8, pack16<__nv_bfloat16>(f));
    }
}

struct BwdWs { size_t plan, dyg, xg, dh, ag, dxg, dgp, G, pool, rvec, dgate, wpart, wgpart, total; int nt; };

BwdWs bwd_ws(const Dims& D) {
    WsCarver w;
    w.take(kStatusBytes);
    BwdWs r;
    r.nt = D.d_e / gemm_bf16_bn(D.d_e > 0 ? D.d_e : 64);
    if (r.nt < 1) r.nt = 1;
    r.plan = w.take(plan_bytes(D, true));
    const bool fused = can_fuse_gather(D) && wgrad_can_gather(D.l_p);      // dy and x gathered inside the consumers' TMA loads
    r.dyg = fused ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);
    r.xg = fused ? 0 : w.take((size_t)D.Rmax * D.d * D.esize);
    r.dh = w.take((size_t)D.Rmax * D.d_e * D.esize);
    r.ag = w.take((size_t)D.Rmax * D.d_e * D.esize);
    r.dxg = w.take((size_t)D.Rmax * D.d * D.esize);
    r.dgp = w.take((size_t)D.Rmax * r.nt * sizeof(float));
    r.G = w.take((size_t)D.B * D.m * D.n * sizeof(float));
    r.pool = w.take((size_t)D.B * D.m * D.d * sizeof(float));
    r.rvec = w.take((size_t)D.B * D.m * D.d * sizeof(float));
    r.dgate = w.take((size_t)D.B * D.k * D.c * sizeof(float));
    r.wpart = w.take((size_t)kDwrSplit * D.d * D.n * sizeof(float));
    {   // split-K partials, sized for the larger of the two weight gradients
        const size_t s1 = wgrad_scratch_bytes(D.n, D.d, D.d_e, D.Rmax), s2 = wgrad_scratch_bytes(D.n, D.d_e, D.d, D.Rmax);
        r.wgpart = w.take((s1 > s2 ? s1 : s2) + 1024);
    }
    r.total = w.off;
    return r;
}

}  // namespace

// Router half of a backward pass, shared by the UoME and SMHA backward: per-row partials of d(loss)/d(gate)
// -> dgate per (sample, expert, patch) -> gradient of the router logits G (softmax Jacobians of Eq. 14 and 21)
// -> dW_r (through the pooled token sums) and rvec, the vector every real token of a patch receives in dx.
uoe_status launch_router_backward(const Dims& D, const void* x, const void* W_r, const int* expert_idx,
                                  const int* patch_idx, const float* p_samp, const float* p_patch, const PlanPtrs& P,
                                  const float* dgp, int nt, const RouterBwdScratch& rs, float* dW_r, cudaStream_t stream) {
    if (!D.bf16) return UOE_ERR_UNSUPPORTED;
    if ((size_t)2 * D.n * D.m * sizeof(float) > 40 * 1024) return UOE_ERR_UNSUPPORTED;
    float *G = rs.G, *pool = rs.pool, *rvec = rs.rvec, *dgate = rs.dgate, *wpart = rs.wpart;
    {
        ProfScope ps("dgate", stream);
        const int n_slabs = D.B * D.k * D.c;
        launch_k(dgate_kernel, dim3((n_slabs + 3) / 4), dim3(128), 0, stream, dgp, nt, P.pair_row, patch_idx, n_slabs, D.c, D.m, D.l_p,
                                                           dgate);
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("router_bwd", stream);
        launch_k(router_bwd_kernel, dim3(D.B), dim3(128), (size_t)2 * D.n * D.m * sizeof(float), stream, 
            dgate, expert_idx, patch_idx, p_samp, p_patch, D.n, D.k, D.m, D.c, D.l_p, D.Lv, G);
    }
    UOE_LAUNCHED();
    int CT = 64;
    while (CT > 1 && (CT / 2) * 8 >= D.d) CT /= 2;
    const int nchunks = (D.d + CT * 8 - 1) / (CT * 8);
    dim3 grid((unsigned)(D.B * D.m * nchunks));
    {
        ProfScope ps("pool", stream);
        launch_k(pool_kernel<__nv_bfloat16>, grid, dim3(kThreads), 0, stream, (const __nv_bfloat16*)x, pool, D.L, D.Lv, D.d,
                                                                  D.m, D.l_p, CT, nchunks);
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("dW_r", stream);
        dim3 g2((D.d + kThreads - 1) / kThreads, dwr_split(D.d));
        launch_k(dwr_partial_kernel, g2, dim3(kThreads), 0, stream, pool, G, wpart, D.B * D.m, D.d, D.n);
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("dW_r_sum", stream);
        const int total = D.d * D.n;
        launch_k(dwr_sum_kernel, dim3((total + kThreads - 1) / kThreads), dim3(kThreads), 0, stream, wpart, dW_r, total, dwr_split(D.d));
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("router_dx_vec", stream);
        launch_k(rvec_kernel<__nv_bfloat16>, dim3(D.B * D.m), dim3(kThreads), 0, stream, (const __nv_bfloat16*)W_r, G, rvec, D.d, D.n);
    }
    UOE_LAUNCHED();
    return UOE_OK;
}

size_t router_backward_scratch_bytes(const Dims& D) {
    return align_up((size_t)D.B * D.m * D.n * 4, 1024) + 2 * align_up((size_t)D.B * D.m * D.d * 4, 1024) +
           align_up((size_t)D.B * D.k * D.c * 4, 1024) + align_up((size_t)kDwrSplit * D.d * D.n * 4, 1024);
}

RouterBwdScratch router_backward_scratch(const Dims& D, char* base) {
    RouterBwdScratch r;
    r.G = (float*)base;
    base += align_up((size_t)D.B * D.m * D.n * 4, 1024);
    r.pool = (float*)base;
    base += align_up((size_t)D.B * D.m * D.d * 4, 1024);
    r.rvec = (float*)base;
    base += align_up((size_t)D.B * D.m * D.d * 4, 1024);
    r.dgate = (float*)base;
    base += align_up((size_t)D.B * D.k * D.c * 4, 1024);
    r.wpart = (float*)base;
    return r;
}

size_t mlp_bwd_workspace_bytes(const Dims& D) { return bwd_ws(D).total; }

}  // namespace uoe

using namespace uoe;

extern "C" uoe_status uoe_mlp_backward(const uoe_problem* prob, const void* x, const void* W1, const void* W2,
                                       const void* W_r, const int32_t* expert_idx, const int32_t* patch_idx,
                                       const float* gate, const int32_t* expert_offsets, const float* p_samp,
                                       const float* p_patch, const void* saved_h, const void* dy, void* dx,
                                       float* dW1, float* dW2, float* dW_r, void* ws, size_t ws_bytes,
                                       void* cuda_stream) {
    Dims D;
    uoe_status st = make_dims(prob, D);
    if (st != UOE_OK) return st;
    if (!x || !W1 || !W2 || !W_r || !expert_idx || !patch_idx || !gate || !expert_offsets || !p_samp || !p_patch ||
        !saved_h || !dy || !dx || !dW1 || !dW2 || !dW_r || !ws)
        return UOE_ERR_INVALID_ARG;
    if (D.d_e < 1) return UOE_ERR_INVALID_ARG;
    const void* al[] = {x, W1, W2, saved_h, dy, dx, dW1, dW2, ws};
    for (const void* p : al)
        if (!aligned16(p)) return UOE_ERR_INVALID_ARG;
    // tensor-core path only: bf16, widths that tile the 128-row weight-gradient MMA
    if (!D.bf16 || D.d % 128 != 0 || D.d_e % 128 != 0) return UOE_ERR_UNSUPPORTED;
    if ((size_t)2 * D.n * D.m * sizeof(float) > 40 * 1024) return UOE_ERR_UNSUPPORTED;
    const BwdWs W = bwd_ws(D);
    if (ws_bytes < W.total) return UOE_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const bool use_gate = (prob->flags & UOE_FLAG_GATE) != 0;
    const bool residual = (prob->flags & UOE_FLAG_RESIDUAL) != 0;
    char* base = (char*)ws;
    int* status = (int*)base;
    const PlanPtrs P = plan_ptrs(D, base + W.plan, true);
    // rows of the per-row weights that belong to no pair (region padding) must read as zero
    UOE_CUDA_OK(cudaMemsetAsync(P.row_gate, 0, 2 * align_up((size_t)D.Rmax * 4, 1024), stream));
    void *dyg = base + W.dyg, *xg = base + W.xg, *dh = base + W.dh, *ag = base + W.ag, *dxg = base + W.dxg;
    float* dgp = (float*)(base + W.dgp);
    float* G = (float*)(base + W.G);
    float* pool = (float*)(base + W.pool);
    float* rvec = (float*)(base + W.rvec);
    float* dgate = (float*)(base + W.dgate);
    float* wpart = (float*)(base + W.wpart);

    st = launch_plan(D, expert_idx, patch_idx, gate, expert_offsets, P, status, stream, use_gate);
    if (st != UOE_OK) return st;
    // Eq. 18 for dy and x: either inside the TMA loads of the kernels that consume them, or as routed copies
    const bool fused = can_fuse_gather(D) && wgrad_can_gather(D.l_p);
    if (!fused) {
        st = launch_gather(D, dy, patch_idx, expert_offsets, P, dyg, stream);
        if (st != UOE_OK) return st;
        st = launch_gather(D, x, patch_idx, expert_offsets, P, xg, stream);
        if (st != UOE_OK) return st;
    }
    WgradGather gq, gp;          // dW2 = ag^T dy_g (Q gathered), dW1 = x_g^T dh (P gathered)
    if (fused) {
        gq.gather_q = true; gq.src_patch = P.src_patch; gq.l_p = D.l_p; gq.Bm = D.B * D.m;
        gp.gather_p = true; gp.src_patch = P.src_patch; gp.l_p = D.l_p; gp.Bm = D.B * D.m;
    }

    GemmArgs ga{dyg, W2, nullptr, dh, nullptr, expert_offsets, D.n, D.d, D.d_e, prob->act, true, D.Rmax};
    ga.label = "bwd_da_dh";
    ga.bwd = true; ga.bwd_h = saved_h; ga.row_gate = P.row_gate; ga.row_valid = P.row_valid; ga.dg_part = dgp; ga.C1 = ag;
    if (fused) { ga.gather_x = dy; ga.src_patch = P.src_patch; ga.l_p = D.l_p; ga.Bm = D.B * D.m; }
    st = launch_gemm_bf16(ga, status, stream);
    if (st != UOE_OK) return st;
    st = launch_wgrad_bf16(ag, fused ? dy : dyg, dW2, expert_offsets, D.n, D.d_e, D.d, D.Rmax, "wgrad_W2", status, stream,
                           wgrad_scratch_bytes(D.n, D.d_e, D.d, D.Rmax) ? (float*)(base + W.wgpart) : nullptr, gq);
    if (st != UOE_OK) return st;
    // patches of 128 tokens: dx_g and the combine are one kernel walked by output patch, after the router's term is known
    const bool patch_major = gemm2_patch_can(D, P, nullptr);
    if (!patch_major) {
        GemmArgs gx{dh, W1, nullptr, dxg, nullptr, expert_offsets, D.n, D.d_e, D.d, UOE_ACT_IDENTITY, true, D.Rmax};
        gx.label = "bwd_dx";
        st = launch_gemm_bf16(gx, status, stream);
        if (st != UOE_OK) return st;
    }
    st = launch_wgrad_bf16(fused ? x : xg, dh, dW1, expert_offsets, D.n, D.d, D.d_e, D.Rmax, "wgrad_W1", status, stream,
                           wgrad_scratch_bytes(D.n, D.d, D.d_e, D.Rmax) ? (float*)(base + W.wgpart) : nullptr, gp);
    if (st != UOE_OK) return st;

    if (use_gate) {
        RouterBwdScratch rs{G, pool, rvec, dgate, wpart};
        st = launch_router_backward(D, x, W_r, expert_idx, patch_idx, p_samp, p_patch, P, dgp, W.nt, rs, dW_r, stream);
        if (st != UOE_OK) return st;
    } else {
        UOE_CUDA_OK(cudaMemsetAsync(dW_r, 0, (size_t)D.d * D.n * sizeof(float), stream));
    }
    // dx = dy (selective residual) + the routed input gradients (the gate is already inside dh) + router term
    if (patch_major)
        return launch_gemm2_patch(D, dh, W1, dy, dx, expert_offsets, P, residual, status, stream, true,
                                  use_gate ? rvec : nullptr, "bwd_dx");
    return launch_combine(D, dy, dxg, P, residual, false, dx, stream, use_gate ? rvec : nullptr);
}


namespace uoe {
size_t balance_bwd_workspace_bytes(const Dims& D) { return kStatusBytes + router_backward_scratch_bytes(D); }
}  // namespace uoe

extern "C" uoe_status uoe_route_balance_backward(const uoe_problem* prob, const void* x, const void* W_r,
                                                 const float* p_patch, float alpha, const float* dloss, void* dx,
                                                 float* dW_r, void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims D;
    uoe_status st = make_dims(prob, D);
    if (st != UOE_OK) return st;
    if (!x || !W_r || !p_patch || !dloss || !dx || !dW_r || !ws) return UOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(dx) || !aligned16(ws)) return UOE_ERR_INVALID_ARG;
    if (!D.bf16) return UOE_ERR_UNSUPPORTED;
    if ((size_t)D.n * D.m * sizeof(float) > 36 * 1024) return UOE_ERR_UNSUPPORTED;
    if (ws_bytes < balance_bwd_workspace_bytes(D)) return UOE_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const RouterBwdScratch rs = router_backward_scratch(D, (char*)ws + kStatusBytes);
    {
        ProfScope ps("balance_bwd", stream);
        launch_k(balance_bwd_kernel, dim3(D.B), dim3(128), (size_t)D.n * D.m * sizeof(float), stream, p_patch, dloss, D.Lv, D.n,
                 D.k, D.m, D.l_p, alpha, rs.G);
    }
    UOE_LAUNCHED();
    int CT = 64;
    while (CT > 1 && (CT / 2) * 8 >= D.d) CT /= 2;
    const int nchunks = (D.d + CT * 8 - 1) / (CT * 8);
    {
        ProfScope ps("pool", stream);
        launch_k(pool_kernel<__nv_bfloat16>, dim3((unsigned)(D.B * D.m * nchunks)), dim3(kThreads), 0, stream,
                 (const __nv_bfloat16*)x, rs.pool, D.L, D.Lv, D.d, D.m, D.l_p, CT, nchunks);
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("dW_r", stream);
        launch_k(dwr_partial_kernel, dim3((D.d + kThreads - 1) / kThreads, dwr_split(D.d)), dim3(kThreads), 0, stream, (const float*)rs.pool,
                 (const float*)rs.G, rs.wpart, D.B * D.m, D.d, D.n);
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("dW_r_sum", stream);
        const int total = D.d * D.n;
        launch_k(dwr_sum_kernel, dim3((total + kThreads - 1) / kThreads), dim3(kThreads), 0, stream, (const float*)rs.wpart, dW_r, total, dwr_split(D.d));
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("router_dx_vec", stream);
        launch_k(rvec_kernel<__nv_bfloat16>, dim3(D.B * D.m), dim3(kThreads), 0, stream, (const __nv_bfloat16*)W_r, (const float*)rs.G,
                 rs.rvec, D.d, D.n);
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("spread_rvec", stream);
        launch_k(spread_rvec_kernel, dim3(D.B * D.m), dim3(kThreads), 0, stream, (const float*)rs.rvec, (__nv_bfloat16*)dx, D.L, D.Lv,
                 D.d, D.m, D.l_p);
    }
    UOE_LAUNCHED();
    return UOE_OK;
}
