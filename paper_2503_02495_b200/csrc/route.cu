// uoe_route: router scoring (Eq. 13-14, 21) and fused top-k expert / top-c patch selection
// (Eq. 17, 22-23) in ONE kernel:
//   every CTA streams one (patch, column chunk, row slice) of x (16-byte loads) and leaves the partial dot
//   products  sum_{t} x[t, chunk] . W_r[chunk, i];  it then takes a ticket of its sample, and the CTA that
//   completes a sample runs that sample's selection: fixed-order sum of the partials, both softmaxes,
//   rank-based selection with warp ballots, gates.  The CTA that completes the last sample turns the
//   per-expert loads into row offsets.  Tickets and loads are reset by their last user, so a workspace
//   whose control block was zeroed once (uoe_workspace_init) serves any number of calls.
#include "kernels.cuh"

namespace uoe {

long long g_launch_count = 0;

namespace {

constexpr int kScoreThreads = 256;

// Selection for sample b by one CTA of kScoreThreads threads (all threads call).  pp: n*m floats of shared memory.
__device__ void select_sample(float* pp, const float* __restrict__ partial, int nparts, int b, int B, int Lv, int n, int k,
                              int m, int c, int l_p, int use_gate, int* __restrict__ expert_idx,
                              int* __restrict__ patch_idx, float* __restrict__ gate, float* __restrict__ p_samp,
                              float* __restrict__ p_patch, int* __restrict__ offsets, int* __restrict__ load,
                              int* __restrict__ ticket) {
    constexpr int NT = kScoreThreads;
    __shared__ float ps[32];               // sample gate
    __shared__ int sel[32];                // chosen experts, ascending
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_elig = (Lv + l_p - 1) / l_p;       // patches holding at least one real token (a prefix)

    for (int idx = tid; idx < n * m; idx += NT) {
        const int i = idx / m, j = idx % m;
        const float* p = partial + ((size_t)(b * m + j) * nparts) * n + i;
        float s = 0.f;
        for (int ch = 0; ch < nparts; ++ch) s += __ldcg(p + (size_t)ch * n);     // written by other CTAs: read from L2
        pp[idx] = s;
    }
    __syncthreads();
    if (tid < n) {                          // Eq. 21: mean over the real tokens, then W_r
        float s = 0.f;
        for (int j = 0; j < m; ++j) s += pp[tid * m + j];
        ps[tid] = s / (float)Lv;
    }
    __syncthreads();
    for (int j = tid; j < m; j += NT) {     // Eq. 14: softmax over the experts of patch j
        const int cnt = max(0, min(l_p, Lv - j * l_p));
        float mx = -INFINITY;
        for (int i = 0; i < n; ++i) {
            const float v = cnt > 0 ? pp[i * m + j] / (float)cnt : 0.f;
            pp[i * m + j] = v;
            mx = fmaxf(mx, v);
        }
        float sum = 0.f;
        for (int i = 0; i < n; ++i) { const float e = expf(pp[i * m + j] - mx); pp[i * m + j] = e; sum += e; }
        for (int i = 0; i < n; ++i) {
            const float pr = pp[i * m + j] / sum;
            pp[i * m + j] = pr;
            p_patch[((size_t)b * n + i) * m + j] = pr;
        }
    }
    if (warp == 0) {
        const float v = lane < n ? ps[lane] : -INFINITY;
        float mx = v;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float e = lane < n ? expf(v - mx) : 0.f;
        float sum = e;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const float pr = e / sum;
        if (lane < n) { ps[lane] = pr; p_samp[(size_t)b * n + lane] = pr; }
        // Eq. 22: rank = number of experts that beat this one (larger value, or equal with lower index)
        int rank = 0;
        for (int i = 0; i < n; ++i) {
            const float w = __shfl_sync(0xffffffffu, pr, i);
            rank += (w > pr) || (w == pr && i < lane);
        }
        const bool pick = lane < n && rank < k;
        const unsigned mask = __ballot_sync(0xffffffffu, pick);
        if (pick) {
            const int s = __popc(mask & ((1u << lane) - 1u));
            sel[s] = lane;
            expert_idx[(size_t)b * k + s] = lane;
            atomicAdd(&load[lane], 1);
        }
    }
    __syncthreads();
    const int take = min(c, n_elig);
    for (int s = warp; s < k; s += NT / 32) {       // Eq. 17 for the s-th chosen expert
        const int i = sel[s];
        const float* v_i = pp + i * m;
        int* out_idx = patch_idx + ((size_t)b * k + s) * c;
        float* out_gate = gate + ((size_t)b * k + s) * c;
        int before = 0;
        for (int j0 = 0; j0 < n_elig; j0 += 32) {
            const int j = j0 + lane;
            const bool valid = j < n_elig;
            const float v = valid ? v_i[j] : 0.f;
            int rank = 0;
            if (valid)
                for (int jj = 0; jj < n_elig; ++jj) {
                    const float w = v_i[jj];
                    rank += (w > v) || (w == v && jj < j);
                }
            const bool pick = valid && rank < take;
            const unsigned mask = __ballot_sync(0xffffffffu, pick);
            if (pick) {
                const int pos = before + __popc(mask & ((1u << lane) - 1u));
                out_idx[pos] = j;
                out_gate[pos] = use_gate ? ps[i] * v : 1.0f;
            }
            before += __popc(mask);
        }
        for (int pos = before + lane; pos < c; pos += 32) { out_idx[pos] = -1; out_gate[pos] = 0.f; }
    }
    // Eq. 23 as row offsets: the CTA that completes the last sample turns the loads into a prefix sum
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = (atomicAdd(ticket, 1) == B - 1);
    }
    __syncthreads();
    if (s_last && warp == 0) {
        __threadfence();
        const int rows_per_pair = c * l_p;
        int rows = 0;
        if (lane < n) {
            rows = (__ldcg(load + lane) * rows_per_pair + UOE_ROW_ALIGN - 1) / UOE_ROW_ALIGN * UOE_ROW_ALIGN;
            load[lane] = 0;                 // left at zero for the next call
        }
        if (lane == 0) *ticket = 0;
        int incl = rows;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane < n) offsets[lane] = incl - rows;
        if (lane == n - 1) offsets[n] = incl;
    }
}

// grid B*m * nchunks * rsplit, column chunk fastest: a CTA takes one column chunk of one row slice of a patch,
// and CTAs that run at the same time cover neighbouring chunks of the same rows, so together they read x
// linearly.  CT threads span the columns of the chunk (16 bytes each), 256/CT span rows.
// Dynamic shared memory: the W_r rows of this chunk, CT*V*n elements (staged with cp.async behind the x loads);
// the CTA that ends up running a sample's selection reuses it for the n*m gate values.
template <typename T>
__global__ void __launch_bounds__(kScoreThreads)
route_kernel(const T* __restrict__ x, const T* __restrict__ W_r, float* __restrict__ partial,
             int B, int L, int Lv, int d, int n, int k, int m, int c, int l_p, int CT, int nchunks, int rsplit,
             int rows_per_cta, int use_gate, int* __restrict__ expert_idx, int* __restrict__ patch_idx,
             float* __restrict__ gate, float* __restrict__ p_samp, float* __restrict__ p_patch,
             int* __restrict__ offsets, int* __restrict__ ctl /* word 1: ticket, words 8..: expert loads */,
             int* __restrict__ sample_ticket /* [B] */) {
    pdl_trigger();
    pdl_wait();
    constexpr int V = Vec16<T>::N;
    extern __shared__ uint4 s_w4[];                   // W_r[c0 : c0+cw, :] as stored
    __shared__ float s_cs[kScoreThreads * V];         // per-thread column sums, later the partial dot products
    __shared__ float s_col[64 * V];                   // column sums of the chunk
    const T* s_w = (const T*)s_w4;
    const int nparts = nchunks * rsplit;
    const int bj = blockIdx.x / nparts, part = blockIdx.x % nparts;
    const int chunk = part % nchunks, rs = part / nchunks;
    const int b = bj / m, j = bj % m;
    const int tid = threadIdx.x;
    const int ct = tid % CT, rt = tid / CT, RT = kScoreThreads / CT;
    const int c0 = chunk * CT * V;
    const int cw = min(CT * V, d - c0);               // columns of this chunk (a multiple of V)
    const int col = c0 + ct * V;
    const int row_lo = rs * rows_per_cta;
    const int rows = min(max(0, min(l_p, Lv - j * l_p)), row_lo + rows_per_cta);      // this slice: [row_lo, rows)

    {   // stage the router rows of this chunk: cw*n elements, contiguous and 16-byte aligned
        const uint4* src = (const uint4*)(W_r + (size_t)c0 * n);
        const int nvec = cw * n / V;
        for (int q = tid; q < nvec; q += kScoreThreads)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"((uint32_t)__cvta_generic_to_shared(s_w4 + q)), "l"(src + q) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    }

    float cs[V];
#pragma unroll
    for (int v = 0; v < V; ++v) cs[v] = 0.f;
    if (col < d) {
        const T* base = x + ((size_t)b * L + (size_t)j * l_p) * d + col;
        int r = row_lo + rt;
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
    for (int v = 0; v < V; ++v) s_cs[tid * V + v] = cs[v];
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    for (int cc = tid; cc < cw; cc += kScoreThreads) {      // sum over the row threads, fixed order
        float a = 0.f;
        for (int q = 0; q < RT; ++q) a += s_cs[(q * CT + cc / V) * V + cc % V];
        s_col[cc] = a;
    }
    __syncthreads();
    // dot products with the n router columns: thread (group g, expert i) strides over the chunk's columns
    const int groups = kScoreThreads / n;
    const int i = tid % n, g = tid / n;
    float a = 0.f;
    if (g < groups)
        for (int cc = g; cc < cw; cc += groups) a = fmaf(s_col[cc], to_f32(s_w[cc * n + i]), a);
    s_cs[tid] = a;
    __syncthreads();
    if (tid < n) {
        float sum = 0.f;
        for (int q = 0; q < groups; ++q) sum += s_cs[q * n + tid];
        partial[((size_t)bj * nparts + part) * n + tid] = sum;
        __threadfence();
    }
    // the CTA that completes sample b (all m * nparts partials written) runs its selection
    __shared__ int s_mine;
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const int done = atomicAdd(&sample_ticket[b], 1);
        s_mine = (done == m * nparts - 1);
        if (s_mine) sample_ticket[b] = 0;         // left at zero for the next call
    }
    __syncthreads();
    if (!s_mine) return;
    __threadfence();
    select_sample((float*)s_w4, partial, nparts, b, B, Lv, n, k, m, c, l_p, use_gate, expert_idx, patch_idx, gate, p_samp,
                  p_patch, offsets, ctl + 8, ctl + 1);
}

struct RouteWs { size_t tickets, partial, total; int nchunks, CT, rsplit, rows_per_cta; size_t smem; };

RouteWs route_ws(const Dims& D) {
    const int V = 16 / D.esize;
    int CT = 64;
    while (CT > 1 && (CT / 2) * V >= D.d) CT /= 2;
    const int nchunks = (D.d + CT * V - 1) / (CT * V);
    const int rows_per_cta = 32 * (kScoreThreads / CT);       // at most four 8-deep load batches per thread
    const int rsplit = (D.l_p + rows_per_cta - 1) / rows_per_cta;
    WsCarver w;
    w.take(kStatusBytes);
    RouteWs r;
    r.tickets = w.take((size_t)D.B * sizeof(int));            // inside the control block that is zeroed once
    r.partial = w.take((size_t)D.B * D.m * nchunks * rsplit * D.n * sizeof(float));
    r.rsplit = rsplit;
    r.rows_per_cta = rows_per_cta;
    r.total = w.off;
    r.nchunks = nchunks;
    r.CT = CT;
    const size_t stage = (size_t)CT * 16 * D.n, sel = (size_t)D.n * D.m * sizeof(float);
    r.smem = stage > sel ? stage : sel;
    return r;
}

// Checks shared by uoe_route and uoe_route_static, then the launch.  `base` is the scratch (control block,
// tickets, partials); its control block must have been zero when first used.
uoe_status route_launch(const Dims& D, uint32_t flags, const void* x, const void* W_r, int32_t* expert_idx,
                        int32_t* patch_idx, float* gate, float* p_samp, float* p_patch, int32_t* expert_offsets,
                        char* base, const RouteWs& W, cudaStream_t stream, bool profile) {
    int* ctl = (int*)base;             // word 0 status (unused here), word 1 ticket, words 8.. expert loads
    int* tickets = (int*)(base + W.tickets);
    float* partial = (float*)(base + W.partial);
    const int use_gate = (flags & UOE_FLAG_GATE) ? 1 : 0;
    dim3 grid((unsigned)(D.B * D.m * W.nchunks * W.rsplit));
    if (D.bf16) {
        if (profile) {
            ProfScope ps("route", stream);
            launch_k(route_kernel<__nv_bfloat16>, grid, dim3(kScoreThreads), W.smem, stream, (const __nv_bfloat16*)x,
                     (const __nv_bfloat16*)W_r, partial, D.B, D.L, D.Lv, D.d, D.n, D.k, D.m, D.c, D.l_p, W.CT, W.nchunks,
                     W.rsplit, W.rows_per_cta, use_gate, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets, ctl,
                     tickets);
        } else {
            launch_k(route_kernel<__nv_bfloat16>, grid, dim3(kScoreThreads), W.smem, stream, (const __nv_bfloat16*)x,
                     (const __nv_bfloat16*)W_r, partial, D.B, D.L, D.Lv, D.d, D.n, D.k, D.m, D.c, D.l_p, W.CT, W.nchunks,
                     W.rsplit, W.rows_per_cta, use_gate, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets, ctl,
                     tickets);
        }
    } else {
        ProfScope ps("route", stream);
        launch_k(route_kernel<float>, grid, dim3(kScoreThreads), W.smem, stream, (const float*)x, (const float*)W_r,
                 partial, D.B, D.L, D.Lv, D.d, D.n, D.k, D.m, D.c, D.l_p, W.CT, W.nchunks, W.rsplit, W.rows_per_cta,
                 use_gate, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets, ctl, tickets);
    }
    UOE_LAUNCHED();
    return UOE_OK;
}

uoe_status route_check(const uoe_problem* prob, Dims& D, RouteWs& W, const void* x, const void* W_r,
                       const void* expert_idx, const void* patch_idx, const void* gate, const void* p_samp,
                       const void* p_patch, const void* expert_offsets) {
    uoe_status st = make_dims(prob, D);
    if (st != UOE_OK) return st;
    if (!x || !W_r || !expert_idx || !patch_idx || !gate || !p_samp || !p_patch || !expert_offsets)
        return UOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(W_r)) return UOE_ERR_INVALID_ARG;
    if ((size_t)D.n * D.m * sizeof(float) > 32 * 1024) return UOE_ERR_UNSUPPORTED;   // gate values of a sample in shared memory
    W = route_ws(D);
    if ((long long)D.B * D.m * W.nchunks * W.rsplit > 0x7fffffffll) return UOE_ERR_UNSUPPORTED;
    if (W.tickets + (size_t)D.B * sizeof(int) > kControlBytes) return UOE_ERR_UNSUPPORTED;   // tickets sit in the zeroed block
    return UOE_OK;
}

}  // namespace

size_t route_workspace_bytes(const Dims& D) { return route_ws(D).total; }

}  // namespace uoe

using namespace uoe;

extern "C" uoe_status uoe_route(const uoe_problem* prob, const void* x, const void* W_r, int32_t* expert_idx,
                                int32_t* patch_idx, float* gate, float* p_samp, float* p_patch,
                                int32_t* expert_offsets, void* ws, size_t ws_bytes, void* cuda_stream) {
    Dims D;
    RouteWs W;
    uoe_status st = route_check(prob, D, W, x, W_r, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets);
    if (st != UOE_OK) return st;
    if (!ws || !aligned16(ws)) return UOE_ERR_INVALID_ARG;
    if (ws_bytes < W.total) return UOE_ERR_WORKSPACE;
    return route_launch(D, prob->flags, x, W_r, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets, (char*)ws, W,
                        (cudaStream_t)cuda_stream, true);
}

// ------------------------------------------------------------------------------------------------
// uoe_route_static: the same kernel with its scratch in a built-in device array
// ------------------------------------------------------------------------------------------------

// Scratch of uoe_route_static: the status block (ticket, expert loads) followed by the partial dot
// products.  One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_route_static_scratch[UOE_ROUTE_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char* g_route_static_ptr[kMaxDevices] = {};    // device address of the array, per device

// In host code `g_route_static_scratch` is only a handle; the address a kernel can use comes from
// cudaGetSymbolAddress, asked once per device with that device current.
uoe_status route_static_base(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return UOE_ERR_CUDA;
    if (!g_route_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_route_static_scratch) != cudaSuccess || !p) return UOE_ERR_CUDA;
        g_route_static_ptr[dev] = (unsigned char*)p;
    }
    *out = g_route_static_ptr[dev];
    return UOE_OK;
}
}  // namespace

extern "C" uoe_status uoe_route_static(const uoe_problem* prob, const void* x, const void* W_r,
                                       int32_t* expert_idx, int32_t* patch_idx, float* gate, float* p_samp,
                                       float* p_patch, int32_t* expert_offsets, void* cuda_stream) {
    Dims D;
    RouteWs W;
    uoe_status st = route_check(prob, D, W, x, W_r, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets);
    if (st != UOE_OK) return st;
    if (W.total > (size_t)UOE_ROUTE_STATIC_SCRATCH_BYTES) return UOE_ERR_STATIC_SCRATCH;
    unsigned char* base = nullptr;
    st = route_static_base(&base);
    if (st != UOE_OK) return st;
    // the array starts zeroed (static storage) and the kernel leaves its tickets and expert loads at zero again
    return route_launch(D, prob->flags, x, W_r, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets, (char*)base,
                        W, (cudaStream_t)cuda_stream, false);
}
