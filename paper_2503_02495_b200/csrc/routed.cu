// Data movement around the expert GEMMs: the routing plan, the token gather (Eq. 18 / 24), the
// weighted combine (Eq. 20 / 26 / 40), and the float32 grouped GEMM used by the float32 path.
#include "kernels.cuh"

namespace uoe {
namespace {

constexpr int kThreads = 256;

// ---------------------------------------------------------------------------------------------
// pair rows for many samples: one CTA passes over expert_idx [B,k] once, a warp per expert, 32 samples per step,
// and writes where every (sample, slot) pair's rows start (samples ascending inside an expert's region).  O(B k)
// work in all, where plan_kernel's own scan of the earlier samples is O(B k) per sample.
// ---------------------------------------------------------------------------------------------
constexpr int kPlanScanMaxB = 512;        // up to here every sample's CTA scans the earlier samples itself

__global__ void __launch_bounds__(1024)
plan_rows_kernel(const int* __restrict__ expert_idx, const int* __restrict__ offsets, int B, int n, int k, int l_a,
                 int* __restrict__ pair_row, int* status) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = warp; i < n; i += 32) {
        const int off_i = offsets[i];
        int running = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int slot = -1;
            if (b < B)
                for (int s = 0; s < k; ++s) {
                    const int e = expert_idx[(size_t)b * k + s];
                    if (e < 0 || e >= n) set_status(status, UOE_ERR_DEVICE_INDEX);
                    if (e == i) slot = s;
                }
            const unsigned ball = __ballot_sync(0xffffffffu, slot >= 0);
            if (slot >= 0) pair_row[(size_t)b * k + slot] = off_i + (running + __popc(ball & ((1u << lane) - 1u))) * l_a;
            running += __popc(ball);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// plan: grid B, 128 threads (512 when the backward asks for long per-row arrays), dynamic shared memory 8*k*c bytes.  Everything a sample needs from global memory
// (its routing arrays, the offsets, the expert choices of the samples before it) is fetched in one round of
// independent loads; the rest runs out of shared memory.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512)
plan_kernel(const int* __restrict__ expert_idx, const int* __restrict__ patch_idx, const float* __restrict__ gate,
            const int* __restrict__ offsets, int B, int n, int k, int m, int c, int l_p,
            int* __restrict__ pair_row, int* __restrict__ inv_row, float* __restrict__ inv_gate,
            int* __restrict__ expert_end, int* status, float* __restrict__ row_gate, float* __restrict__ row_valid,
            int Lv, int use_gate, int* __restrict__ src_patch, uint4* __restrict__ tail, long long tail_row_vecs,
            long long rows_max, int rows_given /* pair_row already holds every pair's first row (plan_rows_kernel) */) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ int s_dyn[];
    int* s_pi = s_dyn;                         // [k*c] patch indices of this sample
    float* s_g = (float*)(s_dyn + k * c);      // [k*c] gates
    __shared__ int my_e[32], prow[32], hist[33], offs[34];
    const int b = blockIdx.x, tid = threadIdx.x, NT = blockDim.x;      // NT: 128 or 512 (long per-row arrays)
    const int l_a = c * l_p;
    if (tid < 33) hist[tid] = 0;
    __syncthreads();
    // ---- one round of loads ----
    if (tid < k) {
        int e = expert_idx[b * k + tid];
        if (e < 0 || e >= n) { set_status(status, UOE_ERR_DEVICE_INDEX); e = 0; }
        my_e[tid] = e;
    }
    if (tid <= n) offs[tid] = offsets[tid];
    for (int idx = tid; idx < k * c; idx += NT) {
        const int pj = patch_idx[(size_t)b * k * c + idx];
        if (pj < -1 || pj >= m) set_status(status, UOE_ERR_DEVICE_INDEX);
        s_pi[idx] = pj;
        s_g[idx] = gate[(size_t)b * k * c + idx];
    }
    if (!rows_given) {   // choices of the samples before b, per expert: lane i of each warp counts expert i through ballots
        int acc = 0;
        const int lane = tid & 31;
        for (int i0 = 0; i0 < b * k; i0 += NT) {
            const int idx = i0 + tid;
            const int e = idx < b * k ? expert_idx[idx] : -1;
            for (int i = 0; i < n; ++i) {
                const unsigned msk = __ballot_sync(0xffffffffu, e == i);
                if (lane == i) acc += __popc(msk);
            }
        }
        if (lane < n && acc) atomicAdd(&hist[lane], acc);
    }
    __syncthreads();
    if (tid < k) {
        const int row = rows_given ? pair_row[b * k + tid] : offs[my_e[tid]] + hist[my_e[tid]] * l_a;
        prow[tid] = row;
        if (!rows_given) pair_row[b * k + tid] = row;
    }
    __syncthreads();
    for (int idx = tid; idx < m * k; idx += NT) {          // inverse map: which routed rows feed patch j
        const int j = idx / k, s = idx % k;
        int row = -1;
        float g = 0.f;
        for (int u = 0; u < c; ++u)
            if (s_pi[s * c + u] == j) { row = prow[s] + u * l_p; g = s_g[s * c + u]; }
        inv_row[((size_t)b * m + j) * k + s] = row;
        inv_gate[((size_t)b * m + j) * k + s] = g;
    }
    // source patch of every l_p-row block (used when the GEMM gathers its own A operand)
    for (int idx = tid; idx < k * c; idx += NT) {
        const int s = idx / c, u = idx % c;
        const int pj = s_pi[idx];
        src_patch[prow[s] / l_p + u] = (pj >= 0 && pj < m) ? b * m + pj : -1;
    }
    if (b == B - 1) {          // the last sample has seen every choice: ends of the expert regions, padding blocks
        __shared__ int s_end[32];
        if (rows_given) {      // the last pair of a region starts l_a rows before its end: the largest first row per expert
            if (tid < n) s_end[tid] = offs[tid];
            __syncthreads();
            for (int idx = tid; idx < B * k; idx += NT) {
                const int e = expert_idx[idx];
                if (e >= 0 && e < n) atomicMax(&s_end[e], pair_row[idx] + l_a);
            }
            __syncthreads();
            if (tid < n) expert_end[tid] = s_end[tid];
        } else {
            if (tid < k) atomicAdd(&hist[my_e[tid]], 1);
            __syncthreads();
            if (tid < n) s_end[tid] = expert_end[tid] = offs[tid] + hist[tid] * l_a;
        }
        __syncthreads();
        for (int i = 0; i < n; ++i)
            for (int rb = s_end[i] / l_p + tid; rb < offs[i + 1] / l_p; rb += NT) src_patch[rb] = -1;
    }
    if (tail) {
        const long long r0 = offs[n];
        const long long total = (rows_max - r0) * tail_row_vecs;
        for (long long q = (long long)b * NT + tid; q < total; q += (long long)B * NT)
            tail[r0 * tail_row_vecs + q] = make_uint4(0, 0, 0, 0);
    }
    if (row_gate) {                          // per-row weights for the backward
        for (int idx = tid; idx < k * l_a; idx += NT) {
            const int s = idx / l_a, r = idx % l_a, u = r / l_p;
            const int pj = s_pi[s * c + u];
            const bool real = pj >= 0 && pj < m && pj * l_p + (r % l_p) < Lv;
            const float g = use_gate ? s_g[s * c + u] : 1.0f;
            row_gate[prow[s] + r] = real ? g : 0.f;
            row_valid[prow[s] + r] = real ? 1.f : 0.f;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// gather: grid (B*k*c + n, nsplit); a patch is one contiguous slab of l_p*d elements on both sides
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
gather_kernel(const uint4* __restrict__ src, const int* __restrict__ patch_idx, const int* __restrict__ offsets,
              const int* __restrict__ pair_row, const int* __restrict__ expert_end,
              uint4* __restrict__ dst, int n_slabs, int k, int c, int m, long long slab_vecs /* l_p*d*esize/16 */,
              long long row_vecs /* d*esize/16 */, int l_p, int n, uint4* __restrict__ tail, long long tail_row_vecs,
              long long rows_max) {
    pdl_trigger();
    pdl_wait();
    const int bx = blockIdx.x;
    long long count;                 // 16-byte pieces to write
    const uint4* s = nullptr;
    uint4* o;
    if (bx == n_slabs + n) {         // rows of `tail` that no kernel writes
        const long long r0 = offsets[n];
        o = tail + r0 * tail_row_vecs;
        count = (rows_max - r0) * tail_row_vecs;
    } else if (bx < n_slabs) {
        const int pair = bx / c, u = bx % c, b = pair / k;
        const int j = patch_idx[bx];
        o = dst + ((long long)pair_row[pair] + (long long)u * l_p) * row_vecs;
        count = slab_vecs;
        if (j >= 0 && j < m) s = src + ((long long)b * m + j) * slab_vecs;
    } else {
        const int i = bx - n_slabs;
        const long long r0 = expert_end[i], r1 = offsets[i + 1];
        o = dst + r0 * row_vecs;
        count = (r1 - r0) * row_vecs;
    }
    const long long per = (count + gridDim.y - 1) / gridDim.y;
    const long long lo = per * blockIdx.y, hi = min(count, lo + per);
    if (s) {
        long long i = lo + threadIdx.x;
        for (; i + 3 * kThreads < hi; i += 4 * kThreads) {
            uint4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = ld_stream16(s + i + q * kThreads);
#pragma unroll
            for (int q = 0; q < 4; ++q) st_stream16(o + i + q * kThreads, v[q]);
        }
        for (; i < hi; i += kThreads) st_stream16(o + i, ld_stream16(s + i));
    } else {
        const uint4 z = make_uint4(0, 0, 0, 0);
        for (long long i = lo + threadIdx.x; i < hi; i += kThreads) st_stream16(o + i, z);
    }
}

// ---------------------------------------------------------------------------------------------
// combine: grid (B*m, row groups)
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads)
combine_kernel(const T* __restrict__ x, const T* __restrict__ z, const int* __restrict__ inv_row,
               const float* __restrict__ inv_gate, T* __restrict__ y, int L, int Lv, int d, int m, int k,
               int l_p, int residual, int use_gate, int rows_per_cta, const float* __restrict__ rvec,
               const int* __restrict__ pair_row /* not null: inv_row holds offsets from the pair's first row */,
               const float* __restrict__ gate_bkc /* not null: whole samples per expert (slot u is patch u): no inverse map,
                                                     weights from the router's gate array [B,k,c] */, int c) {
    pdl_trigger();
    pdl_wait();
    constexpr int V = Vec16<T>::N;
    __shared__ int srow[32];
    __shared__ float sg[32];
    const int bj = blockIdx.x, b = bj / m, j = bj % m;
    const int r0 = blockIdx.y * rows_per_cta, r1 = min(l_p, r0 + rows_per_cta);
    if (threadIdx.x < k) {
        if (gate_bkc) {          // Eq. 26: the token's row in every chosen expert follows from its position alone
            srow[threadIdx.x] = j * l_p < Lv ? pair_row[(size_t)b * k + threadIdx.x] + j * l_p : -1;
            sg[threadIdx.x] = use_gate ? gate_bkc[((size_t)b * k + threadIdx.x) * c + j] : 1.0f;
        } else {
            const int rel = inv_row[(size_t)bj * k + threadIdx.x];
            const int base = pair_row ? pair_row[(size_t)b * k + threadIdx.x] : 0;
            srow[threadIdx.x] = rel >= 0 ? rel + base : -1;
            sg[threadIdx.x] = use_gate ? inv_gate[(size_t)bj * k + threadIdx.x] : 1.0f;
        }
    }
    __syncthreads();
    const int vpr = d / V;
    const int total = (r1 - r0) * vpr;
    for (int idx = threadIdx.x; idx < total; idx += kThreads) {
        const int r = r0 + idx / vpr, cv = idx % vpr;
        const int t = j * l_p + r;
        const size_t xo = ((size_t)b * L + t) * d + (size_t)cv * V;
        // the loads of a round (x and up to four slots) are issued together, then added in ascending slot order
        const bool real = t < Lv;
        uint4 xv = make_uint4(0, 0, 0, 0), q[4];
        if (residual) xv = ld_stream16(x + xo);
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (real && u < k && srow[u] >= 0) q[u] = ld_stream16(z + ((size_t)(srow[u] + r)) * d + (size_t)cv * V);
        float acc[V];
        unpack16<T>(xv, acc);
        if (real) {
            for (int s0 = 0; s0 < k; s0 += 4) {
                if (s0 > 0) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (s0 + u < k && srow[s0 + u] >= 0)
                            q[u] = ld_stream16(z + ((size_t)(srow[s0 + u] + r)) * d + (size_t)cv * V);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (s0 + u < k && srow[s0 + u] >= 0) {
                        float f[V];
                        unpack16<T>(q[u], f);
                        const float g = sg[s0 + u];
#pragma unroll
                        for (int v = 0; v < V; ++v) acc[v] = fmaf(g, f[v], acc[v]);
                    }
                }
            }
            if (rvec) {
                const float* rp = rvec + (size_t)bj * d + (size_t)cv * V;
#pragma unroll
                for (int v = 0; v < V; v += 4) {
                    const float4 rq = *(const float4*)(rp + v);
                    acc[v] += rq.x; acc[v + 1] += rq.y; acc[v + 2] += rq.z; acc[v + 3] += rq.w;
                }
            }
        }
        st_stream16(y + xo, pack16<T>(acc));
    }
}

// ---------------------------------------------------------------------------------------------
// float32 grouped GEMM (FFMA): 64x64 tile, 16-deep K step, 4x4 outputs per thread
// ---------------------------------------------------------------------------------------------
constexpr int BM = 64, BN = 64, BK = 16;

__global__ void __launch_bounds__(256)
gemm_f32_kernel(const float* __restrict__ A, const float* __restrict__ W, const float* __restrict__ bias,
                float* __restrict__ C, float* __restrict__ pre, const int* __restrict__ offsets, int n, int K, int N,
                int act, int b_kmajor) {
    pdl_trigger();
    pdl_wait();
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int total_rows = offsets[n];
    const int row0 = blockIdx.x * BM;
    if (row0 >= total_rows) return;
    int e = 0;
    while (e + 1 < n && row0 >= offsets[e + 1]) ++e;       // regions are multiples of 128 rows: no tile straddles
    const int col0 = blockIdx.y * BN;
    const float* We = W + (size_t)e * K * N;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        for (int idx = threadIdx.x; idx < BM * BK; idx += 256) {
            const int r = idx / BK, kk = idx % BK;
            As[kk][r] = (k0 + kk < K) ? A[(size_t)(row0 + r) * K + k0 + kk] : 0.f;
        }
        for (int idx = threadIdx.x; idx < BK * BN; idx += 256) {
            int kk, cc;
            if (b_kmajor) { cc = idx / BK; kk = idx % BK; } else { kk = idx / BN; cc = idx % BN; }
            float v = 0.f;
            if (k0 + kk < K && col0 + cc < N)
                v = b_kmajor ? We[(size_t)(col0 + cc) * K + k0 + kk] : We[(size_t)(k0 + kk) * N + col0 + cc];
            Bs[kk][cc] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], bb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bb[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const size_t r = (size_t)row0 + ty * 4 + i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int cc = col0 + tx * 4 + j;
            if (cc >= N) continue;
            float v = acc[i][j];
            if (bias) v += bias[(size_t)e * N + cc];
            if (pre) pre[r * N + cc] = v;
            C[r * N + cc] = act_apply(v, act);
        }
    }
}

}  // namespace

uoe_status launch_plan(const Dims& D, const int* expert_idx, const int* patch_idx, const float* gate,
                       const int* offsets, const PlanPtrs& P, int* status, cudaStream_t s, bool use_gate, void* tail,
                       long long tail_row_bytes) {
    const size_t smem = (size_t)D.k * D.c * 8;
    if (smem > 32 * 1024) return UOE_ERR_UNSUPPORTED;      // a sample's routing arrays live in shared memory
    const bool many = D.B > kPlanScanMaxB;
    if (many) {
        ProfScope ps("plan_rows", s);
        launch_k(plan_rows_kernel, dim3(1), dim3(1024), 0, s, expert_idx, offsets, D.B, D.n, D.k, D.l_a, P.pair_row, status);
        UOE_LAUNCHED();
    }
    ProfScope ps("plan", s);
    const int threads = (P.row_gate && (long long)D.k * D.l_a >= 4096) ? 512 : 128;      // the backward's per-row weights: k*l_a rows per sample
    launch_k(plan_kernel, dim3(D.B), dim3(threads), smem, s, expert_idx, patch_idx, gate, offsets, D.B, D.n, D.k, D.m, D.c, D.l_p,
                                    P.pair_row, P.inv_row, P.inv_gate, P.expert_end, status, P.row_gate, P.row_valid,
                                    D.Lv, use_gate ? 1 : 0, P.src_patch, (uint4*)tail, tail_row_bytes / 16, D.Rmax, many ? 1 : 0);
    UOE_LAUNCHED();
    return UOE_OK;
}

uoe_status launch_gather(const Dims& D, const void* src, const int* patch_idx, const int* offsets,
                         const PlanPtrs& P, void* dst, cudaStream_t s, void* tail, long long tail_row_bytes) {
    const long long row_vecs = (long long)D.d * D.esize / 16;
    const long long slab_vecs = row_vecs * D.l_p;
    const int n_slabs = D.B * D.k * D.c;
    int nsplit = (int)((slab_vecs * 16 + 16383) / 16384);
    if (nsplit < 1) nsplit = 1;
    if (nsplit > 128) nsplit = 128;
    dim3 grid(n_slabs + D.n + (tail ? 1 : 0), nsplit);
    ProfScope ps("gather", s);
    launch_k(gather_kernel, grid, dim3(kThreads), 0, s, (const uint4*)src, patch_idx, offsets, P.pair_row, P.expert_end,
                                            (uint4*)dst, n_slabs, D.k, D.c, D.m, slab_vecs, row_vecs, D.l_p, D.n,
                                            (uint4*)tail, tail_row_bytes / 16, D.Rmax);
    UOE_LAUNCHED();
    return UOE_OK;
}

uoe_status launch_combine(const Dims& D, const void* x, const void* z, const PlanPtrs& P, bool residual,
                          bool use_gate, void* y, cudaStream_t s, const float* rvec) {
    // 16-byte vectors per thread: two for small outputs (short dependent chains, many CTAs in flight: these launches are
    // bound by latency), four to eight once the output is tens of MB (fewer, longer CTAs: less set-up per byte; measured
    // 35 -> 31 us at 44 MB, 198 -> 183 us at 268 MB)
    const long long out_bytes = (long long)D.B * D.L * D.d * D.esize;
    const int vecs = out_bytes < (32ll << 20) ? 2 : (out_bytes < (128ll << 20) ? 4 : 8);
    int rows_per_cta = (int)(vecs * kThreads * 16 / ((long long)D.d * D.esize));
    if (rows_per_cta < 1) rows_per_cta = 1;
    if (rows_per_cta > D.l_p) rows_per_cta = D.l_p;
    dim3 grid(D.B * D.m, (D.l_p + rows_per_cta - 1) / rows_per_cta);
    const bool ident = P.inv_relative && P.identity_patches && P.gate != nullptr;
    ProfScope ps("combine", s);
    if (D.bf16)
        launch_k(combine_kernel<__nv_bfloat16>, grid, dim3(kThreads), 0, s, 
            (const __nv_bfloat16*)x, (const __nv_bfloat16*)z, P.inv_row, P.inv_gate, (__nv_bfloat16*)y, D.L, D.Lv,
            D.d, D.m, D.k, D.l_p, residual ? 1 : 0, use_gate ? 1 : 0, rows_per_cta, rvec,
            P.inv_relative ? (const int*)P.pair_row : (const int*)nullptr, ident ? P.gate : (const float*)nullptr, D.c);
    else
        launch_k(combine_kernel<float>, grid, dim3(kThreads), 0, s, (const float*)x, (const float*)z, P.inv_row, P.inv_gate,
                                                       (float*)y, D.L, D.Lv, D.d, D.m, D.k, D.l_p,
                                                       residual ? 1 : 0, use_gate ? 1 : 0, rows_per_cta, rvec,
                                                       P.inv_relative ? (const int*)P.pair_row : (const int*)nullptr,
                                                       ident ? P.gate : (const float*)nullptr, D.c);
    UOE_LAUNCHED();
    return UOE_OK;
}

uoe_status launch_gemm_f32(const GemmArgs& g, cudaStream_t s) {
    dim3 grid((unsigned)((g.rows_max + BM - 1) / BM), (g.N + BN - 1) / BN);
    ProfScope ps(g.label, s);
    launch_k(gemm_f32_kernel, grid, dim3(256), 0, s, (const float*)g.A, (const float*)g.W, (const float*)g.bias, (float*)g.C,
                                         (float*)g.pre, g.offsets, g.n, g.K, g.N, g.act, g.b_kmajor ? 1 : 0);
    UOE_LAUNCHED();
    return UOE_OK;
}

}  // namespace uoe
