// uoe_route: router scoring (Eq. 13-14, 21) and fused top-k expert / top-c patch selection (Eq. 17, 22-23).
//   Every CTA streams one (patch, column chunk, row slice) of x with 16-byte loads, sums its rows per column and
//   multiplies the sums by W_r, so that only scores leave the CTA.  The CTA that completes a sample (a ticket per
//   sample) runs that sample's selection: both softmaxes, rank-based selection with warp ballots, gates; the CTA that
//   completes the last sample turns the per-expert loads into row offsets.  One kernel for small inputs (64-thread
//   CTAs when the patches are many and tiny); for large inputs a first kernel that only streams and a second with one
//   CTA per sample.  Tickets and loads are reset by their last user, so a scratch area whose control block was
//   zeroed once (uoe_workspace_init, or the static array of uoe_route_static) serves any number of calls of any shapes.
// Also here: uoe_route_balance (Eq. 15-16, 42-44) and uoe_route_static.
#include "kernels.cuh"

namespace uoe {

long long g_launch_count = 0;

namespace {

constexpr int kScoreThreads = 256;

// Selection for sample b by one CTA of NT threads (all threads call).  pp: n*m floats of shared memory.
// Written for a short dependent chain (the router is latency-bound on all but the largest inputs): three phases
// separated by CTA barriers, then the ticket.
//   A  a warp works 32/np2 patches at a time (np2 = n rounded up to a power of two), one lane per (patch, expert):
//      adds the parts of the score in ascending order, softmax over the experts of the patch through segment
//      shuffles (Eq. 14), first-stage counts of Eq. 15 when the capacity is dynamic; the raw scores are summed per
//      expert on the side for the sample gate
//   B  warp 0: sample gate (Eq. 21), top-k experts (Eq. 22); the other warps write p_patch
//   C  a warp per chosen expert: top-c patches by rank counting (Eq. 17), gates, the inverse map of the plan
// The CTA that completes the last sample (a ticket) turns every sample's expert set (one bit mask per sample, masks[B]
// in the scratch area) into per-expert row offsets (Eq. 23) and, for the plan, each pair's first row.
template <int NT>
__device__ void select_sample(float* pp, const float* __restrict__ partial, int nparts, int b, int B, int Lv, int n, int k,
                              int m, int c, int l_p,
                              int sel_flags /* bit 0: gate weights, bit 1: dynamic capacity, bit 2: general path only */,
                              int* __restrict__ expert_idx,
                              int* __restrict__ patch_idx, float* __restrict__ gate, float* __restrict__ p_samp,
                              float* __restrict__ p_patch, int* __restrict__ offsets, unsigned* __restrict__ masks,
                              int* __restrict__ ticket, const PlanPtrs plan,
                              const float* local_scores = nullptr /* [m,n] in shared memory: used instead of `partial` */) {
    constexpr int NW = NT / 32;
    constexpr int kMaskCache = 1024;       // samples whose masks the last CTA keeps in shared memory
    __shared__ float ps[32];               // sample gate
    __shared__ float s_raw[NW][32];        // per warp: sum over its patches of the raw scores, per expert
    __shared__ int sel[32];                // chosen experts, ascending
    __shared__ int cnts[32];               // Eq. 16: patches each expert receives in the first routing stage; later: samples per expert
    __shared__ int s_last;
    __shared__ unsigned s_masks[kMaskCache];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int use_gate = sel_flags & 1, dynamic_c = (sel_flags >> 1) & 1;
    if (tid < 32) cnts[tid] = 0;
    const int n_elig = (Lv + l_p - 1) / l_p;       // patches holding at least one real token (a prefix)
    // the single-mode cases: every sample uses all experts (Eq. 12-20) / a chosen expert takes the whole sample (Eq. 21-26)
    const bool all_experts = !(sel_flags & 4) && k == n;
    const bool all_patches = !(sel_flags & 4) && !dynamic_c && c >= n_elig;
    int np2 = 1;
    while (np2 < n) np2 <<= 1;
    const int G = 32 / np2;                         // patches a warp works at a time
    if (dynamic_c) __syncthreads();                 // cnts is zero before the first count

    // ---- A ----
    {
        const int seg = lane / np2, i = lane % np2, seg_base = lane - i;
        float raw_acc = 0.f;
        for (int j0 = warp * G; j0 < m; j0 += NW * G) {
            const int j = j0 + seg;
            const bool valid = j < m && i < n;
            float s = 0.f;
            if (valid) {
                if (local_scores) {
                    s = local_scores[j * n + i];
                } else {
                    // written by other CTAs: read from L2, eight loads in flight, added in ascending order
                    const float* p = partial + ((size_t)(b * m + j) * nparts) * n + i;
                    int ch = 0;
                    for (; ch + 7 < nparts; ch += 8) {
                        float t[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) t[u] = __ldcg(p + (size_t)(ch + u) * n);
#pragma unroll
                        for (int u = 0; u < 8; ++u) s += t[u];
                    }
                    for (; ch < nparts; ++ch) s += __ldcg(p + (size_t)ch * n);
                }
            }
            raw_acc += s;
            const int cnt = valid ? max(0, min(l_p, Lv - j * l_p)) : 0;
            const float g = valid ? (cnt > 0 ? s / (float)cnt : 0.f) : -INFINITY;       // Eq. 13: mean over the patch's real tokens
            float mx = g;
            for (int o = np2 >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float e = valid ? expf(g - mx) : 0.f;
            float sum = e;
            for (int o = np2 >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            const float pr = e / sum;                    // (lanes outside the problem: 0/0, never used)
            if (valid) pp[i * m + j] = pr;
            if (dynamic_c) {                        // Eq. 15: every real patch goes to its k best experts (ties: lower index)
                int rank = 0;
                for (int q = 0; q < n; ++q) {
                    const float w = __shfl_sync(0xffffffffu, pr, seg_base + q);
                    rank += (w > pr) || (w == pr && q < i);
                }
                if (valid && j < n_elig && rank < k) atomicAdd(&cnts[i], 1);
            }
        }
        for (int o = np2; o < 32; o <<= 1) raw_acc += __shfl_xor_sync(0xffffffffu, raw_acc, o);     // over the warp's segments
        if (lane < n) s_raw[warp][lane] = raw_acc;
    }
    __syncthreads();

    // ---- B ----
    if (warp == 0) {
        float v = -INFINITY;
        if (lane < n) {                         // Eq. 21: mean over the real tokens, then W_r
            float s = 0.f;
#pragma unroll
            for (int q = 0; q < NW; ++q) s += s_raw[q][lane];
            v = s / (float)Lv;
        }
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
        if (!all_experts)
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
        }
        if (lane == 0) masks[b] = mask;
    }
    if (NW == 1 || warp > 0) {
        const int t0 = NW == 1 ? tid : tid - 32, nt = NW == 1 ? NT : NT - 32;
        for (int idx = t0; idx < n * m; idx += nt) p_patch[(size_t)b * n * m + idx] = pp[idx];
    }
    __syncthreads();

    // ---- C ----
    int take = min(c, n_elig);
    if (dynamic_c) {                        // Eq. 16: c = the largest first-stage count, capped by the slots available
        int c_dyn = 0;
        for (int i = 0; i < n; ++i) c_dyn = max(c_dyn, cnts[i]);
        take = min(take, c_dyn);
    }
    for (int s = warp; s < k; s += NW) {            // Eq. 17 for the s-th chosen expert
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
            if (!all_patches)
            for (int jj0 = 0; jj0 < n_elig; jj0 += 8) {      // eight broadcast reads at a time
                float w[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) w[u] = jj0 + u < n_elig ? v_i[jj0 + u] : -INFINITY;
#pragma unroll
                for (int u = 0; u < 8; ++u) rank += (w[u] > v) || (w[u] == v && jj0 + u < j);
            }
            const bool pick = valid && rank < take;
            const unsigned mask = __ballot_sync(0xffffffffu, pick);
            const int pos = before + __popc(mask & ((1u << lane) - 1u));
            const float g = use_gate ? ps[i] * v : 1.0f;
            if (pick) {
                out_idx[pos] = j;
                out_gate[pos] = g;
            }
            if (plan.inv_row && valid && !all_patches) {        // the inverse of Eq. 18, relative to the pair's first routed row
                plan.inv_row[((size_t)b * m + j) * k + s] = pick ? pos * l_p : -1;
                plan.inv_gate[((size_t)b * m + j) * k + s] = pick ? g : 0.f;
            }
            before += __popc(mask);
        }
        for (int pos = before + lane; pos < c; pos += 32) { out_idx[pos] = -1; out_gate[pos] = 0.f; }
        if (plan.inv_row && !all_patches)
            for (int j = n_elig + lane; j < m; j += 32) {       // patches of pad tokens only
                plan.inv_row[((size_t)b * m + j) * k + s] = -1;
                plan.inv_gate[((size_t)b * m + j) * k + s] = 0.f;
            }
    }

    // ---- the CTA that completes the last sample: Eq. 23 as row offsets, and the part of the routing plan that needs
    //      every sample's choice (where every pair's rows start, which pair owns every slot of every expert's region) ----
    if (all_experts) {
        // every expert's region holds the B samples in order: nothing here depends on another sample, no ticket
        const int l_a = c * l_p;
        const int region = (B * l_a + UOE_ROW_ALIGN - 1) / UOE_ROW_ALIGN * UOE_ROW_ALIGN;
        if (plan.pair_row && tid < n) {
            plan.pair_row[(size_t)b * k + tid] = tid * region + b * l_a;
            plan.slot_pair[(size_t)tid * B + b] = b * k + tid;
        }
        if (b == 0) {
            if (tid <= n) offsets[tid] = tid * region;
            if (plan.pair_row && tid < n) plan.expert_end[tid] = tid * region + B * l_a;
            if (plan.pair_row && plan.tail) {
                const long long r0 = (long long)n * region, r1 = min(plan.rows_max, r0 + 128);
                for (long long q = tid; q < (r1 - r0) * plan.tail_row_vecs; q += NT) plan.tail[r0 * plan.tail_row_vecs + q] = make_uint4(0, 0, 0, 0);
            }
        }
        return;
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = (atomicAdd(ticket, 1) == B - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) *ticket = 0;              // left at zero for the next call
    if (tid < 32) cnts[tid] = 0;
    __syncthreads();
    for (int b2 = tid; b2 < B; b2 += NT) {           // samples per expert
        unsigned mk = __ldcg(masks + b2);
        if (b2 < kMaskCache) s_masks[b2] = mk;
        while (mk) {
            const int i = __ffs(mk) - 1;
            mk &= mk - 1;
            atomicAdd(&cnts[i], 1);
        }
    }
    __syncthreads();
    const int l_a = c * l_p;
    const int rows = lane < n ? (cnts[lane] * l_a + UOE_ROW_ALIGN - 1) / UOE_ROW_ALIGN * UOE_ROW_ALIGN : 0;
    int incl = rows;                        // every warp scans for itself
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    const int total_rows = __shfl_sync(0xffffffffu, incl, n - 1);
    if (warp == 0) {
        if (lane < n) offsets[lane] = incl - rows;
        if (lane == 0) offsets[n] = total_rows;
    }
    if (plan.pair_row) {                    // a warp per expert, 32 samples per step: rows inside a region ascend with the sample
        for (int i = warp; i < n; i += NW) {
            const int off_i = __shfl_sync(0xffffffffu, incl - rows, i);
            int running = 0;
            for (int b0 = 0; b0 < B; b0 += 32) {
                const int b2 = b0 + lane;
                const unsigned mk = b2 < B ? (b2 < kMaskCache ? s_masks[b2] : __ldcg(masks + b2)) : 0u;
                const bool mine = (mk >> i) & 1u;
                const unsigned ball = __ballot_sync(0xffffffffu, mine);
                if (mine) {        // the chosen experts of a sample ascend: expert i sits in slot #(chosen experts below i)
                    const int s = __popc(mk & ((1u << i) - 1u));
                    const int q = running + __popc(ball & ((1u << lane) - 1u));
                    plan.pair_row[(size_t)b2 * k + s] = off_i + q * l_a;
                    plan.slot_pair[(size_t)i * B + q] = b2 * k + s;
                }
                running += __popc(ball);
            }
            if (lane == 0) plan.expert_end[i] = off_i + running * l_a;
        }
        if (plan.tail) {
            const long long r0 = total_rows, r1 = min(plan.rows_max, r0 + 128);
            for (long long q = tid; q < (r1 - r0) * plan.tail_row_vecs; q += NT) plan.tail[r0 * plan.tail_row_vecs + q] = make_uint4(0, 0, 0, 0);
        }
    }
}

// Scoring (Eq. 13, 21) and selection, in one kernel or two.  Grid B*m * nchunks * rsplit, column chunk fastest: a CTA
// takes one column chunk of one row slice of a patch (CT threads span the columns of the chunk, 16 bytes each, NT/CT
// span rows).  CTAs that run at the same time cover neighbouring chunks of the same rows, so together they read x
// linearly.  The CTA first asks for the rows of W_r that belong to its columns (cp.async into shared memory, landing
// behind the x loads), sums its rows of x per column, and multiplies the column sums by those rows: n partial scores,
// score_part[patch, part, i], are all that leaves the CTA -- pooled activations never reach global memory.
//   TICKET   the CTA that completes a sample (a ticket per sample, m * parts arrivals) runs its selection, which adds
//            the parts in ascending order.  One launch: for small inputs.
//   !TICKET  the kernel does nothing but stream and dot, and route_select_kernel (one CTA per sample) follows.  For
//            large inputs, where a second launch costs less than CTAs that carry the selection code and its registers.
// Dynamic shared memory: max(n*m floats for the selection, the CTA's block of W_r rows).

template <typename T, bool TICKET, int NT>
__global__ void __launch_bounds__(NT, NT == 64 ? (TICKET ? 16 : 32) : (TICKET ? 5 : 6))
route_kernel(const T* __restrict__ x, const T* __restrict__ W_r, float* __restrict__ scores, int B, int L, int Lv, int d,
             int n, int k, int m, int c, int l_p, int CT, int nchunks, int rsplit, int rows_per_cta, int use_gate,
             int* __restrict__ expert_idx, int* __restrict__ patch_idx, float* __restrict__ gate,
             float* __restrict__ p_samp, float* __restrict__ p_patch, int* __restrict__ offsets,
             int* __restrict__ ctl /* word 1: ticket */, int* __restrict__ sample_ticket /* [B] */, unsigned* __restrict__ masks /* [B] */,
             const PlanPtrs plan /* all null: no plan is written */) {
    pdl_trigger();
    pdl_wait();
    constexpr int V = Vec16<T>::N;
    extern __shared__ uint4 s_dyn4[];
    __shared__ __align__(16) float s_cs[NT * V];                    // column sums across row threads; later pooled columns, dot partials
    __shared__ int s_mine;
    const int tid = threadIdx.x;
    const int nparts = nchunks * rsplit;
    const int bj = blockIdx.x / nparts;
    const int b = bj / m, j = bj % m;
    const int part = blockIdx.x % nparts;
    const int chunk = part % nchunks, rs = part / nchunks;
    const int c0 = chunk * CT * V, cw = min(CT * V, d - c0);          // this CTA's columns: [c0, c0 + cw)

    {   // the W_r rows of these columns: cw * n consecutive elements (cw and the rows' start are multiples of V elements)
        const int nvec = cw * n * (int)sizeof(T) / 16;
        const uint4* src = (const uint4*)(W_r + (size_t)c0 * n);
        for (int q = tid; q < nvec; q += NT)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" :: "r"((uint32_t)__cvta_generic_to_shared(s_dyn4 + q)), "l"(src + q) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    }

    // ---- column sums of this CTA's rows ----
    const int ct = tid % CT, rt = tid / CT, RT = NT / CT;
    const int col = c0 + ct * V;
    float cs[V];
    {
        const int row_lo = rs * rows_per_cta;
        const int rows = min(max(0, min(l_p, Lv - j * l_p)), row_lo + rows_per_cta);      // this slice: [row_lo, rows)
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
        if (RT > 1) {                           // sum over the row threads, fixed order
#pragma unroll
            for (int v = 0; v < V; ++v) s_cs[tid * V + v] = cs[v];
            __syncthreads();
            if (rt == 0)
                for (int q = 1; q < RT; ++q)
#pragma unroll
                    for (int v = 0; v < V; ++v) cs[v] += s_cs[(q * CT + ct) * V + v];
        }
    }

    // ---- score_part[bj, part, :] = column sums . W_r rows, out of shared memory; thread (group g, expert i) strides
    //      over the CTA's columns ----
    if (rt == 0 && col < d) {
#pragma unroll
        for (int v = 0; v < V; ++v) s_cs[ct * V + v] = cs[v];       // the slot this thread itself wrote above: no one else reads it
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    {
        const int groups = NT / n;
        const int i = tid % n, g = tid / n;
        const T* s_w = (const T*)s_dyn4;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        if (g < groups) {           // four independent chains, then the tail: a fixed summation order
            int cc = g;
            for (; cc + 3 * groups < cw; cc += 4 * groups) {
                a0 = fmaf(s_cs[cc], to_f32(s_w[cc * n + i]), a0);
                a1 = fmaf(s_cs[cc + groups], to_f32(s_w[(cc + groups) * n + i]), a1);
                a2 = fmaf(s_cs[cc + 2 * groups], to_f32(s_w[(cc + 2 * groups) * n + i]), a2);
                a3 = fmaf(s_cs[cc + 3 * groups], to_f32(s_w[(cc + 3 * groups) * n + i]), a3);
            }
            for (; cc < cw; cc += groups) a0 = fmaf(s_cs[cc], to_f32(s_w[cc * n + i]), a0);
        }
        __syncthreads();
        s_cs[tid] = (a0 + a1) + (a2 + a3);
        __syncthreads();
        if (tid < n) {
            float sum = 0.f;
            for (int q = 0; q < groups; ++q) sum += s_cs[q * n + tid];
            scores[((size_t)bj * nparts + part) * n + tid] = sum;
            __threadfence();
        }
    }
    if constexpr (TICKET) {
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            s_mine = (atomicAdd(&sample_ticket[b], 1) == m * nparts - 1);
            if (s_mine) sample_ticket[b] = 0;         // left at zero for the next call
        }
        __syncthreads();
        if (!s_mine) return;
        __threadfence();
        // ---- this CTA completed sample b ----
        select_sample<NT>((float*)s_dyn4, scores, nparts, b, B, Lv, n, k, m, c, l_p, use_gate, expert_idx, patch_idx, gate, p_samp,
                          p_patch, offsets, masks, ctl + 1, plan);
    }
}

// One CTA per sample, for many samples of few small patches (image-sized inputs: a sample is a few hundred KB and
// there are at least as many samples as SMs).  The CTA's thread groups (CT column threads each) take the sample's
// patches in turn, a thread summing all rows of its 16-byte column piece, so no partial result crosses a thread; the
// pooled patches meet W_r (staged once per CTA) in shared memory and the selection follows in the same CTA: no scores
// in global memory, no ticket per sample, one launch.
constexpr int kSampleThreads = 512;

template <typename T>
__global__ void __launch_bounds__(kSampleThreads, 2)
route_sample_kernel(const T* __restrict__ x, const T* __restrict__ W_r, int B, int L, int Lv, int d, int n, int k, int m, int c,
                    int l_p, int CT, int use_gate, int* __restrict__ expert_idx, int* __restrict__ patch_idx,
                    float* __restrict__ gate, float* __restrict__ p_samp, float* __restrict__ p_patch,
                    int* __restrict__ offsets, int* __restrict__ ctl, unsigned* __restrict__ masks, const PlanPtrs plan) {
    pdl_trigger();
    pdl_wait();
    constexpr int V = Vec16<T>::N;
    constexpr int NT = kSampleThreads;
    extern __shared__ uint4 s_dyn4[];
    const int wbytes = (d * n * (int)sizeof(T) + 15) / 16 * 16;
    const T* s_w = (const T*)s_dyn4;                                          // W_r [d, n]
    float* s_pool = (float*)((char*)s_dyn4 + wbytes);                         // [m, d] column sums of every patch
    float* s_sc = s_pool + (size_t)m * d;                                     // [m, n] scores
    float* s_pp = s_sc + (size_t)m * n;                                       // [n, m] gate values (selection)
    const int tid = threadIdx.x, b = blockIdx.x;
    {
        const int nvec = d * n * (int)sizeof(T) / 16;
        const uint4* src = (const uint4*)W_r;
        for (int q = tid; q < nvec; q += NT)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" :: "r"((uint32_t)__cvta_generic_to_shared(s_dyn4 + q)), "l"(src + q) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    // ---- column sums: group g takes patches g, g + G, ... ----
    const int G = NT / CT, g = tid / CT, col = (tid % CT) * V;
    for (int j = g; j < m; j += G) {
        const int rows = max(0, min(l_p, Lv - j * l_p));
        float cs[V];
#pragma unroll
        for (int v = 0; v < V; ++v) cs[v] = 0.f;
        if (col < d) {
            const T* base = x + ((size_t)b * L + (size_t)j * l_p) * d + col;
            int r = 0;
            for (; r + 7 < rows; r += 8) {
                uint4 q[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) q[u] = ld_stream16(base + (size_t)(r + u) * d);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float f[V];
                    unpack16<T>(q[u], f);
#pragma unroll
                    for (int v = 0; v < V; ++v) cs[v] += f[v];
                }
            }
            for (; r < rows; ++r) {
                float f[V];
                unpack16<T>(ld_stream16(base + (size_t)r * d), f);
#pragma unroll
                for (int v = 0; v < V; ++v) cs[v] += f[v];
            }
#pragma unroll
            for (int v = 0; v < V; ++v) s_pool[(size_t)j * d + col + v] = cs[v];
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // ---- scores[j, i] = pooled patch j . W_r[:, i]: `parts` threads per score, columns dealt round robin, summed by a
    //      fixed shuffle tree ----
    int parts = 1;
    while (parts < 32 && 2 * parts * m * n <= NT) parts <<= 1;
    for (int p0 = 0; p0 < m * n; p0 += NT / parts) {
        const int p = p0 + tid / parts, sub = tid % parts;
        float acc = 0.f;
        if (p < m * n) {
            const int j = p / n, i = p % n;
            const float* pj = s_pool + (size_t)j * d;
            for (int cc = sub; cc < d; cc += parts) acc = fmaf(pj[cc], to_f32(s_w[cc * n + i]), acc);
        }
        for (int o = parts >> 1; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (p < m * n && sub == 0) s_sc[p] = acc;
    }
    __syncthreads();
    select_sample<NT>(s_pp, nullptr, 1, b, B, Lv, n, k, m, c, l_p, use_gate, expert_idx, patch_idx, gate, p_samp, p_patch, offsets,
                      masks, ctl + 1, plan, s_sc);
}

// Selection as a kernel of its own (after a route_kernel launch without tickets): grid B, one CTA per sample.
__global__ void __launch_bounds__(kScoreThreads)
route_select_kernel(const float* __restrict__ scores, int nparts, int B, int Lv, int n, int k, int m, int c, int l_p,
                    int use_gate, int* __restrict__ expert_idx, int* __restrict__ patch_idx, float* __restrict__ gate,
                    float* __restrict__ p_samp, float* __restrict__ p_patch, int* __restrict__ offsets,
                    int* __restrict__ ctl, unsigned* __restrict__ masks, const PlanPtrs plan) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ float s_sel[];
    select_sample<kScoreThreads>(s_sel, scores, nparts, blockIdx.x, B, Lv, n, k, m, c, l_p, use_gate, expert_idx, patch_idx, gate,
                                 p_samp, p_patch, offsets, masks, ctl + 1, plan);
}

struct RouteWs { size_t tickets, scores, total; int nchunks, CT, rsplit, rows_per_cta; size_t smem, wb; bool two_kernels, small_ctas, per_sample; size_t sample_smem; };

constexpr int kWblkBytes = 16384;       // shared memory for a CTA's rows of W_r
constexpr size_t kMaskOffset = kControlBytes / 2;      // control block: status block, sample tickets [B]; second half: expert masks [B]

RouteWs route_ws(const Dims& D) {
    const int V = 16 / D.esize;
    int CT = kScoreThreads;
    // the fewest column threads that still cover d, and few enough that their rows of W_r fit the staging block
    while (CT > 1 && ((CT / 2) * V >= D.d || (size_t)CT * V * D.n * D.esize > (size_t)kWblkBytes)) CT /= 2;
    const int nchunks = (D.d + CT * V - 1) / (CT * V);
    const int rows_per_cta = 32 * (kScoreThreads / CT);       // at most four 8-deep load batches per thread
    const int rsplit = (D.l_p + rows_per_cta - 1) / rows_per_cta;
    // The control block has a fixed size whatever the problem: status block, then the sample tickets.  Data starts
    // behind it, so no problem shape ever writes data where another shape keeps its tickets, and a scratch area
    // zeroed once serves calls of any shapes in any order.
    RouteWs r;
    r.tickets = kStatusBytes;
    WsCarver w;
    w.take(kControlBytes);
    // a second launch pays off once the first moves enough bytes that it should do nothing but stream
    r.two_kernels = nchunks * rsplit > 1 && (size_t)D.B * D.L * D.d * D.esize >= ((size_t)64 << 20);
    r.scores = w.take((size_t)D.B * D.m * nchunks * rsplit * D.n * sizeof(float));
    r.rsplit = rsplit;
    r.rows_per_cta = rows_per_cta;
    r.total = w.off;
    r.nchunks = nchunks;
    r.CT = CT;
    const size_t sel = (size_t)D.n * D.m * sizeof(float);
    r.wb = (size_t)(CT * V < D.d ? CT * V : D.d) * D.n * D.esize;
    // Many small patches (a patch is one CTA's work and a few KB): 64-thread CTAs with exactly the shared memory they
    // need, so that all of them are resident at once and the per-CTA chain (loads, dots, ticket) is paid once.
    r.small_ctas = nchunks * rsplit == 1 && D.d <= 64 * V && D.l_p <= 32 && (size_t)D.d * D.n * D.esize <= (size_t)kWblkBytes &&
                   (long long)D.B * D.m >= 1024;
    if (r.small_ctas) {
        r.CT = 64;
        r.rows_per_cta = D.l_p;
    }
    // they also hand the selection to a second launch: thousands of CTAs would otherwise each pay a fence and a ticket
    if (r.small_ctas) r.two_kernels = true;
    // ... unless a whole sample is one CTA's work (route_sample_kernel): at least one CTA per SM, patches of one column
    // chunk, at most 64 rows per thread, everything of a sample in half an SM's shared memory
    {
        int CTs = 1;
        while (CTs * V < D.d) CTs <<= 1;
        const int Gs = CTs <= kSampleThreads ? kSampleThreads / CTs : 0;
        r.sample_smem = ((size_t)D.d * D.n * D.esize + 15) / 16 * 16 + ((size_t)D.m * D.d + 2 * (size_t)D.m * D.n) * sizeof(float);
        r.per_sample = Gs >= 1 && D.B >= 128 && D.l_p <= 32 && ((D.m + Gs - 1) / Gs) * D.l_p <= 64 && r.sample_smem <= 100 * 1024 &&
                       (size_t)D.B * D.L * D.d * D.esize < ((size_t)64 << 20);
        if (r.per_sample) r.CT = CTs;
    }
    r.smem = r.two_kernels ? r.wb : (sel > r.wb ? sel : r.wb);
    return r;
}

// The launch shared by uoe_route and uoe_route_static.  `base` is the scratch (control block with the tickets, then
// the scores); its control block must have been zero when first used.
uoe_status route_launch(const Dims& D, uint32_t flags, const void* x, const void* W_r, int32_t* expert_idx,
                        int32_t* patch_idx, float* gate, float* p_samp, float* p_patch, int32_t* expert_offsets,
                        char* base, const RouteWs& W, cudaStream_t stream, bool profile, const PlanPtrs& plan = PlanPtrs()) {
    const size_t smem0 = W.smem;
    int* ctl = (int*)base;             // word 0 status (unused here), word 1 ticket
    int* tickets = (int*)(base + W.tickets);
    unsigned* masks = (unsigned*)(base + kMaskOffset);      // every sample's expert set; data, at a place no ticket ever uses
    float* scores = (float*)(base + W.scores);
    const int use_gate = ((flags & UOE_FLAG_GATE) ? 1 : 0) | ((flags & UOE_FLAG_DYNAMIC_C) ? 2 : 0) |
                         ((flags & UOE_FLAG_GENERAL_PATH) ? 4 : 0);                                       // selection flags
    dim3 grid((unsigned)(D.B * D.m * W.nchunks * W.rsplit));
#define UOE_ROUTE_ARGS(T) (const T*)x, (const T*)W_r, scores, D.B, D.L, D.Lv, D.d, D.n, D.k, D.m, D.c, D.l_p, W.CT, \
        W.nchunks, W.rsplit, W.rows_per_cta, use_gate, expert_idx, patch_idx, gate, p_samp, p_patch, expert_offsets, ctl, \
        tickets, masks, plan
#define UOE_ROUTE_LAUNCH(T, TICKET, NT, SMEM) \
        launch_k(route_kernel<T, TICKET, NT>, grid, dim3(NT), SMEM, stream, UOE_ROUTE_ARGS(T))
    cudaError_t e;
    if (W.per_sample) {
        static DeviceOnce once_bf16, once_f32;
        const uoe_status so = D.bf16 ? smem_opt_in(once_bf16, route_sample_kernel<__nv_bfloat16>, 100 * 1024)
                                     : smem_opt_in(once_f32, route_sample_kernel<float>, 100 * 1024);
        if (so != UOE_OK) return so;
        ProfScope ps(profile ? "route" : nullptr, stream);
        if (D.bf16)
            e = launch_k(route_sample_kernel<__nv_bfloat16>, dim3(D.B), dim3(kSampleThreads), W.sample_smem, stream, (const __nv_bfloat16*)x,
                         (const __nv_bfloat16*)W_r, D.B, D.L, D.Lv, D.d, D.n, D.k, D.m, D.c, D.l_p, W.CT, use_gate, expert_idx, patch_idx,
                         gate, p_samp, p_patch, expert_offsets, ctl, masks, plan);
        else
            e = launch_k(route_sample_kernel<float>, dim3(D.B), dim3(kSampleThreads), W.sample_smem, stream, (const float*)x,
                         (const float*)W_r, D.B, D.L, D.Lv, D.d, D.n, D.k, D.m, D.c, D.l_p, W.CT, use_gate, expert_idx, patch_idx,
                         gate, p_samp, p_patch, expert_offsets, ctl, masks, plan);
        if (e != cudaSuccess) return UOE_ERR_CUDA;
        UOE_LAUNCHED();
        return UOE_OK;
    }
    {
        ProfScope ps(profile ? "route" : nullptr, stream);
        if (W.small_ctas) e = D.bf16 ? UOE_ROUTE_LAUNCH(__nv_bfloat16, false, 64, W.smem) : UOE_ROUTE_LAUNCH(float, false, 64, W.smem);
        else if (W.two_kernels) e = D.bf16 ? UOE_ROUTE_LAUNCH(__nv_bfloat16, false, kScoreThreads, W.smem) : UOE_ROUTE_LAUNCH(float, false, kScoreThreads, W.smem);
        else e = D.bf16 ? UOE_ROUTE_LAUNCH(__nv_bfloat16, true, kScoreThreads, smem0) : UOE_ROUTE_LAUNCH(float, true, kScoreThreads, smem0);
    }
#undef UOE_ROUTE_LAUNCH
#undef UOE_ROUTE_ARGS
    if (e != cudaSuccess) return UOE_ERR_CUDA;
    UOE_LAUNCHED();
    if (!W.two_kernels) return UOE_OK;
    {
        ProfScope ps(profile ? "route_select" : nullptr, stream);
        const size_t sel = (size_t)D.n * D.m * sizeof(float);
        e = launch_k(route_select_kernel, dim3(D.B), dim3(kScoreThreads), sel, stream, (const float*)scores, W.nchunks * W.rsplit,
                     D.B, D.Lv, D.n, D.k, D.m, D.c, D.l_p, use_gate, expert_idx, patch_idx, gate, p_samp, p_patch,
                     expert_offsets, ctl, masks, plan);
    }
    if (e != cudaSuccess) return UOE_ERR_CUDA;
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
    if ((size_t)D.n * D.m * sizeof(float) > 36 * 1024) return UOE_ERR_UNSUPPORTED;   // gate values of a sample in shared memory
    W = route_ws(D);
    if ((long long)D.B * D.m * W.nchunks * W.rsplit > 0x7fffffffll) return UOE_ERR_UNSUPPORTED;
    if (W.tickets + (size_t)D.B * sizeof(int) > kMaskOffset) return UOE_ERR_UNSUPPORTED;   // tickets and expert masks must fit the control block
    return UOE_OK;
}

}  // namespace

size_t route_workspace_bytes(const Dims& D) { return route_ws(D).total; }

bool route_can_plan(const Dims&) { return true; }

uoe_status route_run(const uoe_problem* prob, const void* x, const void* W_r, const RoutingPtrs& r, char* scratch,
                     cudaStream_t stream, const PlanPtrs* plan) {
    Dims D;
    RouteWs W;
    uoe_status st = route_check(prob, D, W, x, W_r, r.expert_idx, r.patch_idx, r.gate, r.p_samp, r.p_patch, r.expert_offsets);
    if (st != UOE_OK) return st;
    if (plan && !route_can_plan(D)) return UOE_ERR_UNSUPPORTED;
    return route_launch(D, prob->flags, x, W_r, r.expert_idx, r.patch_idx, r.gate, r.p_samp, r.p_patch, r.expert_offsets, scratch,
                        W, stream, true, plan ? *plan : PlanPtrs());
}

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
// uoe_route_balance: Eq. 15-16 and 42-44 from the patch gate that uoe_route wrote
// ------------------------------------------------------------------------------------------------
namespace uoe {
namespace {
// grid B, 128 threads, dynamic shared memory n*m floats.
__global__ void __launch_bounds__(128)
balance_kernel(const float* __restrict__ p_patch, int Lv, int n, int k, int m, int l_p, float alpha,
               float* __restrict__ lb_loss, int* __restrict__ expert_count, int* __restrict__ c_dyn) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ float pp[];          // [n][m]
    __shared__ int cnts[32];
    __shared__ float Pm[32];
    const int b = blockIdx.x, tid = threadIdx.x;
    const int n_elig = (Lv + l_p - 1) / l_p;       // patches holding at least one real token (a prefix)
    for (int idx = tid; idx < n * m; idx += 128) pp[idx] = p_patch[(size_t)b * n * m + idx];
    if (tid < 32) cnts[tid] = 0;
    __syncthreads();
    for (int j = tid; j < n_elig; j += 128) {      // Eq. 15: patch j goes to its k best experts (ties: lower index)
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
    if (tid < n) {                                  // Eq. 44: mean gate of expert i over the real patches, fixed order
        float s = 0.f;
        for (int j = 0; j < n_elig; ++j) s += pp[tid * m + j];
        Pm[tid] = s / (float)n_elig;
    }
    __syncthreads();
    if (tid < n && expert_count) expert_count[(size_t)b * n + tid] = cnts[tid];
    if (tid == 0) {
        int cmax = 0;
        float loss = 0.f;
        const float fs = (float)n / ((float)k * (float)n_elig);                       // Eq. 43
        for (int i = 0; i < n; ++i) { cmax = max(cmax, cnts[i]); loss += fs * (float)cnts[i] * Pm[i]; }
        if (c_dyn) c_dyn[b] = cmax;                                                     // Eq. 16
        if (lb_loss) lb_loss[b] = alpha * loss;                                         // Eq. 42
    }
}
}  // namespace
}  // namespace uoe

extern "C" uoe_status uoe_route_balance(const uoe_problem* prob, const float* p_patch, float alpha, float* lb_loss,
                                        int32_t* expert_count, int32_t* c_dyn, void* cuda_stream) {
    Dims D;
    uoe_status st = make_dims(prob, D);
    if (st != UOE_OK) return st;
    if (!p_patch || (!lb_loss && !expert_count && !c_dyn)) return UOE_ERR_INVALID_ARG;
    const size_t smem = (size_t)D.n * D.m * sizeof(float);
    if (smem > 36 * 1024) return UOE_ERR_UNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaError_t e;
    {
        ProfScope ps("route_balance", stream);
        e = launch_k(balance_kernel, dim3(D.B), dim3(128), smem, stream, p_patch, D.Lv, D.n, D.k, D.m, D.l_p, alpha, lb_loss,
                     expert_count, c_dyn);
    }
    if (e != cudaSuccess) return UOE_ERR_CUDA;
    UOE_LAUNCHED();
    return UOE_OK;
}

// ------------------------------------------------------------------------------------------------
// uoe_route_static: the same kernel with its scratch in a built-in device array
// ------------------------------------------------------------------------------------------------

// Scratch of uoe_route_static: the control block (tickets, expert loads) followed by the scores and the pooled
// column sums.  One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_route_static_scratch[UOE_ROUTE_STATIC_SCRATCH_BYTES];

namespace {
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
