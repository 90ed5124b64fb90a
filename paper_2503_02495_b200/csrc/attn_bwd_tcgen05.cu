// Backward of the selective multi-head attention core (derivative of Eq. 33-34 with the masks of Eq. 41 and
// Fig. 4).  For every (sample, chosen expert) pair and head, with P = softmax(q k^T / sqrt(d_h) + mask),
// o = P v and the upstream gradient do:
//   dv = P^T do,   dP = do v^T,   dS = P * (dP - delta) / sqrt(d_h)  with  delta_r = sum_c do[r,c] o[r,c],
//   dq = dS k,     dk = dS^T q.
// P is rebuilt from q, k and the saved log-sum-exp of each query row, so nothing of size l_a x l_a is stored.
//
// Two launches of one kernel template, each CTA owning one 128-row output tile, so that every output element
// is accumulated by a single CTA in a fixed order (no atomics):
//   DQ = false  CTA = (key tile j, head, pair): K_j, V_j stay in shared memory, the query tiles stream through;
//               dV_j += P^T dO_i and dK_j += dS^T Q_i accumulate in TMEM over i
//   DQ = true   CTA = (query tile i, head, pair): Q_i, dO_i stay, the key tiles stream; dQ_i += dS K_j
// Per streamed tile:  S = Q K^T and dP = dO V^T (tcgen05.mma 128x128x64 each, accumulators in TMEM), then two
// threads per query row (TMEM lane = row; warps 0-3 take keys 0-63 of the tile, warps 4-7 keys 64-127) form P and
// dS in 32-column pieces, round them to bf16 and write them to shared memory in the 128B-swizzled layout, where they are the A operands of the second MMAs (read
// K-major for dQ, MN-major, i.e. transposed, for dV / dK).
// Masks as in the forward kernel: key c is kept iff c < n_valid (real keys are a prefix of the gathered order)
// and, with the causal flag, c <= query row; query rows >= l_a of a tile belong to the next pair and are dropped.
#include "kernels.cuh"
#include "tc.cuh"
#include "tmap.cuh"

namespace uoe {
namespace {

using namespace tc;

constexpr int T = 128, DH = 64;
constexpr int kThreads = 256;
constexpr int TILE_BYTES = T * DH * 2;            // 16 KB: a [128 x 64] bf16 tile
constexpr int SQ_BYTES = 2 * TILE_BYTES;          // a [128 x 128] bf16 matrix as two swizzled halves

template <bool DQ> struct BCfg {
    // fixed pair of tiles, two stages of streamed pairs, dS (and P for the dK/dV pass)
    static constexpr int SMEM = 2 * TILE_BYTES + 4 * TILE_BYTES + (DQ ? 1 : 2) * SQ_BYTES + 1024 + 256;
};

struct BCtl {
    uint64_t bar_fix, bar_ld[2], bar_s, bar_o;
    uint32_t tmem_base;
    int abort_flag;
};

template <bool DQ>
__global__ void __launch_bounds__(kThreads)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO,
                __nv_bfloat16* __restrict__ out0 /* DQ: dq; else dk */, __nv_bfloat16* __restrict__ out1 /* dv */,
                int ld_out /* elements per row of the output buffers */, const float* __restrict__ lse,
                const float* __restrict__ delta, const int* __restrict__ pair_row, const int* __restrict__ patch_idx,
                int c, int l_p, int Lv, int l_a, int heads, int causal, float scale_log2, float inv_sqrt_dh,
                int* status) {
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sF0 = smem;                           // fixed: DQ ? Q_i : K_j
    uint8_t* sF1 = sF0 + TILE_BYTES;               // fixed: DQ ? dO_i : V_j
    uint8_t* sS0 = sF1 + TILE_BYTES;               // streamed, 2 stages: DQ ? K_j : Q_i
    uint8_t* sS1 = sS0 + 2 * TILE_BYTES;           // streamed, 2 stages: DQ ? V_j : dO_i
    uint8_t* sDS = sS1 + 2 * TILE_BYTES;           // dS [q][keys]
    uint8_t* sP = sDS + SQ_BYTES;                  // P  [q][keys] (dK/dV pass only)
    BCtl* ctl = (BCtl*)(sDS + (DQ ? 1 : 2) * SQ_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;
    __shared__ int s_nvalid;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, head = blockIdx.y, pair = blockIdx.z;

    if (warp == 0) tmem_alloc(&ctl->tmem_base, 512);       // S [0,128), dP [128,256), accumulators [256,384)
    pdl_wait();
    const int row_base = pair_row[pair];
    if (tid == 0) {
        mbar_init(&ctl->bar_fix, 1);
        mbar_init(&ctl->bar_ld[0], 1);
        mbar_init(&ctl->bar_ld[1], 1);
        mbar_init(&ctl->bar_s, 1);
        mbar_init(&ctl->bar_o, 1);
        ctl->abort_flag = 0;
        fence_barrier_init();
        int nv = 0;
        for (int u = 0; u < c; ++u) {
            const int j = patch_idx[(size_t)pair * c + u];
            if (j >= 0) nv += max(0, min(l_p, Lv - j * l_p));
        }
        s_nvalid = nv;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int n_valid = s_nvalid;
    const int kv_end = min(n_valid, l_a);
    const int n_q = (l_a + T - 1) / T, n_kv = (kv_end + T - 1) / T;
    const int col_h = head * DH;

    // streamed tiles [first, last]
    int first, last;
    if (DQ) { first = 0; last = causal ? min(tile, n_kv - 1) : n_kv - 1; }
    else { first = causal ? tile : 0; last = (tile < n_kv) ? n_q - 1 : -1; }
    const int n_it = last - first + 1;             // may be <= 0: nothing to accumulate, the tile's output is zero

    const CUtensorMap* tmS0 = DQ ? &tmK : &tmQ;
    const CUtensorMap* tmS1 = DQ ? &tmV : &tmDO;
    if (tid == 0 && n_it > 0) {
        mbar_arrive_expect_tx(&ctl->bar_fix, 2 * TILE_BYTES);
        tma_load_2d(sF0, DQ ? &tmQ : &tmK, col_h, row_base + tile * T, &ctl->bar_fix);
        tma_load_2d(sF1, DQ ? &tmDO : &tmV, col_h, row_base + tile * T, &ctl->bar_fix);
        for (int t = 0; t < 2 && t < n_it; ++t) {
            mbar_arrive_expect_tx(&ctl->bar_ld[t], 2 * TILE_BYTES);
            tma_load_2d(sS0 + t * TILE_BYTES, tmS0, col_h, row_base + (first + t) * T, &ctl->bar_ld[t]);
            tma_load_2d(sS1 + t * TILE_BYTES, tmS1, col_h, row_base + (first + t) * T, &ctl->bar_ld[t]);
        }
    }

    constexpr uint32_t idesc_s = instr_desc_bf16(T, T, false, false);        // S, dP: both operands K-major
    constexpr uint32_t idesc_q = instr_desc_bf16(T, DH, false, true);        // dQ = dS K: A K-major, B MN-major
    constexpr uint32_t idesc_t = instr_desc_bf16(T, DH, true, true);         // dV = P^T dO, dK = dS^T Q: both MN-major
    const int quarter = warp & 3, hsel = warp >> 2;                          // TMEM lane quarter; half of the keys / channels
    const int trow = quarter * 32 + lane;                                    // TMEM lane = row inside the tile
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    bool ok = true;

    float my_lse2 = 0.f, my_delta = 0.f;
    if (DQ) {
        const int qrow = tile * T + trow;
        if (qrow < l_a) {
            my_lse2 = lse[(size_t)(row_base + qrow) * heads + head] * 1.4426950408889634f;
            my_delta = delta[(size_t)(row_base + qrow) * heads + head];
        }
    }

    for (int it = 0; it < n_it; ++it) {
        const int st = it & 1, cur = first + it;
        const int q_tile = DQ ? tile : cur, k_tile = DQ ? cur : tile;
        // ---- S = Q K^T, dP = dO V^T ----
        if (tid == 0) {
            if (it == 0) ok = mbar_wait(&ctl->bar_fix, 0, abort_flag, status);
            ok = mbar_wait(&ctl->bar_ld[st], (it >> 1) & 1, abort_flag, status) && ok;
            tc_fence_after();
            const uint32_t f0 = smem_u32(sF0), f1 = smem_u32(sF1);
            const uint32_t s0 = smem_u32(sS0 + st * TILE_BYTES), s1 = smem_u32(sS1 + st * TILE_BYTES);
            const uint32_t qa = DQ ? f0 : s0, ka = DQ ? s0 : f0, doa = DQ ? f1 : s1, va = DQ ? s1 : f1;
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
                mma_bf16(tmem_base, smem_desc(qa + ks * 32, 16, 1024), smem_desc(ka + ks * 32, 16, 1024), idesc_s, ks != 0);
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
                mma_bf16(tmem_base + 128, smem_desc(doa + ks * 32, 16, 1024), smem_desc(va + ks * 32, 16, 1024), idesc_s, ks != 0);
            mma_commit(&ctl->bar_s);
        }
        ok = mbar_wait(&ctl->bar_s, it & 1, abort_flag, status);
        if (!__all_sync(0xffffffffu, ok && !*abort_flag)) break;
        tc_fence_after();
        // every MMA issued before this commit has completed, the previous iteration's second group included:
        // its stage and the P / dS buffers are free again
        if (tid == 0 && it >= 1 && it + 1 < n_it) {
            const int ns = (it + 1) & 1;
            mbar_arrive_expect_tx(&ctl->bar_ld[ns], 2 * TILE_BYTES);
            tma_load_2d(sS0 + ns * TILE_BYTES, tmS0, col_h, row_base + (cur + 1) * T, &ctl->bar_ld[ns]);
            tma_load_2d(sS1 + ns * TILE_BYTES, tmS1, col_h, row_base + (cur + 1) * T, &ctl->bar_ld[ns]);
        }

        // ---- P and dS for this thread's query row ----
        const int qrow = q_tile * T + trow;
        if (!DQ) {
            my_lse2 = 0.f; my_delta = 0.f;
            if (qrow < l_a) {
                my_lse2 = lse[(size_t)(row_base + qrow) * heads + head] * 1.4426950408889634f;
                my_delta = delta[(size_t)(row_base + qrow) * heads + head];
            }
        }
        const int kv0 = k_tile * T;
        const int keep_cols = (qrow < l_a ? min(kv_end, causal ? qrow + 1 : kv_end) : 0) - kv0;     // kept columns of this key tile
        const int sw = trow & 7;
#pragma unroll 1
        for (int ch = 2 * hsel; ch < 2 * hsel + 2; ++ch) {
            float s_v[32], dp_v[32];
            tmem_ld32(t_lane + ch * 32, (uint32_t*)s_v);
            tmem_ld32(t_lane + 128 + ch * 32, (uint32_t*)dp_v);
            tmem_ld_wait();
            // (one limit per row covers the three masks -- rows past the pair, keys past the real ones, the causal
            // triangle --: tested clause by clause per element the test becomes branches per element)
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const bool keep = ch * 32 + j < keep_cols;
                const float p = keep ? ex2_approx(fmaf(s_v[j], scale_log2, -my_lse2)) : 0.f;
                s_v[j] = p;
                dp_v[j] = keep ? p * (dp_v[j] - my_delta) * inv_sqrt_dh : 0.f;
            }
            const int half = ch >> 1;                       // 64-key half of the [128 x 128] matrix
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {                // 16-byte pieces of 8 bf16
                const int cc = (ch & 1) * 4 + q8;
                uint4 w;
                w.x = pack_bf16x2(dp_v[q8 * 8 + 0], dp_v[q8 * 8 + 1]); w.y = pack_bf16x2(dp_v[q8 * 8 + 2], dp_v[q8 * 8 + 3]);
                w.z = pack_bf16x2(dp_v[q8 * 8 + 4], dp_v[q8 * 8 + 5]); w.w = pack_bf16x2(dp_v[q8 * 8 + 6], dp_v[q8 * 8 + 7]);
                *(uint4*)(sDS + half * TILE_BYTES + trow * 128 + ((cc ^ sw) << 4)) = w;
                if (!DQ) {
                    w.x = pack_bf16x2(s_v[q8 * 8 + 0], s_v[q8 * 8 + 1]); w.y = pack_bf16x2(s_v[q8 * 8 + 2], s_v[q8 * 8 + 3]);
                    w.z = pack_bf16x2(s_v[q8 * 8 + 4], s_v[q8 * 8 + 5]); w.w = pack_bf16x2(s_v[q8 * 8 + 6], s_v[q8 * 8 + 7]);
                    *(uint4*)(sP + half * TILE_BYTES + trow * 128 + ((cc ^ sw) << 4)) = w;
                }
            }
        }
        fence_async_smem();                  // generic-proxy writes of P / dS -> visible to the tensor core
        tc_fence_before();
        __syncthreads();

        // ---- accumulate: dQ += dS K   |   dV += P^T dO, dK += dS^T Q ----
        if (tid == 0) {
            tc_fence_after();
            const uint32_t ds = smem_u32(sDS);
            const uint32_t s0 = smem_u32(sS0 + st * TILE_BYTES), s1 = smem_u32(sS1 + st * TILE_BYTES);
            if (DQ) {
#pragma unroll
                for (int ks = 0; ks < T / 16; ++ks)
                    mma_bf16(tmem_base + 256, smem_desc(ds + (ks >> 2) * TILE_BYTES + (ks & 3) * 32, 16, 1024),
                             smem_desc(s0 + ks * 2048, 8192, 1024), idesc_q, (it | ks) != 0);
            } else {
                const uint32_t pp = smem_u32(sP);
#pragma unroll
                for (int ks = 0; ks < T / 16; ++ks)       // contraction over the 128 query rows, 16 per step
                    mma_bf16(tmem_base + 320, smem_desc(pp + ks * 2048, TILE_BYTES, 1024),
                             smem_desc(s1 + ks * 2048, 8192, 1024), idesc_t, (it | ks) != 0);
#pragma unroll
                for (int ks = 0; ks < T / 16; ++ks)
                    mma_bf16(tmem_base + 256, smem_desc(ds + ks * 2048, TILE_BYTES, 1024),
                             smem_desc(s0 + ks * 2048, 8192, 1024), idesc_t, (it | ks) != 0);
            }
            if (it == n_it - 1) mma_commit(&ctl->bar_o);
        }
    }

    // ---- write the tile's rows: bf16, zero where nothing was accumulated ----
    bool have = n_it > 0 && ok && !*abort_flag;
    if (n_it > 0) {
        const bool done = mbar_wait(&ctl->bar_o, 0, abort_flag, status) && !*abort_flag;
        have = __all_sync(0xffffffffu, have && done);
        tc_fence_after();
    }
    const int orow = tile * T + trow;
    {
        float acc[DH / 2];                                   // this thread's 32 of the row's 64 channels
#pragma unroll 1
        for (int which = 0; which < (DQ ? 1 : 2); ++which) {
            if (have) {                                      // warp-uniform
                tmem_ld32(t_lane + 256 + which * 64 + hsel * 32, (uint32_t*)acc);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int i = 0; i < DH / 2; ++i) acc[i] = 0.f;
            }
            if (orow < l_a) {
                __nv_bfloat16* out = (which == 0 ? out0 : out1) + (size_t)(row_base + orow) * ld_out + col_h + hsel * 32;
#pragma unroll
                for (int ch = 0; ch < DH / 16; ++ch) {
                    uint4 w;
                    w.x = pack_bf16x2(acc[ch * 8 + 0], acc[ch * 8 + 1]); w.y = pack_bf16x2(acc[ch * 8 + 2], acc[ch * 8 + 3]);
                    w.z = pack_bf16x2(acc[ch * 8 + 4], acc[ch * 8 + 5]); w.w = pack_bf16x2(acc[ch * 8 + 6], acc[ch * 8 + 7]);
                    ((uint4*)out)[ch] = w;
                }
            }
        }
    }
    if (tid == 0 && *abort_flag && n_it > 0) {           // let copies that may still be in flight land (bounded)
        mbar_wait(&ctl->bar_fix, 0, abort_flag, status);
        for (int t = 0; t < 2 && t < n_it; ++t) mbar_try_wait(&ctl->bar_ld[t], 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

// q, k, v, dout: [rows_max, d_g] bf16 routed buffers; dq, dk, dv: bf16 with ld_out elements per row;
// lse, delta: [rows_max, heads] float32 (lse as written by the forward kernel, natural logarithm).
uoe_status launch_attention_backward(const Dims& D, const void* q, const void* k, const void* v, const void* dout,
                                     const float* lse, const float* delta, void* dq, void* dk, void* dv, int ld_out,
                                     const int* pair_row, const int* patch_idx, bool causal, int* status,
                                     cudaStream_t s) {
    if (D.d_h != DH) return UOE_ERR_UNSUPPORTED;
    static DeviceOnce once_kv, once_q;
    {
        uoe_status st = smem_opt_in(once_kv, attn_bwd_kernel<false>, BCfg<false>::SMEM);
        if (st == UOE_OK) st = smem_opt_in(once_q, attn_bwd_kernel<true>, BCfg<true>::SMEM);
        if (st != UOE_OK) return st;
    }
    if ((long long)D.B * D.k > 65535) return UOE_ERR_UNSUPPORTED;      // pairs ride on grid.z
    CUtensorMap tm[4];
    const void* ptrs[4] = {q, k, v, dout};
    for (int i = 0; i < 4; ++i) {
        const uint64_t dims[2] = {(uint64_t)D.d_g, (uint64_t)D.Rmax};
        const uint64_t str[1] = {(uint64_t)D.d_g * 2};
        const uint32_t box[2] = {DH, 128};
        if (!make_tmap(&tm[i], ptrs[i], 2, dims, str, box)) return UOE_ERR_CUDA;
    }
    const int heads = D.d_g / DH;
    dim3 grid((D.l_a + T - 1) / T, heads, D.B * D.k);
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)D.d_h);
    const float inv_sqrt_dh = 1.0f / sqrtf((float)D.d_h);
    {
        ProfScope ps("attn_bwd_dkdv", s);
        launch_k(attn_bwd_kernel<false>, grid, dim3(kThreads), BCfg<false>::SMEM, s, tm[0], tm[1], tm[2], tm[3],
                 (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, ld_out, lse, delta, pair_row, patch_idx, D.c, D.l_p, D.Lv, D.l_a,
                 heads, causal ? 1 : 0, scale_log2, inv_sqrt_dh, status);
    }
    UOE_LAUNCHED();
    {
        ProfScope ps("attn_bwd_dq", s);
        launch_k(attn_bwd_kernel<true>, grid, dim3(kThreads), BCfg<true>::SMEM, s, tm[0], tm[1], tm[2], tm[3],
                 (__nv_bfloat16*)dq, (__nv_bfloat16*)nullptr, ld_out, lse, delta, pair_row, patch_idx, D.c, D.l_p, D.Lv,
                 D.l_a, heads, causal ? 1 : 0, scale_log2, inv_sqrt_dh, status);
    }
    UOE_LAUNCHED();
    return UOE_OK;
}

}  // namespace uoe
