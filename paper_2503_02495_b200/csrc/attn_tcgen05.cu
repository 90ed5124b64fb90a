// Selective multi-head attention core (Eq. 33-34 with the masks of Eq. 41 and Fig. 4): for every
// (sample, chosen expert) pair and every head of that expert, softmax(q k^T / sqrt(d_h) + mask) v over
// the pair's l_a gathered tokens.
//
// One CTA per (128-query tile, head, pair).  q, k, v are rows of the routed buffers [rows, d_g] (bf16),
// so the pair's tokens are contiguous.  Per 128-key tile:
//   S = Q K^T      tcgen05.mma 128x128x64, both operands K-major from TMA, accumulator in TMEM
//   softmax        two threads per query row (TMEM lane = row; warps 0-3 take keys 0-63 of the tile, warps 4-7
//                  keys 64-127): tile maxima exchanged through shared memory, running max in both threads,
//                  each keeps the sum of its own half; P rounded to bf16 and written to shared memory in the
//                  128B-swizzled K-major layout (each thread's half is one [128 x 64] operand tile)
//   O_t = P V      tcgen05.mma 128x64x128, V as the MN-major operand, fresh TMEM accumulator,
//                  then O = alpha * O + O_t in registers, 32 of the 64 channels per thread; S of the next key
//                  tile is issued right behind P V into a second TMEM buffer, so it runs under this update
// Masks: the real keys of a pair are a prefix of its gathered order (patches ascending, pad tokens at
// the end of the sample), so key c is kept iff c < n_valid, and with the causal flag iff also
// c <= query row (the shared lower triangle of Fig. 4).
#include "kernels.cuh"
#include "tc.cuh"
#include "tmap.cuh"

namespace uoe {
namespace {

using namespace tc;

constexpr int TQ = 128, TK = 128, DH = 64;
constexpr int kAttnThreads = 256;
constexpr int TILE_BYTES = 128 * DH * 2;          // 16 KB: a [128 x 64] bf16 tile
constexpr int ATTN_SMEM = TILE_BYTES * (1 + 2 + 2 + 2) + 1024 + 256;
constexpr int kFuseMaxD = 512;                               // fused output projection: z tile [128 x d] fp32 fills TMEM
constexpr int ATTN_SMEM_FUSED = ATTN_SMEM + 1024 + kFuseMaxD * DH * 2;      // + the expert's W^o slice [64 x d] behind the control block

struct AttnCtl {
    uint64_t bar_q, bar_kv[2], bar_s, bar_o, bar_w, bar_z;
    uint32_t tmem_base;
    int abort_flag;
};

// FUSE_O (one head per expert, d <= 512): the output projection of Eq. 35 runs in the same CTA.  The expert's W^o
// slice [64 x d] is fetched by TMA at kernel start; after the last key tile the normalised o tile goes to shared
// memory (bf16, swizzled, in place of Q), z = o W^o_i [128 x d] is accumulated over the whole of TMEM (S and O_t are
// no longer needed) and written to Z instead of o to O.
template <bool FUSE_O>
__global__ void __launch_bounds__(kAttnThreads)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
            const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
            const int* __restrict__ pair_row, const int* __restrict__ patch_idx, int c, int l_p, int Lv, int l_a,
            int d_g, int heads, int causal, float scale_log2, int* status,
            const __grid_constant__ CUtensorMap tmWo, const int* __restrict__ expert_idx, __nv_bfloat16* __restrict__ Z,
            int d) {
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + TILE_BYTES;                 // 2 stages
    uint8_t* sV = sK + 2 * TILE_BYTES;             // 2 stages
    uint8_t* sP = sV + 2 * TILE_BYTES;             // [128 x 128] bf16 as two [128 x 64] swizzled halves
    AttnCtl* ctl = (AttnCtl*)(sP + 2 * TILE_BYTES);
    uint8_t* sW = sP + 2 * TILE_BYTES + 1024;       // FUSE_O: W^o slice as d/64 boxes of [64 x 64], 8 KB each
    volatile int* abort_flag = &ctl->abort_flag;
    __shared__ int s_nvalid;
    __shared__ float s_xch[2][TQ];               // per row: the two half-tile maxima, later the two half sums

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int qt = blockIdx.x, head = blockIdx.y, pair = blockIdx.z;
    const int q0 = qt * TQ;

    if (warp == 0) tmem_alloc(&ctl->tmem_base, 512);       // S: two buffers, columns [0,128) and [128,256); O_t: [256,320)
    pdl_wait();                                             // from here on: data written by earlier kernels
    const int row_base = pair_row[pair];
    if (tid == 0) {
        mbar_init(&ctl->bar_q, 1);
        mbar_init(&ctl->bar_kv[0], 1);
        mbar_init(&ctl->bar_kv[1], 1);
        mbar_init(&ctl->bar_s, 1);
        mbar_init(&ctl->bar_o, 1);
        mbar_init(&ctl->bar_w, 1);
        mbar_init(&ctl->bar_z, 1);
        ctl->abort_flag = 0;
        fence_barrier_init();
        // real keys of this pair: sum over its slots of the real tokens in the slot's patch
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

    int kv_end = min(n_valid, l_a);
    if (causal) kv_end = min(kv_end, q0 + TQ);
    const int n_kv = (kv_end + TK - 1) / TK;               // >= 1: every pair holds a real token
    const int col_h = head * DH;

    if (tid == 0) {
        mbar_arrive_expect_tx(&ctl->bar_q, TILE_BYTES);
        tma_load_2d(sQ, &tmQ, col_h, row_base + q0, &ctl->bar_q);
        for (int t = 0; t < 2 && t < n_kv; ++t) {
            mbar_arrive_expect_tx(&ctl->bar_kv[t], 2 * TILE_BYTES);
            tma_load_2d(sK + t * TILE_BYTES, &tmK, col_h, row_base + t * TK, &ctl->bar_kv[t]);
            tma_load_2d(sV + t * TILE_BYTES, &tmV, col_h, row_base + t * TK, &ctl->bar_kv[t]);
        }
        if (FUSE_O) {                        // the expert's W^o slice, needed only after the last key tile
            const int e = expert_idx[pair];
            mbar_arrive_expect_tx(&ctl->bar_w, (uint32_t)d * DH * 2);
            for (int nb = 0; nb < d / 64; ++nb) tma_load_3d(sW + nb * 8192, &tmWo, nb * 64, 0, e, &ctl->bar_w);
        }
    }

    constexpr uint32_t idesc_s = instr_desc_bf16(TQ, TK, false, false);
    constexpr uint32_t idesc_o = instr_desc_bf16(TQ, DH, false, true);
    const int quarter = warp & 3, hsel = warp >> 2;        // TMEM lane quarter of this warp; which half of the keys / channels
    const int trow = quarter * 32 + lane;                  // row of the tile (TMEM lane)
    const int qrow = q0 + trow;                            // query index inside the pair
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    constexpr int HK = TK / 2, HD = DH / 2;

    float o_acc[HD];
#pragma unroll
    for (int i = 0; i < HD; ++i) o_acc[i] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;                  // l_run: sum over this thread's half of the keys
    bool ok = true;

    for (int it = 0; it < n_kv; ++it) {
        const int st = it & 1;
        // ---- S = Q K^T (issued here for the first tile only; later tiles are issued behind the previous P V) ----
        if (tid == 0 && it == 0) {
            ok = mbar_wait(&ctl->bar_q, 0, abort_flag, status);
            ok = mbar_wait(&ctl->bar_kv[0], 0, abort_flag, status) && ok;
            tc_fence_after();
            const uint32_t qa = smem_u32(sQ), ka = smem_u32(sK);
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
                mma_bf16(tmem_base, smem_desc(qa + ks * 32, 16, 1024), smem_desc(ka + ks * 32, 16, 1024), idesc_s, ks != 0);
            mma_commit(&ctl->bar_s);
        }
        ok = mbar_wait(&ctl->bar_s, it & 1, abort_flag, status);
        if (!__all_sync(0xffffffffu, ok && !*abort_flag)) break;
        tc_fence_after();

        // ---- online softmax for this row ----
        const int kv0 = it * TK + hsel * HK;
        float s_row[HK];
#pragma unroll
        for (int ch = 0; ch < HK / 32; ++ch)
            tmem_ld32(t_lane + (it & 1) * 128 + hsel * HK + ch * 32, (uint32_t*)(s_row + ch * 32));
        tmem_ld_wait();
        float m_new = m_run;
#pragma unroll
        for (int j = 0; j < HK; ++j) {
            const int col = kv0 + j;
            const bool keep = col < n_valid && col < l_a && (!causal || col <= qrow);
            s_row[j] = keep ? s_row[j] * scale_log2 : -INFINITY;
            m_new = fmaxf(m_new, s_row[j]);
        }
        s_xch[hsel][trow] = m_new;            // read by the row's other thread; rewritten only after the next barrier
        __syncthreads();
        m_new = fmaxf(m_new, s_xch[hsel ^ 1][trow]);
        // a row with no kept key so far keeps m = -inf; exp2(-inf - (-inf)) is avoided by the guard
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = exp2f(m_run - m_use);
        float l_add = 0.f;
        uint8_t* prow = sP + hsel * TILE_BYTES + (size_t)trow * 128;
        const int sw = trow & 7;
#pragma unroll
        for (int ch = 0; ch < HK / 8; ++ch) {                 // 16-byte chunks of 8 bf16
            float p[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) { p[q] = exp2f(s_row[ch * 8 + q] - m_use); l_add += p[q]; }
            uint4 w;
            w.x = pack_bf16x2(p[0], p[1]); w.y = pack_bf16x2(p[2], p[3]);
            w.z = pack_bf16x2(p[4], p[5]); w.w = pack_bf16x2(p[6], p[7]);
            *(uint4*)(prow + ((ch ^ sw) << 4)) = w;
        }
        l_run = l_run * alpha + l_add;
        m_run = m_new;
        fence_async_smem();                  // generic-proxy writes of P -> visible to the tensor core
        tc_fence_before();
        __syncthreads();

        // ---- O_t = P V, and behind it S of the next tile into the other S buffer (it runs under the O update) ----
        if (tid == 0) {
            tc_fence_after();
            const uint32_t pa = smem_u32(sP), va = smem_u32(sV + st * TILE_BYTES);
#pragma unroll
            for (int ks = 0; ks < TK / 16; ++ks)
                mma_bf16(tmem_base + 256, smem_desc(pa + (ks >> 2) * TILE_BYTES + (ks & 3) * 32, 16, 1024),
                         smem_desc(va + ks * 2048, 8192, 1024), idesc_o, ks != 0);
            mma_commit(&ctl->bar_o);
            if (it + 1 < n_kv) {
                const int ns = (it + 1) & 1;
                ok = mbar_wait(&ctl->bar_kv[ns], ((it + 1) >> 1) & 1, abort_flag, status) && ok;
                tc_fence_after();
                const uint32_t qa = smem_u32(sQ), ka = smem_u32(sK + ns * TILE_BYTES);
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks)
                    mma_bf16(tmem_base + ns * 128, smem_desc(qa + ks * 32, 16, 1024), smem_desc(ka + ks * 32, 16, 1024), idesc_s,
                             ks != 0);
                mma_commit(&ctl->bar_s);
            }
        }
        ok = mbar_wait(&ctl->bar_o, it & 1, abort_flag, status);
        if (!__all_sync(0xffffffffu, ok && !*abort_flag)) break;
        tc_fence_after();
        if (tid == 0 && it + 2 < n_kv) {     // both MMAs that read this stage are done: refill it
            mbar_arrive_expect_tx(&ctl->bar_kv[st], 2 * TILE_BYTES);
            tma_load_2d(sK + st * TILE_BYTES, &tmK, col_h, row_base + (it + 2) * TK, &ctl->bar_kv[st]);
            tma_load_2d(sV + st * TILE_BYTES, &tmV, col_h, row_base + (it + 2) * TK, &ctl->bar_kv[st]);
        }
        {
            float o_t[HD];
            tmem_ld32(t_lane + 256 + hsel * HD, (uint32_t*)o_t);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < HD; ++i) o_acc[i] = o_acc[i] * alpha + o_t[i];
        }
        tc_fence_before();                   // S and O_t are read; the next iteration may overwrite them
    }

    s_xch[hsel][trow] = l_run;                // the last read of the maxima lies before the last P barrier
    __syncthreads();
    l_run += s_xch[hsel ^ 1][trow];
    const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
    if (lse && hsel == 0 && qrow < l_a && !*abort_flag) lse[(size_t)(row_base + qrow) * heads + head] = (m_run + log2f(l_run)) * 0.69314718055994531f;
    if (!FUSE_O) {
        if (qrow < l_a && !*abort_flag) {
            __nv_bfloat16* out = O + (size_t)(row_base + qrow) * d_g + col_h + hsel * HD;
#pragma unroll
            for (int ch = 0; ch < HD / 8; ++ch) {
                uint4 w;
                w.x = pack_bf16x2(o_acc[ch * 8 + 0] * inv, o_acc[ch * 8 + 1] * inv);
                w.y = pack_bf16x2(o_acc[ch * 8 + 2] * inv, o_acc[ch * 8 + 3] * inv);
                w.z = pack_bf16x2(o_acc[ch * 8 + 4] * inv, o_acc[ch * 8 + 5] * inv);
                w.w = pack_bf16x2(o_acc[ch * 8 + 6] * inv, o_acc[ch * 8 + 7] * inv);
                ((uint4*)out)[ch] = w;
            }
        }
    } else {
        // ---- z = o W^o_i (Eq. 35): o tile -> shared memory (in place of Q), one MMA group over all of TMEM ----
        {
            const int sw = trow & 7;
#pragma unroll
            for (int ch = 0; ch < HD / 8; ++ch) {
                uint4 w;
                w.x = pack_bf16x2(o_acc[ch * 8 + 0] * inv, o_acc[ch * 8 + 1] * inv);
                w.y = pack_bf16x2(o_acc[ch * 8 + 2] * inv, o_acc[ch * 8 + 3] * inv);
                w.z = pack_bf16x2(o_acc[ch * 8 + 4] * inv, o_acc[ch * 8 + 5] * inv);
                w.w = pack_bf16x2(o_acc[ch * 8 + 6] * inv, o_acc[ch * 8 + 7] * inv);
                *(uint4*)(sQ + trow * 128 + (((hsel * (HD / 8) + ch) ^ sw) << 4)) = w;
            }
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0 && !*abort_flag) {
            ok = mbar_wait(&ctl->bar_w, 0, abort_flag, status);
            tc_fence_after();
            const uint32_t oa = smem_u32(sQ), wa = smem_u32(sW);
            for (int n0 = 0; n0 < d; n0 += 256) {            // up to 256 output columns per MMA
                const int nn = min(256, d - n0);
                const uint32_t idesc_z = instr_desc_bf16(TQ, nn, false, true);
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks)
                    mma_bf16(tmem_base + n0, smem_desc(oa + ks * 32, 16, 1024), smem_desc(wa + (n0 / 64) * 8192 + ks * 2048, 8192, 1024),
                             idesc_z, ks != 0);
            }
            mma_commit(&ctl->bar_z);
        }
        ok = mbar_wait(&ctl->bar_z, 0, abort_flag, status);
        if (__all_sync(0xffffffffu, ok && !*abort_flag)) {
            tc_fence_after();
            // each warp stages a [32 rows x 64 columns] piece in shared memory (in place of P) and writes it out with
            // eight lanes per row, so that every store instruction covers whole 128-byte row segments; the two warps
            // of a lane quarter take alternate 64-column groups
            uint8_t* stg = sP + warp * 4096;
            const int wrow0 = q0 + quarter * 32;                  // first query row of this warp's piece
#pragma unroll 1
            for (int g = hsel; g < d / 64; g += 2) {
                float zf[64];
                tmem_ld32(t_lane + g * 64, (uint32_t*)zf);
                tmem_ld32(t_lane + g * 64 + 32, (uint32_t*)(zf + 32));
                tmem_ld_wait();
                __syncwarp();                                     // the previous piece has been read back
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    uint4 w;
                    w.x = pack_bf16x2(zf[ch * 8 + 0], zf[ch * 8 + 1]); w.y = pack_bf16x2(zf[ch * 8 + 2], zf[ch * 8 + 3]);
                    w.z = pack_bf16x2(zf[ch * 8 + 4], zf[ch * 8 + 5]); w.w = pack_bf16x2(zf[ch * 8 + 6], zf[ch * 8 + 7]);
                    *(uint4*)(stg + lane * 128 + ((ch ^ (lane & 7)) << 4)) = w;
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = i * 4 + (lane >> 3), ch = lane & 7;
                    if (wrow0 + r < l_a) {
                        const uint4 w = *(const uint4*)(stg + r * 128 + ((ch ^ (r & 7)) << 4));
                        *(uint4*)(Z + (size_t)(row_base + wrow0 + r) * d + g * 64 + ch * 8) = w;
                    }
                }
            }
        }
    }
    if (tid == 0 && *abort_flag) {           // let copies that may still be in flight land (bounded)
        mbar_wait(&ctl->bar_q, 0, abort_flag, status);
        for (int t = 0; t < 2 && t < n_kv; ++t) mbar_try_wait(&ctl->bar_kv[t], 0);
        if (FUSE_O) mbar_wait(&ctl->bar_w, 0, abort_flag, status);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

// Rotary position embedding on the rotary part of q and k (Eq. 32): in every head the last d_r channels are rotated
// in pairs (2i, 2i+1) by the angle t * 10000^(-2i/d_r), t = the token's position in its sample (so the score of a
// query-key pair depends on their distance in the sample, whichever patches were selected); sign = -1 rotates
// back (the backward of a rotation).  a, b: [rows, ld] bf16, rotated in place.  grid (pairs, chunks), one thread
// per (row of the pair, head).
namespace {
__global__ void __launch_bounds__(256)
rope_kernel(__nv_bfloat16* __restrict__ a, __nv_bfloat16* __restrict__ b, int ld, const int* __restrict__ pair_row,
            const int* __restrict__ patch_idx, int c, int l_p, int l_a, int heads, int d_h, int d_r, float sign) {
    pdl_trigger();
    pdl_wait();
    const int pair = blockIdx.x;
    const int idx = blockIdx.y * 256 + threadIdx.x;
    if (idx >= l_a * heads) return;
    const int lr = idx / heads, head = idx % heads;
    const int j = patch_idx[(size_t)pair * c + lr / l_p];
    if (j < 0) return;                                   // unused slot: zero rows stay zero
    const float t = (float)(j * l_p + lr % l_p);
    const size_t off = (size_t)(pair_row[pair] + lr) * ld + head * d_h + (d_h - d_r);
    uint32_t* pa = (uint32_t*)(a + off);                 // one 32-bit word = one rotated pair
    uint32_t* pb = (uint32_t*)(b + off);
    const float step = -2.0f * 13.287712379549449f / (float)d_r;      // log2(10000)
    for (int i = 0; i < d_r / 2; ++i) {
        float sn, cs;
        sincosf(t * exp2f(step * (float)i), &sn, &cs);
        sn *= sign;
        const uint32_t wa = pa[i], wb = pb[i];
        const float a0 = __uint_as_float(wa << 16), a1 = __uint_as_float(wa & 0xFFFF0000u);
        const float b0 = __uint_as_float(wb << 16), b1 = __uint_as_float(wb & 0xFFFF0000u);
        pa[i] = pack_bf16x2(a0 * cs - a1 * sn, a0 * sn + a1 * cs);
        pb[i] = pack_bf16x2(b0 * cs - b1 * sn, b0 * sn + b1 * cs);
    }
}
}  // namespace

uoe_status launch_rope(const Dims& D, void* a, void* b, int ld, const int* pair_row, const int* patch_idx, bool inverse,
                       cudaStream_t s) {
    if (D.d_rope <= 0) return UOE_OK;
    const int heads = D.d_g / D.d_h;
    dim3 grid(D.B * D.k, (D.l_a * heads + 255) / 256);
    ProfScope ps(inverse ? "rope_bwd" : "rope", s);
    launch_k(rope_kernel, grid, dim3(256), 0, s, (__nv_bfloat16*)a, (__nv_bfloat16*)b, ld, pair_row, patch_idx, D.c, D.l_p,
             D.l_a, heads, D.d_h, D.d_rope, inverse ? -1.0f : 1.0f);
    UOE_LAUNCHED();
    return UOE_OK;
}

// q, k, v, o: [rows_max, d_g] bf16 routed buffers.  If Wo is not null (one head per expert, d <= 512, d % 64 == 0)
// the output projection is fused: o is not written and z [rows_max, d] receives o W^o_i of every routed row.
bool attention_can_fuse_out(const Dims& D) { return D.d_g == DH && D.d <= kFuseMaxD && D.d % 64 == 0; }

uoe_status launch_attention(const Dims& D, const void* q, const void* k, const void* v, void* o, float* lse,
                            const int* pair_row, const int* patch_idx, bool causal, int* status, cudaStream_t s,
                            const void* Wo, const int* expert_idx, void* z) {
    if (D.d_h != DH) return UOE_ERR_UNSUPPORTED;
    if ((long long)D.B * D.k > 65535) return UOE_ERR_UNSUPPORTED;      // pairs ride on grid.z
    const bool fuse = Wo != nullptr;
    if (fuse && (!attention_can_fuse_out(D) || !expert_idx || !z)) return UOE_ERR_INVALID_ARG;
    static DeviceOnce once_plain, once_fused;
    {
        uoe_status st = smem_opt_in(once_plain, attn_kernel<false>, ATTN_SMEM);
        if (st == UOE_OK) st = smem_opt_in(once_fused, attn_kernel<true>, ATTN_SMEM_FUSED);
        if (st != UOE_OK) return st;
    }
    CUtensorMap tm[3], tmWo;
    const void* ptrs[3] = {q, k, v};
    for (int i = 0; i < 3; ++i) {
        const uint64_t dims[2] = {(uint64_t)D.d_g, (uint64_t)D.Rmax};
        const uint64_t str[1] = {(uint64_t)D.d_g * 2};
        const uint32_t box[2] = {DH, 128};
        if (!make_tmap(&tm[i], ptrs[i], 2, dims, str, box)) return UOE_ERR_CUDA;
    }
    tmWo = tm[0];
    if (fuse) {       // W^o [n, d_g, d]: boxes of 64 output columns x 64 contraction rows of one expert
        const uint64_t dims[3] = {(uint64_t)D.d, (uint64_t)D.d_g, (uint64_t)D.n};
        const uint64_t str[2] = {(uint64_t)D.d * 2, (uint64_t)D.d * D.d_g * 2};
        const uint32_t box[3] = {64, DH, 1};
        if (!make_tmap(&tmWo, Wo, 3, dims, str, box)) return UOE_ERR_CUDA;
    }
    const int heads = D.d_g / DH;
    dim3 grid((D.l_a + TQ - 1) / TQ, heads, D.B * D.k);
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)D.d_h);
    ProfScope ps("attention", s);
    if (fuse)
        launch_k(attn_kernel<true>, grid, dim3(kAttnThreads), ATTN_SMEM_FUSED, s, tm[0], tm[1], tm[2], (__nv_bfloat16*)o, lse, pair_row,
                 patch_idx, D.c, D.l_p, D.Lv, D.l_a, D.d_g, heads, causal ? 1 : 0, scale_log2, status, tmWo, expert_idx,
                 (__nv_bfloat16*)z, D.d);
    else
        launch_k(attn_kernel<false>, grid, dim3(kAttnThreads), ATTN_SMEM, s, tm[0], tm[1], tm[2], (__nv_bfloat16*)o, lse, pair_row,
                 patch_idx, D.c, D.l_p, D.Lv, D.l_a, D.d_g, heads, causal ? 1 : 0, scale_log2, status, tmWo, (const int*)nullptr,
                 (__nv_bfloat16*)nullptr, D.d);
    UOE_LAUNCHED();
    return UOE_OK;
}

}  // namespace uoe
