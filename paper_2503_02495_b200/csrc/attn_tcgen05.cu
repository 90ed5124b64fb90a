// Selective multi-head attention core (Eq. 33-34 with the masks of Eq. 41 and Fig. 4): for every
// (sample, chosen expert) pair and every head of that expert, softmax(q k^T / sqrt(d_h) + mask) v over
// the pair's l_a gathered tokens, and optionally the expert's output projection (Eq. 35) in the same kernel.
//
// q, k, v are rows of the routed buffers [rows, d_g] (bf16), so a pair's tokens are contiguous.  A unit of work is
// one 128-query tile of one head of one pair; its keys come in 128-key tiles.
//
// Two kernels:
//   attn_stream_kernel   many units (at least two per SM).  A persistent CTA (one per SM) holds two independent
//     pipelines, each with its own TMA warp, its own MMA-issuing warp, four softmax warps (one thread per query row),
//     its own Q buffer, two K/V stages, P buffer and TMEM columns, and each working units of its own:
//       TMA warp      Q tile of the unit, then K and V of each key tile into the two-stage ring; with the fused output
//                     projection also the expert's W^o in 192-column chunks through the same ring
//       MMA warp      S = Q K^T (128x128x64) into the pipeline's TMEM accumulator, issued as soon as the softmax warps
//                     have taken the previous S out; when they have written P, O_t = P V (128x64x128) into a second
//                     accumulator; at the end z chunks = o W^o (128x192x64)
//       softmax warps row maximum (first pass over S in TMEM), then p = 2^(s*c - m) in 32-column pieces (second pass),
//                     rounded to bf16 into shared memory in the swizzled K-major layout; O = alpha*O + O_t in
//                     registers, taken one key tile late, so that P V runs under the next tile's exponentials
//     The pipelines only meet in the tensor and special-function units of their SM: while one computes exponentials
//     or drains its output, the other's MMAs and loads run, and a pipeline's next Q, K, V are in flight while it
//     still works the current unit.
//   attn_tile_kernel     few units (fewer than two per SM): one CTA per unit, all eight warps on its softmax (two
//     threads per query row), S of the next key tile issued behind P V, the output projection as one MMA group over
//     all of TMEM.  With one unit per SM there is nothing to overlap a unit with, so the whole CTA works the unit.
// Masks: the real keys of a pair are a prefix of its gathered order (patches ascending, pad tokens at
// the end of the sample), so key c is kept iff c < n_valid, and with the causal flag iff also
// c <= query row (the shared lower triangle of Fig. 4).  Only tiles that cross one of the two limits test them.
#include "kernels.cuh"
#include "tc.cuh"
#include "tmap.cuh"

#include <type_traits>

namespace uoe {
namespace {

using namespace tc;

constexpr int TQ = 128, TK = 128, DH = 64;
constexpr int TILE_BYTES = 128 * DH * 2;          // 16 KB: a [128 x 64] bf16 tile
constexpr int kSoftmaxWarps = 4;                  // per pipeline: 128 threads, one per query row
constexpr int kAttnThreads = 2 * (kSoftmaxWarps + 2) * 32;      // 384
constexpr int kFuseMaxD = 512;
constexpr int ZCHUNK = 192;                       // output columns of one z = o W^o step: the S and O_t accumulators together

// shared memory of one pipeline
constexpr int PIPE_Q = 0;                          // Q tile
constexpr int PIPE_KV = TILE_BYTES;                // 2 stages x (K | V); a W^o chunk takes the K half of a stage
constexpr int PIPE_P = PIPE_KV + 4 * TILE_BYTES;   // P [128 x 128] as two swizzled halves; later the o tile and the staging of z
constexpr int PIPE_BYTES = PIPE_P + 2 * TILE_BYTES;            // 112 KB
constexpr int ATTN_SMEM = 2 * PIPE_BYTES + 2048 /*control*/ + 1024 /*alignment slack*/;      // 227 KB, all of an SM

struct PipeCtl {
    uint64_t q_full, q_empty, kv_full[2], kv_empty[2], acc_full, acc_empty, p_full, o_full, o_ready;
    int row_base, n_valid, expert, pad;
};
struct AttnCtl {
    PipeCtl pipe[2];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(AttnCtl) <= 2048, "control block");
static_assert(2 * PIPE_BYTES + 2048 + 1024 <= 232448, "shared memory of one SM");

struct AttnArgs {
    __nv_bfloat16* O;           // [rows, d_g] (not fused)
    __nv_bfloat16* Z;           // [rows, d]   (fused output projection)
    float* lse;                 // [rows, heads] or null
    const int* pair_row;        // [pairs]
    const int* patch_idx;       // [pairs, c]
    const int* expert_idx;      // [pairs] (fused)
    int pairs, c, l_p, Lv, l_a, d_g, heads, causal, d, n_qt;
    float scale_log2;
    int* status;
};


template <bool FUSE_O>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_stream_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmWo, const AttnArgs a) {
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    AttnCtl* ctl = (AttnCtl*)(smem + 2 * PIPE_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;
    int* status = a.status;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // warps 0-3: softmax of pipeline 0, 4-7: softmax of pipeline 1 (warp % 4 = the TMEM lane quarter a warp may read),
    // 8, 9: TMA warps, 10, 11: MMA warps
    const int g = warp < 8 ? warp / kSoftmaxWarps : (warp & 1);
    const int role = warp < 8 ? 0 : (warp < 10 ? 1 : 2);
    uint8_t* pbase = smem + g * PIPE_BYTES;
    uint8_t* sQ = pbase + PIPE_Q;
    uint8_t* sKV = pbase + PIPE_KV;
    uint8_t* sP = pbase + PIPE_P;
    PipeCtl* pc = &ctl->pipe[g];

    if (tid == 0) {
        for (int q = 0; q < 2; ++q) {
            PipeCtl* c = &ctl->pipe[q];
            mbar_init(&c->q_full, 1);
            mbar_init(&c->q_empty, 1 + kSoftmaxWarps);
            for (int t = 0; t < 2; ++t) { mbar_init(&c->kv_full[t], 1); mbar_init(&c->kv_empty[t], 1); }
            mbar_init(&c->acc_full, 1);
            mbar_init(&c->acc_empty, 32 * kSoftmaxWarps);
            mbar_init(&c->p_full, 32 * kSoftmaxWarps);
            mbar_init(&c->o_full, 1);
            mbar_init(&c->o_ready, 32 * kSoftmaxWarps);
        }
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmQ);
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
        if (FUSE_O) prefetch_tmap(&tmWo);
    }
    if (warp == 8) tmem_alloc(&ctl->tmem_base, 512);       // per pipeline 256 columns: S / z chunk [0,128), O_t [128,192)
    pdl_wait();                                             // from here on: data written by earlier kernels
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_pipe = ctl->tmem_base + g * 256;

    // ---- the units of this pipeline ----
    const int n_units = a.pairs * a.heads * a.n_qt;
    const int u_first = (int)blockIdx.x * 2 + g, u_step = 2 * (int)gridDim.x;
    constexpr int t_first = 0, t_step = 1;
    auto kv_tiles = [&](int q0, int n_valid) {              // key tiles the unit has in all
        int kv_end = min(n_valid, a.l_a);
        if (a.causal) kv_end = min(kv_end, q0 + TQ);
        return (kv_end + TK - 1) / TK;
    };
    const int n_zchunk = FUSE_O ? (a.d + ZCHUNK - 1) / ZCHUNK : 0;
    auto wait = [&](uint64_t* bar, uint32_t parity) { return mbar_wait(bar, parity, abort_flag, status) && !*abort_flag; };
    // the same for the one-thread roles (TMA, MMA), which sit on the critical path between the softmax warps' steps:
    // they poll without letting the hardware suspend them first
    auto wait1 = [&](uint64_t* bar, uint32_t parity) { return mbar_wait_spin(bar, parity, abort_flag, status) && !*abort_flag; };

    if (role == 1) {
        // =========================== TMA warp ===========================
        uint32_t q_cnt = 0, kv_cnt = 0;
        bool ok = true;
        for (int u = u_first; u < n_units && ok; u += u_step) {
            const int qt = u % a.n_qt, head = (u / a.n_qt) % a.heads, pair = u / (a.n_qt * a.heads);
            // real keys of this pair: sum over its slots of the real tokens in the slot's patch
            int nv = 0;
            for (int s0 = lane; s0 < a.c; s0 += 32) {
                const int j = a.patch_idx[(size_t)pair * a.c + s0];
                if (j >= 0) nv += max(0, min(a.l_p, a.Lv - j * a.l_p));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) nv += __shfl_xor_sync(0xffffffffu, nv, o);
            const int row_base = a.pair_row[pair];
            const int expert = FUSE_O ? a.expert_idx[pair] : 0;
            const int q0 = qt * TQ, col_h = head * DH;
            const int n_kv = kv_tiles(q0, nv);
            const bool mine = t_first < n_kv;
            if (lane == 0) {
                ok = wait1(&pc->q_empty, (q_cnt & 1) ^ 1);
                if (ok) {
                    pc->row_base = row_base; pc->n_valid = nv; pc->expert = expert;
                    if (mine) {
                        mbar_arrive_expect_tx(&pc->q_full, TILE_BYTES);
                        tma_load_2d(sQ, &tmQ, col_h, row_base + q0, &pc->q_full);
                    } else {
                        mbar_arrive(&pc->q_full);
                    }
                }
                ++q_cnt;
                for (int t = t_first; t < n_kv && ok; t += t_step) {
                    const int st = kv_cnt & 1;
                    ok = wait1(&pc->kv_empty[st], ((kv_cnt >> 1) & 1) ^ 1);
                    if (!ok) break;
                    uint8_t* stage = sKV + st * 2 * TILE_BYTES;
                    mbar_arrive_expect_tx(&pc->kv_full[st], 2 * TILE_BYTES);
                    tma_load_2d(stage, &tmK, col_h, row_base + t * TK, &pc->kv_full[st]);
                    tma_load_2d(stage + TILE_BYTES, &tmV, col_h, row_base + t * TK, &pc->kv_full[st]);
                    ++kv_cnt;
                }
                if (FUSE_O && mine) {          // W^o in chunks
                    for (int zc = 0; zc < n_zchunk && ok; ++zc) {
                        const int n0 = zc * ZCHUNK, nn = min(ZCHUNK, a.d - n0);
                        const int st = kv_cnt & 1;
                        ok = wait1(&pc->kv_empty[st], ((kv_cnt >> 1) & 1) ^ 1);
                        if (!ok) break;
                        uint8_t* stage = sKV + st * 2 * TILE_BYTES;
                        mbar_arrive_expect_tx(&pc->kv_full[st], (uint32_t)nn * DH * 2);
                        for (int nb = 0; nb < nn / 64; ++nb) tma_load_3d(stage + nb * 8192, &tmWo, n0 + nb * 64, 0, expert, &pc->kv_full[st]);
                        ++kv_cnt;
                    }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (lane == 0 && *abort_flag) {          // let copies that may still be in flight land (bounded)
            if (q_cnt > 0) mbar_wait(&pc->q_full, (q_cnt - 1) & 1, abort_flag, status);
            for (uint32_t t = (kv_cnt > 2 ? kv_cnt - 2 : 0); t < kv_cnt; ++t) mbar_wait(&pc->kv_full[t & 1], (t >> 1) & 1, abort_flag, status);
        }
    } else if (role == 2) {
        // =========================== MMA warp ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc_bf16(TQ, TK, false, false);
            constexpr uint32_t idesc_o = instr_desc_bf16(TQ, DH, false, true);
            uint32_t q_cnt = 0, kv_cnt = 0, acc_cnt = 0, p_cnt = 0, ready_cnt = 0;
            bool ok = true;
            for (int u = u_first; u < n_units && ok; u += u_step) {
                const int qt = u % a.n_qt;
                ok = wait1(&pc->q_full, q_cnt & 1);
                ++q_cnt;
                if (!ok) break;
                const int n_kv = kv_tiles(qt * TQ, pc->n_valid);
                if (t_first >= n_kv) { mbar_arrive(&pc->q_empty); continue; }
                tc_fence_after();
                const uint32_t qa = smem_u32(sQ), pa = smem_u32(sP);
                // S of a key tile is issued as soon as its K has landed and the softmax warps have taken the previous S out
                // of the accumulator -- ahead of the previous tile's P V, which has to wait for P -- so the next S is
                // ready when the softmax warps come back for it
                auto issue_s = [&](uint32_t stage_cnt, bool last) {
                    const int st = stage_cnt & 1;
                    if (!(wait1(&pc->kv_full[st], (stage_cnt >> 1) & 1) && wait1(&pc->acc_empty, (acc_cnt & 1) ^ 1))) return false;
                    tc_fence_after();
                    const uint32_t ka = smem_u32(sKV + st * 2 * TILE_BYTES);
#pragma unroll
                    for (int ks = 0; ks < DH / 16; ++ks)
                        mma_bf16(tmem_pipe, smem_desc(qa + ks * 32, 16, 1024), smem_desc(ka + ks * 32, 16, 1024), idesc_s, ks != 0);
                    mma_commit(&pc->acc_full);
                    ++acc_cnt;
                    if (last) mma_commit(&pc->q_empty);       // the unit's last use of Q
                    return true;
                };
                ok = issue_s(kv_cnt, t_first + t_step >= n_kv);
                for (int t = t_first; t < n_kv && ok; t += t_step) {
                    const int st = kv_cnt & 1;
                    if (t + t_step < n_kv) {
                        ok = issue_s(kv_cnt + 1, t + 2 * t_step >= n_kv);
                        if (!ok) break;
                    }
                    ok = wait1(&pc->p_full, p_cnt & 1);
                    ++p_cnt;
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t va = smem_u32(sKV + st * 2 * TILE_BYTES) + TILE_BYTES;
#pragma unroll
                    for (int ks = 0; ks < TK / 16; ++ks)
                        mma_bf16(tmem_pipe + 128, smem_desc(pa + (ks >> 2) * TILE_BYTES + (ks & 3) * 32, 16, 1024),
                                 smem_desc(va + ks * 2048, 8192, 1024), idesc_o, ks != 0);
                    mma_commit(&pc->o_full);
                    mma_commit(&pc->kv_empty[st]);
                    ++kv_cnt;
                }
                if (FUSE_O && ok) {
                    // z = o W^o_i (Eq. 35): the o tile sits where P was, chunk by chunk into the S accumulator
                    ok = wait1(&pc->o_ready, ready_cnt & 1);
                    ++ready_cnt;
                    for (int zc = 0; zc < n_zchunk && ok; ++zc) {
                        const int nn = min(ZCHUNK, a.d - zc * ZCHUNK);
                        const int st = kv_cnt & 1;
                        ok = wait1(&pc->kv_full[st], (kv_cnt >> 1) & 1) && wait1(&pc->acc_empty, (acc_cnt & 1) ^ 1);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t wa = smem_u32(sKV + st * 2 * TILE_BYTES);
                        const uint32_t idesc_z = instr_desc_bf16(TQ, nn, false, true);
#pragma unroll
                        for (int ks = 0; ks < DH / 16; ++ks)
                            mma_bf16(tmem_pipe, smem_desc(pa + ks * 32, 16, 1024), smem_desc(wa + ks * 2048, 8192, 1024), idesc_z, ks != 0);
                        mma_commit(&pc->acc_full);
                        mma_commit(&pc->kv_empty[st]);
                        ++acc_cnt;
                        ++kv_cnt;
                    }
                }
            }
        }
    } else {
        // =========================== softmax warps ===========================
        const int quarter = warp & 3;
        const int trow = quarter * 32 + lane;                  // row of the tile (TMEM lane)
        const uint32_t t_lane = tmem_pipe + ((uint32_t)(quarter * 32) << 16);
        const int sw = trow & 7;
        uint32_t q_cnt = 0, acc_cnt = 0, o_cnt = 0;
        bool ok = true;
        for (int u = u_first; u < n_units && ok; u += u_step) {
            const int qt = u % a.n_qt, head = (u / a.n_qt) % a.heads;
            ok = __all_sync(0xffffffffu, wait(&pc->q_full, q_cnt & 1));
            ++q_cnt;
            if (!ok) break;
            const int row_base = pc->row_base, n_valid = pc->n_valid;
            __syncwarp();
            if (lane == 0) mbar_arrive(&pc->q_empty);
            const int q0 = qt * TQ, qrow = q0 + trow;
            const int n_kv = kv_tiles(q0, n_valid);
            if (t_first >= n_kv) continue;
            const int kv_lim = min(n_valid, a.l_a);

            float o_acc[DH];
#pragma unroll
            for (int i = 0; i < DH; ++i) o_acc[i] = 0.f;
            float m_run = -INFINITY, l_run = 0.f, alpha_pending = 1.f;
            bool pending = false;
            // O += alpha * O + O_t of the previous key tile (its P V has had a whole softmax to finish)
            auto take_o = [&]() {
                bool w = __all_sync(0xffffffffu, wait(&pc->o_full, o_cnt & 1));
                ++o_cnt;
                if (!w) return false;
                tc_fence_after();
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float o_t[32];
                    tmem_ld32(t_lane + 128 + h * 32, (uint32_t*)o_t);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o_acc[h * 32 + i] = fmaf(o_acc[h * 32 + i], alpha_pending, o_t[i]);
                }
                return true;
            };

            for (int t = t_first; t < n_kv && ok; t += t_step) {
                ok = __all_sync(0xffffffffu, wait(&pc->acc_full, acc_cnt & 1));
                ++acc_cnt;
                if (!ok) break;
                tc_fence_after();
                const int kv0 = t * TK;
                const bool masked = kv0 + TK > kv_lim || (a.causal && kv0 + TK - 1 > q0);
                // columns of this tile that the row keeps: one limit covers both masks (real keys are a prefix, and so is
                // the causal triangle of a row)
                const int keep_cols = min(kv_lim, a.causal ? qrow + 1 : kv_lim) - kv0;
                // ---- first pass: the row's maximum over the tile ----
                float mx = -INFINITY;
#pragma unroll
                for (int ch = 0; ch < TK / 32; ++ch) {
                    float s[32];
                    tmem_ld32(t_lane + ch * 32, (uint32_t*)s);
                    tmem_ld_wait();
                    if (masked) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) mx = fmaxf(mx, ch * 32 + j < keep_cols ? s[j] : -INFINITY);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) mx = fmaxf(mx, s[j]);
                    }
                }
                const float m_new = fmaxf(m_run, mx * a.scale_log2);
                // a row with no kept key so far keeps m = -inf; 2^(-inf - (-inf)) is avoided by the guard
                const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                const float alpha = ex2_approx(m_run - m_use);
                if (pending) { ok = take_o(); if (!ok) break; }
                // ---- second pass: p = 2^(s c - m), bf16, into shared memory (swizzled K-major, two [128 x 64] halves) ----
                float l_add = 0.f;
                // (the mask test is a template argument: tested per element at run time it becomes a branch per element)
                auto second_pass = [&](auto mask_tag) {
                    constexpr bool MASKED = decltype(mask_tag)::value;
#pragma unroll
                    for (int ch = 0; ch < TK / 32; ++ch) {
                        float s[32];
                        tmem_ld32(t_lane + ch * 32, (uint32_t*)s);
                        tmem_ld_wait();
                        if (ch == TK / 32 - 1) {            // S is in registers: the accumulator may take the next S
                            tc_fence_before();
                            mbar_arrive(&pc->acc_empty);
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            float p = ex2_approx(fmaf(s[j], a.scale_log2, -m_use));
                            if constexpr (MASKED) p = ch * 32 + j < keep_cols ? p : 0.f;
                            s[j] = p;
                            l_add += p;
                        }
                        uint8_t* prow = sP + (ch >> 1) * TILE_BYTES + (size_t)trow * 128;
#pragma unroll
                        for (int c8 = 0; c8 < 4; ++c8) {
                            uint4 w;
                            w.x = pack_bf16x2(s[c8 * 8 + 0], s[c8 * 8 + 1]); w.y = pack_bf16x2(s[c8 * 8 + 2], s[c8 * 8 + 3]);
                            w.z = pack_bf16x2(s[c8 * 8 + 4], s[c8 * 8 + 5]); w.w = pack_bf16x2(s[c8 * 8 + 6], s[c8 * 8 + 7]);
                            *(uint4*)(prow + ((((ch & 1) * 4 + c8) ^ sw) << 4)) = w;
                        }
                    }
                };
                if (masked) second_pass(std::true_type{});
                else second_pass(std::false_type{});
                l_run = fmaf(l_run, alpha, l_add);
                m_run = m_new;
                alpha_pending = alpha;
                pending = true;
                fence_async_smem();                  // generic-proxy writes of P -> visible to the tensor core
                mbar_arrive(&pc->p_full);
            }
            if (!ok) break;
            if (pending) { ok = take_o(); if (!ok) break; }

            const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
            if (a.lse && qrow < a.l_a) a.lse[(size_t)(row_base + qrow) * a.heads + head] = (m_run + log2f(l_run)) * 0.69314718055994531f;
            if (!FUSE_O) {
                if (qrow < a.l_a) {
                    __nv_bfloat16* out = a.O + (size_t)(row_base + qrow) * a.d_g + head * DH;
#pragma unroll
                    for (int ch = 0; ch < DH / 8; ++ch) {
                        uint4 w;
                        w.x = pack_bf16x2(o_acc[ch * 8 + 0] * inv, o_acc[ch * 8 + 1] * inv);
                        w.y = pack_bf16x2(o_acc[ch * 8 + 2] * inv, o_acc[ch * 8 + 3] * inv);
                        w.z = pack_bf16x2(o_acc[ch * 8 + 4] * inv, o_acc[ch * 8 + 5] * inv);
                        w.w = pack_bf16x2(o_acc[ch * 8 + 6] * inv, o_acc[ch * 8 + 7] * inv);
                        ((uint4*)out)[ch] = w;
                    }
                }
            } else {
                // ---- z = o W^o_i (Eq. 35): the normalised o tile as the A operand where P was (bf16, swizzled) ----
#pragma unroll
                for (int ch = 0; ch < DH / 8; ++ch) {
                    uint4 w;
                    w.x = pack_bf16x2(o_acc[ch * 8 + 0] * inv, o_acc[ch * 8 + 1] * inv);
                    w.y = pack_bf16x2(o_acc[ch * 8 + 2] * inv, o_acc[ch * 8 + 3] * inv);
                    w.z = pack_bf16x2(o_acc[ch * 8 + 4] * inv, o_acc[ch * 8 + 5] * inv);
                    w.w = pack_bf16x2(o_acc[ch * 8 + 6] * inv, o_acc[ch * 8 + 7] * inv);
                    *(uint4*)(sP + trow * 128 + ((ch ^ sw) << 4)) = w;
                }
                fence_async_smem();
                mbar_arrive(&pc->o_ready);
                // each warp stages a [32 rows x 64 columns] piece in the free half of P's place and writes it out with
                // eight lanes per row, so that every store instruction covers whole 128-byte row segments
                uint8_t* stg = sP + TILE_BYTES + quarter * 4096;
                const int wrow0 = q0 + quarter * 32;                  // first query row of this warp's piece
                for (int zc = 0; zc < n_zchunk && ok; ++zc) {
                    const int n0 = zc * ZCHUNK, nn = min(ZCHUNK, a.d - n0);
                    ok = __all_sync(0xffffffffu, wait(&pc->acc_full, acc_cnt & 1));
                    ++acc_cnt;
                    if (!ok) break;
                    tc_fence_after();
                    for (int g64 = 0; g64 < nn / 64; ++g64) {
                        float zf[64];
                        tmem_ld32(t_lane + g64 * 64, (uint32_t*)zf);
                        tmem_ld32(t_lane + g64 * 64 + 32, (uint32_t*)(zf + 32));
                        tmem_ld_wait();
                        if (g64 == nn / 64 - 1) {
                            tc_fence_before();
                            mbar_arrive(&pc->acc_empty);
                        }
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
                            if (wrow0 + r < a.l_a) {
                                const uint4 w = *(const uint4*)(stg + r * 128 + ((ch ^ (r & 7)) << 4));
                                *(uint4*)(a.Z + (size_t)(row_base + wrow0 + r) * a.d + n0 + g64 * 64 + ch * 8) = w;
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(ctl->tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------
// one CTA per unit
// ------------------------------------------------------------------------------------------------
constexpr int kTileThreads = 256;
constexpr int TILE_SMEM = TILE_BYTES * (1 + 2 + 2 + 2) + 1024 + 256;
constexpr int TILE_SMEM_FUSED = TILE_SMEM + 1024 + kFuseMaxD * DH * 2;      // + the expert's W^o slice [64 x d] behind the control block

struct TileCtl {
    uint64_t bar_q, bar_kv[2], bar_s, bar_o, bar_w, bar_z;
    uint32_t tmem_base;
    int abort_flag;
};

// FUSE_O (one head per expert, d <= 512): the output projection of Eq. 35 runs in the same CTA.  The expert's W^o
// slice [64 x d] is fetched by TMA at kernel start; after the last key tile the normalised o tile goes to shared
// memory (bf16, swizzled, in place of Q), z = o W^o_i [128 x d] is accumulated over the whole of TMEM (S and O_t are
// no longer needed) and written to Z instead of o to O.
template <bool FUSE_O>
__global__ void __launch_bounds__(kTileThreads)
attn_tile_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
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
    TileCtl* ctl = (TileCtl*)(sP + 2 * TILE_BYTES);
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
        // columns of this thread's half tile that the row keeps: one limit covers both masks (the real keys are a
        // prefix, and so is the causal triangle of a row); tiles inside both limits skip the test
        const int keep_cols = min(min(n_valid, l_a), causal ? qrow + 1 : l_a) - kv0;
        const bool masked = it * TK + TK > min(n_valid, l_a) || (causal && it * TK + TK - 1 > q0);
        if (masked) {
#pragma unroll
            for (int j = 0; j < HK; ++j) {
                s_row[j] = j < keep_cols ? s_row[j] * scale_log2 : -INFINITY;
                m_new = fmaxf(m_new, s_row[j]);
            }
        } else {
#pragma unroll
            for (int j = 0; j < HK; ++j) {
                s_row[j] *= scale_log2;
                m_new = fmaxf(m_new, s_row[j]);
            }
        }
        s_xch[hsel][trow] = m_new;            // read by the row's other thread; rewritten only after the next barrier
        __syncthreads();
        m_new = fmaxf(m_new, s_xch[hsel ^ 1][trow]);
        // a row with no kept key so far keeps m = -inf; exp2(-inf - (-inf)) is avoided by the guard
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = ex2_approx(m_run - m_use);
        float l_add = 0.f;
        uint8_t* prow = sP + hsel * TILE_BYTES + (size_t)trow * 128;
        const int sw = trow & 7;
#pragma unroll
        for (int ch = 0; ch < HK / 8; ++ch) {                 // 16-byte chunks of 8 bf16
            float p[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) { p[q] = ex2_approx(s_row[ch * 8 + q] - m_use); l_add += p[q]; }
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
    const bool fuse = Wo != nullptr;
    if (fuse && (!attention_can_fuse_out(D) || !expert_idx || !z)) return UOE_ERR_INVALID_ARG;
    static DeviceOnce once_plain, once_fused, once_tile_plain, once_tile_fused;
    {
        uoe_status st = smem_opt_in(once_plain, attn_stream_kernel<false>, ATTN_SMEM);
        if (st == UOE_OK) st = smem_opt_in(once_fused, attn_stream_kernel<true>, ATTN_SMEM);
        if (st == UOE_OK) st = smem_opt_in(once_tile_plain, attn_tile_kernel<false>, TILE_SMEM);
        if (st == UOE_OK) st = smem_opt_in(once_tile_fused, attn_tile_kernel<true>, TILE_SMEM_FUSED);
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
    const int heads = D.d_g / DH, n_qt = (D.l_a + TQ - 1) / TQ;
    const long long pairs = (long long)D.B * D.k, units = pairs * heads * n_qt;
    if (units > 0x7fffffffll) return UOE_ERR_UNSUPPORTED;
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)D.d_h);
    ProfScope ps("attention", s);
    cudaError_t e;
    if (units >= 2ll * sm_count()) {          // enough units to keep two pipelines per SM fed
        AttnArgs a;
        a.O = (__nv_bfloat16*)o; a.Z = (__nv_bfloat16*)z; a.lse = lse;
        a.pair_row = pair_row; a.patch_idx = patch_idx; a.expert_idx = expert_idx;
        a.pairs = (int)pairs; a.c = D.c; a.l_p = D.l_p; a.Lv = D.Lv; a.l_a = D.l_a; a.d_g = D.d_g; a.heads = heads;
        a.causal = causal ? 1 : 0; a.d = D.d; a.n_qt = n_qt;
        a.scale_log2 = scale_log2;
        a.status = status;
        const long long want = (units + 1) / 2;
        const int grid = (int)(want < sm_count() ? want : sm_count());
        if (fuse) e = launch_k(attn_stream_kernel<true>, dim3(grid), dim3(kAttnThreads), ATTN_SMEM, s, tm[0], tm[1], tm[2], tmWo, a);
        else e = launch_k(attn_stream_kernel<false>, dim3(grid), dim3(kAttnThreads), ATTN_SMEM, s, tm[0], tm[1], tm[2], tmWo, a);
    } else {
        if (pairs > 65535) return UOE_ERR_UNSUPPORTED;      // (cannot happen: fewer than two units per SM)
        dim3 grid(n_qt, heads, (unsigned)pairs);
        if (fuse)
            e = launch_k(attn_tile_kernel<true>, grid, dim3(kTileThreads), TILE_SMEM_FUSED, s, tm[0], tm[1], tm[2], (__nv_bfloat16*)o, lse,
                         pair_row, patch_idx, D.c, D.l_p, D.Lv, D.l_a, D.d_g, heads, causal ? 1 : 0, scale_log2, status, tmWo, expert_idx,
                         (__nv_bfloat16*)z, D.d);
        else
            e = launch_k(attn_tile_kernel<false>, grid, dim3(kTileThreads), TILE_SMEM, s, tm[0], tm[1], tm[2], (__nv_bfloat16*)o, lse,
                         pair_row, patch_idx, D.c, D.l_p, D.Lv, D.l_a, D.d_g, heads, causal ? 1 : 0, scale_log2, status, tmWo,
                         (const int*)nullptr, (__nv_bfloat16*)nullptr, D.d);
    }
    if (e != cudaSuccess) return UOE_ERR_CUDA;
    UOE_LAUNCHED();
    return UOE_OK;
}

}  // namespace uoe
