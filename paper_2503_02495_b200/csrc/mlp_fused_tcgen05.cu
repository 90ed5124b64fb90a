// UoME expert MLP in one kernel (Eq. 38-39) for narrow experts (d_e = 256, d <= 512):
//
//   z[r, :] = phi( A[r, :] @ W1[e(r)] ) @ W2[e(r)],   r over the routed rows, e(r) = expert whose region holds r
//
// The hidden tile [128 x 256] never leaves the SM: GEMM1 accumulates it in TMEM, the epilogue warps apply phi and
// write it to shared memory as the bf16 A operand of GEMM2, whose [128 x d] result goes back to TMEM and out by
// TMA stores.  One persistent CTA per SM walks the 128-row tiles (expert regions are padded to 128 rows).
//   warp 0      TMA producer: per 64-wide K step of GEMM1 an A block [128 x 64] (from a routed buffer, or gathered
//               from x with one box per source patch, Eq. 18) and a W1 block [64 x 256]; then per 64-row K step of
//               GEMM2 a W2 block [64 x up to 256]; one three-stage ring serves both, so W2 and the next tile's
//               operands are fetched while the epilogue works
//   warp 1      MMA issuer: tcgen05.mma 128 x 256 x 16 into TMEM columns [0, 256) (hidden tile), then
//               128 x N x 16 into [256, 512) (output columns 0-255) and, for d > 256, into [0, 256) again (the
//               hidden tile has been consumed by then)
//   warps 2-9   epilogue, two warps per TMEM lane quarter sharing the 64-column groups: hidden tile -> (optional
//               store of the pre-activation) -> phi -> bf16 -> swizzled K-major tile in shared memory; output tile
//               -> bf16 -> [32 x 64] pieces staged in the same shared memory (GEMM2 has finished reading it) -> TMA
//               tensor stores
#include "kernels.cuh"
#include "tc.cuh"
#include "tmap.cuh"

namespace uoe {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64, DE = 256;
constexpr int A_BYTES = BM * BK * 2;              // 16 KB
constexpr int B_BYTES = BK * 256 * 2;             // 32 KB: [64 x 256]
constexpr int STAGE = A_BYTES + B_BYTES;
constexpr int STAGES = 3;
constexpr int HID_BYTES = BM * DE * 2;            // 64 KB: phi(h) as four [128 x 64] swizzled tiles
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int SMEM = STAGES * STAGE + HID_BYTES + 1024 /*align slack*/ + 1024 /*control*/;

struct FCtl {
    uint64_t full[STAGES], empty[STAGES], bar_h, bar_a, bar_z, bar_done;
    uint32_t tmem_base;
    int abort_flag;
    int offs[34];
    int tstart[34];
};

__global__ void __launch_bounds__(THREADS, 1)
mlp_fused_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmX,
                 const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW2,
                 const __grid_constant__ CUtensorMap tmZ, __nv_bfloat16* __restrict__ pre,
                 const int* __restrict__ offsets, int n, int d, int act, int* status,
                 const SrcMap smap, int l_p, int Bm,
                 const __nv_bfloat16* __restrict__ b1 /* [n, 256] or null */, const __nv_bfloat16* __restrict__ b2 /* [n, d] or null */) {
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sHid = smem + STAGES * STAGE;
    FCtl* ctl = (FCtl*)(sHid + HID_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        mbar_init(&ctl->bar_h, 1);
        mbar_init(&ctl->bar_a, 32 * EPI_WARPS);
        mbar_init(&ctl->bar_z, 1);
        mbar_init(&ctl->bar_done, 32 * EPI_WARPS);
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmX);
        prefetch_tmap(&tmW1);
        prefetch_tmap(&tmW2);
        prefetch_tmap(&tmZ);
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, 512);
    pdl_wait();                     // everything above touches only this CTA's own resources
    if (warp == 2) {                // offsets and the row-tile prefix over experts (n <= 31)
        int o = 0;
        if (lane <= n) o = offsets[lane];
        const int o1 = __shfl_down_sync(0xffffffffu, o, 1);
        const int tiles = lane < n ? (o1 - o) / BM : 0;
        int incl = tiles;
#pragma unroll
        for (int dd = 1; dd < 32; dd <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, dd);
            if (lane >= dd) incl += v;
        }
        if (lane <= n) ctl->offs[lane] = o;
        if (lane < n) ctl->tstart[lane] = incl - tiles;
        if (lane == n - 1) ctl->tstart[n] = incl;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int total_tiles = ctl->tstart[n];
    const int kb1 = d / BK;                     // K steps of GEMM1
    constexpr int kb2 = DE / BK;                // K steps of GEMM2 (per output half)
    const int nh = d > 256 ? 2 : 1;             // output halves of up to 256 columns

    auto locate = [&](int tile, int& e, int& row0) {
        e = 0;
        while (e + 1 < n && tile >= ctl->tstart[e + 1]) ++e;
        row0 = ctl->offs[e] + (tile - ctl->tstart[e]) * BM;
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_parity = 0;
        bool stop = false;
        auto acquire = [&](uint32_t bytes) -> bool {       // waits for the stage to be free, arms its barrier
            int ok = 1;
            if (lane == 0) ok = (mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag, status) && !*abort_flag) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) return false;
            if (lane == 0) mbar_arrive_expect_tx(&ctl->full[stage], bytes);
            __syncwarp();
            return true;
        };
        auto advance = [&]() {
            issued |= 1u << stage;
            issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
        };
        const bool gathered = smap.on();
        const int nbox_a = gathered ? BM / l_p : 1;                         // <= 16
        // where a tile's rows come from (two dependent look-ups in global memory when A is gathered): found for the
        // next tile while this tile's first W2 blocks are in flight and the ring is full anyway
        int e_next = 0, row0_next = 0, src_next = 0;
        auto look_up = [&](int tile) {
            if (tile >= total_tiles) return;
            locate(tile, e_next, row0_next);
            if (gathered && lane < nbox_a) src_next = src_of(smap, row0_next + lane * l_p, e_next, ctl->offs[e_next], Bm);   // Bm: zero-filled box
        };
        look_up(blockIdx.x);
        for (int tile = blockIdx.x; tile < total_tiles && !stop; tile += gridDim.x) {
            const int e = e_next, row0 = row0_next, my_src = src_next;
            bool looked = false;
            for (int kb = 0; kb < kb1 && !stop; ++kb) {
                if (!acquire(STAGE)) { stop = true; break; }
                uint8_t* sa = smem + stage * STAGE;
                uint8_t* sb = sa + A_BYTES;
                if (lane < nbox_a) {
                    if (gathered) tma_load_3d(sa + lane * l_p * 128, &tmX, kb * BK, 0, my_src, &ctl->full[stage]);
                    else tma_load_2d(sa, &tmA, kb * BK, row0, &ctl->full[stage]);
                }
                if (lane >= 16 && lane < 20)
                    tma_load_3d(sb + (lane - 16) * 8192, &tmW1, (lane - 16) * 64, kb * BK, e, &ctl->full[stage]);
                advance();
            }
            for (int j = 0; j < nh && !stop; ++j) {
                const int nbox = min(256, d - j * 256) / 64;
                for (int kb = 0; kb < kb2; ++kb) {
                    if (!acquire((uint32_t)nbox * 8192)) { stop = true; break; }
                    uint8_t* sb = smem + stage * STAGE + A_BYTES;
                    if (lane < nbox) tma_load_3d(sb + lane * 8192, &tmW2, j * 256 + lane * 64, kb * BK, e, &ctl->full[stage]);
                    advance();
                    if (!looked && j * kb2 + kb + 1 == STAGES) { look_up(tile + gridDim.x); looked = true; }
                }
            }
            if (!looked) look_up(tile + gridDim.x);
        }
        if (lane == 0 && *abort_flag) {      // let this CTA's own copies land before it exits
            for (int s = 0; s < STAGES; ++s)
                if (issued & (1u << s)) mbar_wait(&ctl->full[s], (issued_parity >> s) & 1, abort_flag, status);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            constexpr uint32_t idesc_h = instr_desc_bf16(BM, DE, false, true);
            int stage = 0;
            uint32_t phase = 0;
            bool stop = false;
            int i = 0;                                   // tiles done by this CTA
            for (int tile = blockIdx.x; tile < total_tiles && !stop; tile += gridDim.x, ++i) {
                // d > 256: the hidden tile shares its TMEM columns with the second output half of the previous tile
                if (nh == 2 && i > 0 && (!mbar_wait(&ctl->bar_done, (i - 1) & 1, abort_flag, status) || *abort_flag)) break;
                tc_fence_after();
                for (int kb = 0; kb < kb1; ++kb) {
                    if (!mbar_wait(&ctl->full[stage], phase, abort_flag, status) || *abort_flag) { stop = true; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + stage * STAGE), sb = sa + A_BYTES;
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks)
                        mma_bf16(tmem_base, smem_desc(sa + ks * 32, 16, 1024), smem_desc(sb + ks * 2048, 8192, 1024), idesc_h,
                                 (kb | ks) != 0);
                    mma_commit(&ctl->empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (stop) break;
                mma_commit(&ctl->bar_h);
                // phi(h) is in shared memory; d <= 256: the output columns [256, 512) of the previous tile are drained
                if (!mbar_wait(&ctl->bar_a, i & 1, abort_flag, status) || *abort_flag) break;
                if (nh == 1 && i > 0 && (!mbar_wait(&ctl->bar_done, (i - 1) & 1, abort_flag, status) || *abort_flag)) break;
                tc_fence_after();
                const uint32_t ha = smem_u32(sHid);
                for (int j = 0; j < nh && !stop; ++j) {
                    const int ncols = min(256, d - j * 256);
                    const uint32_t idesc_z = instr_desc_bf16(BM, ncols, false, true);
                    const uint32_t d_tmem = tmem_base + (j == 0 ? 256 : 0);
                    for (int kb = 0; kb < kb2; ++kb) {
                        if (!mbar_wait(&ctl->full[stage], phase, abort_flag, status) || *abort_flag) { stop = true; break; }
                        tc_fence_after();
                        const uint32_t sb = smem_u32(smem + stage * STAGE) + A_BYTES;
#pragma unroll
                        for (int ks = 0; ks < BK / 16; ++ks)
                            mma_bf16(d_tmem, smem_desc(ha + kb * (BM * 128) + ks * 32, 16, 1024),
                                     smem_desc(sb + ks * 2048, 8192, 1024), idesc_z, (kb | ks) != 0);
                        mma_commit(&ctl->empty[stage]);
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                }
                if (stop) break;
                mma_commit(&ctl->bar_z);
            }
        }
    } else {
        // ---------------- epilogue: warps w and w + 4 drain TMEM lane quarter w % 4, alternate 64-column groups ----------------
        const int quarter = warp & 3;
        const int wsel = (warp - 2) >> 2;
        const int trow = quarter * 32 + lane;                 // row of the tile = TMEM lane
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        uint8_t* stg = sHid + (warp - 2) * 4096;              // this warp's [32 x 64] staging piece (output phase)
        auto pack8 = [](const float* f) {
            uint4 w;
            w.x = pack_bf16x2(f[0], f[1]); w.y = pack_bf16x2(f[2], f[3]);
            w.z = pack_bf16x2(f[4], f[5]); w.w = pack_bf16x2(f[6], f[7]);
            return w;
        };
        int i = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++i) {
            int e, row0;
            locate(tile, e, row0);
            bool ready = mbar_wait(&ctl->bar_h, i & 1, abort_flag, status) && !*abort_flag;
            // every warp's output pieces of the previous tile have left shared memory
            if (i > 0) ready = mbar_wait(&ctl->bar_done, (i - 1) & 1, abort_flag, status) && ready && !*abort_flag;
            if (!__all_sync(0xffffffffu, ready)) break;      // warp-uniform: tcgen05.ld below is warp-collective
            tc_fence_after();
            // ---- hidden tile: phi, bf16, K-major swizzled [128 x 64] tiles ----
#pragma unroll 1
            for (int g = wsel; g < DE / 64; g += 2) {
                uint32_t v[64];
                tmem_ld32(t_lane + g * 64, v);
                tmem_ld32(t_lane + g * 64 + 32, v + 32);
                tmem_ld_wait();
                float f[64];
#pragma unroll
                for (int q = 0; q < 64; ++q) f[q] = __uint_as_float(v[q]);
                if (b1) {                                    // the expert's bias row of the first layer
                    const uint4* bp = (const uint4*)(b1 + (size_t)e * DE + g * 64);
#pragma unroll
                    for (int q8 = 0; q8 < 8; ++q8) {
                        float bv[8];
                        unpack16<__nv_bfloat16>(bp[q8], bv);
#pragma unroll
                        for (int q = 0; q < 8; ++q) f[8 * q8 + q] += bv[q];
                    }
                }
                if (pre) {
                    uint4* dst = (uint4*)(pre + (size_t)(row0 + trow) * DE + g * 64);
#pragma unroll
                    for (int c = 0; c < 8; ++c) dst[c] = pack8(f + 8 * c);
                }
                act_apply_n<64>(f, act);
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    *(uint4*)(sHid + g * (BM * 128) + trow * 128 + ((c ^ (trow & 7)) << 4)) = pack8(f + 8 * c);
            }
            fence_async_smem();                  // generic-proxy writes -> visible to the tensor core
            tc_fence_before();
            mbar_arrive(&ctl->bar_a);

            // ---- output tile ----
            const bool zr = mbar_wait(&ctl->bar_z, i & 1, abort_flag, status) && !*abort_flag;
            if (!__all_sync(0xffffffffu, zr)) break;
            tc_fence_after();
            const int wrow0 = row0 + quarter * 32;
#pragma unroll 1
            for (int g = wsel; g < d / 64; g += 2) {
                const uint32_t col = g < 4 ? 256 + g * 64 : (g - 4) * 64;
                uint32_t v[64];
                tmem_ld32(t_lane + col, v);
                tmem_ld32(t_lane + col + 32, v + 32);
                tmem_ld_wait();
                if (lane == 0) bulk_wait_read();          // the previous store has finished reading the piece
                __syncwarp();
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float f[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) f[q] = __uint_as_float(v[8 * c + q]);
                    if (b2) {                                // the expert's bias row of the second layer
                        float bv[8];
                        unpack16<__nv_bfloat16>(*(const uint4*)(b2 + (size_t)e * d + g * 64 + 8 * c), bv);
#pragma unroll
                        for (int q = 0; q < 8; ++q) f[q] += bv[q];
                    }
                    *(uint4*)(stg + lane * 128 + ((c ^ (lane & 7)) << 4)) = pack8(f);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { tma_store_2d(&tmZ, stg, g * 64, wrow0); bulk_commit(); }
            }
            if (lane == 0) bulk_wait_read();              // the pieces may be overwritten by the next hidden tile
            __syncwarp();
            tc_fence_before();
            mbar_arrive(&ctl->bar_done);
        }
    }
    if (warp >= 2 && lane == 0) bulk_wait_all();       // this warp's tensor stores are complete
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

bool mlp_can_fuse(const Dims& D) { return D.bf16 && D.d_e == DE && D.d % 64 == 0 && D.d <= 512 && D.n <= 31; }

// A: routed rows [rows_max, d] (or gathered from gather_x through src_patch), W1 [n, d, 256], W2 [n, 256, d],
// z [rows_max, d]; pre (optional) [rows_max, 256] receives the pre-activation; b1 [n, 256], b2 [n, d] optional biases.
uoe_status launch_mlp_fused(const Dims& D, const void* A, const void* W1, const void* W2, void* z, void* pre,
                            const int* offsets, int act, const void* gather_x, const SrcMap& map, int* status,
                            cudaStream_t s, const void* b1, const void* b2) {
    if (!mlp_can_fuse(D) || D.Rmax % BM != 0) return UOE_ERR_UNSUPPORTED;
    if (gather_x && (!map.on() || D.l_p < 8 || D.l_p % 8 != 0 || BM % D.l_p != 0)) return UOE_ERR_INVALID_ARG;
    static DeviceOnce once;
    {
        const uoe_status st = smem_opt_in(once, mlp_fused_kernel, SMEM);
        if (st != UOE_OK) return st;
    }
    CUtensorMap tmA, tmX, tmW1, tmW2, tmZ;
    if (gather_x) {       // x as [Bm patches, l_p rows, d]
        const uint64_t dims[3] = {(uint64_t)D.d, (uint64_t)D.l_p, (uint64_t)D.B * D.m};
        const uint64_t str[2] = {(uint64_t)D.d * 2, (uint64_t)D.d * 2 * D.l_p};
        const uint32_t box[3] = {BK, (uint32_t)D.l_p, 1};
        if (!make_tmap(&tmX, gather_x, 3, dims, str, box)) return UOE_ERR_CUDA;
        tmA = tmX;
    } else {
        const uint64_t dims[2] = {(uint64_t)D.d, (uint64_t)D.Rmax};
        const uint64_t str[1] = {(uint64_t)D.d * 2};
        const uint32_t box[2] = {BK, BM};
        if (!make_tmap(&tmA, A, 2, dims, str, box)) return UOE_ERR_CUDA;
        tmX = tmA;
    }
    {                     // W1 [n, d, 256] and W2 [n, 256, d]: boxes of 64 columns x 64 contraction rows of one expert
        const uint64_t dims1[3] = {(uint64_t)DE, (uint64_t)D.d, (uint64_t)D.n};
        const uint64_t str1[2] = {(uint64_t)DE * 2, (uint64_t)D.d * DE * 2};
        const uint64_t dims2[3] = {(uint64_t)D.d, (uint64_t)DE, (uint64_t)D.n};
        const uint64_t str2[2] = {(uint64_t)D.d * 2, (uint64_t)D.d * DE * 2};
        const uint32_t box[3] = {64, BK, 1};
        if (!make_tmap(&tmW1, W1, 3, dims1, str1, box)) return UOE_ERR_CUDA;
        if (!make_tmap(&tmW2, W2, 3, dims2, str2, box)) return UOE_ERR_CUDA;
    }
    {                     // z as [rows_max, d], written in [32 rows x 64 columns] pieces
        const uint64_t dims[2] = {(uint64_t)D.d, (uint64_t)D.Rmax};
        const uint64_t str[1] = {(uint64_t)D.d * 2};
        const uint32_t box[2] = {64, 32};
        if (!make_tmap(&tmZ, z, 2, dims, str, box)) return UOE_ERR_CUDA;
    }
    const long long max_tiles = D.Rmax / BM;
    int grid = (int)(max_tiles < sm_count() ? max_tiles : sm_count());
    if (grid < 1) grid = 1;
    ProfScope ps("mlp_fused", s);
    launch_k(mlp_fused_kernel, dim3(grid), dim3(THREADS), (size_t)SMEM, s, tmA, tmX, tmW1, tmW2, tmZ, (__nv_bfloat16*)pre, offsets,
             D.n, D.d, act, status, gather_x ? map : SrcMap(), D.l_p, (int)(D.B * D.m), (const __nv_bfloat16*)b1,
             (const __nv_bfloat16*)b2);
    UOE_LAUNCHED();
    return UOE_OK;
}

}  // namespace uoe
