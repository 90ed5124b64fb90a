// Second expert layer and combine in one kernel, walked by output patch (Eq. 39-40), for patches of exactly 128 tokens:
//
//   y[b, 128 j + r, :] = x[b, 128 j + r, :] + sum over the experts i that selected patch j of  a'_i[row_i + r, :] @ W2[i]
//
// where a' = gate * phi(h) is what the first layer wrote (the product is linear in it, so the combine weight of Eq. 40
// is applied there, one value per 128-row block) and row_i is the first routed row of the patch in expert i's region
// (the plan's inverse map).  A 128-row GEMM tile is one patch, so the CTA that owns output tile (patch, 256 columns)
// runs the K loops of all selecting experts into one TMEM accumulator, in ascending slot order, adds x in the epilogue
// and stores y: the per-expert outputs z never reach memory and the sum over experts stays in float32.  Pad tokens and
// patches nobody selected get y = x (or 0 without the residual).
// The backward uses the same kernel for dx (derivative of Eq. 38 and 40): a' is dh (the gate is inside it), the weights
// are W1 read K-major ([n, d, d_e]: dx_g = dh W1^T), x is dy, and the router's per-patch vector is added on real tokens.
// A tile costs as many K loops as its patch has experts (none to k), so the tiles are handed out as the CTAs get to
// them: a CTA's first tile is its own index, every further one comes from a counter in the workspace's control block
// that the producer warp advances (which CTA computes a tile varies from run to run; the result does not, every tile
// being computed whole, in a fixed order, by one CTA).  The last CTA to finish leaves the counters at zero.
//   warp 0      TMA producer: per 64-wide K step an A block [128 x 64] of a' and a W2 block [64 x 256] (one box each)
//   warp 1      MMA issuer: tcgen05.mma 128 x 256 x 16, two accumulator sets (the epilogue of a tile runs under the
//               next tile's main loop)
//   warps 2-9   epilogue, two per TMEM lane quarter, 128 columns each: accumulator + x -> bf16 -> swizzled staging ->
//               TMA tensor stores
#include "kernels.cuh"
#include "tc.cuh"
#include "tmap.cuh"

namespace uoe {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64, BN = 256;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE = A_BYTES + B_BYTES;
constexpr int STAGES = 4;
constexpr int EPI_WARPS = 8, THREADS = 64 + 32 * EPI_WARPS, STG_BYTES = 32 * 128;
constexpr int SMEM = STAGES * STAGE + 1024 + 1024 + EPI_WARPS * STG_BYTES;
constexpr int KMAX = 8;            // experts per sample this kernel handles
constexpr int kSchedSlots = 4;     // tiles the producer may run ahead of the slowest consumer
constexpr int kSchedWord = 64;     // words [64, 66) of the workspace's control block: next tile, CTAs finished (zero between launches)

struct PCtl {
    uint64_t full[STAGES], empty[STAGES], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort_flag;
    int offs[34];
    uint64_t sfull[kSchedSlots], sempty[kSchedSlots];
    int sched_tile[kSchedSlots];   // tiles handed from the producer warp to the MMA thread and the epilogue warps
};

template <bool B_KMAJOR>
__global__ void __launch_bounds__(THREADS, 1)
gemm2_patch_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const __grid_constant__ CUtensorMap tmY, const __nv_bfloat16* __restrict__ x,
                   const int* __restrict__ inv_row, const int* __restrict__ pair_row, int inv_relative,
                   const int* __restrict__ offsets, int n, int Bm, int m, int k, int K, int N, int Lv, int residual,
                   int* status, int* __restrict__ sched /* [2], zero between launches */,
                   const float* __restrict__ rvec /* [patches, N] added on real tokens, or null */) {
    pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    PCtl* ctl = (PCtl*)(smem + STAGES * STAGE);
    volatile int* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], 32 * EPI_WARPS); }
        for (int q = 0; q < kSchedSlots; ++q) { mbar_init(&ctl->sfull[q], 1); mbar_init(&ctl->sempty[q], 1 + EPI_WARPS); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        prefetch_tmap(&tmY);
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, 2 * BN);
    pdl_wait();                     // everything above touches only this CTA's own resources
    if (warp == 2 && lane <= n) ctl->offs[lane] = offsets[lane];
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    const int n_tiles = N / BN, kb_per = K / BK;
    const int total_tiles = Bm * n_tiles;           // column tiles of a patch are adjacent: its A blocks are read from L2
    // first routed row of patch p in slot s, or -1
    auto row_of = [&](int p, int s) {
        int r = inv_row[(size_t)p * k + s];
        if (r >= 0 && inv_relative) r += pair_row[(p / m) * k + s];
        return r;
    };

    // consumer side of the tile hand-off (one thread per consumer warp): this CTA's next tile, or >= total_tiles at the end
    auto next_tile = [&](int& slot, uint32_t& sphase) {
        int tile = total_tiles;
        if (mbar_wait(&ctl->sfull[slot], sphase, abort_flag, status) && !*abort_flag) {
            tile = ctl->sched_tile[slot];
            mbar_arrive(&ctl->sempty[slot]);
        }
        if (++slot == kSchedSlots) { slot = 0; sphase ^= 1; }
        return tile;
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_parity = 0;
        bool stop = false;
        int slot = 0;
        uint32_t sphase = 0;
        for (bool first = true; !stop; first = false) {
            int tile = total_tiles;
            if (lane == 0) {       // hand the next tile (or the end marker) to the consumers
                if (mbar_wait(&ctl->sempty[slot], sphase ^ 1, abort_flag, status) && !*abort_flag) {
                    tile = first ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(sched, 1);
                    if (tile > total_tiles) tile = total_tiles;
                }
                ctl->sched_tile[slot] = tile;
                mbar_arrive(&ctl->sfull[slot]);
            }
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (++slot == kSchedSlots) { slot = 0; sphase ^= 1; }
            if (tile >= total_tiles) break;
            const int p = tile / n_tiles, n0 = (tile % n_tiles) * BN;
            int rows[KMAX];
#pragma unroll
            for (int s = 0; s < KMAX; ++s) rows[s] = s < k ? row_of(p, s) : -1;
#pragma unroll
            for (int s = 0; s < KMAX; ++s) {
                if (rows[s] < 0 || stop) continue;
                int e = 0;                                  // the expert whose region holds the rows
                while (e + 1 < n && rows[s] >= ctl->offs[e + 1]) ++e;
                for (int kb = 0; kb < kb_per; ++kb) {
                    int ok = 1;
                    if (lane == 0) ok = (mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag, status) && !*abort_flag) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { stop = true; break; }
                    uint8_t* sa = smem + stage * STAGE;
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&ctl->full[stage], STAGE);
                        tma_load_2d(sa, &tmA, kb * BK, rows[s], &ctl->full[stage]);
                        if (B_KMAJOR) tma_load_3d(sa + A_BYTES, &tmB, kb * BK, n0, e, &ctl->full[stage]);
                        else tma_load_4d(sa + A_BYTES, &tmB, 0, kb * BK, n0 / 64, e, &ctl->full[stage]);
                    }
                    issued |= 1u << stage;
                    issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
        if (lane == 0 && *abort_flag) {      // let this CTA's own copies land before it exits
            for (int s = 0; s < STAGES; ++s)
                if (issued & (1u << s)) mbar_wait(&ctl->full[s], (issued_parity >> s) & 1, abort_flag, status);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            constexpr uint32_t idesc = instr_desc_bf16(BM, BN, false, !B_KMAJOR);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool stop = false;
            int slot = 0;
            uint32_t sphase = 0;
            while (!stop) {
                const int tile = next_tile(slot, sphase);
                if (tile >= total_tiles) break;
                const int p = tile / n_tiles;
                int cnt = 0;
                for (int s = 0; s < k; ++s) cnt += inv_row[(size_t)p * k + s] >= 0 ? 1 : 0;
                if (!mbar_wait(&ctl->tempty[acc], acc_phase ^ 1, abort_flag, status) || *abort_flag) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                const int steps = cnt * kb_per;
                for (int i = 0; i < steps; ++i) {
                    if (!mbar_wait(&ctl->full[stage], phase, abort_flag, status) || *abort_flag) { stop = true; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + stage * STAGE), sb = sa + A_BYTES;
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks)
                        mma_bf16(d_tmem, smem_desc(sa + ks * 32, 16, 1024),
                                 B_KMAJOR ? smem_desc(sb + ks * 32, 16, 1024) : smem_desc(sb + ks * 2048, 8192, 1024), idesc, (i | ks) != 0);
                    mma_commit(&ctl->empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (stop) break;
                mma_commit(&ctl->tfull[acc]);          // (no MMA issued for a patch nobody selected: arrives at once)
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ---------------- epilogue ----------------
        const int quarter = warp & 3, wsel = (warp - 2) >> 2;
        int acc = 0;
        uint32_t acc_phase = 0;
        uint8_t* stg = smem + STAGES * STAGE + 1024 + (warp - 2) * STG_BYTES;
        int slot = 0;
        uint32_t sphase = 0;
        for (;;) {
            int tile = 0;
            if (lane == 0) tile = next_tile(slot, sphase);
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (tile >= total_tiles) break;
            const int p = tile / n_tiles, n0 = (tile % n_tiles) * BN;
            int cnt = 0;
            for (int s = 0; s < k; ++s) cnt += inv_row[(size_t)p * k + s] >= 0 ? 1 : 0;
            const bool ready = mbar_wait(&ctl->tfull[acc], acc_phase, abort_flag, status) && !*abort_flag;
            if (!__all_sync(0xffffffffu, ready)) break;      // warp-uniform: tcgen05.ld below is warp-collective
            tc_fence_after();
            const int r = quarter * 32 + lane;
            const bool real = (p % m) * BM + r < Lv;         // a real token (pad tokens: y = x)
            const size_t grow = (size_t)p * BM + r;          // row of x and y
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
#pragma unroll 1
            for (int g = wsel * 2; g < wsel * 2 + 2; ++g) {
                float f[64];
                if (cnt > 0) {
                    uint32_t v[64];
                    tmem_ld32(taddr + g * 64, v);
                    tmem_ld32(taddr + g * 64 + 32, v + 32);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 64; ++q) f[q] = real ? __uint_as_float(v[q]) : 0.f;
                } else {
#pragma unroll
                    for (int q = 0; q < 64; ++q) f[q] = 0.f;
                }
                if (rvec && real) {
                    const float4* rp = (const float4*)(rvec + (size_t)p * N + n0 + g * 64);
#pragma unroll
                    for (int q4 = 0; q4 < 16; ++q4) {
                        const float4 rq = rp[q4];
                        f[4 * q4] += rq.x; f[4 * q4 + 1] += rq.y; f[4 * q4 + 2] += rq.z; f[4 * q4 + 3] += rq.w;
                    }
                }
                if (residual) {
                    const uint4* xp = (const uint4*)(x + grow * N + n0 + g * 64);
#pragma unroll
                    for (int q8 = 0; q8 < 8; ++q8) {
                        float xv[8];
                        unpack16<__nv_bfloat16>(xp[q8], xv);
#pragma unroll
                        for (int q = 0; q < 8; ++q) f[8 * q8 + q] += xv[q];
                    }
                }
                if (lane == 0) bulk_wait_read();          // the previous store has finished reading the piece
                __syncwarp();
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {
                    uint4 w;
                    w.x = pack_bf16x2(f[8 * c8], f[8 * c8 + 1]); w.y = pack_bf16x2(f[8 * c8 + 2], f[8 * c8 + 3]);
                    w.z = pack_bf16x2(f[8 * c8 + 4], f[8 * c8 + 5]); w.w = pack_bf16x2(f[8 * c8 + 6], f[8 * c8 + 7]);
                    *(uint4*)(stg + lane * 128 + ((c8 ^ (lane & 7)) << 4)) = w;
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { tma_store_2d(&tmY, stg, n0 + g * 64, p * BM + quarter * 32); bulk_commit(); }
            }
            tc_fence_before();
            mbar_arrive(&ctl->tempty[acc]);
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
    }
    if (warp >= 2 && lane == 0) bulk_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, 2 * BN);
    }
    if (threadIdx.x == 0) {         // this CTA's last fetch lies before the barrier above: the last CTA to get here resets
        __threadfence();
        if (atomicAdd(sched + 1, 1) == (int)gridDim.x - 1) {
            sched[0] = 0;
            sched[1] = 0;
            __threadfence();
        }
    }
}

// blk[r / 128] = combine weight of the 128-row block that starts at routed row r, for every selected (patch, slot)
__global__ void __launch_bounds__(256)
block_gate_kernel(const int* __restrict__ inv_row, const float* __restrict__ inv_gate, const int* __restrict__ pair_row,
                  int inv_relative, int total, int k, int m, int use_gate, float* __restrict__ blk) {
    pdl_trigger();
    pdl_wait();
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx >= total) return;
    int r = inv_row[idx];
    if (r < 0) return;
    if (inv_relative) r += pair_row[(idx / k / m) * k + idx % k];
    blk[r >> 7] = use_gate ? inv_gate[idx] : 1.0f;
}

}  // namespace

bool gemm2_patch_can(const Dims& D, const PlanPtrs& P, const void* b2) {
    return D.bf16 && D.l_p == BM && D.d % BN == 0 && D.d_e % BK == 0 && D.k <= KMAX && D.n <= 32 && !b2 && P.inv_row &&
           P.inv_gate && !P.identity_patches && (!P.inv_relative || P.pair_row);
}

uoe_status launch_block_gate(const Dims& D, const PlanPtrs& P, bool use_gate, float* blk, cudaStream_t s) {
    const int total = D.B * D.m * D.k;
    ProfScope ps("block_gate", s);
    launch_k(block_gate_kernel, dim3((total + 255) / 256), dim3(256), 0, s, (const int*)P.inv_row, (const float*)P.inv_gate,
             (const int*)P.pair_row, P.inv_relative ? 1 : 0, total, D.k, D.m, use_gate ? 1 : 0, blk);
    UOE_LAUNCHED();
    return UOE_OK;
}

uoe_status launch_gemm2_patch(const Dims& D, const void* a, const void* W2, const void* x, void* y, const int* offsets,
                              const PlanPtrs& P, bool residual, int* status, cudaStream_t s, bool w_kmajor,
                              const float* rvec, const char* label) {
    if (!status) return UOE_ERR_INVALID_ARG;       // the tile counters live in the control block behind the status word
    static DeviceOnce once[2];
    {
        const uoe_status st = w_kmajor ? smem_opt_in(once[1], gemm2_patch_kernel<true>, SMEM)
                                       : smem_opt_in(once[0], gemm2_patch_kernel<false>, SMEM);
        if (st != UOE_OK) return st;
    }
    CUtensorMap tmA, tmB, tmY;
    {
        const uint64_t dims[2] = {(uint64_t)D.d_e, (uint64_t)D.Rmax};
        const uint64_t str[1] = {(uint64_t)D.d_e * 2};
        const uint32_t box[2] = {BK, BM};
        if (!make_tmap(&tmA, a, 2, dims, str, box)) return UOE_ERR_CUDA;
    }
    if (w_kmajor) {       // W [n, d, d_e]: rows of the output dimension, the contraction contiguous
        const uint64_t dims[3] = {(uint64_t)D.d_e, (uint64_t)D.d, (uint64_t)D.n};
        const uint64_t str[2] = {(uint64_t)D.d_e * 2, (uint64_t)D.d_e * D.d * 2};
        const uint32_t box[3] = {BK, BN, 1};
        if (!make_tmap(&tmB, W2, 3, dims, str, box)) return UOE_ERR_CUDA;
    } else {              // W2 [n, d_e, d] as [n][d/64 column blocks][d_e][64]
        const uint64_t dims[4] = {64, (uint64_t)D.d_e, (uint64_t)D.d / 64, (uint64_t)D.n};
        const uint64_t str[3] = {(uint64_t)D.d * 2, 128, (uint64_t)D.d_e * D.d * 2};
        const uint32_t box[4] = {64, BK, BN / 64, 1};
        if (!make_tmap(&tmB, W2, 4, dims, str, box)) return UOE_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)D.d, (uint64_t)D.B * D.L};
        const uint64_t str[1] = {(uint64_t)D.d * 2};
        const uint32_t box[2] = {64, 32};
        if (!make_tmap(&tmY, y, 2, dims, str, box)) return UOE_ERR_CUDA;
    }
    const long long tiles = (long long)D.B * D.m * (D.d / BN);
    const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
    ProfScope ps(label, s);
    auto go = [&](auto kern) {
        launch_k(kern, dim3(grid), dim3(THREADS), (size_t)SMEM, s, tmA, tmB, tmY, (const __nv_bfloat16*)x,
                 (const int*)P.inv_row, (const int*)P.pair_row, P.inv_relative ? 1 : 0, offsets, D.n, D.B * D.m, D.m, D.k, D.d_e,
                 D.d, D.Lv, residual ? 1 : 0, status, status + kSchedWord, rvec);
    };
    if (w_kmajor) go(gemm2_patch_kernel<true>);
    else go(gemm2_patch_kernel<false>);
    UOE_LAUNCHED();
    return UOE_OK;
}

}  // namespace uoe
