// Per-expert weight gradients on the tcgen05 tensor cores (derivative of Eq. 38-39 with respect to
// A^I_i and A^O_i):   dW[e] [M, N] = P_e^T Q_e,   P_e [rows_e, M], Q_e [rows_e, N] the rows of expert e's
// region in two routed buffers.  The contraction runs over the ragged row count of each expert, so both
// operands are "MN-major" for the MMA: a K step is 64 consecutive rows, each row contributing 128 bytes
// (64 elements) per swizzled box.
//
// Persistent CTAs walk (expert, 128-row tile of M, BN-column tile of N); warp roles and the two-buffer
// TMEM accumulator are the same as in the forward grouped GEMM.  The output is float32 and overwritten
// (each epilogue warp stages [32 rows x 32 columns] in swizzled shared memory and issues one TMA tensor
// store); an expert with no rows gets zeros.
// A tile's cost is its expert's row count, so the tile list is ordered by descending row count and handed out
// longest first: a CTA's first tile is its own index, every further one comes from a counter in the workspace's
// control block that the producer warp advances when it is ready for more work (greedy list scheduling: the CTAs
// finish within one cheap tile of each other whatever the load skew).  Which CTA computes a tile varies from run to
// run; the result does not, because every output tile is computed whole, in a fixed K order, by one CTA.  The last
// CTA to finish leaves the counters at zero for the next launch.
#include "kernels.cuh"
#include "tc.cuh"
#include "tmap.cuh"

namespace uoe {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64;
constexpr int A_BLOCK_BYTES = BM * BK * 2;
constexpr int kSchedSlots = 4;       // tiles the producer may run ahead of the slowest consumer
constexpr int kSchedWord = 64;       // words [64, 66) of the workspace's control block: next tile, CTAs finished

// MT = 2: 256 x BN output tiles (two 128-row accumulators fed by the same Q stage), one accumulator set
// drained by eight epilogue warps; MT = 1: 128 x BN tiles with two accumulator sets.
template <int BN, int MT> struct WCfg {
    static constexpr int A_BYTES = MT * A_BLOCK_BYTES;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE = A_BYTES + B_BYTES;
    static constexpr int STAGES = (MT == 2) ? 3 : ((BN == 256) ? 4 : (BN == 128 ? 6 : 8));
    static constexpr int NACC = (MT == 2) ? 1 : 2;
    static constexpr int TMEM_COLS = 2 * BN;
    static constexpr int EPI_WARPS = 4 * MT;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr int STG_BYTES = 32 * 128;
    static constexpr int SMEM = STAGES * STAGE + 1024 + 1024 + EPI_WARPS * STG_BYTES;
};

struct WCtl {
    uint64_t full[8], empty[8], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort_flag;
    int offs[34];
    int perm[32];                  // experts by descending row count
    uint64_t sfull[kSchedSlots], sempty[kSchedSlots];
    int sched_tile[kSchedSlots];   // tiles handed from the producer warp to the MMA thread and the epilogue warps
};

template <int BN, int MT>
__global__ void __launch_bounds__(WCfg<BN, MT>::THREADS, 1)
wgrad_kernel(const __grid_constant__ CUtensorMap tmP, const __grid_constant__ CUtensorMap tmQ,
             const __grid_constant__ CUtensorMap tmW, const int* __restrict__ offsets, int n, int M, int N,
             int ksplit, int* status, int gather_p, int gather_q, const int* __restrict__ src_patch, int l_p, int Bm,
             int* __restrict__ sched /* [2], zero between launches */) {
    pdl_trigger();
    using Cf = WCfg<BN, MT>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    WCtl* ctl = (WCtl*)(smem + Cf::STAGES * Cf::STAGE);
    volatile int* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cf::STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], 32 * Cf::EPI_WARPS); }
        for (int q = 0; q < kSchedSlots; ++q) { mbar_init(&ctl->sfull[q], 1); mbar_init(&ctl->sempty[q], 1 + Cf::EPI_WARPS); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmP);
        prefetch_tmap(&tmQ);
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, Cf::TMEM_COLS);
    pdl_wait();                     // everything above touches only this CTA's own resources
    if (warp == 2) {               // offsets, and the experts ranked by row count (n <= 32)
        const int o = offsets[min(lane, n)], o1 = offsets[min(lane + 1, n)];
        const int rows = lane < n ? o1 - o : -1;
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const int rj = __shfl_sync(0xffffffffu, rows, j);
            rank += (rj > rows || (rj == rows && j < lane)) ? 1 : 0;
        }
        if (lane < n) { ctl->offs[lane] = o; ctl->perm[rank] = lane; }
        if (lane == n - 1) ctl->offs[n] = o1;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    constexpr int TM = MT * BM;
    const int m_tiles = M / TM, n_tiles = N / BN;
    const int per_expert = m_tiles * n_tiles;
    const int total_tiles = n * per_expert * ksplit;
    // tile -> expert, output tile, and the slice [kb_lo, kb_lo + kb_cnt) of the expert's 64-row K blocks that split
    // `ks` of the contraction covers (ksplit = 1: all of them); split ks writes its own copy of the output
    auto decode = [&](int tile, int& e, int& m0, int& n0, int& ks, int& kb_lo, int& kb_cnt) {
        ks = tile % ksplit;
        const int t2 = tile / ksplit;
        e = ctl->perm[t2 / per_expert];
        const int rem = t2 % per_expert;
        m0 = (rem / n_tiles) * TM;
        n0 = (rem % n_tiles) * BN;
        const int num_kb = (ctl->offs[e + 1] - ctl->offs[e]) / BK;
        const int per = (num_kb + ksplit - 1) / ksplit;
        kb_lo = ks * per;
        kb_cnt = max(0, min(num_kb, kb_lo + per) - kb_lo);
    };

    // Consumer side of the tile hand-off (one thread per consumer warp calls it): the next tile of this CTA, or a value
    // >= total_tiles when there is none (also after a wait ran out).
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
        // TMA producer: lane 0 runs the pipeline, the 64-wide boxes are issued one per lane
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_parity = 0;
        bool stop = false;
        const int sub_rows = (gather_p || gather_q) ? min(l_p, BK) : BK, nsub = BK / sub_rows;
        // Source patches of a gathered operand: l_p is a power of two that divides 128, so the slab `sub` of K block kb
        // of a region that starts at routed row r0 lies in routed patch r0 / l_p + (64 kb + sub_rows sub) / l_p.  The
        // warp keeps a window of 32 consecutive entries of src_patch in its lanes and reads them with a shuffle: a
        // look-up in global memory in front of every copy would set the pace of the whole ring.
        const int lp_shift = __ffs(l_p) - 1;
        const int my_sub = nsub == 1 ? 0 : (lane & 15) % nsub;
        const bool gathers = gather_p || gather_q;
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
            int e, m0, n0, ks, kb_lo, num_kb;
            decode(tile, e, m0, n0, ks, kb_lo, num_kb);
            const int r0 = ctl->offs[e] + kb_lo * BK;
            const int patch_end = gathers ? (r0 + num_kb * BK + l_p - 1) >> lp_shift : 0;     // routed patches of this tile's rows
            int win0 = r0 >> lp_shift;
            int win = (gathers && win0 + lane < patch_end) ? src_patch[win0 + lane] : 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                int src = 0, prow = 0;
                if (gathers) {
                    const int row = r0 + kb * BK;
                    if (((row + BK - 1) >> lp_shift) >= win0 + 32) {      // (uniform) the block's last slab is past the window
                        win0 = row >> lp_shift;
                        win = win0 + lane < patch_end ? src_patch[win0 + lane] : 0;
                    }
                    src = __shfl_sync(0xffffffffu, win, (((row + my_sub * sub_rows) >> lp_shift) - win0) & 31);
                    if (src < 0) src = Bm;                                // no patch: the zero-filled box past the end
                    prow = (row + my_sub * sub_rows) & (l_p - 1);
                }
                int ok = 1;
                if (lane == 0) ok = (mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag, status) && !*abort_flag) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { stop = true; break; }
                uint8_t* sa = smem + stage * Cf::STAGE;
                uint8_t* sb = sa + Cf::A_BYTES;
                if (lane == 0) mbar_arrive_expect_tx(&ctl->full[stage], Cf::STAGE);
                __syncwarp();
                // An operand is a tensor of [column blocks of 64][rows][64 columns], so one copy brings all the column
                // blocks of a stage (the pace of this loop is set by the number of copies it issues, not by their bytes).
                // A gathered operand (Eq. 18 inside the contraction) comes from the source tensor
                // [Bm patches][column blocks][l_p rows][64]: the 64 routed rows of a K block are 64 / sub_rows slabs of
                // sub_rows rows, each inside one patch; with one slab it is one copy as well, with more the boxes are one
                // column block wide and lane (block, slab) issues its own.
                const int row = r0 + kb * BK;
                if (lane < 16) {
                    if (!gather_p) {
                        if (lane == 0) tma_load_3d(sa, &tmP, 0, row, m0 / 64, &ctl->full[stage]);
                    } else if (lane < (nsub == 1 ? 1 : (TM / 64) * nsub)) {
                        const int cb = nsub == 1 ? 0 : lane / nsub;
                        tma_load_4d(sa + cb * 8192 + my_sub * sub_rows * 128, &tmP, 0, prow, m0 / 64 + cb, src, &ctl->full[stage]);
                    }
                } else {
                    const int l2 = lane - 16;
                    if (!gather_q) {
                        if (l2 == 0) tma_load_3d(sb, &tmQ, 0, row, n0 / 64, &ctl->full[stage]);
                    } else if (l2 < (nsub == 1 ? 1 : (BN / 64) * nsub)) {
                        const int cb = nsub == 1 ? 0 : l2 / nsub;
                        tma_load_4d(sb + cb * 8192 + my_sub * sub_rows * 128, &tmQ, 0, prow, n0 / 64 + cb, src, &ctl->full[stage]);
                    }
                }
                issued |= 1u << stage;
                issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                if (++stage == Cf::STAGES) { stage = 0; phase ^= 1; }
            }
        }
        if (lane == 0 && *abort_flag) {
            for (int s = 0; s < Cf::STAGES; ++s)
                if (issued & (1u << s)) mbar_wait(&ctl->full[s], (issued_parity >> s) & 1, abort_flag, status);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_bf16(BM, BN, true, true);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool stop = false;
            int slot = 0;
            uint32_t sphase = 0;
            while (!stop) {
                const int tile = next_tile(slot, sphase);
                if (tile >= total_tiles) break;
                int e, m0, n0, ks, kb_lo, num_kb;
                decode(tile, e, m0, n0, ks, kb_lo, num_kb);
                if (!mbar_wait(&ctl->tempty[acc], acc_phase ^ 1, abort_flag, status) || *abort_flag) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&ctl->full[stage], phase, abort_flag, status) || *abort_flag) { stop = true; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + stage * Cf::STAGE);
                    const uint32_t sb = sa + Cf::A_BYTES;
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks) {
                        const uint64_t bd = smem_desc(sb + ks * 2048, 8192, 1024);
#pragma unroll
                        for (int h = 0; h < MT; ++h)
                            mma_bf16(d_tmem + h * BN, smem_desc(sa + h * A_BLOCK_BYTES + ks * 2048, 8192, 1024), bd, idesc,
                                     (kb | ks) != 0);
                    }
                    mma_commit(&ctl->empty[stage]);
                    if (++stage == Cf::STAGES) { stage = 0; phase ^= 1; }
                }
                if (stop) break;
                mma_commit(&ctl->tfull[acc]);
                if (++acc == Cf::NACC) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        int acc = 0;
        uint32_t acc_phase = 0;
        int slot = 0;
        uint32_t sphase = 0;
        for (;;) {
            int tile = 0;
            if (lane == 0) tile = next_tile(slot, sphase);
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (tile >= total_tiles) break;
            int e, m0, n0, ks, kb_lo, num_kb;
            decode(tile, e, m0, n0, ks, kb_lo, num_kb);
            const bool ready = mbar_wait(&ctl->tfull[acc], acc_phase, abort_flag, status) && !*abort_flag;
            if (!__all_sync(0xffffffffu, ready)) break;
            tc_fence_after();
            const int wrow0 = (ks * n + e) * M + m0 + half * BM + quarter * 32;   // first row of this warp's piece in [ksplit*n*M, N]
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (MT == 2 ? half * BN : acc * BN);
            uint8_t* stg = smem + Cf::STAGES * Cf::STAGE + 1024 + (warp - 2) * Cf::STG_BYTES;
            // the TMEM read of the next piece is in flight while this one is staged and stored
            uint32_t v[32];
            if (num_kb > 0) {
                tmem_ld32(taddr, v);
            } else {
#pragma unroll
                for (int q = 0; q < 32; ++q) v[q] = 0u;
            }
#pragma unroll 1
            for (int ch = 0; ch < BN / 32; ++ch) {
                if (num_kb > 0) tmem_ld_wait();
                if (lane == 0) bulk_wait_read();      // the previous store has finished reading the piece
                __syncwarp();
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *(uint4*)(stg + lane * 128 + ((q ^ (lane & 7)) << 4)) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                if (num_kb > 0 && ch + 1 < BN / 32) tmem_ld32(taddr + (ch + 1) * 32, v);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { tma_store_2d(&tmW, stg, n0 + ch * 32, wrow0); bulk_commit(); }
            }
            tc_fence_before();
            mbar_arrive(&ctl->tempty[acc]);
            if (++acc == Cf::NACC) { acc = 0; acc_phase ^= 1; }
        }
    }
    if (warp >= 2 && lane == 0) bulk_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, Cf::TMEM_COLS);
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

// dW = sum over the K splits of their partial outputs, ascending split order.  float4 pieces.
__global__ void __launch_bounds__(256)
wgrad_reduce_kernel(const float4* __restrict__ part, float4* __restrict__ dW, long long vecs, int ksplit) {
    pdl_trigger();
    pdl_wait();
    for (long long q = (long long)blockIdx.x * 256 + threadIdx.x; q < vecs; q += (long long)gridDim.x * 256) {
        float4 a = part[q];
        for (int s = 1; s < ksplit; ++s) {
            const float4 t = part[(long long)s * vecs + q];
            a.x += t.x; a.y += t.y; a.z += t.z; a.w += t.w;
        }
        dW[q] = a;
    }
}

template <int BN, int MT>
uoe_status launch_w(const void* P, const void* Q, float* dW, const int* offsets, int n, int M, int N,
                    long long rows_max, const char* label, int* status, cudaStream_t s, int ksplit, float* part,
                    const WgradGather& g) {
    using Cf = WCfg<BN, MT>;
    static DeviceOnce once;
    auto kern = wgrad_kernel<BN, MT>;
    {
        const uoe_status st = smem_opt_in(once, kern, Cf::SMEM);
        if (st != UOE_OK) return st;
    }
    // operands as [column blocks of 64][rows][64 columns]; a gathered one as [Bm patches][column blocks][l_p rows][64]
    CUtensorMap tmP, tmQ;
    const int sub_rows = g.l_p < BK ? g.l_p : BK;
    auto operand_map = [&](CUtensorMap* tm, const void* base, int cols, int tile_cols, bool gathered) {
        if (gathered) {
            const uint64_t dims[4] = {64, (uint64_t)g.l_p, (uint64_t)cols / 64, (uint64_t)g.Bm};
            const uint64_t str[3] = {(uint64_t)cols * 2, 128, (uint64_t)cols * 2 * g.l_p};
            const uint32_t box[4] = {64, (uint32_t)sub_rows, (uint32_t)(sub_rows == BK ? tile_cols / 64 : 1), 1};
            return make_tmap(tm, base, 4, dims, str, box);
        }
        const uint64_t dims[3] = {64, (uint64_t)rows_max, (uint64_t)cols / 64};
        const uint64_t str[2] = {(uint64_t)cols * 2, 128};
        const uint32_t box[3] = {64, BK, (uint32_t)tile_cols / 64};
        return make_tmap(tm, base, 3, dims, str, box);
    };
    if (!operand_map(&tmP, P, M, MT * BM, g.gather_p) || !operand_map(&tmQ, Q, N, BN, g.gather_q)) return UOE_ERR_CUDA;
    CUtensorMap tmW;      // the output (or the per-split partial outputs) as [ksplit*n*M, N] float32, [32 x 32] pieces
    {
        const uint64_t dims[2] = {(uint64_t)N, (uint64_t)ksplit * n * M};
        const uint64_t str[1] = {(uint64_t)N * 4};
        const uint32_t wbox[2] = {32, 32};
        if (!make_tmap(&tmW, ksplit > 1 ? part : dW, 2, dims, str, wbox, CU_TENSOR_MAP_DATA_TYPE_FLOAT32)) return UOE_ERR_CUDA;
    }
    const long long tiles = (long long)n * (M / (MT * BM)) * (N / BN) * ksplit;
    int grid = (int)(tiles < sm_count() ? tiles : sm_count());
    ProfScope ps(label, s);
    launch_k(kern, grid, dim3(Cf::THREADS), Cf::SMEM, s, tmP, tmQ, tmW, offsets, n, M, N, ksplit, status, g.gather_p ? 1 : 0,
             g.gather_q ? 1 : 0, g.src_patch, g.l_p, g.Bm, status + kSchedWord);
    UOE_LAUNCHED();
    if (ksplit > 1) {
        const long long vecs = (long long)n * M * N / 4;
        launch_k(wgrad_reduce_kernel, dim3((unsigned)((vecs + 255) / 256 < 1184 ? (vecs + 255) / 256 : 1184)), dim3(256), 0, s,
                 (const float4*)part, (float4*)dW, vecs, ksplit);
        UOE_LAUNCHED();
    }
    return UOE_OK;
}

}  // namespace

// How many ways the contraction is split: weight gradients with few output tiles (small M x N per expert) leave most
// SMs idle and give each busy one a long serial K loop, so their rows are split across CTAs into partial outputs
// that a second kernel adds in a fixed order.  1 = no split.
int wgrad_ksplit(int n, int M, int N, long long rows_max) {
    const int bn = gemm_bf16_bn(N);
    const long long tiles = (long long)n * (M / BM) * (N / bn);
    if (tiles < 1 || n < 1 || tiles >= sm_count()) return 1;      // (shapes the kernel does not cover are refused later)
    long long ks = (2ll * sm_count() + tiles - 1) / tiles;
    const long long avg_kb = rows_max / ((long long)n * BK);        // 64-row K blocks per expert on average
    if (ks > avg_kb / 4) ks = avg_kb / 4;                            // at least four K blocks per split
    if (ks > 32) ks = 32;
    return ks < 2 ? 1 : (int)ks;
}

size_t wgrad_scratch_bytes(int n, int M, int N, long long rows_max) {
    const int ks = wgrad_ksplit(n, M, N, rows_max);
    return ks > 1 ? (size_t)ks * n * M * N * sizeof(float) : 0;
}

uoe_status launch_wgrad_bf16(const void* P, const void* Q, float* dW, const int* offsets, int n, int M, int N,
                             long long rows_max, const char* label, int* status, cudaStream_t s, float* part,
                             const WgradGather& g) {
    if (!status) return UOE_ERR_INVALID_ARG;       // the tile counters live in the control block behind the status word
    if (M % BM != 0 || N % 64 != 0 || n > 32) return UOE_ERR_UNSUPPORTED;
    if ((g.gather_p || g.gather_q) && (!g.src_patch || !wgrad_can_gather(g.l_p))) return UOE_ERR_INVALID_ARG;
    const int bn = gemm_bf16_bn(N);
    const int ks = part ? wgrad_ksplit(n, M, N, rows_max) : 1;
    // 256-row output tiles when the weight matrices are large enough to keep every SM busy with them
    if (bn == 256 && M % 256 == 0 && (long long)n * (M / 256) * (N / 256) >= 2 * sm_count())
        return launch_w<256, 2>(P, Q, dW, offsets, n, M, N, rows_max, label, status, s, 1, nullptr, g);
    if (bn == 256) return launch_w<256, 1>(P, Q, dW, offsets, n, M, N, rows_max, label, status, s, ks, part, g);
    if (bn == 128) return launch_w<128, 1>(P, Q, dW, offsets, n, M, N, rows_max, label, status, s, ks, part, g);
    return launch_w<64, 1>(P, Q, dW, offsets, n, M, N, rows_max, label, status, s, ks, part, g);
}

}  // namespace uoe
