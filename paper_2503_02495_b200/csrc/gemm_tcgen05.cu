// bf16 grouped expert GEMM on the tcgen05 tensor cores (Eq. 19 / 38 / 39: every expert applies its own
// weight slice to the rows routed to it).
//
//   C[r, :] = epilogue( A[r, :] @ W[e(r)] ),  r over the routed rows, e(r) = expert whose region holds r
//
// One persistent CTA per SM walks the (row tile, BN-column tile) list; expert regions are padded to 128
// rows, so a 128-row block never straddles two experts.  Warp roles:
//   warp 0      TMA producer (lane 0 runs the pipeline; boxes of a stage that need separate copies are issued one per
//               lane): A tile [MT*128 x 64] and B tile [64 x BN] per K step into a 128B-swizzled ring
//   warp 1      MMA issuer: tcgen05.mma 128 x BN x 16 into TMEM accumulators
//   warps 2..   epilogue: tcgen05.ld the accumulator (one row per thread), activation, bf16, then a
//               [32 rows x 64 columns] piece per warp staged in swizzled shared memory and written with one
//               TMA tensor store (full 128-byte lines instead of 16-byte scattered stores)
// Three tile shapes:
//   MT = 1  128-row tiles, two TMEM accumulators: the epilogue of tile t overlaps the main loop of tile t+1
//   PAIR    256-row tiles worked by a cluster of two CTAs (tcgen05 cta_group::2): CTA r of the pair loads row block r
//           of A and half r of the B tile's columns, the even CTA issues 256 x BN x 16 MMAs that read both CTAs'
//           shared memory and write 128 rows into each CTA's TMEM.  A third fewer operand bytes per flop than MT = 1,
//           and each CTA still keeps two accumulator sets, so the epilogue runs under the next main loop; one barrier
//           round covers 128 columns of K.  Taken, forward and backward, whenever there are at least two such tiles
//           per SM and K is a multiple of 128.
//   MT = 2  256-row tiles in one CTA (two 128-row accumulators fed by the same B stage): the same operand bytes per
//           flop, but one accumulator set, so the drain of a tile is exposed; left for K that is not a multiple of
//           128.  A 256-row unit at the end of an expert region may hold a single 128-row block ("half tile").
// Every stage is filled by as few copies as its layout allows (one box for a routed A tile, one for a B tile: the
// weights [n, K, N] are mapped as [n][N/64 column blocks][K][64]); only a gathered A needs a box per source patch.
// The A operand is either a routed buffer (2-D tensor map) or gathered on the fly from x, one TMA box per
// source patch (Eq. 18 inside the GEMM).
#include "kernels.cuh"
#include "tc.cuh"
#include "tmap.cuh"

namespace uoe {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64;
constexpr int A_BLOCK_BYTES = BM * BK * 2;     // 16 KB per 128-row block

template <int BN, int MT, bool BWD = false, bool PAIR = false> struct Cfg {
    static_assert(!PAIR || (MT == 1 && BN == 256), "CTA pairs: 128 rows and half of a 256-column B tile per CTA");
    static constexpr int UNIT = PAIR ? 2 : MT;                     // 128-row blocks per row tile
    static constexpr int A_BYTES = MT * A_BLOCK_BYTES;
    static constexpr int B_BYTES = (PAIR ? BN / 2 : BN) * BK * 2;  // per CTA
    static constexpr int KSUB = PAIR ? 2 : 1;                      // 64-wide K blocks per stage (one barrier round)
    static constexpr int SUB = A_BYTES + B_BYTES;
    static constexpr int STAGE = KSUB * SUB;
    static constexpr int STAGES = PAIR ? 3 : (MT == 2) ? 3 : ((BN == 256 || BN == 192) ? 4 : (BN == 128 ? 6 : 8));
    static constexpr int NACC = (MT == 2) ? 1 : 2;                 // accumulator sets in TMEM
    static constexpr int ACC_STRIDE = (BN == 192) ? 256 : BN;      // TMEM columns between the two accumulator sets
    static constexpr int TMEM_COLS = 2 * ACC_STRIDE;               // MT=1: two sets; MT=2: one set of two blocks
    // eight epilogue warps: with 256-row tiles one per (row block, TMEM lane quarter); with 128-row tiles two per lane
    // quarter, each draining half of the columns (the long backward epilogue keeps four: its registers would not fit)
    static constexpr int EPI_WARPS = (MT == 2 || !BWD) ? 8 : 4;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr int STG_BYTES = 32 * 128;                     // one epilogue warp's staging piece
    static constexpr int SMEM = STAGES * STAGE + 1024 /*align slack*/ + 1024 /*barriers, offsets*/ + EPI_WARPS * STG_BYTES;
};

struct Ctl {                       // lives behind the stage ring
    uint64_t full[8], empty[8], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort_flag;
    int offs[34];
    int tstart[34];                // first row tile of each expert (prefix sum), tstart[n] = number of row tiles
};

template <int BN, bool B_KMAJOR, bool BWD, int MT, bool PAIR>
__global__ void __launch_bounds__(Cfg<BN, MT, BWD, PAIR>::THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                 const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
                 __nv_bfloat16* __restrict__ C0, __nv_bfloat16* __restrict__ C1, __nv_bfloat16* __restrict__ C2,
                 __nv_bfloat16* __restrict__ pre, const int* __restrict__ offsets,
                 int n, int K, int N, int nmat, int act, int* status, const __nv_bfloat16* __restrict__ bwd_h,
                 const float* __restrict__ row_gate, const float* __restrict__ row_valid, float* __restrict__ dg_part,
                 const __nv_bfloat16* __restrict__ bias /* [n, N] or null: added before the activation (forward epilogue) */,
                 const float* __restrict__ blk_scale /* [rows / 128] or null: factor on the activated output (forward epilogue) */,
                 const __grid_constant__ CUtensorMap tmX, const SrcMap smap, int l_p, int Bm,
                 const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmC1,
                 const __grid_constant__ CUtensorMap tmC2, const __grid_constant__ CUtensorMap tmPre) {
    pdl_trigger();
    using Cf = Cfg<BN, MT, BWD, PAIR>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    Ctl* ctl = (Ctl*)(smem + Cf::STAGES * Cf::STAGE);
    volatile int* abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = PAIR ? (int)cluster_ctarank() : 0;            // CTA of the pair; rank 0 issues the MMAs
    const int worker = PAIR ? blockIdx.x >> 1 : blockIdx.x;        // index of this CTA (pair) among the tile walkers
    const int workers = PAIR ? gridDim.x >> 1 : gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cf::STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        // (pairs: the epilogue threads of both CTAs arrive on rank 0's barrier)
        for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tfull[a], 1); mbar_init(&ctl->tempty[a], (PAIR ? 2 : 1) * 32 * Cf::EPI_WARPS); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB0);
        prefetch_tmap(&tmX);
        prefetch_tmap(&tmC0);
        if (nmat > 1 || BN == 192) { prefetch_tmap(&tmB1); prefetch_tmap(&tmB2); prefetch_tmap(&tmC1); prefetch_tmap(&tmC2); }
        if (BWD) prefetch_tmap(&tmC1);
    }
    if (warp == 1) {
        if constexpr (PAIR) tmem_alloc_pair(&ctl->tmem_base, Cf::TMEM_COLS);
        else tmem_alloc(&ctl->tmem_base, Cf::TMEM_COLS);
    }
    pdl_wait();                     // everything above touches only this CTA's own resources
    if (warp == 2) {                // offsets and the row-tile prefix over experts (n <= 31 here)
        int o = 0;
        if (lane <= n) o = offsets[lane];
        const int o1 = __shfl_down_sync(0xffffffffu, o, 1);
        const int blocks = lane < n ? (o1 - o) / BM : 0;
        const int tiles = (blocks + Cf::UNIT - 1) / Cf::UNIT;
        int incl = tiles;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += v;
        }
        if (lane <= n) ctl->offs[lane] = o;
        if (lane < n) ctl->tstart[lane] = incl - tiles;
        if (lane == n - 1) ctl->tstart[n] = incl;
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();     // the other CTA's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    // tile index -> (row tile, matrix, column tile); the matrices share the A tile, so they are adjacent
    // BN = 192 is the "three 64-wide matrices side by side" tile: the B stage holds one 64-column box of each of the
    // three weight tensors and the three 64-column pieces of the accumulator go to the three outputs, so the A tile is
    // loaded once for q, k and v
    constexpr bool SIDE3 = BN == 192;
    const int n_tiles_mat = SIDE3 ? 1 : N / BN;
    const int n_tiles = SIDE3 ? 1 : n_tiles_mat * nmat;
    const int num_kb = K / (BK * Cf::KSUB);
    const int total_tiles = ctl->tstart[n] * n_tiles;

    // row tile -> expert, first row, number of 128-row blocks it holds.  A CTA's tiles come in ascending order, so the
    // search starts at the expert of its previous tile (e is carried by the caller, 0 before the first tile).
    auto locate = [&](int row_tile, int& e, int& row0, int& blocks) {
        while (e + 1 < n && row_tile >= ctl->tstart[e + 1]) ++e;
        const int i = row_tile - ctl->tstart[e];
        row0 = ctl->offs[e] + i * (Cf::UNIT * BM);
        blocks = min(Cf::UNIT, (ctl->offs[e + 1] - row0) / BM);
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        uint32_t phase = 0;
        uint32_t issued = 0, issued_parity = 0;      // per stage: a load is in flight with this parity
        bool stop = false;
        constexpr int BN_CTA = PAIR ? BN / 2 : BN;              // B columns this CTA loads
        // one copy per operand and stage wherever the rows of a stage are consecutive in memory: the pace of this loop is
        // set by the number of copies it issues.  W [n, K, N] is mapped as [n][N/64 column blocks][K][64], so a box holds
        // all the column blocks of a tile; the three side-by-side matrices take one copy each.
        constexpr int nbox_b = SIDE3 ? 3 : 1;
        const CUtensorMap* tmB_lane = lane == 0 ? &tmB0 : (lane == 1 ? &tmB1 : &tmB2);
        int e = 0;
        for (int tile = worker; tile < total_tiles && !stop; tile += workers) {
            int row0, blocks;
            locate(tile / n_tiles, e, row0, blocks);
            const int mat = (tile % n_tiles) / n_tiles_mat, col0 = ((tile % n_tiles) % n_tiles_mat) * BN;
            const CUtensorMap* tmB = mat == 0 ? &tmB0 : (mat == 1 ? &tmB1 : &tmB2);
            // pairs: this CTA loads row block `rank` (none if the tile holds one block: its MMA rows are never stored)
            const int my_blocks = PAIR ? (rank < blocks ? 1 : 0) : blocks;
            const int arow0 = row0 + rank * BM;
            const bool gathered = smap.on();
            const int nbox_a = gathered ? my_blocks * (BM / l_p) : (my_blocks > 0 ? 1 : 0);   // <= 32; a routed buffer: one box
            int my_src = 0;                                                     // source patch of this lane's box
            {
                const int bx = PAIR ? lane % 16 : lane;       // (pairs: lanes 16.. copy the round's second sub-block)
                if (gathered && bx < nbox_a) my_src = src_of(smap, arow0 + bx * l_p, e, ctl->offs[e], Bm);
            }
            // (pairs: both CTAs' bytes; a routed buffer's box is always MT blocks high, rows past the tile included)
            const uint32_t stage_bytes = Cf::KSUB * ((gathered || PAIR ? blocks : MT) * A_BLOCK_BYTES + (PAIR ? 2 : 1) * Cf::B_BYTES);
            for (int kb = 0; kb < num_kb; ++kb) {
                int ok = 1;
                if (lane == 0) ok = (mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag, status) && !*abort_flag) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { stop = true; break; }
                uint8_t* sa = smem + stage * Cf::STAGE;
                uint8_t* sb = sa + Cf::A_BYTES;
                if (lane == 0 && rank == 0) mbar_arrive_expect_tx(&ctl->full[stage], stage_bytes);
                __syncwarp();
                if constexpr (PAIR) {
                    const uint32_t full0 = map_to_cta(&ctl->full[stage], 0);    // rank 0's barrier counts both CTAs' bytes
                    const int bcol0 = col0 + rank * BN_CTA;
                    // lane (j, box): sub-block j of the round; the sub-blocks' copies leave in the same instruction
                    {
                        const int j = lane / 16, bx = lane % 16;              // KSUB = 2
                        const int k0 = (kb * Cf::KSUB + j) * BK;
                        uint8_t* sa_j = sa + j * Cf::SUB;
                        uint8_t* sb_j = sa_j + Cf::A_BYTES;
                        if (bx < nbox_a) {
                            if (gathered) tma_load_3d_pair(sa_j + bx * l_p * 128, &tmX, k0, 0, my_src, full0);
                            else tma_load_2d_pair(sa_j, &tmA, k0, arow0, full0);
                        }
                        if (bx == 0) {
                            if (B_KMAJOR) tma_load_3d_pair(sb_j, tmB, k0, bcol0, e, full0);
                            else tma_load_4d_pair(sb_j, tmB, 0, k0, bcol0 / 64, e, full0);
                        }
                    }
                } else {
                    if (lane < nbox_a) {
                        if (gathered) tma_load_3d(sa + lane * l_p * 128, &tmX, kb * BK, 0, my_src, &ctl->full[stage]);
                        else tma_load_2d(sa, &tmA, kb * BK, row0, &ctl->full[stage]);
                    }
                    if (lane < nbox_b) {
                        if (SIDE3) tma_load_4d(sb + lane * 8192, tmB_lane, 0, kb * BK, 0, e, &ctl->full[stage]);
                        else if (B_KMAJOR) tma_load_3d(sb, tmB, kb * BK, col0, e, &ctl->full[stage]);
                        else tma_load_4d(sb, tmB, 0, kb * BK, col0 / 64, e, &ctl->full[stage]);
                    }
                }
                issued |= 1u << stage;
                issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                if (++stage == Cf::STAGES) { stage = 0; phase ^= 1; }
            }
        }
        if (lane == 0 && rank == 0 && *abort_flag) {      // let the copies counted by this CTA's barriers land before it exits
            for (int s = 0; s < Cf::STAGES; ++s)
                if (issued & (1u << s)) mbar_wait(&ctl->full[s], (issued_parity >> s) & 1, abort_flag, status);
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---------------- MMA issuer ----------------
            constexpr uint32_t idesc = instr_desc_bf16(PAIR ? 2 * BM : BM, BN, false, !B_KMAJOR);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool stop = false;
            int e = 0;
            for (int tile = worker; tile < total_tiles && !stop; tile += workers) {
                int row0, blocks;
                locate(tile / n_tiles, e, row0, blocks);
                if (!mbar_wait(&ctl->tempty[acc], acc_phase ^ 1, abort_flag, status) || *abort_flag) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * Cf::ACC_STRIDE;        // MT=2: acc is always 0, block h at column h*BN
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&ctl->full[stage], phase, abort_flag, status) || *abort_flag) { stop = true; break; }
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < Cf::KSUB * (BK / 16); ++ks) {
                        const uint32_t sa = smem_u32(smem + stage * Cf::STAGE + (ks / (BK / 16)) * Cf::SUB);
                        const uint32_t sb = sa + Cf::A_BYTES;
                        const int kq = ks % (BK / 16);
                        const uint64_t bd = B_KMAJOR ? smem_desc(sb + kq * 32, 16, 1024)
                                                     : smem_desc(sb + kq * 2048, 8192, 1024);
                        if constexpr (PAIR) {
                            mma_bf16_pair(d_tmem, smem_desc(sa + kq * 32, 16, 1024), bd, idesc, (kb | ks) != 0);
                        } else {
#pragma unroll
                            for (int h = 0; h < MT; ++h)
                                if (h < blocks)
                                    mma_bf16(d_tmem + h * BN, smem_desc(sa + h * A_BLOCK_BYTES + kq * 32, 16, 1024), bd, idesc,
                                             (kb | ks) != 0);
                        }
                    }
                    if constexpr (PAIR) mma_commit_pair(&ctl->empty[stage]);       // frees the stage in both CTAs
                    else mma_commit(&ctl->empty[stage]);
                    if (++stage == Cf::STAGES) { stage = 0; phase ^= 1; }
                }
                if (stop) break;
                if constexpr (PAIR) mma_commit_pair(&ctl->tfull[acc]);
                else mma_commit(&ctl->tfull[acc]);
                if (++acc == Cf::NACC) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ---------------- epilogue: warp w drains TMEM lane quarter w % 4 of 128-row block (w-2)/4 (256-row tiles) or,
        // with 128-row tiles and eight warps, of column half (w-2)/4 ----------------
        const int quarter = warp & 3;
        const int wsel = (warp - 2) >> 2;
        const int half = PAIR ? rank : (MT == 2 ? wsel : 0);  // 128-row block this warp drains
        constexpr int G = BN / 64;                            // 64-column groups of the accumulator
        constexpr bool SPLIT_COLS = MT == 1 && Cf::EPI_WARPS == 8;
        const int g_lo = SPLIT_COLS ? wsel * ((G + 1) / 2) : 0;
        const int g_hi = SPLIT_COLS ? min(G, g_lo + (G + 1) / 2) : G;
        int acc = 0;
        uint32_t acc_phase = 0;
        auto pack8 = [](const float* f) {
            uint4 w;
            w.x = pack_bf16x2(f[0], f[1]); w.y = pack_bf16x2(f[2], f[3]);
            w.z = pack_bf16x2(f[4], f[5]); w.w = pack_bf16x2(f[6], f[7]);
            return w;
        };
        uint8_t* stg = smem + Cf::STAGES * Cf::STAGE + 1024 + (warp - 2) * Cf::STG_BYTES;
        // 64 values of this thread's row -> bf16 -> this warp's staging piece (row = lane, 128B swizzle) -> TMA store
        auto stage_store = [&](const float* f, const CUtensorMap* tm, int c0, int r0) {
            if (lane == 0) bulk_wait_read();          // the previous store has finished reading the piece
            __syncwarp();
#pragma unroll
            for (int c = 0; c < 8; ++c) *(uint4*)(stg + lane * 128 + ((c ^ (lane & 7)) << 4)) = pack8(f + 8 * c);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) { tma_store_2d(tm, stg, c0, r0); bulk_commit(); }
        };
        int e = 0;
        for (int tile = worker; tile < total_tiles; tile += workers) {
            int row0, blocks;
            locate(tile / n_tiles, e, row0, blocks);
            const int mat = (tile % n_tiles) / n_tiles_mat, col0 = ((tile % n_tiles) % n_tiles_mat) * BN;
            const CUtensorMap* tmC = mat == 0 ? &tmC0 : (mat == 1 ? &tmC1 : &tmC2);
            const bool ready = mbar_wait(&ctl->tfull[acc], acc_phase, abort_flag, status) && !*abort_flag;
            if (!__all_sync(0xffffffffu, ready)) break;      // warp-uniform: tcgen05.ld below is warp-collective
            tc_fence_after();
            if (half < blocks) {
                const int wrow0 = row0 + half * BM + quarter * 32;       // first row of this warp's piece
                const size_t row = (size_t)wrow0 + lane;
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (MT == 2 ? half * BN : acc * Cf::ACC_STRIDE);
                if constexpr (BWD) {
                    const float rg = row_gate[row], rv = row_valid[row];
                    float dsum = 0.f;
#pragma unroll 1
                    for (int g = 0; g < BN / 64; ++g) {
                        uint32_t v[64];
                        tmem_ld32(taddr + g * 64, v);
                        tmem_ld32(taddr + g * 64 + 32, v + 32);
                        const uint4* hp = (const uint4*)(bwd_h + row * N + col0 + g * 64);
                        uint4 hv[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) hv[q] = hp[q];
                        tmem_ld_wait();
                        float dh[64], ag[64];
#pragma unroll
                        for (int q = 0; q < 8; ++q) unpack16<__nv_bfloat16>(hv[q], dh + 8 * q);     // h
                        act_and_deriv_n<64>(dh, ag, dh, act);                                         // ag = phi(h), dh = phi'(h)
#pragma unroll
                        for (int q = 0; q < 64; ++q) {
                            const float u = __uint_as_float(v[q]);
                            dsum = fmaf(u, ag[q], dsum);
                            dh[q] = rg * u * dh[q];
                            ag[q] = rg * ag[q];
                        }
                        stage_store(dh, &tmC0, col0 + g * 64, wrow0);
                        stage_store(ag, &tmC1, col0 + g * 64, wrow0);
                    }
                    dg_part[row * n_tiles_mat + (col0 / BN)] = rv * dsum;
                } else {
#pragma unroll 1
                    for (int g = g_lo; g < g_hi; ++g) {
                        uint32_t v[64];
                        tmem_ld32(taddr + g * 64, v);
                        tmem_ld32(taddr + g * 64 + 32, v + 32);
                        tmem_ld_wait();
                        float f[64];
#pragma unroll
                        for (int q = 0; q < 64; ++q) f[q] = __uint_as_float(v[q]);
                        if (bias) {                                  // the expert's bias row (the in-place bias of the batched product)
                            const uint4* bp = (const uint4*)(bias + (size_t)e * N + (SIDE3 ? 0 : col0) + g * 64);
#pragma unroll
                            for (int q8 = 0; q8 < 8; ++q8) {
                                float bv[8];
                                unpack16<__nv_bfloat16>(bp[q8], bv);
#pragma unroll
                                for (int q = 0; q < 8; ++q) f[8 * q8 + q] += bv[q];
                            }
                        }
                        if (pre) stage_store(f, &tmPre, col0 + g * 64, wrow0);
                        act_apply_n<64>(f, act);
                        if (blk_scale) {
                            const float sc = blk_scale[(row0 + half * BM) >> 7];
#pragma unroll
                            for (int q = 0; q < 64; ++q) f[q] *= sc;
                        }
                        if (SIDE3) stage_store(f, g == 0 ? &tmC0 : (g == 1 ? &tmC1 : &tmC2), 0, wrow0);
                        else stage_store(f, tmC, col0 + g * 64, wrow0);
                    }
                }
            }
            tc_fence_before();
            if constexpr (PAIR) mbar_arrive_cluster(map_to_cta(&ctl->tempty[acc], 0));
            else mbar_arrive(&ctl->tempty[acc]);
            if (++acc == Cf::NACC) { acc = 0; acc_phase ^= 1; }
        }
    }
    if (warp >= 2 && lane == 0) bulk_wait_all();       // this warp's tensor stores are complete
    tc_fence_before();
    __syncthreads();
    // pairs: neither CTA leaves (or gives up its TMEM) while the other may still arrive on its barriers or its MMAs
    // may still read this CTA's shared memory
    if constexpr (PAIR) cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        if constexpr (PAIR) tmem_dealloc_pair(tmem_base, Cf::TMEM_COLS);
        else tmem_dealloc(tmem_base, Cf::TMEM_COLS);
    }
}

template <int BN, bool B_KMAJOR, bool BWD, int MT, bool PAIR = false>
uoe_status launch_one(const GemmArgs& g, int* status, cudaStream_t s) {
    using Cf = Cfg<BN, MT, BWD, PAIR>;
    static DeviceOnce once;
    static DeviceValue pairs_cache;    // CTA pairs that can be resident at once, per device
    auto kern = gemm_bf16_kernel<BN, B_KMAJOR, BWD, MT, PAIR>;
    {
        const uoe_status st = smem_opt_in(once, kern, Cf::SMEM);
        if (st != UOE_OK) return st;
    }
    int max_pairs = 0;
    if (PAIR) {
        const int dev = current_device();
        if (!pairs_cache.has(dev)) {
            int v = 0;
            UOE_CUDA_OK(max_resident_pairs(kern, Cf::THREADS, Cf::SMEM, &v));
            if (v < 1) return UOE_ERR_CUDA;
            pairs_cache.set(dev, v);
        }
        max_pairs = pairs_cache.get(dev);
    }
    CUtensorMap tmA, tmB[3], tmX;
    if (g.gather_x) {     // x as [Bm patches, l_p rows, K]; the 2-D map of A is unused
        const uint64_t dims[3] = {(uint64_t)g.K, (uint64_t)g.l_p, (uint64_t)g.Bm};
        const uint64_t str[2] = {(uint64_t)g.K * 2, (uint64_t)g.K * 2 * g.l_p};
        const uint32_t box[3] = {BK, (uint32_t)g.l_p, 1};
        if (!make_tmap(&tmX, g.gather_x, 3, dims, str, box)) return UOE_ERR_CUDA;
        tmA = tmX;
    } else {
        const uint64_t dims[2] = {(uint64_t)g.K, (uint64_t)g.rows_max};
        const uint64_t str[1] = {(uint64_t)g.K * 2};
        const uint32_t box[2] = {BK, (uint32_t)(MT * BM)};      // all the 128-row blocks of a tile in one box
        if (!make_tmap(&tmA, g.A, 2, dims, str, box)) return UOE_ERR_CUDA;
        tmX = tmA;
    }
    const int nmat = g.nmat < 1 ? 1 : g.nmat;
    const void* Ws[3] = {g.W, g.W1 ? g.W1 : g.W, g.W2 ? g.W2 : g.W};
    for (int q = 0; q < 3; ++q) {
        if (B_KMAJOR) {       // W [n, N, K]
            const uint64_t dims[3] = {(uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.n};
            const uint64_t str[2] = {(uint64_t)g.K * 2, (uint64_t)g.K * g.N * 2};
            const uint32_t box[3] = {BK, PAIR ? BN / 2 : BN, 1};
            if (!make_tmap(&tmB[q], Ws[q], 3, dims, str, box)) return UOE_ERR_CUDA;
        } else {              // W [n, K, N] as [n][N/64 column blocks][K][64]
            const uint64_t dims[4] = {64, (uint64_t)g.K, (uint64_t)g.N / 64, (uint64_t)g.n};
            const uint64_t str[3] = {(uint64_t)g.N * 2, 128, (uint64_t)g.K * g.N * 2};
            const uint32_t box[4] = {64, BK, (uint32_t)(BN == 192 ? 1 : (PAIR ? BN / 2 : BN) / 64), 1};
            if (!make_tmap(&tmB[q], Ws[q], 4, dims, str, box)) return UOE_ERR_CUDA;
        }
    }
    // outputs as [rows_max, N], written in [32 rows x 64 columns] pieces
    CUtensorMap tmC[3], tmPre;
    {
        const uint64_t dims[2] = {(uint64_t)g.N, (uint64_t)g.rows_max};
        const uint64_t str[1] = {(uint64_t)g.N * 2};
        const uint32_t box[2] = {64, 32};
        const void* Cs[3] = {g.C, g.C1 ? g.C1 : g.C, g.C2 ? g.C2 : g.C};
        for (int q = 0; q < 3; ++q)
            if (!make_tmap(&tmC[q], Cs[q], 2, dims, str, box)) return UOE_ERR_CUDA;
        if (!make_tmap(&tmPre, g.pre ? g.pre : g.C, 2, dims, str, box)) return UOE_ERR_CUDA;
    }
    long long max_tiles = ((g.rows_max / BM + Cf::UNIT - 1) / Cf::UNIT + g.n) * (BN == 192 ? 1 : (g.N / BN) * nmat);
    const int walkers = PAIR ? max_pairs : sm_count();
    int grid = (int)(max_tiles < walkers ? max_tiles : walkers);
    if (grid < 1) grid = 1;
    if (PAIR) grid *= 2;
    SrcMap smap;          // how the rows of a gathered A are found
    if (g.gather_x) {
        if (g.map.on()) smap = g.map;
        else { smap.src_patch = g.src_patch; smap.l_p = g.l_p; }
    }
    ProfScope ps(g.label, s);
    auto launch = [&](auto... a) {
        if constexpr (PAIR) return launch_k_pairs(a...);
        else return launch_k(a...);
    };
    launch(kern, dim3(grid), dim3(Cf::THREADS), (size_t)Cf::SMEM, s, tmA, tmB[0], tmB[1], tmB[2], (__nv_bfloat16*)g.C, (__nv_bfloat16*)g.C1,
                                             (__nv_bfloat16*)g.C2, (__nv_bfloat16*)g.pre, g.offsets, g.n, g.K, g.N,
                                             nmat, g.act, status, (const __nv_bfloat16*)g.bwd_h, g.row_gate, g.row_valid,
                                             g.dg_part, (const __nv_bfloat16*)g.bias, g.blk_scale, tmX, smap, g.l_p, g.Bm, tmC[0],
                                             tmC[1], tmC[2], tmPre);
    UOE_LAUNCHED();
    return UOE_OK;
}

template <bool B_KMAJOR, bool BWD>
uoe_status dispatch(const GemmArgs& g, int* status, cudaStream_t s) {
    const int bn = gemm_bf16_bn(g.N);
    // 256-row tiles pay off when every SM still gets several of them and the K loop is long enough to be
    // bound by operand delivery rather than by the prologue
    const long long tiles256 = (g.rows_max / 256) * (g.N / 256);
    // the backward epilogue is long: it stays on 128-row accumulators, whose drain overlaps the next tile's main loop,
    // and takes its 256-row tiles from CTA pairs when there are enough of them for every pair of SMs
    if constexpr (BWD) {
        if (bn == 256 && g.K % 128 == 0 && tiles256 >= 2 * sm_count()) return launch_one<256, B_KMAJOR, BWD, 1, true>(g, status, s);
    }
    if constexpr (!BWD) {
        if (bn == 256 && g.K % 128 == 0 && tiles256 >= 2 * sm_count()) return launch_one<256, B_KMAJOR, BWD, 1, true>(g, status, s);
        if (bn == 256 && g.K >= 1024 && tiles256 >= 2 * sm_count()) return launch_one<256, B_KMAJOR, BWD, 2>(g, status, s);
    }
    if (bn == 256) return launch_one<256, B_KMAJOR, BWD, 1>(g, status, s);
    if (bn == 128) return launch_one<128, B_KMAJOR, BWD, 1>(g, status, s);
    return launch_one<64, B_KMAJOR, BWD, 1>(g, status, s);
}

}  // namespace

uoe_status launch_gemm_bf16(const GemmArgs& g, int* status, cudaStream_t s) {
    if (g.K % BK != 0 || g.N % 64 != 0 || g.nmat > 3) return UOE_ERR_UNSUPPORTED;
    if ((g.bias || g.blk_scale) && (g.bwd || g.nmat > 1)) return UOE_ERR_UNSUPPORTED;      // a bias row per expert, a factor per block: plain forward GEMMs only
    if (g.nmat > 1 && g.pre) return UOE_ERR_UNSUPPORTED;
    if (g.gather_x && ((!g.src_patch && !g.map.on()) || g.l_p < 8 || g.l_p % 8 != 0 || BM % g.l_p != 0)) return UOE_ERR_INVALID_ARG;
    if (g.rows_max % BM != 0 || g.n > 31) return UOE_ERR_UNSUPPORTED;
    if (g.bwd) {          // backward epilogue: weights are read K-major ([n, N, K])
        if (!g.b_kmajor || !g.bwd_h || !g.row_gate || !g.row_valid || !g.dg_part || !g.C1 || g.nmat > 1)
            return UOE_ERR_INVALID_ARG;
        return dispatch<true, true>(g, status, s);
    }
    if (g.nmat == 3 && g.N == 64 && !g.b_kmajor && !g.pre) return launch_one<192, false, false, 1>(g, status, s);
    if (g.b_kmajor) return dispatch<true, false>(g, status, s);
    return dispatch<false, false>(g, status, s);
}

}  // namespace uoe
