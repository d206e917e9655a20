// Tensor-core GEMM for sm_100a: C[m,n] (+)= epilogue(sum_k A(m,k) B(n,k)), bf16 operands, fp32
// accumulation in tensor memory.
//
// Persistent CTAs (one per SM) walk the list of 128 x BN output tiles.  Warp 0 streams 64-deep k slices of
// A and B into a ring of shared-memory stages with TMA (128-byte swizzle); warp 1 issues tcgen05.mma
// (M=128, N=BN, K=16) on the landed stages into one of two TMEM accumulator stages and commits each smem
// stage back to the producer; warps 2-17 read a finished accumulator from TMEM (tcgen05.ld, four warps per
// 32-lane quadrant), release it, apply the epilogue and store rows to global memory with 32-byte stores,
// while the MMA warp is already filling the other accumulator stage.
// Either operand may be K-major (contraction index contiguous) or MN-major; the layer needs K/K (forward),
// K/MN (input gradients) and MN/MN (weight gradients, contraction over tokens or over an expert's rows).
//
// Every wait on an mbarrier is bounded: when the bound is hit the CTA records BIGMAC_ERR_TIMEOUT in the
// status word, stops waiting, and still releases its tensor memory before it exits.
#include <cstdlib>

#include "tc_common.cuh"

namespace bigmac {

using namespace tc;

namespace {

// Persistent kernel: gridDim.x CTAs (one per SM) walk the tile list with stride gridDim.x.  The
// accumulator is double-buffered in tensor memory (2 x BN columns), so the epilogue of tile i overlaps
// the MMAs of tile i+1.
// GATHER: the rows of the (K-major) A tile are gathered (TcParams::gather_rows) by two extra warps with 16-byte
// asynchronous copies into the layout a TMA box would have, instead of one TMA box per k slice: warp g of them owns
// rows 64 g .. 64 g + 63 of the tile, lane l piece l & 7 of rows (l >> 3) + 4 j; every thread arrives on the stage's
// "full" barrier when its copies have landed.
template <int BN, int STAGES, bool A_KMAJOR, bool B_KMAJOR, bool TMA_EPI, bool GATHER = false>
__global__ void __launch_bounds__(GATHER ? kThreadsGather : kThreadsV2, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_z,
               const __grid_constant__ CUtensorMap map_b2, const TcParams p) {
    constexpr uint32_t A_BYTES = BM * BK * 2;
    constexpr uint32_t B_BYTES = BN * BK * 2;
    constexpr uint32_t CHUNK_BYTES = 64 * BK * 2;            // one 64-wide MN-major box
    constexpr uint32_t TMEM_COLS = 2 * BN;
    constexpr uint32_t STAGING_BYTES = TMA_EPI ? kEpiWarps * 2 * kBoxBytes : 0;   // per epilogue warp: a box for C, one for Z

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + STAGES * A_BYTES;
    uint8_t* staging = smem + STAGES * (A_BYTES + B_BYTES);
    uint64_t* full_bar = (uint64_t*)(staging + STAGING_BYTES);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tmem_full_bar = empty_bar + STAGES;            // [2]
    uint64_t* tmem_empty_bar = tmem_full_bar + 2;            // [2]
    uint64_t* z_bar = tmem_empty_bar + 2;                    // [kEpiWarps]: sigma' boxes prefetched by TMA (EPI_DACT)
    uint32_t* tmem_slot = (uint32_t*)(z_bar + kEpiWarps);
    volatile int* dead = (volatile int*)(tmem_slot + 1);
    static_assert(!GATHER || A_KMAJOR, "gathered rows: K-major A");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 32) {                                 // the maps are on their way while the barriers are set up
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        prefetch_tensormap(&map_c);
        prefetch_tensormap(&map_z);
        prefetch_tensormap(&map_b2);
    }

    if (threadIdx.x == 0) {
        // a gathered slice completes on the B box's bytes and on the arrival of every gathering thread
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], GATHER ? 1 + kGatherWarps * 32 : 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&tmem_full_bar[s], 1); mbar_init(&tmem_empty_bar[s], kEpiWarps); }
        for (int s = 0; s < kEpiWarps; ++s) mbar_init(&z_bar[s], 1);
        *dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    // Chained launch: everything above touched no global memory and may have run while the kernel before this one in
    // the stream was still working.  Tensor memory is held, so the next kernel of the stream may be set up in turn;
    // from the wait on, the predecessor's results are complete.
    grid_dependency_launch();
    grid_dependency_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    int tiles_m, tiles_n;
    const int total = total_tiles(p, BN, tiles_m, tiles_n);

    if (GATHER && warp >= 2 + kEpiWarps) {
        // ------------------------------------------------------------------ gathered A rows (two warps)
        const int piece = lane & 7;
        const int row0 = (warp - 2 - kEpiWarps) * (BM / kGatherWarps) + (lane >> 3);
        constexpr int ROWS = BM / kGatherWarps / 4;          // rows per lane: row0 + 4 j
        const uint8_t* src = (const uint8_t*)p.gather_src + piece * 16;
        const int64_t ld_bytes = p.gather_ld * 2;
        uint32_t s = 0, phase = 1;
        for (int t = blockIdx.x; t < total; t += gridDim.x) {
            const Tile tl = get_tile(p, BN, t, tiles_m, tiles_n);
            const uint8_t* from[ROWS];                       // this tile's source rows (null: a zero row)
#pragma unroll
            for (int j = 0; j < ROWS; ++j) {
                const int g = p.gather_rows[tl.m0 + row0 + 4 * j];
                from[j] = g < 0 ? nullptr : src + (int64_t)(g / p.gather_div) * ld_bytes;
            }
            for (int kb = 0; kb < tl.num_kb; ++kb, s = (s + 1 == STAGES ? 0 : s + 1), phase ^= (s == 0)) {
                mbar_wait_lean(&empty_bar[s], phase, dead, p.status);
                const uint32_t base = smem_u32(smem_a + s * A_BYTES);
                const int k0_bytes = kb * BK * 2;
#pragma unroll
                for (int j = 0; j < ROWS; ++j) {
                    const int row = row0 + 4 * j;
                    cp_async_16(base + row * 128 + ((piece ^ (row & 7)) << 4), from[j] ? from[j] + k0_bytes : src, from[j] ? 16u : 0u);
                }
                cp_async_arrive(&full_bar[s]);
            }
        }
    } else if (warp == 0 && GATHER) {
        // ------------------------------------------------------------------ TMA producer of B beside the gathered A rows
        if (lane == 0) {
            uint32_t s = 0, phase = 1;
            for (int t = blockIdx.x; t < total; t += gridDim.x) {
                const Tile tl = get_tile(p, BN, t, tiles_m, tiles_n);
                for (int kb = 0; kb < tl.num_kb; ++kb, s = (s + 1 == STAGES ? 0 : s + 1), phase ^= (s == 0)) {
                    mbar_wait_lean(&empty_bar[s], phase, dead, p.status);
                    mbar_expect_tx(&full_bar[s], B_BYTES);
                    tma_load_2d(smem_b + s * B_BYTES, &map_b, &full_bar[s], kb * BK, tl.expert * p.b_rows_per_expert + tl.n0);
                }
            }
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t s = 0, phase = 1;                     // stage and the parity its "empty" barrier is waited on with
            // the next tile is looked up (a global load for grouped rows) before this tile's loads are issued, so
            // that its latency does not sit between two tiles
            Tile nxt = get_tile(p, BN, blockIdx.x < total ? blockIdx.x : 0, tiles_m, tiles_n);
            for (int t = blockIdx.x; t < total; t += gridDim.x) {
                const Tile tl = nxt;
                if (t + (int)gridDim.x < total) nxt = get_tile(p, BN, t + gridDim.x, tiles_m, tiles_n);
                for (int kb = 0; kb < tl.num_kb; ++kb, s = (s + 1 == STAGES ? 0 : s + 1), phase ^= (s == 0)) {
                    mbar_wait_lean(&empty_bar[s], phase, dead, p.status);
                    mbar_expect_tx(&full_bar[s], A_BYTES + B_BYTES);
                    const int k0 = tl.k_row0 + kb * BK;
                    uint8_t* a_dst = smem_a + s * A_BYTES;
                    uint8_t* b_dst = smem_b + s * B_BYTES;
                    if (A_KMAJOR) {
                        tma_load_2d(a_dst, &map_a, &full_bar[s], k0, tl.m0);
                    } else {
#pragma unroll
                        for (int c = 0; c < BM / 64; ++c)
                            tma_load_2d(a_dst + c * CHUNK_BYTES, &map_a, &full_bar[s], tl.m0 + 64 * c, k0);
                    }
                    if (B_KMAJOR) {
                        if (p.n_split >= 0 && tl.n0 >= p.n_split) tma_load_2d(b_dst, &map_b2, &full_bar[s], k0, tl.n0 - p.n_split);
                        else tma_load_2d(b_dst, &map_b, &full_bar[s], k0, tl.expert * p.b_rows_per_expert + tl.n0);
                    } else {
                        const bool second = p.b2_first_kb >= 0 && kb >= p.b2_first_kb;     // dense only
                        const CUtensorMap* mb = second ? &map_b2 : &map_b;
                        const int kb_row = second ? (kb - p.b2_first_kb) * BK : tl.expert * p.b_rows_per_expert + k0;
#pragma unroll
                        for (int c = 0; c < BN / 64; ++c)
                            tma_load_2d(b_dst + c * CHUNK_BYTES, mb, &full_bar[s], tl.n0 + 64 * c, kb_row);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BN, !A_KMAJOR, !B_KMAJOR);
            // descriptors of stage 0; the address field (16-byte units, bits 0-13) takes stage and k-step offsets by addition
            const uint64_t da0 = A_KMAJOR ? smem_desc(smem_u32(smem_a), 16, 1024) : smem_desc(smem_u32(smem_a), CHUNK_BYTES, 1024);
            const uint64_t db0 = B_KMAJOR ? smem_desc(smem_u32(smem_b), 16, 1024) : smem_desc(smem_u32(smem_b), CHUNK_BYTES, 1024);
            constexpr uint32_t kStepA = (A_KMAJOR ? UMMA_K * 2 : UMMA_K * 128) >> 4, kStepB = (B_KMAJOR ? UMMA_K * 2 : UMMA_K * 128) >> 4;
            const bool uniform_k = p.group != GROUP_K && p.split_k <= 1;     // every tile contracts over all of K
            uint32_t stage = 0, phase = 0, local = 0;
            for (int t = blockIdx.x; t < total; t += gridDim.x, ++local) {
                const int num_kb = uniform_k ? (p.K + BK - 1) / BK : get_tile(p, BN, t, tiles_m, tiles_n).num_kb;
                const uint32_t acc = local & 1;
                mbar_wait_lean(&tmem_empty_bar[acc], ((local >> 1) & 1) ^ 1, dead, p.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    mbar_wait_lean(&full_bar[stage], phase, dead, p.status);
                    if (GATHER) fence_async_smem();        // the gathered rows were written through the generic proxy
                    tc_fence_after();
                    const uint64_t da = da0 + stage * (A_BYTES >> 4), db = db0 + stage * (B_BYTES >> 4);
                    umma_bf16(d_tmem, da, db, idesc, kb != 0);
#pragma unroll
                    for (int kk = 1; kk < BK / UMMA_K; ++kk) umma_bf16(d_tmem, da + kk * kStepA, db + kk * kStepB, idesc, 1);
                    umma_commit(&empty_bar[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (num_kb > 0) umma_commit(&tmem_full_bar[acc]);
                else mbar_arrive(&tmem_full_bar[acc]);
            }
        }
    } else if (warp < 2 + kEpiWarps) {
        // ------------------------------------------------------------------ epilogue (warps 2..17)
        const int quad = warp & 3;                     // TMEM lanes 32*quad .. 32*quad+31
        constexpr int COLS_PER_WARP = BN / (kEpiWarps / 4);
        constexpr int CHUNKS = COLS_PER_WARP / 32;
        const int part = (warp - 2) >> 2;              // which COLS_PER_WARP-wide slice of the tile's columns
        uint8_t* box_c = staging + (warp - 2) * 2 * kBoxBytes;
        uint8_t* box_z = box_c + kBoxBytes;
        const int esz = p.out_f32 ? 4 : 2;
        const bool vec_ok = ((p.ldc * esz) % 32 == 0) && ((p.c_stride * esz) % 32 == 0) && (p.ldc % 16 == 0) &&
                            (((uintptr_t)p.C) % 32 == 0) && (((uintptr_t)p.Z) % 32 == 0) && (p.Z == nullptr || p.ldc % 32 == 0);
        // EPI_DACT with staged stores: the warp's saved sigma' box (32 rows x its 64 columns) of the next tile is
        // fetched by TMA into box_z one tile ahead, so its DRAM latency is hidden behind the MMAs and the stores.
        static_assert(!TMA_EPI || CHUNKS == 2, "the sigma' box holds two 32-column chunks");
        const bool z_prefetch = TMA_EPI && p.epilogue == EPI_DACT;
        uint64_t* my_z_bar = &z_bar[warp - 2];
        uint32_t z_count = 0;
        auto issue_z = [&](const Tile& tile) {
            if (lane == 0) {
                mbar_expect_tx(my_z_bar, kBoxBytesZ);
                tma_load_2d(box_z, &map_z, my_z_bar, tile.n0 + part * COLS_PER_WARP, tile.m0 + quad * 32);
            }
        };
        uint32_t local = 0;
        const int step_m = (int)gridDim.x / tiles_n, step_n = (int)gridDim.x - step_m * tiles_n;
        TileWalk1 tw;
        walk1_init(tw, blockIdx.x, tiles_n);
        Tile nxt = tw.t < total ? walk1_tile(p, BN, tw, tiles_m, tiles_n) : Tile{};
        if (z_prefetch && tw.t < total) issue_z(nxt);
        for (; tw.t < total; ++local) {
            const Tile tl = nxt;
            const int t = tw.t;
            walk1_next(tw, gridDim.x, step_m, step_n, tiles_n);                   // tw / nxt now describe the next tile
            if (tw.t < total) nxt = walk1_tile(p, BN, tw, tiles_m, tiles_n);
            const uint32_t acc = local & 1;
            mbar_wait_lean(&tmem_full_bar[acc], (local >> 1) & 1, dead, p.status);
            tc_fence_after();
            const int row = tl.m0 + quad * 32 + lane;
            const bool row_ok = row < tl.m_limit;
            const int64_t row_off = tl.c_base + (int64_t)row * p.ldc;
            const uint32_t t_addr = tmem_base + acc * BN + ((uint32_t)(quad * 32) << 16) + (uint32_t)(part * COLS_PER_WARP);
#pragma unroll 1
            for (int c = 0; c < CHUNKS; ++c) {
                float v[32];
                if (tl.num_kb > 0) {
                    tmem_load_32_nowait(t_addr + c * 32, (uint32_t*)v);
                    tmem_load_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0.0f;
                }
                if (c == CHUNKS - 1) {                 // accumulator fully read: hand the TMEM stage back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tmem_empty_bar[acc]);
                }
                const int col0 = tl.n0 + part * COLS_PER_WARP + c * 32;
                if (col0 >= p.N) continue;             // uniform across the warp
                if (p.bias) add_bias32(v, p.bias + (int64_t)tl.expert * p.bias_stride + col0);   // N is a multiple of 32 here
                if (TMA_EPI) {
                    if (lane == 0) tma_store_wait_read();        // previous boxes of this warp have left smem
                    __syncwarp();
                    if (z_prefetch) {
                        if (c == 0) {
                            mbar_wait_lean(my_z_bar, z_count & 1, dead, p.status);
                            ++z_count;
                        }
                        uint32_t w[8];
                        load_row_u8(box_z, lane, c, w);
                        if (c == CHUNKS - 1) {             // box read by every lane: fetch the next tile's
                            fence_async_smem();
                            __syncwarp();
                            if (t + (int)gridDim.x < total) issue_z(nxt);
                        }
                        mul_by_sig32(v, w);
                    }
                    stage_row_chunk(p, v, box_c, box_z, lane, c);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        const int row0 = tl.expert * p.c_rows_per_expert + tl.m0 + quad * 32;
                        tma_store_2d(&map_c, box_c, col0, row0);
                        if (p.epilogue == EPI_ACT && p.Z && c == CHUNKS - 1) tma_store_2d(&map_z, box_z, col0 - 32, row0);
                        tma_store_commit();
                    }
                } else if (row_ok) {
                    if (p.n_split >= 0 && tl.n0 >= p.n_split) {          // second output: fp32, its own leading dimension
                        TcParams p2 = p;
                        p2.C = p.C2; p2.ldc = p.ldc2; p2.N = p.N2; p2.out_f32 = 1; p2.epilogue = EPI_NONE; p2.accumulate = 0;
                        const bool vec2 = (p.ldc2 % 8 == 0) && (((uintptr_t)p.C2) % 32 == 0);
                        // a split contraction writes partial results: both outputs then share one fp32 matrix (ldc2 == ldc)
                        const int64_t part2 = p.split_k > 1 ? tl.c_base : 0;
                        store_row_chunk(p2, v, part2 + (int64_t)row * p.ldc2, col0 - p.n_split, vec2);
                    } else {
                        store_row_chunk(p, v, row_off, col0, vec_ok);
                    }
                }
            }
        }
        if (TMA_EPI && lane == 0) tma_store_wait_read();          // the boxes have left shared memory; the writes land before the grid ends
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int BN, int STAGES, bool AK, bool BKM, bool TMA_EPI, bool GATHER = false>
cudaError_t launch(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const CUtensorMap& mz,
                   const CUtensorMap& mb2, const TcParams& p, int max_tiles, cudaStream_t stream) {
    constexpr size_t smem = STAGES * (BM * BK * 2 + BN * BK * 2) + (TMA_EPI ? kEpiWarps * 2 * kBoxBytes : 0) +
                            (2 * STAGES + 4 + kEpiWarps) * 8 + 16 + 1024;
    static PerDeviceOnce once;
    auto kernel = gemm_tc_kernel<BN, STAGES, AK, BKM, TMA_EPI, GATHER>;
    int dev;
    if (once.needed(&dev)) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        once.mark(dev);
    }
    const int grid = max_tiles < sm_count() ? max_tiles : sm_count();
    return launch_chained(kernel, grid, GATHER ? kThreadsGather : kThreadsV2, smem, stream, ma, mb, mc, mz, mb2, p);
}

template <int BN, int STAGES, bool TMA_EPI>
cudaError_t dispatch(const GemmArgs& g, int* status, cudaStream_t stream) {
    const int E = g.group == GROUP_NONE ? 1 : g.num_experts;
    CUtensorMap ma, mb;
    bool ok = true;
    TcParams p{};
    // A: [M,K] (K-major) or [K,M] (MN-major).  In GROUP_K, K is the row extent of the padded grouped buffers.
    const bool gather = g.gather_rows != nullptr;           // A's rows are gathered by the producer warp: no tensor map for A
    if (gather && (!g.a_kmajor || !g.b_kmajor || g.group != GROUP_M || g.B2 || g.C2 || g.split_k > 1 || g.K % BK ||
                   (g.lda * 2) % 16 || (uintptr_t)g.A % 16))
        return cudaErrorInvalidValue;
    if (gather) ok &= make_map(&ma, g.A, (uint64_t)g.K, 1, (uint64_t)g.lda, BK, 1);       // placeholder, never used
    else if (g.a_kmajor) ok &= make_map(&ma, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, BM);
    else ok &= make_map(&ma, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda, 64, BK);
    // B: dense [N,K] / [K,N]; grouped weights are E consecutive such matrices (b_stride elements apart).
    const uint64_t rows_per = g.group == GROUP_M ? (uint64_t)(g.b_stride / g.ldb) : 0;
    if (g.b_kmajor)
        ok &= make_map(&mb, g.B, (uint64_t)g.K, g.group == GROUP_M ? rows_per * E : (uint64_t)g.N, (uint64_t)g.ldb, BK, BN);
    else
        ok &= make_map(&mb, g.B, (uint64_t)g.N, g.group == GROUP_M ? rows_per * E : (uint64_t)g.K, (uint64_t)g.ldb, 64, BK);
    // Optional second B tensor (MN-major only): contraction rows k >= b2_first_k come from B2[k - b2_first_k, :].
    CUtensorMap mb2 = mb;
    p.b2_first_kb = -1;
    if (g.B2 && !g.C2) {
        if (g.b_kmajor || g.group != GROUP_NONE || g.b2_first_k % BK) return cudaErrorInvalidValue;
        ok &= make_map(&mb2, g.B2, (uint64_t)g.N, (uint64_t)(g.K - g.b2_first_k), (uint64_t)g.ldb2, 64, BK);
        // the first tensor ends where the second begins
        ok &= make_map(&mb, g.B, (uint64_t)g.N, (uint64_t)g.b2_first_k, (uint64_t)g.ldb, 64, BK);
        p.b2_first_kb = g.b2_first_k / BK;
    }
    p.n_split = -1;
    if (g.C2) {      // second K-major B tensor feeding a second (fp32) output
        if (!g.b_kmajor || g.group != GROUP_NONE || g.n_split % BN || TMA_EPI || g.B2 == nullptr ||
            (g.split_k > 1 && (!g.out_f32 || g.ldc2 != g.ldc)))
            return cudaErrorInvalidValue;
        ok &= make_map(&mb2, g.B2, (uint64_t)g.K, (uint64_t)g.N2, (uint64_t)g.ldb2, BK, BN);
        ok &= make_map(&mb, g.B, (uint64_t)g.K, (uint64_t)g.n_split, (uint64_t)g.ldb, BK, BN);
        p.n_split = g.n_split; p.C2 = g.C2; p.ldc2 = g.ldc2; p.N2 = g.N2;
    }
    // Outputs through TMA stores: bf16, no read-modify-write, 16-byte aligned rows; per-expert outputs (GROUP_K)
    // only when a row tile cannot run into the next expert's rows.
    const bool tma_store = TMA_EPI;
    const bool tma_possible = !g.out_f32 && !g.accumulate && g.split_k <= 1 && (g.ldc % 8 == 0) && ((uintptr_t)g.C % 16 == 0) &&
                           ((uintptr_t)g.Z % 16 == 0) && (g.group != GROUP_K || (g.M % BM == 0 && g.c_stride == (int64_t)g.M * g.ldc));
    if (TMA_EPI && !tma_possible) return cudaErrorInvalidValue;
    CUtensorMap mc = ma, mz = ma;
    if (tma_store) {
        const uint64_t c_rows = g.group == GROUP_K ? (uint64_t)g.M * E : (uint64_t)g.M;
        ok &= make_map(&mc, g.C, (uint64_t)g.N, c_rows, (uint64_t)g.ldc, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
        if ((g.epilogue == EPI_ACT && g.Z) || g.epilogue == EPI_DACT)
            ok &= make_map_u8(&mz, g.Z, (uint64_t)g.N, c_rows, (uint64_t)g.ldc, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    }
    if (!ok) return cudaErrorInvalidValue;
    p.tma_store = tma_store ? 1 : 0;
    p.split_k = (g.group == GROUP_NONE && g.split_k > 1) ? g.split_k : 1;
    p.c_rows_per_expert = g.group == GROUP_K ? g.M : 0;
    p.b_rows_per_expert = (int)rows_per;
    p.C = g.C; p.Z = g.Z; p.ldc = g.ldc; p.c_stride = g.c_stride; p.M = g.M; p.N = g.N; p.K = g.K;
    p.out_f32 = g.out_f32; p.accumulate = g.accumulate; p.epilogue = g.epilogue; p.act = g.act; p.group = g.group;
    p.num_experts = E; p.tile_expert = g.tile_expert; p.n_tiles = g.n_tiles; p.poffsets = g.poffsets; p.status = status;
    p.epi_parts = 4;
    p.bias = g.group == GROUP_M ? g.bias : nullptr; p.bias_stride = g.bias_stride;
    if (p.bias && (g.N % 32 || ((uintptr_t)g.bias % 16) || g.bias_stride % 4)) return cudaErrorInvalidValue;
    p.gather_rows = g.gather_rows; p.gather_src = g.A; p.gather_ld = g.lda; p.gather_div = g.gather_div > 0 ? g.gather_div : 1;
    const int64_t tiles = (int64_t)((g.N + BN - 1) / BN) * ((g.M + BM - 1) / BM) * (g.group == GROUP_K ? E : p.split_k);
    const int max_tiles = tiles > (1 << 30) ? (1 << 30) : (int)tiles;
    if (gather) return launch<BN, STAGES, true, true, TMA_EPI, true>(ma, mb, mc, mz, mb2, p, max_tiles, stream);
    if (g.a_kmajor && g.b_kmajor) return launch<BN, STAGES, true, true, TMA_EPI>(ma, mb, mc, mz, mb2, p, max_tiles, stream);
    if (g.a_kmajor && !g.b_kmajor) return launch<BN, STAGES, true, false, TMA_EPI>(ma, mb, mc, mz, mb2, p, max_tiles, stream);
    if (!g.a_kmajor && !g.b_kmajor) return launch<BN, STAGES, false, false, TMA_EPI>(ma, mb, mc, mz, mb2, p, max_tiles, stream);
    return cudaErrorNotSupported;
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }
int gemm_tc_sm_count() { return sm_count(); }

namespace {
// One thread waits, with the pipelines' bounded wait and a short limit, on a barrier nobody arrives at: the wait
// runs out, the status word is set and the kernel returns.
__global__ void expire_wait_kernel(int* status) {
    __shared__ uint64_t bar;
    __shared__ int dead_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        dead_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(&bar, 0, &dead_flag, status, 1u << 12);
    }
}
}  // namespace

cudaError_t launch_expire_wait(int* status, cudaStream_t stream) {
    expire_wait_kernel<<<1, 32, 0, stream>>>(status);
    return cudaGetLastError();
}

cudaError_t gemm_tc(const GemmArgs& g, int* status, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0) return cudaSuccess;
    // Where it pays, the problem runs on CTA pairs (each SM stages half of B); the tc_pair debug switch disables that.
    const bool pair_enabled = switches().tc_pair != 0;
    const bool want_pair = g.gather_rows ? false          // gathered rows: the one-CTA kernel
                           : g.force_kernel == 2 ? gemm_tc_pair_supported(g)
                           : g.force_kernel == 1 ? false : (pair_enabled && gemm_tc_pair_preferred(g));
    if (want_pair) return gemm_tc_pair(g, status, stream);
    // Output-heavy problems (wide rows: activations, ascend, dx) stage their stores through shared memory and
    // TMA, which costs one pipeline stage; contraction-heavy ones keep the deeper pipeline and store directly.
    const bool staged = switches().staged_stores && !g.C2 && tma_epilogue_possible(g) && g.N >= 1024 && g.N % 256 == 0 &&
                        (g.epilogue != EPI_DACT || g.group != GROUP_K);
    if (g.N >= 256) return staged ? dispatch<256, 3, true>(g, status, stream) : dispatch<256, 4, false>(g, status, stream);
    return dispatch<128, 6, false>(g, status, stream);
}

}  // namespace bigmac
