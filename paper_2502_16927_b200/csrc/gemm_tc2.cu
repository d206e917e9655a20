// Tensor-core GEMM on CTA pairs (tcgen05 cta_group::2): C[m,n] (+)= epilogue(sum_k A(m,k) B(n,k)).
//
// Two CTAs of a cluster (two neighbouring SMs) own one 256 x BN output tile: CTA r holds rows 128r..128r+127
// of A and columns (BN/2)r.. of B in its shared memory, and the 128 x BN accumulator of its rows in its own
// tensor memory.  One tcgen05.mma.cta_group::2 (M=256, N=BN, K=16), issued by the pair's leader (CTA 0),
// multiplies both CTAs' A rows with the B halves of both, so every SM stages only half of B: 32 KB instead of
// 48 KB per 64-deep k slice for the same tensor-core work, which is what bounds the one-CTA kernel.
// Protocol per k slice: each CTA's producer waits for its own "empty" barrier and issues its TMA loads, which
// all complete on the LEADER's "full" barrier (armed by the leader with the bytes of both CTAs); the leader's
// MMA warp waits there, issues the MMAs and commits with a multicast arrive onto the "empty" barrier of both
// CTAs.  Accumulators are double-buffered: "tmem_full" is signalled in both CTAs by a multicast commit, and the
// epilogue warps of both CTAs arrive on the leader's "tmem_empty" when they have read their half.
// No TMA multicast is used.  Everything else (epilogues, grouping, split contraction) is as in gemm_tc.cu.
#include <cstdlib>

#include "tc_pair.cuh"

namespace bigmac {

using namespace tc;

namespace {

// Work item of one CTA pair: rows m0.. (CTA 0) and m0+128.. (CTA 1) of problem `expert`.
struct PairTile {
    int m0, n0, expert, k_row0, num_kb, m_limit, halves;
    int64_t c_base;
};

// pairs of 128-row tiles: dense problems pair consecutive row tiles; expert-grouped rows pair tiles inside one
// expert (an expert with an odd number of tiles ends with a half-used pair).  s_pp[e] = pairs before expert e.
__device__ __forceinline__ PairTile get_pair_tile(const TcParams& p, int BN, int w, int pairs_m, int tiles_n, const int32_t* s_pp) {
    PairTile t;
    const int per = pairs_m * tiles_n;
    const int e = (p.group == GROUP_K || p.split_k > 1) ? w / per : 0;
    const int r = w - e * per;
    const int pair = r / tiles_n;
    t.n0 = (r % tiles_n) * BN;
    t.m0 = pair * 2 * BM;
    t.expert = p.group == GROUP_K ? e : 0;
    t.k_row0 = 0;
    t.num_kb = (p.K + BK - 1) / BK;
    t.m_limit = p.M;
    t.halves = 2;
    t.c_base = 0;
    if (p.group == GROUP_NONE && p.split_k > 1) {
        const int per_part = (t.num_kb + p.split_k - 1) / p.split_k;
        t.k_row0 = e * per_part * BK;
        t.num_kb = max(0, min(per_part, t.num_kb - e * per_part));
        t.c_base = (int64_t)e * p.M * p.ldc;
    } else if (p.group == GROUP_M) {
        int lo = 0, hi = p.num_experts;                        // largest x with s_pp[x] <= pair
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_pp[mid] <= pair) lo = mid; else hi = mid;
        }
        const int32_t* s_off = s_pp + p.num_experts + 1;       // the padded offsets, staged beside the prefix
        const int first = s_off[lo] / kPad, count = (s_off[lo + 1] - s_off[lo]) / kPad;
        const int j = pair - s_pp[lo];
        t.expert = lo;
        t.m0 = (first + 2 * j) * BM;
        t.halves = min(2, count - 2 * j);
    } else if (p.group == GROUP_K) {
        const int32_t* s_off = s_pp + p.num_experts + 1;
        t.k_row0 = s_off[e];
        t.num_kb = (s_off[e + 1] - t.k_row0) / BK;
        t.c_base = (int64_t)e * p.c_stride;
    }
    return t;
}

// Walks the work items of one pair, w = cluster_id, cluster_id + num_clusters, ...  For dense and row-grouped
// problems the (row pair, column tile) indices and the expert are carried along instead of being recomputed from
// w: the lookup (two integer divisions and a binary search, run by every warp at every tile) took about 1500 of
// the 8500 cycles an epilogue warp spends per output-heavy tile.
struct TileWalk {
    int w, pair, n, lo;
};

__device__ __forceinline__ void walk_init(TileWalk& tw, int cluster_id, int tiles_n) {
    tw.w = cluster_id;
    tw.pair = cluster_id / tiles_n;
    tw.n = cluster_id - tw.pair * tiles_n;
    tw.lo = 0;
}

__device__ __forceinline__ void walk_next(TileWalk& tw, int num_clusters, int step_pair, int step_n, int tiles_n) {
    tw.w += num_clusters;
    tw.pair += step_pair;
    tw.n += step_n;
    if (tw.n >= tiles_n) { tw.n -= tiles_n; ++tw.pair; }
}

__device__ __forceinline__ PairTile walk_tile(const TcParams& p, int BN, TileWalk& tw, int pairs_m, int tiles_n, const int32_t* s_pp) {
    if (p.group == GROUP_K || p.split_k > 1) return get_pair_tile(p, BN, tw.w, pairs_m, tiles_n, s_pp);
    PairTile t;
    t.n0 = tw.n * BN;
    t.m0 = tw.pair * 2 * BM;
    t.expert = 0;
    t.k_row0 = 0;
    t.num_kb = (p.K + BK - 1) / BK;
    t.m_limit = p.M;
    t.halves = 2;
    t.c_base = 0;
    if (p.group == GROUP_M) {
        const int32_t* s_off = s_pp + p.num_experts + 1;
        while (tw.lo + 1 < p.num_experts && s_pp[tw.lo + 1] <= tw.pair) ++tw.lo;     // pairs only grow along the walk
        const int first = s_off[tw.lo] / kPad, count = (s_off[tw.lo + 1] - s_off[tw.lo]) / kPad;
        const int j = tw.pair - s_pp[tw.lo];
        t.expert = tw.lo;
        t.m0 = (first + 2 * j) * BM;
        t.halves = min(2, count - 2 * j);
    }
    return t;
}

template <int BN, int STAGES, bool A_KMAJOR, bool B_KMAJOR, bool TMA_EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreadsV2, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_z,
                    const __grid_constant__ CUtensorMap map_b2, const TcParams p) {
    constexpr int BH = BN / 2;                               // B rows (output columns) staged by each CTA
    constexpr uint32_t A_BYTES = BM * BK * 2;
    constexpr uint32_t B_BYTES = BH * BK * 2;
    constexpr uint32_t CHUNK_BYTES = 64 * BK * 2;            // one 64-wide MN-major box
    constexpr uint32_t TMEM_COLS = 2 * BN;
    constexpr uint32_t STAGING_BYTES = TMA_EPI ? kEpiWarps * 2 * kBoxBytes : 0;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + STAGES * A_BYTES;
    uint8_t* staging = smem + STAGES * (A_BYTES + B_BYTES);
    uint64_t* full_bar = (uint64_t*)(staging + STAGING_BYTES);   // waited on in the leader only
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tmem_full_bar = empty_bar + STAGES;            // [2]
    uint64_t* tmem_empty_bar = tmem_full_bar + 2;            // [2], the leader's are used
    uint64_t* z_bar = tmem_empty_bar + 2;                    // [kEpiWarps]
    uint32_t* tmem_slot = (uint32_t*)(z_bar + kEpiWarps);
    volatile int* dead = (volatile int*)(tmem_slot + 1);
    int32_t* s_pp = (int32_t*)(tmem_slot + 4);               // [E + 1] pair prefix (GROUP_M), then [E + 1] padded offsets:
                                                             // every role looks tiles up here, not in global memory

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    if (threadIdx.x == 32) {                                 // the maps are on their way while the barriers are set up
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        prefetch_tensormap(&map_c);
        prefetch_tensormap(&map_z);
        prefetch_tensormap(&map_b2);
    }

    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&tmem_full_bar[s], 1); mbar_init(&tmem_empty_bar[s], 2 * kEpiWarps); }
        for (int s = 0; s < kEpiWarps; ++s) mbar_init(&z_bar[s], 1);
        *dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                      // the peer's barriers exist before anything signals them
    // Chained launch: everything above touched no global memory and may have run while the kernel before this one in
    // the stream was still working.  Tensor memory is held, so the next kernel of the stream may be set up in turn;
    // from the wait on, the predecessor's results are complete.
    grid_dependency_launch();
    grid_dependency_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // ---- work list
    const int tiles_n = (p.N + BN - 1) / BN;
    int pairs_m = (p.M + 2 * BM - 1) / (2 * BM);
    if (p.group != GROUP_NONE && p.poffsets) {
        int32_t* s_off = s_pp + p.num_experts + 1;
        for (int e = threadIdx.x; e <= p.num_experts; e += blockDim.x) s_off[e] = p.poffsets[e];
        __syncthreads();
        if (threadIdx.x == 0 && p.group == GROUP_M) {
            int run = 0;
            for (int e = 0; e < p.num_experts; ++e) {
                s_pp[e] = run;
                run += ((s_off[e + 1] - s_off[e]) / kPad + 1) / 2;
            }
            s_pp[p.num_experts] = run;
        }
    }
    __syncthreads();                                         // the pair prefix is in shared memory
    if (p.group == GROUP_M) pairs_m = s_pp[p.num_experts];
    const int total = pairs_m * tiles_n * (p.group == GROUP_K ? p.num_experts : p.split_k);
    const int step_pair = num_clusters / tiles_n, step_n = num_clusters - step_pair * tiles_n;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t s = 0, phase = 1;                     // stage and the parity its "empty" barrier is waited on with
            TileWalk tw;
            for (walk_init(tw, cluster_id, tiles_n); tw.w < total; walk_next(tw, num_clusters, step_pair, step_n, tiles_n)) {
                const PairTile tl = walk_tile(p, BN, tw, pairs_m, tiles_n, s_pp);
                const int my_m0 = tl.m0 + (int)rank * BM;
                const int my_n0 = tl.n0 + (int)rank * BH;
                for (int kb = 0; kb < tl.num_kb; ++kb, s = (s + 1 == STAGES ? 0 : s + 1), phase ^= (s == 0)) {
                    mbar_wait_lean(&empty_bar[s], phase, dead, p.status);
                    if (leader) mbar_expect_tx(&full_bar[s], 2 * (A_BYTES + B_BYTES));
                    const uint32_t bar = map_to_cta(&full_bar[s], 0);
                    const int k0 = tl.k_row0 + kb * BK;
                    uint8_t* a_dst = smem_a + s * A_BYTES;
                    uint8_t* b_dst = smem_b + s * B_BYTES;
                    if (A_KMAJOR) {
                        tma_load_2d_pair(a_dst, &map_a, bar, k0, my_m0);
                    } else {
#pragma unroll
                        for (int c = 0; c < BM / 64; ++c) tma_load_2d_pair(a_dst + c * CHUNK_BYTES, &map_a, bar, my_m0 + 64 * c, k0);
                    }
                    if (B_KMAJOR) {
                        if (p.n_split >= 0 && tl.n0 >= p.n_split) tma_load_2d_pair(b_dst, &map_b2, bar, k0, my_n0 - p.n_split);
                        else tma_load_2d_pair(b_dst, &map_b, bar, k0, tl.expert * p.b_rows_per_expert + my_n0);
                    } else {
                        const bool second = p.b2_first_kb >= 0 && kb >= p.b2_first_kb;     // dense only
                        const CUtensorMap* mb = second ? &map_b2 : &map_b;
                        const int kb_row = second ? (kb - p.b2_first_kb) * BK : tl.expert * p.b_rows_per_expert + k0;
#pragma unroll
                        for (int c = 0; c < BH / 64; ++c) tma_load_2d_pair(b_dst + c * CHUNK_BYTES, mb, bar, my_n0 + 64 * c, kb_row);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread of the leader CTA)
        if (leader && lane == 0) {
            constexpr uint32_t idesc = instr_desc_pair(BN, !A_KMAJOR, !B_KMAJOR);
            // descriptors of stage 0; the address field (16-byte units, bits 0-13) takes stage and k-step offsets by addition
            const uint64_t da0 = A_KMAJOR ? smem_desc(smem_u32(smem_a), 16, 1024) : smem_desc(smem_u32(smem_a), CHUNK_BYTES, 1024);
            const uint64_t db0 = B_KMAJOR ? smem_desc(smem_u32(smem_b), 16, 1024) : smem_desc(smem_u32(smem_b), CHUNK_BYTES, 1024);
            constexpr uint32_t kStepA = (A_KMAJOR ? UMMA_K * 2 : UMMA_K * 128) >> 4, kStepB = (B_KMAJOR ? UMMA_K * 2 : UMMA_K * 128) >> 4;
            uint32_t stage = 0, phase = 0, local = 0;
            TileWalk tw;
            for (walk_init(tw, cluster_id, tiles_n); tw.w < total; walk_next(tw, num_clusters, step_pair, step_n, tiles_n), ++local) {
                const PairTile tl = walk_tile(p, BN, tw, pairs_m, tiles_n, s_pp);
                const uint32_t acc = local & 1;
                mbar_wait_lean(&tmem_empty_bar[acc], ((local >> 1) & 1) ^ 1, dead, p.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < tl.num_kb; ++kb) {
                    mbar_wait_lean(&full_bar[stage], phase, dead, p.status);
                    tc_fence_after();
                    const uint64_t da = da0 + stage * (A_BYTES >> 4), db = db0 + stage * (B_BYTES >> 4);
                    umma_bf16_pair(d_tmem, da, db, idesc, kb != 0);
#pragma unroll
                    for (int kk = 1; kk < BK / UMMA_K; ++kk) umma_bf16_pair(d_tmem, da + kk * kStepA, db + kk * kStepB, idesc, 1);
                    umma_commit_pair(&empty_bar[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (tl.num_kb > 0) {
                    umma_commit_pair(&tmem_full_bar[acc]);
                } else {                                       // nothing to contract: zero accumulators, signal directly
                    mbar_arrive(&tmem_full_bar[acc]);
                    mbar_arrive_cluster(map_to_cta(&tmem_full_bar[acc], 1));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..17, both CTAs)
        const int quad = warp & 3;
        constexpr int COLS_PER_WARP = BN / (kEpiWarps / 4);
        constexpr int CHUNKS = COLS_PER_WARP / 32;
        const int part = (warp - 2) >> 2;
        uint8_t* box_c = staging + (warp - 2) * 2 * kBoxBytes;
        uint8_t* box_z = box_c + kBoxBytes;
        const int esz = p.out_f32 ? 4 : 2;
        const bool vec_ok = ((p.ldc * esz) % 32 == 0) && ((p.c_stride * esz) % 32 == 0) && (p.ldc % 16 == 0) &&
                            (((uintptr_t)p.C) % 32 == 0) && (((uintptr_t)p.Z) % 32 == 0) && (p.Z == nullptr || p.ldc % 32 == 0);
        const uint32_t leader_tmem_empty[2] = {map_to_cta(&tmem_empty_bar[0], 0), map_to_cta(&tmem_empty_bar[1], 0)};
        const bool z_prefetch = TMA_EPI && p.epilogue == EPI_DACT;
        uint64_t* my_z_bar = &z_bar[warp - 2];
        uint32_t z_count = 0;
        static_assert(!TMA_EPI || CHUNKS == 2, "the sigma' box holds two 32-column chunks");
        auto issue_z = [&](const PairTile& tile) {           // the warp's 32 rows x 64 columns of saved sigma'
            if (lane == 0) {
                mbar_expect_tx(my_z_bar, kBoxBytesZ);
                tma_load_2d(box_z, &map_z, my_z_bar, tile.n0 + part * COLS_PER_WARP, tile.m0 + (int)rank * BM + quad * 32);
            }
        };
        uint32_t local = 0;
        TileWalk tw;
        walk_init(tw, cluster_id, tiles_n);
        PairTile nxt = tw.w < total ? walk_tile(p, BN, tw, pairs_m, tiles_n, s_pp) : PairTile{};
        if (z_prefetch && tw.w < total) issue_z(nxt);
        // Plain epilogues have time to spare: two of the four warps of a lane quadrant do all its columns and the other
        // two stay out of the MMA thread's way (expert GEMM2 / dxg -3 %, ascend -6 %, a plain K = 512 grouped GEMM -9 %;
        // with one warp per quadrant the short-K launches become epilogue-bound, with an activation two are too few).
        const int part_step = p.epilogue == EPI_NONE ? p.epi_parts : 4;
        if (part < part_step)
        for (; tw.w < total; ++local) {
            const PairTile tl = nxt;
            const int w = tw.w;
            walk_next(tw, num_clusters, step_pair, step_n, tiles_n);            // tw / nxt now describe the next item
            if (tw.w < total) nxt = walk_tile(p, BN, tw, pairs_m, tiles_n, s_pp);
            const uint32_t acc = local & 1;
            mbar_wait_lean(&tmem_full_bar[acc], (local >> 1) & 1, dead, p.status);
            tc_fence_after();
            const int my_m0 = tl.m0 + (int)rank * BM;
            const int row = my_m0 + quad * 32 + lane;
            const bool half_ok = (int)rank < tl.halves;
            const bool row_ok = half_ok && row < tl.m_limit;
            const int64_t row_off = tl.c_base + (int64_t)row * p.ldc;
            for (int pp = part; pp < 4; pp += part_step) {
            const uint32_t t_addr = tmem_base + acc * BN + ((uint32_t)(quad * 32) << 16) + (uint32_t)(pp * COLS_PER_WARP);
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
                if (c == CHUNKS - 1) {                 // accumulator half fully read: tell the leader's MMA warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(leader_tmem_empty[acc]);
                }
                const int col0 = tl.n0 + pp * COLS_PER_WARP + c * 32;
                if (col0 >= p.N) continue;             // uniform across the warp
                if (p.bias) add_bias32(v, p.bias + (int64_t)tl.expert * p.bias_stride + col0);   // N is a multiple of 32 here
                if (TMA_EPI) {
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                    if (z_prefetch) {
                        if (c == 0) {
                            mbar_wait_lean(my_z_bar, z_count & 1, dead, p.status);
                            ++z_count;
                        }
                        uint32_t wz[8];
                        load_row_u8(box_z, lane, c, wz);
                        if (c == CHUNKS - 1) {             // box read by every lane: fetch the next tile's
                            fence_async_smem();
                            __syncwarp();
                            if (w + num_clusters < total) issue_z(nxt);
                        }
                        mul_by_sig32(v, wz);
                    }
                    stage_row_chunk(p, v, box_c, box_z, lane, c);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0 && half_ok && my_m0 < tl.m_limit) {
                        const int row0 = tl.expert * p.c_rows_per_expert + my_m0 + quad * 32;
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
        }
        if (TMA_EPI && lane == 0) tma_store_wait_read();          // the boxes have left shared memory; the writes land before the grid ends
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                      // nobody leaves while the peer may still touch this CTA
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

template <int BN, int STAGES, bool AK, bool BKM, bool TMA_EPI>
cudaError_t launch_pair(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const CUtensorMap& mz,
                        const CUtensorMap& mb2, const TcParams& p, int64_t max_items, cudaStream_t stream) {
    constexpr size_t kMaxSmem = 232448;                      // 227 KB: the most a CTA can have on sm_100
    const size_t smem = STAGES * (BM * BK * 2 + (BN / 2) * BK * 2) + (TMA_EPI ? kEpiWarps * 2 * kBoxBytes : 0) +
                        (2 * STAGES + 4 + kEpiWarps) * 8 + 16 + 2 * (size_t)(p.num_experts + 1) * 4 + 1024;
    if (smem > kMaxSmem) return cudaErrorInvalidConfiguration;
    static PerDeviceOnce once;
    auto kernel = gemm_tc_pair_kernel<BN, STAGES, AK, BKM, TMA_EPI>;
    int dev;
    if (once.needed(&dev)) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
        if (e != cudaSuccess) return e;
        once.mark(dev);
    }
    int64_t clusters = sm_count() / 2;
    if (max_items < clusters) clusters = max_items;
    if (clusters < 1) clusters = 1;
    return launch_chained(kernel, (unsigned)(2 * clusters), kThreadsV2, smem, stream, ma, mb, mc, mz, mb2, p);
}

template <int BN, int STAGES, bool TMA_EPI>
cudaError_t dispatch_pair(const GemmArgs& g, int* status, cudaStream_t stream) {
    constexpr int BH = BN / 2;
    const int E = g.group == GROUP_NONE ? 1 : g.num_experts;
    CUtensorMap ma, mb;
    bool ok = true;
    TcParams p{};
    if (g.a_kmajor) ok &= make_map(&ma, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, BM);
    else ok &= make_map(&ma, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda, 64, BK);
    const uint64_t rows_per = g.group == GROUP_M ? (uint64_t)(g.b_stride / g.ldb) : 0;
    if (g.b_kmajor)
        ok &= make_map(&mb, g.B, (uint64_t)g.K, g.group == GROUP_M ? rows_per * E : (uint64_t)g.N, (uint64_t)g.ldb, BK, BH);
    else
        ok &= make_map(&mb, g.B, (uint64_t)g.N, g.group == GROUP_M ? rows_per * E : (uint64_t)g.K, (uint64_t)g.ldb, 64, BK);
    CUtensorMap mb2 = mb;
    p.b2_first_kb = -1;
    if (g.B2 && !g.C2) {
        if (g.b_kmajor || g.group != GROUP_NONE || g.b2_first_k % BK) return cudaErrorInvalidValue;
        ok &= make_map(&mb2, g.B2, (uint64_t)g.N, (uint64_t)(g.K - g.b2_first_k), (uint64_t)g.ldb2, 64, BK);
        ok &= make_map(&mb, g.B, (uint64_t)g.N, (uint64_t)g.b2_first_k, (uint64_t)g.ldb, 64, BK);
        p.b2_first_kb = g.b2_first_k / BK;
    }
    p.n_split = -1;
    if (g.C2) {      // second K-major B tensor feeding a second (fp32) output
        if (!g.b_kmajor || g.group != GROUP_NONE || g.n_split % BN || TMA_EPI || g.B2 == nullptr ||
            (g.split_k > 1 && (!g.out_f32 || g.ldc2 != g.ldc)))
            return cudaErrorInvalidValue;
        ok &= make_map(&mb2, g.B2, (uint64_t)g.K, (uint64_t)g.N2, (uint64_t)g.ldb2, BK, BH);
        ok &= make_map(&mb, g.B, (uint64_t)g.K, (uint64_t)g.n_split, (uint64_t)g.ldb, BK, BH);
        p.n_split = g.n_split; p.C2 = g.C2; p.ldc2 = g.ldc2; p.N2 = g.N2;
    }
    if (TMA_EPI && !tma_epilogue_possible(g)) return cudaErrorInvalidValue;
    CUtensorMap mc = ma, mz = ma;
    if (TMA_EPI) {
        const uint64_t c_rows = g.group == GROUP_K ? (uint64_t)g.M * E : (uint64_t)g.M;
        ok &= make_map(&mc, g.C, (uint64_t)g.N, c_rows, (uint64_t)g.ldc, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
        if ((g.epilogue == EPI_ACT && g.Z) || g.epilogue == EPI_DACT)
            ok &= make_map_u8(&mz, g.Z, (uint64_t)g.N, c_rows, (uint64_t)g.ldc, 64, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    }
    if (!ok) return cudaErrorInvalidValue;
    p.tma_store = TMA_EPI ? 1 : 0;
    p.split_k = (g.group == GROUP_NONE && g.split_k > 1) ? g.split_k : 1;
    p.c_rows_per_expert = g.group == GROUP_K ? g.M : 0;
    p.b_rows_per_expert = (int)rows_per;
    p.C = g.C; p.Z = g.Z; p.ldc = g.ldc; p.c_stride = g.c_stride; p.M = g.M; p.N = g.N; p.K = g.K;
    p.out_f32 = g.out_f32; p.accumulate = g.accumulate; p.epilogue = g.epilogue; p.act = g.act; p.group = g.group;
    p.num_experts = E; p.tile_expert = g.tile_expert; p.n_tiles = g.n_tiles; p.poffsets = g.poffsets; p.status = status;
    p.epi_parts = epi_parts_default(g.epi_parts);
    p.bias = g.group == GROUP_M ? g.bias : nullptr; p.bias_stride = g.bias_stride;
    if (p.bias && (g.N % 32 || ((uintptr_t)g.bias % 16) || g.bias_stride % 4)) return cudaErrorInvalidValue;
    // upper bound on work items (the kernel derives the exact count on the device for grouped rows)
    const int64_t pairs = g.group == GROUP_M ? ((g.M + BM - 1) / BM + 1) / 2 + E : (g.M + 2 * BM - 1) / (2 * BM);
    const int64_t items = pairs * ((g.N + BN - 1) / BN) * (g.group == GROUP_K ? E : p.split_k);
    if (g.a_kmajor && g.b_kmajor) return launch_pair<BN, STAGES, true, true, TMA_EPI>(ma, mb, mc, mz, mb2, p, items, stream);
    if (g.a_kmajor && !g.b_kmajor) return launch_pair<BN, STAGES, true, false, TMA_EPI>(ma, mb, mc, mz, mb2, p, items, stream);
    if (!g.a_kmajor && !g.b_kmajor) return launch_pair<BN, STAGES, false, false, TMA_EPI>(ma, mb, mc, mz, mb2, p, items, stream);
    return cudaErrorNotSupported;
}

}  // namespace

// GROUP_M needs the padded offsets (to pair row tiles inside an expert).
bool gemm_tc_pair_supported(const GemmArgs& g) {
    if (g.N < 256) return false;                                  // narrow outputs stay on the one-CTA kernel
    if (g.group == GROUP_M && !g.poffsets) return false;
    if (g.C2 && (g.n_split % 256 || !g.b_kmajor || !g.a_kmajor)) return false;   // second output: whole tiles of it
    return true;
}

// Measured on B200 (interleaved A/B at the large workload's shapes, after the MMA-issue thread was made lean): pairs
// are 3-20 % faster on every shape (each SM stages half of B) but one: the training expert GEMM1, whose epilogue
// (activation, sigma' quantisation, two output streams) keeps the issue slots so busy that one MMA-issuing thread per
// SM instead of one per pair is worth 2.5 % (0.615-0.626 vs 0.633-0.642 ms in three interleaved runs).
bool gemm_tc_pair_preferred(const GemmArgs& g) {
    return gemm_tc_pair_supported(g) && !(g.epilogue == EPI_ACT && g.Z != nullptr);
}

cudaError_t gemm_tc_pair(const GemmArgs& g, int* status, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0) return cudaSuccess;
    const bool staged = switches().staged_stores && !g.C2 && tma_epilogue_possible(g) && g.N >= 1024 && g.N % 256 == 0 &&
                        (g.epilogue != EPI_DACT || g.group != GROUP_K);
    // 32 KB per stage and CTA: 5 stages beside the 64 KB store staging (4 if the expert tables are long), 6 without it
    if (!staged) return dispatch_pair<256, 6, false>(g, status, stream);
    const int E = g.group == GROUP_NONE ? 1 : g.num_experts;
    return E <= 192 ? dispatch_pair<256, 5, true>(g, status, stream) : dispatch_pair<256, 4, true>(g, status, stream);
}

}  // namespace bigmac
