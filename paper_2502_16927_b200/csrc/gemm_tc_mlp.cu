// Inference forward of the experts in one kernel: u = sigma(xg W1_e^T) W2_e^T per 128-row tile of an expert's
// segment (Eq. 4), with the hidden activations never leaving the SM.  For low widths r <= 256.
//
// The hidden width h is walked in chunks of 64.  Per chunk c, on one CTA:
//   GEMM1   acc1[c % 4] (128 x 64 fp32, tensor memory) = X (128 x r, shared memory, loaded once per tile)
//                                                        x W1_e[64 c .. 64 c + 63, :]^T
//   sigma   16 epilogue warps read acc1 (tcgen05.ld), apply the activation, and write the bf16 result into shared
//           memory in the K-major 128-byte-swizzled layout a tcgen05.mma A operand has (A2[c % 2], 128 x 64)
//   GEMM2   acc2 (128 x r fp32, tensor memory) += A2[c % 2] x W2_e[:, 64 c .. 64 c + 63]^T
// GEMM1 runs two chunks ahead of GEMM2 (four acc1 buffers), so that the activation of two chunks is in flight
// while the tensor pipe works on a third.  Tensor memory: 4 x 64 + r <= 512 columns.  Shared memory at
// r = 256: X 64 KB, W1 and W2 chunks double-buffered 2 x 32 KB each, A2 2 x 16 KB = 224 KB.  After the last chunk
// the 16 warps store acc2 as bf16 rows of u; the next tile's GEMM1s run meanwhile, only its first GEMM2 waits.
// All waits are bounded (status word); the tile -> expert table is read one tile ahead.
// Limit (measured with clock stamps around every wait of the MMA warp): a chunk takes about 1.8 us where the
// tensor pipe needs 0.5.  The waits are short; the time goes into issuing the chunk's 16 + 4 tcgen05.mma
// instructions, about 100 cycles each whatever their size, and GEMM1's are only N = 64 wide (32-64 cycles of
// tensor work each).  A variant on CTA pairs (half the weight bytes per SM, four chunks in flight) ran at the same
// speed, so loads are not what limits it.  A 128-wide chunk would halve the instruction count but leaves no room to
// double-buffer the activated chunk beside X in shared memory at r = 256.  The layer therefore uses this kernel
// only on short tile lists (decode-sized batches), where it saves a launch and the HBM round trip of the
// activations; on long lists the two separate GEMMs (N = 256 instructions) are faster.
#include "tc_pair.cuh"

namespace bigmac {

using namespace tc;

namespace {

constexpr int BH = 64;                                   // hidden chunk
constexpr int kMlpEpiWarps = 16;
constexpr int kAcc1 = 4;                                 // acc1 buffers; GEMM1 runs kAhead chunks ahead of GEMM2
constexpr int kAhead = 2;
constexpr int kFirstEpiWarp = 3;                         // warp 0: X and W1 loads, warp 1: MMA issue, warp 2: W2 loads
constexpr int kMlpThreads = (kFirstEpiWarp + kMlpEpiWarps) * 32;

struct MlpParams {
    void* U;             // [rows, r] bf16
    int r, h, act;
    int b1_rows_per_expert, b2_rows_per_expert;          // h, r
    const int32_t* tile_expert;
    const int32_t* n_tiles;
    int max_tiles;
    int* status;
};

// Arrive on a barrier of another CTA of the cluster, making this thread's earlier stores into that CTA visible to
// whoever acquires the barrier at cluster scope.
__device__ __forceinline__ void mbar_arrive_release_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_cluster_16B(uint32_t cluster_addr, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// SPLIT: a pair of CTAs (a cluster) shares every tile: CTA 0 walks the first half of the hidden chunks, CTA 1 the
// second, so that a short tile list (a few hundred tokens: one tile per expert, far fewer tiles than SMs) streams
// its weights through twice as many SMs.  CTA 1 hands its 128 x r fp32 partial result to CTA 0 through CTA 0's
// shared memory (the X and W1 buffers, free once CTA 0's last GEMM1 of the tile is done: 128 r 2 + 2 x 64 r 2 bytes
// = 128 r 4), CTA 0 adds it to its own and stores the tile.
template <bool SPLIT>
__device__ __forceinline__ void fused_mlp_body(const CUtensorMap& map_x, const CUtensorMap& map_w1, const CUtensorMap& map_w2,
                                               const MlpParams& p) {
    const int KB1 = p.r / BK;                            // 64-deep k slices of GEMM1
    const uint32_t X_BYTES = (uint32_t)KB1 * BM * BK * 2;
    const uint32_t W1_BYTES = (uint32_t)KB1 * BH * BK * 2;
    const uint32_t W2_BYTES = (uint32_t)p.r * BH * 2;
    constexpr uint32_t A2_BYTES = BM * BH * 2;
    constexpr uint32_t TMEM_COLS = 512;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* s_x = smem;
    uint8_t* s_w1 = s_x + X_BYTES;                       // [2]
    uint8_t* s_w2 = s_w1 + 2 * W1_BYTES;                 // [2]
    uint8_t* s_a2 = s_w2 + 2 * W2_BYTES;                 // [2]
    uint64_t* bars = (uint64_t*)(s_a2 + 2 * A2_BYTES);
    uint64_t* x_full = bars;            uint64_t* x_empty = bars + 1;
    uint64_t* w1_full = bars + 2;       uint64_t* w1_empty = bars + 4;
    uint64_t* w2_full = bars + 6;       uint64_t* w2_empty = bars + 8;
    uint64_t* acc1_full = bars + 10;    uint64_t* acc1_empty = bars + 14;      // [kAcc1] each
    uint64_t* a2_full = bars + 18;      uint64_t* a2_empty = bars + 20;
    uint64_t* acc2_full = bars + 22;    uint64_t* acc2_empty = bars + 23;
    uint64_t* peer_free = bars + 24;                     // SPLIT, in CTA 1: CTA 0's X and W1 buffers may be written
    uint64_t* partial_full = bars + 25;                  // SPLIT, in CTA 0: CTA 1's partial result has arrived
    uint64_t* tile_done = bars + 26;                     // SPLIT, in CTA 0: the partial result has been read
    uint32_t* tmem_slot = (uint32_t*)(bars + 27);
    volatile int* dead = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 32) {                                 // the maps are on their way while the barriers are set up
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w1);
        prefetch_tensormap(&map_w2);
    }

    if (threadIdx.x == 0) {
        mbar_init(x_full, 1); mbar_init(x_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&w1_full[s], 1); mbar_init(&w1_empty[s], 1);
            mbar_init(&w2_full[s], 1); mbar_init(&w2_empty[s], 1);
            mbar_init(&a2_full[s], kMlpEpiWarps); mbar_init(&a2_empty[s], 1);
        }
        for (int s = 0; s < kAcc1; ++s) { mbar_init(&acc1_full[s], 1); mbar_init(&acc1_empty[s], kMlpEpiWarps); }
        mbar_init(acc2_full, 1); mbar_init(acc2_empty, kMlpEpiWarps);
        mbar_init(peer_free, 1); mbar_init(partial_full, kMlpEpiWarps); mbar_init(tile_done, kMlpEpiWarps);
        *dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (SPLIT) cluster_sync_all();                        // the peer's barriers exist before anything signals them
    // Chained launch: everything above touched no global memory and may have run while the kernel before this one in
    // the stream was still working.  Tensor memory is held, so the next kernel of the stream may be set up in turn;
    // from the wait on, the predecessor's results are complete.
    grid_dependency_launch();
    grid_dependency_wait();
    const uint32_t tmem_base = *tmem_slot;
    const int total = min(*p.n_tiles, p.max_tiles);
    const uint32_t crank = SPLIT ? cluster_ctarank() : 0u;
    const int first = SPLIT ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, stride = SPLIT ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int chunks = SPLIT ? p.h / BH / 2 : p.h / BH;   // this CTA's chunks of a tile: cbase, cbase + 1, ...
    const int cbase = SPLIT ? (int)crank * chunks : 0;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: X and the W1 chunks
        if (lane == 0) {
            uint32_t g = 0, tl = 0;
            int next_e = first < total ? p.tile_expert[first] : 0;
            for (int t = first; t < total; t += stride, ++tl) {
                const int e = next_e;
                if (t + stride < total) next_e = p.tile_expert[t + stride];
                mbar_wait(x_empty, (tl & 1) ^ 1, dead, p.status);
                // CTA 0 of a pair: X and W1 buffers hold the peer's partial result until the epilogue has read it
                if (SPLIT && crank == 0 && tl > 0) mbar_wait(tile_done, (tl - 1) & 1, dead, p.status);
                mbar_expect_tx(x_full, X_BYTES);
                for (int kb = 0; kb < KB1; ++kb) tma_load_2d(s_x + kb * (BM * BK * 2), &map_x, x_full, kb * BK, t * BM);
                for (int c = 0; c < chunks; ++c, ++g) {
                    const int s = g & 1;
                    mbar_wait(&w1_empty[s], ((g >> 1) & 1) ^ 1, dead, p.status);
                    mbar_expect_tx(&w1_full[s], W1_BYTES);
                    for (int kb = 0; kb < KB1; ++kb)
                        tma_load_2d(s_w1 + s * W1_BYTES + kb * (BH * BK * 2), &map_w1, &w1_full[s], kb * BK,
                                    e * p.b1_rows_per_expert + (cbase + c) * BH);
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ TMA producer: the W2 chunks (its own
        // thread: a W2 buffer frees only when GEMM2 two chunks back is done, and the W1 loads must not queue behind that)
        if (lane == 0) {
            uint32_t g = 0;
            int next_e = first < total ? p.tile_expert[first] : 0;
            for (int t = first; t < total; t += stride) {
                const int e = next_e;
                if (t + stride < total) next_e = p.tile_expert[t + stride];
                for (int c = 0; c < chunks; ++c, ++g) {
                    const int s = g & 1;
                    mbar_wait(&w2_empty[s], ((g >> 1) & 1) ^ 1, dead, p.status);
                    mbar_expect_tx(&w2_full[s], W2_BYTES);
                    tma_load_2d(s_w2 + s * W2_BYTES, &map_w2, &w2_full[s], (cbase + c) * BH, e * p.b2_rows_per_expert);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc1 = instr_desc(BH, false, false);
        const uint32_t idesc2 = instr_desc(p.r, false, false);
        const uint32_t acc2_tmem = tmem_base + kAcc1 * BH;
        // Descriptors of the buffers' first bytes; the address field (bits 0-13, in 16-byte units) takes offsets by plain
        // addition, which keeps the instruction stream of this warp short: it shares its scheduler with four busy
        // epilogue warps, and with descriptors rebuilt per MMA the issue of one chunk's MMAs took longer than the MMAs.
        const uint64_t desc_x = smem_desc(smem_u32(s_x), 16, 1024), desc_w1 = smem_desc(smem_u32(s_w1), 16, 1024);
        const uint64_t desc_w2 = smem_desc(smem_u32(s_w2), 16, 1024), desc_a2 = smem_desc(smem_u32(s_a2), 16, 1024);
        uint32_t g = 0, tl = 0;
        // GEMM2 of global chunk gp (chunk cp of tile number tile_no)
        auto gemm2 = [&](uint32_t gp, int cp, uint32_t tile_no) {
            const int s = gp & 1;
            const uint32_t ph = (gp >> 1) & 1;
            mbar_spin(&w2_full[s], ph, dead, p.status);
            mbar_spin(&a2_full[s], ph, dead, p.status);
            if (cp == 0) mbar_spin(acc2_empty, (tile_no & 1) ^ 1, dead, p.status);
            tc_fence_after();
            if (lane == 0) {
                const uint64_t da = desc_a2 + ((s * A2_BYTES) >> 4), db = desc_w2 + ((s * W2_BYTES) >> 4);
#pragma unroll
                for (int kk = 0; kk < BH / UMMA_K; ++kk)
                    umma_bf16(acc2_tmem, da + ((kk * UMMA_K * 2) >> 4), db + ((kk * UMMA_K * 2) >> 4), idesc2, (cp | kk) != 0);
                umma_commit(&a2_empty[s]);
                umma_commit(&w2_empty[s]);
            }
            __syncwarp();
        };
        // GEMM1 of global chunk gc (chunk c of the current tile)
        auto gemm1 = [&](uint32_t gc, int c) {
            const int s = gc & 1, a = gc & (kAcc1 - 1);
            mbar_spin(&w1_full[s], (gc >> 1) & 1, dead, p.status);
            mbar_spin(&acc1_empty[a], ((gc / kAcc1) & 1) ^ 1, dead, p.status);
            tc_fence_after();
            if (lane == 0) {
                const uint32_t d_tmem = tmem_base + a * BH;
                for (int kb = 0; kb < KB1; ++kb) {
                    const uint64_t da = desc_x + ((kb * (BM * BK * 2)) >> 4);
                    const uint64_t db = desc_w1 + ((s * W1_BYTES + kb * (BH * BK * 2)) >> 4);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)
                        umma_bf16(d_tmem, da + ((kk * UMMA_K * 2) >> 4), db + ((kk * UMMA_K * 2) >> 4), idesc1, (kb | kk) != 0);
                }
                umma_commit(&w1_empty[s]);
                umma_commit(&acc1_full[a]);
                if (c == chunks - 1) umma_commit(x_empty);
            }
            __syncwarp();
        };
        for (int t = first; t < total; t += stride, ++tl) {
            mbar_spin(x_full, tl & 1, dead, p.status);
            for (int c = 0; c < kAhead && c < chunks; ++c) gemm1(g + c, c);
            for (int c = 0; c < chunks; ++c, ++g) {
                if (c + kAhead < chunks) gemm1(g + kAhead, c + kAhead);
                gemm2(g, c, tl);
            }
            if (lane == 0) umma_commit(acc2_full);
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 3..18)
        const int quad = warp & 3;                       // TMEM lanes 32*quad ..
        const int cpart = (warp - kFirstEpiWarp) >> 2;   // 16 of the chunk's 64 columns
        const int row_in_tile = quad * 32 + lane;
        uint32_t g = 0, tl = 0;
        for (int t = first; t < total; t += stride, ++tl) {
            for (int c = 0; c < chunks; ++c, ++g) {
                const int s = g & 1, a = g & (kAcc1 - 1);
                const uint32_t ph = (g >> 1) & 1;
                mbar_spin(&acc1_full[a], (g / kAcc1) & 1, dead, p.status);
                tc_fence_after();
                // the tile's last GEMM1 is done: nothing reads this CTA's X and W1 buffers any more, the peer may write
                if (SPLIT && crank == 0 && c == chunks - 1 && warp == kFirstEpiWarp && lane == 0)
                    mbar_arrive_cluster(map_to_cta(peer_free, 1));
                float v[16];
                tmem_load_16_nowait(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(a * BH + cpart * 16), (uint32_t*)v);
                tmem_load_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc1_empty[a]);
                act_chunk_any<false, 16>(p.act, v, nullptr);
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) w[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
                mbar_spin(&a2_empty[s], ph ^ 1, dead, p.status);       // GEMM2 two chunks back has read this buffer
                uint8_t* row = s_a2 + s * A2_BYTES + row_in_tile * 128;
                const int sw = row_in_tile & 7;                         // 128-byte swizzle: 16-byte piece j of a row sits at j ^ (row % 8)
                st_shared_16B(row + (((2 * cpart) ^ sw) << 4), w[0], w[1], w[2], w[3]);
                st_shared_16B(row + (((2 * cpart + 1) ^ sw) << 4), w[4], w[5], w[6], w[7]);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&a2_full[s]);
            }
            // the tile's output: acc2 (128 x r) -> bf16 rows of u
            mbar_spin(acc2_full, tl & 1, dead, p.status);
            tc_fence_after();
            const int cols = p.r / 4;                                   // per warp: 16, 32, 48 or 64
            __nv_bfloat16* out = (__nv_bfloat16*)p.U + ((int64_t)t * BM + row_in_tile) * p.r + cpart * cols;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(kAcc1 * BH + cpart * cols);
            // SPLIT: the partial result sits in CTA 0's X / W1 buffers as 16-byte pieces [column / 4][row] (neighbouring
            // lanes, i.e. rows, at neighbouring addresses)
            const int piece0 = cpart * (cols / 4);
            if (SPLIT && crank == 1) {
                mbar_wait_cluster(peer_free, tl & 1, dead, p.status);
                const uint32_t dst = map_to_cta(s_x, 0);
                for (int j = 0; j < cols; j += 16) {
                    float v[16];
                    tmem_load_16_nowait(t_addr + j, (uint32_t*)v);
                    tmem_load_wait();
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        st_cluster_16B(dst + (uint32_t)(((piece0 + j / 4 + q) * BM + row_in_tile) * 16), v[4 * q], v[4 * q + 1],
                                       v[4 * q + 2], v[4 * q + 3]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive_release_cluster(map_to_cta(partial_full, 0));
            } else {
                if (SPLIT) mbar_wait_cluster(partial_full, tl & 1, dead, p.status);
                for (int j = 0; j < cols; j += 16) {
                    float v[16];
                    tmem_load_16_nowait(t_addr + j, (uint32_t*)v);
                    tmem_load_wait();
                    if (SPLIT) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float4 o = *(const float4*)(s_x + ((piece0 + j / 4 + q) * BM + row_in_tile) * 16);
                            v[4 * q] += o.x; v[4 * q + 1] += o.y; v[4 * q + 2] += o.z; v[4 * q + 3] += o.w;
                        }
                    }
                    uint32_t w[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) w[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
                    st_global_32B(out + j, w);
                }
                if (SPLIT) {                                 // these reads come before the next tile's TMA writes
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tile_done);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc2_empty);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (SPLIT) cluster_sync_all();                        // nobody leaves while the peer may still signal or write here
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

__global__ void __launch_bounds__(kMlpThreads, 1)
fused_mlp_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w1,
                 const __grid_constant__ CUtensorMap map_w2, const MlpParams p) {
    fused_mlp_body<false>(map_x, map_w1, map_w2, p);
}
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kMlpThreads, 1)
fused_mlp_split_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w1,
                       const __grid_constant__ CUtensorMap map_w2, const MlpParams p) {
    fused_mlp_body<true>(map_x, map_w1, map_w2, p);
}

}  // namespace

bool fused_mlp_supported(int r, int h, int dtype) {
    return dtype == BIGMAC_BF16 && r >= 64 && r <= 256 && r % 64 == 0 && h >= 64 && h % 64 == 0;
}

// xg [max_rows, r] grouped padded rows, w1 [E, h, r], w2 [E, r, h], u [max_rows, r]; tiles of 128 rows, tile -> expert
// and the live tile count on the device.
cudaError_t launch_fused_mlp(const void* xg, const void* w1, const void* w2, void* u, int64_t max_rows, int r, int h, int E,
                             int act, const int32_t* tile_expert, const int32_t* n_tiles, int* status, cudaStream_t stream) {
    if (max_rows <= 0) return cudaSuccess;
    CUtensorMap mx, m1, m2;
    bool ok = make_map(&mx, xg, (uint64_t)r, (uint64_t)max_rows, (uint64_t)r, BK, BM);
    ok &= make_map(&m1, w1, (uint64_t)r, (uint64_t)E * h, (uint64_t)r, BK, BH);
    ok &= make_map(&m2, w2, (uint64_t)h, (uint64_t)E * r, (uint64_t)h, BH, (uint32_t)r);
    if (!ok) return cudaErrorInvalidValue;
    MlpParams p{};
    p.U = u; p.r = r; p.h = h; p.act = act; p.b1_rows_per_expert = h; p.b2_rows_per_expert = r;
    p.tile_expert = tile_expert; p.n_tiles = n_tiles; p.max_tiles = (int)(max_rows / BM); p.status = status;
    const int kb1 = r / BK;
    const size_t smem = (size_t)kb1 * BM * BK * 2 + 2 * (size_t)kb1 * BH * BK * 2 + 2 * (size_t)r * BH * 2 + 2 * (size_t)BM * BH * 2 +
                        27 * 8 + 16 + 1024;
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        cudaError_t e = cudaFuncSetAttribute(fused_mlp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(fused_mlp_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
        if (e != cudaSuccess) return e;
        once.mark(dev);
    }
    if (p.max_tiles <= 0) return cudaSuccess;
    // at most one tile per SM and an even number of hidden chunks: two SMs per tile, half of the chunks each
    if (p.max_tiles <= sm_count() && (h / BH) % 2 == 0) {
        const int pairs = p.max_tiles < sm_count() / 2 ? p.max_tiles : sm_count() / 2;
        return launch_chained(fused_mlp_split_kernel, 2 * pairs, kMlpThreads, smem, stream, mx, m1, m2, p);
    }
    const int grid = p.max_tiles < sm_count() ? p.max_tiles : sm_count();
    return launch_chained(fused_mlp_kernel, grid, kMlpThreads, smem, stream, mx, m1, m2, p);
}

}  // namespace bigmac
