// Tensor-core GEMM for sm_100a: C[m,n] (+)= epilogue(sum_k A(m,k) B(n,k)), bf16 operands, fp32
// accumulation in tensor memory.
//
// One CTA computes one 128 x BN output tile.  Warp 0 streams 64-deep k slices of A and B into a ring of
// shared-memory stages with TMA (128-byte swizzle); warp 1 issues tcgen05.mma (M=128, N=BN, K=16) on the
// landed stages and commits each stage back to the producer; warps 2-5 read the finished accumulator from
// TMEM (tcgen05.ld, one 32-lane quadrant per warp), apply the epilogue and store rows to global memory.
// Either operand may be K-major (contraction index contiguous) or MN-major; the layer needs K/K (forward),
// K/MN (input gradients) and MN/MN (weight gradients, contraction over tokens or over an expert's rows).
//
// Every wait on an mbarrier is bounded: when the bound is hit the CTA records BIGMAC_ERR_TIMEOUT in the
// status word, stops waiting, and still releases its tensor memory before it exits.
#include <cuda.h>

#include "internal.h"
#include "act.cuh"

namespace bigmac {

namespace {

constexpr int BM = 128;          // UMMA M
constexpr int BK = 64;           // bf16 elements per k slice = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int kThreads = 192;
constexpr uint32_t kWaitLimit = 1u << 22;

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
// Bounded wait.  `dead` is a CTA-wide flag in shared memory: once any wait ran out nobody waits again.
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, volatile int* dead, int* status) {
    if (*dead) return;
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if ((i & 1023u) == 1023u && *dead) return;
    }
    *dead = 1;
    atomicExch(status, 1);
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_load_32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
//   K-major tile:  rows of 128 bytes (64 k), 8-row groups 1024 bytes apart (SBO); LBO unused.
//   MN-major tile: k rows of 128 bytes (64 m/n), 8-k groups 1024 bytes apart (SBO), consecutive
//                  64-wide m/n chunks `lbo_bytes` apart (LBO).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffff) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;          // version
    d |= (uint64_t)2 << 61;          // SWIZZLE_128B
    return d;
}

// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, M = 128, N = bn.
__host__ __device__ constexpr uint32_t instr_desc(int bn, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

struct TcParams {
    void* C;
    void* Z;
    int64_t ldc, c_stride;
    int M, N, K;
    int b_rows_per_expert;       // rows of the B tensor map per expert (GROUP_M); 0 if dense
    int out_f32, accumulate, epilogue, act, group;
    const int32_t* tile_expert;
    const int32_t* n_tiles;
    const int32_t* poffsets;
    int* status;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&p);
}

// Epilogue for 32 consecutive columns [col0, col0+32) of one output row.
__device__ __forceinline__ void store_row_chunk(const TcParams& p, float* v, int64_t row_off, int col0, bool vec_ok) {
    const int ncols = min(32, p.N - col0);
    if (ncols <= 0) return;
    __nv_bfloat16* Zb = (__nv_bfloat16*)p.Z;
    if (vec_ok && ncols == 32) {
        const int64_t off = row_off + col0;
        if (p.epilogue == EPI_ACT) {
            if (Zb) {
                uint4* zp = (uint4*)(Zb + off);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    zp[i] = make_uint4(pack_bf16(v[8 * i], v[8 * i + 1]), pack_bf16(v[8 * i + 2], v[8 * i + 3]),
                                       pack_bf16(v[8 * i + 4], v[8 * i + 5]), pack_bf16(v[8 * i + 6], v[8 * i + 7]));
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = act_apply(p.act, v[i]);
        } else if (p.epilogue == EPI_DACT) {
            const uint4* zp = (const uint4*)(Zb + off);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 z = zp[i];
                const uint32_t w[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    v[8 * i + 2 * j] *= act_grad(p.act, bf16_lo(w[j]));
                    v[8 * i + 2 * j + 1] *= act_grad(p.act, bf16_hi(w[j]));
                }
            }
        }
        if (p.out_f32) {
            float4* cp = (float4*)((float*)p.C + off);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float4 o = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                if (p.accumulate) { const float4 c = cp[i]; o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w; }
                cp[i] = o;
            }
        } else {
            uint4* cp = (uint4*)((__nv_bfloat16*)p.C + off);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (p.accumulate) {
                    const uint4 c = cp[i];
                    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) { v[8 * i + 2 * j] += bf16_lo(w[j]); v[8 * i + 2 * j + 1] += bf16_hi(w[j]); }
                }
                cp[i] = make_uint4(pack_bf16(v[8 * i], v[8 * i + 1]), pack_bf16(v[8 * i + 2], v[8 * i + 3]),
                                   pack_bf16(v[8 * i + 4], v[8 * i + 5]), pack_bf16(v[8 * i + 6], v[8 * i + 7]));
            }
        }
        return;
    }
    for (int i = 0; i < ncols; ++i) {        // ragged edge or unaligned rows: scalar
        const int64_t off = row_off + col0 + i;
        float x = v[i];
        if (p.epilogue == EPI_ACT) {
            if (Zb) Zb[off] = __float2bfloat16(x);
            x = act_apply(p.act, x);
        } else if (p.epilogue == EPI_DACT) {
            x *= act_grad(p.act, __bfloat162float(Zb[off]));
        }
        if (p.out_f32) {
            float* C = (float*)p.C;
            C[off] = p.accumulate ? C[off] + x : x;
        } else {
            __nv_bfloat16* C = (__nv_bfloat16*)p.C;
            C[off] = __float2bfloat16(p.accumulate ? __bfloat162float(C[off]) + x : x);
        }
    }
}

template <int BN, int STAGES, bool A_KMAJOR, bool B_KMAJOR>
__global__ void __launch_bounds__(kThreads, 2)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcParams p) {
    constexpr uint32_t A_BYTES = BM * BK * 2;
    constexpr uint32_t B_BYTES = BN * BK * 2;
    constexpr uint32_t CHUNK_BYTES = 64 * BK * 2;            // one 64-wide MN-major box
    constexpr uint32_t TMEM_COLS = BN < 32 ? 32 : BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + STAGES * A_BYTES;
    uint64_t* full_bar = (uint64_t*)(smem + STAGES * (A_BYTES + B_BYTES));
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tmem_full_bar = empty_bar + STAGES;
    uint32_t* tmem_slot = (uint32_t*)(tmem_full_bar + 1);
    volatile int* dead = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN;
    const int m0 = blockIdx.y * BM;

    // ---- which problem does this CTA own?
    int expert = 0, k_row0 = 0, num_kb = (p.K + BK - 1) / BK, m_limit = p.M;
    int64_t c_base = 0;
    if (p.group == GROUP_M) {
        const int live = *p.n_tiles;
        if ((int)blockIdx.y >= live) return;
        expert = p.tile_expert[blockIdx.y];
        m_limit = min(p.M, live * kPad);
    } else if (p.group == GROUP_K) {
        expert = blockIdx.z;
        k_row0 = p.poffsets[expert];
        num_kb = (p.poffsets[expert + 1] - k_row0) / BK;
        c_base = (int64_t)expert * p.c_stride;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(tmem_full_bar, 1);
        *dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % STAGES;
                mbar_wait(&empty_bar[s], ((kb / STAGES) & 1) ^ 1, dead, p.status);
                mbar_expect_tx(&full_bar[s], A_BYTES + B_BYTES);
                const int k0 = k_row0 + kb * BK;
                uint8_t* a_dst = smem_a + s * A_BYTES;
                uint8_t* b_dst = smem_b + s * B_BYTES;
                if (A_KMAJOR) {
                    tma_load_2d(a_dst, &map_a, &full_bar[s], k0, m0);
                } else {
#pragma unroll
                    for (int c = 0; c < BM / 64; ++c) tma_load_2d(a_dst + c * CHUNK_BYTES, &map_a, &full_bar[s], m0 + 64 * c, k0);
                }
                if (B_KMAJOR) {
                    tma_load_2d(b_dst, &map_b, &full_bar[s], k0, expert * p.b_rows_per_expert + n0);
                } else {
#pragma unroll
                    for (int c = 0; c < BN / 64; ++c)
                        tma_load_2d(b_dst + c * CHUNK_BYTES, &map_b, &full_bar[s], n0 + 64 * c,
                                    expert * p.b_rows_per_expert + k0);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = instr_desc(BN, !A_KMAJOR, !B_KMAJOR);
        for (int kb = 0; kb < num_kb; ++kb) {
            const int s = kb % STAGES;
            mbar_wait(&full_bar[s], (kb / STAGES) & 1, dead, p.status);
            tc_fence_after();
            if (lane == 0) {
                const uint32_t a_addr = smem_u32(smem_a + s * A_BYTES);
                const uint32_t b_addr = smem_u32(smem_b + s * B_BYTES);
#pragma unroll
                for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                    const uint64_t da = A_KMAJOR ? smem_desc(a_addr + kk * UMMA_K * 2, 16, 1024)
                                                 : smem_desc(a_addr + kk * UMMA_K * 128, CHUNK_BYTES, 1024);
                    const uint64_t db = B_KMAJOR ? smem_desc(b_addr + kk * UMMA_K * 2, 16, 1024)
                                                 : smem_desc(b_addr + kk * UMMA_K * 128, CHUNK_BYTES, 1024);
                    umma_bf16(tmem_base, da, db, idesc, (kb | kk) != 0);
                }
                umma_commit(&empty_bar[s]);
            }
            __syncwarp();
        }
        if (lane == 0) {
            if (num_kb > 0) umma_commit(tmem_full_bar);
            else mbar_arrive(tmem_full_bar);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quad = warp & 3;                     // TMEM lanes 32*quad .. 32*quad+31
        mbar_wait(tmem_full_bar, 0, dead, p.status);
        tc_fence_after();
        const int row = m0 + quad * 32 + lane;
        const bool row_ok = row < m_limit;
        const int64_t row_off = c_base + (int64_t)row * p.ldc;
        const int esz = p.out_f32 ? 4 : 2;
        const bool vec_ok = ((p.ldc * esz) % 16 == 0) && ((c_base * esz) % 16 == 0) && (p.ldc % 8 == 0);
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            if (n0 + c * 32 >= p.N) break;               // uniform across the warp
            float v[32];
            if (num_kb > 0) {
                tmem_load_32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(c * 32), (uint32_t*)v);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = 0.0f;
            }
            if (row_ok) store_row_chunk(p, v, row_off, n0 + c * 32, vec_ok);
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return (EncodeTiledFn)sym;
    }();
    return fn;
}

// 2-D bf16 tensor map: `inner` contiguous elements per row, `rows` rows `ld` elements apart.
bool make_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t ld, uint32_t box_inner,
              uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {inner, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {box_inner, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int STAGES, bool AK, bool BKM>
cudaError_t launch(const CUtensorMap& ma, const CUtensorMap& mb, const TcParams& p, dim3 grid, cudaStream_t stream) {
    constexpr size_t smem = STAGES * (BM * BK * 2 + BN * BK * 2) + (2 * STAGES + 1) * 8 + 16 + 1024;
    static bool configured = false;
    auto kernel = gemm_tc_kernel<BN, STAGES, AK, BKM>;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kernel<<<grid, kThreads, smem, stream>>>(ma, mb, p);
    return cudaGetLastError();
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }

cudaError_t gemm_tc(const GemmArgs& g, int* status, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0) return cudaSuccess;
    constexpr int BN = 128, STAGES = 3;
    const int E = g.group == GROUP_NONE ? 1 : g.num_experts;
    CUtensorMap ma, mb;
    bool ok = true;
    TcParams p{};
    p.b_rows_per_expert = 0;
    // A: [M,K] (K-major) or [K,M] (MN-major).  In GROUP_K the contraction rows are the padded grouped rows.
    const uint64_t a_k_extent = g.group == GROUP_K ? (uint64_t)g.K : (uint64_t)g.K;
    if (g.a_kmajor) ok &= make_map(&ma, g.A, a_k_extent, (uint64_t)g.M, (uint64_t)g.lda, BK, BM);
    else ok &= make_map(&ma, g.A, (uint64_t)g.M, a_k_extent, (uint64_t)g.lda, 64, BK);
    // B: dense [N,K] / [K,N]; grouped weights are E consecutive such matrices (b_stride elements apart).
    if (g.b_kmajor) {
        const uint64_t rows_per = g.group == GROUP_M ? (uint64_t)(g.b_stride / g.ldb) : (uint64_t)g.N;
        ok &= make_map(&mb, g.B, (uint64_t)g.K, g.group == GROUP_M ? rows_per * E : (uint64_t)g.N, (uint64_t)g.ldb, BK, BN);
        p.b_rows_per_expert = g.group == GROUP_M ? (int)rows_per : 0;
    } else {
        const uint64_t rows_per = g.group == GROUP_M ? (uint64_t)(g.b_stride / g.ldb) : (uint64_t)g.K;
        ok &= make_map(&mb, g.B, (uint64_t)g.N, g.group == GROUP_M ? rows_per * E : (uint64_t)g.K, (uint64_t)g.ldb, 64, BK);
        p.b_rows_per_expert = g.group == GROUP_M ? (int)rows_per : 0;
    }
    if (!ok) return cudaErrorInvalidValue;
    p.C = g.C; p.Z = g.Z; p.ldc = g.ldc; p.c_stride = g.c_stride; p.M = g.M; p.N = g.N; p.K = g.K;
    p.out_f32 = g.out_f32; p.accumulate = g.accumulate; p.epilogue = g.epilogue; p.act = g.act; p.group = g.group;
    p.tile_expert = g.tile_expert; p.n_tiles = g.n_tiles; p.poffsets = g.poffsets; p.status = status;
    dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.group == GROUP_K ? E : 1);
    if (g.a_kmajor && g.b_kmajor) return launch<BN, STAGES, true, true>(ma, mb, p, grid, stream);
    if (g.a_kmajor && !g.b_kmajor) return launch<BN, STAGES, true, false>(ma, mb, p, grid, stream);
    if (!g.a_kmajor && !g.b_kmajor) return launch<BN, STAGES, false, false>(ma, mb, p, grid, stream);
    return cudaErrorNotSupported;
}

}  // namespace bigmac
