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
#include <cuda.h>

#include "internal.h"
#include "act.cuh"

namespace bigmac {

namespace {

constexpr int BM = 128;          // UMMA M
constexpr int BK = 64;           // bf16 elements per k slice = one 128-byte swizzle row
constexpr int UMMA_K = 16;
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

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(smem_u32(src))
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void ld_shared_16B(const void* ptr, uint32_t* w) {
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(smem_u32(ptr)));
}
__device__ __forceinline__ void st_shared_16B(void* ptr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(smem_u32(ptr)), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
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

__device__ __forceinline__ void tmem_load_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_load_32_nowait(uint32_t taddr, uint32_t* v) {
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
    int out_f32, accumulate, epilogue, act, group, num_experts;
    int tma_store;               // bf16 outputs leave through shared memory and TMA stores (map_c / map_z)
    int c_rows_per_expert;       // rows of the C tensor map per expert (GROUP_K); 0 otherwise
    int split_k;                 // dense only: the contraction is cut into split_k parts, part s writes C + s*M*ldc
    int b2_first_kb;             // k slices from this one on come from the second B tensor (map_b2); <0: none
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
__device__ __forceinline__ void st_global_32B(void* ptr, const uint32_t* w) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(ptr), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}
__device__ __forceinline__ void ld_global_32B(const void* ptr, uint32_t* w) {
    asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(ptr));
}

__device__ __forceinline__ float fast_rcp(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float fast_ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

// sigma(z) and sigma'(z) together.  For GELU(erf) the two share one exponential: with s = |z|/sqrt2,
// erf(s) = 1 - (a1 t + ... + a5 t^5) exp(-s^2), t = 1/(1 + 0.3275911 s) (absolute error below 1.5e-7, far
// inside bf16 resolution), Phi(z) = 1 - q or q with q = poly * exp(-z^2/2) / 2, phi(z) = exp(-z^2/2)/sqrt(2 pi).
__device__ __forceinline__ void act_pair(int act, float z, float& a, float& g) {
    if (act == BIGMAC_ACT_GELU_ERF) {
        const float t = fast_rcp(fmaf(0.23164190f, fabsf(z), 1.0f));          // 0.3275911 / sqrt 2
        float poly = fmaf(t, 0.5307027145f, -0.7265760135f);                    // coefficients halved
        poly = fmaf(t, poly, 0.7107068705f);
        poly = fmaf(t, poly, -0.142248368f);
        poly = fmaf(t, poly, 0.127414796f);
        const float e = fast_ex2(-0.72134752f * z * z);                            // exp(-z^2 / 2)
        const float q = poly * t * e;
        const float cdf = z >= 0.0f ? 1.0f - q : q;
        a = z * cdf;
        g = fmaf(z * e, 0.39894228f, cdf);
    } else if (act == BIGMAC_ACT_RELU) {
        a = z > 0.0f ? z : 0.0f;
        g = z > 0.0f ? 1.0f : 0.0f;
    } else {
        a = act_apply(act, z);
        g = act_grad(act, z);
    }
}

// Activation of 32 accumulator values in place; with WITH_G the 32 sigma' values are packed to bf16 pairs in wg.
// The activation is a compile-time constant here so that the switch is taken once per chunk, not per element.
template <int ACT, bool WITH_G>
__device__ __forceinline__ void act_chunk(float* v, uint32_t* wg) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float a0, g0, a1, g1;
        act_pair(ACT, v[2 * i], a0, g0);
        act_pair(ACT, v[2 * i + 1], a1, g1);
        v[2 * i] = a0; v[2 * i + 1] = a1;
        if (WITH_G) wg[i] = pack_bf16(g0, g1);
    }
}
template <bool WITH_G>
__device__ __forceinline__ void act_chunk_any(int act, float* v, uint32_t* wg) {
    switch (act) {
        case BIGMAC_ACT_GELU_ERF: act_chunk<BIGMAC_ACT_GELU_ERF, WITH_G>(v, wg); break;
        case BIGMAC_ACT_RELU: act_chunk<BIGMAC_ACT_RELU, WITH_G>(v, wg); break;
        case BIGMAC_ACT_GELU_TANH: act_chunk<BIGMAC_ACT_GELU_TANH, WITH_G>(v, wg); break;
        default: act_chunk<BIGMAC_ACT_IDENTITY, WITH_G>(v, wg); break;
    }
}

// Epilogue for 32 consecutive columns [col0, col0+32) of one output row held in v[0..31].
__device__ __forceinline__ void store_row_chunk(const TcParams& p, float* v, int64_t row_off, int col0, bool vec_ok) {
    const int ncols = min(32, p.N - col0);
    if (ncols <= 0) return;
    __nv_bfloat16* Zb = (__nv_bfloat16*)p.Z;
    if (vec_ok && ncols == 32) {
        const int64_t off = row_off + col0;
        if (p.epilogue == EPI_ACT) {
            if (Zb) {
                uint32_t w[16];
                act_chunk_any<true>(p.act, v, w);
                st_global_32B(Zb + off, w);
                st_global_32B(Zb + off + 16, w + 8);
            } else {
                act_chunk_any<false>(p.act, v, nullptr);
            }
        } else if (p.epilogue == EPI_DACT) {
            uint32_t w[16];
            ld_global_32B(Zb + off, w);
            ld_global_32B(Zb + off + 16, w + 8);
#pragma unroll
            for (int i = 0; i < 16; ++i) { v[2 * i] *= bf16_lo(w[i]); v[2 * i + 1] *= bf16_hi(w[i]); }
        }
        if (p.out_f32) {
            float* cp = (float*)p.C + off;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t w[8];
                if (p.accumulate) {
                    ld_global_32B(cp + 8 * i, w);
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[8 * i + j] += __uint_as_float(w[j]);
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) w[j] = __float_as_uint(v[8 * i + j]);
                st_global_32B(cp + 8 * i, w);
            }
        } else {
            __nv_bfloat16* cp = (__nv_bfloat16*)p.C + off;
            uint32_t w[16];
            if (p.accumulate) {
                ld_global_32B(cp, w);
                ld_global_32B(cp + 16, w + 8);
#pragma unroll
                for (int i = 0; i < 16; ++i) { v[2 * i] += bf16_lo(w[i]); v[2 * i + 1] += bf16_hi(w[i]); }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
            st_global_32B(cp, w);
            st_global_32B(cp + 16, w + 8);
        }
        return;
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) {           // ragged edge or unaligned rows: scalar (unrolled: v stays in registers)
        if (i >= ncols) break;
        const int64_t off = row_off + col0 + i;
        float x = v[i];
        if (p.epilogue == EPI_ACT) {
            float g;
            act_pair(p.act, x, x, g);
            if (Zb) Zb[off] = __float2bfloat16(g);
        } else if (p.epilogue == EPI_DACT) {
            x *= __bfloat162float(Zb[off]);
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

// One 32-row x 32-column bf16 box of an output in shared memory, laid out for a TMA store with the 64-byte
// swizzle: row `lane` occupies 64 bytes, its 16-byte piece j sits at piece j ^ ((lane >> 1) & 3), which makes
// the 32 lanes' 16-byte stores conflict-free.
__device__ __forceinline__ void stage_row_bf16(uint8_t* box, int lane, const uint32_t* w /*16 packed pairs*/) {
    uint8_t* row = box + lane * 64;
    const int sw = (lane >> 1) & 3;
#pragma unroll
    for (int j = 0; j < 4; ++j) st_shared_16B(row + ((j ^ sw) << 4), w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
}

// Epilogue of 32 columns through shared memory: v -> (sigma', sigma) or v * Z or v, packed to bf16 into the
// warp's staging boxes.  Returns nothing; the caller fences and issues the TMA stores.
__device__ __forceinline__ void stage_row_chunk(const TcParams& p, float* v, uint8_t* box_c, uint8_t* box_z, int lane,
                                                int64_t row_off, int col0, bool row_ok) {
    uint32_t w[16];
    if (p.epilogue == EPI_ACT) {
        if (p.Z) {
            act_chunk_any<true>(p.act, v, w);
            stage_row_bf16(box_z, lane, w);
        } else {
            act_chunk_any<false>(p.act, v, nullptr);
        }
    }   // EPI_DACT: the caller has already multiplied by the prefetched sigma'
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
    stage_row_bf16(box_c, lane, w);
}

// What one CTA works on next: output tile (m0, n0) of problem `expert`, contraction rows
// [k_row0, k_row0 + 64*num_kb).
struct Tile {
    int m0, n0, expert, k_row0, num_kb, m_limit;
    int64_t c_base;
};

__device__ __forceinline__ int total_tiles(const TcParams& p, int BN, int& tiles_m, int& tiles_n) {
    tiles_n = (p.N + BN - 1) / BN;
    tiles_m = p.group == GROUP_M ? min(*p.n_tiles, (p.M + BM - 1) / BM) : (p.M + BM - 1) / BM;
    return tiles_m * tiles_n * (p.group == GROUP_K ? p.num_experts : p.split_k);
}

__device__ __forceinline__ Tile get_tile(const TcParams& p, int BN, int t, int tiles_m, int tiles_n) {
    Tile tl;
    const int per = tiles_m * tiles_n;
    const int e = (p.group == GROUP_K || p.split_k > 1) ? t / per : 0;     // expert, or part of a split contraction
    const int r = t - e * per;
    tl.m0 = (r / tiles_n) * BM;
    tl.n0 = (r % tiles_n) * BN;
    tl.expert = p.group == GROUP_K ? e : 0;
    tl.k_row0 = 0;
    tl.num_kb = (p.K + BK - 1) / BK;
    tl.m_limit = p.M;
    tl.c_base = 0;
    if (p.group != GROUP_K && p.split_k > 1) {
        const int per_part = (tl.num_kb + p.split_k - 1) / p.split_k;
        tl.k_row0 = e * per_part * BK;
        tl.num_kb = max(0, min(per_part, tl.num_kb - e * per_part));
        tl.c_base = (int64_t)e * p.M * p.ldc;
    }
    if (p.group == GROUP_M) {
        tl.expert = p.tile_expert[r / tiles_n];
        tl.m_limit = min(p.M, tiles_m * kPad);
    } else if (p.group == GROUP_K) {
        tl.k_row0 = p.poffsets[e];
        tl.num_kb = (p.poffsets[e + 1] - tl.k_row0) / BK;
        tl.c_base = (int64_t)e * p.c_stride;
    }
    return tl;
}

constexpr int kEpiWarps = 16;
constexpr uint32_t kBoxBytes = 32 * 64;                  // 32 rows x 32 bf16 columns
constexpr int kThreadsV2 = (2 + kEpiWarps) * 32;

// Persistent kernel: gridDim.x CTAs (one per SM) walk the tile list with stride gridDim.x.  The
// accumulator is double-buffered in tensor memory (2 x BN columns), so the epilogue of tile i overlaps
// the MMAs of tile i+1.
template <int BN, int STAGES, bool A_KMAJOR, bool B_KMAJOR, bool TMA_EPI>
__global__ void __launch_bounds__(kThreadsV2, 1)
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

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int tiles_m, tiles_n;
    const int total = total_tiles(p, BN, tiles_m, tiles_n);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&tmem_full_bar[s], 1); mbar_init(&tmem_empty_bar[s], kEpiWarps); }
        for (int s = 0; s < kEpiWarps; ++s) mbar_init(&z_bar[s], 1);
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
            uint32_t it = 0;
            for (int t = blockIdx.x; t < total; t += gridDim.x) {
                const Tile tl = get_tile(p, BN, t, tiles_m, tiles_n);
                for (int kb = 0; kb < tl.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    mbar_wait(&empty_bar[s], ((it / STAGES) & 1) ^ 1, dead, p.status);
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
                        tma_load_2d(b_dst, &map_b, &full_bar[s], k0, tl.expert * p.b_rows_per_expert + tl.n0);
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
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = instr_desc(BN, !A_KMAJOR, !B_KMAJOR);
        uint32_t it = 0, local = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++local) {
            const Tile tl = get_tile(p, BN, t, tiles_m, tiles_n);
            const uint32_t acc = local & 1;
            mbar_wait(&tmem_empty_bar[acc], ((local >> 1) & 1) ^ 1, dead, p.status);
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * BN;
            for (int kb = 0; kb < tl.num_kb; ++kb, ++it) {
                const int s = it % STAGES;
                mbar_wait(&full_bar[s], (it / STAGES) & 1, dead, p.status);
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
                        umma_bf16(d_tmem, da, db, idesc, (kb | kk) != 0);
                    }
                    umma_commit(&empty_bar[s]);
                }
                __syncwarp();
            }
            if (lane == 0) {
                if (tl.num_kb > 0) umma_commit(&tmem_full_bar[acc]);
                else mbar_arrive(&tmem_full_bar[acc]);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..17)
        const int quad = warp & 3;                     // TMEM lanes 32*quad .. 32*quad+31
        constexpr int COLS_PER_WARP = BN / (kEpiWarps / 4);
        constexpr int CHUNKS = COLS_PER_WARP / 32;
        const int part = (warp - 2) >> 2;              // which COLS_PER_WARP-wide slice of the tile's columns
        uint8_t* box_c = staging + (warp - 2) * 2 * kBoxBytes;
        uint8_t* box_z = box_c + kBoxBytes;
        const int esz = p.out_f32 ? 4 : 2;
        const bool vec_ok = ((p.ldc * esz) % 32 == 0) && ((p.c_stride * esz) % 32 == 0) && (p.ldc % 16 == 0) &&
                            (((uintptr_t)p.C) % 32 == 0) && (((uintptr_t)p.Z) % 32 == 0);
        // EPI_DACT with staged stores: the saved sigma' box of the next chunk is fetched by TMA into box_z one
        // chunk ahead (across tiles too), so its DRAM latency is hidden behind the MMAs and the previous chunk.
        const bool z_prefetch = TMA_EPI && p.epilogue == EPI_DACT;
        uint64_t* my_z_bar = &z_bar[warp - 2];
        uint32_t z_count = 0;
        auto issue_z = [&](const Tile& tile, int c) {
            if (lane == 0) {
                mbar_expect_tx(my_z_bar, kBoxBytes);
                tma_load_2d(box_z, &map_z, my_z_bar, tile.n0 + part * COLS_PER_WARP + c * 32, tile.m0 + quad * 32);
            }
        };
        if (z_prefetch && (int)blockIdx.x < total) issue_z(get_tile(p, BN, blockIdx.x, tiles_m, tiles_n), 0);
        uint32_t local = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++local) {
            const Tile tl = get_tile(p, BN, t, tiles_m, tiles_n);
            const uint32_t acc = local & 1;
            mbar_wait(&tmem_full_bar[acc], (local >> 1) & 1, dead, p.status);
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
                if (TMA_EPI) {
                    if (lane == 0) tma_store_wait_read();        // previous boxes of this warp have left smem
                    __syncwarp();
                    if (z_prefetch) {
                        mbar_wait(my_z_bar, z_count & 1, dead, p.status);
                        ++z_count;
                        uint32_t w[16];
                        const uint8_t* zrow = box_z + lane * 64;
                        const int sw = (lane >> 1) & 3;
#pragma unroll
                        for (int j = 0; j < 4; ++j) ld_shared_16B(zrow + ((j ^ sw) << 4), w + 4 * j);
                        fence_async_smem();
                        __syncwarp();
                        if (c + 1 < CHUNKS) issue_z(tl, c + 1);
                        else if (t + (int)gridDim.x < total) issue_z(get_tile(p, BN, t + gridDim.x, tiles_m, tiles_n), 0);
#pragma unroll
                        for (int i = 0; i < 16; ++i) { v[2 * i] *= bf16_lo(w[i]); v[2 * i + 1] *= bf16_hi(w[i]); }
                    }
                    stage_row_chunk(p, v, box_c, box_z, lane, row_off, col0, row_ok);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        const int row0 = tl.expert * p.c_rows_per_expert + tl.m0 + quad * 32;
                        tma_store_2d(&map_c, box_c, col0, row0);
                        if (p.epilogue == EPI_ACT && p.Z) tma_store_2d(&map_z, box_z, col0, row0);
                        tma_store_commit();
                    }
                } else if (row_ok) {
                    store_row_chunk(p, v, row_off, col0, vec_ok);
                }
            }
        }
        if (TMA_EPI && lane == 0) tma_store_wait_all();
    }
    tc_fence_before();
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
              uint32_t box_rows, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {inner, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {box_inner, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int n = []() {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
            return 148;
        return v;
    }();
    return n;
}

template <int BN, int STAGES, bool AK, bool BKM, bool TMA_EPI>
cudaError_t launch(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const CUtensorMap& mz,
                   const CUtensorMap& mb2, const TcParams& p, int max_tiles, cudaStream_t stream) {
    constexpr size_t smem = STAGES * (BM * BK * 2 + BN * BK * 2) + (TMA_EPI ? kEpiWarps * 2 * kBoxBytes : 0) +
                            (2 * STAGES + 4 + kEpiWarps) * 8 + 16 + 1024;
    static bool configured = false;
    auto kernel = gemm_tc_kernel<BN, STAGES, AK, BKM, TMA_EPI>;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int grid = max_tiles < sm_count() ? max_tiles : sm_count();
    kernel<<<grid, kThreadsV2, smem, stream>>>(ma, mb, mc, mz, mb2, p);
    return cudaGetLastError();
}

template <int BN, int STAGES, bool TMA_EPI>
cudaError_t dispatch(const GemmArgs& g, int* status, cudaStream_t stream) {
    const int E = g.group == GROUP_NONE ? 1 : g.num_experts;
    CUtensorMap ma, mb;
    bool ok = true;
    TcParams p{};
    // A: [M,K] (K-major) or [K,M] (MN-major).  In GROUP_K, K is the row extent of the padded grouped buffers.
    if (g.a_kmajor) ok &= make_map(&ma, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, BM);
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
    if (g.B2) {
        if (g.b_kmajor || g.group != GROUP_NONE || g.b2_first_k % BK) return cudaErrorInvalidValue;
        ok &= make_map(&mb2, g.B2, (uint64_t)g.N, (uint64_t)(g.K - g.b2_first_k), (uint64_t)g.ldb2, 64, BK);
        // the first tensor ends where the second begins
        ok &= make_map(&mb, g.B, (uint64_t)g.N, (uint64_t)g.b2_first_k, (uint64_t)g.ldb, 64, BK);
        p.b2_first_kb = g.b2_first_k / BK;
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
            ok &= make_map(&mz, g.Z, (uint64_t)g.N, c_rows, (uint64_t)g.ldc, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    }
    if (!ok) return cudaErrorInvalidValue;
    p.tma_store = tma_store ? 1 : 0;
    p.split_k = (g.group == GROUP_NONE && g.split_k > 1) ? g.split_k : 1;
    p.c_rows_per_expert = g.group == GROUP_K ? g.M : 0;
    p.b_rows_per_expert = (int)rows_per;
    p.C = g.C; p.Z = g.Z; p.ldc = g.ldc; p.c_stride = g.c_stride; p.M = g.M; p.N = g.N; p.K = g.K;
    p.out_f32 = g.out_f32; p.accumulate = g.accumulate; p.epilogue = g.epilogue; p.act = g.act; p.group = g.group;
    p.num_experts = E; p.tile_expert = g.tile_expert; p.n_tiles = g.n_tiles; p.poffsets = g.poffsets; p.status = status;
    const int64_t tiles = (int64_t)((g.N + BN - 1) / BN) * ((g.M + BM - 1) / BM) * (g.group == GROUP_K ? E : p.split_k);
    const int max_tiles = tiles > (1 << 30) ? (1 << 30) : (int)tiles;
    if (g.a_kmajor && g.b_kmajor) return launch<BN, STAGES, true, true, TMA_EPI>(ma, mb, mc, mz, mb2, p, max_tiles, stream);
    if (g.a_kmajor && !g.b_kmajor) return launch<BN, STAGES, true, false, TMA_EPI>(ma, mb, mc, mz, mb2, p, max_tiles, stream);
    if (!g.a_kmajor && !g.b_kmajor) return launch<BN, STAGES, false, false, TMA_EPI>(ma, mb, mc, mz, mb2, p, max_tiles, stream);
    return cudaErrorNotSupported;
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }
int gemm_tc_sm_count() { return sm_count(); }

// Can this problem's output leave through shared memory and TMA stores?
bool tma_epilogue_possible(const GemmArgs& g) {
    return !g.out_f32 && !g.accumulate && g.split_k <= 1 && (g.ldc % 8 == 0) && ((uintptr_t)g.C % 16 == 0) &&
           ((uintptr_t)g.Z % 16 == 0) &&
           (g.group != GROUP_K || (g.M % BM == 0 && g.c_stride == (int64_t)g.M * g.ldc));
}

cudaError_t gemm_tc(const GemmArgs& g, int* status, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0) return cudaSuccess;
    // Output-heavy problems (wide rows: activations, ascend, dx) stage their stores through shared memory and
    // TMA, which costs one pipeline stage; contraction-heavy ones keep the deeper pipeline and store directly.
    const bool staged = tma_epilogue_possible(g) && g.N >= 1024 && g.N % 256 == 0 && (g.epilogue != EPI_DACT || g.group != GROUP_K);
    if (g.N >= 256) return staged ? dispatch<256, 3, true>(g, status, stream) : dispatch<256, 4, false>(g, status, stream);
    return dispatch<128, 6, false>(g, status, stream);
}

}  // namespace bigmac
