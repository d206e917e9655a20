// Shared pieces of the tcgen05 GEMM kernels: PTX wrappers (mbarrier, TMA, tcgen05), descriptors, the epilogue
// arithmetic and store paths, tile enumeration, and the host-side tensor-map helpers.
#pragma once
#include <cuda.h>

#include <cstdlib>

#include "internal.h"
#include "act.cuh"
#include "switches.h"

namespace bigmac {
namespace tc {

constexpr int kEpiWarps = 16;
constexpr uint32_t kBoxBytes = 32 * 64;                  // 32 rows x 32 bf16 columns
constexpr uint32_t kBoxBytesZ = 32 * 64;                 // 32 rows x 64 sigma' bytes (two chunks)
constexpr int kThreadsV2 = (2 + kEpiWarps) * 32;
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
// Non-blocking test of a phase (try_wait may park the thread for a while before it looks again; a chain of short
// dependent steps polls with this one instead).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ void mbar_spin(uint64_t* bar, uint32_t parity, volatile int* dead, int* status) {
    if (*dead) return;
    for (uint32_t i = 0; i < (kWaitLimit << 4); ++i) {
        if (mbar_test_wait(bar, parity)) return;
        if ((i & 4095u) == 4095u && *dead) return;
    }
    *dead = 1;
    atomicExch(status, 1);
}
// Bounded wait.  `dead` is a CTA-wide flag in shared memory: once any wait ran out nobody waits again.
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, volatile int* dead, int* status,
                                          uint32_t limit = kWaitLimit) {
    if (*dead) return;
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if ((i & 1023u) == 1023u && *dead) return;
    }
    *dead = 1;
    atomicExch(status, 1);
}

// The same wait with acquire at cluster scope: for barriers that guard data the other CTA of a pair wrote.
__device__ __forceinline__ void mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* dead, int* status) {
    if (*dead) return;
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.b32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
        if (done) return;
        if ((i & 1023u) == 1023u && *dead) return;
    }
    *dead = 1;
    atomicExch(status, 1);
}

// The wait of a single-thread role (producer, MMA issuer) whose barrier is usually complete already: one try, and
// only then the bounded loop with its flag checks.  These threads set the pace of the mainloop: with the general
// wait, descriptors rebuilt per MMA and modulo arithmetic per k slice, the MMA issuer took 745 cycles per slice
// where the tensor pipe needs 512.
__device__ __forceinline__ void mbar_wait_lean(uint64_t* bar, uint32_t parity, volatile int* dead, int* status) {
    if (mbar_try_wait(bar, parity)) return;
    mbar_wait(bar, parity, dead, status);
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
// Ask for a tensor map to be fetched now (the first TMA copy through a map otherwise waits for the fetch).
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
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

// ---- gathered operand rows (dispatch fused into a contraction's operand load)
// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros (the source is not read).
__device__ __forceinline__ void cp_async_16(uint32_t dst_smem, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// Arrive on an mbarrier of this CTA once all asynchronous copies this thread has issued so far have landed (the
// arrival is counted in the barrier's expected count: .noinc).
__device__ __forceinline__ void cp_async_arrive(uint64_t* bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Gathered operand rows are copied by kGatherWarps extra warps (the last warps of the CTA), 64 threads that each
// arrive on the stage's "full" barrier when their copies have landed; the MMA thread passes a proxy fence between
// that barrier and its first MMA on the stage (the copies are generic-proxy writes, the MMA reads through the async one).
constexpr int kGatherWarps = 2;
constexpr int kThreadsGather = kThreadsV2 + kGatherWarps * 32;

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
__device__ __forceinline__ void tmem_load_16_nowait(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
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
    int epi_parts;               // plain epilogues: this many (1, 2 or 4) of the four epilogue warps of a lane quadrant work
    const float* bias;           // GROUP_M: fp32 bias of expert e at bias + e*bias_stride, added before the epilogue; or null
    int64_t bias_stride;
    int n_split;                 // output columns from this one on come from map_b2 (K-major) and go to C2 (fp32); <0: none
    float* C2;
    int64_t ldc2;
    int N2;
    const int32_t* tile_expert;
    const int32_t* n_tiles;
    const int32_t* poffsets;
    // gathered A rows (dispatch fused into the operand load; K-major A, GROUP_M): row m of A is row
    // gather_rows[m] / gather_div of the matrix at gather_src (row stride gather_ld elements), zeros where
    // gather_rows[m] < 0 (padding rows); null = A is read as it lies
    const int32_t* gather_rows;
    const void* gather_src;
    int64_t gather_ld;
    int gather_div;
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

// Packed fp32 pairs (sm_100 f32x2 arithmetic): one instruction issue for two elements.
typedef unsigned long long f32x2_t;
__device__ __forceinline__ f32x2_t pk2(float a, float b) { f32x2_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ void upk2(f32x2_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ f32x2_t fma2(f32x2_t a, f32x2_t b, f32x2_t c) { f32x2_t d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d; }
__device__ __forceinline__ f32x2_t mul2(f32x2_t a, f32x2_t b) { f32x2_t d; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ f32x2_t add2(f32x2_t a, f32x2_t b) { f32x2_t d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }

// GELU(erf) and its derivative for two elements at once, with one special-function instruction per element (the
// A&S form above needs two, and the special-function pipe is the scarcest one in the epilogue).
// Phi(z) = sat(1/2 + z P(z^2)) with P the degree-8 weighted-minimax fit of (Phi(z) - 1/2) / z on |z| <= 4 (absolute
// error 4.5e-6 in Phi there).  The degree is even and the leading coefficient positive, so beyond the fitted range
// z P(z^2) only grows in magnitude and the saturating multiply-add pins Phi to 0 or 1 by itself (Phi(4) = 1 - 3.2e-5;
// checked up to |z| = 300, and z^2 or P overflowing to +inf saturates the same way): no clamp of the argument is
// needed.  The error of Phi stays below 3.2e-5 everywhere and that of z Phi(z) below 1.1e-4, a small fraction of a
// bf16 rounding step of the result.  phi(z) = exp(-z^2/2) / sqrt(2 pi) comes from one ex2.  Multiply-adds are
// issued as packed pairs.
constexpr float kPhiC0 = 0.39892274141311646f, kPhiC1 = -0.06641065329313278f, kPhiC2 = 0.009877530857920647f,
                kPhiC3 = -0.0011339453049004078f, kPhiC4 = 9.891336230793968e-05f, kPhiC5 = -6.295678304013563e-06f,
                kPhiC6 = 2.7166481686435873e-07f, kPhiC7 = -7.0053451928231425e-09f, kPhiC8 = 8.06635314098969e-11f;
__device__ __forceinline__ float fma_sat(float a, float b, float c) { float d; asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c)); return d; }
__device__ __forceinline__ void gelu_pair2(float z0, float z1, float& a0, float& a1, float& g0, float& g1) {
    const f32x2_t z = pk2(z0, z1);
    const f32x2_t w = mul2(z, z);
    f32x2_t P = fma2(w, pk2(kPhiC8, kPhiC8), pk2(kPhiC7, kPhiC7));
    P = fma2(w, P, pk2(kPhiC6, kPhiC6));
    P = fma2(w, P, pk2(kPhiC5, kPhiC5));
    P = fma2(w, P, pk2(kPhiC4, kPhiC4));
    P = fma2(w, P, pk2(kPhiC3, kPhiC3));
    P = fma2(w, P, pk2(kPhiC2, kPhiC2));
    P = fma2(w, P, pk2(kPhiC1, kPhiC1));
    P = fma2(w, P, pk2(kPhiC0, kPhiC0));
    float p0, p1;
    upk2(P, p0, p1);
    const f32x2_t cdf = pk2(fma_sat(z0, p0, 0.5f), fma_sat(z1, p1, 0.5f));
    float x0, x1;
    upk2(mul2(w, pk2(-0.72134752f, -0.72134752f)), x0, x1);
    const f32x2_t e = pk2(fast_ex2(x0), fast_ex2(x1));                                   // exp(-z^2 / 2)
    upk2(mul2(z, cdf), a0, a1);
    upk2(fma2(mul2(z, e), pk2(0.39894228f, 0.39894228f), cdf), g0, g1);
}

// sigma' is saved as one byte per element: q = round(200 sigma' + 27), i.e. sigma' = (q - 27) / 200 on [-0.135, 1.14]
// (GELU' lies in [-0.129, 1.129]; 0 and 1, all that ReLU needs, are exact).  The step 0.005 gives an absolute error
// of at most 0.0025 (rms 0.0014, about 0.23 % of sigma's rms - the size of a bf16 rounding) at half the bytes.
// Rounding uses the 2^23 trick: the low byte of float(2^23 + 27 + 200 g) is q.
constexpr float kSigScale = 200.0f, kSigMagic = 8388608.0f + 27.0f, kSigStep = 0.005f;
__device__ __forceinline__ uint32_t sig_quant4(float g0, float g1, float g2, float g3) {
    const f32x2_t scale = pk2(kSigScale, kSigScale), magic = pk2(kSigMagic, kSigMagic);
    float f0, f1, f2, f3;
    upk2(fma2(pk2(g0, g1), scale, magic), f0, f1);
    upk2(fma2(pk2(g2, g3), scale, magic), f2, f3);
    const uint32_t b0 = __float_as_uint(f0), b1 = __float_as_uint(f1), b2 = __float_as_uint(f2), b3 = __float_as_uint(f3);
    return __byte_perm(__byte_perm(b0, b1, 0x0040), __byte_perm(b2, b3, 0x0040), 0x5410);
}
__device__ __forceinline__ uint8_t sig_quant1(float g) { return (uint8_t)(__float_as_uint(fmaf(g, kSigScale, kSigMagic)) & 0xffu); }
template <int I>
__device__ __forceinline__ float sig_dequant(uint32_t word) {     // byte I of word -> sigma'
    const uint32_t bits = __byte_perm(word, 0x4B000000u, 0x7650 + I);
    return (__uint_as_float(bits) - kSigMagic) * kSigStep;
}
__device__ __forceinline__ float sig_dequant1(uint8_t q) { return ((float)q - 27.0f) * kSigStep; }
// v[0..31] *= sigma' from 8 words of 4 bytes: byte -> float bits by a permute, then (f - magic) (exact), * step and
// the product with v as packed pairs (two elements per issued instruction).
__device__ __forceinline__ void mul_by_sig32(float* v, const uint32_t* w) {
    const f32x2_t step = pk2(kSigStep, kSigStep), neg_magic = pk2(-kSigMagic, -kSigMagic);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t b0 = __byte_perm(w[i], 0x4B000000u, 0x7650), b1 = __byte_perm(w[i], 0x4B000000u, 0x7651);
        const uint32_t b2 = __byte_perm(w[i], 0x4B000000u, 0x7652), b3 = __byte_perm(w[i], 0x4B000000u, 0x7653);
        const f32x2_t s01 = mul2(add2(pk2(__uint_as_float(b0), __uint_as_float(b1)), neg_magic), step);
        const f32x2_t s23 = mul2(add2(pk2(__uint_as_float(b2), __uint_as_float(b3)), neg_magic), step);
        upk2(mul2(pk2(v[4 * i], v[4 * i + 1]), s01), v[4 * i], v[4 * i + 1]);
        upk2(mul2(pk2(v[4 * i + 2], v[4 * i + 3]), s23), v[4 * i + 2], v[4 * i + 3]);
    }
}

// Activation of 32 accumulator values in place; with WITH_G the 32 sigma' values are packed, one byte each, in wg[0..7].
// The activation is a compile-time constant here so that the switch is taken once per chunk, not per element.
template <int ACT, bool WITH_G, int COUNT = 32>
__device__ __forceinline__ void act_chunk(float* v, uint32_t* wg) {
#pragma unroll
    for (int i = 0; i < COUNT / 4; ++i) {
        float a[4], g[4];
        if (ACT == BIGMAC_ACT_GELU_ERF) {
            gelu_pair2(v[4 * i], v[4 * i + 1], a[0], a[1], g[0], g[1]);
            gelu_pair2(v[4 * i + 2], v[4 * i + 3], a[2], a[3], g[2], g[3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) act_pair(ACT, v[4 * i + j], a[j], g[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) v[4 * i + j] = a[j];
        if (WITH_G) wg[i] = sig_quant4(g[0], g[1], g[2], g[3]);
    }
}
template <bool WITH_G, int COUNT = 32>
__device__ __forceinline__ void act_chunk_any(int act, float* v, uint32_t* wg) {
    switch (act) {
        case BIGMAC_ACT_GELU_ERF: act_chunk<BIGMAC_ACT_GELU_ERF, WITH_G, COUNT>(v, wg); break;
        case BIGMAC_ACT_RELU: act_chunk<BIGMAC_ACT_RELU, WITH_G, COUNT>(v, wg); break;
        case BIGMAC_ACT_GELU_TANH: act_chunk<BIGMAC_ACT_GELU_TANH, WITH_G, COUNT>(v, wg); break;
        default: act_chunk<BIGMAC_ACT_IDENTITY, WITH_G, COUNT>(v, wg); break;
    }
}

// v[0..31] += b[0..31] (32 consecutive fp32 bias values, 16-byte aligned; every lane reads the same addresses).
__device__ __forceinline__ void add_bias32(float* v, const float* __restrict__ b) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 q = __ldg((const float4*)b + i);
        v[4 * i] += q.x; v[4 * i + 1] += q.y; v[4 * i + 2] += q.z; v[4 * i + 3] += q.w;
    }
}

// Epilogue for 32 consecutive columns [col0, col0+32) of one output row held in v[0..31].
__device__ __forceinline__ void store_row_chunk(const TcParams& p, float* v, int64_t row_off, int col0, bool vec_ok) {
    const int ncols = min(32, p.N - col0);
    if (ncols <= 0) return;
    uint8_t* Zb = (uint8_t*)p.Z;                 // sigma', one byte per element
    if (vec_ok && ncols == 32) {
        const int64_t off = row_off + col0;
        if (p.epilogue == EPI_ACT) {
            if (Zb) {
                uint32_t w[8];
                act_chunk_any<true>(p.act, v, w);
                st_global_32B(Zb + off, w);
            } else {
                act_chunk_any<false>(p.act, v, nullptr);
            }
        } else if (p.epilogue == EPI_DACT) {
            uint32_t w[8];
            ld_global_32B(Zb + off, w);
            mul_by_sig32(v, w);
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
            if (Zb) Zb[off] = sig_quant1(g);
        } else if (p.epilogue == EPI_DACT) {
            x *= sig_dequant1(Zb[off]);
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

// The sigma' bytes of two consecutive 32-column chunks share one box of 32 rows x 64 bytes (64-byte swizzle, like
// the bf16 box), so that every row segment a TMA copy moves to or from DRAM is 64 bytes: with 32-byte segments
// the byte tensor ran at well under half the bandwidth of the bf16 one.  `half` = which 32 of the 64 columns.
__device__ __forceinline__ void stage_row_u8(uint8_t* box, int lane, int half, const uint32_t* w /*8 words*/) {
    uint8_t* row = box + lane * 64;
    const int sw = (lane >> 1) & 3;
    st_shared_16B(row + (((2 * half) ^ sw) << 4), w[0], w[1], w[2], w[3]);
    st_shared_16B(row + (((2 * half + 1) ^ sw) << 4), w[4], w[5], w[6], w[7]);
}
__device__ __forceinline__ void load_row_u8(const uint8_t* box, int lane, int half, uint32_t* w /*8 words*/) {
    const uint8_t* row = box + lane * 64;
    const int sw = (lane >> 1) & 3;
    ld_shared_16B(row + (((2 * half) ^ sw) << 4), w);
    ld_shared_16B(row + (((2 * half + 1) ^ sw) << 4), w + 4);
}

// Epilogue of 32 columns through shared memory: v -> (sigma', sigma) or v * Z or v, packed to bf16 into the
// warp's staging boxes.  Returns nothing; the caller fences and issues the TMA stores.
__device__ __forceinline__ void stage_row_chunk(const TcParams& p, float* v, uint8_t* box_c, uint8_t* box_z, int lane,
                                                int zhalf) {
    uint32_t w[16];
    if (p.epilogue == EPI_ACT) {
        if (p.Z) {
            act_chunk_any<true>(p.act, v, w);
            stage_row_u8(box_z, lane, zhalf, w);
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

// The same for the epilogue warps of the one-CTA kernel, which walk t = first, first + stride, ...: for dense and
// row-grouped problems (row tile, column tile) are carried along (no divisions per tile) and the tile -> expert
// table is not read (only the loads need the expert; the outputs of a row-grouped problem are addressed by row).
struct TileWalk1 {
    int t, mt, nt;
};
__device__ __forceinline__ void walk1_init(TileWalk1& w, int first, int tiles_n) {
    w.t = first;
    w.mt = first / tiles_n;
    w.nt = first - w.mt * tiles_n;
}
__device__ __forceinline__ void walk1_next(TileWalk1& w, int stride, int step_m, int step_n, int tiles_n) {
    w.t += stride;
    w.mt += step_m;
    w.nt += step_n;
    if (w.nt >= tiles_n) { w.nt -= tiles_n; ++w.mt; }
}
__device__ __forceinline__ Tile walk1_tile(const TcParams& p, int BN, const TileWalk1& w, int tiles_m, int tiles_n) {
    if (p.group == GROUP_K || p.split_k > 1) return get_tile(p, BN, w.t, tiles_m, tiles_n);
    Tile tl;
    tl.m0 = w.mt * BM;
    tl.n0 = w.nt * BN;
    tl.expert = (p.bias && p.group == GROUP_M) ? p.tile_expert[w.mt] : 0;     // only the bias needs the expert here
    tl.k_row0 = 0;
    tl.num_kb = (p.K + BK - 1) / BK;
    tl.m_limit = p.group == GROUP_M ? min(p.M, tiles_m * kPad) : p.M;
    tl.c_base = 0;
    return tl;
}



// ------------------------------------------------------------------------------------------ host side
// Working epilogue warps per lane quadrant for plain epilogues: the request, else the debug switch, else 2.
inline int epi_parts_default(int requested) {
    const int sw = switches().epi_parts;
    const int v = requested ? requested : sw ? sw : 2;
    return (v == 1 || v == 2) ? v : 4;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
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
// 2-D byte tensor map (the saved sigma'): `inner` bytes per row, rows `ld` bytes apart, no swizzle.
inline bool make_map_u8(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t ld, uint32_t box_inner,
                        uint32_t box_rows, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {inner, rows};
    const cuuint64_t strides[1] = {ld};
    const cuuint32_t box[2] = {box_inner, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool make_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t ld, uint32_t box_inner,
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

inline int sm_count() {
    static int cached[64] = {};
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] > 0) return cached[dev];
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    cached[dev] = v;
    return v;
}

// Can this problem's output leave through shared memory and TMA stores?
inline bool tma_epilogue_possible(const GemmArgs& g) {
    return !g.out_f32 && !g.accumulate && g.split_k <= 1 && (g.ldc % 8 == 0) && ((uintptr_t)g.C % 16 == 0) &&
           ((uintptr_t)g.Z % 16 == 0) && (g.Z == nullptr || g.ldc % 16 == 0) &&
           (g.group != GROUP_K || (g.M % BM == 0 && g.c_stride == (int64_t)g.M * g.ldc));
}

}  // namespace tc
}  // namespace bigmac
