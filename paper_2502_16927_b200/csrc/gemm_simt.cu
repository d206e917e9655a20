// Plain FMA GEMM: C[m,n] (+)= epilogue(sum_k A(m,k) B(n,k)), fp32 accumulation in a fixed order.
// This is the arithmetic of the fp32 layer (tensor cores have no true-fp32 mode, and the routing
// margin and the 1e-4 tolerance of that path need one) and a debugging reference for the bf16 path.
// 64x64 output tile per block, 16-deep k slices staged in shared memory, 4x4 outputs per thread.
#include "internal.h"
#include "act.cuh"

namespace bigmac {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <typename T> __device__ __forceinline__ float ld(const T* p) { return (float)*p; }

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
    grid_dependency_wait();
    grid_dependency_launch();
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN + 4];
    const T* A = (const T*)g.A;
    const T* B = (const T*)g.B;
    int64_t c_base = 0;
    const float* bias = nullptr;
    int m_limit = g.M, k_begin = 0, k_end = g.K;
    const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
    if (g.group == GROUP_M) {
        const int tile = m0 / kPad;
        if (tile >= *g.n_tiles) return;
        B += (int64_t)g.tile_expert[tile] * g.b_stride;
        if (g.bias) bias = g.bias + (int64_t)g.tile_expert[tile] * g.bias_stride;
        m_limit = min(g.M, *g.n_tiles * kPad);
    } else if (g.group == GROUP_K) {
        const int e = blockIdx.z;
        k_begin = g.poffsets[e];
        k_end = g.poffsets[e + 1];
        c_base = (int64_t)e * g.c_stride;
    }
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    float acc[4][4] = {};
    for (int k0 = k_begin; k0 < k_end; k0 += TK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = tid + i * 256;
            int m, kk;
            if (g.a_kmajor) { kk = idx % TK; m = idx / TK; } else { m = idx % TM; kk = idx / TM; }
            const int gm = m0 + m, gk = k0 + kk;
            float v = 0.0f;
            if (gm < m_limit && gk < k_end) v = g.a_kmajor ? ld(A + (int64_t)gm * g.lda + gk) : ld(A + (int64_t)gk * g.lda + gm);
            As[kk][m] = v;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = tid + i * 256;
            int n, kk;
            if (g.b_kmajor) { kk = idx % TK; n = idx / TK; } else { n = idx % TN; kk = idx / TN; }
            const int gn = n0 + n, gk = k0 + kk;
            float v = 0.0f;
            if (gn < g.N && gk < k_end) v = g.b_kmajor ? ld(B + (int64_t)gn * g.ldb + gk) : ld(B + (int64_t)gk * g.ldb + gn);
            Bs[kk][n] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= m_limit) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= g.N) continue;
            const int64_t off = c_base + (int64_t)gm * g.ldc + gn;
            float v = acc[i][j];
            if (bias) v += bias[gn];
            if (g.epilogue == EPI_ACT) {
                if (g.Z) ((T*)g.Z)[off] = (T)act_grad(g.act, v);
                v = act_apply(g.act, v);
            } else if (g.epilogue == EPI_DACT) {
                v *= (float)((const T*)g.Z)[off];
            }
            if (g.out_f32) {
                float* C = (float*)g.C;
                C[off] = g.accumulate ? C[off] + v : v;
            } else {
                T* C = (T*)g.C;
                C[off] = (T)(g.accumulate ? (float)C[off] + v : v);
            }
        }
    }
}

}  // namespace

cudaError_t gemm_simt(const GemmArgs& g, int dtype, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0) return cudaSuccess;
    dim3 grid((g.M + TM - 1) / TM, (g.N + TN - 1) / TN, g.group == GROUP_K ? g.num_experts : 1);
    if (dtype == BIGMAC_BF16)
        (void)launch_chained(gemm_simt_kernel<__nv_bfloat16>, grid, 256, 0, stream, g);
    else
        (void)launch_chained(gemm_simt_kernel<float>, grid, 256, 0, stream, g);
    return cudaGetLastError();
}

}  // namespace bigmac
