// Small-batch (decode-shaped) inference forward of the BigMac layer in ONE cooperative kernel.
//
// For a handful of tokens the layer is a chain of matrix-vector products that is bound by streaming the touched
// weights once (W'_down, W_gate, the selected experts' W1/W2, W'_up) and by launch latency; ten separate launches
// cost far more than the arithmetic.  All SMs walk five phases separated by grid-wide barriers:
//   A  [x' | logits] = x [W'_down ; W_gate]^T           one warp per weight row, all tokens at once
//   B  top-k + softmax gate values                       one warp per token
//   C  a = sigma(W1_e x')  for every routed slot          eight weight rows per warp task
//   D  u = W2_e a                                         four weight rows per warp task
//   E  y' = sum_j p_j u_j ;  y = W'_up y'                 eight weight rows per warp task
// Weights are read as 16-byte vectors, products accumulate in fp32, intermediates stay fp32 in scratch.
// The grid barrier is a bounded spin on a global counter (cooperative launch guarantees co-residency); if the
// bound is ever hit the kernel records BIGMAC_ERR_TIMEOUT in the status word and runs on, so it always ends.
#include "internal.h"
#include "act.cuh"

namespace bigmac {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kDecodeThreads = 256;
constexpr int kDecodeMaxTokens = 16;

struct DecodeArgs {
    const __nv_bfloat16 *x, *w_gate, *w_down, *w1, *w2, *w_up;
    const float* b_gate;
    __nv_bfloat16* y;
    float *logits, *x_lo, *a, *u;      // scratch: [T,E], [T,r], [T*k,h], [T*k,r]
    int32_t* topk_idx;
    float* topk_w;
    unsigned* barrier;                 // zero before the launch
    int* status;
    int T, d, r, h, E, k, act;
};

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(kFull, v, off);
    return v;
}

// All CTAs of the (cooperative) grid meet here; `phase` counts the barriers passed so far.
__device__ __forceinline__ void grid_barrier(unsigned* counter, unsigned phase, int* status) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        const unsigned target = (phase + 1) * gridDim.x;
        unsigned seen = 0;
        for (uint32_t i = 0; i < (1u << 24); ++i) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter));
            if (seen >= target) break;
        }
        if (seen < target) atomicExch(status, 1);
        __threadfence();
    }
    __syncthreads();
}

// dot products of ROWS consecutive weight rows (each `n` bf16, row-major, `ld` apart) with `nv` fp32 vectors
// v[t*v_ld + 0..n) held in shared or global memory; lanes stride over 16-byte pieces.  out[row][t] valid in all lanes.
template <int ROWS, int NV>
__device__ __forceinline__ void rows_dot(const __nv_bfloat16* w, int64_t ld, int n, const float* v, int v_ld, int nv,
                                         float (&out)[ROWS][NV]) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int i = 0; i < ROWS; ++i)
#pragma unroll
        for (int t = 0; t < NV; ++t) out[i][t] = 0.0f;
    for (int c = lane; c < n / 8; c += 32) {
        uint4 wv[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) wv[i] = *reinterpret_cast<const uint4*>(w + i * ld + c * 8);
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            float wf[8];
            unpack8(wv[i], wf);
#pragma unroll
            for (int t = 0; t < NV; ++t) {
                if (t < nv) {
                    const float4 v0 = *reinterpret_cast<const float4*>(v + (int64_t)t * v_ld + c * 8);
                    const float4 v1 = *reinterpret_cast<const float4*>(v + (int64_t)t * v_ld + c * 8 + 4);
                    float acc = out[i][t];
                    acc = fmaf(wf[0], v0.x, acc); acc = fmaf(wf[1], v0.y, acc); acc = fmaf(wf[2], v0.z, acc); acc = fmaf(wf[3], v0.w, acc);
                    acc = fmaf(wf[4], v1.x, acc); acc = fmaf(wf[5], v1.y, acc); acc = fmaf(wf[6], v1.z, acc); acc = fmaf(wf[7], v1.w, acc);
                    out[i][t] = acc;
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < ROWS; ++i)
#pragma unroll
        for (int t = 0; t < NV; ++t) out[i][t] = warp_sum(out[i][t]);
}

// A: one weight row of [W'_down ; W_gate] per warp, against the (at most NV) tokens staged in `xs` as fp32 [T,d].
template <int NV>
__device__ __forceinline__ void phase_a(const DecodeArgs& p, const float* xs, int gwarp, int nwarps) {
    const int lane = threadIdx.x & 31;
    for (int j = gwarp; j < p.r + p.E; j += nwarps) {
        const __nv_bfloat16* row = j < p.r ? p.w_down + (int64_t)j * p.d : p.w_gate + (int64_t)(j - p.r) * p.d;
        float acc[1][NV];
        rows_dot<1, NV>(row, p.d, p.d, xs, p.d, p.T, acc);
        float mine = 0.0f;                                  // lane t keeps token t's value
#pragma unroll
        for (int t = 0; t < NV; ++t) mine = lane == t ? acc[0][t] : mine;
        if (lane < p.T) {
            if (j < p.r) p.x_lo[lane * p.r + j] = mine;
            else p.logits[lane * p.E + (j - p.r)] = mine + (p.b_gate ? p.b_gate[j - p.r] : 0.0f);
        }
    }
}

// E: eight rows of W'_up per warp task against y' [T,r] staged in `ys`.
template <int NV>
__device__ __forceinline__ void phase_e(const DecodeArgs& p, const float* ys, int gwarp, int nwarps) {
    const int lane = threadIdx.x & 31;
    for (int task = gwarp; task < p.d / 8; task += nwarps) {
        const int c0 = task * 8;
        float acc[8][NV];
        rows_dot<8, NV>(p.w_up + (int64_t)c0 * p.r, p.r, p.r, ys, p.r, p.T, acc);
#pragma unroll
        for (int t = 0; t < NV; ++t) {
            float v = acc[0][t];
#pragma unroll
            for (int i = 1; i < 8; ++i) v = lane == i ? acc[i][t] : v;
            if (lane < 8 && t < p.T) p.y[(int64_t)t * p.d + c0 + lane] = __float2bfloat16(v);
        }
    }
}

__global__ void __launch_bounds__(kDecodeThreads, 1) decode_forward_kernel(const DecodeArgs p) {
    extern __shared__ float smem_f[];                       // phase A: x as fp32 [T,d]; C: x' [T,r]; E: y' [T,r]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warps_per_cta = kDecodeThreads / 32;
    const int gwarp = blockIdx.x * warps_per_cta + warp, nwarps = gridDim.x * warps_per_cta;
    const int T = p.T, N = p.T * p.k;

    // ---- A: descend + gate logits (the gate reads x, not x')
    for (int i = threadIdx.x; i < T * p.d; i += kDecodeThreads) smem_f[i] = __bfloat162float(p.x[i]);
    __syncthreads();
    switch (T <= 1 ? 1 : T <= 2 ? 2 : T <= 4 ? 4 : T <= 8 ? 8 : 16) {
        case 1: phase_a<1>(p, smem_f, gwarp, nwarps); break;
        case 2: phase_a<2>(p, smem_f, gwarp, nwarps); break;
        case 4: phase_a<4>(p, smem_f, gwarp, nwarps); break;
        case 8: phase_a<8>(p, smem_f, gwarp, nwarps); break;
        default: phase_a<16>(p, smem_f, gwarp, nwarps); break;
    }
    grid_barrier(p.barrier, 0, p.status);

    // ---- B: top-k by (logit descending, expert id ascending), softmax over the k kept logits
    if (gwarp < T) {
        const int t = gwarp;
        const float* l = p.logits + (int64_t)t * p.E;
        uint32_t taken = 0;                                 // bit i: expert lane + 32*i already chosen
        float top = 0.0f, part = 0.0f;
        for (int j = 0; j < p.k; ++j) {
            float best = -INFINITY;
            int best_e = 0x7fffffff;                         // "no candidate yet"; k <= E, so every round ends with a real id
            for (int i = 0, e = lane; e < p.E; ++i, e += 32) {
                float v = l[e];
                v = v == v ? v : -INFINITY;                  // NaN is ordered as -inf
                if (!((taken >> i) & 1u) && (best_e == 0x7fffffff || v > best)) { best = v; best_e = e; }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const float ov = __shfl_xor_sync(kFull, best, off);
                const int oe = __shfl_xor_sync(kFull, best_e, off);
                if (ov > best || (ov == best && oe < best_e)) { best = ov; best_e = oe; }
            }
            if (best_e != 0x7fffffff && (best_e & 31) == lane) taken |= 1u << (best_e >> 5);
            if (j == 0) top = best;
            const float ex = top == -INFINITY ? 1.0f : expf(best - top);   // only -inf logits kept: 1/k each
            part += ex;
            if (lane == 0) { p.topk_idx[t * p.k + j] = best_e; p.topk_w[t * p.k + j] = ex; }
        }
        __syncwarp();
        for (int j = lane; j < p.k; j += 32) p.topk_w[t * p.k + j] /= part;
    }
    grid_barrier(p.barrier, 1, p.status);

    // ---- C: a = sigma(W1_e x') per routed slot
    for (int i = threadIdx.x; i < T * p.r; i += kDecodeThreads) smem_f[i] = p.x_lo[i];
    __syncthreads();
    {
        const int groups = p.h / 8;                          // h is a multiple of 8
        for (int task = gwarp; task < N * groups; task += nwarps) {
            const int s = task / groups, q0 = (task % groups) * 8;
            const int e = p.topk_idx[s], t = s / p.k;
            float acc[8][1];
            rows_dot<8, 1>(p.w1 + ((int64_t)e * p.h + q0) * p.r, p.r, p.r, smem_f + t * p.r, p.r, 1, acc);
            if (lane < 8) {
                float z = acc[0][0];
#pragma unroll
                for (int i = 1; i < 8; ++i) z = lane == i ? acc[i][0] : z;
                p.a[(int64_t)s * p.h + q0 + lane] = act_apply(p.act, z);
            }
        }
    }
    grid_barrier(p.barrier, 2, p.status);

    // ---- D: u = W2_e a per routed slot
    {
        const int groups = p.r / 4;
        for (int task = gwarp; task < N * groups; task += nwarps) {
            const int s = task / groups, c0 = (task % groups) * 4;
            const int e = p.topk_idx[s];
            float acc[4][1];
            rows_dot<4, 1>(p.w2 + ((int64_t)e * p.r + c0) * p.h, p.h, p.h, p.a + (int64_t)s * p.h, p.h, 1, acc);
            if (lane < 4) {
                float v = acc[0][0];
#pragma unroll
                for (int i = 1; i < 4; ++i) v = lane == i ? acc[i][0] : v;
                p.u[(int64_t)s * p.r + c0 + lane] = v;
            }
        }
    }
    grid_barrier(p.barrier, 3, p.status);

    // ---- E: combine in slot order, then ascend
    for (int i = threadIdx.x; i < T * p.r; i += kDecodeThreads) {
        const int t = i / p.r, c = i % p.r;
        float acc = 0.0f;
        for (int j = 0; j < p.k; ++j) acc = fmaf(p.topk_w[t * p.k + j], p.u[(int64_t)(t * p.k + j) * p.r + c], acc);
        smem_f[i] = acc;
    }
    __syncthreads();
    switch (T <= 1 ? 1 : T <= 2 ? 2 : T <= 4 ? 4 : T <= 8 ? 8 : 16) {
        case 1: phase_e<1>(p, smem_f, gwarp, nwarps); break;
        case 2: phase_e<2>(p, smem_f, gwarp, nwarps); break;
        case 4: phase_e<4>(p, smem_f, gwarp, nwarps); break;
        case 8: phase_e<8>(p, smem_f, gwarp, nwarps); break;
        default: phase_e<16>(p, smem_f, gwarp, nwarps); break;
    }
}

}  // namespace

bool decode_forward_supported(int T, int d, int r, int h, int E, int k, int dtype) {
    (void)k;
    return dtype == BIGMAC_BF16 && T >= 1 && T <= kDecodeMaxTokens && (int64_t)T * d <= 32768 && d % 8 == 0 && r % 8 == 0 &&
           h % 8 == 0 && E <= 1024;
}

cudaError_t launch_decode_forward(const void* x, const bigmac_weights_t* W, void* y, float* logits, float* x_lo, float* a,
                                  float* u, int32_t* topk_idx, float* topk_w, unsigned* barrier, int* status, int T, int d,
                                  int r, int h, int E, int k, int act, int num_sms, cudaStream_t stream) {
    DecodeArgs p;
    p.x = (const __nv_bfloat16*)x; p.w_gate = (const __nv_bfloat16*)W->w_gate; p.w_down = (const __nv_bfloat16*)W->w_down;
    p.w1 = (const __nv_bfloat16*)W->w1; p.w2 = (const __nv_bfloat16*)W->w2; p.w_up = (const __nv_bfloat16*)W->w_up;
    p.b_gate = W->b_gate; p.y = (__nv_bfloat16*)y; p.logits = logits; p.x_lo = x_lo; p.a = a; p.u = u;
    p.topk_idx = topk_idx; p.topk_w = topk_w; p.barrier = barrier; p.status = status;
    p.T = T; p.d = d; p.r = r; p.h = h; p.E = E; p.k = k; p.act = act;
    const size_t smem = sizeof(float) * (size_t)T * (d > r ? d : r);
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        cudaError_t e = cudaFuncSetAttribute(decode_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4);
        if (e != cudaSuccess) return e;
        once.mark(dev);
    }
    cudaError_t err = cudaMemsetAsync(barrier, 0, sizeof(unsigned), stream);
    if (err != cudaSuccess) return err;
    void* args[] = {(void*)&p};
    return cudaLaunchCooperativeKernel((const void*)decode_forward_kernel, dim3(num_sms), dim3(kDecodeThreads), args, smem,
                                       stream);
}

}  // namespace bigmac
