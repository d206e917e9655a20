// Load-balancing loss of the paper's pre-training recipe (Table 5: aux_loss with coefficient alpha) and its
// gradient with respect to the gate logits.  The paper prints no formula; the conventional one is used:
//
//     L_aux = alpha * E * sum_e f_e P_e ,   f_e = (slots that chose e) / (T k) ,
//     P_e   = (1/T) sum_t p[t,e] ,          p[t,:] = softmax over ALL E experts of the gate logits (+ gate bias)
//     dL_aux/dl[t,e] = (alpha E / T) p[t,e] (f_e - sum_j f_j p[t,j])            (f is piecewise constant)
//
// Both kernels give block b a contiguous range of tokens and each of its warps a contiguous sub-range; a warp
// handles one token at a time (lanes stride over the experts) and adds into its own row of shared memory, lane l
// owning the experts e with e % 32 == l, so every sum has a fixed order.  E <= 1024.
#include "internal.h"

namespace bigmac {

namespace {

constexpr unsigned kFull = 0xffffffffu;
// Warps per block: 8 where the shared-memory rows of the backward kernel ((2 W + 1) E floats) stay under 48 KB.
inline int aux_warps(int E) { return E <= 512 ? 8 : 4; }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, off));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(kFull, v, off);
    return v;
}

// Row maximum and 1 / sum exp(l - max) of one token's logits.
__device__ __forceinline__ void softmax_stats(const float* __restrict__ l, const float* __restrict__ b, int E, int lane,
                                              float& m, float& inv_sum) {
    float mx = -INFINITY;
    for (int e = lane; e < E; e += 32) mx = fmaxf(mx, l[e] + (b ? b[e] : 0.0f));
    m = warp_max(mx);
    float sum = 0.0f;
    for (int e = lane; e < E; e += 32) sum += expf(l[e] + (b ? b[e] : 0.0f) - m);
    inv_sum = 1.0f / warp_sum(sum);
}

__device__ __forceinline__ void token_range(int T, int warp, int& t0, int& t1) {
    const int warps = blockDim.x >> 5;
    const int per_warp = (T + (int)gridDim.x * warps - 1) / ((int)gridDim.x * warps);
    const int64_t first = ((int64_t)blockIdx.x * warps + warp) * per_warp;
    t0 = (int)(first < T ? first : T);
    t1 = (int)(first + per_warp < T ? first + per_warp : T);
}

// partial[b][e] = sum over the tokens of block b of p[t,e]
__global__ void __launch_bounds__(256) aux_prob_sums_kernel(const float* __restrict__ logits,
                                                                       const float* __restrict__ b_gate, int T, int E,
                                                                       float* __restrict__ partial) {
    grid_dependency_wait();
    grid_dependency_launch();
    extern __shared__ float acc[];                   // [warps][E]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    for (int i = threadIdx.x; i < warps * E; i += blockDim.x) acc[i] = 0.0f;
    __syncthreads();
    float* mine = acc + warp * E;
    int t0, t1;
    token_range(T, warp, t0, t1);
    for (int t = t0; t < t1; ++t) {
        const float* l = logits + (int64_t)t * E;
        float m, inv;
        softmax_stats(l, b_gate, E, lane, m, inv);
        for (int e = lane; e < E; e += 32) mine[e] += expf(l[e] + (b_gate ? b_gate[e] : 0.0f) - m) * inv;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        float total = 0.0f;
        for (int w = 0; w < warps; ++w) total += acc[w * E + e];
        partial[(int64_t)blockIdx.x * E + e] = total;
    }
}

// loss = coef * E * sum_e f_e P_e   (one block).  Thread (g, e) adds the chunks g, g + groups, ... of expert e in order
// (neighbouring threads read neighbouring experts), thread e then adds its groups in order; a fixed tree over the experts.
__global__ void __launch_bounds__(1024) aux_loss_final_kernel(const float* __restrict__ partial,
                                                              const int32_t* __restrict__ counts_chosen, int chunks, int T,
                                                              int E, int k, float coef, float* __restrict__ loss) {
    grid_dependency_wait();
    grid_dependency_launch();
    __shared__ float part[1024];
    __shared__ float term[1024];
    const int groups = 1024 / E, g = threadIdx.x / E, e = threadIdx.x - g * E;      // E <= 1024: at least one group
    if (g < groups) {
        float acc = 0.0f;
        for (int i = g; i < chunks; i += groups) acc += partial[(int64_t)i * E + e];
        part[g * E + e] = acc;
    }
    __syncthreads();
    float v = 0.0f;
    if ((int)threadIdx.x < E) {
        float P = 0.0f;
        for (int q = 0; q < groups; ++q) P += part[q * E + threadIdx.x];
        v = ((float)counts_chosen[threadIdx.x] / ((float)T * (float)k)) * (P / (float)T);
    }
    term[threadIdx.x] = v;
    __syncthreads();
    for (int half = 512; half > 0; half >>= 1) {
        if ((int)threadIdx.x < half) term[threadIdx.x] += term[threadIdx.x + half];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[0] = coef * (float)E * term[0];
}

// Softmax-over-k backward (as in the plain gate backward) plus the gradient of the load-balancing loss.
template <typename T>
__global__ void __launch_bounds__(256) gate_bwd_aux_kernel(float* __restrict__ dp, const float* __restrict__ topk_w,
                                                                      const int32_t* __restrict__ topk_idx,
                                                                      const int32_t* __restrict__ counts_chosen,
                                                                      const float* __restrict__ logits,
                                                                      const float* __restrict__ b_gate, float coef,
                                                                      T* __restrict__ dlogits, float* __restrict__ aux_partial,
                                                                      int n_tokens, int E, int width, int ld, int k) {
    grid_dependency_wait();
    grid_dependency_launch();
    extern __shared__ float smem[];                  // [warps][E] column sums, [warps][E] the row being built, [E] f
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    float* acc = smem;
    float* rows = smem + warps * E;
    float* f = rows + warps * E;
    for (int i = threadIdx.x; i < warps * E; i += blockDim.x) acc[i] = 0.0f;
    const float inv_nk = 1.0f / ((float)n_tokens * (float)k);
    for (int e = threadIdx.x; e < E; e += blockDim.x) f[e] = (float)counts_chosen[e] * inv_nk;
    __syncthreads();
    float* mine = acc + warp * E;
    float* row = rows + warp * E;
    const float scale = coef * (float)E / (float)n_tokens;
    int t0, t1;
    token_range(n_tokens, warp, t0, t1);
    for (int t = t0; t < t1; ++t) {
        const float* l = logits + (int64_t)t * E;
        float m, inv;
        softmax_stats(l, b_gate, E, lane, m, inv);
        float fp = 0.0f;
        for (int e = lane; e < E; e += 32) {
            const float p = expf(l[e] + (b_gate ? b_gate[e] : 0.0f) - m) * inv;
            row[e] = p;
            fp = fmaf(f[e], p, fp);
        }
        fp = warp_sum(fp);
        for (int e = lane; e < E; e += 32) {
            const float g = scale * row[e] * (f[e] - fp);
            row[e] = g;
            mine[e] += g;
        }
        // the top-k part: g = sum_i p_i dp_i, dl_j = p_j (dp_j - g)
        const float* pw = topk_w + (int64_t)t * k;
        float* gp = dp + (int64_t)t * k;
        float part = 0.0f;
        for (int j = lane; j < k; j += 32) part = fmaf(pw[j], gp[j], part);
        part = warp_sum(part);
        __syncwarp();
        for (int j = lane; j < k; j += 32) {
            const float dl = pw[j] * (gp[j] - part);
            const int e = topk_idx[(int64_t)t * k + j];
            if ((unsigned)e < (unsigned)E) row[e] += dl;  // the k experts of a token are distinct
            gp[j] = dl;                               // fp32 copy per slot, for the bias gradient
        }
        __syncwarp();
        T* out = dlogits + (int64_t)t * ld;
        for (int e = lane; e < width; e += 32) out[e] = (T)(e < E ? row[e] : 0.0f);
        __syncwarp();
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        float total = 0.0f;
        for (int w = 0; w < warps; ++w) total += acc[w * E + e];
        aux_partial[(int64_t)blockIdx.x * E + e] = total;
    }
}

}  // namespace

cudaError_t launch_aux_loss(const float* logits, const float* b_gate, const int32_t* counts_chosen, int T, int E, int k,
                            float coef, float* partial, float* loss, cudaStream_t stream) {
    if (T == 0) return cudaMemsetAsync(loss, 0, sizeof(float), stream);
    const int warps = aux_warps(E);
    (void)launch_chained(aux_prob_sums_kernel, kAuxChunks, warps * 32, sizeof(float) * warps * E, stream, logits, b_gate, T, E, partial);
    (void)launch_chained(aux_loss_final_kernel, 1, 1024, 0, stream, partial, counts_chosen, kAuxChunks, T, E, k, coef, loss);
    return cudaGetLastError();
}

cudaError_t launch_gate_bwd_aux(float* dp, const Tables& tb, void* dlogits, const float* logits, const float* b_gate,
                                float coef, float* aux_partial, int T, int E, int width, int ld, int k, int dtype,
                                cudaStream_t stream) {
    if (T == 0) return cudaSuccess;
    const int warps = aux_warps(E);
    const size_t smem = sizeof(float) * (2 * warps + 1) * E;          // at most 36 KB (E <= 1024)
    if (dtype == BIGMAC_BF16)
        (void)launch_chained(gate_bwd_aux_kernel<__nv_bfloat16>, kAuxChunks, warps * 32, smem, stream, 
            dp, tb.topk_w, tb.topk_idx, tb.counts_chosen, logits, b_gate, coef, (__nv_bfloat16*)dlogits, aux_partial, T, E,
            width, ld, k);
    else
        (void)launch_chained(gate_bwd_aux_kernel<float>, kAuxChunks, warps * 32, smem, stream, 
            dp, tb.topk_w, tb.topk_idx, tb.counts_chosen, logits, b_gate, coef, (float*)dlogits, aux_partial, T, E, width, ld, k);
    return cudaGetLastError();
}

}  // namespace bigmac
