// Row-move kernels of the exchange stage: dispatch (token rows -> expert-grouped rows), combine
// (gate-weighted return to token order) and their backward twins.  All rows move as 16-byte vectors;
// one warp owns one destination row, so every output element is written once and summed in a fixed
// order (deterministic, no atomics).
#include "internal.h"

namespace bigmac {

namespace {

constexpr unsigned kFull = 0xffffffffu;

template <typename T> struct Vec;          // 16 bytes of T
template <> struct Vec<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ uint4 pack(const float* f) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ uint4 pack(const float* f) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t*>(&p);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ int warp_global_id() { return blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); }

// Each warp moves kDispatchRows consecutive grouped rows: all row indices are read first, then every
// 16-byte load of the rows is issued before the first store, so many loads are in flight per lane.
constexpr int kDispatchRows = 4;
__global__ void __launch_bounds__(256) dispatch_kernel(const uint4* __restrict__ src, uint4* __restrict__ grouped,
                                                       const int32_t* __restrict__ slot_of_prow,
                                                       const int32_t* __restrict__ n_tiles, int k, int vecs_per_row,
                                                       int64_t max_prows) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int64_t prow0 = (int64_t)warp_global_id() * kDispatchRows;
    int64_t live = (int64_t)(*n_tiles) * kPad;              // a multiple of kDispatchRows
    if (live > max_prows) live = max_prows;
    if (prow0 >= live) return;
    const int lane = threadIdx.x & 31;
    int s[kDispatchRows];
#pragma unroll
    for (int i = 0; i < kDispatchRows; ++i) s[i] = slot_of_prow[prow0 + i];
    for (int c0 = 0; c0 < vecs_per_row; c0 += 64) {
        uint4 v[kDispatchRows][2];
#pragma unroll
        for (int i = 0; i < kDispatchRows; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int c = c0 + lane + 32 * j;
                v[i][j] = (s[i] >= 0 && c < vecs_per_row) ? src[(int64_t)(s[i] / k) * vecs_per_row + c] : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
        for (int i = 0; i < kDispatchRows; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int c = c0 + lane + 32 * j;
                if (c < vecs_per_row) grouped[(prow0 + i) * vecs_per_row + c] = v[i][j];
            }
    }
}

// MAY_DROP: slots may carry row -1 (dropped under a capacity limit) and are then left out; without it the loop has no
// branch and the k row loads of a token are issued together.
template <typename T, bool MAY_DROP>
__global__ void __launch_bounds__(256) combine_kernel(const uint4* __restrict__ grouped, uint4* __restrict__ dst,
                                                      const float* __restrict__ w,
                                                      const int32_t* __restrict__ prow_of_slot, int n_tokens, int k,
                                                      int vecs_per_row, int dst_vecs_per_row) {
    grid_dependency_wait();
    grid_dependency_launch();
    constexpr int V = Vec<T>::kElems;
    const int t = warp_global_id();
    if (t >= n_tokens) return;
    const int lane = threadIdx.x & 31;
    for (int c = lane; c < vecs_per_row; c += 32) {
        float acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = 0.0f;
        for (int j = 0; j < k; ++j) {                      // slot order: fixed summation order
            const int64_t s = (int64_t)t * k + j;
            int prow = prow_of_slot[s];
            if (MAY_DROP && prow < 0) continue;             // dropped under a capacity limit: absent from the sum
            if (!MAY_DROP) prow = max(prow, 0);             // dropless rows are never negative; keeps the address in range if one were
            const float p = w ? w[s] : 1.0f;
            float f[V];
            Vec<T>::unpack(grouped[(int64_t)prow * vecs_per_row + c], f);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] = fmaf(p, f[i], acc[i]);
        }
        dst[(int64_t)t * dst_vecs_per_row + c] = Vec<T>::pack(acc);
    }
}

template <typename T>
__global__ void __launch_bounds__(256) combine_bwd_kernel(const uint4* __restrict__ dy_lo, const uint4* __restrict__ u,
                                                          uint4* __restrict__ du, float* __restrict__ dp,
                                                          const int32_t* __restrict__ slot_of_prow,
                                                          const float* __restrict__ topk_w,
                                                          const int32_t* __restrict__ n_tiles, int k, int vecs_per_row,
                                                          int64_t max_prows) {
    grid_dependency_wait();
    grid_dependency_launch();
    constexpr int V = Vec<T>::kElems;
    const int64_t prow = warp_global_id();
    int64_t live = (int64_t)(*n_tiles) * kPad;
    if (live > max_prows) live = max_prows;
    if (prow >= live) return;
    const int lane = threadIdx.x & 31;
    const int s = slot_of_prow[prow];
    uint4* out = du + prow * vecs_per_row;
    if (s < 0) {
        for (int c = lane; c < vecs_per_row; c += 32) out[c] = make_uint4(0, 0, 0, 0);
        return;
    }
    const float p = topk_w[s];
    const uint4* g = dy_lo + (int64_t)(s / k) * vecs_per_row;
    const uint4* ur = u + prow * vecs_per_row;
    float dot = 0.0f;
    for (int c = lane; c < vecs_per_row; c += 32) {
        float a[V], b[V], o[V];
        Vec<T>::unpack(g[c], a);
        Vec<T>::unpack(ur[c], b);
#pragma unroll
        for (int i = 0; i < V; ++i) { dot = fmaf(a[i], b[i], dot); o[i] = p * a[i]; }
        out[c] = Vec<T>::pack(o);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(kFull, dot, off);
    if (lane == 0) dp[s] = dot;
}

template <typename T>
__global__ void __launch_bounds__(256) gate_bwd_kernel(float* __restrict__ dp, const float* __restrict__ topk_w,
                                                       const int32_t* __restrict__ topk_idx, T* __restrict__ dlogits,
                                                       int n_tokens, int E, int width, int ld, int k) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int t = warp_global_id();
    if (t >= n_tokens) return;
    const int lane = threadIdx.x & 31;
    const float* p = topk_w + (int64_t)t * k;
    float* g = dp + (int64_t)t * k;
    float part = 0.0f;
    for (int j = lane; j < k; j += 32) part = fmaf(p[j], g[j], part);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(kFull, part, off);
    T* row = dlogits + (int64_t)t * ld;
    for (int e = lane; e < width; e += 32) row[e] = (T)0.0f;
    __syncwarp();
    for (int j = lane; j < k; j += 32) {
        const float dl = p[j] * (g[j] - part);
        const int e = topk_idx[(int64_t)t * k + j];
        if ((unsigned)e < (unsigned)E) row[e] = (T)dl;
        g[j] = dl;                                   // fp32 copy per slot, for the bias gradient
    }
}

// Bias gradient db[e] = sum over slots routed to e of dl[slot], from the fp32 per-slot values, in two
// deterministic stages.  Block b owns a contiguous range of slots, its warps contiguous sub-ranges; a warp walks
// its range 32 slots at a time and lane l adds, in slot order, the values of the experts e with e % 32 == l into
// the warp's row of shared memory.  The block then adds its warps' rows in order.
__global__ void __launch_bounds__(256) colsum_slots_kernel(const float* __restrict__ dl, const int32_t* __restrict__ topk_idx,
                                                           float* __restrict__ partial, int64_t N, int E) {
    grid_dependency_wait();
    grid_dependency_launch();
    extern __shared__ float warp_acc[];              // [8][E]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 8 * E; i += blockDim.x) warp_acc[i] = 0.0f;
    __syncthreads();
    const int64_t per_warp = ((N + (int64_t)gridDim.x * 8 - 1) / ((int64_t)gridDim.x * 8) + 31) / 32 * 32;
    const int64_t s0 = ((int64_t)blockIdx.x * 8 + warp) * per_warp;
    const int64_t s1 = s0 + per_warp < N ? s0 + per_warp : N;
    float* mine = warp_acc + warp * E;
    for (int64_t base = s0; base < s1; base += 32) {
        const int64_t s = base + lane;
        const int e = s < s1 ? topk_idx[s] : -1;
        const float v = s < s1 ? dl[s] : 0.0f;
#pragma unroll 8
        for (int i = 0; i < 32; ++i) {
            const int ei = __shfl_sync(kFull, e, i);
            const float vi = __shfl_sync(kFull, v, i);
            if (ei >= 0 && (ei & 31) == lane) mine[ei] += vi;
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        float total = 0.0f;
        for (int w = 0; w < 8; ++w) total += warp_acc[w * E + e];
        partial[(int64_t)blockIdx.x * E + e] = total;
    }
}

// One warp per column: lane l adds chunks l, l + 32, ... in order, then a fixed shuffle tree adds the lanes.
// `partial2` (nullable): a second array with chunks2 rows, added after the first.
__global__ void __launch_bounds__(256) colsum_final_kernel(const float* __restrict__ partial, const float* __restrict__ partial2,
                                                           float* __restrict__ out, int chunks, int chunks2, int cols,
                                                           int accumulate) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (c >= cols) return;
    float total = 0.0f;
    for (int i = lane; i < chunks; i += 32) total += partial[(int64_t)i * cols + c];
    if (partial2)
        for (int i = lane; i < chunks2; i += 32) total += partial2[(int64_t)i * cols + c];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
    if (lane == 0) out[c] = accumulate ? out[c] + total : total;
}

template <typename T>
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float* __restrict__ ws, int parts, int M, int N,
                                                            T* __restrict__ dst1, int m_split, T* __restrict__ dst2, int m2,
                                                            int accumulate) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;     // N is a multiple of 4
    if (i >= (int64_t)(m_split + m2) * N) return;
    const int m = (int)(i / N);
    float4 acc = *(const float4*)(ws + i);
    for (int s = 1; s < parts; ++s) {
        const float4 v = *(const float4*)(ws + (int64_t)s * M * N + i);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    T* dst = m < m_split ? dst1 + i : dst2 + (i - (int64_t)m_split * N);
    if (!(m < m_split ? dst1 : dst2)) return;
    if (accumulate) { acc.x += (float)dst[0]; acc.y += (float)dst[1]; acc.z += (float)dst[2]; acc.w += (float)dst[3]; }
    dst[0] = (T)acc.x; dst[1] = (T)acc.y; dst[2] = (T)acc.z; dst[3] = (T)acc.w;
}

// [x' | logits] from the fp32 partial results of a descend launch whose contraction was cut into parts (few tokens:
// the launch has too few output tiles to fill the SMs otherwise).  ws is [parts][T][r + E]; the first r columns of a
// row are added in part order and rounded to bf16 (x'), the other E stay fp32 (the gate logits).  r, E multiples of 4.
__global__ void __launch_bounds__(256) descend_reduce_kernel(const float* __restrict__ ws, int parts, int T, int r, int E,
                                                             __nv_bfloat16* __restrict__ x_lo, float* __restrict__ logits) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int n = r + E;
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= (int64_t)T * n) return;
    const int t = (int)(i / n), c = (int)(i - (int64_t)t * n);
    float4 acc = *(const float4*)(ws + i);
    for (int s = 1; s < parts; ++s) {
        const float4 v = *(const float4*)(ws + (int64_t)s * T * n + i);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    if (c < r) {
        __nv_bfloat162* dst = (__nv_bfloat162*)(x_lo + (int64_t)t * r + c);
        dst[0] = __floats2bfloat162_rn(acc.x, acc.y);
        dst[1] = __floats2bfloat162_rn(acc.z, acc.w);
    } else {
        *(float4*)(logits + (int64_t)t * E + (c - r)) = acc;
    }
}

// Per-expert column sums (expert-bias gradients), in two deterministic steps so that one long segment does not
// serialise.  Step 1, block (cg, e, s): slice s of kColsumSlices equal row ranges of expert e's padded segment; 32
// column-threads x 8 row-lanes, a thread adds rows lane, lane + 8, ... of its 16-byte column vector in order, then the
// 8 row-lanes are added in order -> partial[e][s][:].  Step 2 adds the slices in order.
template <typename T>
__global__ void __launch_bounds__(256) grouped_colsum_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ poffsets,
                                                             float* __restrict__ partial, int vecs_per_row) {
    grid_dependency_wait();
    grid_dependency_launch();
    constexpr int V = Vec<T>::kElems;
    __shared__ float part[8][32 * V];
    const int e = blockIdx.y, slice = blockIdx.z, ct = threadIdx.x & 31, rl = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + ct;
    const int64_t r0 = poffsets[e], rows = poffsets[e + 1] - r0;
    const int64_t per = (rows + kColsumSlices - 1) / kColsumSlices;
    const int64_t first = r0 + slice * per, last = min(r0 + rows, first + per);
    float acc[V];
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] = 0.0f;
    if (c < vecs_per_row) {
        int64_t row = first + rl;
        for (; row + 24 < last; row += 32) {           // four rows in flight per thread
            uint4 q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) q[u] = src[(row + 8 * u) * vecs_per_row + c];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float f[V];
                Vec<T>::unpack(q[u], f);
#pragma unroll
                for (int i = 0; i < V; ++i) acc[i] += f[i];
            }
        }
        for (; row < last; row += 8) {
            float f[V];
            Vec<T>::unpack(src[row * vecs_per_row + c], f);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] += f[i];
        }
    }
#pragma unroll
    for (int i = 0; i < V; ++i) part[rl][ct * V + i] = acc[i];
    __syncthreads();
    const int width = vecs_per_row * V;
    for (int j = threadIdx.x; j < 32 * V; j += blockDim.x) {
        const int col = blockIdx.x * 32 * V + j;
        if (col >= width) continue;
        float total = 0.0f;
        for (int q = 0; q < 8; ++q) total += part[q][j];
        partial[((int64_t)e * kColsumSlices + slice) * width + col] = total;
    }
}
__global__ void __launch_bounds__(256) grouped_colsum_final_kernel(const float* __restrict__ partial, float* __restrict__ out,
                                                                   int64_t n, int width, int accumulate) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;      // i = e * width + col
    if (i >= n) return;
    const int64_t e = i / width, col = i - e * width;
    float total = 0.0f;
    for (int s = 0; s < kColsumSlices; ++s) total += partial[(e * kColsumSlices + s) * width + col];
    out[i] = accumulate ? out[i] + total : total;
}

inline int elem_bytes(int dtype) { return dtype == BIGMAC_BF16 ? 2 : 4; }
inline unsigned warp_blocks(int64_t warps) { return (unsigned)((warps + 7) / 8); }

}  // namespace

cudaError_t launch_dispatch(const void* src, void* grouped, const Tables& tb, int k, int width, int dtype,
                            int64_t max_prows, cudaStream_t stream) {
    if (max_prows == 0) return cudaSuccess;
    const int vecs = width * elem_bytes(dtype) / 16;
    return launch_chained(dispatch_kernel, warp_blocks((max_prows + kDispatchRows - 1) / kDispatchRows), 256, 0, stream, (const uint4*)src, (uint4*)grouped, tb.slot_of_prow,
                          tb.n_tiles, k, vecs, max_prows);
}

cudaError_t launch_combine(const void* grouped, void* dst, const float* w, const int32_t* prow_of_slot, int T, int k,
                           int width, int dtype, cudaStream_t stream, int dst_ld, bool may_drop) {
    if (T == 0) return cudaSuccess;
    const int vecs = width * elem_bytes(dtype) / 16;
    const int dvecs = (dst_ld ? dst_ld : width) * elem_bytes(dtype) / 16;
    const uint4* src = (const uint4*)grouped;
    uint4* out = (uint4*)dst;
    if (dtype == BIGMAC_BF16) {
        if (may_drop) return launch_chained(combine_kernel<__nv_bfloat16, true>, warp_blocks(T), 256, 0, stream, src, out, w, prow_of_slot, T, k, vecs, dvecs);
        return launch_chained(combine_kernel<__nv_bfloat16, false>, warp_blocks(T), 256, 0, stream, src, out, w, prow_of_slot, T, k, vecs, dvecs);
    } else {
        if (may_drop) return launch_chained(combine_kernel<float, true>, warp_blocks(T), 256, 0, stream, src, out, w, prow_of_slot, T, k, vecs, dvecs);
        return launch_chained(combine_kernel<float, false>, warp_blocks(T), 256, 0, stream, src, out, w, prow_of_slot, T, k, vecs, dvecs);
    }
    return cudaGetLastError();
}

cudaError_t launch_combine_bwd(const void* dy_lo, const void* u, void* du, float* dp, const Tables& tb, int k,
                               int width, int dtype, int64_t max_prows, cudaStream_t stream) {
    if (max_prows == 0) return cudaSuccess;
    const int vecs = width * elem_bytes(dtype) / 16;
    if (dtype == BIGMAC_BF16)
        (void)launch_chained(combine_bwd_kernel<__nv_bfloat16>, warp_blocks(max_prows), 256, 0, stream, 
            (const uint4*)dy_lo, (const uint4*)u, (uint4*)du, dp, tb.slot_of_prow, tb.topk_w, tb.n_tiles, k, vecs,
            max_prows);
    else
        (void)launch_chained(combine_bwd_kernel<float>, warp_blocks(max_prows), 256, 0, stream, 
            (const uint4*)dy_lo, (const uint4*)u, (uint4*)du, dp, tb.slot_of_prow, tb.topk_w, tb.n_tiles, k, vecs,
            max_prows);
    return cudaGetLastError();
}

cudaError_t launch_gate_bwd(float* dp, const Tables& tb, void* dlogits, int T, int E, int width, int ld, int k,
                            int dtype, cudaStream_t stream) {
    if (T == 0) return cudaSuccess;
    if (dtype == BIGMAC_BF16)
        (void)launch_chained(gate_bwd_kernel<__nv_bfloat16>, warp_blocks(T), 256, 0, stream, dp, tb.topk_w, tb.topk_idx,
                                                                          (__nv_bfloat16*)dlogits, T, E, width, ld, k);
    else
        (void)launch_chained(gate_bwd_kernel<float>, warp_blocks(T), 256, 0, stream, dp, tb.topk_w, tb.topk_idx, (float*)dlogits, T, E, width, ld, k);
    return cudaGetLastError();
}

cudaError_t launch_gate_colsum(const float* dl_slot, const Tables& tb, float* db, float* partial, int64_t N, int E,
                               bool accumulate, cudaStream_t stream, const float* aux_partial) {
    (void)launch_chained(colsum_slots_kernel, kColsumChunks, 256, sizeof(float) * 8 * E, stream, dl_slot, tb.topk_idx, partial, N, E);
    (void)launch_chained(colsum_final_kernel, (unsigned)((E + 7) / 8), 256, 0, stream, partial, aux_partial, db, kColsumChunks, kAuxChunks, E, accumulate);
    return cudaGetLastError();
}

cudaError_t launch_grouped_colsum(const void* src, const int32_t* poffsets, float* out, float* partial, int E, int width,
                                  int dtype, bool accumulate, cudaStream_t stream) {
    if (E == 0 || width == 0) return cudaSuccess;
    const int vecs = width * elem_bytes(dtype) / 16;
    dim3 grid((unsigned)((vecs + 31) / 32), (unsigned)E, (unsigned)kColsumSlices);
    if (dtype == BIGMAC_BF16)
        (void)launch_chained(grouped_colsum_kernel<__nv_bfloat16>, grid, 256, 0, stream, (const uint4*)src, poffsets, partial, vecs);
    else
        (void)launch_chained(grouped_colsum_kernel<float>, grid, 256, 0, stream, (const uint4*)src, poffsets, partial, vecs);
    const int64_t n = (int64_t)E * width;
    (void)launch_chained(grouped_colsum_final_kernel, (unsigned)((n + 255) / 256), 256, 0, stream, partial, out, n, width, accumulate ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_descend_reduce(const float* ws, int parts, int T, int r, int E, void* x_lo, float* logits,
                                  cudaStream_t stream) {
    const int64_t quads = (int64_t)T * (r + E) / 4;
    if (quads == 0) return cudaSuccess;
    return launch_chained(descend_reduce_kernel, (unsigned)((quads + 255) / 256), 256, 0, stream, ws, parts, T, r, E, (__nv_bfloat16*)x_lo, logits);
}

cudaError_t launch_splitk_reduce(const float* ws, int parts, int M, int N, void* dst1, int m_split, void* dst2, int m2,
                                 int dtype, bool accumulate, cudaStream_t stream) {
    const int64_t quads = (int64_t)(m_split + m2) * N / 4;
    if (quads == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((quads + 255) / 256);
    if (dtype == BIGMAC_BF16)
        (void)launch_chained(splitk_reduce_kernel<__nv_bfloat16>, blocks, 256, 0, stream, ws, parts, M, N, (__nv_bfloat16*)dst1, m_split,
                                                                      (__nv_bfloat16*)dst2, m2, accumulate);
    else
        (void)launch_chained(splitk_reduce_kernel<float>, blocks, 256, 0, stream, ws, parts, M, N, (float*)dst1, m_split, (float*)dst2, m2,
                                                               accumulate);
    return cudaGetLastError();
}

}  // namespace bigmac
