// Small-batch (decode-shaped) inference forward of the BigMac layer in ONE cooperative kernel.
//
// For a handful of tokens the layer is a chain of matrix-vector products that is bound by streaming the touched
// weights once (W'_down, W_gate, the selected experts' W1/W2, W'_up) and by launch latency; ten separate launches
// cost far more than the arithmetic.  All SMs walk five phases with three grid-wide barriers (after A, C and D):
//   A  [x' | logits] = x [W'_down ; W_gate]^T           a CTA owns a few weight rows, its sixteen warps a sixteenth of
//                                                        the contraction each, tokens four at a time
//   B  top-k + softmax gate values                       one warp per token, repeated by every CTA into its own
//                                                        shared memory (a few KB of logits from L2: cheaper than a barrier)
//   C  a = sigma(W1_e x')  for every routed slot          sixteen weight rows per warp task
//   D  u = W2_e a                                         four weight rows per warp task
//   E  y' = sum_j p_j u_j ;  y = W'_up y'                 two weight rows per warp task
// Weights are read as 16-byte vectors, up to sixteen of them in flight per lane before the first is used (the
// kernel is bound by latency chains and by instruction fetch, not by arithmetic); products accumulate in fp32,
// intermediates stay fp32 in scratch.
// The grid barrier is a bounded spin on a global counter (cooperative launch guarantees co-residency); if the
// bound is ever hit the kernel records BIGMAC_ERR_TIMEOUT in the status word and runs on, so it always ends.
#include "internal.h"
#include "act.cuh"

namespace bigmac {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kDecodeThreads = 512;
constexpr int kDecodeMaxExperts = 256;      // top-k keeps a token's logits in registers: 8 per lane
constexpr int kDecodeMaxSlots = 2048;        // T k: every CTA keeps all slots' expert ids and gate values
constexpr int kDecodeMaxTokens = 16;

struct DecodeArgs {
    const __nv_bfloat16 *x, *w_gate, *w_down, *w1, *w2, *w_up;
    const float* b_gate;
    __nv_bfloat16* y;
    float *logits, *x_lo, *a, *u;      // scratch: [T,E], [T,r], [T*k,h], [T*k,r]
    int32_t* topk_idx;
    float* topk_w;
    unsigned* barrier;                 // zero before the launch; the kernel leaves it zero
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

// All CTAs of the (cooperative) grid meet here; `phase` counts the barriers passed so far.  One thread per CTA arrives
// with a release at GPU scope (the block barrier before it makes the CTA's writes part of what is released) and
// spins with acquire loads; the block barrier after it hands what was acquired to the other threads.
__device__ __forceinline__ void grid_barrier(unsigned* counter, unsigned phase, int* status) {
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
        const unsigned target = (phase + 1) * gridDim.x;
        unsigned seen = 0;
        for (uint32_t i = 0; i < (1u << 24); ++i) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
        }
        if (seen < target) atomicExch(status, 1);
    }
    __syncthreads();
}

// Partial dot products of ROWS consecutive weight rows (bf16, row-major, `ld` apart) over their 16-byte pieces
// [piece0, piece0 + npieces) with the fp32 vectors vp[0 .. nv); lanes stride over the pieces, U pieces per row and
// round: the ROWS * U loads of a round are issued before any of them is used.  With SPLIT the vectors are in the
// two-plane layout of split_index (elements 8c .. 8c+3 of a vector at float4 number c, elements 8c+4 .. 8c+7 at
// float4 number `plane` + c): neighbouring lanes then read neighbouring 16 bytes of shared memory, where the natural
// layout costs a two-way bank conflict on every load.  out[row * NV + t] is this lane's share; the caller sums
// over the lanes (warp_reduce_scatter).
template <int ROWS, int NV, int U, bool SPLIT>
__device__ __forceinline__ void rows_dot(const __nv_bfloat16* w, int64_t ld, int piece0, int npieces, const float* const (&vp)[NV],
                                         int plane, int nv, float (&out)[ROWS * NV]) {
    const int lane = threadIdx.x & 31, end = piece0 + npieces;
#pragma unroll
    for (int i = 0; i < ROWS * NV; ++i) out[i] = 0.0f;
    for (int c0 = piece0 + lane; c0 < end; c0 += 32 * U) {
        uint4 wv[U][ROWS];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + 32 * u;
#pragma unroll
            for (int i = 0; i < ROWS; ++i)
                wv[u][i] = c < end ? __ldg(reinterpret_cast<const uint4*>(w + i * ld) + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + 32 * u;
            if (c < end) {
#pragma unroll
                for (int t = 0; t < NV; ++t) {
                    if (t < nv) {
                        const float4* vt = reinterpret_cast<const float4*>(vp[t]);
                        const float4 v0 = SPLIT ? vt[c] : vt[2 * c];
                        const float4 v1 = SPLIT ? vt[plane + c] : vt[2 * c + 1];
#pragma unroll
                        for (int i = 0; i < ROWS; ++i) {
                            float wf[8];
                            unpack8(wv[u][i], wf);
                            float acc = out[i * NV + t];
                            acc = fmaf(wf[0], v0.x, acc); acc = fmaf(wf[1], v0.y, acc); acc = fmaf(wf[2], v0.z, acc); acc = fmaf(wf[3], v0.w, acc);
                            acc = fmaf(wf[4], v1.x, acc); acc = fmaf(wf[5], v1.y, acc); acc = fmaf(wf[6], v1.z, acc); acc = fmaf(wf[7], v1.w, acc);
                            out[i * NV + t] = acc;
                        }
                    }
                }
            }
        }
    }
}

// Where element e of a staged vector of n elements sits in the two-plane layout (see rows_dot).
__device__ __forceinline__ int split_index(int e, int n) { return ((e >> 2) & 1) * (n >> 1) + ((e >> 3) << 2) + (e & 3); }

// Sums each of the N values (a power of two, at most 32) over the warp's lanes with N - 1 + log2(32 / N) shuffles
// instead of 5 N: every halving step a lane hands half of its values to its partner and keeps the sums of the
// other half.  Returns the total of value number lane / (32 / N); v is used up.  The order of the additions is fixed.
template <int N>
__device__ __forceinline__ float warp_reduce_scatter(float* v) {
    const int lane = threadIdx.x & 31;
    int off = 16;
#pragma unroll
    for (int cnt = N; cnt > 1; cnt >>= 1, off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < cnt / 2; ++i) {
            const float send = upper ? v[i] : v[i + cnt / 2];
            const float keep = upper ? v[i + cnt / 2] : v[i];
            v[i] = keep + __shfl_xor_sync(kFull, send, off);
        }
    }
    float total = v[0];
#pragma unroll
    for (int o = 16 / N; o > 0; o >>= 1) total += __shfl_xor_sync(kFull, total, o);
    return total;
}

// The kernel runs every piece of its code once or a few times per launch, so code size is time (instruction fetch
// was the largest stall with one fully unrolled copy per token count): tokens are walked four at a time by a loop
// around one small copy of each phase, and the weights of a task are read again for each group of four (from L1).
constexpr int kTokenGroup = 4;

// A: rows of [W'_down ; W_gate] against the tokens staged in `xs` as fp32 [T,d] (two-plane layout).  CTA b owns rows
// b, b + grid, ...; a warp takes one sixteenth of the contraction of four of them at a time (x leaves shared memory
// once per four rows), the sixteen pieces meet in shared memory and are added in order.
__device__ __forceinline__ void phase_a(const DecodeArgs& p, const float* xs, float* part_sums) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kDecodeThreads / 32, ROWS = 4;
    const int R = p.r + p.E, G = gridDim.x, per_cta = (R + G - 1) / G;
    const int pieces = p.d / 8, per_part = (pieces + kWarps - 1) / kWarps;
    const int piece0 = min(pieces, warp * per_part), end = min(pieces, piece0 + per_part);
    for (int first = 0; first < per_cta; first += ROWS) {
        // rows j0, j0 + G, ...: W'_down and W_gate are two arrays, so the four rows are addressed one by one; a row
        // past the end is replaced by a valid one and its result dropped
        const int j0 = blockIdx.x + G * first;
        const uint4* rows[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            int j = j0 + G * i;
            if (first + i >= per_cta || j >= R) j = 0;
            rows[i] = reinterpret_cast<const uint4*>(j < p.r ? p.w_down + (int64_t)j * p.d : p.w_gate + (int64_t)(j - p.r) * p.d);
        }
        bool first_round = true;                             // at least one round, so that every slot below is written
        for (int cb = piece0; cb < end || first_round; cb += 32, first_round = false) {
            const int c = cb + lane;
            uint4 wv[ROWS];
#pragma unroll
            for (int i = 0; i < ROWS; ++i) wv[i] = c < end ? __ldg(rows[i] + c) : make_uint4(0u, 0u, 0u, 0u);
            for (int t0 = 0; t0 < p.T; t0 += kTokenGroup) {
                float acc[ROWS * kTokenGroup];
#pragma unroll
                for (int i = 0; i < ROWS * kTokenGroup; ++i) acc[i] = 0.0f;
                if (c < end) {
#pragma unroll
                    for (int t = 0; t < kTokenGroup; ++t) {
                        if (t0 + t < p.T) {
                            const float4* vt = reinterpret_cast<const float4*>(xs + (int64_t)(t0 + t) * p.d);
                            const float4 v0 = vt[c], v1 = vt[pieces + c];
#pragma unroll
                            for (int i = 0; i < ROWS; ++i) {
                                float wf[8];
                                unpack8(wv[i], wf);
                                float a = 0.0f;
                                a = fmaf(wf[0], v0.x, a); a = fmaf(wf[1], v0.y, a); a = fmaf(wf[2], v0.z, a); a = fmaf(wf[3], v0.w, a);
                                a = fmaf(wf[4], v1.x, a); a = fmaf(wf[5], v1.y, a); a = fmaf(wf[6], v1.z, a); a = fmaf(wf[7], v1.w, a);
                                acc[i * kTokenGroup + t] = a;
                            }
                        }
                    }
                }
                const float mine = warp_reduce_scatter<ROWS * kTokenGroup>(acc);   // (row, token) = lane / 2 / 4, % 4
                if (!(lane & 1)) {
                    float* slot = part_sums + ((lane >> 3) * kWarps + warp) * 16 + t0 + ((lane >> 1) & 3);
                    *slot = first_round ? mine : *slot + mine;
                }
            }
        }
        __syncthreads();
        if (threadIdx.x < ROWS * 16) {
            const int i = threadIdx.x / 16, t = threadIdx.x % 16, j = j0 + G * i;
            if (first + i < per_cta && j < R && t < p.T) {
                float sum = 0.0f;
                for (int q = 0; q < kWarps; ++q) sum += part_sums[(i * kWarps + q) * 16 + t];
                if (j < p.r) p.x_lo[t * p.r + j] = sum;
                else p.logits[t * p.E + (j - p.r)] = sum + (p.b_gate ? p.b_gate[j - p.r] : 0.0f);
            }
        }
        __syncthreads();
    }
}

// E: two rows of W'_up per warp task against y' [T,r] staged in `ys` (two-plane layout).
__device__ __forceinline__ void phase_e(const DecodeArgs& p, const float* ys, int gwarp, int nwarps) {
    constexpr int ROWS = 2;
    const int lane = threadIdx.x & 31;
    for (int task = gwarp; task < p.d / ROWS; task += nwarps) {
        const int c0 = task * ROWS;
        for (int t0 = 0; t0 < p.T; t0 += kTokenGroup) {
            float acc[ROWS * kTokenGroup];
            const float* vp[kTokenGroup];
#pragma unroll
            for (int t = 0; t < kTokenGroup; ++t) vp[t] = ys + (int64_t)min(t0 + t, p.T - 1) * p.r;
            rows_dot<ROWS, kTokenGroup, 2, true>(p.w_up + (int64_t)c0 * p.r, p.r, 0, p.r / 8, vp, p.r / 8,
                                                min(kTokenGroup, p.T - t0), acc);
            const float v = warp_reduce_scatter<ROWS * kTokenGroup>(acc);     // (row, token) = lane / 4 / 4, % 4
            const int t = t0 + ((lane >> 2) & 3);
            if (!(lane & 3) && t < p.T) p.y[(int64_t)t * p.d + c0 + (lane >> 4)] = __float2bfloat16(v);
        }
    }
}

__global__ void __launch_bounds__(kDecodeThreads, 1) decode_forward_kernel(const DecodeArgs p) {
    extern __shared__ float smem_f[];                       // phase A: x as fp32 [T,d]; C: x' [T,r]; E: y' [T,r]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warps_per_cta = kDecodeThreads / 32;
    const int gwarp = warp * gridDim.x + blockIdx.x, nwarps = gridDim.x * warps_per_cta;   // neighbouring tasks on different SMs
    const int T = p.T, N = p.T * p.k;

    int* s_idx = reinterpret_cast<int*>(smem_f + T * max(p.d, p.r));     // [T k] expert of every slot
    float* s_w = reinterpret_cast<float*>(s_idx + N);                      // [T k] its gate value
    float* part_sums = s_w + N;                                            // [4 rows][16 warps][16 tokens] phase A's pieces

    // ---- A: descend + gate logits (the gate reads x, not x')
    // every CTA stages the same bytes: each starts somewhere else in them, or all SMs ask the same L2 lines at once
    for (int i0 = threadIdx.x; i0 < T * p.d / 8; i0 += kDecodeThreads) {  // d is a multiple of 8, x 16-byte aligned
        const int i = (i0 + blockIdx.x * 224) % (T * p.d / 8);
        float f[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(p.x) + i), f);
        const int t = i / (p.d / 8), c = i % (p.d / 8);
        float4* vt = reinterpret_cast<float4*>(smem_f + (int64_t)t * p.d);
        vt[c] = make_float4(f[0], f[1], f[2], f[3]);
        vt[p.d / 8 + c] = make_float4(f[4], f[5], f[6], f[7]);
    }
    __syncthreads();
    phase_a(p, smem_f, part_sums);
    grid_barrier(p.barrier, 0, p.status);

    // ---- B: top-k by (logit descending, expert id ascending), softmax over the k kept logits.  Every CTA does all
    // tokens for itself (warp t: token t); CTA 0 also writes the tables the caller may ask for.
    if (warp < T) {
        const int t = warp;
        const float* l = p.logits + (int64_t)t * p.E;
        float mine[kDecodeMaxExperts / 32];                  // logits of experts lane, lane + 32, ...
#pragma unroll
        for (int i = 0; i < kDecodeMaxExperts / 32; ++i) {
            const int e = lane + 32 * i;
            const float v = e < p.E ? __ldcg(l + e) : 0.0f;
            mine[i] = v == v ? v : -INFINITY;                // NaN is ordered as -inf
        }
        uint32_t taken = 0;                                  // bit i: expert lane + 32 i already chosen
        float top = 0.0f, part = 0.0f;
        for (int j0 = 0; j0 < p.k; j0 += 32) {               // winner j stays with lane j - j0 until the stores
            float my_ex = 0.0f;
            int my_e = 0;
            for (int j = j0; j < min(p.k, j0 + 32); ++j) {
                float best = -INFINITY;
                int best_e = 0x7fffffff;                     // "no candidate yet"; k <= E, so every round ends with a real id
#pragma unroll
                for (int i = 0; i < kDecodeMaxExperts / 32; ++i) {
                    const int e = lane + 32 * i;
                    if (e < p.E && !((taken >> i) & 1u) && (best_e == 0x7fffffff || mine[i] > best)) { best = mine[i]; best_e = e; }
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
                if (lane == j - j0) { my_ex = ex; my_e = best_e; }
            }
            if (j0 + lane < p.k) { s_idx[t * p.k + j0 + lane] = my_e; s_w[t * p.k + j0 + lane] = my_ex; }
        }
        __syncwarp();
        for (int j = lane; j < p.k; j += 32) {
            const float w = s_w[t * p.k + j] / part;
            s_w[t * p.k + j] = w;
            if (blockIdx.x == 0) { p.topk_idx[t * p.k + j] = s_idx[t * p.k + j]; p.topk_w[t * p.k + j] = w; }
        }
    }

    // ---- C: a = sigma(W1_e x') per routed slot.  (Grouping the slots by expert, so that a weight byte is read once
    // however many tokens chose the expert, was measured slower at every T <= 16: the repeats are L2 hits, and the
    // lists, the smaller tasks and the wider reductions cost more than they save.)
    for (int i = threadIdx.x; i < T * p.r / 4; i += kDecodeThreads) {
        const int t = i / (p.r / 4), c = 4 * (i % (p.r / 4));
        *reinterpret_cast<float4*>(smem_f + t * p.r + split_index(c, p.r)) = __ldcg(reinterpret_cast<const float4*>(p.x_lo) + i);
    }
    __syncthreads();
    {
        constexpr int ROWS = 16;
        const int groups = p.h / ROWS;                       // h is a multiple of 16
        for (int task = gwarp; task < N * groups; task += nwarps) {
            const int s = task / groups, q0 = (task % groups) * ROWS;
            const int e = s_idx[s];
            const float* vp[1] = {smem_f + (s / p.k) * p.r};
            float acc[ROWS];
            rows_dot<ROWS, 1, 1, true>(p.w1 + ((int64_t)e * p.h + q0) * p.r, p.r, 0, p.r / 8, vp, p.r / 8, 1, acc);
            const float z = warp_reduce_scatter<ROWS>(acc);            // row lane / 2
            if (!(lane & 1)) p.a[(int64_t)s * p.h + q0 + lane / 2] = act_apply(p.act, z);
        }
    }
    grid_barrier(p.barrier, 1, p.status);

    // ---- D: u = W2_e a per routed slot
    {
        const int groups = p.r / 4;
        for (int task = gwarp; task < N * groups; task += nwarps) {
            const int s = task / groups, c0 = (task % groups) * 4;
            const int e = s_idx[s];
            const float* vp[1] = {p.a + (int64_t)s * p.h};
            float acc[4];
            rows_dot<4, 1, 4, false>(p.w2 + ((int64_t)e * p.r + c0) * p.h, p.h, 0, p.h / 8, vp, 0, 1, acc);
            const float v = warp_reduce_scatter<4>(acc);               // row lane / 8
            if (!(lane & 7)) p.u[(int64_t)s * p.r + c0 + lane / 8] = v;
        }
    }
    grid_barrier(p.barrier, 2, p.status);

    // ---- E: combine in slot order, then ascend
    for (int i0 = threadIdx.x; i0 < T * p.r / 4; i0 += kDecodeThreads) {   // four columns per thread, 16-byte loads
        const int i = (i0 + blockIdx.x * 224) % (T * p.r / 4);              // as in phase A: CTAs start at different places
        const int t = i / (p.r / 4), c = 4 * (i % (p.r / 4));
        float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        for (int j0 = 0; j0 < p.k; j0 += 8) {                // eight loads in flight, added in slot order
            float4 uj[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                uj[q] = j0 + q < p.k ? __ldcg(reinterpret_cast<const float4*>(p.u + (int64_t)(t * p.k + j0 + q) * p.r + c))
                                     : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (j0 + q < p.k) {
                    const float w = s_w[t * p.k + j0 + q];
                    acc.x = fmaf(w, uj[q].x, acc.x); acc.y = fmaf(w, uj[q].y, acc.y);
                    acc.z = fmaf(w, uj[q].z, acc.z); acc.w = fmaf(w, uj[q].w, acc.w);
                }
            }
        }
        *reinterpret_cast<float4*>(smem_f + t * p.r + split_index(c, p.r)) = acc;
    }
    __syncthreads();
    phase_e(p, smem_f, gwarp, nwarps);
    // a fourth round of arrivals: whoever comes last knows that nobody reads the word any more and zeroes it for the
    // next launch (also after a wait that gave up: every CTA arrives four times whatever happens)
    __syncthreads();
    if (threadIdx.x == 0 && atomicAdd(p.barrier, 1u) == 4u * gridDim.x - 1u) atomicExch(p.barrier, 0u);
}

}  // namespace

bool decode_forward_supported(int T, int d, int r, int h, int E, int k, int dtype) {
    return dtype == BIGMAC_BF16 && T >= 1 && T <= kDecodeMaxTokens && (int64_t)T * d <= 32768 && d % 8 == 0 && r % 8 == 0 &&
           h % 16 == 0 && E <= kDecodeMaxExperts && T * k <= kDecodeMaxSlots;
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
    const size_t smem = sizeof(float) * (size_t)T * (d > r ? d : r) + (size_t)T * k * (sizeof(int) + sizeof(float)) +
                        sizeof(float) * 4 * (kDecodeThreads / 32) * 16;
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        cudaError_t e = cudaFuncSetAttribute(decode_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4 + kDecodeMaxSlots * 8 + 4 * (kDecodeThreads / 32) * 16 * 4);
        if (e != cudaSuccess) return e;
        once.mark(dev);
    }
    void* args[] = {(void*)&p};
    return cudaLaunchCooperativeKernel((const void*)decode_forward_kernel, dim3(num_sms), dim3(kDecodeThreads), args, smem,
                                       stream);
}

}  // namespace bigmac
