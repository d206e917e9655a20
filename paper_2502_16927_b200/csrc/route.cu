// Routing kernels: per-token top-k with softmax gate values, and the deterministic stable counting
// sort of routed slots by expert that lays out the dropless dispatch (the on-device stand-in for the
// send layout of the first All-to-All).
#include "internal.h"

namespace bigmac {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kNoExpert = 0x7fffffff;          // "no candidate yet" in the arg-max rounds; never written out

// One warp per token.  Lane l holds experts l, l+32, ...  k rounds of warp arg-max under the order
// (logit descending, expert id ascending); gate values are the softmax over the k winners.
// KREG: k <= 32, the j-th winner stays in a register of lane j until one coalesced store at the end; otherwise
// the winners pass through the output arrays.
// Non-finite logits: NaN is ordered as -inf, and a round that finds only -inf among the experts not yet chosen takes
// the lowest such id, so every id written lies in [0, E) whatever the logits hold (k <= E).  A token whose kept
// logits are all -inf gets the gate value 1/k on each.
template <int VPL, bool KREG>
__global__ void __launch_bounds__(256) topk_kernel(const float* __restrict__ logits, const float* __restrict__ b_gate,
                                                   int T, int E, int k, int32_t* __restrict__ topk_idx,
                                                   float* __restrict__ topk_w) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    const float* row = logits + (size_t)t * E;
    float v[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        const int e = lane + 32 * i;
        const float x = e < E ? row[e] + (b_gate ? b_gate[e] : 0.0f) : -INFINITY;
        v[i] = x == x ? x : -INFINITY;             // NaN is ordered as -inf
    }
    int32_t* out_idx = topk_idx + (size_t)t * k;
    float* out_w = topk_w + (size_t)t * k;
    float my_v = -INFINITY;
    int my_e = 0;
    uint32_t taken = 0;                            // bit i: expert lane + 32 i already chosen
    for (int j = 0; j < k; ++j) {
        float best = -INFINITY;
        int best_e = kNoExpert;
#pragma unroll
        for (int i = 0; i < VPL; ++i) {            // ascending expert id within the lane: strict > keeps the lowest id
            const int e = lane + 32 * i;
            if (e < E && !((taken >> i) & 1u) && (best_e == kNoExpert || v[i] > best)) { best = v[i]; best_e = e; }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(kFull, best, off);
            const int oe = __shfl_xor_sync(kFull, best_e, off);
            if (ov > best || (ov == best && oe < best_e)) { best = ov; best_e = oe; }
        }
        if (best_e != kNoExpert && (best_e & 31) == lane) taken |= 1u << (best_e >> 5);
        if (KREG) {
            if (lane == j) { my_v = best; my_e = best_e; }
        } else if (lane == 0) {
            out_idx[j] = best_e;
            out_w[j] = best;                       // raw logit for now
        }
    }
    if (KREG) {
        const float top = __shfl_sync(kFull, my_v, 0);
        const float ex = lane < k ? (top == -INFINITY ? 1.0f : expf(my_v - top)) : 0.0f;
        float part = ex;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(kFull, part, off);
        if (lane < k) {
            out_idx[lane] = my_e;
            out_w[lane] = ex / part;
        }
        return;
    }
    __syncwarp();
    const float top = out_w[0];
    const bool none = top == -INFINITY;
    float part = 0.0f;
    for (int j = lane; j < k; j += 32) part += none ? 1.0f : expf(out_w[j] - top);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(kFull, part, off);
    for (int j = lane; j < k; j += 32) out_w[j] = (none ? 1.0f : expf(out_w[j] - top)) / part;
}

// Four tokens per warp, eight lanes per token, for k <= 8 and E a multiple of 32 up to 256: lane l of a group
// holds the experts 4 (l + 8 i) + c (one float4 per i), the arg-max tree has three levels, and the j-th winner
// stays in lane j of the group until one store.  Same order (logit descending, expert id ascending).
template <int Q>   // float4 loads per lane: E = 32 Q
__global__ void __launch_bounds__(256) topk8_kernel(const float* __restrict__ logits, const float* __restrict__ b_gate,
                                                    int T, int k, int32_t* __restrict__ topk_idx,
                                                    float* __restrict__ topk_w) {
    grid_dependency_wait();
    grid_dependency_launch();
    constexpr int E = 32 * Q;
    const int lane = threadIdx.x & 31, sub = lane & 7;
    const int t = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 4 + (lane >> 3);
    const bool live = t < T;
    const float4* row = reinterpret_cast<const float4*>(logits + (size_t)(live ? t : 0) * E);
    float v[4 * Q];
#pragma unroll
    for (int i = 0; i < Q; ++i) {
        float4 x = row[sub + 8 * i];
        if (b_gate) {
            const float4 b = reinterpret_cast<const float4*>(b_gate)[sub + 8 * i];
            x.x += b.x; x.y += b.y; x.z += b.z; x.w += b.w;
        }
        v[4 * i] = x.x; v[4 * i + 1] = x.y; v[4 * i + 2] = x.z; v[4 * i + 3] = x.w;
    }
#pragma unroll
    for (int i = 0; i < 4 * Q; ++i) v[i] = v[i] == v[i] ? v[i] : -INFINITY;     // NaN is ordered as -inf
    float my_v = -INFINITY;
    int my_e = 0;
    uint32_t taken = 0;                            // bit i: this lane's i-th expert already chosen
    for (int j = 0; j < k; ++j) {
        float best = -INFINITY;
        int best_e = kNoExpert;
#pragma unroll
        for (int i = 0; i < 4 * Q; ++i) {          // ascending expert id within the lane: strict > keeps the lowest id
            const int e = 4 * (sub + 8 * (i >> 2)) + (i & 3);
            if (!((taken >> i) & 1u) && (best_e == kNoExpert || v[i] > best)) { best = v[i]; best_e = e; }
        }
#pragma unroll
        for (int off = 4; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(kFull, best, off);
            const int oe = __shfl_xor_sync(kFull, best_e, off);
            if (ov > best || (ov == best && oe < best_e)) { best = ov; best_e = oe; }
        }
#pragma unroll
        for (int i = 0; i < 4 * Q; ++i)
            if (4 * (sub + 8 * (i >> 2)) + (i & 3) == best_e) taken |= 1u << i;
        if (sub == j) { my_v = best; my_e = best_e; }
    }
    const float top = __shfl_sync(kFull, my_v, lane & 24);
    const float ex = sub < k ? (top == -INFINITY ? 1.0f : expf(my_v - top)) : 0.0f;
    float part = ex;
#pragma unroll
    for (int off = 4; off > 0; off >>= 1) part += __shfl_xor_sync(kFull, part, off);
    if (live && sub < k) {
        topk_idx[(size_t)t * k + sub] = my_e;
        topk_w[(size_t)t * k + sub] = ex / part;
    }
}

// Pass 1 of the counting sort.  Block b owns slots [b*kSortChunk, (b+1)*kSortChunk); it writes, per
// slot, the number of earlier slots of the same block routed to the same expert, and per expert the
// block's count.  Warps own consecutive sub-chunks, so the order is the slot order.
__global__ void __launch_bounds__(256) sort_local_kernel(const int32_t* __restrict__ topk_idx, int64_t N, int E,
                                                         int32_t* __restrict__ local_rank,
                                                         int32_t* __restrict__ block_counts) {
    grid_dependency_wait();
    grid_dependency_launch();
    extern __shared__ int32_t warp_run[];            // [8][E]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 8 * E; i += blockDim.x) warp_run[i] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kSortChunk + warp * (kSortChunk / 8);
    int32_t my_rank[kSortChunk / 256];
#pragma unroll
    for (int it = 0; it < kSortChunk / 256; ++it) {
        const int64_t s = base + it * 32 + lane;
        int e = s < N ? topk_idx[s] : -1;
        if ((unsigned)e >= (unsigned)E) e = -1;      // an id outside [0, E) (never written by the top-k kernels) counts nowhere
        const unsigned peers = __match_any_sync(kFull, e);
        const int leader = __ffs(peers) - 1;
        int old = 0;
        if (lane == leader && e >= 0) {
            old = warp_run[warp * E + e];
            warp_run[warp * E + e] = old + __popc(peers);
        }
        old = __shfl_sync(kFull, old, leader);
        my_rank[it] = old + __popc(peers & ((1u << lane) - 1u));
        __syncwarp();
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {   // exclusive scan over the 8 warps
        int run = 0;
        for (int w = 0; w < 8; ++w) {
            const int c = warp_run[w * E + e];
            warp_run[w * E + e] = run;
            run += c;
        }
        block_counts[(size_t)blockIdx.x * E + e] = run;
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < kSortChunk / 256; ++it) {
        const int64_t s = base + it * 32 + lane;
        if (s >= N) continue;
        const int e = topk_idx[s];
        local_rank[s] = (unsigned)e < (unsigned)E ? warp_run[warp * E + e] + my_rank[it] : 0;
    }
}

// Pass 2 (one block): per expert an exclusive scan of the block counts, then offsets, padded offsets
// and the tile -> expert map.
__global__ void __launch_bounds__(1024) sort_scan_kernel(int32_t* __restrict__ block_counts, int n_blocks, int E,
                                                         int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                                         int32_t* __restrict__ poffsets,
                                                         int32_t* __restrict__ tile_expert,
                                                         int32_t* __restrict__ n_tiles, int cap,
                                                         int32_t* __restrict__ counts_chosen) {
    grid_dependency_wait();
    grid_dependency_launch();
    __shared__ int32_t s_cnt[kMaxExperts];
    __shared__ int32_t s_poff[kMaxExperts + 1];
    __shared__ int32_t s_part[1024];
    // thread (part, e) owns a contiguous range of blocks of expert e: range sums, then the exclusive scan inside
    // the range starting from the sum of the ranges before it (two dependent passes instead of one long one)
    const int parts = E >= (int)blockDim.x ? 1 : min(16, min((int)blockDim.x / E, max(n_blocks, 1)));
    const int per = (n_blocks + parts - 1) / parts;
    for (int e0 = 0; e0 < E; e0 += blockDim.x / parts) {
        const int e = e0 + threadIdx.x % (blockDim.x / parts), part = threadIdx.x / (blockDim.x / parts);
        const bool mine = e < E && part < parts;
        const int b0 = min(n_blocks, part * per), b1 = min(n_blocks, b0 + per);
        int sum = 0;
        if (mine) {
            int b = b0;
            for (; b + 8 <= b1; b += 8) {
                int c[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) c[i] = block_counts[(size_t)(b + i) * E + e];
#pragma unroll
                for (int i = 0; i < 8; ++i) sum += c[i];
            }
            for (; b < b1; ++b) sum += block_counts[(size_t)b * E + e];
        }
        __syncthreads();                            // s_part of the previous round has been read
        if (part < parts) s_part[part * (blockDim.x / parts) + threadIdx.x % (blockDim.x / parts)] = sum;
        __syncthreads();
        if (mine) {
            int run = 0, total = 0;
            for (int q = 0; q < parts; ++q) {
                const int v = s_part[q * (blockDim.x / parts) + threadIdx.x % (blockDim.x / parts)];
                if (q < part) run += v;
                total += v;
            }
            if (part == 0) {                        // an expert keeps at most `cap` of the slots that chose it
                const int kept = min(total, cap);
                s_cnt[e] = kept;
                counts[e] = kept;
                if (counts_chosen) counts_chosen[e] = total;
            }
            int b = b0;
            for (; b + 8 <= b1; b += 8) {
                int c[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) c[i] = block_counts[(size_t)(b + i) * E + e];
#pragma unroll
                for (int i = 0; i < 8; ++i) { block_counts[(size_t)(b + i) * E + e] = run; run += c[i]; }
            }
            for (; b < b1; ++b) {
                const int c = block_counts[(size_t)b * E + e];
                block_counts[(size_t)b * E + e] = run;
                run += c;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int off = 0, poff = 0;
        for (int e = 0; e < E; ++e) {
            offsets[e] = off;
            s_poff[e] = poff;
            off += s_cnt[e];
            poff += (s_cnt[e] + kPad - 1) / kPad * kPad;
        }
        offsets[E] = off;
        s_poff[E] = poff;
        *n_tiles = poff / kPad;
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E; e += blockDim.x) poffsets[e] = s_poff[e];
    for (int e = threadIdx.x; e < E; e += blockDim.x)
        for (int tile = s_poff[e] / kPad; tile < s_poff[e + 1] / kPad; ++tile) tile_expert[tile] = e;
}

// Pass 3: final positions.  A slot whose rank among the slots of its expert is `cap` or more is dropped (-1).
__global__ void __launch_bounds__(256) sort_place_kernel(const int32_t* __restrict__ topk_idx, int64_t N, int E,
                                                         const int32_t* __restrict__ block_base,
                                                         const int32_t* __restrict__ offsets,
                                                         const int32_t* __restrict__ poffsets,
                                                         int32_t* __restrict__ prow_of_slot /* in: local rank */,
                                                         int32_t* __restrict__ row_of_slot,
                                                         int32_t* __restrict__ slot_of_row,
                                                         int32_t* __restrict__ slot_of_prow, int cap,
                                                         int* __restrict__ status) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= N) return;
    const int e = topk_idx[s];
    if ((unsigned)e >= (unsigned)E) {               // second line of defence: the slot goes nowhere, the call reports it
        row_of_slot[s] = -1;
        prow_of_slot[s] = -1;
        if (status) atomicExch(status, 2);
        return;
    }
    const int within = block_base[(size_t)(s / kSortChunk) * E + e] + prow_of_slot[s];
    if (within >= cap) {
        row_of_slot[s] = -1;
        prow_of_slot[s] = -1;
        return;
    }
    const int row = offsets[e] + within;
    const int prow = poffsets[e] + within;
    row_of_slot[s] = row;
    slot_of_row[row] = (int32_t)s;
    prow_of_slot[s] = prow;
    slot_of_prow[prow] = (int32_t)s;
}

// All three passes (and the fill of slot_of_prow) in ONE block, for the few thousand slots of decode-shaped batches,
// where four launches cost more than the work.  1024 threads; chunk c holds slots [1024 c, 1024 (c + 1)), warp w of
// it the 32 slots from 1024 c + 32 w: ranks inside a warp by match_any, across the warps of a chunk by a scan over the
// per-warp counts, across chunks by the running per-expert totals - the same stable order as the three-pass sort.
__global__ void __launch_bounds__(1024) tables_small_kernel(const int32_t* __restrict__ topk_idx, int N, int E, int cap, int P,
                                                            int32_t* __restrict__ counts, int32_t* __restrict__ counts_chosen,
                                                            int32_t* __restrict__ offsets, int32_t* __restrict__ poffsets,
                                                            int32_t* __restrict__ tile_expert, int32_t* __restrict__ n_tiles,
                                                            int32_t* __restrict__ prow_of_slot, int32_t* __restrict__ row_of_slot,
                                                            int32_t* __restrict__ slot_of_row, int32_t* __restrict__ slot_of_prow,
                                                            int* __restrict__ status) {
    grid_dependency_wait();
    grid_dependency_launch();
    extern __shared__ int32_t sm[];                  // [32][E] per-warp counts of the chunk, [E] totals so far, 2 x [E+1]: 35 E + 2 ints
    int32_t* warp_run = sm;
    int32_t* total = sm + 32 * E;
    int32_t* s_off = total + E;
    int32_t* s_poff = s_off + E + 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < P; i += blockDim.x) slot_of_prow[i] = -1;
    if (cap < N)
        for (int i = threadIdx.x; i < N; i += blockDim.x) slot_of_row[i] = -1;
    for (int e = threadIdx.x; e < E; e += blockDim.x) total[e] = 0;
    const int chunks = (N + 1023) / 1024;
    int32_t rank_of[kSmallTablesMaxSlots / 1024];    // this thread's slot of every chunk: rank among its expert's slots
#pragma unroll
    for (int c = 0; c < kSmallTablesMaxSlots / 1024; ++c) {
        if (c >= chunks) break;                      // uniform
        for (int i = threadIdx.x; i < 32 * E; i += blockDim.x) warp_run[i] = 0;
        __syncthreads();
        const int s = c * 1024 + threadIdx.x;
        int e = s < N ? topk_idx[s] : -1;
        if ((unsigned)e >= (unsigned)E) e = -1;      // an id outside [0, E) counts nowhere
        const unsigned peers = __match_any_sync(kFull, e);
        if (e >= 0 && lane == __ffs(peers) - 1) warp_run[warp * E + e] = __popc(peers);
        const int in_warp = __popc(peers & ((1u << lane) - 1u));
        __syncthreads();
        for (int x = threadIdx.x; x < E; x += blockDim.x) {      // exclusive scan over the warps, on top of the earlier chunks
            int run = total[x];
            for (int w = 0; w < 32; ++w) {
                const int n = warp_run[w * E + x];
                warp_run[w * E + x] = run;
                run += n;
            }
            total[x] = run;
        }
        __syncthreads();
        rank_of[c] = e >= 0 ? warp_run[warp * E + e] + in_warp : 0;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int off = 0, poff = 0;
        for (int e = 0; e < E; ++e) {
            const int kept = min(total[e], cap);
            s_off[e] = off;
            s_poff[e] = poff;
            off += kept;
            poff += (kept + kPad - 1) / kPad * kPad;
        }
        s_off[E] = off;
        s_poff[E] = poff;
        *n_tiles = poff / kPad;
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E; e += blockDim.x) { offsets[e] = s_off[e]; poffsets[e] = s_poff[e]; }
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        counts[e] = min(total[e], cap);
        if (counts_chosen) counts_chosen[e] = total[e];
        for (int tile = s_poff[e] / kPad; tile < s_poff[e + 1] / kPad; ++tile) tile_expert[tile] = e;
    }
#pragma unroll
    for (int c = 0; c < kSmallTablesMaxSlots / 1024; ++c) {
        if (c >= chunks) break;
        const int s = c * 1024 + threadIdx.x;
        if (s >= N) continue;
        const int e = topk_idx[s], within = rank_of[c];
        const bool bad = (unsigned)e >= (unsigned)E;
        if (bad && status) atomicExch(status, 2);
        if (bad || within >= cap) {
            row_of_slot[s] = -1;
            prow_of_slot[s] = -1;
            continue;
        }
        const int row = s_off[e] + within, prow = s_poff[e] + within;
        row_of_slot[s] = row;
        slot_of_row[row] = s;
        prow_of_slot[s] = prow;
        slot_of_prow[prow] = s;
    }
}

}  // namespace

cudaError_t launch_topk(const float* logits, const float* b_gate, int T, int E, int k, int32_t* topk_idx,
                        float* topk_w, cudaStream_t stream) {
    if (T == 0) return cudaSuccess;
    const int warps = 8;
    if (k <= 8 && E % 32 == 0 && E <= 256 && ((uintptr_t)logits % 16 == 0) && ((uintptr_t)b_gate % 16 == 0)) {
        const unsigned blocks = (unsigned)((T + 4 * warps - 1) / (4 * warps));
        switch (E / 32) {
            case 1: return launch_chained(topk8_kernel<1>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
            case 2: return launch_chained(topk8_kernel<2>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
            case 3: return launch_chained(topk8_kernel<3>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
            case 4: return launch_chained(topk8_kernel<4>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
            case 5: return launch_chained(topk8_kernel<5>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
            case 6: return launch_chained(topk8_kernel<6>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
            case 7: return launch_chained(topk8_kernel<7>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
            default: return launch_chained(topk8_kernel<8>, blocks, warps * 32, 0, stream, logits, b_gate, T, k, topk_idx, topk_w);
        }
        return cudaGetLastError();
    }
    dim3 grid((T + warps - 1) / warps), block(warps * 32);
    const int vpl = (E + 31) / 32;
#define BIGMAC_TOPK(V)                                                                                   \
    do {                                                                                                 \
        if (k <= 32) return launch_chained(topk_kernel<V, true>, grid, block, 0, stream, logits, b_gate, T, E, k, topk_idx, topk_w);  \
        else return launch_chained(topk_kernel<V, false>, grid, block, 0, stream, logits, b_gate, T, E, k, topk_idx, topk_w);          \
    } while (0)
    if (vpl <= 1) BIGMAC_TOPK(1);
    else if (vpl <= 2) BIGMAC_TOPK(2);
    else if (vpl <= 4) BIGMAC_TOPK(4);
    else if (vpl <= 8) BIGMAC_TOPK(8);
    else if (vpl <= 16) BIGMAC_TOPK(16);
    else BIGMAC_TOPK(32);
#undef BIGMAC_TOPK
    return cudaGetLastError();
}

cudaError_t launch_tables(const Tables& tb, int T, int E, int k, int cap, cudaStream_t stream, int* status) {
    const int64_t N = (int64_t)T * k;
    const int64_t P = padded_rows_max(N, E);
    if (tables_kernel_count(N, E) == 1) {
        return launch_chained(tables_small_kernel, 1, 1024, sizeof(int32_t) * (35 * E + 2), stream, tb.topk_idx, (int)N, E, cap,
                              (int)P, tb.counts, tb.counts_chosen, tb.offsets, tb.poffsets, tb.tile_expert, tb.n_tiles,
                              tb.prow_of_slot, tb.row_of_slot, tb.slot_of_row, tb.slot_of_prow, status);
    }
    cudaError_t err = cudaMemsetAsync(tb.slot_of_prow, 0xff, sizeof(int32_t) * P, stream);
    if (err != cudaSuccess) return err;
    if (cap < N) {                                   // rows past the kept ones exist only under a capacity limit
        err = cudaMemsetAsync(tb.slot_of_row, 0xff, sizeof(int32_t) * N, stream);
        if (err != cudaSuccess) return err;
    }
    const int nb = sort_blocks(N);
    if (nb > 0) {
        err = launch_chained(sort_local_kernel, nb, 256, sizeof(int32_t) * 8 * E, stream, tb.topk_idx, N, E, tb.prow_of_slot,
                             tb.block_counts);
        if (err != cudaSuccess) return err;
    }
    err = launch_chained(sort_scan_kernel, 1, 1024, 0, stream, tb.block_counts, nb, E, tb.counts, tb.offsets, tb.poffsets,
                         tb.tile_expert, tb.n_tiles, cap, tb.counts_chosen);
    if (err != cudaSuccess) return err;
    if (N > 0)
        err = launch_chained(sort_place_kernel, (unsigned)((N + 255) / 256), 256, 0, stream, tb.topk_idx, N, E, tb.block_counts,
                             tb.offsets, tb.poffsets, tb.prow_of_slot, tb.row_of_slot, tb.slot_of_row, tb.slot_of_prow, cap,
                             status);
    return err;
}

}  // namespace bigmac
