// Per-expert weight-gradient contraction on CTA pairs, balanced under any expert load:
//     C_e[m,n] (+)= sum over the rows k of expert e of A[k,m] B[k,n]        (A, B row-major [rows, M] / [rows, N])
//
// Dropless routing gives experts very different numbers of rows, and a static round-robin of (expert, tile) items
// leaves the SMs that drew the popular experts' tiles working long after the others.  Here
//   - an expert whose contraction is long compared with the balanced share of an SM pair is cut into parts along
//     its rows (plan below); a part writes its fp32 partial result into a workspace slot, and a second kernel
//     adds the parts in order (and zero-fills the outputs of experts without rows, which get no work item);
//   - work items (expert, part, output tile) are handed out dynamically: the leader CTA's producer thread takes
//     the next item from a device counter, one item ahead of need, and passes its description on through a ring
//     in shared memory of both CTAs.  Items are numbered expert by expert, so pairs that run at the same time
//     share operands through L2 exactly as under the static order.
// How a role learns the item: the leader's producer writes ring entry i % kRing in both CTAs (the peer's by
// remote stores) and then arrives on that entry's barrier in each CTA (release at cluster scope for the peer);
// every reader - the peer's producer, the MMA warp, the epilogue warps of both CTAs - waits for that barrier
// (acquire) before it reads the entry.  The end of the list is an entry with num_kb < 0.
// Every item has at least one k slice, so the producer runs at most STAGES items ahead of the MMA warp, which
// runs at most two accumulators ahead of the epilogue: kRing = 16 entries are never overwritten while in use.
// The counter is left at zero by the last pair to finish, ready for the next launch on the stream.
// Mainloop, barriers and accumulator double-buffering are those of gemm_tc2.cu (both operands MN-major).
//
// GATHER: the rows of B are not read from a grouped copy but gathered (the dispatch fused into this operand load: for
// dW1 the rows of B are rows of x', row k of the grouped order being row gather_rows[k] / gather_div of x', zeros on
// padding rows).  The producer thread of each CTA then issues the TMA boxes of A only, and two extra warps per CTA
// follow the item ring and copy this CTA's 128 columns of the 64 gathered rows of every k slice with 16-byte
// asynchronous copies into the swizzled MN-major layout.  Each copying thread arrives on the stage's barrier when its
// copies have landed: in the leader CTA on the "full" barrier itself, in the peer on a barrier of its own that a relay
// thread (the peer's otherwise idle MMA-warp thread) waits on before it passes a proxy fence and arrives, with release
// at cluster scope, on the leader's "full" barrier; the MMA thread acquires at cluster scope and passes a proxy fence.
#include "tc_pair.cuh"

namespace bigmac {

using namespace tc;

namespace {

constexpr int kRing = 16;
constexpr int BN = 256;
constexpr int STAGES = 6;

struct Item {
    int m0, n0, expert, k_row0, num_kb, slot;
};

// Split plan, a pure function of the padded offsets: parts[e] = 0 for an expert without rows, else the number
// of parts its rows are cut into; pp = exclusive prefix of parts, ss = exclusive prefix of the parts of split
// experts (their workspace slots).  With `per` output tiles per expert on `pairs` CTA pairs the balanced share
// is total_kb * per / pairs k slices; parts are at most a quarter of it (at least 8 slices) long, and the
// length grows until the split experts' parts fit the kGroupKSlots workspace slots.
// Called by all lanes of one warp (32-bit arithmetic throughout: the plan sits in front of the first load).
__device__ void groupk_plan(const int32_t* poffsets, int E, int per, int pairs, int32_t* pp, int32_t* ss) {
    const int lane = threadIdx.x & 31;
    const int total_kb = poffsets[E] / BK;
    int len = (int)(((long long)total_kb * per) / (4 * pairs));
    if (len < 8) len = 8;
    for (int iter = 0; iter < 40; ++iter) {
        int slots = 0;
        for (int e = lane; e < E; e += 32) {
            const int kb = (poffsets[e + 1] - poffsets[e]) / BK;
            if (kb > len) slots += (kb + len - 1) / len;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) slots += __shfl_xor_sync(0xffffffffu, slots, off);
        if (slots <= kGroupKSlots) break;
        len += len / 2;
    }
    if (lane == 0) {
        int run = 0, slot = 0, lo = poffsets[0];
        for (int e = 0; e < E; ++e) {
            const int hi = poffsets[e + 1];
            const int kb = (hi - lo) / BK;
            lo = hi;
            int parts = kb == 0 ? 0 : 1;
            if (kb > len) {
                const int want = (kb + len - 1) / len;
                if (slot + want <= kGroupKSlots) parts = want;
            }
            pp[e] = run;
            ss[e] = slot;
            run += parts;
            if (parts > 1) slot += parts;
        }
        pp[E] = run;
        ss[E] = slot;
    }
}

template <bool GATHER>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GATHER ? kThreadsGather : kThreadsV2, 1)
gemm_tc_groupk_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcParams p,
                      int* __restrict__ sched, float* __restrict__ ws, int32_t* __restrict__ plan_out) {
    constexpr int BH = BN / 2;
    constexpr uint32_t A_BYTES = BM * BK * 2;
    constexpr uint32_t B_BYTES = BH * BK * 2;
    constexpr uint32_t CHUNK_BYTES = 64 * BK * 2;
    constexpr uint32_t TMEM_COLS = 2 * BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + STAGES * A_BYTES;
    uint64_t* full_bar = (uint64_t*)(smem + STAGES * (A_BYTES + B_BYTES));
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tmem_full_bar = empty_bar + STAGES;            // [2]
    uint64_t* tmem_empty_bar = tmem_full_bar + 2;            // [2], the leader's are used
    uint64_t* ring_bar = tmem_empty_bar + 2;                 // [kRing], one per ring entry
    Item* ring = (Item*)(ring_bar + kRing);                  // [kRing]
    uint32_t* tmem_slot = (uint32_t*)(ring + kRing);
    volatile int* dead = (volatile int*)(tmem_slot + 1);
    int32_t* s_pp = (int32_t*)(tmem_slot + 4);               // [E + 1] parts before expert e
    int32_t* s_ss = s_pp + p.num_experts + 1;                // [E + 1] workspace slots before expert e
    int32_t* s_off = s_ss + p.num_experts + 1;               // [E + 1] padded row offsets (a copy: the scheduler reads them per item)
    uint64_t* gfull_bar = (uint64_t*)(((uintptr_t)(s_off + p.num_experts + 1) + 7) & ~(uintptr_t)7);   // [STAGES] peer CTA: its gathered rows landed (GATHER)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    if (threadIdx.x == 32) {                                 // the maps are on their way while the barriers are set up
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    const bool leader = rank == 0;
    const int num_clusters = gridDim.x >> 1;
    const int tiles_n = (p.N + BN - 1) / BN, pairs_m = (p.M + 2 * BM - 1) / (2 * BM);
    const int per = pairs_m * tiles_n;

    if (threadIdx.x == 0) {
        // a gathered slice completes on the A boxes' bytes, on the leader's copying threads and on the peer's relay thread
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], GATHER ? 2 + kGatherWarps * 32 : 1); mbar_init(&empty_bar[s], 1); }
        if (GATHER)
            for (int s = 0; s < STAGES; ++s) mbar_init(&gfull_bar[s], kGatherWarps * 32);
        for (int s = 0; s < 2; ++s) { mbar_init(&tmem_full_bar[s], 1); mbar_init(&tmem_empty_bar[s], 2 * kEpiWarps); }
        for (int s = 0; s < kRing; ++s) mbar_init(&ring_bar[s], 1);
        *dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    // Chained launch: everything above touched no global memory and may have run while the kernel before this one in
    // the stream was still working.  Tensor memory is held, so the next kernel of the stream may be set up in turn;
    // from the wait on, the predecessor's results are complete.
    grid_dependency_launch();
    grid_dependency_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // the offsets come to shared memory in one round trip; the plan is computed from there
    for (int e = threadIdx.x; e <= p.num_experts; e += blockDim.x) s_off[e] = p.poffsets[e];
    __syncthreads();
    if (warp == 0) groupk_plan(s_off, p.num_experts, per, num_clusters, s_pp, s_ss);
    __syncthreads();
    const int total = s_pp[p.num_experts] * per;
    if (blockIdx.x == 0)     // the plan, for the finishing kernel
        for (int e = threadIdx.x; e <= p.num_experts; e += blockDim.x) { plan_out[e] = s_pp[e]; plan_out[p.num_experts + 1 + e] = s_ss[e]; }

    auto load_stage = [&](const Item& t, int kb, uint32_t it) {
        const int s = it % STAGES;
        mbar_wait_lean(&empty_bar[s], ((it / STAGES) & 1) ^ 1, dead, p.status);
        if (leader) mbar_expect_tx(&full_bar[s], GATHER ? 2 * A_BYTES : 2 * (A_BYTES + B_BYTES));
        const uint32_t bar = map_to_cta(&full_bar[s], 0);
        const int k0 = t.k_row0 + kb * BK;
        const int my_m0 = t.m0 + (int)rank * BM, my_n0 = t.n0 + (int)rank * BH;
        uint8_t* a_dst = smem_a + s * A_BYTES;
        uint8_t* b_dst = smem_b + s * B_BYTES;
#pragma unroll
        for (int c = 0; c < BM / 64; ++c) tma_load_2d_pair(a_dst + c * CHUNK_BYTES, &map_a, bar, my_m0 + 64 * c, k0);
        if (GATHER) return;                                  // the rows of B are gathered by the copying warps
#pragma unroll
        for (int c = 0; c < BH / 64; ++c) tma_load_2d_pair(b_dst + c * CHUNK_BYTES, &map_b, bar, my_n0 + 64 * c, k0);
    };

    if (GATHER && warp >= 2 + kEpiWarps) {
        // ---------------------------------------------------------- gathered B rows (two warps per CTA)
        const int gw = warp - 2 - kEpiWarps;                    // rows 32 gw .. 32 gw + 31 of every slice
        const int piece = lane & 7, chunk = (lane >> 3) & 1, r0 = lane >> 4;
        const uint8_t* src = (const uint8_t*)p.gather_src + chunk * 128 + piece * 16;
        const int64_t ld_bytes = p.gather_ld * 2;
        uint32_t it = 0;
        for (uint32_t i = 0;; ++i) {
            mbar_wait_cluster(&ring_bar[i % kRing], (i / kRing) & 1, dead, p.status);
            const Item t = ring[i % kRing];
            if (t.num_kb < 0 || *dead) break;
            const uint8_t* col = src + (int64_t)(t.n0 + (int)rank * BH) * 2;
            int idx = p.gather_rows[t.k_row0 + 32 * gw + lane];     // lane j: the source of row 32 gw + j of the slice
            for (int kb = 0; kb < t.num_kb; ++kb, ++it) {
                const int s = it % STAGES;
                const int tok = idx < 0 ? -1 : idx / p.gather_div;
                if (kb + 1 < t.num_kb) idx = p.gather_rows[t.k_row0 + (kb + 1) * BK + 32 * gw + lane];   // one slice ahead
                mbar_wait_lean(&empty_bar[s], ((it / STAGES) & 1) ^ 1, dead, p.status);
                const uint32_t base = smem_u32(smem_b + s * B_BYTES) + chunk * CHUNK_BYTES;
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const int j = r0 + 2 * q, kr = 32 * gw + j;
                    const int tk = __shfl_sync(0xffffffffu, tok, j);
                    cp_async_16(base + kr * 128 + ((piece ^ (kr & 7)) << 4), tk < 0 ? col : col + (int64_t)tk * ld_bytes, tk < 0 ? 0u : 16u);
                }
                cp_async_arrive(leader ? &full_bar[s] : &gfull_bar[s]);
            }
        }
    } else if (GATHER && warp == 1 && !leader) {
        // ---------------------------------------------------------- relay (peer CTA): gathered rows landed -> leader's barrier
        if (lane == 0) {
            const uint32_t leader_full = map_to_cta(full_bar, 0);
            uint32_t it = 0;
            for (uint32_t i = 0;; ++i) {
                mbar_wait_cluster(&ring_bar[i % kRing], (i / kRing) & 1, dead, p.status);
                const int num_kb = ring[i % kRing].num_kb;
                if (num_kb < 0 || *dead) break;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % STAGES;
                    mbar_wait_lean(&gfull_bar[s], (it / STAGES) & 1, dead, p.status);
                    fence_async_smem();
                    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(leader_full + s * 8u) : "memory");
                }
            }
        }
    } else if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            if (leader) {
                // ---------------------------------------------------------- scheduler + TMA producer (leader)
                const uint32_t peer_ring = map_to_cta(ring, 1), peer_bar = map_to_cta(ring_bar, 1);
                int w = atomicAdd(sched, 1);
                for (uint32_t i = 0;; ++i) {
                    Item t;
                    t.num_kb = -1; t.m0 = t.n0 = t.expert = t.k_row0 = 0; t.slot = -1;
                    if (w < total) {
                        const int pi = w / per, r = w - pi * per;
                        int lo = 0, hi = p.num_experts;                    // largest e with s_pp[e] <= pi
                        while (hi - lo > 1) {
                            const int mid = (lo + hi) >> 1;
                            if (s_pp[mid] <= pi) lo = mid; else hi = mid;
                        }
                        const int part = pi - s_pp[lo], parts = s_pp[lo + 1] - s_pp[lo];
                        const int row0 = s_off[lo], kb_e = (s_off[lo + 1] - row0) / BK;
                        const int kb0 = parts > 1 ? part * kb_e / parts : 0, kb1 = parts > 1 ? (part + 1) * kb_e / parts : kb_e;   // kb_e < 2^24, parts <= 32
                        t.expert = lo;
                        t.m0 = (r / tiles_n) * 2 * BM;
                        t.n0 = (r % tiles_n) * BN;
                        t.k_row0 = row0 + kb0 * BK;
                        t.num_kb = kb1 - kb0;
                        t.slot = parts > 1 ? s_ss[lo] + part : -1;
                    }
                    const int e = i % kRing;
                    ring[e] = t;
                    mbar_arrive(&ring_bar[e]);
                    const uint32_t dst = peer_ring + e * (uint32_t)sizeof(Item);
                    asm volatile("st.shared::cluster.v2.b32 [%0], {%1, %2};" ::"r"(dst), "r"(t.m0), "r"(t.n0) : "memory");
                    asm volatile("st.shared::cluster.v2.b32 [%0], {%1, %2};" ::"r"(dst + 8), "r"(t.expert), "r"(t.k_row0) : "memory");
                    asm volatile("st.shared::cluster.v2.b32 [%0], {%1, %2};" ::"r"(dst + 16), "r"(t.num_kb), "r"(t.slot) : "memory");
                    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(peer_bar + e * 8u) : "memory");
                    if (t.num_kb < 0) break;                               // end of the list
                    w = atomicAdd(sched, 1);                               // the next item, fetched behind this one's loads
                    for (int kb = 0; kb < t.num_kb; ++kb, ++it) load_stage(t, kb, it);
                }
                // the last pair to get here leaves both counters at zero for the next launch
                __threadfence();
                if (atomicAdd(sched + 1, 1) == num_clusters - 1) {
                    sched[0] = 0;
                    sched[1] = 0;
                    __threadfence();
                }
            } else {
                // ---------------------------------------------------------- TMA producer (peer)
                for (uint32_t i = 0;; ++i) {
                    const int e = i % kRing;
                    mbar_wait_cluster(&ring_bar[e], (i / kRing) & 1, dead, p.status);
                    const Item t = ring[e];
                    if (t.num_kb < 0 || *dead) break;
                    for (int kb = 0; kb < t.num_kb; ++kb, ++it) load_stage(t, kb, it);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread of the leader CTA)
        if (leader && lane == 0) {
            constexpr uint32_t idesc = instr_desc_pair(BN, true, true);
            const uint64_t da0 = smem_desc(smem_u32(smem_a), CHUNK_BYTES, 1024), db0 = smem_desc(smem_u32(smem_b), CHUNK_BYTES, 1024);
            constexpr uint32_t kStep = (UMMA_K * 128) >> 4;
            uint32_t stage = 0, phase = 0;
            for (uint32_t local = 0;; ++local) {
                const uint32_t acc = local & 1;
                mbar_wait_cluster(&ring_bar[local % kRing], (local / kRing) & 1, dead, p.status);
                const int num_kb = ring[local % kRing].num_kb;
                if (num_kb < 0 || *dead) break;
                mbar_wait_lean(&tmem_empty_bar[acc], ((local >> 1) & 1) ^ 1, dead, p.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (GATHER) {                      // the peer's relay releases at cluster scope; gathered rows are generic-proxy writes
                        mbar_wait_cluster(&full_bar[stage], phase, dead, p.status);
                        fence_async_smem();
                    } else {
                        mbar_wait_lean(&full_bar[stage], phase, dead, p.status);
                    }
                    tc_fence_after();
                    const uint64_t da = da0 + stage * (A_BYTES >> 4), db = db0 + stage * (B_BYTES >> 4);
                    umma_bf16_pair(d_tmem, da, db, idesc, kb != 0);
#pragma unroll
                    for (int kk = 1; kk < BK / UMMA_K; ++kk) umma_bf16_pair(d_tmem, da + kk * kStep, db + kk * kStep, idesc, 1);
                    umma_commit_pair(&empty_bar[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                umma_commit_pair(&tmem_full_bar[acc]);
            }
        }
    } else if (warp < 2 + kEpiWarps) {
        // ------------------------------------------------------------------ epilogue (warps 2..17, both CTAs)
        const int quad = warp & 3;
        constexpr int COLS_PER_WARP = BN / (kEpiWarps / 4);
        constexpr int CHUNKS = COLS_PER_WARP / 32;
        const int part = (warp - 2) >> 2;
        const bool vec_ok = (p.ldc % 16 == 0) && ((p.c_stride * 2) % 32 == 0) && (((uintptr_t)p.C) % 32 == 0);
        const uint32_t leader_tmem_empty[2] = {map_to_cta(&tmem_empty_bar[0], 0), map_to_cta(&tmem_empty_bar[1], 0)};
        // as in the pair kernel: p.epi_parts of the four warps of a lane quadrant do all its columns, the others leave
        const int part_step = p.epi_parts;
        if (part < part_step)
        for (uint32_t local = 0;; ++local) {
            const uint32_t acc = local & 1;
            mbar_wait_cluster(&ring_bar[local % kRing], (local / kRing) & 1, dead, p.status);
            const Item t = ring[local % kRing];
            if (t.num_kb < 0 || *dead) break;
            mbar_wait_lean(&tmem_full_bar[acc], (local >> 1) & 1, dead, p.status);
            tc_fence_after();
            const int row = t.m0 + (int)rank * BM + quad * 32 + lane;
            const bool row_ok = row < p.M;
            // whole contraction: the expert's gradient; one part of it: the part's fp32 slot in the workspace
            const int64_t row_off = (t.slot >= 0 ? (int64_t)t.slot * p.M * p.ldc : (int64_t)t.expert * p.c_stride) + (int64_t)row * p.ldc;
            for (int pp = part; pp < 4; pp += part_step) {
            const uint32_t t_addr = tmem_base + acc * BN + ((uint32_t)(quad * 32) << 16) + (uint32_t)(pp * COLS_PER_WARP);
#pragma unroll 1
            for (int c = 0; c < CHUNKS; ++c) {
                float v[32];
                tmem_load_32_nowait(t_addr + c * 32, (uint32_t*)v);
                tmem_load_wait();
                if (c == CHUNKS - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(leader_tmem_empty[acc]);
                }
                const int col0 = t.n0 + pp * COLS_PER_WARP + c * 32;
                if (col0 < p.N && row_ok) {
                    if (t.slot >= 0) {
                        TcParams p2 = p;
                        p2.C = ws; p2.out_f32 = 1; p2.accumulate = 0;
                        store_row_chunk(p2, v, row_off, col0, p.ldc % 8 == 0);
                    } else {
                        store_row_chunk(p, v, row_off, col0, vec_ok);
                    }
                }
            }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// C_e = sum of the parts of a split expert, in part order (+ C_e when accumulating); C_e = 0 for an expert
// without rows (unless accumulating).  plan = [pp (E+1) | ss (E+1)] as left by the contraction kernel.
__global__ void __launch_bounds__(256) groupk_finish_kernel(const float* __restrict__ ws, const int32_t* __restrict__ plan,
                                                            __nv_bfloat16* __restrict__ C, int64_t c_stride, int64_t mn,
                                                            int E, int accumulate) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int e = blockIdx.y;
    const int parts = plan[e + 1] - plan[e];
    if (parts == 1 || (parts == 0 && accumulate)) return;
    const float* base = ws + (int64_t)plan[E + 1 + e] * mn;
    __nv_bfloat16* dst = C + (int64_t)e * c_stride;
    for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < mn; i += (int64_t)gridDim.x * blockDim.x * 8) {
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
        for (int s = 0; s < parts; ++s) {
            const float4 v0 = *(const float4*)(base + (int64_t)s * mn + i), v1 = *(const float4*)(base + (int64_t)s * mn + i + 4);
            acc[0] += v0.x; acc[1] += v0.y; acc[2] += v0.z; acc[3] += v0.w;
            acc[4] += v1.x; acc[5] += v1.y; acc[6] += v1.z; acc[7] += v1.w;
        }
        uint4 out;
        if (accumulate) {
            out = *(const uint4*)(dst + i);
            const uint32_t* w = (const uint32_t*)&out;
#pragma unroll
            for (int j = 0; j < 4; ++j) { acc[2 * j] += bf16_lo(w[j]); acc[2 * j + 1] += bf16_hi(w[j]); }
        }
        out.x = pack_bf16(acc[0], acc[1]); out.y = pack_bf16(acc[2], acc[3]);
        out.z = pack_bf16(acc[4], acc[5]); out.w = pack_bf16(acc[6], acc[7]);
        *(uint4*)(dst + i) = out;
    }
}

}  // namespace

bool gemm_tc_groupk_supported(const GemmArgs& g) {
    return g.group == GROUP_K && !g.a_kmajor && !g.b_kmajor && g.N >= 256 && g.ldc == g.N && g.N % 8 == 0 && !g.out_f32 &&
           g.epilogue == EPI_NONE && g.poffsets && g.c_stride == (int64_t)g.M * g.N && ((uintptr_t)g.C % 16 == 0) &&
           g.num_experts <= kMaxExperts;
}

size_t gemm_tc_groupk_ws_bytes(int M, int N, int E) {
    return (size_t)kGroupKSlots * M * N * sizeof(float) + 2 * (size_t)(E + 1) * sizeof(int32_t) + 256;
}

// ws: gemm_tc_groupk_ws_bytes(M, N, E) bytes, 256-byte aligned; sched: two ints, zero between launches.
cudaError_t gemm_tc_groupk(const GemmArgs& g, int* status, int* sched, void* ws, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0 || g.num_experts <= 0) return cudaSuccess;
    const int E = g.num_experts;
    CUtensorMap ma, mb;
    const bool gather = g.gather_rows != nullptr;            // B's rows are gathered by the producer warps: no tensor map for B
    if (gather && ((g.ldb * 2) % 16 || (uintptr_t)g.B % 16 || g.N % 128)) return cudaErrorInvalidValue;
    bool ok = make_map(&ma, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda, 64, BK);
    ok &= gather ? make_map(&mb, g.B, (uint64_t)g.N, 1, (uint64_t)g.ldb, 64, 1)         // placeholder, never used
                 : make_map(&mb, g.B, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.ldb, 64, BK);
    if (!ok) return cudaErrorInvalidValue;
    TcParams p{};
    p.C = g.C; p.ldc = g.ldc; p.c_stride = g.c_stride; p.M = g.M; p.N = g.N; p.K = g.K;
    p.accumulate = g.accumulate; p.epilogue = EPI_NONE; p.group = GROUP_K; p.num_experts = E; p.poffsets = g.poffsets;
    p.status = status; p.split_k = 1; p.b2_first_kb = -1; p.n_split = -1; p.epi_parts = epi_parts_default(g.epi_parts);
    p.gather_rows = g.gather_rows; p.gather_src = g.B; p.gather_ld = g.ldb; p.gather_div = g.gather_div > 0 ? g.gather_div : 1;
    float* slots = (float*)ws;
    int32_t* plan = (int32_t*)((char*)ws + (((size_t)kGroupKSlots * g.M * g.N * sizeof(float) + 255) & ~(size_t)255));
    constexpr size_t kMaxSmem = 232448;
    const size_t smem = STAGES * (BM * BK * 2 + (BN / 2) * BK * 2) + (2 * STAGES + 4 + kRing) * 8 + kRing * sizeof(Item) + 16 +
                        3 * (size_t)(E + 1) * 4 + 8 + STAGES * 8 + 1024;
    if (smem > kMaxSmem) return cudaErrorInvalidConfiguration;
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_groupk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_groupk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
        if (e != cudaSuccess) return e;
        once.mark(dev);
    }
    const int clusters = sm_count() / 2 > 0 ? sm_count() / 2 : 1;
    if (gather) return launch_chained(gemm_tc_groupk_kernel<true>, 2 * clusters, kThreadsGather, smem, stream, ma, mb, p, sched, slots, plan);
    return launch_chained(gemm_tc_groupk_kernel<false>, 2 * clusters, kThreadsV2, smem, stream, ma, mb, p, sched, slots, plan);
}

// Second step of gemm_tc_groupk (same g, same ws, same stream): adds the parts of split experts, zero-fills the
// gradients of experts without rows.
cudaError_t gemm_tc_groupk_finish(const GemmArgs& g, void* ws, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0 || g.num_experts <= 0) return cudaSuccess;
    const int E = g.num_experts;
    float* slots = (float*)ws;
    int32_t* plan = (int32_t*)((char*)ws + (((size_t)kGroupKSlots * g.M * g.N * sizeof(float) + 255) & ~(size_t)255));
    const int64_t mn = (int64_t)g.M * g.N;
    dim3 grid((unsigned)((mn / 8 + 255) / 256 < 64 ? (mn / 8 + 255) / 256 : 64), (unsigned)E);
    return launch_chained(groupk_finish_kernel, grid, 256, 0, stream, slots, plan, (__nv_bfloat16*)g.C, g.c_stride, mn, E, g.accumulate ? 1 : 0);
}

}  // namespace bigmac
