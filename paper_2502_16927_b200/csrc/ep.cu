// Expert-parallel entry points of libbigmac (Fig. 2c; Eq. 1 with the row width h replaced by r h): every rank holds
// the shared projections and the gate in full and E/size experts; the two All-to-All exchanges are row puts and gets
// over peer memory at the low width r, issued by the kernels in this file.  A rank's kernels never wait on another
// rank's: the phases are separate calls and the caller puts a barrier between them.
//
// Row placement.  Expert e is owned by rank q = e / El (El = E / size) and holds, in q's grouped buffers, the rows
// of all ranks' slots that chose it: rank 0's first, then rank 1's, ..., each rank's in its own slot order, which
// is the stable order of one layer applied to the concatenation of the ranks' batches.  Segments are padded to
// kPad rows like everywhere else.  With counts_all[p][e] known to every rank, a rank computes on its own where
// each of its slots lands:  row = poffset_q(e) + sum_{p' < rank} counts_all[p'][e] + (rank of the slot among this
// rank's slots of e).  No sizes ever reach the host.
#include <cmath>

#include "layer_common.h"

using namespace bigmac;
using namespace bigmac::detail;

namespace bigmac {
namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kMaxRanks = BIGMAC_EP_MAX_RANKS;

struct Peers { void* p[kMaxRanks]; };

__device__ __forceinline__ int warp_global_id() { return blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); }

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
template <typename T> struct Row;          // 16 bytes of T as floats
template <> struct Row<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ uint4 pack(const float* f) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
};
template <> struct Row<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) { unpack8(v, f); }
    static __device__ __forceinline__ uint4 pack(const float* f) { return pack8(f); }
};

// One block.  From counts_all [size, E]: where this rank's slots of every expert start at their owner (send_base),
// and the tables of the segments this rank owns (padded offsets, tile -> local expert, tiles in use).
// A count matrix that cannot be right (a negative entry, or more rows for one owner than its buffers hold: the caller
// skipped the all-gather, or passed another step's) must not turn into stores outside the buffers: the kernel then
// records kBadCounts in the status word and publishes an empty layout (send_base -1, no tiles), which every later
// kernel of the step treats as "nothing to move".
constexpr int kBadCounts = 2;
__global__ void __launch_bounds__(1024) ep_layout_kernel(const int32_t* __restrict__ counts_all, int size, int rank, int E, int El,
                                                         int64_t max_rows, int* __restrict__ status,
                                                         int32_t* __restrict__ send_base, int32_t* __restrict__ poff_own,
                                                         int32_t* __restrict__ tile_expert_own, int32_t* __restrict__ n_tiles_own) {
    __shared__ int s_bad;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    __shared__ int32_t s_total[kMaxExperts];     // rows of expert e over all ranks
    __shared__ int32_t s_before[kMaxExperts];    // ... of the ranks before this one
    __shared__ int32_t s_poff[kMaxExperts];      // padded offset of expert e in its owner's buffers
    __shared__ int32_t s_end[kMaxRanks];         // padded rows in use at owner q
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        int total = 0, before = 0;
        for (int p = 0; p < size; ++p) {
            const int c = counts_all[(size_t)p * E + e];
            if (c < 0 || (int64_t)c > max_rows) { s_bad = 1; continue; }
            total += c;                          // at most size * max_rows: no overflow
            if (p < rank) before += c;
        }
        s_total[e] = total;
        s_before[e] = before;
    }
    __syncthreads();
    if ((int)threadIdx.x < size) {               // owner q: prefix over its experts
        const int q = threadIdx.x;
        int64_t poff = 0;
        for (int j = 0; j < El; ++j) {
            s_poff[q * El + j] = (int32_t)(poff < max_rows ? poff : max_rows);
            poff += ((int64_t)s_total[q * El + j] + kPad - 1) / kPad * kPad;
        }
        if (poff > max_rows) s_bad = 1;
        s_end[q] = (int32_t)(poff < max_rows ? poff : max_rows);
    }
    __syncthreads();
    if (s_bad) {
        for (int e = threadIdx.x; e < E; e += blockDim.x) send_base[e] = -1;
        for (int j = threadIdx.x; j <= El; j += blockDim.x) poff_own[j] = 0;
        if (threadIdx.x == 0) { *n_tiles_own = 0; atomicExch(status, kBadCounts); }
        return;
    }
    for (int e = threadIdx.x; e < E; e += blockDim.x) send_base[e] = s_poff[e] + s_before[e];
    for (int j = threadIdx.x; j <= El; j += blockDim.x) poff_own[j] = j < El ? s_poff[rank * El + j] : s_end[rank];
    if (threadIdx.x == 0) *n_tiles_own = s_end[rank] / kPad;
    for (int j = threadIdx.x; j < El; j += blockDim.x) {
        const int first = s_poff[rank * El + j] / kPad;
        const int last = (j + 1 < El ? s_poff[rank * El + j + 1] : s_end[rank]) / kPad;
        for (int tile = first; tile < last; ++tile) tile_expert_own[tile] = j;
    }
}

// Zero the padding rows of this rank's segments in two buffers (no peer ever writes there).  Block j: local expert j.
__global__ void __launch_bounds__(256) ep_zero_padding_kernel(uint4* __restrict__ buf_a, uint4* __restrict__ buf_b,
                                                              const int32_t* __restrict__ poff_own,
                                                              const int32_t* __restrict__ counts_all, int size, int rank, int E,
                                                              int El, int vecs) {
    const int j = blockIdx.x;
    int64_t total = 0;
    for (int p = 0; p < size; ++p) {
        const int c = counts_all[(size_t)p * E + rank * El + j];
        if (c < 0) return;                           // rejected by ep_layout_kernel: the layout is empty
        total += c;
    }
    const int64_t first = (int64_t)poff_own[j] + total, last = poff_own[j + 1];
    if (first >= last) return;                       // no padding rows (or an empty layout)
    const int64_t n = (last - first) * vecs;
    for (int64_t i = threadIdx.x; i < n; i += blockDim.x) {
        buf_a[first * vecs + i] = make_uint4(0, 0, 0, 0);
        buf_b[first * vecs + i] = make_uint4(0, 0, 0, 0);
    }
}

// First exchange.  One warp per slot of this rank: its row of x' goes to the owner's grouped buffer.
__global__ void __launch_bounds__(256) ep_put_rows_kernel(const uint4* __restrict__ src, Peers dst, const int32_t* __restrict__ topk_idx,
                                                          const int32_t* __restrict__ row_of_slot, const int32_t* __restrict__ offsets,
                                                          const int32_t* __restrict__ send_base, int32_t* __restrict__ dest_row,
                                                          int64_t N, int k, int El, int vecs, int E) {
    const int64_t s = warp_global_id();
    if (s >= N) return;
    const int lane = threadIdx.x & 31;
    const int e = topk_idx[s];
    const int base = (unsigned)e < (unsigned)E ? send_base[e] : -1;   // an id outside [0, E): treated like an empty layout
    if (base < 0) {                                  // empty layout (see ep_layout_kernel): nothing moves
        if (lane == 0) dest_row[s] = -1;
        return;
    }
    const int dest = base + row_of_slot[s] - offsets[e];
    if (lane == 0) dest_row[s] = dest;
    const uint4* from = src + (s / k) * vecs;
    uint4* to = (uint4*)dst.p[e / El] + (int64_t)dest * vecs;
    for (int c = lane; c < vecs; c += 32) to[c] = from[c];
}

// Second exchange (and, with w == nullptr, the gather of dxg in the backward pass).  One warp per token:
// dst[t,:] = sum_j w[s] * buf_{owner(s)}[dest_row[s],:], slots in order, fp32 accumulation.
template <typename T>
__global__ void __launch_bounds__(256) ep_get_combine_kernel(Peers src, uint4* __restrict__ dst, const float* __restrict__ w,
                                                             const int32_t* __restrict__ topk_idx,
                                                             const int32_t* __restrict__ dest_row, int n_tokens, int k, int El,
                                                             int vecs, int dst_vecs) {
    constexpr int V = Row<T>::kElems;
    const int t = warp_global_id();
    if (t >= n_tokens) return;
    const int lane = threadIdx.x & 31;
    for (int c = lane; c < vecs; c += 32) {
        float acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = 0.0f;
        for (int j = 0; j < k; ++j) {
            const int64_t s = (int64_t)t * k + j;
            const int row = dest_row[s];
            if (row < 0) continue;                       // empty layout
            const float p = w ? w[s] : 1.0f;
            float f[V];
            Row<T>::unpack(((const uint4*)src.p[topk_idx[s] / El])[(int64_t)row * vecs + c], f);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] = fmaf(p, f[i], acc[i]);
        }
        dst[(int64_t)t * dst_vecs + c] = Row<T>::pack(acc);
    }
}

// Backward of the combine, from the token's side.  One warp per slot: dp[s] = <dy'[t], u at the owner> (get),
// du at the owner = p[s] dy'[t] (put).
template <typename T>
__global__ void __launch_bounds__(256) ep_combine_bwd_kernel(const uint4* __restrict__ dy_lo, Peers u, Peers du, float* __restrict__ dp,
                                                             const float* __restrict__ topk_w, const int32_t* __restrict__ topk_idx,
                                                             const int32_t* __restrict__ dest_row, int64_t N, int k, int El, int vecs) {
    constexpr int V = Row<T>::kElems;
    const int64_t s = warp_global_id();
    if (s >= N) return;
    const int lane = threadIdx.x & 31;
    const int q = topk_idx[s] / El;
    const int64_t row = dest_row[s];
    if (row < 0) {                                   // empty layout
        if (lane == 0) dp[s] = 0.0f;
        return;
    }
    const float p = topk_w[s];
    const uint4* g = dy_lo + (s / k) * vecs;
    const uint4* ur = (const uint4*)u.p[q] + row * vecs;
    uint4* out = (uint4*)du.p[q] + row * vecs;
    float dot = 0.0f;
    for (int c = lane; c < vecs; c += 32) {
        float a[V], b[V], o[V];
        Row<T>::unpack(g[c], a);
        Row<T>::unpack(ur[c], b);
#pragma unroll
        for (int i = 0; i < V; ++i) { dot = fmaf(a[i], b[i], dot); o[i] = p * a[i]; }
        out[c] = Row<T>::pack(o);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(kFull, dot, off);
    if (lane == 0) dp[s] = dot;
}

inline unsigned warp_blocks(int64_t warps) { return (unsigned)((warps + 7) / 8); }

// ---- host side ---------------------------------------------------------------------------------------------

struct EpDims {
    int T, d, r, h, E, El, k, dtype, size, rank;
    int64_t N, P, Pep;   // this rank's slots, its local padded bound (tables), the bound on rows it can receive
    int E64, z_es, ldcat;
    bool cdac;           // Eq. 3 layer: no shared projections, rows travel at the full width d (r == d)
};

struct EpBuffers {
    Tables tb;                                    // this rank's slots sorted by (global) expert
    int32_t *send_base, *dest_row;                // [E], [N]
    int32_t *poff_own, *tile_expert_own, *n_tiles_own;
    void *x_lo, *y_lo, *z, *a;                    // saved
    float* logits;                                // scratch (route)
    void *dy_lo, *dz, *dcat, *dx_lo, *dlogits;    // scratch (backward)
    float *dp, *colsum_part, *splitk_ws;
};

int ep_dims(const bigmac_layer* L, int32_t T, int size, int rank, EpDims* out) {
    const bigmac_config_t& c = L->cfg;
    if (size < 1 || size > kMaxRanks || rank < 0 || rank >= size) return BIGMAC_ERR_INVALID_ARG;
    if (c.E % size) return BIGMAC_ERR_INVALID_ARG;
    if (c.capacity_factor > 0 || c.aux_loss_coef > 0 || (c.flags & (BIGMAC_FLAG_GATE_LOW | BIGMAC_FLAG_EXPERT_BIAS)))
        return BIGMAC_ERR_UNSUPPORTED;
    if ((int64_t)size * c.max_tokens * c.k > (int64_t)1 << 30) return BIGMAC_ERR_UNSUPPORTED;
    EpDims m{};
    m.T = T; m.d = c.d; m.r = c.r; m.h = c.h; m.E = c.E; m.El = c.E / size; m.k = c.k; m.dtype = c.dtype;
    m.size = size; m.rank = rank;
    m.N = (int64_t)T * c.k;
    m.P = padded_rows_max(m.N, c.E);
    m.Pep = padded_rows_max((int64_t)size * c.max_tokens * c.k, m.El);
    m.E64 = (c.E + 63) / 64 * 64;
    m.z_es = sigma_as_bytes(L) ? 1 : (int)esize(c.dtype);
    m.cdac = (c.flags & BIGMAC_FLAG_CDAC) != 0;
    m.ldcat = m.cdac ? m.E64 : m.r + m.E64;
    *out = m;
    return BIGMAC_OK;
}

// The owner-side items come first and their sizes do not depend on T: the two expert phases are called without it.
void carve_ep_saved(Carver& cv, const EpDims& m, EpBuffers& b) {
    const size_t es = esize(m.dtype);
    b.poff_own = cv.take<int32_t>(m.El + 1);
    b.tile_expert_own = cv.take<int32_t>(m.Pep / kPad);
    b.n_tiles_own = cv.take<int32_t>(1);
    b.z = cv.take_bytes((size_t)m.Pep * m.h * m.z_es);
    b.a = cv.take_bytes((size_t)m.Pep * m.h * es);
    b.tb.counts = cv.take<int32_t>(m.E);
    b.tb.offsets = cv.take<int32_t>(m.E + 1);
    b.tb.poffsets = cv.take<int32_t>(m.E + 1);
    b.tb.n_tiles = cv.take<int32_t>(1);
    b.tb.counts_chosen = cv.take<int32_t>(m.E);
    b.send_base = cv.take<int32_t>(m.E);
    b.tb.topk_idx = cv.take<int32_t>(m.N);
    b.tb.topk_w = cv.take<float>(m.N);
    b.tb.row_of_slot = cv.take<int32_t>(m.N);
    b.tb.slot_of_row = cv.take<int32_t>(m.N);
    b.tb.prow_of_slot = cv.take<int32_t>(m.N);
    b.tb.slot_of_prow = cv.take<int32_t>(m.P);
    b.tb.tile_expert = cv.take<int32_t>(m.P / kPad);
    b.dest_row = cv.take<int32_t>(m.N);
    b.x_lo = cv.take_bytes((size_t)m.T * m.r * es);
    b.y_lo = cv.take_bytes((size_t)m.T * m.r * es);
}

void carve_ep_scratch(Carver& cv, const EpDims& m, EpBuffers& b) {
    const size_t es = esize(m.dtype);
    b.dz = m.z_es == 1 ? cv.take_bytes((size_t)m.Pep * m.h * es) : nullptr;
    const size_t dense_ws = (size_t)kMaxSplitK * m.ldcat * m.d * sizeof(float);
    const size_t expert_ws = m.dtype == BIGMAC_BF16 ? gemm_tc_groupk_ws_bytes(m.r, m.h, m.El) : 0;
    b.splitk_ws = (float*)cv.take_bytes(dense_ws > expert_ws ? dense_ws : expert_ws);
    b.colsum_part = cv.take<float>((size_t)kColsumChunks * m.E);
    b.logits = cv.take<float>((size_t)m.T * m.E);
    b.tb.block_counts = cv.take<int32_t>((size_t)(sort_blocks(m.N) + 1) * m.E);
    b.dy_lo = cv.take_bytes((size_t)m.T * m.r * es);
    b.dcat = cv.take_bytes((size_t)m.T * m.ldcat * es);
    b.dx_lo = m.cdac ? nullptr : b.dcat;                              // Eq. 3: dx' is dx itself
    b.dlogits = m.cdac ? b.dcat : (char*)b.dcat + (size_t)m.r * es;
    b.dp = cv.take<float>(m.N);
}

size_t ep_saved_bytes(const EpDims& m) { Carver cv(nullptr); EpBuffers b{}; carve_ep_saved(cv, m, b); return cv.total(); }
size_t ep_scratch_bytes(const EpDims& m) { Carver cv(nullptr); EpBuffers b{}; carve_ep_scratch(cv, m, b); return cv.total(); }

// Argument checks shared by the phases; fills the dims and carves both workspaces.
int ep_enter(const bigmac_layer* L, int32_t T, const bigmac_ep_t* ep, void* saved, void* scratch, size_t scratch_bytes,
             bool need_scratch, EpDims* m, EpBuffers* b) {
    BIGMAC_TRY(check_call(L, T));
    if (!ep || !ep->counts_all || !saved || !aligned(saved, 256)) return BIGMAC_ERR_INVALID_ARG;
    BIGMAC_TRY(ep_dims(L, T, ep->size, ep->rank, m));
    for (int q = 0; q < ep->size; ++q)
        if (!ep->xg[q] || !ep->u[q] || !ep->du[q] || !ep->dxg[q] || !aligned(ep->xg[q], 16) || !aligned(ep->u[q], 16) ||
            !aligned(ep->du[q], 16) || !aligned(ep->dxg[q], 16))
            return BIGMAC_ERR_INVALID_ARG;
    Carver cv(saved);
    carve_ep_saved(cv, *m, *b);
    if (need_scratch) {
        if (!scratch || !aligned(scratch, 256)) return BIGMAC_ERR_INVALID_ARG;
        if (scratch_bytes < ep_scratch_bytes(*m)) return BIGMAC_ERR_WORKSPACE;
        Carver cs(scratch);
        carve_ep_scratch(cs, *m, *b);
    }
    return BIGMAC_OK;
}

Peers peers_of(void* const* bufs, int size) {
    Peers p{};
    for (int q = 0; q < size; ++q) p.p[q] = bufs[q];
    return p;
}

int check_shared_weights(const bigmac_weights_t* W, bool experts, bool cdac = false) {
    if (!W) return BIGMAC_ERR_INVALID_ARG;
    if (experts) return (W->w1 && W->w2 && aligned(W->w1, 16) && aligned(W->w2, 16)) ? BIGMAC_OK : BIGMAC_ERR_INVALID_ARG;
    if (!W->w_gate || !aligned(W->w_gate, 16) || !aligned(W->b_gate, 4)) return BIGMAC_ERR_INVALID_ARG;
    if (cdac) return BIGMAC_OK;
    if (!W->w_down || !W->w_up || !aligned(W->w_down, 16) || !aligned(W->w_up, 16)) return BIGMAC_ERR_INVALID_ARG;
    return BIGMAC_OK;
}

}  // namespace
}  // namespace bigmac

extern "C" {

int bigmac_ep_buffer_bytes(const bigmac_layer_t* L, int32_t size, size_t* bytes) {
    if (!L || !bytes) return BIGMAC_ERR_INVALID_ARG;
    EpDims m;
    BIGMAC_TRY(ep_dims(L, 0, size, 0, &m));
    *bytes = (size_t)m.Pep * m.r * esize(m.dtype);
    return BIGMAC_OK;
}

int bigmac_ep_workspace_bytes(const bigmac_layer_t* L, int32_t T, int32_t size, size_t* scratch_bytes, size_t* saved_bytes) {
    if (!L || !scratch_bytes || !saved_bytes || T < 0 || T > L->cfg.max_tokens) return BIGMAC_ERR_INVALID_ARG;
    EpDims m;
    BIGMAC_TRY(ep_dims(L, T, size, 0, &m));
    *scratch_bytes = ep_scratch_bytes(m);
    *saved_bytes = ep_saved_bytes(m);
    return BIGMAC_OK;
}

int bigmac_ep_route(bigmac_layer_t* L, const void* x, int32_t T, const bigmac_weights_t* W, const bigmac_ep_t* ep,
                    bigmac_routing_t* routing_out, void* saved, void* scratch, size_t scratch_bytes, void* stream) {
    EpDims m;
    EpBuffers b{};
    BIGMAC_TRY(ep_enter(L, T, ep, saved, scratch, scratch_bytes, true, &m, &b));
    BIGMAC_TRY(check_shared_weights(W, false, m.cdac));
    cudaStream_t st = (cudaStream_t)stream;
    int32_t* my_counts = ep->counts_all + (size_t)m.rank * m.E;
    if (T == 0) {                                    // this rank brings nothing: its row of the count matrix is zero
        BIGMAC_CUDA(cudaMemsetAsync(my_counts, 0, sizeof(int32_t) * m.E, st));
        return BIGMAC_OK;
    }
    if (!x || !aligned(x, 16)) return BIGMAC_ERR_INVALID_ARG;
    const int bn_desc = (m.r + m.E) >= 256 ? 256 : 128;
    if (m.cdac) {                                    // Eq. 3: logits only; the rows that travel are the tokens themselves,
        GemmArgs g;                                  // kept in `saved` so that the dispatch phase needs no x
        g.A = x; g.lda = m.d; g.B = W->w_gate; g.ldb = m.d; g.C = b.logits; g.ldc = m.E;
        g.M = m.T; g.N = m.E; g.K = m.d; g.out_f32 = true;
        BIGMAC_TRY(gemm(L, G_LOGITS, g, st));
        BIGMAC_CUDA(cudaMemcpyAsync(b.x_lo, x, (size_t)m.T * m.d * esize(m.dtype), cudaMemcpyDeviceToDevice, st));
    } else if (m.dtype == BIGMAC_BF16 && L->use_tc && L->tc_mask == ~0u && m.r % bn_desc == 0) {
        GemmArgs g;                                  // [x' | logits] = x [W'_down ; W_gate]^T in one pass over x
        g.A = x; g.lda = m.d; g.B = W->w_down; g.ldb = m.d; g.C = b.x_lo; g.ldc = m.r;
        g.B2 = W->w_gate; g.ldb2 = m.d; g.n_split = m.r; g.C2 = b.logits; g.ldc2 = m.E; g.N2 = m.E;
        g.M = m.T; g.N = m.r + m.E; g.K = m.d;
        BIGMAC_TRY(gemm(L, G_DESCEND, g, st));
    } else {
        GemmArgs g;
        g.A = x; g.lda = m.d; g.B = W->w_gate; g.ldb = m.d; g.C = b.logits; g.ldc = m.E;
        g.M = m.T; g.N = m.E; g.K = m.d; g.out_f32 = true;
        BIGMAC_TRY(gemm(L, G_LOGITS, g, st));
        GemmArgs q;
        q.A = x; q.lda = m.d; q.B = W->w_down; q.ldb = m.d; q.C = b.x_lo; q.ldc = m.r;
        q.M = m.T; q.N = m.r; q.K = m.d;
        BIGMAC_TRY(gemm(L, G_DESCEND, q, st));
    }
    { Stage s(L, S_TOPK, st); BIGMAC_CUDA(launch_topk(b.logits, W->b_gate, m.T, m.E, m.k, b.tb.topk_idx, b.tb.topk_w, st)); }
    { Stage s(L, S_TABLES, st, tables_kernel_count(m.N, m.E)); BIGMAC_CUDA(launch_tables(b.tb, m.T, m.E, m.k, kNoCapacity, st, L->status)); }
    BIGMAC_CUDA(cudaMemcpyAsync(my_counts, b.tb.counts, sizeof(int32_t) * m.E, cudaMemcpyDeviceToDevice, st));
    if (routing_out) {
        const cudaMemcpyKind kind = cudaMemcpyDeviceToDevice;
        if (routing_out->topk_idx) BIGMAC_CUDA(cudaMemcpyAsync(routing_out->topk_idx, b.tb.topk_idx, sizeof(int32_t) * m.N, kind, st));
        if (routing_out->topk_w) BIGMAC_CUDA(cudaMemcpyAsync(routing_out->topk_w, b.tb.topk_w, sizeof(float) * m.N, kind, st));
        if (routing_out->counts) BIGMAC_CUDA(cudaMemcpyAsync(routing_out->counts, b.tb.counts, sizeof(int32_t) * m.E, kind, st));
        if (routing_out->offsets) BIGMAC_CUDA(cudaMemcpyAsync(routing_out->offsets, b.tb.offsets, sizeof(int32_t) * (m.E + 1), kind, st));
        if (routing_out->row_of_slot) BIGMAC_CUDA(cudaMemcpyAsync(routing_out->row_of_slot, b.tb.row_of_slot, sizeof(int32_t) * m.N, kind, st));
        if (routing_out->slot_of_row) BIGMAC_CUDA(cudaMemcpyAsync(routing_out->slot_of_row, b.tb.slot_of_row, sizeof(int32_t) * m.N, kind, st));
        if (routing_out->counts_chosen) BIGMAC_CUDA(cudaMemcpyAsync(routing_out->counts_chosen, b.tb.counts, sizeof(int32_t) * m.E, kind, st));
        if (routing_out->aux_loss) BIGMAC_CUDA(cudaMemsetAsync(routing_out->aux_loss, 0, sizeof(float), st));
    }
    return BIGMAC_OK;
}

int bigmac_ep_dispatch(bigmac_layer_t* L, int32_t T, const bigmac_ep_t* ep, void* saved, void* stream) {
    EpDims m;
    EpBuffers b{};
    BIGMAC_TRY(ep_enter(L, T, ep, saved, nullptr, 0, false, &m, &b));
    cudaStream_t st = (cudaStream_t)stream;
    const int vecs = m.r * (int)esize(m.dtype) / 16;
    Stage s(L, S_DISPATCH, st, T > 0 ? 3 : 2);
    ep_layout_kernel<<<1, 1024, 0, st>>>(ep->counts_all, m.size, m.rank, m.E, m.El, m.Pep, L->status, b.send_base, b.poff_own,
                                         b.tile_expert_own, b.n_tiles_own);
    ep_zero_padding_kernel<<<m.El, 256, 0, st>>>((uint4*)ep->xg[m.rank], (uint4*)ep->du[m.rank], b.poff_own, ep->counts_all, m.size,
                                                 m.rank, m.E, m.El, vecs);
    if (T > 0)
        ep_put_rows_kernel<<<warp_blocks(m.N), 256, 0, st>>>((const uint4*)b.x_lo, peers_of(ep->xg, m.size), b.tb.topk_idx,
                                                            b.tb.row_of_slot, b.tb.offsets, b.send_base, b.dest_row, m.N, m.k, m.El,
                                                            vecs, m.E);
    BIGMAC_CUDA(cudaGetLastError());
    return BIGMAC_OK;
}

int bigmac_ep_experts(bigmac_layer_t* L, const bigmac_weights_t* W, const bigmac_ep_t* ep, void* saved, void* stream) {
    EpDims m;
    EpBuffers b{};
    BIGMAC_TRY(ep_enter(L, 0, ep, saved, nullptr, 0, false, &m, &b));
    BIGMAC_TRY(check_shared_weights(W, true));
    cudaStream_t st = (cudaStream_t)stream;
    {   // a = sigma(xg W1_e^T) over the received rows; saves sigma'(z)
        GemmArgs g;
        g.A = ep->xg[m.rank]; g.lda = m.r; g.B = W->w1; g.ldb = m.r; g.b_stride = (int64_t)m.h * m.r;
        g.C = b.a; g.Z = b.z; g.ldc = m.h; g.M = (int)m.Pep; g.N = m.h; g.K = m.r;
        g.epilogue = EPI_ACT; g.act = L->cfg.act; g.group = GROUP_M; g.num_experts = m.El;
        g.tile_expert = b.tile_expert_own; g.n_tiles = b.n_tiles_own; g.poffsets = b.poff_own;
        BIGMAC_TRY(gemm(L, G_EXPERT1, g, st));
    }
    {   // u = a W2_e^T
        GemmArgs g;
        g.A = b.a; g.lda = m.h; g.B = W->w2; g.ldb = m.h; g.b_stride = (int64_t)m.r * m.h;
        g.C = ep->u[m.rank]; g.ldc = m.r; g.M = (int)m.Pep; g.N = m.r; g.K = m.h;
        g.group = GROUP_M; g.num_experts = m.El; g.tile_expert = b.tile_expert_own; g.n_tiles = b.n_tiles_own; g.poffsets = b.poff_own;
        BIGMAC_TRY(gemm(L, G_EXPERT2, g, st));
    }
    return BIGMAC_OK;
}

int bigmac_ep_combine(bigmac_layer_t* L, int32_t T, const bigmac_weights_t* W, const bigmac_ep_t* ep, void* y, void* saved,
                      void* stream) {
    EpDims m;
    EpBuffers b{};
    BIGMAC_TRY(ep_enter(L, T, ep, saved, nullptr, 0, false, &m, &b));
    BIGMAC_TRY(check_shared_weights(W, false, m.cdac));
    if (T == 0) return BIGMAC_OK;
    if (!y || !aligned(y, 16)) return BIGMAC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int vecs = m.r * (int)esize(m.dtype) / 16;
    uint4* y_lo = (uint4*)(m.cdac ? y : b.y_lo);     // Eq. 3: the weighted sum is the output
    {
        Stage s(L, S_COMBINE, st);
        if (m.dtype == BIGMAC_BF16)
            ep_get_combine_kernel<__nv_bfloat16><<<warp_blocks(T), 256, 0, st>>>(peers_of(ep->u, m.size), y_lo, b.tb.topk_w,
                                                                                b.tb.topk_idx, b.dest_row, T, m.k, m.El, vecs, vecs);
        else
            ep_get_combine_kernel<float><<<warp_blocks(T), 256, 0, st>>>(peers_of(ep->u, m.size), y_lo, b.tb.topk_w,
                                                                        b.tb.topk_idx, b.dest_row, T, m.k, m.El, vecs, vecs);
        BIGMAC_CUDA(cudaGetLastError());
    }
    if (m.cdac) return BIGMAC_OK;
    GemmArgs g;                                      // y = y' W'_up
    g.A = b.y_lo; g.lda = m.r; g.B = W->w_up; g.ldb = m.r; g.C = y; g.ldc = m.d;
    g.M = m.T; g.N = m.d; g.K = m.r;
    return gemm(L, G_ASCEND, g, st);
}

int bigmac_ep_backward_combine(bigmac_layer_t* L, const void* dy, int32_t T, const bigmac_weights_t* W, const bigmac_ep_t* ep,
                               const bigmac_grads_t* G, int accumulate, void* saved, void* scratch, size_t scratch_bytes,
                               void* stream) {
    EpDims m;
    EpBuffers b{};
    BIGMAC_TRY(ep_enter(L, T, ep, saved, scratch, scratch_bytes, true, &m, &b));
    BIGMAC_TRY(check_shared_weights(W, false, m.cdac));
    if (!G) return BIGMAC_ERR_INVALID_ARG;
    if (T == 0) return BIGMAC_OK;
    if (!dy || !aligned(dy, 16) || !aligned(G->dw_up, 16)) return BIGMAC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const bool acc = accumulate != 0;
    const bool fused = m.dtype == BIGMAC_BF16 && L->use_tc && L->tc_mask == ~0u;
    const void* dy_lo = m.cdac ? dy : b.dy_lo;       // Eq. 3: dy' is dy
    if (!m.cdac) {   // dy' = dy W_up
        GemmArgs g;
        g.A = dy; g.lda = m.d; g.B = W->w_up; g.ldb = m.r; g.b_kmajor = false; g.C = b.dy_lo; g.ldc = m.r;
        g.M = m.T; g.N = m.r; g.K = m.d;
        BIGMAC_TRY(gemm(L, G_DY_LO, g, st));
    }
    if (G->dw_up && !m.cdac) {   // dW_up[c,c'] = sum_t dy[t,c] y'[t,c']   (this rank's tokens)
        GemmArgs g;
        g.A = dy; g.lda = m.d; g.a_kmajor = false; g.B = b.y_lo; g.ldb = m.r; g.b_kmajor = false;
        g.C = G->dw_up; g.ldc = m.r; g.M = m.d; g.N = m.r; g.K = m.T; g.accumulate = acc;
        if (fused) {
            g.split_k = choose_split_k(g.M, g.N, g.K); g.C = b.splitk_ws; g.out_f32 = true; g.accumulate = false;
            BIGMAC_TRY(gemm(L, G_DW_UP, g, st));
            Stage s(L, S_SPLITK_REDUCE, st);
            BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, m.d, m.r, G->dw_up, m.d, nullptr, 0, m.dtype, acc, st));
        } else {
            BIGMAC_TRY(gemm(L, G_DW_UP, g, st));
        }
    }
    const int vecs = m.r * (int)esize(m.dtype) / 16;
    {
        Stage s(L, S_COMBINE_BWD, st);
        if (m.dtype == BIGMAC_BF16)
            ep_combine_bwd_kernel<__nv_bfloat16><<<warp_blocks(m.N), 256, 0, st>>>((const uint4*)dy_lo, peers_of(ep->u, m.size),
                                                                                  peers_of(ep->du, m.size), b.dp, b.tb.topk_w,
                                                                                  b.tb.topk_idx, b.dest_row, m.N, m.k, m.El, vecs);
        else
            ep_combine_bwd_kernel<float><<<warp_blocks(m.N), 256, 0, st>>>((const uint4*)dy_lo, peers_of(ep->u, m.size),
                                                                          peers_of(ep->du, m.size), b.dp, b.tb.topk_w, b.tb.topk_idx,
                                                                          b.dest_row, m.N, m.k, m.El, vecs);
        BIGMAC_CUDA(cudaGetLastError());
    }
    { Stage s(L, S_GATE_BWD, st); BIGMAC_CUDA(launch_gate_bwd(b.dp, b.tb, b.dlogits, m.T, m.E, m.E64, m.ldcat, m.k, m.dtype, st)); }
    return BIGMAC_OK;
}

int bigmac_ep_backward_experts(bigmac_layer_t* L, const bigmac_weights_t* W, const bigmac_ep_t* ep, const bigmac_grads_t* G,
                               int accumulate, void* saved, void* scratch, size_t scratch_bytes, void* stream) {
    EpDims m;
    EpBuffers b{};
    BIGMAC_TRY(ep_enter(L, 0, ep, saved, scratch, scratch_bytes, true, &m, &b));
    BIGMAC_TRY(check_shared_weights(W, true));
    if (!G || !aligned(G->dw1, 16) || !aligned(G->dw2, 16)) return BIGMAC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const bool acc = accumulate != 0;
    void* du = ep->du[m.rank];
    {   // dz = (du W2_e) * sigma'(z)
        GemmArgs g;
        g.A = du; g.lda = m.r; g.B = W->w2; g.ldb = m.h; g.b_kmajor = false; g.b_stride = (int64_t)m.r * m.h;
        g.C = b.dz ? b.dz : b.z; g.Z = b.z; g.ldc = m.h; g.M = (int)m.Pep; g.N = m.h; g.K = m.r;
        g.epilogue = EPI_DACT; g.act = L->cfg.act; g.group = GROUP_M; g.num_experts = m.El;
        g.tile_expert = b.tile_expert_own; g.n_tiles = b.n_tiles_own; g.poffsets = b.poff_own;
        BIGMAC_TRY(gemm(L, G_DZ, g, st));
    }
    void* dz = b.dz ? b.dz : b.z;
    if (G->dw2) {
        GemmArgs g;
        g.A = du; g.lda = m.r; g.a_kmajor = false; g.B = b.a; g.ldb = m.h; g.b_kmajor = false;
        g.C = G->dw2; g.ldc = m.h; g.c_stride = (int64_t)m.r * m.h; g.M = m.r; g.N = m.h; g.K = (int)m.Pep;
        g.group = GROUP_K; g.num_experts = m.El; g.poffsets = b.poff_own; g.accumulate = acc;
        BIGMAC_TRY(expert_weight_grad(L, G_DW2, g, b.splitk_ws, st));
    }
    {   // dxg = dz W1_e
        GemmArgs g;
        g.A = dz; g.lda = m.h; g.B = W->w1; g.ldb = m.r; g.b_kmajor = false; g.b_stride = (int64_t)m.h * m.r;
        g.C = ep->dxg[m.rank]; g.ldc = m.r; g.M = (int)m.Pep; g.N = m.r; g.K = m.h;
        g.group = GROUP_M; g.num_experts = m.El; g.tile_expert = b.tile_expert_own; g.n_tiles = b.n_tiles_own; g.poffsets = b.poff_own;
        BIGMAC_TRY(gemm(L, G_DXG, g, st));
    }
    if (G->dw1) {
        GemmArgs g;
        g.A = dz; g.lda = m.h; g.a_kmajor = false; g.B = ep->xg[m.rank]; g.ldb = m.r; g.b_kmajor = false;
        g.C = G->dw1; g.ldc = m.r; g.c_stride = (int64_t)m.h * m.r; g.M = m.h; g.N = m.r; g.K = (int)m.Pep;
        g.group = GROUP_K; g.num_experts = m.El; g.poffsets = b.poff_own; g.accumulate = acc;
        BIGMAC_TRY(expert_weight_grad(L, G_DW1, g, b.splitk_ws, st));
    }
    return BIGMAC_OK;
}

int bigmac_ep_backward_dispatch(bigmac_layer_t* L, const void* x, int32_t T, const bigmac_weights_t* W, const bigmac_ep_t* ep,
                                void* dx, const bigmac_grads_t* G, int accumulate, void* saved, void* scratch,
                                size_t scratch_bytes, void* stream) {
    EpDims m;
    EpBuffers b{};
    BIGMAC_TRY(ep_enter(L, T, ep, saved, scratch, scratch_bytes, true, &m, &b));
    BIGMAC_TRY(check_shared_weights(W, false, m.cdac));
    if (!G) return BIGMAC_ERR_INVALID_ARG;
    if (T == 0) return BIGMAC_OK;
    if (!x || !dx || !aligned(x, 16) || !aligned(dx, 16) || !aligned(G->dw_gate, 16) || !aligned(G->dw_down, 16) ||
        !aligned(G->db_gate, 4))
        return BIGMAC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const bool acc = accumulate != 0;
    const bool fused = m.dtype == BIGMAC_BF16 && L->use_tc && L->tc_mask == ~0u;
    const int vecs = m.r * (int)esize(m.dtype) / 16, dvecs = m.ldcat * (int)esize(m.dtype) / 16;
    uint4* gather_to = (uint4*)(m.cdac ? dx : b.dx_lo);          // Eq. 3: the gathered rows are dx (before the gate's share)
    const int gather_ld = m.cdac ? vecs : dvecs;
    {   // dx'[t] = sum_j dxg[row of slot (t,j) at its owner]
        Stage s(L, S_DXLO_GATHER, st);
        if (m.dtype == BIGMAC_BF16)
            ep_get_combine_kernel<__nv_bfloat16><<<warp_blocks(T), 256, 0, st>>>(peers_of(ep->dxg, m.size), gather_to, nullptr,
                                                                                b.tb.topk_idx, b.dest_row, T, m.k, m.El, vecs, gather_ld);
        else
            ep_get_combine_kernel<float><<<warp_blocks(T), 256, 0, st>>>(peers_of(ep->dxg, m.size), gather_to, nullptr,
                                                                        b.tb.topk_idx, b.dest_row, T, m.k, m.El, vecs, gather_ld);
        BIGMAC_CUDA(cudaGetLastError());
    }
    if (m.cdac) {
        {   // dx += dl W_gate
            GemmArgs g;
            g.A = b.dlogits; g.lda = m.ldcat; g.B = W->w_gate; g.ldb = m.d; g.b_kmajor = false; g.C = dx; g.ldc = m.d;
            g.M = m.T; g.N = m.d; g.K = m.E; g.accumulate = true;
            BIGMAC_TRY(gemm(L, G_DX_GATE, g, st));
        }
        if (G->dw_gate) {   // dW_gate = dl^T x
            GemmArgs g;
            g.A = b.dlogits; g.lda = m.ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.M = m.E; g.N = m.d; g.K = m.T;
            if (fused) {
                g.C = b.splitk_ws; g.ldc = m.d; g.out_f32 = true; g.M = m.ldcat; g.split_k = choose_split_k(g.M, g.N, g.K);
                BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
                Stage s(L, S_SPLITK_REDUCE, st);
                BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, m.ldcat, m.d, G->dw_gate, m.E, nullptr, 0, m.dtype, acc, st));
            } else {
                g.C = G->dw_gate; g.ldc = m.d; g.accumulate = acc;
                BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
            }
        }
        if (G->db_gate) { Stage s(L, S_COLSUM, st, 2); BIGMAC_CUDA(launch_gate_colsum(b.dp, b.tb, G->db_gate, b.colsum_part, m.N, m.E, acc, st)); }
        return BIGMAC_OK;
    }
    if (fused) {
        {   // dx = [dx' | dl] [W_down ; W_gate]
            GemmArgs g;
            g.A = b.dcat; g.lda = m.ldcat; g.B = W->w_down; g.ldb = m.d; g.b_kmajor = false;
            g.B2 = W->w_gate; g.ldb2 = m.d; g.b2_first_k = m.r;
            g.C = dx; g.ldc = m.d; g.M = m.T; g.N = m.d; g.K = m.r + m.E;
            BIGMAC_TRY(gemm(L, G_DX, g, st));
        }
        if (G->dw_down || G->dw_gate) {
            GemmArgs g;
            g.A = b.dcat; g.lda = m.ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.C = b.splitk_ws; g.ldc = m.d; g.out_f32 = true; g.M = m.ldcat; g.N = m.d; g.K = m.T;
            g.split_k = choose_split_k(g.M, g.N, g.K);
            BIGMAC_TRY(gemm(L, G_DW_DOWN, g, st));
            Stage s(L, S_SPLITK_REDUCE, st);
            BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, m.ldcat, m.d, G->dw_down, m.r, G->dw_gate, m.E, m.dtype, acc, st));
        }
    } else {
        {
            GemmArgs g;
            g.A = b.dx_lo; g.lda = m.ldcat; g.B = W->w_down; g.ldb = m.d; g.b_kmajor = false; g.C = dx; g.ldc = m.d;
            g.M = m.T; g.N = m.d; g.K = m.r;
            BIGMAC_TRY(gemm(L, G_DX, g, st));
        }
        {
            GemmArgs g;
            g.A = b.dlogits; g.lda = m.ldcat; g.B = W->w_gate; g.ldb = m.d; g.b_kmajor = false; g.C = dx; g.ldc = m.d;
            g.M = m.T; g.N = m.d; g.K = m.E; g.accumulate = true;
            BIGMAC_TRY(gemm(L, G_DX_GATE, g, st));
        }
        if (G->dw_down) {
            GemmArgs g;
            g.A = b.dx_lo; g.lda = m.ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.C = G->dw_down; g.ldc = m.d; g.M = m.r; g.N = m.d; g.K = m.T; g.accumulate = acc;
            BIGMAC_TRY(gemm(L, G_DW_DOWN, g, st));
        }
        if (G->dw_gate) {
            GemmArgs g;
            g.A = b.dlogits; g.lda = m.ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.C = G->dw_gate; g.ldc = m.d; g.M = m.E; g.N = m.d; g.K = m.T; g.accumulate = acc;
            BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
        }
    }
    if (G->db_gate) { Stage s(L, S_COLSUM, st, 2); BIGMAC_CUDA(launch_gate_colsum(b.dp, b.tb, G->db_gate, b.colsum_part, m.N, m.E, acc, st)); }
    return BIGMAC_OK;
}

}  // extern "C"
