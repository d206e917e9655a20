// C-ABI entry points of libbigmac: argument checks, workspace carving and the launch sequence of the
// BigMac DCCA MoE layer (Eq. 2 / Eq. 4), forward and backward.  No device allocation, no stream
// synchronisation and no host-visible data dependence inside route / forward / backward: segment sizes
// stay on the device.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "layer_common.h"
#include "switches.h"

namespace bigmac {
Switches& switches() {
    static Switches s;
    return s;
}
}  // namespace bigmac

using namespace bigmac;
using namespace bigmac::detail;

namespace bigmac {
namespace detail {

struct Buffers {
    Tables tb;
    float* logits;
    void *x_lo, *xg, *z, *a, *u, *y_lo;                 // forward intermediates
    void *dy_lo, *du, *dxg; float* dp;                   // backward intermediates
    void* dz;            // [P,h]: its own buffer when sigma' is saved as bytes, else written over sigma'
    void* dcat;          // [T, r + E64]: dx' in columns [0, r), the dense gate gradient dl in columns [r, r + E64)
    void *dx_lo, *dlogits;                               // views into dcat (row stride r + E64)
    float* colsum_part;  // [kColsumChunks + kAuxChunks, E]: partial column sums of the top-k part, then of the load-balancing part
    float* aux_part;     // [kAuxChunks, E] forward scratch of the load-balancing loss
    float* aux_loss;     // [1] saved: L_aux of the batch
    float* logits_saved; // [T,E] saved copy of the gate logits (only with a load-balancing loss)
    float* splitk_ws;    // fp32 partial results of the split weight-gradient contractions
    float* descend_ws;   // few tokens: fp32 partial results [parts][T][r + E] of the split descend + logits launch
    float* bias_ws;      // fp32 row-slice sums of the expert-bias gradients (a region of their own: they run on the second stream)
};

struct Dims {
    int T, d, r, h, E, k, dtype;
    int64_t N, P;
    int E64;   // leading dimension of the dense [T,E] gate-gradient matrix (E rounded up to 64)
    int z_es;  // bytes per saved sigma'(z) element: 1 on the tensor-core path (quantised), else the dtype's
    bool cdac; // Eq. 3 layer: no descend / ascend projections, r == d
    int ldcat; // row stride of dcat: r + E64, or E64 alone without projections (dx' then goes straight to dx)
    bool gate_low; // the gate reads x' (w_gate [E,r])
    bool bias;     // experts have biases b1 [E,h], b2 [E,r]
    int cap;   // rows an expert keeps at most (Table 5's capacity factor); kNoCapacity = dropless
    float aux; // coefficient of the load-balancing loss (Table 5), 0 = none
};


Dims dims_of(const bigmac_layer* L, int T) {
    const bigmac_config_t& c = L->cfg;
    Dims m{T, c.d, c.r, c.h, c.E, c.k, c.dtype, (int64_t)T * c.k, 0};
    m.P = padded_rows_max(m.N, c.E);
    m.E64 = (c.E + 63) / 64 * 64;
    m.z_es = sigma_as_bytes(L) ? 1 : (int)esize(c.dtype);
    m.cdac = (c.flags & BIGMAC_FLAG_CDAC) != 0;
    m.ldcat = m.cdac ? m.E64 : m.r + m.E64;
    m.gate_low = (c.flags & BIGMAC_FLAG_GATE_LOW) != 0;
    m.bias = (c.flags & BIGMAC_FLAG_EXPERT_BIAS) != 0;
    m.cap = kNoCapacity;
    if (c.capacity_factor > 0) {                     // C = ceil((f * (T k)) / E), evaluated in double in this order
        const double rows = std::ceil(c.capacity_factor * (double)m.N / (double)c.E);
        if (rows < (double)m.N) m.cap = (int)rows;
    }
    m.aux = (float)c.aux_loss_coef;
    return m;
}

// What a training forward hands to its backward.
void carve_saved(Carver& cv, const Dims& m, Buffers& b, bool with_z) {
    const size_t es = esize(m.dtype);
    b.tb.topk_idx = cv.take<int32_t>(m.N);
    b.tb.topk_w = cv.take<float>(m.N);
    b.tb.counts = cv.take<int32_t>(m.E);
    b.tb.offsets = cv.take<int32_t>(m.E + 1);
    b.tb.poffsets = cv.take<int32_t>(m.E + 1);
    b.tb.row_of_slot = cv.take<int32_t>(m.N);
    b.tb.slot_of_row = cv.take<int32_t>(m.N);
    b.tb.prow_of_slot = cv.take<int32_t>(m.N);
    b.tb.slot_of_prow = cv.take<int32_t>(m.P);
    b.tb.tile_expert = cv.take<int32_t>(m.P / kPad);
    b.tb.n_tiles = cv.take<int32_t>(1);
    b.x_lo = m.cdac ? nullptr : cv.take_bytes((size_t)m.T * m.r * es);     // without projections x' is x itself
    b.xg = cv.take_bytes((size_t)m.P * m.r * es);
    b.z = with_z ? cv.take_bytes((size_t)m.P * m.h * m.z_es) : nullptr;
    b.a = cv.take_bytes((size_t)m.P * m.h * es);
    b.u = cv.take_bytes((size_t)m.P * m.r * es);
    b.y_lo = m.cdac ? nullptr : cv.take_bytes((size_t)m.T * m.r * es);     // ... and y' is y
    b.tb.counts_chosen = cv.take<int32_t>(m.E);
    b.aux_loss = cv.take<float>(1);
    b.logits_saved = (with_z && m.aux > 0) ? cv.take<float>((size_t)m.T * m.E) : nullptr;
}

void carve_route_scratch(Carver& cv, const Dims& m, Buffers& b) {
    b.logits = cv.take<float>((size_t)m.T * m.E);
    b.tb.block_counts = cv.take<int32_t>((size_t)(sort_blocks(m.N) + 1) * m.E);
    b.aux_part = m.aux > 0 ? cv.take<float>((size_t)kAuxChunks * m.E) : nullptr;
}

void carve_backward_scratch(Carver& cv, const Dims& m, Buffers& b) {
    const size_t es = esize(m.dtype);
    b.dy_lo = m.cdac ? nullptr : cv.take_bytes((size_t)m.T * m.r * es);
    b.du = cv.take_bytes((size_t)m.P * m.r * es);
    b.dxg = cv.take_bytes((size_t)m.P * m.r * es);
    b.dz = m.z_es == 1 ? cv.take_bytes((size_t)m.P * m.h * es) : nullptr;
    b.dcat = cv.take_bytes((size_t)m.T * m.ldcat * es);
    b.dx_lo = m.cdac ? nullptr : b.dcat;
    b.dlogits = (b.dcat && !m.cdac) ? (char*)b.dcat + (size_t)m.r * es : b.dcat;
    b.dp = cv.take<float>(m.N);
    b.colsum_part = cv.take<float>((size_t)(kColsumChunks + kAuxChunks) * m.E);
    // fp32 partial results: of the split dense contractions, and of the parts of long experts in dW1 / dW2
    const size_t dense_ws = (size_t)kMaxSplitK * m.ldcat * m.d * sizeof(float);
    const size_t expert_ws = m.dtype == BIGMAC_BF16 ? gemm_tc_groupk_ws_bytes(m.r, m.h, m.E) : 0;
    const size_t bias_ws = m.bias ? (size_t)m.E * kColsumSlices * (m.h > m.r ? m.h : m.r) * sizeof(float) : 0;
    b.splitk_ws = (float*)cv.take_bytes(dense_ws > expert_ws ? dense_ws : expert_ws);
    b.bias_ws = bias_ws ? (float*)cv.take_bytes(bias_ws) : nullptr;
}

// Few tokens: the descend + gate-logits launch has a handful of output tiles, each walking all of d; its contraction
// is then cut into parts (fp32 partial results, added by a small kernel) so that the SMs share the weight streaming.
// A function of the shape only: every call of a handle with the same T takes the same path.
int descend_split_parts(const Dims& m) {
    if (m.T > 1024 || m.E % 4 || m.dtype != BIGMAC_BF16) return 1;
    return choose_split_k(m.T, m.r + m.E, m.d);
}
void carve_descend_split(Carver& cv, const Dims& m, Buffers& b) {
    const int parts = descend_split_parts(m);
    b.descend_ws = parts > 1 ? cv.take<float>((size_t)parts * m.T * (m.r + m.E)) : nullptr;
}

size_t forward_scratch_bytes(const Dims& m, bool training) {
    Carver cv(nullptr);
    Buffers b{};
    carve_route_scratch(cv, m, b);
    carve_descend_split(cv, m, b);
    if (!training) carve_saved(cv, m, b, false);
    return cv.total();
}
size_t backward_scratch_bytes(const Dims& m) {
    Carver cv(nullptr);
    Buffers b{};
    carve_backward_scratch(cv, m, b);
    return cv.total();
}
size_t saved_bytes_of(const Dims& m) {
    Carver cv(nullptr);
    Buffers b{};
    carve_saved(cv, m, b, true);
    return cv.total();
}


int check_weights(const bigmac_layer* L, const bigmac_weights_t* W) {
    if (!W || !W->w_gate || !W->w1 || !W->w2) return BIGMAC_ERR_INVALID_ARG;
    if (!aligned(W->w_gate, 16) || !aligned(W->w1, 16) || !aligned(W->w2, 16) || !aligned(W->b_gate, 4))
        return BIGMAC_ERR_INVALID_ARG;
    if (L && (L->cfg.flags & BIGMAC_FLAG_EXPERT_BIAS) && (!W->b1 || !W->b2 || !aligned(W->b1, 16) || !aligned(W->b2, 16)))
        return BIGMAC_ERR_INVALID_ARG;
    if (L && (L->cfg.flags & BIGMAC_FLAG_CDAC)) return BIGMAC_OK;             // no shared projections
    if (!W->w_down || !W->w_up || !aligned(W->w_down, 16) || !aligned(W->w_up, 16)) return BIGMAC_ERR_INVALID_ARG;
    return BIGMAC_OK;
}

int gemm(const bigmac_layer* L, int id, const GemmArgs& g, cudaStream_t st) {
    Stage stage(L, id, st);
    cudaError_t err;
    const bool sigma_pair = id == G_EXPERT1 || id == G_DZ;      // these two must agree on the sigma' format
    if (L->cfg.dtype == BIGMAC_BF16 && L->use_tc && ((L->tc_mask >> id) & 1u) && (!sigma_pair || L->tc_mask == ~0u))
        err = gemm_tc(g, L->status, st);
    else
        err = gemm_simt(g, L->cfg.dtype, st);
    return err == cudaSuccess ? BIGMAC_OK : BIGMAC_ERR_CUDA;
}

// Number of parts to cut a dense contraction of `num_kb` k slices into so that tiles * parts fills the SMs:
// minimises waves * slices-per-part (ties: fewer parts).
int choose_split_k(int M, int N, int K) {
    // the weight-gradient contractions (both operands MN-major, N >= 256) run on CTA pairs: 256-row tiles, SMs/2 units
    const bool pairs = N >= 256;
    const int bn = N >= 256 ? 256 : 128, bm = pairs ? 256 : 128;
    const int64_t tiles = (int64_t)((M + bm - 1) / bm) * ((N + bn - 1) / bn);
    const int num_kb = (K + 63) / 64, units = pairs ? gemm_tc_sm_count() / 2 : gemm_tc_sm_count();
    int best = 1;
    int64_t best_cost = -1;
    for (int s = 1; s <= kMaxSplitK && s <= num_kb; ++s) {
        const int64_t cost = ((tiles * s + units - 1) / units) * ((num_kb + s - 1) / s);
        if (best_cost < 0 || cost < best_cost) { best = s; best_cost = cost; }
    }
    return best;
}

// Steps F2-F3 from the gate logits: top-k with softmax gate values, dispatch layout (under the capacity limit, if
// any), load-balancing loss.
int route_from_logits(const bigmac_layer* L, const Dims& m, const bigmac_weights_t* W, Buffers& b, cudaStream_t st) {
    { Stage s(L, S_TOPK, st); BIGMAC_CUDA(launch_topk(b.logits, W->b_gate, m.T, m.E, m.k, b.tb.topk_idx, b.tb.topk_w, st)); }
    { Stage s(L, S_TABLES, st, tables_kernel_count(m.N, m.E)); BIGMAC_CUDA(launch_tables(b.tb, m.T, m.E, m.k, m.cap, st, L->status)); }
    if (m.aux > 0) {
        Stage s(L, S_AUX_LOSS, st, 2);
        BIGMAC_CUDA(launch_aux_loss(b.logits, W->b_gate, b.tb.counts_chosen, m.T, m.E, m.k, m.aux, b.aux_part, b.aux_loss, st));
        if (b.logits_saved)
            BIGMAC_CUDA(cudaMemcpyAsync(b.logits_saved, b.logits, sizeof(float) * (size_t)m.T * m.E, cudaMemcpyDeviceToDevice, st));
    }
    return BIGMAC_OK;
}

// Steps F1-F3: gate logits on x, top-k with softmax gate values, dispatch layout.
int run_routing(const bigmac_layer* L, const Dims& m, const void* x, const bigmac_weights_t* W, Buffers& b,
                cudaStream_t st) {
    GemmArgs g;
    if (m.gate_low) {                                // the gate reads x': descend first, logits from its stored value
        GemmArgs q;
        q.A = x; q.lda = m.d; q.B = W->w_down; q.ldb = m.d; q.C = b.x_lo; q.ldc = m.r;
        q.M = m.T; q.N = m.r; q.K = m.d;
        BIGMAC_TRY(gemm(L, G_DESCEND, q, st));
        g.A = b.x_lo; g.lda = m.r; g.B = W->w_gate; g.ldb = m.r; g.K = m.r;
    } else {
        g.A = x; g.lda = m.d; g.B = W->w_gate; g.ldb = m.d; g.K = m.d;
    }
    g.C = b.logits; g.ldc = m.E; g.M = m.T; g.N = m.E; g.out_f32 = true;
    BIGMAC_TRY(gemm(L, G_LOGITS, g, st));
    return route_from_logits(L, m, W, b, st);
}

// Calls that keep no saved state (bigmac_route, the inference forward): the tables the caller asked for are produced
// in the caller's arrays themselves (same element types and layouts as the internal ones), so nothing is copied.
void alias_routing(Buffers& b, const bigmac_routing_t* out) {
    if (!out) return;
    if (out->topk_idx) b.tb.topk_idx = out->topk_idx;
    if (out->topk_w) b.tb.topk_w = out->topk_w;
    if (out->counts) b.tb.counts = out->counts;
    if (out->offsets) b.tb.offsets = out->offsets;
    if (out->row_of_slot) b.tb.row_of_slot = out->row_of_slot;
    if (out->slot_of_row) b.tb.slot_of_row = out->slot_of_row;
    if (out->counts_chosen) b.tb.counts_chosen = out->counts_chosen;
    if (out->aux_loss) b.aux_loss = out->aux_loss;
}

// Copies the tables into the caller's arrays (a training forward keeps its own copy in `saved` for the backward);
// members that alias_routing pointed at the caller's arrays are already in place.
int export_routing(const Dims& m, const Buffers& b, bigmac_routing_t* out, cudaStream_t st) {
    if (!out) return BIGMAC_OK;
    const cudaMemcpyKind kind = cudaMemcpyDeviceToDevice;
    if (out->topk_idx && out->topk_idx != b.tb.topk_idx)
        BIGMAC_CUDA(cudaMemcpyAsync(out->topk_idx, b.tb.topk_idx, sizeof(int32_t) * m.N, kind, st));
    if (out->topk_w && out->topk_w != b.tb.topk_w) BIGMAC_CUDA(cudaMemcpyAsync(out->topk_w, b.tb.topk_w, sizeof(float) * m.N, kind, st));
    if (out->counts && out->counts != b.tb.counts) BIGMAC_CUDA(cudaMemcpyAsync(out->counts, b.tb.counts, sizeof(int32_t) * m.E, kind, st));
    if (out->offsets && out->offsets != b.tb.offsets)
        BIGMAC_CUDA(cudaMemcpyAsync(out->offsets, b.tb.offsets, sizeof(int32_t) * (m.E + 1), kind, st));
    if (out->row_of_slot && out->row_of_slot != b.tb.row_of_slot)
        BIGMAC_CUDA(cudaMemcpyAsync(out->row_of_slot, b.tb.row_of_slot, sizeof(int32_t) * m.N, kind, st));
    if (out->slot_of_row && out->slot_of_row != b.tb.slot_of_row)
        BIGMAC_CUDA(cudaMemcpyAsync(out->slot_of_row, b.tb.slot_of_row, sizeof(int32_t) * m.N, kind, st));
    if (out->counts_chosen && out->counts_chosen != b.tb.counts_chosen)
        BIGMAC_CUDA(cudaMemcpyAsync(out->counts_chosen, b.tb.counts_chosen, sizeof(int32_t) * m.E, kind, st));
    if (out->aux_loss) {
        if (m.aux <= 0) BIGMAC_CUDA(cudaMemsetAsync(out->aux_loss, 0, sizeof(float), st));
        else if (out->aux_loss != b.aux_loss) BIGMAC_CUDA(cudaMemcpyAsync(out->aux_loss, b.aux_loss, sizeof(float), kind, st));
    }
    return BIGMAC_OK;
}

int check_call(const bigmac_layer* L, int32_t T) {
    if (!L) return BIGMAC_ERR_INVALID_ARG;
    if (T < 0 || T > L->cfg.max_tokens) return BIGMAC_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return BIGMAC_ERR_CUDA;
    if (dev != L->device) return BIGMAC_ERR_STATE;
    return BIGMAC_OK;
}

// Does the per-expert weight gradient run on the balanced kernel (dynamic work items, long experts in parts)?
bool uses_groupk(const bigmac_layer* L, int id, const GemmArgs& g) {
    const bool enabled = switches().groupk != 0;
    const bool tc = L->cfg.dtype == BIGMAC_BF16 && L->use_tc && ((L->tc_mask >> id) & 1u);
    // below about 16 k slices of work per CTA pair the items are too short for dynamic hand-out to pay (measured:
    // +10 us per launch at 1024 tokens of the medium shape, -31 % at 16384 tokens with Zipf loads)
    const int64_t tiles = (int64_t)((g.M + 255) / 256) * ((g.N + 255) / 256);
    const bool enough = (L->cfg.flags & BIGMAC_FLAG_DYNAMIC_WGRAD) ||
                        (int64_t)(g.K / 64) * tiles >= 16 * (int64_t)(gemm_tc_sm_count() / 2);
    return enabled && tc && enough && gemm_tc_groupk_supported(g);
}

// dW1_e[q,c'] = sum over the rows of expert e of dz[row,q] xg[row,c'] as a contraction request (xg: the grouped rows,
// or with gather_rows the ungrouped matrix they are copies of).
GemmArgs dw1_request(const Dims& m, const void* dz, const void* rows, const Tables& tb, void* dw1, bool acc) {
    GemmArgs g;
    g.A = dz; g.lda = m.h; g.a_kmajor = false; g.B = rows; g.ldb = m.r; g.b_kmajor = false;
    g.C = dw1; g.ldc = m.r; g.c_stride = (int64_t)m.h * m.r; g.M = m.h; g.N = m.r; g.K = (int)m.P;
    g.group = GROUP_K; g.num_experts = m.E; g.poffsets = tb.poffsets; g.accumulate = acc;
    return g;
}

// Is the dispatch fused into its consumers' operand loads (F5 of the forward disappears as a launch, the grouped
// copy xg of x' is never written)?  Inference: expert GEMM1 gathers the rows of x' itself.  Training: so does the
// weight gradient dW1, when it runs on the balanced kernel (the statically scheduled kernels read a grouped copy).
// A pure function of the handle, T and the debug switches: a training forward and its backward must see the same
// switches.
bool dispatch_is_fused(const bigmac_layer* L, const Dims& m, bool training) {
    if (!switches().fuse_dispatch || !sigma_as_bytes(L) || m.r % 64) return false;
    if (!training) {
        const bool short_list = m.P / kPad <= 2 * (int64_t)gemm_tc_sm_count();
        const bool mlp_fused = !m.bias && (switches().fused_mlp == 2 || (switches().fused_mlp == 1 && short_list)) &&
                               fused_mlp_supported(m.r, m.h, m.dtype);
        return !mlp_fused;
    }
    if (m.r % 128) return false;
    Tables shape_only{};                                     // the kernel choice depends on shapes and alignment only:
    void* const somewhere = (void*)(uintptr_t)256;           // stand-ins that are tested for presence and alignment, never read
    shape_only.poffsets = (int32_t*)somewhere;
    return uses_groupk(L, G_DW1, dw1_request(m, somewhere, somewhere, shape_only, somewhere, false));
}

// Per-expert weight gradient (contraction over the expert's rows): on the tensor-core path the balanced kernel
// (dynamic work items, long experts in parts), else the generic grouped contraction.
int expert_weight_grad(const bigmac_layer* L, int id, const GemmArgs& g, float* splitk_ws, cudaStream_t st) {
    if (uses_groupk(L, id, g)) {
        { Stage stage(L, id, st); BIGMAC_CUDA(gemm_tc_groupk(g, L->status, L->status + 2, splitk_ws, st)); }
        { Stage stage(L, S_SPLITK_REDUCE, st); BIGMAC_CUDA(gemm_tc_groupk_finish(g, splitk_ws, st)); }
        return BIGMAC_OK;
    }
    return gemm(L, id, g, st);
}

}  // namespace detail
}  // namespace bigmac

extern "C" {

int bigmac_layer_create(const bigmac_config_t* cfg, bigmac_layer_t** out) {
    if (!cfg || !out) return BIGMAC_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->d <= 0 || cfg->r <= 0 || cfg->h <= 0 || cfg->E <= 0 || cfg->k <= 0 || cfg->max_tokens < 0)
        return BIGMAC_ERR_INVALID_ARG;
    if (cfg->k > cfg->E) return BIGMAC_ERR_INVALID_ARG;
    if (cfg->dtype != BIGMAC_F32 && cfg->dtype != BIGMAC_BF16) return BIGMAC_ERR_INVALID_ARG;
    if (cfg->act < BIGMAC_ACT_RELU || cfg->act > BIGMAC_ACT_IDENTITY) return BIGMAC_ERR_INVALID_ARG;
    if (cfg->flags & ~(BIGMAC_FLAG_SIMT_GEMM | BIGMAC_FLAG_CDAC | BIGMAC_FLAG_DYNAMIC_WGRAD | BIGMAC_FLAG_GATE_LOW |
                       BIGMAC_FLAG_EXPERT_BIAS))
        return BIGMAC_ERR_INVALID_ARG;
    if ((cfg->flags & BIGMAC_FLAG_CDAC) && cfg->r != cfg->d) return BIGMAC_ERR_INVALID_ARG;
    if ((cfg->flags & BIGMAC_FLAG_CDAC) && (cfg->flags & BIGMAC_FLAG_GATE_LOW)) return BIGMAC_ERR_INVALID_ARG;
    if (!(cfg->capacity_factor >= 0) || !(cfg->aux_loss_coef >= 0) || std::isinf(cfg->capacity_factor) ||
        std::isinf(cfg->aux_loss_coef))
        return BIGMAC_ERR_INVALID_ARG;
    if ((cfg->flags & BIGMAC_FLAG_GATE_LOW) && cfg->aux_loss_coef > 0) return BIGMAC_ERR_UNSUPPORTED;
    if (cfg->E > kMaxExperts) return BIGMAC_ERR_UNSUPPORTED;
    if ((int64_t)cfg->max_tokens * cfg->k > (int64_t)1 << 30) return BIGMAC_ERR_UNSUPPORTED;
    const int vec = cfg->dtype == BIGMAC_BF16 ? 8 : 4;     // rows move as 16-byte vectors
    if (cfg->d % vec || cfg->r % vec || cfg->h % vec) return BIGMAC_ERR_UNSUPPORTED;
    if (cfg->dtype == BIGMAC_BF16 && (cfg->d % 64 || cfg->r % 64 || cfg->h % 64)) return BIGMAC_ERR_UNSUPPORTED;
    bigmac_layer* L = new (std::nothrow) bigmac_layer();
    if (!L) return BIGMAC_ERR_CUDA;
    L->cfg = *cfg;
    L->use_tc = cfg->dtype == BIGMAC_BF16 && !(cfg->flags & BIGMAC_FLAG_SIMT_GEMM);
    L->tc_mask = switches().tc_mask;
    if (cudaGetDevice(&L->device) != cudaSuccess || cudaMalloc((void**)&L->status, 4 * sizeof(int)) != cudaSuccess ||
        cudaMemset(L->status, 0, 4 * sizeof(int)) != cudaSuccess) {
        delete L;
        return BIGMAC_ERR_CUDA;
    }
    if (L->use_tc && !gemm_tc_available()) {
        cudaFree(L->status);
        delete L;
        return BIGMAC_ERR_UNSUPPORTED;
    }
    // the backward pass's second stream and its fork / join events; without them the pass runs on one stream
    bool side_ok = cudaStreamCreateWithFlags(&L->side, cudaStreamNonBlocking) == cudaSuccess;
    for (cudaEvent_t& e : L->fork_join)
        side_ok = side_ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
    if (!side_ok) {
        for (cudaEvent_t& e : L->fork_join)
            if (e) { cudaEventDestroy(e); e = nullptr; }
        if (L->side) { cudaStreamDestroy(L->side); L->side = nullptr; }
        cudaGetLastError();
    }
    *out = L;
    return BIGMAC_OK;
}

int bigmac_layer_destroy(bigmac_layer_t* L) {
    if (!L) return BIGMAC_ERR_INVALID_ARG;
    for (cudaEvent_t e : L->ev) cudaEventDestroy(e);
    for (cudaEvent_t e : L->fork_join)
        if (e) cudaEventDestroy(e);
    if (L->side) cudaStreamDestroy(L->side);
    cudaFree(L->status);
    delete L;
    return BIGMAC_OK;
}

int bigmac_workspace_bytes(const bigmac_layer_t* L, int32_t T, int training, size_t* scratch_bytes,
                           size_t* saved_bytes) {
    if (!L || !scratch_bytes || !saved_bytes || T < 0 || T > L->cfg.max_tokens) return BIGMAC_ERR_INVALID_ARG;
    const Dims m = dims_of(L, T);
    size_t s = forward_scratch_bytes(m, training != 0);
    if (training) {
        const size_t bw = backward_scratch_bytes(m);
        if (bw > s) s = bw;
    }
    *scratch_bytes = s;
    *saved_bytes = training ? saved_bytes_of(m) : 0;
    return BIGMAC_OK;
}

int bigmac_route(bigmac_layer_t* L, const void* x, int32_t T, const bigmac_weights_t* W, bigmac_routing_t* out,
                 void* scratch, size_t scratch_bytes, void* stream) {
    BIGMAC_TRY(check_call(L, T));
    if (!out) return BIGMAC_ERR_INVALID_ARG;
    BIGMAC_TRY(check_weights(L, W));
    if (T == 0) return BIGMAC_OK;
    if (!x || !aligned(x, 16) || !scratch || !aligned(scratch, 256)) return BIGMAC_ERR_INVALID_ARG;
    const Dims m = dims_of(L, T);
    if (scratch_bytes < forward_scratch_bytes(m, false)) return BIGMAC_ERR_WORKSPACE;
    Carver cv(scratch);
    Buffers b{};
    carve_route_scratch(cv, m, b);
    carve_saved(cv, m, b, false);
    alias_routing(b, out);
    cudaStream_t st = (cudaStream_t)stream;
    BIGMAC_TRY(run_routing(L, m, x, W, b, st));
    return export_routing(m, b, out, st);
}

int bigmac_forward(bigmac_layer_t* L, const void* x, int32_t T, const bigmac_weights_t* W, void* y,
                   bigmac_routing_t* routing_out, void* saved, void* scratch, size_t scratch_bytes, void* stream) {
    BIGMAC_TRY(check_call(L, T));
    BIGMAC_TRY(check_weights(L, W));
    if (T == 0) return BIGMAC_OK;
    if (!x || !y || !aligned(x, 16) || !aligned(y, 16) || !scratch || !aligned(scratch, 256) ||
        !aligned(saved, 256))
        return BIGMAC_ERR_INVALID_ARG;
    const bool training = saved != nullptr;
    const Dims m = dims_of(L, T);
    if (scratch_bytes < forward_scratch_bytes(m, training)) return BIGMAC_ERR_WORKSPACE;
    Buffers b{};
    Carver cs(scratch);
    carve_route_scratch(cs, m, b);
    carve_descend_split(cs, m, b);
    if (training) {
        Carver cv(saved);
        carve_saved(cv, m, b, true);
    } else {
        carve_saved(cs, m, b, false);
        alias_routing(b, routing_out);
    }
    cudaStream_t st = (cudaStream_t)stream;
    const bigmac_config_t& c = L->cfg;

    // A few tokens, inference: the whole forward in one cooperative kernel (weight streaming, no tensor cores)
    if (!training && !m.cdac && !m.gate_low && !m.bias && m.cap == kNoCapacity && m.aux == 0 && sigma_as_bytes(L) &&
        decode_forward_supported(m.T, m.d, m.r, m.h, m.E, m.k, m.dtype)) {
        {
            Stage s(L, S_DECODE, st);
            BIGMAC_CUDA(launch_decode_forward(x, W, y, b.logits, (float*)b.xg, (float*)b.a, (float*)b.u, b.tb.topk_idx,
                                              b.tb.topk_w, (unsigned*)(L->status + 1), L->status, m.T, m.d, m.r, m.h, m.E,
                                              m.k, c.act, gemm_tc_sm_count(), st));
        }
        if (routing_out) {
            { Stage s(L, S_TABLES, st, tables_kernel_count(m.N, m.E)); BIGMAC_CUDA(launch_tables(b.tb, m.T, m.E, m.k, m.cap, st, L->status)); }
            BIGMAC_TRY(export_routing(m, b, routing_out, st));
        }
        return BIGMAC_OK;
    }
    // F1 + F4 in one pass over x when the tile grid allows it: [x' | logits] = x [W'_down ; W_gate]^T, logits in fp32
    const int bn_desc = (m.r + m.E) >= 256 ? 256 : 128;
    const bool fuse_gate = !m.cdac && !m.gate_low && c.dtype == BIGMAC_BF16 && L->use_tc && L->tc_mask == ~0u && m.r % bn_desc == 0;
    if (fuse_gate) {
        GemmArgs g;
        g.A = x; g.lda = m.d; g.B = W->w_down; g.ldb = m.d; g.C = b.x_lo; g.ldc = m.r;
        g.B2 = W->w_gate; g.ldb2 = m.d; g.n_split = m.r; g.C2 = b.logits; g.ldc2 = m.E; g.N2 = m.E;
        g.M = m.T; g.N = m.r + m.E; g.K = m.d;
        if (b.descend_ws) {                                   // few tokens: contraction in parts, then [x' | logits] from them
            g.split_k = descend_split_parts(m); g.out_f32 = true;
            g.C = b.descend_ws; g.ldc = m.r + m.E; g.C2 = b.descend_ws + m.r; g.ldc2 = m.r + m.E;
            BIGMAC_TRY(gemm(L, G_DESCEND, g, st));
            Stage s(L, S_SPLITK_REDUCE, st);
            BIGMAC_CUDA(launch_descend_reduce(b.descend_ws, g.split_k, m.T, m.r, m.E, b.x_lo, b.logits, st));
        } else {
            BIGMAC_TRY(gemm(L, G_DESCEND, g, st));
        }
        BIGMAC_TRY(route_from_logits(L, m, W, b, st));
    } else {
        BIGMAC_TRY(run_routing(L, m, x, W, b, st));                               // F1-F3
    }
    BIGMAC_TRY(export_routing(m, b, routing_out, st));
    if (m.cdac) b.x_lo = const_cast<void*>(x);                                    // Eq. 3: experts read the token itself
    if (!fuse_gate && !m.cdac && !m.gate_low) {                                   // F4 descend: x' = x W'_down
        GemmArgs g;
        g.A = x; g.lda = m.d; g.B = W->w_down; g.ldb = m.d; g.C = b.x_lo; g.ldc = m.r;
        g.M = m.T; g.N = m.r; g.K = m.d;
        BIGMAC_TRY(gemm(L, G_DESCEND, g, st));
    }
    // F5 dispatch at width r - unless it is fused into its consumers: expert GEMM1's producer warp then gathers the
    // rows of x' itself (slot_of_prow names the token of every grouped row, -1 the zero padding rows) and the grouped
    // copy xg is never written.
    const bool short_list = m.P / kPad <= 2 * (int64_t)gemm_tc_sm_count();
    const bool mlp_fused_ = !training && !m.bias && (switches().fused_mlp == 2 || (switches().fused_mlp == 1 && short_list)) &&
                            sigma_as_bytes(L) && fused_mlp_supported(m.r, m.h, m.dtype);
    const bool gather_dispatch = dispatch_is_fused(L, m, training);
    if (!gather_dispatch) { Stage s(L, S_DISPATCH, st); BIGMAC_CUDA(launch_dispatch(b.x_lo, b.xg, b.tb, m.k, m.r, m.dtype, m.P, st)); }
    // Inference, low width r <= 256, up to two row tiles per SM: F6 + F7 in one kernel, the hidden activations stay on
    // the SM.  On long tile lists the two separate GEMMs are faster (the fused kernel is bound by the issue of its many
    // narrow MMA instructions): measured 0.375 vs 0.329 ms forward at the medium workload, 0.099 vs 0.106 ms at 512
    // decode tokens.  The fused_mlp debug switch forces it off (0) / on (2).
    if (mlp_fused_) {
        Stage s(L, S_FUSED_MLP, st);
        BIGMAC_CUDA(launch_fused_mlp(b.xg, W->w1, W->w2, b.u, m.P, m.r, m.h, m.E, c.act, b.tb.tile_expert, b.tb.n_tiles,
                                     L->status, st));
    } else {
        {                                                                             // F6 a = sigma(xg W1_e^T); saves sigma'(z)
            GemmArgs g;
            g.A = b.xg; g.lda = m.r; g.B = W->w1; g.ldb = m.r; g.b_stride = (int64_t)m.h * m.r;
            if (gather_dispatch) { g.A = b.x_lo; g.gather_rows = b.tb.slot_of_prow; g.gather_div = m.k; }
            g.C = b.a; g.Z = b.z; g.ldc = m.h; g.M = (int)m.P; g.N = m.h; g.K = m.r;
            g.epilogue = EPI_ACT; g.act = c.act; g.group = GROUP_M; g.num_experts = m.E;
            g.tile_expert = b.tb.tile_expert; g.n_tiles = b.tb.n_tiles; g.poffsets = b.tb.poffsets;
            if (m.bias) { g.bias = W->b1; g.bias_stride = m.h; }
            BIGMAC_TRY(gemm(L, G_EXPERT1, g, st));
        }
        {                                                                             // F7 u = a W2_e^T
            GemmArgs g;
            g.A = b.a; g.lda = m.h; g.B = W->w2; g.ldb = m.h; g.b_stride = (int64_t)m.r * m.h;
            g.C = b.u; g.ldc = m.r; g.M = (int)m.P; g.N = m.r; g.K = m.h;
            g.group = GROUP_M; g.num_experts = m.E; g.tile_expert = b.tb.tile_expert; g.n_tiles = b.tb.n_tiles; g.poffsets = b.tb.poffsets;
            if (m.bias) { g.bias = W->b2; g.bias_stride = m.r; }
            BIGMAC_TRY(gemm(L, G_EXPERT2, g, st));
        }
    }
    if (m.cdac) b.y_lo = y;                                                       // Eq. 3: the weighted sum is the output
    { Stage s(L, S_COMBINE, st); BIGMAC_CUDA(launch_combine(b.u, b.y_lo, b.tb.topk_w, b.tb.prow_of_slot, m.T, m.k, m.r, m.dtype, st, 0, m.cap != kNoCapacity)); }  // F8
    if (!m.cdac) {                                                                // F9 ascend: y = y' W'_up
        GemmArgs g;
        g.A = b.y_lo; g.lda = m.r; g.B = W->w_up; g.ldb = m.r; g.C = y; g.ldc = m.d;
        g.M = m.T; g.N = m.d; g.K = m.r;
        BIGMAC_TRY(gemm(L, G_ASCEND, g, st));
    }
    return BIGMAC_OK;
}

static int backward_launches(bigmac_layer_t* L, const void* x, const void* dy, int32_t T, const bigmac_weights_t* W,
                             void* saved, void* dx, const bigmac_grads_t* G, int accumulate, void* scratch,
                             size_t scratch_bytes, void* stream);

int bigmac_backward(bigmac_layer_t* L, const void* x, const void* dy, int32_t T, const bigmac_weights_t* W,
                    void* saved, void* dx, const bigmac_grads_t* G, int accumulate, void* scratch,
                    size_t scratch_bytes, void* stream) {
    if (L) L->side_forked = false;
    const int rc = backward_launches(L, x, dy, T, W, saved, dx, G, accumulate, scratch, scratch_bytes, stream);
    if (rc != BIGMAC_OK && L && L->side_forked) {
        // a launch failed after work was forked to the second stream: join it, so that the caller's stream (and a
        // capture in progress) is not left with an open fork and nothing of this call outlives its return unordered
        if (cudaEventRecord(L->fork_join[9], L->side) == cudaSuccess) cudaStreamWaitEvent((cudaStream_t)stream, L->fork_join[9], 0);
    }
    return rc;
}

static int backward_launches(bigmac_layer_t* L, const void* x, const void* dy, int32_t T, const bigmac_weights_t* W,
                             void* saved, void* dx, const bigmac_grads_t* G, int accumulate, void* scratch,
                             size_t scratch_bytes, void* stream) {
    BIGMAC_TRY(check_call(L, T));
    BIGMAC_TRY(check_weights(L, W));
    if (!G) return BIGMAC_ERR_INVALID_ARG;
    if (T == 0) return BIGMAC_OK;
    if (!x || !dy || !dx || !saved || !scratch || !aligned(x, 16) || !aligned(dy, 16) || !aligned(dx, 16) ||
        !aligned(saved, 256) || !aligned(scratch, 256))
        return BIGMAC_ERR_INVALID_ARG;
    if (!aligned(G->dw_gate, 16) || !aligned(G->dw_down, 16) || !aligned(G->dw1, 16) || !aligned(G->dw2, 16) ||
        !aligned(G->dw_up, 16) || !aligned(G->db_gate, 4))
        return BIGMAC_ERR_INVALID_ARG;
    if ((L->cfg.flags & BIGMAC_FLAG_EXPERT_BIAS) && (!aligned(G->db1, 4) || !aligned(G->db2, 4))) return BIGMAC_ERR_INVALID_ARG;
    const Dims m = dims_of(L, T);
    if (scratch_bytes < backward_scratch_bytes(m)) return BIGMAC_ERR_WORKSPACE;
    Buffers b{};
    {
        Carver cv(saved);
        carve_saved(cv, m, b, true);
        Carver cs(scratch);
        carve_backward_scratch(cs, m, b);
    }
    cudaStream_t st = (cudaStream_t)stream;
    const bigmac_config_t& c = L->cfg;
    const bool acc = accumulate != 0;

    // Overlap (the overlap debug switch turns it off): dW_up, the gate backward with the bias-gradient column sums, the dx' gather
    // and [dW_down ; dW_gate] go to a second stream, forked from and joined back into the caller's stream with events, so that they run beside launches they
    // do not depend on.  Everything that shares the fp32 workspace stays ordered.
    const bool overlap_on = switches().overlap != 0;
    // (not while per-stage events are recorded: a stage timed beside another stream's launches would not be its own time)
    const bool overlap = overlap_on && L->side && !L->prof_on && !m.cdac;
    cudaStream_t sd = st;
    if (overlap) {
        sd = L->side;
        BIGMAC_CUDA(cudaEventRecord(L->fork_join[0], st));
        BIGMAC_CUDA(cudaStreamWaitEvent(sd, L->fork_join[0], 0));
        L->side_forked = true;
    }
    if (m.cdac) b.dy_lo = const_cast<void*>(dy);
    if (!m.cdac) {   // dy' = dy W_up                                   [T,d] x [d,r]
        GemmArgs g;
        g.A = dy; g.lda = m.d; g.B = W->w_up; g.ldb = m.r; g.b_kmajor = false; g.C = b.dy_lo; g.ldc = m.r;
        g.M = m.T; g.N = m.r; g.K = m.d;
        BIGMAC_TRY(gemm(L, G_DY_LO, g, st));
    }
    const bool fused = L->cfg.dtype == BIGMAC_BF16 && L->use_tc && L->tc_mask == ~0u;
    const int ldcat = m.ldcat;
    if (G->dw_up && !m.cdac) {   // dW_up[c,c'] = sum_t dy[t,c] y'[t,c']
        GemmArgs g;
        g.A = dy; g.lda = m.d; g.a_kmajor = false; g.B = b.y_lo; g.ldb = m.r; g.b_kmajor = false;
        g.C = G->dw_up; g.ldc = m.r; g.M = m.d; g.N = m.r; g.K = m.T; g.accumulate = acc;
        if (fused) {   // contraction over all tokens, few output tiles: split it, reduce the parts in order
            g.split_k = choose_split_k(g.M, g.N, g.K); g.C = b.splitk_ws; g.out_f32 = true; g.accumulate = false;
            BIGMAC_TRY(gemm(L, G_DW_UP, g, sd));
            Stage s(L, S_SPLITK_REDUCE, sd);
            BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, m.d, m.r, G->dw_up, m.d, nullptr, 0, m.dtype, acc, sd));
        } else {
            BIGMAC_TRY(gemm(L, G_DW_UP, g, sd));
        }
    }
    if (overlap) BIGMAC_CUDA(cudaEventRecord(L->fork_join[1], sd));          // dW_up done: the fp32 workspace is free again
    // du = p dy'[t], dp = <dy'[t], u>; then the softmax-over-k backward
    if (m.cap != kNoCapacity) BIGMAC_CUDA(cudaMemsetAsync(b.dp, 0, sizeof(float) * m.N, st));   // dropped slots: dp = 0
    { Stage s(L, S_COMBINE_BWD, st); BIGMAC_CUDA(launch_combine_bwd(b.dy_lo, b.u, b.du, b.dp, b.tb, m.k, m.r, m.dtype, m.P, st)); }
    // The gate backward (dp -> dl) and the gate-bias column sums feed only dx, dW_gate and db_gate at the end of the pass:
    // with the second stream they run beside the expert contractions instead of in front of them.
    if (overlap) {
        BIGMAC_CUDA(cudaEventRecord(L->fork_join[2], st));
        BIGMAC_CUDA(cudaStreamWaitEvent(sd, L->fork_join[2], 0));
    }
    float* aux_part = nullptr;                                                    // column sums of dL_aux/dl, for db_gate
    if (m.aux > 0) {
        aux_part = b.colsum_part + (size_t)kColsumChunks * m.E;
        Stage s(L, S_GATE_BWD, sd);
        BIGMAC_CUDA(launch_gate_bwd_aux(b.dp, b.tb, b.dlogits, b.logits_saved, W->b_gate, m.aux, aux_part, m.T, m.E, m.E64,
                                        ldcat, m.k, m.dtype, sd));
    } else {
        Stage s(L, S_GATE_BWD, sd);
        BIGMAC_CUDA(launch_gate_bwd(b.dp, b.tb, b.dlogits, m.T, m.E, m.E64, ldcat, m.k, m.dtype, sd));
    }
    bool colsum_done = false;
    if (overlap) {
        if (G->db_gate) {
            Stage s(L, S_COLSUM, sd, 2);
            BIGMAC_CUDA(launch_gate_colsum(b.dp, b.tb, G->db_gate, b.colsum_part, m.N, m.E, acc, sd, aux_part));
        }
        BIGMAC_CUDA(cudaEventRecord(L->fork_join[3], sd));
        colsum_done = true;
    }
    {   // dz = (du W2_e) * sigma'(z); the forward saved sigma'(z) in the z buffer, dz is written over it
        GemmArgs g;
        g.A = b.du; g.lda = m.r; g.B = W->w2; g.ldb = m.h; g.b_kmajor = false; g.b_stride = (int64_t)m.r * m.h;
        g.C = b.dz ? b.dz : b.z; g.Z = b.z; g.ldc = m.h; g.M = (int)m.P; g.N = m.h; g.K = m.r;
        g.epilogue = EPI_DACT; g.act = c.act; g.group = GROUP_M; g.num_experts = m.E;
        g.tile_expert = b.tb.tile_expert; g.n_tiles = b.tb.n_tiles; g.poffsets = b.tb.poffsets;
        BIGMAC_TRY(gemm(L, G_DZ, g, st));
    }
    void* dz = b.dz ? b.dz : b.z;
    if (overlap) BIGMAC_CUDA(cudaStreamWaitEvent(st, L->fork_join[1], 0));    // from here on the fp32 workspace is used again
    if (m.bias) {   // db1_e = sum_rows dz[row,:], db2_e = sum_rows du[row,:]  (padding rows hold zeros)
        // Two HBM-bound passes over dz and du that nothing later in the pass reads: with the second stream they run
        // beside the tensor-bound dW2 / dxg (joined with the dx' gather), on slice sums in a region of their own.
        cudaStream_t sb = st;
        if (overlap) {
            BIGMAC_CUDA(cudaEventRecord(L->fork_join[8], st));
            BIGMAC_CUDA(cudaStreamWaitEvent(sd, L->fork_join[8], 0));
            sb = sd;
        }
        Stage s(L, S_COLSUM, sb, 2 * ((G->db1 ? 1 : 0) + (G->db2 ? 1 : 0)));
        if (G->db1) BIGMAC_CUDA(launch_grouped_colsum(dz, b.tb.poffsets, G->db1, b.bias_ws, m.E, m.h, m.dtype, acc, sb));
        if (G->db2) BIGMAC_CUDA(launch_grouped_colsum(b.du, b.tb.poffsets, G->db2, b.bias_ws, m.E, m.r, m.dtype, acc, sb));
    }
    if (G->dw2) {   // dW2_e[c',q] = sum_rows du[row,c'] a[row,q]
        GemmArgs g;
        g.A = b.du; g.lda = m.r; g.a_kmajor = false; g.B = b.a; g.ldb = m.h; g.b_kmajor = false;
        g.C = G->dw2; g.ldc = m.h; g.c_stride = (int64_t)m.r * m.h; g.M = m.r; g.N = m.h; g.K = (int)m.P;
        g.group = GROUP_K; g.num_experts = m.E; g.poffsets = b.tb.poffsets; g.accumulate = acc;
        BIGMAC_TRY(expert_weight_grad(L, G_DW2, g, b.splitk_ws, st));
    }
    {   // dxg = dz W1_e
        GemmArgs g;
        g.A = dz; g.lda = m.h; g.B = W->w1; g.ldb = m.r; g.b_kmajor = false; g.b_stride = (int64_t)m.h * m.r;
        g.C = b.dxg; g.ldc = m.r; g.M = (int)m.P; g.N = m.r; g.K = m.h;
        g.group = GROUP_M; g.num_experts = m.E; g.tile_expert = b.tb.tile_expert; g.n_tiles = b.tb.n_tiles; g.poffsets = b.tb.poffsets;
        BIGMAC_TRY(gemm(L, G_DXG, g, st));
    }
    if (overlap) {   // dx'[t] = sum_j dxg[row of slot (t,j)]: an HBM-bound gather beside the tensor-bound dW1
        BIGMAC_CUDA(cudaEventRecord(L->fork_join[4], st));
        BIGMAC_CUDA(cudaStreamWaitEvent(sd, L->fork_join[4], 0));
        { Stage s(L, S_DXLO_GATHER, sd); BIGMAC_CUDA(launch_combine(b.dxg, b.dx_lo, nullptr, b.tb.prow_of_slot, m.T, m.k, m.r, m.dtype, sd, ldcat, m.cap != kNoCapacity)); }
        BIGMAC_CUDA(cudaEventRecord(L->fork_join[5], sd));
    }
    if (G->dw1) {   // dW1_e[q,c'] = sum_rows dz[row,q] xg[row,c']
        GemmArgs g = dw1_request(m, dz, b.xg, b.tb, G->dw1, acc);
        if (dispatch_is_fused(L, m, true)) {     // no grouped copy exists: the contraction gathers the rows of x' (Eq. 3: of x)
            g.B = m.cdac ? x : b.x_lo;
            g.gather_rows = b.tb.slot_of_prow;
            g.gather_div = m.k;
        }
        BIGMAC_TRY(expert_weight_grad(L, G_DW1, g, b.splitk_ws, st));
    }
    if (m.cdac) {
        // Eq. 3: dx = sum_j dxg[row of slot (t,j)] + dl W_gate; dW_gate = dl^T x
        { Stage s(L, S_DXLO_GATHER, st); BIGMAC_CUDA(launch_combine(b.dxg, dx, nullptr, b.tb.prow_of_slot, m.T, m.k, m.d, m.dtype, st, 0, m.cap != kNoCapacity)); }
        {
            GemmArgs g;
            g.A = b.dlogits; g.lda = ldcat; g.B = W->w_gate; g.ldb = m.d; g.b_kmajor = false; g.C = dx; g.ldc = m.d;
            g.M = m.T; g.N = m.d; g.K = m.E; g.accumulate = true;
            BIGMAC_TRY(gemm(L, G_DX_GATE, g, st));
        }
        if (G->dw_gate) {
            GemmArgs g;
            g.A = b.dlogits; g.lda = ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.M = m.E; g.N = m.d; g.K = m.T;
            if (fused) {
                g.C = b.splitk_ws; g.ldc = m.d; g.out_f32 = true; g.M = ldcat; g.split_k = choose_split_k(g.M, g.N, g.K);
                BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
                Stage s(L, S_SPLITK_REDUCE, st);
                BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, ldcat, m.d, G->dw_gate, m.E, nullptr, 0, m.dtype, acc, st));
            } else {
                g.C = G->dw_gate; g.ldc = m.d; g.accumulate = acc;
                BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
            }
        }
        if (G->db_gate) { Stage s(L, S_COLSUM, st, 2); BIGMAC_CUDA(launch_gate_colsum(b.dp, b.tb, G->db_gate, b.colsum_part, m.N, m.E, acc, st, aux_part)); }
        return BIGMAC_OK;
    }
    // dx'[t] = sum_j dxg[row of slot (t,j)]   (the transpose of the dispatch gather)
    if (overlap) {
        BIGMAC_CUDA(cudaStreamWaitEvent(st, L->fork_join[5], 0));             // join: the gather ...
        BIGMAC_CUDA(cudaStreamWaitEvent(st, L->fork_join[3], 0));             // ... and the gate backward with its column sums
    } else {
        Stage s(L, S_DXLO_GATHER, st);
        BIGMAC_CUDA(launch_combine(b.dxg, b.dx_lo, nullptr, b.tb.prow_of_slot, m.T, m.k, m.r, m.dtype, st, ldcat, m.cap != kNoCapacity));
    }
    if (m.gate_low) {
        // The gate read x': its gradient joins dx' (dx' += dl W_gate, W_gate [E,r]) before the descend projection;
        // dW_gate = dl^T x'.
        {
            GemmArgs g;
            g.A = b.dlogits; g.lda = ldcat; g.B = W->w_gate; g.ldb = m.r; g.b_kmajor = false; g.C = b.dx_lo; g.ldc = ldcat;
            g.M = m.T; g.N = m.r; g.K = m.E; g.accumulate = true;
            BIGMAC_TRY(gemm(L, G_DX_GATE, g, st));
        }
        {   // dx = dx' W_down
            GemmArgs g;
            g.A = b.dx_lo; g.lda = ldcat; g.B = W->w_down; g.ldb = m.d; g.b_kmajor = false; g.C = dx; g.ldc = m.d;
            g.M = m.T; g.N = m.d; g.K = m.r;
            BIGMAC_TRY(gemm(L, G_DX, g, st));
        }
        if (G->dw_down) {   // dW_down[c',c] = sum_t dx'[t,c'] x[t,c]
            GemmArgs g;
            g.A = b.dx_lo; g.lda = ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.M = m.r; g.N = m.d; g.K = m.T;
            if (fused) {
                g.C = b.splitk_ws; g.ldc = m.d; g.out_f32 = true; g.split_k = choose_split_k(g.M, g.N, g.K);
                BIGMAC_TRY(gemm(L, G_DW_DOWN, g, st));
                Stage s(L, S_SPLITK_REDUCE, st);
                BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, m.r, m.d, G->dw_down, m.r, nullptr, 0, m.dtype, acc, st));
            } else {
                g.C = G->dw_down; g.ldc = m.d; g.accumulate = acc;
                BIGMAC_TRY(gemm(L, G_DW_DOWN, g, st));
            }
        }
        if (G->dw_gate) {   // dW_gate[e,c'] = sum_t dl[t,e] x'[t,c']
            GemmArgs g;
            g.A = b.dlogits; g.lda = ldcat; g.a_kmajor = false; g.B = b.x_lo; g.ldb = m.r; g.b_kmajor = false;
            g.N = m.r; g.K = m.T;
            if (fused) {
                g.M = m.E64; g.C = b.splitk_ws; g.ldc = m.r; g.out_f32 = true; g.split_k = choose_split_k(g.M, g.N, g.K);
                BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
                Stage s(L, S_SPLITK_REDUCE, st);
                BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, m.E64, m.r, G->dw_gate, m.E, nullptr, 0, m.dtype, acc, st));
            } else {
                g.M = m.E; g.C = G->dw_gate; g.ldc = m.r; g.accumulate = acc;
                BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
            }
        }
        if (!colsum_done && G->db_gate) { Stage s(L, S_COLSUM, st, 2); BIGMAC_CUDA(launch_gate_colsum(b.dp, b.tb, G->db_gate, b.colsum_part, m.N, m.E, acc, st, aux_part)); }
        return BIGMAC_OK;
    }
    if (fused) {
        // dx and [dW_down ; dW_gate] share only their input [dx' | dl]: with the second stream the weight gradient's CTAs
        // move in as those of dx leave.  The caller's stream has finished dW1 here, so the fp32 workspace is free.
        cudaStream_t sw = st;
        if (overlap && (G->dw_down || G->dw_gate)) {
            BIGMAC_CUDA(cudaEventRecord(L->fork_join[6], st));
            BIGMAC_CUDA(cudaStreamWaitEvent(sd, L->fork_join[6], 0));
            sw = sd;
        }
        {   // dx = [dx' | dl] [W_down ; W_gate]: one contraction over r + E
            GemmArgs g;
            g.A = b.dcat; g.lda = ldcat; g.B = W->w_down; g.ldb = m.d; g.b_kmajor = false;
            g.B2 = W->w_gate; g.ldb2 = m.d; g.b2_first_k = m.r;
            g.C = dx; g.ldc = m.d; g.M = m.T; g.N = m.d; g.K = m.r + m.E;
            BIGMAC_TRY(gemm(L, G_DX, g, st));
        }
        if (G->dw_down || G->dw_gate) {   // [dW_down ; dW_gate] = [dx' | dl]^T x: x is read once for both
            GemmArgs g;
            g.A = b.dcat; g.lda = ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.C = b.splitk_ws; g.ldc = m.d; g.out_f32 = true; g.M = ldcat; g.N = m.d; g.K = m.T;
            g.split_k = choose_split_k(g.M, g.N, g.K);
            BIGMAC_TRY(gemm(L, G_DW_DOWN, g, sw));
            Stage s(L, S_SPLITK_REDUCE, sw);
            BIGMAC_CUDA(launch_splitk_reduce(b.splitk_ws, g.split_k, ldcat, m.d, G->dw_down, m.r, G->dw_gate, m.E, m.dtype,
                                             acc, sw));
        }
        if (sw != st) {
            BIGMAC_CUDA(cudaEventRecord(L->fork_join[7], sd));
            BIGMAC_CUDA(cudaStreamWaitEvent(st, L->fork_join[7], 0));
        }
    } else {
        {   // dx = dx' W_down
            GemmArgs g;
            g.A = b.dx_lo; g.lda = ldcat; g.B = W->w_down; g.ldb = m.d; g.b_kmajor = false; g.C = dx; g.ldc = m.d;
            g.M = m.T; g.N = m.d; g.K = m.r;
            BIGMAC_TRY(gemm(L, G_DX, g, st));
        }
        {   // dx += dl W_gate
            GemmArgs g;
            g.A = b.dlogits; g.lda = ldcat; g.B = W->w_gate; g.ldb = m.d; g.b_kmajor = false; g.C = dx; g.ldc = m.d;
            g.M = m.T; g.N = m.d; g.K = m.E; g.accumulate = true;
            BIGMAC_TRY(gemm(L, G_DX_GATE, g, st));
        }
        if (G->dw_down) {   // dW_down[c',c] = sum_t dx'[t,c'] x[t,c]
            GemmArgs g;
            g.A = b.dx_lo; g.lda = ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.C = G->dw_down; g.ldc = m.d; g.M = m.r; g.N = m.d; g.K = m.T; g.accumulate = acc;
            BIGMAC_TRY(gemm(L, G_DW_DOWN, g, st));
        }
        if (G->dw_gate) {   // dW_gate[e,c] = sum_t dl[t,e] x[t,c]
            GemmArgs g;
            g.A = b.dlogits; g.lda = ldcat; g.a_kmajor = false; g.B = x; g.ldb = m.d; g.b_kmajor = false;
            g.C = G->dw_gate; g.ldc = m.d; g.M = m.E; g.N = m.d; g.K = m.T; g.accumulate = acc;
            BIGMAC_TRY(gemm(L, G_DW_GATE, g, st));
        }
    }
    if (!colsum_done && G->db_gate) {
        Stage s(L, S_COLSUM, st, 2);
        BIGMAC_CUDA(launch_gate_colsum(b.dp, b.tb, G->db_gate, b.colsum_part, m.N, m.E, acc, st, aux_part));
    }
    return BIGMAC_OK;
}

int bigmac_device_status(bigmac_layer_t* L, void* stream) {
    if (!L) return BIGMAC_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int word = 0;
    if (cudaMemcpyAsync(&word, L->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(L->status, 0, sizeof(int), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
        return BIGMAC_ERR_CUDA;
    if (word != 0) {
        // a kernel gave up on a wait: its work counters and the grid-barrier word may be mid-count; back to rest
        if (cudaMemsetAsync(L->status + 1, 0, 3 * sizeof(int), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
            return BIGMAC_ERR_CUDA;
    }
    if (word == 2) return BIGMAC_ERR_STATE;            // an expert-parallel count matrix that cannot be right, or an expert id outside [0, E)
    return word == 0 ? BIGMAC_OK : BIGMAC_ERR_TIMEOUT;
}

const char* bigmac_status_string(int status) {
    switch (status) {
        case BIGMAC_OK: return "ok";
        case BIGMAC_ERR_INVALID_ARG: return "invalid argument";
        case BIGMAC_ERR_UNSUPPORTED: return "unsupported configuration";
        case BIGMAC_ERR_WORKSPACE: return "workspace too small";
        case BIGMAC_ERR_CUDA: return "CUDA error";
        case BIGMAC_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case BIGMAC_ERR_STATE: return "handle used on the wrong device, an expert-parallel count matrix that cannot be right, or an expert id outside [0, E) in the routing tables";
        case BIGMAC_ERR_TOO_LARGE: return "problem exceeds the fixed scratch array of bigmac_route_static";
        default: return "unknown status";
    }
}

int bigmac_exchange_rows(bigmac_layer_t* L, const void* saved, int32_t T, int32_t width, const void* src,
                         void* grouped, size_t grouped_bytes, void* dst, int which, void* stream) {
    BIGMAC_TRY(check_call(L, T));
    if (!saved || !grouped || width <= 0 || which < 0 || which > 2 || !aligned(saved, 256) ||
        !aligned(grouped, 16) || !aligned(src, 16) || !aligned(dst, 16))
        return BIGMAC_ERR_INVALID_ARG;
    if ((which != 1 && !src) || (which != 0 && !dst)) return BIGMAC_ERR_INVALID_ARG;
    const size_t es = esize(L->cfg.dtype);
    if ((width * es) % 16) return BIGMAC_ERR_UNSUPPORTED;
    if (T == 0) return BIGMAC_OK;
    const Dims m = dims_of(L, T);
    if (grouped_bytes < (size_t)m.P * width * es) return BIGMAC_ERR_WORKSPACE;
    Buffers b{};
    Carver cv(const_cast<void*>(saved));
    carve_saved(cv, m, b, true);
    cudaStream_t st = (cudaStream_t)stream;
    if (which != 1) { Stage s(L, S_DISPATCH, st); BIGMAC_CUDA(launch_dispatch(src, grouped, b.tb, m.k, width, m.dtype, m.P, st)); }
    if (which != 0) {
        Stage s(L, S_COMBINE, st);
        BIGMAC_CUDA(launch_combine(grouped, dst, b.tb.topk_w, b.tb.prow_of_slot, m.T, m.k, width, m.dtype, st, 0, m.cap != kNoCapacity));
    }
    return BIGMAC_OK;
}

}  // extern "C"

// ---- routing without caller-provided scratch ----------------------------------------------------------
// The intermediates of the routing step live in this file-scope device array.  In host code its name is
// only a stand-in for the symbol, never a device address: the address is resolved once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what the kernels are given.
static __device__ __align__(256) unsigned char g_route_static_scratch[BIGMAC_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};

// Device address of the array on the current device (which the caller has checked to be `device`).
int static_scratch_address(int device, void** ptr) {
    if (device < 0 || device >= kMaxDevices) return BIGMAC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_route_static_scratch) != cudaSuccess || !p) return BIGMAC_ERR_CUDA;
        g_static_ptr[device] = p;
    }
    *ptr = g_static_ptr[device];
    return BIGMAC_OK;
}

// Only what routing needs: logits, counting-sort counters and the tables (no float intermediates).
void carve_route_only(Carver& cv, const Dims& m, Buffers& b) {
    carve_route_scratch(cv, m, b);
    b.tb.topk_idx = cv.take<int32_t>(m.N);
    b.tb.topk_w = cv.take<float>(m.N);
    b.tb.counts = cv.take<int32_t>(m.E);
    b.tb.offsets = cv.take<int32_t>(m.E + 1);
    b.tb.poffsets = cv.take<int32_t>(m.E + 1);
    b.tb.row_of_slot = cv.take<int32_t>(m.N);
    b.tb.slot_of_row = cv.take<int32_t>(m.N);
    b.tb.prow_of_slot = cv.take<int32_t>(m.N);
    b.tb.slot_of_prow = cv.take<int32_t>(m.P);
    b.tb.tile_expert = cv.take<int32_t>(m.P / kPad);
    b.tb.n_tiles = cv.take<int32_t>(1);
    b.tb.counts_chosen = cv.take<int32_t>(m.E);
    b.aux_loss = cv.take<float>(1);
    if (m.gate_low) b.x_lo = cv.take_bytes((size_t)m.T * m.r * esize(m.dtype));   // the gate reads x'
}

}  // namespace

extern "C" {

int bigmac_route_static(bigmac_layer_t* L, const void* x, int32_t T, const bigmac_weights_t* W,
                        bigmac_routing_t* out, void* stream) {
    BIGMAC_TRY(check_call(L, T));
    if (!out) return BIGMAC_ERR_INVALID_ARG;
    BIGMAC_TRY(check_weights(L, W));
    if (T == 0) return BIGMAC_OK;
    if (!x || !aligned(x, 16)) return BIGMAC_ERR_INVALID_ARG;
    const Dims m = dims_of(L, T);
    {
        Carver measure(nullptr);
        Buffers b{};
        carve_route_only(measure, m, b);
        if (measure.total() > (size_t)BIGMAC_STATIC_SCRATCH_BYTES) return BIGMAC_ERR_TOO_LARGE;
    }
    void* base = nullptr;
    BIGMAC_TRY(static_scratch_address(L->device, &base));
    Carver cv(base);
    Buffers b{};
    carve_route_only(cv, m, b);
    alias_routing(b, out);
    cudaStream_t st = (cudaStream_t)stream;
    BIGMAC_TRY(run_routing(L, m, x, W, b, st));
    return export_routing(m, b, out, st);
}

int bigmac_profile_enable(bigmac_layer_t* L, int on) {
    if (!L) return BIGMAC_ERR_INVALID_ARG;
    if (on && L->ev.empty()) {
        L->ev.resize(2 * kEventPairs);
        for (cudaEvent_t& e : L->ev)
            if (cudaEventCreate(&e) != cudaSuccess) return BIGMAC_ERR_CUDA;
    }
    L->prof_on = on != 0;
    L->launches = 0;
    L->dropped = 0;
    L->ev_slot.clear();
    std::memset(L->ms, 0, sizeof(L->ms));
    std::memset(L->calls, 0, sizeof(L->calls));
    return BIGMAC_OK;
}

int bigmac_profile_read(bigmac_layer_t* L, void* stream, bigmac_profile_t* out) {
    if (!L || !out) return BIGMAC_ERR_INVALID_ARG;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BIGMAC_ERR_CUDA;
    for (size_t i = 0; i < L->ev_slot.size(); ++i) {
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, L->ev[2 * i], L->ev[2 * i + 1]) == cudaSuccess) L->ms[L->ev_slot[i]] += ms;
    }
    L->ev_slot.clear();
    out->launches = L->launches;
    out->dropped = L->dropped;
    out->n_slots = S_COUNT;
    std::memcpy(out->ms, L->ms, sizeof(L->ms));
    std::memcpy(out->calls, L->calls, sizeof(L->calls));
    return BIGMAC_OK;
}

const char* bigmac_profile_slot_name(int slot) { return slot >= 0 && slot < S_COUNT ? kSlotNames[slot] : ""; }

// ---- debug / unit-test entry point (declared in bigmac_debug.h) --------------------------------------
int bigmac_debug_gemm(bigmac_layer_t* L, const bigmac_debug_gemm_t* q, int use_tensor_cores, void* stream) {
    if (!L || !q) return BIGMAC_ERR_INVALID_ARG;
    GemmArgs g;
    g.A = q->A; g.B = q->B; g.C = q->C; g.Z = q->Z; g.lda = q->lda; g.ldb = q->ldb; g.ldc = q->ldc;
    g.M = q->M; g.N = q->N; g.K = q->K; g.a_kmajor = q->a_kmajor != 0; g.b_kmajor = q->b_kmajor != 0;
    g.out_f32 = q->out_f32 != 0; g.accumulate = q->accumulate != 0; g.epilogue = q->epilogue; g.act = q->act;
    g.group = q->group; g.num_experts = q->num_experts; g.b_stride = q->b_stride; g.c_stride = q->c_stride;
    g.tile_expert = q->tile_expert; g.n_tiles = q->n_tiles; g.poffsets = q->poffsets;
    L->launches += 1;
    g.force_kernel = use_tensor_cores == 2 ? 1 : use_tensor_cores >= 3 ? 2 : 0;
    g.epi_parts = use_tensor_cores == 4 ? 2 : use_tensor_cores == 5 ? 1 : use_tensor_cores == 3 ? 4 : 0;
    cudaError_t err = use_tensor_cores ? gemm_tc(g, L->status, (cudaStream_t)stream)
                                       : gemm_simt(g, L->cfg.dtype, (cudaStream_t)stream);
    return err == cudaSuccess ? BIGMAC_OK : BIGMAC_ERR_CUDA;
}

int bigmac_debug_set(const char* name, int value) {
    if (!name) return BIGMAC_ERR_INVALID_ARG;
    Switches& sw = switches();
    if (!std::strcmp(name, "overlap")) sw.overlap = value;
    else if (!std::strcmp(name, "tc_pair")) sw.tc_pair = value;
    else if (!std::strcmp(name, "groupk")) sw.groupk = value;
    else if (!std::strcmp(name, "fused_mlp")) sw.fused_mlp = value;
    else if (!std::strcmp(name, "epi_parts")) sw.epi_parts = value;
    else if (!std::strcmp(name, "staged_stores")) sw.staged_stores = value;
    else if (!std::strcmp(name, "chain")) sw.chain = value;
    else if (!std::strcmp(name, "fuse_dispatch")) sw.fuse_dispatch = value;
    else if (!std::strcmp(name, "tc_mask")) sw.tc_mask = (unsigned)value;
    else if (!std::strcmp(name, "defaults")) sw = Switches();
    else return BIGMAC_ERR_INVALID_ARG;
    return BIGMAC_OK;
}

int bigmac_debug_expire_wait(bigmac_layer_t* L, void* stream) {
    if (!L) return BIGMAC_ERR_INVALID_ARG;
    L->launches += 1;
    return launch_expire_wait(L->status, (cudaStream_t)stream) == cudaSuccess ? BIGMAC_OK : BIGMAC_ERR_CUDA;
}

}  // extern "C"
