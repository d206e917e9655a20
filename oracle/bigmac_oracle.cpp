// CPU oracle for the BigMac DCCA Mixture-of-Experts layer.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, per-token / per-row evaluation in fp64 of what the layer computes, written
// from the paper's equations.  It shares no code with the CUDA library and must never sit on
// the product path: only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
//
// The layer (Eq. 2 with the BigMac expert of Eq. 4; the gate reads the full-width token x, as the
// text after Eq. 2 chooses):
//     x' = x W'_down ;   y' = sum_{i in T} p_i(x) E_i(x') ;   y = y' W'_up ;
//     E_i(v) = sigma(v W_{i,up}) W_{i,down}
// Storage convention: every weight is [out_features, in_features], row-major, so "v W" above is
// out[o] = sum_i v[i] * W[o][i].  Names: w_down [r,d], w1 = W_{i,up} [E,h,r], w2 = W_{i,down} [E,r,h],
// w_up [d,r], w_gate [E,d], b_gate [E] (optional).
//
// Readings where the paper is silent (all listed in the design notes): linear gate; top-k by
// (logit descending, expert id ascending); gate weights = softmax over the k selected logits;
// dropless routing; no biases except the optional gate bias; rows of an expert's segment in
// ascending slot id (slot s = t*k + j).
//
// Training-recipe variants of the pre-training configuration (Table 5: capacity factor 1.2, load-balancing loss
// with coefficient 0.001), for which the paper prints no formula; the conventional ones are taken:
//   capacity: an expert keeps the first C = ceil(f T k / E) of the slots that chose it, in slot order; a dropped
//   slot adds nothing to y' (gate values are not renormalised) and receives no gradient;
//   load-balancing loss: L_aux = alpha E sum_e f_e P_e, f_e = slots that chose e / (T k) (before dropping),
//   P_e = mean over tokens of the softmax of the logits over all E experts; gradient through P only.
// `keep` arguments below are per-slot bytes (1 = kept, 0 = dropped), NULL = every slot kept (dropless).
//
// Inputs are float arrays holding values exactly representable in the workload dtype; they are
// widened to double before any arithmetic and nothing is rounded afterwards.
//
// Parity pins (tests, CPU only): top-k against a full library sort, gate weights against a library
// softmax, tables against a library stable argsort and a brute-force count, E=1/k=1 and
// shared-expert special cases against a 4-matmul MLP, identity-expert case against the two
// projections alone, per-token against grouped evaluation, gradients against central finite
// differences and the adjoint identity; capacity tables against a brute-force per-expert list, the dropped
// forward against the E=1, k=1 case (rows past C are zero, the others a plain MLP) and against the dropless
// forward minus the dropped slots' terms, the load-balancing loss against its closed forms (equal logits: alpha;
// collapse onto one expert: alpha E) and its gradient against central differences.  Float values of y and of the gradients on random data
// have no printed example in the paper: "parity unpinned" by the paper for those, pinned only by
// the special cases above.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>

namespace {

enum { ACT_RELU = 0, ACT_GELU_ERF = 1, ACT_GELU_TANH = 2, ACT_IDENTITY = 3 };

const double kSqrt2 = 1.41421356237309504880;
const double kSqrt2OverPi = 0.79788456080286535588;
const double kInvSqrt2Pi = 0.39894228040143267794;

// sigma of Eq. 4.
double act_f(int act, double z) {
    switch (act) {
        case ACT_RELU: return z > 0.0 ? z : 0.0;
        case ACT_GELU_ERF: return 0.5 * z * (1.0 + std::erf(z / kSqrt2));
        case ACT_GELU_TANH: return 0.5 * z * (1.0 + std::tanh(kSqrt2OverPi * (z + 0.044715 * z * z * z)));
        default: return z;
    }
}

// d sigma / dz.  ReLU' is 0 at z = 0.
double act_df(int act, double z) {
    switch (act) {
        case ACT_RELU: return z > 0.0 ? 1.0 : 0.0;
        case ACT_GELU_ERF: {
            double Phi = 0.5 * (1.0 + std::erf(z / kSqrt2));
            double phi = kInvSqrt2Pi * std::exp(-0.5 * z * z);
            return Phi + z * phi;
        }
        case ACT_GELU_TANH: {
            double w = kSqrt2OverPi * (z + 0.044715 * z * z * z);
            double th = std::tanh(w);
            double dw = kSqrt2OverPi * (1.0 + 3.0 * 0.044715 * z * z);
            return 0.5 * (1.0 + th) + 0.5 * z * (1.0 - th * th) * dw;
        }
        default: return 1.0;
    }
}

// out[o] = sum_i v[i] * W[o][i]      (W is [n_out, n_in] floats, widened per element)
void matvec(const double* v, const float* W, int n_out, int n_in, double* out) {
    for (int o = 0; o < n_out; ++o) {
        const float* row = W + (size_t)o * n_in;
        double acc = 0.0;
        for (int i = 0; i < n_in; ++i) acc += v[i] * (double)row[i];
        out[o] = acc;
    }
}

// out[i] = sum_o g[o] * W[o][i]      (the transpose product, for gradients w.r.t. the input)
void matvec_t(const double* g, const float* W, int n_out, int n_in, double* out) {
    for (int i = 0; i < n_in; ++i) out[i] = 0.0;
    for (int o = 0; o < n_out; ++o) {
        const float* row = W + (size_t)o * n_in;
        double go = g[o];
        for (int i = 0; i < n_in; ++i) out[i] += go * (double)row[i];
    }
}

// Round to the nearest bf16 value (ties to even), via float.
double round_bf16(double v) {
    float f = (float)v;
    uint32_t bits;
    std::memcpy(&bits, &f, 4);
    bits = (bits + 0x7fffu + ((bits >> 16) & 1u)) & 0xffff0000u;
    std::memcpy(&f, &bits, 4);
    return (double)f;
}

// The pre-activation at which sigma' is evaluated in the backward pass.  ReLU' is a discrete decision
// (z > 0): when `decide_bf16` is set it is taken the way the BF16 kernels take it, from x' rounded to
// bf16, so that both sides decide on the same numbers; every other quantity stays exact.
void decision_preact(const double* x_lo, const double* z_exact, const float* w1_e, int r, int h, int act,
                     int decide_bf16, double* z_dec, const float* b1_e = nullptr) {
    if (!decide_bf16 || act != ACT_RELU) {
        std::memcpy(z_dec, z_exact, sizeof(double) * h);
        return;
    }
    std::vector<double> xr(r);
    for (int c = 0; c < r; ++c) xr[c] = round_bf16(x_lo[c]);
    matvec(xr.data(), w1_e, h, r, z_dec);
    if (b1_e)
        for (int q = 0; q < h; ++q) z_dec[q] += (double)b1_e[q];
}

void widen(const float* src, int n, double* dst) {
    for (int i = 0; i < n; ++i) dst[i] = (double)src[i];
}

// One routed slot of one token through expert e (Eq. 4):  z = x' W1_e^T, a = sigma(z), u = a W2_e^T.
// Variant with expert biases (Eq. 4 has none; Table 3's parameter count has a bias-like term): z += b1_e, u += b2_e;
// b1_e [h] / b2_e [r] are NULL without them.
void expert_forward(const double* x_lo, const float* w1_e, const float* w2_e, int r, int h, int act,
                    double* z, double* a, double* u, const float* b1_e = nullptr, const float* b2_e = nullptr) {
    matvec(x_lo, w1_e, h, r, z);
    if (b1_e)
        for (int q = 0; q < h; ++q) z[q] += (double)b1_e[q];
    for (int q = 0; q < h; ++q) a[q] = act_f(act, z[q]);
    matvec(a, w2_e, r, h, u);
    if (b2_e)
        for (int c = 0; c < r; ++c) u[c] += (double)b2_e[c];
}

}  // namespace

extern "C" {

// Gate logits: l[t,e] = sum_c x[t,c] W_g[e,c] (+ b_g[e]).  The gate reads x, not x' (text after Eq. 2).
void oracle_gate_logits(const float* x, const float* w_gate, const float* b_gate, int T, int d, int E,
                        double* logits) {
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        std::vector<double> xt(d);
        widen(x + (size_t)t * d, d, xt.data());
        matvec(xt.data(), w_gate, E, d, logits + (size_t)t * E);
        if (b_gate)
            for (int e = 0; e < E; ++e) logits[(size_t)t * E + e] += (double)b_gate[e];
    }
}

// Variant (the choice the text after Eq. 2 mentions and sets aside): the gate reads the low-width token,
// l[t,e] = sum_c x'[t,c] W_g[e,c] (+ b_g[e]) with W_g [E,r] and x' = x W'_down.  round_bf16: x' is rounded to bf16
// first, as the BF16 kernels hold it, so that the discrete top-k choice is taken on the same numbers on both sides.
void oracle_gate_logits_low(const float* x, const float* w_down, const float* w_gate, const float* b_gate, int T, int d,
                            int r, int E, int round_x_lo_bf16, double* logits) {
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        std::vector<double> xt(d), x_lo(r);
        widen(x + (size_t)t * d, d, xt.data());
        matvec(xt.data(), w_down, r, d, x_lo.data());
        if (round_x_lo_bf16)
            for (int c = 0; c < r; ++c) x_lo[c] = round_bf16(x_lo[c]);
        matvec(x_lo.data(), w_gate, E, r, logits + (size_t)t * E);
        if (b_gate)
            for (int e = 0; e < E; ++e) logits[(size_t)t * E + e] += (double)b_gate[e];
    }
}

// Top-k set T of Eq. 2 and the gate values p_i: experts ordered by (logit descending, id ascending),
// first k kept in that order; p = softmax over the k kept logits (so the p of a token sum to 1).
// Non-finite logits (the paper is silent; a diverging run produces them): NaN is ordered as -inf, so that the order
// is total and ties among -inf fall to the lower id; a token whose k kept logits are all -inf gets p = 1/k each.
// Every id written lies in [0, E).
void oracle_topk(const double* logits, int T, int E, int k, int32_t* topk_idx, double* topk_p) {
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        std::vector<double> l(logits + (size_t)t * E, logits + (size_t)(t + 1) * E);
        for (int e = 0; e < E; ++e)
            if (std::isnan(l[e])) l[e] = -INFINITY;
        std::vector<int> order(E);
        std::iota(order.begin(), order.end(), 0);
        std::stable_sort(order.begin(), order.end(), [&l](int a, int b) { return l[a] > l[b]; });
        const double m = l[order[0]];
        double denom = 0.0;
        for (int j = 0; j < k; ++j) denom += std::isinf(m) && m < 0 ? 1.0 : std::exp(l[order[j]] - m);
        for (int j = 0; j < k; ++j) {
            topk_idx[(size_t)t * k + j] = order[j];
            topk_p[(size_t)t * k + j] = (std::isinf(m) && m < 0 ? 1.0 : std::exp(l[order[j]] - m)) / denom;
        }
    }
}

// Dropless dispatch layout (the on-device stand-in for the first All-to-All): a stable counting sort
// of slot ids s = t*k + j by expert id.
void oracle_tables(const int32_t* topk_idx, int T, int k, int E, int32_t* counts, int32_t* offsets,
                   int32_t* row_of_slot, int32_t* slot_of_row) {
    const int64_t N = (int64_t)T * k;
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (int64_t s = 0; s < N; ++s) counts[topk_idx[s]] += 1;
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
    std::vector<int32_t> seen(E, 0);   // slots already placed per expert = #{s' < s : idx[s'] = e}
    for (int64_t s = 0; s < N; ++s) {
        int e = topk_idx[s];
        int32_t row = offsets[e] + seen[e];
        seen[e] += 1;
        row_of_slot[s] = row;
        slot_of_row[row] = (int32_t)s;
    }
}

// Dispatch layout under a capacity of `cap` rows per expert (Table 5's capacity factor; cap = ceil(f T k / E) is
// computed by the caller): the stable counting sort above, except that a slot whose rank among the slots of its
// expert is >= cap is dropped: keep[s] = 0, row_of_slot[s] = -1.  counts / offsets describe the kept rows,
// counts_chosen the slots before dropping; slot_of_row[row] = -1 for row >= offsets[E].
void oracle_tables_capacity(const int32_t* topk_idx, int T, int k, int E, int cap, int32_t* counts_chosen,
                            int32_t* counts, int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row,
                            uint8_t* keep) {
    const int64_t N = (int64_t)T * k;
    for (int e = 0; e < E; ++e) counts_chosen[e] = 0;
    for (int64_t s = 0; s < N; ++s) counts_chosen[topk_idx[s]] += 1;
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) {
        counts[e] = std::min(counts_chosen[e], cap);
        offsets[e + 1] = offsets[e] + counts[e];
    }
    for (int64_t row = 0; row < N; ++row) slot_of_row[row] = -1;
    std::vector<int32_t> seen(E, 0);
    for (int64_t s = 0; s < N; ++s) {
        const int e = topk_idx[s];
        const int32_t rank = seen[e];
        seen[e] += 1;
        keep[s] = rank < cap ? 1 : 0;
        if (keep[s]) {
            row_of_slot[s] = offsets[e] + rank;
            slot_of_row[offsets[e] + rank] = (int32_t)s;
        } else {
            row_of_slot[s] = -1;
        }
    }
}

// Load-balancing loss (Table 5, coefficient alpha) and its gradient with respect to the gate logits:
//   p[t,:] = softmax over all E of l[t,:] ;  P_e = (1/T) sum_t p[t,e] ;  f_e = #{slots with topk_idx = e} / (T k) ;
//   L_aux = alpha E sum_e f_e P_e ;  dL/dl[t,e] = (alpha E / T) p[t,e] (f_e - sum_j f_j p[t,j])   (f held constant).
// dlogits [T,E] may be NULL.
void oracle_aux_loss(const double* logits, const int32_t* topk_idx, int T, int E, int k, double alpha,
                     double* loss, double* dlogits) {
    std::vector<double> f(E, 0.0), P(E, 0.0), p((size_t)T * E);
    for (int64_t s = 0; s < (int64_t)T * k; ++s) f[topk_idx[s]] += 1.0;
    for (int e = 0; e < E; ++e) f[e] /= (double)T * k;
    for (int t = 0; t < T; ++t) {
        const double* l = logits + (size_t)t * E;
        double m = l[0], denom = 0.0;
        for (int e = 1; e < E; ++e) m = std::max(m, l[e]);
        for (int e = 0; e < E; ++e) denom += std::exp(l[e] - m);
        for (int e = 0; e < E; ++e) {
            p[(size_t)t * E + e] = std::exp(l[e] - m) / denom;
            P[e] += p[(size_t)t * E + e] / T;
        }
    }
    double acc = 0.0;
    for (int e = 0; e < E; ++e) acc += f[e] * P[e];
    *loss = alpha * E * acc;
    if (!dlogits) return;
    for (int t = 0; t < T; ++t) {
        const double* pt = &p[(size_t)t * E];
        double fp = 0.0;
        for (int e = 0; e < E; ++e) fp += f[e] * pt[e];
        for (int e = 0; e < E; ++e) dlogits[(size_t)t * E + e] = alpha * E / T * pt[e] * (f[e] - fp);
    }
}

// Forward, token by token, exactly as Eq. 2 is written.  `tokens` selects n token ids (NULL = 0..n-1).
// Outputs are indexed by position in `tokens`.  z_out / u_out may be NULL.
void oracle_forward_tokens(const float* x, const float* w_down, const float* w1, const float* w2,
                           const float* w_up, const int32_t* topk_idx, const double* topk_p,
                           const int32_t* tokens, int n, int d, int r, int h, int E, int k, int act,
                           double* x_lo_out, double* y_lo_out, double* y_out, double* z_out, double* u_out,
                           const uint8_t* keep, const float* b1, const float* b2) {
    (void)E;
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < n; ++i) {
        const int t = tokens ? tokens[i] : i;
        std::vector<double> xt(d), x_lo(r), z(h), a(h), u(r), y_lo(r, 0.0);
        widen(x + (size_t)t * d, d, xt.data());
        matvec(xt.data(), w_down, r, d, x_lo.data());                       // x' = x W'_down
        for (int j = 0; j < k; ++j) {                                       // sum over i in T
            const int e = topk_idx[(size_t)t * k + j];
            const double p = topk_p[(size_t)t * k + j];
            expert_forward(x_lo.data(), w1 + (size_t)e * h * r, w2 + (size_t)e * r * h, r, h, act,
                           z.data(), a.data(), u.data(), b1 ? b1 + (size_t)e * h : nullptr, b2 ? b2 + (size_t)e * r : nullptr);
            if (!keep || keep[(size_t)t * k + j])
                for (int c = 0; c < r; ++c) y_lo[c] += p * u[c];           // p_i(x) E_i(x'); nothing from a dropped slot
            if (z_out) std::memcpy(z_out + ((size_t)i * k + j) * h, z.data(), sizeof(double) * h);
            if (u_out) std::memcpy(u_out + ((size_t)i * k + j) * r, u.data(), sizeof(double) * r);
        }
        if (x_lo_out) std::memcpy(x_lo_out + (size_t)i * r, x_lo.data(), sizeof(double) * r);
        if (y_lo_out) std::memcpy(y_lo_out + (size_t)i * r, y_lo.data(), sizeof(double) * r);
        if (y_out) matvec(y_lo.data(), w_up, d, r, y_out + (size_t)i * d);  // y = y' W'_up
    }
}

// Forward the way a dispatching implementation evaluates it: descend all tokens, gather the r-wide
// rows into expert segments (dispatch), run every expert over its segment, combine by slot with the
// gate weights, ascend.  Must agree with oracle_forward_tokens; it also exercises the tables.
void oracle_forward_grouped(const float* x, const float* w_down, const float* w1, const float* w2,
                            const float* w_up, const double* topk_p, const int32_t* offsets,
                            const int32_t* row_of_slot, const int32_t* slot_of_row, int T, int d, int r,
                            int h, int E, int k, int act, double* xg_out, double* y_lo_out, double* y_out,
                            const float* b1, const float* b2) {
    const int64_t N = (int64_t)T * k;
    std::vector<double> x_lo((size_t)T * r), xg((size_t)N * r), ug((size_t)N * r);
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        std::vector<double> xt(d);
        widen(x + (size_t)t * d, d, xt.data());
        matvec(xt.data(), w_down, r, d, &x_lo[(size_t)t * r]);
    }
    for (int64_t row = 0; row < offsets[E]; ++row) {                        // dispatch (offsets[E] = N when dropless)
        const int t = slot_of_row[row] / k;
        std::memcpy(&xg[(size_t)row * r], &x_lo[(size_t)t * r], sizeof(double) * r);
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int e = 0; e < E; ++e) {                                           // experts over segments
        std::vector<double> z(h), a(h);
        for (int row = offsets[e]; row < offsets[e + 1]; ++row)
            expert_forward(&xg[(size_t)row * r], w1 + (size_t)e * h * r, w2 + (size_t)e * r * h, r, h, act,
                           z.data(), a.data(), &ug[(size_t)row * r], b1 ? b1 + (size_t)e * h : nullptr,
                           b2 ? b2 + (size_t)e * r : nullptr);
    }
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {                                           // combine + ascend
        std::vector<double> y_lo(r, 0.0);
        for (int j = 0; j < k; ++j) {
            const int64_t s = (int64_t)t * k + j;
            const double p = topk_p[s];
            if (row_of_slot[s] < 0) continue;                               // dropped under a capacity limit
            const double* u = &ug[(size_t)row_of_slot[s] * r];
            for (int c = 0; c < r; ++c) y_lo[c] += p * u[c];
        }
        if (y_lo_out) std::memcpy(y_lo_out + (size_t)t * r, y_lo.data(), sizeof(double) * r);
        if (y_out) matvec(y_lo.data(), w_up, d, r, y_out + (size_t)t * d);
    }
    if (xg_out) std::memcpy(xg_out, xg.data(), sizeof(double) * xg.size());
}

// Backward of the scalar L = sum(y * dy), token by token (chain rule through Eq. 2 / Eq. 4; the
// discrete top-k choice carries no gradient, the gate weights do).  Per selected token i (id t):
//   dy' = dy W_up ; per slot j: dp_j = <dy', u_j>, du_j = p_j dy', da_j = du_j W2, dz_j = da_j * sigma'(z_j),
//   dx' = sum_j dz_j W1 ; softmax-over-k: g = sum_i p_i dp_i, dl_j = p_j (dp_j - g) ;
//   dx = dx' W_down + sum_j dl_j W_g[e_j]     (gate on x';  with gate_low: dx = (dx' + sum_j dl_j W_g[e_j]) W_down).
// Outputs (any may be NULL) are indexed by position in `tokens`.
void oracle_backward_tokens(const float* x, const float* dy, const float* w_gate, const float* w_down,
                            const float* w1, const float* w2, const float* w_up, const int32_t* topk_idx,
                            const double* topk_p, const int32_t* tokens, int n, int d, int r, int h, int E,
                            int k, int act, int decide_bf16, double* dx_out, double* dx_lo_out,
                            double* dlogit_out, double* dy_lo_out, const uint8_t* keep, int gate_low,
                            const float* b1, const float* b2) {
    (void)E;
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < n; ++i) {
        const int t = tokens ? tokens[i] : i;
        std::vector<double> xt(d), dyt(d), x_lo(r), dy_lo(r), z(h), zd(h), a(h), u(r), du(r), da(h), dz(h), tmp(r),
            dx_lo(r, 0.0), dp(k), dl(k), dx(d), gate_part(d, 0.0);
        widen(x + (size_t)t * d, d, xt.data());
        widen(dy + (size_t)t * d, d, dyt.data());
        matvec(xt.data(), w_down, r, d, x_lo.data());
        matvec_t(dyt.data(), w_up, d, r, dy_lo.data());
        for (int j = 0; j < k; ++j) {
            const int e = topk_idx[(size_t)t * k + j];
            const double p = topk_p[(size_t)t * k + j];
            const float* w1_e = w1 + (size_t)e * h * r;
            const float* w2_e = w2 + (size_t)e * r * h;
            if (keep && !keep[(size_t)t * k + j]) { dp[j] = 0.0; continue; }   // a dropped slot is absent from y'
            const float* b1_e = b1 ? b1 + (size_t)e * h : nullptr;
            expert_forward(x_lo.data(), w1_e, w2_e, r, h, act, z.data(), a.data(), u.data(), b1_e,
                           b2 ? b2 + (size_t)e * r : nullptr);
            double acc = 0.0;
            for (int c = 0; c < r; ++c) acc += dy_lo[c] * u[c];
            dp[j] = acc;
            for (int c = 0; c < r; ++c) du[c] = p * dy_lo[c];
            matvec_t(du.data(), w2_e, r, h, da.data());
            decision_preact(x_lo.data(), z.data(), w1_e, r, h, act, decide_bf16, zd.data(), b1_e);
            for (int q = 0; q < h; ++q) dz[q] = da[q] * act_df(act, zd[q]);
            matvec_t(dz.data(), w1_e, h, r, tmp.data());
            for (int c = 0; c < r; ++c) dx_lo[c] += tmp[c];
        }
        double g = 0.0;
        for (int j = 0; j < k; ++j) g += topk_p[(size_t)t * k + j] * dp[j];
        for (int j = 0; j < k; ++j) dl[j] = topk_p[(size_t)t * k + j] * (dp[j] - g);
        if (gate_low) {       // the gate read x' (W_g is [E,r]): its gradient joins dx' before the descend projection
            for (int j = 0; j < k; ++j) {
                const float* wg = w_gate + (size_t)topk_idx[(size_t)t * k + j] * r;
                for (int c = 0; c < r; ++c) dx_lo[c] += dl[j] * (double)wg[c];
            }
        }
        matvec_t(dx_lo.data(), w_down, r, d, dx.data());
        if (!gate_low) {
            for (int j = 0; j < k; ++j) {
                const float* wg = w_gate + (size_t)topk_idx[(size_t)t * k + j] * d;
                for (int c = 0; c < d; ++c) gate_part[c] += dl[j] * (double)wg[c];
            }
            for (int c = 0; c < d; ++c) dx[c] += gate_part[c];
        }
        if (dx_out) std::memcpy(dx_out + (size_t)i * d, dx.data(), sizeof(double) * d);
        if (dx_lo_out) std::memcpy(dx_lo_out + (size_t)i * r, dx_lo.data(), sizeof(double) * r);
        if (dlogit_out) std::memcpy(dlogit_out + (size_t)i * k, dl.data(), sizeof(double) * k);
        if (dy_lo_out) std::memcpy(dy_lo_out + (size_t)i * r, dy_lo.data(), sizeof(double) * r);
    }
}

// Weight gradients of one expert e over its segment of rows [offsets[e], offsets[e+1]):
//   dW2_e[c,q] = sum_rows du[c] a[q] ;  dW1_e[q,c] = sum_rows dz[q] x'[c].
// An expert that received no rows gets exactly zero gradients.
void oracle_backward_expert(const float* x, const float* dy, const float* w_down, const float* w1,
                            const float* w2, const float* w_up, const double* topk_p, const int32_t* offsets,
                            const int32_t* slot_of_row, int e, int d, int r, int h, int k, int act,
                            int decide_bf16, double* dw1_e, double* dw2_e, const float* b1, const float* b2,
                            double* db1_e, double* db2_e) {
    std::fill(dw1_e, dw1_e + (size_t)h * r, 0.0);
    std::fill(dw2_e, dw2_e + (size_t)r * h, 0.0);
    if (db1_e) std::fill(db1_e, db1_e + h, 0.0);       // db1_e[q] = sum_rows dz[q] ;  db2_e[c] = sum_rows du[c]
    if (db2_e) std::fill(db2_e, db2_e + r, 0.0);
    const float* b1_e = b1 ? b1 + (size_t)e * h : nullptr;
    const float* b2_e = b2 ? b2 + (size_t)e * r : nullptr;
    const float* w1_e = w1 + (size_t)e * h * r;
    const float* w2_e = w2 + (size_t)e * r * h;
    std::vector<double> xt(d), dyt(d), x_lo(r), dy_lo(r), z(h), zd(h), a(h), u(r), du(r), da(h), dz(h);
    for (int row = offsets[e]; row < offsets[e + 1]; ++row) {
        const int s = slot_of_row[row];
        const int t = s / k;
        const double p = topk_p[s];
        widen(x + (size_t)t * d, d, xt.data());
        widen(dy + (size_t)t * d, d, dyt.data());
        matvec(xt.data(), w_down, r, d, x_lo.data());
        matvec_t(dyt.data(), w_up, d, r, dy_lo.data());
        expert_forward(x_lo.data(), w1_e, w2_e, r, h, act, z.data(), a.data(), u.data(), b1_e, b2_e);
        for (int c = 0; c < r; ++c) du[c] = p * dy_lo[c];
        matvec_t(du.data(), w2_e, r, h, da.data());
        decision_preact(x_lo.data(), z.data(), w1_e, r, h, act, decide_bf16, zd.data(), b1_e);
        for (int q = 0; q < h; ++q) dz[q] = da[q] * act_df(act, zd[q]);
        if (db1_e)
            for (int q = 0; q < h; ++q) db1_e[q] += dz[q];
        if (db2_e)
            for (int c = 0; c < r; ++c) db2_e[c] += du[c];
        for (int c = 0; c < r; ++c)
            for (int q = 0; q < h; ++q) dw2_e[(size_t)c * h + q] += du[c] * a[q];
        for (int q = 0; q < h; ++q)
            for (int c = 0; c < r; ++c) dw1_e[(size_t)q * r + c] += dz[q] * x_lo[c];
    }
}

// dW1 [E,h,r] and dW2 [E,r,h] of every expert (experts are independent: one thread each).
void oracle_backward_all_experts(const float* x, const float* dy, const float* w_down, const float* w1,
                                 const float* w2, const float* w_up, const double* topk_p, const int32_t* offsets,
                                 const int32_t* slot_of_row, int E, int d, int r, int h, int k, int act,
                                 int decide_bf16, double* dw1, double* dw2, const float* b1, const float* b2,
                                 double* db1, double* db2) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int e = 0; e < E; ++e)
        oracle_backward_expert(x, dy, w_down, w1, w2, w_up, topk_p, offsets, slot_of_row, e, d, r, h, k, act,
                               decide_bf16, dw1 + (size_t)e * h * r, dw2 + (size_t)e * r * h, b1, b2,
                               db1 ? db1 + (size_t)e * h : nullptr, db2 ? db2 + (size_t)e * r : nullptr);
}

// Gradients of the shared matrices, as sums over all tokens of outer products of per-token vectors
// (which the caller obtains from oracle_forward_tokens / oracle_backward_tokens):
//   dW_up[c,c'] = sum_t dy[t,c] y'[t,c'] ;  dW_down[c',c] = sum_t dx'[t,c'] x[t,c] ;
//   dW_g[e,c]   = sum_t dl[t,e] x[t,c]   ;  db_g[e]      = sum_t dl[t,e]   (dl is zero off the top-k set).
void oracle_backward_shared(const float* x, const float* dy, const double* y_lo, const double* dx_lo,
                            const int32_t* topk_idx, const double* dlogit, int T, int d, int r, int E, int k,
                            double* dw_up, double* dw_down, double* dw_gate, double* db_gate) {
#pragma omp parallel for schedule(static)
    for (int c = 0; c < d; ++c) {
        double* out = dw_up + (size_t)c * r;
        for (int cc = 0; cc < r; ++cc) out[cc] = 0.0;
        for (int t = 0; t < T; ++t) {
            const double g = (double)dy[(size_t)t * d + c];
            const double* yl = y_lo + (size_t)t * r;
            for (int cc = 0; cc < r; ++cc) out[cc] += g * yl[cc];
        }
    }
#pragma omp parallel for schedule(static)
    for (int cc = 0; cc < r; ++cc) {
        double* out = dw_down + (size_t)cc * d;
        for (int c = 0; c < d; ++c) out[c] = 0.0;
        for (int t = 0; t < T; ++t) {
            const double g = dx_lo[(size_t)t * r + cc];
            const float* xt = x + (size_t)t * d;
            for (int c = 0; c < d; ++c) out[c] += g * (double)xt[c];
        }
    }
#pragma omp parallel for schedule(static)
    for (int e = 0; e < E; ++e) {
        double* out = dw_gate + (size_t)e * d;
        for (int c = 0; c < d; ++c) out[c] = 0.0;
        double bsum = 0.0;
        for (int t = 0; t < T; ++t)
            for (int j = 0; j < k; ++j) {
                if (topk_idx[(size_t)t * k + j] != e) continue;
                const double g = dlogit[(size_t)t * k + j];
                const float* xt = x + (size_t)t * d;
                for (int c = 0; c < d; ++c) out[c] += g * (double)xt[c];
                bsum += g;
            }
        if (db_gate) db_gate[e] = bsum;
    }
}

}  // extern "C"
