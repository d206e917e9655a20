/* bigmac.h - C ABI of the BigMac DCCA Mixture-of-Experts layer for NVIDIA B200 (sm_100a).
 *
 * The layer (paper, Eq. 2, with the BigMac expert of Eq. 4; the gate reads the full-width token x,
 * as the text following Eq. 2 chooses):
 *
 *     x' = x W'_down ;   y' = sum_{i in T} p_i(x) E_i(x') ;   y = y' W'_up ;
 *     E_i(v) = sigma(v W_{i,up}) W_{i,down}
 *
 * T is the set of the top_k experts of the token, p_i its gate values.  Tokens travel between the
 * shared projections and the experts at the low width r; on one GPU the two All-to-All exchanges of
 * Fig. 2c become a dispatch into expert-grouped row segments and a gate-weighted combine back to
 * token order.  Routing is dropless (section "Enabling Dropless Token Routing"): every token reaches
 * exactly k experts and segments have variable length.
 *
 * Symbols (paper's Table 2 in brackets): T tokens [b*s], d model width [h], r low width [r*h],
 * h expert hidden width, E experts [e], k experts per token [top_k], N = T*k routed rows.
 *
 * Conventions
 *  - Every tensor pointer is CALLER-OWNED DEVICE memory, 16-byte aligned, row-major, dense, and is
 *    borrowed only for the stream-ordered duration of the call.  Configuration structs and the
 *    output-size pointers are HOST memory.
 *  - Weights are stored [out_features, in_features] (the contraction index is contiguous):
 *    w_gate [E,d], w_down [r,d], w1 [E,h,r] (W_{i,up}), w2 [E,r,h] (W_{i,down}), w_up [d,r].
 *  - dtype BIGMAC_F32: all float tensors are fp32 and all arithmetic is fp32 FMA.
 *    dtype BIGMAC_BF16: x, y, dy, dx, weights, weight gradients and intermediates are bf16, products
 *    accumulate in fp32 on the tensor cores; gate logits, gate weights and the gate bias stay fp32.
 *    The BF16 path requires d, r and h to be multiples of 64.
 *  - Where the paper is silent: the gate is linear, l = x w_gate^T (+ b_gate); the k experts are
 *    chosen by (logit descending, expert id ascending); p is the softmax over the k chosen logits,
 *    so the p of one token sum to 1; there are no biases other than the optional gate bias.
 *  - The library never allocates device memory in route/forward/backward, never synchronises the
 *    stream (bigmac_device_status excepted) and orders everything after the work already on the stream
 *    passed in (a cudaStream_t as void*) and before whatever the caller puts there next.  bigmac_backward
 *    runs a few launches that do not depend on each other on a second stream owned by the handle, forked
 *    from and joined back into the caller's stream with events (stream capture sees an ordinary fork and
 *    join; if a launch fails after the fork the second stream is joined back before the error is returned).
 *    One handle serves one stream at a time.  The kernels of a call are launched with programmatic stream
 *    serialisation (each is set up while its predecessor still runs and waits for it before it touches memory):
 *    results and ordering against other work on the stream are those of plain launches.
 *  - Behaviour does not depend on the environment: the library reads no environment variable.  Measurement and
 *    debugging aids (per-stage timing, single contractions, kernel-choice switches) are declared in
 *    bigmac_debug.h and are not part of this interface.
 *  - Non-finite values are not trapped and propagate as in any matrix product, with one guarantee: routing never
 *    writes an expert id outside [0, E).  A NaN gate logit is ordered as -inf; when only -inf logits are left among
 *    the experts not yet chosen the lowest such id is taken (its gate value is 0, or 1/k if all k are -inf).
 *  - Return value: BIGMAC_OK (0) or a negative bigmac_status_t.  On an argument error nothing is
 *    launched.  Nothing throws, aborts or traps; problems detected on the device (a bounded wait that
 *    ran out) are recorded in a status word read by bigmac_device_status.
 */
#ifndef BIGMAC_H_
#define BIGMAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bigmac_layer bigmac_layer_t; /* opaque, library-owned */

typedef enum {
    BIGMAC_OK = 0,
    BIGMAC_ERR_INVALID_ARG = -1,
    BIGMAC_ERR_UNSUPPORTED = -2,
    BIGMAC_ERR_WORKSPACE = -3,
    BIGMAC_ERR_CUDA = -4,
    BIGMAC_ERR_TIMEOUT = -5,
    BIGMAC_ERR_STATE = -6,
    BIGMAC_ERR_TOO_LARGE = -7 /* problem exceeds the fixed scratch of bigmac_route_static */
} bigmac_status_t;

typedef enum { BIGMAC_F32 = 0, BIGMAC_BF16 = 1 } bigmac_dtype_t;

/* sigma of Eq. 4.  GELU_ERF: z/2 (1 + erf(z/sqrt 2)); GELU_TANH: the tanh approximation with
 * coefficient 0.044715; IDENTITY exists for tests. */
typedef enum {
    BIGMAC_ACT_RELU = 0,
    BIGMAC_ACT_GELU_ERF = 1,
    BIGMAC_ACT_GELU_TANH = 2,
    BIGMAC_ACT_IDENTITY = 3
} bigmac_act_t;

/* flags */
#define BIGMAC_FLAG_SIMT_GEMM 1u /* BF16 only: run every contraction on the plain FMA kernels (debug aid) */
/* The conventional fine-grained MoE layer the paper compares with (Eq. 3, the communicate-descend-ascend-
 * communicate structure): y = sum_{i in T} p_i(x) E_i(x) with experts that map d -> h -> d themselves, so tokens are
 * dispatched and combined at the full width d and there are no shared projections.  Requires r == d; w_down, w_up,
 * dw_down and dw_up are ignored (may be NULL); w1 is [E,h,d], w2 is [E,d,h].  Same routing, same kernels, same
 * entry points: the like-for-like single-GPU counterpart of the BigMac layer (parameter parity: h = r'h'/d for a
 * BigMac layer with low width r' and expert hidden width h'). */
#define BIGMAC_FLAG_CDAC 2u
/* BF16 tensor-core path: run the per-expert weight gradients on the dynamically scheduled kernel (work items handed
 * out at run time, long experts contracted in parts) whatever the problem size.  Without the flag that kernel is
 * used when there is enough work per SM pair for it to pay, else the statically scheduled one. */
#define BIGMAC_FLAG_DYNAMIC_WGRAD 4u
/* The gate reads the low-width token x' = x W'_down instead of x (the alternative the text after Eq. 2 mentions and
 * sets aside): l = x' w_gate^T (+ b_gate) with w_gate and dw_gate of shape [E,r].  In the backward pass the gate's
 * gradient joins dx' before the descend projection.  Not together with BIGMAC_FLAG_CDAC (there x' is x:
 * INVALID_ARG) nor with a load-balancing loss (UNSUPPORTED). */
#define BIGMAC_FLAG_GATE_LOW 8u
/* Expert biases (Eq. 4 has none; Table 3's parameter count has a bias-like term): E_i(v) = sigma(v W_{i,up} + b1_i)
 * W_{i,down} + b2_i with fp32 b1 [E,h] and b2 [E,r] in bigmac_weights_t (required with this flag, ignored without)
 * and fp32 gradients db1 / db2 in bigmac_grads_t (nullable).  The small-batch and fused-expert inference kernels are
 * bypassed.  Not with expert parallelism (UNSUPPORTED). */
#define BIGMAC_FLAG_EXPERT_BIAS 16u

/* The two training-recipe settings of the paper's pre-training configuration (Table 5: capacity factor 1.2,
 * load-balancing loss with coefficient 0.001).  Both are off (0) in the layer the paper advocates and measures,
 * which is dropless; the paper prints no formula for either, so the conventional ones are used:
 *
 *  capacity_factor f > 0: an expert keeps at most C = ceil(f * T * k / E) rows per call; of the slots that chose
 *    it, the first C in slot order (token ascending, then choice) are kept, the others are dropped.  A dropped
 *    slot contributes nothing to y' (its gate value is NOT redistributed: the p of a token are still the softmax
 *    over its k chosen logits) and receives no gradient.  Conventional implementations pad every expert to C rows;
 *    here segments stay as long as the kept rows, which gives the same result.
 *
 *  aux_loss_coef alpha > 0: L_aux = alpha * E * sum_e f_e P_e, with f_e = (slots that chose e, before dropping)
 *    / (T k) and P_e the mean over tokens of the softmax of the gate logits over ALL E experts.  The forward
 *    writes L_aux; the backward adds dL_aux/dl (through P only; f is piecewise constant) to the gate gradient,
 *    i.e. it returns the gradients of  sum(y * dy) + L_aux. */
typedef struct {
    int32_t d, r, h, E, k; /* 1 <= k <= E */
    int32_t max_tokens;    /* largest T any call will pass */
    int32_t dtype;         /* bigmac_dtype_t */
    int32_t act;           /* bigmac_act_t */
    uint32_t flags;
    double capacity_factor; /* 0 = dropless (Eq. 2 as written); else > 0; C = ceil((f * (T k)) / E) in double */
    double aux_loss_coef;   /* 0 = no load-balancing loss; else > 0 */
} bigmac_config_t;

typedef struct {
    const void *w_gate;   /* [E,d]   ([E,r] with BIGMAC_FLAG_GATE_LOW) */
    const float *b_gate;  /* [E] fp32, or NULL */
    const void *w_down;   /* [r,d]   W'_down of Eq. 2 */
    const void *w1;       /* [E,h,r] W_{i,up} of Eq. 4 */
    const void *w2;       /* [E,r,h] W_{i,down} of Eq. 4 */
    const void *w_up;     /* [d,r]   W'_up of Eq. 2 */
    const float *b1;      /* [E,h] fp32, BIGMAC_FLAG_EXPERT_BIAS only */
    const float *b2;      /* [E,r] fp32, BIGMAC_FLAG_EXPERT_BIAS only */
} bigmac_weights_t;

/* Gradient buffers, same shapes and dtype as the weights; db_gate fp32 [E] or NULL. */
typedef struct {
    void *dw_gate;
    float *db_gate;
    void *dw_down, *dw1, *dw2, *dw_up;
    float *db1, *db2;     /* [E,h], [E,r] fp32, BIGMAC_FLAG_EXPERT_BIAS only (nullable) */
} bigmac_grads_t;

/* Routing tables.  Flat slot id s = t*k + j (j-th choice of token t).
 *   topk_idx[s]    expert of slot s, slots of a token in descending-logit order
 *   topk_w[s]      gate value p of slot s (fp32)
 *   counts[e]      rows routed to expert e;  offsets = exclusive prefix sum, offsets[E] = T*k
 *   row_of_slot[s] = offsets[e] + #{s' < s : topk_idx[s'] = e}  (stable counting sort by expert)
 *   slot_of_row    its inverse
 * With a capacity factor: counts[e] = kept rows = min(chosen, C), offsets[E] = all kept rows, row_of_slot[s] = -1
 * for a dropped slot, slot_of_row[row] = -1 for row >= offsets[E]; counts_chosen[e] = slots that chose e before
 * dropping (equal to counts without a capacity factor).
 *   aux_loss[0]    L_aux of this batch (fp32; 0 when aux_loss_coef = 0)
 * Any member may be NULL if the caller does not want that table. */
typedef struct {
    int32_t *topk_idx;      /* [T*k] */
    float *topk_w;          /* [T*k] */
    int32_t *counts;        /* [E]   */
    int32_t *offsets;       /* [E+1] */
    int32_t *row_of_slot;   /* [T*k] */
    int32_t *slot_of_row;   /* [T*k] */
    int32_t *counts_chosen; /* [E]   */
    float *aux_loss;        /* [1]   */
} bigmac_routing_t;

/* Validate the configuration and create a handle on the current CUDA device.  Allocates one small
 * device status word (no other device memory is owned by the handle), one stream and ten events.
 * Errors: INVALID_ARG (null pointers, non-positive sizes, k > E, unknown enums, a negative or non-finite
 * capacity_factor or aux_loss_coef), UNSUPPORTED (BF16
 * with d, r or h not a multiple of 64; E > 1024), CUDA. */
int bigmac_layer_create(const bigmac_config_t *cfg, bigmac_layer_t **out);
int bigmac_layer_destroy(bigmac_layer_t *L);

/* Bytes the caller must provide for a call with T tokens: `scratch_bytes` of scratch (contents
 * undefined before and after a call) and, for a training forward and its backward, `saved_bytes`
 * of saved state.  Both pointers must be 256-byte aligned.  training: 0 = inference forward,
 * 1 = training forward / backward. */
int bigmac_workspace_bytes(const bigmac_layer_t *L, int32_t T, int training, size_t *scratch_bytes,
                           size_t *saved_bytes);

/* Routing only: gate logits on x (text after Eq. 2), top-k, gate values, and the dispatch layout that
 * stands in for the first All-to-All (dropless).  x [T,d].  Integer tables have exactly one correct
 * value.  T = 0 is a no-op. */
int bigmac_route(bigmac_layer_t *L, const void *x, int32_t T, const bigmac_weights_t *W,
                 bigmac_routing_t *out, void *scratch, size_t scratch_bytes, void *stream);

/* Forward of Eq. 2 / Eq. 4: y [T,d] from x [T,d].  routing_out (nullable) receives the tables.
 * saved = NULL runs the inference forward; otherwise `saved` (saved_bytes of the training query)
 * receives what bigmac_backward needs. */
int bigmac_forward(bigmac_layer_t *L, const void *x, int32_t T, const bigmac_weights_t *W, void *y,
                   bigmac_routing_t *routing_out, void *saved, void *scratch, size_t scratch_bytes,
                   void *stream);

/* Backward of the same layer for an upstream gradient dy [T,d] (chain rule through Eq. 2 / Eq. 4):
 * dx [T,d] (through both the projections and the gate weights; the discrete top-k choice carries no
 * gradient) and every weight gradient in G (members may be NULL to skip one).  `x`, `W`, `T` and
 * `saved` must be those of the training forward.  accumulate = 0 overwrites the gradients (experts
 * that received no token get zeros), 1 adds to them.  `saved` may be modified. */
int bigmac_backward(bigmac_layer_t *L, const void *x, const void *dy, int32_t T, const bigmac_weights_t *W,
                    void *saved, void *dx, const bigmac_grads_t *G, int accumulate, void *scratch,
                    size_t scratch_bytes, void *stream);

/* Synchronise `stream` and return the device status word (BIGMAC_OK; BIGMAC_ERR_TIMEOUT if a
 * bounded wait inside a kernel ran out, in which case outputs of that call are undefined;
 * BIGMAC_ERR_STATE if bigmac_ep_dispatch found a count matrix that cannot be right - a negative entry or
 * more rows than an owner's buffers hold - in which case that step moved and computed nothing and no
 * memory outside the buffers was touched).  The word is cleared by the call. */
int bigmac_device_status(bigmac_layer_t *L, void *stream);

const char *bigmac_status_string(int status);

/* ---- Expert parallelism: the deployment the paper measures (Fig. 2c; Eq. 1 with the row width h replaced by
 * r h) ------------------------------------------------------------------------------------------------------
 * `size` ranks, one GPU each.  Every rank holds the shared matrices (w_gate, b_gate, w_down, w_up) in full and
 * E/size experts: rank q owns experts [q E/size, (q+1) E/size), and its w1 / w2 / dw1 / dw2 hold only those
 * ([E/size,h,r], [E/size,r,h]).  Every rank brings its own T tokens (T may differ between ranks).  The result is
 * that of ONE layer applied to all ranks' tokens together (rank 0's first, then rank 1's, ...).
 *
 * The two All-to-All exchanges of Fig. 2c are made by the ranks' own kernels over peer memory, at the low width
 * r: a rank PUTS the r-wide row x' of each of its slots straight into the segment of the owning rank's grouped
 * buffer, and later GETS the expert output u of that row from there (weighted by its gate value); the backward pass
 * puts du and gets dxg the same way.  Per rank and direction k T r (size-1)/size elements cross the links, against
 * k T d (size-1)/size for a layer that exchanges full-width rows (Eq. 1).  Rows land in the owner's local memory
 * first; its grouped GEMMs read only local memory.  No host-visible sizes, no device allocation, no stream
 * synchronisation inside the calls.
 *
 * Exchange buffers: four per rank (xg, u, du, dxg), bigmac_ep_buffer_bytes() each, caller-owned, 256-byte aligned,
 * and mapped into every rank's address space (peer access within a process, CUDA IPC or symmetric memory between
 * processes): entry [q] of each array below is rank q's buffer as THIS rank addresses it.  counts_all is local
 * memory, [size, E]: bigmac_ep_route writes this rank's row, the caller gathers the other ranks' rows into it (an
 * all-gather of E integers per rank) before bigmac_ep_dispatch.
 *
 * Order of calls on every rank, with a barrier over all ranks' streams wherever "|" stands (each call only
 * enqueues work on `stream`; the barrier must order that work, e.g. a collective on the same streams):
 *     route  | (all-gather of counts) dispatch | experts | combine            -> y
 *     backward_combine | backward_experts | backward_dispatch                -> dx, gradients
 * `saved` (and, across the three backward calls, `scratch`) must keep their contents between the calls of a step.
 * The gradients of the shared matrices that the backward returns are this rank's share (the sum over its own
 * tokens): the caller adds them over the ranks, as for any data-parallel layer; dw1 / dw2 are complete.
 * With BIGMAC_FLAG_CDAC the same calls run the conventional layer of Eq. 3 under expert parallelism: no shared
 * projections, the rows that travel are the tokens themselves at the full width d (Eq. 1 as written), w1 / w2 of the
 * owned experts are [E/size,h,d] / [E/size,d,h], w_down / w_up and their gradients are ignored.
 * Not supported together with a capacity factor, a load-balancing loss, BIGMAC_FLAG_GATE_LOW or
 * BIGMAC_FLAG_EXPERT_BIAS (BIGMAC_ERR_UNSUPPORTED). */
#define BIGMAC_EP_MAX_RANKS 8
typedef struct {
    int32_t rank, size;                 /* 0 <= rank < size <= BIGMAC_EP_MAX_RANKS, E % size == 0 */
    int32_t *counts_all;                /* [size, E] device memory of this rank */
    void *xg[BIGMAC_EP_MAX_RANKS];      /* rows x' received by rank q     [rows, r] */
    void *u[BIGMAC_EP_MAX_RANKS];       /* expert outputs of rank q       [rows, r] */
    void *du[BIGMAC_EP_MAX_RANKS];      /* gradients received by rank q   [rows, r] */
    void *dxg[BIGMAC_EP_MAX_RANKS];     /* input gradients of rank q      [rows, r] */
} bigmac_ep_t;

/* Bytes of ONE exchange buffer when no rank brings more than the handle's max_tokens tokens (worst case: every
 * slot of every rank is routed to this rank's experts). */
int bigmac_ep_buffer_bytes(const bigmac_layer_t *L, int32_t size, size_t *bytes);
/* Scratch and saved bytes of the expert-parallel calls (both 256-byte aligned, as for bigmac_workspace_bytes). */
int bigmac_ep_workspace_bytes(const bigmac_layer_t *L, int32_t T, int32_t size, size_t *scratch_bytes,
                              size_t *saved_bytes);
/* x' = x W'_down and the gate logits, top-k, gate values, this rank's slots sorted by expert; writes row `rank` of
 * ep->counts_all.  routing_out (nullable) receives this rank's local tables (counts / offsets / rows local). */
int bigmac_ep_route(bigmac_layer_t *L, const void *x, int32_t T, const bigmac_weights_t *W, const bigmac_ep_t *ep,
                    bigmac_routing_t *routing_out, void *saved, void *scratch, size_t scratch_bytes, void *stream);
/* Layout of every owner's segments from counts_all, zero fill of this rank's padding rows, first exchange: x' rows
 * of this rank's slots -> xg of the owners. */
int bigmac_ep_dispatch(bigmac_layer_t *L, int32_t T, const bigmac_ep_t *ep, void *saved, void *stream);
/* This rank's experts over the rows it received: u = sigma(xg W1_e^T) W2_e^T (Eq. 4).  W->w1 / w2: owned experts. */
int bigmac_ep_experts(bigmac_layer_t *L, const bigmac_weights_t *W, const bigmac_ep_t *ep, void *saved, void *stream);
/* Second exchange and the rest of Eq. 2: y' = sum_j p_j u[row of slot j at its owner], y = y' W'_up. */
int bigmac_ep_combine(bigmac_layer_t *L, int32_t T, const bigmac_weights_t *W, const bigmac_ep_t *ep, void *y,
                      void *saved, void *stream);
/* dy' = dy W_up, dW_up; per slot dp = <dy', u at its owner> (get) and du = p dy' -> du of the owner (put); gate
 * backward.  G members may be NULL. */
int bigmac_ep_backward_combine(bigmac_layer_t *L, const void *dy, int32_t T, const bigmac_weights_t *W,
                               const bigmac_ep_t *ep, const bigmac_grads_t *G, int accumulate, void *saved,
                               void *scratch, size_t scratch_bytes, void *stream);
/* This rank's experts, backward, over the rows it holds: dz, dW2, dxg, dW1 (G->dw1 / dw2: owned experts). */
int bigmac_ep_backward_experts(bigmac_layer_t *L, const bigmac_weights_t *W, const bigmac_ep_t *ep,
                               const bigmac_grads_t *G, int accumulate, void *saved, void *scratch,
                               size_t scratch_bytes, void *stream);
/* dx' = sum_j dxg[row of slot j at its owner] (get), dx, dW_down, dW_gate, db_gate (this rank's share). */
int bigmac_ep_backward_dispatch(bigmac_layer_t *L, const void *x, int32_t T, const bigmac_weights_t *W,
                                const bigmac_ep_t *ep, void *dx, const bigmac_grads_t *G, int accumulate,
                                void *saved, void *scratch, size_t scratch_bytes, void *stream);

/* bigmac_route for callers that cannot provide scratch memory.  (The paper has no counterpart: this is
 * a deployment variant of the routing step, not part of the method.)
 *
 * Who needs it: a host program that has handed all free device memory to its own pool, a latency-critical
 * loop that must not run into cudaMalloc's implicit device synchronisation, or a plug-in that is given
 * nothing but input and output pointers and has no allocator to ask.  Such callers cannot size and
 * allocate the `scratch` buffer that bigmac_route wants.  This entry point computes exactly the same tables
 * from the same inputs, but keeps its intermediates (gate logits, counting-sort counters, the internal
 * padded tables) in a fixed array of BIGMAC_STATIC_SCRATCH_BYTES that is part of the library image: every
 * GPU that loads the library holds that much memory until the process exits.
 *
 *  - It allocates nothing: no cudaMalloc / cudaFree, no allocating library routine.  The caller still passes
 *    x, the weights and the output tables (device memory, as for bigmac_route).
 *  - Limit: the routing intermediates of (T, E, k) must fit the array: about
 *    4*T*E + 24*T*k + 4*E*(T*k/1024) + 1.2 KB * E bytes, plus 4.8 KB * E with a load-balancing loss and T*r
 *    elements with BIGMAC_FLAG_GATE_LOW (the return code is the authority: the exact carve includes 256-byte
 *    alignment of every region); a larger problem is rejected with BIGMAC_ERR_TOO_LARGE and nothing is launched.
 *  - The first call on a device resolves the array's device address (once per device, with that device
 *    current) and keeps it for the later ones.
 *  - All calls share the one array, and it keeps the previous call's contents (everything a call reads it
 *    has written itself first).  Two calls that overlap on the GPU - different streams, or different
 *    handles - race on it: serialise them. */
#define BIGMAC_STATIC_SCRATCH_BYTES (8u << 20)
int bigmac_route_static(bigmac_layer_t *L, const void *x, int32_t T, const bigmac_weights_t *W,
                        bigmac_routing_t *out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* BIGMAC_H_ */
