// Internal declarations shared by the translation units of libbigmac (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "bigmac.h"
#include "switches.h"

namespace bigmac {

// Chained launches.  A kernel launched through launch_chained may be set up (its CTAs placed, their prologue run)
// while the kernel before it in the stream is still running; it must call grid_dependency_wait() before it reads
// or writes any global memory - that call returns once the predecessor has completed and its writes are visible.
// grid_dependency_launch() lets the successor's set-up begin; a kernel that allocates tensor memory calls it only
// after its allocation (a successor's CTA on the same SM could otherwise take the columns first and then wait for
// this kernel for ever).  Launched plainly, both calls do nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = switches().chain ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

constexpr int kPad = 128;          // expert segments are padded to multiples of this many rows internally
constexpr int kMaxExperts = 1024;

// ---------------------------------------------------------------------------------------------
// GEMM request:  C[m,n] (+)= epilogue( sum_k A(m,k) * B(n,k) )
//   a_kmajor: A(m,k) = A[m*lda + k], else A[k*lda + m].   b_kmajor: B(n,k) = B[n*ldb + k], else B[k*ldb + n].
//   C is row-major [M, ldc].
// Grouping (the experts' variable-length row segments, padded to kPad rows; tables live on the device):
//   GROUP_NONE  one dense problem.
//   GROUP_M     rows of A and C are the padded grouped rows; row tile i (kPad rows) belongs to expert
//               tile_expert[i] (only the first *n_tiles tiles exist); B of expert e starts at B + e*b_stride.
//   GROUP_K     one problem per expert e with the contraction running over its padded rows
//               [poffsets[e], poffsets[e+1]) of A and B; C of expert e starts at C + e*c_stride.
// ---------------------------------------------------------------------------------------------
enum GroupMode { GROUP_NONE = 0, GROUP_M = 1, GROUP_K = 2 };
enum Epilogue {
    EPI_NONE = 0,   // C = acc
    EPI_ACT = 1,    // Z = sigma'(acc) (if Z != nullptr), C = sigma(acc)
    EPI_DACT = 2,   // C = acc * Z[m,n]               (Z holds sigma'(z) from the forward; C may alias Z)
};

struct GemmArgs {
    const void* A = nullptr; const void* B = nullptr; void* C = nullptr;
    void* Z = nullptr;                  // sigma'(z), [M, ldc] like C, element type = input dtype
    int64_t lda = 0, ldb = 0, ldc = 0;
    int M = 0, N = 0, K = 0;            // GROUP_M: M = upper bound on padded rows; GROUP_K: K = row extent of A and B
    bool a_kmajor = true, b_kmajor = true;
    bool out_f32 = false;               // C is fp32 regardless of the input dtype
    bool accumulate = false;            // C += result
    int epilogue = EPI_NONE;
    int act = 0;
    int group = GROUP_NONE;
    int num_experts = 0;
    int64_t b_stride = 0, c_stride = 0; // elements
    const int32_t* tile_expert = nullptr;
    const int32_t* n_tiles = nullptr;
    const int32_t* poffsets = nullptr;
    // Tensor-core path only, dense problems only:
    const void* B2 = nullptr;           // second MN-major B: contraction rows k >= b2_first_k read B2[(k - b2_first_k)*ldb2 + n]
    int64_t ldb2 = 0;
    int b2_first_k = 0;                 // multiple of 64
    // ... or, with K-major B: output columns n >= n_split use rows of B2 (n - n_split) and are written as fp32 to
    // C2[m*ldc2 + n - n_split] for n - n_split < N2 (n_split a multiple of the tile width; N = n_split + N2).
    int n_split = -1;
    float* C2 = nullptr;
    int64_t ldc2 = 0;
    int N2 = 0;
    int split_k = 1;                    // > 1: part s of the contraction writes its partial result (fp32) to C + s*M*ldc
    int force_kernel = 0;               // measurement aid: 1 = one-CTA kernel, 2 = CTA-pair kernel, 0 = default choice
    int epi_parts = 0;                  // measurement aid: epilogue warps per lane quadrant that work (1, 2 or 4); 0 = default choice
    // Tensor-core path, GROUP_M with K-major A: the rows of A are gathered (the dispatch fused into the operand load):
    // row m of A is row gather_rows[m] / gather_div of A itself (which then is the ungrouped matrix, lda its row
    // stride), zeros where gather_rows[m] < 0.  Null: A holds the grouped rows.
    const int32_t* gather_rows = nullptr;
    int gather_div = 1;
    // GROUP_M only: fp32 bias added to the accumulator before the epilogue, column n of a row of expert e gets
    // bias[e*bias_stride + n] (16-byte aligned, bias_stride a multiple of 4)
    const float* bias = nullptr;
    int64_t bias_stride = 0;
};

// fp32-FMA GEMM for either dtype (dtype: bigmac_dtype_t of A, B, Z and - unless out_f32 - C).
cudaError_t gemm_simt(const GemmArgs& g, int dtype, cudaStream_t stream);
// tcgen05 / TMEM / TMA GEMM, bf16 inputs, fp32 accumulation.  `status` is the device status word.
cudaError_t gemm_tc(const GemmArgs& g, int* status, cudaStream_t stream);
bool gemm_tc_available();
// Per-expert weight-gradient contraction (GROUP_K, both operands MN-major, bf16 output) with dynamically scheduled
// work items and long experts cut into parts (gemm_tc_groupk.cu).  ws: gemm_tc_groupk_ws_bytes() bytes, 256-byte
// aligned; sched: two device ints that are zero between launches (the kernel leaves them so).
constexpr int kGroupKSlots = 32;
bool gemm_tc_groupk_supported(const GemmArgs& g);
size_t gemm_tc_groupk_ws_bytes(int M, int N, int E);
cudaError_t gemm_tc_groupk(const GemmArgs& g, int* status, int* sched, void* ws, cudaStream_t stream);
cudaError_t gemm_tc_groupk_finish(const GemmArgs& g, void* ws, cudaStream_t stream);   // always after gemm_tc_groupk
// Inference forward of the experts in one kernel for r <= 256 (gemm_tc_mlp.cu): u = sigma(xg W1_e^T) W2_e^T per
// 128-row tile, hidden activations kept on the SM.
bool fused_mlp_supported(int r, int h, int dtype);
cudaError_t launch_fused_mlp(const void* xg, const void* w1, const void* w2, void* u, int64_t max_rows, int r, int h, int E,
                             int act, const int32_t* tile_expert, const int32_t* n_tiles, int* status, cudaStream_t stream);
// CTA-pair variant (tcgen05 cta_group::2) for outputs at least 256 wide.
bool gemm_tc_pair_supported(const GemmArgs& g);
bool gemm_tc_pair_preferred(const GemmArgs& g);
cudaError_t gemm_tc_pair(const GemmArgs& g, int* status, cudaStream_t stream);
int gemm_tc_sm_count();
// Test aid: a one-thread kernel whose bounded barrier wait runs out after a short limit and records it in `status`.
cudaError_t launch_expire_wait(int* status, cudaStream_t stream);

// ---------------------------------------------------------------------------------------------
// Routing tables held in device memory (internal superset of bigmac_routing_t).
// ---------------------------------------------------------------------------------------------
struct Tables {
    int32_t* topk_idx;      // [N]
    float* topk_w;          // [N]
    int32_t* counts;        // [E]
    int32_t* offsets;       // [E+1]   canonical (unpadded)
    int32_t* poffsets;      // [E+1]   padded to kPad
    int32_t* row_of_slot;   // [N]     canonical
    int32_t* slot_of_row;   // [N]
    int32_t* prow_of_slot;  // [N]     row in the padded grouped buffers
    int32_t* slot_of_prow;  // [P]     -1 on padding rows
    int32_t* tile_expert;   // [P/kPad]
    int32_t* n_tiles;       // [1]     number of kPad-row tiles in use
    int32_t* block_counts;  // [n_blocks, E] scratch of the counting sort
    int32_t* counts_chosen; // [E]     slots that chose the expert, before any dropping (nullable)
};

// Per-device one-time launch configuration (function attributes are per device; a process may use several).
struct PerDeviceOnce {
    unsigned long long done = 0;           // bit d: configured on device d (d < 64)
    // true if `fn` still has to run on the current device
    bool needed(int* device_out) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *device_out = -1; return true; }
        *device_out = dev;
        return !((done >> dev) & 1ull);
    }
    void mark(int dev) { if (dev >= 0) done |= 1ull << dev; }
};

inline int64_t padded_rows_max(int64_t N, int E) { return ((N + kPad - 1) / kPad + E) * (int64_t)kPad; }
constexpr int kSortChunk = 1024;   // slots per block of the counting sort
inline int sort_blocks(int64_t N) { return (int)((N + kSortChunk - 1) / kSortChunk); }

// logits [T,E] fp32 (+ b_gate) -> topk_idx, topk_w.
cudaError_t launch_topk(const float* logits, const float* b_gate, int T, int E, int k, int32_t* topk_idx,
                        float* topk_w, cudaStream_t stream);
// topk_idx -> every other table (deterministic stable counting sort of slots by expert).  `cap`: rows an expert
// keeps at most (the capacity of Table 5's capacity factor; kNoCapacity = dropless); a slot whose rank among the
// slots of its expert is cap or more gets row_of_slot = prow_of_slot = -1, counts / offsets describe kept rows.
constexpr int kNoCapacity = 0x7fffffff;
// Few slots and experts: one single-block kernel does the whole sort; else three passes (and a fill).  Measured with
// per-stage events (E = 64): 512 slots 10.6 us against 20.7 us, 4096 slots 19.4 against 20.4: the limit is where it pays.
constexpr int kSmallTablesMaxSlots = 2048, kSmallTablesMaxExperts = 256;
inline int tables_kernel_count(int64_t N, int E) {
    return (N > 0 && N <= kSmallTablesMaxSlots && E <= kSmallTablesMaxExperts) ? 1 : 3;
}
// `status` (nullable): the handle's status word; an expert id outside [0, E) - which the top-k kernels never write -
// is placed nowhere (row -1) and recorded there as 2.
cudaError_t launch_tables(const Tables& tb, int T, int E, int k, int cap, cudaStream_t stream, int* status = nullptr);

// Row moves.  `width` elements of the dtype per row; all row pointers 16-byte aligned.
// grouped[prow,:] = src[slot_of_prow[prow]/k,:], zeros on padding rows, for prow < n_tiles*kPad.
cudaError_t launch_dispatch(const void* src, void* grouped, const Tables& tb, int k, int width, int dtype,
                            int64_t max_prows, cudaStream_t stream);
// dst[t,:] = sum_j w[t*k+j] * grouped[prow_of_slot[t*k+j],:]   (w == nullptr: unit weights), fp32 accumulation;
// with may_drop, slots with prow_of_slot < 0 (dropped under a capacity limit) are left out of the sum.
// dst rows are `dst_ld` elements apart (0: dense, = width).
cudaError_t launch_combine(const void* grouped, void* dst, const float* w, const int32_t* prow_of_slot, int T,
                           int k, int width, int dtype, cudaStream_t stream, int dst_ld = 0, bool may_drop = false);
// Backward of the combine: du[prow,:] = p[s] * dy_lo[t,:] (zeros on padding), dp[s] = <dy_lo[t,:], u[prow,:]>.
cudaError_t launch_combine_bwd(const void* dy_lo, const void* u, void* du, float* dp, const Tables& tb, int k,
                               int width, int dtype, int64_t max_prows, cudaStream_t stream);
// Softmax-over-k backward: g = sum_i p_i dp_i, dl_j = p_j (dp_j - g); writes the dense [T,E] matrix
// (zeros off the top-k set, and in the padding columns E..width-1) in the dtype, rows `ld` elements apart, and
// leaves the fp32 dl_j in dp[slot].
cudaError_t launch_gate_bwd(float* dp, const Tables& tb, void* dlogits, int T, int E, int width, int ld, int k,
                            int dtype, cudaStream_t stream);
// Load-balancing loss (Table 5; conventional form, the paper prints none):
//   L_aux = coef * E * sum_e f_e P_e,  f_e = counts_chosen[e] / (T k),  P_e = mean_t softmax_E(logits[t,:] + b_gate)[e].
// Forward: loss[0] = L_aux; `partial` holds kAuxChunks * E floats of scratch.  Deterministic summation order.
constexpr int kAuxChunks = 1184;
cudaError_t launch_aux_loss(const float* logits, const float* b_gate, const int32_t* counts_chosen, int T, int E, int k,
                            float coef, float* partial, float* loss, cudaStream_t stream);
// launch_gate_bwd plus dL_aux/dl: dlogits[t,e] = (top-k part) + (coef E / T) p[t,e] (f_e - sum_j f_j p[t,j]); the
// column sums of the second term go to aux_partial [kAuxChunks, E] for launch_gate_colsum.
cudaError_t launch_gate_bwd_aux(float* dp, const Tables& tb, void* dlogits, const float* logits, const float* b_gate,
                                float coef, float* aux_partial, int T, int E, int width, int ld, int k, int dtype,
                                cudaStream_t stream);
// db[e] (+)= sum over the slots routed to e of dl_slot[slot] (the fp32 per-slot gate gradients launch_gate_bwd
// leaves in dp); `partial` holds kColsumChunks * E floats of scratch.  Deterministic summation order.
constexpr int kColsumChunks = 296;
// aux_partial (nullable): a second array, [kAuxChunks, E], of partial column sums added in (launch_gate_bwd_aux).
cudaError_t launch_gate_colsum(const float* dl_slot, const Tables& tb, float* db, float* partial, int64_t N, int E,
                               bool accumulate, cudaStream_t stream, const float* aux_partial = nullptr);
// Per-expert column sums of a grouped matrix (the expert-bias gradients): out[e, c] (+)= sum over the padded rows of
// expert e of src[row, c] (padding rows hold zeros), fp32, fixed summation order.  width a multiple of 8 (bf16) / 4;
// partial: E * kColsumSlices * width floats of scratch.
constexpr int kColsumSlices = 32;
cudaError_t launch_grouped_colsum(const void* src, const int32_t* poffsets, float* out, float* partial, int E, int width,
                                  int dtype, bool accumulate, cudaStream_t stream);
// Sum the `parts` fp32 partial results ws[s][m][n] of a split contraction in the order s = 0, 1, ... and write
// rows [0, m_split) to dst1 [m_split, N] and rows [m_split, m_split + m2) to dst2 [m2, N] (dst2 may be null),
// in the dtype, adding to the destination if `accumulate`.
cudaError_t launch_splitk_reduce(const float* ws, int parts, int M, int N, void* dst1, int m_split, void* dst2, int m2,
                                 int dtype, bool accumulate, cudaStream_t stream);
// [x' (bf16) | logits (fp32)] from the [parts][T][r + E] fp32 partial results of a split descend launch (r, E % 4 == 0).
cudaError_t launch_descend_reduce(const float* ws, int parts, int T, int r, int E, void* x_lo, float* logits,
                                  cudaStream_t stream);

// Small-batch inference forward in one cooperative kernel (bf16, T <= 16): scratch logits [T,E], x_lo [T,r],
// a [T*k,h], u [T*k,r] fp32; writes y, topk_idx, topk_w.  `barrier` is one device word owned by the handle.
bool decode_forward_supported(int T, int d, int r, int h, int E, int k, int dtype);
cudaError_t launch_decode_forward(const void* x, const bigmac_weights_t* W, void* y, float* logits, float* x_lo, float* a,
                                  float* u, int32_t* topk_idx, float* topk_w, unsigned* barrier, int* status, int T, int d,
                                  int r, int h, int E, int k, int act, int num_sms, cudaStream_t stream);

}  // namespace bigmac
