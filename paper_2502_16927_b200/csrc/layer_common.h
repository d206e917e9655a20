// Pieces of the layer's host code shared by its translation units (layer.cu: the one-GPU entry points; ep.cu: the
// expert-parallel ones): the handle, the stage ids, launch accounting, workspace carving and the GEMM front door.
#pragma once
#include <cstdlib>
#include <cstring>
#include <vector>

#include "internal.h"
#include "bigmac_debug.h"

struct bigmac_layer {
    bigmac_config_t cfg;
    int device;
    int* status;        // device status word; status[1] is the grid-barrier counter of the small-batch kernel,
                        // status[2..3] the work counters of the per-expert weight-gradient kernel (zero at rest)
    bool use_tc;        // bf16 contractions on tcgen05
    unsigned tc_mask;   // debug: bit i set = contraction i runs on tcgen05 (the tc_mask switch at creation)
    // second stream of the backward pass (created on first use): launches that do not depend on each other and lean
    // on different units (a tensor-bound weight gradient beside an HBM-bound row move) run side by side
    cudaStream_t side = nullptr;
    cudaEvent_t fork_join[10] = {};     // [9]: joins the second stream back when a call fails after its fork
    bool side_forked = false;          // the running bigmac_backward has put work on `side`
    // measurement aid
    bool prof_on = false;
    uint64_t launches = 0;
    uint32_t dropped = 0;
    std::vector<cudaEvent_t> ev;       // pool of start/stop pairs
    std::vector<int> ev_slot;          // stage of each recorded pair
    float ms[BIGMAC_PROFILE_SLOTS] = {};
    uint32_t calls[BIGMAC_PROFILE_SLOTS] = {};
};

namespace bigmac {
namespace detail {

// Contraction ids (bits of tc_mask).
enum { G_LOGITS = 0, G_DESCEND, G_EXPERT1, G_EXPERT2, G_ASCEND, G_DY_LO, G_DW_UP, G_DZ, G_DW2, G_DXG, G_DW1,
       G_DX, G_DX_GATE, G_DW_DOWN, G_DW_GATE,
       S_TOPK, S_TABLES, S_DISPATCH, S_COMBINE, S_COMBINE_BWD, S_GATE_BWD, S_DXLO_GATHER, S_COLSUM, S_SPLITK_REDUCE,
       S_DECODE, S_FUSED_MLP, S_AUX_LOSS, S_COUNT };
const char* const kSlotNames[S_COUNT] = {
    "gemm_logits", "gemm_descend", "gemm_expert1", "gemm_expert2", "gemm_ascend", "gemm_dy_lo", "gemm_dw_up",
    "gemm_dz", "gemm_dw2", "gemm_dxg", "gemm_dw1", "gemm_dx", "gemm_dx_gate", "gemm_dw_down", "gemm_dw_gate",
    "topk", "tables", "dispatch", "combine", "combine_bwd", "gate_bwd", "dxlo_gather", "colsum",
    "splitk_reduce", "decode_forward", "fused_expert_mlp", "aux_loss"};
constexpr size_t kEventPairs = 8192;
constexpr int kMaxSplitK = 8;

// Counts the launches of one stage and, while profiling, brackets them with an event pair.
struct Stage {
    bigmac_layer* L;
    cudaStream_t st;
    cudaEvent_t stop = nullptr;
    Stage(const bigmac_layer* layer, int slot, cudaStream_t stream, int kernels = 1)
        : L(const_cast<bigmac_layer*>(layer)), st(stream) {
        L->launches += kernels;
        if (!L->prof_on) return;
        const size_t i = L->ev_slot.size();
        if (i >= kEventPairs) { L->dropped += kernels; return; }
        L->ev_slot.push_back(slot);
        L->calls[slot] += kernels;
        cudaEventRecord(L->ev[2 * i], st);
        stop = L->ev[2 * i + 1];
    }
    ~Stage() { if (stop) cudaEventRecord(stop, st); }
};

inline size_t esize(int dtype) { return dtype == BIGMAC_BF16 ? 2 : 4; }

// Hands out 256-byte-aligned regions of one buffer; with base == nullptr it only measures.
struct Carver {
    char* base;
    size_t used = 0;
    explicit Carver(void* b) : base((char*)b) {}
    template <typename T> T* take(size_t count) {
        used = (used + 255) & ~(size_t)255;
        T* p = base ? (T*)(base + used) : nullptr;
        used += count * sizeof(T);
        return p;
    }
    void* take_bytes(size_t bytes) { return take<char>(bytes); }
    size_t total() const { return (used + 255) & ~(size_t)255; }
};


inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p & (a - 1)) == 0; }
// The tensor-core kernels save sigma' as one byte per element; that needs expert GEMM1 and dz on the same side.
inline bool sigma_as_bytes(const bigmac_layer* L) { return L->cfg.dtype == BIGMAC_BF16 && L->use_tc && L->tc_mask == ~0u; }

// One contraction on the path the handle selects (tcgen05 or fp32 FMA), counted and timed as stage `id`.
int gemm(const bigmac_layer* L, int id, const GemmArgs& g, cudaStream_t st);
// Parts to cut a dense contraction over K into so that tiles * parts fills the SMs.
int choose_split_k(int M, int N, int K);
// Per-expert weight gradient (contraction over the expert's rows); splitk_ws: the fp32 workspace of the handle's call.
int expert_weight_grad(const bigmac_layer* L, int id, const GemmArgs& g, float* splitk_ws, cudaStream_t st);
int check_call(const bigmac_layer* L, int32_t T);

#define BIGMAC_TRY(expr)                        \
    do {                                        \
        int _s = (expr);                        \
        if (_s != BIGMAC_OK) return _s;         \
    } while (0)
#define BIGMAC_CUDA(expr)                                   \
    do {                                                    \
        if ((expr) != cudaSuccess) return BIGMAC_ERR_CUDA;  \
    } while (0)


}  // namespace detail
}  // namespace bigmac
