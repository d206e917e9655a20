/* bigmac_debug.h - measurement, unit-test and debugging aids of libbigmac.  Not needed to use the layer and not part
 * of its interface (bigmac.h): run ONE contraction in isolation, run the exchange kernels at any row width, time
 * the stages of a call, switch kernel choices, make a bounded wait run out.  The paper has no counterpart; the
 * contractions it implies are the matrix products of Eq. 2 and Eq. 4 and of their chain-rule gradients.
 *
 * bigmac_debug_gemm:
 *
 *   C[m,n] (+)= epilogue( sum_k A(m,k) * B(n,k) ),  fp32 accumulation
 *   a_kmajor: A(m,k) = A[m*lda + k], else A[k*lda + m];  b_kmajor: B(n,k) = B[n*ldb + k], else B[k*ldb + n].
 *   group 0: dense.  group 1: rows are expert-grouped segments padded to 128 rows, row tile i belongs to
 *   expert tile_expert[i], only *n_tiles tiles exist, B of expert e at B + e*b_stride.  group 2: one
 *   problem per expert with k running over rows [poffsets[e], poffsets[e+1]), C of expert e at C + e*c_stride.
 *   epilogue 0: none; 1: Z = sigma'(acc) (if Z), C = sigma(acc); 2: C = acc * Z.  On the tensor-core kernels Z holds
 *   sigma' as one byte per element, q = round(200 sigma' + 27); on the plain FMA kernel Z has the layer's dtype.
 * All pointers are device memory (tables included), 16-byte aligned.  use_tensor_cores: 0 = plain FMA kernel,
 * 1 = tensor cores (default kernel choice), 2 = force the one-CTA kernel, 3 / 4 / 5 = force the CTA-pair kernel with
 * four / two / one working epilogue warps per lane quadrant (plain epilogues only; the default choice is two);
 * non-zero values require a BF16 handle.  Returns a bigmac_status_t.
 */
#ifndef BIGMAC_DEBUG_H_
#define BIGMAC_DEBUG_H_
#include "bigmac.h"
#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    const void *A, *B;
    void *C, *Z;
    int64_t lda, ldb, ldc;
    int32_t M, N, K;
    int32_t a_kmajor, b_kmajor, out_f32, accumulate, epilogue, act, group, num_experts;
    int64_t b_stride, c_stride;
    const int32_t *tile_expert, *n_tiles, *poffsets;
} bigmac_debug_gemm_t;

int bigmac_debug_gemm(bigmac_layer_t *L, const bigmac_debug_gemm_t *q, int use_tensor_cores, void *stream);

/* Test aid for the failure path of the device-side waits: launches a one-thread kernel that waits, with the same
 * bounded wait the TMA / MMA pipelines use but a limit of 4096 polls, on a barrier nobody arrives at.  The wait runs
 * out, the kernel records it in the handle's status word and returns normally (no trap, no fault): the next
 * bigmac_device_status returns BIGMAC_ERR_TIMEOUT and the handle and the context stay usable. */
int bigmac_debug_expire_wait(bigmac_layer_t *L, void *stream);

/* Measurement aid for the dispatch/combine stage (Eq. 1: bytes through the exchange are proportional
 * to the row width): run the standalone dispatch and combine kernels on rows of `width` elements of
 * the layer's dtype.  width = r is BigMac's exchange; width = d is what a fine-grained layer of equal
 * E and k moves.  src [T,width] -> grouped [rows_padded,width] -> dst [T,width] with the gate values
 * of the routing held in `saved` (from a training forward of the same T).  which: 0 = dispatch only,
 * 1 = combine only (grouped must hold data), 2 = both. */
int bigmac_exchange_rows(bigmac_layer_t *L, const void *saved, int32_t T, int32_t width, const void *src,
                         void *grouped, size_t grouped_bytes, void *dst, int which, void *stream);

/* Measurement aid: per-stage device timing and a launch counter.  While enabled, every kernel the
 * library launches is bracketed by a pair of CUDA events on the caller's stream (no synchronisation) and
 * counted.  bigmac_profile_read synchronises `stream`, adds the elapsed time of every bracket recorded
 * since the last read to its stage's slot and returns the totals; the bracket pool holds 8192 launches
 * between reads, later ones are counted in `dropped` and not timed.  The paper has no counterpart. */
#define BIGMAC_PROFILE_SLOTS 32
typedef struct {
    uint64_t launches;                      /* kernels launched since enable */
    uint32_t dropped;                       /* launches not timed because the pool was full */
    int32_t n_slots;                        /* slots in use */
    float ms[BIGMAC_PROFILE_SLOTS];         /* summed device time per stage */
    uint32_t calls[BIGMAC_PROFILE_SLOTS];   /* launches per stage */
} bigmac_profile_t;
int bigmac_profile_enable(bigmac_layer_t *L, int on);
int bigmac_profile_read(bigmac_layer_t *L, void *stream, bigmac_profile_t *out);
const char *bigmac_profile_slot_name(int slot);

/* Process-wide switches for A/B measurements and for isolating a kernel in a test.  The defaults are the product;
 * nothing but this call changes them (the library reads no environment variable).  Not thread-safe against running
 * calls: set switches between calls.
 *   "overlap" 0/1        backward pass on one stream / independent launches on the handle's second stream (default 1)
 *   "tc_pair" 0/1        never / where faster: the CTA-pair tcgen05 kernel (default 1)
 *   "groupk" 0/1         never / where it pays: the dynamically scheduled per-expert weight-gradient kernel (default 1)
 *   "fused_mlp" 0/1/2    inference expert GEMM1 + sigma + GEMM2 in one kernel never / on short tile lists / always (default 1)
 *   "epi_parts" 0/1/2/4  working epilogue warps per lane quadrant of plain epilogues (0 = default choice, 2)
 *   "chain" 0/1          kernels launched with programmatic stream serialisation (set-up overlaps the predecessor) (default 1)
 *   "staged_stores" 0/1  wide bf16 outputs by 32-byte direct stores / through shared-memory boxes and TMA stores (default 1)
 *   "fuse_dispatch" 0/1  standalone dispatch kernel / the dispatch fused into its consumers: expert GEMM1 and the weight
 *                        gradient dW1 gather the rows of x' themselves, no grouped copy is written (default 0: measured slower)
 *   "tc_mask" bits       bit i: contraction i runs on tcgen05, else on the FMA kernel; read when a handle is created
 *   "defaults"           every switch back to its default (value ignored)
 * Returns BIGMAC_ERR_INVALID_ARG for an unknown name. */
int bigmac_debug_set(const char *name, int value);

#ifdef __cplusplus
}
#endif
#endif /* BIGMAC_DEBUG_H_ */
