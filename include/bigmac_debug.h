/* bigmac_debug.h - unit-test entry point of libbigmac: run ONE contraction of the layer in isolation.
 * Not needed to use the layer.  The paper has no counterpart; the contractions it implies are the
 * matrix products of Eq. 2 and Eq. 4 and of their chain-rule gradients.
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

#ifdef __cplusplus
}
#endif
#endif /* BIGMAC_DEBUG_H_ */
