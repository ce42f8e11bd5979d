/* pop_kernels.h - kernel-level entry points of the POP prefill library (C ABI).
 *
 * Each call runs ONE step of the path declared in pop.h on caller-owned device buffers, so that
 * every kernel can be checked against the oracle's statement of the same step and timed alone.
 * Conventions are those of pop.h: device pointers are borrowed, `stream` is a cudaStream_t, calls
 * are asynchronous, the return value is a pop_status, and an error enqueues nothing.
 */
#ifndef POP_KERNELS_H_
#define POP_KERNELS_H_

#include "pop.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Projection GEMM of a decoder layer (paper Eq. 1-2: the "x W" products), batched:
 *   D[g][m][n] = sum_k A[g][m][k] * B[g][n][k],  g < batch, bf16 operands, fp32 accumulation.
 * A: device bf16, row stride lda, batch stride a_bs (elements; 0 = densely packed); B likewise.
 * epilogue: 0 store bf16, 1 store fp32, 2 fp32 out += D (residual add of Eq. 1),
 *           3 gated FFN: rows of B come in blocks of 256 (128 gate rows, then the 128 matching up
 *             rows), out bf16 column f = act(gate_f) * up_f for f < n_valid (act 0 SiLU, 1 tanh-GELU).
 * out: row stride ldo, batch stride o_bs, in elements of the output type.
 * Requires K, lda, ldb multiples of 8, 16-byte aligned pointers, N a multiple of 8 (256 for epilogue 3). */
int pop_k_gemm(const void* A, int64_t lda, int64_t a_bs, const void* B, int64_t ldb, int64_t b_bs, void* out,
               int64_t ldo, int64_t o_bs, int32_t M, int32_t N, int32_t K, int32_t batch, int32_t epilogue,
               int32_t act, int32_t n_valid, void* stream);

/* Synchronise the stream, then read and clear the library's device status word. */
int pop_k_status(void* stream);

/* Kernel launches enqueued by this library since the last pop_k_reset_launch_count(). */
int64_t pop_k_launch_count(void);
void pop_k_reset_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* POP_KERNELS_H_ */
