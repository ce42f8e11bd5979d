// Shared host/device declarations of the POP prefill library (internal).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/pop.h"

namespace pop {

typedef __nv_bfloat16 bf16;

// Device status word shared by all kernels of the library (file-scope in status.cu). Kernels
// raise it with atomicMin to a negative pop_status; pop_last_status reads and clears it.
int* status_word();                 // device address, valid for the current device
int read_and_clear_status(cudaStream_t s);

// Launch counter (host side): every kernel launch of the library goes through count_launch().
void count_launch();
int64_t launch_count();
void reset_launch_count();

// Tensor-map encoding through the driver entry point (no link-time dependency on libcuda).
// 3-D bf16 tensor [dim2][dim1][dim0] with dim0 contiguous; strides in elements; 128-byte swizzle;
// box = [1][box1][box0]; box0 must be 64 (128 bytes).
int make_tmap_bf16_3d(CUtensorMap* out, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                      uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box0, uint32_t box1);
// 5-D bf16 tensor, used for the paged KV pools [layer][page][slot][head][hd].
int make_tmap_bf16_5d(CUtensorMap* out, const void* base, const uint64_t dims[5], const uint64_t strides_elems[4],
                      const uint32_t box[5]);

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ------------------------------------------------------------------------------------ GEMM
// D[g][m][n] = sum_k A[g][m][k] * B[g][n][k]   (bf16 operands, fp32 accumulation on tcgen05)
enum GemmEpilogue {
  EPI_STORE_BF16 = 0,   // out bf16 [M][ldo]
  EPI_STORE_F32 = 1,    // out fp32 [M][ldo]
  EPI_ADD_F32 = 2,      // out fp32 [M][ldo] += D  (residual add)
  EPI_GATED_BF16 = 3    // B rows come in blocks of 256: 128 gate rows then the matching 128 up rows;
                        // out bf16 [M][ldo], column f = act(gate_f) * up_f, for f < n_valid
};
struct GemmArgs {
  const bf16* A; int64_t lda; int64_t a_batch_stride;   // elements
  const bf16* B; int64_t ldb; int64_t b_batch_stride;
  void* out; int64_t ldo; int64_t out_batch_stride;     // elements of the output type
  int M, N, K, batch;
  int epilogue;
  int act;          // EPI_GATED_BF16: 0 SiLU, 1 tanh-GELU
  int n_valid;      // EPI_GATED_BF16: number of valid output columns (d_ffn); others: ignored
};
int launch_gemm(const GemmArgs& a, cudaStream_t stream);

}  // namespace pop
