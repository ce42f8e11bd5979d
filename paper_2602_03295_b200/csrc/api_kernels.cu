// C-ABI wrappers for the kernel-level entry points declared in pop_kernels.h.
#include "common.cuh"
#include "../../include/pop_kernels.h"

using namespace pop;

extern "C" {

int pop_k_gemm(const void* A, int64_t lda, int64_t a_bs, const void* B, int64_t ldb, int64_t b_bs, void* out,
               int64_t ldo, int64_t o_bs, int32_t M, int32_t N, int32_t K, int32_t batch, int32_t epilogue,
               int32_t act, int32_t n_valid, void* stream) {
  GemmArgs a;
  a.A = static_cast<const bf16*>(A); a.lda = lda; a.a_batch_stride = a_bs;
  a.B = static_cast<const bf16*>(B); a.ldb = ldb; a.b_batch_stride = b_bs;
  a.out = out; a.ldo = ldo; a.out_batch_stride = o_bs;
  a.M = M; a.N = N; a.K = K; a.batch = batch;
  a.epilogue = epilogue; a.act = act; a.n_valid = n_valid;
  return launch_gemm(a, static_cast<cudaStream_t>(stream));
}

const char* pop_strerror(int status) {
  switch (status) {
    case POP_OK: return "ok";
    case POP_E_INVALID: return "invalid argument";
    case POP_E_NOSPACE: return "buffer too small";
    case POP_E_CUDA: return "CUDA call failed";
    case POP_E_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case POP_E_MISSING: return "a required tensor is missing";
  }
  return "unknown status";
}

int pop_k_status(void* stream) { return read_and_clear_status(static_cast<cudaStream_t>(stream)); }
int64_t pop_k_launch_count(void) { return launch_count(); }
void pop_k_reset_launch_count(void) { reset_launch_count(); }

}  // extern "C"
