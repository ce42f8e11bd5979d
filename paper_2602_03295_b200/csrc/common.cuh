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

// Optional per-kernel timing: when enabled, every launch wrapper brackets its kernel with CUDA
// events on the launching stream; prof_summary() synchronises them and sums by kind.
enum ProfKind { PROF_GEMM = 0, PROF_ATTENTION = 1, PROF_ELEMENTWISE = 2, PROF_GEMV = 3, PROF_DECODE_ATTN = 4,
                PROF_KINDS = 5 };
void prof_enable(bool on);
bool prof_enabled();
struct ProfScope {   // records the start event on construction, the end event on destruction
  ProfScope(int kind, double work, cudaStream_t s);
  ~ProfScope();
  int kind; double work; cudaStream_t stream; cudaEvent_t e0, e1; bool active;
};
int prof_summary(int kind, double* total_ms, double* total_work, int64_t* launches);   // clears that kind

// Chained launches of the single-row (boundary token / decode) kernels. A kernel launched with
// launch_chained may become resident while the kernel before it on the stream is still running;
// it calls chain_trigger() at its top (its own successor may then be made resident) and
// chain_wait() before it reads anything an earlier kernel wrote and before it writes anything:
// chain_wait() returns when the preceding kernel has completed and its writes are visible. Every
// kernel of a chain waits, so completion is transitive. Before the wait a kernel touches only data
// that no kernel ever writes (weights, gains, block tables). A kernel launched the ordinary way
// after a chained one is ordered after it as usual. POP_CHAINED_LAUNCH=0 in the environment turns
// the early residency off (the kernels then run strictly one after the other).
bool chained_launch_enabled();
#ifdef __CUDACC__
__device__ __forceinline__ void chain_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <typename... P, typename... A>
inline cudaError_t launch_chained(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                  A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chained_launch_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}
// The same with thread-block clusters of (1, cluster_y, 1) CTAs.
template <typename... P, typename... A>
inline cudaError_t launch_chained_cluster(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                          unsigned cluster_y, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = cluster_y;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chained_launch_enabled() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}
#endif

// Tensor-map encoding through the driver entry point (no link-time dependency on libcuda).
// 3-D bf16 tensor [dim2][dim1][dim0] with dim0 contiguous; strides in elements; 128-byte swizzle;
// box = [1][box1][box0]; box0 must be 64 (128 bytes).
int make_tmap_bf16_3d(CUtensorMap* out, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                      uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box0, uint32_t box1);
// 3-D fp32 tensor [dim2][dim1][dim0], 128-byte swizzle, box = [1][box1][32] (32 floats = 128 bytes): the
// GEMM's output tiles
// 3-D byte tensor (FP8 operands), 128-byte swizzle, box = [1][box1][128]
int make_tmap_u8_3d(CUtensorMap* out, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                    uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t box1);
int make_tmap_f32_3d(CUtensorMap* out, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                     uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box1);
// rank-`rank` (3..5) bf16 tensor, dims/strides/box given innermost first (strides in elements, for
// dims 1..rank-1), 128-byte swizzle. Used for Q and for the paged KV pools [page][slot][head][hd].
int make_tmap_bf16_nd(CUtensorMap* out, const void* base, int rank, const uint64_t dims[5],
                      const uint64_t strides_elems[4], const uint32_t box[5]);

// page sizes the attention tiles can walk: 16, 32, 64 or a multiple of 128 positions
inline bool page_size_ok(int ps) { return ps == 16 || ps == 32 || ps == 64 || (ps >= 128 && ps % 128 == 0); }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ------------------------------------------------------------------------------------ GEMM
// D[g][m][n] = sum_k A[g][m][k] * B[g][n][k]   (bf16 operands, fp32 accumulation on tcgen05)
enum GemmEpilogue {
  EPI_STORE_BF16 = 0,   // out bf16 [M][ldo]
  EPI_STORE_F32 = 1,    // out fp32 [M][ldo]
  EPI_ADD_F32 = 2,      // out fp32 [M][ldo] += D  (residual add)
  EPI_GATED_BF16 = 3,   // B rows come in blocks of 256: 128 gate rows then the matching 128 up rows;
                        // out bf16 [M][ldo], column f = act(gate_f) * up_f, for f < n_valid
  EPI_QKV_ROPE = 4      // columns are heads [q heads | k heads | v heads] * hd: per-head norm, RoPE and the
                        // paged-cache write happen in the epilogue (GemmArgs::rope describes where to)
};
struct RopeArgs;
struct GemmArgs {
  const bf16* A; int64_t lda; int64_t a_batch_stride;   // elements
  const bf16* B; int64_t ldb; int64_t b_batch_stride;
  void* out; int64_t ldo; int64_t out_batch_stride;     // elements of the output type
  int M, N, K, batch;
  int epilogue;
  int act;          // EPI_GATED_BF16: 0 SiLU, 1 tanh-GELU
  int n_valid;      // EPI_GATED_BF16: number of valid output columns (d_ffn); others: ignored
  const RopeArgs* rope;   // EPI_QKV_ROPE only (its in / ld_in fields are unused; groups == batch)
  // RMSNorm folded around the GEMMs (batch == 1 only). A residual GEMM (EPI_ADD_F32) can also emit
  // the next GEMM's operand hn = bf16(x_new * gain_next), NOT yet normalised, and per n-tile the
  // row sums of x_new^2 (ss_out[row * ss_ld + n_tile], summed later in a fixed order, so results
  // do not depend on timing). The consuming GEMM scales its rows by
  // rsqrt(sum_i ss_in[row * ss_in_ld + i] / norm_d + norm_eps) before its own epilogue.
  bf16* hn_out; int64_t ld_hn; const float* gain_next; float* ss_out; int ss_ld;
  const float* ss_in; int ss_cnt; int ss_in_ld; int norm_d; float norm_eps;
  // FP8 operands (batch == 1, no folded norm): A and B point at E4M3 codes, lda / ldb /
  // K count codes (multiples of 16), and the accumulator is scaled by a_scale[row] * *b_scale (device)
  // before the epilogue proper
  bool fp8; const float* a_scale; const float* b_scale;
};
int launch_gemm(const GemmArgs& a, cudaStream_t stream);

// ------------------------------------------------------------------------------------ attention
// out[b][i][h][:] = softmax_j(q[b][i][h] . k[b][j][g(h)] / sqrt(hd)) v[b][j][g(h)] over cache positions
// j <= q_pos0 + i (and j > q_pos0 + i - window when window > 0), g(h) = h * n_kv / n_q.
struct AttnArgs {
  const bf16* q; int64_t ldq;            // [batch*seq_len][ldq], head h at column h*head_dim
  const bf16* k_pool; const bf16* v_pool; // one layer of the paged cache: [num_pages][page_size][n_kv][hd]
  const int32_t* block_table;            // device [batch][max_pages_per_seq]
  bf16* out; int64_t ldo;                // [batch*seq_len][ldo]
  int batch, seq_len, q_pos0, kv_len;
  // ragged batches: device int32 [batch + 1] prefix sums of the sequence lengths over packed rows;
  // sequence b then has cu[b+1] - cu[b] query rows and as many cache positions (seq_len / kv_len
  // give the maximum over the batch, q_pos0 must be 0); null = every sequence has seq_len rows
  const int32_t* cu_seqlens;
  int total_rows;                        // rows of q / out when packed (0 = batch * seq_len)
  int n_q_heads, n_kv_heads, head_dim;
  int page_size, num_pages, max_pages_per_seq;
  int window;
};
int launch_attention(const AttnArgs& a, cudaStream_t stream);

// ------------------------------------------------------------------------------------ elementwise
int launch_embed(const int32_t* tokens, const bf16* table, const bf16* embeds, float* x, int rows, int d, int vocab,
                 cudaStream_t s);
// out[g][row][:] = x[row][:] * rsqrt(mean(x[row]^2) + eps) * gain[g][:]; bf16 or fp32 output
int launch_rmsnorm(const float* x, int64_t ldx, const float* gain, int64_t gain_stride, void* out, int64_t ldo,
                   int64_t out_group_stride, int rows, int d, int groups, float eps, bool out_f32, cudaStream_t s);
// x[row][:] += rmsnorm(t[row][:]) * gain
int launch_postnorm_add(float* x, int64_t ldx, const float* t, int64_t ldt, const float* gain, int rows, int d,
                        float eps, cudaStream_t s);
// table[pos][j] = (cos, sin)(pos * theta^(-2j/hd)), pos < n_pos, j < hd/2
// rows for positions first_pos .. first_pos + n_pos - 1
int launch_rope_table(float2* table, int n_pos, int hd, float theta, cudaStream_t s, int first_pos = 0,
                      const int32_t* first_pos_dev = nullptr);   // device value overrides first_pos when given
struct RopeArgs {
  const float* in; int64_t ld_in; int64_t in_group_stride;   // fp32 rows [q heads | k heads | v heads] * hd
  bf16* q_out; int64_t ldq;                                  // may be null when n_q == 0
  bf16* k_pool; bf16* v_pool; int64_t pool_layer_stride;     // pools [layer][page][slot][n_kv][hd]
  int layer0;                                                // cache layer (0-based) of group 0
  const int32_t* block_table; int max_pages_per_seq; int page_size;
  const float* q_gain; const float* k_gain; int64_t gain_group_stride;   // per-head norm gains or null
  const float2* table; int table_pos0;                      // table row 0 holds position table_pos0
  int n_q, n_kv, hd;
  int rows, rows_per_seq, rows_written, pos0, groups;
  float eps;
  // ragged batches (null = uniform). In the GEMM epilogue: packed row r belongs to the sequence b with
  // cu[b] <= r < cu[b+1], position r - cu[b]; the last `skip_last` positions of each sequence are not
  // written. In launch_rope_cache it is only used for boundary rows (rows == batch): row b sits at
  // position cu[b+1] - cu[b] - 1.
  const int32_t* cu_seqlens; int batch; int skip_last;
  // boundary / decode rows only: the position is read from device memory at run time (a step that is
  // replayed from a captured graph with an advancing position); the table then holds that one row
  const int32_t* pos_dev;
  // pages per layer of the pools. Block-table entries live on the device, so only the kernel can
  // check them: with num_pages > 0 an entry outside [0, num_pages) is never turned into an address;
  // the row is skipped and the status word raised to POP_E_INVALID. 0 = unknown (no check).
  int num_pages;
};
int launch_rope_cache(const RopeArgs& a, cudaStream_t s);
int launch_gather_rows(const float* src, float* dst, int batch, int d, int rows_per_seq, int row, cudaStream_t s);
// dst[b][:] = src[cu[b+1] - 1][:]: the last row of every packed sequence
// tok[b] = index of the largest logit of row b (lowest index among equals), also stored at out[b * out_ld + *step]
int launch_argmax(const float* logits, int64_t ld, int vocab, int batch, int32_t* tok, int32_t* out, int out_ld,
                  const int32_t* step, cudaStream_t s);
// counters[0] = a, counters[1] = b; and counters[0] += 1, counters[1] += 1
int launch_set_counters(int32_t* counters, int a, int b, cudaStream_t s);
int launch_bump_counters(int32_t* counters, cudaStream_t s);
int launch_gather_last_rows(const float* src, float* dst, int batch, int d, const int32_t* cu, cudaStream_t s);

// ------------------------------------------------------------------------------------ FP8 operands
// out[row][:] = e4m3(LN(x[row]) * 448 / amax_row), scale[row] = amax_row / 448 (LN = RMSNorm with `gain`)
int launch_rmsnorm_e4m3(const float* x, int64_t ldx, const float* gain, uint8_t* out, int64_t ldo, float* scale,
                        int rows, int d, float eps, cudaStream_t s);
// rows of bf16 values -> codes and one scale per row (d <= 16384); out may alias in (row by row in place)
int launch_quant_rows_e4m3(const bf16* in, int64_t ld_in, uint8_t* out, int64_t ld_out, float* scale, int rows, int d,
                           cudaStream_t s);
// out[i] = e4m3(w[i] * 448 / amax), *scale = amax / 448 over the n elements; scratch: 4 bytes
int launch_quantize_weights_e4m3(const bf16* w, int64_t n, uint8_t* out, float* scale, unsigned int* scratch,
                                 cudaStream_t s);

// ------------------------------------------------------------------------------------ boundary path
struct GemvArgs {
  const void* x; int64_t ldx; bool x_f32;    // [B][K] bf16 or fp32
  const void* w; int64_t ldw;                // [N][K] bf16; or E4M3 codes (w_fp8, bf16 x only, K and ldw
                                             // multiples of 16) with the matrix's scale at *w_scale (device)
  void* out; int64_t ldo;                    // mode 0: fp32 store; 2: fp32 +=; 3: gated -> bf16 [B][n_valid]
  int B, N, K, mode, act, n_valid;
  bool w_fp8; const float* w_scale;
};
int launch_gemv(const GemvArgs& a, cudaStream_t s);
struct DecAttnArgs {
  const bf16* q; int64_t ldq;
  const bf16* k_pool; const bf16* v_pool;    // one layer of the cache
  const int32_t* block_table; int max_pages_per_seq; int page_size;
  float* partial;                            // [batch][n_q][splits][hd + 2] fp32 scratch
  bf16* out; int64_t ldo;
  int batch, n_q, n_kv, head_dim, kv_len, window;
  int kv_first;                // first cache position the query may attend to (0: all; a layer whose
                               // earlier rows were never generated)
  const int32_t* cu_seqlens;   // ragged: sequence b has cu[b+1] - cu[b] cache positions (kv_len = their maximum)
  const int32_t* pos_dev;      // run-time cache length - 1 (see RopeArgs::pos_dev)
  // optional [batch][n_kv] int32, all zero before the call and all zero again after it: with it the
  // attention kernel merges its own splits (one launch); without, a second kernel does
  int32_t* counters;
  int num_pages;               // pages in the pool, for the device-side block-table check (0 = no check)
  // Optional: finish the projection inside the attention kernel instead of a kernel of its own. With
  // `qkv` set (fp32 rows [q heads | k heads | v heads] * hd, one per sequence, straight from the QKV
  // GEMV) every CTA applies the per-head norm (gains or null) and the rotary row to its own query
  // heads, and the CTA whose key range holds the newest position does the same for that position's
  // key, appends key and value to the (then writable) pools and takes them from there; `q` is unused.
  const float* qkv; int64_t ld_qkv;
  const float* q_gain; const float* k_gain;
  const float2* table; int table_pos0;   // as in RopeArgs
  float eps;
  // With `qkv`: true when the cache rows of the older positions, the block table and pos_dev / cu_seqlens
  // were written at least two launches back on the stream (the library's own chain of kernels): the
  // kernel then starts loading the cache before it waits for its predecessor. False: it waits first.
  bool cache_settled;
};
int decode_attn_splits(int kv_len, int window, int n_kv, int batch);
int launch_decode_attention(const DecAttnArgs& a, cudaStream_t s);

}  // namespace pop
