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

/* pop_k_gemm (batch 1, epilogues 0-3) with the layer's RMSNorm (the LN of paper Eq. 1-2) folded
 * around it, so that no separate pass over the residual stream is needed:
 *  - producer side, epilogue 2 only, when hn_out != NULL: besides out += D the call writes
 *    hn_out[m][n] = bf16(out_new[m][n] * gain_next[n]) (row stride ld_hn) -- the next GEMM's operand,
 *    not yet normalised -- and ss_out[m * ss_ld + n / 256] = sum over that 256-column tile of
 *    out_new[m][n]^2 (ss_ld >= ceil(N / 256));
 *  - consumer side, when ss_in != NULL: every row m of D is multiplied by
 *    rsqrt(sum_{i < ss_cnt} ss_in[m * ss_in_ld + i] / norm_d + norm_eps) before the epilogue acts
 *    (for epilogue 3 before the activation). The partial sums are added in index order, so the
 *    result does not depend on scheduling.
 * Pass NULL for the side not wanted. */
int pop_k_gemm_norm(const void* A, int64_t lda, const void* B, int64_t ldb, void* out, int64_t ldo, int32_t M,
                    int32_t N, int32_t K, int32_t epilogue, int32_t act, int32_t n_valid, void* hn_out, int64_t ld_hn,
                    const float* gain_next, float* ss_out, int32_t ss_ld, const float* ss_in, int32_t ss_cnt,
                    int32_t ss_in_ld, int32_t norm_d, float norm_eps, void* stream);

/* The fused form of the QKV projection and pop_k_rope_cache (paper Eq. 2-3; Eq. 14 for pruned
 * layers): D[g] = A[g] W[g]^T with W's rows ordered [q heads | k heads | v heads] * hd, and in the
 * GEMM's epilogue the optional per-head RMSNorm (q, k), RoPE (q, k), rounding to bf16, q -> q_out
 * [M][ldq] (n_q may be 0: no query, as for pruned layers), k and v -> cache layer layer0 + g.
 * A bf16 [batch][M][lda] (batch stride a_bs, 0 = packed), W bf16 [batch][(n_q+2 n_kv) hd][ldw].
 * Row / position / cache conventions and the remaining arguments are those of pop_k_rope_cache;
 * M must be a multiple of rows_per_seq. Nothing of the fp32 projection goes through memory. */
int pop_k_gemm_qkv_rope(const void* A, int64_t lda, int64_t a_bs, const void* W, int64_t ldw, int64_t w_bs, int32_t M,
                        int32_t K, int32_t batch, void* q_out, int64_t ldq, void* k_pool, void* v_pool,
                        int64_t pool_layer_stride, int32_t layer0, const int32_t* block_table,
                        int32_t max_pages_per_seq, int32_t page_size, const float* q_gain, const float* k_gain,
                        int64_t gain_gs, const void* table, int32_t n_q, int32_t n_kv, int32_t head_dim,
                        int32_t rows_per_seq, int32_t rows_written, int32_t pos0, float eps, void* stream);

/* Causal GQA attention of a decoder layer over the paged cache (paper Eq. 1, Attn(x_l, K, V) after
 * the append of Eq. 3): for sequence b, query row i (absolute position q_pos0 + i) and head h,
 *   out[b][i][h] = sum_j softmax_j(q[b][i][h] . k[b][j][g] / sqrt(hd)) v[b][j][g],  g = h*n_kv/n_q,
 * over cache positions j <= q_pos0 + i, and j > q_pos0 + i - window when window > 0.
 * q: device bf16 [batch*seq_len][ldq] (head h at column h*hd); k_pool/v_pool: ONE layer of the
 * cache, bf16 [num_pages][page_size][n_kv][hd]; block_table as in pop_kv_cache_t; out: bf16
 * [batch*seq_len][ldo]. kv_len = valid cache positions (>= q_pos0 + seq_len). hd in {64,128,256}; page_size as in pop.h. */
int pop_k_attention(const void* q, int64_t ldq, const void* k_pool, const void* v_pool, const int32_t* block_table,
                    void* out, int64_t ldo, int32_t batch, int32_t seq_len, int32_t q_pos0, int32_t kv_len,
                    int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t page_size, int32_t num_pages,
                    int32_t max_pages_per_seq, int32_t window, void* stream);

/* FP8 operands for the projections of paper Eq. 1-2. The paper fixes no number format and names
 * stage-aware quantisation as a direction (Sec. 6); this is the OCP E4M3 format (1-4-3 bits, bias 7,
 * largest value 448, no infinities), round to nearest even, saturating, with one scale per
 * activation row and one per weight matrix: value = code * scale.
 *
 * pop_k_rmsnorm_e4m3: y = LN(x[r]) as pop_k_rmsnorm computes it in fp32; out[r][:] = e4m3(y * 448 /
 *   max|y|) as bytes (row stride ldo bytes, a multiple of 16), scale[r] = max|y| / 448 (1 for a zero row).
 * pop_k_quant_rows_e4m3: rows of stored bf16 values (row stride ld_in elements, d <= 16384 a multiple of 8):
 *   out[r][:] = e4m3(in[r][:] * 448 / max|in[r]|) (row stride ld_out bytes, a multiple of 16), scale[r] as
 *   above. out may be in itself (each row's codes then fill the first d bytes of the row).
 * pop_k_quantize_e4m3: the same for a whole bf16 array of n elements (n a multiple of 8) with one
 *   scale: out[i] = e4m3(w[i] * 448 / max|w|), *scale = max|w| / 448. scratch4: 4 device bytes.
 * pop_k_gemm_e4m3: D[m][n] = a_scale[m] * *b_scale * sum_k A[m][k] * B[n][k] on the codes (fp32
 *   accumulation on the tensor cores, kind f8f6f4), then epilogue 0, 1, 2 or 3 of pop_k_gemm. lda,
 *   ldb, K count codes and are multiples of 16; pointers 16-byte aligned; a_scale, b_scale device fp32. */
/* pop_k_gemv with E4M3 weights (the single-position passes of Sec. 3.3 / the decode stage stream half the
 * bytes): out[b][n] = *w_scale * sum_k x[b][k] * W[n][k], x bf16 [B][ldx] unquantised, W codes [N][ldw]
 * (K and ldw multiples of 16), w_scale device fp32. Modes as pop_k_gemv. */
int pop_k_gemv_e4m3(const void* x, int64_t ldx, const void* w, int64_t ldw, const float* w_scale, void* out,
                    int64_t ldo, int32_t B, int32_t N, int32_t K, int32_t mode, int32_t act, int32_t n_valid,
                    void* stream);
int pop_k_rmsnorm_e4m3(const float* x, int64_t ldx, const float* gain, void* out, int64_t ldo, float* scale,
                       int32_t rows, int32_t d, float eps, void* stream);
int pop_k_quant_rows_e4m3(const void* in, int64_t ld_in, void* out, int64_t ld_out, float* scale, int32_t rows,
                          int32_t d, void* stream);
int pop_k_quantize_e4m3(const void* w, int64_t n, void* out, float* scale, void* scratch4, void* stream);
int pop_k_gemm_e4m3(const void* A, int64_t lda, const float* a_scale, const void* B, int64_t ldb,
                    const float* b_scale, void* out, int64_t ldo, int32_t M, int32_t N, int32_t K, int32_t epilogue,
                    int32_t act, int32_t n_valid, void* stream);

/* RMSNorm, the LN of paper Eq. 2 / Eq. 14: out[g][r][:] = x[r][:] * rsqrt(mean(x[r]^2)+eps) * gain[g][:].
 * x fp32 [rows][ldx]; gain fp32, group g at gain + g*gain_stride; out bf16 (out_f32 = 0) or fp32,
 * group stride out_gs elements. */
int pop_k_rmsnorm(const float* x, int64_t ldx, const float* gain, int64_t gain_stride, void* out, int64_t ldo,
                  int64_t out_gs, int32_t rows, int32_t d, int32_t groups, float eps, int32_t out_f32, void* stream);

/* Rotary table: table[pos][j] = (cos, sin)(pos * theta^(-2j/hd)) as float2, pos < n_pos, j < hd/2. */
int pop_k_rope_table(void* table, int32_t n_pos, int32_t head_dim, float theta, void* stream);

/* KV generation and append (paper Eq. 2-3; Eq. 14 when applied to a pruned layer): rows of fp32
 * projections [q heads | k heads | v heads] * hd get the optional per-head RMSNorm (q, k), RoPE
 * (q, k), rounding to bf16; q goes to q_out [rows][ldq], k and v into cache layer layer0 + g of
 * the pools [layer][page][slot][n_kv][hd] (pool_layer_stride elements per layer). Row r belongs to
 * sequence r / rows_per_seq at position pos0 + r % rows_per_seq; rows with r % rows_per_seq >=
 * rows_written are skipped. n_q may be 0 (pruned layers: no query). */
int pop_k_rope_cache(const float* in, int64_t ld_in, int64_t in_gs, void* q_out, int64_t ldq, void* k_pool,
                     void* v_pool, int64_t pool_layer_stride, int32_t layer0, const int32_t* block_table,
                     int32_t max_pages_per_seq, int32_t page_size, const float* q_gain, const float* k_gain,
                     int64_t gain_gs, const void* table, int32_t n_q, int32_t n_kv, int32_t head_dim, int32_t rows,
                     int32_t rows_per_seq, int32_t rows_written, int32_t pos0, int32_t groups, float eps,
                     void* stream);

/* Weight-streaming GEMV of the boundary-token path (paper Sec. 3.3) and of the output head:
 * out[b][n] = sum_k x[b][k] * W[n][k] for a few rows b. x bf16 or fp32 (x_f32) [B][ldx]; W bf16
 * [N][ldw]. mode 0: fp32 store; 2: fp32 +=; 3: gated (W rows in 128-gate/128-up blocks) -> bf16. */
int pop_k_gemv(const void* x, int64_t ldx, int32_t x_f32, const void* w, int64_t ldw, void* out, int64_t ldo,
               int32_t B, int32_t N, int32_t K, int32_t mode, int32_t act, int32_t n_valid, void* stream);

/* Single-query attention of the boundary token (paper Sec. 3.3; one query per sequence at position
 * kv_len-1) over one cache layer, split over the keys. n_q / n_kv <= 8; head_dim 64, 128 or 256.
 * partial: device scratch of batch * n_q * 64 * (hd + 2) floats, contents irrelevant before and after.
 * counters: optional device int32 [batch * n_kv]. If given they must all be zero when the call's
 * kernels start and are all zero again when they end (so one zeroed array serves any number of
 * calls on one stream); the attention kernel then merges its own splits and the call is a single
 * launch. Null: a second kernel merges them. Both ways give the same bits. With few splits per sequence
 * and kv head (short caches, several sequences) the splits run as one thread-block cluster and merge
 * through distributed shared memory; partial and counters are then not touched (POP_DEC_CLUSTER=0 in the
 * environment turns that form off). */
int pop_k_decode_attention(const void* q, int64_t ldq, const void* k_pool, const void* v_pool,
                           const int32_t* block_table, int32_t max_pages_per_seq, int32_t page_size, float* partial,
                           int32_t* counters, void* out, int64_t ldo, int32_t batch, int32_t n_q, int32_t n_kv,
                           int32_t head_dim, int32_t kv_len, int32_t window, void* stream);

/* pop_k_decode_attention with the end of the projection folded in (paper Eq. 2-3 for the one new
 * position, then Attn of Eq. 1; Sec. 3.3): instead of finished queries the kernel takes the fp32 row
 * qkv[b] = [q heads | k heads | v heads] * head_dim of every sequence (ld_qkv floats apart), applies the
 * per-head RMSNorm (q_gain / k_gain: fp32 [head_dim], or both NULL for none; eps) and the rotary row
 * of position kv_len - 1 (table: device float2 [head_dim / 2] pairs (cos, sin) of that one position) to
 * the queries and the key, appends key and value at position kv_len - 1 of the cache (k_pool and
 * v_pool are WRITTEN here: one layer, [num_pages][page_size][n_kv][head_dim]), and attends over
 * positions max(0, kv_len - window) .. kv_len - 1 (window 0: all). counters (device int32
 * [batch * n_kv], zero before and after) are required: the call is a single launch. A block-table
 * entry outside [0, num_pages) is never dereferenced; the status word is raised to POP_E_INVALID.
 * This is the form the boundary-token / decode path of pop_prefill and pop_decode_step runs. */
int pop_k_decode_attention_qkv(const float* qkv, int64_t ld_qkv, const float* q_gain, const float* k_gain, float eps,
                               const void* rope_row, void* k_pool, void* v_pool, const int32_t* block_table,
                               int32_t max_pages_per_seq, int32_t page_size, int32_t num_pages, float* partial,
                               int32_t* counters, void* out, int64_t ldo, int32_t batch, int32_t n_q, int32_t n_kv,
                               int32_t head_dim, int32_t kv_len, int32_t window, void* stream);

/* The same single-query attention as pop_k_decode_attention for callers that have no way to hand
 * over a scratch buffer because they cannot allocate device memory at the point of the call: code
 * running inside a host callback or a real-time serving loop where cudaMalloc is forbidden, or a
 * process that received all its device buffers (inputs and outputs only) from another owner and
 * has no allocator of its own. (The paper has no counterpart: this is a packaging variant, not a
 * step of the method.) The split-KV partials go to a fixed array of POP_STATIC_SCRATCH_FLOATS
 * floats (16 MiB) that is part of the library image, so every GPU that loads the library holds it
 * until the process ends. The call allocates and frees nothing, neither through CUDA nor any other
 * library. Arguments, layouts and results are those of pop_k_decode_attention minus `partial`.
 *  - Limit: batch * n_q * splits * (head_dim + 2) <= POP_STATIC_SCRATCH_FLOATS, where splits =
 *    min(64, SMs / (n_kv * batch), ceil(span / 64)), at least 1, and span = min(kv_len, window or
 *    kv_len); a larger problem is refused with POP_E_NOSPACE and nothing is enqueued (e.g. 512
 *    sequences x 32 heads x hd 128 fit at any length; 1024 such sequences do not).
 *  - The first call on each device looks up the array's device address (one runtime query with
 *    that device current, result kept); make that first call before starting any stream capture.
 *  - All calls share the one array, which keeps whatever the previous call left. Each call
 *    overwrites every slot it later reads, so no clearing is needed, but two calls whose kernels
 *    may overlap on the GPU (different streams without an ordering between them) race on it:
 *    serialise them. Calls on one stream are safe. The arrival counters of the split merge sit in a
 *    second fixed array (4096 entries, one per sequence and kv head; with more than that a second
 *    kernel merges the splits instead); it is not reachable from the host, starts at zero when the
 *    library is loaded and every launch leaves it at zero again.
 * Errors: POP_E_INVALID (null pointer, bad head_dim or head counts), POP_E_NOSPACE (over the limit,
 * or block table too short), POP_E_CUDA. */
#define POP_STATIC_SCRATCH_FLOATS (4 * 1024 * 1024)
int pop_k_decode_attention_static(const void* q, int64_t ldq, const void* k_pool, const void* v_pool,
                                  const int32_t* block_table, int32_t max_pages_per_seq, int32_t page_size,
                                  void* out, int64_t ldo, int32_t batch, int32_t n_q, int32_t n_kv,
                                  int32_t head_dim, int32_t kv_len, int32_t window, void* stream);

/* Synchronise the stream, then read and clear the library's device status word. */
int pop_k_status(void* stream);

/* Self-test of the library's failure path (no counterpart in the paper). Every device-side wait of
 * the GEMM and attention kernels (on an mbarrier that a TMA copy or a tensor-core commit completes)
 * is bounded: when it runs out, the kernel raises the status word to POP_E_DEVICE_TIMEOUT, unwinds and
 * returns, and kernels launched while the word is raised return at once. This call launches one small
 * kernel that performs that very wait on a barrier nothing arrives at, for at most limit_cycles SM
 * cycles (1 .. 1 000 000, i.e. well under a millisecond; POP_E_INVALID otherwise), so the path can be
 * exercised without a fault, a trap or an endless loop: afterwards pop_k_status returns
 * POP_E_DEVICE_TIMEOUT once and POP_OK from then on. */
int pop_k_wait_selftest(int64_t limit_cycles, void* stream);

/* Per-kernel timing for benchmarks. pop_k_profile(1) makes every launch of this library record a
 * CUDA-event pair on its stream; pop_k_profile_summary waits for the recorded events of one kind
 * (0 projection GEMM, 1 prefill attention, 2 elementwise, 3 GEMV, 4 decode attention), returns
 * their summed duration in ms, their summed algorithmic work (flops for kinds 0-1, bytes
 * otherwise) and their count, and forgets them. Off by default; costs nothing when off. */
void pop_k_profile(int32_t enable);
int pop_k_profile_summary(int32_t kind, double* total_ms, double* total_work, int64_t* launches);

/* Kernel launches enqueued by this library since the last pop_k_reset_launch_count(). */
int64_t pop_k_launch_count(void);
void pop_k_reset_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* POP_KERNELS_H_ */
