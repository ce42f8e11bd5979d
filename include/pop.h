/* pop.h - C ABI of the POP (Prefill-Only Pruning) prefill library for NVIDIA B200 (sm_100a).
 *
 * The library evaluates the prefill stage of a decoder-only transformer in two ways:
 *
 *   pop_full_prefill  the standard prefill: all L layers over the prompt x_1..x_N
 *                     (paper Sec. 2.1, Eq. 1-3), logits of the last prompt position;
 *   pop_prefill       POP's pruned prefill (paper Sec. 3.3): layers 1..L_keep run in full; each
 *                     deeper layer only stores k = RoPE(LN(H) W^K), v = LN(H) W^V computed from the
 *                     state H leaving the kept stack (Eq. 14) and passes H on unchanged (Eq. 15);
 *                     the last prompt token x_N is then run through ALL L layers as the first
 *                     decode step (boundary handling), so its logits use the whole model.
 *
 * Conventions
 *   - Every pointer named dev_* or documented "device" is CUDA device memory owned by the caller.
 *     The library borrows it; it allocates no device memory of its own and frees none.
 *   - `stream` is a cudaStream_t passed as void*. Calls enqueue work on it and return without
 *     synchronising (pop_last_status is the exception).
 *   - Return value: POP_OK (0) or a negative pop_status code. Arguments are checked before the first
 *     launch: POP_E_INVALID and POP_E_NOSPACE mean nothing was enqueued and nothing written. POP_E_CUDA
 *     (a launch or runtime call failed part-way) may leave earlier kernels of the call queued; the
 *     outputs are then undefined.
 *   - One device per process: the library caches per-process launch attributes and the address of its
 *     device status word for the device that is current at the first call. Replicas on several GPUs
 *     run as one process per GPU.
 *   - Matrices are row-major bf16 [out_features, in_features] (y = x W^T). Norm gains are fp32.
 *   - Sequences of a batch have equal length; positions are 0-based.
 */
#ifndef POP_H_
#define POP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  POP_OK = 0,
  POP_E_INVALID = -1,        /* null pointer, size out of range, shape inconsistent with the config */
  POP_E_NOSPACE = -2,        /* weight arena, workspace or KV pages too small */
  POP_E_CUDA = -3,           /* a CUDA runtime / driver call or a launch failed */
  POP_E_DEVICE_TIMEOUT = -4, /* a bounded device-side wait expired (seen through pop_last_status) */
  POP_E_MISSING = -5         /* pop_load_weights: a required tensor was not supplied */
} pop_status;

typedef struct pop_model pop_model_t; /* opaque */

/* Model shape. struct_size must be sizeof(pop_config_t) (guards against ABI drift). */
typedef struct {
  uint32_t struct_size;
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rms_eps;
  float rope_theta;
  int32_t act;          /* 0: SiLU-gated FFN, 1: tanh-GELU-gated FFN */
  int32_t qk_norm;      /* 1: per-head RMSNorm on q and k between projection and RoPE */
  int32_t post_norms;   /* 1: RMSNorm on the attention and FFN outputs before the residual add */
  int32_t window;       /* sliding-window size in keys, own position included; 0: all layers global */
  int32_t global_every; /* with window > 0: 1-based layer l is global iff l % global_every == 0 */
} pop_config_t;

/* One named weight tensor handed to pop_load_weights.
 * name: "embed", "final_norm", "lm_head", or "layers.<l>.<t>" with 1-based l and t one of
 *   ln_in, wq, wk, wv, wo, ln_ffn, w_gate, w_up, w_down, q_norm, k_norm, post_attn_norm, post_ffn_norm.
 * dev_ptr: device memory, contiguous; dtype 0 = bf16 (matrices), 1 = fp32 (norm gains). */
typedef struct {
  const char* name;
  const void* dev_ptr;
  int32_t dtype;
  int32_t ndim;
  int64_t shape[2];
} pop_tensor_t;

/* Paged KV cache, caller-owned device memory.
 * k_pool, v_pool: bf16 [n_layers][num_pages][page_size][n_kv_heads][head_dim].
 * block_table:    device int32 [batch][max_pages_per_seq]; entry (b, j) is the page that holds
 *                 positions j*page_size .. (j+1)*page_size-1 of sequence b.
 * page_size must be 16, 32, 64 or a multiple of 128, so that no 128-position attention tile
 * straddles pages unevenly. Entries of a page beyond seq_len are left untouched. */
typedef struct {
  void* k_pool;
  void* v_pool;
  const int32_t* block_table;
  int32_t page_size, num_pages, max_pages_per_seq;
} pop_kv_cache_t;

/* Prompt. tokens: device int32 [batch][seq_len]. embeds: device bf16 [batch][seq_len][d_model] or
 * NULL; when given, a position whose token id is negative takes its input row from embeds (visual
 * or other pre-computed embeddings) instead of the embedding table. Token ids live on the device, so
 * the host cannot check them: an id >= vocab, or a negative id while embeds is NULL, makes that
 * position's input a row of zeros, raises the device status word to POP_E_INVALID (the remaining
 * kernels of the call return without computing) and is reported by pop_last_status. */
typedef struct {
  const int32_t* tokens;
  const void* embeds;
} pop_input_t;

/* Bytes of device memory pop_load_weights needs for the repacked weights of `cfg`. */
size_t pop_weight_arena_bytes(const pop_config_t* cfg);

/* Repack the given tensors into dev_arena (fused QKV, tile-interleaved gate/up, concatenated K/V
 * projections for the pruned-layer pass) on `stream` and return a model handle. The source tensors
 * may be released once the stream has drained. Errors: POP_E_INVALID, POP_E_NOSPACE, POP_E_MISSING,
 * POP_E_CUDA. The handle (host memory) is released with pop_free; the arena stays the caller's. */
int pop_load_weights(const pop_config_t* cfg, const pop_tensor_t* tensors, int32_t n_tensors,
                     void* dev_arena, size_t arena_bytes, void* stream, pop_model_t** out);

/* Scratch bytes a prefill of `batch` sequences of `seq_len` tokens needs (activations, fp32
 * residual stream, rotary table, split-KV partials). */
size_t pop_workspace_bytes(const pop_model_t* m, int32_t seq_len, int32_t batch);

/* Lend the library a workspace of `bytes` bytes (device, 1024-byte aligned). It is used by every
 * later prefill call until replaced; calls that overlap on the GPU must not share one. */
int pop_set_workspace(pop_model_t* m, void* dev_ws, size_t bytes);

/* POP pruned prefill with boundary handling (paper Sec. 3.3, Eq. 14-15). 1 <= L_keep <= n_layers.
 * On completion kv_cache_out holds seq_len entries for EVERY layer and sequence: layers <= L_keep
 * and position seq_len-1 of all layers from full layer evaluations, positions 0..seq_len-2 of
 * layers > L_keep from the independent K/V projections of H. logits_out: device fp32
 * [batch][vocab], the next-token logits at the last prompt position. L_keep == n_layers gives
 * exactly pop_full_prefill. */
int pop_prefill(pop_model_t* m, const pop_input_t* tokens_or_embeds, int32_t seq_len, int32_t batch,
                int32_t L_keep, pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream);

/* Standard full-depth prefill of the unpruned model (paper Sec. 2.1, Eq. 1-3; the reference path
 * POP is compared with in Sec. 4.3). Same outputs as pop_prefill. */
int pop_full_prefill(pop_model_t* m, const pop_input_t* tokens_or_embeds, int32_t seq_len, int32_t batch,
                     pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream);

/* pop_prefill for a batch of sequences of DIFFERENT lengths (the paper batches real prompts, Sec. 4.3:
 * batch 8; padding is not part of the method, so none is used): the sequences are packed back to
 * back, tokens_or_embeds->tokens is device int32 [sum of lengths] (embeds, if given, device bf16
 * [sum of lengths][d_model]), seq_lens is a HOST array of `batch` lengths (each >= 1). Sequence b
 * uses row b of the block table and gets seq_lens[b] cache entries in every layer; its boundary
 * token is its own last token, and logits_out[b] are the next-token logits after it. The
 * workspace must be sized for (max length, batch). Other conventions and errors as pop_prefill. */
int pop_prefill_ragged(pop_model_t* m, const pop_input_t* tokens_or_embeds, const int32_t* seq_lens, int32_t batch,
                       int32_t L_keep, pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream);

/* pop_prefill for an explicitly given pruned set S_skip (paper Eq. 4 and Eq. 14-15; the shallow /
 * interleaved selections of the ablation in Sec. 4.4): skip is a HOST array of n_layers bytes,
 * skip[l-1] != 0 meaning layer l only stores its K/V projections of the state that reaches it and
 * hands that state on unchanged. Evaluated in the paper's literal two phases (prompt positions
 * through the layers, then the last prompt token through ALL layers as a decode step), so it costs
 * n_layers boundary passes where pop_prefill needs n_layers - L_keep; for the deep-suffix set the
 * two calls agree to rounding. Outputs, conventions and errors as pop_prefill. */
int pop_prefill_skip(pop_model_t* m, const pop_input_t* tokens_or_embeds, int32_t seq_len, int32_t batch,
                     const uint8_t* skip, pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream);

/* FP8 operands for the four projections of every kept layer (QKV, output, gate/up, down). The paper
 * runs unquantised models and names stage-aware quantisation as a direction (Sec. 6); this is that
 * second precision, off by default. pop_enable_fp8 writes E4M3 copies of those weight matrices (one
 * scale per matrix) into dev_arena (caller's device memory, 1024-byte aligned, at least
 * pop_fp8_arena_bytes(m); it must stay valid while enabled; d_model, q_dim, d_ffn multiples of 16 and
 * q_dim, d_ffn <= 16384, POP_E_INVALID otherwise). While enabled, pop_prefill, pop_full_prefill,
 * pop_prefill_chunked and pop_prefill_ragged turn the rows entering those projections into E4M3
 * codes with one scale per row (the normalised rows straight from the norm, the stored bf16
 * attention output and gated activation in place) and run the four GEMMs on the codes (fp32
 * accumulation; scales applied to the accumulator before the usual epilogue). The single-position
 * passes -- the boundary token's deep layers, pop_decode_step, pop_generate_greedy -- stream the
 * E4M3 weights (half the bytes) and keep bf16 activations. Attention and the pruned layers' Eq. 14
 * projections keep bf16 operands. pop_prefill_skip and pop_prefill_ablation (the literal two-phase
 * evaluation) return POP_E_INVALID while it is enabled. dev_arena = NULL disables it. */
size_t pop_fp8_arena_bytes(const pop_model_t* m);
int pop_enable_fp8(pop_model_t* m, void* dev_arena, size_t bytes, void* stream);

/* pop_prefill evaluated chunk by chunk over the positions: chunk_len positions of every sequence
 * at a time through the kept layers (Eq. 1-3, attending over the cache entries the earlier chunks
 * stored) and the pruned layers' projections (Eq. 14-15), the boundary token (Sec. 3.3) with the
 * last chunk. By causality this is the same function as pop_prefill; what changes is the
 * workspace: pop_workspace_bytes(m, chunk_len, batch) suffices whatever seq_len is, so prompts far
 * beyond what a one-shot workspace allows fit (seq_len <= 2^24). Inputs, outputs and errors as
 * pop_prefill; chunk_len >= 1 (a multiple of 128 keeps the attention tiles full; larger than
 * seq_len means one chunk). */
int pop_prefill_chunked(pop_model_t* m, const pop_input_t* tokens_or_embeds, int32_t seq_len, int32_t batch,
                        int32_t L_keep, int32_t chunk_len, pop_kv_cache_t* kv_cache_out, float* logits_out,
                        void* stream);

/* The two component ablations of the paper's Sec. 4.4.1 (the design-choice ablation table) on top
 * of pop_prefill_skip; flags is a combination of
 *   POP_NO_BOUNDARY  no boundary handling: the last prompt token is processed by the pruned
 *                    prefill model like every other position (pruned layers store their Eq. 14
 *                    projections for all seq_len positions, there is no full-depth pass for the last
 *                    token) and logits_out comes from the state that leaves the pruned model there;
 *   POP_NO_INDEP_KV  no independent KV projections: pruned layers generate no cache entries for the prompt
 *                    (their rows of positions 0..seq_len-2 are left untouched); in the last token's
 *                    full-depth pass such a layer attends to position seq_len-1 only. Later decode
 *                    steps must keep that horizon: use pop_decode_step_from.
 * flags = 0 is pop_prefill_skip. Other arguments, outputs and errors as pop_prefill_skip;
 * POP_E_INVALID for unknown flag bits. */
#define POP_NO_BOUNDARY 1
#define POP_NO_INDEP_KV 2
int pop_prefill_ablation(pop_model_t* m, const pop_input_t* tokens_or_embeds, int32_t seq_len, int32_t batch,
                         const uint8_t* skip, int32_t flags, pop_kv_cache_t* kv_cache_out, float* logits_out,
                         void* stream);

/* pop_decode_step with an attention horizon per layer: layer_first_pos is a HOST array of n_layers
 * int32; layer l attends to cache positions layer_first_pos[l-1] .. pos only (and within its window,
 * if it has one). After pop_prefill_ablation(POP_NO_INDEP_KV) on seq_len = N tokens the pruned layers
 * take N-1 (N if POP_NO_BOUNDARY was set as well: they then hold nothing of the prompt), the others 0
 * (paper Sec. 4.4.1: in those layers only the last prompt token and the generated tokens are visible). NULL = pop_decode_step. POP_E_INVALID if an entry is negative
 * or beyond pos. */
int pop_decode_step_from(pop_model_t* m, const int32_t* tokens, int32_t pos, int32_t batch,
                         const int32_t* layer_first_pos, pop_kv_cache_t* kv_cache, float* logits_out, void* stream);

/* One decode step of the FULL model over the cache a prefill left (the decode stage D of paper
 * Sec. 3.2, Eq. 11, which Sec. 3.3 keeps at full depth): tokens is device int32 [batch], the token of
 * each sequence at position `pos` = number of entries its cache already holds. Every layer
 * appends its k, v at `pos` (Eq. 2-3), attends over positions 0..pos (the window in local
 * layers), and logits_out (device fp32 [batch][vocab]) receives the next-token logits. After
 * pop_prefill(seq_len = N) the first call uses pos = N. The cache must have room for pos + 1
 * positions per sequence (POP_E_NOSPACE otherwise); the workspace of any earlier prefill with the
 * same batch is large enough. Errors as pop_prefill. */
int pop_decode_step(pop_model_t* m, const int32_t* tokens, int32_t pos, int32_t batch, pop_kv_cache_t* kv_cache,
                    float* logits_out, void* stream);

/* Greedy generation on the device (the decode stage of paper Sec. 3.2, Eq. 11, run as a loop): starting from
 * first_tokens (device int32 [batch], the token of each sequence at position pos0 -- normally the
 * arg-max of the prefill's logits), n_steps times: one full-model decode step as pop_decode_step,
 * then the arg-max of its logits (lowest index among equal values) becomes the next token.
 * tokens_out (device int32 [batch][n_steps]) receives the generated tokens: tokens_out[b][i] is
 * the token at position pos0 + i + 1. logits_scratch is device fp32 [batch][vocab] (it holds the
 * last step's logits afterwards). One step is captured into a CUDA graph whose kernels read the
 * position from device memory, and that graph is launched n_steps times on `stream`, so the host
 * issues n_steps graph launches instead of n_steps x (7 n_layers + 5) kernel launches (9 per layer for a model with post-norms). The call
 * creates and destroys a stream and a graph of its own (host-side objects; no device memory).
 * Not available while pop_k_profile is on. The cache must have room for pos0 + n_steps positions. */
int pop_generate_greedy(pop_model_t* m, const int32_t* first_tokens, int32_t pos0, int32_t n_steps, int32_t batch,
                        pop_kv_cache_t* kv_cache, int32_t* tokens_out, float* logits_scratch, void* stream);

/* The hidden states the last pop_prefill / pop_full_prefill call with the same (seq_len, batch) left in
 * the workspace, copied out on `stream` (either pointer may be NULL, not both):
 *   hidden_out  device fp32 [batch][seq_len][d_model]: the residual stream leaving the last layer that
 *               ran over the whole prompt. After pop_prefill this is x_{L_keep+1}; its rows 0..seq_len-2
 *               are the state H every pruned layer projects (paper Eq. 14) and hands on unchanged
 *               (Eq. 15). After pop_full_prefill it is x_{L+1} of Eq. 1.
 *   last_out    device fp32 [batch][d_model]: the last prompt position after ALL n_layers layers (the
 *               boundary token's state, paper Sec. 3.3), i.e. the input of the final norm.
 * Meaningful only until the next call that uses the workspace. Errors: POP_E_INVALID, POP_E_NOSPACE
 * (no workspace, or one too small for these sizes), POP_E_CUDA. */
int pop_read_hidden(pop_model_t* m, int32_t seq_len, int32_t batch, float* hidden_out, float* last_out,
                    void* stream);

/* Synchronise `stream`, then read and clear the device status word: POP_OK, POP_E_DEVICE_TIMEOUT if
 * a kernel gave up on a bounded wait, POP_E_INVALID if a kernel met an unusable token id, or
 * POP_E_CUDA. Once the word is raised the library's GEMM and attention kernels return at once, so
 * the outputs of that call (and of calls queued behind it) are undefined until it is read. */
int pop_last_status(pop_model_t* m, void* stream);

/* Number of kernel launches the last prefill call on this model enqueued. */
int64_t pop_last_launch_count(const pop_model_t* m);

void pop_free(pop_model_t* m);
const char* pop_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* POP_H_ */
