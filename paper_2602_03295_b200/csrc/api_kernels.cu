// C-ABI wrappers for the kernel-level entry points declared in pop_kernels.h.
#include "common.cuh"
#include "../../include/pop_kernels.h"

using namespace pop;

extern "C" {

int pop_k_gemm(const void* A, int64_t lda, int64_t a_bs, const void* B, int64_t ldb, int64_t b_bs, void* out,
               int64_t ldo, int64_t o_bs, int32_t M, int32_t N, int32_t K, int32_t batch, int32_t epilogue,
               int32_t act, int32_t n_valid, void* stream) {
  GemmArgs a{};
  a.A = static_cast<const bf16*>(A); a.lda = lda; a.a_batch_stride = a_bs;
  a.B = static_cast<const bf16*>(B); a.ldb = ldb; a.b_batch_stride = b_bs;
  a.out = out; a.ldo = ldo; a.out_batch_stride = o_bs;
  a.M = M; a.N = N; a.K = K; a.batch = batch;
  a.epilogue = epilogue; a.act = act; a.n_valid = n_valid;
  return launch_gemm(a, static_cast<cudaStream_t>(stream));
}

int pop_k_gemm_e4m3(const void* A, int64_t lda, const float* a_scale, const void* B, int64_t ldb,
                    const float* b_scale, void* out, int64_t ldo, int32_t M, int32_t N, int32_t K, int32_t epilogue,
                    int32_t act, int32_t n_valid, void* stream) {
  GemmArgs a{};
  a.A = static_cast<const bf16*>(A); a.lda = lda;
  a.B = static_cast<const bf16*>(B); a.ldb = ldb;
  a.out = out; a.ldo = ldo;
  a.M = M; a.N = N; a.K = K; a.batch = 1;
  a.epilogue = epilogue; a.act = act; a.n_valid = n_valid;
  a.fp8 = true; a.a_scale = a_scale; a.b_scale = b_scale;
  if (epilogue != EPI_STORE_BF16 && epilogue != EPI_STORE_F32 && epilogue != EPI_ADD_F32 &&
      epilogue != EPI_GATED_BF16)
    return POP_E_INVALID;
  return launch_gemm(a, static_cast<cudaStream_t>(stream));
}

int pop_k_rmsnorm_e4m3(const float* x, int64_t ldx, const float* gain, void* out, int64_t ldo, float* scale,
                       int32_t rows, int32_t d, float eps, void* stream) {
  return launch_rmsnorm_e4m3(x, ldx, gain, static_cast<uint8_t*>(out), ldo, scale, rows, d, eps,
                             static_cast<cudaStream_t>(stream));
}

int pop_k_quant_rows_e4m3(const void* in, int64_t ld_in, void* out, int64_t ld_out, float* scale, int32_t rows,
                          int32_t d, void* stream) {
  return launch_quant_rows_e4m3(static_cast<const bf16*>(in), ld_in, static_cast<uint8_t*>(out), ld_out, scale, rows, d,
                                static_cast<cudaStream_t>(stream));
}

int pop_k_quantize_e4m3(const void* w, int64_t n, void* out, float* scale, void* scratch4, void* stream) {
  return launch_quantize_weights_e4m3(static_cast<const bf16*>(w), n, static_cast<uint8_t*>(out), scale,
                                      static_cast<unsigned int*>(scratch4), static_cast<cudaStream_t>(stream));
}

int pop_k_gemm_norm(const void* A, int64_t lda, const void* B, int64_t ldb, void* out, int64_t ldo, int32_t M,
                    int32_t N, int32_t K, int32_t epilogue, int32_t act, int32_t n_valid, void* hn_out, int64_t ld_hn,
                    const float* gain_next, float* ss_out, int32_t ss_ld, const float* ss_in, int32_t ss_cnt,
                    int32_t ss_in_ld, int32_t norm_d, float norm_eps, void* stream) {
  GemmArgs a{};
  a.A = static_cast<const bf16*>(A); a.lda = lda;
  a.B = static_cast<const bf16*>(B); a.ldb = ldb;
  a.out = out; a.ldo = ldo;
  a.M = M; a.N = N; a.K = K; a.batch = 1;
  a.epilogue = epilogue; a.act = act; a.n_valid = n_valid;
  a.hn_out = static_cast<bf16*>(hn_out); a.ld_hn = ld_hn; a.gain_next = gain_next; a.ss_out = ss_out; a.ss_ld = ss_ld;
  a.ss_in = ss_in; a.ss_cnt = ss_cnt; a.ss_in_ld = ss_in_ld; a.norm_d = norm_d; a.norm_eps = norm_eps;
  if (epilogue == EPI_QKV_ROPE) return POP_E_INVALID;
  return launch_gemm(a, static_cast<cudaStream_t>(stream));
}

int pop_k_gemm_qkv_rope(const void* A, int64_t lda, int64_t a_bs, const void* W, int64_t ldw, int64_t w_bs, int32_t M,
                        int32_t K, int32_t batch, void* q_out, int64_t ldq, void* k_pool, void* v_pool,
                        int64_t pool_layer_stride, int32_t layer0, const int32_t* block_table,
                        int32_t max_pages_per_seq, int32_t page_size, const float* q_gain, const float* k_gain,
                        int64_t gain_gs, const void* table, int32_t n_q, int32_t n_kv, int32_t head_dim,
                        int32_t rows_per_seq, int32_t rows_written, int32_t pos0, float eps, void* stream) {
  RopeArgs r{};
  r.q_out = static_cast<bf16*>(q_out); r.ldq = ldq;
  r.k_pool = static_cast<bf16*>(k_pool); r.v_pool = static_cast<bf16*>(v_pool);
  r.pool_layer_stride = pool_layer_stride; r.layer0 = layer0;
  r.block_table = block_table; r.max_pages_per_seq = max_pages_per_seq; r.page_size = page_size;
  r.q_gain = q_gain; r.k_gain = k_gain; r.gain_group_stride = gain_gs;
  r.table = static_cast<const float2*>(table);
  r.n_q = n_q; r.n_kv = n_kv; r.hd = head_dim;
  r.rows = M; r.rows_per_seq = rows_per_seq; r.rows_written = rows_written; r.pos0 = pos0; r.groups = batch;
  r.eps = eps;
  GemmArgs a{};
  a.A = static_cast<const bf16*>(A); a.lda = lda; a.a_batch_stride = a_bs;
  a.B = static_cast<const bf16*>(W); a.ldb = ldw; a.b_batch_stride = w_bs;
  a.M = M; a.N = (n_q + 2 * n_kv) * head_dim; a.K = K; a.batch = batch;
  a.epilogue = EPI_QKV_ROPE; a.rope = &r;
  return launch_gemm(a, static_cast<cudaStream_t>(stream));
}

int pop_k_attention(const void* q, int64_t ldq, const void* k_pool, const void* v_pool, const int32_t* block_table,
                    void* out, int64_t ldo, int32_t batch, int32_t seq_len, int32_t q_pos0, int32_t kv_len,
                    int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t page_size, int32_t num_pages,
                    int32_t max_pages_per_seq, int32_t window, void* stream) {
  AttnArgs a{};
  a.q = static_cast<const bf16*>(q); a.ldq = ldq;
  a.k_pool = static_cast<const bf16*>(k_pool); a.v_pool = static_cast<const bf16*>(v_pool);
  a.block_table = block_table; a.out = static_cast<bf16*>(out); a.ldo = ldo;
  a.batch = batch; a.seq_len = seq_len; a.q_pos0 = q_pos0; a.kv_len = kv_len;
  a.n_q_heads = n_q_heads; a.n_kv_heads = n_kv_heads; a.head_dim = head_dim;
  a.page_size = page_size; a.num_pages = num_pages; a.max_pages_per_seq = max_pages_per_seq; a.window = window;
  return launch_attention(a, static_cast<cudaStream_t>(stream));
}

int pop_k_rmsnorm(const float* x, int64_t ldx, const float* gain, int64_t gain_stride, void* out, int64_t ldo,
                  int64_t out_gs, int32_t rows, int32_t d, int32_t groups, float eps, int32_t out_f32, void* stream) {
  if (!x || !gain || !out) return POP_E_INVALID;
  return launch_rmsnorm(x, ldx, gain, gain_stride, out, ldo, out_gs, rows, d, groups, eps, out_f32 != 0,
                        static_cast<cudaStream_t>(stream));
}

int pop_k_rope_table(void* table, int32_t n_pos, int32_t head_dim, float theta, void* stream) {
  if (!table || n_pos < 1 || head_dim < 2) return POP_E_INVALID;
  return launch_rope_table(static_cast<float2*>(table), n_pos, head_dim, theta, static_cast<cudaStream_t>(stream));
}

int pop_k_rope_cache(const float* in, int64_t ld_in, int64_t in_gs, void* q_out, int64_t ldq, void* k_pool,
                     void* v_pool, int64_t pool_layer_stride, int32_t layer0, const int32_t* block_table,
                     int32_t max_pages_per_seq, int32_t page_size, const float* q_gain, const float* k_gain,
                     int64_t gain_gs, const void* table, int32_t n_q, int32_t n_kv, int32_t head_dim, int32_t rows,
                     int32_t rows_per_seq, int32_t rows_written, int32_t pos0, int32_t groups, float eps,
                     void* stream) {
  if (!in || !k_pool || !v_pool || !block_table || !table || (n_q > 0 && !q_out)) return POP_E_INVALID;
  RopeArgs r{};
  r.in = in; r.ld_in = ld_in; r.in_group_stride = in_gs;
  r.q_out = static_cast<bf16*>(q_out); r.ldq = ldq;
  r.k_pool = static_cast<bf16*>(k_pool); r.v_pool = static_cast<bf16*>(v_pool);
  r.pool_layer_stride = pool_layer_stride; r.layer0 = layer0;
  r.block_table = block_table; r.max_pages_per_seq = max_pages_per_seq; r.page_size = page_size;
  r.q_gain = q_gain; r.k_gain = k_gain; r.gain_group_stride = gain_gs;
  r.table = static_cast<const float2*>(table);
  r.n_q = n_q; r.n_kv = n_kv; r.hd = head_dim;
  r.rows = rows; r.rows_per_seq = rows_per_seq; r.rows_written = rows_written; r.pos0 = pos0; r.groups = groups;
  r.eps = eps;
  return launch_rope_cache(r, static_cast<cudaStream_t>(stream));
}

int pop_k_gemv(const void* x, int64_t ldx, int32_t x_f32, const void* w, int64_t ldw, void* out, int64_t ldo,
               int32_t B, int32_t N, int32_t K, int32_t mode, int32_t act, int32_t n_valid, void* stream) {
  GemvArgs v{};
  v.x = x; v.ldx = ldx; v.x_f32 = x_f32 != 0; v.w = static_cast<const bf16*>(w); v.ldw = ldw;
  v.out = out; v.ldo = ldo; v.B = B; v.N = N; v.K = K; v.mode = mode; v.act = act; v.n_valid = n_valid;
  return launch_gemv(v, static_cast<cudaStream_t>(stream));
}

int pop_k_gemv_e4m3(const void* x, int64_t ldx, const void* w, int64_t ldw, const float* w_scale, void* out,
                    int64_t ldo, int32_t B, int32_t N, int32_t K, int32_t mode, int32_t act, int32_t n_valid,
                    void* stream) {
  GemvArgs v{};
  v.x = x; v.ldx = ldx; v.x_f32 = false; v.w = w; v.ldw = ldw; v.w_fp8 = true; v.w_scale = w_scale;
  v.out = out; v.ldo = ldo; v.B = B; v.N = N; v.K = K; v.mode = mode; v.act = act; v.n_valid = n_valid;
  return launch_gemv(v, static_cast<cudaStream_t>(stream));
}

int pop_k_decode_attention(const void* q, int64_t ldq, const void* k_pool, const void* v_pool,
                           const int32_t* block_table, int32_t max_pages_per_seq, int32_t page_size, float* partial,
                           int32_t* counters, void* out, int64_t ldo, int32_t batch, int32_t n_q, int32_t n_kv,
                           int32_t head_dim, int32_t kv_len, int32_t window, void* stream) {
  DecAttnArgs a{};
  a.counters = counters;
  a.q = static_cast<const bf16*>(q); a.ldq = ldq;
  a.k_pool = static_cast<const bf16*>(k_pool); a.v_pool = static_cast<const bf16*>(v_pool);
  a.block_table = block_table; a.max_pages_per_seq = max_pages_per_seq; a.page_size = page_size;
  a.partial = partial; a.out = static_cast<bf16*>(out); a.ldo = ldo;
  a.batch = batch; a.n_q = n_q; a.n_kv = n_kv; a.head_dim = head_dim; a.kv_len = kv_len; a.window = window;
  return launch_decode_attention(a, static_cast<cudaStream_t>(stream));
}

int pop_k_decode_attention_qkv(const float* qkv, int64_t ld_qkv, const float* q_gain, const float* k_gain, float eps,
                               const void* rope_row, void* k_pool, void* v_pool, const int32_t* block_table,
                               int32_t max_pages_per_seq, int32_t page_size, int32_t num_pages, float* partial,
                               int32_t* counters, void* out, int64_t ldo, int32_t batch, int32_t n_q, int32_t n_kv,
                               int32_t head_dim, int32_t kv_len, int32_t window, void* stream) {
  if (!qkv || !rope_row || !counters || (q_gain == nullptr) != (k_gain == nullptr)) return POP_E_INVALID;
  if (batch < 1 || page_size < 1 || num_pages < 1 || kv_len < 1) return POP_E_INVALID;
  if ((int64_t)ceil_div(kv_len, page_size) > max_pages_per_seq) return POP_E_NOSPACE;
  DecAttnArgs a{};
  a.counters = counters;
  a.qkv = qkv; a.ld_qkv = ld_qkv; a.q_gain = q_gain; a.k_gain = k_gain; a.eps = eps;
  a.table = static_cast<const float2*>(rope_row); a.table_pos0 = kv_len - 1;
  a.k_pool = static_cast<const bf16*>(k_pool); a.v_pool = static_cast<const bf16*>(v_pool);
  a.block_table = block_table; a.max_pages_per_seq = max_pages_per_seq; a.page_size = page_size;
  a.num_pages = num_pages;
  a.partial = partial; a.out = static_cast<bf16*>(out); a.ldo = ldo;
  a.batch = batch; a.n_q = n_q; a.n_kv = n_kv; a.head_dim = head_dim; a.kv_len = kv_len; a.window = window;
  return launch_decode_attention(a, static_cast<cudaStream_t>(stream));
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
void pop_k_profile(int32_t enable) { prof_enable(enable != 0); }
int pop_k_profile_summary(int32_t kind, double* total_ms, double* total_work, int64_t* launches) {
  return prof_summary(kind, total_ms, total_work, launches);
}
int64_t pop_k_launch_count(void) { return launch_count(); }
void pop_k_reset_launch_count(void) { reset_launch_count(); }

}  // extern "C"
