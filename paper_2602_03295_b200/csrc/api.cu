// Model-level entry points of pop.h: weight repacking, workspace layout, and the two prefill
// procedures (standard full-depth prefill; POP pruned prefill with boundary handling).
#include "common.cuh"

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using namespace pop;

namespace {

constexpr size_t kAlign = 1024;
constexpr int kMaxPrunedChunk = 16;   // pruned layers whose K/V projections run as one batched GEMM

struct LayerOffsets {   // byte offsets inside one layer block of the arena
  size_t wqkv, wo, wgu, wd, ln_in, ln_ffn, post_attn, post_ffn, q_norm, k_norm, total;
};

struct Workspace {
  float* x;          // [M][d] residual stream, fp32
  bf16* hn;          // [chunk][M][d] normalised activations (GEMM operand)
  float* qkv;        // unused (kept for layout stability)
  bf16* q;           // [M][q_dim]
  bf16* ao;          // [M][q_dim] attention output
  bf16* act;         // [M][F] gated activation
  float* t;          // [M][d] sublayer output of post-norm models
  float2* rope;      // [N][hd/2]
  float* xb;         // [B][d] boundary rows
  float* tb;         // [B][d]
  float* hb32;       // [B][d]
  bf16* hb;          // [B][d]
  float* qkvb;       // [B][qkv_dim]
  bf16* qb;          // unused (kept for layout stability): the decode attention finishes the queries itself
  bf16* ob;          // [B][q_dim]
  bf16* ab;          // [B][F]
  float* partial;    // [B][n_q][64][hd+2]
  float2* rope1;     // [hd/2] rotary row of the one position a decode step works on
  int32_t* cu;       // [B+1] packed-row prefix sums of a ragged batch
  int32_t* ctr;      // [2] device counters of the greedy loop: position, step
  int32_t* tok;      // [B] current token of every sequence in the greedy loop
  int32_t* dec_ctr;  // [B][n_kv] arrival counters of the decode attention's split merge (zero between launches)
  float* a_scale;    // [M] row scales of FP8 activations
  size_t total;
};

}  // namespace

struct pop_model {
  pop_config_t cfg;
  char* arena;
  size_t arena_bytes;
  LayerOffsets lo;
  size_t layer_stride;     // bytes
  size_t off_embed, off_lm_head, off_final_norm;
  int f_pad;
  int q_dim, kv_dim, qkv_dim;
  void* ws;
  size_t ws_bytes;
  int64_t last_launches;
  // FP8 copies of the kept layers' widest matrices (caller's memory, filled by pop_enable_fp8):
  // per layer E4M3 codes of wqkv [qkv_dim][d], the fused gate/up matrix [2 f_pad][d], wo [d][q_dim]
  // and w_down [d][d_ffn], then per layer four fp32 scales (same order)
  uint8_t* fp8;            // null = bf16 operands everywhere
  size_t fp8_layer_bytes;  // codes of one layer
  float* fp8_scales;       // [n_layers][4]
};

namespace {

bool config_ok(const pop_config_t* c) {
  if (!c || c->struct_size != sizeof(pop_config_t)) return false;
  if (c->n_layers < 1 || c->d_model < 8 || c->d_model % 8 || c->n_q_heads < 1 || c->n_kv_heads < 1) return false;
  if (c->n_q_heads % c->n_kv_heads || c->n_q_heads / c->n_kv_heads > 8) return false;
  if (c->head_dim != 64 && c->head_dim != 128 && c->head_dim != 256) return false;
  if (c->d_ffn < 8 || c->d_ffn % 8 || c->vocab < 1) return false;
  if (!(c->rms_eps >= 0.f) || !(c->rope_theta > 0.f)) return false;
  if (c->act < 0 || c->act > 1 || c->window < 0 || c->global_every < 0) return false;
  return true;
}

void layout(const pop_config_t& c, pop_model* m) {
  m->q_dim = c.n_q_heads * c.head_dim;
  m->kv_dim = c.n_kv_heads * c.head_dim;
  m->qkv_dim = m->q_dim + 2 * m->kv_dim;
  m->f_pad = (c.d_ffn + 127) / 128 * 128;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, kAlign); return r; };
  const size_t d = c.d_model;
  m->lo.wqkv = take((size_t)m->qkv_dim * d * 2);
  m->lo.wo = take(d * m->q_dim * 2);
  m->lo.wgu = take((size_t)2 * m->f_pad * d * 2);
  m->lo.wd = take(d * (size_t)c.d_ffn * 2);
  m->lo.ln_in = take(d * 4);
  m->lo.ln_ffn = take(d * 4);
  m->lo.post_attn = take(d * 4);
  m->lo.post_ffn = take(d * 4);
  m->lo.q_norm = take((size_t)c.head_dim * 4);
  m->lo.k_norm = take((size_t)c.head_dim * 4);
  m->lo.total = o;
  m->layer_stride = o;
  size_t g = (size_t)c.n_layers * m->layer_stride;
  m->off_embed = g; g = align_up(g + (size_t)c.vocab * d * 2, kAlign);
  m->off_lm_head = g; g = align_up(g + (size_t)c.vocab * d * 2, kAlign);
  m->off_final_norm = g; g = align_up(g + d * 4, kAlign);
  m->arena_bytes = g;
}

inline char* layer_base(const pop_model* m, int layer1) { return m->arena + (size_t)(layer1 - 1) * m->layer_stride; }
template <class T>
inline T* lp(const pop_model* m, int layer1, size_t off) { return reinterpret_cast<T*>(layer_base(m, layer1) + off); }

int layer_window(const pop_config_t& c, int layer1) {
  if (c.window <= 0) return 0;
  if (c.global_every > 0 && layer1 % c.global_every == 0) return 0;
  return c.window;
}

Workspace carve(const pop_model* m, char* base, int N, int B) {
  const pop_config_t& c = m->cfg;
  const size_t M = (size_t)B * N, d = c.d_model;
  const int chunk = std::min(kMaxPrunedChunk, std::max(1, c.n_layers - 1));
  Workspace w;
  size_t o = 0;
  auto take = [&](size_t bytes) { char* r = base + o; o = align_up(o + bytes, kAlign); return r; };
  w.x = (float*)take(M * d * 4);
  w.hn = (bf16*)take((size_t)chunk * M * d * 2);
  w.qkv = nullptr;   // projections never pass through memory in fp32: the GEMM epilogue finishes them
  w.q = (bf16*)take(M * m->q_dim * 2);
  w.ao = (bf16*)take(M * m->q_dim * 2);
  w.act = (bf16*)take(M * (size_t)c.d_ffn * 2);
  w.t = (float*)take(c.post_norms ? M * d * 4 : 0);
  w.rope = (float2*)take((size_t)N * (c.head_dim / 2) * 8);
  w.xb = (float*)take((size_t)B * d * 4);
  w.tb = (float*)take((size_t)B * d * 4);
  w.hb32 = (float*)take((size_t)B * d * 4);
  w.hb = (bf16*)take((size_t)B * d * 2);
  w.qkvb = (float*)take((size_t)B * m->qkv_dim * 4);
  w.qb = (bf16*)take((size_t)B * m->q_dim * 2);
  w.ob = (bf16*)take((size_t)B * m->q_dim * 2);
  w.ab = (bf16*)take((size_t)B * c.d_ffn * 2);
  w.partial = (float*)take((size_t)B * c.n_q_heads * 64 * (c.head_dim + 2) * 4);
  w.rope1 = (float2*)take((size_t)(c.head_dim / 2) * 8);
  w.cu = (int32_t*)take((size_t)(B + 1) * 4);
  w.ctr = (int32_t*)take(2 * 4);
  w.tok = (int32_t*)take((size_t)B * 4);
  w.dec_ctr = (int32_t*)take((size_t)B * c.n_kv_heads * 4);
  w.a_scale = (float*)take(M * 4);
  w.total = o;
  return w;
}

#define POP_TRY(expr)            \
  do {                           \
    int rc__ = (expr);           \
    if (rc__ != POP_OK) return rc__; \
  } while (0)

// one full decoder layer (paper Eq. 1-3) on all M = B*N rows of the residual stream
// Ragged batches: `cu` (device prefix sums, B + 1 entries) and `rows` (total packed rows) replace the
// uniform B x N layout; N is then the longest sequence.
// Chunked prefill: the N rows of every sequence are its positions pos0 .. pos0 + N - 1 (the cache
// already holds positions < pos0 of this layer; w.rope holds the rotary rows of these N positions).
int full_layer(pop_model* m, const Workspace& w, int l, int N, int B, const pop_kv_cache_t* kc, cudaStream_t s,
               const int32_t* cu = nullptr, int rows = 0, int pos0 = 0) {
  const pop_config_t& c = m->cfg;
  const int M = cu ? rows : B * N, d = c.d_model;
  const int64_t pool_layer_stride = (int64_t)kc->num_pages * kc->page_size * m->kv_dim;
  const bool fp8 = m->fp8 != nullptr;
  const uint8_t* w8 = fp8 ? m->fp8 + (size_t)(l - 1) * m->fp8_layer_bytes : nullptr;
  if (fp8)
    POP_TRY(launch_rmsnorm_e4m3(w.x, d, lp<float>(m, l, m->lo.ln_in), (uint8_t*)w.hn, d, w.a_scale, M, d, c.rms_eps, s));
  else
    POP_TRY(launch_rmsnorm(w.x, d, lp<float>(m, l, m->lo.ln_in), 0, w.hn, d, 0, M, d, 1, c.rms_eps, false, s));
  // QKV projection with per-head norm, RoPE and the cache append (Eq. 2-3) in the GEMM's epilogue
  RopeArgs r{};
  r.q_out = w.q; r.ldq = m->q_dim;
  r.k_pool = (bf16*)kc->k_pool; r.v_pool = (bf16*)kc->v_pool; r.pool_layer_stride = pool_layer_stride;
  r.layer0 = l - 1; r.block_table = kc->block_table; r.max_pages_per_seq = kc->max_pages_per_seq;
  r.page_size = kc->page_size; r.num_pages = kc->num_pages;
  r.q_gain = c.qk_norm ? lp<float>(m, l, m->lo.q_norm) : nullptr;
  r.k_gain = c.qk_norm ? lp<float>(m, l, m->lo.k_norm) : nullptr;
  // the epilogue indexes the table by absolute position: hand it the address row 0 would have
  r.table = w.rope - (int64_t)pos0 * (c.head_dim / 2); r.n_q = c.n_q_heads; r.n_kv = c.n_kv_heads; r.hd = c.head_dim;
  r.rows = M; r.rows_per_seq = N; r.rows_written = N; r.pos0 = pos0; r.groups = 1; r.eps = c.rms_eps;
  r.cu_seqlens = cu; r.batch = B; r.skip_last = 0;
  GemmArgs g{};
  g.A = w.hn; g.lda = d; g.B = lp<bf16>(m, l, m->lo.wqkv); g.ldb = d;
  g.M = M; g.N = m->qkv_dim; g.K = d; g.batch = 1; g.epilogue = EPI_QKV_ROPE; g.rope = &r;
  if (fp8) {
    g.fp8 = true; g.B = (const bf16*)w8; g.a_scale = w.a_scale; g.b_scale = m->fp8_scales + 4 * (l - 1);
  }
  POP_TRY(launch_gemm(g, s));
  AttnArgs a{};
  a.q = w.q; a.ldq = m->q_dim;
  a.k_pool = (const bf16*)kc->k_pool + (int64_t)(l - 1) * pool_layer_stride;
  a.v_pool = (const bf16*)kc->v_pool + (int64_t)(l - 1) * pool_layer_stride;
  a.block_table = kc->block_table; a.out = w.ao; a.ldo = m->q_dim;
  a.batch = B; a.seq_len = N; a.q_pos0 = pos0; a.kv_len = pos0 + N; a.cu_seqlens = cu; a.total_rows = cu ? M : 0;
  a.n_q_heads = c.n_q_heads; a.n_kv_heads = c.n_kv_heads; a.head_dim = c.head_dim;
  a.page_size = kc->page_size; a.num_pages = kc->num_pages; a.max_pages_per_seq = kc->max_pages_per_seq;
  a.window = layer_window(c, l);
  POP_TRY(launch_attention(a, s));
  // O projection + residual
  g = GemmArgs{};
  g.A = w.ao; g.lda = m->q_dim; g.B = lp<bf16>(m, l, m->lo.wo); g.ldb = m->q_dim;
  g.M = M; g.N = d; g.K = m->q_dim; g.batch = 1;
  if (fp8) {
    // the stored bf16 rows become codes in place (a row's codes fill the first half of its bytes)
    POP_TRY(launch_quant_rows_e4m3(w.ao, m->q_dim, (uint8_t*)w.ao, 2 * (int64_t)m->q_dim, w.a_scale, M, m->q_dim, s));
    g.fp8 = true; g.lda = 2 * (int64_t)m->q_dim; g.a_scale = w.a_scale;
    g.B = (const bf16*)(w8 + ((size_t)m->qkv_dim + 2 * (size_t)m->f_pad) * d);
    g.b_scale = m->fp8_scales + 4 * (l - 1) + 2;
  }
  if (c.post_norms) {
    g.out = w.t; g.ldo = d; g.epilogue = EPI_STORE_F32;
    POP_TRY(launch_gemm(g, s));
    POP_TRY(launch_postnorm_add(w.x, d, w.t, d, lp<float>(m, l, m->lo.post_attn), M, d, c.rms_eps, s));
  } else {
    g.out = w.x; g.ldo = d; g.epilogue = EPI_ADD_F32;
    POP_TRY(launch_gemm(g, s));
  }
  // gated FFN + residual
  if (fp8)
    POP_TRY(launch_rmsnorm_e4m3(w.x, d, lp<float>(m, l, m->lo.ln_ffn), (uint8_t*)w.hn, d, w.a_scale, M, d, c.rms_eps, s));
  else
    POP_TRY(launch_rmsnorm(w.x, d, lp<float>(m, l, m->lo.ln_ffn), 0, w.hn, d, 0, M, d, 1, c.rms_eps, false, s));
  g = GemmArgs{};
  g.A = w.hn; g.lda = d; g.B = lp<bf16>(m, l, m->lo.wgu); g.ldb = d;
  g.out = w.act; g.ldo = c.d_ffn; g.M = M; g.N = 2 * m->f_pad; g.K = d; g.batch = 1;
  g.epilogue = EPI_GATED_BF16; g.act = c.act; g.n_valid = c.d_ffn;
  if (fp8) {
    g.fp8 = true; g.B = (const bf16*)(w8 + (size_t)m->qkv_dim * d); g.a_scale = w.a_scale;
    g.b_scale = m->fp8_scales + 4 * (l - 1) + 1;
  }
  POP_TRY(launch_gemm(g, s));
  g = GemmArgs{};
  g.A = w.act; g.lda = c.d_ffn; g.B = lp<bf16>(m, l, m->lo.wd); g.ldb = c.d_ffn;
  g.M = M; g.N = d; g.K = c.d_ffn; g.batch = 1;
  if (fp8) {
    POP_TRY(launch_quant_rows_e4m3(w.act, c.d_ffn, (uint8_t*)w.act, 2 * (int64_t)c.d_ffn, w.a_scale, M, c.d_ffn, s));
    g.fp8 = true; g.lda = 2 * (int64_t)c.d_ffn; g.a_scale = w.a_scale;
    g.B = (const bf16*)(w8 + ((size_t)m->qkv_dim + 2 * (size_t)m->f_pad + (size_t)m->q_dim) * d);
    g.b_scale = m->fp8_scales + 4 * (l - 1) + 3;
  }
  if (c.post_norms) {
    g.out = w.t; g.ldo = d; g.epilogue = EPI_STORE_F32;
    POP_TRY(launch_gemm(g, s));
    POP_TRY(launch_postnorm_add(w.x, d, w.t, d, lp<float>(m, l, m->lo.post_ffn), M, d, c.rms_eps, s));
  } else {
    g.out = w.x; g.ldo = d; g.epilogue = EPI_ADD_F32;
    POP_TRY(launch_gemm(g, s));
  }
  return POP_OK;
}

// Independent K/V projections of pruned layers l0..l0+n-1 (paper Eq. 14) from the state H held in
// w.x, for positions 0..N-2 of every sequence; the state itself is left unchanged (Eq. 15).
int pruned_kv(pop_model* m, const Workspace& w, int l0, int n, int N, int B, const pop_kv_cache_t* kc,
              cudaStream_t s, const int32_t* cu = nullptr, int rows = 0, bool write_last = false, int pos0 = 0) {
  const pop_config_t& c = m->cfg;
  const int M = cu ? rows : B * N, d = c.d_model;
  const int64_t pool_layer_stride = (int64_t)kc->num_pages * kc->page_size * m->kv_dim;
  POP_TRY(launch_rmsnorm(w.x, d, lp<float>(m, l0, m->lo.ln_in), (int64_t)(m->layer_stride / 4), w.hn, d,
                         (int64_t)M * d, M, d, n, c.rms_eps, false, s));
  RopeArgs r{};
  r.q_out = nullptr; r.ldq = 0;
  r.k_pool = (bf16*)kc->k_pool; r.v_pool = (bf16*)kc->v_pool; r.pool_layer_stride = pool_layer_stride;
  r.layer0 = l0 - 1; r.block_table = kc->block_table; r.max_pages_per_seq = kc->max_pages_per_seq;
  r.page_size = kc->page_size; r.num_pages = kc->num_pages;
  r.q_gain = nullptr;
  r.k_gain = c.qk_norm ? lp<float>(m, l0, m->lo.k_norm) : nullptr;
  r.gain_group_stride = (int64_t)(m->layer_stride / 4);
  r.table = w.rope - (int64_t)pos0 * (c.head_dim / 2); r.n_q = 0; r.n_kv = c.n_kv_heads; r.hd = c.head_dim;
  r.rows = M; r.rows_per_seq = N; r.rows_written = write_last ? N : N - 1; r.pos0 = pos0; r.groups = n;
  r.eps = c.rms_eps;
  r.cu_seqlens = cu; r.batch = B; r.skip_last = write_last ? 0 : 1;
  // ONE batched GEMM over the pruned layers (the layer is the batch dimension of both operands);
  // its epilogue applies each layer's K norm and RoPE and writes the layer's cache entries
  GemmArgs g{};
  g.A = w.hn; g.lda = d; g.a_batch_stride = (int64_t)M * d;
  g.B = lp<bf16>(m, l0, m->lo.wqkv) + (int64_t)m->q_dim * d; g.ldb = d;
  g.b_batch_stride = (int64_t)(m->layer_stride / 2);
  g.M = M; g.N = 2 * m->kv_dim; g.K = d; g.batch = n; g.epilogue = EPI_QKV_ROPE; g.rope = &r;
  return launch_gemm(g, s);
}

// Boundary token as a decode step of layer l (paper Sec. 3.3): one row per sequence in w.xb.
// `table` holds rotary rows starting at position `table_pos0`.
int boundary_layer(pop_model* m, const Workspace& w, int l, int N, int B, const pop_kv_cache_t* kc,
                   const float2* table, int table_pos0, cudaStream_t s, const int32_t* cu = nullptr,
                   const int32_t* pos_dev = nullptr, int kv_first = 0) {
  const pop_config_t& c = m->cfg;
  const int d = c.d_model;
  const int64_t pool_layer_stride = (int64_t)kc->num_pages * kc->page_size * m->kv_dim;
  POP_TRY(launch_rmsnorm(w.xb, d, lp<float>(m, l, m->lo.ln_in), 0, w.hb, d, 0, B, d, 1, c.rms_eps, false, s));
  GemvArgs v{};
  v.x = w.hb; v.ldx = d; v.x_f32 = false; v.w = lp<bf16>(m, l, m->lo.wqkv); v.ldw = d;
  v.out = w.qkvb; v.ldo = m->qkv_dim; v.B = B; v.N = m->qkv_dim; v.K = d; v.mode = 0;
  // with FP8 enabled the single-position passes stream the E4M3 copies of the four matrices (half the
  // bytes) and keep their bf16 activations
  const uint8_t* w8 = m->fp8 ? m->fp8 + (size_t)(l - 1) * m->fp8_layer_bytes : nullptr;
  const float* sc8 = m->fp8 ? m->fp8_scales + 4 * (l - 1) : nullptr;
  if (w8) { v.w = w8; v.w_fp8 = true; v.w_scale = sc8; }
  POP_TRY(launch_gemv(v, s));
  // per-head norm, RoPE and the cache append of the new position happen inside the attention kernel
  DecAttnArgs a{};
  a.qkv = w.qkvb; a.ld_qkv = m->qkv_dim;
  a.q_gain = c.qk_norm ? lp<float>(m, l, m->lo.q_norm) : nullptr;
  a.k_gain = c.qk_norm ? lp<float>(m, l, m->lo.k_norm) : nullptr;
  a.table = table; a.table_pos0 = table_pos0; a.eps = c.rms_eps;
  a.cache_settled = true;   // the QKV GEMV sits between this launch and whatever wrote the cache
  a.k_pool = (const bf16*)kc->k_pool + (int64_t)(l - 1) * pool_layer_stride;
  a.v_pool = (const bf16*)kc->v_pool + (int64_t)(l - 1) * pool_layer_stride;
  a.block_table = kc->block_table; a.max_pages_per_seq = kc->max_pages_per_seq; a.page_size = kc->page_size;
  a.partial = w.partial; a.out = w.ob; a.ldo = m->q_dim;
  a.batch = B; a.n_q = c.n_q_heads; a.n_kv = c.n_kv_heads; a.head_dim = c.head_dim; a.kv_len = N;
  a.cu_seqlens = cu; a.pos_dev = pos_dev; a.counters = w.dec_ctr;
  a.kv_first = kv_first; a.num_pages = kc->num_pages;
  a.window = layer_window(c, l);
  POP_TRY(launch_decode_attention(a, s));
  v = GemvArgs{};
  v.x = w.ob; v.ldx = m->q_dim; v.w = lp<bf16>(m, l, m->lo.wo); v.ldw = m->q_dim; v.B = B; v.N = d; v.K = m->q_dim;
  if (w8) {
    v.w = w8 + ((size_t)m->qkv_dim + 2 * (size_t)m->f_pad) * d; v.w_fp8 = true; v.w_scale = sc8 + 2;
  }
  if (c.post_norms) {
    v.out = w.tb; v.ldo = d; v.mode = 0;
    POP_TRY(launch_gemv(v, s));
    POP_TRY(launch_postnorm_add(w.xb, d, w.tb, d, lp<float>(m, l, m->lo.post_attn), B, d, c.rms_eps, s));
  } else {
    v.out = w.xb; v.ldo = d; v.mode = 2;
    POP_TRY(launch_gemv(v, s));
  }
  POP_TRY(launch_rmsnorm(w.xb, d, lp<float>(m, l, m->lo.ln_ffn), 0, w.hb, d, 0, B, d, 1, c.rms_eps, false, s));
  v = GemvArgs{};
  v.x = w.hb; v.ldx = d; v.w = lp<bf16>(m, l, m->lo.wgu); v.ldw = d; v.out = w.ab; v.ldo = c.d_ffn;
  v.B = B; v.N = 2 * m->f_pad; v.K = d; v.mode = 3; v.act = c.act; v.n_valid = c.d_ffn;
  if (w8) { v.w = w8 + (size_t)m->qkv_dim * d; v.w_fp8 = true; v.w_scale = sc8 + 1; }
  POP_TRY(launch_gemv(v, s));
  v = GemvArgs{};
  v.x = w.ab; v.ldx = c.d_ffn; v.w = lp<bf16>(m, l, m->lo.wd); v.ldw = c.d_ffn; v.B = B; v.N = d; v.K = c.d_ffn;
  if (w8) {
    v.w = w8 + ((size_t)m->qkv_dim + 2 * (size_t)m->f_pad + (size_t)m->q_dim) * d; v.w_fp8 = true; v.w_scale = sc8 + 3;
  }
  if (c.post_norms) {
    v.out = w.tb; v.ldo = d; v.mode = 0;
    POP_TRY(launch_gemv(v, s));
    POP_TRY(launch_postnorm_add(w.xb, d, w.tb, d, lp<float>(m, l, m->lo.post_ffn), B, d, c.rms_eps, s));
  } else {
    v.out = w.xb; v.ldo = d; v.mode = 2;
    POP_TRY(launch_gemv(v, s));
  }
  return POP_OK;
}

int run_prefill(pop_model* m, const pop_input_t* in, int N, int B, int L_keep, pop_kv_cache_t* kc, float* logits,
                cudaStream_t s) {
  if (!m || !in || !in->tokens || !kc || !kc->k_pool || !kc->v_pool || !kc->block_table || !logits)
    return POP_E_INVALID;
  const pop_config_t& c = m->cfg;
  if (N < 1 || B < 1 || L_keep < 1 || L_keep > c.n_layers) return POP_E_INVALID;
  if ((int64_t)N * B > (int64_t)1 << 24) return POP_E_INVALID;
  if (!page_size_ok(kc->page_size) || kc->num_pages < 1) return POP_E_INVALID;
  if ((int64_t)ceil_div(N, kc->page_size) > kc->max_pages_per_seq) return POP_E_NOSPACE;
  if ((int64_t)ceil_div(N, kc->page_size) * B > kc->num_pages) return POP_E_NOSPACE;
  if (!m->ws) return POP_E_NOSPACE;
  const Workspace w = carve(m, (char*)m->ws, N, B);
  if (w.total > m->ws_bytes) return POP_E_NOSPACE;
  // the workspace is the caller's between calls: the split-merge counters start from zero in every call
  if (cudaMemsetAsync(w.dec_ctr, 0, (size_t)B * m->cfg.n_kv_heads * 4, s) != cudaSuccess) return POP_E_CUDA;
  const int64_t launches0 = launch_count();
  const int M = B * N, d = c.d_model;

  POP_TRY(launch_rope_table(w.rope, N, c.head_dim, c.rope_theta, s));
  POP_TRY(launch_embed(in->tokens, (const bf16*)(m->arena + m->off_embed), (const bf16*)in->embeds, w.x, M, d,
                       c.vocab, s));
  for (int l = 1; l <= L_keep; ++l) POP_TRY(full_layer(m, w, l, N, B, kc, s));
  if (L_keep < c.n_layers) {
    if (N > 1) {
      for (int l0 = L_keep + 1; l0 <= c.n_layers; l0 += kMaxPrunedChunk) {
        const int n = std::min(kMaxPrunedChunk, c.n_layers - l0 + 1);
        POP_TRY(pruned_kv(m, w, l0, n, N, B, kc, s));
      }
    }
    POP_TRY(launch_gather_rows(w.x, w.xb, B, d, N, N - 1, s));
    for (int l = L_keep + 1; l <= c.n_layers; ++l) POP_TRY(boundary_layer(m, w, l, N, B, kc, w.rope, 0, s));
  } else {
    POP_TRY(launch_gather_rows(w.x, w.xb, B, d, N, N - 1, s));
  }
  // final norm (kept in fp32) and output head on the last prompt position
  POP_TRY(launch_rmsnorm(w.xb, d, (const float*)(m->arena + m->off_final_norm), 0, w.hb32, d, 0, B, d, 1, c.rms_eps,
                         true, s));
  GemvArgs v{};
  v.x = w.hb32; v.ldx = d; v.x_f32 = true; v.w = (const bf16*)(m->arena + m->off_lm_head); v.ldw = d;
  v.out = logits; v.ldo = c.vocab; v.B = B; v.N = c.vocab; v.K = d; v.mode = 0;
  POP_TRY(launch_gemv(v, s));
  m->last_launches = launch_count() - launches0;
  return POP_OK;
}

// pop_prefill evaluated chunk by chunk over the positions (workspace for chunk_len rows per sequence
// instead of N): by causality, positions p0 .. p0+n-1 of a kept layer need the layer's cache entries
// of positions < p0 (already stored by the earlier chunks, Eq. 3) and nothing of later positions;
// Eq. 14 is per position. The last chunk carries the boundary token exactly as pop_prefill does.
int run_prefill_chunked(pop_model* m, const pop_input_t* in, int N, int B, int L_keep, int C, pop_kv_cache_t* kc,
                        float* logits, cudaStream_t s) {
  if (!m || !in || !in->tokens || !kc || !kc->k_pool || !kc->v_pool || !kc->block_table || !logits)
    return POP_E_INVALID;
  const pop_config_t& c = m->cfg;
  if (N < 1 || B < 1 || C < 1 || L_keep < 1 || L_keep > c.n_layers) return POP_E_INVALID;
  if (C > N) C = N;
  if ((int64_t)C * B > (int64_t)1 << 24 || N > (1 << 24)) return POP_E_INVALID;
  if (!page_size_ok(kc->page_size) || kc->num_pages < 1) return POP_E_INVALID;
  if ((int64_t)ceil_div(N, kc->page_size) > kc->max_pages_per_seq) return POP_E_NOSPACE;
  if ((int64_t)ceil_div(N, kc->page_size) * B > kc->num_pages) return POP_E_NOSPACE;
  if (!m->ws) return POP_E_NOSPACE;
  const Workspace w = carve(m, (char*)m->ws, C, B);
  if (w.total > m->ws_bytes) return POP_E_NOSPACE;
  if (cudaMemsetAsync(w.dec_ctr, 0, (size_t)B * m->cfg.n_kv_heads * 4, s) != cudaSuccess) return POP_E_CUDA;
  const int64_t launches0 = launch_count();
  const int d = c.d_model;
  const bf16* table = (const bf16*)(m->arena + m->off_embed);
  for (int p0 = 0; p0 < N; p0 += C) {
    const int n = std::min(C, N - p0);
    const bool last = p0 + n == N;
    POP_TRY(launch_rope_table(w.rope, n, c.head_dim, c.rope_theta, s, p0));
    for (int b = 0; b < B; ++b) {
      const int64_t row0 = (int64_t)b * N + p0;
      POP_TRY(launch_embed(in->tokens + row0, table, in->embeds ? (const bf16*)in->embeds + row0 * d : nullptr,
                           w.x + (int64_t)b * n * d, n, d, c.vocab, s));
    }
    for (int l = 1; l <= L_keep; ++l) POP_TRY(full_layer(m, w, l, n, B, kc, s, nullptr, 0, p0));
    if (L_keep < c.n_layers && (!last || n > 1)) {
      // every position but the boundary token (the last row of the last chunk) gets its Eq. 14 entries
      for (int l0 = L_keep + 1; l0 <= c.n_layers; l0 += kMaxPrunedChunk) {
        const int np = std::min(kMaxPrunedChunk, c.n_layers - l0 + 1);
        POP_TRY(pruned_kv(m, w, l0, np, n, B, kc, s, nullptr, 0, !last, p0));
      }
    }
    if (last) {
      POP_TRY(launch_gather_rows(w.x, w.xb, B, d, n, n - 1, s));
      for (int l = L_keep + 1; l <= c.n_layers; ++l) POP_TRY(boundary_layer(m, w, l, N, B, kc, w.rope, p0, s));
    }
  }
  POP_TRY(launch_rmsnorm(w.xb, d, (const float*)(m->arena + m->off_final_norm), 0, w.hb32, d, 0, B, d, 1, c.rms_eps,
                         true, s));
  GemvArgs v{};
  v.x = w.hb32; v.ldx = d; v.x_f32 = true; v.w = (const bf16*)(m->arena + m->off_lm_head); v.ldw = d;
  v.out = logits; v.ldo = c.vocab; v.B = B; v.N = c.vocab; v.K = d; v.mode = 0;
  POP_TRY(launch_gemv(v, s));
  m->last_launches = launch_count() - launches0;
  return POP_OK;
}

// pop_prefill for sequences of different lengths, packed back to back (no padding rows).
int run_prefill_ragged(pop_model* m, const pop_input_t* in, const int32_t* seq_lens, int B, int L_keep,
                       pop_kv_cache_t* kc, float* logits, cudaStream_t s) {
  if (!m || !in || !in->tokens || !seq_lens || !kc || !kc->k_pool || !kc->v_pool || !kc->block_table || !logits)
    return POP_E_INVALID;
  const pop_config_t& c = m->cfg;
  if (B < 1 || B > 4096 || L_keep < 1 || L_keep > c.n_layers) return POP_E_INVALID;
  std::vector<int32_t> cu(B + 1, 0);
  int N = 0;
  for (int b = 0; b < B; ++b) {
    if (seq_lens[b] < 1) return POP_E_INVALID;
    if ((int64_t)cu[b] + seq_lens[b] > (int64_t)1 << 24) return POP_E_INVALID;
    cu[b + 1] = cu[b] + seq_lens[b];
    N = std::max(N, (int)seq_lens[b]);
  }
  const int T = cu[B];
  if (!page_size_ok(kc->page_size) || kc->num_pages < 1) return POP_E_INVALID;
  if ((int64_t)ceil_div(N, kc->page_size) > kc->max_pages_per_seq) return POP_E_NOSPACE;
  if (!m->ws) return POP_E_NOSPACE;
  const Workspace w = carve(m, (char*)m->ws, N, B);        // laid out for B x N rows >= T
  if (w.total > m->ws_bytes) return POP_E_NOSPACE;
  // the workspace is the caller's between calls: the split-merge counters start from zero in every call
  if (cudaMemsetAsync(w.dec_ctr, 0, (size_t)B * m->cfg.n_kv_heads * 4, s) != cudaSuccess) return POP_E_CUDA;
  const int64_t launches0 = launch_count();
  const int d = c.d_model;
  // the prefix sums travel through the stream like everything else (the host vector is pageable
  // memory, which the runtime stages before returning)
  if (cudaMemcpyAsync(w.cu, cu.data(), (size_t)(B + 1) * 4, cudaMemcpyHostToDevice, s) != cudaSuccess) return POP_E_CUDA;
  POP_TRY(launch_rope_table(w.rope, N, c.head_dim, c.rope_theta, s));
  POP_TRY(launch_embed(in->tokens, (const bf16*)(m->arena + m->off_embed), (const bf16*)in->embeds, w.x, T, d,
                       c.vocab, s));
  for (int l = 1; l <= L_keep; ++l) POP_TRY(full_layer(m, w, l, N, B, kc, s, w.cu, T));
  if (L_keep < c.n_layers) {
    if (T > B) {      // some sequence has more than its boundary token
      for (int l0 = L_keep + 1; l0 <= c.n_layers; l0 += kMaxPrunedChunk) {
        const int n = std::min(kMaxPrunedChunk, c.n_layers - l0 + 1);
        POP_TRY(pruned_kv(m, w, l0, n, N, B, kc, s, w.cu, T));
      }
    }
    POP_TRY(launch_gather_last_rows(w.x, w.xb, B, d, w.cu, s));
    for (int l = L_keep + 1; l <= c.n_layers; ++l) POP_TRY(boundary_layer(m, w, l, N, B, kc, w.rope, 0, s, w.cu));
  } else {
    POP_TRY(launch_gather_last_rows(w.x, w.xb, B, d, w.cu, s));
  }
  POP_TRY(launch_rmsnorm(w.xb, d, (const float*)(m->arena + m->off_final_norm), 0, w.hb32, d, 0, B, d, 1, c.rms_eps,
                         true, s));
  GemvArgs v{};
  v.x = w.hb32; v.ldx = d; v.x_f32 = true; v.w = (const bf16*)(m->arena + m->off_lm_head); v.ldw = d;
  v.out = logits; v.ldo = c.vocab; v.B = B; v.N = c.vocab; v.K = d; v.mode = 0;
  POP_TRY(launch_gemv(v, s));
  m->last_launches = launch_count() - launches0;
  return POP_OK;
}

// POP prefill for an arbitrary pruned set S_skip (paper Eq. 4, Eq. 14-15; the layer-selection
// ablation of Sec. 4.4), in the paper's literal two phases: phase 1 walks the layers over the
// prompt, a kept layer in full, a pruned layer storing only its K/V projections of the state that
// reaches it; phase 2 runs the boundary token through ALL layers as a decode step, which also
// overwrites whatever phase 1 left at the last position of each layer's cache.
int run_prefill_skip(pop_model* m, const pop_input_t* in, int N, int B, const uint8_t* skip, int flags,
                     pop_kv_cache_t* kc, float* logits, cudaStream_t s) {
  if (flags & ~(POP_NO_BOUNDARY | POP_NO_INDEP_KV)) return POP_E_INVALID;
  const bool boundary = !(flags & POP_NO_BOUNDARY), indep_kv = !(flags & POP_NO_INDEP_KV);
  if (!m || !in || !in->tokens || !skip || !kc || !kc->k_pool || !kc->v_pool || !kc->block_table || !logits)
    return POP_E_INVALID;
  if (m->fp8) return POP_E_INVALID;   // FP8 operands: not in the literal two-phase evaluation
  const pop_config_t& c = m->cfg;
  if (N < 1 || B < 1 || (int64_t)N * B > (int64_t)1 << 24) return POP_E_INVALID;
  if (!page_size_ok(kc->page_size) || kc->num_pages < 1) return POP_E_INVALID;
  if ((int64_t)ceil_div(N, kc->page_size) > kc->max_pages_per_seq) return POP_E_NOSPACE;
  if ((int64_t)ceil_div(N, kc->page_size) * B > kc->num_pages) return POP_E_NOSPACE;
  if (!m->ws) return POP_E_NOSPACE;
  const Workspace w = carve(m, (char*)m->ws, N, B);
  if (w.total > m->ws_bytes) return POP_E_NOSPACE;
  // the workspace is the caller's between calls: the split-merge counters start from zero in every call
  if (cudaMemsetAsync(w.dec_ctr, 0, (size_t)B * m->cfg.n_kv_heads * 4, s) != cudaSuccess) return POP_E_CUDA;
  const int64_t launches0 = launch_count();
  const int M = B * N, d = c.d_model;
  POP_TRY(launch_rope_table(w.rope, N, c.head_dim, c.rope_theta, s));
  POP_TRY(launch_embed(in->tokens, (const bf16*)(m->arena + m->off_embed), (const bf16*)in->embeds, w.x, M, d,
                       c.vocab, s));
  if (boundary) POP_TRY(launch_gather_rows(w.x, w.xb, B, d, N, N - 1, s));   // x_1 of the boundary token, kept for phase 2
  if (N > 1 || !boundary) {
    for (int l = 1; l <= c.n_layers; ++l) {
      if (!skip[l - 1]) POP_TRY(full_layer(m, w, l, N, B, kc, s));
      else if (indep_kv) POP_TRY(pruned_kv(m, w, l, 1, N, B, kc, s, nullptr, 0, !boundary));
    }
  }
  if (boundary) {
    // without independent KV projections a pruned layer holds nothing before position N-1
    for (int l = 1; l <= c.n_layers; ++l)
      POP_TRY(boundary_layer(m, w, l, N, B, kc, w.rope, 0, s, nullptr, nullptr,
                             (!indep_kv && skip[l - 1]) ? N - 1 : 0));
  } else {
    // the last token went through the pruned model with all the others: its logits come from there
    POP_TRY(launch_gather_rows(w.x, w.xb, B, d, N, N - 1, s));
  }
  POP_TRY(launch_rmsnorm(w.xb, d, (const float*)(m->arena + m->off_final_norm), 0, w.hb32, d, 0, B, d, 1, c.rms_eps,
                         true, s));
  GemvArgs v{};
  v.x = w.hb32; v.ldx = d; v.x_f32 = true; v.w = (const bf16*)(m->arena + m->off_lm_head); v.ldw = d;
  v.out = logits; v.ldo = c.vocab; v.B = B; v.N = c.vocab; v.K = d; v.mode = 0;
  POP_TRY(launch_gemv(v, s));
  m->last_launches = launch_count() - launches0;
  return POP_OK;
}

// The kernels of one decode step. The position comes from the host (`pos`) or, when `pos_dev` is
// given, from device memory at run time.
int decode_body(pop_model* m, const Workspace& w, const int32_t* tokens, int pos, const int32_t* pos_dev, int B,
                pop_kv_cache_t* kc, float* logits, cudaStream_t s, const int32_t* layer_first_pos = nullptr) {
  const pop_config_t& c = m->cfg;
  const int d = c.d_model;
  POP_TRY(launch_rope_table(w.rope1, 1, c.head_dim, c.rope_theta, s, pos, pos_dev));
  POP_TRY(launch_embed(tokens, (const bf16*)(m->arena + m->off_embed), nullptr, w.xb, B, d, c.vocab, s));
  for (int l = 1; l <= c.n_layers; ++l)
    POP_TRY(boundary_layer(m, w, l, pos + 1, B, kc, w.rope1, pos, s, nullptr, pos_dev,
                           layer_first_pos ? layer_first_pos[l - 1] : 0));
  POP_TRY(launch_rmsnorm(w.xb, d, (const float*)(m->arena + m->off_final_norm), 0, w.hb32, d, 0, B, d, 1, c.rms_eps,
                         true, s));
  GemvArgs v{};
  v.x = w.hb32; v.ldx = d; v.x_f32 = true; v.w = (const bf16*)(m->arena + m->off_lm_head); v.ldw = d;
  v.out = logits; v.ldo = c.vocab; v.B = B; v.N = c.vocab; v.K = d; v.mode = 0;
  return launch_gemv(v, s);
}

// One decode step of the full model (the decode stage of paper Sec. 3.2, Eq. 11): every sequence's token at position `pos`
// (= entries already in the cache) goes through all L layers as the boundary token does.
int run_decode(pop_model* m, const int32_t* tokens, int pos, int B, pop_kv_cache_t* kc, float* logits,
               cudaStream_t s, const int32_t* layer_first_pos = nullptr) {
  if (!m || !tokens || !kc || !kc->k_pool || !kc->v_pool || !kc->block_table || !logits) return POP_E_INVALID;
  const pop_config_t& c = m->cfg;
  if (layer_first_pos)
    for (int l = 0; l < c.n_layers; ++l)
      if (layer_first_pos[l] < 0 || layer_first_pos[l] > pos) return POP_E_INVALID;
  if (pos < 0 || B < 1 || pos > (1 << 24)) return POP_E_INVALID;
  if (!page_size_ok(kc->page_size) || kc->num_pages < 1) return POP_E_INVALID;
  if ((int64_t)ceil_div(pos + 1, kc->page_size) > kc->max_pages_per_seq) return POP_E_NOSPACE;
  if ((int64_t)ceil_div(pos + 1, kc->page_size) * B > kc->num_pages) return POP_E_NOSPACE;
  if (!m->ws) return POP_E_NOSPACE;
  const Workspace w = carve(m, (char*)m->ws, 1, B);
  if (w.total > m->ws_bytes) return POP_E_NOSPACE;
  // the workspace is the caller's between calls: the split-merge counters start from zero in every call
  if (cudaMemsetAsync(w.dec_ctr, 0, (size_t)B * m->cfg.n_kv_heads * 4, s) != cudaSuccess) return POP_E_CUDA;
  const int64_t launches0 = launch_count();
  POP_TRY(decode_body(m, w, tokens, pos, nullptr, B, kc, logits, s, layer_first_pos));
  m->last_launches = launch_count() - launches0;
  return POP_OK;
}

// Greedy generation on the device: the decode step and the arg-max that feeds the next one are
// captured once into a CUDA graph whose kernels read the position from device memory, and the graph
// is replayed n_steps times on the caller's stream.
int run_generate(pop_model* m, const int32_t* first_tokens, int pos0, int n_steps, int B, pop_kv_cache_t* kc,
                 int32_t* tokens_out, float* logits, cudaStream_t s) {
  if (!m || !first_tokens || !kc || !kc->k_pool || !kc->v_pool || !kc->block_table || !tokens_out || !logits)
    return POP_E_INVALID;
  const pop_config_t& c = m->cfg;
  if (pos0 < 0 || B < 1 || n_steps < 1 || (int64_t)pos0 + n_steps > (1 << 24)) return POP_E_INVALID;
  if (prof_enabled()) return POP_E_INVALID;            // per-launch events cannot be recorded into a graph
  if (!page_size_ok(kc->page_size) || kc->num_pages < 1) return POP_E_INVALID;
  if ((int64_t)ceil_div(pos0 + n_steps, kc->page_size) > kc->max_pages_per_seq) return POP_E_NOSPACE;
  if (!m->ws) return POP_E_NOSPACE;
  const Workspace w = carve(m, (char*)m->ws, 1, B);
  if (w.total > m->ws_bytes) return POP_E_NOSPACE;
  // the workspace is the caller's between calls: the split-merge counters start from zero in every call
  if (cudaMemsetAsync(w.dec_ctr, 0, (size_t)B * m->cfg.n_kv_heads * 4, s) != cudaSuccess) return POP_E_CUDA;
  const int64_t launches0 = launch_count();
  if (cudaMemcpyAsync(w.tok, first_tokens, (size_t)B * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return POP_E_CUDA;
  POP_TRY(launch_set_counters(w.ctr, pos0, 0, s));
  // capture one step on a stream of the library's own
  cudaStream_t cs = nullptr;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  if (cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) != cudaSuccess) return POP_E_CUDA;
  int rc = POP_OK;
  if (cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal) != cudaSuccess) rc = POP_E_CUDA;
  if (rc == POP_OK) {
    rc = decode_body(m, w, w.tok, 0, w.ctr, B, kc, logits, cs);
    if (rc == POP_OK) rc = launch_argmax(logits, c.vocab, c.vocab, B, w.tok, tokens_out, n_steps, w.ctr + 1, cs);
    if (rc == POP_OK) rc = launch_bump_counters(w.ctr, cs);
    if (cudaStreamEndCapture(cs, &graph) != cudaSuccess || graph == nullptr) rc = rc == POP_OK ? POP_E_CUDA : rc;
  }
  if (rc == POP_OK && cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) rc = POP_E_CUDA;
  for (int i = 0; i < n_steps && rc == POP_OK; ++i)
    if (cudaGraphLaunch(exec, s) != cudaSuccess) rc = POP_E_CUDA;
  // an executable graph in flight is released when its last launch has completed
  if (exec) cudaGraphExecDestroy(exec);
  if (graph) cudaGraphDestroy(graph);
  cudaStreamDestroy(cs);
  cudaGetLastError();
  m->last_launches = launch_count() - launches0;
  return rc;
}

struct NameRef { int layer; std::string t; };
bool parse_name(const char* name, NameRef* out) {
  if (!name) return false;
  if (strncmp(name, "layers.", 7) == 0) {
    char* end = nullptr;
    long l = strtol(name + 7, &end, 10);
    if (!end || *end != '.' || l < 1) return false;
    out->layer = (int)l;
    out->t = end + 1;
    return true;
  }
  out->layer = 0;
  out->t = name;
  return true;
}

}  // namespace

extern "C" {

size_t pop_weight_arena_bytes(const pop_config_t* cfg) {
  if (!config_ok(cfg)) return 0;
  pop_model tmp{};
  layout(*cfg, &tmp);
  return tmp.arena_bytes;
}

int pop_load_weights(const pop_config_t* cfg, const pop_tensor_t* tensors, int32_t n_tensors, void* dev_arena,
                     size_t arena_bytes, void* stream, pop_model_t** out) {
  if (!config_ok(cfg) || !tensors || n_tensors < 1 || !dev_arena || !out) return POP_E_INVALID;
  if (reinterpret_cast<uintptr_t>(dev_arena) % kAlign) return POP_E_INVALID;
  pop_model* m = new (std::nothrow) pop_model{};
  if (!m) return POP_E_INVALID;
  m->cfg = *cfg;
  layout(*cfg, m);
  if (arena_bytes < m->arena_bytes) { delete m; return POP_E_NOSPACE; }
  m->arena = static_cast<char*>(dev_arena);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const pop_config_t& c = *cfg;
  const size_t d = c.d_model;
  const int L = c.n_layers;
  const int n_layer_kinds = 13;
  std::vector<char> seen((size_t)L * n_layer_kinds + 3, 0);
  static const char* kinds[13] = {"ln_in", "wq", "wk", "wv", "wo", "ln_ffn", "w_gate", "w_up", "w_down",
                                  "q_norm", "k_norm", "post_attn_norm", "post_ffn_norm"};
  bool cuda_ok = true;
  auto copy = [&](void* dst, const void* src, size_t bytes) {
    if (cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess) cuda_ok = false;
  };
  // zero the padded gate/up blocks first
  if (m->f_pad != c.d_ffn)
    for (int l = 1; l <= L; ++l)
      if (cudaMemsetAsync(layer_base(m, l) + m->lo.wgu, 0, (size_t)2 * m->f_pad * d * 2, s) != cudaSuccess)
        cuda_ok = false;
  int rc = POP_OK;
  for (int i = 0; i < n_tensors && rc == POP_OK; ++i) {
    const pop_tensor_t& t = tensors[i];
    NameRef nr;
    if (!t.dev_ptr || !parse_name(t.name, &nr)) { rc = POP_E_INVALID; break; }
    auto want = [&](int dtype, int64_t s0, int64_t s1) {
      if (t.dtype != dtype) return false;
      if (s1 == 0) return t.ndim == 1 && t.shape[0] == s0;
      return t.ndim == 2 && t.shape[0] == s0 && t.shape[1] == s1;
    };
    if (nr.layer == 0) {
      if (nr.t == "embed") {
        if (!want(0, c.vocab, d)) { rc = POP_E_INVALID; break; }
        copy(m->arena + m->off_embed, t.dev_ptr, (size_t)c.vocab * d * 2);
        seen[(size_t)L * n_layer_kinds + 0] = 1;
      } else if (nr.t == "lm_head") {
        if (!want(0, c.vocab, d)) { rc = POP_E_INVALID; break; }
        copy(m->arena + m->off_lm_head, t.dev_ptr, (size_t)c.vocab * d * 2);
        seen[(size_t)L * n_layer_kinds + 1] = 1;
      } else if (nr.t == "final_norm") {
        if (!want(1, d, 0)) { rc = POP_E_INVALID; break; }
        copy(m->arena + m->off_final_norm, t.dev_ptr, d * 4);
        seen[(size_t)L * n_layer_kinds + 2] = 1;
      } else {
        rc = POP_E_INVALID;
      }
      continue;
    }
    if (nr.layer > L) { rc = POP_E_INVALID; break; }
    int kind = -1;
    for (int k = 0; k < n_layer_kinds; ++k)
      if (nr.t == kinds[k]) kind = k;
    if (kind < 0) { rc = POP_E_INVALID; break; }
    char* lb = layer_base(m, nr.layer);
    const size_t F = c.d_ffn;
    switch (kind) {
      case 0: if (!want(1, d, 0)) rc = POP_E_INVALID; else copy(lb + m->lo.ln_in, t.dev_ptr, d * 4); break;
      case 1: if (!want(0, m->q_dim, d)) rc = POP_E_INVALID; else copy(lb + m->lo.wqkv, t.dev_ptr, (size_t)m->q_dim * d * 2); break;
      case 2: if (!want(0, m->kv_dim, d)) rc = POP_E_INVALID;
              else copy(lb + m->lo.wqkv + (size_t)m->q_dim * d * 2, t.dev_ptr, (size_t)m->kv_dim * d * 2); break;
      case 3: if (!want(0, m->kv_dim, d)) rc = POP_E_INVALID;
              else copy(lb + m->lo.wqkv + (size_t)(m->q_dim + m->kv_dim) * d * 2, t.dev_ptr, (size_t)m->kv_dim * d * 2); break;
      case 4: if (!want(0, d, m->q_dim)) rc = POP_E_INVALID; else copy(lb + m->lo.wo, t.dev_ptr, d * m->q_dim * 2); break;
      case 5: if (!want(1, d, 0)) rc = POP_E_INVALID; else copy(lb + m->lo.ln_ffn, t.dev_ptr, d * 4); break;
      case 6:
      case 7: {
        // gate rows [128t, 128t+128) -> arena rows [256t, 256t+128); up rows -> [256t+128, 256t+256)
        if (!want(0, F, d)) { rc = POP_E_INVALID; break; }
        char* dst = lb + m->lo.wgu + (kind == 7 ? (size_t)128 * d * 2 : 0);
        const size_t full_blocks = F / 128, tail = F % 128;
        if (full_blocks &&
            cudaMemcpy2DAsync(dst, (size_t)256 * d * 2, t.dev_ptr, (size_t)128 * d * 2, (size_t)128 * d * 2,
                              full_blocks, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
          cuda_ok = false;
        if (tail)
          copy(dst + full_blocks * 256 * d * 2, (const char*)t.dev_ptr + full_blocks * 128 * d * 2, tail * d * 2);
        break;
      }
      case 8: if (!want(0, d, F)) rc = POP_E_INVALID; else copy(lb + m->lo.wd, t.dev_ptr, d * F * 2); break;
      case 9: if (!want(1, c.head_dim, 0)) rc = POP_E_INVALID; else copy(lb + m->lo.q_norm, t.dev_ptr, (size_t)c.head_dim * 4); break;
      case 10: if (!want(1, c.head_dim, 0)) rc = POP_E_INVALID; else copy(lb + m->lo.k_norm, t.dev_ptr, (size_t)c.head_dim * 4); break;
      case 11: if (!want(1, d, 0)) rc = POP_E_INVALID; else copy(lb + m->lo.post_attn, t.dev_ptr, d * 4); break;
      case 12: if (!want(1, d, 0)) rc = POP_E_INVALID; else copy(lb + m->lo.post_ffn, t.dev_ptr, d * 4); break;
    }
    if (rc == POP_OK) seen[(size_t)(nr.layer - 1) * n_layer_kinds + kind] = 1;
  }
  if (rc == POP_OK && !cuda_ok) rc = POP_E_CUDA;
  if (rc == POP_OK) {
    for (int l = 0; l < L && rc == POP_OK; ++l)
      for (int k = 0; k < n_layer_kinds; ++k) {
        const bool needed = k <= 8 || ((k == 9 || k == 10) && c.qk_norm) || (k >= 11 && c.post_norms);
        if (needed && !seen[(size_t)l * n_layer_kinds + k]) rc = POP_E_MISSING;
      }
    for (int k = 0; k < 3; ++k)
      if (!seen[(size_t)L * n_layer_kinds + k]) rc = POP_E_MISSING;
  }
  if (rc != POP_OK) { delete m; return rc; }
  *out = m;
  return POP_OK;
}

size_t pop_workspace_bytes(const pop_model_t* m, int32_t seq_len, int32_t batch) {
  if (!m || seq_len < 1 || batch < 1) return 0;
  return carve(m, nullptr, seq_len, batch).total;
}

int pop_set_workspace(pop_model_t* m, void* dev_ws, size_t bytes) {
  if (!m || !dev_ws || reinterpret_cast<uintptr_t>(dev_ws) % kAlign) return POP_E_INVALID;
  m->ws = dev_ws;
  m->ws_bytes = bytes;
  return POP_OK;
}

static size_t fp8_layer_codes(const pop_model* m) {
  const size_t d = m->cfg.d_model;
  return ((size_t)m->qkv_dim + 2 * (size_t)m->f_pad + (size_t)m->q_dim + (size_t)m->cfg.d_ffn) * d;
}

size_t pop_fp8_arena_bytes(const pop_model_t* m) {
  if (!m) return 0;
  return align_up(fp8_layer_codes(m), kAlign) * m->cfg.n_layers + align_up((size_t)m->cfg.n_layers * 4 * 4 + 4, kAlign);
}

int pop_enable_fp8(pop_model_t* m, void* dev_arena, size_t bytes, void* stream) {
  if (!m) return POP_E_INVALID;
  if (!dev_arena) {
    m->fp8 = nullptr;
    return POP_OK;
  }
  const pop_config_t& c = m->cfg;
  if (reinterpret_cast<uintptr_t>(dev_arena) % kAlign) return POP_E_INVALID;
  // code rows are GEMM operands (16-byte granules), activation rows are quantised by one CTA each
  if (c.d_model % 16 || m->q_dim % 16 || c.d_ffn % 16 || c.d_ffn > 16384 || m->q_dim > 16384) return POP_E_INVALID;
  if (bytes < pop_fp8_arena_bytes(m)) return POP_E_NOSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t d = c.d_model;
  const size_t layer = align_up(fp8_layer_codes(m), kAlign);
  uint8_t* base = static_cast<uint8_t*>(dev_arena);
  float* scales = reinterpret_cast<float*>(base + layer * c.n_layers);
  unsigned int* scratch = reinterpret_cast<unsigned int*>(scales + 4 * c.n_layers);
  for (int l = 1; l <= c.n_layers; ++l) {
    uint8_t* dst = base + layer * (l - 1);
    float* sc = scales + 4 * (l - 1);
    POP_TRY(launch_quantize_weights_e4m3(lp<bf16>(m, l, m->lo.wqkv), (int64_t)m->qkv_dim * d, dst, sc, scratch, s));
    dst += (size_t)m->qkv_dim * d;
    POP_TRY(launch_quantize_weights_e4m3(lp<bf16>(m, l, m->lo.wgu), (int64_t)2 * m->f_pad * d, dst, sc + 1, scratch, s));
    dst += (size_t)2 * m->f_pad * d;
    POP_TRY(launch_quantize_weights_e4m3(lp<bf16>(m, l, m->lo.wo), (int64_t)m->q_dim * d, dst, sc + 2, scratch, s));
    dst += (size_t)m->q_dim * d;
    POP_TRY(launch_quantize_weights_e4m3(lp<bf16>(m, l, m->lo.wd), (int64_t)c.d_ffn * d, dst, sc + 3, scratch, s));
  }
  m->fp8 = base;
  m->fp8_layer_bytes = layer;
  m->fp8_scales = scales;
  return POP_OK;
}

int pop_prefill(pop_model_t* m, const pop_input_t* in, int32_t seq_len, int32_t batch, int32_t L_keep,
                pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream) {
  return run_prefill(m, in, seq_len, batch, L_keep, kv_cache_out, logits_out, static_cast<cudaStream_t>(stream));
}

int pop_full_prefill(pop_model_t* m, const pop_input_t* in, int32_t seq_len, int32_t batch,
                     pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream) {
  if (!m) return POP_E_INVALID;
  return run_prefill(m, in, seq_len, batch, m->cfg.n_layers, kv_cache_out, logits_out,
                     static_cast<cudaStream_t>(stream));
}

int pop_prefill_ragged(pop_model_t* m, const pop_input_t* in, const int32_t* seq_lens, int32_t batch, int32_t L_keep,
                       pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream) {
  return run_prefill_ragged(m, in, seq_lens, batch, L_keep, kv_cache_out, logits_out,
                            static_cast<cudaStream_t>(stream));
}

int pop_prefill_skip(pop_model_t* m, const pop_input_t* in, int32_t seq_len, int32_t batch, const uint8_t* skip,
                     pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream) {
  return run_prefill_skip(m, in, seq_len, batch, skip, 0, kv_cache_out, logits_out,
                          static_cast<cudaStream_t>(stream));
}

int pop_prefill_chunked(pop_model_t* m, const pop_input_t* in, int32_t seq_len, int32_t batch, int32_t L_keep,
                        int32_t chunk_len, pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream) {
  return run_prefill_chunked(m, in, seq_len, batch, L_keep, chunk_len, kv_cache_out, logits_out,
                             static_cast<cudaStream_t>(stream));
}

int pop_prefill_ablation(pop_model_t* m, const pop_input_t* in, int32_t seq_len, int32_t batch, const uint8_t* skip,
                         int32_t flags, pop_kv_cache_t* kv_cache_out, float* logits_out, void* stream) {
  return run_prefill_skip(m, in, seq_len, batch, skip, flags, kv_cache_out, logits_out,
                          static_cast<cudaStream_t>(stream));
}

int pop_decode_step_from(pop_model_t* m, const int32_t* tokens, int32_t pos, int32_t batch,
                         const int32_t* layer_first_pos, pop_kv_cache_t* kv_cache, float* logits_out, void* stream) {
  return run_decode(m, tokens, pos, batch, kv_cache, logits_out, static_cast<cudaStream_t>(stream),
                    layer_first_pos);
}

int pop_decode_step(pop_model_t* m, const int32_t* tokens, int32_t pos, int32_t batch, pop_kv_cache_t* kv_cache,
                    float* logits_out, void* stream) {
  return run_decode(m, tokens, pos, batch, kv_cache, logits_out, static_cast<cudaStream_t>(stream));
}

int pop_generate_greedy(pop_model_t* m, const int32_t* first_tokens, int32_t pos0, int32_t n_steps, int32_t batch,
                        pop_kv_cache_t* kv_cache, int32_t* tokens_out, float* logits_scratch, void* stream) {
  return run_generate(m, first_tokens, pos0, n_steps, batch, kv_cache, tokens_out, logits_scratch,
                      static_cast<cudaStream_t>(stream));
}

int pop_read_hidden(pop_model_t* m, int32_t seq_len, int32_t batch, float* hidden_out, float* last_out,
                    void* stream) {
  if (!m || seq_len < 1 || batch < 1 || (!hidden_out && !last_out)) return POP_E_INVALID;
  if (!m->ws) return POP_E_NOSPACE;
  const Workspace w = carve(m, (char*)m->ws, seq_len, batch);
  if (w.total > m->ws_bytes) return POP_E_NOSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t d = m->cfg.d_model;
  if (hidden_out && cudaMemcpyAsync(hidden_out, w.x, (size_t)batch * seq_len * d * 4, cudaMemcpyDeviceToDevice, s) !=
                        cudaSuccess)
    return POP_E_CUDA;
  if (last_out && cudaMemcpyAsync(last_out, w.xb, (size_t)batch * d * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return POP_E_CUDA;
  return POP_OK;
}

int pop_last_status(pop_model_t* m, void* stream) {
  if (!m) return POP_E_INVALID;
  return read_and_clear_status(static_cast<cudaStream_t>(stream));
}

int64_t pop_last_launch_count(const pop_model_t* m) { return m ? m->last_launches : 0; }

void pop_free(pop_model_t* m) { delete m; }

}  // extern "C"
