// Bandwidth-bound kernels around the tensor-core GEMMs: embedding gather, RMSNorm (the LN of
// paper Eq. 2 / Eq. 14), the rotary table, RoPE + per-head norm + paged cache write (Eq. 2-3, and
// Eq. 14 for pruned layers), and the post-norm residual add of post-norm models.
#include "common.cuh"

namespace pop {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// block-wide sum, result broadcast to every thread; `red` holds >= 32 floats
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  const int nw = (blockDim.x + 31) >> 5;
  float t = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
  if (w == 0) {
    t = warp_sum(t);
    if (l == 0) red[0] = t;
  }
  __syncthreads();
  return red[0];
}

// ------------------------------------------------------------------------------ embedding
// A token id the host cannot see may be unusable: negative with no embedding rows supplied, or
// >= vocab. Such a row becomes zeros, nothing is dereferenced for it, and the status word is raised
// to POP_E_INVALID (the kernels queued behind then return at once; the caller reads the word).
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const bf16* __restrict__ table,
                             const bf16* __restrict__ embeds, float* __restrict__ x, int d, int vocab,
                             int* __restrict__ status) {
  const int row = blockIdx.x;
  const int tok = tokens[row];
  float* dst = x + (int64_t)row * d;
  if ((tok < 0 && embeds == nullptr) || tok >= vocab) {
    if (threadIdx.x == 0) atomicMin(status, (int)POP_E_INVALID);
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4)
      *reinterpret_cast<float4*>(dst + c) = make_float4(0.f, 0.f, 0.f, 0.f);
    return;
  }
  const bf16* src = (tok >= 0) ? table + (int64_t)tok * d : embeds + (int64_t)row * d;
  for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
    const uint4 raw = *reinterpret_cast<const uint4*>(src + c);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
    float4 a, b;
    float2 f;
    f = __bfloat1622float2(h[0]); a.x = f.x; a.y = f.y;
    f = __bfloat1622float2(h[1]); a.z = f.x; a.w = f.y;
    f = __bfloat1622float2(h[2]); b.x = f.x; b.y = f.y;
    f = __bfloat1622float2(h[3]); b.z = f.x; b.w = f.y;
    *reinterpret_cast<float4*>(dst + c) = a;
    *reinterpret_cast<float4*>(dst + c + 4) = b;
  }
}

// ------------------------------------------------------------------------------ RMSNorm
// out[g][row][:] = x[row][:] * rsqrt(mean(x^2) + eps) * gain[g][:], g = blockIdx.y.
// OUT_F32: write fp32 (final norm feeding the output head), else bf16 (GEMM operand).
template <bool OUT_F32>
__global__ void rmsnorm_kernel(const float* __restrict__ x, int64_t ldx, const float* __restrict__ gain,
                               int64_t gain_stride, void* __restrict__ out, int64_t ldo, int64_t out_group_stride,
                               int d, float eps) {
  // The first RN_CACHE float4 per thread of the row and of the gain stay in registers (rows up to
  // 16 * blockDim floats are read exactly once); longer rows re-read their remainder from L1/L2.
  constexpr int RN_CACHE = 4;
  __shared__ float red[32];
  chain_trigger();
  // Rows are walked from the last to the first: the kernel that produced x wrote its highest rows last,
  // so those are the ones still in L2, and the GEMM that consumes the output starts at row 0, which this
  // order writes last.
  const int row = gridDim.x - 1 - blockIdx.x, g = blockIdx.y;
  const float* xr = x + (int64_t)row * ldx;
  const float* gr = gain + (int64_t)g * gain_stride;
  const int step = blockDim.x * 4;
  // gains are weights, never written by a kernel: their loads go out before the wait on the producer of x
  float4 gv[RN_CACHE];
#pragma unroll
  for (int i = 0; i < RN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    gv[i] = c < d ? *reinterpret_cast<const float4*>(gr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  chain_wait();
  float4 xv[RN_CACHE];
#pragma unroll
  for (int i = 0; i < RN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    xv[i] = c < d ? *reinterpret_cast<const float4*>(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < RN_CACHE; ++i) {
    const float4 v = xv[i];
    if (threadIdx.x * 4 + i * step < d) ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  for (int c = threadIdx.x * 4 + RN_CACHE * step; c < d; c += step) {
    const float4 v = *reinterpret_cast<const float4*>(xr + c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, red);
  const float rstd = rsqrtf(ss / (float)d + eps);
  auto emit = [&](int c, const float4& v, const float4& w) {
    const float a = v.x * rstd * w.x, b = v.y * rstd * w.y, c2 = v.z * rstd * w.z, e = v.w * rstd * w.w;
    if (OUT_F32) {
      float* o = reinterpret_cast<float*>(out) + (int64_t)g * out_group_stride + (int64_t)row * ldo + c;
      *reinterpret_cast<float4*>(o) = make_float4(a, b, c2, e);
    } else {
      bf16* o = reinterpret_cast<bf16*>(out) + (int64_t)g * out_group_stride + (int64_t)row * ldo + c;
      __nv_bfloat162 p0 = __floats2bfloat162_rn(a, b), p1 = __floats2bfloat162_rn(c2, e);
      uint2 w2;
      w2.x = *reinterpret_cast<uint32_t*>(&p0);
      w2.y = *reinterpret_cast<uint32_t*>(&p1);
      *reinterpret_cast<uint2*>(o) = w2;
    }
  };
#pragma unroll
  for (int i = 0; i < RN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    if (c < d) emit(c, xv[i], gv[i]);
  }
  for (int c = threadIdx.x * 4 + RN_CACHE * step; c < d; c += step)
    emit(c, *reinterpret_cast<const float4*>(xr + c), *reinterpret_cast<const float4*>(gr + c));
}

// x[row][:] += rmsnorm(t[row][:]) * gain      (post-norm models: norm of the sublayer output)
__global__ void postnorm_add_kernel(float* __restrict__ x, int64_t ldx, const float* __restrict__ t, int64_t ldt,
                                    const float* __restrict__ gain, int d, float eps) {
  // the sublayer output row stays in registers (rows up to 16 floats per thread are read once)
  constexpr int PN_CACHE = 4;
  __shared__ float red[32];
  chain_trigger();
  const int row = blockIdx.x;
  const float* tr = t + (int64_t)row * ldt;
  float* xr = x + (int64_t)row * ldx;
  const int step = blockDim.x * 4;
  float4 gv[PN_CACHE];                      // weights: loaded before the wait on the producer of t
#pragma unroll
  for (int i = 0; i < PN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    gv[i] = c < d ? *reinterpret_cast<const float4*>(gain + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  chain_wait();
  float4 tv[PN_CACHE], xv[PN_CACHE];
#pragma unroll
  for (int i = 0; i < PN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    tv[i] = c < d ? *reinterpret_cast<const float4*>(tr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    xv[i] = c < d ? *reinterpret_cast<const float4*>(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < PN_CACHE; ++i) {
    const float4 v = tv[i];
    if (threadIdx.x * 4 + i * step < d) ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  for (int c = threadIdx.x * 4 + PN_CACHE * step; c < d; c += step) {
    const float4 v = *reinterpret_cast<const float4*>(tr + c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, red);
  const float rstd = rsqrtf(ss / (float)d + eps);
#pragma unroll
  for (int i = 0; i < PN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    if (c < d) {
      const float4 v = tv[i], w = gv[i];
      float4 o = xv[i];
      o.x += v.x * rstd * w.x; o.y += v.y * rstd * w.y; o.z += v.z * rstd * w.z; o.w += v.w * rstd * w.w;
      *reinterpret_cast<float4*>(xr + c) = o;
    }
  }
  for (int c = threadIdx.x * 4 + PN_CACHE * step; c < d; c += step) {
    const float4 v = *reinterpret_cast<const float4*>(tr + c);
    const float4 w = *reinterpret_cast<const float4*>(gain + c);
    float4 o = *reinterpret_cast<float4*>(xr + c);
    o.x += v.x * rstd * w.x; o.y += v.y * rstd * w.y; o.z += v.z * rstd * w.z; o.w += v.w * rstd * w.w;
    *reinterpret_cast<float4*>(xr + c) = o;
  }
}

// ------------------------------------------------------------------------------ rotary table
// table[pos][j] = (cos, sin)(pos * theta^(-2j/hd)), evaluated in fp64, stored fp32.
__global__ void rope_table_kernel(float2* __restrict__ table, int n_pos, int half, double theta, int first_pos,
                                  const int32_t* __restrict__ first_pos_dev) {
  if (first_pos_dev != nullptr) first_pos = *first_pos_dev;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pos * half) return;
  const int pos = i / half, j = i - pos * half;
  const double inv = exp2(-(2.0 * j / (2.0 * half)) * log2(theta));
  double s, c;
  sincos((double)(first_pos + pos) * inv, &s, &c);
  table[i] = make_float2((float)c, (float)s);
}

// ------------------------------------------------------------------------------ RoPE + cache write
// One warp per (row, head). Input row layout (fp32): [n_q heads | n_kv heads (k) | n_kv heads (v)] * hd.
// q heads: optional per-head RMSNorm, RoPE, -> q_out bf16. k heads: optional norm, RoPE, -> K pool.
// v heads: -> V pool. Row r of group g maps to sequence b = r / rows_per_seq, position pos0 + r % rows_per_seq;
// rows with (r % rows_per_seq) >= rows_written are skipped (pruned layers skip the boundary position).
struct RopeDev {
  const float* in; int64_t ld_in; int64_t in_group_stride;
  bf16* q_out; int64_t ldq;
  bf16* k_pool; bf16* v_pool; int64_t pool_layer_stride;   // elements per layer of a pool
  int layer0;                                              // cache layer of group 0
  const int32_t* block_table; int max_pages_per_seq; int page_size;
  const float* q_gain; const float* k_gain; int64_t gain_group_stride;
  const float2* table; int table_pos0;                      // [pos - table_pos0][hd/2]
  int n_q, n_kv, hd;
  int rows, rows_per_seq, rows_written, pos0;
  float eps;
  const int32_t* cu;      // boundary rows of a ragged batch: row b sits at position cu[b+1] - cu[b] - 1
  const int32_t* pos_dev; // run-time position of all rows; table row 0 is that position
  int num_pages;          // block-table entries are checked against it when > 0
  int* status;            // device status word
};

template <int HD>
__global__ void rope_cache_kernel(const RopeDev p) {
  chain_trigger();
  chain_wait();
  constexpr int PER = HD / 64;            // rotation pairs per lane
  const int warps_per_block = blockDim.x >> 5;
  const int heads = p.n_q + 2 * p.n_kv;
  const int64_t item = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int g = blockIdx.y;
  if (item >= (int64_t)p.rows * heads) return;
  const int row = (int)(item / heads);
  const int h = (int)(item - (int64_t)row * heads);
  const int b = row / p.rows_per_seq;
  const int i = row - b * p.rows_per_seq;
  if (i >= p.rows_written) return;
  const int pos = p.pos_dev ? *p.pos_dev : (p.cu ? p.cu[b + 1] - p.cu[b] - 1 : p.pos0 + i);
  const int table_row = p.pos_dev ? 0 : pos - p.table_pos0;
  const float* src = p.in + (int64_t)g * p.in_group_stride + (int64_t)row * p.ld_in + (int64_t)h * HD;
  float lo[PER], hi[PER];                 // elements j and j + HD/2, j = lane + 32*u
#pragma unroll
  for (int u = 0; u < PER; ++u) {
    lo[u] = src[lane + 32 * u];
    hi[u] = src[lane + 32 * u + HD / 2];
  }
  const bool is_q = h < p.n_q;
  const bool is_v = h >= p.n_q + p.n_kv;
  if (!is_v) {
    const float* gain = is_q ? p.q_gain : p.k_gain;
    if (gain != nullptr) {
      gain += (int64_t)g * p.gain_group_stride;
      float ss = 0.f;
#pragma unroll
      for (int u = 0; u < PER; ++u) ss += lo[u] * lo[u] + hi[u] * hi[u];
      ss = warp_sum(ss);
      const float rstd = rsqrtf(ss / (float)HD + p.eps);
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        lo[u] = lo[u] * rstd * gain[lane + 32 * u];
        hi[u] = hi[u] * rstd * gain[lane + 32 * u + HD / 2];
      }
    }
#pragma unroll
    for (int u = 0; u < PER; ++u) {
      const float2 cs = p.table[(int64_t)table_row * (HD / 2) + lane + 32 * u];
      const float a = lo[u] * cs.x - hi[u] * cs.y;
      const float c = hi[u] * cs.x + lo[u] * cs.y;
      lo[u] = a;
      hi[u] = c;
    }
  }
  bf16* dst;
  if (is_q) {
    dst = p.q_out + (int64_t)row * p.ldq + (int64_t)h * HD;
  } else {
    const int kvh = is_v ? h - p.n_q - p.n_kv : h - p.n_q;
    const int page = p.block_table[(int64_t)b * p.max_pages_per_seq + pos / p.page_size];
    if (p.num_pages > 0 && (unsigned)page >= (unsigned)p.num_pages) {
      if (lane == 0) atomicMin(p.status, (int)POP_E_INVALID);     // never turned into an address
      return;
    }
    const int slot = pos % p.page_size;
    bf16* pool = (is_v ? p.v_pool : p.k_pool) + (int64_t)(p.layer0 + g) * p.pool_layer_stride;
    dst = pool + (((int64_t)page * p.page_size + slot) * p.n_kv + kvh) * HD;
  }
#pragma unroll
  for (int u = 0; u < PER; ++u) {
    dst[lane + 32 * u] = __float2bfloat16_rn(lo[u]);
    dst[lane + 32 * u + HD / 2] = __float2bfloat16_rn(hi[u]);
  }
}

// gather boundary rows: dst[b][:] = src[b * rows_per_seq + row][:]
__global__ void gather_rows_kernel(const float* __restrict__ src, float* __restrict__ dst, int d, int rows_per_seq,
                                   int row) {
  const float* s = src + ((int64_t)blockIdx.x * rows_per_seq + row) * d;
  float* o = dst + (int64_t)blockIdx.x * d;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4)
    *reinterpret_cast<float4*>(o + c) = *reinterpret_cast<const float4*>(s + c);
}

// dst[b][:] = src[cu[b+1] - 1][:]
__global__ void gather_last_rows_kernel(const float* __restrict__ src, float* __restrict__ dst, int d,
                                        const int32_t* __restrict__ cu) {
  const float* s = src + (int64_t)(cu[blockIdx.x + 1] - 1) * d;
  float* o = dst + (int64_t)blockIdx.x * d;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4)
    *reinterpret_cast<float4*>(o + c) = *reinterpret_cast<const float4*>(s + c);
}

// greedy choice: index of the largest logit of a row, the lowest index among equal values
__global__ void argmax_kernel(const float* __restrict__ logits, int64_t ld, int vocab, int32_t* __restrict__ tok,
                              int32_t* __restrict__ out, int out_ld, const int32_t* __restrict__ step) {
  __shared__ float sv[32];
  __shared__ int si[32];
  const float* row = logits + (int64_t)blockIdx.x * ld;
  float best = -INFINITY;
  int idx = 0x7fffffff;
  for (int i = threadIdx.x; i < vocab; i += blockDim.x) {
    const float v = row[i];
    if (v > best || (v == best && i < idx)) { best = v; idx = i; }
  }
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (ov > best || (ov == best && oi < idx)) { best = ov; idx = oi; }
  }
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = idx; }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int nw = blockDim.x >> 5;
    best = threadIdx.x < nw ? sv[threadIdx.x] : -INFINITY;
    idx = threadIdx.x < nw ? si[threadIdx.x] : 0x7fffffff;
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      if (ov > best || (ov == best && oi < idx)) { best = ov; idx = oi; }
    }
    if (threadIdx.x == 0) {
      if (idx == 0x7fffffff) idx = 0;          // a row without any finite value
      tok[blockIdx.x] = idx;
      if (out != nullptr) out[(int64_t)blockIdx.x * out_ld + (step ? *step : 0)] = idx;
    }
  }
}
__global__ void set_counters_kernel(int32_t* c, int a, int b) { c[0] = a; c[1] = b; }
__global__ void bump_counters_kernel(int32_t* c) { c[0] += 1; c[1] += 1; }

}  // namespace

int launch_embed(const int32_t* tokens, const bf16* table, const bf16* embeds, float* x, int rows, int d, int vocab,
                 cudaStream_t s) {
  if (d % 8) return POP_E_INVALID;
  int* status = status_word();
  if (!status) return POP_E_CUDA;
  ProfScope prof(PROF_ELEMENTWISE, (double)rows * d * 6, s);
  embed_kernel<<<rows, 256, 0, s>>>(tokens, table, embeds, x, d, vocab, status);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_rmsnorm(const float* x, int64_t ldx, const float* gain, int64_t gain_stride, void* out, int64_t ldo,
                   int64_t out_group_stride, int rows, int d, int groups, float eps, bool out_f32, cudaStream_t s) {
  if (d % 4 || ldx % 4 || ldo % 4 || rows < 1 || groups < 1) return POP_E_INVALID;
  dim3 grid(rows, groups);
  const int threads = d >= 2048 ? 256 : 128;
  ProfScope prof(PROF_ELEMENTWISE, (double)rows * d * (4.0 + groups * (out_f32 ? 4.0 : 2.0)), s);
  if (out_f32)
    launch_chained(rmsnorm_kernel<true>, grid, dim3(threads), 0, s, x, ldx, gain, gain_stride, out, ldo,
                   out_group_stride, d, eps);
  else
    launch_chained(rmsnorm_kernel<false>, grid, dim3(threads), 0, s, x, ldx, gain, gain_stride, out, ldo,
                   out_group_stride, d, eps);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_postnorm_add(float* x, int64_t ldx, const float* t, int64_t ldt, const float* gain, int rows, int d,
                        float eps, cudaStream_t s) {
  if (d % 4 || ldx % 4 || ldt % 4) return POP_E_INVALID;
  ProfScope prof(PROF_ELEMENTWISE, (double)rows * d * 12, s);
  launch_chained(postnorm_add_kernel, dim3(rows), dim3(d >= 2048 ? 256 : 128), 0, s, x, ldx, t, ldt, gain, d, eps);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_rope_table(float2* table, int n_pos, int hd, float theta, cudaStream_t s, int first_pos,
                      const int32_t* first_pos_dev) {
  const int total = n_pos * (hd / 2);
  rope_table_kernel<<<ceil_div(total, 256), 256, 0, s>>>(table, n_pos, hd / 2, (double)theta, first_pos, first_pos_dev);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_rope_cache(const RopeArgs& a, cudaStream_t s) {
  RopeDev p;
  p.in = a.in; p.ld_in = a.ld_in; p.in_group_stride = a.in_group_stride;
  p.q_out = a.q_out; p.ldq = a.ldq;
  p.k_pool = a.k_pool; p.v_pool = a.v_pool; p.pool_layer_stride = a.pool_layer_stride;
  p.layer0 = a.layer0;
  p.block_table = a.block_table; p.max_pages_per_seq = a.max_pages_per_seq; p.page_size = a.page_size;
  p.q_gain = a.q_gain; p.k_gain = a.k_gain; p.gain_group_stride = a.gain_group_stride;
  p.table = a.table; p.table_pos0 = a.table_pos0;
  p.n_q = a.n_q; p.n_kv = a.n_kv; p.hd = a.hd;
  p.rows = a.rows; p.rows_per_seq = a.rows_per_seq; p.rows_written = a.rows_written; p.pos0 = a.pos0;
  p.eps = a.eps;
  p.cu = a.cu_seqlens;
  p.pos_dev = a.pos_dev;
  p.num_pages = a.num_pages;
  p.status = status_word();
  if (!p.status) return POP_E_CUDA;
  if ((a.cu_seqlens != nullptr || a.pos_dev != nullptr) && a.rows_per_seq != 1) return POP_E_INVALID;
  const int heads = a.n_q + 2 * a.n_kv;
  const int64_t items = (int64_t)a.rows * heads;
  dim3 grid((unsigned)((items + 7) / 8), a.groups);
  ProfScope prof(PROF_ELEMENTWISE, (double)items * a.groups * a.hd * 6, s);
  switch (a.hd) {
    case 64: launch_chained(rope_cache_kernel<64>, grid, dim3(256), 0, s, p); break;
    case 128: launch_chained(rope_cache_kernel<128>, grid, dim3(256), 0, s, p); break;
    case 256: launch_chained(rope_cache_kernel<256>, grid, dim3(256), 0, s, p); break;
    default: return POP_E_INVALID;
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_gather_rows(const float* src, float* dst, int batch, int d, int rows_per_seq, int row, cudaStream_t s) {
  gather_rows_kernel<<<batch, 256, 0, s>>>(src, dst, d, rows_per_seq, row);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_argmax(const float* logits, int64_t ld, int vocab, int batch, int32_t* tok, int32_t* out, int out_ld,
                  const int32_t* step, cudaStream_t s) {
  argmax_kernel<<<batch, 1024, 0, s>>>(logits, ld, vocab, tok, out, out_ld, step);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}
int launch_set_counters(int32_t* counters, int a, int b, cudaStream_t s) {
  set_counters_kernel<<<1, 1, 0, s>>>(counters, a, b);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}
int launch_bump_counters(int32_t* counters, cudaStream_t s) {
  bump_counters_kernel<<<1, 1, 0, s>>>(counters);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_gather_last_rows(const float* src, float* dst, int batch, int d, const int32_t* cu, cudaStream_t s) {
  gather_last_rows_kernel<<<batch, 256, 0, s>>>(src, dst, d, cu);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

}  // namespace pop
