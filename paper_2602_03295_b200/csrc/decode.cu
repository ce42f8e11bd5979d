// Bandwidth-bound kernels of the boundary-token path (paper Sec. 3.3: the last prompt token is the
// first decode step of the full model) and of the output head: weight-streaming GEMV for a handful
// of rows, and single-query attention over the paged cache with split-KV partials.
#include "common.cuh"
#include "../../include/pop_kernels.h"

#include <mutex>

namespace pop {
namespace {

constexpr int GEMV_MAXB = 8;     // rows (sequences) handled per pass
constexpr int GEMV_R = 2;        // weight rows per warp

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ float act_fn(float g, int act) {
  if (act == 0) return g / (1.0f + expf(-g));
  const float c = 0.7978845608028654f;
  return 0.5f * g * (1.0f + tanhf(c * (g + 0.044715f * g * g * g)));
}

struct GemvDev {
  const void* x; int64_t ldx;      // [B][K] bf16 or fp32
  const bf16* w; int64_t ldw;      // [N][K]
  void* out; int64_t ldo;
  int B, N, K;
  int mode;                        // 0 store fp32, 2 fp32 +=, 3 gated -> bf16
  int act, n_valid;
};

// Each warp owns GEMV_R weight rows (mode 3: GEMV_R gate rows and their up rows) and streams them
// once with 16-byte loads; the few activation rows come through L1.
template <bool X_F32>
__global__ void __launch_bounds__(256) gemv_kernel(const GemvDev p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const bool gated = p.mode == 3;
  constexpr int R = GEMV_R;
  const int n_out = gated ? p.N / 2 : p.N;        // logical output rows
  const int o0 = warp * R;
  if (o0 >= n_out) return;
  // weight rows for output o: plain -> o; gated -> gate row (o/128)*256 + o%128, up row +128
  const bf16* wr[R * 2];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int o = min(o0 + r, n_out - 1);
    const int64_t row = gated ? (int64_t)(o >> 7) * 256 + (o & 127) : o;
    wr[r] = p.w + row * p.ldw;
    wr[R + r] = p.w + (row + 128) * p.ldw;
  }
  float acc[R * 2][GEMV_MAXB];
#pragma unroll
  for (int r = 0; r < R * 2; ++r)
#pragma unroll
    for (int b = 0; b < GEMV_MAXB; ++b) acc[r][b] = 0.f;

  for (int k = lane * 8; k < p.K; k += 256) {
    float wf[R * 2][8];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      unpack8(ld_stream(wr[r] + k), wf[r]);
      if (gated) unpack8(ld_stream(wr[R + r] + k), wf[R + r]);
    }
#pragma unroll
    for (int b = 0; b < GEMV_MAXB; ++b) {
      if (b < p.B) {
        float xf[8];
        if (X_F32) {
          const float* xp = reinterpret_cast<const float*>(p.x) + (int64_t)b * p.ldx + k;
          const float4 a = *reinterpret_cast<const float4*>(xp);
          const float4 c = *reinterpret_cast<const float4*>(xp + 4);
          xf[0] = a.x; xf[1] = a.y; xf[2] = a.z; xf[3] = a.w;
          xf[4] = c.x; xf[5] = c.y; xf[6] = c.z; xf[7] = c.w;
        } else {
          unpack8(*reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(p.x) + (int64_t)b * p.ldx + k), xf);
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[r][b] = fmaf(wf[r][e], xf[e], acc[r][b]);
          if (gated) {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[R + r][b] = fmaf(wf[R + r][e], xf[e], acc[R + r][b]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
#pragma unroll
    for (int b = 0; b < GEMV_MAXB; ++b) {
      if (b < p.B) {
        float v = warp_sum(acc[r][b]);
        float u = gated ? warp_sum(acc[R + r][b]) : 0.f;
        const int o = o0 + r;
        if (lane == 0 && o < n_out) {
          if (p.mode == 0) {
            reinterpret_cast<float*>(p.out)[(int64_t)b * p.ldo + o] = v;
          } else if (p.mode == 2) {
            reinterpret_cast<float*>(p.out)[(int64_t)b * p.ldo + o] += v;
          } else if (o < p.n_valid) {
            reinterpret_cast<bf16*>(p.out)[(int64_t)b * p.ldo + o] = __float2bfloat16_rn(act_fn(v, p.act) * u);
          }
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------ decode attention
// One CTA per (kv head, split, sequence): the G = n_q/n_kv query heads of the group attend over a
// contiguous chunk of cache positions; each warp walks positions, lanes split head_dim. Partials
// (max, sum, unnormalised output) go to scratch and are merged by the combine kernel.
struct DecAttnDev {
  const bf16* q; int64_t ldq;              // [B][n_q*hd], one query per sequence at position kv_len-1
  const bf16* k_pool; const bf16* v_pool;  // one layer: [page][slot][n_kv][hd]
  const int32_t* block_table; int max_pages_per_seq; int page_size;
  float* partial;                          // [B][n_q][splits][hd + 2]
  bf16* out; int64_t ldo;                  // [B][n_q*hd]
  int n_q, n_kv, kv_len, window, splits;
  float scale_log2;
};

constexpr int DEC_MAXG = 8;

template <int HD>
__global__ void __launch_bounds__(128) dec_attn_kernel(const DecAttnDev p) {
  constexpr int PER = HD / 32;             // elements per lane
  const int kvh = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
  const int G = p.n_q / p.n_kv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int lo = p.window > 0 ? max(0, p.kv_len - p.window) : 0;
  const int span = p.kv_len - lo;
  const int chunk = (span + p.splits - 1) / p.splits;
  const int j0 = lo + split * chunk;
  const int j1 = min(p.kv_len, j0 + chunk);

  float qv[DEC_MAXG][PER];
#pragma unroll
  for (int g = 0; g < DEC_MAXG; ++g)
    if (g < G) {
      const bf16* qp = p.q + (int64_t)b * p.ldq + (int64_t)(kvh * G + g) * HD + lane * PER;
#pragma unroll
      for (int e = 0; e < PER; ++e) qv[g][e] = __bfloat162float(qp[e]) * p.scale_log2;
    }
  float m[DEC_MAXG], l[DEC_MAXG], o[DEC_MAXG][PER];
#pragma unroll
  for (int g = 0; g < DEC_MAXG; ++g) {
    m[g] = -INFINITY;
    l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < PER; ++e) o[g][e] = 0.f;
  }
  const int32_t* bt = p.block_table + (int64_t)b * p.max_pages_per_seq;
  for (int j = j0 + warp; j < j1; j += 4) {
    const int page = bt[j / p.page_size];
    const int64_t off = (((int64_t)page * p.page_size + j % p.page_size) * p.n_kv + kvh) * HD + lane * PER;
    float kf[PER], vf[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      kf[e] = __bfloat162float(p.k_pool[off + e]);
      vf[e] = __bfloat162float(p.v_pool[off + e]);
    }
#pragma unroll
    for (int g = 0; g < DEC_MAXG; ++g)
      if (g < G) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < PER; ++e) s = fmaf(qv[g][e], kf[e], s);
        s = warp_sum(s);
        const float mn = fmaxf(m[g], s);
        const float f = exp2f(m[g] - mn);      // exp2f(-inf) = 0 on the first key
        const float pj = exp2f(s - mn);
        // the probability meets V as bf16, as it does in the prefill kernel's P.V product
        const float pr = __bfloat162float(__float2bfloat16_rn(pj));
        l[g] = l[g] * f + pj;
#pragma unroll
        for (int e = 0; e < PER; ++e) o[g][e] = fmaf(pr, vf[e], o[g][e] * f);
        m[g] = mn;
      }
  }
  // merge the 4 warps of the CTA through shared memory
  __shared__ float sm_m[4][DEC_MAXG], sm_l[4][DEC_MAXG];
  __shared__ float sm_o[4][DEC_MAXG][HD];
#pragma unroll
  for (int g = 0; g < DEC_MAXG; ++g)
    if (g < G) {
      if (lane == 0) {
        sm_m[warp][g] = m[g];
        sm_l[warp][g] = l[g];
      }
#pragma unroll
      for (int e = 0; e < PER; ++e) sm_o[warp][g][lane * PER + e] = o[g][e];
    }
  __syncthreads();
  for (int idx = threadIdx.x; idx < G * HD; idx += blockDim.x) {
    const int g = idx / HD, e = idx - g * HD;
    float mm = -INFINITY;
    for (int w = 0; w < 4; ++w) mm = fmaxf(mm, sm_m[w][g]);
    float ll = 0.f, oo = 0.f;
    for (int w = 0; w < 4; ++w) {
      const float f = (sm_m[w][g] == -INFINITY) ? 0.f : exp2f(sm_m[w][g] - mm);
      ll += sm_l[w][g] * f;
      oo += sm_o[w][g][e] * f;
    }
    float* dst = p.partial + (((int64_t)b * p.n_q + kvh * G + g) * p.splits + split) * (HD + 2);
    dst[2 + e] = oo;
    if (e == 0) {
      dst[0] = mm;
      dst[1] = ll;
    }
  }
}

template <int HD>
__global__ void dec_combine_kernel(const DecAttnDev p) {
  const int h = blockIdx.x, b = blockIdx.y;
  const float* src = p.partial + ((int64_t)b * p.n_q + h) * p.splits * (HD + 2);
  float mm = -INFINITY;
  for (int s = 0; s < p.splits; ++s) mm = fmaxf(mm, src[s * (HD + 2)]);
  float ll = 0.f;
  for (int s = 0; s < p.splits; ++s) {
    const float ms = src[s * (HD + 2)];
    if (ms > -INFINITY) ll += src[s * (HD + 2) + 1] * exp2f(ms - mm);
  }
  for (int e = threadIdx.x; e < HD; e += blockDim.x) {
    float oo = 0.f;
    for (int s = 0; s < p.splits; ++s) {
      const float ms = src[s * (HD + 2)];
      if (ms > -INFINITY) oo += src[s * (HD + 2) + 2 + e] * exp2f(ms - mm);
    }
    p.out[(int64_t)b * p.ldo + (int64_t)h * HD + e] = __float2bfloat16_rn(oo / ll);
  }
}

}  // namespace

int launch_gemv(const GemvArgs& a, cudaStream_t s) {
  if (!a.x || !a.w || !a.out || a.B < 1 || a.N < 1 || a.K < 1) return POP_E_INVALID;
  if (a.K % 8 || a.ldw % 8 || a.ldx % 8) return POP_E_INVALID;
  if (a.mode == 3 && (a.N % 256 || a.n_valid > a.N / 2)) return POP_E_INVALID;
  const int n_out = a.mode == 3 ? a.N / 2 : a.N;
  const int warps = ceil_div(n_out, GEMV_R);
  const int blocks = ceil_div(warps, 8);
  const int elt = a.x_f32 ? 4 : 2;
  for (int b0 = 0; b0 < a.B; b0 += GEMV_MAXB) {
    GemvDev p;
    p.x = static_cast<const char*>(a.x) + (int64_t)b0 * a.ldx * elt;
    p.ldx = a.ldx;
    p.w = a.w; p.ldw = a.ldw;
    p.out = static_cast<char*>(a.out) + (int64_t)b0 * a.ldo * (a.mode == 3 ? 2 : 4);
    p.ldo = a.ldo;
    p.B = a.B - b0 < GEMV_MAXB ? a.B - b0 : GEMV_MAXB;
    p.N = a.N; p.K = a.K; p.mode = a.mode; p.act = a.act; p.n_valid = a.n_valid;
    ProfScope prof(PROF_GEMV, (double)a.N * a.K * 2, s);
    if (a.x_f32) gemv_kernel<true><<<blocks, 256, 0, s>>>(p);
    else gemv_kernel<false><<<blocks, 256, 0, s>>>(p);
    count_launch();
  }
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int decode_attn_splits(int kv_len, int window) {
  const int span = window > 0 && window < kv_len ? window : kv_len;
  int s = ceil_div(span, 256);
  return s < 1 ? 1 : (s > 64 ? 64 : s);
}

int launch_decode_attention(const DecAttnArgs& a, cudaStream_t s) {
  if (!a.q || !a.k_pool || !a.v_pool || !a.block_table || !a.partial || !a.out) return POP_E_INVALID;
  if (a.n_q % a.n_kv || a.n_q / a.n_kv > DEC_MAXG || a.kv_len < 1) return POP_E_INVALID;
  DecAttnDev p;
  p.q = a.q; p.ldq = a.ldq;
  p.k_pool = a.k_pool; p.v_pool = a.v_pool;
  p.block_table = a.block_table; p.max_pages_per_seq = a.max_pages_per_seq; p.page_size = a.page_size;
  p.partial = a.partial; p.out = a.out; p.ldo = a.ldo;
  p.n_q = a.n_q; p.n_kv = a.n_kv; p.kv_len = a.kv_len; p.window = a.window;
  p.splits = decode_attn_splits(a.kv_len, a.window);
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)a.head_dim);
  dim3 grid(a.n_kv, p.splits, a.batch), grid2(a.n_q, a.batch);
  const int span = (a.window > 0 && a.window < a.kv_len) ? a.window : a.kv_len;
  ProfScope prof(PROF_DECODE_ATTN, (double)a.batch * span * a.n_kv * a.head_dim * 4, s);
  switch (a.head_dim) {
    case 64:
      dec_attn_kernel<64><<<grid, 128, 0, s>>>(p);
      dec_combine_kernel<64><<<grid2, 64, 0, s>>>(p);
      break;
    case 128:
      dec_attn_kernel<128><<<grid, 128, 0, s>>>(p);
      dec_combine_kernel<128><<<grid2, 128, 0, s>>>(p);
      break;
    case 256:
      dec_attn_kernel<256><<<grid, 128, 0, s>>>(p);
      dec_combine_kernel<256><<<grid2, 128, 0, s>>>(p);
      break;
    default: return POP_E_INVALID;
  }
  count_launch();
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

}  // namespace pop

// ------------------------------------------------------------------------------ allocation-free variant
// Split-KV partials of pop_k_decode_attention_static live here instead of in a caller buffer.
// The array is part of the loaded module: every GPU that loads this library carries it until the
// process exits. POP_STATIC_SCRATCH_FLOATS (pop_kernels.h) states its size.
namespace pop {
namespace {

static __device__ __align__(256) float g_dec_static_scratch[POP_STATIC_SCRATCH_FLOATS];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float* g_static_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device. In host code the array's name is only
// a handle for the runtime, not something a kernel can dereference, so the address is looked up
// once per device (with that device current) and remembered.
int static_scratch(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return POP_E_CUDA;
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_dec_static_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return POP_E_CUDA;
    }
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return POP_OK;
}

}  // namespace
}  // namespace pop

extern "C" int pop_k_decode_attention_static(const void* q, int64_t ldq, const void* k_pool, const void* v_pool,
                                             const int32_t* block_table, int32_t max_pages_per_seq,
                                             int32_t page_size, void* out, int64_t ldo, int32_t batch, int32_t n_q,
                                             int32_t n_kv, int32_t head_dim, int32_t kv_len, int32_t window,
                                             void* stream) {
  using namespace pop;
  if (!q || !k_pool || !v_pool || !block_table || !out) return POP_E_INVALID;
  if (batch < 1 || n_q < 1 || n_kv < 1 || kv_len < 1 || page_size < 1 || window < 0) return POP_E_INVALID;
  if (n_q % n_kv || n_q / n_kv > DEC_MAXG) return POP_E_INVALID;
  if (head_dim != 64 && head_dim != 128 && head_dim != 256) return POP_E_INVALID;
  if ((int64_t)ceil_div(kv_len, page_size) > max_pages_per_seq) return POP_E_NOSPACE;
  DecAttnDev p;
  p.splits = decode_attn_splits(kv_len, window);
  // every (sequence, query head, split) owns head_dim + 2 floats of the shared array
  const int64_t need = (int64_t)batch * n_q * p.splits * (head_dim + 2);
  if (need > (int64_t)POP_STATIC_SCRATCH_FLOATS) return POP_E_NOSPACE;
  float* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != POP_OK) return rc;
  p.q = static_cast<const bf16*>(q); p.ldq = ldq;
  p.k_pool = static_cast<const bf16*>(k_pool); p.v_pool = static_cast<const bf16*>(v_pool);
  p.block_table = block_table; p.max_pages_per_seq = max_pages_per_seq; p.page_size = page_size;
  p.partial = scratch;
  p.out = static_cast<bf16*>(out); p.ldo = ldo;
  p.n_q = n_q; p.n_kv = n_kv; p.kv_len = kv_len; p.window = window;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)head_dim);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The first kernel writes every partial slot the second one reads (all splits of all heads, also
  // the empty ones), so nothing left in the array by an earlier call is ever consumed and no
  // clearing is needed between calls.
  dim3 grid(n_kv, p.splits, batch), grid2(n_q, batch);
  switch (head_dim) {
    case 64:
      dec_attn_kernel<64><<<grid, 128, 0, s>>>(p);
      dec_combine_kernel<64><<<grid2, 64, 0, s>>>(p);
      break;
    case 128:
      dec_attn_kernel<128><<<grid, 128, 0, s>>>(p);
      dec_combine_kernel<128><<<grid2, 128, 0, s>>>(p);
      break;
    default:
      dec_attn_kernel<256><<<grid, 128, 0, s>>>(p);
      dec_combine_kernel<256><<<grid2, 128, 0, s>>>(p);
      break;
  }
  count_launch();
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}
