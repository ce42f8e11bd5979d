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
// once with 16-byte loads, GEMV_U k-steps (8 or 16 loads per lane) in flight at a time; the few
// activation rows come through L1. NB = activation rows handled (1, 2, 4 or 8).
constexpr int GEMV_U = 4;

template <bool X_F32>
__device__ __forceinline__ void load_x8(const void* x, int64_t off, float (&xf)[8]) {
  if (X_F32) {
    const float* xp = reinterpret_cast<const float*>(x) + off;
    const float4 a = *reinterpret_cast<const float4*>(xp);
    const float4 c = *reinterpret_cast<const float4*>(xp + 4);
    xf[0] = a.x; xf[1] = a.y; xf[2] = a.z; xf[3] = a.w;
    xf[4] = c.x; xf[5] = c.y; xf[6] = c.z; xf[7] = c.w;
  } else {
    unpack8(*reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(x) + off), xf);
  }
}

template <bool X_F32, int NB, bool GATED>
__global__ void __launch_bounds__(256) gemv_kernel(const GemvDev p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  constexpr int R = GEMV_R;
  constexpr int RW = GATED ? 2 * R : R;           // weight rows streamed per warp
  const int n_out = GATED ? p.N / 2 : p.N;        // logical output rows
  const int o0 = warp * R;
  if (o0 >= n_out) return;
  // weight rows for output o: plain -> o; gated -> gate row (o/128)*256 + o%128, up row +128
  const bf16* wr[RW];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int o = min(o0 + r, n_out - 1);
    const int64_t row = GATED ? (int64_t)(o >> 7) * 256 + (o & 127) : o;
    wr[r] = p.w + row * p.ldw;
    if (GATED) wr[R + r] = p.w + (row + 128) * p.ldw;
  }
  float acc[RW][NB];
#pragma unroll
  for (int r = 0; r < RW; ++r)
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[r][b] = 0.f;

  for (int k0 = lane * 8; k0 < p.K; k0 += 256 * GEMV_U) {
    uint4 wraw[GEMV_U][RW];
#pragma unroll
    for (int u = 0; u < GEMV_U; ++u) {
      const int k = k0 + u * 256;
#pragma unroll
      for (int r = 0; r < RW; ++r)
        wraw[u][r] = (k < p.K) ? ld_stream(wr[r] + k) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < GEMV_U; ++u) {
      const int k = k0 + u * 256;
      if (k < p.K) {
        float wf[RW][8];
#pragma unroll
        for (int r = 0; r < RW; ++r) unpack8(wraw[u][r], wf[r]);
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          if (b < p.B) {
            float xf[8];
            load_x8<X_F32>(p.x, (int64_t)b * p.ldx + k, xf);
#pragma unroll
            for (int r = 0; r < RW; ++r)
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[r][b] = fmaf(wf[r][e], xf[e], acc[r][b]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      if (b < p.B) {
        float v = warp_sum(acc[r][b]);
        float u = GATED ? warp_sum(acc[GATED ? R + r : r][b]) : 0.f;
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

template <bool X_F32, bool GATED>
void launch_gemv_nb(const GemvDev& p, int blocks, cudaStream_t s) {
  if (p.B <= 1) gemv_kernel<X_F32, 1, GATED><<<blocks, 256, 0, s>>>(p);
  else if (p.B <= 2) gemv_kernel<X_F32, 2, GATED><<<blocks, 256, 0, s>>>(p);
  else if (p.B <= 4) gemv_kernel<X_F32, 4, GATED><<<blocks, 256, 0, s>>>(p);
  else gemv_kernel<X_F32, 8, GATED><<<blocks, 256, 0, s>>>(p);
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
  const int32_t* cu;                       // ragged: sequence b has cu[b+1] - cu[b] cache positions
  const int32_t* pos_dev;                  // run-time cache length - 1
};

constexpr int DEC_MAXG = 8;
constexpr int DEC_UNROLL = 4;     // keys per lane group whose K and V loads are in flight together

template <int HD>
struct DecCfg {
  static constexpr int LPK = HD / 8;                   // lanes per key: each lane holds 8 elements (16 bytes)
  static constexpr int KPW = 32 / LPK;                 // keys per warp per pass
  static constexpr int WARPS = (HD == 256) ? 4 : 8;
};

template <int HD, int GMAX>
__global__ void __launch_bounds__(DecCfg<HD>::WARPS * 32) dec_attn_kernel(const DecAttnDev p) {
  using C = DecCfg<HD>;
  constexpr int LPK = C::LPK, KPW = C::KPW, WARPS = C::WARPS;
  const int kvh = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
  const int G = p.n_q / p.n_kv;   // <= GMAX
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPK;                          // which key of the pass this lane group reads
  const int e0 = (lane % LPK) * 8;                     // first head_dim element of this lane
  const int kv_len = p.pos_dev ? *p.pos_dev + 1 : (p.cu ? p.cu[b + 1] - p.cu[b] : p.kv_len);
  const int lo = p.window > 0 ? max(0, kv_len - p.window) : 0;
  const int span = kv_len - lo;
  const int chunk = (span + p.splits - 1) / p.splits;
  const int j0 = lo + split * chunk;
  const int j1 = min(kv_len, j0 + chunk);

  float qv[GMAX][8];
#pragma unroll
  for (int g = 0; g < GMAX; ++g)
    if (g < G) {
      float t[8];
      unpack8(*reinterpret_cast<const uint4*>(p.q + (int64_t)b * p.ldq + (int64_t)(kvh * G + g) * HD + e0), t);
#pragma unroll
      for (int e = 0; e < 8; ++e) qv[g][e] = t[e] * p.scale_log2;
    }
  float m[GMAX], l[GMAX], o[GMAX][8];
#pragma unroll
  for (int g = 0; g < GMAX; ++g) {
    m[g] = -INFINITY;
    l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) o[g][e] = 0.f;
  }
  const int32_t* bt = p.block_table + (int64_t)b * p.max_pages_per_seq;
  constexpr int STRIDE = WARPS * KPW;                  // keys the CTA covers per pass
  // the trip count depends on the warp only, never on the lane: every lane reaches the shuffles
  for (int jw = j0 + warp * KPW; jw < j1; jw += STRIDE * DEC_UNROLL) {
    const int jb = jw + sub;
    uint4 kraw[DEC_UNROLL], vraw[DEC_UNROLL];
#pragma unroll
    for (int u = 0; u < DEC_UNROLL; ++u) {
      const int j = jb + u * STRIDE;
      kraw[u] = make_uint4(0, 0, 0, 0);
      vraw[u] = make_uint4(0, 0, 0, 0);
      if (j < j1) {
        const int page = bt[j / p.page_size];
        const int64_t off = (((int64_t)page * p.page_size + j % p.page_size) * p.n_kv + kvh) * HD + e0;
        kraw[u] = ld_stream(p.k_pool + off);
        vraw[u] = ld_stream(p.v_pool + off);
      }
    }
#pragma unroll
    for (int u = 0; u < DEC_UNROLL; ++u) {
      const bool valid = jb + u * STRIDE < j1;   // uniform within a lane group
      {
        float kf[8], vf[8];
        unpack8(kraw[u], kf);
        unpack8(vraw[u], vf);
#pragma unroll
        for (int g = 0; g < GMAX; ++g)
          if (g < G) {
            float sc = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) sc = fmaf(qv[g][e], kf[e], sc);
#pragma unroll
            for (int w = LPK / 2; w > 0; w >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, w);
            if (!valid) sc = -INFINITY;            // a key past the chunk contributes nothing
            const float mn = fmaxf(m[g], sc);
            if (mn == -INFINITY) continue;         // nothing seen yet by this lane group
            const float f = exp2f(m[g] - mn);      // exp2f(-inf) = 0 on the first key
            const float pj = exp2f(sc - mn);
            // the probability meets V as bf16, as it does in the prefill kernel's P.V product
            const float pr = __bfloat162float(__float2bfloat16_rn(pj));
            l[g] = l[g] * f + pj;
#pragma unroll
            for (int e = 0; e < 8; ++e) o[g][e] = fmaf(pr, vf[e], o[g][e] * f);
            m[g] = mn;
          }
      }
    }
  }
  __syncwarp();
  // merge the lane groups of a warp (they walked different keys), then the warps through shared memory
#pragma unroll
  for (int g = 0; g < GMAX; ++g)
    if (g < G) {
#pragma unroll
      for (int w = LPK; w < 32; w <<= 1) {
        const float mo = __shfl_xor_sync(0xffffffffu, m[g], w);
        const float lo2 = __shfl_xor_sync(0xffffffffu, l[g], w);
        const float mn = fmaxf(m[g], mo);
        const float fa = (m[g] == -INFINITY) ? 0.f : exp2f(m[g] - mn);
        const float fb = (mo == -INFINITY) ? 0.f : exp2f(mo - mn);
        l[g] = l[g] * fa + lo2 * fb;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float oo = __shfl_xor_sync(0xffffffffu, o[g][e], w);
          o[g][e] = o[g][e] * fa + oo * fb;
        }
        m[g] = mn;
      }
    }
  __shared__ float sm_m[WARPS][GMAX], sm_l[WARPS][GMAX];
  __shared__ float sm_o[WARPS][GMAX][HD];
#pragma unroll
  for (int g = 0; g < GMAX; ++g)
    if (g < G) {
      if (lane == 0) {
        sm_m[warp][g] = m[g];
        sm_l[warp][g] = l[g];
      }
      if (sub == 0) {
#pragma unroll
        for (int e = 0; e < 8; ++e) sm_o[warp][g][e0 + e] = o[g][e];
      }
    }
  __syncthreads();
  for (int idx = threadIdx.x; idx < G * HD; idx += blockDim.x) {
    const int g = idx / HD, e = idx - g * HD;
    float mm = -INFINITY;
    for (int w = 0; w < WARPS; ++w) mm = fmaxf(mm, sm_m[w][g]);
    float ll = 0.f, oo = 0.f;
    for (int w = 0; w < WARPS; ++w) {
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
void launch_dec_attn(const DecAttnDev& p, dim3 grid, int G, cudaStream_t s) {
  constexpr int T = DecCfg<HD>::WARPS * 32;
  if (G <= 1) dec_attn_kernel<HD, 1><<<grid, T, 0, s>>>(p);
  else if (G <= 2) dec_attn_kernel<HD, 2><<<grid, T, 0, s>>>(p);
  else if (G <= 4) dec_attn_kernel<HD, 4><<<grid, T, 0, s>>>(p);
  else dec_attn_kernel<HD, 8><<<grid, T, 0, s>>>(p);
}

template <int HD>
__global__ void dec_combine_kernel(const DecAttnDev p) {
  // one CTA per (head, sequence); splits <= 64. The split weights exp2(m_s - max m) are computed
  // once (thread s handles split s), then every thread sums its output elements over the splits
  // with independent loads.
  __shared__ float wgt[64];
  __shared__ float inv_l;
  const int h = blockIdx.x, b = blockIdx.y;
  const float* src = p.partial + ((int64_t)b * p.n_q + h) * p.splits * (HD + 2);
  if (threadIdx.x < 32) {
    const int s0 = threadIdx.x, s1 = threadIdx.x + 32;
    const float m0 = s0 < p.splits ? src[s0 * (HD + 2)] : -INFINITY;
    const float m1 = s1 < p.splits ? src[s1 * (HD + 2)] : -INFINITY;
    const float l0 = s0 < p.splits ? src[s0 * (HD + 2) + 1] : 0.f;
    const float l1 = s1 < p.splits ? src[s1 * (HD + 2) + 1] : 0.f;
    float mm = fmaxf(m0, m1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
    const float w0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - mm);
    const float w1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - mm);
    wgt[s0] = w0;
    wgt[s1] = w1;
    const float ll = warp_sum(l0 * w0 + l1 * w1);
    if (threadIdx.x == 0) inv_l = 1.0f / ll;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < HD; e += blockDim.x) {
    float oo = 0.f;
#pragma unroll 8
    for (int s = 0; s < p.splits; ++s) oo = fmaf(src[s * (HD + 2) + 2 + e], wgt[s], oo);
    p.out[(int64_t)b * p.ldo + (int64_t)h * HD + e] = __float2bfloat16_rn(oo * inv_l);
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
    if (a.mode == 3) {
      if (a.x_f32) launch_gemv_nb<true, true>(p, blocks, s);
      else launch_gemv_nb<false, true>(p, blocks, s);
    } else {
      if (a.x_f32) launch_gemv_nb<true, false>(p, blocks, s);
      else launch_gemv_nb<false, false>(p, blocks, s);
    }
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
  p.cu = a.cu_seqlens;
  p.pos_dev = a.pos_dev;
  p.splits = a.pos_dev ? 64 : decode_attn_splits(a.kv_len, a.window);
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)a.head_dim);
  dim3 grid(a.n_kv, p.splits, a.batch), grid2(a.n_q, a.batch);
  const int span = (a.window > 0 && a.window < a.kv_len) ? a.window : a.kv_len;
  ProfScope prof(PROF_DECODE_ATTN, (double)a.batch * span * a.n_kv * a.head_dim * 4, s);
  switch (a.head_dim) {
    case 64:
      launch_dec_attn<64>(p, grid, p.n_q / p.n_kv, s);
      dec_combine_kernel<64><<<grid2, 64, 0, s>>>(p);
      break;
    case 128:
      launch_dec_attn<128>(p, grid, p.n_q / p.n_kv, s);
      dec_combine_kernel<128><<<grid2, 128, 0, s>>>(p);
      break;
    case 256:
      launch_dec_attn<256>(p, grid, p.n_q / p.n_kv, s);
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
  p.cu = nullptr;
  p.pos_dev = nullptr;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)head_dim);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The first kernel writes every partial slot the second one reads (all splits of all heads, also
  // the empty ones), so nothing left in the array by an earlier call is ever consumed and no
  // clearing is needed between calls.
  dim3 grid(n_kv, p.splits, batch), grid2(n_q, batch);
  switch (head_dim) {
    case 64:
      launch_dec_attn<64>(p, grid, p.n_q / p.n_kv, s);
      dec_combine_kernel<64><<<grid2, 64, 0, s>>>(p);
      break;
    case 128:
      launch_dec_attn<128>(p, grid, p.n_q / p.n_kv, s);
      dec_combine_kernel<128><<<grid2, 128, 0, s>>>(p);
      break;
    default:
      launch_dec_attn<256>(p, grid, p.n_q / p.n_kv, s);
      dec_combine_kernel<256><<<grid2, 128, 0, s>>>(p);
      break;
  }
  count_launch();
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}
