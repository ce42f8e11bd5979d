// Bandwidth-bound kernels of the boundary-token path (paper Sec. 3.3: the last prompt token is the
// first decode step of the full model) and of the output head: weight-streaming GEMV for a handful
// of rows, and single-query attention over the paged cache with split-KV partials.
#include "common.cuh"
#include "ptx.cuh"
#include "../../include/pop_kernels.h"

#include <cstdlib>
#include <mutex>

namespace pop {
namespace {

constexpr int GEMV_MAXB = 8;     // rows (sequences) handled per pass
constexpr int GEMV_R = 2;        // weight rows per warp
constexpr int GEMV_RG = 1;       // gated form: gate rows per warp (each with its up row)

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// 8 bf16 -> fp32 with a shift and a mask per pair: a bf16 is the upper half of the fp32 of the same
// value, and the integer pipe is wider than the conversion unit
__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// 16 E4M3 codes -> fp32 (exact: every E4M3 value is an fp16 value)
__device__ __forceinline__ void unpack16_e4m3(const uint4& raw, float (&f)[16]) {
  const uint16_t* h = reinterpret_cast<const uint16_t*>(&raw);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(h[j]));
    const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&h2));
    f[2 * j] = t.x;
    f[2 * j + 1] = t.y;
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
  const void* w; int64_t ldw;      // [N][K] bf16, or E4M3 codes (W8 kernels) whose common scale is *w_scale
  const float* w_scale;
  void* out; int64_t ldo;
  int B, N, K;
  int mode;                        // 0 store fp32, 2 fp32 +=, 3 gated -> bf16
  int act, n_valid;
};

// Each warp owns GEMV_R weight rows (mode 3: GEMV_RG gate rows and their up rows) and streams them
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

// KS = warps of a CTA that share the same rows and split K between them (KS consecutive warps act
// as one group of 32 KS lanes); their partial sums meet in shared memory in a fixed order. Few
// output rows with KS = 1 would leave most of the SMs' load slots empty.
// W8: the weights are E4M3 codes (16 per 16-byte load instead of 8 bf16), the activations stay as they
// are; the sums are scaled by the matrix's scale at the end.
template <bool X_F32, int NB, bool GATED, int KS, bool W8 = false>
__global__ void __launch_bounds__(256) gemv_kernel(const GemvDev p) {
  constexpr int EL = W8 ? 16 : 8;                 // weight elements per 16-byte load
  constexpr int WBYTES = W8 ? 1 : 2;
  const int lane = threadIdx.x & 31;
  const int wic = threadIdx.x >> 5;                         // warp in CTA
  const int slice = wic % KS;
  const int warp = blockIdx.x * ((blockDim.x >> 5) / KS) + wic / KS;   // row group
  constexpr int R = GATED ? GEMV_RG : GEMV_R;
  constexpr int RW = GATED ? 2 * R : R;           // weight rows streamed per warp
  const int n_out = GATED ? p.N / 2 : p.N;        // logical output rows
  const int o0 = warp * R;
  chain_trigger();
  if (KS == 1 && o0 >= n_out) return;
  // weight rows for output o: plain -> o; gated -> gate row (o/128)*256 + o%128, up row +128
  const char* wr[RW];                             // byte addresses of the rows
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int o = min(o0 + r, n_out - 1);
    const int64_t row = GATED ? (int64_t)(o >> 7) * 256 + (o & 127) : o;
    wr[r] = static_cast<const char*>(p.w) + row * p.ldw * WBYTES;
    if (GATED) wr[R + r] = static_cast<const char*>(p.w) + (row + 128) * p.ldw * WBYTES;
  }
  float acc[RW][NB];
#pragma unroll
  for (int r = 0; r < RW; ++r)
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[r][b] = 0.f;

  // the first batch of weight loads goes out before the wait on the preceding kernel: weights are
  // never written by a kernel, the activations may be
  auto load_batch = [&](uint4 (&wraw)[GEMV_U][RW], int k0) {
#pragma unroll
    for (int u = 0; u < GEMV_U; ++u) {
      const int k = k0 + u * 32 * EL * KS;
#pragma unroll
      for (int r = 0; r < RW; ++r)
        wraw[u][r] = (k < p.K) ? ld_stream(wr[r] + (int64_t)k * WBYTES) : make_uint4(0, 0, 0, 0);
    }
  };
  int k0 = (slice * 32 + lane) * EL;
  uint4 wraw[GEMV_U][RW];
  if (k0 < p.K) load_batch(wraw, k0);
  chain_wait();
  while (k0 < p.K) {
#pragma unroll
    for (int u = 0; u < GEMV_U; ++u) {
      const int k = k0 + u * 32 * EL * KS;
      if (k < p.K) {
        float wf[RW][EL];
#pragma unroll
        for (int r = 0; r < RW; ++r) {
          if constexpr (W8) unpack16_e4m3(wraw[u][r], wf[r]);
          else unpack8(wraw[u][r], wf[r]);
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          if (b < p.B) {
#pragma unroll
            for (int hh = 0; hh < EL / 8; ++hh) {
              float xf[8];
              load_x8<X_F32>(p.x, (int64_t)b * p.ldx + k + hh * 8, xf);
#pragma unroll
              for (int r = 0; r < RW; ++r)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[r][b] = fmaf(wf[r][hh * 8 + e], xf[e], acc[r][b]);
            }
          }
        }
      }
    }
    k0 += 32 * EL * KS * GEMV_U;
    if (k0 < p.K) load_batch(wraw, k0);
  }
  if (KS > 1) {
    // slice 0 of every group adds the other slices' sums in slice order
    __shared__ float part[8][RW][NB];
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        acc[r][b] = warp_sum(acc[r][b]);
        if (lane == 0) part[wic][r][b] = acc[r][b];
      }
    __syncthreads();
    if (slice != 0 || o0 >= n_out) return;
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        float v = 0.f;
#pragma unroll
        for (int sl = 0; sl < KS; ++sl) v += part[wic + sl][r][b];
        acc[r][b] = v;
      }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      if (b < p.B) {
        float v = KS > 1 ? acc[r][b] : warp_sum(acc[r][b]);
        float u = GATED ? (KS > 1 ? acc[GATED ? R + r : r][b] : warp_sum(acc[GATED ? R + r : r][b])) : 0.f;
        if (W8) {
          const float ws = *p.w_scale;
          v *= ws;
          u *= ws;
        }
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

// The tensor-core GEMV costs the same for 1 to 8 activation rows; the scalar one is faster for one or
// two rows and several times slower for eight (c2 shapes, 8 rows, us per launch alone and cold, scalar /
// tensor-core: QKV 34.7 / 17.6, O 36.6 / 14.3, gate-up 126 / 48, down 106 / 32). POP_GEMV_MMA=0 keeps the
// scalar kernel everywhere.
constexpr int GEMV_MMA_MIN_ROWS = 3;
bool gemv_mma_enabled() {
  const char* e = getenv("POP_GEMV_MMA");
  return !(e && e[0] == '0');
}

template <bool X_F32, bool GATED, int KS, bool W8>
void launch_gemv_nb(const GemvDev& p, int blocks, int threads, cudaStream_t s) {
  if (p.B <= 1) launch_chained(gemv_kernel<X_F32, 1, GATED, KS, W8>, dim3(blocks), dim3(threads), 0, s, p);
  else if (p.B <= 2) launch_chained(gemv_kernel<X_F32, 2, GATED, KS, W8>, dim3(blocks), dim3(threads), 0, s, p);
  else if (p.B <= 4) launch_chained(gemv_kernel<X_F32, 4, GATED, KS, W8>, dim3(blocks), dim3(threads), 0, s, p);
  else launch_chained(gemv_kernel<X_F32, 8, GATED, KS, W8>, dim3(blocks), dim3(threads), 0, s, p);
}

template <bool X_F32, bool GATED, bool W8 = false>
void launch_gemv_ks(const GemvDev& p, int row_warps, int ks, cudaStream_t s) {
  // the slices of a row group sit in one CTA of 8 warps; without a K split the warps are
  // independent and CTAs of 4 warps spread more evenly over the SMs (fewer, shorter stragglers)
  const int wpc = ks == 1 ? 4 : 8;
  const int blocks = ceil_div(row_warps * ks, wpc);
  switch (ks) {
    case 8: launch_gemv_nb<X_F32, GATED, 8, W8>(p, blocks, 256, s); break;
    case 4: launch_gemv_nb<X_F32, GATED, 4, W8>(p, blocks, 256, s); break;
    case 2: launch_gemv_nb<X_F32, GATED, 2, W8>(p, blocks, 256, s); break;
    default: launch_gemv_nb<X_F32, GATED, 1, W8>(p, blocks, wpc * 32, s); break;
  }
}

// ------------------------------------------------------------------------------ tensor-core GEMV
// bf16 activations x bf16 weights on the warp-level MMA (m16n8k16): the weight rows are the M side, the
// (up to 8) activation rows the N side. A lane (g = lane / 4, t = lane % 4) loads 16 bytes = 8 consecutive
// k of weight rows g and g + 8 and of activation row g at the same k offset 32 s + 8 t; the four
// register pairs of each load feed two MMAs as (a0, a2) / (a1, a3) / (b0, b1). The k index inside an
// MMA is then a permutation of the real one, the same for A and B, which a dot product does not see.
// One instruction does the work of 256 conversions and FMAs of the scalar kernel, and the sums come
// out complete in the accumulator: no shuffles. Gated form: rows g are gate rows, rows g + 8 their
// up rows, so one thread ends up with both sums of an output.
// KS warps of a CTA share a row group and take k-steps s = slice, slice + KS, ...
constexpr int MMA_U = 4;     // k-steps per batch of loads (two batches in flight)

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// X32: the activations are fp32 (the output head's input). Each value goes in as two bf16, its rounding and
// the rounding of what the first one missed, through two MMAs on the same weights: the product keeps
// about 16 bits of the activation instead of 8.
template <bool GATED, int KS, bool X32>
__global__ void __launch_bounds__(256) gemv_mma_kernel(const GemvDev p) {
  constexpr int GPC = 8 / KS;                       // row groups a CTA works on at a time
  const int lane = threadIdx.x & 31, wic = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int slice = wic % KS;
  const int n_out = GATED ? p.N / 2 : p.N;
  const int n_groups = (n_out + (GATED ? 8 : 16) - 1) / (GATED ? 8 : 16);
  const int n_rounds = (n_groups + GPC - 1) / GPC;  // rounds of GPC groups; this CTA takes blockIdx.x, + gridDim.x, ..
  const int my_rounds = n_rounds > (int)blockIdx.x ? (n_rounds - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int n_steps = p.K / 32;
  // batches of MMA_U k-steps per round, the same for every slice (steps past the end are skipped), so
  // that the warps of a CTA finish a round together; batches are numbered through all the rounds and
  // two of them are always in flight, also across the end of a round
  const int nb_round = ((n_steps + KS - 1) / KS + MMA_U - 1) / MMA_U;
  const int n_batches = my_rounds * nb_round;
  chain_trigger();
  const bf16* xr = static_cast<const bf16*>(p.x) + (int64_t)g * p.ldx + t * 8;
  const float* xr32 = static_cast<const float*>(p.x) + (int64_t)g * p.ldx + t * 8;
  const bool has_x = g < p.B;
  auto group_of = [&](int round_i) { return ((int)blockIdx.x + round_i * (int)gridDim.x) * GPC + wic / KS; };
  float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
  uint4 wa[2][MMA_U], wb[2][MMA_U];
  // load side: walks the same (round, batch) sequence two batches ahead of the compute side
  const bf16* wlo = nullptr;
  const bf16* whi = nullptr;
  int l_ri = 0, l_lb = 0;
  auto set_rows = [&](int round_i) {
    const int group = group_of(round_i);
    // rows of this lane; past the end they repeat the last row (loaded, never stored)
    int64_t r_lo, r_hi;
    if (GATED) {
      const int o = min(group * 8 + g, n_out - 1);
      r_lo = (int64_t)(o >> 7) * 256 + (o & 127);
      r_hi = r_lo + 128;
    } else {
      r_lo = min(group * 16 + g, n_out - 1);
      r_hi = min(group * 16 + g + 8, n_out - 1);
    }
    wlo = static_cast<const bf16*>(p.w) + r_lo * p.ldw + t * 8;
    whi = static_cast<const bf16*>(p.w) + r_hi * p.ldw + t * 8;
  };
  if (my_rounds > 0) set_rows(0);
  auto load_next = [&](int buf) {
    if (l_ri >= my_rounds) return;
#pragma unroll
    for (int u = 0; u < MMA_U; ++u) {
      const int s = slice + KS * (l_lb * MMA_U + u);
      if (s < n_steps) {
        wa[buf][u] = ld_stream(wlo + s * 32);
        wb[buf][u] = ld_stream(whi + s * 32);
      }
    }
    if (++l_lb == nb_round) {
      l_lb = 0;
      if (++l_ri < my_rounds) set_rows(l_ri);
    }
  };
  // the first two batches of weight loads go out before the wait on the preceding kernel
  load_next(0);
  load_next(1);
  chain_wait();
  __shared__ float part[8][32][4];
  int buf = 0, lb = 0, ri = 0;
  for (int fb = 0; fb < n_batches; ++fb) {
#pragma unroll
    for (int u = 0; u < MMA_U; ++u) {
      const int s = slice + KS * (lb * MMA_U + u);
      if (s < n_steps) {
        const uint4 a = buf ? wa[1][u] : wa[0][u], b = buf ? wb[1][u] : wb[0][u];
        if (X32) {
          float xf[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          if (has_x) {
            const float4 x0 = *reinterpret_cast<const float4*>(xr32 + s * 32);
            const float4 x1 = *reinterpret_cast<const float4*>(xr32 + s * 32 + 4);
            xf[0] = x0.x; xf[1] = x0.y; xf[2] = x0.z; xf[3] = x0.w;
            xf[4] = x1.x; xf[5] = x1.y; xf[6] = x1.z; xf[7] = x1.w;
          }
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(xf[2 * i], xf[2 * i + 1]);
            const float2 hf = __bfloat1622float2(h);
            const __nv_bfloat162 l = __floats2bfloat162_rn(xf[2 * i] - hf.x, xf[2 * i + 1] - hf.y);
            hi[i] = *reinterpret_cast<const uint32_t*>(&h);
            lo[i] = *reinterpret_cast<const uint32_t*>(&l);
          }
          mma_bf16_16816(d0, a.x, b.x, a.y, b.y, hi[0], hi[1]);
          mma_bf16_16816(d1, a.z, b.z, a.w, b.w, hi[2], hi[3]);
          mma_bf16_16816(d0, a.x, b.x, a.y, b.y, lo[0], lo[1]);
          mma_bf16_16816(d1, a.z, b.z, a.w, b.w, lo[2], lo[3]);
        } else {
          const uint4 xv = has_x ? *reinterpret_cast<const uint4*>(xr + s * 32) : make_uint4(0, 0, 0, 0);
          mma_bf16_16816(d0, a.x, b.x, a.y, b.y, xv.x, xv.y);
          mma_bf16_16816(d1, a.z, b.z, a.w, b.w, xv.z, xv.w);
        }
      }
    }
    if (buf) load_next(1); else load_next(0);
    buf ^= 1;
    if (++lb < nb_round) continue;
    // ---- end of a round: the sums of this warp's rows are complete (up to the K split)
    float c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      c[i] = d0[i] + d1[i];
      d0[i] = d1[i] = 0.f;
    }
    const int group = group_of(ri);
    bool store = true;
    if (KS > 1) {
      // slice 0 of every group adds the other slices' sums in slice order
      __syncthreads();                               // the previous round's sums have been read
#pragma unroll
      for (int i = 0; i < 4; ++i) part[wic][lane][i] = c[i];
      __syncthreads();
      store = slice == 0;
      if (store) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float v = 0.f;
#pragma unroll
          for (int sl = 0; sl < KS; ++sl) v += part[wic + sl][lane][i];
          c[i] = v;
        }
      }
    }
    if (store) {
      // c[0], c[1]: row g (gated: gate sum) for sequences 2t, 2t + 1; c[2], c[3]: row g + 8 (gated: up sum)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int b = 2 * t + j;
        if (b >= p.B) continue;
        if (GATED) {
          const int o = group * 8 + g;
          if (o < n_out && o < p.n_valid)
            reinterpret_cast<bf16*>(p.out)[(int64_t)b * p.ldo + o] = __float2bfloat16_rn(act_fn(c[j], p.act) * c[2 + j]);
        } else {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int o = group * 16 + g + 8 * h;
            if (o >= n_out) continue;
            float* dst = reinterpret_cast<float*>(p.out) + (int64_t)b * p.ldo + o;
            if (p.mode == 0) *dst = c[2 * h + j];
            else *dst += c[2 * h + j];
          }
        }
      }
    }
    lb = 0;
    ++ri;
  }
}

template <bool GATED, bool X32>
void launch_gemv_mma(const GemvDev& p, int ks, cudaStream_t s) {
  const int n_out = GATED ? p.N / 2 : p.N;
  const int groups = ceil_div(n_out, GATED ? 8 : 16);
  const int rounds = ceil_div(groups * ks, 8);
  // two CTAs fit an SM (registers); each walks its rounds with the load pipeline kept full between them
  static int slots = 0;
  if (slots == 0) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      n = 148;
    slots = 2 * n;
  }
  const int blocks = rounds < slots ? rounds : slots;
  switch (ks) {
    case 8: launch_chained(gemv_mma_kernel<GATED, 8, X32>, dim3(blocks), dim3(256), 0, s, p); break;
    case 4: launch_chained(gemv_mma_kernel<GATED, 4, X32>, dim3(blocks), dim3(256), 0, s, p); break;
    case 2: launch_chained(gemv_mma_kernel<GATED, 2, X32>, dim3(blocks), dim3(256), 0, s, p); break;
    default: launch_chained(gemv_mma_kernel<GATED, 1, X32>, dim3(blocks), dim3(256), 0, s, p); break;
  }
}

// ------------------------------------------------------------------------------ decode attention
// One CTA per (kv head, split, sequence): the G = n_q/n_kv query heads of the group attend over a
// contiguous chunk of cache positions. The chunk is cut into groups of 16 keys that the warps
// take in turn. A warp streams the K and V rows of its groups into its own ring of shared-memory
// stages with 16-byte asynchronous copies (several groups in flight), and computes on the warp-level
// tensor-core path with the keys on the M side, so that no MMA row is padding:
//     S^T [16 keys x 8 heads]  = K [16 x hd] . Q^T [hd x 8]            (hd/16 MMAs, Q^T kept in registers)
//     O^T [hd x 8 heads]      += V^T [hd x 16 keys] . P^T [16 x 8]     (hd/16 MMAs)
// P^T reaches the second product as bf16 (as it does in the prefill kernel), moved from the
// accumulator layout to the B-operand layout by an 8x8 transpose across the warp. Heads G..7 are
// zero columns. Partials (max, sum, unnormalised output) go to scratch and are merged by the combine kernel.
struct DecAttnDev {
  const bf16* q; int64_t ldq;              // [B][n_q*hd], one query per sequence at position kv_len-1
  const bf16* k_pool; const bf16* v_pool;  // one layer: [page][slot][n_kv][hd]
  const int32_t* block_table; int max_pages_per_seq; int page_size;
  float* partial;                          // [B][n_q][splits][hd + 2]
  bf16* out; int64_t ldo;                  // [B][n_q*hd]
  int n_q, n_kv, kv_len, window, splits;
  int kv_first;                            // positions before this one are never attended to
  float scale_log2;
  const int32_t* cu;                       // ragged: sequence b has cu[b+1] - cu[b] cache positions
  const int32_t* pos_dev;                  // run-time cache length - 1
  // [B][n_kv] arrival counters, zero before the launch and zero again after it: the last CTA of a
  // (sequence, kv head) to finish merges the splits itself. Null: the combine kernel does it.
  unsigned int* counters;
  int num_pages;                           // block-table entries are checked against it when > 0
  int* status;                             // device status word
  // projection finished in this kernel (see DecAttnArgs::qkv); null = q holds finished queries
  const float* qkv; int64_t ld_qkv;
  const float* q_gain; const float* k_gain;
  const float2* table; int table_pos0;
  float eps;
  bool cache_settled;                      // see DecAttnArgs
};

constexpr int DEC_MAXG = 8;       // query heads per kv head: the N extent of one MMA

template <int HD>
struct DecCfg {
  static constexpr int KT = 16;                        // keys per stage (the M extent of one MMA)
  static constexpr int WARPS = (HD == 256) ? 4 : 8;
  static constexpr int ROWB = HD * 2;                  // bytes of one head's cache row
  static constexpr int CH = ROWB / 16;                 // 16-byte chunks per row
  static constexpr int STAGE = 2 * KT * ROWB;          // K rows, then V rows
  static constexpr int NST = (HD == 64) ? 6 : 3;       // stages per warp
  static constexpr int SMEM = WARPS * NST * STAGE;     // 192 KB
  static constexpr int MERGE_FLOATS = WARPS * DEC_MAXG * (HD + 2);
  static constexpr int XCHG_FLOATS = DEC_MAXG * (HD + 2);       // a CTA's result, read by its cluster
  static_assert((MERGE_FLOATS + DEC_MAXG * 65 + XCHG_FLOATS) * 4 <= SMEM, "the merges reuse the ring");
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  // src_bytes 0 writes 16 zero bytes and reads nothing
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// 8x8 transpose of 16-bit elements across the warp (thread i holds row i/4, columns 2(i%4), 2(i%4)+1)
__device__ __forceinline__ uint32_t movm_t(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
// D[16x8] += A[16x16] . B[16x8], bf16 operands, fp32 accumulate
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Merge of the split partials of heads h_first .. h_first + n_heads - 1 of sequence b, by all
// threads of the CTA (splits <= 64). Per head one warp computes the split weights exp2(m_s - max m)
// (lane s handles splits s and s + 32), then every thread sums its output elements over the splits
// with independent loads. Partials are read past L1: other CTAs of the same launch may have written them.
template <int HD>
__device__ __forceinline__ void dec_combine_heads(const DecAttnDev& p, int b, int h_first, int n_heads,
                                                  float* wgt /* [n_heads][64] */, float* inv_l /* [n_heads] */) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  for (int g = warp; g < n_heads; g += n_warps) {
    const float* src = p.partial + ((int64_t)b * p.n_q + h_first + g) * p.splits * (HD + 2);
    const int s0 = lane, s1 = lane + 32;
    const float m0 = s0 < p.splits ? __ldcg(src + s0 * (HD + 2)) : -INFINITY;
    const float m1 = s1 < p.splits ? __ldcg(src + s1 * (HD + 2)) : -INFINITY;
    const float l0 = s0 < p.splits ? __ldcg(src + s0 * (HD + 2) + 1) : 0.f;
    const float l1 = s1 < p.splits ? __ldcg(src + s1 * (HD + 2) + 1) : 0.f;
    float mm = fmaxf(m0, m1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
    const float w0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - mm);
    const float w1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - mm);
    wgt[g * 64 + s0] = w0;
    wgt[g * 64 + s1] = w1;
    const float ll = warp_sum(l0 * w0 + l1 * w1);
    if (lane == 0) inv_l[g] = 1.0f / ll;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < n_heads * HD; idx += blockDim.x) {
    const int g = idx / HD, e = idx - g * HD;
    const float* src = p.partial + ((int64_t)b * p.n_q + h_first + g) * p.splits * (HD + 2) + 2 + e;
    float oo = 0.f;
#pragma unroll 8
    for (int sp = 0; sp < p.splits; ++sp) oo = fmaf(__ldcg(src + sp * (HD + 2)), wgt[g * 64 + sp], oo);
    p.out[(int64_t)b * p.ldo + (int64_t)(h_first + g) * HD + e] = __float2bfloat16_rn(oo * inv_l[g]);
  }
}

// CL: the splits of a (sequence, kv head) form one thread-block cluster and merge through distributed
// shared memory (no partials in global memory, no counters).
template <int HD, bool CL>
__global__ void __launch_bounds__(DecCfg<HD>::WARPS * 32) dec_attn_kernel(const DecAttnDev p) {
  using C = DecCfg<HD>;
  constexpr int KT = C::KT, WARPS = C::WARPS, ROWB = C::ROWB, CH = C::CH, NST = C::NST, NT = HD / 16;
  constexpr uint32_t FULL = 0xffffffffu;
  extern __shared__ __align__(128) uint8_t dec_smem[];
  chain_trigger();
  // Finished queries and the newest cache row come from the kernel just before this one. When this
  // kernel finishes the projection itself (p.qkv) inside the library's chain of kernels, only the fp32
  // projection row does: the cache rows of the older positions, the block table and the run-time
  // length were written at least two kernels back, i.e. by kernels that are complete (every kernel of
  // a chain waits for its predecessor), so the first loads of the cache go out before the wait and
  // overlap the predecessor's tail.
  const bool early = p.qkv != nullptr && p.cache_settled;
  if (!early) chain_wait();
  const int kvh = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
  const int G = p.n_q / p.n_kv;   // <= DEC_MAXG
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kv_len = p.pos_dev ? *p.pos_dev + 1 : (p.cu ? p.cu[b + 1] - p.cu[b] : p.kv_len);
  const int lo = max(p.window > 0 ? max(0, kv_len - p.window) : 0, min(p.kv_first, kv_len - 1));
  const int span = kv_len - lo;
  const int chunk = (span + p.splits - 1) / p.splits;
  const int j0 = lo + split * chunk;
  const int j1 = min(kv_len, j0 + chunk);
  // groups of KT keys; warp w takes groups w, w + WARPS, ...  (counts depend on the warp only)
  const int n_groups = j1 > j0 ? (j1 - j0 + KT - 1) / KT : 0;
  const int n_mine = n_groups > warp ? (n_groups - warp + WARPS - 1) / WARPS : 0;

  const int32_t* bt = p.block_table + (int64_t)b * p.max_pages_per_seq;
  __shared__ __align__(16) bf16 q_fin[DEC_MAXG * HD];
  // this thread's two heads are 2 (lane%4) and 2 (lane%4) + 1, its keys of a group lane/4 and lane/4 + 8
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  float o[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;

  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(dec_smem) + warp * (NST * C::STAGE);

  auto issue = [&](int it) {
    const int jg = j0 + (warp + it * WARPS) * KT;
    const uint32_t st = ring + (it % NST) * C::STAGE;
    // lanes 0..15 (and again 16..31) each find the pool row of one key of the group; -1 past the chunk
    const int jk = jg + (lane & 15);
    int row = -1;
    if (jk < j1) {
      const int page = bt[jk / p.page_size];
      if (p.num_pages > 0 && (unsigned)page >= (unsigned)p.num_pages)
        atomicMin(p.status, (int)POP_E_INVALID);     // never turned into an address: the key reads as zeros
      else
        row = page * p.page_size + jk % p.page_size;
    }
#pragma unroll
    for (int i = 0; i < KT * CH / 32; ++i) {
      const int idx = i * 32 + lane;
      const int key = idx / CH, ch = idx % CH;
      const int r = __shfl_sync(FULL, row, key);
      const int64_t off = r < 0 ? 0 : ((int64_t)r * p.n_kv + kvh) * HD + ch * 8;
      const int nbytes = r < 0 ? 0 : 16;
      // 16-byte chunks of a row are permuted by the key's low bits: the 8 rows one matrix load
      // touches fall in different banks
      const uint32_t dst = st + key * ROWB + ((ch ^ (key & 7)) << 4);
      cp_async16(dst, p.k_pool + off, nbytes);
      cp_async16(dst + KT * ROWB, p.v_pool + off, nbytes);
    }
  };

  // the newest position's group (the last one of the range that holds it) has to wait for the append
  const bool holds_new = p.qkv != nullptr && kv_len - 1 >= j0 && kv_len - 1 < j1;
  int deferred = -1;
#pragma unroll
  for (int i = 0; i < NST; ++i) {
    if (i < n_mine) {
      if (holds_new && warp == (n_groups - 1) % WARPS && i == n_mine - 1) deferred = i;
      else issue(i);
    }
    cp_async_commit();
  }
  if (early) chain_wait();
  if (p.qkv != nullptr) {
    // Finish the projection here: per-head norm, rotary row of the newest position kv_len - 1. Every
    // CTA does its own G query heads (to shared memory); the CTA whose range holds that position also
    // does the key, and writes key and value into the cache before any of its warps loads that range.
    constexpr int PER = HD / 64;
    const int pos = kv_len - 1;
    const bool owner = pos >= j0 && pos < j1;
    const float* row = p.qkv + (int64_t)b * p.ld_qkv;
    const int q_dim = p.n_q * HD, kv_dim = p.n_kv * HD;
    const float2* trow = p.table + (int64_t)(p.pos_dev ? 0 : pos - p.table_pos0) * (HD / 2);
    for (int it = warp; it < G + (owner ? 2 : 0); it += WARPS) {
      const bool is_q = it < G, is_k = it == G;
      const float* src = row + (is_q ? (int64_t)(kvh * G + it) * HD
                                     : (is_k ? (int64_t)q_dim + kvh * HD : (int64_t)q_dim + kv_dim + kvh * HD));
      float lo[PER], hi[PER];
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        lo[u] = src[lane + 32 * u];
        hi[u] = src[lane + 32 * u + HD / 2];
      }
      if (is_q || is_k) {
        const float* gain = is_q ? p.q_gain : p.k_gain;
        if (gain != nullptr) {
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
          const float2 cs = trow[lane + 32 * u];
          const float a = lo[u] * cs.x - hi[u] * cs.y;
          const float c = hi[u] * cs.x + lo[u] * cs.y;
          lo[u] = a;
          hi[u] = c;
        }
      }
      bf16* dst;
      if (is_q) {
        dst = q_fin + it * HD;
      } else {
        const int page = bt[pos / p.page_size];
        if (p.num_pages > 0 && (unsigned)page >= (unsigned)p.num_pages) {
          if (lane == 0) atomicMin(p.status, (int)POP_E_INVALID);     // never turned into an address
          continue;
        }
        bf16* pool = const_cast<bf16*>(is_k ? p.k_pool : p.v_pool);
        dst = pool + (((int64_t)page * p.page_size + pos % p.page_size) * p.n_kv + kvh) * HD;
      }
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        dst[lane + 32 * u] = __float2bfloat16_rn(lo[u]);
        dst[lane + 32 * u + HD / 2] = __float2bfloat16_rn(hi[u]);
      }
    }
    __threadfence();      // the cache rows are read back below through asynchronous copies
    __syncthreads();
    if (deferred >= 0) {
      issue(deferred);
      cp_async_commit();
    }
  }
  // Q^T as the B operand: thread holds head lane/4, dims 16 ks + 2 (lane%4) + {0, 1} and + 8
  uint32_t qb[NT][2];
  {
    const int g = lane >> 2;
    const bf16* qrow = (p.qkv != nullptr ? q_fin + (g < G ? g : 0) * HD
                                         : p.q + (int64_t)b * p.ldq + (int64_t)(kvh * G + (g < G ? g : 0)) * HD) +
                       (lane & 3) * 2;
#pragma unroll
    for (int ks = 0; ks < NT; ++ks) {
      qb[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16) : 0u;
      qb[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8) : 0u;
    }
  }
  // matrix-load addresses of this lane (lane = 8 * matrix + row of the matrix)
  const int mi = lane >> 3, r8 = lane & 7;
  const uint32_t k_lane = ((mi & 1) * 8 + r8) * ROWB;          // K: matrices (keys 0-7 | 8-15) x (chunk 2ks | 2ks+1)
  const uint32_t v_lane = KT * ROWB + ((mi >> 1) * 8 + r8) * ROWB;   // V: matrices (chunk 2t | 2t+1) x (keys 0-7 | 8-15)
  const int kr = lane >> 2;

  for (int it = 0; it < n_mine; ++it) {
    if (it == deferred) cp_async_wait<0>();      // its copies were committed after the others
    else cp_async_wait<NST - 1>();
    __syncwarp();
    const uint32_t st = ring + (it % NST) * C::STAGE;
    const int jg = j0 + (warp + it * WARPS) * KT;
    float s[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};   // two chains of dependent MMAs
#pragma unroll
    for (int ks = 0; ks < NT; ks += 2) {
      uint32_t a[4], a2[4];
      ldsm_x4(a, st + k_lane + (((2 * ks + (mi >> 1)) ^ r8) << 4));
      ldsm_x4(a2, st + k_lane + (((2 * ks + 2 + (mi >> 1)) ^ r8) << 4));
      mma_16816(s, a, qb[ks][0], qb[ks][1]);
      mma_16816(sb, a2, qb[ks + 1][0], qb[ks + 1][1]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) s[i] += sb[i];
    const bool v0 = jg + kr < j1, v1 = jg + kr + 8 < j1;   // keys past the chunk contribute nothing
    const float s0 = v0 ? s[0] * p.scale_log2 : -INFINITY, s1 = v0 ? s[1] * p.scale_log2 : -INFINITY;
    const float s2 = v1 ? s[2] * p.scale_log2 : -INFINITY, s3 = v1 ? s[3] * p.scale_log2 : -INFINITY;
    float x0 = fmaxf(s0, s2), x1 = fmaxf(s1, s3);
#pragma unroll
    for (int w = 4; w < 32; w <<= 1) {
      x0 = fmaxf(x0, __shfl_xor_sync(FULL, x0, w));
      x1 = fmaxf(x1, __shfl_xor_sync(FULL, x1, w));
    }
    // the first key of a group is always inside the chunk, so the new maxima are finite
    const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);
    const float f0 = exp2f(m0 - n0), f1 = exp2f(m1 - n1);   // exp2f(-inf) = 0 on the first group
    const float p0 = exp2f(s0 - n0), p1 = exp2f(s1 - n1), p2 = exp2f(s2 - n0), p3 = exp2f(s3 - n1);
    l0 = l0 * f0 + (p0 + p2);
    l1 = l1 * f1 + (p1 + p3);
    m0 = n0;
    m1 = n1;
    if (__any_sync(FULL, f0 != 1.f || f1 != 1.f)) {
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        o[t][0] *= f0; o[t][1] *= f1; o[t][2] *= f0; o[t][3] *= f1;
      }
    }
    const uint32_t pb0 = movm_t(pack_bf16x2(p0, p1));   // keys 0-7 of the group
    const uint32_t pb1 = movm_t(pack_bf16x2(p2, p3));   // keys 8-15
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      uint32_t a[4];
      ldsm_x4_t(a, st + v_lane + (((2 * t + (mi & 1)) ^ r8) << 4));
      mma_16816(o[t], a, pb0, pb1);
    }
    __syncwarp();                                         // every lane is done with the stage
    if (it + NST < n_mine) issue(it + NST);
    cp_async_commit();
  }
  cp_async_wait<0>();
#pragma unroll
  for (int w = 4; w < 32; w <<= 1) {
    l0 += __shfl_xor_sync(FULL, l0, w);
    l1 += __shfl_xor_sync(FULL, l1, w);
  }
  __syncthreads();                                        // all rings are idle: reuse them for the merge
  float* sm_m = reinterpret_cast<float*>(dec_smem);       // [WARPS][8]
  float* sm_l = sm_m + WARPS * DEC_MAXG;                  // [WARPS][8]
  float* sm_o = sm_l + WARPS * DEC_MAXG;                  // [WARPS][8][HD]
  {
    const int h0 = (lane & 3) * 2;
    if (lane < 4) {
      sm_m[warp * DEC_MAXG + h0] = m0; sm_m[warp * DEC_MAXG + h0 + 1] = m1;
      sm_l[warp * DEC_MAXG + h0] = l0; sm_l[warp * DEC_MAXG + h0 + 1] = l1;
    }
    float* so = sm_o + (warp * DEC_MAXG + h0) * HD;
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      so[t * 16 + kr] = o[t][0];
      so[HD + t * 16 + kr] = o[t][1];
      so[t * 16 + kr + 8] = o[t][2];
      so[HD + t * 16 + kr + 8] = o[t][3];
    }
  }
  __syncthreads();
  float* xchg = reinterpret_cast<float*>(dec_smem) + C::MERGE_FLOATS + DEC_MAXG * 65;   // [G] m | [G] l | [G][HD] o
  for (int idx = threadIdx.x; idx < G * HD; idx += blockDim.x) {
    const int g = idx / HD, e = idx - g * HD;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) mm = fmaxf(mm, sm_m[w * DEC_MAXG + g]);
    float ll = 0.f, oo = 0.f;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) {
      const float mw = sm_m[w * DEC_MAXG + g];
      const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - mm);
      ll += sm_l[w * DEC_MAXG + g] * f;
      oo += sm_o[(w * DEC_MAXG + g) * HD + e] * f;
    }
    if (CL) {
      xchg[2 * DEC_MAXG + g * HD + e] = oo;
      if (e == 0) {
        xchg[g] = mm;
        xchg[DEC_MAXG + g] = ll;
      }
    } else {
      float* dst = p.partial + (((int64_t)b * p.n_q + kvh * G + g) * p.splits + split) * (HD + 2);
      dst[2 + e] = oo;
      if (e == 0) {
        dst[0] = mm;
        dst[1] = ll;
      }
    }
  }
  if (CL) {
    // every CTA of the cluster finishes a slice of the G * HD outputs from all the CTAs' results
    cluster_arrive();
    cluster_wait();
    const int cs = p.splits;                        // cluster size = number of splits
    const int per = (G * HD + cs - 1) / cs;
    const int first = (int)cluster_ctarank() * per;
    const uint32_t xa = smem_u32(xchg);
    for (int idx = first + threadIdx.x; idx < min(first + per, G * HD); idx += blockDim.x) {
      const int g = idx / HD, e = idx - g * HD;
      float mr[16], lr[16], orr[16];
#pragma unroll
      for (int r = 0; r < 16; ++r) {
        if (r < cs) {
          const uint32_t base = mapa_u32(xa, (uint32_t)r);
          asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(mr[r]) : "r"(base + 4u * g));
          asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(lr[r]) : "r"(base + 4u * (DEC_MAXG + g)));
          asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(orr[r]) : "r"(base + 4u * (2 * DEC_MAXG + g * HD + e)));
        } else {
          mr[r] = -INFINITY; lr[r] = 0.f; orr[r] = 0.f;
        }
      }
      float mm = -INFINITY;
#pragma unroll
      for (int r = 0; r < 16; ++r) mm = fmaxf(mm, mr[r]);
      float ll = 0.f, oo = 0.f;
#pragma unroll
      for (int r = 0; r < 16; ++r) {
        const float f = (mr[r] == -INFINITY) ? 0.f : exp2f(mr[r] - mm);
        ll = fmaf(lr[r], f, ll);
        oo = fmaf(orr[r], f, oo);
      }
      p.out[(int64_t)b * p.ldo + (int64_t)(kvh * G + g) * HD + e] = __float2bfloat16_rn(oo / ll);
    }
    // nobody leaves while a neighbour may still read its shared memory
    cluster_arrive();
    cluster_wait();
    return;
  }
  if (p.counters == nullptr) return;
  // the last CTA of this (sequence, kv head) to get here merges the splits; the counter wraps back to 0
  __shared__ int is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int old = atomicInc(p.counters + (int64_t)b * p.n_kv + kvh, (unsigned int)p.splits - 1u);
    is_last = old == (unsigned int)p.splits - 1u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  float* wgt = reinterpret_cast<float*>(dec_smem) + C::MERGE_FLOATS;
  dec_combine_heads<HD>(p, b, kvh * G, G, wgt, wgt + DEC_MAXG * 64);
}

template <int HD>
int launch_dec_attn(const DecAttnDev& p, dim3 grid, cudaStream_t s) {
  using C = DecCfg<HD>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(dec_attn_kernel<HD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM) !=
        cudaSuccess)
      return POP_E_CUDA;
    configured = true;
  }
  if (launch_chained(dec_attn_kernel<HD, false>, grid, dim3(C::WARPS * 32), (size_t)C::SMEM, s, p) != cudaSuccess)
    return POP_E_CUDA;
  return POP_OK;
}

// Clusters of `cs` CTAs (the splits of one (sequence, kv head)) that this device can hold at once, 0 if
// the kernel cannot be launched that way. Looked up once per head_dim and cluster size.
template <int HD>
int dec_cluster_capacity(int cs) {
  using C = DecCfg<HD>;
  static int cap[17] = {};          // 0: not looked at, -1: unusable
  if (cs < 2 || cs > 16) return 0;
  if (cap[cs] != 0) return cap[cs] < 0 ? 0 : cap[cs];
  cap[cs] = -1;
  if (cudaFuncSetAttribute(dec_attn_kernel<HD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM) != cudaSuccess ||
      (cs > 8 && cudaFuncSetAttribute(dec_attn_kernel<HD, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) !=
                     cudaSuccess)) {
    cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1, cs, 1);
  cfg.blockDim = dim3(C::WARPS * 32);
  cfg.dynamicSmemBytes = C::SMEM;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = cs;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, dec_attn_kernel<HD, true>, &cfg) != cudaSuccess || n < 1) {
    cudaGetLastError();
    return 0;
  }
  cap[cs] = n;
  return n;
}

bool dec_cluster_enabled() {
  const char* e = getenv("POP_DEC_CLUSTER");       // "0": always merge the splits through global memory
  return !(e && e[0] == '0');
}

template <int HD>
__global__ void dec_combine_kernel(const DecAttnDev p) {
  // one CTA per (head, sequence)
  __shared__ float wgt[64];
  __shared__ float inv_l;
  chain_trigger();
  chain_wait();
  dec_combine_heads<HD>(p, blockIdx.y, blockIdx.x, 1, wgt, &inv_l);
}

}  // namespace

int launch_gemv(const GemvArgs& a, cudaStream_t s) {
  if (!a.x || !a.w || !a.out || a.B < 1 || a.N < 1 || a.K < 1) return POP_E_INVALID;
  if (a.K % 8 || a.ldw % 8 || a.ldx % 8) return POP_E_INVALID;
  if (a.w_fp8 && (a.x_f32 || !a.w_scale || a.K % 16 || a.ldw % 16)) return POP_E_INVALID;
  const int el = a.w_fp8 ? 16 : 8;
  if (a.mode == 3 && (a.N % 256 || a.n_valid > a.N / 2)) return POP_E_INVALID;
  const int n_out = a.mode == 3 ? a.N / 2 : a.N;
  const int warps = ceil_div(n_out, a.mode == 3 ? GEMV_RG : GEMV_R);
  // split K between the warps of a CTA while the warps of the doubled split still fit 1.5 times the
  // GPU's resident warps (148 SMs x 64; 1 and 2 measured slower on the decode step)
  int ks = 1;
  while (ks < 8 && warps * ks * 4 <= 148 * 64 * 3 && a.K >= 32 * el * ks * 2) ks *= 2;
  const int elt = a.x_f32 ? 4 : 2;
  for (int b0 = 0; b0 < a.B; b0 += GEMV_MAXB) {
    GemvDev p;
    p.x = static_cast<const char*>(a.x) + (int64_t)b0 * a.ldx * elt;
    p.ldx = a.ldx;
    p.w = a.w; p.ldw = a.ldw; p.w_scale = a.w_scale;
    p.out = static_cast<char*>(a.out) + (int64_t)b0 * a.ldo * (a.mode == 3 ? 2 : 4);
    p.ldo = a.ldo;
    p.B = a.B - b0 < GEMV_MAXB ? a.B - b0 : GEMV_MAXB;
    p.N = a.N; p.K = a.K; p.mode = a.mode; p.act = a.act; p.n_valid = a.n_valid;
    ProfScope prof(PROF_GEMV, (double)a.N * a.K * (a.w_fp8 ? 1 : 2), s);
    if (!a.w_fp8 && a.K % 32 == 0 && p.B >= GEMV_MMA_MIN_ROWS && gemv_mma_enabled()) {
      // K split over the 8 warps of a CTA while every warp keeps at least two batches of k-steps
      int mks = 1;
      while (mks < 8 && a.K / 32 >= 2 * MMA_U * mks * 2) mks *= 2;
      if (a.mode == 3) {
        if (a.x_f32) launch_gemv_mma<true, true>(p, mks, s);
        else launch_gemv_mma<true, false>(p, mks, s);
      } else {
        if (a.x_f32) launch_gemv_mma<false, true>(p, mks, s);
        else launch_gemv_mma<false, false>(p, mks, s);
      }
      count_launch();
      continue;
    }
    if (a.mode == 3) {
      if (a.w_fp8) launch_gemv_ks<false, true, true>(p, warps, ks, s);
      else if (a.x_f32) launch_gemv_ks<true, true>(p, warps, ks, s);
      else launch_gemv_ks<false, true>(p, warps, ks, s);
    } else {
      if (a.w_fp8) launch_gemv_ks<false, false, true>(p, warps, ks, s);
      else if (a.x_f32) launch_gemv_ks<true, false>(p, warps, ks, s);
      else launch_gemv_ks<false, false>(p, warps, ks, s);
    }
    count_launch();
  }
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

// Split count: as many CTAs as the GPU has SMs (one CTA fills an SM's shared memory), never more
// than 64 (the combine kernel's limit) nor so many that a CTA gets less than one 16-key group per
// warp. kv_len < 1 means "not known on the host" (the length is read on the device).
int decode_attn_splits(int kv_len, int window, int n_kv, int batch) {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      n = 148;
    sms = n;
  }
  int s = sms / (n_kv * batch > 0 ? n_kv * batch : 1);
  if (s > 64) s = 64;
  if (kv_len >= 1) {
    const int span = window > 0 && window < kv_len ? window : kv_len;
    const int by_len = ceil_div(span, 64);
    if (s > by_len) s = by_len;
  }
  return s < 1 ? 1 : s;
}

template <int HD>
int launch_dec_pair(const DecAttnDev& p0, int batch, cudaStream_t s) {
  // Cluster form: the splits of a (sequence, kv head) are one thread-block cluster of 2, 4, 8 or 16 CTAs
  // that merge through distributed shared memory. Taken when that keeps at least 0.8 of the CTAs the
  // free split count would give and the device holds all the clusters at once: short caches and
  // batches of several sequences (2 splits: 9.0 -> 7.7 us per launch). With one long sequence the
  // device does not hold eight 16-CTA clusters of this size, and eight 8-CTA clusters (64 CTAs instead of
  // 144) measured 1.2 % slower per decode step, so that case keeps the merge through global memory.
  if (dec_cluster_enabled() && p0.splits >= 2) {
    int cs = 2;
    while (cs * 2 <= p0.splits && cs < 16) cs *= 2;
    if (cs * 5 >= p0.splits * 4 && dec_cluster_capacity<HD>(cs) >= p0.n_kv * batch) {
      using C = DecCfg<HD>;
      DecAttnDev p = p0;
      p.splits = cs;
      if (launch_chained_cluster(dec_attn_kernel<HD, true>, dim3(p.n_kv, cs, batch), dim3(C::WARPS * 32),
                                 (size_t)C::SMEM, s, (unsigned)cs, p) != cudaSuccess) {
        cudaGetLastError();
        return POP_E_CUDA;
      }
      count_launch();
      return POP_OK;
    }
  }
  const DecAttnDev& p = p0;
  dim3 grid(p.n_kv, p.splits, batch), grid2(p.n_q, batch);
  const int rc = launch_dec_attn<HD>(p, grid, s);
  if (rc != POP_OK) return rc;
  count_launch();
  if (p.counters == nullptr) {
    launch_chained(dec_combine_kernel<HD>, grid2, dim3(HD < 128 ? HD : 128), 0, s, p);
    count_launch();
  }
  return POP_OK;
}

int launch_dec_by_head_dim(const DecAttnDev& p, int head_dim, int batch, cudaStream_t s) {
  int rc = POP_E_INVALID;
  switch (head_dim) {
    case 64: rc = launch_dec_pair<64>(p, batch, s); break;
    case 128: rc = launch_dec_pair<128>(p, batch, s); break;
    case 256: rc = launch_dec_pair<256>(p, batch, s); break;
    default: return POP_E_INVALID;
  }
  if (rc != POP_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_decode_attention(const DecAttnArgs& a, cudaStream_t s) {
  if ((!a.q && !a.qkv) || !a.k_pool || !a.v_pool || !a.block_table || !a.partial || !a.out) return POP_E_INVALID;
  if (a.qkv && !a.table) return POP_E_INVALID;
  if (a.n_q % a.n_kv || a.n_q / a.n_kv > DEC_MAXG || a.kv_len < 1) return POP_E_INVALID;
  DecAttnDev p;
  p.qkv = a.qkv; p.ld_qkv = a.ld_qkv; p.q_gain = a.q_gain; p.k_gain = a.k_gain;
  p.table = a.table; p.table_pos0 = a.table_pos0; p.eps = a.eps; p.cache_settled = a.cache_settled;
  p.q = a.q; p.ldq = a.ldq;
  p.k_pool = a.k_pool; p.v_pool = a.v_pool;
  p.block_table = a.block_table; p.max_pages_per_seq = a.max_pages_per_seq; p.page_size = a.page_size;
  p.partial = a.partial; p.out = a.out; p.ldo = a.ldo;
  p.n_q = a.n_q; p.n_kv = a.n_kv; p.kv_len = a.kv_len; p.window = a.window;
  p.kv_first = a.kv_first < 0 ? 0 : a.kv_first;
  p.cu = a.cu_seqlens;
  p.pos_dev = a.pos_dev;
  p.counters = reinterpret_cast<unsigned int*>(a.counters);
  p.num_pages = a.num_pages;
  p.status = status_word();
  if (!p.status) return POP_E_CUDA;
  p.splits = decode_attn_splits(a.pos_dev ? 0 : a.kv_len, a.window, a.n_kv, a.batch);
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)a.head_dim);
  const int span = (a.window > 0 && a.window < a.kv_len) ? a.window : a.kv_len;
  ProfScope prof(PROF_DECODE_ATTN, (double)a.batch * span * a.n_kv * a.head_dim * 4, s);
  return launch_dec_by_head_dim(p, a.head_dim, a.batch, s);
}

}  // namespace pop

// ------------------------------------------------------------------------------ allocation-free variant
// Split-KV partials of pop_k_decode_attention_static live here instead of in a caller buffer.
// The array is part of the loaded module: every GPU that loads this library carries it until the
// process exits. POP_STATIC_SCRATCH_FLOATS (pop_kernels.h) states its size.
namespace pop {
namespace {

static __device__ __align__(256) float g_dec_static_scratch[POP_STATIC_SCRATCH_FLOATS];
// arrival counters of the split merge, one per (sequence, kv head): zero when the module is loaded,
// and every launch leaves them at zero again
constexpr int kStaticCounters = 4096;
static __device__ unsigned int g_dec_static_counters[kStaticCounters];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float* g_static_ptr[kMaxDevices] = {};
unsigned int* g_static_ctr[kMaxDevices] = {};

// Device address of the scratch array on the current device. In host code the array's name is only
// a handle for the runtime, not something a kernel can dereference, so the address is looked up
// once per device (with that device current) and remembered.
int static_scratch(float** out, unsigned int** counters) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return POP_E_CUDA;
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    float* ptr = nullptr;
    unsigned int* ctr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_dec_static_scratch) != cudaSuccess || ptr == nullptr ||
        cudaGetSymbolAddress((void**)&ctr, g_dec_static_counters) != cudaSuccess || ctr == nullptr) {
      cudaGetLastError();
      return POP_E_CUDA;
    }
    g_static_ptr[dev] = ptr;
    g_static_ctr[dev] = ctr;
  }
  *out = g_static_ptr[dev];
  *counters = g_static_ctr[dev];
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
  p.splits = decode_attn_splits(kv_len, window, n_kv, batch);
  // every (sequence, query head, split) owns head_dim + 2 floats of the shared array
  const int64_t need = (int64_t)batch * n_q * p.splits * (head_dim + 2);
  if (need > (int64_t)POP_STATIC_SCRATCH_FLOATS) return POP_E_NOSPACE;
  float* scratch = nullptr;
  unsigned int* counters = nullptr;
  const int rc = static_scratch(&scratch, &counters);
  if (rc != POP_OK) return rc;
  p.q = static_cast<const bf16*>(q); p.ldq = ldq;
  p.k_pool = static_cast<const bf16*>(k_pool); p.v_pool = static_cast<const bf16*>(v_pool);
  p.block_table = block_table; p.max_pages_per_seq = max_pages_per_seq; p.page_size = page_size;
  p.num_pages = 0;
  p.status = nullptr;
  p.qkv = nullptr; p.ld_qkv = 0; p.q_gain = p.k_gain = nullptr; p.table = nullptr; p.table_pos0 = 0; p.eps = 0.f; p.cache_settled = false;
  p.partial = scratch;
  p.out = static_cast<bf16*>(out); p.ldo = ldo;
  p.n_q = n_q; p.n_kv = n_kv; p.kv_len = kv_len; p.window = window;
  p.kv_first = 0;
  p.cu = nullptr;
  p.pos_dev = nullptr;
  // with a counter per (sequence, kv head) the attention kernel merges its own splits
  p.counters = (int64_t)batch * n_kv <= kStaticCounters ? counters : nullptr;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)head_dim);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Every partial slot that the merge reads is written first by this call's own CTAs (all splits of
  // all heads, also the empty ones), so nothing left in the array by an earlier call is ever
  // consumed and no clearing is needed between calls.
  return launch_dec_by_head_dim(p, head_dim, batch, s);
}
