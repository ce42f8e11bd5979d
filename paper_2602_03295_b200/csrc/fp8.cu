// FP8 (OCP E4M3) operands for the kept layers' widest projections: quantisation kernels. One scale per
// activation row (computed where the row is normalised), one per weight matrix (computed once at load).
// The paper names stage-aware quantisation as a direction (Sec. 6) and fixes no format.
#include "common.cuh"

namespace pop {
namespace {

constexpr float E4M3_MAX = 448.0f;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// two fp32 values -> two E4M3 codes (round to nearest even, saturating), `lo` in the low byte
__device__ __forceinline__ uint16_t cvt_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t cvt_e4m3x4(float a, float b, float c, float d) {
  return (uint32_t)cvt_e4m3x2(a, b) | ((uint32_t)cvt_e4m3x2(c, d) << 16);
}

// RMSNorm with an E4M3 result: y = x * rsqrt(mean(x^2) + eps) * gain in fp32, amax = max |y| over the row,
// codes e4m3(y * (448 / amax)), scale[row] = amax / 448 (1 for a row of zeros). The row and the gain stay
// in registers (rows up to 16 floats per thread; longer rows re-read their remainder). Since the row
// scale rstd is positive, max |y| = rstd * max |x * gain|: the sum of squares and that maximum are
// reduced over the block in one pass.
constexpr int QN_CACHE = 4;
__global__ void rmsnorm_e4m3_kernel(const float* __restrict__ x, int64_t ldx, const float* __restrict__ gain,
                                    uint8_t* __restrict__ out, int64_t ldo, float* __restrict__ scale, int d,
                                    float eps) {
  __shared__ float red_s[32], red_m[32];
  const int row = blockIdx.x;
  const float* xr = x + (int64_t)row * ldx;
  const int step = blockDim.x * 4;
  float4 yv[QN_CACHE];                      // x, then x * gain
  float4 gv[QN_CACHE];
  float ss = 0.f, am = 0.f;
  // all loads first (a zero row element contributes nothing to either reduction), the arithmetic after:
  // the eight loads of a thread are in flight together
#pragma unroll
  for (int i = 0; i < QN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    gv[i] = c < d ? *reinterpret_cast<const float4*>(gain + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    yv[i] = c < d ? *reinterpret_cast<const float4*>(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int i = 0; i < QN_CACHE; ++i) {
    const float4 v = yv[i], g = gv[i];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    yv[i] = make_float4(v.x * g.x, v.y * g.y, v.z * g.z, v.w * g.w);
    am = fmaxf(am, fmaxf(fmaxf(fabsf(yv[i].x), fabsf(yv[i].y)), fmaxf(fabsf(yv[i].z), fabsf(yv[i].w))));
  }
  for (int c = threadIdx.x * 4 + QN_CACHE * step; c < d; c += step) {
    const float4 v = *reinterpret_cast<const float4*>(xr + c);
    const float4 g = *reinterpret_cast<const float4*>(gain + c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    am = fmaxf(am, fmaxf(fmaxf(fabsf(v.x * g.x), fabsf(v.y * g.y)), fmaxf(fabsf(v.z * g.z), fabsf(v.w * g.w))));
  }
  // one block-wide pass for both values
  ss = warp_sum_f(ss);
  am = warp_max(am);
  const int wp = threadIdx.x >> 5, ln = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  if (ln == 0) {
    red_s[wp] = ss;
    red_m[wp] = am;
  }
  __syncthreads();
  ss = warp_sum_f(ln < nw ? red_s[ln] : 0.f);
  am = warp_max(ln < nw ? red_m[ln] : 0.f);
  const float rstd = rsqrtf(ss / (float)d + eps);
  const float amax = am * rstd;             // max |y|
  // y * (448 / amax) = (x * gain) * (rstd * 448 / amax)
  const float k = amax > 0.f ? rstd * (E4M3_MAX / amax) : 0.f;
  if (threadIdx.x == 0) scale[row] = amax > 0.f ? amax / E4M3_MAX : 1.0f;
  uint8_t* orow = out + (int64_t)row * ldo;
#pragma unroll
  for (int i = 0; i < QN_CACHE; ++i) {
    const int c = threadIdx.x * 4 + i * step;
    if (c < d) *reinterpret_cast<uint32_t*>(orow + c) = cvt_e4m3x4(yv[i].x * k, yv[i].y * k, yv[i].z * k, yv[i].w * k);
  }
  for (int c = threadIdx.x * 4 + QN_CACHE * step; c < d; c += step) {
    const float4 v = *reinterpret_cast<const float4*>(xr + c);
    const float4 g = *reinterpret_cast<const float4*>(gain + c);
    *reinterpret_cast<uint32_t*>(orow + c) = cvt_e4m3x4(v.x * g.x * k, v.y * g.y * k, v.z * g.z * k, v.w * g.w * k);
  }
}

// Rows of stored bf16 activations (attention output, gated FFN activation) -> E4M3 codes with one scale per
// row: amax = max |row|, codes e4m3(v * (448 / amax)), scale = amax / 448. The whole row sits in registers
// (up to 8 x 8 values per thread) before the first code is written, so `out` may be the row's own memory.
constexpr int QR_CACHE = 8;
__global__ void __launch_bounds__(256) quant_rows_bf16_e4m3_kernel(const bf16* in, int64_t ld_in, uint8_t* out,
                                                                   int64_t ld_out, float* __restrict__ scale, int d) {
  __shared__ float red_m[8];
  const int row = blockIdx.x;
  const bf16* ir = in + (int64_t)row * ld_in;
  uint4 raw[QR_CACHE];
  float am = 0.f;
#pragma unroll
  for (int i = 0; i < QR_CACHE; ++i) {           // all loads of the row first
    const int c = (i * 256 + threadIdx.x) * 8;
    raw[i] = c < d ? *reinterpret_cast<const uint4*>(ir + c) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int i = 0; i < QR_CACHE; ++i) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw[i]);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(h[j]);
      am = fmaxf(am, fmaxf(fabsf(f.x), fabsf(f.y)));
    }
  }
  am = warp_max(am);
  if ((threadIdx.x & 31) == 0) red_m[threadIdx.x >> 5] = am;
  __syncthreads();                           // also: every thread holds its part of the row by now
  am = warp_max((threadIdx.x & 31) < 8 ? red_m[threadIdx.x & 31] : 0.f);
  const float inv = am > 0.f ? E4M3_MAX / am : 1.0f;
  if (threadIdx.x == 0) scale[row] = am > 0.f ? am / E4M3_MAX : 1.0f;
  uint8_t* orow = out + (int64_t)row * ld_out;
#pragma unroll
  for (int i = 0; i < QR_CACHE; ++i) {
    const int c = (i * 256 + threadIdx.x) * 8;
    if (c < d) {
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw[i]);
      float f[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 t = __bfloat1622float2(h[j]);
        f[2 * j] = t.x * inv;
        f[2 * j + 1] = t.y * inv;
      }
      uint2 o;
      o.x = cvt_e4m3x4(f[0], f[1], f[2], f[3]);
      o.y = cvt_e4m3x4(f[4], f[5], f[6], f[7]);
      *reinterpret_cast<uint2*>(orow + c) = o;
    }
  }
}

// weight matrices, once per model: amax over the matrix (non-negative floats order like their bit patterns),
// then codes e4m3(w * (448 / amax)) and scale = amax / 448
__global__ void amax_bf16_kernel(const bf16* __restrict__ w, int64_t n, unsigned int* __restrict__ amax_bits) {
  float m = 0.f;
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < n; i += (int64_t)gridDim.x * blockDim.x * 8) {
    const uint4 raw = *reinterpret_cast<const uint4*>(w + i);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(h[j]);
      m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
    }
  }
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) atomicMax(amax_bits, __float_as_uint(m));
}
__global__ void quant_bf16_e4m3_kernel(const bf16* __restrict__ w, int64_t n, const unsigned int* __restrict__ amax_bits,
                                       uint8_t* __restrict__ out, float* __restrict__ scale) {
  const float amax = __uint_as_float(*amax_bits);
  const float inv = amax > 0.f ? E4M3_MAX / amax : 1.0f;
  if (blockIdx.x == 0 && threadIdx.x == 0) *scale = amax > 0.f ? amax / E4M3_MAX : 1.0f;
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < n; i += (int64_t)gridDim.x * blockDim.x * 8) {
    const uint4 raw = *reinterpret_cast<const uint4*>(w + i);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
    float f[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 t = __bfloat1622float2(h[j]);
      f[2 * j] = t.x * inv;
      f[2 * j + 1] = t.y * inv;
    }
    uint2 o;
    o.x = cvt_e4m3x4(f[0], f[1], f[2], f[3]);
    o.y = cvt_e4m3x4(f[4], f[5], f[6], f[7]);
    *reinterpret_cast<uint2*>(out + i) = o;
  }
}

}  // namespace

int launch_rmsnorm_e4m3(const float* x, int64_t ldx, const float* gain, uint8_t* out, int64_t ldo, float* scale,
                        int rows, int d, float eps, cudaStream_t s) {
  if (!x || !gain || !out || !scale || d % 4 || ldx % 4 || ldo % 16 || rows < 1) return POP_E_INVALID;
  ProfScope prof(PROF_ELEMENTWISE, (double)rows * d * 5.0, s);
  rmsnorm_e4m3_kernel<<<rows, d >= 2048 ? 256 : 128, 0, s>>>(x, ldx, gain, out, ldo, scale, d, eps);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_quant_rows_e4m3(const bf16* in, int64_t ld_in, uint8_t* out, int64_t ld_out, float* scale, int rows, int d,
                           cudaStream_t s) {
  if (!in || !out || !scale || rows < 1 || d < 8 || d % 8 || ld_in % 8 || ld_out % 16) return POP_E_INVALID;
  if (d > QR_CACHE * 256 * 8) return POP_E_INVALID;     // the row must fit the registers of one CTA
  ProfScope prof(PROF_ELEMENTWISE, (double)rows * d * 3.0, s);
  quant_rows_bf16_e4m3_kernel<<<rows, 256, 0, s>>>(in, ld_in, out, ld_out, scale, d);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

int launch_quantize_weights_e4m3(const bf16* w, int64_t n, uint8_t* out, float* scale, unsigned int* scratch,
                                 cudaStream_t s) {
  if (!w || !out || !scale || !scratch || n < 8 || n % 8) return POP_E_INVALID;
  if (cudaMemsetAsync(scratch, 0, 4, s) != cudaSuccess) return POP_E_CUDA;
  const int blocks = (int)std::min<int64_t>(148 * 8, (n / 8 + 255) / 256);
  amax_bf16_kernel<<<blocks, 256, 0, s>>>(w, n, scratch);
  quant_bf16_e4m3_kernel<<<blocks, 256, 0, s>>>(w, n, scratch, out, scale);
  count_launch();
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

}  // namespace pop
